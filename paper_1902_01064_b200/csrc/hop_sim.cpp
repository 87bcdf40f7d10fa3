// Host-side deterministic simulation of the Hop queue protocol (paper Sections 4 and 5).
//
// The paper describes the protocol with FIFO update queues and token queues.  A queue-free
// formulation is used here: everything a worker can observe about a neighbour follows from two
// facts, the iteration the neighbour is in and the list of iterations it has entered (and so
// sent, Fig. alg2: Send happens on entering an iteration):
//   * Recv(k) of worker i may take from in-neighbour j the newest entered iteration v <= k of j
//     (one queue per iteration slot keeps newer ones out of reach, Section 6); it is usable iff
//     v >= k - s (Section 4.4).  Recv completes once |N_in(i)| - N_buw(i) in-neighbours (self
//     counts) are usable and then takes every usable one (Fig. alg4: needed + extras).
//   * What a Recv dequeued is gone from the queue.  Under HOP_STALE_NEW_ONLY (Eq. 2's index set, Fig. alg3's
//     test on what this call dequeued) a usable update enters the Reduce only if it is newer than the
//     one the worker's previous Recv saw from that neighbour; one mark per in-edge keeps that.
//   * TokenQ(j->i).size() = Iter(j) - Iter(i) + max_ig (proof of Theorem 2), so "a token is
//     available from every out-neighbour" is Iter(j) >= Iter(i) + 1 - max_ig for all of them, and
//     the straggler test of Section 5 (how many tokens the out-neighbours hold for me) is
//     min_j Iter(j) - Iter(i) - 1 iterations behind the slowest out-neighbour.
// In the serial approach of Section 3.2 (Compute, Apply, Send, Recv, Reduce) an iteration's update leaves when its
// Compute ends instead of when the iteration is entered; tokens move as before.
// Time is integer ticks; only Compute takes time.  Transitions that fall on the same tick are
// resolved in rounds: every worker whose inputs changed in the previous round decides from the
// state that round left, then all decisions are committed.
#include <algorithm>
#include <queue>
#include <string>
#include <vector>

#include "hop_internal.h"

namespace {

enum Phase : int8_t { COMPUTE, WAIT_RECV, WAIT_TOKEN, WAIT_JUMP_RECV, DONE };

struct Decision {
    enum Kind : int8_t { NONE, APPLIED, ENTER, PLAN_JUMP, JUMP } kind = NONE;
    int32_t target = 0;
    std::vector<std::pair<int32_t, int32_t>> got;   // (neighbour, version)
    std::vector<int32_t> seen;                      // per in-edge of the worker: usable version this Recv saw, -1 none
};

struct Sim {
    const HopGraph& g;
    const HopSimParams& p;
    const uint64_t* ticks;
    int32_t iters;
    int32_t N;
    std::vector<int32_t> iter;                      // iteration a worker is in
    std::vector<Phase> phase;
    std::vector<int32_t> jump_to;
    std::vector<int32_t> applied;                   // newest iteration whose Reduce/Apply is done (-1: none)
    std::vector<std::vector<int32_t>> entered;      // iterations whose update a worker has sent, ascending
    std::vector<std::vector<int64_t>> entered_seq;  // global order of those Send events (arrival order at every receiver)
    std::vector<int32_t> reduced;                   // per in-edge: newest version the receiver's completed Recvs have seen
    int64_t send_seq = 0;
    uint64_t now = 0;
    using Ev = std::pair<uint64_t, int32_t>;
    std::priority_queue<Ev, std::vector<Ev>, std::greater<Ev>> compute_end;
    // output
    std::vector<std::vector<int32_t>> r_nbr, r_ver, r_num;   // per (level*N + worker)
    hop_trace& out;

    Sim(const HopGraph& g_, const HopSimParams& p_, const uint64_t* t, int32_t it, hop_trace& o)
        : g(g_), p(p_), ticks(t), iters(it), N(g_.N), iter(N, 0), phase(N, COMPUTE), jump_to(N, 0), applied(N, -1),
          entered(N), entered_seq(N), reduced(g_.in_idx.size(), -1), r_nbr((size_t)it * N), r_ver((size_t)it * N), r_num((size_t)it * N), out(o) {}

    int32_t newest_entered_upto(int32_t j, int32_t level) const {
        const auto& e = entered[j];
        auto it = std::upper_bound(e.begin(), e.end(), level);
        return it == e.begin() ? -1 : *(it - 1);
    }

    void send(int32_t i, int32_t k) {
        entered[i].push_back(k);
        entered_seq[i].push_back(send_seq++);
    }

    void enter(int32_t i, int32_t k) {
        iter[i] = k;
        if (!p.serial_send) send(i, k);
        phase[i] = COMPUTE;
        compute_end.push({now + ticks[(size_t)i * iters + k], i});
    }

    bool try_recv(int32_t i, int32_t level, int32_t own_version, Decision& d) const {
        d.got.clear();
        const int32_t a = g.in_ptr[i], e = g.in_ptr[i + 1];
        d.seen.assign(e - a, -1);
        for (int32_t t = a; t < e; ++t) {
            const int32_t j = g.in_idx[t];
            if (j == i && own_version >= 0) { d.got.push_back({j, own_version}); continue; }
            const int32_t v = newest_entered_upto(j, level);
            if (v >= 0 && v >= level - p.s) { d.got.push_back({j, v}); d.seen[t - a] = v; }
        }
        const int32_t need = (e - a) - p.b[i];
        if ((int32_t)d.got.size() < need) return false;
        if (p.backup_exact && (int32_t)d.got.size() > need) {
            // keep the own update plus the neighbours whose first usable update (iteration >= level - s) was sent
            // earliest: the first |N_in| - b entries a FIFO dequeue would return
            std::vector<std::pair<int64_t, int32_t>> order;   // (send order of first usable update, neighbour)
            for (auto [j, v] : d.got) {
                if (j == i) continue;
                const auto& en = entered[j];
                const size_t pos = std::lower_bound(en.begin(), en.end(), std::max(0, level - p.s)) - en.begin();
                order.push_back({entered_seq[j][pos], j});
            }
            std::sort(order.begin(), order.end());
            std::vector<uint8_t> keep(N, 0);
            keep[i] = 1;
            for (int32_t t = 0; t < need - 1; ++t) keep[order[t].second] = 1;
            std::vector<std::pair<int32_t, int32_t>> kept;
            for (auto jv : d.got) if (keep[jv.first]) kept.push_back(jv);
            d.got.swap(kept);
        }
        if (!p.stale_reuse) {
            // only updates newer than what an earlier Recv of this worker already took out of the queue
            std::vector<std::pair<int32_t, int32_t>> fresh;
            for (auto jv : d.got) {
                const int32_t t = (int32_t)(std::lower_bound(g.in_idx.begin() + a, g.in_idx.begin() + e, jv.first) - g.in_idx.begin());
                if (jv.first == i || jv.second > reduced[t]) fresh.push_back(jv);
            }
            d.got.swap(fresh);
        }
        return true;
    }

    void recv_done(int32_t i, const Decision& d) {
        const int32_t a = g.in_ptr[i];
        for (size_t t = 0; t < d.seen.size(); ++t)
            if (d.seen[t] >= 0) reduced[a + t] = d.seen[t];
    }

    Decision decide(int32_t i) const {
        Decision d;
        const int32_t k = iter[i];
        switch (phase[i]) {
        case WAIT_RECV:
            if (try_recv(i, k, -1, d)) d.kind = Decision::APPLIED;
            break;
        case WAIT_TOKEN: {
            int32_t slowest = INT32_MAX, least_applied = INT32_MAX;
            bool any = false;
            for (int32_t t = g.out_ptr[i]; t < g.out_ptr[i + 1]; ++t) {
                const int32_t j = g.out_idx[t];
                if (j == i) continue;
                any = true;
                slowest = std::min(slowest, iter[j]);
                least_applied = std::min(least_applied, applied[j]);
            }
            if (p.notify_ack) {   // NOTIFY-ACK: every out-neighbour has acknowledged (reduced) iteration k-1
                if (!any || least_applied >= k - 1) { d.kind = Decision::ENTER; d.target = k + 1; }
                break;
            }
            if (p.max_skip > 0 && any) {
                const int32_t behind = slowest - (k + 1);
                const int32_t skip = std::min(std::min(behind, p.max_skip), (iters - 1) - (k + 1));
                if (behind >= 1 && skip >= 1) { d.kind = Decision::PLAN_JUMP; d.target = k + 1 + skip; break; }
            }
            if (!any || p.max_ig == 0 || slowest >= k + 1 - p.max_ig) { d.kind = Decision::ENTER; d.target = k + 1; }
            break;
        }
        case WAIT_JUMP_RECV:
            if (try_recv(i, jump_to[i] - 1, k + 1, d)) { d.kind = Decision::JUMP; d.target = jump_to[i]; }
            break;
        default: break;
        }
        return d;
    }

    void record(int32_t op, int32_t level, int32_t i, const Decision& d, int32_t own_as) {
        const size_t r = (size_t)level * N + i;
        out.op[r] = op;
        int32_t den = 0;
        for (auto [j, v] : d.got) {
            const int32_t veff = (j == i && own_as >= 0) ? own_as : v;
            const int32_t w = p.weight_mode == HOP_W_UNIFORM ? 1 : veff - (level - p.s) + 1;
            r_nbr[r].push_back(j); r_ver[r].push_back(v); r_num[r].push_back(w);
            den += w;
        }
        out.den[r] = den;
    }

    // marks the workers whose next decision may depend on worker i having entered an iteration
    void touch_neighbours(int32_t i, std::vector<uint8_t>& dirty) const {
        for (int32_t t = g.out_ptr[i]; t < g.out_ptr[i + 1]; ++t) dirty[g.out_idx[t]] = 1;
        for (int32_t t = g.in_ptr[i]; t < g.in_ptr[i + 1]; ++t) dirty[g.in_idx[t]] = 1;
    }

    int run(std::string& err) {
        out.levels = iters; out.N = N;
        out.op.assign((size_t)iters * N, HOP_OP_IDLE);
        out.den.assign((size_t)iters * N, 0);
        for (int32_t i = 0; i < N; ++i) enter(i, 0);
        int32_t done = 0;
        std::vector<uint8_t> dirty(N, 0), next_dirty(N, 0);
        std::vector<std::pair<int32_t, Decision>> acts;
        while (done < N) {
            if (compute_end.empty()) {
                err = "protocol deadlock at tick " + std::to_string(now) + ": no worker is computing and " +
                      std::to_string(N - done) + " are unfinished";
                return HOP_E_DEADLOCK;
            }
            now = compute_end.top().first;
            std::fill(dirty.begin(), dirty.end(), 0);
            while (!compute_end.empty() && compute_end.top().first == now) {
                const int32_t i = compute_end.top().second;
                compute_end.pop();
                phase[i] = WAIT_RECV;
                dirty[i] = 1;
                if (p.serial_send) { send(i, iter[i]); touch_neighbours(i, dirty); }
            }
            for (;;) {
                acts.clear();
                for (int32_t i = 0; i < N; ++i)
                    if (dirty[i]) {
                        Decision d = decide(i);
                        if (d.kind != Decision::NONE) acts.emplace_back(i, std::move(d));
                    }
                if (acts.empty()) break;
                std::fill(next_dirty.begin(), next_dirty.end(), 0);
                for (auto& [i, d] : acts) {
                    const int32_t k = iter[i];
                    next_dirty[i] = 1;
                    switch (d.kind) {
                    case Decision::APPLIED:
                        record(HOP_OP_NORMAL, k, i, d, -1);
                        recv_done(i, d);
                        applied[i] = k;
                        if (p.notify_ack) touch_neighbours(i, next_dirty);   // an ACK may release an in-neighbour
                        if (k == iters - 1) { phase[i] = DONE; ++done; } else phase[i] = WAIT_TOKEN;
                        break;
                    case Decision::ENTER:
                        enter(i, d.target);
                        touch_neighbours(i, next_dirty);
                        break;
                    case Decision::PLAN_JUMP:
                        jump_to[i] = d.target;
                        phase[i] = WAIT_JUMP_RECV;
                        break;
                    case Decision::JUMP:
                        record(HOP_OP_JUMP, d.target - 1, i, d, d.target - 1);
                        recv_done(i, d);
                        enter(i, d.target);
                        touch_neighbours(i, next_dirty);
                        break;
                    default: break;
                    }
                }
                dirty.swap(next_dirty);
            }
        }
        out.makespan = now;
        out.ptr.assign((size_t)iters * N + 1, 0);
        for (size_t r = 0; r < (size_t)iters * N; ++r) {
            out.ptr[r + 1] = out.ptr[r] + (int64_t)r_nbr[r].size();
            out.nbr.insert(out.nbr.end(), r_nbr[r].begin(), r_nbr[r].end());
            out.ver.insert(out.ver.end(), r_ver[r].begin(), r_ver[r].end());
            out.num.insert(out.num.end(), r_num[r].begin(), r_num[r].end());
        }
        return HOP_OK;
    }
};

}  // namespace

int hop_simulate(const HopGraph& g, const HopSimParams& p, const uint64_t* ticks, int32_t iters,
                 hop_trace& out, std::string& err) {
    for (size_t t = 0; t < (size_t)g.N * iters; ++t)
        if (ticks[t] == 0) { err = "compute time of 0 ticks"; return HOP_E_ARG; }
    if (p.notify_ack && p.max_skip > 0) { err = "NOTIFY-ACK has no iteration skipping"; return HOP_E_ARG; }
    if (p.max_skip > 0 && p.max_ig == 0) { err = "skipping reads token counts: token queues (max_ig >= 1) required"; return HOP_E_ARG; }
    Sim sim(g, p, ticks, iters, out);
    return sim.run(err);
}
