// Trace objects, host-side validation of trace records against the protocol's rules, and the
// construction of the per-level device tables (distinct consumed slices, per-worker entries).
#include <algorithm>
#include <cstring>
#include <string>
#include <unordered_map>
#include <vector>

#include "hop_internal.h"

static std::string g_trace_err;
const char* hop_trace_last_error() { return g_trace_err.c_str(); }

extern "C" int hop_trace_create(hop_trace** out, int32_t levels, int32_t N, const int32_t* op,
                                const int64_t* ptr, const int32_t* nbr, const int32_t* ver,
                                const int32_t* num, const int32_t* den) {
    if (!out || levels < 0 || N <= 0 || !op || !ptr || !den) { g_trace_err = "hop_trace_create: bad argument"; return HOP_E_ARG; }
    const size_t R = (size_t)levels * N;
    if (ptr[0] != 0) { g_trace_err = "hop_trace_create: ptr[0] must be 0"; return HOP_E_ARG; }
    for (size_t r = 0; r < R; ++r)
        if (ptr[r + 1] < ptr[r]) { g_trace_err = "hop_trace_create: ptr must be non-decreasing"; return HOP_E_ARG; }
    const int64_t E = ptr[R];
    if (E > 0 && (!nbr || !ver || !num)) { g_trace_err = "hop_trace_create: null entry arrays"; return HOP_E_ARG; }
    hop_trace* t = new hop_trace;
    t->levels = levels; t->N = N;
    t->op.assign(op, op + R);
    t->ptr.assign(ptr, ptr + R + 1);
    t->den.assign(den, den + R);
    t->nbr.assign(nbr, nbr + E);
    t->ver.assign(ver, ver + E);
    t->num.assign(num, num + E);
    *out = t;
    return HOP_OK;
}

extern "C" int hop_trace_dims(const hop_trace* t, int32_t* levels, int32_t* N, int64_t* entries, uint64_t* makespan) {
    if (!t) return HOP_E_ARG;
    if (levels) *levels = t->levels;
    if (N) *N = t->N;
    if (entries) *entries = (int64_t)t->nbr.size();
    if (makespan) *makespan = t->makespan;
    return HOP_OK;
}

extern "C" int hop_trace_export(const hop_trace* t, int32_t* op, int64_t* ptr, int32_t* nbr, int32_t* ver,
                                int32_t* num, int32_t* den) {
    if (!t) return HOP_E_ARG;
    auto cp = [](auto* dst, const auto& v) { if (dst && !v.empty()) std::memcpy(dst, v.data(), v.size() * sizeof(v[0])); };
    cp(op, t->op); cp(ptr, t->ptr); cp(nbr, t->nbr); cp(ver, t->ver); cp(num, t->num); cp(den, t->den);
    return HOP_OK;
}

extern "C" int hop_trace_destroy(hop_trace* t) { delete t; return HOP_OK; }

// One level of records checked against the rules the protocol guarantees.  `newest[i]` is the
// newest version worker i holds before the level and is advanced; `sent` (optional, [N][levels])
// marks the iterations a worker entered, i.e. the versions other workers may consume; `taken`
// (optional, one per in-edge, -1 = nothing yet) is the newest version the receiver has consumed over
// that edge and is advanced: a FIFO queue never hands out an older update after a newer one, and
// under HOP_STALE_NEW_ONLY never the same one twice.
int hop_validate_level(const HopGraph& g, const HopSimParams& p, int32_t level, const int32_t* op,
                       const int64_t* ptr, const int32_t* nbr, const int32_t* ver, const int32_t* num,
                       const int32_t* den, std::vector<int32_t>& newest,
                       std::vector<std::vector<uint8_t>>* sent, std::vector<int32_t>* taken, std::string& err) {
    const int32_t N = g.N;
    auto fail = [&](int32_t i, const std::string& what) {
        err = "trace record (level " + std::to_string(level) + ", worker " + std::to_string(i) + "): " + what;
        return HOP_E_TRACE;
    };
    std::vector<int32_t> seen(N, -1);
    for (int32_t i = 0; i < N; ++i) {
        const int64_t a = ptr[i], e = ptr[i + 1];
        const int32_t o = op[i];
        if (o == HOP_OP_IDLE) {
            if (e != a) return fail(i, "IDLE record with entries");
            continue;
        }
        if (o != HOP_OP_NORMAL && o != HOP_OP_JUMP) return fail(i, "unknown op");
        if (o == HOP_OP_NORMAL && newest[i] != level) return fail(i, "NORMAL but the worker does not hold version " + std::to_string(level));
        if (o == HOP_OP_JUMP && !(newest[i] <= level && newest[i] >= level - p.s)) return fail(i, "JUMP but the held version is outside [k-s, k]");
        const int32_t d = g.in_ptr[i + 1] - g.in_ptr[i];
        // Fig. alg4's count is about usable updates; with s > 0 and HOP_STALE_NEW_ONLY the Reduce may hold fewer
        // (only those that arrived since the previous Recv, Eq. 2), down to the own update alone
        const bool may_be_fewer = p.s > 0 && !p.stale_reuse;
        if (!may_be_fewer && e - a < d - p.b[i]) return fail(i, "fewer than |N_in| - b consumed updates");
        if (e - a > d) return fail(i, "more consumed updates than in-neighbours");
        int64_t sum = 0;
        bool own = false;
        const auto nb_begin = g.in_idx.begin() + g.in_ptr[i], nb_end = g.in_idx.begin() + g.in_ptr[i + 1];
        auto walk = nb_begin;            // records usually list neighbours in ascending order, like the graph: one merge pass
        for (int64_t t = a; t < e; ++t) {
            const int32_t j = nbr[t], v = ver[t];
            if (j < 0 || j >= N) return fail(i, "neighbour id out of range");
            while (walk != nb_end && *walk < j) ++walk;
            const auto edge = (walk != nb_end && *walk == j) ? walk : std::lower_bound(nb_begin, nb_end, j);
            if (edge == nb_end || *edge != j)
                return fail(i, "consumed worker " + std::to_string(j) + " is not an in-neighbour");
            if (seen[j] == i) return fail(i, "neighbour consumed twice");
            seen[j] = i;
            if (v < level - p.s || v > level || v < 0) return fail(i, "version " + std::to_string(v) + " outside the staleness window [k-s, k]");
            if (j == i) {
                own = true;
                if (v != newest[i]) return fail(i, "own entry must name the version the worker holds");
            } else if (sent && !(*sent)[j][v]) {
                return fail(i, "version " + std::to_string(v) + " of worker " + std::to_string(j) + " was never sent");
            }
            if (taken && j != i) {
                int32_t& last = (*taken)[edge - g.in_idx.begin()];
                if (v < last) return fail(i, "version " + std::to_string(v) + " of worker " + std::to_string(j) + " is older than one consumed before");
                if (v == last && !p.stale_reuse)
                    return fail(i, "version " + std::to_string(v) + " of worker " + std::to_string(j) + " was consumed before (HOP_STALE_NEW_ONLY reduces an update once)");
                last = v;
            }
            if (num[t] <= 0) return fail(i, "non-positive weight numerator");
            sum += num[t];
        }
        if (!own) return fail(i, "own update missing");
        if (sum != den[i]) return fail(i, "numerators do not sum to the denominator");
    }
    for (int32_t i = 0; i < N; ++i)
        if (op[i] != HOP_OP_IDLE) newest[i] = level + 1;
    return HOP_OK;
}

// Device tables of one level: the distinct consumed (worker, version) slices in first-use order and,
// per active worker, its entries as (slice index, float weight).
void hop_build_level(const HopGraph& g, int32_t s, int32_t level, const int32_t* op, const int64_t* ptr,
                     const int32_t* nbr, const int32_t* ver, const int32_t* num, const int32_t* den,
                     HopLevelHost& out) {
    const int32_t N = g.N, S = s + 1;
    std::vector<int32_t> slice_of((size_t)N * S, -1);
    out = HopLevelHost();
    const size_t n_ent = (size_t)(ptr[N] - ptr[0]) + 3 * (size_t)N;      // entries plus per-record padding
    out.ents.reserve(n_ent); out.ent_slice.reserve(n_ent); out.ent_num.reserve(n_ent);
    out.recs.reserve(N); out.rec_den.reserve(N); out.grad_workers.reserve(N); out.src_row.reserve(std::min(n_ent, (size_t)N * S));
    for (int32_t i = 0; i < N; ++i) {
        if (op[i] == HOP_OP_IDLE) continue;
        HopRecord r{};
        r.worker = i;
        r.out_row = i * S + (level + 1) % S;
        r.ent_begin = (int32_t)out.ents.size();
        r.ent_count = (int32_t)(ptr[i + 1] - ptr[i]);
        if (op[i] == HOP_OP_NORMAL) {
            r.g_stage = out.nG++;
            r.cur_row = i * S + level % S;
            out.grad_workers.push_back(i);
        } else {
            r.g_stage = -1;
            r.cur_row = -1;
            ++out.nJump;
        }
        r.self_u = -1;
        for (int64_t t = ptr[i]; t < ptr[i + 1]; ++t) {
            const int32_t row = nbr[t] * S + ver[t] % S;
            if (slice_of[row] < 0) { slice_of[row] = out.U++; out.src_row.push_back(row); }
            if (nbr[t] == i) r.self_u = slice_of[row];      // slice index for now; scaled by the tile width when planned
            out.ents.push_back({slice_of[row], (float)num[t] / (float)den[i]});
            out.ent_slice.push_back(slice_of[row]);
            out.ent_num.push_back(num[t]);
        }
        out.rec_den.push_back(den[i]);
        out.sumC += r.ent_count;
        // Entries are padded to a multiple of four per record with weight-0 terms on the record's first slice
        // (adding 0 * x changes nothing), so that the mix kernels run whole groups of four without a remainder loop.
        while (r.ent_count % 4 != 0 && r.ent_count > 0) {
            out.ents.push_back({out.ents[r.ent_begin].u, 0.0f});
            out.ent_slice.push_back(out.ent_slice[r.ent_begin]);
            out.ent_num.push_back(0);
            ++r.ent_count;
        }
        out.recs.push_back(r);
    }
    out.nA = (int32_t)out.recs.size();
}
