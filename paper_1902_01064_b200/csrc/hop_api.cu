// C ABI of libhop_b200.so: context, options, buffer binding, trace upload, level execution.
#include <cuda_runtime.h>
#include <nvtx3/nvToolsExt.h>

#include <algorithm>
#include <cmath>
#include <cstdio>
#include <cstring>
#include <string>
#include <map>
#include <utility>
#include <vector>

#include "hop_internal.h"

const char* hop_trace_last_error();

struct hop_ctx {
    HopGraph g;
    HopSimParams sp;
    int64_t P = 0;
    int32_t s = 0;
    // options
    double lr = 0.1, momentum = 0.0, sigma = 1e-3, weight_decay = 0.0;
    int32_t loss = HOP_LOSS_HINGE;
    bool serial = false;             // serial approach: Apply before Send (Section 3.2)
    int32_t grad_mode = HOP_GRAD_EXTERNAL, mix_kernel = HOP_MIX_AUTO;
    uint64_t grad_seed = 0;
    int64_t col_offset = 0;
    // bound device memory (borrowed)
    float *X = nullptr, *M = nullptr, *G = nullptr;
    cudaStream_t stream = nullptr;
    bool bound = false;
    // SVM data (borrowed) + coefficient scratch (owned)
    const float *svmA = nullptr, *svmY = nullptr, *svmVal = nullptr;
    const int64_t* svmRowPtr = nullptr;
    const int32_t* svmCol = nullptr;
    int32_t svmR = 0, svmB = 0;
    float* coef = nullptr;
    double* margins = nullptr;       // [N][batch] margins of the current minibatches (split-phase stepping)
    bool mid_step = false;           // hop_step_begin done, hop_step_end pending
    // loaded trace (owned device tables)
    std::vector<HopLevelHost> levels;
    float* d_tcw = nullptr;         // tensor-core path: weight numerators, row tables, padded slice rows
    HopTcRow* d_tcrows = nullptr;
    int32_t* d_tcsrc = nullptr;
    alignas(64) unsigned char tc_mapX[128], tc_mapG[128], tc_mapY[8 * 128];   // TMA tensor maps over X, G, output slots
    int32_t tc_slots = 0;
    bool tc_maps_ready = false;
    // hop_run: instantiated CUDA graphs of level ranges, keyed by (first level, count)
    bool nvtx = false;              // one NVTX range per level around the enqueue calls (tracing aid)
    bool use_graph = true;
    struct Graph { cudaGraphExec_t exec; int64_t launches; };
    std::map<std::pair<int32_t, int32_t>, Graph> graphs;
    int32_t* d_i32 = nullptr;       // src_row and grad_workers of all levels
    HopRecord* d_rec = nullptr;
    HopEntry* d_ent = nullptr;
    bool loaded = false;
    hop_trace loaded_trace;         // host copy: the levels are planned again when an option that shapes the plan changes
    // streaming mode (hop_step_host): pinned staging + device copy of one level
    void* h_stage = nullptr; void* d_stage = nullptr; size_t stage_cap = 0;
    float* h_probe = nullptr; size_t probe_cap = 0;
    // progress
    int32_t level = 0;
    std::vector<int32_t> newest;
    std::vector<std::vector<uint8_t>> sent;   // [N][level] worker entered (sent) that iteration
    std::vector<int32_t> taken;               // per in-edge: newest version consumed over it (hop_step_host validation)
    int32_t* d_err = nullptr;
    int sm_count = 0;
    int64_t launches = 0;
    // optional per-kernel-class timing with CUDA events on the bound stream
    bool timing = false;
    std::vector<cudaEvent_t> ev_pool;
    size_t ev_used = 0;
    struct Span { size_t a, b; int kind; int64_t bytes; };
    std::vector<Span> spans;
    std::string err;
};

static std::string g_create_err;

#define HOP_FAIL(ctx, code, msg) do { (ctx)->err = (msg); return (code); } while (0)
#define HOP_CUDA(ctx, call) do { cudaError_t e_ = (call); if (e_ != cudaSuccess) { \
    (ctx)->err = std::string(#call) + ": " + cudaGetErrorString(e_); return HOP_E_CUDA; } } while (0)

extern "C" const char* hop_last_error(const hop_ctx* ctx) {
    if (ctx) return ctx->err.c_str();
    const char* t = hop_trace_last_error();
    return g_create_err.empty() ? t : g_create_err.c_str();
}

extern "C" int hop_create(hop_ctx** out, const int32_t* in_ptr, const int32_t* in_idx, int32_t N, int64_t P,
                          int32_t s, int32_t b, int32_t max_skip) {
    g_create_err.clear();
    auto fail = [&](int code, const std::string& m) { g_create_err = "hop_create: " + m; return code; };
    if (!out || !in_ptr || !in_idx) return fail(HOP_E_ARG, "null pointer");
    if (N <= 0 || P <= 0 || s < 0 || b < 0 || max_skip < 0) return fail(HOP_E_ARG, "N, P must be positive; s, b, max_skip non-negative");
    if ((int64_t)N * (s + 1) > (1 << 30)) return fail(HOP_E_ARG, "N*(s+1) too large");
    if (max_skip > s + 1) return fail(HOP_E_GRAPH, "max_skip > s+1: the jumper's parameters would leave its version ring");
    if (in_ptr[0] != 0) return fail(HOP_E_GRAPH, "in_ptr[0] != 0");
    hop_ctx* c = new hop_ctx;
    c->g.N = N;
    c->g.in_ptr.assign(in_ptr, in_ptr + N + 1);
    std::vector<std::vector<int32_t>> outs(N);
    for (int32_t i = 0; i < N; ++i) {
        if (in_ptr[i + 1] < in_ptr[i]) { delete c; return fail(HOP_E_GRAPH, "in_ptr not monotone"); }
        std::vector<int32_t> nb(in_idx + in_ptr[i], in_idx + in_ptr[i + 1]);
        std::sort(nb.begin(), nb.end());
        if (std::adjacent_find(nb.begin(), nb.end()) != nb.end()) { delete c; return fail(HOP_E_GRAPH, "duplicate in-neighbour at worker " + std::to_string(i)); }
        if (!nb.empty() && (nb.front() < 0 || nb.back() >= N)) { delete c; return fail(HOP_E_GRAPH, "neighbour id out of range at worker " + std::to_string(i)); }
        if (!std::binary_search(nb.begin(), nb.end(), i)) { delete c; return fail(HOP_E_GRAPH, "worker " + std::to_string(i) + " has no self-loop"); }
        if (b >= (int32_t)nb.size()) { delete c; return fail(HOP_E_GRAPH, "b >= |N_in(" + std::to_string(i) + ")|"); }
        for (int32_t j : nb) outs[j].push_back(i);
        c->g.in_idx.insert(c->g.in_idx.end(), nb.begin(), nb.end());
    }
    c->g.out_ptr.assign(1, 0);
    for (int32_t j = 0; j < N; ++j) {
        c->g.out_idx.insert(c->g.out_idx.end(), outs[j].begin(), outs[j].end());
        c->g.out_ptr.push_back((int32_t)c->g.out_idx.size());
    }
    c->P = P; c->s = s;
    c->sp.s = s; c->sp.max_ig = std::max(1, s); c->sp.max_skip = max_skip; c->sp.weight_mode = HOP_W_UNIFORM;
    c->sp.b.assign(N, b);
    c->newest.assign(N, 0);
    c->sent.assign(N, {});
    c->taken.assign(c->g.in_idx.size(), -1);
    *out = c;
    return HOP_OK;
}

// Kernel arguments (pointers, learning rate, tables) are baked into captured graphs: drop them on any change.
static void drop_graphs(hop_ctx* c) {
    for (auto& kv : c->graphs) cudaGraphExecDestroy(kv.second.exec);
    c->graphs.clear();
}

static void free_trace_tables(hop_ctx* c) {
    drop_graphs(c);
    if (c->d_i32) cudaFree(c->d_i32);
    if (c->d_rec) cudaFree(c->d_rec);
    if (c->d_ent) cudaFree(c->d_ent);
    if (c->d_tcw) cudaFree(c->d_tcw);
    if (c->d_tcrows) cudaFree(c->d_tcrows);
    if (c->d_tcsrc) cudaFree(c->d_tcsrc);
    c->d_i32 = nullptr; c->d_rec = nullptr; c->d_ent = nullptr;
    c->d_tcw = nullptr; c->d_tcrows = nullptr; c->d_tcsrc = nullptr;
    c->levels.clear();
    c->loaded = false;
    c->mid_step = false;
}

extern "C" int hop_destroy(hop_ctx* c) {
    if (!c) return HOP_OK;
    free_trace_tables(c);
    if (c->coef) cudaFree(c->coef);
    if (c->margins) cudaFree(c->margins);
    if (c->d_err) cudaFree(c->d_err);
    if (c->d_stage) cudaFree(c->d_stage);
    if (c->h_stage) cudaFreeHost(c->h_stage);
    if (c->h_probe) cudaFreeHost(c->h_probe);
    for (cudaEvent_t e : c->ev_pool) cudaEventDestroy(e);
    delete c;
    return HOP_OK;
}

static int set_option_value(hop_ctx* c, int key, double v) {
    if (key == HOP_OPT_USE_GRAPH) { c->use_graph = v != 0.0; return HOP_OK; }
    if (key == HOP_OPT_NVTX) { c->nvtx = v != 0.0; return HOP_OK; }
    if (key == HOP_OPT_NOTIFY_ACK) { c->sp.notify_ack = v != 0.0; return HOP_OK; }
    if (key == HOP_OPT_WEIGHT_DECAY) {
        if (v < 0) HOP_FAIL(c, HOP_E_ARG, "hop_set_option: weight decay must be non-negative");
        c->weight_decay = v;
        return HOP_OK;
    }
    if (key == HOP_OPT_LOSS) {
        if (v != HOP_LOSS_HINGE && v != HOP_LOSS_LOG) HOP_FAIL(c, HOP_E_ARG, "hop_set_option: unknown loss");
        c->loss = (int32_t)v;
        return HOP_OK;
    }
    if (key == HOP_OPT_APPROACH) {
        if (v != HOP_APPROACH_PARALLEL && v != HOP_APPROACH_SERIAL) HOP_FAIL(c, HOP_E_ARG, "hop_set_option: unknown approach");
        c->serial = v == HOP_APPROACH_SERIAL;
        c->sp.serial_send = c->serial ? 1 : 0;
        return HOP_OK;
    }
    if (key == HOP_OPT_STALE_REDUCE) {
        if (v != HOP_STALE_NEW_ONLY && v != HOP_STALE_REUSE) HOP_FAIL(c, HOP_E_ARG, "hop_set_option: unknown stale-reduce mode");
        c->sp.stale_reuse = v == HOP_STALE_REUSE;
        return HOP_OK;
    }
    if (key == HOP_OPT_BACKUP_MODE) {
        if (v != HOP_BACKUP_AT_LEAST && v != HOP_BACKUP_EXACT) HOP_FAIL(c, HOP_E_ARG, "hop_set_option: unknown backup mode");
        c->sp.backup_exact = (int32_t)v;
        return HOP_OK;
    }
    if (key >= HOP_OPT_BACKUP_OF_WORKER) {
        const int i = key - HOP_OPT_BACKUP_OF_WORKER;
        if (i < 0 || i >= c->g.N) HOP_FAIL(c, HOP_E_ARG, "hop_set_option: worker index out of range");
        const int d = c->g.in_ptr[i + 1] - c->g.in_ptr[i];
        if (v < 0 || v >= d || v != std::floor(v)) HOP_FAIL(c, HOP_E_GRAPH, "hop_set_option: N_buw(i) must be an integer in [0, |N_in(i)|)");
        c->sp.b[i] = (int32_t)v;
        return HOP_OK;
    }
    switch (key) {
    case HOP_OPT_MAX_IG:
        if (v < 0 || v != std::floor(v)) HOP_FAIL(c, HOP_E_ARG, "hop_set_option: max_ig must be a non-negative integer");
        c->sp.max_ig = (int32_t)v; break;
    case HOP_OPT_LR: c->lr = v; break;
    case HOP_OPT_MOMENTUM: c->momentum = v; break;
    case HOP_OPT_WEIGHT_MODE:
        if (v != HOP_W_UNIFORM && v != HOP_W_STALE_LINEAR) HOP_FAIL(c, HOP_E_ARG, "hop_set_option: unknown weight mode");
        c->sp.weight_mode = (int32_t)v; break;
    case HOP_OPT_GRAD_MODE:
        if (v < 0 || v > 3 || v != std::floor(v)) HOP_FAIL(c, HOP_E_ARG, "hop_set_option: unknown gradient mode");
        c->grad_mode = (int32_t)v; break;
    case HOP_OPT_GRAD_SEED:
        if (v < 0 || v >= 9007199254740992.0 || v != std::floor(v)) HOP_FAIL(c, HOP_E_ARG, "hop_set_option: seed must be an integer in [0, 2^53)");
        c->grad_seed = (uint64_t)v; break;
    case HOP_OPT_GRAD_SIGMA: c->sigma = v; break;
    case HOP_OPT_MIX_KERNEL:
        if (v < 0 || v > 3 || v != std::floor(v)) HOP_FAIL(c, HOP_E_ARG, "hop_set_option: unknown mix kernel");
        c->mix_kernel = (int32_t)v; break;
    case HOP_OPT_COL_OFFSET:
        if (v < 0 || v != std::floor(v) || std::fmod(v, 4.0) != 0.0) HOP_FAIL(c, HOP_E_ARG, "hop_set_option: column offset must be a non-negative multiple of 4");
        c->col_offset = (int64_t)v; break;
    default: HOP_FAIL(c, HOP_E_ARG, "hop_set_option: unknown key " + std::to_string(key));
    }
    return HOP_OK;
}

static int load_trace_impl(hop_ctx* c, const hop_trace& t, bool rewind, bool validate);

// What plan_level bakes into a loaded level: staged rows, tile width, kernel choice, the gradient rows of the dense path.
struct PlanShape {
    bool mom, decay, serial; int32_t grad_mode, mix_kernel;
    bool operator==(const PlanShape& o) const {
        return mom == o.mom && decay == o.decay && serial == o.serial && grad_mode == o.grad_mode && mix_kernel == o.mix_kernel;
    }
};
static PlanShape plan_shape(const hop_ctx* c) {
    return PlanShape{c->momentum != 0.0, c->weight_decay != 0.0, c->serial, c->grad_mode, c->mix_kernel};
}

extern "C" int hop_set_option(hop_ctx* c, int key, double v) {
    if (!c) return HOP_E_ARG;
    if (!std::isfinite(v)) HOP_FAIL(c, HOP_E_ARG, "hop_set_option: the value must be finite");
    if (c->mid_step) HOP_FAIL(c, HOP_E_STATE, "hop_set_option: a hop_step_begin is waiting for its hop_step_end");
    drop_graphs(c);
    const PlanShape before = plan_shape(c);
    const double old_mom = c->momentum, old_wd = c->weight_decay;
    const bool old_serial = c->serial;
    const int32_t old_gm = c->grad_mode, old_mk = c->mix_kernel;
    const int rc = set_option_value(c, key, v);
    if (rc) return rc;
    if (c->loaded && !(plan_shape(c) == before)) {
        // the loaded levels were planned for the old setting: plan and upload them again, keeping the position
        const int rr = load_trace_impl(c, c->loaded_trace, false, false);      // it passed the validation when it was loaded
        if (rr) {            // not plannable under the new setting: keep the old one (tables untouched)
            const std::string why = c->err;
            c->momentum = old_mom; c->weight_decay = old_wd; c->serial = old_serial; c->grad_mode = old_gm; c->mix_kernel = old_mk;
            c->err = "hop_set_option: the loaded trace cannot be planned with this value (" + why + "); option unchanged";
            return rr;
        }
    }
    return HOP_OK;
}

extern "C" int hop_sim_run(hop_ctx* c, const uint64_t* ticks, int32_t iters, hop_trace** out) {
    if (!c || !ticks || !out || iters <= 0) { if (c) c->err = "hop_sim_run: bad argument"; return HOP_E_ARG; }
    hop_trace* t = new hop_trace;
    const int rc = hop_simulate(c->g, c->sp, ticks, iters, *t, c->err);
    if (rc != HOP_OK) { delete t; return rc; }
    *out = t;
    return HOP_OK;
}

// ---- device ------------------------------------------------------------------------------------
static int ensure_device(hop_ctx* c) {
    if (c->d_err) return HOP_OK;
    int dev = 0;
    HOP_CUDA(c, cudaGetDevice(&dev));
    HOP_CUDA(c, cudaDeviceGetAttribute(&c->sm_count, cudaDevAttrMultiProcessorCount, dev));
    HOP_CUDA(c, cudaMalloc(&c->d_err, sizeof(int32_t)));
    HOP_CUDA(c, cudaMemset(c->d_err, 0, sizeof(int32_t)));
    return HOP_OK;
}

extern "C" int hop_bind_buffers(hop_ctx* c, float* X, float* M, float* G, void* stream) {
    if (!c) return HOP_E_ARG;
    if (!X) HOP_FAIL(c, HOP_E_ARG, "hop_bind_buffers: X is null");
    if (((uintptr_t)X | (uintptr_t)M | (uintptr_t)G) & 15) HOP_FAIL(c, HOP_E_ARG, "hop_bind_buffers: pointers must be 16-byte aligned");
    const int rc = ensure_device(c);
    if (rc) return rc;
    c->X = X; c->M = M; c->G = G; c->stream = (cudaStream_t)stream; c->bound = true;
    c->tc_maps_ready = false;
    drop_graphs(c);
    return HOP_OK;
}

static int alloc_coef(hop_ctx* c, int32_t R, int32_t B) {
    if (R <= 0 || B <= 0 || R % B != 0) HOP_FAIL(c, HOP_E_ARG, "SVM shard: rows_per_worker must be a positive multiple of batch");
    const int rc = ensure_device(c);
    if (rc) return rc;
    drop_graphs(c);      // captured kernels hold the old scratch and data pointers
    if (c->mid_step) HOP_FAIL(c, HOP_E_STATE, "SVM shard: a hop_step_begin is waiting for its hop_step_end");
    if (c->coef) { cudaFree(c->coef); c->coef = nullptr; }
    if (c->margins) { cudaFree(c->margins); c->margins = nullptr; }
    HOP_CUDA(c, cudaMalloc(&c->coef, (size_t)c->g.N * B * sizeof(float)));
    HOP_CUDA(c, cudaMalloc(&c->margins, (size_t)c->g.N * B * sizeof(double)));
    HOP_CUDA(c, cudaMemset(c->margins, 0, (size_t)c->g.N * B * sizeof(double)));
    c->svmR = R; c->svmB = B;
    return HOP_OK;
}

extern "C" int hop_bind_svm_dense(hop_ctx* c, const float* A, const float* y, int32_t R, int32_t B) {
    if (!c) return HOP_E_ARG;
    if (!A || !y) HOP_FAIL(c, HOP_E_ARG, "hop_bind_svm_dense: null pointer");
    const int rc = alloc_coef(c, R, B);
    if (rc) return rc;
    c->svmA = A; c->svmY = y;
    return HOP_OK;
}

extern "C" int hop_bind_svm_csr(hop_ctx* c, const int64_t* row_ptr, const int32_t* col, const float* val,
                                const float* y, int32_t R, int32_t B) {
    if (!c) return HOP_E_ARG;
    if (!row_ptr || !col || !val || !y) HOP_FAIL(c, HOP_E_ARG, "hop_bind_svm_csr: null pointer");
    const int rc = alloc_coef(c, R, B);
    if (rc) return rc;
    c->svmRowPtr = row_ptr; c->svmCol = col; c->svmVal = val; c->svmY = y;
    return HOP_OK;
}

// Tile width and kernel for one level: as many columns per tile as the staged rows leave room for.
static int plan_level(hop_ctx* c, HopLevelHost& L, bool allow_tensor = true) {
    // In the serial approach gradient, momentum and weight decay are applied to x_k before the mix, which then only averages.
    const bool use_g = c->grad_mode != HOP_GRAD_SVM_CSR && !c->serial;
    const bool mom = c->momentum != 0.0 && !c->serial;
    const bool decay = c->weight_decay != 0.0 && !c->serial;
    const int nG = use_g ? L.nG : 0;
    L.stage_rows = L.U + nG * (mom ? 2 : 1);
    int kernel = c->mix_kernel;
    // Tensor-core path: dense levels only (a contraction over <= 256 distinct slices for <= 128 workers).
    // (momentum and weight decay do not keep a level off it: the update direction is then formed in G by a pre-pass)
    const bool tc_ok = allow_tensor && c->g.N <= 128 && L.U <= 256 && L.nA > 0 && c->P % 128 == 0 &&
                       (use_g || L.nG == 0 || c->serial) &&
                       hop_dense_tc_smem((L.U + 31) / 32 * 32) > 0;
    const bool dense = L.nA >= 32 && L.sumC >= 32 * (int64_t)L.nA;
    if (tc_ok && (kernel == HOP_MIX_TENSOR || (kernel == HOP_MIX_AUTO && dense))) {
        L.kernel = HOP_MIX_TENSOR;
        L.tile_w = 128;
        L.stage_rows = L.U;
        L.Kpad = (L.U + 31) / 32 * 32;
        L.tc_w.assign((size_t)L.Kpad * 128, 0.f);
        L.tc_rows.assign(128, HopTcRow{-1, -1, 1.f});
        L.tc_src.assign(L.Kpad, L.src_row[0]);
        std::copy(L.src_row.begin(), L.src_row.end(), L.tc_src.begin());
        for (size_t a = 0; a < L.recs.size(); ++a) {
            const HopRecord& r = L.recs[a];
            const int i = r.worker;
            L.tc_rows[i] = HopTcRow{r.out_row, (r.g_stage >= 0 && use_g) ? i : -1, 1.0f / (float)L.rec_den[a]};
            for (int t = r.ent_begin; t < r.ent_begin + r.ent_count; ++t) {
                if (L.ent_num[t] == 0) continue;                 // padding entry
                const int u = L.ent_slice[t];
                // A^T in the K-major core-matrix layout the MMA reads: [u/4][i/8][i%8][u%4]
                L.tc_w[(size_t)(u / 4) * 512 + (i / 8) * 32 + (i % 8) * 4 + (u % 4)] = (float)L.ent_num[t];
            }
        }
        L.alg_bytes = 4 * c->P * ((int64_t)L.U + nG + L.nA);
        return HOP_OK;
    }
    const int rows = std::max(1, L.stage_rows);
    const int64_t tb = ((int64_t)L.recs.size() * sizeof(HopRecord) + (int64_t)L.ents.size() * sizeof(HopEntry) + 127) / 128 * 128;
    const bool tables_fit = tb <= hop_mix_table_limit();
    const bool unaligned = c->P % 4 != 0;
    // The bulk-copy kernel takes any P; with P % 4 != 0 it needs its tables in shared memory and a staged row of w + 4 floats.
    if (kernel == HOP_MIX_AUTO || kernel == HOP_MIX_TENSOR) kernel = (!unaligned || tables_fit) ? HOP_MIX_BULK : HOP_MIX_STAGED;
    if (kernel == HOP_MIX_BULK && unaligned && !tables_fit)
        HOP_FAIL(c, HOP_E_UNSUPPORTED, "the bulk-copy mix kernel with P not a multiple of 4 needs the level's tables to fit shared memory");
    const bool padded = kernel == HOP_MIX_BULK && unaligned;
    L.table_smem = (kernel == HOP_MIX_BULK && tables_fit) ? (int32_t)tb : 0;
    const int64_t budget = (hop_mix_smem_budget(kernel) - L.table_smem) / hop_mix_stages(kernel);
    int64_t w = budget / ((int64_t)rows * 4) - (padded ? 4 : 0);
    const int unit = (!unaligned || padded) ? 4 : 1;
    if (w >= 128) w = std::min<int64_t>(1024, w / 128 * 128);
    else if (w >= 32) w = w / 32 * 32;
    else w = w / unit * unit;
    if (w < unit) HOP_FAIL(c, HOP_E_UNSUPPORTED, "a level consumes more distinct slices than shared memory can stage");
    const int64_t Pr = (c->P + unit - 1) / unit * unit;
    w = std::min<int64_t>(w, Pr);
    L.tile_w = (int32_t)w;
    L.kernel = kernel;
    // slice index -> float offset of the slice's element 0 in a staged tile (padded rows: stride w + 4, plus the distance of
    // the row's first element from the 16-byte boundary below it, the same for every tile since w is a multiple of 4)
    const int64_t stride = w + (padded ? 4 : 0);
    auto offset_of = [&](int32_t slice) { return (int32_t)(slice * stride + (padded ? (((int64_t)L.src_row[slice] * c->P) & 3) : 0)); };
    for (HopEntry& e : L.ents) e.u = offset_of(e.u);
    for (HopRecord& r : L.recs) if (r.self_u >= 0) r.self_u = offset_of(r.self_u);
    // every distinct consumed slice once + gradient once + result once (+ momentum read and write)
    L.alg_bytes = 4 * c->P * ((int64_t)L.U + nG + L.nA + (mom ? 2 * (int64_t)nG : 0));
    return HOP_OK;
}

static int ensure_tc_maps(hop_ctx* c);

extern "C" int hop_load_trace(hop_ctx* c, const hop_trace* t) {
    if (!c || !t) return HOP_E_ARG;
    if (!c->bound) HOP_FAIL(c, HOP_E_STATE, "hop_load_trace: bind buffers first");
    if (t->N != c->g.N) HOP_FAIL(c, HOP_E_TRACE, "hop_load_trace: trace has a different number of workers");
    return load_trace_impl(c, *t, true, true);
}

// Validates, plans and uploads; rewind = false keeps the current level (the same trace planned again).
static int load_trace_impl(hop_ctx* c, const hop_trace& trace, bool rewind, bool validate) {
    const hop_trace* t = &trace;
    const int32_t N = t->N, L = t->levels;
    std::vector<int32_t> newest(N, 0);
    std::vector<std::vector<uint8_t>> sent(N, std::vector<uint8_t>(L, 0));
    for (int32_t k = 0; k < L; ++k)
        for (int32_t i = 0; i < N; ++i) sent[i][k] = t->op[(size_t)k * N + i] == HOP_OP_NORMAL;
    std::vector<HopLevelHost> levels(L);
    std::vector<int32_t> taken(c->g.in_idx.size(), -1);
    for (int32_t k = 0; k < L; ++k) {
        const size_t r = (size_t)k * N;
        const int rc = !validate ? HOP_OK : hop_validate_level(c->g, c->sp, k, &t->op[r], &t->ptr[r], t->nbr.data(), t->ver.data(),
                                                                t->num.data(), &t->den[r], newest, &sent, &taken, c->err);
        if (rc) return rc;
        hop_build_level(c->g, c->s, k, &t->op[r], &t->ptr[r], t->nbr.data(), t->ver.data(), t->num.data(), &t->den[r], levels[k]);
        const int rc2 = plan_level(c, levels[k]);
        if (rc2) return rc2;
    }
    std::vector<int32_t> h_i32; std::vector<HopRecord> h_rec; std::vector<HopEntry> h_ent;
    std::vector<float> h_tcw; std::vector<HopTcRow> h_tcrows; std::vector<int32_t> h_tcsrc;
    for (auto& Lv : levels) {
        if (Lv.kernel == HOP_MIX_TENSOR) {
            Lv.off_tcw = (int64_t)h_tcw.size(); h_tcw.insert(h_tcw.end(), Lv.tc_w.begin(), Lv.tc_w.end());
            Lv.off_tcrows = (int64_t)h_tcrows.size(); h_tcrows.insert(h_tcrows.end(), Lv.tc_rows.begin(), Lv.tc_rows.end());
            Lv.off_tcsrc = (int64_t)h_tcsrc.size(); h_tcsrc.insert(h_tcsrc.end(), Lv.tc_src.begin(), Lv.tc_src.end());
            Lv.tc_w.clear(); Lv.tc_w.shrink_to_fit();
        }
        Lv.off_src = (int64_t)h_i32.size(); h_i32.insert(h_i32.end(), Lv.src_row.begin(), Lv.src_row.end());
        Lv.off_gw = (int64_t)h_i32.size(); h_i32.insert(h_i32.end(), Lv.grad_workers.begin(), Lv.grad_workers.end());
        Lv.off_rec = (int64_t)h_rec.size(); h_rec.insert(h_rec.end(), Lv.recs.begin(), Lv.recs.end());
        Lv.off_ent = (int64_t)h_ent.size(); h_ent.insert(h_ent.end(), Lv.ents.begin(), Lv.ents.end());
    }
    free_trace_tables(c);
    HOP_CUDA(c, cudaMalloc(&c->d_i32, std::max<size_t>(1, h_i32.size()) * sizeof(int32_t)));
    HOP_CUDA(c, cudaMalloc(&c->d_rec, std::max<size_t>(1, h_rec.size()) * sizeof(HopRecord)));
    HOP_CUDA(c, cudaMalloc(&c->d_ent, std::max<size_t>(1, h_ent.size()) * sizeof(HopEntry)));
    HOP_CUDA(c, cudaMemcpyAsync(c->d_i32, h_i32.data(), h_i32.size() * sizeof(int32_t), cudaMemcpyHostToDevice, c->stream));
    HOP_CUDA(c, cudaMemcpyAsync(c->d_rec, h_rec.data(), h_rec.size() * sizeof(HopRecord), cudaMemcpyHostToDevice, c->stream));
    HOP_CUDA(c, cudaMemcpyAsync(c->d_ent, h_ent.data(), h_ent.size() * sizeof(HopEntry), cudaMemcpyHostToDevice, c->stream));
    if (!h_tcw.empty()) {
        HOP_CUDA(c, cudaMalloc(&c->d_tcw, h_tcw.size() * sizeof(float)));
        HOP_CUDA(c, cudaMalloc(&c->d_tcrows, h_tcrows.size() * sizeof(HopTcRow)));
        HOP_CUDA(c, cudaMalloc(&c->d_tcsrc, h_tcsrc.size() * sizeof(int32_t)));
        HOP_CUDA(c, cudaMemcpyAsync(c->d_tcw, h_tcw.data(), h_tcw.size() * sizeof(float), cudaMemcpyHostToDevice, c->stream));
        HOP_CUDA(c, cudaMemcpyAsync(c->d_tcrows, h_tcrows.data(), h_tcrows.size() * sizeof(HopTcRow), cudaMemcpyHostToDevice, c->stream));
        HOP_CUDA(c, cudaMemcpyAsync(c->d_tcsrc, h_tcsrc.data(), h_tcsrc.size() * sizeof(int32_t), cudaMemcpyHostToDevice, c->stream));
        const int mrc = ensure_tc_maps(c);
        if (mrc) return mrc;
    }
    HOP_CUDA(c, cudaStreamSynchronize(c->stream));   // the host vectors go out of scope
    c->levels = std::move(levels);
    c->sent = std::move(sent);
    c->loaded = true;
    c->mid_step = false;
    if (&trace != &c->loaded_trace) c->loaded_trace = trace;
    if (rewind) {
        c->level = 0;
        std::fill(c->newest.begin(), c->newest.end(), 0);
        std::fill(c->taken.begin(), c->taken.end(), -1);
    }
    return HOP_OK;
}

static int check_mode(hop_ctx* c) {
    const bool mom = c->momentum != 0.0;
    if (mom && !c->M) HOP_FAIL(c, HOP_E_STATE, "momentum != 0 but no momentum buffer bound");
    if (c->grad_mode != HOP_GRAD_SVM_CSR && !c->G) HOP_FAIL(c, HOP_E_STATE, "this gradient mode needs a dense gradient buffer G");
    if (c->grad_mode == HOP_GRAD_SVM_CSR && mom) HOP_FAIL(c, HOP_E_UNSUPPORTED, "momentum with the CSR SVM mode is not implemented");
    if (c->grad_mode == HOP_GRAD_SVM_CSR && c->serial && c->weight_decay != 0.0)
        HOP_FAIL(c, HOP_E_UNSUPPORTED, "weight decay with the CSR SVM mode in the serial approach is not implemented");
    if (c->grad_mode == HOP_GRAD_SVM_CSR && !c->svmRowPtr) HOP_FAIL(c, HOP_E_STATE, "CSR SVM mode without hop_bind_svm_csr");
    if (c->grad_mode == HOP_GRAD_SVM_DENSE && !c->svmA) HOP_FAIL(c, HOP_E_STATE, "dense SVM mode without hop_bind_svm_dense");
    return HOP_OK;
}

static int mark(hop_ctx* c, size_t* idx) {
    if (c->ev_used == c->ev_pool.size()) {
        cudaEvent_t e;
        HOP_CUDA(c, cudaEventCreate(&e));
        c->ev_pool.push_back(e);
    }
    *idx = c->ev_used++;
    HOP_CUDA(c, cudaEventRecord(c->ev_pool[*idx], c->stream));
    return HOP_OK;
}
#define HOP_SPAN_BEGIN() do { if (c->timing) { int r_ = mark(c, &t0); if (r_) return r_; } } while (0)
#define HOP_SPAN_END(kind, bytes) do { if (c->timing) { int r_ = mark(c, &t1); if (r_) return r_; \
    c->spans.push_back({t0, t1, (kind), (int64_t)(bytes)}); } } while (0)

// Enqueues the kernels of one level.
struct TcPtrs { const float* w; const HopTcRow* rows; const int32_t* src; };   // device tables of the dense path

static int ensure_tc_maps(hop_ctx* c) {
    if (c->tc_maps_ready) return HOP_OK;
    c->tc_slots = (c->s + 1 <= 8) ? c->s + 1 : 0;
    const int me = hop_dense_tc_make_maps(c->X, (int64_t)c->g.N * (c->s + 1), c->G, c->g.N, c->P, c->tc_mapX, c->tc_mapG,
                                          c->tc_mapY, c->tc_slots);
    if (me) HOP_FAIL(c, HOP_E_CUDA, std::string("tensor map for the dense path: ") + cudaGetErrorString((cudaError_t)me));
    c->tc_maps_ready = true;
    return HOP_OK;
}

// phase 0: the whole level.  phase 1: the gradient phase only (SVM modes stop after the partial margins).
// phase 2: the rest (SVM modes start from the margins the caller has summed over the column shards).
// chained: the operation in front of this level on the stream is the previous level of the same hop_run call (a kernel of
// this library), not something the caller enqueued.
struct NvtxLevelRange {         // "hop level k" on the host timeline while the level's kernels are enqueued
    bool on;
    NvtxLevelRange(bool enabled, int level, int phase) : on(enabled) {
        if (!on) return;
        char name[48];
        snprintf(name, sizeof name, phase == 0 ? "hop level %d" : (phase == 1 ? "hop level %d (begin)" : "hop level %d (end)"), level);
        nvtxRangePushA(name);
    }
    ~NvtxLevelRange() { if (on) nvtxRangePop(); }
};

static int run_level(hop_ctx* c, const HopLevelHost& L, const HopLevelDev& lv, const TcPtrs& tc, int phase = 0, bool chained = false) {
    NvtxLevelRange range(c->nvtx, lv.level, phase);
    size_t t0 = 0, t1 = 0;
    HopLaunchCfg cfg{};
    cfg.X = c->X; cfg.M = c->M; cfg.G = c->G; cfg.P = c->P; cfg.N = c->g.N; cfg.s = c->s;
    cfg.lr = (float)c->lr; cfg.mu = (float)c->momentum; cfg.wd = (float)c->weight_decay; cfg.loss = c->loss; cfg.tile_w = L.tile_w;
    cfg.use_g = c->grad_mode != HOP_GRAD_SVM_CSR;
    cfg.sm_count = c->sm_count; cfg.err_word = c->d_err; cfg.stream = c->stream;
    cfg.table_smem = L.table_smem; cfg.n_ents = (int32_t)L.ents.size();
    int e = hop_checked_set_fence(cfg);
    if (e) HOP_FAIL(c, HOP_E_CUDA, std::string("checked build, buffer ranges: ") + cudaGetErrorString((cudaError_t)e));
    bool grad_kernel_in_front = false;      // a gradient kernel of this library was launched by this call, right before the mix
    if (L.nG > 0 && c->grad_mode != HOP_GRAD_EXTERNAL) {
        HOP_SPAN_BEGIN();
        switch (c->grad_mode) {
        case HOP_GRAD_SYNTHETIC:
            if (phase != 2) { e = hop_launch_synth_grad(cfg, lv, c->grad_seed, (float)c->sigma, c->col_offset); c->launches += 1; grad_kernel_in_front = true; }
            break;
        case HOP_GRAD_SVM_DENSE:
            e = hop_launch_svm_dense(cfg, lv, c->svmA, c->svmY, c->svmR, c->svmB, c->coef, c->margins, phase);
            c->launches += (phase == 1 || (phase == 0 && hop_svm_dense_is_fused(c->P, c->svmB))) ? 1 : 2;
            grad_kernel_in_front = true; break;
        case HOP_GRAD_SVM_CSR:
            // parallel approach inside hop_run: the margin kernel is a programmatic dependent of the previous level's last
            // kernel (it fetches its static row data while that kernel drains, then waits), and the mix-update of it.  Not
            // for the first level of a call: what the caller enqueued in front may still be writing the row data.
            cfg.dependent = (phase == 0 && !c->serial && chained) ? 1 : 0;
            e = hop_launch_svm_csr_coef(cfg, lv, c->svmRowPtr, c->svmCol, c->svmVal, c->svmY, c->svmR, c->svmB, c->coef, c->margins, phase);
            c->launches += 1; grad_kernel_in_front = true; break;
        default: break;
        }
        if (e) HOP_FAIL(c, HOP_E_CUDA, std::string("gradient kernel launch: ") + cudaGetErrorString((cudaError_t)e));
        HOP_SPAN_END(0, 0);
    }
    if (phase == 1) return HOP_OK;
    if (c->serial && L.nG > 0) {      // Apply on x_k before it is sent: dense update kernel, or the sparse apply on slot k
        HOP_SPAN_BEGIN();
        if (c->grad_mode == HOP_GRAD_SVM_CSR)
            e = hop_launch_svm_csr_apply(cfg, lv, c->svmRowPtr, c->svmCol, c->svmVal, c->svmR, c->svmB, c->coef, 0);
        else
            e = hop_launch_apply_dense(cfg, lv);
        c->launches += 1;
        if (e) HOP_FAIL(c, HOP_E_CUDA, std::string("apply launch: ") + cudaGetErrorString((cudaError_t)e));
        HOP_SPAN_END(2, 0);
        cfg.use_g = 0; cfg.mu = 0.f; cfg.wd = 0.f;      // the mix only averages
        grad_kernel_in_front = false;                   // the apply kernel in front writes X
    }
    // None of the gradient kernels writes X or M, and each was launched with a full dependency on everything before it:
    // the mix may fetch its X and M rows while such a kernel drains (it waits before it reads G and before it stores).
    cfg.early_x = grad_kernel_in_front ? 1 : 0;
    if (L.kernel == HOP_MIX_TENSOR && L.nG > 0 && cfg.use_g && (cfg.mu != 0.f || cfg.wd != 0.f)) {
        // the dense path's epilogue applies -lr * G only: momentum and weight decay go into G first (cfg.mu / cfg.wd are
        // already 0 here in the serial approach, where the apply kernel has done it all)
        HOP_SPAN_BEGIN();
        e = hop_launch_direction_dense(cfg, lv);
        c->launches += 1;
        if (e) HOP_FAIL(c, HOP_E_CUDA, std::string("update direction launch: ") + cudaGetErrorString((cudaError_t)e));
        HOP_SPAN_END(2, 0);
    }
    if (L.nA > 0) {
        HOP_SPAN_BEGIN();
        if (L.kernel == HOP_MIX_TENSOR)
            e = hop_launch_mix_dense_tc(cfg, c->tc_mapX, c->tc_mapG,
                                        (L.nA == c->g.N && c->tc_slots > 0) ? c->tc_mapY + 128 * ((lv.level + 1) % (c->s + 1)) : nullptr,
                                        tc.w, tc.rows, tc.src, L.Kpad, L.tc_rows.data());
        else
            e = (L.kernel == HOP_MIX_BULK) ? hop_launch_mix_bulk(cfg, lv) : hop_launch_mix_staged(cfg, lv);
        c->launches += 1;
        if (e) HOP_FAIL(c, HOP_E_CUDA, std::string("mix kernel launch: ") + cudaGetErrorString((cudaError_t)e));
        HOP_SPAN_END(1, L.alg_bytes);
    }
    if (L.nG > 0 && c->grad_mode == HOP_GRAD_SVM_CSR && !c->serial) {
        HOP_SPAN_BEGIN();
        // launched with a full dependency: with the sparse apply a dependent as well (a chain of three programmatic edges
        // per level) a level of the 16-worker CSR workload took 44.0 us instead of 37.2 us in graph replay (measured)
        cfg.dependent = 0;
        e = hop_launch_svm_csr_apply(cfg, lv, c->svmRowPtr, c->svmCol, c->svmVal, c->svmR, c->svmB, c->coef, 1);
        c->launches += 1;
        if (e) HOP_FAIL(c, HOP_E_CUDA, std::string("sparse apply launch: ") + cudaGetErrorString((cudaError_t)e));
        HOP_SPAN_END(2, 0);
    }
    return HOP_OK;
}

static int step_phase(hop_ctx* c, int phase) {
    if (!c->bound || !c->loaded) HOP_FAIL(c, HOP_E_STATE, "hop_step_begin/end: bind buffers and load a trace first");
    if (c->level >= (int32_t)c->levels.size()) HOP_FAIL(c, HOP_E_STATE, "hop_step_begin/end: past the end of the trace");
    if ((phase == 1) == c->mid_step) HOP_FAIL(c, HOP_E_STATE, "hop_step_begin and hop_step_end must alternate");
    int rc = check_mode(c);
    if (rc) return rc;
    const HopLevelHost& L = c->levels[c->level];
    HopLevelDev lv{c->d_i32 + L.off_src, c->d_rec + L.off_rec, c->d_ent + L.off_ent, c->d_i32 + L.off_gw, L.U, L.nA, L.nG, c->level};
    rc = run_level(c, L, lv, TcPtrs{c->d_tcw + L.off_tcw, c->d_tcrows + L.off_tcrows, c->d_tcsrc + L.off_tcsrc}, phase);
    if (rc) return rc;
    c->mid_step = phase == 1;
    if (phase == 2) {
        for (const HopRecord& r : L.recs) c->newest[r.worker] = c->level + 1;
        c->level += 1;
    }
    return HOP_OK;
}

extern "C" int hop_step_begin(hop_ctx* c, double** margins, int64_t* count) {
    if (!c) return HOP_E_ARG;
    const int rc = step_phase(c, 1);
    if (rc) return rc;
    const bool svm = c->grad_mode == HOP_GRAD_SVM_DENSE || c->grad_mode == HOP_GRAD_SVM_CSR;
    if (margins) *margins = svm ? c->margins : nullptr;
    if (count) *count = svm ? (int64_t)c->g.N * c->svmB : 0;
    return HOP_OK;
}

extern "C" int hop_step_end(hop_ctx* c) {
    if (!c) return HOP_E_ARG;
    return step_phase(c, 2);
}

extern "C" int hop_step(hop_ctx* c) {
    if (!c) return HOP_E_ARG;
    if (c->mid_step) HOP_FAIL(c, HOP_E_STATE, "hop_step: a hop_step_begin is waiting for its hop_step_end");
    if (!c->bound || !c->loaded) HOP_FAIL(c, HOP_E_STATE, "hop_step: bind buffers and load a trace first");
    if (c->level >= (int32_t)c->levels.size()) HOP_FAIL(c, HOP_E_STATE, "hop_step: past the end of the trace");
    int rc = check_mode(c);
    if (rc) return rc;
    const HopLevelHost& L = c->levels[c->level];
    HopLevelDev lv{c->d_i32 + L.off_src, c->d_rec + L.off_rec, c->d_ent + L.off_ent, c->d_i32 + L.off_gw,
                   L.U, L.nA, L.nG, c->level};
    rc = run_level(c, L, lv, TcPtrs{c->d_tcw + L.off_tcw, c->d_tcrows + L.off_tcrows, c->d_tcsrc + L.off_tcsrc});
    if (rc) return rc;
    for (const HopRecord& r : L.recs) c->newest[r.worker] = c->level + 1;
    c->level += 1;
    return HOP_OK;
}

static int enqueue_level(hop_ctx* c, int32_t k, bool chained) {
    const HopLevelHost& L = c->levels[k];
    HopLevelDev lv{c->d_i32 + L.off_src, c->d_rec + L.off_rec, c->d_ent + L.off_ent, c->d_i32 + L.off_gw, L.U, L.nA, L.nG, k};
    return run_level(c, L, lv, TcPtrs{c->d_tcw + L.off_tcw, c->d_tcrows + L.off_tcrows, c->d_tcsrc + L.off_tcsrc}, 0, chained);
}

extern "C" int hop_run(hop_ctx* c, int32_t n_levels) {
    if (!c) return HOP_E_ARG;
    if (!c->bound || !c->loaded) HOP_FAIL(c, HOP_E_STATE, "hop_run: bind buffers and load a trace first");
    if (c->mid_step) HOP_FAIL(c, HOP_E_STATE, "hop_run: a hop_step_begin is waiting for its hop_step_end");
    if (n_levels < 0 || c->level + n_levels > (int32_t)c->levels.size()) HOP_FAIL(c, HOP_E_STATE, "hop_run: past the end of the trace");
    if (n_levels == 0) return HOP_OK;
    int rc = check_mode(c);
    if (rc) return rc;
    const int32_t first = c->level;
    // Graph replay needs a capturable stream (not the legacy default stream), no per-kernel event timing,
    // and a gradient source that is part of the library (an external G changes between levels).
    const bool graph = c->use_graph && c->stream != nullptr && !c->timing && c->grad_mode != HOP_GRAD_EXTERNAL && n_levels > 1 &&
                       !hop_checked_build();      // the checked build copies its buffer ranges from pageable memory: not capturable
    if (!graph) {
        for (int32_t k = first; k < first + n_levels; ++k)
            if ((rc = enqueue_level(c, k, k > first))) return rc;
    } else {
        auto key = std::make_pair(first, n_levels);
        auto it = c->graphs.find(key);
        if (it == c->graphs.end()) {
            const int64_t launches_before = c->launches;
            HOP_CUDA(c, cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeRelaxed));
            for (int32_t k = first; k < first + n_levels && !rc; ++k) rc = enqueue_level(c, k, k > first);
            cudaGraph_t g = nullptr;
            const cudaError_t ce = cudaStreamEndCapture(c->stream, &g);
            const int64_t in_graph = c->launches - launches_before;
            c->launches = launches_before;
            if (rc) { if (g) cudaGraphDestroy(g); return rc; }
            if (ce != cudaSuccess) { c->err = std::string("hop_run: stream capture: ") + cudaGetErrorString(ce); return HOP_E_CUDA; }
            cudaGraphExec_t ex = nullptr;
            const cudaError_t ie = cudaGraphInstantiate(&ex, g, 0);
            cudaGraphDestroy(g);
            if (ie != cudaSuccess) { c->err = std::string("hop_run: graph instantiation: ") + cudaGetErrorString(ie); return HOP_E_CUDA; }
            it = c->graphs.emplace(key, hop_ctx::Graph{ex, in_graph}).first;
        }
        HOP_CUDA(c, cudaGraphLaunch(it->second.exec, c->stream));
        c->launches += it->second.launches;
    }
    for (int32_t k = first; k < first + n_levels; ++k)
        for (const HopRecord& r : c->levels[k].recs) c->newest[r.worker] = k + 1;
    c->level = first + n_levels;
    return HOP_OK;
}

extern "C" int hop_step_host(hop_ctx* c, const int32_t* op, const int64_t* ptr, const int32_t* nbr, const int32_t* ver,
                             const int32_t* num, const int32_t* den, float* probe_dst, int64_t probe_len) {
    if (!c) return HOP_E_ARG;
    if (!op || !ptr || !den) HOP_FAIL(c, HOP_E_ARG, "hop_step_host: null pointer");
    if (!c->bound) HOP_FAIL(c, HOP_E_STATE, "hop_step_host: bind buffers first");
    if (c->mid_step) HOP_FAIL(c, HOP_E_STATE, "hop_step_host: a hop_step_begin is waiting for its hop_step_end");
    if (probe_len < 0 || probe_len > c->P) HOP_FAIL(c, HOP_E_ARG, "hop_step_host: probe_len out of range");
    int rc = check_mode(c);
    if (rc) return rc;
    const int32_t N = c->g.N, k = c->level;
    if (ptr[0] != 0) HOP_FAIL(c, HOP_E_ARG, "hop_step_host: ptr[0] must be 0");
    for (int32_t i = 0; i < N; ++i) {
        if ((int32_t)c->sent[i].size() <= k) c->sent[i].resize(k + 1, 0);
        c->sent[i][k] = op[i] == HOP_OP_NORMAL;
    }
    std::vector<int32_t> newest = c->newest, taken = c->taken;
    rc = hop_validate_level(c->g, c->sp, k, op, ptr, nbr, ver, num, den, newest, &c->sent, &taken, c->err);
    if (rc) return rc;
    HopLevelHost L;
    hop_build_level(c->g, c->s, k, op, ptr, nbr, ver, num, den, L);
    rc = plan_level(c, L);
    if (rc) return rc;
    const bool tcl = L.kernel == HOP_MIX_TENSOR;
    if (tcl && (rc = ensure_tc_maps(c))) return rc;
    // pack [src_row | grad_workers | recs | ents] into one pinned buffer, one H2D copy
    const size_t b_src = L.src_row.size() * 4, b_gw = L.grad_workers.size() * 4;
    const size_t o_gw = b_src, o_rec = (o_gw + b_gw + 15) / 16 * 16, b_rec = L.recs.size() * sizeof(HopRecord);
    const size_t o_ent = o_rec + b_rec, b_ent = L.ents.size() * sizeof(HopEntry);
    // dense path: weight numerators (16-byte aligned for the bulk copy), row table, padded slice rows
    const size_t o_tcw = (o_ent + b_ent + 127) / 128 * 128, b_tcw = tcl ? L.tc_w.size() * sizeof(float) : 0;
    const size_t o_tcr = o_tcw + b_tcw, b_tcr = tcl ? L.tc_rows.size() * sizeof(HopTcRow) : 0;
    const size_t o_tcs = (o_tcr + b_tcr + 15) / 16 * 16, b_tcs = tcl ? L.tc_src.size() * sizeof(int32_t) : 0;
    const size_t total = std::max<size_t>(16, o_tcs + b_tcs);
    if (total > c->stage_cap) {
        if (c->d_stage) cudaFree(c->d_stage);
        if (c->h_stage) cudaFreeHost(c->h_stage);
        c->d_stage = nullptr; c->h_stage = nullptr; c->stage_cap = 0;
        const size_t cap = std::max<size_t>(total * 2, 1 << 16);
        HOP_CUDA(c, cudaMalloc(&c->d_stage, cap));
        HOP_CUDA(c, cudaMallocHost(&c->h_stage, cap));
        c->stage_cap = cap;
    }
    if ((size_t)probe_len > c->probe_cap) {
        if (c->h_probe) cudaFreeHost(c->h_probe);
        c->h_probe = nullptr; c->probe_cap = 0;
        HOP_CUDA(c, cudaMallocHost((void**)&c->h_probe, (size_t)probe_len * sizeof(float)));
        c->probe_cap = (size_t)probe_len;
    }
    unsigned char* h = (unsigned char*)c->h_stage;
    if (b_src) std::memcpy(h, L.src_row.data(), b_src);
    if (b_gw) std::memcpy(h + o_gw, L.grad_workers.data(), b_gw);
    if (b_rec) std::memcpy(h + o_rec, L.recs.data(), b_rec);
    if (b_ent) std::memcpy(h + o_ent, L.ents.data(), b_ent);
    if (b_tcw) std::memcpy(h + o_tcw, L.tc_w.data(), b_tcw);
    if (b_tcr) std::memcpy(h + o_tcr, L.tc_rows.data(), b_tcr);
    if (b_tcs) std::memcpy(h + o_tcs, L.tc_src.data(), b_tcs);
    HOP_CUDA(c, cudaMemcpyAsync(c->d_stage, h, total, cudaMemcpyHostToDevice, c->stream));
    unsigned char* d = (unsigned char*)c->d_stage;
    HopLevelDev lv{(const int32_t*)d, (const HopRecord*)(d + o_rec), (const HopEntry*)(d + o_ent), (const int32_t*)(d + o_gw),
                   L.U, L.nA, L.nG, k};
    rc = run_level(c, L, lv, TcPtrs{(const float*)(d + o_tcw), (const HopTcRow*)(d + o_tcr), (const int32_t*)(d + o_tcs)});
    if (rc) return rc;
    c->newest = newest;
    c->taken.swap(taken);
    c->level += 1;
    if (probe_dst && probe_len > 0) {
        const float* src = c->X + ((int64_t)0 * (c->s + 1) + c->newest[0] % (c->s + 1)) * c->P;
        HOP_CUDA(c, cudaMemcpyAsync(c->h_probe, src, (size_t)probe_len * sizeof(float), cudaMemcpyDeviceToHost, c->stream));
    }
    HOP_CUDA(c, cudaStreamSynchronize(c->stream));
    if (probe_dst && probe_len > 0) std::memcpy(probe_dst, c->h_probe, (size_t)probe_len * sizeof(float));
    return HOP_OK;
}

extern "C" int hop_set_level(hop_ctx* c, int32_t level) {
    if (!c) return HOP_E_ARG;
    if (level < 0 || (c->loaded && level > (int32_t)c->levels.size())) HOP_FAIL(c, HOP_E_ARG, "hop_set_level: out of range");
    c->mid_step = false;
    std::fill(c->taken.begin(), c->taken.end(), -1);    // hop_step_host's per-edge order check starts afresh
    // newest version held by each worker after levels [0, level)
    std::fill(c->newest.begin(), c->newest.end(), 0);
    if (c->loaded)
        for (int32_t k = 0; k < level; ++k)
            for (const HopRecord& r : c->levels[k].recs) c->newest[r.worker] = k + 1;
    c->level = level;
    return HOP_OK;
}

extern "C" int hop_newest_version(hop_ctx* c, int32_t worker, int32_t* version) {
    if (!c || !version) return HOP_E_ARG;
    if (worker < 0 || worker >= c->g.N) HOP_FAIL(c, HOP_E_ARG, "hop_newest_version: worker out of range");
    *version = c->newest[worker];
    return HOP_OK;
}

extern "C" int hop_write_params(hop_ctx* c, int32_t worker, int32_t version, const float* src) {
    if (!c) return HOP_E_ARG;
    if (!src || version < 0 || worker < -1 || worker >= c->g.N) HOP_FAIL(c, HOP_E_ARG, "hop_write_params: bad argument");
    if (!c->bound) HOP_FAIL(c, HOP_E_STATE, "hop_write_params: bind buffers first");
    const int S = c->s + 1;
    const int lo = worker < 0 ? 0 : worker, hi = worker < 0 ? c->g.N : worker + 1;
    for (int i = lo; i < hi; ++i)
        HOP_CUDA(c, cudaMemcpyAsync(c->X + ((int64_t)i * S + version % S) * c->P, src, (size_t)c->P * sizeof(float),
                                    cudaMemcpyHostToDevice, c->stream));
    HOP_CUDA(c, cudaStreamSynchronize(c->stream));
    return HOP_OK;
}

extern "C" int hop_read_params(hop_ctx* c, int32_t worker, int32_t version, float* dst) {
    if (!c) return HOP_E_ARG;
    if (!dst || worker < 0 || worker >= c->g.N || version < -1) HOP_FAIL(c, HOP_E_ARG, "hop_read_params: bad argument");
    if (!c->bound) HOP_FAIL(c, HOP_E_STATE, "hop_read_params: bind buffers first");
    const int S = c->s + 1;
    const int v = version < 0 ? c->newest[worker] : version;
    HOP_CUDA(c, cudaMemcpyAsync(dst, c->X + ((int64_t)worker * S + v % S) * c->P, (size_t)c->P * sizeof(float),
                                cudaMemcpyDeviceToHost, c->stream));
    HOP_CUDA(c, cudaStreamSynchronize(c->stream));
    return HOP_OK;
}

extern "C" int hop_read_status(hop_ctx* c, int32_t* word) {
    if (!c || !word) return HOP_E_ARG;
    *word = 0;
    if (!c->d_err) return HOP_OK;
    HOP_CUDA(c, cudaStreamSynchronize(c->stream));
    HOP_CUDA(c, cudaMemcpy(word, c->d_err, sizeof(int32_t), cudaMemcpyDeviceToHost));
    if (*word != 0) {
        static const char* what[] = {"unknown", "mix_bulk_kernel: a tile's copies did not arrive", "mix_bulk_kernel: no stage became free",
                                     "mix_dense_tc_kernel: a pipeline wait ran out",
                                     "checked build: an access outside the bound buffers was refused"};
        const int code = (*word >> 24) & 0xff;
        HOP_FAIL(c, HOP_E_DEVICE, std::string("a kernel reported -- ") + what[code >= 1 && code <= 4 ? code : 0] +
                                  " (status word " + std::to_string(*word) + ", detail " + std::to_string(*word & 0xffffff) + ")");
    }
    return HOP_OK;
}

extern "C" int hop_build_is_checked(void) { return hop_checked_build() ? 1 : 0; }

extern "C" int hop_clear_status(hop_ctx* c) {
    if (!c) return HOP_E_ARG;
    if (!c->d_err) return HOP_OK;
    HOP_CUDA(c, cudaMemsetAsync(c->d_err, 0, sizeof(int32_t), c->stream));
    return HOP_OK;
}

extern "C" int hop_selftest_bounded_wait(hop_ctx* c, int32_t polls, int32_t detail) {
    if (!c) return HOP_E_ARG;
    if (polls < 1 || polls > 65536) HOP_FAIL(c, HOP_E_ARG, "hop_selftest_bounded_wait: polls must be in [1, 65536]");
    if (!c->bound) HOP_FAIL(c, HOP_E_STATE, "hop_selftest_bounded_wait: bind buffers first");
    const int e = hop_launch_wait_selftest(c->d_err, (uint32_t)polls, detail, c->stream);
    if (e) HOP_FAIL(c, HOP_E_CUDA, std::string("self-test launch: ") + cudaGetErrorString((cudaError_t)e));
    c->launches += 1;
    return HOP_OK;
}

extern "C" int hop_level_stats(hop_ctx* c, int32_t level, int64_t* out) {
    if (!c || !out) return HOP_E_ARG;
    if (!c->loaded || level < 0 || level >= (int32_t)c->levels.size()) HOP_FAIL(c, HOP_E_ARG, "hop_level_stats: no such level");
    const HopLevelHost& L = c->levels[level];
    out[0] = L.U; out[1] = L.nG; out[2] = L.nJump; out[3] = L.sumC; out[4] = L.tile_w; out[5] = L.kernel;
    out[6] = L.stage_rows; out[7] = L.alg_bytes;
    out[8] = L.kernel == HOP_MIX_TENSOR ? (int64_t)2 * 2 * 128 * L.Kpad * c->P : 0;   // two TF32 passes, M x N x K = P x 128 x Kpad
    out[9] = L.Kpad;
    return HOP_OK;
}

extern "C" int hop_timing_enable(hop_ctx* c, int32_t on) {
    if (!c) return HOP_E_ARG;
    c->timing = on != 0;
    c->spans.clear();
    c->ev_used = 0;
    return HOP_OK;
}

extern "C" int hop_timing_read(hop_ctx* c, double* ms, int64_t* launches, int64_t* mix_bytes) {
    if (!c || !ms || !launches || !mix_bytes) return HOP_E_ARG;
    for (int k = 0; k < 3; ++k) { ms[k] = 0.0; launches[k] = 0; }
    *mix_bytes = 0;
    if (c->bound) HOP_CUDA(c, cudaStreamSynchronize(c->stream));
    for (const auto& sp : c->spans) {
        float t = 0.f;
        HOP_CUDA(c, cudaEventElapsedTime(&t, c->ev_pool[sp.a], c->ev_pool[sp.b]));
        ms[sp.kind] += t;
        launches[sp.kind] += 1;
        if (sp.kind == 1) *mix_bytes += sp.bytes;
    }
    c->spans.clear();
    c->ev_used = 0;
    return HOP_OK;
}

extern "C" int hop_launch_count(hop_ctx* c, int64_t* n) {
    if (!c || !n) return HOP_E_ARG;
    *n = c->launches;
    return HOP_OK;
}
