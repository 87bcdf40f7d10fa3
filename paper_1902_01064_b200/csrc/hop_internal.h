// Internal declarations shared by the translation units of libhop_b200.so.
#pragma once
#include <cstdint>
#include <string>
#include <vector>

#include "hop.h"

struct hop_trace {
    int32_t levels = 0, N = 0;
    uint64_t makespan = 0;
    std::vector<int32_t> op;    // [levels*N]
    std::vector<int64_t> ptr;   // [levels*N+1]
    std::vector<int32_t> nbr, ver, num;
    std::vector<int32_t> den;   // [levels*N]
};

// ---- device-side tables of one level (built on the host, uploaded once) -------------------------
struct HopRecord {          // one active (NORMAL or JUMP) worker of a level
    int32_t worker;
    int32_t out_row;        // row of X that receives x_{k+1,i}: worker*(s+1) + (k+1) mod (s+1)
    int32_t ent_begin;      // first entry (relative to the level's entry array)
    int32_t ent_count;
    int32_t g_stage;        // index among the level's NORMAL workers, -1 for JUMP
    int32_t cur_row;        // row of X holding x_{k,i} (gradient input); -1 for JUMP
    int32_t self_u;         // float offset of the worker's own consumed slice inside a staged tile (weight decay)
    int32_t pad1;
};
struct alignas(8) HopEntry {
    int32_t u;              // float offset of the slice's row inside a staged tile: slice index * tile width
    float w;                // float(num) / float(den)
};

struct HopTcRow {           // per worker, for the tensor-core dense path
    int32_t out_row;        // row of X receiving the result, -1 if the worker is idle in this level
    int32_t g_row;          // row of G to apply (= worker), -1 for none
    float inv_den;          // 1 / weight denominator (row scaling)
};

struct HopLevelHost {
    int32_t U = 0, nA = 0, nG = 0, nJump = 0;
    int64_t sumC = 0;
    std::vector<int32_t> src_row;       // [U] rows of X
    std::vector<HopRecord> recs;        // [nA]
    std::vector<HopEntry> ents;
    std::vector<int32_t> grad_workers;  // [nG] workers with a NORMAL record
    std::vector<int32_t> ent_slice, ent_num, rec_den;   // integer view of the entries (slice index, numerator), per-record denominator
    // tensor-core dense path (only when planned): numerators in the MMA's shared-memory layout, row table, padded slice rows
    int32_t Kpad = 0;
    std::vector<float> tc_w;
    std::vector<HopTcRow> tc_rows;
    std::vector<int32_t> tc_src;
    int64_t off_tcw = 0, off_tcrows = 0, off_tcsrc = 0;
    // offsets into the uploaded arrays
    int64_t off_src = 0, off_rec = 0, off_ent = 0, off_gw = 0;
    // launch plan
    int32_t tile_w = 0, kernel = 0, stage_rows = 0, table_smem = 0;
    int64_t alg_bytes = 0;
};

struct HopLevelDev {        // passed by value to the kernels
    const int32_t* src_row;
    const HopRecord* recs;
    const HopEntry* ents;
    const int32_t* grad_workers;
    int32_t U, nA, nG, level;
};

struct HopGraph {
    int32_t N = 0;
    std::vector<int32_t> in_ptr, in_idx;    // in-neighbours, self included
    std::vector<int32_t> out_ptr, out_idx;  // out-neighbours, self included
};

struct HopSimParams {
    int32_t s, max_ig /*0 = none*/, max_skip, weight_mode;
    int32_t notify_ack = 0;     // NOTIFY-ACK back-pressure (Section 3.3) instead of token queues
    int32_t backup_exact = 0;   // keep exactly |N_in| - b updates (own + earliest senders) instead of every usable one
    int32_t serial_send = 0;    // serial approach: the update of iteration k is sent when Compute(k) ends, not on entering k
    int32_t stale_reuse = 0;    // 1: a usable update an earlier Recv already returned is reduced again (HOP_STALE_REUSE)
    std::vector<int32_t> b;
};

// hop_sim.cpp
int hop_simulate(const HopGraph& g, const HopSimParams& p, const uint64_t* ticks, int32_t iters,
                 hop_trace& out, std::string& err);
// hop_trace.cpp
int hop_validate_level(const HopGraph& g, const HopSimParams& p, int32_t level, const int32_t* op,
                       const int64_t* ptr, const int32_t* nbr, const int32_t* ver, const int32_t* num,
                       const int32_t* den, std::vector<int32_t>& newest,
                       std::vector<std::vector<uint8_t>>* sent, std::vector<int32_t>* taken, std::string& err);
void hop_build_level(const HopGraph& g, int32_t s, int32_t level, const int32_t* op, const int64_t* ptr,
                     const int32_t* nbr, const int32_t* ver, const int32_t* num, const int32_t* den,
                     HopLevelHost& out);

// Opt a kernel into the largest dynamic shared-memory size once per device instead of before every launch
// (the call is not a stream operation, so this also keeps it out of stream capture).
#ifdef __CUDACC__
template <auto Kernel>
static inline cudaError_t hop_allow_max_smem() {
    static bool done[64] = {};
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64) return cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
    if (!done[dev]) {
        e = cudaFuncSetAttribute(Kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, 227 * 1024);
        if (e != cudaSuccess) return e;
        done[dev] = true;
    }
    return cudaSuccess;
}
#endif

// hop_kernels.cu : launchers.  All return a cudaError_t cast to int.
struct HopLaunchCfg {
    float* X; float* M; float* G;
    int64_t P;
    int32_t N, s;
    float lr, mu;
    float wd;           // weight decay lambda: lambda * x_{k,i} joins the gradient of NORMAL records
    int32_t loss;       // 0 hinge, 1 log (SVM modes)
    int32_t tile_w;
    int32_t use_g;      // dense gradient rows are applied
    int32_t sm_count;
    int32_t* err_word;  // device
    int32_t table_smem; // bytes of shared memory holding the level's records + entries (0 = read from global)
    int32_t n_ents;
    int32_t early_x;    // the mix launch may overlap the tail of the gradient kernel launched just before it (which writes
                        // neither X nor M): programmatic dependent launch
    int32_t dependent;  // CSR SVM kernels: launch as a programmatic dependent of the kernel in front (the kernel waits before it
                        // touches anything that kernel, or one before it, may still be writing)
    void* stream;
};
int hop_launch_mix_staged(const HopLaunchCfg& c, const HopLevelDev& lv);
int hop_launch_mix_bulk(const HopLaunchCfg& c, const HopLevelDev& lv);
int hop_launch_synth_grad(const HopLaunchCfg& c, const HopLevelDev& lv, uint64_t seed, float sigma, int64_t col_offset);
// phase 0 = whole gradient; 1 = partial margins into `margins` only; 2 = coefficients from `margins`, then the rest
int hop_launch_svm_dense(const HopLaunchCfg& c, const HopLevelDev& lv, const float* A, const float* y,
                         int32_t R, int32_t B, float* coef, double* margins, int phase);
int hop_launch_svm_csr_coef(const HopLaunchCfg& c, const HopLevelDev& lv, const int64_t* row_ptr, const int32_t* col,
                            const float* val, const float* y, int32_t R, int32_t B, float* coef, double* margins, int phase);
// slot_shift 1: apply to x_{k+1} after the mix (parallel approach); 0: to x_k before it (serial approach)
int hop_launch_svm_csr_apply(const HopLaunchCfg& c, const HopLevelDev& lv, const int64_t* row_ptr, const int32_t* col,
                             const float* val, int32_t R, int32_t B, const float* coef, int32_t slot_shift);
// serial approach, dense gradients: x_k <- x_k - lr * d in place for the level's NORMAL workers
int hop_launch_apply_dense(const HopLaunchCfg& c, const HopLevelDev& lv);
// dense (tensor-core) path with momentum or weight decay: G <- update direction, in place, before the mix
int hop_launch_direction_dense(const HopLaunchCfg& c, const HopLevelDev& lv);
bool hop_svm_dense_is_fused(int64_t P, int32_t B);   // the dense SVM gradient of a level is one launch instead of two
int hop_checked_set_fence(const HopLaunchCfg& c);     // checked build only (no-op otherwise): bound-buffer ranges for the kernels
bool hop_checked_build();
int hop_launch_wait_selftest(int32_t* err_word, uint32_t polls, int32_t detail, void* stream);
int hop_mix_smem_budget(int kernel);   // usable dynamic shared memory per CTA for the kernel
int hop_mix_stages(int kernel);
int hop_mix_table_limit();
// hop_dense_tc.cu
size_t hop_dense_tc_smem(int Kpad);
int hop_dense_tc_make_maps(float* X, int64_t ring_rows, const float* G, int32_t N, int64_t P, void* mapX, void* mapG,
                           void* mapY, int32_t n_slots);   // 128-byte blobs; mapY holds n_slots of them
// mapY = the output slot's map when every worker is active in the level, else nullptr (row-by-row stores);
// host_rows = the host copy of tbl (its per-worker constants travel as kernel parameters)
int hop_launch_mix_dense_tc(const HopLaunchCfg& c, const void* mapX, const void* mapG, const void* mapY, const float* Wk,
                            const HopTcRow* tbl, const int32_t* src_row, int Kpad, const HopTcRow* host_rows);
