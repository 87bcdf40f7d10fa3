// Dense-graph mixing on the 5th-generation tensor cores (tcgen05, accumulators in tensor memory).
//
// For an all-to-all graph every worker consumes ~N slices, so the level is a contraction
//     Y[i][p] = (1/den_i) * sum_u A[i][u] * Xs[u][p]  -  lr * G[i][p]
// over the K = U_k distinct consumed (worker, version) rows, with A[i][u] the integer weight numerator
// of Eq. 2 (or 1 for the plain mean of Fig. alg4) and den_i their sum (Reduce of Fig. alg3 / alg4, Apply
// of Fig. alg0).  float32 accuracy from TF32 tensor cores by operand splitting (3xTF32): X = X_hi + X_lo
// with both parts TF32-exact, W = diag(1/den) * A with A's small integers TF32-exact, so A_lo == 0, the
// W_lo * X_hi term of 3xTF32 vanishes identically and two MMA passes remain: A*X_hi and A*X_lo.  They go to
// two separate accumulators (the first is a sum of exact 13-bit products, the second is tiny), added in
// float32 in the epilogue where the row scaling 1/den_i is applied.
//
// Roles inside one persistent thread block (one per SM), tile = 128 parameter columns x all workers:
//   warp 0      producer: cp.async.bulk of the 32 raw X row pieces of a K-chunk into shared memory
//   warp 1      MMA issue (one elected lane): tcgen05.mma kind::tf32, M=128 (columns) x N=128 (workers) x K=8,
//               A operand (X_hi / X_lo) from tensor memory, B operand (A^T, resident) from shared memory
//   warps 4-7   converters: lane = column; read the raw chunk from shared memory, split hi/lo with
//               cvt.rna.tf32, tcgen05.st into the A stages in tensor memory
//   warps 8-11  epilogue: tcgen05.ld both accumulators, add, release them, then y = acc/den - lr*g with
//               coalesced 128-byte loads of G and stores of Y per (warp, worker)
// Tensor memory (512 columns): D_hi 0..127, D_lo 128..255, four A stages of 64 columns (hi 32 + lo 32).
// Every wait is bounded; a time-out sets the error word and lets the block run to its normal exit,
// where tensor memory is released.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>

#include "hop_internal.h"

namespace {

constexpr int kTile = 128;          // parameter columns per tile = MMA M
constexpr int kChunk = 32;          // K rows per pipeline stage
constexpr int kStages = 4;
constexpr int kThreads = 12 * 32;
constexpr uint32_t kSpin = 1u << 20;
constexpr int kRawStageBytes = kChunk * kTile * 4;          // 16 KB
enum : int32_t { ERR_TC_WAIT = 3 << 24 };

__device__ __forceinline__ uint32_t s32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mb_init(uint64_t* b, uint32_t c) { asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(s32(b)), "r"(c)); }
__device__ __forceinline__ void mb_expect_tx(uint64_t* b, uint32_t n) { asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(s32(b)), "r"(n) : "memory"); }
__device__ __forceinline__ void mb_arrive(uint64_t* b) { asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(s32(b)) : "memory"); }
__device__ __forceinline__ bool mb_try(uint64_t* b, uint32_t ph) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}" : "=r"(ok) : "r"(s32(b)), "r"(ph) : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool mb_wait(uint64_t* b, uint32_t ph, volatile int* abort_flag) {
    for (uint32_t it = 0; it < kSpin; ++it) {
        if (mb_try(b, ph)) return true;
        if (it > 32) __nanosleep(40);
        if ((it & 1023) == 1023 && *abort_flag) return false;
    }
    return false;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(s32(dst)), "l"(src), "r"(bytes), "r"(s32(bar)) : "memory");
}
__device__ __forceinline__ uint32_t to_tf32(float x) { uint32_t r; asm("cvt.rna.tf32.f32 %0, %1;" : "=r"(r) : "f"(x)); return r; }

// Shared-memory matrix descriptor, K-major, no swizzle: 8x(16 B) core matrices; leading-dimension byte
// offset = distance between core matrices adjacent in K, stride byte offset = distance between 8-row
// groups; bits 46-47 = 1 (descriptor version of this architecture); layout type 0.
__device__ __forceinline__ uint64_t smem_desc(uint32_t addr, uint32_t lbo, uint32_t sbo) {
    return (uint64_t)((addr & 0x3FFFF) >> 4) | ((uint64_t)(lbo >> 4) << 16) | ((uint64_t)(sbo >> 4) << 32) | (1ull << 46);
}
// Instruction descriptor: D = F32 (bits 4-5 = 1), A = B = TF32 (format 2 at bits 7-9 and 10-12), both K-major,
// N >> 3 at bits 17-22, M >> 4 at bits 24-28.
constexpr uint32_t kIdesc = (1u << 4) | (2u << 7) | (2u << 10) | ((128u >> 3) << 17) | ((128u >> 4) << 24);

__device__ __forceinline__ void mma_tf32_ts(uint32_t d_tmem, uint32_t a_tmem, uint64_t b_desc, uint32_t accumulate) {
    asm volatile("{\n.reg .pred p;\nsetp.ne.b32 p, %4, 0;\ntcgen05.mma.cta_group::1.kind::tf32 [%0], [%1], %2, %3, p;\n}"
                 ::"r"(d_tmem), "r"(a_tmem), "l"(b_desc), "r"(kIdesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void mma_commit(uint64_t* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(s32(bar)) : "memory");
}
__device__ __forceinline__ void fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tmem_st32(uint32_t taddr, const uint32_t (&v)[32]) {
    asm volatile("tcgen05.st.sync.aligned.32x32b.x32.b32 [%0], {%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,%16,"
                 "%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31,%32};"
                 ::"r"(taddr), "r"(v[0]), "r"(v[1]), "r"(v[2]), "r"(v[3]), "r"(v[4]), "r"(v[5]), "r"(v[6]), "r"(v[7]), "r"(v[8]), "r"(v[9]),
                 "r"(v[10]), "r"(v[11]), "r"(v[12]), "r"(v[13]), "r"(v[14]), "r"(v[15]), "r"(v[16]), "r"(v[17]), "r"(v[18]), "r"(v[19]),
                 "r"(v[20]), "r"(v[21]), "r"(v[22]), "r"(v[23]), "r"(v[24]), "r"(v[25]), "r"(v[26]), "r"(v[27]), "r"(v[28]), "r"(v[29]),
                 "r"(v[30]), "r"(v[31]) : "memory");
}
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float (&v)[32]) {
    uint32_t r[32];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x32.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15,"
                 "%16,%17,%18,%19,%20,%21,%22,%23,%24,%25,%26,%27,%28,%29,%30,%31}, [%32];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]), "=r"(r[8]), "=r"(r[9]),
                   "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]), "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]),
                   "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]), "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]),
                   "=r"(r[30]), "=r"(r[31]) : "r"(taddr) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}

struct TcSmem {                       // control block at the start of dynamic shared memory
    uint64_t raw_full[kStages], raw_empty[kStages], a_full[kStages], a_empty[kStages];
    uint64_t acc_full, acc_empty, w_full;
    uint32_t tmem_base;
    int abort_flag;
    HopTcRow rows[128];
};

__global__ void __launch_bounds__(kThreads, 1)
mix_dense_tc_kernel(float* __restrict__ X, const float* __restrict__ G, int64_t P, float lr, const float* __restrict__ Wk,
                    const HopTcRow* __restrict__ tbl, const int32_t* __restrict__ src_row, int Kpad,
                    int32_t* __restrict__ err_word) {
    extern __shared__ __align__(1024) unsigned char smem[];
    TcSmem* cb = reinterpret_cast<TcSmem*>(smem);
    float* Wsm = reinterpret_cast<float*>(smem + 4096);                        // Kpad * 512 bytes, canonical K-major
    float* raw = reinterpret_cast<float*>(smem + 4096 + (size_t)Kpad * 512);   // kStages x [32][128] floats
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t tiles = P / kTile;
    const int nchunks = Kpad / kChunk;
    volatile int* abort_flag = &cb->abort_flag;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mb_init(&cb->raw_full[s], 1); mb_init(&cb->raw_empty[s], 4); mb_init(&cb->a_full[s], 4); mb_init(&cb->a_empty[s], 1); }
        mb_init(&cb->acc_full, 1); mb_init(&cb->acc_empty, 4); mb_init(&cb->w_full, 1);
        cb->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    for (int i = tid; i < 128; i += kThreads) cb->rows[i] = tbl[i];
    if (warp == 2) {   // tensor-memory allocation: all 512 columns, by one warp, which also frees them
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(s32(&cb->tmem_base)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem = cb->tmem_base;
    const uint32_t kDhi = 0, kDlo = 128, kA0 = 256;

    if (warp == 0) {
        // ------------------------------------------------ producer
        if (lane == 0) {
            mb_expect_tx(&cb->w_full, (uint32_t)Kpad * 512u);
            bulk_g2s(Wsm, Wk, (uint32_t)Kpad * 512u, &cb->w_full);
        }
        int64_t q = 0;
        bool ok = true;
        for (int64_t tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
            for (int c = 0; c < nchunks && ok; ++c, ++q) {
                const int s = (int)(q % kStages);
                const uint32_t ph = (uint32_t)((q / kStages) & 1);
                if (!mb_wait(&cb->raw_empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
                if (lane == 0) mb_expect_tx(&cb->raw_full[s], kRawStageBytes);
                __syncwarp();
                const int u = c * kChunk + lane;
                bulk_g2s(raw + (size_t)s * (kChunk * kTile) + lane * kTile, X + (int64_t)src_row[u] * P + tile * kTile,
                         kTile * 4u, &cb->raw_full[s]);
            }
        }
        if (!ok && lane == 0) { atomicCAS(err_word, 0, ERR_TC_WAIT | 1); cb->abort_flag = 1; }
    } else if (warp == 1) {
        // ------------------------------------------------ MMA issue
        if (lane == 0) {
            bool ok = mb_wait(&cb->w_full, 0, abort_flag);
            int64_t q = 0, tcount = 0;
            const uint32_t wbase = s32(Wsm);
            for (int64_t tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tcount) {
                if (!mb_wait(&cb->acc_empty, (uint32_t)((tcount & 1) ^ 1), abort_flag)) { ok = false; break; }
                fence_after();
                for (int c = 0; c < nchunks; ++c, ++q) {
                    const int s = (int)(q % kStages);
                    if (!mb_wait(&cb->a_full[s], (uint32_t)((q / kStages) & 1), abort_flag)) { ok = false; break; }
                    fence_after();
                    const uint32_t a_hi = tmem + kA0 + s * 64, a_lo = a_hi + 32;
#pragma unroll
                    for (int j = 0; j < kChunk / 8; ++j) {
                        // B operand: 8 K-columns of A^T = two core-matrix columns, 2048 bytes apart; 8-row groups 128 bytes apart
                        const uint64_t bd = smem_desc(wbase + (uint32_t)(c * (kChunk / 4) + j * 2) * 2048u, 2048u, 128u);
                        const uint32_t acc = (c > 0 || j > 0) ? 1u : 0u;
                        mma_tf32_ts(tmem + kDhi, a_hi + j * 8, bd, acc);
                        mma_tf32_ts(tmem + kDlo, a_lo + j * 8, bd, acc);
                    }
                    mma_commit(&cb->a_empty[s]);
                }
                if (!ok) break;
                mma_commit(&cb->acc_full);
            }
            if (!ok) { atomicCAS(err_word, 0, ERR_TC_WAIT | 2); cb->abort_flag = 1; }
        }
    } else if (warp >= 4 && warp < 8) {
        // ------------------------------------------------ converters (lane quarter = warp % 4)
        const int col = (warp - 4) * 32 + lane;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        int64_t q = 0;
        bool ok = true;
        for (int64_t tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
            for (int c = 0; c < nchunks; ++c, ++q) {
                const int s = (int)(q % kStages);
                const uint32_t ph = (uint32_t)((q / kStages) & 1);
                if (!mb_wait(&cb->raw_full[s], ph, abort_flag) || !mb_wait(&cb->a_empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
                fence_after();
                const float* r = raw + (size_t)s * (kChunk * kTile) + col;
                uint32_t hi[32], lo[32];
#pragma unroll
                for (int u = 0; u < 32; ++u) {
                    const float x = r[u * kTile];
                    hi[u] = to_tf32(x);
                    lo[u] = to_tf32(x - __uint_as_float(hi[u]));
                }
                const uint32_t a_hi = tmem + lane_base + kA0 + s * 64;
                tmem_st32(a_hi, hi);
                tmem_st32(a_hi + 32, lo);
                asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
                fence_before();
                __syncwarp();
                if (lane == 0) { mb_arrive(&cb->a_full[s]); mb_arrive(&cb->raw_empty[s]); }
            }
        }
        if (!ok && lane == 0) { atomicCAS(err_word, 0, ERR_TC_WAIT | 3); cb->abort_flag = 1; }
    } else if (warp >= 8) {
        // ------------------------------------------------ epilogue (lane quarter = warp % 4)
        const int col = (warp - 8) * 32 + lane;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        int64_t tcount = 0;
        bool ok = true;
        for (int64_t tile = blockIdx.x; tile < tiles; tile += gridDim.x, ++tcount) {
            if (!mb_wait(&cb->acc_full, (uint32_t)(tcount & 1), abort_flag)) { ok = false; break; }
            fence_after();
            float acc[128];
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                float h[32], l[32];
                tmem_ld32(tmem + lane_base + kDhi + b * 32, h);
                tmem_ld32(tmem + lane_base + kDlo + b * 32, l);
#pragma unroll
                for (int i = 0; i < 32; ++i) acc[b * 32 + i] = h[i] + l[i];
            }
            fence_before();
            __syncwarp();
            if (lane == 0) mb_arrive(&cb->acc_empty);       // the next tile's MMAs may overwrite the accumulators now
            const int64_t c0 = tile * kTile + col;
#pragma unroll
            for (int b = 0; b < 128; b += 16) {
                float g[16];
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const HopTcRow rw = cb->rows[b + i];
                    g[i] = (rw.g_row >= 0) ? __ldcs(G + (int64_t)rw.g_row * P + c0) : 0.f;
                }
#pragma unroll
                for (int i = 0; i < 16; ++i) {
                    const HopTcRow rw = cb->rows[b + i];
                    if (rw.out_row >= 0) X[(int64_t)rw.out_row * P + c0] = fmaf(-lr, g[i], __fdiv_rn(acc[b + i], rw.den));
                }
            }
        }
        if (!ok && lane == 0) { atomicCAS(err_word, 0, ERR_TC_WAIT | 4); cb->abort_flag = 1; }
    }
    fence_before();
    __syncthreads();
    if (warp == 2) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, 512;" ::"r"(tmem) : "memory");
}

}  // namespace

size_t hop_dense_tc_smem(int Kpad) { return 4096 + (size_t)Kpad * 512 + (size_t)kStages * kRawStageBytes; }

int hop_launch_mix_dense_tc(const HopLaunchCfg& c, const float* Wk, const HopTcRow* tbl, const int32_t* src_row, int Kpad) {
    const size_t smem = hop_dense_tc_smem(Kpad);
    cudaError_t e = cudaFuncSetAttribute(mix_dense_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return (int)e;
    const int64_t tiles = c.P / kTile;
    const int grid = (int)std::min<int64_t>(tiles, (int64_t)c.sm_count);
    mix_dense_tc_kernel<<<grid, kThreads, smem, (cudaStream_t)c.stream>>>(c.X, c.G, c.P, c.lr, Wk, tbl, src_row, Kpad, c.err_word);
    return (int)cudaGetLastError();
}
