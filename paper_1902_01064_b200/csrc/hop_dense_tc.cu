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
//   warps 0, 2  producers: the 16 raw X row pieces of a K-chunk as four TMA tile::gather4 loads (4 arbitrary rows
//               of the ring per instruction), two per warp: a warp issues at ~27 ns per row fetched (measured)
//   warp 1      MMA issue (one elected lane): tcgen05.mma kind::tf32, M=128 (columns) x N=128 (workers) x K=8,
//               A operand (X_hi / X_lo) from tensor memory, B operand (A^T, resident) from shared memory
//   warp 3      gradient loader and result storer: the tile's N x 128 piece of G comes in, and the finished results
//               leave, in quarters of 32 workers (2-D TMA boxes; one bulk row copy per active worker when some
//               workers are idle in the level); a quarter is refilled as soon as its results have been read out
//   warps 4-11  converters, two groups taking alternate chunks: lane = column; read the raw chunk from shared
//               memory, split hi/lo with round-to-nearest TF32 splitting, tcgen05.st into the A stages
//   warps 12-19 epilogue, two groups owning 64 workers each: tcgen05.ld both accumulators, add, release them, then
//               y = acc/den - lr*g written over g in shared memory, quarter by quarter
// Tensor memory (512 columns): D_hi 0..127, D_lo 128..255, four A stages of 64 columns (two chunks of hi 16 + lo 16).
// Shared memory: control block, A^T (Kpad x 512 B), four (or two) 16 KB gradient / result quarters, 3..8 raw stages of 8 KB.
// Every wait is bounded; a time-out sets the error word and lets the block run to its normal exit,
// where tensor memory is released.
#include <cuda.h>            // CUtensorMap and the cuTensorMapEncodeTiled prototype only; no libcuda link
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstring>

#include "hop_internal.h"

namespace {

constexpr int kTile = 128;          // parameter columns per tile = MMA M
constexpr int kChunk = 16;          // K rows per pipeline stage
constexpr int kStages = 8;          // most raw shared-memory stages (3..8, chosen by the host)
constexpr int kAStages = 4;         // tensor-memory A stages of two chunks each (one per converter group)
constexpr int kThreads = 20 * 32;
constexpr uint32_t kSpin = 1u << 20;
constexpr int kRawStageBytes = kChunk * kTile * 4;          // 8 KB
constexpr int kGQuarterBytes = 32 * kTile * 4;              // 16 KB: 32 workers x 128 columns of gradients / results
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
// TMA tensor-map loads (2-D, no swizzle).  x is the column (multiple of 4 floats: 16-byte rule), y the row.
__device__ __forceinline__ void tma_gather4(void* dst, const CUtensorMap* map, int x, int y0, int y1, int y2, int y3, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cta.global.tile::gather4.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5, %6}], [%7];"
                 ::"r"(s32(dst)), "l"(map), "r"(x), "r"(y0), "r"(y1), "r"(y2), "r"(y3), "r"(s32(bar)) : "memory");
}
__device__ __forceinline__ void tma_tile2d(void* dst, const CUtensorMap* map, int x, int y, uint64_t* bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cta.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(s32(dst)), "l"(map), "r"(x), "r"(y), "r"(s32(bar)) : "memory");
}
// Round to TF32 (10 explicit mantissa bits), nearest with ties away from zero, on the integer pipe: add half
// an ulp to the magnitude and clear the 13 low bits.  Same result as cvt.rna.tf32.f32 for finite inputs, but
// that conversion instruction issues at a fraction of the integer rate and made the converter warps the
// slowest stage (measured).
__device__ __forceinline__ uint32_t to_tf32(float x) { return (__float_as_uint(x) + 0x1000u) & 0xFFFFE000u; }

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
// 16 columns of both accumulators for this thread's lane, added: one wait for the two loads.
__device__ __forceinline__ void tmem_ld16_sum(uint32_t t_hi, uint32_t t_lo, float* out) {
    uint32_t h[16], l[16];
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(h[0]), "=r"(h[1]), "=r"(h[2]), "=r"(h[3]), "=r"(h[4]), "=r"(h[5]), "=r"(h[6]), "=r"(h[7]), "=r"(h[8]), "=r"(h[9]),
                   "=r"(h[10]), "=r"(h[11]), "=r"(h[12]), "=r"(h[13]), "=r"(h[14]), "=r"(h[15]) : "r"(t_hi) : "memory");
    asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                 : "=r"(l[0]), "=r"(l[1]), "=r"(l[2]), "=r"(l[3]), "=r"(l[4]), "=r"(l[5]), "=r"(l[6]), "=r"(l[7]), "=r"(l[8]), "=r"(l[9]),
                   "=r"(l[10]), "=r"(l[11]), "=r"(l[12]), "=r"(l[13]), "=r"(l[14]), "=r"(l[15]) : "r"(t_lo) : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
    for (int i = 0; i < 16; ++i) out[i] = __uint_as_float(h[i]) + __uint_as_float(l[i]);
}

struct TcRowConsts {
    float inv_den[128];                  // 1 / (sum of the worker's integer weights)
    uint32_t active_mask[4], g_mask[4];  // bit i of word i/32: worker i writes a result / applies a gradient
};

struct TcSmem {                       // control block at the start of dynamic shared memory
    uint64_t raw_full[kStages], raw_empty[kStages], a_full[kStages], a_empty[kStages];
    uint64_t acc_full, acc_empty, w_full;
    uint64_t g_full[4], y_full[4];        // one pair per quarter (32 workers) of the gradient / result tile
    uint32_t tmem_base;
    int abort_flag;
    alignas(16) int32_t src[256];         // ring row of each of the K consumed slices (read by the producers for every chunk)
    HopTcRow rows[128];
};
static_assert(sizeof(TcSmem) <= 4096, "control block");

__global__ void __launch_bounds__(kThreads, 1)
mix_dense_tc_kernel(const __grid_constant__ CUtensorMap mapX, const __grid_constant__ CUtensorMap mapG,
                    const __grid_constant__ CUtensorMap mapY, int box_store,
                    float* __restrict__ X, int64_t P, int n_workers, float lr, const float* __restrict__ Wk,
                    const HopTcRow* __restrict__ tbl, const int32_t* __restrict__ src_row, int Kpad, int raw_stages, int g_bufs,
                    int32_t* __restrict__ err_word, const __grid_constant__ TcRowConsts rc) {
    extern __shared__ __align__(1024) unsigned char smem[];
    TcSmem* cb = reinterpret_cast<TcSmem*>(smem);
    float* Wsm = reinterpret_cast<float*>(smem + 4096);                        // Kpad * 512 bytes, canonical K-major
    // Gradient / result quarters of [32 workers][128 columns]: four buffers (one per quarter of the tile), or two (one per
    // epilogue group, used for its two quarters in turn) when the weight matrix leaves too little room for raw stages
    float* Gsm = reinterpret_cast<float*>(smem + 4096 + (size_t)Kpad * 512);
    float* raw = Gsm + g_bufs * 32 * kTile;                                    // raw_stages x [16][128] floats
    auto g_buf = [&](int q) -> float* { return Gsm + (g_bufs == 4 ? q : (q >> 1)) * 32 * kTile; };
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int64_t tiles = P / kTile;
    const int nchunks = Kpad / kChunk;
    volatile int* abort_flag = &cb->abort_flag;

    if (tid == 0) {
        for (int s = 0; s < kStages; ++s) { mb_init(&cb->raw_full[s], 2); mb_init(&cb->raw_empty[s], 4); mb_init(&cb->a_full[s], 8); mb_init(&cb->a_empty[s], 1); }
        mb_init(&cb->acc_full, 1); mb_init(&cb->acc_empty, 8); mb_init(&cb->w_full, 1);
        for (int q = 0; q < 4; ++q) { mb_init(&cb->g_full[q], 1); mb_init(&cb->y_full[q], 4); }
        cb->abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    for (int i = tid; i < 128; i += kThreads) cb->rows[i] = tbl[i];
    for (int i = tid; i < Kpad; i += kThreads) cb->src[i] = src_row[i];
    if (warp == 2) {   // tensor-memory allocation: all 512 columns, by one warp, which also frees them
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], 512;" ::"r"(s32(&cb->tmem_base)) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem = cb->tmem_base;
    const uint32_t kDhi = 0, kDlo = 128, kA0 = 256;

    if (warp == 0 || warp == 2) {
        // ------------------------------------------------ producers: two warps, two gather4 loads each per chunk
        // (a warp issues its TMA loads one after the other, ~27 ns per row fetched: one warp alone cannot keep up)
        const int half = warp >> 1;
        if (warp == 0 && lane == 0) {
            mb_expect_tx(&cb->w_full, (uint32_t)Kpad * 512u);
            bulk_g2s(Wsm, Wk, (uint32_t)Kpad * 512u, &cb->w_full);
        }
        int s = 0;             // raw stage and its phase bit, advanced by hand (raw_stages is not a power of two)
        uint32_t ph = 0;
        bool ok = true;
        for (int64_t tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x) {
            for (int c = 0; c < nchunks && ok; ++c) {
                if (!mb_wait(&cb->raw_empty[s], ph ^ 1u, abort_flag)) { ok = false; break; }
                if (lane == 0) mb_expect_tx(&cb->raw_full[s], kRawStageBytes / 2);
                __syncwarp();
                if (lane < 2) {
                    const int r4 = half * 2 + lane;                 // which group of four rows of the chunk
                    const int u = c * kChunk + r4 * 4;
                    const int4 rows4 = *reinterpret_cast<const int4*>(&cb->src[u]);
                    tma_gather4(raw + (size_t)s * (kChunk * kTile) + r4 * 4 * kTile, &mapX, (int)(tile * kTile),
                                rows4.x, rows4.y, rows4.z, rows4.w, &cb->raw_full[s]);
                }
                if (++s == raw_stages) { s = 0; ph ^= 1u; }
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
                // One wait, fence and commit per pair of chunks: waiting, fencing and committing cost this thread
                // more than the four MMAs of a chunk take on the tensor pipe (measured), and this thread sets the
                // pace of the main loop.
                for (int c = 0; c < nchunks; c += 2, ++q) {
                    const int s = (int)(q % kAStages);
                    if (!mb_wait(&cb->a_full[s], (uint32_t)((q / kAStages) & 1), abort_flag)) { ok = false; break; }
                    fence_after();
#pragma unroll
                    for (int h = 0; h < 2; ++h) {
                        const uint32_t a_hi = tmem + kA0 + s * 64 + h * 32, a_lo = a_hi + 16;
#pragma unroll
                        for (int j = 0; j < kChunk / 8; ++j) {
                            // B operand: 8 K-columns of A^T = two core-matrix columns, 2048 bytes apart; 8-row groups 128 bytes apart
                            const uint64_t bd = smem_desc(wbase + (uint32_t)((c + h) * (kChunk / 4) + j * 2) * 2048u, 2048u, 128u);
                            const uint32_t acc = (c > 0 || h > 0 || j > 0) ? 1u : 0u;
                            mma_tf32_ts(tmem + kDhi, a_hi + j * 8, bd, acc);
                            mma_tf32_ts(tmem + kDlo, a_lo + j * 8, bd, acc);
                        }
                    }
                    mma_commit(&cb->a_empty[s]);
                }
                if (!ok) break;
                mma_commit(&cb->acc_full);
            }
            if (!ok) { atomicCAS(err_word, 0, ERR_TC_WAIT | 2); cb->abort_flag = 1; }
        }
    } else if (warp == 3) {
        // ------------------------------------------------ gradient loader and result storer.  The gradient / result
        // tile is handled in quarters of 32 workers: g_full[q] tells the epilogue that quarter q holds the gradients
        // of its tile, y_full[q] tells this warp that the results have replaced them.  This warp then sends the
        // quarter out, waits until the copy engine has read it, and refills it with the next tile's gradients, so
        // the epilogue warps never wait for a store (as one chain load -> compute -> store took 4.4 of 5.8 us per
        // tile, measured).  Without gradients the refill is a plain arrival: g_full then only says "free".
        const bool has_g = (rc.g_mask[0] | rc.g_mask[1] | rc.g_mask[2] | rc.g_mask[3]) != 0;
        const int nq = (n_workers + 31) / 32;
        const uint32_t qbytes = (uint32_t)min(32, n_workers) * kTile * 4u;      // the box of the map; rows out of range arrive as zeros
        auto refill = [&](int q, int64_t tile) {
            if (has_g) {
                mb_expect_tx(&cb->g_full[q], qbytes);
                tma_tile2d(g_buf(q), &mapG, (int)(tile * kTile), q * 32, &cb->g_full[q]);
            } else {
                mb_arrive(&cb->g_full[q]);
            }
        };
        // With two buffers a buffer serves quarters 2h and 2h+1 of a tile in turn: the even quarters go first, and
        // what a buffer is refilled with after a store is the next quarter that lives in it.
        const int n_even = (nq + 1) / 2;
        if (lane == 0 && (int64_t)blockIdx.x < tiles)
            for (int q = 0; q < nq; q += (g_bufs == 4 ? 1 : 2)) refill(q, blockIdx.x);
        // With four buffers the refill of a quarter is deferred by one step: this warp issues the next quarter's store
        // first and only then waits until the copy engine has read the previous one (wait_group.read 1).  Waiting after
        // every store put ~1 us per quarter, four times per tile, on this warp alone: the kernel ran at 4.6 us per tile
        // even without any gradient traffic (measured).  Every lane commits one group per quarter (empty for lanes
        // that store nothing), so the group counts agree across the warp.
        const bool defer = g_bufs == 4;
        int pend_q = -1;
        int64_t pend_tile = 0;
        int64_t tcount = 0;
        bool ok = true;
        for (int64_t tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tcount) {
            for (int i = 0; i < nq; ++i) {
                const int q = g_bufs == 4 ? i : (i < n_even ? 2 * i : 2 * (i - n_even) + 1);
                if (!mb_wait(&cb->y_full[q], (uint32_t)(tcount & 1), abort_flag)) { ok = false; break; }
                if (box_store) {
                    if (lane == 0)     // all workers active: one box [32 workers x 128] into the output slot
                        asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.tile.bulk_group [%0, {%1, %2}], [%3];"
                                     ::"l"(&mapY), "r"((int)(tile * kTile)), "r"(q * 32), "r"(s32(g_buf(q))) : "memory");
                } else {               // one 512-byte row copy per active worker of the quarter
                    const HopTcRow rw = cb->rows[q * 32 + lane];
                    if (rw.out_row >= 0)
                        asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;"
                                     ::"l"(X + (int64_t)rw.out_row * P + tile * kTile), "r"(s32(g_buf(q) + lane * kTile)), "r"(kTile * 4) : "memory");
                }
                asm volatile("cp.async.bulk.commit_group;" ::: "memory");
                if (!defer) {
                    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
                    __syncwarp();          // the quarter has been read out of shared memory
                    if (lane == 0) {
                        if (!(q & 1) && q + 1 < nq) refill(q + 1, tile);
                        else if (tile + gridDim.x < tiles) refill(q & ~1, tile + gridDim.x);
                    }
                } else {
                    if (pend_q >= 0) {
                        asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
                        __syncwarp();      // the previous quarter has been read out of shared memory
                        if (lane == 0 && pend_tile + gridDim.x < tiles) refill(pend_q, pend_tile + gridDim.x);
                    }
                    pend_q = q;
                    pend_tile = tile;
                }
            }
        }
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // this thread's stores have reached global memory
        if (!ok && lane == 0) { atomicCAS(err_word, 0, ERR_TC_WAIT | 5); cb->abort_flag = 1; }
    } else if (warp >= 4 && warp < 12) {
        // ------------------------------------------------ converters (lane quarter = warp % 4): two groups of four
        // warps, the first takes the even chunks, the second the odd ones; a tensor-memory stage holds one chunk of
        // each (32 columns per group: hi 16 + lo 16).  With one group the converter warps, at one busy warp per
        // scheduler, ran at ~0.2 instructions per cycle and set the pace of the block (measured).
        const int par = (warp - 4) >> 2;
        const int col = ((warp - 4) & 3) * 32 + lane;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const int64_t my_tiles = (int64_t)blockIdx.x < tiles ? (tiles - blockIdx.x + gridDim.x - 1) / gridDim.x : 0;
        const int64_t total = my_tiles * nchunks;
        bool ok = true;
        // The tensor-memory store of a chunk is left in flight while this warp's next chunk is fetched from shared
        // memory; the chunk is published to the MMA warp (a_full) once tcgen05.wait::st has covered it.
        int pending = -1;
        auto publish = [&]() {
            asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory");
            fence_before();
            __syncwarp();
            if (lane == 0) mb_arrive(&cb->a_full[pending]);
            pending = -1;
        };
        int rs = par;              // raw stage of chunk q and its phase bit, advanced by hand (3 <= raw_stages <= 8)
        uint32_t rph = 0;
        for (int64_t q = par; q < total; q += 2) {
            const int s = (int)((q >> 1) & (kAStages - 1));
            // With an odd number of raw stages a stage alternates between the two groups, and this group may get here
            // before the other one has even seen the stage's previous chunk: the parity test on raw_full would then
            // pass on that older phase.  So first make sure the previous chunk of the stage has been released.
            if (pending >= 0 && !(mb_try(&cb->raw_empty[rs], rph ^ 1u) && mb_try(&cb->raw_full[rs], rph))) publish();   // nothing to overlap with
            if (!mb_wait(&cb->raw_empty[rs], rph ^ 1u, abort_flag)) { ok = false; break; }
            if (!mb_wait(&cb->raw_full[rs], rph, abort_flag)) { ok = false; break; }
            const float* r = raw + (size_t)rs * (kChunk * kTile) + col;
            float x[kChunk];
#pragma unroll
            for (int u = 0; u < kChunk; ++u) x[u] = r[u * kTile];
            if (pending >= 0) publish();
            if (!mb_wait(&cb->a_empty[s], (uint32_t)((((q >> 1) / kAStages) & 1) ^ 1), abort_flag)) { ok = false; break; }
            fence_after();
            uint32_t v[2 * kChunk];                      // hi in columns 0..15 of this group's half of the stage, lo in 16..31
#pragma unroll
            for (int u = 0; u < kChunk; ++u) {
                v[u] = to_tf32(x[u]);
                v[kChunk + u] = to_tf32(x[u] - __uint_as_float(v[u]));
            }
            __syncwarp();
            if (lane == 0) mb_arrive(&cb->raw_empty[rs]);   // the raw chunk is in registers
            tmem_st32(tmem + lane_base + kA0 + s * 64 + par * 32, v);
            pending = s;
            rs += 2;
            if (rs >= raw_stages) { rs -= raw_stages; rph ^= 1u; }
        }
        if (pending >= 0) publish();
        if (!ok && lane == 0) { atomicCAS(err_word, 0, ERR_TC_WAIT | 3); cb->abort_flag = 1; }
    } else if (warp >= 12) {
        // ------------------------------------------------ epilogue (lane quarter = warp % 4): two groups of four warps,
        // the first owns workers 0..63 (quarters 0, 1 of the tile), the second workers 64..127 (quarters 2, 3).
        // The loop over the workers has to be unrolled (the accumulators are registers), and the unrolled code is
        // what every tile streams through the instruction cache: one copy serves both groups (the group only
        // moves base addresses), and the usual quarter, where every worker is active and has a gradient, has a
        // body without the mask tests.
        const int half = (warp - 12) >> 2;
        const int col = ((warp - 12) & 3) * 32 + lane;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const int nq = (n_workers + 31) / 32;
        int64_t tcount = 0;
        bool ok = true;
        for (int64_t tile = blockIdx.x; tile < tiles && ok; tile += gridDim.x, ++tcount) {
            if (!mb_wait(&cb->acc_full, (uint32_t)(tcount & 1), abort_flag)) { ok = false; break; }
            fence_after();
            float acc[64];
            if (half * 2 < nq) {
#pragma unroll
                for (int j = 0; j < 4; ++j) tmem_ld16_sum(tmem + lane_base + kDhi + half * 64 + j * 16, tmem + lane_base + kDlo + half * 64 + j * 16, acc + j * 16);
            }
            fence_before();
            __syncwarp();
            if (lane == 0) mb_arrive(&cb->acc_empty);   // the next tile's MMAs may overwrite the accumulators now
            // y = acc/den - lr*g replaces g in the shared tile (column-per-thread: conflict-free), then the tile leaves
            // through the copy engine: per-thread 4-byte global stores of 128 different rows were the slowest part of
            // the kernel by far (measured).
#pragma unroll
            for (int qq = 0; qq < 2; ++qq) {
                const int q = half * 2 + qq;
                if (q < nq && ok) {
                    if (!mb_wait(&cb->g_full[q], (uint32_t)(tcount & 1), abort_flag)) { ok = false; }
                    else {
                        float* Gq = g_buf(q) + col;
                        const float* dq = rc.inv_den + q * 32;
                        const uint32_t amq = rc.active_mask[q], gmq = rc.g_mask[q];
                        // Batches of 8 rows, the gradients of the next batch fetched before the stores of this one:
                        // the compiler cannot prove that the stores do not alias later loads, and a load-store-load
                        // chain per row cost ~100 cycles per row (measured).
                        float g[8], gn[8];
                        if (amq == 0xffffffffu && gmq == 0u) {
                            // no gradient in this kernel at all (serial approach, jump-only levels): scale and store;
                            // through the masked body below this took 4.3 us per tile instead of 1 (measured)
#pragma unroll
                            for (int b = 0; b < 32; ++b) Gq[b * kTile] = acc[qq * 32 + b] * dq[b];
                        } else if (amq == 0xffffffffu && gmq == 0xffffffffu) {
#pragma unroll
                            for (int i = 0; i < 8; ++i) g[i] = Gq[i * kTile];
#pragma unroll
                            for (int b = 0; b < 32; b += 8) {
                                if (b + 8 < 32) {
#pragma unroll
                                    for (int i = 0; i < 8; ++i) gn[i] = Gq[(b + 8 + i) * kTile];
                                }
#pragma unroll
                                for (int i = 0; i < 8; ++i) Gq[(b + i) * kTile] = fmaf(-lr, g[i], acc[qq * 32 + b + i] * dq[b + i]);
#pragma unroll
                                for (int i = 0; i < 8; ++i) g[i] = gn[i];
                            }
                        } else {
#pragma unroll
                            for (int i = 0; i < 8; ++i) g[i] = Gq[i * kTile];   // stale but unused when the row has no gradient
#pragma unroll
                            for (int b = 0; b < 32; b += 8) {
                                if (b + 8 < 32) {
#pragma unroll
                                    for (int i = 0; i < 8; ++i) gn[i] = Gq[(b + 8 + i) * kTile];
                                }
#pragma unroll
                                for (int i = 0; i < 8; ++i) {
                                    const float gv = ((gmq >> (b + i)) & 1u) ? g[i] : 0.f;
                                    if ((amq >> (b + i)) & 1u) Gq[(b + i) * kTile] = fmaf(-lr, gv, acc[qq * 32 + b + i] * dq[b + i]);
                                }
#pragma unroll
                                for (int i = 0; i < 8; ++i) g[i] = gn[i];
                            }
                        }
                        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // results visible to the copy engine
                        __syncwarp();
                        if (lane == 0) mb_arrive(&cb->y_full[q]);
                    }
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

// Four gradient / result buffers while at least seven raw stages fit beside them, else two (32 KB more for raw
// stages).  Two buffers put a load latency inside each epilogue group's chain, which costs ~10 % when the raw stages
// were not the limit (K = 192, measured); with five or fewer raw stages the stages matter more (K >= 224).
static void tc_layout(int Kpad, int* g_bufs, int* raw_stages) {
    const long free_bytes = 227L * 1024 - 4096 - (long)Kpad * 512;
    const long st4 = std::min<long>(kStages, (free_bytes - 4 * kGQuarterBytes) / kRawStageBytes);
    const long st2 = std::min<long>(kStages, (free_bytes - 2 * kGQuarterBytes) / kRawStageBytes);
    *g_bufs = st4 >= kStages - 1 ? 4 : 2;
    *raw_stages = (int)std::max(0L, *g_bufs == 4 ? st4 : st2);
}
// 0 when the level does not fit (fewer than 3 raw stages)
size_t hop_dense_tc_smem(int Kpad) {
    int gb, st;
    tc_layout(Kpad, &gb, &st);
    return st < 3 ? 0 : 4096 + (size_t)Kpad * 512 + (size_t)gb * kGQuarterBytes + (size_t)st * kRawStageBytes;
}

// Tensor maps: X as [N*(s+1) rows][P] with a one-row box of 128 columns (the tile::gather4 form loads four
// such rows), G as [N rows][P] with a min(32, N) x 128 box (one quarter of a tile).  cuTensorMapEncodeTiled is looked up through the
// runtime so that the library does not link against the driver.
// mapY[slot]: the rows {i*(s+1) + slot} of X, i.e. the output slot of a level, as an [N rows][P] tensor with row
// stride (s+1)*P and the same box as G (n_slots maps of 128 bytes each).
int hop_dense_tc_make_maps(float* X, int64_t ring_rows, const float* G, int32_t N, int64_t P, void* mapX, void* mapG,
                           void* mapY, int32_t n_slots) {
    typedef CUresult (*EncodeFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                 const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    static EncodeFn encode = nullptr;
    if (!encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
        if (e != cudaSuccess) return (int)e;
        if (!fn || q != cudaDriverEntryPointSuccess) return (int)cudaErrorNotSupported;
        encode = (EncodeFn)fn;
    }
    alignas(64) CUtensorMap m;
    const cuuint32_t estr[2] = {1, 1};
    {
        const cuuint64_t dims[2] = {(cuuint64_t)P, (cuuint64_t)ring_rows};
        const cuuint64_t strides[1] = {(cuuint64_t)P * 4};
        const cuuint32_t box[2] = {(cuuint32_t)kTile, 1};
        if (encode(&m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, X, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return (int)cudaErrorInvalidValue;
        std::memcpy(mapX, &m, sizeof(m));
    }
    if (G) {
        const cuuint64_t dims[2] = {(cuuint64_t)P, (cuuint64_t)N};
        const cuuint64_t strides[1] = {(cuuint64_t)P * 4};
        const cuuint32_t box[2] = {(cuuint32_t)kTile, (cuuint32_t)std::min(32, N)};
        if (encode(&m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<float*>(G), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return (int)cudaErrorInvalidValue;
    }
    std::memcpy(mapG, &m, sizeof(m));
    const int64_t S = ring_rows / N;
    for (int slot = 0; slot < n_slots; ++slot) {
        const cuuint64_t dims[2] = {(cuuint64_t)P, (cuuint64_t)N};
        const cuuint64_t strides[1] = {(cuuint64_t)S * P * 4};
        const cuuint32_t box[2] = {(cuuint32_t)kTile, (cuuint32_t)std::min(32, N)};
        if (encode(&m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, X + (int64_t)slot * P, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_NONE, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) != CUDA_SUCCESS)
            return (int)cudaErrorInvalidValue;
        std::memcpy((unsigned char*)mapY + 128 * slot, &m, sizeof(m));
    }
    return 0;
}

int hop_launch_mix_dense_tc(const HopLaunchCfg& c, const void* mapX, const void* mapG, const void* mapY, const float* Wk,
                            const HopTcRow* tbl, const int32_t* src_row, int Kpad, const HopTcRow* host_rows) {
    alignas(64) CUtensorMap mx, mg, my;
    std::memcpy(&mx, mapX, sizeof(mx));
    std::memcpy(&mg, mapG, sizeof(mg));
    std::memcpy(&my, mapY ? mapY : mapX, sizeof(my));
    TcRowConsts rc{};
    for (int i = 0; i < 128; ++i) {
        rc.inv_den[i] = host_rows[i].inv_den;
        rc.active_mask[i >> 5] |= (uint32_t)(host_rows[i].out_row >= 0) << (i & 31);
        rc.g_mask[i >> 5] |= (uint32_t)(host_rows[i].g_row >= 0) << (i & 31);
    }
    const size_t smem = hop_dense_tc_smem(Kpad);
    int gb, st;
    tc_layout(Kpad, &gb, &st);
    cudaError_t e = hop_allow_max_smem<mix_dense_tc_kernel>();
    if (e != cudaSuccess) return (int)e;
    const int64_t tiles = c.P / kTile;
    const int grid = (int)std::min<int64_t>(tiles, (int64_t)c.sm_count);
    mix_dense_tc_kernel<<<grid, kThreads, smem, (cudaStream_t)c.stream>>>(mx, mg, my, mapY ? 1 : 0, c.X, c.P, c.N, c.lr, Wk, tbl, src_row, Kpad,
                                                                          st, gb, c.err_word, rc);
    return (int)cudaGetLastError();
}
