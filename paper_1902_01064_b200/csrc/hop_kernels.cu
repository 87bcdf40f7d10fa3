// CUDA kernels of the Hop hot path for sm_100a.
//
//   mix_staged / mix_bulk   fused Recv-Reduce-Apply for one level: x_{k+1,i} = sum w * x_{v,j} - lr * d
//                           (Fig. alg0 steps 2-3, Reduce of Fig. alg4 / Eq. 2), SGD or momentum, weight decay
//   synth_grad              G[i][p] = sigma * normal(seed, i, k, p)
//   svm_margin_* / svm_dense_grad / svm_dense_fused / svm_csr_apply   hinge- or log-loss linear model gradient and sparse Apply
//   apply_dense             serial approach (Section 3.2): x_k <- x_k - lr * d before the level's Reduce
//   direction_dense         G <- update direction (momentum, weight decay) ahead of the dense-graph kernel
//   wait_selftest           a bounded wait that runs out, for the status-word path
// (the dense-graph tensor-core kernel lives in hop_dense_tc.cu)
//
// In-place ring: version k+1 of a worker overwrites the slot of version k-s, which other workers may
// consume in the same level.  A thread block therefore owns a column tile for ALL workers: it first
// brings every distinct consumed slice of the tile into shared memory, then writes.  Blocks own
// disjoint columns, so no other ordering is needed, and every distinct slice is read once.
#include <cuda_runtime.h>
#include <algorithm>
#include <cstdint>

#include "hop_internal.h"

namespace {

constexpr int kStagedThreads = 512;
constexpr int kConsumerWarps = 16;
constexpr int kProducerWarps = 8;   // a warp issues ~25-40 ns per small bulk copy, so several issue in parallel.  Measured with
                                    // 16 consumer warps: 4 / 6 / 8 producer warps 6.64 / 6.33 / 6.70 TB/s (and 12+6 6.64, 12+10 6.30,
                                    // 14+10 6.65, 10+10 6.63): every split but the two with 22 warps in all is within 1.5 %
constexpr int kBulkThreads = 32 * (kConsumerWarps + kProducerWarps);
constexpr int kBulkStages = 2;
constexpr uint32_t kSpinLimit = 1u << 22;

enum : int32_t { ERR_FULL_WAIT = 1 << 24, ERR_EMPTY_WAIT = 2 << 24, ERR_BOUNDS = 4 << 24 };

// Checked build (-DHOP_CHECKED, a separate library used by the tests; compute-sanitizer's place): every global-memory
// source of a bulk copy or cp.async, and every gather of the SVM kernels, is first tested against the bound buffers
// X, M and G.  An access outside them is recorded (status code 4, detail = which site) and skipped, never made.
#ifdef HOP_CHECKED
struct HopFence { const char* lo[3]; const char* hi[3]; int32_t* err; };
__device__ HopFence g_fence;
__device__ __forceinline__ bool fence_ok(const void* p, size_t bytes, int site) {
    const char* a = static_cast<const char*>(p);
#pragma unroll
    for (int k = 0; k < 3; ++k)
        if (g_fence.lo[k] != nullptr && a >= g_fence.lo[k] && a + bytes <= g_fence.hi[k]) return true;
    if (g_fence.err != nullptr) atomicCAS(g_fence.err, 0, ERR_BOUNDS | site);
    return false;
}
#define HOP_FENCE(ptr, bytes, site) do { if (!fence_ok((ptr), (bytes), (site))) return; } while (0)
#define HOP_FENCE_OR(ptr, bytes, site, fallback) (fence_ok((ptr), (bytes), (site)) ? *(ptr) : (fallback))
#define HOP_FENCED(ptr, bytes, site) fence_ok((ptr), (bytes), (site))
#else
#define HOP_FENCE(ptr, bytes, site) do { } while (0)
#define HOP_FENCE_OR(ptr, bytes, site, fallback) (*(ptr))
#define HOP_FENCED(ptr, bytes, site) true
#endif

// ------------------------------------------------------------------------------------------------
// Consumer math shared by both mix kernels: one warp produces the tile of one record.
// stage: [rows][w] floats; rows [0,U) consumed slices, [U,U+nG) gradients, [U+nG,U+2nG) momentum.
// ALIGNED = false (VEC = 4 only): the rows of X and M are not 16-byte aligned in global memory (P % 4 != 0), so the
// results leave as guarded scalar stores; shared memory is aligned either way.
template <int VEC, bool MOMENTUM, bool DECAY, bool ALIGNED = true>
__device__ __forceinline__ void reduce_apply_record(const HopRecord& r, const HopEntry* __restrict__ ents,
                                                    const float* __restrict__ stage, int w, int wd, int U, int nG,
                                                    bool use_g, float lr, float mu, float lam, float* __restrict__ X,
                                                    float* __restrict__ M, int64_t P, int64_t c0, int lane) {
    const HopEntry* e = ents + r.ent_begin;
    const int n = r.ent_count;
    float* out = X + (int64_t)r.out_row * P + c0;
    const bool grad = use_g && r.g_stage >= 0;
    // weight decay: lambda * x_{k,i} joins the gradient; x_{k,i} is the worker's own consumed slice.  With a sparse
    // gradient (no dense row) only the decay term is applied here, the data term by the sparse apply.
    const bool decay = DECAY && r.g_stage >= 0 && r.self_u >= 0;   // DECAY is a template flag: the common path carries no trace of it
    const float* grow = stage + (int64_t)(U + (grad ? r.g_stage : 0)) * w;
    const float* mrow = stage + (int64_t)(U + nG + (grad ? r.g_stage : 0)) * w;
    float* mout = MOMENTUM ? (M + (int64_t)r.worker * P + c0) : nullptr;
    for (int c = lane * VEC; c < wd; c += 32 * VEC) {
        if constexpr (VEC == 4) {
            float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
            const float* sc = stage + c;
            int t = 0;
#define HOP_FMA4(W, V) acc.x = fmaf(W, V.x, acc.x); acc.y = fmaf(W, V.y, acc.y); acc.z = fmaf(W, V.z, acc.z); acc.w = fmaf(W, V.w, acc.w)
            for (; t + 4 <= n; t += 4) {      // loads first, then the multiply-adds in entry order
                const HopEntry e0 = e[t], e1 = e[t + 1], e2 = e[t + 2], e3 = e[t + 3];
                const float4 v0 = *reinterpret_cast<const float4*>(sc + e0.u);
                const float4 v1 = *reinterpret_cast<const float4*>(sc + e1.u);
                const float4 v2 = *reinterpret_cast<const float4*>(sc + e2.u);
                const float4 v3 = *reinterpret_cast<const float4*>(sc + e3.u);
                HOP_FMA4(e0.w, v0); HOP_FMA4(e1.w, v1); HOP_FMA4(e2.w, v2); HOP_FMA4(e3.w, v3);
            }
            for (; t < n; ++t) {
                const HopEntry en = e[t];
                const float4 v = *reinterpret_cast<const float4*>(sc + en.u);
                HOP_FMA4(en.w, v);
            }
#undef HOP_FMA4
            if (decay && !grad) {
                const float4 xs = *reinterpret_cast<const float4*>(sc + r.self_u);
                const float k = -lr * lam;
                acc.x = fmaf(k, xs.x, acc.x); acc.y = fmaf(k, xs.y, acc.y); acc.z = fmaf(k, xs.z, acc.z); acc.w = fmaf(k, xs.w, acc.w);
            }
            if (grad) {
                float4 g = *reinterpret_cast<const float4*>(grow + c);
                if (decay) {
                    const float4 xs = *reinterpret_cast<const float4*>(sc + r.self_u);
                    g.x = fmaf(lam, xs.x, g.x); g.y = fmaf(lam, xs.y, g.y); g.z = fmaf(lam, xs.z, g.z); g.w = fmaf(lam, xs.w, g.w);
                }
                if constexpr (MOMENTUM) {
                    const float4 m = *reinterpret_cast<const float4*>(mrow + c);
                    g.x = fmaf(mu, m.x, g.x); g.y = fmaf(mu, m.y, g.y);
                    g.z = fmaf(mu, m.z, g.z); g.w = fmaf(mu, m.w, g.w);
                    if constexpr (ALIGNED) {
                        *reinterpret_cast<float4*>(mout + c) = g;
                    } else {
                        const float gv[4] = {g.x, g.y, g.z, g.w};
#pragma unroll
                        for (int q = 0; q < 4; ++q) if (c + q < wd) mout[c + q] = gv[q];
                    }
                }
                acc.x = fmaf(-lr, g.x, acc.x); acc.y = fmaf(-lr, g.y, acc.y);
                acc.z = fmaf(-lr, g.z, acc.z); acc.w = fmaf(-lr, g.w, acc.w);
            }
            if constexpr (ALIGNED) {
                *reinterpret_cast<float4*>(out + c) = acc;
            } else {
                const float av[4] = {acc.x, acc.y, acc.z, acc.w};
#pragma unroll
                for (int q = 0; q < 4; ++q) if (c + q < wd) out[c + q] = av[q];
            }
        } else {
            float acc = 0.f;
            for (int t = 0; t < n; ++t) {
                const HopEntry en = e[t];
                acc = fmaf(en.w, stage[en.u + c], acc);
            }
            if (decay && !grad) acc = fmaf(-lr * lam, stage[r.self_u + c], acc);
            if (grad) {
                float g = grow[c];
                if (decay) g = fmaf(lam, stage[r.self_u + c], g);
                if constexpr (MOMENTUM) {
                    g = fmaf(mu, mrow[c], g);
                    mout[c] = g;
                }
                acc = fmaf(-lr, g, acc);
            }
            out[c] = acc;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// mix_staged: the general kernel, for any P.  Persistent blocks, two shared-memory stages filled with cp.async by all
// threads (one warp per staged row), block-wide barriers: the copies of the next tile are in flight while this tile
// is computed.  MODE 0: P % 4 == 0, 16-byte copies, vector math and stores.  MODE 1: any P with a tile width that is
// a multiple of 4: 4-byte copies (the rows are not 16-byte aligned in global memory, the staged copy is), vector
// math, scalar stores.  MODE 2: scalar everything (tile widths below 32 that are not multiples of 4).
__device__ __forceinline__ void cp_async_4(float* dst, const float* src) {
    HOP_FENCE(src, 4, 1);
    asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_16(float* dst, const float* src) {
    HOP_FENCE(src, 16, 2);
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"((uint32_t)__cvta_generic_to_shared(dst)), "l"(src) : "memory");
}
template <int MODE, bool MOMENTUM, bool DECAY>
__global__ void __launch_bounds__(kStagedThreads, 1)
mix_staged_kernel(float* __restrict__ X, float* __restrict__ M, const float* __restrict__ G, int64_t P, int w,
                  int use_g, float lr, float mu, float lam, HopLevelDev lv) {
    extern __shared__ __align__(16) float smem[];
    constexpr int kWarps = kStagedThreads / 32;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nG = use_g ? lv.nG : 0;
    const int rows = lv.U + nG * (MOMENTUM ? 2 : 1);
    const int64_t stage_floats = (int64_t)rows * w;
    const int64_t tiles = (P + w - 1) / w;
    auto fetch = [&](int64_t tile, int stage) {
        const int64_t c0 = tile * w;
        const int wd = (int)min((int64_t)w, P - c0);
        float* dst0 = smem + stage * stage_floats;
        for (int r = warp; r < rows; r += kWarps) {
            const float* src;
            if (r < lv.U) src = X + (int64_t)lv.src_row[r] * P;
            else if (r < lv.U + nG) src = G + (int64_t)lv.grad_workers[r - lv.U] * P;
            else src = M + (int64_t)lv.grad_workers[r - lv.U - nG] * P;
            src += c0;
            float* dst = dst0 + (int64_t)r * w;
            if constexpr (MODE == 0) {
                for (int c = lane * 4; c < wd; c += 128) cp_async_16(dst + c, src + c);
            } else {
                for (int c = lane; c < wd; c += 32) cp_async_4(dst + c, src + c);
            }
        }
    };
    int n = 0;
    if ((int64_t)blockIdx.x < tiles) fetch(blockIdx.x, 0);
    asm volatile("cp.async.commit_group;" ::: "memory");
    for (int64_t tile = blockIdx.x; tile < tiles; tile += gridDim.x, ++n) {
        const int64_t next = tile + gridDim.x;
        if (next < tiles) fetch(next, (n + 1) & 1);
        asm volatile("cp.async.commit_group;" ::: "memory");          // one group per iteration, empty or not
        asm volatile("cp.async.wait_group 1;" ::: "memory");          // this tile's copies (of this thread) have landed
        __syncthreads();                                               // ... and everybody else's
        const int64_t c0 = tile * w;
        const int wd = (int)min((int64_t)w, P - c0);
        const float* st = smem + (n & 1) * stage_floats;
        for (int a = warp; a < lv.nA; a += kWarps) {
            if constexpr (MODE == 0)
                reduce_apply_record<4, MOMENTUM, DECAY, true>(lv.recs[a], lv.ents, st, w, wd, lv.U, nG, use_g != 0, lr, mu, lam, X, M, P, c0, lane);
            else if constexpr (MODE == 1)
                reduce_apply_record<4, MOMENTUM, DECAY, false>(lv.recs[a], lv.ents, st, w, wd, lv.U, nG, use_g != 0, lr, mu, lam, X, M, P, c0, lane);
            else
                reduce_apply_record<1, MOMENTUM, DECAY>(lv.recs[a], lv.ents, st, w, wd, lv.U, nG, use_g != 0, lr, mu, lam, X, M, P, c0, lane);
        }
        __syncthreads();                                               // the stage may be refilled by the next iteration
    }
    asm volatile("cp.async.wait_group 0;" ::: "memory");
}

// ------------------------------------------------------------------------------------------------
// mbarrier / bulk-copy helpers (PTX ISA: mbarrier, cp.async.bulk)
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n.reg .pred p;\nmbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\nselp.u32 %0, 1, 0, p;\n}"
                 : "=r"(ok) : "r"(smem_u32(bar)), "r"(parity) : "memory");
    return ok != 0;
}
// Bounded wait: gives up after kSpinLimit polls so that a lost copy can never hang the GPU.  A failed poll is followed
// by a sleep of SLEEP_NS: a poll returns after ~50 ns, and back-to-back polling by the waiting warps made up about
// half of all instructions the kernel executed (ncu: 1150 polls per tile).
template <int SLEEP_NS>
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity) {
    for (uint32_t it = 0; it < kSpinLimit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        __nanosleep(SLEEP_NS);
    }
    return false;
}
__device__ __forceinline__ void bulk_g2s(void* dst, const void* src, uint32_t bytes, uint64_t* bar) {
    HOP_FENCE(src, bytes, 3);      // a skipped copy leaves the barrier short: the bounded waits end the kernel
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(smem_u32(dst)), "l"(src), "r"(bytes), "r"(smem_u32(bar)) : "memory");
}

// Programmatic dependent launch (PTX griddepcontrol): a kernel launched with the programmatic-serialization attribute may
// start while the kernel in front of it in the stream is still running, once every block of that kernel has executed
// launch_dependents (or exited); dependency_wait then blocks until that kernel has completed and its writes are visible.
// Without the attribute, or with nothing in front, both are no-ops.
__device__ __forceinline__ void dependency_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void launch_dependents() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Self-test of the bounded wait: one warp waits on a barrier that nothing will ever complete, gives up after `polls`
// polls, records ERR_FULL_WAIT with `detail` and returns -- the path a lost copy would take in mix_bulk_kernel.
__global__ void __launch_bounds__(32)
wait_selftest_kernel(int32_t* __restrict__ err_word, uint32_t polls, int32_t detail) {
    __shared__ uint64_t bar;
    if (threadIdx.x == 0) {
        mbar_init(&bar, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    bool done = false;
    for (uint32_t it = 0; it < polls && !done; ++it) {
        done = mbar_try_wait(&bar, 0);
        if (!done) __nanosleep(32);
    }
    if (!done && threadIdx.x == 0) atomicCAS(err_word, 0, ERR_FULL_WAIT | (detail & 0xffffff));
}

// A record as the bulk kernel keeps it in shared memory: everything that does not depend on the tile is worked out
// once per block (the generic record costs ~60 instructions per tile and record in address arithmetic and flags).
struct alignas(16) BulkRec {
    int64_t out_off;        // out_row * P
    int32_t ent_begin;      // first entry (a multiple of 4: entries are padded per record)
    int32_t groups;         // entries / 4
    int32_t g_off;          // float offset of the gradient row inside a staged tile, -1 without gradient
    int32_t self_off;       // float offset of the worker's own consumed slice when weight decay applies, else -1
    int32_t worker;
    int32_t pad;
};
static_assert(sizeof(BulkRec) == sizeof(HopRecord), "the two record forms share the table space");

// Reduce + Apply for one record and one tile from the shared-memory tables: whole groups of four entries, two
// entries per 16-byte table load, the four slice loads of a group ahead of its multiply-adds (in entry order).
template <bool MOMENTUM, bool DECAY>
__device__ __forceinline__ void bulk_record(const BulkRec& r, const int4* __restrict__ ents2, const float* __restrict__ stage,
                                            int w, int wd, int nG, float lr, float mu, float lam, float* __restrict__ Xc,
                                            float* __restrict__ Mc, int64_t P, int lane) {
    // Both loops stay rolled: unrolled by the compiler (four copies plus a remainder switch) they cost ~20 more
    // instructions and 9 more branches per record and a larger instruction footprint (measured).
#pragma unroll 1
    for (int c = lane * 4; c < wd; c += 128) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        const float* sc = stage + c;
        const int4* e = ents2 + (r.ent_begin >> 1);
#define HOP_FMA4(W, V) acc.x = fmaf(W, V.x, acc.x); acc.y = fmaf(W, V.y, acc.y); acc.z = fmaf(W, V.z, acc.z); acc.w = fmaf(W, V.w, acc.w)
#pragma unroll 1
        for (int g = 0; g < r.groups; ++g, e += 2) {
            const int4 e01 = e[0], e23 = e[1];             // (offset, weight) x 2 each
            const float4 v0 = *reinterpret_cast<const float4*>(sc + e01.x);
            const float4 v1 = *reinterpret_cast<const float4*>(sc + e01.z);
            const float4 v2 = *reinterpret_cast<const float4*>(sc + e23.x);
            const float4 v3 = *reinterpret_cast<const float4*>(sc + e23.z);
            const float w0 = __int_as_float(e01.y), w1 = __int_as_float(e01.w), w2 = __int_as_float(e23.y), w3 = __int_as_float(e23.w);
            HOP_FMA4(w0, v0); HOP_FMA4(w1, v1); HOP_FMA4(w2, v2); HOP_FMA4(w3, v3);
        }
#undef HOP_FMA4
        if (DECAY && r.self_off >= 0 && r.g_off < 0) {
            const float4 xs = *reinterpret_cast<const float4*>(sc + r.self_off);
            const float k = -lr * lam;
            acc.x = fmaf(k, xs.x, acc.x); acc.y = fmaf(k, xs.y, acc.y); acc.z = fmaf(k, xs.z, acc.z); acc.w = fmaf(k, xs.w, acc.w);
        }
        if (r.g_off >= 0) {
            float4 g = *reinterpret_cast<const float4*>(sc + r.g_off);
            if (DECAY && r.self_off >= 0) {
                const float4 xs = *reinterpret_cast<const float4*>(sc + r.self_off);
                g.x = fmaf(lam, xs.x, g.x); g.y = fmaf(lam, xs.y, g.y); g.z = fmaf(lam, xs.z, g.z); g.w = fmaf(lam, xs.w, g.w);
            }
            if constexpr (MOMENTUM) {
                const float4 m = *reinterpret_cast<const float4*>(sc + r.g_off + nG * w);
                g.x = fmaf(mu, m.x, g.x); g.y = fmaf(mu, m.y, g.y);
                g.z = fmaf(mu, m.z, g.z); g.w = fmaf(mu, m.w, g.w);
                *reinterpret_cast<float4*>(Mc + (int64_t)r.worker * P + c) = g;
            }
            acc.x = fmaf(-lr, g.x, acc.x); acc.y = fmaf(-lr, g.y, acc.y);
            acc.z = fmaf(-lr, g.z, acc.z); acc.w = fmaf(-lr, g.w, acc.w);
        }
        *reinterpret_cast<float4*>(Xc + r.out_off + c) = acc;
    }
}

// The same for parameter counts that are not multiples of 4 (ALIGNED = false): a slice's staged copy starts at the 16-byte
// boundary below its first element, so element c of the tile sits `shift` floats into its staged row (the shift is
// folded into the table offsets) and is not 16-byte aligned in general: a lane takes every 32nd column with scalar
// shared-memory loads (the same number of shared-memory wavefronts as the vector form, four times the load instructions)
// and scalar, coalesced global stores.  Same multiply-adds in the same order.
template <bool MOMENTUM, bool DECAY>
__device__ __forceinline__ void bulk_record_scalar(const BulkRec& r, const int4* __restrict__ ents2, const float* __restrict__ stage,
                                                   int ws, int wd, int nG, float lr, float mu, float lam, float* __restrict__ Xc,
                                                   float* __restrict__ Mc, int64_t P, int lane) {
    // a lane takes columns cb, cb + 32, cb + 64, cb + 96 per round, so that the table loads and the loop are shared by four
    // outputs as in the vector form; columns past the tile's width are predicated off (loads included: they could leave the stage)
#pragma unroll 1
    for (int cb = lane; cb < wd; cb += 128) {
        float acc[4] = {0.f, 0.f, 0.f, 0.f};
        const float* sc = stage + cb;
        const bool on[4] = {true, cb + 32 < wd, cb + 64 < wd, cb + 96 < wd};
        const int4* e = ents2 + (r.ent_begin >> 1);
#pragma unroll 1
        for (int g = 0; g < r.groups; ++g, e += 2) {
            const int4 e01 = e[0], e23 = e[1];
            float v[4][4];
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                v[j][0] = on[j] ? sc[e01.x + 32 * j] : 0.f; v[j][1] = on[j] ? sc[e01.z + 32 * j] : 0.f;
                v[j][2] = on[j] ? sc[e23.x + 32 * j] : 0.f; v[j][3] = on[j] ? sc[e23.z + 32 * j] : 0.f;
            }
            const float w0 = __int_as_float(e01.y), w1 = __int_as_float(e01.w), w2 = __int_as_float(e23.y), w3 = __int_as_float(e23.w);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                acc[j] = fmaf(w0, v[j][0], acc[j]); acc[j] = fmaf(w1, v[j][1], acc[j]);
                acc[j] = fmaf(w2, v[j][2], acc[j]); acc[j] = fmaf(w3, v[j][3], acc[j]);
            }
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            if (!on[j]) continue;
            const int c = cb + 32 * j;
            const float* scj = sc + 32 * j;
            float a = acc[j];
            if (DECAY && r.self_off >= 0 && r.g_off < 0) a = fmaf(-lr * lam, scj[r.self_off], a);
            if (r.g_off >= 0) {
                float g = scj[r.g_off];
                if (DECAY && r.self_off >= 0) g = fmaf(lam, scj[r.self_off], g);
                if constexpr (MOMENTUM) {
                    g = fmaf(mu, scj[r.g_off + nG * ws], g);
                    Mc[(int64_t)r.worker * P + c] = g;
                }
                a = fmaf(-lr, g, a);
            }
            Xc[r.out_off + c] = a;
        }
    }
}

// mix_bulk: persistent blocks; the first kProducerWarps warps are producers (asynchronous bulk copies of
// every staged row of the next tile, rows dealt round-robin to the producer lanes, completion counted
// in bytes on an mbarrier), the other kConsumerWarps warps consume.  Two stages.
// 16-byte aligned base pointers (bulk copies move multiples of 16 bytes from 16-byte boundaries).  ALIGNED: P % 4 == 0, every
// row piece is such a copy.  !ALIGNED: any P; a row piece is fetched from the 16-byte boundary below its first element
// into a staged row of w + 4 floats (never past the end of the buffer it lies in: the last one to three floats of a
// buffer come by plain loads), consumers use bulk_record_scalar, early_x is not used, the tables must be in shared memory.
// early_x != 0: the launch carries the programmatic-serialization attribute and the kernel in front of it in the stream
// (the level's gradient kernel) writes neither X nor M: barrier set-up, the tables and the X / M rows of the first
// kBulkStages tiles are then fetched while that kernel is still draining; the gradient rows and every store come
// after dependency_wait.  early_x == 0: everything comes after it.
template <bool MOMENTUM, bool DECAY, bool ALIGNED = true>
__global__ void __launch_bounds__(kBulkThreads, 1)
mix_bulk_kernel(float* __restrict__ X, float* __restrict__ M, const float* __restrict__ G, int64_t P, int w,
                int use_g, float lr, float mu, float lam, HopLevelDev lv, int table_bytes, int n_ents,
                int32_t* __restrict__ err_word, int early_x, int ring_rows, int n_workers) {
    extern __shared__ __align__(128) unsigned char smem_raw[];
    uint64_t* full = reinterpret_cast<uint64_t*>(smem_raw);
    uint64_t* empty = full + kBulkStages;
    float* stage0 = reinterpret_cast<float*>(smem_raw + 128 + table_bytes);
    // the level's records and entries are read once per tile by every consumer warp: keep them on chip, the records
    // in the tile-independent form (when the tables do not fit, the consumers use the generic records in global memory)
    BulkRec* srec = reinterpret_cast<BulkRec*>(smem_raw + 128);
    const int4* sent2 = reinterpret_cast<const int4*>(srec + lv.nA);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int nG = use_g ? lv.nG : 0;
    const int rows = lv.U + nG * (MOMENTUM ? 2 : 1);
    const int ws = ALIGNED ? w : w + 4;                    // floats per staged row
    const int64_t stage_floats = (int64_t)rows * ws;
    const int64_t tiles = (P + w - 1) / w;
    launch_dependents();     // a kernel behind that was launched as a dependent (a CSR margin kernel) may fetch its static data
    if (!(ALIGNED && early_x)) dependency_wait();
    if (tid == 0) {
        for (int s = 0; s < kBulkStages; ++s) { mbar_init(&full[s], kProducerWarps); mbar_init(&empty[s], kConsumerWarps); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    __syncthreads();
    if (warp < kProducerWarps) {
        // ---------------- producers: row r goes to warp r % kProducerWarps, lane (r / kProducerWarps) % 32, so that
        // every warp issues the same number of copies (+-1): a warp issues them one after the other, ~30-40 ns
        // each, and the busiest warp sets the pace (measured)
        const int my_rows = (rows - warp + kProducerWarps - 1) / kProducerWarps;
        // a lane's rows are the same for every tile: the first kHoist source addresses are formed once (the row
        // tables are in global memory; reading them per tile would put a global-load latency before every copy)
        constexpr int kHoist = 2;
        auto row_src = [&](int r) -> const float* {
            if (r < lv.U) return X + (int64_t)lv.src_row[r] * P;
            if (r < lv.U + nG) return G + (int64_t)lv.grad_workers[r - lv.U] * P;
            return M + (int64_t)lv.grad_workers[r - lv.U - nG] * P;
        };
        const float* src_h[kHoist];
#pragma unroll
        for (int h = 0; h < kHoist; ++h) {
            const int r = warp + (lane + 32 * h) * kProducerWarps;
            src_h[h] = r < rows ? row_src(r) : nullptr;
        }
        int64_t n = 0;
        bool ok = true;
        // which == 0: every row of this lane; 1: all but the gradient rows; 2: the gradient rows only
        auto issue = [&](int64_t tile, int s, int which) {
            const int64_t c0 = tile * w;
            const int wd = (int)min((int64_t)w, P - c0);
            float* dst = stage0 + s * stage_floats;
            if constexpr (ALIGNED) {
                const uint32_t bytes = (uint32_t)wd * 4u;
                if (which != 2) {
                    if (lane == 0) mbar_expect_tx(&full[s], bytes * (uint32_t)my_rows);
                    __syncwarp();
                }
                auto wanted = [&](int r) { return which == 0 || ((r >= lv.U && r < lv.U + nG) == (which == 2)); };
#pragma unroll
                for (int h = 0; h < kHoist; ++h) {
                    const int r = warp + (lane + 32 * h) * kProducerWarps;
                    if (src_h[h] && wanted(r)) bulk_g2s(dst + r * w, src_h[h] + c0, bytes, &full[s]);
                }
                for (int r = warp + (lane + 32 * kHoist) * kProducerWarps; r < rows; r += 32 * kProducerWarps)
                    if (wanted(r)) bulk_g2s(dst + (int64_t)r * w, row_src(r) + c0, bytes, &full[s]);
            } else {
                // which is always 0 here.  A piece starts `a` floats above a 16-byte boundary: copy from that boundary, a
                // whole number of 16-byte units; the staged row then holds the tile's element c at index a + c.
                uint32_t mine = 0;
                auto fetch = [&](int r, const float* rowbase) {
                    const float* src = rowbase + c0;
                    const uint32_t a = (uint32_t)((reinterpret_cast<uintptr_t>(src) >> 2) & 3u);
                    const float* src0 = src - a;
                    uint32_t n = (a + (uint32_t)wd + 3u) & ~3u;
                    float* d = dst + (int64_t)r * ws;
                    const float* end = r < lv.U ? X + (int64_t)ring_rows * P : (r < lv.U + nG ? G : M) + (int64_t)n_workers * P;
                    if (src0 + n > end) {                       // last piece of the buffer: its last 1-3 floats by plain loads
                        n -= 4;
                        for (const float* q = src0 + n; q < end; ++q) d[q - src0] = *q;
                    }
                    if (n) { bulk_g2s(d, src0, n * 4u, &full[s]); mine += n * 4u; }
                };
#pragma unroll
                for (int h = 0; h < kHoist; ++h)
                    if (src_h[h]) fetch(warp + (lane + 32 * h) * kProducerWarps, src_h[h]);
                for (int r = warp + (lane + 32 * kHoist) * kProducerWarps; r < rows; r += 32 * kProducerWarps) fetch(r, row_src(r));
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) mine += __shfl_xor_sync(0xffffffffu, mine, o);
                __syncwarp();                                   // the plain stores above are ordered before lane 0's arrival
                if (lane == 0) mbar_expect_tx(&full[s], mine);  // bytes may complete before they are expected: the count is signed
            }
        };
        int64_t tile = blockIdx.x;
        if (ALIGNED && early_x) {
            // the first tiles' X and M rows while the gradient kernel may still be writing G (both stages are free)
            int pre = 0;
            for (int64_t t = tile; t < tiles && pre < kBulkStages; t += gridDim.x, ++pre) issue(t, pre, 1);
            dependency_wait();
            for (int q = 0; q < pre; ++q, tile += gridDim.x, ++n) issue(tile, q, 2);
        }
        for (; tile < tiles && ok; tile += gridDim.x, ++n) {
            const int s = (int)(n % kBulkStages);
            const uint32_t ph = (uint32_t)((n / kBulkStages) & 1);
            if (!mbar_wait<256>(&empty[s], ph ^ 1u)) { ok = false; if (lane == 0) atomicCAS(err_word, 0, ERR_EMPTY_WAIT | (int)(tile & 0xffffff)); break; }
            issue(tile, s, 0);
        }
        // drain: do not leave while copies into this block's shared memory are still in flight
        if (ok) {
            const int64_t issued = n;
            for (int64_t m = (issued > kBulkStages ? issued - kBulkStages : 0); m < issued; ++m)
                mbar_wait<256>(&full[m % kBulkStages], (uint32_t)((m / kBulkStages) & 1));
        }
    } else {
        // ---------------- consumers
        const int cw = warp - kProducerWarps;
        // The tables are built by the consumer warps alone, behind a barrier of their own, while the producers are
        // already fetching the first tiles.
        if (table_bytes > 0) {
            constexpr int kConsumerThreads = 32 * kConsumerWarps;
            const int ct = tid - 32 * kProducerWarps;
            for (int i = ct; i < lv.nA; i += kConsumerThreads) {
                const HopRecord r = lv.recs[i];
                const bool grad = use_g != 0 && r.g_stage >= 0;
                BulkRec b;
                b.out_off = (int64_t)r.out_row * P;
                b.ent_begin = r.ent_begin;
                b.groups = r.ent_count >> 2;
                b.g_off = grad ? (lv.U + r.g_stage) * ws + (ALIGNED ? 0 : (int)(((int64_t)r.worker * P) & 3)) : -1;
                b.self_off = (DECAY && r.g_stage >= 0 && r.self_u >= 0) ? r.self_u : -1;
                b.worker = r.worker;
                b.pad = 0;
                srec[i] = b;
            }
            int2* sent = reinterpret_cast<int2*>(srec + lv.nA);
            const int2* ge = reinterpret_cast<const int2*>(lv.ents);
            for (int i = ct; i < n_ents; i += kConsumerThreads) sent[i] = ge[i];
            asm volatile("bar.sync 1, %0;" ::"n"(kConsumerThreads) : "memory");
        }
        if (ALIGNED && early_x) dependency_wait();      // no store before the kernel in front has finished (it may read the slot written here)
        int64_t n = 0;
        for (int64_t tile = blockIdx.x; tile < tiles; tile += gridDim.x, ++n) {
            const int s = (int)(n % kBulkStages);
            const uint32_t ph = (uint32_t)((n / kBulkStages) & 1);
            if (!mbar_wait<32>(&full[s], ph)) { if (lane == 0) atomicCAS(err_word, 0, ERR_FULL_WAIT | (int)(tile & 0xffffff)); break; }
            const int64_t c0 = tile * w;
            const int wd = (int)min((int64_t)w, P - c0);
            const float* st = stage0 + s * stage_floats;
            if (table_bytes > 0) {
#pragma unroll 1
                for (int a = cw; a < lv.nA; a += kConsumerWarps) {
                    if constexpr (ALIGNED)
                        bulk_record<MOMENTUM, DECAY>(srec[a], sent2, st, w, wd, nG, lr, mu, lam, X + c0, MOMENTUM ? M + c0 : nullptr, P, lane);
                    else
                        bulk_record_scalar<MOMENTUM, DECAY>(srec[a], sent2, st, ws, wd, nG, lr, mu, lam, X + c0, MOMENTUM ? M + c0 : nullptr, P, lane);
                }
            } else if constexpr (ALIGNED) {
                for (int a = cw; a < lv.nA; a += kConsumerWarps)
                    reduce_apply_record<4, MOMENTUM, DECAY>(lv.recs[a], lv.ents, st, w, wd, lv.U, nG, use_g != 0, lr, mu, lam, X, M, P, c0, lane);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&empty[s]);
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Philox4x32-10 (Salmon et al., SC'11): multipliers and Weyl key increments from the publication.
__device__ __forceinline__ void philox4x32_10(uint32_t c0, uint32_t c1, uint32_t c2, uint32_t c3, uint32_t k0, uint32_t k1,
                                              uint32_t (&o)[4]) {
    constexpr uint32_t M0 = 0xD2511F53u, M1 = 0xCD9E8D57u, W0 = 0x9E3779B9u, W1 = 0xBB67AE85u;
#pragma unroll
    for (int r = 0; r < 10; ++r) {
        const uint64_t p0 = (uint64_t)M0 * c0, p1 = (uint64_t)M1 * c2;     // one wide multiply each
        const uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        const uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        c0 = hi1 ^ c1 ^ k0; c1 = lo1; c2 = hi0 ^ c3 ^ k1; c3 = lo0;
        k0 += W0; k1 += W1;
    }
    o[0] = c0; o[1] = c1; o[2] = c2; o[3] = c3;
}
// Box-Muller on 23-bit uniforms u = (n + 1/2) / 2^23 (exact in float32), scaled by sigma.  The kernel is
// instruction-bound, so: the uniforms are built by placing the 23 random bits in the mantissa of a float in
// [1, 2) (no integer-to-float conversion); the hardware approximations lg2 / sqrt / sin / cos are used on purpose
// (error <= 3 ulp for the logarithm, 2 ulp for the root, <= 2^-21.4 absolute for sine and cosine on [-pi, pi]:
// a normal deviate moves by < 5e-6, a parameter by < 1e-9 per step after scaling by sigma and the learning rate).
__device__ __forceinline__ void box_muller(uint32_t ra, uint32_t rb, float sigma, float& z0, float& z1) {
    const float f1 = __uint_as_float(0x3f800000u | (ra >> 9));        // 1 + n1 * 2^-23
    const float f2 = __uint_as_float(0x3f800000u | (rb >> 9));        // 1 + n2 * 2^-23
    const float u1 = f1 - 0.99999994f;                                // f1 - (1 - 2^-24) = (n1 + 1/2) * 2^-23, exact
    // angle - pi = 2 pi u2 - pi = 2 pi f2 - 3 pi + pi 2^-23 in one multiply-add; with both constants rounded to float the
    // angle is off by at most 3.5e-7 rad over all 2^23 values of n2 (checked exhaustively) and stays inside (-pi, pi)
    const float a = fmaf(f2, 6.2831855f, -9.424778f);
    float l2, rad, sn, cs;
    asm("lg2.approx.ftz.f32 %0, %1;" : "=f"(l2) : "f"(u1));
    asm("sqrt.approx.ftz.f32 %0, %1;" : "=f"(rad) : "f"(l2 * -1.3862943611198906f));   // sqrt(-2 ln u1)
    __sincosf(a, &sn, &cs);
    rad *= -sigma;                                                    // cos(a) = -cos(a - pi), sin likewise
    z0 = rad * cs; z1 = rad * sn;
}

// Four independent Philox blocks per thread (groups q, q + 256, q + 512, q + 768 of four columns): the ten rounds of one block are
// a serial dependency chain; interleaved chains keep the issue slots busy (2.1 -> 1.7 ms per launch, measured).  A thread block
// covers kGradChunks consecutive chunks of 1024 groups, so that the launch and drain of a block are spread over more work.
constexpr int kGradChunks = 4;
__global__ void __launch_bounds__(256)
synth_grad_kernel(float* __restrict__ G, int64_t P, HopLevelDev lv, uint32_t k0, uint32_t k1, float sigma, int64_t col_offset) {
    launch_dependents();      // the mix-update kernel behind may set itself up; it waits before it touches G
    const int worker = lv.grad_workers[blockIdx.y];
    float* row = G + (int64_t)worker * P;
    const bool vec = (P & 3) == 0;
    const uint64_t gq0 = (uint64_t)(col_offset / 4);
#pragma unroll 1
    for (int it = 0; it < kGradChunks; ++it) {
        const int64_t q0 = ((int64_t)blockIdx.x * kGradChunks + it) * 1024 + threadIdx.x;   // local group of 4 columns
        if (q0 * 4 >= P) break;
        uint32_t o[4][4];
#pragma unroll
        for (int h = 0; h < 4; ++h)
            philox4x32_10((uint32_t)(gq0 + q0 + h * 256), (uint32_t)worker, (uint32_t)lv.level, 6u, k0, k1, o[h]);
#pragma unroll
        for (int h = 0; h < 4; ++h) {
            const int64_t c = (q0 + h * 256) * 4;
            if (c >= P) continue;
            float z[4];
            box_muller(o[h][0], o[h][1], sigma, z[0], z[1]);
            box_muller(o[h][2], o[h][3], sigma, z[2], z[3]);
            if (vec) {
                *reinterpret_cast<float4*>(row + c) = make_float4(z[0], z[1], z[2], z[3]);
            } else {
                for (int e = 0; e < 4 && c + e < P; ++e) row[c + e] = z[e];
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// Hinge-loss SVM.  One warp per minibatch row: margin = a_r . x_{k,i} accumulated in double (the
// active-set test y*margin < 1 is then decided as in exact arithmetic up to ~1e-16), reduced with
// warp shuffles; coef_r = -y_r/B if active else 0.
__device__ __forceinline__ double warp_sum(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// d(loss)/d(margin) of one row: hinge -y/B on the active set (y*m < 1, strict), log loss -y / (B (1 + e^{y m})).
__device__ __forceinline__ float loss_coefficient(float y, double m, int B, int loss) {
    if (loss == 0) return ((double)y * m < 1.0) ? -y / (float)B : 0.f;
    return (float)(-(double)y / ((double)B * (1.0 + exp((double)y * m))));
}

// When launched as a programmatic dependent of the previous level's last kernel, the row's column indices and values
// (static data) are fetched before dependency_wait and the parameter gather comes after it; launch_dependents comes
// after the wait too, so that the mix-update kernel behind cannot start before everything in front has finished.
constexpr int kCsrPrefetch = 4;      // elements per lane held in registers: rows of up to 128 stored elements in one round
__global__ void __launch_bounds__(256)
svm_margin_csr_kernel(const float* __restrict__ X, int64_t P, int S, HopLevelDev lv, const int64_t* __restrict__ row_ptr,
                      const int32_t* __restrict__ col, const float* __restrict__ val, const float* __restrict__ y,
                      int R, int B, int loss, float* __restrict__ coef, double* __restrict__ margins_out) {
    const int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const bool live = gw < lv.nG * B;
    int worker = 0, r = 0;
    int64_t row = 0, t0 = 0, t1 = 0;
    int32_t pc[kCsrPrefetch];
    float pv[kCsrPrefetch];
    if (live) {
        const int a = gw / B;
        r = gw - a * B;
        worker = lv.grad_workers[a];
        row = (int64_t)worker * R + (int64_t)(lv.level % (R / B)) * B + r;
        t0 = row_ptr[row] + lane;
        t1 = row_ptr[row + 1];
#pragma unroll
        for (int q = 0; q < kCsrPrefetch; ++q) {
            const int64_t t = t0 + 32 * q;
            pc[q] = t < t1 ? col[t] : 0;
            pv[q] = t < t1 ? val[t] : 0.f;
        }
    }
    dependency_wait();
    launch_dependents();
    if (!live) return;
    const float* x = X + ((int64_t)worker * S + lv.level % S) * P;
    double m = 0.0;
    float xv[kCsrPrefetch];
#pragma unroll
    for (int q = 0; q < kCsrPrefetch; ++q) xv[q] = (t0 + 32 * q < t1) ? HOP_FENCE_OR(x + pc[q], 4, 4, 0.f) : 0.f;   // the gathers in flight together
#pragma unroll
    for (int q = 0; q < kCsrPrefetch; ++q)
        if (t0 + 32 * q < t1) m += (double)pv[q] * (double)xv[q];                           // a lane's elements in their order
    for (int64_t t = t0 + 32 * kCsrPrefetch; t < t1; t += 32) m += (double)val[t] * (double)HOP_FENCE_OR(x + col[t], 4, 4, 0.f);
    m = warp_sum(m);
    if (lane == 0) {
        if (margins_out) margins_out[(int64_t)worker * B + r] = m;     // partial margin over this shard's columns
        else coef[(int64_t)worker * B + r] = loss_coefficient(y[row], m, B, loss);
    }
}

// Coefficients from margins that were summed over column shards (one thread per minibatch row).
__global__ void __launch_bounds__(256)
svm_coef_from_margins_kernel(const double* __restrict__ margins, HopLevelDev lv, const float* __restrict__ y, int R, int B,
                             int loss, float* __restrict__ coef) {
    launch_dependents();
    const int t = blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= lv.nG * B) return;
    const int a = t / B, r = t - a * B;
    const int worker = lv.grad_workers[a];
    const int64_t row = (int64_t)worker * R + (int64_t)(lv.level % (R / B)) * B + r;
    coef[(int64_t)worker * B + r] = loss_coefficient(y[row], margins[(int64_t)worker * B + r], B, loss);
}

__global__ void __launch_bounds__(256)
svm_margin_dense_kernel(const float* __restrict__ X, int64_t P, int S, HopLevelDev lv, const float* __restrict__ A,
                        const float* __restrict__ y, int R, int B, int loss, float* __restrict__ coef,
                        double* __restrict__ margins_out) {
    const int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (gw >= lv.nG * B) return;
    const int a = gw / B, r = gw - a * B;
    const int worker = lv.grad_workers[a];
    const int64_t row = (int64_t)worker * R + (int64_t)(lv.level % (R / B)) * B + r;
    const float* x = X + ((int64_t)worker * S + lv.level % S) * P;
    const float* arow = A + row * P;
    double m = 0.0;
    for (int64_t p = lane; p < P; p += 32) m += (double)arow[p] * (double)x[p];
    m = warp_sum(m);
    if (lane == 0) {
        if (margins_out) margins_out[(int64_t)worker * B + r] = m;
        else coef[(int64_t)worker * B + r] = loss_coefficient(y[row], m, B, loss);
    }
}

// g[i][p] = sum_r coef_r * A[r][p]; one thread per column, rows of the minibatch in order.
__global__ void __launch_bounds__(256)
svm_dense_grad_kernel(float* __restrict__ G, int64_t P, HopLevelDev lv, const float* __restrict__ A, int R, int B,
                      const float* __restrict__ coef) {
    launch_dependents();
    const int worker = lv.grad_workers[blockIdx.y];
    const int64_t p = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (p >= P) return;
    const float* a0 = A + ((int64_t)worker * R + (int64_t)(lv.level % (R / B)) * B) * P + p;
    const float* cf = coef + (int64_t)worker * B;
    float g = 0.f;
    int r = 0;
    for (; r + 8 <= B; r += 8) {          // eight independent loads in flight, the multiply-adds in row order
        float a[8], c[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) { a[i] = a0[(int64_t)(r + i) * P]; c[i] = cf[r + i]; }
#pragma unroll
        for (int i = 0; i < 8; ++i) g = fmaf(c[i], a[i], g);
    }
    for (; r < B; ++r) g = fmaf(cf[r], a0[(int64_t)r * P], g);
    G[(int64_t)worker * P + p] = g;
}

// Margins, coefficients and gradient of one worker's minibatch in one block (small problems: the three steps as separate
// launches cost more in launch latency than in work).  Same arithmetic in the same order as svm_margin_dense_kernel
// followed by svm_dense_grad_kernel: a warp per row for the margins, a thread per column for the gradient.
// The kernel is latency-bound (a few KB per worker): up to 32 warps take one minibatch row each, so all margins cost
// one round of loads, and a gradient thread keeps 32 rows in flight.
constexpr int kFusedSvmThreads = 1024;
__global__ void __launch_bounds__(kFusedSvmThreads)
svm_dense_fused_kernel(const float* __restrict__ X, float* __restrict__ G, int64_t P, int S, HopLevelDev lv,
                       const float* __restrict__ A, const float* __restrict__ y, int R, int B, int loss) {
    extern __shared__ float s_coef[];      // [B]
    launch_dependents();
    const int worker = lv.grad_workers[blockIdx.x];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, warps = blockDim.x >> 5;
    const int64_t row0 = (int64_t)worker * R + (int64_t)(lv.level % (R / B)) * B;
    const float* x = X + ((int64_t)worker * S + lv.level % S) * P;
    for (int r = warp; r < B; r += warps) {
        const float* arow = A + (row0 + r) * P;
        double m = 0.0;
        for (int64_t p = lane; p < P; p += 32) m += (double)arow[p] * (double)x[p];
        m = warp_sum(m);
        if (lane == 0) s_coef[r] = loss_coefficient(y[row0 + r], m, B, loss);
    }
    __syncthreads();
    for (int64_t p = threadIdx.x; p < P; p += blockDim.x) {
        const float* a0 = A + row0 * P + p;
        float g = 0.f;
        int r = 0;
        for (; r + 32 <= B; r += 32) {        // the loads first, then the multiply-adds in row order
            float a[32];
#pragma unroll
            for (int i = 0; i < 32; ++i) a[i] = a0[(int64_t)(r + i) * P];
#pragma unroll
            for (int i = 0; i < 32; ++i) g = fmaf(s_coef[r + i], a[i], g);
        }
        for (; r + 8 <= B; r += 8) {
            float a[8];
#pragma unroll
            for (int i = 0; i < 8; ++i) a[i] = a0[(int64_t)(r + i) * P];
#pragma unroll
            for (int i = 0; i < 8; ++i) g = fmaf(s_coef[r + i], a[i], g);
        }
        for (; r < B; ++r) g = fmaf(s_coef[r], a0[(int64_t)r * P], g);
        G[(int64_t)worker * P + p] = g;
    }
}

// Sparse Apply after the dense mix: x_{k+1,i}[col] -= lr * coef_r * val, one warp per row.  As a programmatic dependent of
// the mix-update kernel it fetches the row's static data first and touches the coefficients and X only after dependency_wait.
__global__ void __launch_bounds__(256)
svm_csr_apply_kernel(float* __restrict__ X, int64_t P, int S, float lr, HopLevelDev lv, const int64_t* __restrict__ row_ptr,
                     const int32_t* __restrict__ col, const float* __restrict__ val, int R, int B,
                     const float* __restrict__ coef, int slot_shift) {
    launch_dependents();
    const int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    const bool live = gw < lv.nG * B;
    int worker = 0, r = 0;
    int64_t t0 = 0, t1 = 0;
    int32_t pc[kCsrPrefetch];
    float pv[kCsrPrefetch];
    if (live) {
        const int a = gw / B;
        r = gw - a * B;
        worker = lv.grad_workers[a];
        const int64_t row = (int64_t)worker * R + (int64_t)(lv.level % (R / B)) * B + r;
        t0 = row_ptr[row] + lane;
        t1 = row_ptr[row + 1];
#pragma unroll
        for (int q = 0; q < kCsrPrefetch; ++q) {
            const int64_t t = t0 + 32 * q;
            pc[q] = t < t1 ? col[t] : -1;
            pv[q] = t < t1 ? val[t] : 0.f;
        }
    }
    dependency_wait();
    if (!live) return;
    const float cf = coef[(int64_t)worker * B + r];
    if (cf == 0.f) return;
    float* x = X + ((int64_t)worker * S + (lv.level + slot_shift) % S) * P;
    const float scale = -lr * cf;
#pragma unroll
    for (int q = 0; q < kCsrPrefetch; ++q)
        if (pc[q] >= 0 && HOP_FENCED(x + pc[q], 4, 5)) atomicAdd(x + pc[q], scale * pv[q]);
    for (int64_t t = t0 + 32 * kCsrPrefetch; t < t1; t += 32)
        if (HOP_FENCED(x + col[t], 4, 5)) atomicAdd(x + col[t], scale * val[t]);
}

// Serial approach (Compute, Apply, then Send): x_k <- x_k - lr * d in place for the level's NORMAL workers, with
// d = g (+ lambda x_k), through the momentum buffer when there is one.  One float4 per thread.
template <bool MOMENTUM>
__global__ void __launch_bounds__(256)
apply_dense_kernel(float* __restrict__ X, float* __restrict__ M, const float* __restrict__ G, int64_t P, int S, float lr,
                   float mu, float lam, HopLevelDev lv) {
    const int worker = lv.grad_workers[blockIdx.y];
    const int64_t c = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (c >= P) return;
    float* x = X + ((int64_t)worker * S + lv.level % S) * P + c;
    const float* g = G + (int64_t)worker * P + c;
    float* m = MOMENTUM ? M + (int64_t)worker * P + c : nullptr;
    const int n = (int)min((int64_t)4, P - c);
    if (n == 4 && (P & 3) == 0) {
        float4 xv = *reinterpret_cast<float4*>(x), gv = *reinterpret_cast<const float4*>(g);
        gv.x = fmaf(lam, xv.x, gv.x); gv.y = fmaf(lam, xv.y, gv.y); gv.z = fmaf(lam, xv.z, gv.z); gv.w = fmaf(lam, xv.w, gv.w);
        if constexpr (MOMENTUM) {
            const float4 mv = *reinterpret_cast<float4*>(m);
            gv.x = fmaf(mu, mv.x, gv.x); gv.y = fmaf(mu, mv.y, gv.y); gv.z = fmaf(mu, mv.z, gv.z); gv.w = fmaf(mu, mv.w, gv.w);
            *reinterpret_cast<float4*>(m) = gv;
        }
        xv.x = fmaf(-lr, gv.x, xv.x); xv.y = fmaf(-lr, gv.y, xv.y); xv.z = fmaf(-lr, gv.z, xv.z); xv.w = fmaf(-lr, gv.w, xv.w);
        *reinterpret_cast<float4*>(x) = xv;
    } else {
        for (int e = 0; e < n; ++e) {
            float gv = fmaf(lam, x[e], g[e]);
            if constexpr (MOMENTUM) { gv = fmaf(mu, m[e], gv); m[e] = gv; }
            x[e] = fmaf(-lr, gv, x[e]);
        }
    }
}

// Update direction in place for the dense (tensor-core) path, whose epilogue applies -lr * G only: G <- g + lambda * x_k, through
// the momentum buffer when there is one (m <- mu * m + G; G <- m), for the level's NORMAL workers.  One float4 per thread.
template <bool MOMENTUM>
__global__ void __launch_bounds__(256)
direction_dense_kernel(const float* __restrict__ X, float* __restrict__ M, float* __restrict__ G, int64_t P, int S,
                       float mu, float lam, HopLevelDev lv) {
    const int worker = lv.grad_workers[blockIdx.y];
    const int64_t c = ((int64_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (c >= P) return;
    const float* x = X + ((int64_t)worker * S + lv.level % S) * P + c;
    float* g = G + (int64_t)worker * P + c;
    float* m = MOMENTUM ? M + (int64_t)worker * P + c : nullptr;
    const int n = (int)min((int64_t)4, P - c);
    if (n == 4 && (P & 3) == 0) {
        float4 gv = *reinterpret_cast<const float4*>(g);
        if (lam != 0.f) {
            const float4 xv = *reinterpret_cast<const float4*>(x);
            gv.x = fmaf(lam, xv.x, gv.x); gv.y = fmaf(lam, xv.y, gv.y); gv.z = fmaf(lam, xv.z, gv.z); gv.w = fmaf(lam, xv.w, gv.w);
        }
        if constexpr (MOMENTUM) {
            const float4 mv = *reinterpret_cast<const float4*>(m);
            gv.x = fmaf(mu, mv.x, gv.x); gv.y = fmaf(mu, mv.y, gv.y); gv.z = fmaf(mu, mv.z, gv.z); gv.w = fmaf(mu, mv.w, gv.w);
            *reinterpret_cast<float4*>(m) = gv;
        }
        *reinterpret_cast<float4*>(g) = gv;
    } else {
        for (int e = 0; e < n; ++e) {
            float gv = lam != 0.f ? fmaf(lam, x[e], g[e]) : g[e];
            if constexpr (MOMENTUM) { gv = fmaf(mu, m[e], gv); m[e] = gv; }
            g[e] = gv;
        }
    }
}

constexpr int kStagedStages = 2;
size_t staged_smem(const HopLaunchCfg& c, const HopLevelDev& lv) {
    const int nG = c.use_g ? lv.nG : 0;
    const int rows = lv.U + nG * (c.mu != 0.f ? 2 : 1);
    return (size_t)kStagedStages * rows * c.tile_w * sizeof(float);
}

}  // namespace

// Checked build: tells the kernels which address ranges are the bound buffers (stream-ordered, before the level's launches).
int hop_checked_set_fence(const HopLaunchCfg& c) {
#ifdef HOP_CHECKED
    HopFence f{};
    const size_t ring = (size_t)c.N * (c.s + 1) * c.P * sizeof(float), per = (size_t)c.N * c.P * sizeof(float);
    f.lo[0] = reinterpret_cast<const char*>(c.X); f.hi[0] = f.lo[0] + ring;
    f.lo[1] = reinterpret_cast<const char*>(c.M); f.hi[1] = c.M ? f.lo[1] + per : nullptr;
    f.lo[2] = reinterpret_cast<const char*>(c.G); f.hi[2] = c.G ? f.lo[2] + per : nullptr;
    f.err = c.err_word;
    return (int)cudaMemcpyToSymbolAsync(g_fence, &f, sizeof f, 0, cudaMemcpyHostToDevice, (cudaStream_t)c.stream);
#else
    (void)c;
    return 0;
#endif
}
bool hop_checked_build() {
#ifdef HOP_CHECKED
    return true;
#else
    return false;
#endif
}

// One launch for margins + coefficients + gradient when a worker's minibatch is small (B * P floats, read twice).
bool hop_svm_dense_is_fused(int64_t P, int32_t B) { return B <= 4096 && (int64_t)B * P <= 65536; }

int hop_mix_smem_budget(int kernel) { return kernel == HOP_MIX_BULK ? (227 * 1024 - 128) : 200 * 1024; }
int hop_mix_table_limit() { return 32 * 1024; }
int hop_mix_stages(int kernel) { return kernel == HOP_MIX_BULK ? kBulkStages : kStagedStages; }

int hop_launch_mix_staged(const HopLaunchCfg& c, const HopLevelDev& lv) {
    if (lv.nA == 0) return 0;
    const size_t smem = staged_smem(c, lv);
    const int64_t tiles = (c.P + c.tile_w - 1) / c.tile_w;
    const int grid = (int)std::min<int64_t>(tiles, (int64_t)c.sm_count);
    const int mode = (c.P % 4 == 0 && c.tile_w % 4 == 0) ? 0 : (c.tile_w % 4 == 0 ? 1 : 2);
    const bool mom = c.mu != 0.f;
    cudaStream_t st = (cudaStream_t)c.stream;
    cudaError_t e = cudaSuccess;
#define HOP_LAUNCH_STAGED(V, MO, DE)                                                                          \
    do {                                                                                                      \
        e = hop_allow_max_smem<mix_staged_kernel<V, MO, DE>>();                                               \
        if (e == cudaSuccess)                                                                                 \
            mix_staged_kernel<V, MO, DE><<<grid, kStagedThreads, smem, st>>>(c.X, c.M, c.G, c.P, c.tile_w, c.use_g, c.lr, c.mu, c.wd, lv); \
    } while (0)
#define HOP_LAUNCH_STAGED2(V, MO) do { if (c.wd != 0.f) HOP_LAUNCH_STAGED(V, MO, true); else HOP_LAUNCH_STAGED(V, MO, false); } while (0)
#define HOP_LAUNCH_STAGED3(V) do { if (mom) HOP_LAUNCH_STAGED2(V, true); else HOP_LAUNCH_STAGED2(V, false); } while (0)
    if (mode == 0) HOP_LAUNCH_STAGED3(0);
    else if (mode == 1) HOP_LAUNCH_STAGED3(1);
    else HOP_LAUNCH_STAGED3(2);
#undef HOP_LAUNCH_STAGED3
#undef HOP_LAUNCH_STAGED2
#undef HOP_LAUNCH_STAGED
    if (e != cudaSuccess) return (int)e;
    return (int)cudaGetLastError();
}

int hop_launch_mix_bulk(const HopLaunchCfg& c, const HopLevelDev& lv) {
    if (lv.nA == 0) return 0;
    const int nG = c.use_g ? lv.nG : 0;
    const int rows = lv.U + nG * (c.mu != 0.f ? 2 : 1);
    const bool aligned = c.P % 4 == 0;
    if (!aligned && c.table_smem == 0) return (int)cudaErrorInvalidValue;      // the planner never asks for this
    const size_t smem = 128 + (size_t)c.table_smem + (size_t)kBulkStages * rows * (c.tile_w + (aligned ? 0 : 4)) * sizeof(float);
    const int64_t tiles = (c.P + c.tile_w - 1) / c.tile_w;
    const int grid = (int)std::min<int64_t>(tiles, (int64_t)c.sm_count);
    cudaStream_t st = (cudaStream_t)c.stream;
    cudaError_t e = cudaSuccess;
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)grid); lc.blockDim = dim3(kBulkThreads); lc.dynamicSmemBytes = smem; lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    const int early_x = (c.early_x && aligned) ? 1 : 0;
    lc.numAttrs = early_x ? 1 : 0;
#define HOP_LAUNCH_BULK(MO, DE, AL)                                                                           \
    do {                                                                                                      \
        e = hop_allow_max_smem<mix_bulk_kernel<MO, DE, AL>>();                                                \
        if (e == cudaSuccess)                                                                                 \
            e = cudaLaunchKernelEx(&lc, mix_bulk_kernel<MO, DE, AL>, c.X, c.M, (const float*)c.G, c.P, (int)c.tile_w, (int)c.use_g, c.lr, c.mu, \
                                   c.wd, lv, (int)c.table_smem, (int)c.n_ents, c.err_word, early_x, (int)(c.N * (c.s + 1)), (int)c.N); \
    } while (0)
#define HOP_LAUNCH_BULK2(MO, DE) do { if (aligned) HOP_LAUNCH_BULK(MO, DE, true); else HOP_LAUNCH_BULK(MO, DE, false); } while (0)
    const bool mom = c.mu != 0.f, dec = c.wd != 0.f;
    if (mom && dec) HOP_LAUNCH_BULK2(true, true);
    else if (mom) HOP_LAUNCH_BULK2(true, false);
    else if (dec) HOP_LAUNCH_BULK2(false, true);
    else HOP_LAUNCH_BULK2(false, false);
#undef HOP_LAUNCH_BULK2
#undef HOP_LAUNCH_BULK
    if (e != cudaSuccess) return (int)e;
    return (int)cudaGetLastError();
}

int hop_launch_synth_grad(const HopLaunchCfg& c, const HopLevelDev& lv, uint64_t seed, float sigma, int64_t col_offset) {
    if (lv.nG == 0) return 0;
    const int64_t groups = (c.P + 3) / 4;
    dim3 grid((unsigned)((groups + 1024 * kGradChunks - 1) / (1024 * kGradChunks)), (unsigned)lv.nG);
    synth_grad_kernel<<<grid, 256, 0, (cudaStream_t)c.stream>>>(c.G, c.P, lv, (uint32_t)(seed & 0xffffffffu), (uint32_t)(seed >> 32), sigma, col_offset);
    return (int)cudaGetLastError();
}

// phase 0: margins, coefficients (and the dense gradient) in one go.  phase 1: only the partial margins over this
// context's columns, written to `margins`.  phase 2: coefficients from the (summed) margins, then the dense gradient.
int hop_launch_svm_dense(const HopLaunchCfg& c, const HopLevelDev& lv, const float* A, const float* y,
                         int32_t R, int32_t B, float* coef, double* margins, int phase) {
    if (lv.nG == 0) return 0;
    const int warps = lv.nG * B;
    cudaStream_t st = (cudaStream_t)c.stream;
    if (phase == 0 && hop_svm_dense_is_fused(c.P, B)) {
        const int threads = std::min(kFusedSvmThreads, std::max(128, std::max(32 * B, (int)((c.P + 31) / 32 * 32))));
        svm_dense_fused_kernel<<<lv.nG, threads, (size_t)B * sizeof(float), st>>>(c.X, c.G, c.P, c.s + 1, lv, A, y, R, B, c.loss);
        return (int)cudaGetLastError();
    }
    if (phase != 2)
        svm_margin_dense_kernel<<<(warps * 32 + 255) / 256, 256, 0, st>>>(c.X, c.P, c.s + 1, lv, A, y, R, B, c.loss, coef,
                                                                          phase == 1 ? margins : nullptr);
    if (phase == 1) return (int)cudaGetLastError();
    if (phase == 2) svm_coef_from_margins_kernel<<<(warps + 255) / 256, 256, 0, st>>>(margins, lv, y, R, B, c.loss, coef);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return (int)e;
    dim3 grid((unsigned)((c.P + 255) / 256), (unsigned)lv.nG);
    svm_dense_grad_kernel<<<grid, 256, 0, st>>>(c.G, c.P, lv, A, R, B, coef);
    return (int)cudaGetLastError();
}

// One launch with or without the programmatic-serialization attribute (see dependency_wait above).
template <typename... KArgs, typename... Args>
static cudaError_t launch_maybe_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, cudaStream_t st, bool dependent, Args... args) {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = grid; lc.blockDim = block; lc.dynamicSmemBytes = 0; lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = dependent ? 1 : 0;
    return cudaLaunchKernelEx(&lc, kernel, KArgs(args)...);
}

int hop_launch_svm_csr_coef(const HopLaunchCfg& c, const HopLevelDev& lv, const int64_t* row_ptr, const int32_t* col,
                            const float* val, const float* y, int32_t R, int32_t B, float* coef, double* margins, int phase) {
    if (lv.nG == 0) return 0;
    const int warps = lv.nG * B;
    cudaStream_t st = (cudaStream_t)c.stream;
    if (phase != 2) {
        const cudaError_t e = launch_maybe_dependent(svm_margin_csr_kernel, dim3((warps * 32 + 255) / 256), dim3(256), st, c.dependent != 0,
                                                     (const float*)c.X, c.P, (int)(c.s + 1), lv, row_ptr, col, val, y, (int)R, (int)B,
                                                     (int)c.loss, coef, phase == 1 ? margins : (double*)nullptr);
        if (e != cudaSuccess) return (int)e;
    } else {
        svm_coef_from_margins_kernel<<<(warps + 255) / 256, 256, 0, st>>>(margins, lv, y, R, B, c.loss, coef);
    }
    return (int)cudaGetLastError();
}

int hop_launch_svm_csr_apply(const HopLaunchCfg& c, const HopLevelDev& lv, const int64_t* row_ptr, const int32_t* col,
                             const float* val, int32_t R, int32_t B, const float* coef, int32_t slot_shift) {
    if (lv.nG == 0) return 0;
    const int warps = lv.nG * B;
    const cudaError_t e = launch_maybe_dependent(svm_csr_apply_kernel, dim3((warps * 32 + 255) / 256), dim3(256), (cudaStream_t)c.stream,
                                                 c.dependent != 0, c.X, c.P, (int)(c.s + 1), c.lr, lv, row_ptr, col, val, (int)R, (int)B,
                                                 coef, (int)slot_shift);
    if (e != cudaSuccess) return (int)e;
    return (int)cudaGetLastError();
}

int hop_launch_wait_selftest(int32_t* err_word, uint32_t polls, int32_t detail, void* stream) {
    wait_selftest_kernel<<<1, 32, 0, (cudaStream_t)stream>>>(err_word, polls, detail);
    return (int)cudaGetLastError();
}

int hop_launch_direction_dense(const HopLaunchCfg& c, const HopLevelDev& lv) {
    if (lv.nG == 0) return 0;
    dim3 grid((unsigned)(((c.P + 3) / 4 + 255) / 256), (unsigned)lv.nG);
    if (c.mu != 0.f) direction_dense_kernel<true><<<grid, 256, 0, (cudaStream_t)c.stream>>>(c.X, c.M, c.G, c.P, c.s + 1, c.mu, c.wd, lv);
    else direction_dense_kernel<false><<<grid, 256, 0, (cudaStream_t)c.stream>>>(c.X, c.M, c.G, c.P, c.s + 1, c.mu, c.wd, lv);
    return (int)cudaGetLastError();
}

int hop_launch_apply_dense(const HopLaunchCfg& c, const HopLevelDev& lv) {
    if (lv.nG == 0) return 0;
    dim3 grid((unsigned)(((c.P + 3) / 4 + 255) / 256), (unsigned)lv.nG);
    if (c.mu != 0.f) apply_dense_kernel<true><<<grid, 256, 0, (cudaStream_t)c.stream>>>(c.X, c.M, c.G, c.P, c.s + 1, c.lr, c.mu, c.wd, lv);
    else apply_dense_kernel<false><<<grid, 256, 0, (cudaStream_t)c.stream>>>(c.X, c.M, c.G, c.P, c.s + 1, c.lr, c.mu, c.wd, lv);
    return (int)cudaGetLastError();
}
