// hop_svm_csr_sgd_static: the hinge-SVM minibatch step on one parameter vector for callers that
// must not allocate.  The per-row hinge coefficients -- the scratch that hop_step keeps in a
// cudaMalloc'ed buffer -- live here in a fixed device array that is part of the library image.
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdint>
#include <cstring>
#include <string>

#include "hop.h"

// Scratch: one float per minibatch row.  Every GPU that loads the library holds these 64 KiB until
// the process exits.
static __device__ __align__(256) float g_static_coef[HOP_STATIC_MAX_ROWS];

namespace {

constexpr int kMaxDevices = 64;
// Device address of g_static_coef per device.  In host code the array's name is only a handle for
// the runtime, not an address a kernel can use; the address is looked up once per device.
float* g_coef_addr[kMaxDevices] = {};

int fail(int code, const std::string& msg, char* errbuf, int64_t errbuf_len) {
    if (errbuf && errbuf_len > 0) {
        const size_t n = std::min<size_t>(msg.size(), (size_t)errbuf_len - 1);
        std::memcpy(errbuf, msg.data(), n);
        errbuf[n] = 0;
    }
    return code;
}

__device__ __forceinline__ double warp_sum_f64(double v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// One warp per row: margin = a_r . x in double, coef_r = -y_r/rows if y_r * margin < 1 else 0.
__global__ void __launch_bounds__(256)
static_margin_kernel(const float* __restrict__ x, const int64_t* __restrict__ row_ptr, const int32_t* __restrict__ col,
                     const float* __restrict__ val, const float* __restrict__ y, int rows, float* __restrict__ coef) {
    const int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (r >= rows) return;
    double m = 0.0;
    for (int64_t t = row_ptr[r] + lane; t < row_ptr[r + 1]; t += 32) m += (double)val[t] * (double)x[col[t]];
    m = warp_sum_f64(m);
    if (lane == 0) coef[r] = ((double)y[r] * m < 1.0) ? -y[r] / (float)rows : 0.f;
}

// x_out[col] -= lr * coef_r * val, one warp per row.
__global__ void __launch_bounds__(256)
static_apply_kernel(float* __restrict__ x_out, const int64_t* __restrict__ row_ptr, const int32_t* __restrict__ col,
                    const float* __restrict__ val, int rows, float lr, const float* __restrict__ coef) {
    const int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
    if (r >= rows) return;
    const float cf = coef[r];
    if (cf == 0.f) return;
    const float scale = -lr * cf;
    for (int64_t t = row_ptr[r] + lane; t < row_ptr[r + 1]; t += 32) atomicAdd(x_out + col[t], scale * val[t]);
}

}  // namespace

extern "C" int hop_svm_csr_sgd_static(const float* x, float* x_out, int64_t P, const int64_t* row_ptr,
                                      const int32_t* col, const float* val, const float* y, int32_t rows,
                                      float lr, void* cuda_stream, char* errbuf, int64_t errbuf_len) {
    if (errbuf && errbuf_len > 0) errbuf[0] = 0;
    if (!x || !x_out || !row_ptr || !col || !val || !y || P <= 0 || rows <= 0)
        return fail(HOP_E_ARG, "hop_svm_csr_sgd_static: null pointer or non-positive size", errbuf, errbuf_len);
    if (rows > HOP_STATIC_MAX_ROWS)
        return fail(HOP_E_ARG, "hop_svm_csr_sgd_static: " + std::to_string(rows) + " rows exceed the built-in scratch of " +
                    std::to_string(HOP_STATIC_MAX_ROWS) + " rows; use hop_bind_svm_csr + hop_step for larger minibatches",
                    errbuf, errbuf_len);
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess || dev < 0 || dev >= kMaxDevices)
        return fail(HOP_E_CUDA, std::string("hop_svm_csr_sgd_static: cudaGetDevice: ") +
                    (e != cudaSuccess ? cudaGetErrorString(e) : "device index out of range"), errbuf, errbuf_len);
    if (!g_coef_addr[dev]) {   // first call on this device: resolve the array's device address
        float* p = nullptr;
        e = cudaGetSymbolAddress((void**)&p, g_static_coef);
        if (e != cudaSuccess || !p)
            return fail(HOP_E_CUDA, std::string("hop_svm_csr_sgd_static: cudaGetSymbolAddress: ") + cudaGetErrorString(e),
                        errbuf, errbuf_len);
        g_coef_addr[dev] = p;
    }
    float* coef = g_coef_addr[dev];
    cudaStream_t st = (cudaStream_t)cuda_stream;
    const int blocks = (rows * 32 + 255) / 256;
    static_margin_kernel<<<blocks, 256, 0, st>>>(x, row_ptr, col, val, y, rows, coef);
    static_apply_kernel<<<blocks, 256, 0, st>>>(x_out, row_ptr, col, val, rows, lr, coef);
    e = cudaGetLastError();
    if (e != cudaSuccess)
        return fail(HOP_E_CUDA, std::string("hop_svm_csr_sgd_static: kernel launch: ") + cudaGetErrorString(e), errbuf, errbuf_len);
    return HOP_OK;
}
