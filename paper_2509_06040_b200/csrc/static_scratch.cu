// bgrpo_reward_mse_static: the -MSE row reduction of the leaf-reward kernel for callers that cannot hand the
// library a scratch buffer.  Its reduction partials and ticket counters live in a fixed array that is part of the
// loaded library image on every GPU, so the call needs no cudaMalloc from anybody.  The paper has no counterpart;
// this is a deployment convenience.
#include <mutex>

#include "internal.h"

namespace bgrpo {
namespace {

constexpr int kStaticVec = kChunkVec / kStreamThreads;                       // float4 per thread
constexpr size_t kCounterBytes = BGRPO_STATIC_MAX_ROWS * sizeof(unsigned int);
constexpr size_t kPartialSlots = (BGRPO_STATIC_SCRATCH_BYTES - kCounterBytes) / sizeof(double);

// [0, kCounterBytes): one ticket counter per row; the rest: one double per (row, chunk).
static __device__ __align__(256) unsigned char g_static_scratch[BGRPO_STATIC_SCRATCH_BYTES];

// One CTA per (row, chunk of kChunkVec float4).  Thread sums are float over 16 elements, everything above that is
// double; the CTA that draws a row's last ticket adds the row's chunk partials in a fixed order and writes r.
__global__ void __launch_bounds__(kStreamThreads)
reward_mse_static_kernel(const float* __restrict__ rows, const float* __restrict__ target, float* __restrict__ r_out,
                         unsigned char* scratch, int64_t D, int32_t nchunks) {
    unsigned int* counters = reinterpret_cast<unsigned int*>(scratch);
    double* partials = reinterpret_cast<double*>(scratch + kCounterBytes);
    const int chunk = blockIdx.x % nchunks;
    const int row = blockIdx.x / nchunks;
    const int64_t D4 = D >> 2;
    const float4* __restrict__ z = reinterpret_cast<const float4*>(rows + static_cast<int64_t>(row) * D);
    const float4* __restrict__ tg = reinterpret_cast<const float4*>(target);
    float acc = 0.0f;
#pragma unroll
    for (int k = 0; k < kStaticVec; ++k) {
        const int64_t e = static_cast<int64_t>(chunk) * kChunkVec + k * kStreamThreads + threadIdx.x;
        if (e < D4) {
            const float4 a = __ldcs(z + e), t = __ldg(tg + e);
            const float dx = a.x - t.x, dy = a.y - t.y, dz = a.z - t.z, dw = a.w - t.w;
            acc = fmaf(dx, dx, acc);
            acc = fmaf(dy, dy, acc);
            acc = fmaf(dz, dz, acc);
            acc = fmaf(dw, dw, acc);
        }
    }
    __shared__ double red[kStreamThreads / 32];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    double s = static_cast<double>(acc);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_down_sync(0xffffffffu, s, o);
    if (lane == 0) red[warp] = s;
    __syncthreads();
    if (warp != 0) return;
    int last = 0;
    if (lane == 0) {
        double cta = 0.0;
#pragma unroll
        for (int w = 0; w < kStreamThreads / 32; ++w) cta += red[w];
        __stcg(&partials[static_cast<int64_t>(row) * nchunks + chunk], cta);
        __threadfence();
        last = (atomicAdd(&counters[row], 1u) == static_cast<unsigned int>(nchunks) - 1u);
        if (last) __threadfence();
    }
    if (!__shfl_sync(0xffffffffu, last, 0)) return;
    double tot = 0.0;
    for (int c = lane; c < nchunks; c += 32) tot += __ldcg(&partials[static_cast<int64_t>(row) * nchunks + c]);
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) tot += __shfl_down_sync(0xffffffffu, tot, o);
    if (lane == 0) r_out[row] = static_cast<float>(-tot / static_cast<double>(D));
}

constexpr int kMaxDevices = 64;
std::mutex g_setup_mutex;
unsigned char* g_scratch_addr[kMaxDevices] = {nullptr};

// Device address of g_static_scratch on the current device.  In host code the symbol's name is only a handle, not an
// address a kernel can use; the address is asked for once per device, with that device current, and remembered.
cudaError_t static_scratch_address(unsigned char** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_setup_mutex);
    if (!g_scratch_addr[dev]) {
        void* ptr = nullptr;
        e = cudaGetSymbolAddress(&ptr, g_static_scratch);
        if (e != cudaSuccess) return e;
        g_scratch_addr[dev] = static_cast<unsigned char*>(ptr);
    }
    *out = g_scratch_addr[dev];
    return cudaSuccess;
}

}  // namespace
}  // namespace bgrpo

extern "C" {

bgrpo_status bgrpo_reward_mse_static(const float* rows_dev, const float* target_dev, int32_t n_rows, int64_t D,
                                     float* r_out_dev, void* stream) {
    using namespace bgrpo;
    if (!rows_dev || !target_dev || !r_out_dev) return BGRPO_ERR_INVALID_ARG;   // NULL pointer
    if ((reinterpret_cast<uintptr_t>(rows_dev) | reinterpret_cast<uintptr_t>(target_dev)) % 16 != 0)
        return BGRPO_ERR_INVALID_ARG;   // rows_dev and target_dev must be 16-byte aligned
    if (n_rows < 1 || D < 4 || D % 4 != 0) return BGRPO_ERR_INVALID_ARG;   // n_rows must be >= 1 and D a positive multiple of 4
    if (n_rows > BGRPO_STATIC_MAX_ROWS)
        return BGRPO_ERR_CAPACITY;   // n_rows exceeds BGRPO_STATIC_MAX_ROWS: split the call or use bgrpo_leaf_reward_mse
    const int64_t nchunks = (D / 4 + kChunkVec - 1) / kChunkVec;
    if (static_cast<uint64_t>(n_rows) * static_cast<uint64_t>(nchunks) > kPartialSlots)
        return BGRPO_ERR_CAPACITY;   // n_rows * ceil(D/4096) exceeds the built-in scratch: split the call or use bgrpo_leaf_reward_mse
    unsigned char* scratch = nullptr;
    cudaError_t e = static_scratch_address(&scratch);
    if (e != cudaSuccess) return BGRPO_ERR_CUDA;
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    // the array keeps whatever the previous call left: the ticket counters must start at zero, the partials are
    // all rewritten before they are read
    e = cudaMemsetAsync(scratch, 0, static_cast<size_t>(n_rows) * sizeof(unsigned int), s);
    if (e != cudaSuccess) return BGRPO_ERR_CUDA;
    reward_mse_static_kernel<<<static_cast<unsigned int>(n_rows * nchunks), kStreamThreads, 0, s>>>(
        rows_dev, target_dev, r_out_dev, scratch, D, static_cast<int32_t>(nchunks));
    e = cudaGetLastError();
    if (e != cudaSuccess) return BGRPO_ERR_CUDA;
    return BGRPO_OK;
}

}  // extern "C"
