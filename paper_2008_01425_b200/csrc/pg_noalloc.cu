// pg_transposed_product_noalloc: z = X^T p without any allocation.
//
// Some callers cannot allocate device memory at the point where they need this
// product: code running inside a framework's memory-pool callback, a serving
// loop whose memory budget is fixed at start-up, or a region where an
// allocation would synchronise the device (cudaMalloc does) and stall the
// other streams.  For them the row-tile partial sums that the transposed sweep
// needs live in a fixed array inside this library instead of a caller-sized
// workspace.  The price is a size limit and no concurrency: see the header.
#include <cuda_runtime.h>

#include <cstdint>
#include <mutex>

#include "powergossip.h"

namespace {

constexpr int kTileRows = 256;                 // rows summed by one CTA
constexpr int kTileCols = 256;                 // columns per CTA: 64 threads x 4
constexpr long long kScratchFloats = PG_NOALLOC_MAX_PARTIALS;
constexpr int kMaxDevices = 64;
constexpr long long kMaxGridY = 65535;         // CUDA's limit on gridDim.y

// The scratch itself.  Every GPU that loads this library keeps its own copy
// until the process exits.  In host code this name is only a handle for the
// runtime's symbol lookup, never a device address.
static __device__ __align__(256) float g_partials[kScratchFloats];

std::mutex g_mutex;
float* g_partials_addr[kMaxDevices] = {};      // device address of g_partials, per device

// partials[rt][c] = sum over the rows of tile rt of p[r] * X[r][c]
template <bool VEC>
__global__ void __launch_bounds__(256)
xtp_partial_kernel(const float* __restrict__ X, int rows, int cols, long long ld,
                   const float* __restrict__ p, float* __restrict__ partials, int width) {
    __shared__ float s_p[kTileRows];
    __shared__ float s_red[3][kTileCols];
    const int r0 = blockIdx.y * kTileRows;
    const int r1 = min(rows, r0 + kTileRows);
    for (int t = threadIdx.x; t < kTileRows; t += 256) s_p[t] = (r0 + t < r1) ? p[r0 + t] : 0.0f;
    __syncthreads();
    const int tx = threadIdx.x & 63, ty = threadIdx.x >> 6;
    const int c = blockIdx.x * kTileCols + tx * 4;
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
    if (c < cols) {
        for (int r = r0 + ty; r < r1; r += 4) {
            const float pr = s_p[r - r0];
            const float* x = X + (long long)r * ld + c;
            if (VEC) {   // 16-byte rows: cols and ld are multiples of 4, X is 16-byte aligned
                const float4 v = *reinterpret_cast<const float4*>(x);
                a0 = fmaf(pr, v.x, a0); a1 = fmaf(pr, v.y, a1); a2 = fmaf(pr, v.z, a2); a3 = fmaf(pr, v.w, a3);
            } else {
                a0 = fmaf(pr, x[0], a0);
                if (c + 1 < cols) a1 = fmaf(pr, x[1], a1);
                if (c + 2 < cols) a2 = fmaf(pr, x[2], a2);
                if (c + 3 < cols) a3 = fmaf(pr, x[3], a3);
            }
        }
    }
    if (ty > 0) {
        s_red[ty - 1][tx * 4 + 0] = a0; s_red[ty - 1][tx * 4 + 1] = a1;
        s_red[ty - 1][tx * 4 + 2] = a2; s_red[ty - 1][tx * 4 + 3] = a3;
    }
    __syncthreads();
    if (ty == 0 && c < cols) {
        for (int t = 0; t < 3; ++t) {
            a0 += s_red[t][tx * 4 + 0]; a1 += s_red[t][tx * 4 + 1];
            a2 += s_red[t][tx * 4 + 2]; a3 += s_red[t][tx * 4 + 3];
        }
        float* out = partials + (long long)blockIdx.y * width + c;
        out[0] = a0;
        if (c + 1 < cols) out[1] = a1;
        if (c + 2 < cols) out[2] = a2;
        if (c + 3 < cols) out[3] = a3;
    }
}

// z[c] = partials[0][c] + partials[1][c] + ...   (fixed order, fp64 sum)
__global__ void __launch_bounds__(256)
xtp_reduce_kernel(const float* __restrict__ partials, int rtiles, int cols, int width,
                  float* __restrict__ z) {
    const int c = blockIdx.x * 256 + threadIdx.x;
    if (c >= cols) return;
    double s = 0.0;
    for (int rt = 0; rt < rtiles; ++rt) s += (double)partials[(long long)rt * width + c];
    z[c] = (float)s;
}

// Device address of g_partials on the current device, looked up once per device.
int scratch_address(float** out) {
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return PG_ERR_CUDA;
    std::lock_guard<std::mutex> lock(g_mutex);
    if (!g_partials_addr[dev]) {
        float* addr = nullptr;
        const cudaError_t rc = cudaGetSymbolAddress(reinterpret_cast<void**>(&addr), g_partials);
        if (rc != cudaSuccess || !addr) {
            cudaGetLastError();
            return PG_ERR_CUDA;
        }
        g_partials_addr[dev] = addr;
    }
    *out = g_partials_addr[dev];
    return PG_OK;
}

bool on_current_device(const void* ptr) {
    int dev = -1;
    cudaPointerAttributes attr{};
    if (cudaGetDevice(&dev) != cudaSuccess) return false;
    if (cudaPointerGetAttributes(&attr, ptr) != cudaSuccess) {
        cudaGetLastError();
        return false;
    }
    return attr.type == cudaMemoryTypeDevice && attr.device == dev;
}

}  // namespace

extern "C" int pg_transposed_product_noalloc(const float* X_dev, int32_t rows, int32_t cols, int64_t ld,
                                             const float* p_dev, float* z_dev, void* stream_v) {
    if (!X_dev || !p_dev || !z_dev || rows < 1 || cols < 1 || ld < cols) return PG_ERR_INVALID;
    // sizes in 64 bits: cols near INT_MAX must not wrap while being rounded up
    const long long rtiles_ll = (static_cast<long long>(rows) + kTileRows - 1) / kTileRows;
    const long long width_ll = (static_cast<long long>(cols) + 3) / 4 * 4;      // one row of partials
    if (rtiles_ll * width_ll > kScratchFloats) return PG_ERR_TOO_LARGE;
    if (rtiles_ll > kMaxGridY) return PG_ERR_TOO_LARGE;      // row tiles are the launch's second grid dimension
    const int rtiles = static_cast<int>(rtiles_ll);
    const int width = static_cast<int>(width_ll);
    if (!on_current_device(X_dev) || !on_current_device(p_dev) || !on_current_device(z_dev)) return PG_ERR_INVALID;
    float* partials = nullptr;
    const int rc = scratch_address(&partials);
    if (rc != PG_OK) return rc;
    cudaStream_t stream = static_cast<cudaStream_t>(stream_v);
    const dim3 grid((cols + kTileCols - 1) / kTileCols, rtiles);
    const bool vec = cols % 4 == 0 && ld % 4 == 0 && reinterpret_cast<uintptr_t>(X_dev) % 16 == 0;
    // every cell of the scratch that the second kernel reads is written by the
    // first one in this same call, so nothing left over from an earlier call is
    // ever read and nothing needs clearing
    if (vec)
        xtp_partial_kernel<true><<<grid, 256, 0, stream>>>(X_dev, rows, cols, ld, p_dev, partials, width);
    else
        xtp_partial_kernel<false><<<grid, 256, 0, stream>>>(X_dev, rows, cols, ld, p_dev, partials, width);
    // z is written only if the partial sums were really enqueued
    if (cudaGetLastError() != cudaSuccess) return PG_ERR_CUDA;
    xtp_reduce_kernel<<<(cols + 255) / 256, 256, 0, stream>>>(partials, rtiles, cols, width, z_dev);
    if (cudaGetLastError() != cudaSuccess) return PG_ERR_CUDA;
    return PG_OK;
}
