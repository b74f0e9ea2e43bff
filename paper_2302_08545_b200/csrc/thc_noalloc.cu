// thc_prepare_noalloc: the preliminary stage for callers that must not allocate.
//
// Who needs this.  Some hosts of this library run where cudaMalloc is off limits: inside a
// framework's pre-planned memory pool, in a plugin that is handed its buffers and may not
// grow the process's device footprint, or in code that runs while a memory-accounting tool
// has frozen allocations.  thc_prepare needs scratch (one fp64 partial sum per 2^14
// coordinates per worker) and takes it from the caller's workspace, whose size the caller
// has to ask for and allocate; thc_create allocates the context's device block.  This entry
// point needs neither: its scratch is a fixed array in the library's own device image, and it
// takes the few parameters it needs as plain arguments instead of a context.
//
// The price: the array exists on every GPU that loads the library, for the life of the
// process (THC_NOALLOC_SCRATCH_BYTES), inputs larger than it can serve are refused, and all
// calls share it, so two calls that overlap on the GPU (different streams, or different host
// threads) race.  Nothing in it has to start at zero: every slot a call reads is written by
// that call first.
#include "../../include/thc.h"

#include <cuda_runtime.h>
#include <math.h>
#include <stdint.h>

namespace {

constexpr int kChunkLog2Max = 14;            // coordinates summed by one CTA
constexpr int kThreadsNA = 256;
constexpr uint64_t kMaxPartials = THC_NOALLOC_SCRATCH_BYTES / sizeof(double);
constexpr int kMaxDevices = 64;

// The scratch.  In host code this name is only a handle for cudaGetSymbolAddress; kernels
// get the device address as an argument.
static __device__ __align__(256) double g_noalloc_partials[kMaxPartials];

struct PtrArrayNA { const void *p[THC_MAX_WORKERS]; };

__device__ __forceinline__ float4 load4_masked(const float *x, uint64_t j, uint64_t d)
{
    if (j + 4 <= d) return __ldg(reinterpret_cast<const float4 *>(x + j));
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (j + 0 < d) v.x = __ldg(x + j + 0);
    if (j + 1 < d) v.y = __ldg(x + j + 1);
    if (j + 2 < d) v.z = __ldg(x + j + 2);
    if (j + 3 < d) v.w = __ldg(x + j + 3);
    return v;
}

// Sum of squares of one chunk of one worker, fp64, fixed order.
template <bool BF16>
__global__ void __launch_bounds__(kThreadsNA)
noalloc_partial_kernel(PtrArrayNA in, uint64_t d, uint32_t chunk_log2, uint64_t chunks_per_worker,
                       double *__restrict__ partial)
{
    const uint64_t chunk = blockIdx.x;
    const uint32_t wl = blockIdx.y;
    const uint64_t j0 = chunk << chunk_log2;
    const int n4 = 1 << (chunk_log2 - 2);
    double s = 0.0;
    for (int c = threadIdx.x; c < n4; c += kThreadsNA) {
        const uint64_t j = j0 + (uint64_t)c * 4;
        if (j >= d) break;
        float4 v;
        if (BF16) {
            const uint16_t *x = static_cast<const uint16_t *>(in.p[wl]);
            uint32_t w0 = 0, w1 = 0;
            if (j + 4 <= d) {
                const uint2 q = __ldg(reinterpret_cast<const uint2 *>(x + j));
                w0 = q.x; w1 = q.y;
            } else {
                for (int e = 0; e < 4; ++e)
                    if (j + e < d) {
                        const uint32_t h = (uint32_t)__ldg(x + j + e) << ((e & 1) * 16);
                        if (e < 2) w0 |= h; else w1 |= h;
                    }
            }
            v = make_float4(__uint_as_float(w0 << 16), __uint_as_float(w0 & 0xFFFF0000u),
                            __uint_as_float(w1 << 16), __uint_as_float(w1 & 0xFFFF0000u));
        } else {
            v = load4_masked(static_cast<const float *>(in.p[wl]), j, d);
        }
        s = fma((double)v.x, (double)v.x, s);
        s = fma((double)v.y, (double)v.y, s);
        s = fma((double)v.z, (double)v.z, s);
        s = fma((double)v.w, (double)v.w, s);
    }
    __shared__ double red[kThreadsNA / 32];
    for (int off = 16; off > 0; off >>= 1) s += __shfl_down_sync(0xFFFFFFFFu, s, off);
    if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = s;
    __syncthreads();
    if (threadIdx.x == 0) {
        double t = 0.0;
        for (int w = 0; w < kThreadsNA / 32; ++w) t += red[w];
        partial[(uint64_t)wl * chunks_per_worker + chunk] = t;
    }
}

// M per block: one warp per RHT block, fixed summation order.
__global__ void __launch_bounds__(128)
noalloc_final_kernel(const double *__restrict__ partial, uint32_t n, uint64_t nblocks,
                     uint64_t chunks_per_block, uint64_t chunks_per_worker, double t_p, uint32_t k,
                     float *__restrict__ scales, uint32_t *status)
{
    const uint64_t blk = ((uint64_t)blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (blk >= nblocks) return;
    double ell = 0.0;
    for (uint32_t i = 0; i < n; ++i) {
        double s = 0.0;
        const double *p = partial + (uint64_t)i * chunks_per_worker + blk * chunks_per_block;
        for (uint64_t c = lane; c < chunks_per_block; c += 32) s += p[c];
        for (int off = 16; off > 0; off >>= 1) s += __shfl_xor_sync(0xFFFFFFFFu, s, off);
        const double norm = sqrt(s);
        if (norm > ell || norm != norm) ell = norm;
    }
    if (lane != 0) return;
    float M = (float)(t_p * ell / sqrt((double)((uint64_t)1 << k)));
    uint32_t flags = 0;
    if (!isfinite(M)) { M = 0.0f; flags |= THC_STATUS_NONFINITE; }
    if (M == 0.0f) flags |= THC_STATUS_ZERO_BLOCK;
    scales[blk] = M;
    if (flags != 0 && status != nullptr) atomicOr(status, flags);
}

// Device address of the scratch on the current device, looked up once per device.
int scratch_address(double **out)
{
    static double *addr[kMaxDevices];
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return THC_ECUDA;
    if (addr[dev] == nullptr) {
        void *p = nullptr;
        if (cudaGetSymbolAddress(&p, g_noalloc_partials) != cudaSuccess || p == nullptr)
            return THC_ECUDA;
        addr[dev] = static_cast<double *>(p);
    }
    *out = addr[dev];
    return THC_OK;
}

}  // namespace

extern "C" int thc_prepare_noalloc(const void *const *grads, uint32_t n, uint64_t d,
                                   uint32_t log2_block, uint32_t in_dtype, double t_p,
                                   float *scales, uint32_t *status_or_null, void *stream)
{
    if (grads == nullptr || scales == nullptr || n == 0 || n > THC_MAX_WORKERS || d == 0)
        return THC_EINVAL;
    if (log2_block < 3 || log2_block > 22) return THC_EINVAL;
    if (in_dtype != THC_F32 && in_dtype != THC_BF16) return THC_EINVAL;
    if (!(t_p > 0.0) || !isfinite(t_p)) return THC_EINVAL;
    for (uint32_t i = 0; i < n; ++i)
        if (grads[i] == nullptr || (reinterpret_cast<uintptr_t>(grads[i]) & 15u) != 0) return THC_EINVAL;
    if (d > (1ull << 40)) return THC_EINVAL;          // the bound every other entry point applies
    const uint64_t B = 1ull << log2_block;
    const uint64_t d_pad = (d + B - 1) / B * B;
    const uint64_t nblocks = d_pad / B;
    const uint32_t chunk_log2 = log2_block < (uint32_t)kChunkLog2Max ? log2_block : (uint32_t)kChunkLog2Max;
    const uint64_t chunks_per_worker = d_pad >> chunk_log2;
    const uint64_t chunks_per_block = 1ull << (log2_block - chunk_log2);
    if (chunks_per_worker > 0x7FFFFFFFull) return THC_EUNSUPPORTED;
    if ((uint64_t)n * chunks_per_worker > kMaxPartials) return THC_EWORKSPACE;   // beyond the built-in scratch

    double *partial = nullptr;
    const int rc = scratch_address(&partial);     // first call on a device: symbol look-up
    if (rc != THC_OK) return rc;

    cudaStream_t st = static_cast<cudaStream_t>(stream);
    PtrArrayNA in;
    for (uint32_t i = 0; i < THC_MAX_WORKERS; ++i) in.p[i] = i < n ? grads[i] : nullptr;
    const dim3 grid((unsigned)chunks_per_worker, n);
    if (in_dtype == THC_BF16)
        noalloc_partial_kernel<true><<<grid, kThreadsNA, 0, st>>>(in, d, chunk_log2, chunks_per_worker, partial);
    else
        noalloc_partial_kernel<false><<<grid, kThreadsNA, 0, st>>>(in, d, chunk_log2, chunks_per_worker, partial);
    if (cudaGetLastError() != cudaSuccess) return THC_ECUDA;
    noalloc_final_kernel<<<(unsigned)((nblocks + 3) / 4), 128, 0, st>>>(
        partial, n, nblocks, chunks_per_block, chunks_per_worker, t_p, log2_block, scales, status_or_null);
    if (cudaGetLastError() != cudaSuccess) return THC_ECUDA;
    return THC_OK;
}
