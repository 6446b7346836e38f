// lq_vector_norm_static: the L^q norm of one device vector without any allocation.
//
// Some callers cannot allocate device memory at the moment they need a norm: a process whose whole
// device memory was handed to another allocator at start-up (a training framework's caching pool, a
// serving process with fixed partitions), or a latency-critical loop in which the device-wide
// synchronisation that cudaMalloc / cudaFree imply is not acceptable.  A plan (lq_plan_create)
// allocates its tables and reduction scratch, so those callers cannot use lq_layer_norms.  This
// entry point keeps the scratch of the two-stage reduction in a fixed array that is part of the
// library image instead: every GPU that loads the library holds kStaticTiles doubles (32 KB) until
// the process exits.
//
// The array is shared by all calls.  Each call overwrites exactly the entries it reads back, so
// nothing has to be cleared between calls, but two calls that overlap on the GPU (different
// streams, or different host threads) race on it: the caller must order them.
#include <mutex>

#include "lq_internal.cuh"

namespace lq {
namespace {

constexpr int kStaticTiles = 4096;                                    // one fp64 partial per tile
constexpr int kStaticTileBlocks = 32;                                 // blocks of 1024 values per tile
constexpr int64_t kStaticTileCoords = (int64_t)kStaticTileBlocks * kBlockCoords;
constexpr int64_t kStaticMaxCoords = kStaticTiles * kStaticTileCoords;
constexpr int kMaxDevices = 64;

// In host code this name is only a handle for cudaGetSymbolAddress; kernels receive the address.
static __device__ __align__(256) double g_static_partials[kStaticTiles];

std::mutex g_setup_mutex;
double* g_partials_addr[kMaxDevices] = {};

// mode 0: max |v|   1: sum |v|   2: sum v^2   3: sum |v|^q (integer q >= 3)
template <int kMode>
__device__ __forceinline__ void add_term(double& acc, float v, int q)
{
    const double a = fabs((double)v);
    if (kMode == 0)      acc = fmax(acc, a);
    else if (kMode == 1) acc += a;
    else if (kMode == 2) acc = fma(a, a, acc);
    else { double p = a; for (int r = 1; r < q; ++r) p = __dmul_rn(p, a); acc += p; }
}

// One CTA per tile of 32 blocks of 1024 values; a lane takes the float4 at 128 j + 4 lane of
// a block, the same ownership and summation order as the plan-based norm.  A non-finite value
// makes the partial NaN.
template <int kMode>
__global__ void __launch_bounds__(kThreads) static_norm_partial_kernel(const float* __restrict__ v, int64_t n,
                                                                       int q, double* __restrict__ partials)
{
    __shared__ double scratch[kWarps];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int64_t first_block = (int64_t)blockIdx.x * kStaticTileBlocks;
    const int64_t nblocks = (n + kBlockCoords - 1) / kBlockCoords;
    double acc = 0.0;
    int bad = 0;
    for (int b = warp; b < kStaticTileBlocks && first_block + b < nblocks; b += kWarps) {
        const int64_t base = (first_block + b) * kBlockCoords + 4 * lane;
        for (int j = 0; j < 8; ++j) {
            const int64_t pos = base + 128 * j;
            float x[4] = {0.f, 0.f, 0.f, 0.f};
            if (pos + 4 <= n) {
                const float4 t = __ldg(reinterpret_cast<const float4*>(v + pos));
                x[0] = t.x; x[1] = t.y; x[2] = t.z; x[3] = t.w;
            } else {
                for (int e = 0; e < 4; ++e) if (pos + e < n) x[e] = __ldg(v + pos + e);
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (!(fabsf(x[e]) <= 3.402823466e38f)) bad = 1;
                add_term<kMode>(acc, x[e], q);
            }
        }
    }
    bad = __syncthreads_or(bad);
    double r = kMode == 0 ? block_reduce<true>(acc, scratch) : block_reduce<false>(acc, scratch);
    if (bad) r = __longlong_as_double(0x7ff8000000000000LL);
    if (threadIdx.x == 0) partials[blockIdx.x] = r;
}

// Adds the partials in a fixed order, takes the root and rounds to fp32.  status: 0 ok,
// LQ_STATUS_ZERO_NORM, LQ_STATUS_NONFINITE (the norm is reported as 0 in both flagged cases).
__global__ void __launch_bounds__(128) static_norm_finalize_kernel(const double* __restrict__ partials, int ntiles,
                                                                   int q, float* __restrict__ norm_out,
                                                                   uint32_t* __restrict__ status_out)
{
    __shared__ double scratch[4];
    double acc = 0.0;
    int bad = 0;
    for (int i = threadIdx.x; i < ntiles; i += blockDim.x) {
        const double t = partials[i];
        if (!(fabs(t) <= 1.7976931348623157e308)) bad = 1;
        if (q == 0) acc = fmax(acc, t); else acc += t;
    }
    bad = __syncthreads_or(bad);
    const double total = q == 0 ? block_reduce<true>(acc, scratch) : block_reduce<false>(acc, scratch);
    if (threadIdx.x == 0) {
        double n64;
        if (q == 0 || q == 1) n64 = total;
        else if (q == 2)      n64 = sqrt(total);
        else                  n64 = pow(total, 1.0 / (double)q);
        float nf = (float)n64;
        uint32_t st = 0;
        if (bad || !(fabs(n64) <= 1.7976931348623157e308) || !(fabsf(nf) <= 3.402823466e38f)) st = LQ_STATUS_NONFINITE;
        else if (nf < 1.17549435e-38f) st = LQ_STATUS_ZERO_NORM;
        *norm_out = st ? 0.0f : nf;
        if (status_out) *status_out = st;
    }
}

}  // namespace
}  // namespace lq

extern "C" int lq_vector_norm_static(const float* v, int64_t n, int32_t q, float* norm_out,
                                     uint32_t* status_out, void* stream)
{
    using namespace lq;
    if ((!v && n > 0) || !norm_out) return lq_set_error(LQ_EINVAL, "lq_vector_norm_static: v or norm_out is NULL");
    if (n < 0 || n > kStaticMaxCoords)
        return lq_set_error(LQ_EINVAL, "lq_vector_norm_static: n = %lld is outside [0, %lld], the size the "
                            "library's fixed scratch array covers", (long long)n, (long long)kStaticMaxCoords);
    if (q < 0 || q > 16) return lq_set_error(LQ_EINVAL, "lq_vector_norm_static: q must be 0 (infinity norm) or 1..16");
    if (reinterpret_cast<uintptr_t>(v) % 16 != 0)
        return lq_set_error(LQ_EINVAL, "lq_vector_norm_static: v must be 16-byte aligned");

    // once per device: ask the runtime where this device keeps the scratch array
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return lq_set_error(LQ_ECUDA, "cudaGetDevice: %s", cudaGetErrorString(e));
    if (dev < 0 || dev >= kMaxDevices) return lq_set_error(LQ_EINVAL, "device index %d not supported", dev);
    double* partials = nullptr;
    {
        std::lock_guard<std::mutex> lock(g_setup_mutex);
        if (!g_partials_addr[dev]) {
            void* addr = nullptr;
            e = cudaGetSymbolAddress(&addr, g_static_partials);
            if (e != cudaSuccess || !addr)
                return lq_set_error(LQ_ECUDA, "cudaGetSymbolAddress(scratch): %s", cudaGetErrorString(e));
            g_partials_addr[dev] = static_cast<double*>(addr);
        }
        partials = g_partials_addr[dev];
    }

    cudaStream_t s = (cudaStream_t)stream;
    const int ntiles = (int)((n + kStaticTileCoords - 1) / kStaticTileCoords);
    if (ntiles > 0) {
        if (q == 0)      static_norm_partial_kernel<0><<<ntiles, kThreads, 0, s>>>(v, n, q, partials);
        else if (q == 1) static_norm_partial_kernel<1><<<ntiles, kThreads, 0, s>>>(v, n, q, partials);
        else if (q == 2) static_norm_partial_kernel<2><<<ntiles, kThreads, 0, s>>>(v, n, q, partials);
        else             static_norm_partial_kernel<3><<<ntiles, kThreads, 0, s>>>(v, n, q, partials);
        e = cudaGetLastError();
        if (e != cudaSuccess) return lq_set_error(LQ_ECUDA, "static_norm_partial_kernel: %s", cudaGetErrorString(e));
    }
    static_norm_finalize_kernel<<<1, 128, 0, s>>>(partials, ntiles, q, norm_out, status_out);
    e = cudaGetLastError();
    if (e != cudaSuccess) return lq_set_error(LQ_ECUDA, "static_norm_finalize_kernel: %s", cudaGetErrorString(e));
    return LQ_OK;
}
