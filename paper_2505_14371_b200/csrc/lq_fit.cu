// Level update (Algorithm 1 lines 2-7): for each layer, merge the sampled histograms with the
// weights lambda_z = N_z^2 / sum N_z^2 and minimise
//     sum_j int_{l_j}^{l_{j+1}} (l_{j+1} - u)(u - l_j) dF~(u)
// (Section 3.2 of the paper, the minimisation that follows Eq. MQV).  The paper gives the objective
// only; the solver is exact coordinate minimisation: with neighbours a < c fixed, the optimal level
// l solves  F~(l) = F~(c) - int_a^c (u - a)/(c - a) dF~(u).  F~ is piecewise linear (uniform density
// inside a histogram bin), so F~, its first moment and its inverse are closed forms.
//
// Coordinate descent stops at a local minimum, and the objective has several when the density is not log-concave
// (a step density already has two), so the descent runs from two starts, the quantiles of the mass above bin 0 and the
// uniform grid, and the end point with the smaller objective is kept (the uniform start's only if it is smaller by
// more than one part in 10^9, so that rounding does not decide between two copies of the same minimum).
//
// One CTA per layer; odd and even interior levels are updated in two parallel half-sweeps (levels of
// one parity only depend on the other parity).  All arithmetic is fp64 and this file is compiled
// without FMA contraction so that the sequence of roundings is the plain one.
#include "lq_internal.cuh"

namespace lq {

constexpr int kBins = 385;            // bins 0..384 carry density; bin 385 (u = 1) never adds variance
constexpr int kFitThreads = 128;
constexpr int kMaxSweeps = 100;

struct FitSmem {
    double e[kBins + 1];
    double mass[kBins];
    double F[kBins + 1];
    double M1[kBins + 1];
    double M2[kBins + 1];
    double l[kMaxLevels];
    double lb[kMaxLevels];
    double term[kMaxLevels];
    double obj[2];
    double lambda[LQ_MAX_WORKERS];
    double red[kFitThreads / 32];
    double moved;
    int ok;
};

__device__ __forceinline__ double bin_edge(int i)
{
    if (i <= 0) return 0.0;
    const int o = (i - 1) >> 4, m = (i - 1) & 15;
    return ldexp(1.0 + (double)m * 0.0625, o - 24);
}

__device__ int bin_of(const FitSmem& s, double x)
{
    int lo = 0, hi = kBins - 1;
    while (lo < hi) {
        const int mid = (lo + hi + 1) >> 1;
        if (s.e[mid] <= x) lo = mid; else hi = mid - 1;
    }
    return lo;
}

__device__ double cdf(const FitSmem& s, double x, double* m1)
{
    const int i = bin_of(s, x);
    double theta = (x - s.e[i]) / (s.e[i + 1] - s.e[i]);
    if (theta > 1.0) theta = 1.0;
    const double part = s.mass[i] * theta;
    *m1 = s.M1[i] + part * ((s.e[i] + x) * 0.5);
    return s.F[i] + part;
}

// int_0^x u^2 dF~(u); inside a bin int_{e0}^{x} u^2 = (mass in [e0, x]) * (e0^2 + e0 x + x^2) / 3
__device__ double second_moment(const FitSmem& s, double x)
{
    const int i = bin_of(s, x);
    double theta = (x - s.e[i]) / (s.e[i + 1] - s.e[i]);
    if (theta > 1.0) theta = 1.0;
    const double part = s.mass[i] * theta;
    return s.M2[i] + part * ((s.e[i] * s.e[i] + s.e[i] * x + x * x) / 3.0);
}

__device__ double cdf_inv(const FitSmem& s, double y)
{
    int lo = 0, hi = kBins;
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (s.F[mid + 1] > y) hi = mid; else lo = mid + 1;
    }
    if (lo >= kBins) return 1.0;
    double t = (y - s.F[lo]) / s.mass[lo];
    if (t < 0.0) t = 0.0;
    return s.e[lo] + t * (s.e[lo + 1] - s.e[lo]);
}

// Odd/even sweeps of exact coordinate minimisation on the levels l (shared memory), by the whole CTA.
__device__ void descend(FitSmem& s, double* l, int n, int tid)
{
    for (int sweep = 0; sweep < kMaxSweeps; ++sweep) {
        double moved = 0.0;
        for (int parity = 1; parity >= 0; --parity) {
            for (int j = tid; j <= n - 2; j += kFitThreads) {
                if (j < 1 || (j & 1) != parity) continue;
                const double a = l[j - 1], c = l[j + 1];
                if (!(c > a)) continue;
                double m1a, m1c, b;
                const double Fa = cdf(s, a, &m1a), Fc = cdf(s, c, &m1c);
                const double mass_ac = Fc - Fa;
                if (!(mass_ac > 0.0)) b = (a + c) * 0.5;
                else {
                    const double target = Fc - ((m1c - m1a) - a * mass_ac) / (c - a);
                    b = cdf_inv(s, target);
                    if (b < a) b = a;
                    if (b > c) b = c;
                }
                const double rel = fabs(b - l[j]) / (fabs(b) > 1e-300 ? fabs(b) : 1e-300);
                if (rel > moved) moved = rel;
                l[j] = b;
            }
            __syncthreads();
        }
        moved = warp_max(moved);
        if ((tid & 31) == 0) s.red[tid >> 5] = moved;
        __syncthreads();
        if (tid == 0) {
            double mx = s.red[0];
            for (int w = 1; w < kFitThreads / 32; ++w) mx = fmax(mx, s.red[w]);
            s.moved = mx;
        }
        __syncthreads();
        if (s.moved <= 1e-13) break;
    }
    __syncthreads();
}

// The objective at the levels l: interval j gives -(M2(c) - M2(a)) + (a + c)(M1(c) - M1(a)) - a c (F(c) - F(a));
// the intervals are added in order by one thread so that the sum does not depend on the CTA's shape.
__device__ void objective(FitSmem& s, const double* l, int n, int tid, double* out)
{
    for (int j = tid; j + 1 < n; j += kFitThreads) {
        const double a = l[j], c = l[j + 1];
        double m1a, m1c;
        const double Fa = cdf(s, a, &m1a), Fc = cdf(s, c, &m1c);
        const double m2a = second_moment(s, a), m2c = second_moment(s, c);
        s.term[j] = ((a + c) * (m1c - m1a) - (m2c - m2a)) - (a * c) * (Fc - Fa);
    }
    __syncthreads();
    if (tid == 0) {
        double total = 0.0;
        for (int j = 0; j + 1 < n; ++j) total += s.term[j];
        *out = total;
    }
    __syncthreads();
}

// Per-layer mode (member_off == nullptr): CTA m fits layer m.  Shared mode: CTA t fits one sequence for type t,
// whose member layers are member_layer[member_off[t] .. member_off[t+1]) (all with the same level count): the
// histograms of all (sample, member) pairs are merged with weights N^2 (the variance to minimise is
// sum N_s^2 sum_i sigma^2(u_i)), scaled by sum N_s^2 d_s, and the result goes to every member.
__global__ void __launch_bounds__(kFitThreads) fit_levels_kernel(PlanDev p, const uint32_t* __restrict__ hist,
                                                                 const float* __restrict__ norms, int Z,
                                                                 float* __restrict__ levels_stage,
                                                                 const int32_t* __restrict__ member_off,
                                                                 const int32_t* __restrict__ member_layer)
{
    __shared__ FitSmem s;
    const bool shared_fit = member_off != nullptr;
    const int m0 = shared_fit ? member_off[blockIdx.x] : 0, m1 = shared_fit ? member_off[blockIdx.x + 1] : 0;
    if (shared_fit && m1 <= m0) return;
    const int m = shared_fit ? member_layer[m0] : blockIdx.x;
    const LayerDesc L = p.layers[m];
    const int n = L.nlevels;
    if (n < 3) return;
    const int tid = threadIdx.x;

    if (shared_fit) {
        if (tid == 0) {
            double wd = 0.0;
            for (int z = 0; z < Z; ++z)
                for (int j = m0; j < m1; ++j) {
                    const int mm = member_layer[j];
                    const double w = (double)norms[(int64_t)z * p.num_layers + mm];
                    wd += w * w * (double)p.layers[mm].size;
                }
            s.moved = wd;
            s.ok = wd > 0.0;
        }
        __syncthreads();
        if (!s.ok) return;
        const double wd = s.moved;
        for (int i = tid; i <= kBins; i += kFitThreads) s.e[i] = bin_edge(i);
        for (int i = tid; i < kBins; i += kFitThreads) {
            double acc = 0.0;
            for (int z = 0; z < Z; ++z)
                for (int j = m0; j < m1; ++j) {
                    const int mm = member_layer[j];
                    const double w = (double)norms[(int64_t)z * p.num_layers + mm];
                    acc += (w * w) * (double)hist[((int64_t)z * p.num_layers + mm) * LQ_HIST_STRIDE + i];
                }
            s.mass[i] = acc / wd;
        }
        __syncthreads();
    } else {
    if (L.size <= 0) return;

    if (tid == 0) {
        double wsum = 0.0;
        for (int z = 0; z < Z; ++z) {
            const double w = (double)norms[(int64_t)z * p.num_layers + m];
            wsum += w * w;
        }
        s.ok = wsum > 0.0;
        if (s.ok)
            for (int z = 0; z < Z; ++z) {
                const double w = (double)norms[(int64_t)z * p.num_layers + m];
                s.lambda[z] = (w * w) / wsum;
            }
    }
    __syncthreads();
    if (!s.ok) return;

    for (int i = tid; i <= kBins; i += kFitThreads) s.e[i] = bin_edge(i);
    for (int i = tid; i < kBins; i += kFitThreads) {
        double acc = 0.0;
        for (int z = 0; z < Z; ++z)
            acc += s.lambda[z] * (double)hist[((int64_t)z * p.num_layers + m) * LQ_HIST_STRIDE + i];
        s.mass[i] = acc / (double)L.size;
    }
    __syncthreads();
    }
    if (tid == 0) {
        s.F[0] = 0.0; s.M1[0] = 0.0; s.M2[0] = 0.0;
        for (int i = 0; i < kBins; ++i) {
            s.F[i + 1] = s.F[i] + s.mass[i];
            s.M1[i + 1] = s.M1[i] + s.mass[i] * ((s.e[i] + s.e[i + 1]) * 0.5);
            s.M2[i + 1] = s.M2[i] + s.mass[i] * ((s.e[i] * s.e[i] + s.e[i] * s.e[i + 1] + s.e[i + 1] * s.e[i + 1]) / 3.0);
        }
        s.ok = (s.F[kBins] - s.mass[0]) > 0.0;
    }
    __syncthreads();
    if (!s.ok) return;

    const double above = s.F[kBins] - s.mass[0];
    for (int j = tid; j < n; j += kFitThreads) {
        const double frac = (double)j / (double)(n - 1);
        if (j == 0) s.l[j] = s.lb[j] = 0.0;
        else if (j == n - 1) s.l[j] = s.lb[j] = 1.0;
        else {
            s.l[j] = cdf_inv(s, s.mass[0] + above * frac);
            s.lb[j] = frac;
        }
    }
    __syncthreads();

    descend(s, s.l, n, tid);
    descend(s, s.lb, n, tid);
    objective(s, s.l, n, tid, &s.obj[0]);
    objective(s, s.lb, n, tid, &s.obj[1]);
    if (s.obj[1] < s.obj[0] * (1.0 - 1e-9))
        for (int j = 1 + tid; j <= n - 2; j += kFitThreads) s.l[j] = s.lb[j];
    __syncthreads();

    // round to fp32; force strict monotonicity (one ulp and 2^-40 above the level before, one ulp
    // below the level after; serial: order matters)
    if (tid == 0) {
        float* out = levels_stage + (int64_t)m * kLevelStride;
        out[0] = 0.0f; out[n - 1] = 1.0f;
        for (int j = 1; j <= n - 2; ++j) {
            const float f = (float)s.l[j];
            float fl = nextafterf(out[j - 1], 2.0f);
            const float gap = __fadd_rn(out[j - 1], 9.094947017729282e-13f);   // previous level + 2^-40
            if (gap > fl) fl = gap;
            out[j] = f > fl ? f : fl;
        }
        for (int j = n - 2; j >= 1; --j) {
            const float ce = nextafterf(out[j + 1], -1.0f);
            if (out[j] > ce) out[j] = ce;
        }
        for (int jm = m0 + 1; jm < m1; ++jm) {             // the other members of the type receive the same sequence
            float* dst = levels_stage + (int64_t)member_layer[jm] * kLevelStride;
            for (int j = 0; j < n; ++j) dst[j] = out[j];
        }
    }
}

cudaError_t launch_fit(const PlanDev& p, const uint32_t* hist, const float* norms, int num_samples,
                       float* levels_stage, cudaStream_t s)
{
    if (p.num_layers == 0) return cudaSuccess;
    fit_levels_kernel<<<(unsigned)p.num_layers, kFitThreads, 0, s>>>(p, hist, norms, num_samples, levels_stage,
                                                                     nullptr, nullptr);
    return cudaGetLastError();
}

cudaError_t launch_fit_shared(const PlanDev& p, const uint32_t* hist, const float* norms, int num_samples,
                              float* levels_stage, const int32_t* member_off, const int32_t* member_layer,
                              int num_types, cudaStream_t s)
{
    if (num_types == 0) return cudaSuccess;
    fit_levels_kernel<<<(unsigned)num_types, kFitThreads, 0, s>>>(p, hist, norms, num_samples, levels_stage,
                                                                  member_off, member_layer);
    return cudaGetLastError();
}

}  // namespace lq
