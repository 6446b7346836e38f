/*
 * CPU oracle for layer-wise stochastic quantization and the QODA update.
 *
 * TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, single-threaded statement
 * of what the method computes, written from the paper's equations.  It shares no code,
 * header, table or constant generator with the CUDA library and must never be linked
 * into, or called from, the product path.  Only the tests, the smoke check and the
 * benchmark's CPU-baseline leg may use it.
 *
 * Build: gcc -O2 -ffp-contract=off -fno-fast-math -shared -fPIC lq_oracle.c -lm
 * (no contraction, no fast-math: every fp32 operation below is one IEEE-rounded step).
 *
 * Parity status of each part against the paper:
 *   philox, norm, quantizer, pack, histogram, decode/aggregate, QODA update: pinned by
 *     the CPU tests (known-answer vectors, closed forms, brute force, invariants).
 *   level fit (orc_fit_levels): the paper states the objective (Section 3.2, the
 *     variance minimisation after Eq. MQV and the CDF weights) but no solver, so the
 *     solver here is this implementation's own: "parity unpinned" against the paper; it is
 *     pinned only through properties of the objective (descent, stationarity, the
 *     uniform-density closed form, brute-force search on small cases).
 */
#include <math.h>
#include <stdint.h>
#include <stdlib.h>
#include <string.h>

/* ------------------------------------------------------------------------------------
 * Counter-based random numbers: Philox4x32 with 10 rounds (Salmon, Moraes, Dror, Shaw,
 * "Parallel random numbers: as easy as 1, 2, 3", SC'11).  The paper's quantizer needs one
 * independent uniform per coordinate (Section 3.1, definition of q_l(u)); keying the
 * stream on (seed, step, worker, layer, index) is this implementation's choice so that a CPU and a
 * GPU draw the same value for the same coordinate.
 * ---------------------------------------------------------------------------------- */
void orc_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4])
{
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * (uint64_t)c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * (uint64_t)c2;
        uint32_t n0 = (uint32_t)(p1 >> 32) ^ c1 ^ k0;
        uint32_t n1 = (uint32_t)p1;
        uint32_t n2 = (uint32_t)(p0 >> 32) ^ c3 ^ k1;
        uint32_t n3 = (uint32_t)p0;
        c0 = n0; c1 = n1; c2 = n2; c3 = n3;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

/* Uniform in [0,1) for coordinate `index` of (worker, layer) at iteration `step`:
 * key = (seed low, seed high), counter = (index / 4, layer, worker, step), the coordinate
 * takes output word index % 4, and rho = (word >> 9) * 2^-23: the top 23 bits of the word
 * on the grid of fp32 numbers in [0,1) with spacing 2^-23 (exact in fp32). */
float orc_uniform(uint64_t seed, uint32_t step, uint32_t worker, uint32_t layer, uint64_t index)
{
    uint32_t ctr[4] = { (uint32_t)(index >> 2), layer, worker, step };
    uint32_t key[2] = { (uint32_t)seed, (uint32_t)(seed >> 32) };
    uint32_t out[4];
    orc_philox4x32_10(ctr, key, out);
    return (float)(out[index & 3] >> 9) * 1.1920928955078125e-07f; /* 2^-23 */
}

/* ------------------------------------------------------------------------------------
 * L^q norm of one layer (Section 2.2: v is represented by (||v||_q, sign, u)).
 * q = 0 stands for the infinity norm.  Accumulated in fp64, returned rounded to fp32
 * (the message carries the norm as a 32-bit float, Section 3.2).
 * status: 0 ok, 1 zero norm (below the smallest normal float), 2 non-finite.
 * In both flagged cases the returned norm is 0 and the layer's message is all zero.
 * ---------------------------------------------------------------------------------- */
float orc_layer_norm(const float* v, int64_t d, int q, int* status)
{
    double acc = 0.0;
    int bad = 0;
    for (int64_t i = 0; i < d; ++i) {
        double a = fabs((double)v[i]);
        if (!(a <= 3.4028234663852886e38)) bad = 1;      /* NaN or infinity */
        if (q == 0)      { if (a > acc) acc = a; }
        else if (q == 1) acc += a;
        else if (q == 2) acc += a * a;
        else { double p = a; for (int r = 1; r < q; ++r) p *= a; acc += p; }
    }
    double n64;
    if (q == 0 || q == 1) n64 = acc;
    else if (q == 2)      n64 = sqrt(acc);
    else                  n64 = pow(acc, 1.0 / (double)q);
    float n = (float)n64;
    int st = 0;
    if (bad || !(n64 == n64) || isinf(n64) || isinf(n)) st = 2;
    else if (n < 1.17549435e-38f) st = 1;
    if (status) *status = st;
    return st ? 0.0f : n;
}

/* ------------------------------------------------------------------------------------
 * Stochastic quantization of one layer (Section 3.1).  For each coordinate:
 *   u   = min(|v| * (1/N), 1)                       normalised magnitude (Section 2.2)
 *   tau = the largest j <= n-2 with level[j] <= u   (so u = 1 falls in the last interval)
 *   up with probability xi(u) = (u - l_tau) / (l_{tau+1} - l_tau), decided as
 *        rho * (l_{tau+1} - l_tau) < (u - l_tau)     with rho the coordinate's uniform
 *   idx = tau + up,  sign = (v < 0), so both zeros carry sign 0.
 * `near` counts coordinates whose decision is within 1e-6 (relative to the interval)
 * of the threshold.  norm == 0 gives an all-zero message.
 * v points at coordinate `first_index` of the layer and d coordinates are processed, so
 * that a test can quantize a slice of a large layer.
 * ---------------------------------------------------------------------------------- */
void orc_quantize_layer(const float* v, int64_t d, int64_t first_index, float norm,
                        const float* level, int n,
                        uint64_t seed, uint32_t step, uint32_t worker, uint32_t layer,
                        uint8_t* idx, uint8_t* sign, int64_t* near)
{
    int64_t near_count = 0;
    if (!(norm > 0.0f)) {
        memset(idx, 0, (size_t)d); memset(sign, 0, (size_t)d);
        if (near) *near = 0;
        return;
    }
    const float r = 1.0f / norm;
    for (int64_t i = 0; i < d; ++i) {
        float a = fabsf(v[i]);
        float u = a * r;
        if (u > 1.0f) u = 1.0f;
        int tau = 0;
        for (int j = 1; j <= n - 2; ++j) if (level[j] <= u) tau = j;
        float num = u - level[tau];
        float den = level[tau + 1] - level[tau];
        float rho = orc_uniform(seed, step, worker, layer, (uint64_t)(first_index + i));
        float t = rho * den;
        int up = (t < num) ? 1 : 0;
        if (fabsf(t - num) <= 1e-6f * den) ++near_count;
        idx[i] = (uint8_t)(tau + up);
        sign[i] = (uint8_t)(v[i] < 0.0f ? 1 : 0);
    }
    if (near) *near = near_count;
}

/* ------------------------------------------------------------------------------------
 * Fixed-width message layout (Section 3.2: a 32-bit float norm, one sign bit and one
 * integer code per coordinate; Section 7.1 footnote: no entropy code on top).
 * The physical layout is this implementation's:
 *   every coordinate becomes one symbol of b+1 bits, symbol = 2 * idx + sign (sign in bit 0);
 *   a layer of d coordinates is cut into blocks of 1024 coordinates (the last one
 *   zero-padded); a block is (b+1) planes of 32 words; coordinate c of a block belongs to
 *   lane (c/4)%32 and has position p = 4*(c/128) + c%4 in that lane; the 32 symbols of a
 *   lane form one little-endian string of 32*(b+1) bits with symbol p at bit offset
 *   p*(b+1); bit t of that string is bit t%32 of word (t/32)*32 + lane of the block.
 * ---------------------------------------------------------------------------------- */
int64_t orc_packed_words(int64_t d, int b)
{
    return ((d + 1023) / 1024) * 32 * (int64_t)(b + 1);
}

static void locate(int64_t i, int b, int64_t* block_base, int* lane, int* p)
{
    int64_t blk = i / 1024;
    int c = (int)(i % 1024);
    *block_base = blk * 32 * (int64_t)(b + 1);
    *lane = (c / 4) % 32;
    *p = 4 * (c / 128) + c % 4;
}

void orc_pack_layer(const uint8_t* idx, const uint8_t* sign, int64_t d, int b, uint32_t* words)
{
    memset(words, 0, (size_t)orc_packed_words(d, b) * sizeof(uint32_t));
    for (int64_t i = 0; i < d; ++i) {
        int64_t base; int lane, p;
        locate(i, b, &base, &lane, &p);
        unsigned symbol = ((unsigned)idx[i] << 1) | (unsigned)(sign[i] ? 1 : 0);
        for (int bit = 0; bit <= b; ++bit) {
            if ((symbol >> bit) & 1u) {
                int t = p * (b + 1) + bit;           /* position in the lane's bit string */
                words[base + (int64_t)(t / 32) * 32 + lane] |= (uint32_t)1 << (t % 32);
            }
        }
    }
}

void orc_unpack_layer(const uint32_t* words, int64_t d, int b, uint8_t* idx, uint8_t* sign)
{
    for (int64_t i = 0; i < d; ++i) {
        int64_t base; int lane, p;
        locate(i, b, &base, &lane, &p);
        unsigned symbol = 0;
        for (int bit = 0; bit <= b; ++bit) {
            int t = p * (b + 1) + bit;
            symbol |= ((words[base + (int64_t)(t / 32) * 32 + lane] >> (t % 32)) & 1u) << bit;
        }
        idx[i] = (uint8_t)(symbol >> 1);
        sign[i] = (uint8_t)(symbol & 1u);
    }
}

/* ------------------------------------------------------------------------------------
 * Histogram of normalised magnitudes of one layer (Algorithm 1, line 4: estimate the
 * distribution of normalised dual vectors).  The binning is this implementation's: 386 bins,
 * bin 0 = [0, 2^-24), then 16 bins per octave with edges 2^e * (1 + m/16) up to 1,
 * and the last bin holds u = 1 only.  The bin is found here by comparing against the
 * edges, one by one.
 * ---------------------------------------------------------------------------------- */
#define ORC_NUM_BINS 386

double orc_bin_edge(int i)      /* lower edge of bin i, i = 0..386 (edge 385 = 1) */
{
    if (i <= 0) return 0.0;
    if (i > 385) return 1.0 + 1.0 / 16.0;
    int o = (i - 1) / 16, m = (i - 1) % 16;
    return ldexp(1.0 + (double)m / 16.0, -24 + o);
}

void orc_histogram_layer(const float* v, int64_t d, float norm, uint32_t* hist)
{
    if (!(norm > 0.0f)) return;
    double edge[ORC_NUM_BINS + 1];
    for (int i = 0; i <= ORC_NUM_BINS; ++i) edge[i] = orc_bin_edge(i);
    const float r = 1.0f / norm;
    for (int64_t i = 0; i < d; ++i) {
        float u = fabsf(v[i]) * r;
        if (u > 1.0f) u = 1.0f;
        int bin = 0;
        while (bin < ORC_NUM_BINS - 1 && (double)u >= edge[bin + 1]) ++bin;
        hist[bin] += 1u;
    }
}

/* ------------------------------------------------------------------------------------
 * Level fit (Section 3.2: minimise sum_j int_{l_j}^{l_{j+1}} sigma_Q^2(u; l) dF~(u), with
 * F~ the sum of the Z sampled vectors' CDFs weighted by lambda_z = N_z^2 / sum N_z^2).
 * The paper names no solver; this one is this implementation's own ("parity unpinned"):
 *   F~ is taken piecewise linear from the merged histogram (uniform density in a bin);
 *   the mass at u = 1 (last bin) never contributes variance and is left out;
 *   two starts, each followed by the sweeps below: (A) quantiles j/(n-1) of the mass above bin 0,
 *     (B) the uniform grid j/(n-1).  Coordinate descent stops at a local minimum and the objective
 *     has several when the density is not log-concave; the result is the start whose end point has
 *     the smaller objective, B only if it is smaller by more than one part in 10^9;
 *   sweeps: exact coordinate minimisation of one interior level given its neighbours
 *     a < c, i.e. F~(l) = F~(c) - int_a^c (u-a)/(c-a) dF~(u)  (the first-order condition
 *     int_a^l (u-a) dF~ = int_l^c (c-u) dF~), odd levels first, then even levels;
 *   up to 100 sweeps, stopping when no level moved by more than 1e-13 relative;
 *   round to fp32 and force strict monotonicity: each level at least one ulp and at least
 *   2^-40 above the one before, and at least one ulp below the one after.
 * Returns 1 if levels were written, 0 if there was no usable mass (levels untouched).
 * hist is [Z][stride] counts, norms are the Z vectors' fp32 norms, d the layer size.
 * ---------------------------------------------------------------------------------- */
typedef struct {
    double e[ORC_NUM_BINS + 1];       /* bin edges, e[385] = 1 */
    double mass[ORC_NUM_BINS];        /* weighted mass of bins 0..384 (bin 385 unused) */
    double F[ORC_NUM_BINS + 1];       /* cumulative mass at the edges */
    double M1[ORC_NUM_BINS + 1];      /* cumulative first moment at the edges */
    double M2[ORC_NUM_BINS + 1];      /* cumulative second moment at the edges */
} orc_density;

static int find_bin(const orc_density* D, double x)
{
    int lo = 0, hi = 384;             /* largest i in [0,384] with e[i] <= x */
    while (lo < hi) {
        int mid = (lo + hi + 1) / 2;
        if (D->e[mid] <= x) lo = mid; else hi = mid - 1;
    }
    return lo;
}

static double cdf_at(const orc_density* D, double x, double* first_moment)
{
    int i = find_bin(D, x);
    double theta = (x - D->e[i]) / (D->e[i + 1] - D->e[i]);
    if (theta > 1.0) theta = 1.0;
    double part = D->mass[i] * theta;
    if (first_moment) *first_moment = D->M1[i] + part * ((D->e[i] + x) * 0.5);
    return D->F[i] + part;
}

static double cdf_inverse(const orc_density* D, double y)
{
    int lo = 0, hi = 385;             /* smallest i in [0,385] with F[i+1] > y; 385 = none */
    while (lo < hi) {
        int mid = (lo + hi) / 2;
        if (D->F[mid + 1] > y) hi = mid; else lo = mid + 1;
    }
    if (lo >= 385) return 1.0;
    double t = (y - D->F[lo]) / D->mass[lo];
    if (t < 0.0) t = 0.0;
    return D->e[lo] + t * (D->e[lo + 1] - D->e[lo]);
}

/* int_0^x u^2 dF~(u): inside a bin of density m/(e1-e0), int_{e0}^{x} u^2 = part * (e0^2 + e0 x + x^2) / 3 */
static double second_moment_at(const orc_density* D, double x)
{
    int i = find_bin(D, x);
    double theta = (x - D->e[i]) / (D->e[i + 1] - D->e[i]);
    if (theta > 1.0) theta = 1.0;
    double part = D->mass[i] * theta;
    return D->M2[i] + part * ((D->e[i] * D->e[i] + D->e[i] * x + x * x) / 3.0);
}

/* sum_j int_{l_j}^{l_{j+1}} (l_{j+1} - u)(u - l_j) dF~(u) from the cumulative moments:
 * each interval gives -(M2(c) - M2(a)) + (a + c)(M1(c) - M1(a)) - a c (F(c) - F(a)). */
static double density_objective(const orc_density* D, const double* l, int n)
{
    double total = 0.0;
    for (int j = 0; j + 1 < n; ++j) {
        double a = l[j], c = l[j + 1], m1a, m1c;
        double Fa = cdf_at(D, a, &m1a), Fc = cdf_at(D, c, &m1c);
        double m2a = second_moment_at(D, a), m2c = second_moment_at(D, c);
        total += ((a + c) * (m1c - m1a) - (m2c - m2a)) - (a * c) * (Fc - Fa);
    }
    return total;
}

static orc_density D;                 /* single-threaded oracle: static storage is fine */
static int solve_levels(int n, float* level_out);

int orc_fit_levels(const uint32_t* hist, int64_t stride, const float* norms, int Z,
                   int64_t d, int n, float* level_out)
{
    if (n < 3 || d <= 0) return 0;
    double wsum = 0.0;
    for (int z = 0; z < Z; ++z) wsum += (double)norms[z] * (double)norms[z];
    if (!(wsum > 0.0)) return 0;
    for (int i = 0; i <= 385; ++i) D.e[i] = orc_bin_edge(i);
    for (int i = 0; i < 385; ++i) {
        double m = 0.0;
        for (int z = 0; z < Z; ++z) {
            double lambda = ((double)norms[z] * (double)norms[z]) / wsum;
            m += lambda * (double)hist[(int64_t)z * stride + i];
        }
        D.mass[i] = m / (double)d;
    }
    return solve_levels(n, level_out);
}

/* One level sequence for a whole type (Section 3.1: coordinates are split into M types, each with
 * its own sequence; here a type is a set of layers).  The S histograms are those of all (sampled
 * vector, member layer) pairs of the type, sizes[s] and norms[s] the layer size and norm of each.  The
 * variance the fit minimises is sum_s N_s^2 sum_{i in s} sigma_Q^2(u_i), so the merged measure weighs
 * every histogram's counts by N_s^2 (with one member layer this is the CDF weighting of orc_fit_levels);
 * it is scaled by sum_s N_s^2 d_s to total mass one. */
int orc_fit_levels_shared(const uint32_t* hist, int64_t stride, const float* norms, const int64_t* sizes,
                          int S, int n, float* level_out)
{
    if (n < 3) return 0;
    double wd = 0.0;
    for (int s = 0; s < S; ++s) wd += (double)norms[s] * (double)norms[s] * (double)sizes[s];
    if (!(wd > 0.0)) return 0;
    for (int i = 0; i <= 385; ++i) D.e[i] = orc_bin_edge(i);
    for (int i = 0; i < 385; ++i) {
        double m = 0.0;
        for (int s = 0; s < S; ++s)
            m += ((double)norms[s] * (double)norms[s]) * (double)hist[(int64_t)s * stride + i];
        D.mass[i] = m / wd;
    }
    return solve_levels(n, level_out);
}

/* Odd/even sweeps of exact coordinate minimisation from the levels in l. */
static void descend(double* l, int n)
{
    for (int sweep = 0; sweep < 100; ++sweep) {
        double moved = 0.0;
        for (int parity = 1; parity >= 0; --parity) {
            for (int j = 1; j <= n - 2; ++j) {
                if ((j & 1) != parity) continue;
                double a = l[j - 1], c = l[j + 1], b;
                if (!(c > a)) continue;
                double m1a, m1c;
                double Fa = cdf_at(&D, a, &m1a), Fc = cdf_at(&D, c, &m1c);
                double mass_ac = Fc - Fa;
                if (!(mass_ac > 0.0)) b = (a + c) * 0.5;
                else {
                    double target = Fc - ((m1c - m1a) - a * mass_ac) / (c - a);
                    b = cdf_inverse(&D, target);
                    if (b < a) b = a;
                    if (b > c) b = c;
                }
                double rel = fabs(b - l[j]) / (fabs(b) > 1e-300 ? fabs(b) : 1e-300);
                if (rel > moved) moved = rel;
                l[j] = b;
            }
        }
        if (moved <= 1e-13) break;
    }
}

/* The solver proper, on the density left in D. */
static int solve_levels(int n, float* level_out)
{
    D.F[0] = 0.0; D.M1[0] = 0.0; D.M2[0] = 0.0;
    for (int i = 0; i < 385; ++i) {
        D.F[i + 1] = D.F[i] + D.mass[i];
        D.M1[i + 1] = D.M1[i] + D.mass[i] * ((D.e[i] + D.e[i + 1]) * 0.5);
        D.M2[i + 1] = D.M2[i] + D.mass[i] * ((D.e[i] * D.e[i] + D.e[i] * D.e[i + 1] + D.e[i + 1] * D.e[i + 1]) / 3.0);
    }
    double total = D.F[385], above = total - D.mass[0];
    if (!(above > 0.0)) return 0;

    double l[256], lb[256];
    l[0] = 0.0; l[n - 1] = 1.0;
    lb[0] = 0.0; lb[n - 1] = 1.0;
    for (int j = 1; j <= n - 2; ++j) {
        l[j] = cdf_inverse(&D, D.mass[0] + above * ((double)j / (double)(n - 1)));
        lb[j] = (double)j / (double)(n - 1);
    }
    descend(l, n);
    descend(lb, n);
    double obj_a = density_objective(&D, l, n), obj_b = density_objective(&D, lb, n);
    if (obj_b < obj_a * (1.0 - 1e-9))
        for (int j = 1; j <= n - 2; ++j) l[j] = lb[j];

    level_out[0] = 0.0f; level_out[n - 1] = 1.0f;
    for (int j = 1; j <= n - 2; ++j) {
        float f = (float)l[j];
        float floor_ = nextafterf(level_out[j - 1], 2.0f);
        float gap_ = level_out[j - 1] + 9.094947017729282e-13f;     /* previous level + 2^-40 */
        if (gap_ > floor_) floor_ = gap_;
        level_out[j] = f > floor_ ? f : floor_;
    }
    for (int j = n - 2; j >= 1; --j) {
        float ceil_ = nextafterf(level_out[j + 1], -1.0f);
        if (level_out[j] > ceil_) level_out[j] = ceil_;
    }
    return 1;
}

/* Objective of the fit evaluated from the same piecewise-uniform density (used by the
 * tests to check descent against levels that did not come from the solver). */
double orc_fit_objective(const uint32_t* hist, int64_t stride, const float* norms, int Z,
                         int64_t d, const float* level, int n)
{
    double wsum = 0.0, total = 0.0;
    for (int z = 0; z < Z; ++z) wsum += (double)norms[z] * (double)norms[z];
    if (!(wsum > 0.0)) return 0.0;
    for (int i = 0; i < 385; ++i) {
        double m = 0.0;
        for (int z = 0; z < Z; ++z)
            m += (((double)norms[z] * (double)norms[z]) / wsum) * (double)hist[(int64_t)z * stride + i];
        m /= (double)d;
        if (m == 0.0) continue;
        double lo = orc_bin_edge(i), hi = orc_bin_edge(i + 1), dens = m / (hi - lo);
        /* cut the bin at every level that falls inside it and integrate
         * (l_{j+1} - u)(u - l_j) exactly on each piece */
        double x0 = lo;
        while (x0 < hi) {
            int j = 0;
            for (int t = 1; t <= n - 2; ++t) if ((double)level[t] <= x0) j = t;
            double a = level[j], c = level[j + 1];
            double x1 = c < hi ? c : hi;
            if (!(x1 > x0)) break;
            /* int (c-u)(u-a) du = [-(u^3)/3 + (a+c)u^2/2 - a c u] */
            double P0 = -x0 * x0 * x0 / 3.0 + (a + c) * x0 * x0 * 0.5 - a * c * x0;
            double P1 = -x1 * x1 * x1 / 3.0 + (a + c) * x1 * x1 * 0.5 - a * c * x1;
            total += dens * (P1 - P0);
            x0 = x1;
        }
    }
    return total;
}

/* ------------------------------------------------------------------------------------
 * DECODE of one layer (Section 3.2; Algorithm 1 line 15): V^_i = N * sign_i * l_{idx_i},
 * evaluated as one fp32 multiply N * l_idx with the sign applied afterwards.
 * ---------------------------------------------------------------------------------- */
void orc_decode_layer(const uint8_t* idx, const uint8_t* sign, int64_t d, float norm,
                      const float* level, float* out)
{
    for (int64_t i = 0; i < d; ++i) {
        float mag = norm * level[idx[i]];
        out[i] = sign[i] ? -mag : mag;
    }
}

/* Mean of K decoded vectors, accumulated in fp32 in worker order, then scaled by the
 * fp32 reciprocal of K (Algorithm 1 lines 10 and 17: sum_k V^_k / K).
 * decoded is [K][d]. */
void orc_aggregate(const float* decoded, int K, int64_t d, float* gbar)
{
    const float invK = 1.0f / (float)K;
    for (int64_t i = 0; i < d; ++i) {
        float acc = 0.0f;
        for (int k = 0; k < K; ++k) acc = acc + decoded[(int64_t)k * d + i];
        gbar[i] = acc * invK;
    }
}

/* One worker-layer term of the adaptive step size (Eq. general_stepsize:
 * ||V^_{k,s+1/2} - V^_{k,s-1/2}||^2).  The decoded vectors are fp32, and their difference is
 * formed in that precision (one fp32 subtraction per coordinate); the squares of those fp32
 * differences, exact in fp64, are summed in fp64. */
double orc_sq_diff(const float* cur, const float* prev, int64_t d)
{
    double acc = 0.0;
    for (int64_t i = 0; i < d; ++i) {
        float t = cur[i] - (prev ? prev[i] : 0.0f);
        acc += (double)t * (double)t;
    }
    return acc;
}

/* eta_{t+1} = gamma_{t+1} = (1 + S_t)^(-1/2), S_t = S_{t-1} + sum_k ||.||^2 / K^2
 * (Eq. general_stepsize).  Returns the new S; *eta receives the fp32 step size. */
double orc_step_size(double S_prev, double sum_sq_diff, int K, float* eta)
{
    double S = S_prev + sum_sq_diff / ((double)K * (double)K);
    *eta = (float)(1.0 / sqrt(1.0 + S));
    return S;
}

/* Optimistic dual averaging update (Eq. ODA; Algorithm 1 lines 17, 18 and, for the next
 * iteration, line 10), each written as one fp32 operation:
 *   Y_{t+1}   = Y_t - gbar
 *   X_{t+1}   = fma(eta, Y_{t+1}, X_1)
 *   X_{t+3/2} = fma(-eta, gbar, X_{t+1})        (gamma_{t+1} = eta_{t+1})
 * X may be NULL. */
void orc_qoda_update(const float* gbar, const float* X1, float* Y, float* Xhalf, float* X,
                     float eta, int64_t d)
{
    for (int64_t i = 0; i < d; ++i) {
        float y = Y[i] - gbar[i];
        float x = fmaf(eta, y, X1[i]);
        Y[i] = y;
        if (X) X[i] = x;
        Xhalf[i] = fmaf(-eta, gbar[i], x);
    }
}

/* ------------------------------------------------------------------------------------
 * Alternative adaptive step sizes (Eq. Alt; appendix "Analysis in Almost Sure Boundedness
 * Model"):  eta_t = (1 + lambda_{t-2} + mu_{t-2})^(-1/2),  gamma_t = (1 + lambda_{t-2})^(qhat - 1/2),
 * qhat in (0, 1/4], with the running sums (zero for t <= 0)
 *   lambda_t = sum_{s<=t} || (1/K) sum_k V^_{k,s+1/2} ||^2      (the appendix's form: the squared
 *              norm of the aggregate; the main text prints the sum of the workers' squared norms
 *              over K^2 instead)
 *   mu_t     = sum_{s<=t} || X_s - X_{s+1} ||^2.
 * Both norms are taken on fp32 vectors: lambda on the mean gbar the update itself uses, mu on the
 * fp32 difference of the two iterates; the squares, exact in fp64, are summed in fp64.
 * ---------------------------------------------------------------------------------- */
void orc_alt_rates(double lambda, double mu, double qhat, float* eta, float* gamma)
{
    *eta = (float)(1.0 / sqrt(1.0 + lambda + mu));
    *gamma = (float)pow(1.0 + lambda, qhat - 0.5);
}

double orc_sq_norm(const float* g, int64_t d)
{
    double acc = 0.0;
    for (int64_t i = 0; i < d; ++i) acc += (double)g[i] * (double)g[i];
    return acc;
}

/* The optimistic dual averaging update with separate rates (Eq. ODA):
 *   Y_{t+1} = Y_t - gbar,  X_{t+1} = fma(eta, Y_{t+1}, X_1),  X_{t+3/2} = fma(-gamma, gbar, X_{t+1}). */
void orc_qoda_update_rates(const float* gbar, const float* X1, float* Y, float* Xhalf, float* X,
                           float eta, float gamma, int64_t d)
{
    for (int64_t i = 0; i < d; ++i) {
        float y = Y[i] - gbar[i];
        float x = fmaf(eta, y, X1[i]);
        Y[i] = y;
        if (X) X[i] = x;
        Xhalf[i] = fmaf(-gamma, gbar[i], x);
    }
}

/* ------------------------------------------------------------------------------------
 * Code-length accounting (Appendix "Coding Framework").  With F~ the weighted CDF of the
 * layer's normalised coordinates (taken, as in the fit, piecewise linear from the merged
 * histogram, plus the point mass at u = 1 of the last bin), the probability that level j is
 * emitted is  p^_j = int hat_j(u) dF~(u),  hat_j rising linearly from l_{j-1} to l_j and falling
 * linearly from l_j to l_{j+1} (one-sided at j = 0 and j = n-1): stochastic rounding sends u to
 * l_tau with probability (l_{tau+1}-u)/(l_{tau+1}-l_tau) and to l_{tau+1} otherwise.
 * p_out[0..n-1] receives the probabilities (they add up to the total mass, 1).
 * ---------------------------------------------------------------------------------- */
int orc_level_probabilities(const uint32_t* hist, int64_t stride, const float* norms, int Z,
                            int64_t d, const float* level, int n, double* p_out)
{
    for (int j = 0; j < n; ++j) p_out[j] = 0.0;
    if (n < 2 || d <= 0) return 0;
    double wsum = 0.0;
    for (int z = 0; z < Z; ++z) wsum += (double)norms[z] * (double)norms[z];
    if (!(wsum > 0.0)) return 0;
    for (int i = 0; i < ORC_NUM_BINS; ++i) {
        double m = 0.0;
        for (int z = 0; z < Z; ++z)
            m += (((double)norms[z] * (double)norms[z]) / wsum) * (double)hist[(int64_t)z * stride + i];
        m /= (double)d;
        if (m == 0.0) continue;
        if (i == ORC_NUM_BINS - 1) { p_out[n - 1] += m; continue; }      /* the point mass at u = 1 */
        double lo = orc_bin_edge(i), hi = orc_bin_edge(i + 1), dens = m / (hi - lo);
        double x0 = lo;
        while (x0 < hi) {                  /* cut the bin at the levels inside it */
            int j = 0;
            for (int t = 1; t <= n - 2; ++t) if ((double)level[t] <= x0) j = t;
            double a = level[j], c = level[j + 1];
            double x1 = c < hi ? c : hi;
            if (!(x1 > x0)) break;
            /* on [x0, x1] inside [a, c]: int (c-u)/(c-a) du goes to level j, int (u-a)/(c-a) du to level j+1 */
            double len = x1 - x0, mid = 0.5 * (x0 + x1);
            p_out[j]     += dens * len * (c - mid) / (c - a);
            p_out[j + 1] += dens * len * (mid - a) / (c - a);
            x0 = x1;
        }
    }
    return 1;
}

/* Expected message length of one layer in bits as the appendix writes it:
 *   C_q + (1 - p^_0) d + (H + 1) d,   C_q = 32,   H = - sum_{j=1}^{alpha} p^_j log2 p^_j
 * (the sum over the interior levels j = 1 .. n-2, as printed).  *nonzeros receives the expected
 * number of non-zero coordinates (1 - p^_0) d. */
double orc_expected_code_length(const double* p, int n, int64_t d, double* nonzeros)
{
    double H = 0.0;
    for (int j = 1; j <= n - 2; ++j) if (p[j] > 0.0) H -= p[j] * log2(p[j]);
    double nz = (1.0 - p[0]) * (double)d;
    if (nonzeros) *nonzeros = nz;
    return 32.0 + nz + (H + 1.0) * (double)d;
}

/* ------------------------------------------------------------------------------------
 * Lossless prefix code on the level symbols (appendix, "Further Details on Coding Framework":
 * with the symbol frequencies known or estimated, classical Huffman coding).
 *
 * orc_huffman_lengths: code lengths of a Huffman code for n <= 256 symbols with weights w
 * (probabilities or counts).  Every symbol receives a code word, also those of weight zero (an
 * estimated distribution may miss a symbol that then occurs): weights below floor = total * 2^-40
 * are raised to it.  Plain Huffman: repeatedly merge the two lightest trees (ties: the tree whose
 * smallest symbol index is lower comes first); a symbol's length is its depth.  If the longest
 * word exceeds max_len the floor is doubled and the construction repeated (with all weights equal
 * the depth is ceil(log2 n) <= 8, so this ends).  n = 1 gives length 1.
 * ---------------------------------------------------------------------------------- */
int orc_huffman_lengths(const double* w, int n, int max_len, uint8_t* len)
{
    if (n < 1 || n > 256 || max_len < 8 || max_len > 32) return 0;
    if (n == 1) { len[0] = 1; return 1; }
    double total = 0.0;
    for (int i = 0; i < n; ++i) { if (!(w[i] >= 0.0)) return 0; total += w[i]; }
    if (!(total > 0.0)) total = 1.0;
    double floor_w = total * 9.094947017729282e-13;      /* 2^-40 of the total */
    for (;;) {
        double wt[511]; int parent[511]; int lowest[511]; int alive[511];
        int nodes = n;
        for (int i = 0; i < n; ++i) { wt[i] = w[i] > floor_w ? w[i] : floor_w; parent[i] = -1; lowest[i] = i; alive[i] = 1; }
        for (int merges = 0; merges < n - 1; ++merges) {
            int a = -1, b = -1;                           /* the two lightest live trees, a before b */
            for (int i = 0; i < nodes; ++i) {
                if (!alive[i]) continue;
                if (a < 0 || wt[i] < wt[a] || (wt[i] == wt[a] && lowest[i] < lowest[a])) { b = a; a = i; }
                else if (b < 0 || wt[i] < wt[b] || (wt[i] == wt[b] && lowest[i] < lowest[b])) b = i;
            }
            wt[nodes] = wt[a] + wt[b]; parent[nodes] = -1; alive[nodes] = 1;
            lowest[nodes] = lowest[a] < lowest[b] ? lowest[a] : lowest[b];
            parent[a] = nodes; parent[b] = nodes; alive[a] = 0; alive[b] = 0;
            ++nodes;
        }
        int longest = 0;
        for (int i = 0; i < n; ++i) {
            int d = 0;
            for (int v = i; parent[v] >= 0; v = parent[v]) ++d;
            len[i] = (uint8_t)d;
            if (d > longest) longest = d;
        }
        if (longest <= max_len) return 1;
        floor_w *= 2.0;
    }
}

/* Canonical code words from the lengths: symbols ordered by (length, index); the first word is all
 * zeros, each next word is the previous plus one, shifted left when the length grows.  Words are
 * written most significant bit first. */
void orc_canonical_codes(const uint8_t* len, int n, uint32_t* code)
{
    uint32_t next = 0; int prev_len = 0;
    for (int l = 1; l <= 32; ++l)
        for (int i = 0; i < n; ++i)
            if (len[i] == l) {
                next <<= (l - prev_len);
                code[i] = next;
                next += 1; prev_len = l;
            }
}

/* Entropy-coded form of one block of up to 1024 coordinates (the blocks of the fixed-width layout).
 * Stream order: s = 32 * lane + p for lane = 0..31, p = 0..31, which is coordinate
 * c = 128 * (p / 4) + 4 * lane + p % 4 of the block; coordinates c >= count are left out.  Each
 * coordinate contributes its level's code word, most significant bit first, then, when the level
 * index is not 0, one sign bit (appendix: one bit for the sign of each non-zero entry).  Stream bit t
 * is bit t % 32 of word t / 32.  Returns the number of bits; words must hold 1024 * 33 / 32 entries. */
static void put_bit(uint32_t* words, int64_t t, unsigned bit)
{
    if (bit) words[t / 32] |= (uint32_t)1 << (t % 32);
}

int64_t orc_entropy_encode_block(const uint8_t* idx, const uint8_t* sign, int count,
                                 const uint8_t* len, const uint32_t* code, uint32_t* words)
{
    int64_t t = 0;
    memset(words, 0, sizeof(uint32_t) * 1056);
    for (int s = 0; s < 1024; ++s) {
        int lane = s / 32, p = s % 32;
        int c = 128 * (p / 4) + 4 * lane + p % 4;
        if (c >= count) continue;
        int l = len[idx[c]];
        for (int j = l - 1; j >= 0; --j) put_bit(words, t++, (code[idx[c]] >> j) & 1u);
        if (idx[c] != 0) put_bit(words, t++, sign[c] ? 1u : 0u);
    }
    return t;
}

/* Inverse of the above, reading bit by bit: a word of length l is recognised when the bits read so
 * far equal the code of a symbol of that length.  Returns the number of bits consumed, or -1 when the
 * stream holds no valid word. */
int64_t orc_entropy_decode_block(const uint32_t* words, int count, const uint8_t* len, const uint32_t* code,
                                 int n, uint8_t* idx, uint8_t* sign)
{
    int64_t t = 0;
    for (int s = 0; s < 1024; ++s) {
        int lane = s / 32, p = s % 32;
        int c = 128 * (p / 4) + 4 * lane + p % 4;
        if (c >= count) continue;
        uint32_t acc = 0; int l = 0, found = -1;
        while (found < 0) {
            if (l >= 32) return -1;
            acc = (acc << 1) | ((words[t / 32] >> (t % 32)) & 1u); ++t; ++l;
            for (int i = 0; i < n; ++i) if (len[i] == l && code[i] == acc) { found = i; break; }
        }
        idx[c] = (uint8_t)found;
        sign[c] = 0;
        if (found != 0) { sign[c] = (uint8_t)((words[t / 32] >> (t % 32)) & 1u); ++t; }
    }
    return t;
}

/* ------------------------------------------------------------------------------------
 * Elias' recursive ("omega") code of a positive integer (Elias 1975, cited by the appendix on
 * the coding framework for the case where only "smaller values are more frequent" is known).
 * Definition, written out: start from the single bit 0; while value > 1, put the binary
 * representation of value in front and continue with value = (number of bits just written) - 1.
 * bits_out receives the word as '0'/'1' characters (at most 63 + terminator); returns its length.
 * orc_elias_omega_decode reads one word from a '0'/'1' string and returns the value (0 on a
 * malformed word); *used receives the number of characters consumed.
 * ---------------------------------------------------------------------------------- */
int orc_elias_omega(uint64_t value, char* bits_out)
{
    char word[160];
    int end = 159, start = 159;
    word[end] = '\0';
    word[--start] = '0';
    if (value == 0) { bits_out[0] = '\0'; return 0; }
    while (value > 1) {
        int nb = 0;
        for (uint64_t t = value; t; t >>= 1) ++nb;
        for (int i = 0; i < nb; ++i) word[--start] = (char)('0' + (int)((value >> i) & 1u));   /* least significant bit last */
        value = (uint64_t)(nb - 1);
    }
    const int len = end - start;
    memcpy(bits_out, word + start, (size_t)len + 1);
    return len;
}

uint64_t orc_elias_omega_decode(const char* bits, int* used)
{
    uint64_t n = 1;
    int pos = 0;
    for (;;) {
        if (bits[pos] == '0') { ++pos; break; }
        if (bits[pos] != '1') { if (used) *used = pos; return 0; }
        uint64_t v = 0;
        for (uint64_t i = 0; i <= n; ++i) {
            const char ch = bits[pos++];
            if (ch != '0' && ch != '1') { if (used) *used = pos; return 0; }
            v = (v << 1) | (uint64_t)(ch - '0');
        }
        n = v;
    }
    if (used) *used = pos;
    return n;
}
