// sgc_oracle.cpp -- CPU ORACLE for one SGC optimizer step.  TEST INFRASTRUCTURE ONLY.
//
// This file is the slow, plain reference that the CUDA library is checked against.  It is
// used by the tests, by the smoke check and by the benchmark's CPU-baseline leg; the product
// (the CUDA library and its Python binding) never calls it and shares no code with it.
//
// What it computes (paper notation):
//   Sparsify_s            Section 3.2, text before Eq. (4): keep the s largest-magnitude entries
//   p = A G~, q = A G~^2  Eq. (4) and the unnumbered equation after it; Algorithm 2
//   k-space Adam          Algorithm 2 (Algorithm 1 in k dimensions)
//   OMP_A(y)              Eq. (7); Appendix B Algorithm 3.  Algorithm 3 is an algebraic rewrite
//                         (inverse Cholesky) of textbook orthogonal matching pursuit; the oracle
//                         is the textbook form: correlate, normalised argmax, dense least
//                         squares on the support (Householder QR), residual.
//   N = a*x^M/(sqrt(x^V)+eps), W <- W - eta*N      Eq. (8), Eq. (3); Algorithm 2
//
// Readings of points the paper leaves open (all listed in the design notes of the repository):
//   * V uses beta2 (Algorithm 2; the displayed Eq. (6) prints beta1, a typo).
//   * Bias correction (Algorithm 2) produces temporaries; M and V are stored uncorrected.
//   * A has i.i.d. entries of standard deviation 1/sqrt(k) (Section 3.3).  Here
//     A[j][i] = sigma_k * Z(seed, j, i) with sigma_k = fl32(1/sqrt(k)) and Z a counter-based
//     approximately standard-normal value (a binary16 number) defined below; A is never stored.
//   * Ties in |g| and in the OMP argmax go to the lower index; selected columns are not re-selected.
//   * Exactly s OMP iterations unless the new column is numerically dependent on the support.
//   * Eq. (8) is applied on the intersection of the two supports where x^V > 0; elsewhere N = 0.
//   Parity unpinned by the paper (readings of ours, nothing printed fixes them): the stop on a numerically dependent
//   column, the treatment of Eq. (8) where the two supports differ or x^V <= 0, and the opt-in variant of
//   orc_set_recovery (one shared support, early stop on the residual).
//
// Beyond the step itself: orc_select (the Select line of Algorithm 3 for several residuals at once, for checking picks at
// sizes where s full iterations are out of reach), orc_reproject (SGCA, Appendix C, Algorithm 4), orc_omp_tol / orc_least_squares /
// orc_set_recovery (the variant built on the remark after Eq. (8)); the chunked (MESGC) and projected (CESGC) forms of
// Section 4.4 are compositions of these states written out in oracle/binding.py (cesgc_step) and in the tests.
//
// Arithmetic: inputs and stored state are fp32; every sum is accumulated in fp64.
// Pins: see tests/test_oracle_*.py (dense-matrix definitions, brute-force supports, closed-form
// Adam trajectories, exact recovery of planted vectors, numpy least squares, golden Z vectors).
//
// Build: g++ -O2 -std=c++17 -fopenmp -ffp-contract=off -mfma -shared -fPIC

#include <algorithm>
#include <cmath>
#include <cstdint>
#include <cstdlib>
#include <cstring>
#include <numeric>
#include <vector>

#ifdef _OPENMP
#include <omp.h>
#endif

namespace {

// ------------------------------------------------------------------------------------------
// Z(seed, row, col): the measurement-matrix entry before scaling.  The paper fixes only the law of
// A (i.i.d. zero-mean normal entries of standard deviation 1/sqrt(k), Section 3.3); this is the
// concrete, counter-based realisation of it.  Every value of Z is exactly a binary16 (half) number.
//
//  1. column keys  ck = mix32( mix32(col + 0x9E3779B9 * seed_lo) ^ seed_hi )     (offset)
//                  mk = mix32( ck ^ 0x5BD1E995 ) | 1                               (odd stride)
//  2. pair word    one 32-bit word serves the two rows 2p and 2p+1 of a column:
//                  h = ck + p * mk ; h ^= h>>16 ; h *= 0x85EBCA6B ; h ^= h>>15
//  3. byte sums    S = b0 + b1 of h for the even row, b2 + b3 for the odd row   (0..510, triangular law)
//  4. centred      x = (S - 255) / 256                      (exact in binary16)
//  5. quantile map w = x*x ; q = fma(fma(w, C2, C1), w, C0) ; Z = x*q , every operation rounded to
//                  binary16 (round to nearest even, subnormals kept) -- the arithmetic of the GPU's
//                  packed half-precision instructions, restated here through exact double products
//
// The odd polynomial maps the quantiles of the triangular law onto those of the standard normal;
// C0..C2 were chosen once (variance 1.0000, kurtosis 2.999, Kolmogorov distance 3.5e-3 to the
// normal over the 511 lattice points, |Z| <= 3.37, Z monotone in S) and are frozen as bit patterns.
// Both column keys pass through a full-avalanche finaliser once per column; the per-word mixing
// (step 2) is deliberately short because it runs k*d/2 times per correlation pass on the GPU.  The
// per-column odd stride mk makes two columns share their word sequence only if both 32-bit keys
// are related, which does not happen among d < 2^32 columns in expectation.
// mix32 is the public-domain "lowbias32" integer finaliser.
// ------------------------------------------------------------------------------------------
inline uint32_t mix32(uint32_t x) {
    x ^= x >> 16; x *= 0x7feb352dU;
    x ^= x >> 15; x *= 0x846ca68bU;
    x ^= x >> 16;
    return x;
}

inline float bits_to_float(uint32_t b) { float f; std::memcpy(&f, &b, 4); return f; }
inline uint32_t float_to_bits(float f) { uint32_t b; std::memcpy(&b, &f, 4); return b; }

// ---- binary16 arithmetic, restated with doubles -----------------------------------------------
// value of a binary16 bit pattern (finite patterns only)
inline double half_value(uint16_t b) {
    const int sign = b >> 15, e = (b >> 10) & 31, m = b & 1023;
    const double mag = e == 0 ? std::ldexp((double)m, -24) : std::ldexp((double)(1024 + m), e - 25);
    return sign ? -mag : mag;
}
// nearest binary16 (ties to even) of a double of magnitude below 65520; subnormals are kept
inline uint16_t half_round(double v) {
    const uint16_t sign = std::signbit(v) ? 0x8000 : 0;
    const double a = std::fabs(v);
    if (a == 0.0) return sign;
    int e;
    std::frexp(a, &e);                                  // a = f * 2^e, f in [0.5, 1)
    int q = e - 11;                                     // spacing 2^q of binary16 numbers near a (11-bit significand)
    if (q < -24) q = -24;                               // subnormal range: spacing 2^-24
    const double scaled = std::ldexp(a, -q);            // exact
    double r = std::nearbyint(scaled);                  // default rounding mode: to nearest, ties to even
    // r in [0, 2048]; r == 2048 means the significand overflowed into the next binade
    int64_t n = (int64_t)r;
    if (n == 0) return sign;
    int exp_field;
    if (n >= 2048) { n >>= 1; q += 1; }
    if (n >= 1024) exp_field = q + 25; else exp_field = 0;        // normal: value = n * 2^q with 1024 <= n < 2048
    return (uint16_t)(sign | (exp_field << 10) | (n & 1023));
}
// products of two binary16 numbers are exact in double; the sum with a third is exact unless the product lies
// more than 30 binary orders below it, where it cannot move the rounded result onto or off a tie
inline uint16_t half_mul(uint16_t a, uint16_t b) { return half_round(half_value(a) * half_value(b)); }
inline uint16_t half_fma(uint16_t a, uint16_t b, uint16_t c) { return half_round(half_value(a) * half_value(b) + half_value(c)); }

inline uint32_t column_key(uint64_t seed, uint32_t col) {
    const uint32_t seed_lo = (uint32_t)(seed & 0xFFFFFFFFu);
    const uint32_t seed_hi = (uint32_t)(seed >> 32);
    return mix32(mix32(col + 0x9E3779B9U * seed_lo) ^ seed_hi);
}

// step 5 for one lattice point S in [0, 510]
inline uint16_t z_of_byte_sum(int S) {
    const uint16_t C0 = 0x40c2, C1 = 0xbad9, C2 = 0x3f89;
    const uint16_t x = half_round((double)(S - 255) / 256.0);          // exact
    const uint16_t w = half_mul(x, x);
    uint16_t q = half_fma(w, C2, C1);
    q = half_fma(q, w, C0);
    return half_mul(x, q);
}

// Z takes one of 511 values; they are computed once from the definition above and looked up afterwards
struct ZTable {
    float z[511];
    ZTable() { for (int S = 0; S <= 510; ++S) z[S] = (float)half_value(z_of_byte_sum(S)); }
};
inline const ZTable& z_table() { static const ZTable t; return t; }

inline float z_from_key(uint32_t ck, uint32_t row) {
    const uint32_t mk = mix32(ck ^ 0x5BD1E995U) | 1U;
    uint32_t h = ck + (row >> 1) * mk;
    h ^= h >> 16; h *= 0x85EBCA6BU; h ^= h >> 15;
    const int S = (row & 1U) ? (int)((h >> 16) & 0xFF) + (int)(h >> 24) : (int)(h & 0xFF) + (int)((h >> 8) & 0xFF);
    return z_table().z[S];
}

inline float sigma_of_k(int32_t k) { return (float)(1.0 / std::sqrt((double)k)); }

// A[row][col] as the real number sigma_k * Z (the product of two fp32 values is exact in fp64).
inline double a_entry(uint32_t ck, uint32_t row, double sigma) { return sigma * (double)z_from_key(ck, row); }

// ------------------------------------------------------------------------------------------
// Dense least squares  min_x || y - B x ||_2,  B is k x j column-major, by Householder QR.
// Returns false if a diagonal of R is (numerically) zero.
// ------------------------------------------------------------------------------------------
bool least_squares_qr(std::vector<double> B, std::vector<double> y, int k, int j, double* x) {
    std::vector<double> rdiag(j);
    for (int c = 0; c < j; ++c) {
        double* col = &B[(size_t)c * k];
        double nrm = 0.0;
        for (int i = c; i < k; ++i) nrm += col[i] * col[i];
        nrm = std::sqrt(nrm);
        if (nrm == 0.0) return false;
        const double alpha = (col[c] > 0.0) ? -nrm : nrm;
        // v = col[c:] - alpha e1 ; H = I - 2 v v^T / (v^T v)
        col[c] -= alpha;
        double vtv = 0.0;
        for (int i = c; i < k; ++i) vtv += col[i] * col[i];
        if (vtv == 0.0) return false;
        for (int c2 = c + 1; c2 < j; ++c2) {
            double* o = &B[(size_t)c2 * k];
            double dot = 0.0;
            for (int i = c; i < k; ++i) dot += col[i] * o[i];
            const double f = 2.0 * dot / vtv;
            for (int i = c; i < k; ++i) o[i] -= f * col[i];
        }
        {
            double dot = 0.0;
            for (int i = c; i < k; ++i) dot += col[i] * y[i];
            const double f = 2.0 * dot / vtv;
            for (int i = c; i < k; ++i) y[i] -= f * col[i];
        }
        rdiag[c] = alpha;
    }
    // back substitution: R is stored in the upper triangle (strictly above the diagonal) + rdiag
    for (int c = j - 1; c >= 0; --c) {
        double acc = y[c];
        for (int c2 = c + 1; c2 < j; ++c2) acc -= B[(size_t)c2 * k + c] * x[c2];
        if (rdiag[c] == 0.0) return false;
        x[c] = acc / rdiag[c];
    }
    return true;
}

}  // namespace

extern "C" {

// ---- the A definition ---------------------------------------------------------------------
float orc_sigma(int32_t k) { return sigma_of_k(k); }

// out[r * ncols + c] = Z(seed, row0 + r, col0 + c)
// the binary16 arithmetic of the generator, exported so that the tests can pin it
uint16_t orc_half_round(double v) { return half_round(v); }
double orc_half_value(uint16_t b) { return half_value(b); }
uint16_t orc_half_fma(uint16_t a, uint16_t b, uint16_t c) { return half_fma(a, b, c); }
uint16_t orc_half_mul(uint16_t a, uint16_t b) { return half_mul(a, b); }
uint16_t orc_z_of_byte_sum(int32_t S) { return z_of_byte_sum(S); }

void orc_z_block(uint64_t seed, int64_t row0, int64_t nrows, int64_t col0, int64_t ncols, float* out) {
    for (int64_t c = 0; c < ncols; ++c) {
        const uint32_t ck = column_key(seed, (uint32_t)(col0 + c));
        for (int64_t r = 0; r < nrows; ++r) out[r * ncols + c] = z_from_key(ck, (uint32_t)(row0 + r));
    }
}

// ---- a1: Sparsify_s (Section 3.2) ------------------------------------------------------------
// idx/val: the s entries of largest |g| (ties -> lower index), returned in ascending index order.
int32_t orc_sparsify(const float* g, int64_t d, int32_t s, uint32_t* idx, float* val) {
    if (s < 0 || s > d) return -1;
    std::vector<uint32_t> order((size_t)d);
    std::iota(order.begin(), order.end(), 0u);
    auto before = [g](uint32_t a, uint32_t b) {
        const float ma = std::fabs(g[a]), mb = std::fabs(g[b]);
        return (ma > mb) || (ma == mb && a < b);
    };
    std::partial_sort(order.begin(), order.begin() + s, order.end(), before);
    std::vector<uint32_t> top(order.begin(), order.begin() + s);
    std::sort(top.begin(), top.end());
    for (int32_t i = 0; i < s; ++i) { idx[i] = top[i]; val[i] = g[top[i]]; }
    return 0;
}

// ---- a2: p = A G~, q = A G~^2 (Eq. 4 and the equation after it) --------------------------------
void orc_project(uint64_t seed, int32_t k, const uint32_t* idx, const float* val, int32_t s,
                 double* p, double* q) {
    const double sigma = (double)sigma_of_k(k);
    for (int32_t j = 0; j < k; ++j) {
        double accp = 0.0, accq = 0.0;
        for (int32_t i = 0; i < s; ++i) {
            const double a = a_entry(column_key(seed, idx[i]), (uint32_t)j, sigma);
            const double gi = (double)val[i];
            accp += a * gi;
            accq += a * (gi * gi);
        }
        p[j] = accp; q[j] = accq;
    }
}

// ---- a3: k-space Adam (Algorithm 2) -------------------------------------------------
// M,V: stored fp32 state, updated in place (uncorrected).  t is the 1-based step count of THIS step.
// Mhat,Vhat: bias-corrected temporaries in fp64, computed from the stored (rounded) state.
void orc_adam(float* M, float* V, const double* p, const double* q, int32_t k,
              float beta1, float beta2, int64_t t, double* Mhat, double* Vhat) {
    const double b1 = (double)beta1, b2 = (double)beta2;
    const double c1 = 1.0 - std::pow(b1, (double)t), c2 = 1.0 - std::pow(b2, (double)t);
    for (int32_t j = 0; j < k; ++j) {
        M[j] = (float)(b1 * (double)M[j] + (1.0 - b1) * p[j]);
        V[j] = (float)(b2 * (double)V[j] + (1.0 - b2) * q[j]);
        Mhat[j] = (double)M[j] / c1;
        Vhat[j] = (double)V[j] / c2;
    }
}

// ---- a4: x = OMP_A(y) (Eq. 7; Appendix B) -----------------------------------------------------
// Textbook OMP, s iterations.  Outputs (all length s): lam = selected columns in selection order,
// x = least-squares coefficients aligned with lam (final support), top1/top2 = best and
// second-best normalised correlation at each iteration, rnorm = ||r|| AFTER each iteration.
// Returns the number of completed iterations (< s only on a dependent column).
//
// orc_omp_tol is the same recovery with an optional early stop (not in Algorithm 3, which always runs s iterations):
// with residual_tol > 0 the iterations end after the first one that leaves ||r|| <= residual_tol * ||y||.
int32_t orc_omp_tol(uint64_t seed, int64_t d, int32_t k, int32_t s, const double* y, double residual_tol,
                    uint32_t* lam, double* x, double* top1, double* top2, double* rnorm) {
    const double sigma = (double)sigma_of_k(k);
    double ynorm = 0.0;
    for (int32_t row = 0; row < k; ++row) ynorm += y[row] * y[row];
    ynorm = std::sqrt(ynorm);
    std::vector<double> r(y, y + k);
    std::vector<double> cols;            // selected columns of A, column-major k x j
    std::vector<uint8_t> taken((size_t)d, 0);
    int32_t done = 0;
    for (int32_t it = 0; it < s; ++it) {
        // correlate every unselected column with the residual; normalised argmax, lowest index on ties
        int nthreads = 1;
#ifdef _OPENMP
        nthreads = omp_get_max_threads();
#endif
        std::vector<double> tb1(nthreads, -1.0), tb2(nthreads, -1.0);
        std::vector<int64_t> ti1(nthreads, -1);
#pragma omp parallel
        {
            int tid = 0, nt = 1;
#ifdef _OPENMP
            tid = omp_get_thread_num(); nt = omp_get_num_threads();
#endif
            const int64_t lo = d * tid / nt, hi = d * (tid + 1) / nt;
            double b1 = -1.0, b2 = -1.0; int64_t i1 = -1;
            for (int64_t i = lo; i < hi; ++i) {
                if (taken[i]) continue;
                const uint32_t ck = column_key(seed, (uint32_t)i);
                double dot = 0.0, n2 = 0.0;
                for (int32_t j = 0; j < k; ++j) {
                    const double a = a_entry(ck, (uint32_t)j, sigma);
                    dot += a * r[j];
                    n2 += a * a;
                }
                const double c = std::fabs(dot) / std::sqrt(n2);
                if (c > b1) { b2 = b1; b1 = c; i1 = i; }
                else if (c > b2) { b2 = c; }
            }
            tb1[tid] = b1; tb2[tid] = b2; ti1[tid] = i1;
        }
        double b1 = -1.0, b2 = -1.0; int64_t i1 = -1;
        for (int tdx = 0; tdx < nthreads; ++tdx) {       // ascending column ranges: strict > keeps the lowest index
            if (tb1[tdx] > b1) { b2 = std::max(b1, tb2[tdx]); b1 = tb1[tdx]; i1 = ti1[tdx]; }
            else { b2 = std::max(b2, tb1[tdx]); }
        }
        if (i1 < 0) break;
        // extend the support and solve least squares on it
        const int32_t j = it + 1;
        cols.resize((size_t)j * k);
        {
            const uint32_t ck = column_key(seed, (uint32_t)i1);
            for (int32_t row = 0; row < k; ++row) cols[(size_t)it * k + row] = a_entry(ck, (uint32_t)row, sigma);
        }
        std::vector<double> xs(j);
        // dependence test of the new column on the current support (relative residual of its projection)
        if (it > 0) {
            std::vector<double> prev(cols.begin(), cols.begin() + (size_t)it * k);
            std::vector<double> newc(cols.begin() + (size_t)it * k, cols.end());
            std::vector<double> coef(it);
            bool ok = least_squares_qr(prev, newc, k, it, coef.data());
            double res2 = 0.0, n2 = 0.0;
            for (int32_t row = 0; row < k; ++row) {
                double v = newc[row];
                for (int32_t c = 0; c < it; ++c) v -= cols[(size_t)c * k + row] * coef[c];
                res2 += v * v; n2 += newc[row] * newc[row];
            }
            if (!ok || res2 <= 1e-10 * n2) break;
        }
        if (!least_squares_qr(cols, std::vector<double>(y, y + k), k, j, xs.data())) break;
        taken[i1] = 1;
        lam[it] = (uint32_t)i1;
        top1[it] = b1; top2[it] = b2;
        double rn = 0.0;
        for (int32_t row = 0; row < k; ++row) {
            double v = y[row];
            for (int32_t c = 0; c < j; ++c) v -= cols[(size_t)c * k + row] * xs[c];
            r[row] = v; rn += v * v;
        }
        rnorm[it] = std::sqrt(rn);
        for (int32_t c = 0; c < j; ++c) x[c] = xs[c];
        done = j;
        if (residual_tol > 0.0 && rnorm[it] <= residual_tol * ynorm) break;
    }
    for (int32_t c = done; c < s; ++c) { lam[c] = 0xFFFFFFFFu; x[c] = 0.0; top1[c] = top2[c] = rnorm[c] = 0.0; }
    return done;
}

int32_t orc_omp(uint64_t seed, int64_t d, int32_t k, int32_t s, const double* y,
                uint32_t* lam, double* x, double* top1, double* top2, double* rnorm) {
    return orc_omp_tol(seed, d, k, s, y, 0.0, lam, x, top1, top2, rnorm);
}

// The "Select" line of Algorithm 3 (Appendix B) on its own, for a batch of residuals: for every residual r_n, n < n_res,
//   idx[n] = argmax over the columns i in [0, d) outside skip_n of |<A_:i, r_n>| / ||A_:i||_2   (lowest i on exact ties),
// with the best and the second-best score.  skip_n (the columns already in the support of residual n) holds skip_count[n]
// entries at skip[n * skip_stride ...].  Every residual is treated exactly as one iteration of orc_omp_tol treats its
// residual; the batch only lets one generated column of A meet all residuals.  R is n_res x k, row-major.
void orc_select(uint64_t seed, int64_t d, int32_t k, int32_t n_res, const double* R, const uint32_t* skip,
                const int32_t* skip_count, int32_t skip_stride, int64_t* idx, double* best, double* second) {
    const double sigma = (double)sigma_of_k(k);
    std::vector<uint8_t> listed((size_t)d, 0);          // the column is in some residual's skip list
    for (int32_t n = 0; n < n_res; ++n)
        for (int32_t q = 0; skip && q < skip_count[n]; ++q) {
            const uint32_t c = skip[(size_t)n * skip_stride + q];
            if ((int64_t)c < d) listed[c] = 1;
        }
    std::vector<double> Rt((size_t)k * n_res);           // k x n_res: the residuals' entries of one row side by side
    for (int32_t n = 0; n < n_res; ++n)
        for (int32_t j = 0; j < k; ++j) Rt[(size_t)j * n_res + n] = R[(size_t)n * k + j];
    int nthreads = 1;
#ifdef _OPENMP
    nthreads = omp_get_max_threads();
#endif
    std::vector<double> tb1((size_t)nthreads * n_res, -1.0), tb2((size_t)nthreads * n_res, -1.0);
    std::vector<int64_t> ti1((size_t)nthreads * n_res, -1);
#pragma omp parallel
    {
        int tid = 0, nt = 1;
#ifdef _OPENMP
        tid = omp_get_thread_num(); nt = omp_get_num_threads();
#endif
        const int64_t lo = d * tid / nt, hi = d * (tid + 1) / nt;
        double* b1 = &tb1[(size_t)tid * n_res];
        double* b2 = &tb2[(size_t)tid * n_res];
        int64_t* i1 = &ti1[(size_t)tid * n_res];
        std::vector<double> dot(n_res);
        for (int64_t i = lo; i < hi; ++i) {
            const uint32_t ck = column_key(seed, (uint32_t)i);
            std::fill(dot.begin(), dot.end(), 0.0);
            double n2 = 0.0;
            for (int32_t j = 0; j < k; ++j) {
                const double a = a_entry(ck, (uint32_t)j, sigma);
                const double* rj = &Rt[(size_t)j * n_res];
                for (int32_t n = 0; n < n_res; ++n) dot[n] += a * rj[n];
                n2 += a * a;
            }
            const double nrm = std::sqrt(n2);
            for (int32_t n = 0; n < n_res; ++n) {
                if (listed[i]) {
                    bool skipped = false;
                    for (int32_t q = 0; q < skip_count[n]; ++q) skipped = skipped || skip[(size_t)n * skip_stride + q] == (uint32_t)i;
                    if (skipped) continue;
                }
                const double c = std::fabs(dot[n]) / nrm;
                if (c > b1[n]) { b2[n] = b1[n]; b1[n] = c; i1[n] = i; }
                else if (c > b2[n]) { b2[n] = c; }
            }
        }
    }
    for (int32_t n = 0; n < n_res; ++n) {
        double b1 = -1.0, b2 = -1.0; int64_t i1 = -1;
        for (int tdx = 0; tdx < nthreads; ++tdx) {       // ascending column ranges: strict > keeps the lowest index
            const double c1 = tb1[(size_t)tdx * n_res + n], c2 = tb2[(size_t)tdx * n_res + n];
            if (c1 > b1) { b2 = std::max(b1, c2); b1 = c1; i1 = ti1[(size_t)tdx * n_res + n]; }
            else { b2 = std::max(b2, c1); }
        }
        idx[n] = i1; best[n] = b1; second[n] = b2;
    }
}

// Least squares of y on a given support: x = argmin ||y - A_Lambda x||_2 (the last step of every OMP iteration, on
// its own).  The columns must be independent, as the picks of an OMP run are; returns 0, or -1 on an exactly zero pivot.
int32_t orc_least_squares(uint64_t seed, int32_t k, const uint32_t* lam, int32_t n, const double* y, double* x) {
    const double sigma = (double)sigma_of_k(k);
    std::vector<double> cols((size_t)n * k);
    for (int32_t c = 0; c < n; ++c) {
        const uint32_t ck = column_key(seed, lam[c]);
        for (int32_t row = 0; row < k; ++row) cols[(size_t)c * k + row] = a_entry(ck, (uint32_t)row, sigma);
    }
    return least_squares_qr(cols, std::vector<double>(y, y + k), k, n, x) ? 0 : -1;
}

// ---- a5: N = alpha x^M / (sqrt(x^V) + eps) on the common support; W <- W - eta N (Eq. 8, Eq. 3) ---
// upd_idx/upd_val (capacity s): the positions updated (ascending index) and eta*N there (fp64).
// Returns the number of updated positions; *mismatch = number of M-support entries absent from the
// V-support; *negv = number of common entries skipped because x^V <= 0.
int32_t orc_combine_scatter(const uint32_t* lamM, const double* xM, int32_t nM,
                            const uint32_t* lamV, const double* xV, int32_t nV,
                            float alpha, float eps, float lr, float* W,
                            uint32_t* upd_idx, double* upd_val, int32_t* mismatch, int32_t* negv) {
    std::vector<std::pair<uint32_t, double>> out;
    int32_t mis = 0, neg = 0;
    for (int32_t a = 0; a < nM; ++a) {
        int32_t hit = -1;
        for (int32_t b = 0; b < nV; ++b) if (lamV[b] == lamM[a]) { hit = b; break; }
        if (hit < 0) { ++mis; continue; }
        if (!(xV[hit] > 0.0)) { ++neg; continue; }
        const double N = (double)alpha * xM[a] / (std::sqrt(xV[hit]) + (double)eps);
        out.emplace_back(lamM[a], (double)lr * N);
    }
    std::sort(out.begin(), out.end());
    for (size_t i = 0; i < out.size(); ++i) {
        upd_idx[i] = out[i].first; upd_val[i] = out[i].second;
        W[out[i].first] = (float)((double)W[out[i].first] - out[i].second);
    }
    if (mismatch) *mismatch = mis;
    if (negv) *negv = neg;
    return (int32_t)out.size();
}

// ---- the whole step (Algorithm 2 + Eq. 3), composed of the pieces above -----------------------
struct orc_state {
    int64_t d; int32_t k, s; uint64_t seed; float lr, beta1, beta2, eps, alpha; int64_t t;
    std::vector<float> M, V;
    // records of the last step
    std::vector<uint32_t> sel_idx; std::vector<float> sel_val;
    std::vector<double> p, q, Mhat, Vhat;
    std::vector<uint32_t> lamM, lamV; std::vector<double> xM, xV, top1M, top2M, top1V, top2V, rnM, rnV;
    int32_t doneM, doneV, n_upd, mismatch, negv;
    std::vector<uint32_t> upd_idx; std::vector<double> upd_val;
    // opt-in variant of the recovery (orc_set_recovery)
    int32_t shared_support; double residual_tol;
};

orc_state* orc_create(int64_t d, int32_t k, int32_t s, uint64_t seed, float lr, float beta1, float beta2, float eps) {
    if (d < 1 || k < 1 || s < 1 || s > k || s > d || d >= (int64_t)1 << 32) return nullptr;
    orc_state* st = new orc_state();
    st->d = d; st->k = k; st->s = s; st->seed = seed; st->lr = lr; st->beta1 = beta1; st->beta2 = beta2;
    st->eps = eps; st->alpha = 1.0f; st->t = 0;
    st->M.assign(k, 0.0f); st->V.assign(k, 0.0f);
    st->sel_idx.resize(s); st->sel_val.resize(s);
    st->p.resize(k); st->q.resize(k); st->Mhat.resize(k); st->Vhat.resize(k);
    st->lamM.resize(s); st->lamV.resize(s); st->xM.resize(s); st->xV.resize(s);
    st->top1M.resize(s); st->top2M.resize(s); st->top1V.resize(s); st->top2V.resize(s);
    st->rnM.resize(s); st->rnV.resize(s); st->upd_idx.resize(s); st->upd_val.resize(s);
    st->doneM = st->doneV = st->n_upd = st->mismatch = st->negv = 0;
    st->shared_support = 0; st->residual_tol = 0.0;
    return st;
}
void orc_destroy(orc_state* st) { delete st; }
void orc_set_alpha(orc_state* st, float alpha) { st->alpha = alpha; }
// Opt-in variant built on the remark after Eq. (8) that OMP_A(M) and OMP_A(V) have the same non-zero positions:
// shared_support = 1: OMP_A(M^) alone selects the support; x^V is the least-squares fit of V^ on that support.
// residual_tol > 0: a recovery ends early once ||r|| <= residual_tol * ||y|| (see orc_omp_tol).
// The defaults (0, 0.0) are Algorithm 2 as printed.
void orc_set_recovery(orc_state* st, int32_t shared_support, double residual_tol) {
    st->shared_support = shared_support; st->residual_tol = residual_tol;
}

// Steps a1-a3 only (cheap); used when the recovery is sampled.
void orc_step_compress(orc_state* st, const float* grad) {
    st->t += 1;
    orc_sparsify(grad, st->d, st->s, st->sel_idx.data(), st->sel_val.data());
    orc_project(st->seed, st->k, st->sel_idx.data(), st->sel_val.data(), st->s, st->p.data(), st->q.data());
    orc_adam(st->M.data(), st->V.data(), st->p.data(), st->q.data(), st->k, st->beta1, st->beta2, st->t,
             st->Mhat.data(), st->Vhat.data());
}
// Steps a4-a5 on the state left by orc_step_compress.
void orc_step_recover(orc_state* st, float* weight) {
    st->doneM = orc_omp_tol(st->seed, st->d, st->k, st->s, st->Mhat.data(), st->residual_tol, st->lamM.data(),
                            st->xM.data(), st->top1M.data(), st->top2M.data(), st->rnM.data());
    if (st->shared_support) {
        // one support for both moments: the columns OMP_A(M^) selected, in its order
        for (int32_t c = 0; c < st->s; ++c) {
            st->lamV[c] = st->lamM[c]; st->xV[c] = 0.0; st->top1V[c] = st->top2V[c] = st->rnV[c] = 0.0;
        }
        st->doneV = st->doneM;
        if (st->doneM > 0) orc_least_squares(st->seed, st->k, st->lamM.data(), st->doneM, st->Vhat.data(), st->xV.data());
    } else {
        st->doneV = orc_omp_tol(st->seed, st->d, st->k, st->s, st->Vhat.data(), st->residual_tol, st->lamV.data(),
                                st->xV.data(), st->top1V.data(), st->top2V.data(), st->rnV.data());
    }
    st->n_upd = orc_combine_scatter(st->lamM.data(), st->xM.data(), st->doneM, st->lamV.data(), st->xV.data(),
                                    st->doneV, st->alpha, st->eps, st->lr, weight, st->upd_idx.data(),
                                    st->upd_val.data(), &st->mismatch, &st->negv);
}
void orc_step(orc_state* st, const float* grad, float* weight) {
    orc_step_compress(st, grad);
    orc_step_recover(st, weight);
}

// SGCA re-projection (Appendix C, Algorithm 4): with a new matrix A' (here: a new seed),
//   M <- A' OMP_A(M),  V <- A' OMP_A(V),  A <- A'.
// Reading: M and V are the stored moments (bias correction yields temporaries, as everywhere in this oracle); both
// recoveries are run afresh on them with the old A, s iterations each, and the s-sparse results are projected with A'.
void orc_reproject(orc_state* st, uint64_t new_seed) {
    const int32_t k = st->k, s = st->s;
    std::vector<double> y((size_t)k), x((size_t)s), t1((size_t)s), t2((size_t)s), rn((size_t)s), out((size_t)k), unused((size_t)k);
    std::vector<uint32_t> lam((size_t)s);
    std::vector<float> val((size_t)s);
    int32_t done = 0;
    for (int pass = 0; pass < 2; ++pass) {
        std::vector<float>& state = pass == 0 ? st->M : st->V;
        for (int32_t j = 0; j < k; ++j) y[j] = (double)state[j];
        if (pass == 1 && st->shared_support) {
            // the variant of orc_set_recovery: V is fitted on the support found for M
            for (int32_t l = 0; l < s; ++l) x[l] = 0.0;
            if (done > 0) orc_least_squares(st->seed, k, lam.data(), done, y.data(), x.data());
        } else {
            done = orc_omp_tol(st->seed, st->d, k, s, y.data(), st->residual_tol, lam.data(), x.data(), t1.data(), t2.data(),
                               rn.data());
        }
        // A' x with x supported on the recovered columns: sum in fp64 in the order of selection
        for (int32_t j = 0; j < k; ++j) out[j] = 0.0;
        const double sigma = (double)sigma_of_k(k);
        for (int32_t l = 0; l < done; ++l) {
            const uint32_t ck = column_key(new_seed, lam[l]);
            for (int32_t j = 0; j < k; ++j) out[j] += a_entry(ck, (uint32_t)j, sigma) * x[l];
        }
        for (int32_t j = 0; j < k; ++j) state[j] = (float)out[j];
    }
    st->seed = new_seed;
}

// Read-back of the last step's records.  what: see the Python binding for the list.
int32_t orc_get(orc_state* st, int32_t what, void* dst, int64_t bytes) {
    const void* src = nullptr; int64_t n = 0;
    switch (what) {
        case 0: src = &st->t; n = 8; break;
        case 1: src = st->M.data(); n = 4 * (int64_t)st->k; break;
        case 2: src = st->V.data(); n = 4 * (int64_t)st->k; break;
        case 3: src = st->p.data(); n = 8 * (int64_t)st->k; break;
        case 4: src = st->q.data(); n = 8 * (int64_t)st->k; break;
        case 5: src = st->sel_idx.data(); n = 4 * (int64_t)st->s; break;
        case 6: src = st->sel_val.data(); n = 4 * (int64_t)st->s; break;
        case 7: src = st->lamM.data(); n = 4 * (int64_t)st->s; break;
        case 8: src = st->lamV.data(); n = 4 * (int64_t)st->s; break;
        case 9: src = st->xM.data(); n = 8 * (int64_t)st->s; break;
        case 10: src = st->xV.data(); n = 8 * (int64_t)st->s; break;
        case 11: src = st->top1M.data(); n = 8 * (int64_t)st->s; break;
        case 12: src = st->top2M.data(); n = 8 * (int64_t)st->s; break;
        case 13: src = st->top1V.data(); n = 8 * (int64_t)st->s; break;
        case 14: src = st->top2V.data(); n = 8 * (int64_t)st->s; break;
        case 15: src = st->upd_idx.data(); n = 4 * (int64_t)st->s; break;
        case 16: src = st->upd_val.data(); n = 8 * (int64_t)st->s; break;
        case 17: src = &st->n_upd; n = 4; break;
        case 18: src = &st->mismatch; n = 4; break;
        case 19: src = &st->negv; n = 4; break;
        case 20: src = &st->doneM; n = 4; break;
        case 21: src = &st->doneV; n = 4; break;
        case 22: src = st->Mhat.data(); n = 8 * (int64_t)st->k; break;
        case 23: src = st->Vhat.data(); n = 8 * (int64_t)st->k; break;
        case 24: src = st->rnM.data(); n = 8 * (int64_t)st->s; break;
        case 25: src = st->rnV.data(); n = 8 * (int64_t)st->s; break;
        default: return -1;
    }
    if (bytes < n) return -2;
    std::memcpy(dst, src, (size_t)n);
    return 0;
}

int32_t orc_num_threads(void) {
#ifdef _OPENMP
    return omp_get_max_threads();
#else
    return 1;
#endif
}

}  // extern "C"
