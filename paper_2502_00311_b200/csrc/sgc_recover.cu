// a4 + a5: x^M = OMP_A(M^), x^V = OMP_A(V^) (Eq. 7; Appendix B Algorithm 3), then
// N = alpha x^M / (sqrt(x^V) + eps) and W <- W - lr N (Eq. 8, Eq. 3; Algorithm 2).
//
// Algorithm 3 needs, for every pick, the argmax of |<A_i, r>| / ||A_i|| over all d columns ("Projection" and
// "Select"), and A is regenerated rather than stored, so one such argmax costs k*d generated entries.  Two ways
// of getting the picks are implemented; both produce exactly the picks of Algorithm 3.
//
// Lock-step (k_omp, mode 1): one pass over all columns per pick, both residuals (M^ and V^) against every
//   generated entry; fp32 screen, fp64 decision among the near-maximal candidates, then the inverse-Cholesky
//   recurrences of Algorithm 3 (c = F^T g, gamma, new column of F, a_j, x = F a) in fp64 and r = y - A_Lambda x.
//
// Speculative (rounds of speculation kernels, the tensor-core screening pass, k_resolve): OMP first runs on a short
//   candidate list only (the supports of the previous step plus harvested columns), which costs next to
//   nothing, and records the residual before every pick.  ONE pass over all d columns then correlates A with
//   all those residuals at once (sgc_pass.cu) and reports every column whose score comes within the rounding
//   margin of the speculated pick's.  k_resolve walks the picks in order: a pick without a challenger, or one
//   that wins the fp64 rescoring against its challengers, is the true argmax; at the first pick that loses,
//   the global winner (known from the same pass) is forced, the columns reported for that residual join the
//   candidate list and the next round continues from there.  Every round fixes at least one more pick; what is
//   still open after the enqueued rounds, or after any overflow, is finished in lock-step.
//   The speculation itself has three forms, chosen on the device by the length of the list: Algorithm 3 on the
//   list's Gram matrix (k_gram_prepare, k_gram_matrix, k_omp_gram, k_spec_rows; up to kGramList columns), one
//   block per residual correlating the list itself (k_spec_small; up to kSmallList), and k_omp mode 0 beyond.
//
// k_omp is one cooperative kernel for lock-step and long lists: all blocks correlate (phase A), grid barrier,
// blocks 0 and 1 keep the books of M^ and V^ (phase B), grid barrier.  k_scatter applies Eq. (8) on the common
// support.  Several states that share A are recovered together (launch_recover_group): their residuals sit side by
// side in one screened batch, so one pass serves them all.
#include <cooperative_groups.h>
#include <cuda_fp16.h>

#include "sgc_internal.cuh"

namespace cg = cooperative_groups;

namespace sgc {
namespace {

struct OmpArgs {
    uint32_t seed_lo, seed_hi;
    unsigned long long d;
    int k, s;
    unsigned int num_tiles;            // lock-step tiles of kOmpThreads * kCorrCols columns
    double sigma;
    int half_n;                        // residuals per stream in one screening pass
    int rows_wide, rows_narrow;        // rows of the pass that serves both streams / the first stream alone
    double z_harvest, z_floor;         // screening thresholds in units of ||r|| / sqrt(k)
    Cand* corr_cand;                   // [2][grid][kCorrTop]
    const double* y64; double* r64; float* r32;      // r32 viewed as float[2k] (interleaved pairs)
    uint16_t* zsel; uint32_t* lam; double* F; double* acoef; double* x; double* rnorm;
    Counters* cnt; SpecCtl* ctl;
    uint16_t* rt; float* tau; float* inv_scale; unsigned int* rep_count; double* pick_score;
    double* rhist;                     // fp64 copies of the screened residuals (row = m * half_n + position), for the resolve kernel
    // two-level screening
    float* wide_tau; double z_wide; unsigned int* wide_count; unsigned int* wide_bits;
    int mini;                          // 1: speculation ahead of a list pass (at most `depth` picks)
    int depth;
    const uint32_t* cand_list;
    uint16_t* zlist; double* gram; double* p0; int* pick_li;     // Gram path
};

// ------------------------------------------------------------------------------------------------
// small helpers
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ bool better(float sa, uint32_t ia, float sb, uint32_t ib) {
    return (sa > sb) || (sa == sb && ia < ib);
}

// the best two columns seen, and the largest score among all others (what is dropped: the caller can tell whether a
// dropped column could still have mattered)
struct Top2 {
    float s1, s2, s3; uint32_t i1, i2;
    __device__ __forceinline__ void init() { s1 = s2 = s3 = -1.0f; i1 = i2 = kNoColumn; }
    __device__ __forceinline__ void push(float s, uint32_t i) {
        if (i == i1 || i == i2) return;
        if (better(s, i, s1, i1)) { s3 = fmaxf(s3, s2); s2 = s1; i2 = i1; s1 = s; i1 = i; }
        else if (better(s, i, s2, i2)) { s3 = fmaxf(s3, s2); s2 = s; i2 = i; }
        else s3 = fmaxf(s3, s);
    }
};

__device__ __forceinline__ void warp_merge(Top2& t) {
    for (int o = 16; o > 0; o >>= 1) {
        const float a1 = __shfl_xor_sync(0xffffffffu, t.s1, o), a2 = __shfl_xor_sync(0xffffffffu, t.s2, o);
        const uint32_t j1 = __shfl_xor_sync(0xffffffffu, t.i1, o), j2 = __shfl_xor_sync(0xffffffffu, t.i2, o);
        const float a3 = __shfl_xor_sync(0xffffffffu, t.s3, o);
        if (j1 != kNoColumn) t.push(a1, j1);
        if (j2 != kNoColumn) t.push(a2, j2);
        t.s3 = fmaxf(t.s3, a3);
    }
}

__device__ __forceinline__ double warp_sum(double v) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}
__device__ __forceinline__ float warp_sum(float v) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// deterministic block sum (kOmpThreads threads); every thread receives the result.  red: 32 doubles.
__device__ double block_sum(double v, double* red) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    double t = (lane < kOmpThreads / 32) ? red[lane] : 0.0;
    t = warp_sum(t);
    return t;
}

// threshold of a wide list: every column scoring at least z_wide noise deviations against a screened residual (norm rn)
// whose row index is a multiple of 8, in the scaled units of that row
__device__ __forceinline__ float wide_threshold(const OmpArgs& a, double rn) {
    return (float)(a.z_wide * rn / sqrt((double)a.k) * residual_scale(rn));
}

// shared memory of the bookkeeping code (blocks 0 and 1 of k_omp, the only block of k_resolve)
struct BookSmem {
    double red[32];
    float fred[32];
    double gvec[kMaxS];               // Gram column g
    double cvec[kMaxS];               // c = F^T g
    double xs[kMaxS];                 // current coefficients
    double best_dot, best_n2, best_score;
    double cur_rnorm;                 // ||r|| of the residual the next pick is made from
    uint32_t best_idx;
    uint32_t cand_idx[kRescoreCap];
    int n_cand;
    int rescan_n; int rescan_blk[8];  // blocks of the lock-step screen that kept a near-maximal column to themselves
    int hi, extra, dep, stop;         // speculation record of this block's stream
    unsigned int smax_bits;
};

// exact score of one column against a residual: dot = <Z_i, r>, n2 = ||Z_i||^2 (fp64), for every thread
__device__ void rescore_column(const OmpArgs& a, BookSmem& sh, uint32_t idx, const double* r, double* dot_out, double* n2_out) {
    const ColKey key = column_key(a.seed_lo, a.seed_hi, idx);
    double dot = 0.0, n2 = 0.0;
    for (int row = 2 * threadIdx.x; row < a.k; row += 2 * kOmpThreads) {            // one generated word = two rows
        const float2 zz = half2_bits_to_float2(z_pair_from_word(key.ck + (uint32_t)(row >> 1) * key.mk));
        dot += (double)zz.x * r[row];
        n2 += (double)zz.x * (double)zz.x;
        if (row + 1 < a.k) {
            dot += (double)zz.y * r[row + 1];
            n2 += (double)zz.y * (double)zz.y;
        }
    }
    *dot_out = block_sum(dot, sh.red);
    *n2_out = block_sum(n2, sh.red);
}

// fp64 argmax of |<A_i, r>| / ||A_i|| among sh.cand_idx[0..nc), lowest index on ties -> sh.best_*
__device__ void rescore_candidates(const OmpArgs& a, BookSmem& sh, int nc, const double* r) {
    if (threadIdx.x == 0) { sh.best_score = -1.0; sh.best_idx = kNoColumn; sh.best_dot = 0.0; sh.best_n2 = 1.0; }
    __syncthreads();
    for (int c = 0; c < nc; ++c) {
        const uint32_t idx = sh.cand_idx[c];
        double dot, n2;
        rescore_column(a, sh, idx, r, &dot, &n2);
        if (threadIdx.x == 0) {
            const double sc = n2 > 0.0 ? dot * dot / n2 : 0.0;
            if (sc > sh.best_score || (sc == sh.best_score && idx < sh.best_idx)) {
                sh.best_score = sc; sh.best_idx = idx; sh.best_dot = dot; sh.best_n2 = n2;
            }
        }
        __syncthreads();
    }
}

// x = F a and r = y - A_Lambda x for the first v picks (F, a and the stored columns are prefixes of their
// final values, so any earlier state can be rebuilt); r goes to r_out, x to sh.xs (and x_out when given).
// Returns ||r||.
__device__ double rebuild_prefix(const OmpArgs& a, BookSmem& sh, int m, int v, double* r_out, float* r32_out, double* x_out) {
    const int k = a.k, s = a.s;
    const double* y = a.y64 + (size_t)m * k;
    const uint16_t* zs = a.zsel + (size_t)m * s * k;
    const double* F = a.F + (size_t)m * s * s;
    const double* ac = a.acoef + (size_t)m * s;
    __syncthreads();
    if ((int)threadIdx.x < v) {
        const int i = threadIdx.x;
        double acc = 0.0;
#pragma unroll 8
        for (int l = i; l < v; ++l) acc = acc + ac[l] * F[(size_t)i * s + l];
        sh.xs[i] = acc;
        if (x_out) x_out[i] = acc;
    }
    __syncthreads();
    double rn2 = 0.0;
    for (int row = threadIdx.x; row < k; row += kOmpThreads) {
        double acc = 0.0;
#pragma unroll 8
        for (int l = 0; l < v; ++l) acc += sh.xs[l] * (double)half_bits_to_float(zs[(size_t)l * k + row]);
        const double rv = y[row] - a.sigma * acc;
        r_out[row] = rv;
        if (r32_out) r32_out[2 * row + m] = (float)rv;
        rn2 += rv * rv;
    }
    rn2 = block_sum(rn2, sh.red);
    return sqrt(rn2);
}

// residual r (norm rn) becomes row c of stream m of the screened batch: binary16, scaled by a power of two
__device__ void write_rt_row(const OmpArgs& a, int m, int c, const double* r, double rn) {
    const int n = m * a.half_n + c;
    uint16_t* dst = a.rt + (size_t)n * a.k;
    const double sc = residual_scale(rn);
    double* keep = a.rhist + (size_t)n * a.k;
    for (int row = threadIdx.x; row < a.k; row += kOmpThreads) {
        const double rv = r[row];
        dst[row] = half_rn_bits(rv * sc);
        keep[row] = rv;
    }
    if (threadIdx.x == 0) a.inv_scale[n] = (float)(1.0 / sc);
}

// ------------------------------------------------------------------------------------------------
// phase A, lock-step: every column of A against both residuals (thread = kCorrCols columns x all rows)
// ------------------------------------------------------------------------------------------------
__device__ void corr_all_columns(const OmpArgs& a, float2* sr, uint32_t (*mask_idx)[kMaxS], int* mask_n, Top2 (*wtop)[32],
                                 const int* picks) {
    const int k = a.k, s = a.s;
    const float2* r32 = reinterpret_cast<const float2*>(a.r32);
    __syncthreads();
    for (int j = threadIdx.x; j < k; j += kOmpThreads) sr[j] = r32[j];
    if (threadIdx.x == 0) sr[k] = make_float2(0.0f, 0.0f);          // partner of the last row when k is odd
    Top2 best[2];
    best[0].init(); best[1].init();
    constexpr unsigned int kTileCols = kOmpThreads * kCorrCols;
    for (unsigned int tile = blockIdx.x; tile < a.num_tiles; tile += gridDim.x) {
        const unsigned long long col_base = (unsigned long long)tile * kTileCols;
        __syncthreads();
        if (threadIdx.x < 2) mask_n[threadIdx.x] = 0;
        __syncthreads();
        // already selected columns that fall into this tile are excluded from the argmax
        for (int e = threadIdx.x; e < picks[0] + picks[1]; e += kOmpThreads) {
            const int m = e < picks[0] ? 0 : 1;
            const uint32_t l = a.lam[m * s + (m ? e - picks[0] : e)];
            if (l >= col_base && l < col_base + kTileCols) mask_idx[m][atomicAdd(&mask_n[m], 1)] = l;
        }
        uint32_t h[kCorrCols], mk[kCorrCols];
        float am[kCorrCols], av[kCorrCols], an[kCorrCols];
#pragma unroll
        for (int c = 0; c < kCorrCols; ++c) {
            const ColKey key = column_key(a.seed_lo, a.seed_hi, (uint32_t)(col_base + c * kOmpThreads + threadIdx.x));
            h[c] = key.ck; mk[c] = key.mk;
            am[c] = av[c] = an[c] = 0.0f;
        }
        __syncthreads();
#pragma unroll 2
        for (int row = 0; row < k; row += 2) {                      // one generated word = two rows
            const float2 r0 = sr[row], r1 = sr[row + 1];
            const bool both = row + 1 < k;
#pragma unroll
            for (int c = 0; c < kCorrCols; ++c) {
                const float2 z = half2_bits_to_float2(z_pair_from_word(h[c]));
                h[c] += mk[c];
                am[c] = __fmaf_rn(z.x, r0.x, am[c]);
                av[c] = __fmaf_rn(z.x, r0.y, av[c]);
                an[c] = __fmaf_rn(z.x, z.x, an[c]);
                am[c] = __fmaf_rn(z.y, r1.x, am[c]);
                av[c] = __fmaf_rn(z.y, r1.y, av[c]);
                if (both) an[c] = __fmaf_rn(z.y, z.y, an[c]);
            }
        }
#pragma unroll
        for (int c = 0; c < kCorrCols; ++c) {
            const unsigned long long col = col_base + c * kOmpThreads + threadIdx.x;
            if (col >= a.d) continue;
            const float inv = an[c] > 0.0f ? 1.0f / an[c] : 0.0f;
            float sm = am[c] * am[c] * inv, sv = av[c] * av[c] * inv;
            for (int e = 0; e < mask_n[0]; ++e) if (mask_idx[0][e] == (uint32_t)col) sm = -1.0f;
            for (int e = 0; e < mask_n[1]; ++e) if (mask_idx[1][e] == (uint32_t)col) sv = -1.0f;
            if (sm >= 0.0f) best[0].push(sm, (uint32_t)col);
            if (sv >= 0.0f) best[1].push(sv, (uint32_t)col);
        }
    }
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    warp_merge(best[0]);
    warp_merge(best[1]);
    __syncthreads();
    if (lane == 0) { wtop[0][warp] = best[0]; wtop[1][warp] = best[1]; }
    __syncthreads();
    if (warp < 2) {
        Top2 t = wtop[warp][lane];
        warp_merge(t);
        if (lane == 0) {
            Cand* o = a.corr_cand + ((size_t)warp * gridDim.x + blockIdx.x) * kCorrTop;
            o[0].score = t.s1; o[0].idx = t.i1;
            o[1].score = t.s2; o[1].idx = t.i2;
            o[2].score = t.s3; o[2].idx = kNoColumn;        // score of the best column this block did not forward
        }
    }
}

// ------------------------------------------------------------------------------------------------
// phase A, restricted: the candidate list against both residuals (warp = one column, lanes over rows)
// ------------------------------------------------------------------------------------------------
__device__ void corr_candidates(const OmpArgs& a, int n_cand, Top2 (*wtop)[32], const int* picks, float2* sr,
                                uint32_t (*sup)[kMaxS]) {
    const int k = a.k, s = a.s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    // the residual pair and both supports, once per call, in shared memory: every candidate reads them
    {
        const float2* r32 = reinterpret_cast<const float2*>(a.r32);
        for (int row = threadIdx.x; row < k; row += kOmpThreads) sr[row] = r32[row];
        for (int q = threadIdx.x; q < picks[0]; q += kOmpThreads) sup[0][q] = a.lam[q];
        for (int q = threadIdx.x; q < picks[1]; q += kOmpThreads) sup[1][q] = a.lam[s + q];
    }
    __syncthreads();
    const float2* r32 = sr;
    Top2 best[2];
    best[0].init(); best[1].init();
    const int stride = gridDim.x * (kOmpThreads / 32);
    for (int e = warp * gridDim.x + blockIdx.x; e < n_cand; e += stride) {        // neighbours go to different blocks
        const uint32_t col = a.cand_list[e];
        bool t0 = false, t1 = false;
        for (int q = lane; q < picks[0]; q += 32) t0 |= (sup[0][q] == col);
        for (int q = lane; q < picks[1]; q += 32) t1 |= (sup[1][q] == col);
        t0 = __any_sync(0xffffffffu, t0);
        t1 = __any_sync(0xffffffffu, t1);
        const ColKey key = column_key(a.seed_lo, a.seed_hi, col);
        float dm = 0.0f, dv = 0.0f, n2 = 0.0f;
        uint32_t h = key.ck + (uint32_t)lane * key.mk;
        const uint32_t step = 32u * key.mk;
        if ((k & 1) == 0) {
            // both residual pairs of a generated word in one 16-byte read: consecutive lanes, consecutive banks
            const float4* r4 = reinterpret_cast<const float4*>(r32);
#pragma unroll 4
            for (int pr = lane; pr < (k >> 1); pr += 32) {
                const float2 z = half2_bits_to_float2(z_pair_from_word(h));
                h += step;
                const float4 rr = r4[pr];
                dm = __fmaf_rn(z.x, rr.x, dm);
                dv = __fmaf_rn(z.x, rr.y, dv);
                n2 = __fmaf_rn(z.x, z.x, n2);
                dm = __fmaf_rn(z.y, rr.z, dm);
                dv = __fmaf_rn(z.y, rr.w, dv);
                n2 = __fmaf_rn(z.y, z.y, n2);
            }
        } else {
#pragma unroll 4
            for (int row = 2 * lane; row < k; row += 64) {              // one generated word = two rows
                const float2 z = half2_bits_to_float2(z_pair_from_word(h));
                h += step;
                const float2 r0 = r32[row];
                dm = __fmaf_rn(z.x, r0.x, dm);
                dv = __fmaf_rn(z.x, r0.y, dv);
                n2 = __fmaf_rn(z.x, z.x, n2);
                if (row + 1 < k) {
                    const float2 r1 = r32[row + 1];
                    dm = __fmaf_rn(z.y, r1.x, dm);
                    dv = __fmaf_rn(z.y, r1.y, dv);
                    n2 = __fmaf_rn(z.y, z.y, n2);
                }
            }
        }
        dm = warp_sum(dm); dv = warp_sum(dv); n2 = warp_sum(n2);
        const float inv = n2 > 0.0f ? 1.0f / n2 : 0.0f;
        if (!t0) best[0].push(dm * dm * inv, col);
        if (!t1) best[1].push(dv * dv * inv, col);
    }
    __syncthreads();
    if (lane == 0) { wtop[0][warp] = best[0]; wtop[1][warp] = best[1]; }
    __syncthreads();
    if (warp < 2) {
        Top2 t = wtop[warp][lane];
        warp_merge(t);
        if (lane == 0) {
            Cand* o = a.corr_cand + ((size_t)warp * gridDim.x + blockIdx.x) * kCorrTop;
            o[0].score = t.s1; o[0].idx = t.i1;
            o[1].score = t.s2; o[1].idx = t.i2;
            o[2].score = -1.0f; o[2].idx = kNoColumn;       // a speculation: the screening pass judges what was left out
        }
    }
}

__device__ __forceinline__ bool in_support_list(const uint32_t* lam, int n, uint32_t col) {
    for (int q = 0; q < n; ++q) if (lam[q] == col) return true;
    return false;
}

// Lock-step only.  Block `blk` of the screen forwarded its best two columns for residual m, but a third scored inside the
// rescoring window as well (score >= thr).  The bookkeeping block walks that block's tiles again with the arithmetic of
// corr_all_columns (same operations in the same order, hence the same fp32 scores) and appends every free column with
// score >= thr that was not forwarded, so that all of them reach the fp64 decision.  Costs about one screen of a block
// (a 1/gridDim share of the columns), only when it happens.
__device__ void rescan_block(const OmpArgs& a, BookSmem& sh, int m, int j, int blk, float thr, const float2* sr,
                             const Cand* fwd) {
    const int k = a.k;
    const uint32_t f0 = fwd[0].idx, f1 = fwd[1].idx;
    const uint32_t* lam = a.lam + (size_t)m * a.s;
    constexpr unsigned int kTileCols = kOmpThreads * kCorrCols;
    for (unsigned int tile = (unsigned int)blk; tile < a.num_tiles; tile += gridDim.x) {
        const unsigned long long col_base = (unsigned long long)tile * kTileCols;
#pragma unroll 1
        for (int c = 0; c < kCorrCols; ++c) {
            const unsigned long long col = col_base + c * kOmpThreads + threadIdx.x;
            const ColKey key = column_key(a.seed_lo, a.seed_hi, (uint32_t)col);
            uint32_t h = key.ck;
            float acc = 0.0f, an = 0.0f;
            for (int row = 0; row < k; row += 2) {
                const float2 r0 = sr[row], r1 = sr[row + 1];
                const float2 z = half2_bits_to_float2(z_pair_from_word(h));
                h += key.mk;
                acc = __fmaf_rn(z.x, m ? r0.y : r0.x, acc);
                an = __fmaf_rn(z.x, z.x, an);
                acc = __fmaf_rn(z.y, m ? r1.y : r1.x, acc);
                if (row + 1 < k) an = __fmaf_rn(z.y, z.y, an);
            }
            if (col >= a.d) continue;
            const float inv = an > 0.0f ? 1.0f / an : 0.0f;
            const float sc = acc * acc * inv;
            if (sc >= thr && (uint32_t)col != f0 && (uint32_t)col != f1 && !in_support_list(lam, j, (uint32_t)col)) {
                const int slot = atomicAdd(&sh.n_cand, 1);
                if (slot < kRescoreCap) sh.cand_idx[slot] = (uint32_t)col;
            }
        }
    }
    __syncthreads();
}

// ------------------------------------------------------------------------------------------------
// phase B: one pick of Algorithm 3 for residual m (whole block).  The pick is `forced` when given, otherwise
// the fp64 argmax among the screened candidates of phase A.
// Returns 0 = booked, 1 = no candidate left, 2 = the picked column is linearly dependent on the support.
// spec_c >= 0: the pick is speculative and screened as residual spec_c of stream m (score and threshold are
// recorded); spec_next >= 0: the new residual becomes row spec_next of the screened batch.
// ------------------------------------------------------------------------------------------------
__device__ int book_pick(const OmpArgs& a, BookSmem& sh, int m, int j, uint32_t forced, int spec_c, int spec_next,
                         bool final_pick, const Cand* cc, int n_entries, const float2* sr_lock = nullptr) {
    const int k = a.k, s = a.s;
    const double* y = a.y64 + (size_t)m * k;
    double* r = a.r64 + (size_t)m * k;
    uint16_t* zs = a.zsel + (size_t)m * s * k;
    double* F = a.F + (size_t)m * s * s;
    double* xg = a.x + (size_t)m * s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int nc;
    __syncthreads();
    if (forced != kNoColumn) {
        if (threadIdx.x == 0) sh.cand_idx[0] = forced;
        nc = 1;
        __syncthreads();
    } else {
        // ---- 1. screened candidates: everything within 2e-3 (relative, squared scores) of the best fp32 score
        float mx = -1.0f;
        for (int e = threadIdx.x; e < n_entries; e += kOmpThreads) {
            const Cand c = cc[e];
            if (c.idx != kNoColumn) mx = fmaxf(mx, c.score);
        }
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        if (threadIdx.x == 0) { sh.n_cand = 0; sh.rescan_n = 0; }
        if (lane == 0) sh.fred[warp] = mx;
        __syncthreads();
        mx = sh.fred[lane];
        for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
        const float thr = mx - 2e-3f * fabsf(mx);
        for (int e = threadIdx.x; e < n_entries; e += kOmpThreads) {
            const Cand c = cc[e];
            if (c.idx != kNoColumn && c.score >= 0.0f && c.score >= thr) {
                const int slot = atomicAdd(&sh.n_cand, 1);
                if (slot < kRescoreCap) sh.cand_idx[slot] = c.idx;
            } else if (c.idx == kNoColumn && c.score >= 0.0f && c.score >= thr) {
                // a block of the lock-step screen kept a third column inside the rescoring window to itself: its range is
                // screened again below so that the column reaches the fp64 decision (flagged only when that cannot be done)
                const int slot = sr_lock != nullptr ? atomicAdd(&sh.rescan_n, 1) : 8;
                if (slot < 8) sh.rescan_blk[slot] = e / kCorrTop;
                else atomicOr(&a.cnt->status, (unsigned int)SGC_STATUS_CANDIDATE_OVERFLOW);
            }
        }
        __syncthreads();
        if (sr_lock != nullptr) {
            const int n_rescan = sh.rescan_n < 8 ? sh.rescan_n : 8;
            for (int q = 0; q < n_rescan; ++q)
                rescan_block(a, sh, m, j, sh.rescan_blk[q], thr, sr_lock, cc + (size_t)sh.rescan_blk[q] * kCorrTop);
        }
        nc = sh.n_cand;
        if (nc > kRescoreCap) {
            if (threadIdx.x == 0) atomicOr(&a.cnt->status, (unsigned int)SGC_STATUS_CANDIDATE_OVERFLOW);
            nc = kRescoreCap;
        }
        if (nc == 0) return 1;
    }
    // ---- 2. fp64 rescoring: the argmax of |<A_i, r>| / ||A_i|| among the candidates, lowest index on ties
    rescore_candidates(a, sh, nc, r);
    const uint32_t lam_new = sh.best_idx;
    const double dot_r = sh.best_dot, n2_new = sh.best_n2;
    if (spec_c >= 0) {
        // what the screening pass must be able to refute: any column scoring above this pick, up to the margin
        if (threadIdx.x == 0) {
            const double ps = sqrt(sh.best_score), rn = sh.cur_rnorm, unit = rn / sqrt((double)k);
            a.pick_score[(size_t)m * s + j] = ps;
            double t = ps - screen_margin(rn, ps, k);
            if (t > a.z_harvest * unit) t = a.z_harvest * unit;
            if (t < a.z_floor * unit) t = a.z_floor * unit;
            a.tau[m * a.half_n + spec_c] = (float)(t * residual_scale(rn));     // row spec_c was scaled with this norm
            if ((spec_c & 7) == 0) a.wide_tau[(m * a.half_n + spec_c) >> 3] = wide_threshold(a, rn);
            a.lam[(size_t)m * s + j] = lam_new;
        }
    }
    // ---- 3. store the new column (binary16 bits, exact) --------------------------------------------------
    {
        const ColKey key = column_key(a.seed_lo, a.seed_hi, lam_new);
        uint16_t* znew = zs + (size_t)j * k;
        for (int row = 2 * threadIdx.x; row < k; row += 2 * kOmpThreads) {
            const uint32_t z2 = z_pair_from_word(key.ck + (uint32_t)(row >> 1) * key.mk);
            znew[row] = (uint16_t)(z2 & 0xFFFFu);
            if (row + 1 < k) znew[row + 1] = (uint16_t)(z2 >> 16);
        }
    }
    __syncthreads();
    // ---- 4. g = A_Lambda^T a_new  (Gram column; "g_{:,lambda_k}" restricted to the support) --------------
    // warp = one stored column; eight binary16 entries per load when the rows allow it
    const double sig2 = a.sigma * a.sigma;
    {
        const uint16_t* znew = zs + (size_t)j * k;
        const bool vec = (k & 7) == 0;
        for (int l = warp; l < j; l += kOmpThreads / 32) {
            const uint16_t* zl = zs + (size_t)l * k;
            double acc = 0.0;
            if (vec) {
                const uint4* pl = reinterpret_cast<const uint4*>(zl);
                const uint4* pn = reinterpret_cast<const uint4*>(znew);
#pragma unroll 4
                for (int v = lane; v < (k >> 3); v += 32) {
                    const uint4 xa = pl[v], xb = pn[v];
                    const uint32_t wa[4] = {xa.x, xa.y, xa.z, xa.w}, wb[4] = {xb.x, xb.y, xb.z, xb.w};
#pragma unroll
                    for (int e = 0; e < 4; ++e) {                          // products of two binary16 numbers are exact in fp32
                        const float2 fa = half2_bits_to_float2(wa[e]), fb = half2_bits_to_float2(wb[e]);
                        acc += (double)(fa.x * fb.x);
                        acc += (double)(fa.y * fb.y);
                    }
                }
            } else {
#pragma unroll 8
                for (int row = lane; row < k; row += 32)
                    acc += (double)(half_bits_to_float(zl[row]) * half_bits_to_float(znew[row]));
            }
            acc = warp_sum(acc);
            if (lane == 0) sh.gvec[l] = sig2 * acc;
        }
    }
    __syncthreads();
    // ---- 5. c = F^T g ;  F is upper triangular, F(l,i) stored at F[l*s + i]; warp = one entry of c -------
    for (int i = warp; i < j; i += kOmpThreads / 32) {
        double acc = 0.0;
        for (int l = lane; l <= i; l += 32) acc += F[(size_t)l * s + i] * sh.gvec[l];
        acc = warp_sum(acc);
        if (lane == 0) sh.cvec[i] = acc;
    }
    __syncthreads();
    double csq = 0.0;
    if ((int)threadIdx.x < j) csq = sh.cvec[threadIdx.x] * sh.cvec[threadIdx.x];
    csq = block_sum(csq, sh.red);
    // ---- 6. gamma = 1/sqrt(g_ll - c^T c); a dependent column stops this recovery --------------------------
    const double gnn = sig2 * n2_new;
    const double piv = gnn - csq;
    if (!(piv > 1e-10 * gnn)) return 2;
    const double gamma = 1.0 / sqrt(piv);
    // ---- 7. new column of F: [-gamma F c ; gamma]; warp = one row of F ------------------------------------
    for (int i = warp; i < j; i += kOmpThreads / 32) {
        double acc = 0.0;
        for (int l = i + lane; l < j; l += 32) acc += F[(size_t)i * s + l] * sh.cvec[l];
        acc = warp_sum(acc);
        if (lane == 0) F[(size_t)i * s + j] = -gamma * acc;
    }
    if (threadIdx.x == 0) F[(size_t)j * s + j] = gamma;
    // ---- 8. a_j = gamma <a_new, r> ;  x = F a  grows by a_j * F(:, j) -------------------------------------
    const double aj = gamma * a.sigma * dot_r;
    __syncthreads();
    if ((int)threadIdx.x <= j) {
        const int i = threadIdx.x;
        const double xo = (i < j) ? xg[i] : 0.0;
        const double xn = xo + aj * F[(size_t)i * s + j];
        xg[i] = xn;
        sh.xs[i] = xn;
    }
    if (threadIdx.x == 0) { a.acoef[(size_t)m * s + j] = aj; a.lam[(size_t)m * s + j] = lam_new; }
    __syncthreads();
    // ---- 9. r = y - A_Lambda x ---------------------------------------------------------------------------
    double rn2 = 0.0;
    for (int row = threadIdx.x; row < k; row += kOmpThreads) {
        double acc0 = 0.0, acc1 = 0.0, acc2 = 0.0, acc3 = 0.0;     // four chains: the loads of 32 columns are in flight together
        int l = 0;
#pragma unroll 8
        for (; l + 3 <= j; l += 4) {
            acc0 += sh.xs[l] * (double)half_bits_to_float(zs[(size_t)l * k + row]);
            acc1 += sh.xs[l + 1] * (double)half_bits_to_float(zs[(size_t)(l + 1) * k + row]);
            acc2 += sh.xs[l + 2] * (double)half_bits_to_float(zs[(size_t)(l + 2) * k + row]);
            acc3 += sh.xs[l + 3] * (double)half_bits_to_float(zs[(size_t)(l + 3) * k + row]);
        }
        for (; l <= j; ++l) acc0 += sh.xs[l] * (double)half_bits_to_float(zs[(size_t)l * k + row]);
        acc0 += acc2; acc1 += acc3;
        const double rv = y[row] - a.sigma * (acc0 + acc1);
        r[row] = rv;
        a.r32[2 * row + m] = (float)rv;
        rn2 += rv * rv;
    }
    rn2 = block_sum(rn2, sh.red);
    if (spec_next >= 0) write_rt_row(a, m, spec_next, r, sqrt(rn2));      // each thread re-reads the rows it wrote
    if (threadIdx.x == 0) {
        a.rnorm[(size_t)m * s + j] = sqrt(rn2);
        sh.cur_rnorm = sqrt(rn2);
        // a prescribed column, if there was one, is consumed with this pick
        if (final_pick) { a.cnt->done[m] = j + 1; a.ctl->v[m] = j + 1; a.ctl->forced[m] = kNoColumn; }
    }
    __syncthreads();
    return 0;
}

// ------------------------------------------------------------------------------------------------
// the cooperative OMP kernel.  mode 0: speculate on the candidate list; mode 1: lock-step over all columns.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kOmpThreads, 1) k_omp(OmpArgs a, int mode) {
    cg::grid_group grid = cg::this_grid();
    extern __shared__ float2 sr[];                       // residual pair per row (lock-step only)
    __shared__ BookSmem sh;
    __shared__ uint32_t mask_idx[2][kMaxS];
    __shared__ int mask_n[2];
    __shared__ Top2 wtop[2][32];
    volatile SpecCtl* ctl = a.ctl;
    // ---- gate: identical in every block, because nothing below changes the control block before the first barrier
    const int fin[2] = {ctl->finished[0], ctl->finished[1]};
    if (mode == 0) {
        if (!ctl->round_active || ctl->fallback || ctl->n_cand <= kSmallList) return;
        if (a.mini && (ctl->mini_done || (a.wide_count[0] == 0u && a.wide_count[1] == 0u))) return;
    } else if (fin[0] && fin[1]) return;
    const int vc[2] = {ctl->v[0], ctl->v[1]};                            // confirmed picks
    const uint32_t fc[2] = {ctl->forced[0], ctl->forced[1]};             // confirmed winner for pick vc, if any
    const int n_cand = ctl->n_cand;
    const int base[2] = {vc[0] + (fc[0] != kNoColumn ? 1 : 0), vc[1] + (fc[1] != kNoColumn ? 1 : 0)};
    // where this kernel starts: the speculation resumes after the tentative picks (those confirmed against the wide
    // lists only), lock-step after the confirmed ones.  The first pick may be prescribed: confirmed (final) or imposed
    // by a list pass (still speculative).
    int v0[2]; uint32_t first_col[2]; bool first_final[2];
    for (int m = 0; m < 2; ++m) {
        const int tv = ctl->tv[m];
        v0[m] = (mode == 0 && tv > vc[m]) ? tv : vc[m];
        first_final[m] = v0[m] == vc[m] && fc[m] != kNoColumn;
        uint32_t first = 0xFFFFFFFFu;                  // kNoColumn
        if (first_final[m]) first = fc[m];
        else if (mode == 0 && v0[m] == tv) first = ctl->tforced[m];
        first_col[m] = first;
    }
    grid.sync();
    const int mb = blockIdx.x;                           // blocks 0 and 1 keep the books of M^ and V^
    // the first full pass of a step starts the wide lists afresh; later ones add what their residuals bring (the lists then
    // cover the whole path of this step, which is where the next step's path runs, too)
    if (mode == 0 && !a.mini && a.wide_count != nullptr && ctl->rounds == 0) {
        if (mb == 0 && threadIdx.x == 0) a.wide_count[0] = a.wide_count[1] = 0u;
        const size_t words = 2 * (((size_t)a.d + 31) / 32);          // both streams' bitmaps
        for (size_t w = (size_t)blockIdx.x * kOmpThreads + threadIdx.x; w < words; w += (size_t)gridDim.x * kOmpThreads)
            a.wide_bits[w] = 0u;
    }
    if (mb < 2) {
        if (!fin[mb]) {
            // state after the picks made so far (a refuted speculation left later values behind)
            const double rn = rebuild_prefix(a, sh, mb, v0[mb], a.r64 + (size_t)mb * a.k, a.r32, a.x + (size_t)mb * a.s);
            if (threadIdx.x == 0) {
                sh.cur_rnorm = rn;
                if (v0[mb] == 0) a.ctl->ynorm[mb] = rn;
                sh.hi = v0[mb] > base[mb] ? v0[mb] : base[mb]; sh.extra = 0; sh.dep = 0;
                a.ctl->stop[mb] = 0;
            }
            const int c0 = v0[mb] - base[mb];
            if (mode == 0 && !first_final[mb] && c0 >= 0 && c0 < a.half_n) write_rt_row(a, mb, c0, a.r64 + (size_t)mb * a.k, rn);
        } else if (threadIdx.x == 0) {
            a.ctl->stop[mb] = 1;
        }
        if (mode == 0) {
            const int keep = fin[mb] ? 0 : (v0[mb] - base[mb] > 0 ? v0[mb] - base[mb] : 0);   // rows of earlier tentative picks stay
            for (int c = threadIdx.x; c < a.half_n; c += kOmpThreads) {
                a.rep_count[mb * a.half_n + c] = 0u;
                if (c >= keep) {
                    a.tau[mb * a.half_n + c] = __int_as_float(0x7f800000);
                    if ((c & 7) == 0) a.wide_tau[(mb * a.half_n + c) >> 3] = __int_as_float(0x7f800000);
                }
            }
        }
    }
    grid.sync();
    for (int i = 0;; ++i) {
        int jm[2], picks[2];
        bool act[2], need_corr = false;
        for (int m = 0; m < 2; ++m) {
            jm[m] = v0[m] + i;
            act[m] = !fin[m] && jm[m] < a.s && !ctl->stop[m];
            if (mode == 0 && (jm[m] - base[m] >= a.half_n || i >= a.depth)) act[m] = false;
            picks[m] = jm[m] < a.s ? jm[m] : a.s;
            if (act[m] && !(i == 0 && first_col[m] != kNoColumn)) need_corr = true;
        }
        if (!act[0] && !act[1]) break;
        if (need_corr) {
            if (mode == 0) corr_candidates(a, n_cand, wtop, picks, sr, mask_idx);
            else corr_all_columns(a, sr, mask_idx, mask_n, wtop, picks);
        }
        grid.sync();
        if (mb < 2 && act[mb]) {
            const int m = mb, j = jm[m];
            const uint32_t forced = (i == 0) ? first_col[m] : kNoColumn;
            const bool speculative = (mode == 0) && !(i == 0 && first_final[m]);
            const int c = j - base[m];                            // -1 for a confirmed prescribed pick
            const int next = (mode == 0 && c + 1 < a.half_n && j + 1 < a.s) ? c + 1 : -1;
            const int rc = book_pick(a, sh, m, j, forced, speculative ? c : -1, next, !speculative,
                                     a.corr_cand + (size_t)m * gridDim.x * kCorrTop, (int)gridDim.x * kCorrTop,
                                     mode == 1 ? sr : nullptr);
            if (threadIdx.x == 0) {
                if (rc == 0) {
                    sh.hi = j + 1;
                } else if (speculative) {
                    // no candidate left: the current residual is screened without a pick; dependent column: the
                    // pick is screened, and the recovery stops there if the pick is confirmed
                    if (rc == 1) {
                        sh.extra = 1;
                        a.tau[m * a.half_n + c] =
                            (float)(a.z_harvest * sh.cur_rnorm / sqrt((double)a.k) * residual_scale(sh.cur_rnorm));
                        if ((c & 7) == 0) a.wide_tau[(m * a.half_n + c) >> 3] = wide_threshold(a, sh.cur_rnorm);
                    } else { sh.dep = 1; sh.hi = j + 1; }
                    a.ctl->stop[m] = 1;
                } else {
                    // a confirmed pick cannot be made: this recovery ends with j picks
                    a.cnt->stopped[m] = 1;
                    atomicOr(&a.cnt->status, (unsigned int)SGC_STATUS_DEPENDENT_COLUMN);
                    a.cnt->done[m] = j;
                    a.ctl->v[m] = j;
                    a.ctl->finished[m] = 1;
                    a.ctl->stop[m] = 1;
                }
            }
        }
        grid.sync();
    }
    if (mb < 2 && threadIdx.x == 0 && !fin[mb]) {
        if (mode == 0) {
            a.ctl->base[mb] = base[mb];
            a.ctl->hi[mb] = sh.hi < base[mb] ? base[mb] : sh.hi;
            a.ctl->extra[mb] = sh.extra;
            a.ctl->dep[mb] = sh.dep;
            a.ctl->list_exact[mb] = 0;    // only the best two candidates of every block reached the fp64 decision
        } else if (!a.ctl->finished[mb]) {
            a.cnt->done[mb] = a.ctl->v[mb];
            a.ctl->finished[mb] = 1;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// speculation on a short candidate list (at most kSmallList columns): block m runs the whole OMP of residual m
// by itself -- correlation of the list (warp = one column), pick, Algorithm 3 -- without any grid barrier.
// Same records as k_omp mode 0.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kOmpThreads, 1) k_spec_small(OmpArgs a) {
    extern __shared__ float2 sr[];
    __shared__ BookSmem sh;
    __shared__ Cand scored[kSmallList];                  // screen score of every candidate: the pick is exact within the list
    float* rs = reinterpret_cast<float*>(sr);            // the residual of this block's stream, fp32
    volatile SpecCtl* ctl = a.ctl;
    const int n_cand = ctl->n_cand;
    if (!ctl->round_active || ctl->fallback || n_cand > kSmallList || (n_cand <= kGramList && ctl->gram_ok)) return;
    const int m = blockIdx.x, k = a.k, s = a.s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int c = threadIdx.x; c < a.half_n; c += kOmpThreads) {
        a.rep_count[m * a.half_n + c] = 0u;
        a.tau[m * a.half_n + c] = __int_as_float(0x7f800000);
    }
    if (ctl->finished[m]) return;
    const int v0 = ctl->v[m];
    const uint32_t forced0 = ctl->forced[m];
    const int base = v0 + (forced0 != kNoColumn ? 1 : 0);
    const double rn0 = rebuild_prefix(a, sh, m, v0, a.r64 + (size_t)m * k, a.r32, a.x + (size_t)m * s);
    if (threadIdx.x == 0) {
        sh.cur_rnorm = rn0;
        if (v0 == 0) a.ctl->ynorm[m] = rn0;
        sh.hi = base; sh.extra = 0; sh.dep = 0; sh.stop = 0;
    }
    if (forced0 == kNoColumn) write_rt_row(a, m, 0, a.r64 + (size_t)m * k, rn0);
    __syncthreads();
    for (int j = v0; j < s; ++j) {
        const int c = j - base;                                       // -1 for the forced pick
        if (c >= a.half_n || sh.stop) break;
        const uint32_t forced = (j == v0) ? forced0 : kNoColumn;
        if (forced == kNoColumn) {
            // phase A inside the block: every candidate column against this residual
            __syncthreads();
            for (int row = threadIdx.x; row < k; row += kOmpThreads) rs[row] = a.r32[2 * row + m];
            if (threadIdx.x == 0) rs[k] = 0.0f;
            __syncthreads();
            for (int e = warp; e < n_cand; e += kOmpThreads / 32) {
                const uint32_t col = a.cand_list[e];
                bool taken = false;
                for (int q = lane; q < j; q += 32) taken |= (a.lam[(size_t)m * s + q] == col);
                if (__any_sync(0xffffffffu, taken)) {
                    if (lane == 0) { scored[e].score = -1.0f; scored[e].idx = kNoColumn; }
                    continue;
                }
                const ColKey key = column_key(a.seed_lo, a.seed_hi, col);
                float dot = 0.0f, n2 = 0.0f;
                uint32_t h = key.ck + (uint32_t)lane * key.mk;
                const uint32_t step = 32u * key.mk;
                for (int row = 2 * lane; row < k; row += 64) {         // one generated word = two rows
                    const float2 z = half2_bits_to_float2(z_pair_from_word(h));
                    h += step;
                    dot = __fmaf_rn(z.x, rs[row], dot);
                    n2 = __fmaf_rn(z.x, z.x, n2);
                    dot = __fmaf_rn(z.y, rs[row + 1], dot);
                    if (row + 1 < k) n2 = __fmaf_rn(z.y, z.y, n2);
                }
                dot = warp_sum(dot); n2 = warp_sum(n2);
                if (lane == 0) { scored[e].score = n2 > 0.0f ? dot * dot / n2 : 0.0f; scored[e].idx = col; }
            }
            __syncthreads();
        }
        const bool speculative = forced == kNoColumn;
        const int next = (c + 1 < a.half_n && j + 1 < s) ? c + 1 : -1;
        const int rc = book_pick(a, sh, m, j, forced, speculative ? c : -1, next, !speculative, scored, n_cand);
        if (threadIdx.x == 0) {
            if (rc == 0) {
                sh.hi = j + 1;
            } else if (speculative) {
                if (rc == 1) {
                    sh.extra = 1;
                    a.tau[m * a.half_n + c] =
                        (float)(a.z_harvest * sh.cur_rnorm / sqrt((double)k) * residual_scale(sh.cur_rnorm));
                } else { sh.dep = 1; sh.hi = j + 1; }
                sh.stop = 1;
            } else {
                a.cnt->stopped[m] = 1;
                atomicOr(&a.cnt->status, (unsigned int)SGC_STATUS_DEPENDENT_COLUMN);
                a.cnt->done[m] = j;
                a.ctl->v[m] = j;
                a.ctl->finished[m] = 1;
                sh.stop = 1;
            }
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        a.ctl->base[m] = base;
        a.ctl->hi[m] = sh.hi < base ? base : sh.hi;
        a.ctl->extra[m] = sh.extra;
        a.ctl->dep[m] = sh.dep;
        // every list member was scored, and all near-maximal ones decided in fp64 unless their buffer overflowed
        a.ctl->list_exact[m] = (a.cnt->status & (unsigned int)SGC_STATUS_CANDIDATE_OVERFLOW) ? 0 : 1;
    }
}

// ------------------------------------------------------------------------------------------------
// speculation on a very short candidate list (at most kGramList columns): Algorithm 3 as printed in Appendix B,
// i.e. on the Gram matrix G = Z_C^T Z_C of the list and the correlations p = Z_C^T r, which it updates without
// touching the k-dimensional residual.  Four kernels per round:
//   k_gram_prepare  the list's columns as binary16 (zlist) and p0 = Z_C^T y for both residuals
//   k_gram_matrix   G, only when the list has changed since G was computed (in a steady state: never)
//   k_omp_gram      block m: all picks of residual m, O(|C| * j) fp64 work per pick
//   k_spec_rows     one block per pick: the residual r_j = y - A_Lambda x_j it was made from (binary16 row of
//                   the screened batch, norm, threshold), and the picked column for the later kernels
// The records are those of k_omp mode 0 / k_spec_small.  Scores from G differ from scores computed against r_j
// only by fp64 rounding; should that ever flip a pick, the screening pass reports the better column as a
// challenger and k_resolve decides with the directly computed scores.
// ------------------------------------------------------------------------------------------------
constexpr int kGramThreads = 256;
constexpr int kGramSmemN = 96, kGramSmemS = 64;       // list length and support size up to which k_omp_gram stages G and F
constexpr size_t kGramSmemBytes = sizeof(double) * ((size_t)kGramSmemN * kGramSmemN + (size_t)kGramSmemS * kGramSmemS);

__device__ __forceinline__ bool gram_round(volatile SpecCtl* ctl) {
    return ctl->round_active && !ctl->fallback && ctl->gram_ok && ctl->n_cand <= kGramList;
}

__device__ double block_sum_256(double v, double* red) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    double t = (lane < kGramThreads / 32) ? red[lane] : 0.0;
    t = warp_sum(t);
    return t;
}

__global__ void __launch_bounds__(kGramThreads) k_gram_prepare(OmpArgs a) {
    volatile SpecCtl* ctl = a.ctl;
    if (!gram_round(ctl)) return;
    __shared__ double red[32];
    const int n = ctl->n_cand, b = blockIdx.x, k = a.k;
    if (b == 0 && threadIdx.x == 0) {
        a.ctl->gram_todo = (ctl->gram_version != ctl->list_version) ? 1 : 0;
        a.ctl->gram_pending = ctl->list_version;
    }
    if (b >= n) return;
    const ColKey key = column_key(a.seed_lo, a.seed_hi, a.cand_list[b]);
    uint32_t* dst = reinterpret_cast<uint32_t*>(a.zlist + (size_t)b * k);          // k is a multiple of 64 on this path
    double dm = 0.0, dv = 0.0;
    for (int p = threadIdx.x; p < (k >> 1); p += kGramThreads) {
        const uint32_t z2 = z_pair_from_word(key.ck + (uint32_t)p * key.mk);
        dst[p] = z2;
        const float2 z = half2_bits_to_float2(z2);
        dm += (double)z.x * a.y64[2 * p] + (double)z.y * a.y64[2 * p + 1];
        dv += (double)z.x * a.y64[k + 2 * p] + (double)z.y * a.y64[k + 2 * p + 1];
    }
    dm = block_sum_256(dm, red);
    dv = block_sum_256(dv, red);
    if (threadIdx.x == 0) { a.p0[b] = dm; a.p0[kGramList + b] = dv; }
}

__global__ void __launch_bounds__(kGramThreads) k_gram_matrix(OmpArgs a) {
    volatile SpecCtl* ctl = a.ctl;
    if (!gram_round(ctl) || !ctl->gram_todo) return;
    extern __shared__ uint4 colb[];                                   // column b of the list
    const int n = ctl->n_cand, b = blockIdx.x, k = a.k;
    if (b >= n) return;
    const uint4* src = reinterpret_cast<const uint4*>(a.zlist + (size_t)b * k);
    for (int v = threadIdx.x; v < (k >> 3); v += kGramThreads) colb[v] = src[v];
    __syncthreads();
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (int c = b + warp; c < n; c += kGramThreads / 32) {
        const uint4* pc = reinterpret_cast<const uint4*>(a.zlist + (size_t)c * k);
        double acc = 0.0;
#pragma unroll 4
        for (int v = lane; v < (k >> 3); v += 32) {
            const uint4 x = pc[v], y4 = colb[v];
            const uint32_t xw[4] = {x.x, x.y, x.z, x.w}, yw[4] = {y4.x, y4.y, y4.z, y4.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {                              // products of two binary16 numbers are exact in fp32
                const float2 fa = half2_bits_to_float2(xw[e]), fb = half2_bits_to_float2(yw[e]);
                acc += (double)(fa.x * fb.x);
                acc += (double)(fa.y * fb.y);
            }
        }
        acc = warp_sum(acc);
        if (lane == 0) { a.gram[(size_t)b * kGramList + c] = acc; a.gram[(size_t)c * kGramList + b] = acc; }
    }
}

__global__ void __launch_bounds__(kGramThreads, 1) k_omp_gram(OmpArgs a) {
    volatile SpecCtl* ctl = a.ctl;
    if (!gram_round(ctl)) return;
    __shared__ double red[32];
    __shared__ double p[kGramList], gdiag[kGramList];
    __shared__ double xs[kMaxS], gvec[kMaxS], cvec[kMaxS];
    __shared__ int li[kMaxS];
    __shared__ unsigned char taken[kGramList];
    __shared__ int found, best_i, stop, hi_s, extra_s, dep_s;
    __shared__ double wsc[kGramThreads / 32];
    __shared__ uint32_t wcol[kGramThreads / 32];
    __shared__ int widx[kGramThreads / 32];
    static_assert(kGramThreads == kGramList, "one thread per list member");
    const int m = blockIdx.x, s = a.s, n = ctl->n_cand, t = threadIdx.x;
    const int lane = t & 31, warp = t >> 5;
    if (m == 0 && t == 0 && ctl->gram_todo) a.ctl->gram_version = ctl->gram_pending;   // k_gram_matrix has run
    for (int c = t; c < a.half_n; c += kGramThreads) {
        a.rep_count[m * a.half_n + c] = 0u;
        a.tau[m * a.half_n + c] = __int_as_float(0x7f800000);
    }
    if (ctl->finished[m]) return;
    const int v0 = ctl->v[m];
    const uint32_t forced0 = ctl->forced[m];
    const int base = v0 + (forced0 != kNoColumn ? 1 : 0);
    const double sigma = a.sigma, sig2 = sigma * sigma;
    const double* G = a.gram;
    double* F = a.F + (size_t)m * s * s;
    // short lists and supports (the steady state) keep G and F in shared memory: every pick is a chain of a dozen dependent
    // reads of them, each an L2 round trip otherwise.  F is written through to global memory, where later kernels read it.
    extern __shared__ double gram_sm[];
    double* Gs = gram_sm;
    double* Fs = gram_sm + kGramSmemN * kGramSmemN;
    const bool g_sm = n <= kGramSmemN, f_sm = s <= kGramSmemS;
    if (g_sm) for (int e = t; e < n * n; e += kGramThreads) Gs[e] = G[(size_t)(e / n) * kGramList + (e % n)];
    if (f_sm) for (int e = t; e < s * s; e += kGramThreads) Fs[e] = F[e];
#define GRAM_G(r, c) (g_sm ? Gs[(r) * n + (c)] : G[(size_t)(r) * kGramList + (c)])
#define GRAM_F(r, c) (f_sm ? Fs[(r) * s + (c)] : F[(size_t)(r) * s + (c)])
    double* ac = a.acoef + (size_t)m * s;
    uint32_t* lam = a.lam + (size_t)m * s;
    const uint32_t my_col = t < n ? a.cand_list[t] : kNoColumn;
    // list positions of the verified picks (and of the forced one); a missing one sends the step to the direct kernels
    if (t == 0) { found = 0; stop = 0; hi_s = base; extra_s = 0; dep_s = 0; }
    taken[t] = 0;
    __syncthreads();
    int forced_li = -1;
    if (t < n) {
        gdiag[t] = G[(size_t)t * kGramList + t];          // (global: the staged copy is not yet synchronised)
        for (int l = 0; l < v0; ++l) if (lam[l] == my_col) { li[l] = t; taken[t] = 1; atomicAdd(&found, 1); }
        if (forced0 != kNoColumn && my_col == forced0) { li[v0] = t; atomicAdd(&found, 1); }
    }
    __syncthreads();
    if (found != base) {
        if (t == 0) a.ctl->gram_ok = 0;
        return;
    }
    if (forced0 != kNoColumn) forced_li = li[v0];
    for (int i = t; i < v0; i += kGramThreads) {
        double acc = 0.0;
        for (int l = i; l < v0; ++l) acc = acc + ac[l] * GRAM_F(i, l);
        xs[i] = acc;
        a.x[(size_t)m * s + i] = acc;
        a.pick_li[(size_t)m * s + i] = li[i];
    }
    __syncthreads();
    for (int j = v0; j < s; ++j) {
        const int c = j - base;                                         // -1 for the forced pick
        if (c >= a.half_n || stop) break;
        // correlations of the list with the current residual: p = p0 - sigma * G[:, Lambda] x   (G is symmetric)
        double pi = 0.0;
        if (t < n) {
            double acc = 0.0;
#pragma unroll 8
            for (int l = 0; l < j; ++l) acc += GRAM_G(li[l], t) * xs[l];
            pi = a.p0[m * kGramList + t] - sigma * acc;
            p[t] = pi;
        }
        int q;
        const bool forced = (j == v0) && forced0 != kNoColumn;
        if (forced) {
            q = forced_li;
            __syncthreads();
        } else {
            // "Select": argmax of p_i^2 / g_ii over the free list members, lowest column index on ties
            double sc = (t < n && !taken[t] && gdiag[t] > 0.0) ? pi * pi / gdiag[t] : -1.0;
            uint32_t col = sc >= 0.0 ? my_col : kNoColumn;
            int idx = t;
            for (int o = 16; o > 0; o >>= 1) {
                const double s2 = __shfl_xor_sync(0xffffffffu, sc, o);
                const uint32_t c2 = __shfl_xor_sync(0xffffffffu, col, o);
                const int i2 = __shfl_xor_sync(0xffffffffu, idx, o);
                if (s2 > sc || (s2 == sc && c2 < col)) { sc = s2; col = c2; idx = i2; }
            }
            __syncthreads();
            if (lane == 0) { wsc[warp] = sc; wcol[warp] = col; widx[warp] = idx; }
            __syncthreads();
            if (t == 0) {
                double bs = -1.0; uint32_t bc = kNoColumn; int bi = -1;
                for (int w = 0; w < kGramThreads / 32; ++w)
                    if (wsc[w] > bs || (wsc[w] == bs && wcol[w] < bc)) { bs = wsc[w]; bc = wcol[w]; bi = widx[w]; }
                best_i = bs >= 0.0 ? bi : -1;
            }
            __syncthreads();
            q = best_i;
            if (q < 0) {                                                // every list member is in the support already
                if (t == 0) { extra_s = 1; stop = 1; }
                __syncthreads();
                break;
            }
        }
        const double pq = p[q], gqq = gdiag[q];
        if (t == 0) {
            lam[j] = a.cand_list[q];
            li[j] = q;
            a.pick_li[(size_t)m * s + j] = q;
            if (!forced) a.pick_score[(size_t)m * s + j] = fabs(pq) / sqrt(gqq);
        }
        // Gram column of the pick restricted to the support, c = F^T g, pivot
        for (int l = t; l < j; l += kGramThreads) gvec[l] = sig2 * GRAM_G(li[l], q);
        __syncthreads();
        double csq = 0.0;
        for (int i0 = 0; i0 < j; i0 += kGramThreads / 16) {
            const int i = i0 + (t >> 4), sub = t & 15;
            double acc = 0.0;
            if (i < j)
                for (int l = sub; l <= i; l += 16) acc += GRAM_F(l, i) * gvec[l];
            for (int o = 8; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            if (i < j && sub == 0) { cvec[i] = acc; csq += acc * acc; }
        }
        csq = block_sum_256(csq, red);
        const double gnn = sig2 * gqq, piv = gnn - csq;
        if (!(piv > 1e-10 * gnn)) {
            // dependent column: a speculative one is screened and ends the recovery if confirmed; a forced one ends it now
            if (t == 0) {
                if (forced) {
                    a.cnt->stopped[m] = 1;
                    atomicOr(&a.cnt->status, (unsigned int)SGC_STATUS_DEPENDENT_COLUMN);
                    a.cnt->done[m] = j; a.ctl->v[m] = j; a.ctl->finished[m] = 1;
                } else { dep_s = 1; hi_s = j + 1; }
                stop = 1;
            }
            __syncthreads();
            break;
        }
        const double gamma = 1.0 / sqrt(piv);
        for (int i0 = 0; i0 < j; i0 += kGramThreads / 16) {
            const int i = i0 + (t >> 4), sub = t & 15;
            double acc = 0.0;
            if (i < j)
                for (int l = i + sub; l < j; l += 16) acc += GRAM_F(i, l) * cvec[l];
            for (int o = 8; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            if (i < j && sub == 0) { F[(size_t)i * s + j] = -gamma * acc; if (f_sm) Fs[i * s + j] = -gamma * acc; }
        }
        if (t == 0) { F[(size_t)j * s + j] = gamma; if (f_sm) Fs[j * s + j] = gamma; }
        const double aj = gamma * sigma * pq;
        __syncthreads();
        for (int i = t; i <= j; i += kGramThreads) {
            const double xo = (i < j) ? xs[i] : 0.0;
            const double xn = xo + aj * GRAM_F(i, j);
            xs[i] = xn;
            a.x[(size_t)m * s + i] = xn;
        }
        if (t == 0) {
            ac[j] = aj;
            taken[q] = 1;
            hi_s = j + 1;
            if (forced) { a.cnt->done[m] = j + 1; a.ctl->v[m] = j + 1; }
        }
        __syncthreads();
    }
    if (t == 0 && !a.ctl->finished[m]) {
        a.ctl->base[m] = base;
        a.ctl->hi[m] = hi_s < base ? base : hi_s;
        a.ctl->extra[m] = extra_s;
        a.ctl->dep[m] = dep_s;
        a.ctl->list_exact[m] = 1;
    }
}
#undef GRAM_G
#undef GRAM_F

// block (m, c): the state after j = base + c picks of residual m
__global__ void __launch_bounds__(kGramThreads) k_spec_rows(OmpArgs a) {
    volatile SpecCtl* ctl = a.ctl;
    if (!gram_round(ctl)) return;
    __shared__ double red[32];
    __shared__ double xs[kMaxS];
    __shared__ int li[kMaxS];
    const int per = a.half_n + 1;
    const int m = blockIdx.x / per, c = blockIdx.x % per, k = a.k, s = a.s, t = threadIdx.x;
    if (ctl->finished[m]) return;
    const int base = ctl->base[m], hi = ctl->hi[m], extra = ctl->extra[m], dep = ctl->dep[m];
    const int j = base + c;
    if (j > hi || (dep && j == hi)) return;               // a dependent pick leaves no new state behind
    const double* F = a.F + (size_t)m * s * s;
    const double* ac = a.acoef + (size_t)m * s;
    const double* y = a.y64 + (size_t)m * k;
    const int n_coef = j;
    for (int i = t; i < n_coef; i += kGramThreads) {
        double acc = 0.0;
        for (int l = i; l < n_coef; ++l) acc = acc + ac[l] * F[(size_t)i * s + l];
        xs[i] = acc;
        li[i] = a.pick_li[(size_t)m * s + i];
    }
    __syncthreads();
    // the picked column of pick j, for the kernels that rebuild residuals from the stored columns; the block of the first
    // state also stores the column of pick base - 1, which may be a prescribed one that no earlier round has stored
    if (c == 0 && base > 0) {
        const uint32_t* src = reinterpret_cast<const uint32_t*>(a.zlist + (size_t)li[base - 1] * k);
        uint32_t* dst = reinterpret_cast<uint32_t*>(a.zsel + ((size_t)m * s + base - 1) * k);
        for (int pr = t; pr < (k >> 1); pr += kGramThreads) dst[pr] = src[pr];
    }
    if (j < hi) {
        const uint32_t* src = reinterpret_cast<const uint32_t*>(a.zlist + (size_t)a.pick_li[(size_t)m * s + j] * k);
        uint32_t* dst = reinterpret_cast<uint32_t*>(a.zsel + ((size_t)m * s + j) * k);
        for (int pr = t; pr < (k >> 1); pr += kGramThreads) dst[pr] = src[pr];
    }
    const bool screened = c < a.half_n && (j < hi || (j == hi && extra));
    // r_j = y - sigma * Z_Lambda x_j in fp64 (kept for the resolve kernel) and its norm, then (for a screened state) the
    // scaled binary16 row
    const bool has_row = c < a.half_n;
    const int nrow = m * a.half_n + (has_row ? c : 0);
    double* keep = a.rhist + (size_t)nrow * k;
    double rn2 = 0.0;
    for (int row = t; row < k; row += kGramThreads) {
        double acc0 = 0.0, acc1 = 0.0;
        int l = 0;
#pragma unroll 4
        for (; l + 1 < n_coef; l += 2) {
            acc0 += xs[l] * (double)half_bits_to_float(a.zlist[(size_t)li[l] * k + row]);
            acc1 += xs[l + 1] * (double)half_bits_to_float(a.zlist[(size_t)li[l + 1] * k + row]);
        }
        if (l < n_coef) acc0 += xs[l] * (double)half_bits_to_float(a.zlist[(size_t)li[l] * k + row]);
        const double r1 = y[row] - a.sigma * (acc0 + acc1);
        if (has_row) keep[row] = r1;
        rn2 += r1 * r1;
    }
    rn2 = block_sum_256(rn2, red);
    const double rn = sqrt(rn2);
    if (t == 0) {
        if (j == 0) a.ctl->ynorm[m] = rn;
        else a.rnorm[(size_t)m * s + j - 1] = rn;            // ||r|| after pick j-1 (verified entries are rewritten with equal values)
    }
    if (!screened) return;
    const double sc = residual_scale(rn);
    uint16_t* dst = a.rt + (size_t)nrow * k;
    for (int row = t; row < k; row += kGramThreads) dst[row] = half_rn_bits(keep[row] * sc);    // each thread re-reads its own rows
    if (t == 0) {
        a.inv_scale[nrow] = (float)(1.0 / sc);
        const double unit = rn / sqrt((double)k);
        double tau;
        if (j < hi) {
            const double ps = a.pick_score[(size_t)m * s + j];
            tau = ps - screen_margin(rn, ps, k);
            if (tau > a.z_harvest * unit) tau = a.z_harvest * unit;
            if (tau < a.z_floor * unit) tau = a.z_floor * unit;
        } else {
            tau = a.z_harvest * unit;
        }
        a.tau[nrow] = (float)(tau * sc);
    }
}

// ------------------------------------------------------------------------------------------------
// resolve: confirm or refute the speculated picks with the reports of the screening pass
// ------------------------------------------------------------------------------------------------
struct ResolveArgs {
    OmpArgs o;
    const uint2* rep; int rep_cap;
    unsigned int* cand_bits; uint32_t* cand_list; double* rtmp;
    const uint32_t* kept_ring;
    int mini;                              // 1: the reports come from a list pass (two-level screening)
    const unsigned int* wide_count;
};

__device__ __forceinline__ bool in_support(const uint32_t* lam, int n, uint32_t col) {
    for (int q = 0; q < n; ++q) if (lam[q] == col) return true;
    return false;
}

// Collects into sh.cand_idx[start..] the reported columns of one residual that are not in the first n_sup picks,
// differ from `skip`, and score within `window` of the best such report, provided that best reaches `floor_sc`.
// Returns the number of candidates (start included), or -1 on overflow.
__device__ int collect_challengers(BookSmem& sh, const uint2* rep, unsigned int count, const uint32_t* lam, int n_sup,
                                   uint32_t skip, float floor_sc, float window, int start) {
    __syncthreads();
    if (threadIdx.x == 0) { sh.smax_bits = 0u; sh.n_cand = start; }
    __syncthreads();
    for (unsigned int e = threadIdx.x; e < count; e += kOmpThreads) {
        const uint2 rp = rep[e];
        const float sc = __uint_as_float(rp.y);
        if (sc >= floor_sc && rp.x != skip && !in_support(lam, n_sup, rp.x)) atomicMax(&sh.smax_bits, rp.y);   // scores are >= 0
    }
    __syncthreads();
    const unsigned int smax_bits = sh.smax_bits;
    if (smax_bits == 0u) return start;
    const float lo = __uint_as_float(smax_bits) - window;
    for (unsigned int e = threadIdx.x; e < count; e += kOmpThreads) {
        const uint2 rp = rep[e];
        const float sc = __uint_as_float(rp.y);
        if (sc >= floor_sc && sc >= lo && rp.x != skip && !in_support(lam, n_sup, rp.x)) {
            const int slot = atomicAdd(&sh.n_cand, 1);
            if (slot < kRescoreCap) sh.cand_idx[slot] = rp.x;
        }
    }
    __syncthreads();
    const int n = sh.n_cand;
    return n > kRescoreCap ? -1 : n;
}

// appends the columns `cols` that the list does not hold yet; n_s is the running length (shared memory)
__device__ void cand_append(const uint32_t* cols, int n_cols, int* n_s, uint32_t* cand_list, unsigned int* cand_bits) {
    for (int e = threadIdx.x; e < n_cols; e += blockDim.x) {
        const uint32_t col = cols[e];
        if (col == kNoColumn) continue;
        const unsigned int bit = 1u << (col & 31u);
        if (atomicOr(&cand_bits[col >> 5], bit) & bit) continue;
        const int slot = atomicAdd(n_s, 1);
        if (slot < kCandCap) cand_list[slot] = col;
        else atomicAnd(&cand_bits[col >> 5], ~bit);
    }
}

// Cuts the candidate list back to what is certain to matter when `incoming` more columns would let it outgrow kCandKeep:
// the ring of kept index sets and the picks made so far (columns harvested for earlier residuals have lost most of
// their value: the residual has moved on).
__device__ void make_room(const ResolveArgs& ra, int incoming) {
    volatile SpecCtl* ctl = ra.o.ctl;
    __shared__ int n_s;
    __syncthreads();
    const int n0 = ctl->n_cand;
    if (n0 + incoming <= kCandKeep) return;
    for (int e = threadIdx.x; e < n0; e += kOmpThreads) {
        const uint32_t col = ra.cand_list[e];
        atomicAnd(&ra.cand_bits[col >> 5], ~(1u << (col & 31u)));
    }
    if (threadIdx.x == 0) n_s = 0;
    __syncthreads();
    cand_append(ra.kept_ring, ctl->hist_count * ra.o.s, &n_s, ra.cand_list, ra.cand_bits);
    __syncthreads();
    for (int m = 0; m < 2; ++m) {
        cand_append(ra.o.lam + (size_t)m * ra.o.s, ctl->finished[m] ? ra.o.cnt->done[m] : ctl->hi[m], &n_s, ra.cand_list,
                    ra.cand_bits);
        __syncthreads();
    }
    if (threadIdx.x == 0) { ctl->n_cand = n_s < kCandCap ? n_s : kCandCap; ctl->list_version = ctl->list_version + 1; }
    __syncthreads();
}

// the reported columns of one residual that score at least `floor_sc` join the candidate list (the forced winner first)
__device__ void harvest(const ResolveArgs& ra, BookSmem& sh, const uint2* rep, unsigned int count, uint32_t first,
                        float floor_sc = 0.0f) {
    volatile SpecCtl* ctl = ra.o.ctl;
    __shared__ int n_s;
    __syncthreads();
    if (threadIdx.x == 0) n_s = ctl->n_cand;
    __syncthreads();
    if (first != kNoColumn) cand_append(&first, 1, &n_s, ra.cand_list, ra.cand_bits);
    __syncthreads();
    for (unsigned int e = threadIdx.x; e < count; e += kOmpThreads) {
        const uint2 rp = rep[e];
        if (__uint_as_float(rp.y) < floor_sc) continue;
        const uint32_t col = rp.x;
        const unsigned int bit = 1u << (col & 31u);
        if (atomicOr(&ra.cand_bits[col >> 5], bit) & bit) continue;
        const int slot = atomicAdd(&n_s, 1);
        if (slot < kCandCap) ra.cand_list[slot] = col;
        else atomicAnd(&ra.cand_bits[col >> 5], ~bit);
    }
    __syncthreads();
    if (threadIdx.x == 0) { ctl->n_cand = n_s < kCandCap ? n_s : kCandCap; ctl->list_version = ctl->list_version + 1; }
    __syncthreads();
}

// Full mode (reports of a pass over all d columns): confirms the speculated picks in order; the first refuted pick of a
// stream gets its true winner, which becomes final.  Mini mode (reports of a list pass over the wide lists): the same
// walk, but what it establishes is tentative -- tv / tforced tell the next speculation where to resume, while v, forced,
// the round count and everything a finished recovery records are left alone; the next full pass decides on all of it.
__global__ void __launch_bounds__(kOmpThreads, 1) k_resolve(ResolveArgs ra) {
    const OmpArgs& a = ra.o;
    __shared__ BookSmem sh;
    __shared__ int give_up, any_failed;
    volatile SpecCtl* ctl = a.ctl;
    const bool mini = ra.mini != 0;
    if (!ctl->round_active) return;
    if (ctl->fallback || ctl->pass_error) {
        // a wait inside the screening pass ran out: its reports are void, the remaining picks are made in lock-step
        if (threadIdx.x == 0) {
            if (ctl->pass_error) atomicOr(&a.cnt->status, (unsigned int)SGC_STATUS_TIMEOUT);
            ctl->fallback = 1; ctl->round_active = 0;
        }
        return;
    }
    if (mini) {
        if (ctl->mini_done || ctl->n_cand <= kSmallList) return;
        if (ra.wide_count[0] == 0u && ra.wide_count[1] == 0u) {
            if (threadIdx.x == 0) ctl->mini_done = 1;
            return;
        }
    }
    const int s = a.s;
    // Sweep: every block takes its share of the report lists (warp per residual) and notes which picks have a challenger
    // within the margin; the walk below only stops at those.  Nothing of the control block changes before the walk.
    {
        const int gw = blockIdx.x * (kOmpThreads / 32) + (threadIdx.x >> 5), nw = gridDim.x * (kOmpThreads / 32);
        for (int m = 0; m < 2; ++m) {
            if (ctl->finished[m]) continue;
            const int base = ctl->base[m], hi = ctl->hi[m];
            const int lo = (mini && ctl->tv[m] > base) ? ctl->tv[m] : base;
            for (int j = lo + gw; j < hi; j += nw) {
                const int n = m * a.half_n + (j - base);
                const unsigned int count = a.rep_count[n];
                bool hit = count > (unsigned int)ra.rep_cap;             // an overflowed list: the walk gives up there
                if (!hit) {
                    const uint32_t pick = a.lam[(size_t)m * s + j];
                    const double ps = a.pick_score[(size_t)m * s + j];
                    const double rn = j == 0 ? ctl->ynorm[m] : a.rnorm[(size_t)m * s + j - 1];
                    const float floor_sc = (float)ps - (float)screen_margin(rn, ps, a.k);
                    const bool skip_members = ctl->list_exact[m] != 0;
                    const uint2* list = ra.rep + (size_t)n * ra.rep_cap;
                    for (unsigned int e0 = threadIdx.x & 31; e0 < count; e0 += 8 * 32) {
                        uint2 rp8[8];                                    // eight reports in flight per lane
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            const unsigned int e = e0 + 32u * u;
                            rp8[u] = e < count ? list[e] : make_uint2(pick, 0u);
                        }
#pragma unroll
                        for (int u = 0; u < 8; ++u) {
                            const uint2 rp = rp8[u];
                            if (__uint_as_float(rp.y) < floor_sc || rp.x == pick) continue;
                            // a list member lost the exact comparison against the pick during the speculation (or is in the support)
                            if (skip_members && ((ra.cand_bits[rp.x >> 5] >> (rp.x & 31u)) & 1u)) continue;
                            if (!in_support(a.lam + (size_t)m * s, j, rp.x)) hit = true;
                        }
                    }
                    hit = __any_sync(0xffffffffu, hit);
                }
                if ((threadIdx.x & 31) == 0) a.ctl->contested[n] = hit ? 1 : 0;
            }
        }
    }
    // the block that finishes its share last walks the picks (ticket counter, nobody waits)
    __shared__ int last_block;
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) {
        const unsigned int ticket = atomicAdd(&a.ctl->resolve_ticket, 1u);
        last_block = ticket == gridDim.x - 1 ? 1 : 0;
        if (last_block) a.ctl->resolve_ticket = 0u;
    }
    __syncthreads();
    if (!last_block) return;
    __threadfence();
    __shared__ int contested[kPassMaxN];
    for (int n = threadIdx.x; n < kPassMaxN; n += kOmpThreads) contested[n] = ctl->contested[n];
    if (threadIdx.x == 0) {
        give_up = 0; any_failed = 0;
        if (mini) ctl->list_rounds = ctl->list_rounds + 1;
        else {
            ctl->rounds = ctl->rounds + 1;
            // width of the pass whose reports are being resolved (ctl->narrow still names it)
            ctl->pass_rows = ctl->pass_rows + (ctl->narrow ? a.rows_narrow : a.rows_wide);
        }
    }
    __syncthreads();
    for (int m = 0; m < 2; ++m) {
        if (ctl->finished[m]) continue;
        const int base = ctl->base[m], hi = ctl->hi[m], extra = ctl->extra[m], dep = ctl->dep[m];
        const uint32_t* lam = a.lam + (size_t)m * s;
        const int lo = (mini && ctl->tv[m] > base) ? ctl->tv[m] : base;
        int v = lo;
        uint32_t forced = kNoColumn;
        bool failed = false, bad = false;
        for (int j = lo; j < hi && !failed && !bad; ++j) {
            const int n = m * a.half_n + (j - base);
            if (!contested[n]) { v = j + 1; continue; }           // nobody comes close: the pick is the argmax
            const unsigned int count = a.rep_count[n];
            if (count > (unsigned int)ra.rep_cap) { bad = true; break; }
            const uint32_t pick = lam[j];
            const double ps = a.pick_score[(size_t)m * s + j];
            const double rn = j == 0 ? ctl->ynorm[m] : a.rnorm[(size_t)m * s + j - 1];
            const float margin = (float)screen_margin(rn, ps, a.k);
            if (threadIdx.x == 0) sh.cand_idx[0] = pick;
            const int nc = collect_challengers(sh, ra.rep + (size_t)n * ra.rep_cap, count, lam, j, pick, (float)ps - margin,
                                               2.0f * margin, 1);
            if (nc < 0) { bad = true; break; }
            if (nc == 1) { v = j + 1; continue; }                 // nobody comes close: the pick is the argmax
            rescore_candidates(a, sh, nc, a.rhist + (size_t)n * a.k);       // the residual this pick was made from
            if (sh.best_idx == pick) { v = j + 1; continue; }
            forced = sh.best_idx; v = j; failed = true;
            if (!mini && threadIdx.x == 0) ctl->refuted = ctl->refuted + 1;
            make_room(ra, (int)count + 1 + ((hi - j) / kLookAhead) * 1024);
            harvest(ra, sh, ra.rep + (size_t)n * ra.rep_cap, count, forced);
            // look ahead: the later residuals of this speculation are off the true path by a pick or a few, yet close
            // to it, so the columns that come near their picks are the likely picks of the next round
            for (int jj = j + kLookAhead; jj < hi; jj += kLookAhead) {
                const int nn = m * a.half_n + (jj - base);
                const unsigned int cc = a.rep_count[nn];
                if (cc > (unsigned int)ra.rep_cap) continue;
                harvest(ra, sh, ra.rep + (size_t)nn * ra.rep_cap, cc, kNoColumn,
                        (float)(kLookAheadShare * a.pick_score[(size_t)m * s + jj]));        // reports hold unscaled scores
            }

        }
        if (mini) {
            // tentative outcome only
            if (!failed && !bad) v = dep ? hi - 1 : hi;
            __syncthreads();
            if (threadIdx.x == 0) {
                ctl->tv[m] = v;
                ctl->tforced[m] = forced;
                if (failed) { any_failed = 1; ctl->list_refuted = ctl->list_refuted + 1; }
                if (bad) give_up = 1;
            }
            __syncthreads();
            continue;
        }
        if (!failed && !bad) {
            if (dep) {
                // the dependent pick was the true argmax: Algorithm 3 cannot extend the support, this recovery ends
                v = hi - 1;
                if (threadIdx.x == 0) {
                    a.cnt->stopped[m] = 1; a.cnt->done[m] = v; ctl->finished[m] = 1;
                    atomicOr(&a.cnt->status, (unsigned int)SGC_STATUS_DEPENDENT_COLUMN);
                }
            } else if (hi >= s) {
                v = s;
                if (threadIdx.x == 0) { a.cnt->done[m] = s; ctl->finished[m] = 1; }
            } else if (extra) {
                // residual screened without a pick: its best reported column is the next pick
                const int n = m * a.half_n + (hi - base);
                const unsigned int count = a.rep_count[n];
                const double rn = hi == 0 ? ctl->ynorm[m] : a.rnorm[(size_t)m * s + hi - 1];
                const float margin = (float)screen_margin(rn, 8.0 * rn / sqrt((double)a.k), a.k);    // scores near the noise maximum
                int nc = -1;
                if (count >= 1u && count <= (unsigned int)ra.rep_cap)
                    nc = collect_challengers(sh, ra.rep + (size_t)n * ra.rep_cap, count, lam, hi, kNoColumn, 0.0f, 2.0f * margin, 0);
                if (nc <= 0) bad = true;
                else {
                    rescore_candidates(a, sh, nc, a.rhist + (size_t)n * a.k);
                    forced = sh.best_idx; v = hi;
                    make_room(ra, (int)count + 1);
                    harvest(ra, sh, ra.rep + (size_t)n * ra.rep_cap, count, forced);
                }
            } else {
                v = hi;                                           // the pass had no room for more residuals
            }
        }
        __syncthreads();
        if (threadIdx.x == 0) {
            ctl->v[m] = v;
            ctl->forced[m] = forced;
            ctl->tv[m] = v;
            ctl->tforced[m] = kNoColumn;
            if (bad) give_up = 1;
        }
        __syncthreads();
    }
    if (mini) {
        // list passes rest until the next full pass once every screened window is full and nothing in it was refuted, or
        // when the reports overflowed (the full pass has to sort that out)
        if (threadIdx.x == 0 && give_up) ctl->mini_done = 1;
        if (threadIdx.x == 0 && !any_failed && !give_up) {
            bool full = true;
            for (int m = 0; m < 2; ++m) {
                if (ctl->finished[m]) continue;
                const int base = ctl->base[m], hi = ctl->hi[m];
                if (!(hi - base >= a.half_n || hi >= s || ctl->dep[m] || ctl->extra[m])) full = false;
            }
            if (full) ctl->mini_done = 1;
        }
        return;
    }
    if (threadIdx.x == 0) {
        ctl->mini_done = 0;
        if (give_up) {
            ctl->fallback = 1; ctl->round_active = 0;
            atomicOr(&a.cnt->status, (unsigned int)SGC_STATUS_CANDIDATE_OVERFLOW);
        } else if (ctl->finished[0] && ctl->finished[1]) {
            ctl->round_active = 0;
        }
        ctl->narrow = (ctl->finished[1] && !ctl->finished[0]) ? 1 : 0;     // the rows of a pass start with the first stream's
        const int r = ctl->rounds - 1;
        if (r >= 0 && r < kMaxRounds) { ctl->trace[r][0] = ctl->v[0]; ctl->trace[r][1] = ctl->v[1]; ctl->trace[r][2] = ctl->n_cand; }
    }
}

// start of the recovery of one step
__global__ void k_spec_init(SpecCtl* ctl, int speculate, float* wide_tau, int shared) {
    if (threadIdx.x == 0) {
        ctl->tv[0] = ctl->tv[1] = 0;
        ctl->tforced[0] = ctl->tforced[1] = kNoColumn;
        ctl->mini_done = 0; ctl->list_rounds = 0; ctl->list_refuted = 0; ctl->refuted = 0;
        // no wide list unless a long-list speculation asks for one
        if (wide_tau != nullptr) for (int g = 0; g < kPassMaxN / 8; ++g) wide_tau[g] = __int_as_float(0x7f800000);
        ctl->round_active = speculate; ctl->fallback = speculate ? 0 : 1;
        ctl->v[0] = ctl->v[1] = 0;
        ctl->forced[0] = ctl->forced[1] = kNoColumn;
        ctl->finished[0] = 0;
        ctl->finished[1] = shared ? 1 : 0;          // shared support: the second stream makes no picks of its own
        ctl->narrow = shared ? 1 : 0;
        ctl->stop[0] = ctl->stop[1] = 0;
        ctl->rounds = 0; ctl->pass_error = 0; ctl->pass_rows = 0;
        for (int r = 0; r < kMaxRounds; ++r) ctl->trace[r][0] = ctl->trace[r][1] = ctl->trace[r][2] = 0;
        ctl->gram_ok = 1;
        if (ctl->list_version == 0) ctl->list_version = 1;      // a fresh state: no Gram matrix yet
    }
}

// start of the step, after Sparsify_s: M^ and V^ are combinations of the columns kept in this and in earlier steps
// (Eq. 4, 5), so the indices just kept are candidates, and they enter the ring of recent index sets
__global__ void __launch_bounds__(kOmpThreads, 1)
k_cand_begin(SpecCtl* ctl, const uint32_t* sel_idx, int s, uint32_t* kept_ring, int hist_slots, uint32_t* cand_list,
             unsigned int* cand_bits) {
    __shared__ int n_s;
    const int n0 = ctl->n_cand;
    const int slot = ctl->hist_next % hist_slots;
    if (threadIdx.x == 0) n_s = n0;
    for (int e = threadIdx.x; e < s; e += kOmpThreads) kept_ring[(size_t)slot * s + e] = sel_idx[e];
    __syncthreads();
    cand_append(sel_idx, s, &n_s, cand_list, cand_bits);
    __syncthreads();
    if (threadIdx.x == 0) {
        const int n_new = n_s < kCandCap ? n_s : kCandCap;
        if (n_new != n0) { ctl->n_cand = n_new; ctl->list_version = ctl->list_version + 1; }
        ctl->hist_next = (slot + 1) % hist_slots;
        if (ctl->hist_count < hist_slots) ctl->hist_count = ctl->hist_count + 1;
    }
}

// end of the step: the supports found stay (or become) candidates of the next step
__global__ void __launch_bounds__(kOmpThreads, 1)
k_cand_update(SpecCtl* ctl, const Counters* cnt, const uint32_t* lam, int s, uint32_t* cand_list, unsigned int* cand_bits,
              const uint32_t* kept_ring, int* rounds_out) {
    __shared__ int n_s;
    // how many rounds this step took (the enqueued rounds if even they were not enough): sizes the next step's launches
    // bit 8: a list pass refuted a pick (the wide lists earned their keep); bit 9: a full pass refuted a pick
    if (threadIdx.x == 0)
        *rounds_out = (ctl->fallback ? kMaxRounds : ctl->rounds) | (ctl->list_refuted > 0 ? 256 : 0) | (ctl->refuted > 0 ? 512 : 0);
    int n = ctl->n_cand;
    // rebuild from the supports and the ring of kept index sets when the list has outgrown its bound, or when it holds
    // far more than those although a single round confirmed every pick (harvested columns of an earlier cold start)
    const int n_hist = ctl->hist_count * s;
    const bool rebuild = n > kCandKeep || (ctl->rounds <= 1 && !ctl->fallback && n > 4 * s + n_hist);
    if (rebuild) {
        for (int e = threadIdx.x; e < n; e += kOmpThreads) {
            const uint32_t col = cand_list[e];
            atomicAnd(&cand_bits[col >> 5], ~(1u << (col & 31u)));
        }
        n = 0;
    }
    if (threadIdx.x == 0) n_s = n;
    __syncthreads();
    for (int m = 0; m < 2; ++m) {
        cand_append(lam + (size_t)m * s, cnt->done[m] < s ? cnt->done[m] : s, &n_s, cand_list, cand_bits);
        __syncthreads();
    }
    if (rebuild) cand_append(kept_ring, n_hist, &n_s, cand_list, cand_bits);
    __syncthreads();
    if (threadIdx.x == 0) {
        const int n_new = n_s < kCandCap ? n_s : kCandCap;
        if (n_new != ctl->n_cand || n == 0) ctl->list_version = ctl->list_version + 1;     // rebuilt or extended
        ctl->n_cand = n_new;
    }
}

// ------------------------------------------------------------------------------------------------
// Opt-in variant of the recovery (remark after Eq. (8): both recoveries have their non-zeros at the same positions).
// Runs after the recoveries of the step, one block.
//   tol > 0: each recovery is cut after the first pick that left ||r|| <= tol ||y||.  OMP is greedy, so the picks before
//            the cut are those an early-stopping run makes, and the leading block of the inverse Cholesky factor F with
//            the leading coefficients a gives the least-squares fit on them: x = F_j a_j.
//   shared:  the second stream made no picks; x^V = F F^T A_Lambda^T V^ is the least-squares fit of V^ on the support
//            of the first stream (F F^T = (A_Lambda^T A_Lambda)^-1, Appendix B).
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kOmpThreads, 1) k_variant_tail(OmpArgs a, int shared, double tol) {
    __shared__ double red[32];
    __shared__ double u[kMaxS], av[kMaxS];
    __shared__ int cut;
    const int k = a.k, s = a.s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    if (tol > 0.0) {
        for (int m = 0; m < (shared ? 1 : 2); ++m) {
            const double* y = a.y64 + (size_t)m * k;
            double yn2 = 0.0;
            for (int row = threadIdx.x; row < k; row += kOmpThreads) yn2 += y[row] * y[row];
            yn2 = block_sum(yn2, red);
            const int done = a.cnt->done[m];
            if (threadIdx.x == 0) {
                const double bound = tol * sqrt(yn2);
                cut = done;
                for (int j = 0; j < done; ++j) if (a.rnorm[(size_t)m * s + j] <= bound) { cut = j + 1; break; }
            }
            __syncthreads();
            const int n = cut;
            if (n < done) {
                const double* F = a.F + (size_t)m * s * s;
                const double* ac = a.acoef + (size_t)m * s;
                for (int i = threadIdx.x; i < s; i += kOmpThreads) {
                    double acc = 0.0;
                    for (int l = i; l < n; ++l) acc = acc + ac[l] * F[(size_t)i * s + l];
                    a.x[(size_t)m * s + i] = acc;                  // 0 for i >= n
                    if (i >= n) a.rnorm[(size_t)m * s + i] = 0.0;
                }
                if (threadIdx.x == 0) a.cnt->done[m] = n;
            }
            __syncthreads();
        }
    }
    if (shared) {
        const int n = a.cnt->done[0];
        const double* y = a.y64 + (size_t)k;                       // V^
        const double* F = a.F;                                     // factor of the first stream's support
        for (int l = warp; l < n; l += kOmpThreads / 32) {
            const uint16_t* zl = a.zsel + (size_t)l * k;
            double acc = 0.0;
            for (int row = lane; row < k; row += 32) acc += (double)half_bits_to_float(zl[row]) * y[row];
            acc = warp_sum(acc);
            if (lane == 0) u[l] = a.sigma * acc;
        }
        __syncthreads();
        for (int i = threadIdx.x; i < n; i += kOmpThreads) {
            double acc = 0.0;
            for (int l = 0; l <= i; ++l) acc += F[(size_t)l * s + i] * u[l];
            av[i] = acc;
        }
        __syncthreads();
        for (int i = threadIdx.x; i < s; i += kOmpThreads) {
            double acc = 0.0;
            for (int l = i; l < n; ++l) acc += F[(size_t)i * s + l] * av[l];
            a.x[(size_t)s + i] = acc;                              // 0 for i >= n
            a.lam[(size_t)s + i] = i < n ? a.lam[i] : kNoColumn;
            a.rnorm[(size_t)s + i] = 0.0;
        }
        if (threadIdx.x == 0) a.cnt->done[1] = n;
    }
}

// ------------------------------------------------------------------------------------------------
// a5: combine + scatter
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(kBookThreads, 1)
k_scatter(int s, uint32_t* lam, double* x, Counters* __restrict__ cnt, float* __restrict__ W,
          uint32_t* __restrict__ upd_idx, double* __restrict__ upd_val, double alpha, double eps, double lr) {
    __shared__ uint32_t vidx[kMaxS];
    __shared__ double vval[kMaxS];
    __shared__ int flag[kMaxS];
    __shared__ int n_mis, n_neg;
    const int nM = cnt->done[0], nV = cnt->done[1];
    if (threadIdx.x == 0) { n_mis = 0; n_neg = 0; }
    // unpicked slots read as "none"
    for (int i = threadIdx.x; i < s; i += kBookThreads) {
        if (i >= nM) { lam[i] = 0xFFFFFFFFu; x[i] = 0.0; }
        if (i >= nV) { lam[s + i] = 0xFFFFFFFFu; x[s + i] = 0.0; }
    }
    __syncthreads();
    const int a = threadIdx.x;
    flag[a] = 0;
    if (a < nM) {
        const uint32_t li = lam[a];
        int hit = -1;
        for (int b = 0; b < nV; ++b) if (lam[s + b] == li) { hit = b; break; }
        if (hit < 0) atomicAdd(&n_mis, 1);
        else {
            const double xv = x[s + hit];
            if (!(xv > 0.0)) atomicAdd(&n_neg, 1);
            else {
                const double N = alpha * x[a] / (sqrt(xv) + eps);
                vidx[a] = li; vval[a] = lr * N; flag[a] = 1;
            }
        }
    }
    __syncthreads();
    int n_valid = 0;
    if (a < nM && flag[a]) {
        int rank = 0;
        for (int b = 0; b < nM; ++b) if (flag[b] && vidx[b] < vidx[a]) ++rank;
        upd_idx[rank] = vidx[a];
        upd_val[rank] = vval[a];
        W[vidx[a]] = (float)((double)W[vidx[a]] - vval[a]);
    }
    if (threadIdx.x == 0) {
        for (int b = 0; b < nM; ++b) n_valid += flag[b];
        cnt->n_upd = n_valid; cnt->mismatch = n_mis; cnt->negv = n_neg;
        unsigned int bits = 0;
        if (n_mis > 0 || nM != nV) bits |= (unsigned int)SGC_STATUS_SUPPORT_MISMATCH;
        if (n_neg > 0) bits |= (unsigned int)SGC_STATUS_NEGATIVE_V;
        if (bits) atomicOr(&cnt->status, bits);
    }
}

// z with d * P(|N(0,1)| > z) = target (bisection on erfc)
double normal_tail_threshold_impl(double d, double target) {
    double p = target / d;
    if (p > 0.5) p = 0.5;
    double lo = 0.0, hi = 12.0;
    for (int i = 0; i < 80; ++i) {
        const double mid = 0.5 * (lo + hi);
        if (erfc(mid / sqrt(2.0)) > p) lo = mid; else hi = mid;
    }
    return 0.5 * (lo + hi);
}

OmpArgs make_args(const sgc_state* st) {
    OmpArgs a;
    a.seed_lo = (uint32_t)(st->seed & 0xFFFFFFFFu); a.seed_hi = (uint32_t)(st->seed >> 32);
    a.d = (unsigned long long)st->d; a.k = st->k; a.s = st->s;
    const unsigned long long tile_cols = (unsigned long long)kOmpThreads * kCorrCols;
    a.num_tiles = (unsigned int)(((unsigned long long)st->d + tile_cols - 1) / tile_cols);
    a.sigma = (double)(float)(1.0 / sqrt((double)st->k));
    a.half_n = st->pass_n / 2;
    a.rows_wide = st->pass_n; a.rows_narrow = st->pass_n_half;
    a.z_harvest = st->z_harvest; a.z_floor = st->z_floor;
    a.corr_cand = st->corr_cand; a.y64 = st->y64; a.r64 = st->r64; a.r32 = reinterpret_cast<float*>(st->r32);
    a.zsel = st->zsel; a.lam = st->lam; a.F = st->F; a.acoef = st->acoef; a.x = st->x; a.rnorm = st->rnorm;
    a.cnt = st->cnt; a.ctl = st->ctl;
    a.rt = st->rt; a.tau = st->tau; a.inv_scale = st->inv_scale; a.rep_count = st->rep_count; a.pick_score = st->pick_score;
    a.rhist = st->rhist;
    a.cand_list = st->cand_list;
    a.zlist = st->zlist; a.gram = st->gram; a.p0 = st->p0; a.pick_li = st->pick_li;
    a.wide_tau = st->wide_tau; a.z_wide = st->z_wide; a.wide_count = nullptr; a.wide_bits = st->wide_bits; a.mini = 0;
    a.depth = 1 << 30;
    return a;
}

cudaError_t launch_omp(sgc_state* st, const OmpArgs& a, int mode, cudaStream_t stream) {
    OmpArgs args = a;
    int m = mode;
    void* params[2] = {&args, &m};
    return cudaLaunchCooperativeKernel((const void*)k_omp, dim3((unsigned int)st->corr_grid), dim3(kOmpThreads), params,
                                       (size_t)st->corr_smem, stream);
}

}  // namespace

double normal_tail_threshold(double d, double target) { return normal_tail_threshold_impl(d, target); }

cudaError_t configure_recover(sgc_state* st) {
    const size_t smem = ((size_t)st->k + 1) * sizeof(float2);
    // the opt-in shared-memory limit belongs to the kernel, not to a state: it is set to what the largest supported k
    // needs, so that states of any size can live side by side on a device
    constexpr size_t smem_max = ((size_t)kMaxK + 1) * sizeof(float2);
    static_assert(smem_max + 48 * 1024 <= 227 * 1024, "k_omp: dynamic plus static shared memory must fit one SM");
    static_assert((size_t)kMaxK * 2 <= 48 * 1024, "k_gram_matrix stages one binary16 column without opting in");
    cudaError_t e = cudaFuncSetAttribute(k_omp, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max);
    if (e != cudaSuccess) return e;
    int occ = 0;
    e = cudaFuncSetAttribute(k_spec_small, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem_max);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(k_omp_gram, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kGramSmemBytes);
    if (e != cudaSuccess) return e;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_omp, kOmpThreads, smem);
    if (e != cudaSuccess) return e;
    if (occ < 1) return cudaErrorInvalidConfiguration;
    int coop = 0;
    e = cudaDeviceGetAttribute(&coop, cudaDevAttrCooperativeLaunch, st->device);
    if (e != cudaSuccess) return e;
    if (!coop) return cudaErrorNotSupported;
    st->corr_grid = st->sm_count * occ;                  // every block resident: required by the grid barrier
    if (st->corr_grid < 2) return cudaErrorInvalidConfiguration;
    st->corr_smem = (int)smem;
    // speculative recovery: needs whole 64-row chunks of A for the tensor-core pass
    st->spec_ok = (st->k % 64 == 0);
    int half = st->s < 128 ? st->s : 128;
    half = (half + 15) / 16 * 16;
    st->pass_n = 2 * half;
    st->z_harvest = normal_tail_threshold_impl((double)st->d, 3072.0);
    st->z_floor = normal_tail_threshold_impl((double)st->d, 6144.0);
    st->z_wide = normal_tail_threshold_impl((double)st->d, 100000.0);
    if (st->spec_ok) {
        e = pass_configure(kPassMaxN);
        if (e != cudaSuccess) return e;
    }
    return cudaSuccess;
}

cudaError_t finish_recover_setup(sgc_state* st) {
    if (!st->spec_ok) return cudaSuccess;
    cudaError_t e = cudaSuccess;
    for (int g = 1; g <= kPassMaxN / st->pass_n && e == cudaSuccess; ++g)      // one map per number of states in a batch
        e = pass_encode_map(st->tmap[g - 1], st->rt, g * st->pass_n, st->k);
    if (e != cudaSuccess) return e;
    // shared-support variant: only the first stream has residuals to screen, a pass half as wide does
    st->pass_n_half = ((st->pass_n / 2 + 31) / 32) * 32;
    e = pass_encode_map(st->tmap_half, st->rt, st->pass_n_half, st->k);
    if (e != cudaSuccess) return e;
    e = launch_inv_norms(st->seed, (uint64_t)st->d, st->k, st->inv_norm, 0);     // column norms: a property of (seed, k)
    if (e != cudaSuccess) return e;
    return cudaDeviceSynchronize();
}

// Recovery (a4 + a5) of n states that share (d, k, s, seed), hence A.  The states' screened residuals are laid out side by
// side in the screening buffers of the first state of each batch (a batch = as many states as fit kPassMaxN columns), so
// one pass over A serves a whole batch; everything else runs per state.  n = 1 is the plain sgc_step.
static cudaError_t recover_batches(sgc_state* const* sts, float* const* weights, int n, cudaStream_t stream, int* launches) {
    sgc_state* st0 = sts[0];
    bool speculate = true;
    for (int i = 0; i < n; ++i)
        speculate = speculate && sts[i]->spec_ok && sts[i]->spec_ready &&
                    (sts[i]->mode == 2 || (sts[i]->mode == 0 && sts[i]->d >= (1ll << 16)));
    const int per_batch = speculate ? kPassMaxN / st0->pass_n : 1;
    std::vector<OmpArgs> args((size_t)n);
    cudaError_t e = cudaSuccess;
    int n_rounds = 0;
    int mini_rounds = 0;          // rounds that get list passes: the likely ones; the spare rounds behind them stay cheap to enqueue
    for (int i = 0; i < n; ++i) {
        sgc_state* st = sts[i];
        sgc_state* lead = sts[i - i % per_batch];
        const int slot = i % per_batch;
        OmpArgs a = make_args(st);
        // this state's slice of the batch's screening buffers
        a.rt = lead->rt + (size_t)slot * st->pass_n * st->k;
        a.tau = lead->tau + slot * st->pass_n;
        a.inv_scale = lead->inv_scale + slot * st->pass_n;
        a.rep_count = lead->rep_count + slot * st->pass_n;
        args[i] = a;
        {
            PhaseTimer timer(st, stream, kPhaseBook, 1);
            k_spec_init<<<1, 32, 0, stream>>>(st->ctl, speculate ? 1 : 0, st->wide_tau, st->shared_support);
            *launches += 1;
            if (speculate) {
                k_cand_begin<<<1, kOmpThreads, 0, stream>>>(st->ctl, st->sel_idx, st->s, st->kept_ring, st->hist_slots,
                                                            st->cand_list, st->cand_bits);
                *launches += 1;
            }
        }
        // rounds to enqueue: twice what the last finished step needed plus slack (read from pinned memory without
        // synchronising; a stale value only changes how much is enqueued); what they leave open is done in lock-step
        const int hint = speculate ? *reinterpret_cast<volatile int*>(st->h_rounds) : 0;
        const int last = hint & 255;
        int want = last <= 0 ? 8 : 2 * last + 3;
        if (last > 0 && last + 2 > mini_rounds) mini_rounds = last + 2;
        if (last <= 0) mini_rounds = kMaxRounds;
        if (st->max_rounds > 0 && want > st->max_rounds) want = st->max_rounds;
        if (want > n_rounds) n_rounds = want;
        // two-level screening pays where steps need several full passes (recovery picks columns outside the kept sets);
        // it is dropped again when a step needed one pass and its list passes refuted nothing
        if (last >= 3) st->two_level = true;
        else if (last == 1 && !(hint & 256)) st->two_level = false;
    }
    if (n_rounds > kMaxRounds) n_rounds = kMaxRounds;
    const bool two_level = speculate && n == 1 && st0->two_level;
    // A state whose two streams fill a pass of more than kPassFastRows rows, and whose last step had a pick refuted: the
    // refuted stream needs several rounds anyway, and the rows of a speculation beyond its first refuted pick are wasted.
    // Such a step screens half as many residuals per stream and round, in the pass of half the width at half the cost;
    // the stream that is confirmed without contest rides along in two rounds instead of one.
    const bool compact = speculate && n == 1 && st0->pass_n > kPassFastRows && st0->pass_n_half <= kPassFastRows &&
                         (*reinterpret_cast<volatile int*>(st0->h_rounds) & 512) != 0;
    if (compact) {
        args[0].half_n = st0->pass_n_half / 2;
        args[0].rows_wide = args[0].rows_narrow = st0->pass_n_half;
        n_rounds = n_rounds + 1 < kMaxRounds ? n_rounds + 1 : kMaxRounds;
        if (st0->max_rounds > 0 && n_rounds > st0->max_rounds) n_rounds = st0->max_rounds;
    }
    PassWide wide;
    if (two_level) {
        args[0].wide_count = st0->wide_count;
        wide.tau = st0->wide_tau; wide.list = st0->wide_list; wide.count = st0->wide_count; wide.bits = st0->wide_bits;
        wide.cap = kWideCap; wide.half_n = args[0].half_n; wide.ctl = st0->ctl; wide.list_pass = false;
    }
    if (speculate) {
        for (int round = 0; round < n_rounds && e == cudaSuccess; ++round) {
            // list passes first: speculate a few picks ahead, screen the wide lists only, keep what they confirm as
            // tentative picks; every kernel of this loop returns at once when there is nothing (more) to do
            for (int mini = 0; two_level && round < mini_rounds && mini < kMiniRounds && e == cudaSuccess; ++mini) {
                sgc_state* st = st0;
                {
                    PhaseTimer timer(st, stream, kPhaseCorr, 1);
                    OmpArgs am = args[0];
                    am.mini = 1; am.depth = kMiniDepth;
                    e = launch_omp(st, am, 0, stream);
                    *launches += 1;
                }
                if (e != cudaSuccess) break;
                {
                    PhaseTimer timer(st, stream, kPhasePass, 1);
                    const int* gates[kPassMaxBatch] = {&st->ctl->round_active};
                    int* errors[kPassMaxBatch] = {&st->ctl->pass_error};
                    PassWide lp = wide;
                    lp.list_pass = true;
                    const bool two_widths = !compact && st->pass_n_half < st->pass_n;   // the width that ctl->narrow names runs
                    if (compact)
                        e = launch_pass(st->tmap_half, st->seed, (uint64_t)st->d, st->k, st->pass_n_half, st->tau, st->inv_scale,
                                        st->inv_norm, st->rep_count, st->rep, kRepCap, gates, errors, st->sm_count, stream, &lp,
                                        nullptr, 0, st->wait_limit_ns);
                    else
                    e = launch_pass(st->tmap[0], st->seed, (uint64_t)st->d, st->k, st->pass_n, st->tau, st->inv_scale,
                                    st->inv_norm, st->rep_count, st->rep, kRepCap, gates, errors, st->sm_count, stream, &lp,
                                    two_widths ? &st->ctl->narrow : nullptr, 0, st->wait_limit_ns);
                    if (two_widths && e == cudaSuccess) {
                        e = launch_pass(st->tmap_half, st->seed, (uint64_t)st->d, st->k, st->pass_n_half, st->tau,
                                        st->inv_scale, st->inv_norm, st->rep_count, st->rep, kRepCap, gates, errors,
                                        st->sm_count, stream, &lp, &st->ctl->narrow, 1, st->wait_limit_ns);
                        *launches += 1;
                    }
                    *launches += 1;
                }
                if (e != cudaSuccess) break;
                ResolveArgs ra;
                ra.o = args[0];
                ra.rep = st->rep; ra.rep_cap = kRepCap; ra.cand_bits = st->cand_bits; ra.cand_list = st->cand_list;
                ra.rtmp = st->rtmp; ra.kept_ring = st->kept_ring; ra.mini = 1; ra.wide_count = st->wide_count;
                PhaseTimer timer(st, stream, kPhaseBook, 1);
                k_resolve<<<kResolveBlocks, kOmpThreads, 0, stream>>>(ra);
                *launches += 1;
            }
            for (int b0 = 0; b0 < n && e == cudaSuccess; b0 += per_batch) {
                const int nb = n - b0 < per_batch ? n - b0 : per_batch;
                for (int i = b0; i < b0 + nb && e == cudaSuccess; ++i) {
                    sgc_state* st = sts[i];
                    const OmpArgs& a = args[i];
                    PhaseTimer timer(st, stream, kPhaseCorr, 6);
                    k_gram_prepare<<<kGramList, kGramThreads, 0, stream>>>(a);       // very short list: Gram-matrix OMP
                    k_gram_matrix<<<kGramList, kGramThreads, (size_t)st->k * 2, stream>>>(a);
                    k_omp_gram<<<2, kGramThreads, kGramSmemBytes, stream>>>(a);
                    k_spec_rows<<<2 * (a.half_n + 1), kGramThreads, 0, stream>>>(a);
                    k_spec_small<<<2, kOmpThreads, st->corr_smem, stream>>>(a);      // short candidate list
                    e = launch_omp(st, a, 0, stream);                                // long candidate list
                    *launches += 6;
                }
                if (e != cudaSuccess) break;
                sgc_state* lead = sts[b0];
                {
                    PhaseTimer timer(lead, stream, kPhasePass, 1);
                    const int* gates[kPassMaxBatch];
                    int* errors[kPassMaxBatch];
                    for (int q = 0; q < kPassMaxBatch; ++q) {
                        gates[q] = q < nb ? &sts[b0 + q]->ctl->round_active : nullptr;
                        errors[q] = q < nb ? &sts[b0 + q]->ctl->pass_error : nullptr;
                    }
                    // a state on its own: once only its first stream has residuals left (the second recovery is complete, or
                    // the shared-support variant is on), the pass half as wide serves the round; ctl->narrow names the width
                    const bool two_widths = n == 1 && !compact && lead->pass_n_half < lead->pass_n;
                    if (compact)
                        e = launch_pass(lead->tmap_half, lead->seed, (uint64_t)lead->d, lead->k, lead->pass_n_half, lead->tau,
                                        lead->inv_scale, lead->inv_norm, lead->rep_count, lead->rep, kRepCap, gates, errors,
                                        lead->sm_count, stream, two_level ? &wide : nullptr, nullptr, 0, lead->wait_limit_ns);
                    else
                    e = launch_pass(lead->tmap[nb - 1], lead->seed, (uint64_t)lead->d, lead->k, nb * lead->pass_n, lead->tau,
                                    lead->inv_scale, lead->inv_norm, lead->rep_count, lead->rep, kRepCap, gates, errors,
                                    lead->sm_count, stream, two_level ? &wide : nullptr,
                                    two_widths ? &lead->ctl->narrow : nullptr, 0, lead->wait_limit_ns);
                    if (two_widths && e == cudaSuccess) {
                        e = launch_pass(lead->tmap_half, lead->seed, (uint64_t)lead->d, lead->k, lead->pass_n_half, lead->tau,
                                        lead->inv_scale, lead->inv_norm, lead->rep_count, lead->rep, kRepCap, gates, errors,
                                        lead->sm_count, stream, two_level ? &wide : nullptr, &lead->ctl->narrow, 1,
                                        lead->wait_limit_ns);
                        *launches += 1;
                    }
                    *launches += 1;
                }
                for (int i = b0; i < b0 + nb && e == cudaSuccess; ++i) {
                    sgc_state* st = sts[i];
                    ResolveArgs ra;
                    ra.o = args[i];
                    ra.rep = lead->rep + (size_t)(i - b0) * st->pass_n * kRepCap;
                    ra.rep_cap = kRepCap; ra.cand_bits = st->cand_bits; ra.cand_list = st->cand_list; ra.rtmp = st->rtmp;
                    ra.kept_ring = st->kept_ring; ra.mini = 0; ra.wide_count = st->wide_count;
                    PhaseTimer timer(st, stream, kPhaseBook, 1);
                    k_resolve<<<kResolveBlocks, kOmpThreads, 0, stream>>>(ra);
                    *launches += 1;
                }
            }
        }
        if (e != cudaSuccess) return e;
    }
    for (int i = 0; i < n; ++i) {
        sgc_state* st = sts[i];
        {
            PhaseTimer timer(st, stream, kPhaseCorr, 1);
            e = launch_omp(st, args[i], 1, stream);
            *launches += 1;
        }
        if (e != cudaSuccess) return e;
        if (st->shared_support || st->residual_tol > 0.0) {
            PhaseTimer timer(st, stream, kPhaseBook, 1);
            k_variant_tail<<<1, kOmpThreads, 0, stream>>>(args[i], st->shared_support, st->residual_tol);
            *launches += 1;
        }
        PhaseTimer timer(st, stream, kPhaseScatter, 1);
        k_scatter<<<1, kBookThreads, 0, stream>>>(st->s, st->lam, st->x, st->cnt, weights[i], st->upd_idx, st->upd_val,
                                                  (double)st->alpha, (double)st->eps, (double)st->lr);
        *launches += 1;
        if (speculate) {
            k_cand_update<<<1, kOmpThreads, 0, stream>>>(st->ctl, st->cnt, st->lam, st->s, st->cand_list, st->cand_bits,
                                                         st->kept_ring, st->d_rounds);
            *launches += 1;
        }
    }
    return cudaGetLastError();
}

// Which states of a group share passes.  One pass serves a batch of states only while it has room for all their residuals
// (kPassMaxN rows), and the two-level screening -- what keeps the number of passes over all d columns down when the
// recovery picks columns outside the kept sets -- is a single-state scheme.  So a state goes alone when a batch could hold
// nothing beside it, or when its last step needed three or more passes over all columns (the same signal that switches
// its two-level screening on); the others are batched.  The result does not depend on the split.
cudaError_t launch_recover_group(sgc_state* const* sts, float* const* weights, int n, cudaStream_t stream, int* launches) {
    if (n == 1) return recover_batches(sts, weights, 1, stream, launches);
    std::vector<sgc_state*> together;
    std::vector<float*> together_w;
    cudaError_t e = cudaSuccess;
    for (int i = 0; i < n && e == cudaSuccess; ++i) {
        sgc_state* st = sts[i];
        const bool speculates = st->spec_ok && st->spec_ready && (st->mode == 2 || (st->mode == 0 && st->d >= (1ll << 16)));
        const int last = speculates ? (*reinterpret_cast<volatile int*>(st->h_rounds) & 255) : 0;
        const bool alone = speculates && (kPassMaxN / st->pass_n < 2 || st->two_level || last >= 3);
        if (alone) e = recover_batches(&sts[i], &weights[i], 1, stream, launches);
        else { together.push_back(st); together_w.push_back(weights[i]); }
    }
    if (e == cudaSuccess && !together.empty())
        e = recover_batches(together.data(), together_w.data(), (int)together.size(), stream, launches);
    return e;
}

cudaError_t launch_recover(sgc_state* st, float* weight, cudaStream_t stream, int* launches) {
    return recover_batches(&st, &weight, 1, stream, launches);
}

}  // namespace sgc
