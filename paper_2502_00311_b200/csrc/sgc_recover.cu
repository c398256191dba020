// a4 + a5: x^M = OMP_A(M^), x^V = OMP_A(V^) (Eq. 7; Appendix B Algorithm 3), then
// N = alpha x^M / (sqrt(x^V) + eps) and W <- W - lr N (Eq. 8, Eq. 3; Algorithm 2 line 6).
//
// Both recoveries advance in lock-step, one iteration per pair of launches:
//   k_corr   the "Projection" + "Select" lines of Algorithm 3 without the d x d Gram matrix (Appendix B allows
//            the memory-efficient form): every column of A is regenerated tile by tile and correlated with
//            BOTH residuals, scores <A_i, r>^2 / ||A_i||^2 are reduced to the best few per block (fp32 screen);
//   k_book   one block per residual: rescoring of the screened candidates in fp64 (the argmax decision),
//            then the inverse-Cholesky recurrences of Algorithm 3 (c = F^T g, gamma, new column of F,
//            a_j, x = F a) in fp64 and the residual r = y - A_Lambda x.
// k_scatter applies Eq. (8) on the common support and updates W.
#include "sgc_internal.cuh"

namespace sgc {
namespace {

// ------------------------------------------------------------------------------------------------
// correlation pass
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ bool better(float sa, uint32_t ia, float sb, uint32_t ib) {
    return (sa > sb) || (sa == sb && ia < ib);
}

struct Top2 {
    float s1, s2; uint32_t i1, i2;
    __device__ __forceinline__ void init() { s1 = s2 = -1.0f; i1 = i2 = 0xFFFFFFFFu; }
    __device__ __forceinline__ void push(float s, uint32_t i) {
        if (better(s, i, s1, i1)) { s2 = s1; i2 = i1; s1 = s; i1 = i; }
        else if (better(s, i, s2, i2)) { s2 = s; i2 = i; }
    }
};

__device__ __forceinline__ void warp_merge(Top2& t) {
    for (int o = 16; o > 0; o >>= 1) {
        const float a1 = __shfl_xor_sync(0xffffffffu, t.s1, o), a2 = __shfl_xor_sync(0xffffffffu, t.s2, o);
        const uint32_t j1 = __shfl_xor_sync(0xffffffffu, t.i1, o), j2 = __shfl_xor_sync(0xffffffffu, t.i2, o);
        t.push(a1, j1);
        t.push(a2, j2);
    }
}

template <int C>
__global__ void __launch_bounds__(kCorrThreads, 2)
k_corr(uint32_t seed_lo, uint32_t seed_hi, unsigned long long d, int k, int s, const float2* __restrict__ r32,
       const uint32_t* __restrict__ lam, const Counters* __restrict__ cnt, Cand* __restrict__ out,
       unsigned int num_tiles) {
    extern __shared__ float2 sr[];                       // residual pair per row
    __shared__ uint32_t mask_idx[2][kMaxS];
    __shared__ int mask_n[2];
    __shared__ Top2 wtop[2][kCorrThreads / 32];
    for (int j = threadIdx.x; j < k; j += kCorrThreads) sr[j] = r32[j];
    const int done0 = cnt->done[0], done1 = cnt->done[1];
    Top2 best[2];
    best[0].init(); best[1].init();
    constexpr unsigned int kTileCols = kCorrThreads * C;
    for (unsigned int tile = blockIdx.x; tile < num_tiles; tile += gridDim.x) {
        const unsigned long long col_base = (unsigned long long)tile * kTileCols;
        __syncthreads();
        if (threadIdx.x < 2) mask_n[threadIdx.x] = 0;
        __syncthreads();
        // already selected columns that fall into this tile are excluded from the argmax
        for (int e = threadIdx.x; e < done0 + done1; e += kCorrThreads) {
            const int m = e < done0 ? 0 : 1;
            const uint32_t l = lam[m * s + (m ? e - done0 : e)];
            if (l >= col_base && l < col_base + kTileCols) mask_idx[m][atomicAdd(&mask_n[m], 1)] = l;
        }
        uint32_t h[C], mk[C];
        float am[C], av[C], an[C];
#pragma unroll
        for (int c = 0; c < C; ++c) {
            const ColKey key = column_key(seed_lo, seed_hi, (uint32_t)(col_base + c * kCorrThreads + threadIdx.x));
            h[c] = key.ck; mk[c] = key.mk;
            am[c] = av[c] = an[c] = 0.0f;
        }
        __syncthreads();
#pragma unroll 4
        for (int row = 0; row < k; ++row) {
            const float2 rr = sr[row];
#pragma unroll
            for (int c = 0; c < C; ++c) {
                const float z = z_from_word(h[c]);
                h[c] += mk[c];
                am[c] = __fmaf_rn(z, rr.x, am[c]);
                av[c] = __fmaf_rn(z, rr.y, av[c]);
                an[c] = __fmaf_rn(z, z, an[c]);
            }
        }
#pragma unroll
        for (int c = 0; c < C; ++c) {
            const unsigned long long col = col_base + c * kCorrThreads + threadIdx.x;
            if (col >= d) continue;
            const float inv = an[c] > 0.0f ? 1.0f / an[c] : 0.0f;
            float sm = am[c] * am[c] * inv, sv = av[c] * av[c] * inv;
            for (int e = 0; e < mask_n[0]; ++e) if (mask_idx[0][e] == (uint32_t)col) sm = -1.0f;
            for (int e = 0; e < mask_n[1]; ++e) if (mask_idx[1][e] == (uint32_t)col) sv = -1.0f;
            best[0].push(sm, (uint32_t)col);
            best[1].push(sv, (uint32_t)col);
        }
    }
    // block reduction of the two running top-2 lists
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    warp_merge(best[0]);
    warp_merge(best[1]);
    if (lane == 0) { wtop[0][warp] = best[0]; wtop[1][warp] = best[1]; }
    __syncthreads();
    if (warp < 2) {
        Top2 t;
        t.init();
        if (lane < kCorrThreads / 32) t = wtop[warp][lane];
        warp_merge(t);
        if (lane == 0) {
            Cand* o = out + ((size_t)warp * gridDim.x + blockIdx.x) * kCorrTop;
            o[0].score = t.s1; o[0].idx = t.i1;
            o[1].score = t.s2; o[1].idx = t.i2;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// bookkeeping: fp64 argmax among the screened candidates + Algorithm 3 recurrences
// ------------------------------------------------------------------------------------------------
__device__ __forceinline__ double warp_sum(double v) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// deterministic block sum; every thread receives the result.  red: 32 doubles of shared memory.
__device__ double block_sum(double v, double* red) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    v = warp_sum(v);
    __syncthreads();
    if (lane == 0) red[warp] = v;
    __syncthreads();
    double t = (lane < kBookThreads / 32) ? red[lane] : 0.0;
    t = warp_sum(t);
    return t;
}

struct BookArgs {
    uint32_t seed_lo, seed_hi;
    int k, s, corr_grid;
    double sigma;
    const Cand* corr_cand;
    const double* y64; double* r64; float* r32;       // r32 viewed as float[2k] (interleaved pairs)
    uint16_t* zsel; uint32_t* lam; double* F; double* acoef; double* x; double* rnorm;
    Counters* cnt;
};

__global__ void __launch_bounds__(kBookThreads, 1)
k_book(BookArgs a, int iter) {
    const int m = blockIdx.x;                    // 0: M^, 1: V^
    if (a.cnt->stopped[m]) return;
    __shared__ double red[32];
    __shared__ float fred[32];
    __shared__ uint32_t cand_idx[kRescoreCap];
    __shared__ int n_cand;
    __shared__ double gvec[kMaxS];               // Gram column g, then reused
    __shared__ double cvec[kMaxS];               // c = F^T g
    __shared__ double xs[kMaxS];                 // current coefficients
    __shared__ double best_dot, best_n2, best_score;
    __shared__ uint32_t best_idx;
    const int k = a.k, s = a.s, j = iter;
    const double* y = a.y64 + (size_t)m * k;
    double* r = a.r64 + (size_t)m * k;
    uint16_t* zs = a.zsel + (size_t)m * s * k;
    double* F = a.F + (size_t)m * s * s;
    double* xg = a.x + (size_t)m * s;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;

    // ---- 1. screened candidates: everything within 2e-3 (relative, squared scores) of the best fp32 score
    const Cand* cc = a.corr_cand + (size_t)m * a.corr_grid * kCorrTop;
    const int n_entries = a.corr_grid * kCorrTop;
    float mx = -1.0f;
    for (int e = threadIdx.x; e < n_entries; e += kBookThreads) mx = fmaxf(mx, cc[e].score);
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (threadIdx.x == 0) { n_cand = 0; best_score = -1.0; best_idx = 0xFFFFFFFFu; best_dot = 0.0; best_n2 = 1.0; }
    __syncthreads();
    if (lane == 0) fred[warp] = mx;
    __syncthreads();
    mx = fred[lane];
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    const float thr = mx - 2e-3f * fabsf(mx);
    for (int e = threadIdx.x; e < n_entries; e += kBookThreads) {
        const Cand c = cc[e];
        if (c.idx != 0xFFFFFFFFu && c.score >= 0.0f && c.score >= thr) {
            const int slot = atomicAdd(&n_cand, 1);
            if (slot < kRescoreCap) cand_idx[slot] = c.idx;
        }
    }
    __syncthreads();
    int nc = n_cand;
    if (nc > kRescoreCap) {
        if (threadIdx.x == 0) atomicOr(&a.cnt->status, (unsigned int)SGC_STATUS_CANDIDATE_OVERFLOW);
        nc = kRescoreCap;
    }
    if (nc == 0) {          // nothing left to select (cannot happen while fewer than d columns are taken)
        if (threadIdx.x == 0) { a.cnt->stopped[m] = 1; atomicOr(&a.cnt->status, (unsigned int)SGC_STATUS_DEPENDENT_COLUMN); }
        return;
    }
    // ---- 2. fp64 rescoring: the argmax of |<A_i, r>| / ||A_i|| among the candidates, lowest index on ties
    for (int c = 0; c < nc; ++c) {
        const uint32_t idx = cand_idx[c];
        const ColKey key = column_key(a.seed_lo, a.seed_hi, idx);
        double dot = 0.0, n2 = 0.0;
        for (int row = threadIdx.x; row < k; row += kBookThreads) {
            const double z = (double)z_from_word(key.ck + (uint32_t)row * key.mk);
            dot += z * r[row];
            n2 += z * z;
        }
        dot = block_sum(dot, red);
        n2 = block_sum(n2, red);
        if (threadIdx.x == 0) {
            const double sc = n2 > 0.0 ? dot * dot / n2 : 0.0;
            if (sc > best_score || (sc == best_score && idx < best_idx)) {
                best_score = sc; best_idx = idx; best_dot = dot; best_n2 = n2;
            }
        }
        __syncthreads();
    }
    const uint32_t lam_new = best_idx;
    const double dot_r = best_dot, n2_new = best_n2;
    // ---- 3. store the new column (bfloat16 bits, exact) ------------------------------------------------
    {
        const ColKey key = column_key(a.seed_lo, a.seed_hi, lam_new);
        uint16_t* znew = zs + (size_t)j * k;
        for (int row = threadIdx.x; row < k; row += kBookThreads)
            znew[row] = z_bf16_bits(z_from_word(key.ck + (uint32_t)row * key.mk));
    }
    __syncthreads();
    // ---- 4. g = A_Lambda^T a_new  (Gram column; "g_{:,lambda_k}" restricted to the support) --------------
    const double sig2 = a.sigma * a.sigma;
    {
        const uint16_t* znew = zs + (size_t)j * k;
        for (int l = warp; l < j; l += kBookThreads / 32) {
            const uint16_t* zl = zs + (size_t)l * k;
            double acc = 0.0;
            for (int row = lane; row < k; row += 32)
                acc += (double)(bf16_bits_to_float(zl[row]) * bf16_bits_to_float(znew[row]));   // product exact in fp32
            acc = warp_sum(acc);
            if (lane == 0) gvec[l] = sig2 * acc;
        }
    }
    __syncthreads();
    // ---- 5. c = F^T g ;  F is upper triangular, F(l,i) stored at F[l*s + i] ----------------------------
    double csq = 0.0;
    if (threadIdx.x < j) {
        const int i = threadIdx.x;
        double acc = 0.0;
        for (int l = 0; l <= i; ++l) acc += F[(size_t)l * s + i] * gvec[l];
        cvec[i] = acc;
        csq = acc * acc;
    }
    csq = block_sum(csq, red);
    // ---- 6. gamma = 1/sqrt(g_ll - c^T c); a dependent column stops this recovery --------------------------
    const double gnn = sig2 * n2_new;
    const double piv = gnn - csq;
    if (!(piv > 1e-10 * gnn)) {
        if (threadIdx.x == 0) { a.cnt->stopped[m] = 1; atomicOr(&a.cnt->status, (unsigned int)SGC_STATUS_DEPENDENT_COLUMN); }
        return;
    }
    const double gamma = 1.0 / sqrt(piv);
    // ---- 7. new column of F: [-gamma F c ; gamma] ------------------------------------------------------
    __syncthreads();
    if (threadIdx.x < j) {
        const int i = threadIdx.x;
        double acc = 0.0;
        for (int l = i; l < j; ++l) acc += F[(size_t)i * s + l] * cvec[l];
        F[(size_t)i * s + j] = -gamma * acc;
    } else if (threadIdx.x == j) {
        F[(size_t)j * s + j] = gamma;
    }
    // ---- 8. a_j = gamma <a_new, r> ;  x = F a  grows by a_j * F(:, j) -------------------------------------
    const double aj = gamma * a.sigma * dot_r;
    __syncthreads();
    if (threadIdx.x <= j) {
        const int i = threadIdx.x;
        const double xo = (i < j) ? xg[i] : 0.0;
        const double xn = xo + aj * F[(size_t)i * s + j];
        xg[i] = xn;
        xs[i] = xn;
    }
    if (threadIdx.x == 0) { a.acoef[(size_t)m * s + j] = aj; a.lam[(size_t)m * s + j] = lam_new; }
    __syncthreads();
    // ---- 9. r = y - A_Lambda x ---------------------------------------------------------------------------
    double rn2 = 0.0;
    for (int row = threadIdx.x; row < k; row += kBookThreads) {
        double acc = 0.0;
        for (int l = 0; l <= j; ++l) acc += xs[l] * (double)bf16_bits_to_float(zs[(size_t)l * k + row]);
        const double rv = y[row] - a.sigma * acc;
        r[row] = rv;
        a.r32[2 * row + m] = (float)rv;
        rn2 += rv * rv;
    }
    rn2 = block_sum(rn2, red);
    if (threadIdx.x == 0) {
        a.rnorm[(size_t)m * s + j] = sqrt(rn2);
        a.cnt->done[m] = j + 1;
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

}  // namespace

cudaError_t configure_recover(sgc_state* st) {
    const size_t smem = (size_t)st->k * sizeof(float2);
    cudaError_t e = cudaFuncSetAttribute(k_corr<kCorrCols>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    int occ = 0;
    e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&occ, k_corr<kCorrCols>, kCorrThreads, smem);
    if (e != cudaSuccess) return e;
    if (occ < 1) return cudaErrorInvalidConfiguration;
    const unsigned long long tile_cols = (unsigned long long)kCorrThreads * kCorrCols;
    const unsigned long long tiles = ((unsigned long long)st->d + tile_cols - 1) / tile_cols;
    unsigned long long grid = (unsigned long long)st->sm_count * occ;
    if (grid > tiles) grid = tiles;
    st->corr_grid = (int)grid;
    st->corr_smem = (int)smem;
    return cudaSuccess;
}

cudaError_t launch_recover(sgc_state* st, float* weight, cudaStream_t stream, int* launches) {
    const uint32_t seed_lo = (uint32_t)(st->seed & 0xFFFFFFFFu), seed_hi = (uint32_t)(st->seed >> 32);
    const unsigned long long tile_cols = (unsigned long long)kCorrThreads * kCorrCols;
    const unsigned int tiles = (unsigned int)(((unsigned long long)st->d + tile_cols - 1) / tile_cols);
    BookArgs a;
    a.seed_lo = seed_lo; a.seed_hi = seed_hi; a.k = st->k; a.s = st->s; a.corr_grid = st->corr_grid;
    a.sigma = (double)(float)(1.0 / sqrt((double)st->k));
    a.corr_cand = st->corr_cand; a.y64 = st->y64; a.r64 = st->r64; a.r32 = reinterpret_cast<float*>(st->r32);
    a.zsel = st->zsel; a.lam = st->lam; a.F = st->F; a.acoef = st->acoef; a.x = st->x; a.rnorm = st->rnorm;
    a.cnt = st->cnt;
    for (int it = 0; it < st->s; ++it) {
        {
            PhaseTimer timer(st, stream, kPhaseCorr, 1);
            k_corr<kCorrCols><<<st->corr_grid, kCorrThreads, st->corr_smem, stream>>>(
                seed_lo, seed_hi, (unsigned long long)st->d, st->k, st->s, st->r32, st->lam, st->cnt, st->corr_cand, tiles);
        }
        {
            PhaseTimer timer(st, stream, kPhaseBook, 1);
            k_book<<<2, kBookThreads, 0, stream>>>(a, it);
        }
        *launches += 2;
    }
    PhaseTimer timer(st, stream, kPhaseScatter, 1);
    k_scatter<<<1, kBookThreads, 0, stream>>>(st->s, st->lam, st->x, st->cnt, weight, st->upd_idx, st->upd_val,
                                              (double)st->alpha, (double)st->eps, (double)st->lr);
    *launches += 1;
    return cudaGetLastError();
}

}  // namespace sgc
