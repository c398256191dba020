// MESGC (Section 4.4) with small per-chunk problems: c chunks of one flat vector, each an SGC problem of its own
// (own M, V; s_c <= 16 kept entries, k_c <= 128 rows), all sharing the matrix A (k_c x d/c) named by one seed.
// Run chunk by chunk this costs ~25 launches per chunk; here the whole step of all chunks takes 2 + 2 s_c launches:
//   k_chunk_front    block = chunk: exact top-s_c of the chunk (a1), p = A g~, q = A g~^2 and the k-space Adam moments
//                    (a2 + a3), residuals r = y for both moments
//   per OMP iteration (Algorithm 3, all 2c recoveries in lock-step, which is where the shared A pays: a column of A is
//   generated once and meets the residuals of every chunk):
//     k_chunk_corr   thread = one residual, block = 256 residuals x a range of columns: fp32 scores |<A_i,r>| / ||A_i||,
//                    best two columns of the range per residual
//     k_chunk_pick   warp = one recovery: fp64 rescoring of the columns within 2e-3 of the best fp32 score, lowest
//                    index on ties, then the inverse-Cholesky recurrences of Algorithm 3, x, r
//   k_chunk_scatter  warp = chunk: Eq. (8) on the common support, weight update (a5)
// Every record lands in the chunk's own state, so sgc_get works per chunk exactly as after sgc_step.
#include <algorithm>
#include <new>
#include <vector>

#include "sgc_internal.cuh"

namespace sgc {
namespace {

constexpr int kFrontThreads = 512;
constexpr int kCorrBlock = 256;          // residuals per block of k_chunk_corr
constexpr int kChunkMaxS = 16;
constexpr int kChunkMaxK = 128;

struct ChunkArgs {
    const ChunkRef* table;
    int c, k, s, kp;                     // kp: k rounded up to 8, 16, 32, 64 or 128 (row stride of r32)
    long long dc;                        // columns per chunk
    uint32_t seed_lo, seed_hi;
    double sigma;
    float* r32;                          // [2c][kp]
    Cand* cand;                          // [2c][splits][2]
    int splits, cols_per_split;
};

__device__ __forceinline__ double warp_sum_d(double v) {
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// ---- a1 + a2 + a3, one block per chunk -------------------------------------------------------------------
// Top-s of the chunk by the key (|g| bits << 32) | ~index (unique; lowest index wins equal magnitudes): every thread
// keeps the CAP largest keys of its strided share in registers (the s largest of the chunk are among them), then s
// rounds of "largest head of any thread" pop them in descending order.
template <int CAP>
__global__ void __launch_bounds__(kFrontThreads)
k_chunk_front(ChunkArgs a, const float* __restrict__ grad, double b1, double b2, double c1, double c2) {
    __shared__ unsigned long long wmax[kFrontThreads / 32];
    __shared__ unsigned long long sel_key[kChunkMaxS];
    __shared__ ColKey keys[kChunkMaxS];
    __shared__ float vals[kChunkMaxS];
    const int ch = blockIdx.x, s = a.s, k = a.k;
    const ChunkRef ref = a.table[ch];
    const float* g = grad + (size_t)ch * a.dc;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    unsigned long long top[CAP];
#pragma unroll
    for (int q = 0; q < CAP; ++q) top[q] = 0ull;                    // no real key is 0
    const long long nvec = a.dc >> 2;                                // chunks start on 16-byte boundaries, dc % 4 == 0
    for (long long v = threadIdx.x; v < nvec; v += kFrontThreads) {
        const float4 f = __ldcs(reinterpret_cast<const float4*>(g) + v);
        const float e[4] = {f.x, f.y, f.z, f.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const uint32_t i = (uint32_t)(4 * v + u);
            const unsigned long long key = ((unsigned long long)(__float_as_uint(e[u]) & 0x7FFFFFFFu) << 32) | (uint32_t)(~i);
            if (key > top[CAP - 1]) {
#pragma unroll
                for (int q = CAP - 1; q >= 0; --q) {
                    const unsigned long long up = q > 0 ? top[q - 1] : ~0ull;
                    if (key > top[q]) top[q] = key > up ? up : key;
                }
            }
        }
    }
    for (int r = 0; r < s; ++r) {
        unsigned long long m = top[0];
        for (int o = 16; o > 0; o >>= 1) { const unsigned long long t = __shfl_xor_sync(0xffffffffu, m, o); m = t > m ? t : m; }
        if (lane == 0) wmax[warp] = m;
        __syncthreads();
        unsigned long long best = 0ull;
#pragma unroll
        for (int w = 0; w < kFrontThreads / 32; ++w) best = wmax[w] > best ? wmax[w] : best;
        if (top[0] == best && best != 0ull) {                        // keys are unique: exactly one thread pops
#pragma unroll
            for (int q = 0; q + 1 < CAP; ++q) top[q] = top[q + 1];
            top[CAP - 1] = 0ull;
            sel_key[r] = best;
        }
        __syncthreads();
    }
    if (threadIdx.x == 0) {
        // ascending index order, as the records of sgc_step have it
        for (int i = 1; i < s; ++i) {
            const unsigned long long kv = sel_key[i];
            int j = i - 1;
            while (j >= 0 && (uint32_t)(~(uint32_t)sel_key[j]) > (uint32_t)(~(uint32_t)kv)) { sel_key[j + 1] = sel_key[j]; --j; }
            sel_key[j + 1] = kv;
        }
        unsigned int bits = 0u;
        for (int i = 0; i < s; ++i) {
            const uint32_t idx = ~(uint32_t)sel_key[i];
            if ((sel_key[i] >> 32) >= 0x7F800000ull) bits |= (unsigned int)SGC_STATUS_NONFINITE_INPUT;
            const float val = g[idx];
            ref.sel_idx[i] = idx; ref.sel_val[i] = val;
            keys[i] = column_key(a.seed_lo, a.seed_hi, idx);
            vals[i] = val;
        }
        if (bits) atomicOr(&ref.cnt->status, bits);
        ref.cnt->done[0] = ref.cnt->done[1] = 0;
        ref.cnt->stopped[0] = ref.cnt->stopped[1] = 0;
        ref.cnt->n_upd = ref.cnt->mismatch = ref.cnt->negv = 0;
        ref.ctl->round_active = 0; ref.ctl->fallback = 1; ref.ctl->rounds = 0; ref.ctl->list_rounds = 0;
    }
    __syncthreads();
    // a2 + a3: thread = row; fp64 sums in ascending column order (the arithmetic of the one-state kernel, term by term)
    for (int row = threadIdx.x; row < k; row += kFrontThreads) {
        double accp = 0.0, accq = 0.0;
        for (int i = 0; i < s; ++i) {
            const double av = a.sigma * (double)z_at(keys[i], (uint32_t)row);
            const double gv = (double)vals[i];
            accp = accp + av * gv;
            accq = accq + av * (gv * gv);
        }
        ref.p[row] = accp;
        ref.q[row] = accq;
        const float m = (float)(b1 * (double)ref.M[row] + (1.0 - b1) * accp);
        const float v = (float)(b2 * (double)ref.V[row] + (1.0 - b2) * accq);
        ref.M[row] = m;
        ref.V[row] = v;
        const double mh = (double)m / c1, vh = (double)v / c2;      // bias-corrected temporaries; state stays uncorrected
        ref.y64[row] = mh; ref.y64[k + row] = vh;
        ref.r64[row] = mh; ref.r64[k + row] = vh;
        a.r32[(size_t)(2 * ch) * a.kp + row] = (float)mh;
        a.r32[(size_t)(2 * ch + 1) * a.kp + row] = (float)vh;
    }
}

// ---- phase A of one OMP iteration: every column of A against the residuals of all recoveries ------------------
// grid = (column splits, groups of 256 recoveries).  The block walks its columns in tiles: thread t generates column
// t of the tile into shared memory (fp32, with 1 / ||Z_i||), then every thread, which holds the residual of one
// recovery in registers, scores all columns of the tile in ascending order (a strict ">" keeps the lowest index).
// Only the best two columns per recovery leave the block; columns already in the support are skipped when they show up
// as a new best.
template <int KP>
__global__ void __launch_bounds__(kCorrBlock) k_chunk_corr(ChunkArgs a, int iter) {
    constexpr int TC = KP <= 64 ? 256 : 128;                         // columns per tile
    constexpr int ZS = KP + 4;                                       // row stride of a tile column (16-byte multiple)
    extern __shared__ float smem[];
    float* zt = smem;                                                // [TC][ZS]
    float* inv = smem + TC * ZS;                                     // [TC]
    const int res = blockIdx.y * kCorrBlock + threadIdx.x;           // recovery = 2 * chunk + moment
    const bool have = res < 2 * a.c;
    bool active = false;
    const uint32_t* sup = nullptr;
    float rr[KP];
#pragma unroll
    for (int q = 0; q < KP; ++q) rr[q] = 0.0f;
    if (have) {
        const ChunkRef& ref = a.table[res >> 1];
        active = ref.cnt->stopped[res & 1] == 0;
        sup = ref.lam + (size_t)(res & 1) * a.s;
        const float4* src = reinterpret_cast<const float4*>(a.r32 + (size_t)res * KP);
#pragma unroll
        for (int q = 0; q < KP / 4; ++q) { const float4 f = src[q]; rr[4 * q] = f.x; rr[4 * q + 1] = f.y; rr[4 * q + 2] = f.z; rr[4 * q + 3] = f.w; }
    }
    float s1 = -1.0f, s2 = -1.0f;
    uint32_t i1 = kNoColumn, i2 = kNoColumn;
    const long long col0 = (long long)blockIdx.x * a.cols_per_split;
    long long col1 = col0 + a.cols_per_split;
    if (col1 > a.dc) col1 = a.dc;
    for (long long tile = col0; tile < col1; tile += TC) {
        __syncthreads();
        for (int t = threadIdx.x; t < TC; t += kCorrBlock) {
            const long long col = tile + t;
            float n2 = 0.0f;
            float* dst = zt + t * ZS;
            if (col < col1) {
                const ColKey key = column_key(a.seed_lo, a.seed_hi, (uint32_t)col);
                uint32_t h = key.ck;
#pragma unroll 4
                for (int row = 0; row < KP; row += 2) {
                    float2 z = half2_bits_to_float2(z_pair_from_word(h));
                    h += key.mk;
                    if (row >= a.k) z.x = 0.0f;
                    if (row + 1 >= a.k) z.y = 0.0f;
                    dst[row] = z.x; dst[row + 1] = z.y;
                    n2 = __fmaf_rn(z.x, z.x, n2);
                    n2 = __fmaf_rn(z.y, z.y, n2);
                }
            } else {
                for (int row = 0; row < KP; ++row) dst[row] = 0.0f;
            }
            inv[t] = n2 > 0.0f ? 1.0f / sqrtf(n2) : 0.0f;
        }
        __syncthreads();
        if (!active) continue;
        const int n_here = (int)((col1 - tile) < TC ? (col1 - tile) : TC);
        for (int t = 0; t < n_here; ++t) {
            const float4* zc = reinterpret_cast<const float4*>(zt + t * ZS);
            float acc0 = 0.0f, acc1 = 0.0f;
#pragma unroll
            for (int q = 0; q < KP / 4; ++q) {
                const float4 z = zc[q];                              // same address in every thread: a broadcast
                acc0 = __fmaf_rn(z.x, rr[4 * q], acc0);
                acc1 = __fmaf_rn(z.y, rr[4 * q + 1], acc1);
                acc0 = __fmaf_rn(z.z, rr[4 * q + 2], acc0);
                acc1 = __fmaf_rn(z.w, rr[4 * q + 3], acc1);
            }
            const float sc = fabsf(acc0 + acc1) * inv[t];
            if (sc > s2) {
                const uint32_t col = (uint32_t)(tile + t);
                bool taken = false;
                for (int q = 0; q < iter; ++q) taken |= (sup[q] == col);
                if (!taken) {
                    if (sc > s1) { s2 = s1; i2 = i1; s1 = sc; i1 = col; }
                    else { s2 = sc; i2 = col; }
                }
            }
        }
    }
    if (have) {
        Cand* out = a.cand + ((size_t)res * a.splits + blockIdx.x) * 2;
        out[0].score = s1; out[0].idx = i1;
        out[1].score = s2; out[1].idx = i2;
    }
}

// ---- phase B of one OMP iteration: one warp per recovery ---------------------------------------------------
// Argmax among the columns that phase A left within 2e-3 (relative) of the best fp32 score, decided on fp64 scores
// <Z_i, r>^2 / ||Z_i||^2 with the lowest index winning ties; then Algorithm 3 (Appendix B) for the new column:
// g = A_Lambda^T a_new, c = F^T g, gamma = 1 / sqrt(g_ll - c^T c) (a pivot below 1e-10 g_ll ends this recovery),
// new column [-gamma F c; gamma] of F, a_j = gamma <a_new, r>, x = F a, r = y - A_Lambda x.
__global__ void __launch_bounds__(32) k_chunk_pick(ChunkArgs a, int iter) {
    __shared__ double gv[kChunkMaxS], cv[kChunkMaxS], xs[kChunkMaxS];
    __shared__ uint32_t cidx[kRescoreCap];
    __shared__ int n_c;
    const int res = blockIdx.x, m = res & 1, lane = threadIdx.x;
    const ChunkRef ref = a.table[res >> 1];
    if (ref.cnt->stopped[m]) return;
    const int k = a.k, s = a.s, j = iter;
    const Cand* cc = a.cand + (size_t)res * a.splits * 2;
    const int n_entries = a.splits * 2;
    float mx = -1.0f;
    for (int e = lane; e < n_entries; e += 32) if (cc[e].idx != kNoColumn) mx = fmaxf(mx, cc[e].score);
    for (int o = 16; o > 0; o >>= 1) mx = fmaxf(mx, __shfl_xor_sync(0xffffffffu, mx, o));
    if (lane == 0) n_c = 0;
    __syncwarp();
    const float thr = mx - 2e-3f * fabsf(mx);
    for (int e = lane; e < n_entries; e += 32) {
        const Cand c = cc[e];
        if (c.idx != kNoColumn && c.score >= 0.0f && c.score >= thr) {
            const int slot = atomicAdd(&n_c, 1);
            if (slot < kRescoreCap) cidx[slot] = c.idx;
        }
    }
    __syncwarp();
    int nc = n_c;
    if (nc > kRescoreCap) {
        if (lane == 0) atomicOr(&ref.cnt->status, (unsigned int)SGC_STATUS_CANDIDATE_OVERFLOW);
        nc = kRescoreCap;
    }
    double* r = ref.r64 + (size_t)m * k;
    const double* y = ref.y64 + (size_t)m * k;
    if (nc == 0) {                                                   // no column left to pick (d/c = iterations made)
        if (lane == 0) { ref.cnt->stopped[m] = 1; ref.cnt->done[m] = j; }
        return;
    }
    // fp64 scores of the candidates
    double best_sc = -1.0, best_dot = 0.0, best_n2 = 1.0;
    uint32_t best_idx = kNoColumn;
    for (int c = 0; c < nc; ++c) {
        const uint32_t idx = cidx[c];
        const ColKey key = column_key(a.seed_lo, a.seed_hi, idx);
        double dot = 0.0, n2 = 0.0;
        for (int row = 2 * lane; row < k; row += 64) {
            const float2 zz = half2_bits_to_float2(z_pair_from_word(key.ck + (uint32_t)(row >> 1) * key.mk));
            dot += (double)zz.x * r[row];
            n2 += (double)zz.x * (double)zz.x;
            if (row + 1 < k) { dot += (double)zz.y * r[row + 1]; n2 += (double)zz.y * (double)zz.y; }
        }
        dot = warp_sum_d(dot); n2 = warp_sum_d(n2);
        const double sc = n2 > 0.0 ? dot * dot / n2 : 0.0;
        if (sc > best_sc || (sc == best_sc && idx < best_idx)) { best_sc = sc; best_idx = idx; best_dot = dot; best_n2 = n2; }
    }
    // the new column, binary16 bits (exact)
    uint16_t* zs = ref.zsel + (size_t)m * s * k;
    double* F = ref.F + (size_t)m * s * s;
    double* xg = ref.x + (size_t)m * s;
    {
        const ColKey key = column_key(a.seed_lo, a.seed_hi, best_idx);
        uint16_t* znew = zs + (size_t)j * k;
        for (int row = 2 * lane; row < k; row += 64) {
            const uint32_t z2 = z_pair_from_word(key.ck + (uint32_t)(row >> 1) * key.mk);
            znew[row] = (uint16_t)(z2 & 0xFFFFu);
            if (row + 1 < k) znew[row + 1] = (uint16_t)(z2 >> 16);
        }
    }
    __syncwarp();
    const double sig2 = a.sigma * a.sigma;
    const uint16_t* znew = zs + (size_t)j * k;
    for (int l = 0; l < j; ++l) {                                    // g = A_Lambda^T a_new
        const uint16_t* zl = zs + (size_t)l * k;
        double acc = 0.0;
        for (int row = lane; row < k; row += 32) acc += (double)(half_bits_to_float(zl[row]) * half_bits_to_float(znew[row]));
        acc = warp_sum_d(acc);
        if (lane == 0) gv[l] = sig2 * acc;
    }
    __syncwarp();
    double csq = 0.0;
    if (lane < j) {                                                  // c = F^T g (F upper triangular, F(l, i) at F[l*s + i])
        double acc = 0.0;
        for (int l = 0; l <= lane; ++l) acc += F[(size_t)l * s + lane] * gv[l];
        cv[lane] = acc;
        csq = acc * acc;
    }
    csq = warp_sum_d(csq);
    const double gnn = sig2 * best_n2;
    const double piv = gnn - csq;
    if (!(piv > 1e-10 * gnn)) {                                      // dependent column: this recovery ends with j picks
        if (lane == 0) {
            ref.cnt->stopped[m] = 1; ref.cnt->done[m] = j;
            atomicOr(&ref.cnt->status, (unsigned int)SGC_STATUS_DEPENDENT_COLUMN);
        }
        return;
    }
    const double gamma = 1.0 / sqrt(piv);
    __syncwarp();
    if (lane < j) {
        double acc = 0.0;
        for (int l = lane; l < j; ++l) acc += F[(size_t)lane * s + l] * cv[l];
        F[(size_t)lane * s + j] = -gamma * acc;
    } else if (lane == j) {
        F[(size_t)j * s + j] = gamma;
    }
    const double aj = gamma * a.sigma * best_dot;
    __syncwarp();
    if (lane <= j) {
        const double xo = lane < j ? xg[lane] : 0.0;
        const double xn = xo + aj * F[(size_t)lane * s + j];
        xg[lane] = xn;
        xs[lane] = xn;
    }
    if (lane == 0) { ref.acoef[(size_t)m * s + j] = aj; ref.lam[(size_t)m * s + j] = best_idx; }
    __syncwarp();
    double rn2 = 0.0;
    for (int row = lane; row < k; row += 32) {                       // r = y - A_Lambda x
        double acc = 0.0;
        for (int l = 0; l <= j; ++l) acc += xs[l] * (double)half_bits_to_float(zs[(size_t)l * k + row]);
        const double rv = y[row] - a.sigma * acc;
        r[row] = rv;
        a.r32[(size_t)res * a.kp + row] = (float)rv;
        rn2 += rv * rv;
    }
    rn2 = warp_sum_d(rn2);
    if (lane == 0) {
        ref.rnorm[(size_t)m * s + j] = sqrt(rn2);
        ref.cnt->done[m] = j + 1;
    }
}

// ---- a5: Eq. (8) on the common support of the two recoveries of a chunk, one warp per chunk -------------------
__global__ void __launch_bounds__(32) k_chunk_scatter(ChunkArgs a, float* __restrict__ weight, double alpha, double eps, double lr) {
    __shared__ uint32_t vidx[kChunkMaxS];
    __shared__ double vval[kChunkMaxS];
    __shared__ int flag[kChunkMaxS];
    const int ch = blockIdx.x, lane = threadIdx.x, s = a.s;
    const ChunkRef ref = a.table[ch];
    float* W = weight + (size_t)ch * a.dc;
    const int nM = ref.cnt->done[0], nV = ref.cnt->done[1];
    uint32_t* lam = ref.lam;
    double* x = ref.x;
    if (lane < s) {                                                  // unpicked slots read as "none"
        if (lane >= nM) { lam[lane] = kNoColumn; x[lane] = 0.0; }
        if (lane >= nV) { lam[s + lane] = kNoColumn; x[s + lane] = 0.0; }
        flag[lane] = 0;
    }
    __syncwarp();
    bool mis = false, neg = false;
    if (lane < nM) {
        const uint32_t li = lam[lane];
        int hit = -1;
        for (int b = 0; b < nV; ++b) if (lam[s + b] == li) { hit = b; break; }
        if (hit < 0) mis = true;
        else {
            const double xv = x[s + hit];
            if (!(xv > 0.0)) neg = true;
            else {
                const double N = alpha * x[lane] / (sqrt(xv) + eps);
                vidx[lane] = li; vval[lane] = lr * N; flag[lane] = 1;
            }
        }
    }
    __syncwarp();
    const int n_mis = __popc(__ballot_sync(0xffffffffu, mis)), n_neg = __popc(__ballot_sync(0xffffffffu, neg));
    const bool valid = lane < nM && flag[lane];
    const int n_valid = __popc(__ballot_sync(0xffffffffu, valid));
    if (valid) {
        int rank = 0;
        for (int b = 0; b < nM; ++b) if (flag[b] && vidx[b] < vidx[lane]) ++rank;
        ref.upd_idx[rank] = vidx[lane];
        ref.upd_val[rank] = vval[lane];
        W[vidx[lane]] = (float)((double)W[vidx[lane]] - vval[lane]);
    }
    if (lane == 0) {
        ref.cnt->n_upd = n_valid; ref.cnt->mismatch = n_mis; ref.cnt->negv = n_neg;
        unsigned int bits = 0;
        if (n_mis > 0 || nM != nV) bits |= (unsigned int)SGC_STATUS_SUPPORT_MISMATCH;
        if (n_neg > 0) bits |= (unsigned int)SGC_STATUS_NEGATIVE_V;
        if (bits) atomicOr(&ref.cnt->status, bits);
    }
}

}  // namespace

// ---- host side ----------------------------------------------------------------------------------------------
namespace {

int padded_k(int k) { return k <= 8 ? 8 : k <= 16 ? 16 : k <= 32 ? 32 : k <= 64 ? 64 : 128; }

unsigned long long list_key(sgc_state* const* sts, int c) {
    unsigned long long h = 1469598103934665603ull;                   // FNV-1a
    for (int i = 0; i < c; ++i) {                                     // host object and its device allocation
        h ^= (unsigned long long)(uintptr_t)sts[i]; h *= 1099511628211ull;
        h ^= (unsigned long long)(uintptr_t)sts[i]->base; h *= 1099511628211ull;
    }
    return h ^ (unsigned long long)c;
}

template <int KP>
cudaError_t corr_setup(size_t* smem_out) {
    constexpr int TC = KP <= 64 ? 256 : 128;
    const size_t smem = (size_t)(TC * (KP + 4) + TC) * sizeof(float);
    *smem_out = smem;
    return cudaFuncSetAttribute(k_chunk_corr<KP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

template <int KP>
void corr_launch(const ChunkArgs& a, int iter, size_t smem, cudaStream_t stream) {
    dim3 grid((unsigned int)a.splits, (unsigned int)((2 * a.c + kCorrBlock - 1) / kCorrBlock));
    k_chunk_corr<KP><<<grid, kCorrBlock, smem, stream>>>(a, iter);
}

// builds (or reuses) the workspace for this chunk list; the first build synchronises (one allocation, one copy)
cudaError_t ensure_ws(sgc_state* const* sts, int c) {
    sgc_state* st0 = sts[0];
    const unsigned long long key = list_key(sts, c);
    if (st0->chunk_ws && st0->chunk_ws->key == key && st0->chunk_ws->c == c) return cudaSuccess;
    {
        std::vector<sgc_state*> sorted(sts, sts + c);                // a state may appear once only
        std::sort(sorted.begin(), sorted.end());
        for (int i = 1; i < c; ++i) if (sorted[i] == sorted[i - 1]) return cudaErrorInvalidValue;
    }
    free_chunk_ws(st0);
    ChunkWs* ws = new (std::nothrow) ChunkWs();
    if (!ws) return cudaErrorMemoryAllocation;
    ws->c = c; ws->key = key; ws->kp = padded_k(st0->k);
    // column splits: enough blocks for every SM twice over, at least one tile per split
    const int groups = (2 * c + kCorrBlock - 1) / kCorrBlock;
    const int tile = ws->kp <= 64 ? 256 : 128;
    int splits = (2 * st0->sm_count + groups - 1) / groups;
    const long long max_splits = (st0->d + tile - 1) / tile;
    if (splits > max_splits) splits = (int)max_splits;
    if (splits < 1) splits = 1;
    long long per = (st0->d + splits - 1) / splits;
    per = (per + tile - 1) / tile * tile;
    splits = (int)((st0->d + per - 1) / per);
    ws->splits = splits;
    const size_t b_table = ((size_t)c * sizeof(ChunkRef) + 255) / 256 * 256;
    const size_t b_r32 = ((size_t)2 * c * ws->kp * sizeof(float) + 255) / 256 * 256;
    const size_t b_cand = (size_t)2 * c * splits * 2 * sizeof(Cand);
    cudaError_t e = cudaMalloc(&ws->base, b_table + b_r32 + b_cand);
    if (e != cudaSuccess) { delete ws; return e; }
    unsigned char* base = static_cast<unsigned char*>(ws->base);
    ws->table = reinterpret_cast<ChunkRef*>(base);
    ws->r32 = reinterpret_cast<float*>(base + b_table);
    ws->cand = reinterpret_cast<Cand*>(base + b_table + b_r32);
    std::vector<ChunkRef> host((size_t)c);
    for (int i = 0; i < c; ++i) {
        sgc_state* st = sts[i];
        ChunkRef& r = host[i];
        r.M = st->M; r.V = st->V; r.p = st->p; r.q = st->q; r.y64 = st->y64; r.r64 = st->r64;
        r.sel_idx = st->sel_idx; r.sel_val = st->sel_val;
        r.zsel = st->zsel; r.lam = st->lam; r.F = st->F; r.acoef = st->acoef; r.x = st->x; r.rnorm = st->rnorm;
        r.upd_idx = st->upd_idx; r.upd_val = st->upd_val; r.cnt = st->cnt; r.ctl = st->ctl;
    }
    e = cudaMemcpy(ws->table, host.data(), (size_t)c * sizeof(ChunkRef), cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemset(ws->r32, 0, b_r32);         // rows k..kp of every residual stay zero
    if (e != cudaSuccess) { cudaFree(ws->base); delete ws; return e; }
    st0->chunk_ws = ws;
    return cudaSuccess;
}

}  // namespace

void free_chunk_ws(sgc_state* st) {
    if (!st || !st->chunk_ws) return;
    cudaFree(st->chunk_ws->base);
    delete st->chunk_ws;
    st->chunk_ws = nullptr;
}

// The batched path serves chunk lists whose states are alike in everything but their moments: same shape, matrix, step
// count and hyper-parameters, Algorithm 2 as printed, small s and k, and no request for the speculative recovery.
bool chunked_batch_eligible(sgc_state* const* sts, int c) {
    const sgc_state* a = sts[0];
    if (a->s > kChunkMaxS || a->k > kChunkMaxK || (a->d & 3) || a->d >= (1ll << 31) || c > (1 << 20)) return false;
    for (int i = 0; i < c; ++i) {
        const sgc_state* b = sts[i];
        if (b->mode == SGC_MODE_SPECULATIVE || b->shared_support || b->residual_tol > 0.0 || b->profile) return false;
        if (b->d != a->d || b->k != a->k || b->s != a->s || b->seed != a->seed || b->t != a->t || b->lr != a->lr ||
            b->beta1 != a->beta1 || b->beta2 != a->beta2 || b->eps != a->eps || b->alpha != a->alpha || b->device != a->device)
            return false;
    }
    return true;
}

// One step of all chunks (the caller has already advanced every state's step count).
cudaError_t launch_chunked_batch(sgc_state* const* sts, int c, const float* grad, float* weight, cudaStream_t stream,
                                 int* launches) {
    sgc_state* st0 = sts[0];
    cudaError_t e = ensure_ws(sts, c);
    if (e != cudaSuccess) return e;
    const ChunkWs* ws = st0->chunk_ws;
    ChunkArgs a;
    a.table = ws->table; a.c = c; a.k = st0->k; a.s = st0->s; a.kp = ws->kp; a.dc = st0->d;
    a.seed_lo = (uint32_t)(st0->seed & 0xFFFFFFFFu); a.seed_hi = (uint32_t)(st0->seed >> 32);
    a.sigma = (double)(float)(1.0 / sqrt((double)st0->k));
    a.r32 = ws->r32; a.cand = ws->cand; a.splits = ws->splits;
    a.cols_per_split = (int)((st0->d + ws->splits - 1) / ws->splits);
    const int tile = ws->kp <= 64 ? 256 : 128;
    a.cols_per_split = (a.cols_per_split + tile - 1) / tile * tile;
    const double b1 = (double)st0->beta1, b2 = (double)st0->beta2;
    const double c1 = 1.0 - pow(b1, (double)st0->t), c2 = 1.0 - pow(b2, (double)st0->t);
    const int s = st0->s;
    if (s <= 1) k_chunk_front<1><<<c, kFrontThreads, 0, stream>>>(a, grad, b1, b2, c1, c2);
    else if (s <= 2) k_chunk_front<2><<<c, kFrontThreads, 0, stream>>>(a, grad, b1, b2, c1, c2);
    else if (s <= 4) k_chunk_front<4><<<c, kFrontThreads, 0, stream>>>(a, grad, b1, b2, c1, c2);
    else if (s <= 8) k_chunk_front<8><<<c, kFrontThreads, 0, stream>>>(a, grad, b1, b2, c1, c2);
    else k_chunk_front<16><<<c, kFrontThreads, 0, stream>>>(a, grad, b1, b2, c1, c2);
    *launches += 1;
    size_t smem = 0;
    switch (ws->kp) {
        case 8: e = corr_setup<8>(&smem); break;
        case 16: e = corr_setup<16>(&smem); break;
        case 32: e = corr_setup<32>(&smem); break;
        case 64: e = corr_setup<64>(&smem); break;
        default: e = corr_setup<128>(&smem); break;
    }
    if (e != cudaSuccess) return e;
    for (int iter = 0; iter < s; ++iter) {
        switch (ws->kp) {
            case 8: corr_launch<8>(a, iter, smem, stream); break;
            case 16: corr_launch<16>(a, iter, smem, stream); break;
            case 32: corr_launch<32>(a, iter, smem, stream); break;
            case 64: corr_launch<64>(a, iter, smem, stream); break;
            default: corr_launch<128>(a, iter, smem, stream); break;
        }
        k_chunk_pick<<<2 * c, 32, 0, stream>>>(a, iter);
        *launches += 2;
    }
    k_chunk_scatter<<<c, 32, 0, stream>>>(a, weight, (double)st0->alpha, (double)st0->eps, (double)st0->lr);
    *launches += 1;
    return cudaGetLastError();
}

}  // namespace sgc
