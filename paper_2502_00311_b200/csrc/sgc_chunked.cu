// MESGC (Section 4.4) with small per-chunk problems: c chunks of one flat vector, each an SGC problem of its own
// (own M, V; s_c <= 32 kept entries, k_c <= 256 rows), all sharing the matrix A (k_c x d/c) named by one seed.
// Run chunk by chunk this costs ~25 launches per chunk; here the whole step of all chunks takes 2 + 2 s_c launches:
//   k_chunk_front    block = chunk: exact top-s_c of the chunk (a1), p = A g~, q = A g~^2 and the k-space Adam moments
//                    (a2 + a3), residuals r = y for both moments
//   per OMP iteration (Algorithm 3, all 2c recoveries in lock-step, which is where the shared A pays: a column of A is
//   generated once and meets the residuals of every chunk):
//     k_chunk_corr   thread = one residual, block = 256 residuals x a range of columns: fp32 scores |<A_i,r>| / ||A_i||,
//                    best two columns of the range per residual
//     k_chunk_pick   block of 128 threads = one recovery: fp64 rescoring of the columns within 2e-3 of the best fp32 score, lowest
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
constexpr int kChunkMaxS = 32;
constexpr int kChunkMaxK = 256;

struct ChunkArgs {
    const ChunkRef* table;
    int c, k, s, kp;                     // kp: k rounded up to 8, 16, 32, 64, 128 or 256 (row stride of r32)
    long long dc;                        // columns per chunk
    uint32_t seed_lo, seed_hi;
    double sigma;
    float* r32;                          // [2c][kp]
    Cand* cand;                          // [2c][splits][2]
    int splits, cols_per_split;
    int early;                           // the iteration's kernels let their successor's blocks in at once (see after_previous_kernel)
    // tensor-core route (see ChunkWs)
    int kp64;
    uint16_t* rt; float* tau; float* inv_scale; unsigned int* rep_count; uint2* rep;
    double* rnv; unsigned char* unresolved; int* flags;
    double z_rep;
    int epoch0;                          // flags[0] == epoch0 + iteration: that iteration left a recovery unresolved
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
__host__ __device__ constexpr int corr_ks(int kp) { return kp > 64 ? kp / 64 : 1; }   // threads that share the rows of a residual: 64 rows each
__host__ __device__ constexpr int corr_tile(int kp) { return kp <= 64 ? 256 : (kp <= 128 ? 128 : 32); }   // columns per tile
__host__ __device__ constexpr int corr_group(int kp) { return kCorrBlock / corr_ks(kp); }   // recoveries per block

// The two kernels of an iteration are launched with programmatic stream serialization: the blocks of the next kernel may
// become resident while this one is still running, and wait here until it has completed and its writes are visible.
// Nothing of another kernel's output is touched before this call.  (A launch without that attribute passes at once.)
// early: the successor's blocks are let in as soon as this kernel's blocks run, which pays when both grids fit the SMs
// together; otherwise they come in as this kernel's blocks leave (waiting blocks would hold the places of blocks with
// work to do: 0.57 -> 0.82 ms per step at 1024 chunks).
__device__ __forceinline__ void after_previous_kernel(int early) {
    asm volatile("griddepcontrol.wait;" ::: "memory");
    if (early) asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

// launch configuration of such a kernel
struct ChainedLaunch {
    cudaLaunchConfig_t cfg;
    cudaLaunchAttribute attr[1];
    ChainedLaunch(dim3 grid, dim3 block, size_t smem, cudaStream_t stream) : cfg{} {
        cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = stream;
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[0].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr; cfg.numAttrs = 1;
    }
};

// gate != nullptr: the launch is a fallback of the tensor-core route and returns at once unless *gate names this
// iteration (a.epoch): the word holds the epoch of the last iteration that left a recovery unresolved.
template <int KP>
__global__ void __launch_bounds__(kCorrBlock) k_chunk_corr(ChunkArgs a, int iter, const int* gate) {
    after_previous_kernel(a.early);
    if (gate != nullptr && *gate != a.epoch0 + iter) return;
    constexpr int TC = corr_tile(KP);
    constexpr int KS = corr_ks(KP), KL = KP / KS;                    // KS threads hold KL rows of a residual each
    constexpr int ZS = KP + 4 * KS;                                  // stride of a tile column: every row part is followed by four
                                                                     // floats, so that the KS parts a warp reads at once sit in different banks
    extern __shared__ float smem[];
    float* zt = smem;                                                // [TC][ZS]
    float* inv = smem + TC * ZS;                                     // [TC]
    float* n2p = inv + TC;                                           // [GPC][TC] partial ||Z_i||^2
    constexpr int GPC = kCorrBlock / TC, RG = KP / GPC;              // generating threads per column, rows each
    const int h = threadIdx.x % KS;
    const int res = blockIdx.y * (kCorrBlock / KS) + threadIdx.x / KS;     // recovery = 2 * chunk + moment
    const bool have = res < 2 * a.c;
    bool active = false;
    const uint32_t* sup = nullptr;
    float rr[KL];
#pragma unroll
    for (int q = 0; q < KL; ++q) rr[q] = 0.0f;
    if (have) {
        const ChunkRef& ref = a.table[res >> 1];
        active = ref.cnt->stopped[res & 1] == 0;
        sup = ref.lam + (size_t)(res & 1) * a.s;
        const float4* src = reinterpret_cast<const float4*>(a.r32 + (size_t)res * KP + h * KL);
#pragma unroll
        for (int q = 0; q < KL / 4; ++q) { const float4 f = src[q]; rr[4 * q] = f.x; rr[4 * q + 1] = f.y; rr[4 * q + 2] = f.z; rr[4 * q + 3] = f.w; }
    }
    float s1 = -1.0f, s2 = -1.0f;
    uint32_t i1 = kNoColumn, i2 = kNoColumn;
    const long long col0 = (long long)blockIdx.x * a.cols_per_split;
    long long col1 = col0 + a.cols_per_split;
    if (col1 > a.dc) col1 = a.dc;
    for (long long tile = col0; tile < col1; tile += TC) {
        __syncthreads();
        {
            // every thread generates: GPC threads share a column of the tile, RG rows each
            const int t = threadIdx.x % TC, part = threadIdx.x / TC;
            const long long col = tile + t;
            float n2 = 0.0f;
            float* dst = zt + t * ZS;
            if (col < col1) {
                const ColKey key = column_key(a.seed_lo, a.seed_hi, (uint32_t)col);
                uint32_t hw = key.ck + (uint32_t)(part * RG / 2) * key.mk;
#pragma unroll 4
                for (int q = 0; q < RG; q += 2) {
                    const int row = part * RG + q;
                    float2 z = half2_bits_to_float2(z_pair_from_word(hw));
                    hw += key.mk;
                    if (row >= a.k) z.x = 0.0f;
                    if (row + 1 >= a.k) z.y = 0.0f;
                    const int at = row + 4 * (row / KL);
                    dst[at] = z.x; dst[at + 1] = z.y;
                    n2 = __fmaf_rn(z.x, z.x, n2);
                    n2 = __fmaf_rn(z.y, z.y, n2);
                }
            } else {
                for (int q = 0; q < RG; ++q) { const int row = part * RG + q; dst[row + 4 * (row / KL)] = 0.0f; }
            }
            n2p[part * TC + t] = n2;
        }
        __syncthreads();
        if (threadIdx.x < TC) {
            float n2 = 0.0f;
#pragma unroll
            for (int g = 0; g < GPC; ++g) n2 += n2p[g * TC + threadIdx.x];
            inv[threadIdx.x] = n2 > 0.0f ? 1.0f / sqrtf(n2) : 0.0f;
        }
        __syncthreads();
        if (KS == 1 && !active) continue;                            // (with KS > 1 the shuffles below need every lane)
        const int n_here = (int)((col1 - tile) < TC ? (col1 - tile) : TC);
        // the score of tile column t for this thread's recovery (with KS > 1: every lane of the warp calls it)
        auto score = [&](int t) -> float {
            const float4* zc = reinterpret_cast<const float4*>(zt + t * ZS + h * (KL + 4));
            float acc0 = 0.0f, acc1 = 0.0f;
#pragma unroll
            for (int q = 0; q < KL / 4; ++q) {
                const float4 z = zc[q];                              // one address per row part: a broadcast
                acc0 = __fmaf_rn(z.x, rr[4 * q], acc0);
                acc1 = __fmaf_rn(z.y, rr[4 * q + 1], acc1);
                acc0 = __fmaf_rn(z.z, rr[4 * q + 2], acc0);
                acc1 = __fmaf_rn(z.w, rr[4 * q + 3], acc1);
            }
            float dot = acc0 + acc1;
#pragma unroll
            for (int o = 1; o < KS; o <<= 1) dot += __shfl_xor_sync(0xffffffffu, dot, o);   // the other parts of the rows
            return fabsf(dot);
        };
        auto offer = [&](float sc, int t) {                          // columns are offered in ascending order
            if (!(sc > s2)) return;
            const uint32_t col = (uint32_t)(tile + t);
            bool taken = false;
            for (int q = 0; q < iter; ++q) taken |= (sup[q] == col);
            if (taken) return;
            if (sc > s1) { s2 = s1; i2 = i1; s1 = sc; i1 = col; }
            else { s2 = sc; i2 = col; }
        };
        // from 64 rows on, four columns at a time: four independent chains of multiply-adds, and one compare decides
        // for all four whether any of them can enter the best two (with few rows the sweep is short, some lane of the
        // warp nearly always has a new best, and the grouped form only adds work: 63 -> 67 us per step at k_c = 8)
        int t = 0;
        for (; KP >= 64 && t + 4 <= n_here; t += 4) {
            const float4 iv = *reinterpret_cast<const float4*>(inv + t);
            const float sc0 = score(t) * iv.x, sc1 = score(t + 1) * iv.y, sc2 = score(t + 2) * iv.z, sc3 = score(t + 3) * iv.w;
            if (active && fmaxf(fmaxf(sc0, sc1), fmaxf(sc2, sc3)) > s2) {
                offer(sc0, t); offer(sc1, t + 1); offer(sc2, t + 2); offer(sc3, t + 3);
            }
        }
        for (; t < n_here; ++t) {
            const float sc = score(t) * inv[t];
            if (active) offer(sc, t);
        }
    }
    if (have && h == 0) {
        Cand* out = a.cand + ((size_t)res * a.splits + blockIdx.x) * 2;
        out[0].score = s1; out[0].idx = i1;
        out[1].score = s2; out[1].idx = i2;
    }
}

// ---- phase B of one OMP iteration: one block of kPickThreads threads per recovery ---------------------------------------------------
// Argmax among the columns that phase A left within 2e-3 (relative) of the best fp32 score, decided on fp64 scores
// <Z_i, r>^2 / ||Z_i||^2 with the lowest index winning ties; then Algorithm 3 (Appendix B) for the new column:
// g = A_Lambda^T a_new, c = F^T g, gamma = 1 / sqrt(g_ll - c^T c) (a pivot below 1e-10 g_ll ends this recovery),
// new column [-gamma F c; gamma] of F, a_j = gamma <a_new, r>, x = F a, r = y - A_Lambda x.
constexpr int kPickThreads = 128;        // one block per recovery

struct PickSmem {
    double gv[kChunkMaxS], cv[kChunkMaxS], xs[kChunkMaxS];
    double red[2][kPickThreads / 32];
    double csq;
    uint32_t cidx[kRescoreCap];
    int n_c;
    float fred[kPickThreads / 32];
};

// What the update of a pick reads of the recovery's state, fetched in one round trip (pick_stage), lives in dynamic
// shared memory sized by s_c and k_c (pick_dyn_bytes), so that small problems keep many blocks per SM:
// F [s][s], r [k], y [k], x0 [s] as doubles, then the columns z [s * k + 2] (they start at z[0] or z[1]: see pick_columns).
struct PickDyn { double* F; double* r; double* y; double* x0; uint16_t* z; };

__device__ __forceinline__ PickDyn pick_dyn(const ChunkArgs& a) {
    extern __shared__ double pick_mem[];
    PickDyn d;
    d.F = pick_mem; d.r = d.F + a.s * a.s; d.y = d.r + a.k; d.x0 = d.y + a.k;
    d.z = reinterpret_cast<uint16_t*>(d.x0 + a.s);
    return d;
}

size_t pick_dyn_bytes(int s, int k) {
    return (size_t)(s * s + 2 * k + s) * sizeof(double) + ((size_t)(s * k + 2) * sizeof(uint16_t) + 7) / 8 * 8;
}

// Copies the state that pick j of a recovery reads (the j earlier columns, F, x, y and the residual) into shared memory.
// All loads are independent of one another, so they cost one trip to global memory instead of one per phase of the update.
// A block-wide barrier has to follow before pick_finish reads them.
// The staged columns keep the position inside a 32-bit word that they have in global memory, so that they can be copied
// word by word.
__device__ __forceinline__ uint16_t* pick_columns(const PickDyn& dy, const uint16_t* zs) {
    return dy.z + (((uintptr_t)zs >> 1) & 1u);
}

__device__ __forceinline__ void pick_stage(const ChunkArgs& a, const ChunkRef& ref, int m, int j) {
    const int t = threadIdx.x, k = a.k, s = a.s;
    const PickDyn dy = pick_dyn(a);
    const uint16_t* zs = ref.zsel + (size_t)m * s * k;
    {
        uint16_t* zsh = pick_columns(dy, zs);
        const int n = j * k, first = (int)(zsh - dy.z);               // elements before the first whole word: 0 or 1
        if (n > 0) {
            const int words = (n - first) / 2;
            const uint32_t* src = reinterpret_cast<const uint32_t*>(zs + first);
            uint32_t* dst = reinterpret_cast<uint32_t*>(zsh + first);
            for (int w = t; w < words; w += kPickThreads) dst[w] = src[w];
            if (t == 0 && first) zsh[0] = zs[0];
            if (t == 1 && first + 2 * words < n) zsh[n - 1] = zs[n - 1];
        }
    }
    const double* F = ref.F + (size_t)m * s * s;
    for (int e = t; e < j * j; e += kPickThreads) {
        const int l = e / j, i = e - l * j;
        dy.F[l * s + i] = F[(size_t)l * s + i];
    }
    if (t < j) dy.x0[t] = ref.x[(size_t)m * s + t];
    const double* r = ref.r64 + (size_t)m * k;
    const double* y = ref.y64 + (size_t)m * k;
    for (int row = t; row < k; row += kPickThreads) { dy.r[row] = r[row]; dy.y[row] = y[row]; }
}

// sums of two values over the block; every thread receives both
__device__ __forceinline__ void pick_sum2(PickSmem& sh, double& a, double& b) {
    a = warp_sum_d(a); b = warp_sum_d(b);
    __syncthreads();
    if ((threadIdx.x & 31) == 0) { sh.red[0][threadIdx.x >> 5] = a; sh.red[1][threadIdx.x >> 5] = b; }
    __syncthreads();
    a = 0.0; b = 0.0;
#pragma unroll
    for (int w = 0; w < kPickThreads / 32; ++w) { a += sh.red[0][w]; b += sh.red[1][w]; }
}

// largest value over the block; every thread receives it
__device__ __forceinline__ float pick_max(PickSmem& sh, float v) {
    for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
    __syncthreads();
    if ((threadIdx.x & 31) == 0) sh.fred[threadIdx.x >> 5] = v;
    __syncthreads();
    v = sh.fred[0];
#pragma unroll
    for (int w = 1; w < kPickThreads / 32; ++w) v = fmaxf(v, sh.fred[w]);
    return v;
}

// the decision among the nc candidates in sh.cidx and the update of the recovery `res` with the winner as pick j
// (all kPickThreads threads of the block; nc is the same in every thread; pick_stage has run for this recovery)
__device__ void pick_finish(const ChunkArgs& a, const ChunkRef& ref, PickSmem& sh, int res, int j, int nc) {
    double* gv = sh.gv; double* cv = sh.cv; double* xs = sh.xs;
    const uint32_t* cidx = sh.cidx;
    const int m = res & 1, t = threadIdx.x, lane = t & 31, warp = t >> 5, k = a.k, s = a.s;
    double* r = ref.r64 + (size_t)m * k;
    const PickDyn dy = pick_dyn(a);
    const double* y = dy.y;
    if (nc == 0) {                                                   // no column left to pick (d/c = iterations made)
        if (t == 0) { ref.cnt->stopped[m] = 1; ref.cnt->done[m] = j; }
        return;
    }
    __syncthreads();                                                 // the staged state is complete
    // fp64 scores of the candidates
    double best_sc = -1.0, best_dot = 0.0, best_n2 = 1.0;
    uint32_t best_idx = kNoColumn;
    for (int c = 0; c < nc; ++c) {
        const uint32_t idx = cidx[c];
        const ColKey key = column_key(a.seed_lo, a.seed_hi, idx);
        double dot = 0.0, n2 = 0.0;
        for (int row = 2 * t; row < k; row += 2 * kPickThreads) {
            const float2 zz = half2_bits_to_float2(z_pair_from_word(key.ck + (uint32_t)(row >> 1) * key.mk));
            dot += (double)zz.x * dy.r[row];
            n2 += (double)zz.x * (double)zz.x;
            if (row + 1 < k) { dot += (double)zz.y * dy.r[row + 1]; n2 += (double)zz.y * (double)zz.y; }
        }
        pick_sum2(sh, dot, n2);
        const double sc = n2 > 0.0 ? dot * dot / n2 : 0.0;
        if (sc > best_sc || (sc == best_sc && idx < best_idx)) { best_sc = sc; best_idx = idx; best_dot = dot; best_n2 = n2; }
    }
    // the new column, binary16 bits (exact): kept in the state and beside the staged ones
    uint16_t* zs = ref.zsel + (size_t)m * s * k;
    uint16_t* zsh = pick_columns(dy, zs);
    double* F = ref.F + (size_t)m * s * s;
    double* xg = ref.x + (size_t)m * s;
    {
        const ColKey key = column_key(a.seed_lo, a.seed_hi, best_idx);
        uint16_t* znew = zs + (size_t)j * k;
        for (int row = 2 * t; row < k; row += 2 * kPickThreads) {
            const uint32_t z2 = z_pair_from_word(key.ck + (uint32_t)(row >> 1) * key.mk);
            znew[row] = (uint16_t)(z2 & 0xFFFFu);
            zsh[j * k + row] = (uint16_t)(z2 & 0xFFFFu);
            if (row + 1 < k) { znew[row + 1] = (uint16_t)(z2 >> 16); zsh[j * k + row + 1] = (uint16_t)(z2 >> 16); }
        }
    }
    __syncthreads();
    const double sig2 = a.sigma * a.sigma;
    const uint16_t* znew = zsh + j * k;
    for (int l = warp; l < j; l += kPickThreads / 32) {              // g = A_Lambda^T a_new, one earlier column per warp
        const uint16_t* zl = zsh + l * k;
        double acc = 0.0;
        for (int row = lane; row < k; row += 32) acc += (double)(half_bits_to_float(zl[row]) * half_bits_to_float(znew[row]));
        acc = warp_sum_d(acc);
        if (lane == 0) gv[l] = sig2 * acc;
    }
    __syncthreads();
    if (warp == 0) {
        double csq = 0.0;
        if (lane < j) {                                              // c = F^T g (F upper triangular, F(l, i) at F[l*s + i])
            double acc = 0.0;
            for (int l = 0; l <= lane; ++l) acc += dy.F[l * s + lane] * gv[l];
            cv[lane] = acc;
            csq = acc * acc;
        }
        csq = warp_sum_d(csq);
        if (lane == 0) sh.csq = csq;
    }
    __syncthreads();
    const double gnn = sig2 * best_n2;
    const double piv = gnn - sh.csq;
    if (!(piv > 1e-10 * gnn)) {                                      // dependent column: this recovery ends with j picks
        if (t == 0) {
            ref.cnt->stopped[m] = 1; ref.cnt->done[m] = j;
            atomicOr(&ref.cnt->status, (unsigned int)SGC_STATUS_DEPENDENT_COLUMN);
        }
        return;
    }
    const double gamma = 1.0 / sqrt(piv);
    const double aj = gamma * a.sigma * best_dot;
    if (warp == 0) {
        double fj = 0.0;                                             // this lane's entry of the new column of F
        if (lane < j) {
            double acc = 0.0;
            for (int l = lane; l < j; ++l) acc += dy.F[lane * s + l] * cv[l];
            fj = -gamma * acc;
            F[(size_t)lane * s + j] = fj;
        } else if (lane == j) {
            fj = gamma;
            F[(size_t)j * s + j] = fj;
        }
        if (lane <= j) {
            const double xo = lane < j ? dy.x0[lane] : 0.0;
            const double xn = xo + aj * fj;
            xg[lane] = xn;
            xs[lane] = xn;
        }
        if (lane == 0) { ref.acoef[(size_t)m * s + j] = aj; ref.lam[(size_t)m * s + j] = best_idx; }
    }
    __syncthreads();
    double rn2 = 0.0, unused = 0.0;
    for (int row = t; row < k; row += kPickThreads) {                // r = y - A_Lambda x
        double acc = 0.0;
        for (int l = 0; l <= j; ++l) acc += xs[l] * (double)half_bits_to_float(zsh[l * k + row]);
        const double rv = y[row] - a.sigma * acc;
        r[row] = rv;
        a.r32[(size_t)res * a.kp + row] = (float)rv;
        rn2 += rv * rv;
    }
    pick_sum2(sh, rn2, unused);
    if (t == 0) {
        ref.rnorm[(size_t)m * s + j] = sqrt(rn2);
        ref.cnt->done[m] = j + 1;
    }
}

// SIMT route: the candidates are the columns that phase A left within 2e-3 (relative) of the best fp32 score.
// only != nullptr: a second chance for the recoveries that the tensor-core route marked unresolved; skipped unless *gate
// names this iteration.
__global__ void __launch_bounds__(kPickThreads) k_chunk_pick(ChunkArgs a, int iter, const int* gate, const unsigned char* only) {
    __shared__ PickSmem sh;
    after_previous_kernel(a.early);
    if (gate != nullptr && *gate != a.epoch0 + iter) return;
    const int res = blockIdx.x, m = res & 1, t = threadIdx.x;
    if (only != nullptr && !only[res]) return;
    const ChunkRef ref = a.table[res >> 1];
    if (ref.cnt->stopped[m]) return;
    const int j = iter;
    pick_stage(a, ref, m, j);                                    // (pick_max's barriers come before anything reads it)
    const Cand* cc = a.cand + (size_t)res * a.splits * 2;
    const int n_entries = a.splits * 2;
    float mx = -1.0f;
    for (int e = t; e < n_entries; e += kPickThreads) if (cc[e].idx != kNoColumn) mx = fmaxf(mx, cc[e].score);
    if (t == 0) sh.n_c = 0;
    mx = pick_max(sh, mx);                                          // (its barriers also publish n_c = 0)
    const float thr = mx - 2e-3f * fabsf(mx);
    for (int e = t; e < n_entries; e += kPickThreads) {
        const Cand c = cc[e];
        if (c.idx != kNoColumn && c.score >= 0.0f && c.score >= thr) {
            const int slot = atomicAdd(&sh.n_c, 1);
            if (slot < kRescoreCap) sh.cidx[slot] = c.idx;
        }
    }
    __syncthreads();
    int nc = sh.n_c;
    if (nc > kRescoreCap) {
        if (t == 0) atomicOr(&ref.cnt->status, (unsigned int)SGC_STATUS_CANDIDATE_OVERFLOW);
        nc = kRescoreCap;
    }
    pick_finish(a, ref, sh, res, j, nc);
}

// ---- tensor-core route of phase A (k_c > 32) --------------------------------------------------------------------
// The contraction Z^T R of an iteration (all columns of A against the residuals of all recoveries) is what the screening
// pass of sgc_pass.cu computes on the tensor cores: k_chunk_rt lays the residuals out as its binary16 rows (each scaled
// by a power of two, rows k_c.. of the padded height zero) with a report threshold of z_rep noise deviations, the pass
// reports every (column, recovery) pair above it, and k_chunk_pick_rep takes the candidates from the reports: every
// column within twice the pass's error bound of the best report.  Whatever that cannot settle (no report, too many, a
// window that reaches below the threshold, a zero residual) is marked unresolved and goes through the fp32 route.
__global__ void __launch_bounds__(64) k_chunk_rt(ChunkArgs a, int n_rows, int iter) {
    __shared__ double red[2];
    const int row = blockIdx.x, t = threadIdx.x;
    const float inf = __int_as_float(0x7f800000);
    bool live = row < 2 * a.c;
    const ChunkRef* ref = live ? &a.table[row >> 1] : nullptr;
    if (live && ref->cnt->stopped[row & 1]) live = false;
    if (!live) {
        if (t == 0) { a.tau[row] = inf; a.rep_count[row] = 0u; if (row < 2 * a.c) a.unresolved[row] = 0; }
        return;
    }
    const double* r = ref->r64 + (size_t)(row & 1) * a.k;
    double rn2 = 0.0;
    for (int q = t; q < a.k; q += 64) rn2 += r[q] * r[q];
    rn2 = warp_sum_d(rn2);
    if ((t & 31) == 0) red[t >> 5] = rn2;
    __syncthreads();
    const double rn = sqrt(red[0] + red[1]);
    if (!(rn > 0.0) || !isfinite(rn)) {                               // nothing to screen: the fp32 route decides
        if (t == 0) { a.tau[row] = inf; a.rep_count[row] = 0u; a.unresolved[row] = 1; a.flags[0] = a.epoch0 + iter; }   // every writer of an iteration stores the same value
        return;
    }
    const double sc = residual_scale(rn);
    uint16_t* dst = a.rt + (size_t)row * a.kp64;
    for (int q = t; q < a.kp64; q += 64) dst[q] = q < a.k ? half_rn_bits(r[q] * sc) : (uint16_t)0;
    if (t == 0) {
        a.tau[row] = (float)(a.z_rep * rn / sqrt((double)a.k) * sc);
        a.inv_scale[row] = (float)(1.0 / sc);
        a.rep_count[row] = 0u;
        a.rnv[row] = rn;
        a.unresolved[row] = 0;
    }
}

__global__ void __launch_bounds__(kPickThreads) k_chunk_pick_rep(ChunkArgs a, int iter) {
    __shared__ PickSmem sh;
    const int res = blockIdx.x, m = res & 1, t = threadIdx.x, j = iter;
    const ChunkRef ref = a.table[res >> 1];
    if (ref.cnt->stopped[m] || a.unresolved[res]) return;
    pick_stage(a, ref, m, j);
    const unsigned int count = a.rep_count[res];
    const bool timed_out = a.flags[1] != 0;                          // a wait inside a pass of this step ran out: its reports are void
    bool give_up = timed_out || count == 0u || count > (unsigned int)kChunkRepCap;      // the same in every thread
    const uint2* rp = a.rep + (size_t)res * kChunkRepCap;
    const uint32_t* sup = ref.lam + (size_t)m * a.s;
    float smax = -1.0f;
    if (!give_up) {
        for (unsigned int e = t; e < count; e += kPickThreads) {
            const uint2 v = rp[e];
            bool taken = false;
            for (int q = 0; q < j; ++q) taken |= (sup[q] == v.x);
            if (!taken) smax = fmaxf(smax, __uint_as_float(v.y));
        }
        smax = pick_max(sh, smax);
        if (smax < 0.0f) give_up = true;
    }
    float lo = 0.0f;
    if (!give_up) {
        const double rn = a.rnv[res];
        lo = (float)((double)smax - 2.0 * screen_margin(rn, (double)smax, a.kp64));
        // the window must stay above the report threshold, or a column inside it may not have been reported
        if (!((double)lo > a.z_rep * rn / sqrt((double)a.k) * 1.001)) give_up = true;
    }
    if (!give_up) {
        if (t == 0) sh.n_c = 0;
        __syncthreads();
        for (unsigned int e = t; e < count; e += kPickThreads) {
            const uint2 v = rp[e];
            if (__uint_as_float(v.y) < lo) continue;
            bool taken = false;
            for (int q = 0; q < j; ++q) taken |= (sup[q] == v.x);
            if (taken) continue;
            const int slot = atomicAdd(&sh.n_c, 1);
            if (slot < kRescoreCap) sh.cidx[slot] = v.x;
        }
        __syncthreads();
        if (sh.n_c > kRescoreCap) give_up = true;
    }
    if (give_up) {
        if (t == 0) {
            a.unresolved[res] = 1; a.flags[0] = a.epoch0 + iter;
            if (timed_out) atomicOr(&ref.cnt->status, (unsigned int)SGC_STATUS_TIMEOUT);
        }
        return;
    }
    pick_finish(a, ref, sh, res, j, sh.n_c);
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

int padded_k(int k) { return k <= 8 ? 8 : k <= 16 ? 16 : k <= 32 ? 32 : k <= 64 ? 64 : k <= 128 ? 128 : 256; }

unsigned long long list_key(sgc_state* const* sts, int c) {
    unsigned long long h = 1469598103934665603ull;                   // FNV-1a
    for (int i = 0; i < c; ++i) {                                     // host object and its device allocation
        h ^= (unsigned long long)(uintptr_t)sts[i]; h *= 1099511628211ull;
        h ^= (unsigned long long)(uintptr_t)sts[i]->base; h *= 1099511628211ull;
    }
    h ^= sts[0]->seed; h *= 1099511628211ull;                        // the norm table belongs to one matrix
    return h ^ (unsigned long long)c;
}

template <int KP>
cudaError_t corr_setup(size_t* smem_out) {
    constexpr int TC = corr_tile(KP);
    const size_t smem = (size_t)(TC * (KP + 4 * corr_ks(KP)) + TC + kCorrBlock) * sizeof(float);
    *smem_out = smem;
    return cudaFuncSetAttribute(k_chunk_corr<KP>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
}

// blocks of k_chunk_corr<KP> that one SM holds at a time (0 on an error)
template <int KP>
int corr_resident() {
    size_t smem = 0;
    int blocks = 0;
    if (corr_setup<KP>(&smem) != cudaSuccess) return 0;
    if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&blocks, k_chunk_corr<KP>, kCorrBlock, smem) != cudaSuccess) return 0;
    return blocks;
}

int corr_resident(int kp) {
    switch (kp) {
        case 8: return corr_resident<8>();
        case 16: return corr_resident<16>();
        case 32: return corr_resident<32>();
        case 64: return corr_resident<64>();
        case 128: return corr_resident<128>();
        default: return corr_resident<256>();
    }
}

template <int KP>
cudaError_t corr_launch(const ChunkArgs& a, int iter, size_t smem, cudaStream_t stream, const int* gate) {
    dim3 grid((unsigned int)a.splits, (unsigned int)((2 * a.c + corr_group(KP) - 1) / corr_group(KP)));
    ChainedLaunch l(grid, dim3(kCorrBlock), smem, stream);
    return cudaLaunchKernelEx(&l.cfg, k_chunk_corr<KP>, a, iter, gate);
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
    // column splits: as many blocks as the SMs hold at a time (one wave), at least one tile per split
    const int groups = (2 * c + corr_group(ws->kp) - 1) / corr_group(ws->kp);
    const int tile = corr_tile(ws->kp);
    int resident = corr_resident(ws->kp);
    if (resident < 1) { delete ws; return cudaErrorLaunchOutOfResources; }
    int splits = resident * st0->sm_count / groups;
    const long long max_splits = (st0->d + tile - 1) / tile;
    if (splits > max_splits) splits = (int)max_splits;
    if (splits < 1) splits = 1;
    long long per = (st0->d + splits - 1) / splits;
    per = (per + tile - 1) / tile * tile;
    splits = (int)((st0->d + per - 1) / per);
    ws->splits = splits;
    auto up = [](size_t b) { return (b + 255) / 256 * 256; };
    const size_t b_table = up((size_t)c * sizeof(ChunkRef));
    const size_t b_r32 = up((size_t)2 * c * ws->kp * sizeof(float));
    const size_t b_cand = up((size_t)2 * c * splits * 2 * sizeof(Cand));
    // tensor-core route: worth it from k_c = 33 on; bounded by its report lists (n_rows * 16 KB)
    // (a pass has some 40 us of fixed cost: below ~1e9 multiply-adds per iteration the fp32 kernel is quicker)
    ws->tensor = ws->kp >= 64 && 2 * c <= 2048 && (double)st0->d * ws->kp * 2.0 * c >= 1.0e9;
    ws->kp64 = (st0->k + 63) / 64 * 64;
    ws->n_rows = (2 * c + 31) / 32 * 32;
    ws->passes = (ws->n_rows + kPassMaxN - 1) / kPassMaxN;
    size_t b_rt = 0, b_row = 0, b_rep = 0, b_norm = 0, b_rn = 0, b_un = 0, b_flags = 0;
    if (ws->tensor) {
        b_rt = up((size_t)ws->n_rows * ws->kp64 * sizeof(uint16_t));
        b_row = up((size_t)ws->n_rows * sizeof(float));
        b_rep = up((size_t)ws->n_rows * kChunkRepCap * sizeof(uint2));
        b_norm = up((size_t)st0->d * sizeof(uint16_t));
        b_rn = up((size_t)2 * c * sizeof(double));
        b_un = up((size_t)2 * c);
        b_flags = 256;
    }
    cudaError_t e = cudaMalloc(&ws->base, b_table + b_r32 + b_cand + b_rt + 3 * b_row + b_rep + b_norm + b_rn + b_un + b_flags);
    if (e != cudaSuccess) { delete ws; return e; }
    unsigned char* base = static_cast<unsigned char*>(ws->base);
    size_t off = 0;
    ws->table = reinterpret_cast<ChunkRef*>(base + off); off += b_table;
    ws->r32 = reinterpret_cast<float*>(base + off); off += b_r32;
    ws->cand = reinterpret_cast<Cand*>(base + off); off += b_cand;
    if (ws->tensor) {
        ws->rt = reinterpret_cast<uint16_t*>(base + off); off += b_rt;
        ws->tau = reinterpret_cast<float*>(base + off); off += b_row;
        ws->inv_scale = reinterpret_cast<float*>(base + off); off += b_row;
        ws->rep_count = reinterpret_cast<unsigned int*>(base + off); off += b_row;
        ws->rep = reinterpret_cast<uint2*>(base + off); off += b_rep;
        ws->inv_norm = reinterpret_cast<uint16_t*>(base + off); off += b_norm;
        ws->rnv = reinterpret_cast<double*>(base + off); off += b_rn;
        ws->unresolved = base + off; off += b_un;
        ws->flags = reinterpret_cast<int*>(base + off); off += b_flags;
        ws->z_rep = normal_tail_threshold((double)st0->d, 32.0);    // ~32 noise columns per recovery above the threshold
        const int h_flags[3] = {0, 0, 1};
        e = pass_configure(kPassMaxN);
        if (e == cudaSuccess) e = cudaMemset(ws->rt, 0, b_rt);
        if (e == cudaSuccess) e = cudaMemset(ws->unresolved, 0, b_un);
        if (e == cudaSuccess) e = cudaMemcpy(ws->flags, h_flags, sizeof(h_flags), cudaMemcpyHostToDevice);
        for (int p = 0; p < ws->passes && e == cudaSuccess; ++p) {
            const int n_p = ws->n_rows - p * kPassMaxN < kPassMaxN ? ws->n_rows - p * kPassMaxN : kPassMaxN;
            e = pass_encode_map(ws->tmap[p], ws->rt + (size_t)p * kPassMaxN * ws->kp64, n_p, ws->kp64);
        }
        if (e == cudaSuccess) e = launch_inv_norms(st0->seed, (uint64_t)st0->d, st0->k, ws->inv_norm, 0);
        if (e == cudaSuccess) e = cudaDeviceSynchronize();           // the table is ready before any stream uses it
        if (e != cudaSuccess) { cudaFree(ws->base); delete ws; return e; }
    }
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
    if (e == cudaSuccess) e = cudaDeviceSynchronize();               // set-up done before the caller's stream runs on it
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
    {
        const int groups = (2 * c + corr_group(ws->kp) - 1) / corr_group(ws->kp);
        a.early = (ws->splits * groups <= st0->sm_count && 2 * c <= st0->sm_count) ? 1 : 0;
    }
    a.cols_per_split = (int)((st0->d + ws->splits - 1) / ws->splits);
    const int tile = corr_tile(ws->kp);
    a.cols_per_split = (a.cols_per_split + tile - 1) / tile * tile;
    a.kp64 = ws->kp64; a.rt = ws->rt; a.tau = ws->tau; a.inv_scale = ws->inv_scale; a.rep_count = ws->rep_count; a.rep = ws->rep;
    a.rnv = ws->rnv; a.unresolved = ws->unresolved; a.flags = ws->flags; a.z_rep = ws->z_rep;
    // names the iterations of this step in the gate word: 1 + (step count mod 2^20) * 64 + iteration, never 0
    a.epoch0 = 1 + (int)((st0->t & 0xFFFFF) * 64);
    if (ws->tensor) {
        e = cudaMemsetAsync(ws->flags + 1, 0, sizeof(int), stream);      // the time-out flag is per step
        if (e != cudaSuccess) return e;
    }
    const double b1 = (double)st0->beta1, b2 = (double)st0->beta2;
    const double c1 = 1.0 - pow(b1, (double)st0->t), c2 = 1.0 - pow(b2, (double)st0->t);
    const int s = st0->s;
    if (s <= 1) k_chunk_front<1><<<c, kFrontThreads, 0, stream>>>(a, grad, b1, b2, c1, c2);
    else if (s <= 2) k_chunk_front<2><<<c, kFrontThreads, 0, stream>>>(a, grad, b1, b2, c1, c2);
    else if (s <= 4) k_chunk_front<4><<<c, kFrontThreads, 0, stream>>>(a, grad, b1, b2, c1, c2);
    else if (s <= 8) k_chunk_front<8><<<c, kFrontThreads, 0, stream>>>(a, grad, b1, b2, c1, c2);
    else if (s <= 16) k_chunk_front<16><<<c, kFrontThreads, 0, stream>>>(a, grad, b1, b2, c1, c2);
    else k_chunk_front<32><<<c, kFrontThreads, 0, stream>>>(a, grad, b1, b2, c1, c2);
    *launches += 1;
    size_t smem = 0;
    switch (ws->kp) {
        case 8: e = corr_setup<8>(&smem); break;
        case 16: e = corr_setup<16>(&smem); break;
        case 32: e = corr_setup<32>(&smem); break;
        case 64: e = corr_setup<64>(&smem); break;
        case 128: e = corr_setup<128>(&smem); break;
        default: e = corr_setup<256>(&smem); break;
    }
    if (e != cudaSuccess) return e;
    for (int iter = 0; iter < s; ++iter) {
        const int* gate = nullptr;
        if (ws->tensor) {
            // phase A on the tensor cores; the fp32 kernels below then only run for what the reports left open
            k_chunk_rt<<<ws->n_rows, 64, 0, stream>>>(a, ws->n_rows, iter);
            const int* gates[kPassMaxBatch] = {ws->flags + 2};
            int* errors[kPassMaxBatch] = {ws->flags + 1};
            for (int p = 0; p < ws->passes && e == cudaSuccess; ++p) {
                const int n_p = ws->n_rows - p * kPassMaxN < kPassMaxN ? ws->n_rows - p * kPassMaxN : kPassMaxN;
                const size_t r0 = (size_t)p * kPassMaxN;
                e = launch_pass(ws->tmap[p], st0->seed, (uint64_t)st0->d, ws->kp64, n_p, ws->tau + r0, ws->inv_scale + r0,
                                ws->inv_norm, ws->rep_count + r0, ws->rep + r0 * kChunkRepCap, kChunkRepCap, gates, errors,
                                st0->sm_count, stream, nullptr, nullptr, 0, st0->wait_limit_ns);
            }
            if (e != cudaSuccess) return e;
            k_chunk_pick_rep<<<2 * c, kPickThreads, pick_dyn_bytes(s, st0->k), stream>>>(a, iter);
            *launches += 2 + ws->passes;
            gate = ws->flags;
        }
        switch (ws->kp) {
            case 8: e = corr_launch<8>(a, iter, smem, stream, gate); break;
            case 16: e = corr_launch<16>(a, iter, smem, stream, gate); break;
            case 32: e = corr_launch<32>(a, iter, smem, stream, gate); break;
            case 64: e = corr_launch<64>(a, iter, smem, stream, gate); break;
            case 128: e = corr_launch<128>(a, iter, smem, stream, gate); break;
            default: e = corr_launch<256>(a, iter, smem, stream, gate); break;
        }
        {
            ChainedLaunch l(dim3((unsigned int)(2 * c)), dim3(kPickThreads), pick_dyn_bytes(s, st0->k), stream);
            const unsigned char* only = gate ? ws->unresolved : nullptr;
            if (e == cudaSuccess) e = cudaLaunchKernelEx(&l.cfg, k_chunk_pick, a, iter, gate, only);
        }
        if (e != cudaSuccess) return e;
        *launches += 2;
    }
    k_chunk_scatter<<<c, 32, 0, stream>>>(a, weight, (double)st0->alpha, (double)st0->eps, (double)st0->lr);
    *launches += 1;
    return cudaGetLastError();
}

}  // namespace sgc
