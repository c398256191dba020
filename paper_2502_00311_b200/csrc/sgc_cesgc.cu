// CESGC (Section 4.4, "Compute Efficient SGC"): SGC runs on the projected gradient B G (r x n) instead of G (m x n), and
// its update goes back through B^T:  W <- W - eta B^T SGC(B G).  B (r x m, the first r left-singular vectors of a
// gradient, refreshed by the caller every few hundred steps) is an input here; the two projections around the SGC core
// are the kernels of this file.
//   k_cesgc_project   P = B G.  Thread = one column j of G and four rows of B; G is read row by row (coalesced over j),
//                     the rows of B come from shared memory as broadcasts.  Sums are carried as pairs of floats (error-free
//                     product through one FMA, error-free two-term sum: some 44 bits in all; fp64 arithmetic runs at a
//                     64th of the fp32 rate on this part and made this kernel 1.1 ms), and rounded to fp32 once at the
//                     end.  The top-s selection that follows decides on those values; a reference that forms B G in fp64
//                     gets the same fp32 numbers but for a few elements in ten thousand (entries much smaller than
//                     their terms), which differ by one ulp.  Slabs of B and G are staged in shared memory; the next ones travel
//                     through registers while the current ones are worked on.
//   k_cesgc_back      W += B^T U for the r x n matrix U that the SGC core left (U = -eta N has at most s non-zeros):
//                     block = one column of U; columns without a non-zero cost one read of r values.
#include "sgc_internal.cuh"

namespace sgc {
namespace {

constexpr int kProjCols = 32;            // columns of G per block
constexpr int kProjRows = 4;             // rows of B per thread
constexpr int kProjChunk = 64;           // rows of G per staged slab of B
constexpr int kCesgcMaxR = 64;

constexpr int kProjStage = 8;            // floats of each slab that one thread moves (at 256 threads: 64 x 32 floats)

__global__ void __launch_bounds__(kProjCols * (kCesgcMaxR / kProjRows))
k_cesgc_project(const float* __restrict__ B, const float* __restrict__ G, float* __restrict__ P, int r, int m, int n) {
    __shared__ float bs[kCesgcMaxR][kProjChunk];                      // B[:, row0 .. row0 + 64)
    __shared__ float gs[kProjChunk][kProjCols];                       // G[row0 .. row0 + 64, the block's columns]
    const int groups = (r + kProjRows - 1) / kProjRows;
    const int jl = threadIdx.x % kProjCols, ig = threadIdx.x / kProjCols;
    const int j = blockIdx.x * kProjCols + jl;
    const bool work = ig < groups && j < n;
    const int nb = r * kProjChunk, ng = kProjChunk * kProjCols;       // slab sizes
    const int per_b = (nb + blockDim.x - 1) / blockDim.x, per_g = (ng + blockDim.x - 1) / blockDim.x;   // <= kProjStage
    float pb[kProjStage], pg[kProjStage];                             // the next slabs, on their way through registers
    auto fetch = [&](int row0) {
#pragma unroll
        for (int u = 0; u < kProjStage; ++u) {
            const int eb = threadIdx.x + u * blockDim.x, eg = eb;
            pb[u] = 0.0f; pg[u] = 0.0f;
            if (u < per_b && eb < nb) {
                const int i = eb / kProjChunk, q = eb % kProjChunk;
                if (row0 + q < m) pb[u] = B[(size_t)i * m + row0 + q];
            }
            if (u < per_g && eg < ng) {
                const int q = eg / kProjCols, c = eg % kProjCols;
                const int col = blockIdx.x * kProjCols + c;
                if (row0 + q < m && col < n) pg[u] = G[(size_t)(row0 + q) * n + col];
            }
        }
    };
    float hi[kProjRows], lo[kProjRows];
#pragma unroll
    for (int u = 0; u < kProjRows; ++u) hi[u] = lo[u] = 0.0f;
    fetch(0);
    for (int row0 = 0; row0 < m; row0 += kProjChunk) {
        __syncthreads();                                              // the previous slabs have been used up
#pragma unroll
        for (int u = 0; u < kProjStage; ++u) {
            const int e = threadIdx.x + u * blockDim.x;
            if (u < per_b && e < nb) bs[e / kProjChunk][e % kProjChunk] = pb[u];
            if (u < per_g && e < ng) gs[e / kProjCols][e % kProjCols] = pg[u];
        }
        __syncthreads();
        if (row0 + kProjChunk < m) fetch(row0 + kProjChunk);          // in flight while this slab is worked on
        if (!work) continue;
        const int rows = m - row0 < kProjChunk ? m - row0 : kProjChunk;
        for (int q = 0; q < rows; ++q) {
            const float g = gs[q][jl];
#pragma unroll
            for (int u = 0; u < kProjRows; ++u) {
                const float b = bs[ig * kProjRows + u][q];
                const float p = __fmul_rn(b, g);
                const float pe = __fmaf_rn(b, g, -p);                 // b g = p + pe exactly
                const float t = __fadd_rn(hi[u], p);
                const float v = __fsub_rn(t, hi[u]);
                const float te = __fadd_rn(__fsub_rn(hi[u], __fsub_rn(t, v)), __fsub_rn(p, v));   // hi + p = t + te exactly
                hi[u] = t;
                lo[u] = __fadd_rn(lo[u], __fadd_rn(te, pe));
            }
        }
    }
    if (work) {
#pragma unroll
        for (int u = 0; u < kProjRows; ++u) {
            const int i = ig * kProjRows + u;
            if (i < r) P[(size_t)i * n + j] = (float)((double)hi[u] + (double)lo[u]);
        }
    }
}

__global__ void __launch_bounds__(256)
k_cesgc_back(const float* __restrict__ B, const float* __restrict__ U, float* __restrict__ W, int r, int m, int n) {
    __shared__ float us[kCesgcMaxR];
    __shared__ int idx[kCesgcMaxR];
    __shared__ int n_nz;
    const int j = blockIdx.x;
    if (threadIdx.x == 0) n_nz = 0;
    __syncthreads();
    if ((int)threadIdx.x < r) {
        const float u = U[(size_t)threadIdx.x * n + j];
        if (u != 0.0f) { const int slot = atomicAdd(&n_nz, 1); us[slot] = u; idx[slot] = threadIdx.x; }
    }
    __syncthreads();
    const int nz = n_nz;
    if (nz == 0) return;
    // ascending row order of B, whatever order the atomics gave: the sum below does not depend on the schedule
    if (threadIdx.x == 0) {
        for (int a = 1; a < nz; ++a) {
            const int ia = idx[a]; const float ua = us[a];
            int b = a - 1;
            while (b >= 0 && idx[b] > ia) { idx[b + 1] = idx[b]; us[b + 1] = us[b]; --b; }
            idx[b + 1] = ia; us[b + 1] = ua;
        }
    }
    __syncthreads();
    for (int row = threadIdx.x; row < m; row += 256) {
        double acc = 0.0;
        for (int a = 0; a < nz; ++a) acc += (double)B[(size_t)idx[a] * m + row] * (double)us[a];
        float* w = W + (size_t)row * n + j;
        *w = (float)((double)*w + acc);
    }
}

}  // namespace

bool cesgc_shape_ok(int r, int m, int n) { return r >= 1 && r <= kCesgcMaxR && m >= 1 && n >= 1; }

cudaError_t launch_cesgc_project(const float* B, const float* G, float* P, int r, int m, int n, cudaStream_t stream) {
    const int groups = (r + kProjRows - 1) / kProjRows;
    const int threads = kProjCols * groups < 256 ? 256 : kProjCols * groups;      // at least 256: the slabs are staged 8 floats per thread
    k_cesgc_project<<<(n + kProjCols - 1) / kProjCols, threads, 0, stream>>>(B, G, P, r, m, n);
    return cudaGetLastError();
}

cudaError_t launch_cesgc_back(const float* B, const float* U, float* W, int r, int m, int n, cudaStream_t stream) {
    k_cesgc_back<<<n, 256, 0, stream>>>(B, U, W, r, m, n);
    return cudaGetLastError();
}

}  // namespace sgc
