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
//                     through registers while the current ones are worked on.  The rows of G are split over the CTAs of
//                     a thread-block cluster (n / 32 column blocks alone would not fill the SMs); their partial sums
//                     meet in the first CTA through distributed shared memory, added in rank order.
//   k_cesgc_back      W += B^T U for the r x n matrix U that the SGC core left (U = -eta N has at most s non-zeros):
//                     block = one column of U; columns without a non-zero cost one read of r values.
#include "sgc_internal.cuh"

#include <cooperative_groups.h>

namespace cg = cooperative_groups;

namespace sgc {
namespace {

constexpr int kProjCols = 32;            // columns of G per block
constexpr int kProjRows = 4;             // rows of B per thread
constexpr int kProjChunk = 64;           // rows of G per staged slab of B
constexpr int kCesgcMaxR = 64;

constexpr int kProjStage = 8;            // floats of each slab that one thread moves (at 256 threads: 64 x 32 floats)
constexpr int kProjMaxSplit = 8;         // CTAs of a cluster (the portable limit), each with a range of G's rows
constexpr int kProjResident = 4 * 148;   // CTAs of this kernel that the SMs hold at once (64 registers, 256 threads)

__global__ void __launch_bounds__(kProjCols * (kCesgcMaxR / kProjRows), 2)   // 64 registers: four blocks of 256 threads per SM
k_cesgc_project(const float* __restrict__ B, const float* __restrict__ G, float* __restrict__ P, int r, int m, int n) {
    __shared__ __align__(16) float bs[kCesgcMaxR][kProjChunk];       // B[:, row0 .. row0 + 64)
    __shared__ float gs[kProjChunk][kProjCols];                       // G[row0 .. row0 + 64, the block's columns]
    cg::cluster_group cluster = cg::this_cluster();
    const int groups = (r + kProjRows - 1) / kProjRows;
    const int jl = threadIdx.x % kProjCols, ig = threadIdx.x / kProjCols;
    const int j = blockIdx.x * kProjCols + jl;
    const bool work = ig < groups && j < n;
    // this CTA's rows of G: whole slabs, the same number for every CTA of the cluster (the last ranges may be empty)
    const int slabs = (m + kProjChunk - 1) / kProjChunk;
    const int part_rows = (slabs + (int)gridDim.y - 1) / (int)gridDim.y * kProjChunk;
    const int m_begin = (int)blockIdx.y * part_rows;
    const int m_end = m_begin + part_rows < m ? m_begin + part_rows : m;
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
                if (row0 + q < m_end) pb[u] = B[(size_t)i * m + row0 + q];
            }
            if (u < per_g && eg < ng) {
                const int q = eg / kProjCols, c = eg % kProjCols;
                const int col = blockIdx.x * kProjCols + c;
                if (row0 + q < m_end && col < n) pg[u] = G[(size_t)(row0 + q) * n + col];
            }
        }
    };
    float hi[kProjRows], lo[kProjRows];
#pragma unroll
    for (int u = 0; u < kProjRows; ++u) hi[u] = lo[u] = 0.0f;
    fetch(m_begin);
    for (int row0 = m_begin; row0 < m_end; row0 += kProjChunk) {
        __syncthreads();                                              // the previous slabs have been used up
#pragma unroll
        for (int u = 0; u < kProjStage; ++u) {
            const int e = threadIdx.x + u * blockDim.x;
            if (u < per_b && e < nb) bs[e / kProjChunk][e % kProjChunk] = pb[u];
            if (u < per_g && e < ng) gs[e / kProjCols][e % kProjCols] = pg[u];
        }
        __syncthreads();
        if (row0 + kProjChunk < m_end) fetch(row0 + kProjChunk);          // in flight while this slab is worked on
        if (!work) continue;
        // rows of this slab, rounded up to four: what lies beyond m_end was staged as zeros and adds nothing
        const int rows = ((m_end - row0 < kProjChunk ? m_end - row0 : kProjChunk) + 3) & ~3;
        for (int q = 0; q < rows; q += 4) {
            const float g4[4] = {gs[q][jl], gs[q + 1][jl], gs[q + 2][jl], gs[q + 3][jl]};
#pragma unroll
            for (int u = 0; u < kProjRows; ++u) {
                const float4 b4 = *reinterpret_cast<const float4*>(&bs[ig * kProjRows + u][q]);   // one address per warp
                const float bq[4] = {b4.x, b4.y, b4.z, b4.w};
#pragma unroll
                for (int e = 0; e < 4; ++e) {                         // ascending rows of G: the order of the sums is fixed
                    const float p = __fmul_rn(bq[e], g4[e]);
                    const float pe = __fmaf_rn(bq[e], g4[e], -p);     // b g = p + pe exactly
                    const float t = __fadd_rn(hi[u], p);
                    const float v = __fsub_rn(t, hi[u]);
                    const float te = __fadd_rn(__fsub_rn(hi[u], __fsub_rn(t, v)), __fsub_rn(p, v));   // hi + p = t + te exactly
                    hi[u] = t;
                    lo[u] = __fadd_rn(lo[u], __fadd_rn(te, pe));
                }
            }
        }
    }
    // the partial sums of the cluster's CTAs, left in each one's shared memory (the slab of B is done with)
    __syncthreads();
    float* part_hi = &bs[0][0];
    float* part_lo = part_hi + kCesgcMaxR * kProjCols;
    static_assert(2 * kProjCols <= kProjChunk, "two 64 x 32 arrays in the slab of B");
    if (work) {
#pragma unroll
        for (int u = 0; u < kProjRows; ++u) {
            part_hi[(ig * kProjRows + u) * kProjCols + jl] = hi[u];
            part_lo[(ig * kProjRows + u) * kProjCols + jl] = lo[u];
        }
    }
    cluster.sync();
    if (cluster.block_rank() == 0 && work) {
        const unsigned split = cluster.num_blocks();
#pragma unroll
        for (int u = 0; u < kProjRows; ++u) {
            const int i = ig * kProjRows + u;
            if (i >= r) continue;
            double acc = 0.0;
            for (unsigned y = 0; y < split; ++y) {                    // rank order: the result does not depend on the schedule
                const float* h = cluster.map_shared_rank(part_hi, y);
                const float* l = cluster.map_shared_rank(part_lo, y);
                acc += (double)h[i * kProjCols + jl];
                acc += (double)l[i * kProjCols + jl];
            }
            P[(size_t)i * n + j] = (float)acc;
        }
    }
    cluster.sync();                                                   // nobody leaves while its sums may still be read
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
    const int col_blocks = (n + kProjCols - 1) / kProjCols;
    const int slabs = (m + kProjChunk - 1) / kProjChunk;
    int split = kProjResident / col_blocks;                                         // one wave; a function of the shape alone
    if (split > kProjMaxSplit) split = kProjMaxSplit;
    if (split > slabs / 2) split = slabs / 2;                                       // at least two slabs per CTA
    if (split < 1) split = 1;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)col_blocks, (unsigned)split, 1);
    cfg.blockDim = dim3((unsigned)threads, 1, 1);
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = 1; attr[0].val.clusterDim.y = (unsigned)split; attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr; cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, k_cesgc_project, B, G, P, r, m, n);
}

cudaError_t launch_cesgc_back(const float* B, const float* U, float* W, int r, int m, int n, cudaStream_t stream) {
    k_cesgc_back<<<n, 256, 0, stream>>>(B, U, W, r, m, n);
    return cudaGetLastError();
}

}  // namespace sgc
