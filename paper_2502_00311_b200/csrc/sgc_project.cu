// a2 + a3 fused: p = A G~, q = A G~^2 (Eq. 4 and the equation after it; Algorithm 2) followed by the
// k-space Adam moments with bias correction (Algorithm 2).  One thread per row of A; the s selected
// columns of A are regenerated on the fly (k*s entries), sums are carried in fp64 in ascending column order.
#include "sgc_internal.cuh"

namespace sgc {
namespace {

constexpr int kProjThreads = 128;

__global__ void __launch_bounds__(kProjThreads)
k_project_adam(uint32_t seed_lo, uint32_t seed_hi, int k, int s, const uint32_t* __restrict__ sel_idx,
               const float* __restrict__ sel_val, float* __restrict__ M, float* __restrict__ V,
               double* __restrict__ p, double* __restrict__ q, double* __restrict__ y64, double* __restrict__ r64,
               float2* __restrict__ r32, Counters* __restrict__ cnt, double sigma, double b1, double b2, double c1,
               double c2) {
    extern __shared__ unsigned char smem_raw[];
    ColKey* keys = reinterpret_cast<ColKey*>(smem_raw);
    float* vals = reinterpret_cast<float*>(keys + s);
    for (int i = threadIdx.x; i < s; i += kProjThreads) {
        keys[i] = column_key(seed_lo, seed_hi, sel_idx[i]);
        vals[i] = sel_val[i];
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) {            // new step: reset the recovery bookkeeping
        cnt->done[0] = cnt->done[1] = 0;
        cnt->stopped[0] = cnt->stopped[1] = 0;
        cnt->n_upd = cnt->mismatch = cnt->negv = 0;
    }
    __syncthreads();
    const int row = blockIdx.x * kProjThreads + threadIdx.x;
    if (row >= k) return;
    double accp = 0.0, accq = 0.0;
    for (int i = 0; i < s; ++i) {
        const double a = sigma * (double)z_at(keys[i], (uint32_t)row);
        const double g = (double)vals[i];
        accp = accp + a * g;
        accq = accq + a * (g * g);
    }
    p[row] = accp;
    q[row] = accq;
    const float m = (float)(b1 * (double)M[row] + (1.0 - b1) * accp);
    const float v = (float)(b2 * (double)V[row] + (1.0 - b2) * accq);
    M[row] = m;
    V[row] = v;
    const double mh = (double)m / c1, vh = (double)v / c2;   // bias-corrected temporaries; state stays uncorrected
    y64[row] = mh; y64[k + row] = vh;
    r64[row] = mh; r64[k + row] = vh;
    r32[row] = make_float2((float)mh, (float)vh);
}

// SGCA re-projection (Appendix C, Algorithm 4): M <- A' OMP_A(M), V <- A' OMP_A(V) for a new matrix A'.
// OMP is scale-equivariant, OMP_A(M) = (1 - beta1^t) OMP_A(M^), so the recoveries of the step that has just run are
// reused (the paper notes that the results of the first call can be stored): row j of the new state is
// c * sum_l A'[j][lambda_l] x_l over the recovered support, summed in fp64 in the order of selection.
__global__ void __launch_bounds__(kProjThreads)
k_reproject(uint32_t seed_lo, uint32_t seed_hi, int k, int s, const uint32_t* __restrict__ lam, const double* __restrict__ x,
            const Counters* __restrict__ cnt, float* __restrict__ M, float* __restrict__ V, double sigma, double c1, double c2,
            SpecCtl* ctl) {
    extern __shared__ unsigned char smem_raw[];
    ColKey* keys = reinterpret_cast<ColKey*>(smem_raw);
    double* xs = reinterpret_cast<double*>(keys + 2 * s);
    const int done[2] = {cnt->done[0], cnt->done[1]};
    for (int i = threadIdx.x; i < 2 * s; i += kProjThreads) {
        const int m = i / s, l = i % s;
        if (l < done[m]) { keys[i] = column_key(seed_lo, seed_hi, lam[i]); xs[i] = x[i]; }
    }
    if (blockIdx.x == 0 && threadIdx.x == 0) ctl->list_version = ctl->list_version + 1;   // Gram matrix of the old A is void
    __syncthreads();
    const int row = blockIdx.x * kProjThreads + threadIdx.x;
    if (row >= k) return;
    for (int m = 0; m < 2; ++m) {
        double acc = 0.0;
        for (int l = 0; l < done[m]; ++l) acc = acc + sigma * (double)z_at(keys[m * s + l], (uint32_t)row) * xs[m * s + l];
        if (m == 0) M[row] = (float)(c1 * acc); else V[row] = (float)(c2 * acc);
    }
}

__global__ void k_z_block(uint32_t seed_lo, uint32_t seed_hi, long long row0, long long nrows, long long col0,
                          long long ncols, float* __restrict__ out) {
    const long long n = nrows * ncols;
    for (long long e = (long long)blockIdx.x * blockDim.x + threadIdx.x; e < n; e += (long long)gridDim.x * blockDim.x) {
        const long long r = e / ncols, c = e % ncols;
        const ColKey key = column_key(seed_lo, seed_hi, (uint32_t)(col0 + c));
        out[e] = z_at(key, (uint32_t)(row0 + r));
    }
}

}  // namespace

cudaError_t launch_project_adam(sgc_state* st, cudaStream_t stream, int* launches) {
    const double b1 = (double)st->beta1, b2 = (double)st->beta2;
    const double c1 = 1.0 - pow(b1, (double)st->t), c2 = 1.0 - pow(b2, (double)st->t);
    const double sigma = (double)(float)(1.0 / sqrt((double)st->k));
    const int grid = (st->k + kProjThreads - 1) / kProjThreads;
    const size_t smem = (size_t)st->s * (sizeof(ColKey) + sizeof(float));
    PhaseTimer timer(st, stream, kPhaseProject, 1);
    k_project_adam<<<grid, kProjThreads, smem, stream>>>((uint32_t)(st->seed & 0xFFFFFFFFu), (uint32_t)(st->seed >> 32),
                                                         st->k, st->s, st->sel_idx, st->sel_val, st->M, st->V, st->p,
                                                         st->q, st->y64, st->r64, st->r32, st->cnt, sigma, b1, b2, c1, c2);
    *launches += 1;
    return cudaGetLastError();
}

cudaError_t launch_reproject(sgc_state* st, uint64_t new_seed, cudaStream_t stream) {
    const double b1 = (double)st->beta1, b2 = (double)st->beta2;
    const double c1 = 1.0 - pow(b1, (double)st->t), c2 = 1.0 - pow(b2, (double)st->t);
    const double sigma = (double)(float)(1.0 / sqrt((double)st->k));
    const int grid = (st->k + kProjThreads - 1) / kProjThreads;
    const size_t smem = 2 * (size_t)st->s * (sizeof(ColKey) + sizeof(double));
    k_reproject<<<grid, kProjThreads, smem, stream>>>((uint32_t)(new_seed & 0xFFFFFFFFu), (uint32_t)(new_seed >> 32), st->k, st->s,
                                                      st->lam, st->x, st->cnt, st->M, st->V, sigma, c1, c2, st->ctl);
    return cudaGetLastError();
}

cudaError_t launch_z_block(uint64_t seed, int64_t row0, int64_t nrows, int64_t col0, int64_t ncols, float* out,
                           cudaStream_t stream) {
    const long long n = nrows * ncols;
    if (n <= 0) return cudaSuccess;
    long long blocks = (n + 255) / 256;
    if (blocks > 148 * 16) blocks = 148 * 16;
    k_z_block<<<(unsigned int)blocks, 256, 0, stream>>>((uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32), row0, nrows,
                                                        col0, ncols, out);
    return cudaGetLastError();
}

}  // namespace sgc
