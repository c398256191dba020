// a1: G~ = Sparsify_s(G)  (Section 3.2: keep the s entries of largest magnitude, zero the rest).
//
// The answer is the set of the s largest keys  key(i) = (|g_i| bit pattern) << 32 | ~i  (unique; the
// ~i part sends ties to the lower index).  HBM traffic is one read of the gradient:
//   1. k_sample   reads <= 2^18..2^24 strided elements, builds a 12-bit magnitude histogram and derives a
//                 threshold tau under which roughly max(2048, 8s) elements of the whole vector lie above;
//   2. k_filter   streams the gradient once with 128-bit loads and appends every key >= tau to a
//                 candidate list (a few thousand entries);
//   3. k_pick     one block: exact radix select of the s largest candidate keys, sort by index.
// If the candidate list ends up with fewer than s or more than its capacity (degenerate value
// distributions, e.g. all magnitudes equal), k_pick instead runs the same exact radix select over the
// whole gradient (slow, still correct) and reports SGC_STATUS_SELECT_FALLBACK.
#include <mutex>

#include "sgc_internal.cuh"

namespace sgc {
namespace {

constexpr int kSampleThreads = 256;
constexpr int kSampleChunk = 256;

__device__ __forceinline__ uint32_t mag_bits(float g) { return __float_as_uint(g) & 0x7FFFFFFFu; }

__global__ void __launch_bounds__(kSampleThreads)
k_sample(const float* __restrict__ grad, unsigned long long d, unsigned int n_chunks, unsigned int target,
         unsigned int* __restrict__ hist, Counters* __restrict__ cnt, int direct) {
    if (direct) {   // the whole vector fits in the candidate list: no threshold needed
        if (blockIdx.x == 0 && threadIdx.x == 0) { cnt->sel_tau = 0u; cnt->sel_count = 0u; }
        return;
    }
    __shared__ unsigned int sh[kSelBins];
    __shared__ unsigned int part[kSampleThreads];
    __shared__ bool last;
    for (int b = threadIdx.x; b < kSelBins; b += kSampleThreads) sh[b] = 0u;
    __syncthreads();
    for (unsigned int c = blockIdx.x; c < n_chunks; c += gridDim.x) {
        const unsigned long long start = (((unsigned long long)c * d) / n_chunks) & ~3ull;
        const unsigned long long next = (c + 1 == n_chunks) ? d : ((((unsigned long long)(c + 1) * d) / n_chunks) & ~3ull);
        const unsigned long long i = start + threadIdx.x;
        if (i < next && i < start + kSampleChunk) atomicAdd(&sh[mag_bits(__ldg(grad + i)) >> 19], 1u);
    }
    __syncthreads();
    for (int b = threadIdx.x; b < kSelBins; b += kSampleThreads)
        if (sh[b]) atomicAdd(&hist[b], sh[b]);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = (atomicAdd(&cnt->sel_ticket, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!last) return;
    __threadfence();
    // last block: largest bin b such that (number of sampled keys in bins >= b) >= target
    constexpr int per = kSelBins / kSampleThreads;      // 16 bins per thread
    unsigned int mine = 0;
    for (int u = 0; u < per; ++u) mine += __ldcg(&hist[threadIdx.x * per + u]);
    part[threadIdx.x] = mine;
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned int acc = 0, tau = 0;
        int t = kSampleThreads - 1;
        for (; t >= 0; --t) { if (acc + part[t] >= target) break; acc += part[t]; }
        if (t >= 0) {
            int b = t * per + per - 1;
            for (; b >= t * per; --b) { acc += __ldcg(&hist[b]); if (acc >= target) break; }
            tau = (unsigned int)b << 19;
        }
        cnt->sel_tau = tau;
        cnt->sel_count = 0u;
        cnt->sel_ticket = 0u;
    }
    __syncthreads();
    for (int b = threadIdx.x; b < kSelBins; b += kSampleThreads) hist[b] = 0u;    // ready for the next step
}

__device__ __forceinline__ void consider(float g, unsigned long long i, unsigned int tau, unsigned long long* cand,
                                         Counters* cnt) {
    const uint32_t key = mag_bits(g);
    if (key >= tau) {
        if (key >= 0x7F800000u) atomicOr(&cnt->status, (unsigned int)SGC_STATUS_NONFINITE_INPUT);
        const unsigned int slot = atomicAdd(&cnt->sel_count, 1u);
        if (slot < (unsigned int)kSelCap) cand[slot] = ((unsigned long long)key << 32) | (uint32_t)(~(uint32_t)i);
    }
}

__global__ void __launch_bounds__(512)
k_filter(const float* __restrict__ grad, unsigned long long d, unsigned long long* __restrict__ cand,
         Counters* __restrict__ cnt) {
    const unsigned int tau = cnt->sel_tau;
    const unsigned long long n4 = d >> 2;
    const float4* g4 = reinterpret_cast<const float4*>(grad);
    const unsigned long long stride = (unsigned long long)gridDim.x * blockDim.x;
    unsigned long long i = (unsigned long long)blockIdx.x * blockDim.x + threadIdx.x;
    for (; i + 3 * stride < n4; i += 4 * stride) {            // four independent 128-bit loads in flight
        const float4 a = __ldcs(g4 + i), b = __ldcs(g4 + i + stride), c = __ldcs(g4 + i + 2 * stride),
                     e = __ldcs(g4 + i + 3 * stride);
        // largest sign-cleared bit pattern of the 16 values (orders magnitudes; NaN and infinity sort on top)
        const uint32_t m0 = max(max(mag_bits(a.x), mag_bits(a.y)), max(mag_bits(a.z), mag_bits(a.w)));
        const uint32_t m1 = max(max(mag_bits(b.x), mag_bits(b.y)), max(mag_bits(b.z), mag_bits(b.w)));
        const uint32_t m2 = max(max(mag_bits(c.x), mag_bits(c.y)), max(mag_bits(c.z), mag_bits(c.w)));
        const uint32_t m3 = max(max(mag_bits(e.x), mag_bits(e.y)), max(mag_bits(e.z), mag_bits(e.w)));
        const bool hit = max(max(m0, m1), max(m2, m3)) >= tau;
        if (hit) {
            const float v[16] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w, c.x, c.y, c.z, c.w, e.x, e.y, e.z, e.w};
#pragma unroll
            for (int u = 0; u < 16; ++u) consider(v[u], (i + (u >> 2) * stride) * 4 + (u & 3), tau, cand, cnt);
        }
    }
    for (; i < n4; i += stride) {
        const float4 a = __ldcs(g4 + i);
        consider(a.x, i * 4 + 0, tau, cand, cnt); consider(a.y, i * 4 + 1, tau, cand, cnt);
        consider(a.z, i * 4 + 2, tau, cand, cnt); consider(a.w, i * 4 + 3, tau, cand, cnt);
    }
    if (blockIdx.x == 0 && threadIdx.x < (d & 3ull)) {       // ragged tail
        const unsigned long long t = (n4 << 2) + threadIdx.x;
        consider(grad[t], t, tau, cand, cnt);
    }
}

// ---- exact selection of the s largest 64-bit keys by one block ---------------------------------------
constexpr int kPickThreads = 1024;
constexpr int kDigitBits = 11;
constexpr int kDigits = 1 << kDigitBits;

struct CandSource {
    const unsigned long long* cand;
    __device__ __forceinline__ unsigned long long operator()(unsigned long long i) const { return cand[i]; }
};
struct GradSource {
    const float* grad;
    __device__ __forceinline__ unsigned long long operator()(unsigned long long i) const {
        return ((unsigned long long)mag_bits(grad[i]) << 32) | (uint32_t)(~(uint32_t)i);
    }
};

// Returns (in every thread) the s-th largest key of src[0..n).  hist: kDigits words of shared memory.  NT: threads of the block.
template <int NT, class Src>
__device__ unsigned long long block_kth_largest(Src src, unsigned long long n, unsigned int s, unsigned int* hist,
                                                unsigned int* scan, unsigned long long* bcast) {      // bcast: 3 words
    unsigned long long prefix = 0ull, mask = 0ull;
    unsigned int need = s;
    int shift = 64;
    while (shift > 0) {
        const int bits = shift >= kDigitBits ? kDigitBits : shift;
        shift -= bits;
        const unsigned int dm = (1u << bits) - 1u;
        for (int b = threadIdx.x; b < kDigits; b += NT) hist[b] = 0u;
        __syncthreads();
        for (unsigned long long i = threadIdx.x; i < n; i += NT) {
            const unsigned long long key = src(i);
            if ((key & mask) == prefix) atomicAdd(&hist[(unsigned int)(key >> shift) & dm], 1u);
        }
        __syncthreads();
        // scan from the top digit: thread t owns the reversed bins B t .. B t + B - 1
        constexpr int B = kDigits / NT;
        unsigned int r[B];
        unsigned int v = 0;
#pragma unroll
        for (int u = 0; u < B; ++u) { r[u] = hist[kDigits - 1 - (B * (int)threadIdx.x + u)]; v += r[u]; }
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        unsigned int incl = v;
        for (int o = 1; o < 32; o <<= 1) { const unsigned int t = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += t; }
        if (lane == 31) scan[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            unsigned int w = lane < NT / 32 ? scan[lane] : 0u, wi = w;
            for (int o = 1; o < 32; o <<= 1) { const unsigned int t = __shfl_up_sync(0xffffffffu, wi, o); if (lane >= o) wi += t; }
            scan[lane] = wi - w;                            // exclusive offset of each warp
        }
        __syncthreads();
        const unsigned int excl = scan[warp] + incl - v;    // keys in strictly higher bins than mine
        if (excl < need && need <= excl + v) {              // exactly one thread
            unsigned int used = excl, digit = 0, in_bin = 0;
#pragma unroll
            for (int u = 0; u < B; ++u) {
                if (in_bin == 0u && need <= used + r[u]) { digit = kDigits - 1 - (B * threadIdx.x + u); in_bin = r[u]; }
                else if (in_bin == 0u) used += r[u];
            }
            bcast[0] = (unsigned long long)digit;
            bcast[1] = (unsigned long long)(need - used);
            bcast[2] = (unsigned long long)in_bin;
        }
        __syncthreads();
        prefix |= bcast[0] << shift;
        mask |= (unsigned long long)dm << shift;
        need = (unsigned int)bcast[1];
        const bool whole_bin = bcast[2] == bcast[1];        // every key of the boundary bin is wanted: its lowest possible
        __syncthreads();                                    // key (remaining digits zero) is a valid threshold
        if (whole_bin) break;
    }
    return prefix;
}

// shared memory of the exact selection (one block)
struct PickSmem {
    unsigned int hist[kDigits];
    unsigned int scan[32];
    unsigned long long bcast[3];
    uint32_t picked[kMaxS];
    unsigned int n_out;
};

// The s largest keys among `count` candidates (or, when the candidate list cannot serve -- fewer than s entries or an
// overflow -- among all d entries of the gradient: slow, exact, flagged), sorted by index, with their values.
template <int NT>
__device__ void pick_block(PickSmem& sm, const float* __restrict__ grad, unsigned long long d, unsigned int s,
                           const unsigned long long* __restrict__ cand, unsigned int count, Counters* __restrict__ cnt,
                           uint32_t* __restrict__ sel_idx, float* __restrict__ sel_val) {
    const bool use_cand = (count >= s) && (count <= (unsigned int)kSelCap);
    if (threadIdx.x == 0) sm.n_out = 0u;
    for (int i = threadIdx.x; i < kMaxS; i += NT) sm.picked[i] = 0xFFFFFFFFu;
    __syncthreads();
    if (use_cand) {
        CandSource src{cand};
        const unsigned long long kth = block_kth_largest<NT>(src, count, s, sm.hist, sm.scan, sm.bcast);
        for (unsigned int i = threadIdx.x; i < count; i += NT) {
            const unsigned long long key = cand[i];
            if (key >= kth) sm.picked[atomicAdd(&sm.n_out, 1u)] = ~(uint32_t)key;
        }
    } else {
        if (threadIdx.x == 0) atomicOr(&cnt->status, (unsigned int)SGC_STATUS_SELECT_FALLBACK);
        GradSource src{grad};
        const unsigned long long kth = block_kth_largest<NT>(src, d, s, sm.hist, sm.scan, sm.bcast);
        for (unsigned long long i = threadIdx.x; i < d; i += NT) {
            const unsigned long long key = src(i);
            if (key >= kth) {
                if ((key >> 32) >= 0x7F800000ull) atomicOr(&cnt->status, (unsigned int)SGC_STATUS_NONFINITE_INPUT);
                sm.picked[atomicAdd(&sm.n_out, 1u)] = (uint32_t)i;
            }
        }
    }
    __syncthreads();
    // ascending index order: the indices are distinct, so the rank of one among the s kept is its place in the output (every
    // thread reads the same slot at the same time: a broadcast); exactly s slots are in use, the radix selection having
    // stopped on a threshold that s keys reach
    for (unsigned int i = threadIdx.x; i < s; i += NT) {
        const uint32_t idx = sm.picked[i];
        unsigned int rank = 0;
        for (unsigned int q = 0; q < s; ++q) rank += sm.picked[q] < idx ? 1u : 0u;
        sel_idx[rank] = idx;
        sel_val[rank] = grad[idx];
    }
}

// carry_out: the sampled threshold is left for the next call's one-kernel selection, which appends to an empty list
__global__ void __launch_bounds__(kPickThreads)
k_pick(const float* __restrict__ grad, unsigned long long d, unsigned int s, const unsigned long long* __restrict__ cand,
       Counters* __restrict__ cnt, uint32_t* __restrict__ sel_idx, float* __restrict__ sel_val, int carry_out) {
    __shared__ PickSmem sm;
    pick_block<kPickThreads>(sm, grad, d, s, cand, cnt->sel_count, cnt, sel_idx, sel_val);
    if (carry_out && threadIdx.x == 0) {
        cnt->sel_tau_next = cnt->sel_tau;
        cnt->sel_count = 0u;
    }
}

// ---- the one-kernel selection of a warm state ---------------------------------------------------------------
// Gradients of consecutive steps follow nearly the same law, so the threshold tau that left a few thousand survivors
// in one step serves the next: one kernel streams the gradient with the carried tau (one read of d floats, the only
// HBM traffic of a1), counts what lies in the 8 magnitude bins below tau as well (a bin is 1/16 of an octave, so the
// histogram reaches a factor 1.41 below tau), and the block that finishes last derives the next step's tau from that
// histogram and makes the exact pick.  A miss (fewer than s survivors, or more than the list holds: the law moved by
// a factor of several from one step to the next) is served by the same block with the exact selection over the whole
// gradient -- milliseconds instead of microseconds, flagged SGC_STATUS_SELECT_FALLBACK -- which also yields the next tau.
// The first step of a state has no tau and takes the sampled path (k_sample, k_filter, k_pick) instead.
constexpr int kFastLoads = 4;                       // 128-bit loads in flight per thread
constexpr int kFastThreads = 512;                   // three blocks per SM, four loads each: 96 KB in flight per SM
constexpr int kTailBins = 8;                        // histogram bins kept below tau

__device__ __forceinline__ void tail_count(float g, unsigned int floor_key, unsigned int* sh_hist) {
    const uint32_t key = mag_bits(g);
    if (key >= floor_key) atomicAdd(&sh_hist[key >> 19], 1u);
}

__global__ void __launch_bounds__(kFastThreads, 3)
k_select_fast(const float* __restrict__ grad, unsigned long long d, unsigned int s, unsigned int want,
              unsigned long long* __restrict__ cand, unsigned int* __restrict__ hist, Counters* __restrict__ cnt,
              uint32_t* __restrict__ sel_idx, float* __restrict__ sel_val) {
    __shared__ __align__(16) unsigned int sh_hist[kSelBins];
    __shared__ PickSmem sm;
    __shared__ unsigned int part[kFastThreads];
    __shared__ unsigned int next_bin;
    __shared__ bool last;
    unsigned int tau = cnt->sel_tau_next;
    if (tau == 0u) tau = 0x7F800000u;                // nothing usable carried: only non-finite entries pass; the exact path serves
    const unsigned int tau_bin = tau >> 19;
    const unsigned int floor_bin = tau_bin > (unsigned int)kTailBins ? tau_bin - kTailBins : 0u;
    const unsigned int floor_key = floor_bin << 19;
    for (int b = threadIdx.x; b < kSelBins; b += kFastThreads) sh_hist[b] = 0u;
    __syncthreads();
    const unsigned long long n4 = d >> 2;
    const float4* g4 = reinterpret_cast<const float4*>(grad);
    const unsigned long long stride = (unsigned long long)gridDim.x * kFastThreads;
    unsigned long long i = (unsigned long long)blockIdx.x * kFastThreads + threadIdx.x;
    for (; i + (kFastLoads - 1) * stride < n4; i += kFastLoads * stride) {
        float4 v[kFastLoads];
#pragma unroll
        for (int u = 0; u < kFastLoads; ++u) v[u] = __ldcs(g4 + i + u * stride);
        uint32_t m = 0u;
#pragma unroll
        for (int u = 0; u < kFastLoads; ++u)
            m = max(m, max(max(mag_bits(v[u].x), mag_bits(v[u].y)), max(mag_bits(v[u].z), mag_bits(v[u].w))));
        if (m >= floor_key) {
#pragma unroll
            for (int u = 0; u < kFastLoads; ++u) {
                const float e[4] = {v[u].x, v[u].y, v[u].z, v[u].w};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    tail_count(e[c], floor_key, sh_hist);
                    consider(e[c], (i + u * stride) * 4 + c, tau, cand, cnt);
                }
            }
        }
    }
    for (; i < n4; i += stride) {
        const float4 a = __ldcs(g4 + i);
        const float e[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
        for (int c = 0; c < 4; ++c) {
            tail_count(e[c], floor_key, sh_hist);
            consider(e[c], i * 4 + c, tau, cand, cnt);
        }
    }
    if (blockIdx.x == 0 && threadIdx.x < (d & 3ull)) {       // ragged tail
        const unsigned long long t = (n4 << 2) + threadIdx.x;
        tail_count(grad[t], floor_key, sh_hist);
        consider(grad[t], t, tau, cand, cnt);
    }
    __syncthreads();
    for (int b = floor_bin + threadIdx.x; b < kSelBins; b += kFastThreads)
        if (sh_hist[b]) atomicAdd(&hist[b], sh_hist[b]);
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) last = (atomicAdd(&cnt->sel_ticket2, 1u) == gridDim.x - 1);
    __syncthreads();
    if (!last) return;
    __threadfence();
    // ---- last block: next threshold from the histogram, then the exact pick --------------------------------------
    // the histogram comes into shared memory in one parallel read; thread t sums its bins, a block-wide suffix scan finds
    // the thread whose bins hold the crossing, and that thread walks them
    constexpr int per = kSelBins / kFastThreads;        // 8 bins per thread
    unsigned int mine = 0;
    for (int u = 0; u < per; ++u) { const unsigned int c = __ldcg(&hist[threadIdx.x * per + u]); sh_hist[threadIdx.x * per + u] = c; mine += c; }
    const unsigned int count = __ldcg(&cnt->sel_count);
    const bool hit = count >= s && count <= (unsigned int)kSelCap;
    if (threadIdx.x == 0) next_bin = floor_bin;         // when even the whole histogram holds fewer than `want`: its floor
    __syncthreads();
    {
        // keys in the bins of this and of higher threads: suffix sum, first inside each warp (shuffles), then over the warps
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        unsigned int incl = mine;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const unsigned int v = __shfl_down_sync(0xffffffffu, incl, o);
            if (lane + o < 32) incl += v;
        }
        if (lane == 0) part[warp] = incl;                   // the warp's total
        __syncthreads();
        unsigned int higher = 0;
        for (int w = warp + 1; w < kFastThreads / 32; ++w) higher += part[w];
        incl += higher;
        const unsigned int above = incl - mine;
        if (above < want && want <= incl) {              // exactly one thread
            unsigned int acc = above;
            for (int u = per - 1; u >= 0; --u) {
                acc += sh_hist[threadIdx.x * per + u];
                if (acc >= want) { next_bin = threadIdx.x * per + u; break; }
            }
        }
    }
    __syncthreads();
    for (int b = threadIdx.x; b < kSelBins; b += kFastThreads) hist[b] = 0u;    // the next step starts from zero
    const unsigned long long* src = cand;
    if (hit && count <= (unsigned int)(kSelBins / 2)) {
        // a short candidate list is staged in shared memory (the histogram has served its purpose): the digit passes of
        // the exact pick then read it from there
        __syncthreads();
        unsigned long long* staged = reinterpret_cast<unsigned long long*>(sh_hist);
        for (unsigned int e = threadIdx.x; e < count; e += kFastThreads) staged[e] = __ldcg(cand + e);
        __syncthreads();
        src = staged;
    }
    // a miss hands pick_block an empty list: it then selects exactly over the whole gradient and flags the fallback
    pick_block<kFastThreads>(sm, grad, d, s, src, hit ? count : 0u, cnt, sel_idx, sel_val);
    __syncthreads();
    if (threadIdx.x == 0) {
        unsigned int nb = next_bin;
        if (!hit) {
            // next threshold from the result itself: a quarter octave below the smallest kept magnitude
            uint32_t lo = 0xFFFFFFFFu;
            for (unsigned int e = 0; e < s; ++e) lo = min(lo, mag_bits(sel_val[e]));
            nb = (lo >> 19) > 4u ? (lo >> 19) - 4u : 1u;
        }
        if (nb < 1u) nb = 1u;
        cnt->sel_tau_next = nb << 19;
        cnt->sel_count = 0u;
        cnt->sel_ticket2 = 0u;
    }
}

// Launch geometry of the selection for a vector of length d with s kept entries: one definition for every caller.
struct SelectPlan {
    int direct;                 // the whole vector fits in the candidate list: no threshold needed
    unsigned int n_chunks;      // sample: 256-element chunks, between 2^10 and 2^16 of them
    unsigned int target;        // rank in the sample that corresponds to max(2048, 8 s) survivors in the vector
    int sample_grid;
    unsigned int filter_blocks;
    unsigned int want;          // survivors aimed at: max(2048, 8 s)
};

SelectPlan plan_select(unsigned long long d, int s, int sm_count) {
    SelectPlan p;
    p.direct = d <= (unsigned long long)kSelCap;
    unsigned long long n_chunks = d / 16384ull;
    if (n_chunks < 1024ull) n_chunks = 1024ull;
    if (n_chunks > 65536ull) n_chunks = 65536ull;
    unsigned long long n_sample = n_chunks * kSampleChunk;
    if (n_sample > d) n_sample = d;
    unsigned long long want = 8ull * (unsigned long long)s;
    if (want < 2048ull) want = 2048ull;
    unsigned long long target = (want * n_sample + d - 1) / d;       // rank in the sample
    if (target < 32ull) target = 32ull;
    p.want = (unsigned int)want;
    p.n_chunks = (unsigned int)n_chunks;
    p.target = (unsigned int)target;
    p.sample_grid = (int)(n_chunks < 4096ull ? n_chunks / 8 : 512);
    if (p.sample_grid < 1) p.sample_grid = 1;
    const unsigned long long n4 = d >> 2;
    unsigned long long blocks = (n4 + 512ull * 4ull - 1) / (512ull * 4ull);
    const unsigned long long max_blocks = (unsigned long long)sm_count * 4ull;
    if (blocks > max_blocks) blocks = max_blocks;
    if (blocks < 1) blocks = 1;
    p.filter_blocks = (unsigned int)blocks;
    return p;
}

// The launches of the selection on `stream`; hist and the counters must be zero on entry (the kernels leave them so for
// the next call).  warm: a threshold carried from the previous call exists, and the one-kernel selection runs; otherwise
// the sampled path (sample, filter, pick), which leaves its threshold behind when carry_out is set.  `timed` (may be null)
// receives the per-kernel timing when profiling is on.
cudaError_t enqueue_select(const float* grad, unsigned long long d, int s, int sm_count, unsigned int* hist,
                           unsigned long long* cand, Counters* cnt, uint32_t* out_idx, float* out_val, cudaStream_t stream,
                           sgc_state* timed, bool warm, bool carry_out, int* launches) {
    const SelectPlan p = plan_select(d, s, sm_count);
    if (warm && !p.direct) {
        PhaseTimer timer(timed, stream, kPhaseFilter, 1);
        k_select_fast<<<3 * sm_count, kFastThreads, 0, stream>>>(grad, d, (unsigned int)s, p.want, cand, hist, cnt, out_idx, out_val);
        *launches += 1;
        return cudaGetLastError();
    }
    {
        PhaseTimer timer(timed, stream, kPhaseSample, 1);
        k_sample<<<p.direct ? 1 : p.sample_grid, kSampleThreads, 0, stream>>>(grad, d, p.n_chunks, p.target, hist, cnt, p.direct);
    }
    {
        PhaseTimer timer(timed, stream, kPhaseFilter, 1);
        k_filter<<<p.filter_blocks, 512, 0, stream>>>(grad, d, cand, cnt);
    }
    {
        PhaseTimer timer(timed, stream, kPhasePick, 1);
        k_pick<<<1, kPickThreads, 0, stream>>>(grad, d, (unsigned int)s, cand, cnt, out_idx, out_val, carry_out && !p.direct ? 1 : 0);
    }
    *launches += 3;
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_select(sgc_state* st, const float* grad, cudaStream_t stream, int* launches) {
    // the first selection of a state samples its threshold; every later one carries it
    const cudaError_t e = enqueue_select(grad, (unsigned long long)st->d, st->s, st->sm_count, st->sel_hist, st->sel_cand,
                                         st->cnt, st->sel_idx, st->sel_val, stream, st, st->sel_warm, true, launches);
    if (e == cudaSuccess) st->sel_warm = true;
    return e;
}

}  // namespace sgc

// ------------------------------------------------------------------------------------------------
// sgc_sparsify_static: the top-s selection (a1) for callers that must not allocate device memory.
//
// Some hosts of this library cannot call cudaMalloc at the moment they need a selection: a training loop
// whose framework has already claimed all device memory for its own caching allocator (a cudaMalloc from
// a library then fails or fragments the pool), or a latency-critical thread for which cudaMalloc's implicit
// device-wide synchronisation would stall every other stream.  For them the scratch that the selection
// needs (threshold histogram, candidate list, counters: kStaticScratchBytes = 278 784 bytes) lives in a
// file-scope __device__ array that every GPU loading this library holds until the process exits.
//
// The array's name is only a host-side handle; kernels need its device address, which the first call on
// each device obtains with cudaGetSymbolAddress (that first call should therefore happen before any stream
// capture).  The call itself allocates nothing: no cudaMalloc, cudaFree or allocating library routine.
// All calls on one device share the array, and it keeps the previous call's contents: the parts that must
// start at zero are cleared on the caller's stream at the start of every call.  Two calls that overlap on
// the GPU (different streams, or different host threads) race on the array and give undefined results.
// ------------------------------------------------------------------------------------------------
namespace sgc {
namespace {

constexpr size_t kStaticCntOff = 0;                                              // Counters (padded to 256)
constexpr size_t kStaticHistOff = 256;                                           // u32[kSelBins]
constexpr size_t kStaticCandOff = kStaticHistOff + sizeof(unsigned int) * kSelBins;   // u64[kSelCap]
constexpr size_t kStaticScratchBytes = kStaticCandOff + sizeof(unsigned long long) * kSelCap;
static_assert(sizeof(Counters) <= 256, "counter block must fit its slot");
static_assert(kStaticScratchBytes == 278784, "documented size of the static scratch");

static __device__ __align__(256) unsigned char g_static_scratch[kStaticScratchBytes];

constexpr int kMaxDevices = 64;
struct StaticSetup { bool ready; unsigned char* ptr; int sm_count; };
StaticSetup g_static_setup[kMaxDevices];            // zero-initialised; written once per device
std::mutex g_static_mutex;

__global__ void k_copy_status(const Counters* __restrict__ cnt, uint32_t* __restrict__ out) { *out = cnt->status; }

}  // namespace
}  // namespace sgc

extern "C" SGC_API int sgc_sparsify_static(const float* grad, int64_t d, int32_t s, uint32_t* out_idx, float* out_val,
                                           uint32_t* out_status, void* stream) {
    using namespace sgc;
    if (!grad || !out_idx || !out_val) return SGC_ERR_NULL;
    if (d < 1 || s < 1 || (int64_t)s > d || d >= ((int64_t)1 << 32) || s > kMaxS) return SGC_ERR_DIM;
    if ((uintptr_t)grad & 15u) return SGC_ERR_ALIGN;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return (int)e;
    if (dev < 0 || dev >= kMaxDevices) return SGC_ERR_DIM;
    StaticSetup setup;
    {
        std::lock_guard<std::mutex> lock(g_static_mutex);
        if (!g_static_setup[dev].ready) {           // once per device, with that device current
            void* p = nullptr;
            e = cudaGetSymbolAddress(&p, g_static_scratch);
            if (e != cudaSuccess) return (int)e;
            int sms = 0;
            e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
            if (e != cudaSuccess) return (int)e;
            g_static_setup[dev].ptr = static_cast<unsigned char*>(p);
            g_static_setup[dev].sm_count = sms;
            g_static_setup[dev].ready = true;
        }
        setup = g_static_setup[dev];
    }
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    Counters* cnt = reinterpret_cast<Counters*>(setup.ptr + kStaticCntOff);
    unsigned int* hist = reinterpret_cast<unsigned int*>(setup.ptr + kStaticHistOff);
    unsigned long long* cand = reinterpret_cast<unsigned long long*>(setup.ptr + kStaticCandOff);
    // counters and histogram must start at zero; the candidate list is overwritten before it is read
    e = cudaMemsetAsync(setup.ptr, 0, kStaticCandOff, cs);
    if (e != cudaSuccess) return (int)e;
    int launches = 0;
    e = enqueue_select(grad, (unsigned long long)d, s, setup.sm_count, hist, cand, cnt, out_idx, out_val, cs, nullptr, false, false,
                       &launches);
    if (e != cudaSuccess) return (int)e;
    if (out_status) k_copy_status<<<1, 1, 0, cs>>>(cnt, out_status);
    return (int)cudaGetLastError();
}
