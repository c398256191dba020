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

// Returns (in every thread) the s-th largest key of src[0..n).  hist: kDigits words of shared memory.
template <class Src>
__device__ unsigned long long block_kth_largest(Src src, unsigned long long n, unsigned int s, unsigned int* hist,
                                                unsigned int* scan, unsigned long long* bcast) {
    unsigned long long prefix = 0ull, mask = 0ull;
    unsigned int need = s;
    int shift = 64;
    while (shift > 0) {
        const int bits = shift >= kDigitBits ? kDigitBits : shift;
        shift -= bits;
        const unsigned int dm = (1u << bits) - 1u;
        for (int b = threadIdx.x; b < kDigits; b += kPickThreads) hist[b] = 0u;
        __syncthreads();
        for (unsigned long long i = threadIdx.x; i < n; i += kPickThreads) {
            const unsigned long long key = src(i);
            if ((key & mask) == prefix) atomicAdd(&hist[(unsigned int)(key >> shift) & dm], 1u);
        }
        __syncthreads();
        // scan from the top digit: thread t owns reversed bins 2t, 2t+1
        const unsigned int r0 = hist[kDigits - 1 - 2 * threadIdx.x], r1 = hist[kDigits - 2 - 2 * threadIdx.x];
        unsigned int v = r0 + r1;
        const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
        unsigned int incl = v;
        for (int o = 1; o < 32; o <<= 1) { const unsigned int t = __shfl_up_sync(0xffffffffu, incl, o); if (lane >= o) incl += t; }
        if (lane == 31) scan[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            unsigned int w = scan[lane], wi = w;
            for (int o = 1; o < 32; o <<= 1) { const unsigned int t = __shfl_up_sync(0xffffffffu, wi, o); if (lane >= o) wi += t; }
            scan[lane] = wi - w;                            // exclusive offset of each warp
        }
        __syncthreads();
        const unsigned int excl = scan[warp] + incl - v;    // keys in strictly higher bins than mine
        if (excl < need && need <= excl + v) {              // exactly one thread
            unsigned int digit, used;
            if (need <= excl + r0) { digit = kDigits - 1 - 2 * threadIdx.x; used = excl; }
            else { digit = kDigits - 2 - 2 * threadIdx.x; used = excl + r0; }
            bcast[0] = (unsigned long long)digit;
            bcast[1] = (unsigned long long)(need - used);
        }
        __syncthreads();
        prefix |= bcast[0] << shift;
        mask |= (unsigned long long)dm << shift;
        need = (unsigned int)bcast[1];
        __syncthreads();
    }
    return prefix;
}

__global__ void __launch_bounds__(kPickThreads)
k_pick(const float* __restrict__ grad, unsigned long long d, unsigned int s, const unsigned long long* __restrict__ cand,
       Counters* __restrict__ cnt, uint32_t* __restrict__ sel_idx, float* __restrict__ sel_val) {
    __shared__ unsigned int hist[kDigits];
    __shared__ unsigned int scan[32];
    __shared__ unsigned long long bcast[2];
    __shared__ uint32_t picked[kMaxS];
    __shared__ unsigned int n_out;
    const unsigned int count = cnt->sel_count;
    const bool use_cand = (count >= s) && (count <= (unsigned int)kSelCap);
    if (threadIdx.x == 0) n_out = 0u;
    for (int i = threadIdx.x; i < kMaxS; i += kPickThreads) picked[i] = 0xFFFFFFFFu;
    __syncthreads();
    if (use_cand) {
        CandSource src{cand};
        const unsigned long long kth = block_kth_largest(src, count, s, hist, scan, bcast);
        for (unsigned int i = threadIdx.x; i < count; i += kPickThreads) {
            const unsigned long long key = cand[i];
            if (key >= kth) picked[atomicAdd(&n_out, 1u)] = ~(uint32_t)key;
        }
    } else {
        if (threadIdx.x == 0) atomicOr(&cnt->status, (unsigned int)SGC_STATUS_SELECT_FALLBACK);
        GradSource src{grad};
        const unsigned long long kth = block_kth_largest(src, d, s, hist, scan, bcast);
        for (unsigned long long i = threadIdx.x; i < d; i += kPickThreads) {
            const unsigned long long key = src(i);
            if (key >= kth) {
                if ((key >> 32) >= 0x7F800000ull) atomicOr(&cnt->status, (unsigned int)SGC_STATUS_NONFINITE_INPUT);
                picked[atomicAdd(&n_out, 1u)] = (uint32_t)i;
            }
        }
    }
    __syncthreads();
    // ascending index order: bitonic sort of 1024 slots (unused slots hold 0xFFFFFFFF and sink to the end)
    for (unsigned int size = 2; size <= (unsigned int)kMaxS; size <<= 1) {
        for (unsigned int stride = size >> 1; stride > 0; stride >>= 1) {
            const unsigned int i = threadIdx.x, j = i ^ stride;
            if (j > i) {
                const uint32_t a = picked[i], b = picked[j];
                const bool up = ((i & size) == 0);
                if ((a > b) == up) { picked[i] = b; picked[j] = a; }
            }
            __syncthreads();
        }
    }
    if (threadIdx.x < s) {
        const uint32_t idx = picked[threadIdx.x];
        sel_idx[threadIdx.x] = idx;
        sel_val[threadIdx.x] = grad[idx];
    }
}

// Launch geometry of the selection for a vector of length d with s kept entries: one definition for every caller.
struct SelectPlan {
    int direct;                 // the whole vector fits in the candidate list: no threshold needed
    unsigned int n_chunks;      // sample: 256-element chunks, between 2^10 and 2^16 of them
    unsigned int target;        // rank in the sample that corresponds to max(2048, 8 s) survivors in the vector
    int sample_grid;
    unsigned int filter_blocks;
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

// The three launches of the selection on `stream`; hist and the counters must be zero on entry (k_sample leaves them
// so for the next call).  `timed` (may be null) receives the per-kernel timing when profiling is on.
cudaError_t enqueue_select(const float* grad, unsigned long long d, int s, int sm_count, unsigned int* hist,
                           unsigned long long* cand, Counters* cnt, uint32_t* out_idx, float* out_val, cudaStream_t stream,
                           sgc_state* timed) {
    const SelectPlan p = plan_select(d, s, sm_count);
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
        k_pick<<<1, kPickThreads, 0, stream>>>(grad, d, (unsigned int)s, cand, cnt, out_idx, out_val);
    }
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_select(sgc_state* st, const float* grad, cudaStream_t stream, int* launches) {
    *launches += 3;
    return enqueue_select(grad, (unsigned long long)st->d, st->s, st->sm_count, st->sel_hist, st->sel_cand, st->cnt,
                          st->sel_idx, st->sel_val, stream, st);
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
    e = enqueue_select(grad, (unsigned long long)d, s, setup.sm_count, hist, cand, cnt, out_idx, out_val, cs, nullptr);
    if (e != cudaSuccess) return (int)e;
    if (out_status) k_copy_status<<<1, 1, 0, cs>>>(cnt, out_status);
    return (int)cudaGetLastError();
}
