// Screening pass of the recovery (a4): the "Projection" line of Algorithm 3, p = A^T r, for a whole batch of
// residual vectors at once, as one dense contraction  C = A^T R  on the tcgen05 tensor cores.
//
//   A (k x d) is regenerated tile by tile by the CUDA cores straight into shared memory as binary16 (every Z
//   is a binary16 number; the generator's packed f16x2 arithmetic emits two rows per instruction), in the
//   K-major 128-byte-swizzled layout the UMMA descriptors expect;
//   R^T (N x k, binary16, one residual per row, each row scaled by a power of two) arrives chunk by chunk through TMA;
//   accumulators live in tensor memory (fp32, 128 lanes = 128 columns of A, N columns each);
//   the epilogue reads them back with tcgen05.ld, divides by the column norm ||Z_i|| (read from the state's table of
//   1 / ||Z_i||, filled once at creation; only the stand-alone pass of sgc_screen, which has no state, lets its
//   generator threads accumulate the norm as a by-product) and appends every (column, residual) pair whose score
//   |<Z_i, R_n>| / ||Z_i|| reaches the residual's threshold tau_n to that residual's report list.
//
// Nothing of size d is written: the output is the short report lists.  The pass serves two purposes of the
// speculative OMP (see sgc_recover.cu): it verifies that no column outside the candidate set beats a
// speculated pick, and it harvests new candidates.
//
// One persistent CTA per SM; warp roles: 0 = TMA producer, 1 = MMA issuer (owns the tensor-memory
// allocation), 2-5 = epilogue (one per 32-lane quadrant of tensor memory), 6-21 = generators.
// Every wait on an mbarrier is bounded (two seconds unless the caller sets another limit); on expiry the CTA records an
// error, leaves all loops, waits for the matrix operations and copies it still has in flight, frees its tensor memory and
// returns.
#include <cuda.h>

#include <mutex>

#include "sgc_internal.cuh"

namespace sgc {
namespace {

constexpr int kGenWarps = 16;                                // 512 generator threads: two per column of a sweep
constexpr int kFirstGenWarp = 6;                             // warps 2..5 are the epilogue
constexpr int kPassThreads = 32 * (kFirstGenWarp + kGenWarps);   // 704
constexpr int kTileCols = 128;                               // UMMA M: columns of A per accumulator tile
constexpr int kSuperCols = 2 * kTileCols;                    // columns of A per sweep over k
constexpr int kChunkRows = 64;                               // rows of A per pipeline stage (128 B of binary16)
constexpr int kTileBytes = kTileCols * kChunkRows * 2;       // 16384
constexpr int kNormRing = 8;
#ifndef SGC_PASS_SWAP
#define SGC_PASS_SWAP 1
#endif
constexpr bool kPassSwap = SGC_PASS_SWAP != 0;
constexpr unsigned long long kWaitLimitNs = 2000000000ull;   // default bound of every mbarrier wait

struct PassArgs {
    uint32_t seed_lo, seed_hi;
    unsigned long long d;
    int k, n;                    // n: residuals per pass (multiple of 32, <= 256)
    int stages, bufs;            // slots of the ring; accumulator buffers in tensor memory (2 when n <= 128)
    unsigned int num_super;      // ceil(d / 256)
    const float* tau;            // [n] thresholds (+inf = unused residual), in the units of the (scaled) rows of R^T
    const float* inv_scale;      // [n] factor that turns a score back into the caller's units, or nullptr for 1
    const uint16_t* inv_norm;    // [d] 1 / ||Z_i|| as binary16 (TABLE variant); otherwise the generators accumulate the norms
    unsigned int* rep_count;     // [n]
    uint2* rep;                  // [n][rep_cap]  (column, score bits)
    int rep_cap;
    // Two-level screening (single state only).  A full pass also collects, for every 8th residual of each stream,
    // every column scoring at least big_tau[row / 8] into the stream's "wide list" (some 10^5 columns; the bitmap lets a
    // column in once).  A list pass (list_ctl != nullptr) then screens only the columns of the two wide lists: a few
    // percent of the work of a full pass.
    const float* big_tau;        // [n / 8] or nullptr
    uint32_t* big_list;          // [2][big_cap]
    unsigned int* big_count;     // [2]
    unsigned int* big_bits;      // [2] bitmaps over [0, d), one per stream
    int big_cap, big_half;
    const SpecCtl* list_ctl;     // list pass: gate and list lengths come from the control block
    const int* sel; int sel_value;    // optional: the kernel returns at once unless *sel == sel_value (which of two widths runs)
    const int* gate[kPassMaxBatch];   // optional: the kernel returns at once when every *gate is 0 (one per batched state)
    int* error[kPassMaxBatch];        // set to 1 when a wait expired (one per batched state)
    unsigned long long wait_limit_ns; // bound of every mbarrier wait
};

// ---- PTX wrappers ---------------------------------------------------------------------------------------
__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// bounded wait: false when the limit expired or another thread of the CTA already gave up.  sleep_ns > 0 backs
// off between polls so that a waiting warp leaves the issue slots to the generator warps.  The clock is read every
// 64th poll, or at every poll when the limit is so short (under a millisecond) that the caller wants waits to expire.
__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned int sleep_ns,
                                            unsigned long long limit_ns) {
    const uint32_t every = limit_ns < 1000000ull ? 0u : 63u;
    unsigned long long t0 = 0;
    for (uint32_t i = 0;; ++i) {
        if (sleep_ns) __nanosleep(sleep_ns);
        if (mbar_try(bar, parity)) return true;
        if ((i & every) == every) {
            if (*abort_flag) return false;
            const unsigned long long t = global_ns();
            if (t0 == 0) t0 = t;
            else if (t - t0 > limit_ns) { *abort_flag = 1; return false; }
        }
    }
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag, unsigned int sleep_ns,
                                          unsigned long long limit_ns) {
    if (mbar_try(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, abort_flag, sleep_ns, limit_ns);
}
__device__ __forceinline__ void fence_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(map), "r"(bar), "r"(x), "r"(y)
        : "memory");
}

// shared-memory matrix descriptor: K-major operand, 128-byte swizzle, 8-row groups 1024 bytes apart
__device__ __forceinline__ uint64_t umma_desc(uint32_t smem_addr) {
    uint64_t desc = (uint64_t)((smem_addr & 0x3FFFFu) >> 4);
    desc |= (uint64_t)1 << 16;                 // leading byte offset (unused with swizzled K-major): 16 B
    desc |= (uint64_t)(1024 >> 4) << 32;       // stride byte offset between 8-row groups
    desc |= (uint64_t)1 << 46;                 // descriptor version of sm_100
    desc |= (uint64_t)2 << 61;                 // SWIZZLE_128B
    return desc;
}
// instruction descriptor: f16 x f16 -> fp32 (operand formats 0), both operands K-major, M = 128, N = n
__device__ __forceinline__ uint32_t umma_idesc(int n) {
    return (1u << 4) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(kTileCols >> 4) << 24);
}
__device__ __forceinline__ void umma_f16(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t acc) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(acc)
        : "memory");
}
__device__ __forceinline__ void umma_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&v)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void st_shared_v4(uint32_t addr, uint32_t a, uint32_t b, uint32_t c, uint32_t d) {
    asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(a), "r"(b), "r"(c), "r"(d) : "memory");
}

// ---- the kernel -----------------------------------------------------------------------------------------
// dynamic shared memory (after alignment to 1024 bytes):
//   stages x { A tile 0 (16 KB) | A tile 1 (16 KB) | R^T chunk (n x 128 B) }
//   norms  float[kNormRing][256][2]      partial ||Z_i||^2 of the two generator threads of each column
//   tau    float[256], 1 / tau float[256]
//   mbarriers: full[stages], empty[stages], acc_full[2], acc_empty[2], drain;  tensor-memory base;  abort flag
// WIDE: the two-level screening code (wide-list harvest, list passes) is compiled in
// SUB: 64-row chunks of A per slot of the ring, i.e. per hand-off between generators, TMA and MMA issuer (2 when the
// residual block is narrow enough for two slots of 128 rows: half as many barrier rounds per generated entry)
// SWAP (128 residual rows, table of norms, no wide lists): the residual chunk is the M operand and all 256 generated columns
// the N operand of one MMA per 16 rows (instead of two MMAs of N = 128 that both read the residual chunk); the accumulator then
// holds residuals along the lanes and columns of A along the tensor-memory columns
template <bool TABLE, bool WIDE, int SUB, bool SWAP>
__global__ void __launch_bounds__(kPassThreads, 1) k_pass(const __grid_constant__ CUtensorMap tmap, PassArgs a) {
    if (a.gate[0] != nullptr) {
        bool any = false;
#pragma unroll
        for (int q = 0; q < kPassMaxBatch; ++q) any = any || (a.gate[q] != nullptr && *a.gate[q] != 0);
        if (!any) return;
    }
    if (a.sel != nullptr && *a.sel != a.sel_value) return;
    // list pass: the columns are the concatenation of the two wide lists (every block reads the same lengths: nothing
    // writes them while a list pass runs)
    unsigned int list_n0 = 0, list_n = 0, num_super = a.num_super;
    if (WIDE && a.list_ctl != nullptr) {
        const volatile SpecCtl* lc = a.list_ctl;
        if (!lc->round_active || lc->fallback || lc->mini_done || lc->n_cand <= kSmallList) return;
        list_n0 = min(a.big_count[0], (unsigned int)a.big_cap);
        // the half-width pass serves the first stream alone: its own list is all it needs
        list_n = list_n0 + ((a.sel != nullptr && a.sel_value == 1) ? 0u : min(a.big_count[1], (unsigned int)a.big_cap));
        if (list_n == 0) return;
        num_super = (list_n + kSuperCols - 1) / kSuperCols;
        if (blockIdx.x >= num_super) return;
    }
    const bool listed = WIDE && a.list_ctl != nullptr;
    extern __shared__ unsigned char smem_raw[];
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    unsigned char* gen_base = smem_raw + (base - smem_u32(smem_raw));
    const int sub_bytes = 2 * kTileBytes + a.n * 128;      // one 64-row chunk: two tiles of A and the chunk of R^T
    const int stage_bytes = SUB * sub_bytes;
    const uint32_t norms_off = (uint32_t)a.stages * stage_bytes;
    float* norms = reinterpret_cast<float*>(gen_base + norms_off);
    float* tau_s = norms + kNormRing * kSuperCols * 2;
    float* itau_s = tau_s + 256;                                     // 1 / tau: a group of 16 residuals is skipped on one compare
    uint64_t* bars = reinterpret_cast<uint64_t*>(itau_s + 256);
    const uint32_t bar_full = smem_u32(bars), bar_empty = bar_full + 8u * a.stages;
    const uint32_t bar_accf = bar_empty + 8u * a.stages, bar_acce = bar_accf + 16u, bar_drain = bar_acce + 16u;
    uint32_t* tmem_slot = reinterpret_cast<uint32_t*>(bars + 2 * a.stages + 5);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(tmem_slot + 1);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int kc_count = a.k / kChunkRows;

    if (threadIdx.x == 0) {
        for (int s = 0; s < a.stages; ++s) {
            mbar_init(bar_full + 8u * s, kGenWarps + 1);
            mbar_init(bar_empty + 8u * s, 1);
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(bar_accf + 8u * b, 1);
            mbar_init(bar_acce + 8u * b, 4);
        }
        mbar_init(bar_drain, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        fence_async_smem();
    }
    for (int i = threadIdx.x; i < 256; i += kPassThreads) {
        const float tv = i < a.n ? a.tau[i] : __int_as_float(0x7f800000);
        tau_s[i] = tv;
        itau_s[i] = tv > 0.0f ? 1.0f / tv : 3.0e38f;                 // tau = +inf (unused residual) -> 0
    }
    if (warp == 1) {           // tensor memory: all 512 columns (the only CTA on this SM)
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(tmem_slot)), "r"(512u)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = *tmem_slot;
    const int acc_cols = 2 * a.n;              // tensor-memory columns of one accumulator buffer (two tiles)

    if (warp == 0) {
        // ---------------- TMA producer: one chunk of R^T per stage -----------------------------------------
        if (lane == 0) {
            uint32_t st = 0, ph = 0;
            bool ok = true;
            for (unsigned int sweep = blockIdx.x; ok && sweep < num_super; sweep += gridDim.x) {
                for (int kc = 0; kc < kc_count; kc += SUB) {
                    if (!mbar_wait(bar_empty + 8u * st, ph ^ 1u, abort_flag, 256, a.wait_limit_ns)) { ok = false; break; }
                    mbar_arrive_expect_tx(bar_full + 8u * st, (uint32_t)a.n * 128u * SUB);
#pragma unroll
                    for (int u = 0; u < SUB; ++u)
                        tma_load_2d(base + st * stage_bytes + u * sub_bytes + 2 * kTileBytes, &tmap, (kc + u) * kChunkRows, 0,
                                    bar_full + 8u * st);
                    if (++st == (uint32_t)a.stages) { st = 0; ph ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        // ---------------- MMA issuer ----------------------------------------------------------------------
        if (lane == 0) {
            const uint32_t idesc = umma_idesc(a.n);
            const uint32_t idesc_swap = umma_idesc(kSuperCols);      // M = 128 residual rows, N = 256 columns of A
            // descriptors differ only in their start-address field (units of 16 bytes): keep that word per stage
            const uint64_t desc_hi = umma_desc(0) & 0xFFFFFFFF00000000ull;
            const uint32_t desc_lo0 = (uint32_t)(umma_desc(base) & 0xFFFFFFFFull);
            const uint32_t stage_step = (uint32_t)stage_bytes >> 4;
            uint32_t st = 0, ph = 0, sweep_i = 0;
            bool ok = true;
            for (unsigned int sweep = blockIdx.x; ok && sweep < num_super; sweep += gridDim.x, ++sweep_i) {
                const uint32_t buf = sweep_i % a.bufs, use = sweep_i / a.bufs;
                if (!mbar_wait(bar_acce + 8u * buf, (use & 1u) ^ 1u, abort_flag, 32, a.wait_limit_ns)) { ok = false; break; }
                tc_fence_after();
                const uint32_t acc0 = tmem_base + buf * acc_cols, acc1 = acc0 + a.n;
                for (int kc = 0; kc < kc_count; kc += SUB) {
                    if (!mbar_wait(bar_full + 8u * st, ph, abort_flag, 0, a.wait_limit_ns)) { ok = false; break; }
                    tc_fence_after();
#pragma unroll
                    for (int u = 0; u < SUB; ++u) {
                        const uint32_t lo = desc_lo0 + st * stage_step + u * ((uint32_t)sub_bytes >> 4);
                        const uint32_t first = (kc + u) != 0 ? 1u : 0u;
#pragma unroll
                        for (int kk = 0; kk < kChunkRows / 16; ++kk) {
                            const uint64_t bdesc = desc_hi | (uint64_t)(lo + (2 * kTileBytes >> 4) + 2 * kk);
                            if (SWAP) {
                                // D[residual][column] += R_chunk (128 x 16) * Z (256 x 16)^T: both tiles of A are one N operand
                                umma_f16(acc0, bdesc, desc_hi | (uint64_t)(lo + 2 * kk), idesc_swap, kk != 0 ? 1u : first);
                            } else {
                                umma_f16(acc0, desc_hi | (uint64_t)(lo + 2 * kk), bdesc, idesc, kk != 0 ? 1u : first);
                                umma_f16(acc1, desc_hi | (uint64_t)(lo + (kTileBytes >> 4) + 2 * kk), bdesc, idesc, kk != 0 ? 1u : first);
                            }
                        }
                    }
                    umma_commit(bar_empty + 8u * st);        // frees the stage once these MMAs have read it
                    if (++st == (uint32_t)a.stages) { st = 0; ph ^= 1u; }
                }
                if (ok) umma_commit(bar_accf + 8u * buf);    // accumulators of this sweep complete
            }
        }
    } else if (warp < kFirstGenWarp) {
        // ---------------- epilogue: scores against thresholds ----------------------------------------------
        const int quad = warp & 3;
        uint32_t sweep_i = 0;
        bool ok = true;
        for (unsigned int sweep = blockIdx.x; ok && sweep < num_super; sweep += gridDim.x, ++sweep_i) {
            const uint32_t buf = sweep_i % a.bufs, use = sweep_i / a.bufs;
            if (!__all_sync(0xffffffffu, mbar_wait(bar_accf + 8u * buf, use & 1u, abort_flag, 512, a.wait_limit_ns))) { ok = false; break; }
            tc_fence_after();
            if (SWAP) {
                // this thread owns residual n_res; the 256 columns of the sweep run along the tensor-memory columns.  Each
                // epilogue warp keeps its own copy of the sweep's 1 / ||Z_i|| as floats (no barrier between the warps)
                const int n_res = quad * 32 + lane;
                const float tau_n = tau_s[n_res];
                float* inv_w = norms + (size_t)quad * kSuperCols;
                uint32_t* col_w = reinterpret_cast<uint32_t*>(norms + (size_t)(4 + quad) * kSuperCols);   // list pass: the columns
                __syncwarp();
#pragma unroll
                for (int q = 0; q < kSuperCols / 32; ++q) {
                    unsigned long long col = (unsigned long long)sweep * kSuperCols + q * 32 + lane;
                    if (listed) {
                        const unsigned int idx = (unsigned int)col;
                        col = idx < list_n0 ? a.big_list[idx] : (idx < list_n ? a.big_list[(size_t)a.big_cap + idx - list_n0] : a.d);
                        col_w[q * 32 + lane] = (uint32_t)col;
                    }
                    inv_w[q * 32 + lane] = col < a.d ? half_bits_to_float(a.inv_norm[col]) : 0.0f;
                }
                __syncwarp();
                // every 8th residual feeds the wide list of its stream (full passes of the two-level screening)
                const bool feeds = WIDE && a.big_tau != nullptr && !listed && (n_res & 7) == 0;
                const float wide_tau_n = feeds ? a.big_tau[n_res >> 3] : 0.0f;
                // wide-list hits of this warp are queued in shared memory and appended after the sweep, all at once: the two
                // dependent global atomics of an append then cost the warp two round trips per sweep instead of two per hit
                // (the warp's 32 residuals belong to one stream whenever the streams' blocks are multiples of 32 rows)
                uint32_t* queue = reinterpret_cast<uint32_t*>(norms + (size_t)(8 + quad) * kSuperCols);
                const bool queued = WIDE && (a.big_half & 31) == 0;
                if (WIDE && lane == 0) queue[0] = 0u;
                if (WIDE) __syncwarp();
#pragma unroll 1
                for (int c0 = 0; c0 < kSuperCols; c0 += 16) {
                    uint32_t v[16];
                    tmem_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + buf * acc_cols + c0, v);
                    float peak = 0.0f;
                    const float4* in4 = reinterpret_cast<const float4*>(inv_w + c0);
#pragma unroll
                    for (int i4 = 0; i4 < 4; ++i4) {
                        const float4 w = in4[i4];
                        peak = fmaxf(peak, fabsf(__uint_as_float(v[4 * i4])) * w.x);
                        peak = fmaxf(peak, fabsf(__uint_as_float(v[4 * i4 + 1])) * w.y);
                        peak = fmaxf(peak, fabsf(__uint_as_float(v[4 * i4 + 2])) * w.z);
                        peak = fmaxf(peak, fabsf(__uint_as_float(v[4 * i4 + 3])) * w.w);
                    }
                    if (feeds && peak >= wide_tau_n) {
                        const int m = n_res >= a.big_half ? 1 : 0;
                        unsigned int hits = 0u;
#pragma unroll
                        for (int i = 0; i < 16; ++i)
                            hits |= (fabsf(__uint_as_float(v[i])) * inv_w[c0 + i] >= wide_tau_n ? 1u : 0u) << i;
                        while (hits) {
                            const int i = __ffs(hits) - 1;
                            hits &= hits - 1u;
                            const unsigned long long col = (unsigned long long)sweep * kSuperCols + c0 + i;
                            if (queued) {
                                const unsigned int qs = atomicAdd(&queue[0], 1u) + 1u;
                                if (qs < (unsigned int)kSuperCols) { queue[qs] = (uint32_t)col; continue; }
                            }
                            const unsigned int bit = 1u << ((unsigned int)col & 31u);
                            if (!(atomicOr(&a.big_bits[(size_t)m * ((a.d + 31) >> 5) + (col >> 5)], bit) & bit)) {
                                const unsigned int slot = atomicAdd(&a.big_count[m], 1u);
                                if (slot < (unsigned int)a.big_cap) a.big_list[(size_t)m * a.big_cap + slot] = (uint32_t)col;
                            }
                        }
                    }
                    if (!(peak >= tau_n)) continue;
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float inv = inv_w[c0 + i];
                        const float sc = fabsf(__uint_as_float(v[i])) * inv;
                        if (sc >= tau_n && inv > 0.0f) {
                            const unsigned int slot = atomicAdd(&a.rep_count[n_res], 1u);
                            if (slot < (unsigned int)a.rep_cap) {
                                const float out = a.inv_scale ? sc * a.inv_scale[n_res] : sc;
                                const uint32_t col = listed ? col_w[c0 + i] : (uint32_t)((unsigned long long)sweep * kSuperCols + c0 + i);
                                a.rep[(size_t)n_res * a.rep_cap + slot] = make_uint2(col, __float_as_uint(out));
                            }
                        }
                    }
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_acce + 8u * buf);     // the accumulator is free; the queued appends follow
                if (WIDE && queued) {
                    unsigned int qn = queue[0];
                    if (qn > (unsigned int)kSuperCols - 1u) qn = (unsigned int)kSuperCols - 1u;
                    const int m = quad * 32 >= a.big_half ? 1 : 0;
                    for (unsigned int e = 1u + lane; e <= qn; e += 32u) {
                        const unsigned long long col = queue[e];
                        const unsigned int bit = 1u << ((unsigned int)col & 31u);
                        if (!(atomicOr(&a.big_bits[(size_t)m * ((a.d + 31) >> 5) + (col >> 5)], bit) & bit)) {
                            const unsigned int slot = atomicAdd(&a.big_count[m], 1u);
                            if (slot < (unsigned int)a.big_cap) a.big_list[(size_t)m * a.big_cap + slot] = (uint32_t)col;
                        }
                    }
                    __syncwarp();
                }
                continue;
            }
            const float* nr = norms + (size_t)(sweep_i % kNormRing) * kSuperCols * 2;
#pragma unroll 1
            for (int t = 0; t < 2; ++t) {
                const int col_local = t * kTileCols + quad * 32 + lane;
                unsigned long long col = (unsigned long long)sweep * kSuperCols + col_local;
                if (listed) {
                    const unsigned int idx = (unsigned int)col;
                    col = idx < list_n0 ? a.big_list[idx] : (idx < list_n ? a.big_list[(size_t)a.big_cap + idx - list_n0] : a.d);
                }
                float inv = 0.0f;
                if (TABLE) {
                    if (col < a.d) inv = half_bits_to_float(a.inv_norm[col]);
                } else {
                    const float n2 = nr[col_local * 2] + nr[col_local * 2 + 1];
                    if (col < a.d && n2 > 0.0f) inv = 1.0f / sqrtf(n2);
                }
#pragma unroll 1
                for (int c0 = 0; c0 < a.n; c0 += 16) {
                    uint32_t v[16];
                    tmem_ld16(tmem_base + ((uint32_t)(quad * 32) << 16) + buf * acc_cols + t * a.n + c0, v);
                    if (WIDE && a.big_tau != nullptr && !listed && inv > 0.0f) {
                        // every 8th residual feeds the wide list of its stream
                        const bool w0 = fabsf(__uint_as_float(v[0])) * inv >= a.big_tau[c0 >> 3];
                        const bool w8 = fabsf(__uint_as_float(v[8])) * inv >= a.big_tau[(c0 >> 3) + 1];
                        if (w0 || w8) {
                            const unsigned int bit = 1u << ((unsigned int)col & 31u);
                            const int m = c0 >= a.big_half ? 1 : 0;
                            if (!(atomicOr(&a.big_bits[(size_t)m * ((a.d + 31) >> 5) + (col >> 5)], bit) & bit)) {
                                const unsigned int slot = atomicAdd(&a.big_count[m], 1u);
                                if (slot < (unsigned int)a.big_cap) a.big_list[(size_t)m * a.big_cap + slot] = (uint32_t)col;
                            }
                        }
                    }
                    // one compare settles the usual case that none of the 16 residuals reaches its threshold
                    // (|v| inv >= tau  <=>  |v| / tau >= 1 / inv, with a little slack for the rounding of 1 / tau)
                    float peak = 0.0f;
                    {
                        const float4* it4 = reinterpret_cast<const float4*>(itau_s + c0);
#pragma unroll
                        for (int i4 = 0; i4 < 4; ++i4) {
                            const float4 w = it4[i4];
                            peak = fmaxf(peak, fabsf(__uint_as_float(v[4 * i4])) * w.x);
                            peak = fmaxf(peak, fabsf(__uint_as_float(v[4 * i4 + 1])) * w.y);
                            peak = fmaxf(peak, fabsf(__uint_as_float(v[4 * i4 + 2])) * w.z);
                            peak = fmaxf(peak, fabsf(__uint_as_float(v[4 * i4 + 3])) * w.w);
                        }
                    }
                    if (!(peak * inv >= 0.999f)) continue;
#pragma unroll
                    for (int i = 0; i < 16; ++i) {
                        const float sc = fabsf(__uint_as_float(v[i])) * inv;
                        if (sc >= tau_s[c0 + i] && inv > 0.0f) {
                            const unsigned int slot = atomicAdd(&a.rep_count[c0 + i], 1u);
                            if (slot < (unsigned int)a.rep_cap) {
                                const float out = a.inv_scale ? sc * a.inv_scale[c0 + i] : sc;
                                a.rep[(size_t)(c0 + i) * a.rep_cap + slot] = make_uint2((uint32_t)col, __float_as_uint(out));
                            }
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_acce + 8u * buf);
        }
    } else {
        // ---------------- generators: Z tiles as binary16, swizzled K-major ---------------------------------
        const int g = threadIdx.x - kFirstGenWarp * 32;
        const int col_local = g & (kSuperCols - 1), half = g >> 8;
        const int tile = col_local >> 7, m = col_local & (kTileCols - 1);
        const uint32_t row_off = (uint32_t)tile * kTileBytes + (uint32_t)m * 128u;
        const uint32_t sw = (uint32_t)(m & 7);
        uint32_t off[4];                                     // swizzled positions of this thread's four 16-byte chunks
#pragma unroll
        for (int c = 0; c < 4; ++c) off[c] = row_off + ((((uint32_t)(half * 4 + c)) ^ sw) << 4);
        uint32_t st = 0, ph = 0, sweep_i = 0;
        bool ok = true;
        for (unsigned int sweep = blockIdx.x; ok && sweep < num_super; sweep += gridDim.x, ++sweep_i) {
            uint32_t gcol = (uint32_t)((unsigned long long)sweep * kSuperCols + col_local);
            if (listed) gcol = gcol < list_n0 ? a.big_list[gcol] : (gcol < list_n ? a.big_list[(size_t)a.big_cap + gcol - list_n0] : 0u);
            const ColKey key = column_key(a.seed_lo, a.seed_hi, gcol);
            float norm = 0.0f;
            uint32_t h = key.ck + (uint32_t)(half * 16) * key.mk;   // one word per row pair
            const uint32_t skip = 16u * key.mk;                  // the other generator thread of this column owns the next 32 rows
            for (int kc = 0; kc < kc_count; kc += SUB) {
                if (!__all_sync(0xffffffffu, mbar_wait(bar_empty + 8u * st, ph ^ 1u, abort_flag, 0, a.wait_limit_ns))) { ok = false; break; }
#pragma unroll
                for (int u = 0; u < SUB; ++u) {
                const uint32_t dst = base + st * stage_bytes + u * sub_bytes;
#pragma unroll
                for (int c = 0; c < 4; c += 2) {
                    uint32_t w[8];
                    uint32_t n2 = 0u;                            // ||.||^2 of 16 entries as two binary16 partial sums
#pragma unroll
                    for (int e = 0; e < 8; ++e) {
                        w[e] = z_pair_from_word(h);
                        h += key.mk;
                        if (!TABLE) n2 = hfma2(w[e], w[e], n2);
                    }
                    st_shared_v4(dst + off[c], w[0], w[1], w[2], w[3]);
                    st_shared_v4(dst + off[c + 1], w[4], w[5], w[6], w[7]);
                    if (!TABLE) {
                        const float2 part = half2_bits_to_float2(n2);
                        norm += part.x + part.y;
                    }
                }
                h += skip;
                }
                if (!TABLE && kc + SUB >= kc_count) norms[((size_t)(sweep_i % kNormRing) * kSuperCols + col_local) * 2 + half] = norm;
                fence_async_smem();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_full + 8u * st);
                if (++st == (uint32_t)a.stages) { st = 0; ph ^= 1u; }
            }
        }
    }
    // ---------------- tail: everyone meets, tensor memory is returned ---------------------------------------
    tc_fence_before();
    __syncthreads();
    if (*abort_flag) {
        // A wait ran out.  Every role has left its loop, so nothing new is issued from here on; what may still be in
        // flight are the copies of at most `stages` chunks of R^T and the MMAs of as many stages.  The MMAs are waited
        // for explicitly (a commit on a barrier of its own arrives once every MMA this thread issued has completed);
        // the copies (a few KB each, microseconds) get 200 us to land before shared and tensor memory are released.
        if (threadIdx.x == 0)
            for (int q = 0; q < kPassMaxBatch; ++q) if (a.error[q]) atomicExch(a.error[q], 1);
        if (warp == 1 && lane == 0) {
            umma_commit(bar_drain);
            const unsigned long long t0 = global_ns();
            while (!mbar_try(bar_drain, 0u) && global_ns() - t0 < 2000000ull) __nanosleep(1000);
        }
        const unsigned long long t0 = global_ns();
        while (global_ns() - t0 < 200000ull) __nanosleep(1000);
        __syncthreads();
    }
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(512u) : "memory");
    }
}

// 1 / ||Z_i|| for every column, once per state: thread = column, fp32 sum of the exact squares
__global__ void __launch_bounds__(256) k_inv_norms(uint32_t seed_lo, uint32_t seed_hi, unsigned long long d, int k, uint16_t* out) {
    const unsigned long long col = (unsigned long long)blockIdx.x * 256 + threadIdx.x;
    if (col >= d) return;
    const ColKey key = column_key(seed_lo, seed_hi, (uint32_t)col);
    float n2 = 0.0f;
    uint32_t h = key.ck;
#pragma unroll 4
    for (int row = 0; row < k; row += 2) {
        const float2 z = half2_bits_to_float2(z_pair_from_word(h));
        h += key.mk;
        n2 = __fmaf_rn(z.x, z.x, n2);
        if (row + 1 < k) n2 = __fmaf_rn(z.y, z.y, n2);
    }
    const float inv = n2 > 0.0f ? 1.0f / sqrtf(n2) : 0.0f;
    unsigned short bits;
    asm("cvt.rn.f16.f32 %0, %1;" : "=h"(bits) : "f"(inv));
    out[col] = bits;
}

// ---- host side --------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

std::mutex g_encode_mutex;
EncodeTiledFn g_encode = nullptr;

cudaError_t get_encoder(EncodeTiledFn* out) {
    std::lock_guard<std::mutex> lock(g_encode_mutex);
    if (!g_encode) {
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        cudaError_t e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess) return e;
        if (qres != cudaDriverEntryPointSuccess || !fn) return cudaErrorNotSupported;
        g_encode = reinterpret_cast<EncodeTiledFn>(fn);
    }
    *out = g_encode;
    return cudaSuccess;
}

size_t pass_smem_bytes(int n, int slots, int sub) {
    return 1024 + (size_t)slots * sub * (2 * kTileBytes + (size_t)n * 128) + sizeof(float) * (kNormRing * kSuperCols * 2 + 512) +
           8 * (2 * (size_t)slots + 5) + 16;
}

}  // namespace

// 64-row chunks per slot and slots of the ring: four chunks fit beside a residual block of up to 128 rows, three beyond
int pass_sub(int n, int k) { return (n <= 128 && k % (2 * kChunkRows) == 0) ? 2 : 1; }
int pass_slots(int n, int k) { return (n <= 128 ? 4 : 3) / pass_sub(n, k); }

cudaError_t pass_encode_map(void* tmap_out, const void* rt, int n, int k) {
    EncodeTiledFn enc = nullptr;
    cudaError_t e = get_encoder(&enc);
    if (e != cudaSuccess) return e;
    const cuuint64_t gdim[2] = {(cuuint64_t)k, (cuuint64_t)n};
    const cuuint64_t gstride[1] = {(cuuint64_t)k * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kChunkRows, (cuuint32_t)n};
    const cuuint32_t estr[2] = {1, 1};
    const CUresult r = enc(static_cast<CUtensorMap*>(tmap_out), CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(rt), gdim,
                           gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                           CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? cudaSuccess : cudaErrorInvalidValue;
}

template <bool TABLE, bool WIDE, int SUB, bool SWAP = false>
cudaError_t pass_opt_in(int need) {
    return cudaFuncSetAttribute(k_pass<TABLE, WIDE, SUB, SWAP>, cudaFuncAttributeMaxDynamicSharedMemorySize, need);
}

cudaError_t pass_configure(int) {
    static_assert(sizeof(CUtensorMap) == kTensorMapBytes, "tensor map storage");
    size_t need = 0;                              // one setting that serves every width the kernel is launched with
    for (int n = 32; n <= kPassMaxN; n += 32)
        for (int sub = 1; sub <= 2; ++sub) {
            const size_t b = pass_smem_bytes(n, (n <= 128 ? 4 : 3) / sub, sub);
            if ((n <= 128 || sub == 1) && b > need) need = b;
        }
    cudaError_t e = pass_opt_in<false, false, 1>((int)need);
    if (e == cudaSuccess) e = pass_opt_in<false, false, 2>((int)need);
    if (e == cudaSuccess) e = pass_opt_in<true, true, 1>((int)need);
    if (e == cudaSuccess) e = pass_opt_in<true, true, 2>((int)need);
    if (e == cudaSuccess) e = pass_opt_in<true, false, 1>((int)need);
    if (e == cudaSuccess) e = pass_opt_in<true, false, 2>((int)need);
    if (e == cudaSuccess) e = pass_opt_in<true, false, 2, true>((int)need);
    if (e == cudaSuccess) e = pass_opt_in<true, true, 2, true>((int)need);
    return e;
}

cudaError_t launch_inv_norms(uint64_t seed, uint64_t d, int k, uint16_t* out, cudaStream_t stream) {
    k_inv_norms<<<(unsigned int)((d + 255) / 256), 256, 0, stream>>>((uint32_t)(seed & 0xFFFFFFFFu), (uint32_t)(seed >> 32), d, k, out);
    return cudaGetLastError();
}

cudaError_t launch_pass(const void* tmap, uint64_t seed, uint64_t d, int k, int n, const float* tau, const float* inv_scale,
                        const uint16_t* inv_norm, unsigned int* rep_count, uint2* rep, int rep_cap, const int* const* gates,
                        int* const* errors, int sm_count, cudaStream_t stream, const PassWide* wide, const int* sel,
                        int sel_value, unsigned long long wait_limit_ns) {
    PassArgs a;
    a.wait_limit_ns = wait_limit_ns ? wait_limit_ns : kWaitLimitNs;
    a.sel = sel; a.sel_value = sel_value;
    a.seed_lo = (uint32_t)(seed & 0xFFFFFFFFu); a.seed_hi = (uint32_t)(seed >> 32);
    a.d = d; a.k = k; a.n = n;
    const int sub = pass_sub(n, k);
    a.stages = pass_slots(n, k); a.bufs = n <= 128 ? 2 : 1;
    a.num_super = (unsigned int)((d + kSuperCols - 1) / kSuperCols);
    a.tau = tau; a.inv_scale = inv_scale; a.inv_norm = inv_norm; a.rep_count = rep_count; a.rep = rep; a.rep_cap = rep_cap;
    for (int q = 0; q < kPassMaxBatch; ++q) { a.gate[q] = gates ? gates[q] : nullptr; a.error[q] = errors ? errors[q] : nullptr; }
    a.big_tau = nullptr; a.big_list = nullptr; a.big_count = nullptr; a.big_bits = nullptr; a.big_cap = 0; a.big_half = 0;
    a.list_ctl = nullptr;
    if (wide) {
        a.big_tau = wide->tau; a.big_list = wide->list; a.big_count = wide->count; a.big_bits = wide->bits;
        a.big_cap = wide->cap; a.big_half = wide->half_n;
        a.list_ctl = wide->list_pass ? wide->ctl : nullptr;
    }
    unsigned int grid = (unsigned int)sm_count;
    if (grid > a.num_super) grid = a.num_super;
    CUtensorMap map;
    memcpy(&map, tmap, sizeof(map));
    const size_t smem = pass_smem_bytes(n, a.stages, sub);
    if (sub == 2) {
        if (inv_norm && wide && n == kTileCols && kPassSwap) k_pass<true, true, 2, true><<<grid, kPassThreads, smem, stream>>>(map, a);
        else if (inv_norm && wide) k_pass<true, true, 2, false><<<grid, kPassThreads, smem, stream>>>(map, a);
        else if (inv_norm && n == kTileCols && kPassSwap) k_pass<true, false, 2, true><<<grid, kPassThreads, smem, stream>>>(map, a);
        else if (inv_norm) k_pass<true, false, 2, false><<<grid, kPassThreads, smem, stream>>>(map, a);
        else k_pass<false, false, 2, false><<<grid, kPassThreads, smem, stream>>>(map, a);
    } else {
        if (inv_norm && wide) k_pass<true, true, 1, false><<<grid, kPassThreads, smem, stream>>>(map, a);
        else if (inv_norm) k_pass<true, false, 1, false><<<grid, kPassThreads, smem, stream>>>(map, a);
        else k_pass<false, false, 1, false><<<grid, kPassThreads, smem, stream>>>(map, a);
    }
    return cudaGetLastError();
}

}  // namespace sgc
