// Internal declarations of the SGC CUDA library (sm_100a).  Not part of the public C ABI.
#pragma once

#include <cuda_fp16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <string.h>

#include <vector>

#include "sgc.h"

namespace sgc {

// ------------------------------------------------------------------------------------------------
// Measurement matrix: A[j][i] = sigma_k * Z(seed, j, i), never stored (Section 3.3 fixes only the law:
// i.i.d. zero-mean normal entries of standard deviation 1/sqrt(k)).  Every Z is exactly a binary16 number.
//
// Z(seed, row, col); one 32-bit word yields the two rows 2p and 2p+1 of a column:
//   ck = mix32(mix32(col + 0x9E3779B9*seed_lo) ^ seed_hi),  mk = mix32(ck ^ 0x5BD1E995) | 1
//   h  = ck + p*mk;  h ^= h >> 16;  h *= 0x85EBCA6B;  h ^= h >> 15
//   S  = b0 + b1 (even row) or b2 + b3 (odd row), bytes of h;   x = (S - 255)/256
//   w  = x*x;  q = fma(fma(w, C2, C1), w, C0);  Z = x*q        (binary16, round to nearest even)
// A byte pair sum is triangular on 511 lattice points; the odd polynomial maps its quantiles onto the normal's.
// Both rows are evaluated at once with packed half-precision instructions (f16x2).
// ------------------------------------------------------------------------------------------------
constexpr uint32_t kGolden = 0x9E3779B9u;
constexpr uint32_t kMulEntry = 0x85EBCA6Bu;
constexpr uint32_t kStrideSalt = 0x5BD1E995u;
constexpr uint32_t kC0x2 = 0x40c240c2u, kC1x2 = 0xbad9bad9u, kC2x2 = 0x3f893f89u;   // C0, C1, C2 in both halves

__host__ __device__ __forceinline__ uint32_t mix32(uint32_t x) {
    x ^= x >> 16; x *= 0x7feb352du;
    x ^= x >> 15; x *= 0x846ca68bu;
    x ^= x >> 16;
    return x;
}

struct ColKey { uint32_t ck, mk; };

__host__ __device__ __forceinline__ ColKey column_key(uint32_t seed_lo, uint32_t seed_hi, uint32_t col) {
    ColKey c;
    c.ck = mix32(mix32(col + kGolden * seed_lo) ^ seed_hi);
    c.mk = mix32(c.ck ^ kStrideSalt) | 1u;
    return c;
}

__device__ __forceinline__ uint32_t hfma2(uint32_t a, uint32_t b, uint32_t c) {
    uint32_t d;
    asm("fma.rn.f16x2 %0, %1, %2, %3;" : "=r"(d) : "r"(a), "r"(b), "r"(c));
    return d;
}
__device__ __forceinline__ uint32_t hmul2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("mul.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

__device__ __forceinline__ uint32_t hsub2(uint32_t a, uint32_t b) {
    uint32_t d;
    asm("sub.rn.f16x2 %0, %1, %2;" : "=r"(d) : "r"(a), "r"(b));
    return d;
}

// h0 = ck + p*mk (the caller advances it by mk per row pair).  Returns Z of rows 2p (low half) and 2p+1 (high
// half) as two binary16 bit patterns.
__device__ __forceinline__ uint32_t z_pair_from_word(uint32_t h0) {
    uint32_t h = h0;
    h ^= h >> 16; h *= kMulEntry;
    // x = (b0 + b1 - 255)/256 (even row; b2, b3 for the odd row) as a difference of two halves that are planted by byte
    // permutes alone: the half 0x4400 | b is 4 + b/256, so (4 + b0/256) - (4 + (255 - b1)/256) = x, exactly.  The
    // complement of bytes 1 and 3 rides along in the three-input logic operation of the last mixing step.
    h = h ^ (h >> 15) ^ 0xFF00FF00u;
    const uint32_t x = hsub2(__byte_perm(h, 0x44444444u, 0x4240), __byte_perm(h, 0x44444444u, 0x4341));
    const uint32_t w = hmul2(x, x);
    uint32_t q = hfma2(w, kC2x2, kC1x2);
    q = hfma2(q, w, kC0x2);
    return hmul2(x, q);
}

__device__ __forceinline__ float half_bits_to_float(uint32_t b) {
    float f;
    asm("{\n\t.reg .b16 t;\n\tcvt.u16.u32 t, %1;\n\tcvt.f32.f16 %0, t;\n\t}" : "=f"(f) : "r"(b));
    return f;
}
__device__ __forceinline__ float2 half2_bits_to_float2(uint32_t b) {
    float2 f;
    asm("{\n\t.reg .b16 lo, hi;\n\tmov.b32 {lo, hi}, %2;\n\tcvt.f32.f16 %0, lo;\n\tcvt.f32.f16 %1, hi;\n\t}"
        : "=f"(f.x), "=f"(f.y) : "r"(b));
    return f;
}
// Z(row) of the column with key (ck, mk), as binary16 bits / as a float
__device__ __forceinline__ uint32_t z_bits_at(const ColKey& key, uint32_t row) {
    const uint32_t z2 = z_pair_from_word(key.ck + (row >> 1) * key.mk);
    return (row & 1u) ? (z2 >> 16) : (z2 & 0xFFFFu);
}
__device__ __forceinline__ float z_at(const ColKey& key, uint32_t row) { return half_bits_to_float(z_bits_at(key, row)); }

// ------------------------------------------------------------------------------------------------
// limits
// ------------------------------------------------------------------------------------------------
constexpr int kMaxK = 16384;           // rows of A of a state: the lock-step kernel keeps both residuals (8 bytes per row) in shared memory
constexpr int kPassMaxK = 65536;       // rows of A of the stand-alone screening pass (sgc_screen)
constexpr int kMaxS = 1024;
constexpr int kSelCap = 32768;          // candidate slots of the top-s filter
constexpr int kSelBins = 4096;          // 12-bit magnitude histogram of the sample
constexpr int kCorrThreads = 512;       // threads per block of the correlation pass
constexpr int kCorrCols = 2;            // columns per thread and tile
constexpr int kCorrTop = 3;             // slots per block and residual: its best two columns, and the score of its third best
constexpr int kRescoreCap = 16;         // candidates rescored in fp64 per iteration and residual
constexpr int kBookThreads = 1024;
constexpr int kOmpThreads = 1024;       // threads per block of the cooperative OMP kernel
constexpr int kCandCap = 32768;         // candidate columns kept for the restricted (speculative) OMP
constexpr int kCandKeep = 24576;        // the list is rebuilt from the supports once it grows beyond this
constexpr int kSmallList = 768;         // lists up to this length are correlated inside the bookkeeping block
constexpr int kHistSteps = 64;          // steps whose kept indices (Sparsify_s) stay candidates ...
constexpr int kHistColumns = 8192;      // ... as long as they are at most this many columns
constexpr int kLookAhead = 12;          // after a refuted pick, every kLookAhead-th later residual is harvested too
constexpr double kLookAheadShare = 0.78; // ... as far as its columns reach this share of the residual's pick score
constexpr int kWideCap = 2097152;       // columns per wide list (two-level screening)
constexpr int kResolveBlocks = 16;        // blocks of the resolve kernel: all sweep the report lists, the last to finish walks the picks
constexpr int kPassFastRows = 128;      // a pass over up to this many residual rows costs half of a wider one (A is generated once either way)
constexpr int kMiniRounds = 8;          // list passes between two full passes, at most
constexpr int kMiniDepth = 32;          // picks speculated ahead of one list pass
constexpr int kGramList = 256;          // lists up to this length run OMP on their Gram matrix (Algorithm 3 as printed)
constexpr int kRepCap = 8192;           // report slots per residual of one screening pass
constexpr int kPassMaxN = 256;          // residuals per screening pass (UMMA N)
constexpr int kPassMaxBatch = 8;        // states whose residuals one screening pass can serve (kPassMaxN / 32)
constexpr int kMaxRounds = 24;          // speculate / screen / resolve rounds enqueued per step
constexpr int kTensorMapBytes = 128;    // sizeof(CUtensorMap)
// |score computed by the screening pass - exact score| <= (kScreenMargin + k * kScreenAccMargin) * ||r|| + kScreenNormMargin * score:
//   * the residual is rounded to binary16: relative error 2^-11 per element, hence at most 2^-11 ||r|| (4.9e-4) in the
//     normalised score by Cauchy-Schwarz (Z itself is exact in binary16);
//   * the k products are summed in fp32 inside the tensor cores: at most k * 2^-23 * sum |z_i r_i| <= k * 2^-23 ||Z_i|| ||r||
//     whatever the order of the additions and whether intermediate sums are rounded or truncated;
//   * 1 / ||Z_i|| comes from a binary16 table (relative error 2^-11), or is accumulated in short binary16 partial sums by the
//     stand-alone pass (about 1e-4): kScreenNormMargin covers both.
constexpr double kScreenMargin = 4.9e-4;
constexpr double kScreenAccMargin = 1.1920928955078125e-7;      // 2^-23 per row of A
constexpr double kScreenNormMargin = 1.0e-3;

// binary16 residual rows of the screening pass
__device__ __forceinline__ uint16_t half_rn_bits(double v) { return __half_as_ushort(__double2half(v)); }   // nearest even

// bound on |score seen by the screening pass - exact score| for a residual of norm rn over k rows and a score near ps
__device__ __forceinline__ double screen_margin(double rn, double ps, int k) {
    return (kScreenMargin + (double)k * kScreenAccMargin) * rn + kScreenNormMargin * ps;
}

// power-of-two scale that brings a residual of norm rn into [2^12, 2^13): no binary16 overflow, and entries
// down to 2^-26 of the norm stay normal numbers
__device__ __forceinline__ double residual_scale(double rn) {
    if (!(rn > 0.0) || !isfinite(rn)) return 1.0;
    int e;
    frexp(rn, &e);
    return ldexp(1.0, 13 - e);
}

constexpr uint32_t kNoColumn = 0xFFFFFFFFu;

struct Cand { float score; uint32_t idx; };

// device-resident control block of the speculative recovery (one per state)
struct SpecCtl {
    int round_active;       // 1 while another speculate / screen / resolve round is needed
    int fallback;           // 1: the remaining picks are made in lock-step over all columns
    int v[2];               // verified picks per residual (M^, V^)
    uint32_t forced[2];     // column that must become pick v[m] (the verified global winner), or kNoColumn
    int base[2];            // first speculative pick of the current round
    int hi[2];              // one past the last speculative pick of the current round
    int extra[2];           // 1: the residual after pick hi-1 is screened without a pick (harvest + forced winner)
    int dep[2];             // 1: pick hi-1 turned out linearly dependent on the support
    int finished[2];        // recovery of this residual complete
    int n_cand;             // length of the candidate list
    int rounds;             // screening passes that did work in the last step
    int pass_error;         // a wait inside the screening pass expired (reported as SGC_STATUS_TIMEOUT)
    int stop[2];            // scratch of the cooperative kernel: speculation of residual m has ended
    int list_exact[2];      // 1: the last speculation of residual m compared every list member exactly
    int list_version;       // bumped whenever the candidate list changes
    int gram_version;       // list version the stored Gram matrix belongs to
    int gram_pending;       // list version seen by the round in flight
    int gram_todo;          // 1: the Gram matrix must be recomputed in this round
    int gram_ok;            // 0: the Gram path gave up in this step (a pick is missing from the list)
    int tv[2];              // tentative picks: confirmed against the wide lists only (tv >= v)
    uint32_t tforced[2];    // column imposed as pick tv[m] by a list pass, or kNoColumn
    int narrow;             // 1: only the first stream still has residuals to screen: the half-width pass serves the round
    int mini_done;          // 1: list passes rest until the next full pass
    int list_rounds;        // list passes of the last step that were resolved
    int list_refuted;       // picks that those list passes refuted
    int refuted;            // picks that the full passes of this step refuted
    unsigned int resolve_ticket;   // blocks of the resolve kernel that have finished their share of the sweep
    int contested[kPassMaxN];      // per screened residual: some report comes within the margin of its pick (sweep result)
    int pass_rows;          // residual rows that the full passes of the last step screened, summed over the passes
    int hist_count, hist_next;  // ring of the kept index sets of the last steps: valid slots, slot of the next step
    int trace[kMaxRounds][3];   // per round: confirmed picks of both streams and the list length after it
    double ynorm[2];        // ||y|| per residual
};

// device-resident counters of one state
struct Counters {
    unsigned int status;        // sticky SGC_STATUS_* bits
    unsigned int sel_count;     // candidates appended by the filter pass
    unsigned int sel_ticket;    // blocks of the sample pass that have finished
    unsigned int sel_tau;       // threshold on the sign-cleared bit pattern
    int done[2];                // completed OMP iterations per residual (M^, V^)
    int stopped[2];             // 1 once a residual's OMP has stopped early
    int n_upd, mismatch, negv, pad;
    unsigned int sel_tau_next;  // threshold carried to the next step's one-kernel selection (0: none yet)
    unsigned int sel_ticket2;   // blocks of the one-kernel selection that have finished
};

// Batched chunk path (sgc_chunked.cu): the records of one chunk's state, as the batched kernels address them
struct ChunkRef {
    float* M; float* V; double* p; double* q; double* y64; double* r64;
    uint32_t* sel_idx; float* sel_val;
    uint16_t* zsel; uint32_t* lam; double* F; double* acoef; double* x; double* rnorm;
    uint32_t* upd_idx; double* upd_val; Counters* cnt; SpecCtl* ctl;
};
// workspace of the batched chunk path, owned by the first state of the chunk list it was built for
struct ChunkWs {
    void* base;                 // one device allocation holding everything below
    ChunkRef* table;            // [c]
    float* r32;                 // [2c][kp] residuals of all streams (stream = 2 * chunk + moment), rows padded to kp
    Cand* cand;                 // [2c][splits][2] best two columns of every column split, per stream
    int c, kp, splits;
    unsigned long long key;     // names the chunk list (its state pointers) the table was built from
    // tensor-core route of the correlation (k_c > 32): the residuals of all recoveries go through the screening pass
    bool tensor;
    int kp64, n_rows, passes;   // rows of A per column padded to a multiple of 64; residual rows (multiple of 32); passes of <= 256 rows
    uint16_t* rt;               // [n_rows][kp64] binary16 residuals, each scaled by a power of two
    float* tau; float* inv_scale; unsigned int* rep_count;   // [n_rows]
    uint2* rep;                 // [n_rows][kChunkRepCap] (column, score)
    uint16_t* inv_norm;         // [d/c] 1 / ||Z_i|| over the k_c rows, binary16
    double* rnv;                // [2c] ||r|| of every recovery at the start of the iteration
    unsigned char* unresolved;  // [2c] 1: the reports did not settle this recovery's pick; the fp32 route decides it
    int* flags;                 // [0] epoch of the last iteration that left a recovery unresolved, [1] a wait inside a pass of
                                // this step expired, [2] constant 1 (gate)
    double z_rep;               // report threshold in units of ||r|| / sqrt(k_c)
    unsigned char tmap[8][128]; // tensor maps of the row blocks of rt, one per pass
};
constexpr int kChunkRepCap = 2048;      // report slots per residual row of the chunk path

}  // namespace sgc

// the state behind the opaque handle
struct sgc_state {
    int64_t d; int32_t k, s; uint64_t seed; float lr, beta1, beta2, eps, alpha; int64_t t;
    int device; int sm_count;
    cudaStream_t last_stream; bool has_stream;
    int32_t last_launches; bool stepped;
    bool sel_warm;              // a top-s threshold from the previous step is on the device (one-kernel selection)
    int corr_grid, corr_smem;
    int mode;                   // 0 auto, 1 lock-step only, 2 speculative whenever k allows it
    int shared_support;         // 1: OMP(M^) alone selects, V^ is fitted on its support (sgc_set_recovery)
    double residual_tol;        // > 0: recoveries are cut at the first pick that leaves ||r|| <= residual_tol ||y||
    bool spec_ok;               // speculative recovery usable for this (d, k)
    bool spec_ready;            // its buffers exist (second allocation: at creation for d >= 65536, else at sgc_set_mode)
    void* spec_base; size_t spec_bytes;
    int pass_n;                 // residuals per screening pass (multiple of 32, <= 256); pass_n / 2 per residual stream
    double z_harvest, z_floor;  // thresholds of the screening pass in units of ||r|| / sqrt(k)
    double z_wide;              // threshold of the wide lists, same units
    unsigned char tmap[8][128]; // CUtensorMaps of the residual matrix R^T, one per number of states batched into a pass
    unsigned char tmap_half[128]; // the same for a pass over the first stream's residuals alone (shared-support variant)
    int pass_n_half;            // its width: pass_n / 2 rounded up to a multiple of 32
    // optional per-kernel timing (sgc_set_profile)
    bool profile;
    std::vector<cudaEvent_t>* ev_pool; size_t ev_used;
    std::vector<int>* ev_phase;          // phase of each (start, stop) event pair
    float prof_ms[8]; int32_t prof_launches[8];
    // device memory (one allocation, carved)
    void* base; size_t bytes;
    float *M, *V; double *p, *q;
    uint32_t* sel_idx; float* sel_val;
    double *y64, *r64;          // [2][k]
    float2* r32;                // [k] (M^ residual, V^ residual)
    unsigned long long* sel_cand; unsigned int* sel_hist;
    sgc::Cand* corr_cand;       // [2][corr_grid][kCorrTop]
    uint16_t* zsel;             // [2][s][k] selected columns of Z as binary16 bits
    uint32_t* lam;              // [2][s]
    double *F, *acoef, *x, *gvec, *cvec, *rnorm;   // [2][s*s], [2][s] ...
    uint32_t* upd_idx; double* upd_val;
    sgc::Counters* cnt;
    // speculative recovery
    sgc::SpecCtl* ctl;
    uint16_t* rt;               // R^T [pass_n][k] binary16 bits: the residuals screened by one pass, each row scaled
    float* tau;                 // [pass_n] thresholds (in the scaled units of the row)
    float* inv_scale;           // [pass_n] 1 / (power-of-two scale of the row)
    unsigned int* rep_count;    // [pass_n]
    uint2* rep;                 // [pass_n][kRepCap] (column, score bits)
    double* pick_score;         // [2][s] exact score |<Z_i, r>| / ||Z_i|| of every speculative pick
    uint32_t* cand_list;        // [kCandCap]
    unsigned int* cand_bits;    // bitmap over [0, d): membership in cand_list
    double* rtmp;               // [k] scratch residual of the resolve kernel
    double* rhist;              // [pass_n][k] the screened residuals of this state in fp64 (row = stream * rows per stream + position)
    uint16_t* inv_norm;         // [d] 1 / ||Z_i|| as binary16, filled once at creation (the screening pass reads it)
    uint16_t* zlist;            // [kGramList][k] the candidate columns as binary16 (Gram path)
    double* gram;               // [kGramList][kGramList] Z_C^T Z_C
    double* p0;                 // [2][kGramList] Z_C^T y per residual
    int* pick_li;               // [2][s] list position of every pick (Gram path)
    uint32_t* kept_ring;         // [hist_slots][s] kept indices of the last steps (all of them are columns M^ and V^ are made of)
    int hist_slots;
    sgc::ChunkWs* chunk_ws;     // batched chunk path: workspace built for the chunk list that starts with this state
    bool two_level;             // host: wide lists and list passes are in use (steps that need several full passes)
    float* wide_tau;            // [kPassMaxN / 8] thresholds of the wide lists, one per 8th screened residual
    uint32_t* wide_list;        // [2][kWideCap]
    unsigned int* wide_count;   // [2]
    unsigned int* wide_bits;    // [2] bitmaps over [0, d): the column is in the stream's wide list
    unsigned long long wait_limit_ns;   // bound of the waits inside this state's screening passes; 0 = the default
    int max_rounds;             // host: most speculation rounds a step may enqueue; 0 = chosen from the last step's count
    int* h_rounds;              // pinned, device-mapped: rounds the last finished step needed (read without synchronising)
    int* d_rounds;              // device alias of h_rounds
};

namespace sgc {
enum Phase { kPhaseSample = 0, kPhaseFilter = 1, kPhasePick = 2, kPhaseProject = 3, kPhaseCorr = 4, kPhaseBook = 5,
             kPhaseScatter = 6, kPhasePass = 7, kNumPhases = 8 };

// Brackets the launches issued during its lifetime with a pair of events when profiling is on (no state: never).
struct PhaseTimer {
    sgc_state* st; cudaStream_t stream; bool on;
    PhaseTimer(sgc_state* s, cudaStream_t cs, int phase, int n_launches) : st(s), stream(cs), on(s != nullptr && s->profile) {
        if (!on) return;
        while (st->ev_pool->size() < st->ev_used + 2) {
            cudaEvent_t e;
            if (cudaEventCreate(&e) != cudaSuccess) { on = false; return; }
            st->ev_pool->push_back(e);
        }
        st->ev_phase->push_back(phase);
        st->prof_launches[phase] += n_launches;
        cudaEventRecord((*st->ev_pool)[st->ev_used], stream);
    }
    ~PhaseTimer() {
        if (!on) return;
        cudaEventRecord((*st->ev_pool)[st->ev_used + 1], stream);
        st->ev_used += 2;
    }
};

// launchers (each returns the cudaError_t of its launches); defined in the .cu files
cudaError_t launch_select(sgc_state* st, const float* grad, cudaStream_t stream, int* launches);
cudaError_t launch_project_adam(sgc_state* st, cudaStream_t stream, int* launches);
cudaError_t launch_recover(sgc_state* st, float* weight, cudaStream_t stream, int* launches);
cudaError_t launch_reproject(sgc_state* st, uint64_t new_seed, cudaStream_t stream);
cudaError_t launch_recover_group(sgc_state* const* sts, float* const* weights, int n, cudaStream_t stream, int* launches);
cudaError_t launch_z_block(uint64_t seed, int64_t row0, int64_t nrows, int64_t col0, int64_t ncols, float* out,
                           cudaStream_t stream);
// MESGC with small per-chunk problems (s <= 32, k <= 256): the whole step of all chunks in 2 + 2s launches
bool chunked_batch_eligible(sgc_state* const* sts, int c);
cudaError_t launch_chunked_batch(sgc_state* const* sts, int c, const float* grad, float* weight, cudaStream_t stream,
                                 int* launches);
void free_chunk_ws(sgc_state* st);
// CESGC projections (sgc_cesgc.cu): P = B G and W += B^T U
bool cesgc_shape_ok(int r, int m, int n);
cudaError_t launch_cesgc_project(const float* B, const float* G, float* P, int r, int m, int n, cudaStream_t stream);
cudaError_t launch_cesgc_back(const float* B, const float* U, float* W, int r, int m, int n, cudaStream_t stream);
double normal_tail_threshold(double d, double target);   // z with d * P(|N(0,1)| > z) = target
cudaError_t configure_recover(sgc_state* st);   // occupancy / shared-memory set-up at create time
cudaError_t finish_recover_setup(sgc_state* st); // after the workspace exists: tensor map of R^T

// wide lists of the two-level screening (sgc_pass.cu): a full pass fills them, a list pass screens only their columns
struct PassWide {
    const float* tau;            // [n / 8] thresholds of the wide lists (scaled units of rows 0, 8, 16, ...)
    uint32_t* list;              // [2][cap]
    unsigned int* count;         // [2]
    unsigned int* bits;          // [2] bitmaps over [0, d), one per stream: a column enters a list once
    int cap, half_n;
    const SpecCtl* ctl;
    bool list_pass;              // true: screen the lists' columns; false: full pass that feeds the lists
};

// screening pass (sgc_pass.cu)
cudaError_t pass_configure(int n);
cudaError_t pass_encode_map(void* tmap_out, const void* rt, int n, int k);
cudaError_t launch_pass(const void* tmap, uint64_t seed, uint64_t d, int k, int n, const float* tau, const float* inv_scale,
                        const uint16_t* inv_norm, unsigned int* rep_count, uint2* rep, int rep_cap, const int* const* gates,
                        int* const* errors, int sm_count, cudaStream_t stream, const PassWide* wide = nullptr,
                        const int* sel = nullptr, int sel_value = 0, unsigned long long wait_limit_ns = 0);   // 0: the default (2 s)
cudaError_t launch_inv_norms(uint64_t seed, uint64_t d, int k, uint16_t* out, cudaStream_t stream);
}  // namespace sgc
