// C ABI of the SGC library (include/sgc.h): argument checks, state life cycle, step orchestration.
#include <math.h>
#include <atomic>
#include <new>
#include <string.h>

#include "sgc_internal.cuh"

namespace {

inline size_t align_up(size_t v) { return (v + 255) & ~(size_t)255; }

std::atomic<unsigned long long> g_screen_wait_limit_ns{0};      // sgc_screen's bound on the waits of its pass; 0 = default

// a state may only be stepped on the device it was created on
bool on_own_device(const sgc_state* st) {
    int dev = -1;
    return cudaGetDevice(&dev) == cudaSuccess && dev == st->device;
}

template <class T>
T* carve(unsigned char* base, size_t& off, size_t count) {
    T* p = reinterpret_cast<T*>(base + off);
    off = align_up(off + count * sizeof(T));
    return p;
}

// lays out (base == nullptr: only measures) the workspace of a state
size_t layout(sgc_state* st, unsigned char* base) {
    size_t off = 0;
    const size_t k = (size_t)st->k, s = (size_t)st->s;
    st->M = carve<float>(base, off, k);
    st->V = carve<float>(base, off, k);
    st->p = carve<double>(base, off, k);
    st->q = carve<double>(base, off, k);
    st->sel_idx = carve<uint32_t>(base, off, s);
    st->sel_val = carve<float>(base, off, s);
    st->y64 = carve<double>(base, off, 2 * k);
    st->r64 = carve<double>(base, off, 2 * k);
    st->r32 = carve<float2>(base, off, k);
    st->sel_cand = carve<unsigned long long>(base, off, sgc::kSelCap);
    st->sel_hist = carve<unsigned int>(base, off, sgc::kSelBins);
    st->corr_cand = carve<sgc::Cand>(base, off, 2 * (size_t)(st->corr_grid > 32 ? st->corr_grid : 32) * sgc::kCorrTop);
    st->zsel = carve<uint16_t>(base, off, 2 * s * k);
    st->lam = carve<uint32_t>(base, off, 2 * s);
    st->F = carve<double>(base, off, 2 * s * s);
    st->acoef = carve<double>(base, off, 2 * s);
    st->x = carve<double>(base, off, 2 * s);
    st->rnorm = carve<double>(base, off, 2 * s);
    st->upd_idx = carve<uint32_t>(base, off, s);
    st->upd_val = carve<double>(base, off, s);
    st->cnt = carve<sgc::Counters>(base, off, 1);
    st->ctl = carve<sgc::SpecCtl>(base, off, 1);
    return off;
}

// lays out (base == nullptr: only measures) the buffers of the speculative recovery: a second allocation, made at
// creation for states that will use it on their own accord (d >= 65536) and at sgc_set_mode(SGC_MODE_SPECULATIVE)
// for the others, so that thousands of small chunk states do not carry 50 MB each that they never touch
size_t layout_spec(sgc_state* st, unsigned char* base) {
    size_t off = 0;
    const size_t k = (size_t)st->k, s = (size_t)st->s;
    {
        const size_t n = (size_t)sgc::kPassMaxN;          // room for a whole batch of same-A states (sgc_step_group)
        st->rt = carve<uint16_t>(base, off, n * k);
        st->tau = carve<float>(base, off, n);
        st->inv_scale = carve<float>(base, off, n);
        st->rep_count = carve<unsigned int>(base, off, n);
        st->rep = carve<uint2>(base, off, n * sgc::kRepCap);
        st->pick_score = carve<double>(base, off, 2 * s);
        st->cand_list = carve<uint32_t>(base, off, sgc::kCandCap);
        st->cand_bits = carve<unsigned int>(base, off, ((size_t)st->d + 31) / 32);
        st->rtmp = carve<double>(base, off, k);
        st->rhist = carve<double>(base, off, (size_t)st->pass_n * k);
        st->inv_norm = carve<uint16_t>(base, off, (size_t)st->d);
        st->zlist = carve<uint16_t>(base, off, (size_t)sgc::kGramList * k);
        st->gram = carve<double>(base, off, (size_t)sgc::kGramList * sgc::kGramList);
        st->p0 = carve<double>(base, off, 2 * (size_t)sgc::kGramList);
        st->pick_li = carve<int>(base, off, 2 * s);
        st->hist_slots = sgc::kHistColumns / (int)s < sgc::kHistSteps ? sgc::kHistColumns / (int)s : sgc::kHistSteps;
        if (st->hist_slots < 1) st->hist_slots = 1;
        st->kept_ring = carve<uint32_t>(base, off, (size_t)st->hist_slots * s);
        st->wide_tau = carve<float>(base, off, sgc::kPassMaxN / 8);
        st->wide_list = carve<uint32_t>(base, off, 2 * (size_t)sgc::kWideCap);
        st->wide_count = carve<unsigned int>(base, off, 2);
        st->wide_bits = carve<unsigned int>(base, off, 2 * (((size_t)st->d + 31) / 32));
    }
    return off;
}

bool finite_f(float v) { return isfinite(v); }

cudaError_t ensure_spec(sgc_state* st) {
    if (!st->spec_ok || st->spec_ready) return cudaSuccess;
    {
        sgc_state probe = *st;                                       // measuring must not leave pointers behind
        st->spec_bytes = layout_spec(&probe, nullptr);
    }
    cudaError_t e = cudaMalloc(&st->spec_base, st->spec_bytes);
    if (e != cudaSuccess) { st->spec_base = nullptr; return e; }
    layout_spec(st, static_cast<unsigned char*>(st->spec_base));
    e = cudaMemset(st->spec_base, 0, st->spec_bytes);             // empty candidate list, bitmaps, wide lists
    if (e == cudaSuccess) e = sgc::finish_recover_setup(st);      // tensor maps of R^T, column norms (synchronises)
    if (e != cudaSuccess) { cudaFree(st->spec_base); st->spec_base = nullptr; return e; }
    st->spec_ready = true;
    return cudaSuccess;
}

}  // namespace

extern "C" {

SGC_API int sgc_create(sgc_state** out, int64_t d, int32_t k, int32_t s, uint64_t seed, float lr, float beta1, float beta2,
               float eps) {
    if (!out) return SGC_ERR_NULL;
    *out = nullptr;
    if (d < 1 || k < 1 || s < 1 || s > k || (int64_t)s > d || d >= ((int64_t)1 << 32) || k > sgc::kMaxK ||
        s > sgc::kMaxS)
        return SGC_ERR_DIM;
    if (!(beta1 >= 0.0f && beta1 < 1.0f) || !(beta2 >= 0.0f && beta2 < 1.0f) || !(eps > 0.0f) || !finite_f(eps) ||
        !finite_f(lr))
        return SGC_ERR_HYPER;
    sgc_state* st = new (std::nothrow) sgc_state();
    if (!st) return (int)cudaErrorMemoryAllocation;
    memset(st, 0, sizeof(*st));
    st->ev_pool = new (std::nothrow) std::vector<cudaEvent_t>();
    st->ev_phase = new (std::nothrow) std::vector<int>();
    if (!st->ev_pool || !st->ev_phase) { delete st->ev_pool; delete st->ev_phase; delete st; return (int)cudaErrorMemoryAllocation; }
    st->d = d; st->k = k; st->s = s; st->seed = seed; st->lr = lr; st->beta1 = beta1; st->beta2 = beta2; st->eps = eps;
    st->alpha = 1.0f; st->t = 0;
    cudaError_t e = cudaGetDevice(&st->device);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&st->sm_count, cudaDevAttrMultiProcessorCount, st->device);
    if (e == cudaSuccess) e = sgc::configure_recover(st);
    if (e == cudaSuccess) {
        st->bytes = layout(st, nullptr);
        e = cudaMalloc(&st->base, st->bytes);
    }
    if (e == cudaSuccess) {
        layout(st, static_cast<unsigned char*>(st->base));
        e = cudaMemset(st->base, 0, st->bytes);        // M_0 = V_0 = 0, counters, histogram, empty candidate list
    }
    if (e == cudaSuccess && st->d >= ((int64_t)1 << 16)) e = ensure_spec(st);      // SGC_MODE_AUTO speculates from this size on
    if (e == cudaSuccess) {
        e = cudaHostAlloc(reinterpret_cast<void**>(&st->h_rounds), sizeof(int), cudaHostAllocMapped);
        if (e == cudaSuccess) { st->h_rounds[0] = 0; e = cudaHostGetDevicePointer(reinterpret_cast<void**>(&st->d_rounds), st->h_rounds, 0); }
    }
    if (e != cudaSuccess) {
        if (st->base) cudaFree(st->base);
        if (st->spec_base) cudaFree(st->spec_base);
        if (st->h_rounds) cudaFreeHost(st->h_rounds);
        delete st->ev_pool; delete st->ev_phase;
        delete st;
        return (int)e;
    }
    *out = st;
    return SGC_OK;
}

SGC_API int sgc_step(sgc_state* st, const float* grad, float* weight, void* stream) {
    if (!st || !grad || !weight) return SGC_ERR_NULL;
    if (((uintptr_t)grad & 15u) || ((uintptr_t)weight & 15u)) return SGC_ERR_ALIGN;
    if (!on_own_device(st)) return SGC_ERR_DEVICE;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    int launches = 0;
    // t counts the steps whose gradient has entered M and V: it moves once the kernel that updates them is enqueued
    st->t += 1;
    cudaError_t e = sgc::launch_select(st, grad, cs, &launches);
    if (e == cudaSuccess) e = sgc::launch_project_adam(st, cs, &launches);
    if (e != cudaSuccess) { st->t -= 1; return (int)e; }
    e = sgc::launch_recover(st, weight, cs, &launches);
    st->last_stream = cs; st->has_stream = true; st->stepped = true; st->last_launches = launches;
    return (int)e;
}

SGC_API int sgc_step_group(sgc_state* const* states, const float* const* grads, float* const* weights, int32_t n, void* stream) {
    if (!states || !grads || !weights) return SGC_ERR_NULL;
    if (n < 1) return SGC_ERR_DIM;
    for (int32_t i = 0; i < n; ++i) {
        if (!states[i] || !grads[i] || !weights[i]) return SGC_ERR_NULL;
        if (states[i]->d != states[0]->d || states[i]->k != states[0]->k || states[i]->s != states[0]->s ||
            states[i]->seed != states[0]->seed)
            return SGC_ERR_GROUP;
        if (((uintptr_t)grads[i] & 15u) || ((uintptr_t)weights[i] & 15u)) return SGC_ERR_ALIGN;
        for (int32_t j = 0; j < i; ++j) if (states[j] == states[i]) return SGC_ERR_GROUP;
        if (!on_own_device(states[i])) return SGC_ERR_DEVICE;
    }
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    std::vector<int> launches((size_t)n, 0);
    cudaError_t e = cudaSuccess;
    for (int32_t i = 0; i < n && e == cudaSuccess; ++i) {           // a1-a3 per state
        sgc_state* st = states[i];
        st->t += 1;
        e = sgc::launch_select(st, grads[i], cs, &launches[i]);
        if (e == cudaSuccess) e = sgc::launch_project_adam(st, cs, &launches[i]);
        if (e != cudaSuccess) st->t -= 1;                           // this state's moments were not touched
    }
    int shared = 0;
    if (e == cudaSuccess) e = sgc::launch_recover_group(states, weights, n, cs, &shared);   // a4 + a5, passes shared per batch
    for (int32_t i = 0; i < n; ++i) {
        sgc_state* st = states[i];
        st->last_stream = cs; st->has_stream = true; st->stepped = true;
        st->last_launches = launches[i] + (i == 0 ? shared : 0);     // the shared launches are booked on the first state
    }
    return (int)e;
}

SGC_API int sgc_step_chunked(sgc_state* const* states, int32_t c, const float* grad, float* weight, void* stream) {
    if (!states || !grad || !weight) return SGC_ERR_NULL;
    if (c < 1) return SGC_ERR_DIM;
    if (!states[0]) return SGC_ERR_NULL;
    const int64_t dc = states[0]->d;
    if ((dc * 4) % 16 != 0 && c > 1) return SGC_ERR_ALIGN;          // every chunk must start on a 16-byte boundary
    if (((uintptr_t)grad & 15u) || ((uintptr_t)weight & 15u)) return SGC_ERR_ALIGN;
    bool alike = true;
    for (int32_t i = 0; i < c && alike; ++i) {
        if (!states[i]) return SGC_ERR_NULL;
        alike = states[i]->d == dc && states[i]->k == states[0]->k && states[i]->s == states[0]->s && states[i]->seed == states[0]->seed;
        if (!on_own_device(states[i])) return SGC_ERR_DEVICE;
    }
    if (!alike) return SGC_ERR_GROUP;
    if (sgc::chunked_batch_eligible(states, c)) {
        // small per-chunk problems: all chunks in one set of launches (sgc_chunked.cu); a state listed twice is
        // rejected there, when the table of the chunk list is built
        cudaStream_t cs = static_cast<cudaStream_t>(stream);
        for (int32_t i = 0; i < c; ++i) states[i]->t += 1;
        int launches = 0;
        const cudaError_t e = sgc::launch_chunked_batch(states, c, grad, weight, cs, &launches);
        if (e == cudaErrorInvalidValue) { for (int32_t i = 0; i < c; ++i) states[i]->t -= 1; return SGC_ERR_GROUP; }
        if (e != cudaSuccess && launches == 0) { for (int32_t i = 0; i < c; ++i) states[i]->t -= 1; return (int)e; }
        for (int32_t i = 0; i < c; ++i) {
            sgc_state* st = states[i];
            st->last_stream = cs; st->has_stream = true; st->stepped = true;
            st->last_launches = i == 0 ? launches : 0;
        }
        return (int)e;
    }
    std::vector<const float*> gs((size_t)c);
    std::vector<float*> ws((size_t)c);
    for (int32_t i = 0; i < c; ++i) { gs[i] = grad + (size_t)i * dc; ws[i] = weight + (size_t)i * dc; }
    return sgc_step_group(states, gs.data(), ws.data(), c, stream);
}

SGC_API int sgc_cesgc_step(sgc_state* const* states, int32_t c, const float* B, int32_t r, int32_t m, int32_t n,
                           const float* grad, float* weight, float* scratch, void* stream) {
    if (!states || !B || !grad || !weight || !scratch) return SGC_ERR_NULL;
    if (c < 1 || !sgc::cesgc_shape_ok(r, m, n)) return SGC_ERR_DIM;
    if (!states[0]) return SGC_ERR_NULL;
    const int64_t dp = (int64_t)r * n;
    if (dp % c != 0 || states[0]->d != dp / c) return SGC_ERR_DIM;
    if ((uintptr_t)scratch & 15u) return SGC_ERR_ALIGN;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    float* P = scratch;                  // B G
    float* U = scratch + dp;             // the compressed problem's "weights": start at zero, end as -eta N
    cudaError_t e = sgc::launch_cesgc_project(B, grad, P, r, m, n, cs);
    if (e == cudaSuccess) e = cudaMemsetAsync(U, 0, (size_t)dp * sizeof(float), cs);
    if (e != cudaSuccess) return (int)e;
    const int rc = sgc_step_chunked(states, c, P, U, stream);
    if (rc != SGC_OK) return rc;
    return (int)sgc::launch_cesgc_back(B, U, weight, r, m, n, cs);
}

SGC_API int sgc_destroy(sgc_state* st) {
    if (!st) return SGC_OK;
    cudaError_t e = cudaSuccess;
    if (st->has_stream) e = cudaStreamSynchronize(st->last_stream);
    sgc::free_chunk_ws(st);
    if (st->spec_base) cudaFree(st->spec_base);
    cudaError_t e2 = cudaFree(st->base);
    if (st->h_rounds) cudaFreeHost(st->h_rounds);
    for (cudaEvent_t ev : *st->ev_pool) cudaEventDestroy(ev);
    delete st->ev_pool; delete st->ev_phase;
    delete st;
    return (int)(e != cudaSuccess ? e : e2);
}

SGC_API int sgc_set_alpha(sgc_state* st, float alpha) {
    if (!st) return SGC_ERR_NULL;
    if (!finite_f(alpha)) return SGC_ERR_HYPER;
    st->alpha = alpha;
    return SGC_OK;
}

SGC_API int sgc_reproject(sgc_state* st, uint64_t new_seed, void* stream) {
    if (!st) return SGC_ERR_NULL;
    if (!st->stepped) return SGC_ERR_NOSTEP;
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    cudaError_t e = sgc::launch_reproject(st, new_seed, cs);
    st->seed = new_seed;
    if (e == cudaSuccess && st->spec_ready) e = sgc::launch_inv_norms(new_seed, (uint64_t)st->d, st->k, st->inv_norm, cs);
    st->last_stream = cs; st->has_stream = true;
    return (int)e;
}

SGC_API int sgc_set_mode(sgc_state* st, int32_t mode) {
    if (!st) return SGC_ERR_NULL;
    if (mode < SGC_MODE_AUTO || mode > SGC_MODE_SPECULATIVE) return SGC_ERR_WHAT;
    if (mode == SGC_MODE_SPECULATIVE && !st->spec_ok) return SGC_ERR_DIM;
    if (mode == SGC_MODE_SPECULATIVE) {
        const cudaError_t e = ensure_spec(st);                       // small states get their speculative buffers here
        if (e != cudaSuccess) return (int)e;
    }
    st->mode = mode;
    return SGC_OK;
}

SGC_API int sgc_set_recovery(sgc_state* st, int32_t shared_support, double residual_tol) {
    if (!st) return SGC_ERR_NULL;
    if ((shared_support != 0 && shared_support != 1) || !(residual_tol >= 0.0) || !isfinite(residual_tol)) return SGC_ERR_WHAT;
    st->shared_support = shared_support;
    st->residual_tol = residual_tol;
    return SGC_OK;
}

SGC_API int sgc_get(sgc_state* st, int32_t what, void* dst, size_t bytes) {
    if (!st || !dst) return SGC_ERR_NULL;
    const size_t k = (size_t)st->k, s = (size_t)st->s;
    const void* src = nullptr;
    size_t n = 0;
    bool needs_step = true;
    switch (what) {
        case SGC_GET_T: {
            if (bytes < 8) return SGC_ERR_SIZE;
            memcpy(dst, &st->t, 8);
            return SGC_OK;
        }
        case SGC_GET_M: src = st->M; n = 4 * k; needs_step = false; break;
        case SGC_GET_V: src = st->V; n = 4 * k; needs_step = false; break;
        case SGC_GET_SEL_IDX: src = st->sel_idx; n = 4 * s; break;
        case SGC_GET_SEL_VAL: src = st->sel_val; n = 4 * s; break;
        case SGC_GET_P: src = st->p; n = 8 * k; break;
        case SGC_GET_Q: src = st->q; n = 8 * k; break;
        case SGC_GET_LAM_M: src = st->lam; n = 4 * s; break;
        case SGC_GET_LAM_V: src = st->lam + s; n = 4 * s; break;
        case SGC_GET_X_M: src = st->x; n = 8 * s; break;
        case SGC_GET_X_V: src = st->x + s; n = 8 * s; break;
        case SGC_GET_UPD_IDX: src = st->upd_idx; n = 4 * s; break;
        case SGC_GET_UPD_VAL: src = st->upd_val; n = 8 * s; break;
        case SGC_GET_N_UPD: src = &st->cnt->n_upd; n = 4; break;
        case SGC_GET_STATUS: src = &st->cnt->status; n = 4; needs_step = false; break;
        case SGC_GET_MISMATCH: src = &st->cnt->mismatch; n = 4; break;
        case SGC_GET_NEGV: src = &st->cnt->negv; n = 4; break;
        case SGC_GET_DONE_M: src = &st->cnt->done[0]; n = 4; break;
        case SGC_GET_DONE_V: src = &st->cnt->done[1]; n = 4; break;
        case SGC_GET_RNORM_M: src = st->rnorm; n = 8 * s; break;
        case SGC_GET_RNORM_V: src = st->rnorm + s; n = 8 * s; break;
        case SGC_GET_ROUNDS: src = &st->ctl->rounds; n = 4; break;
        case SGC_GET_FALLBACK: src = &st->ctl->fallback; n = 4; break;
        case SGC_GET_N_CAND: src = &st->ctl->n_cand; n = 4; break;
        case SGC_GET_LIST_ROUNDS: src = &st->ctl->list_rounds; n = 4; break;
        case SGC_GET_PASS_ROWS: src = &st->ctl->pass_rows; n = 4; break;
        case SGC_GET_ROUND_TRACE: src = &st->ctl->trace[0][0]; n = 4 * 3 * sgc::kMaxRounds; break;
        default: return SGC_ERR_WHAT;
    }
    if (needs_step && !st->stepped) return SGC_ERR_NOSTEP;
    if (bytes < n) return SGC_ERR_SIZE;
    cudaError_t e = cudaSuccess;
    if (st->has_stream) e = cudaStreamSynchronize(st->last_stream);
    if (e == cudaSuccess) e = cudaMemcpy(dst, src, n, cudaMemcpyDeviceToHost);
    return (int)e;
}

SGC_API int sgc_set_state(sgc_state* st, const float* M, const float* V, int64_t t) {
    if (!st || !M || !V) return SGC_ERR_NULL;
    if (t < 0) return SGC_ERR_DIM;
    cudaError_t e = cudaSuccess;
    if (st->has_stream) e = cudaStreamSynchronize(st->last_stream);
    if (e == cudaSuccess) e = cudaMemcpy(st->M, M, 4 * (size_t)st->k, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) e = cudaMemcpy(st->V, V, 4 * (size_t)st->k, cudaMemcpyHostToDevice);
    if (e == cudaSuccess) st->t = t;
    return (int)e;
}

SGC_API int sgc_clear_status(sgc_state* st) {
    if (!st) return SGC_ERR_NULL;
    cudaError_t e = cudaSuccess;
    if (st->has_stream) e = cudaStreamSynchronize(st->last_stream);
    if (e == cudaSuccess) e = cudaMemset(&st->cnt->status, 0, 4);
    return (int)e;
}

SGC_API int sgc_status(sgc_state* st, uint32_t* out) {
    if (!st || !out) return SGC_ERR_NULL;
    cudaError_t e = cudaSuccess;
    if (st->has_stream) e = cudaStreamSynchronize(st->last_stream);
    if (e == cudaSuccess) e = cudaMemcpy(out, &st->cnt->status, sizeof(uint32_t), cudaMemcpyDeviceToHost);
    return (int)e;
}

SGC_API int sgc_set_wait_limit(sgc_state* st, uint64_t ns) {
    if (st) st->wait_limit_ns = (unsigned long long)ns;
    else g_screen_wait_limit_ns.store((unsigned long long)ns);
    return SGC_OK;
}

SGC_API int sgc_set_max_rounds(sgc_state* st, int32_t rounds) {
    if (!st) return SGC_ERR_NULL;
    if (rounds < 0) return SGC_ERR_DIM;
    st->max_rounds = rounds;
    return SGC_OK;
}

SGC_API int sgc_last_launches(sgc_state* st, int32_t* out) {
    if (!st || !out) return SGC_ERR_NULL;
    *out = st->last_launches;
    return SGC_OK;
}

// folds the recorded event pairs into the per-phase totals (the stream must have drained)
static void drain_profile(sgc_state* st) {
    for (size_t i = 0; i + 1 < st->ev_used; i += 2) {
        float ms = 0.0f;
        if (cudaEventElapsedTime(&ms, (*st->ev_pool)[i], (*st->ev_pool)[i + 1]) == cudaSuccess)
            st->prof_ms[(*st->ev_phase)[i / 2]] += ms;
    }
    st->ev_used = 0;
    st->ev_phase->clear();
}

SGC_API int sgc_set_profile(sgc_state* st, int enable) {
    if (!st) return SGC_ERR_NULL;
    cudaError_t e = cudaSuccess;
    if (st->has_stream) e = cudaStreamSynchronize(st->last_stream);
    st->ev_used = 0;
    st->ev_phase->clear();
    for (int i = 0; i < sgc::kNumPhases; ++i) { st->prof_ms[i] = 0.0f; st->prof_launches[i] = 0; }
    st->profile = enable != 0;
    return (int)e;
}

SGC_API int sgc_get_profile(sgc_state* st, float* ms, int32_t* launches) {
    if (!st || !ms || !launches) return SGC_ERR_NULL;
    cudaError_t e = cudaSuccess;
    if (st->has_stream) e = cudaStreamSynchronize(st->last_stream);
    if (e != cudaSuccess) return (int)e;
    drain_profile(st);
    for (int i = 0; i < sgc::kNumPhases; ++i) { ms[i] = st->prof_ms[i]; launches[i] = st->prof_launches[i]; }
    return SGC_OK;
}

SGC_API int sgc_z_block(uint64_t seed, int64_t row0, int64_t nrows, int64_t col0, int64_t ncols, float* out, void* stream) {
    if (!out) return SGC_ERR_NULL;
    if (row0 < 0 || nrows < 0 || col0 < 0 || ncols < 0 || col0 + ncols > ((int64_t)1 << 32) ||
        row0 + nrows > ((int64_t)1 << 32))
        return SGC_ERR_DIM;
    return (int)sgc::launch_z_block(seed, row0, nrows, col0, ncols, out, static_cast<cudaStream_t>(stream));
}

SGC_API int sgc_screen(uint64_t seed, int64_t d, int32_t k, int32_t n, const uint16_t* rt, const float* tau, uint32_t* rep_count,
                       uint32_t* rep, int32_t rep_cap, int32_t* error_flag, void* stream) {
    if (!rt || !tau || !rep_count || !rep || !error_flag) return SGC_ERR_NULL;
    if (d < 1 || d >= ((int64_t)1 << 32) || k < 64 || k > sgc::kPassMaxK || k % 64 != 0 || n < 32 || n > sgc::kPassMaxN ||
        n % 32 != 0 || rep_cap < 1)
        return SGC_ERR_DIM;
    if (((uintptr_t)rt & 15u) || ((uintptr_t)rep & 7u)) return SGC_ERR_ALIGN;
    int dev = 0, sms = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e == cudaSuccess) e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess) e = sgc::pass_configure(n);
    unsigned char map[sgc::kTensorMapBytes];
    if (e == cudaSuccess) e = sgc::pass_encode_map(map, rt, n, k);
    cudaStream_t cs = static_cast<cudaStream_t>(stream);
    if (e == cudaSuccess) e = cudaMemsetAsync(rep_count, 0, sizeof(uint32_t) * (size_t)n, cs);
    if (e == cudaSuccess) e = cudaMemsetAsync(error_flag, 0, sizeof(int32_t), cs);
    {
        int* errors[sgc::kPassMaxBatch] = {error_flag};
        if (e == cudaSuccess)
            e = sgc::launch_pass(map, seed, (uint64_t)d, k, n, tau, nullptr, nullptr, rep_count, reinterpret_cast<uint2*>(rep), rep_cap,
                                 nullptr, errors, sms, cs, nullptr, nullptr, 0, g_screen_wait_limit_ns.load());
    }
    return (int)e;
}

SGC_API const char* sgc_strerror(int code) {
    switch (code) {
        case SGC_OK: return "success";
        case SGC_ERR_NULL: return "a required pointer is NULL";
        case SGC_ERR_DIM: return "dimension out of range (need 1 <= s <= min(k, d), d < 2^32, k <= 16384, s <= 1024; "
                                 "the speculative recovery and sgc_screen need k to be a multiple of 64)";
        case SGC_ERR_HYPER: return "hyper-parameter out of range (beta in [0,1), eps > 0, finite lr and alpha)";
        case SGC_ERR_ALIGN: return "grad and weight must be 16-byte aligned";
        case SGC_ERR_WHAT: return "unknown record selector";
        case SGC_ERR_SIZE: return "destination buffer too small";
        case SGC_ERR_GROUP: return "states of a group must be distinct and share d, k, s and seed";
        case SGC_ERR_NOSTEP: return "no step has run yet";
        case SGC_ERR_DEVICE: return "the state belongs to another device than the current one";
        default: break;
    }
    if (code > 0) return cudaGetErrorString((cudaError_t)code);
    return "unknown error";
}

SGC_API int sgc_version(void) { return 200; }

}  // extern "C"
