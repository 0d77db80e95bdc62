// The C-ABI entry points: argument validation, workspace planning, kernel-family choice.
// Every function here runs on the host and only enqueues work; see include/obcache.h.
#include "obc_common.cuh"
#include <atomic>
#include <cmath>
#include <cstring>
#include <mutex>
#include <vector>

namespace obc {

static thread_local int g_last_cuda_error = 0;
void set_last_cuda_error(int e) { g_last_cuda_error = e; }

// ---- optional per-kernel event timing ---------------------------------------------------------
namespace {
struct ProfRec { const char* name; cudaEvent_t e0, e1; };
std::mutex g_prof_mu;
std::vector<ProfRec> g_prof;
std::atomic<bool> g_prof_on{false};
}  // namespace

ProfScope::ProfScope(const char* name, cudaStream_t s) : slot(-1), stream(s) {
    if (!g_prof_on.load(std::memory_order_relaxed)) return;
    ProfRec r{name, nullptr, nullptr};
    if (cudaEventCreate(&r.e0) != cudaSuccess || cudaEventCreate(&r.e1) != cudaSuccess) return;
    cudaEventRecord(r.e0, s);
    std::lock_guard<std::mutex> lk(g_prof_mu);
    g_prof.push_back(r);
    slot = (int)g_prof.size() - 1;
}
ProfScope::~ProfScope() {
    if (slot < 0) return;
    std::lock_guard<std::mutex> lk(g_prof_mu);
    if (slot < (int)g_prof.size()) cudaEventRecord(g_prof[slot].e1, stream);
}

namespace {

int elem_size(int dtype) { return dtype == OBC_BF16 ? 2 : 4; }

obc_status check_tensor(const obc_tensor& t, bool need_batch_stride) {
    if (!t.ptr) return OBC_ERR_NULL;
    if (t.dtype != OBC_F32 && t.dtype != OBC_BF16) return OBC_ERR_UNSUPPORTED;
    const long long es = elem_size(t.dtype);
    if (((uintptr_t)t.ptr & 15) != 0) return OBC_ERR_ALIGN;
    if ((t.stride_t * es) % 16 || (t.stride_h * es) % 16 || (t.stride_b * es) % 16) return OBC_ERR_ALIGN;
    if (t.stride_t < kD || t.stride_h < 0 || t.stride_b < 0) return OBC_ERR_SHAPE;
    (void)need_batch_stride;
    return OBC_OK;
}

TensorView view(const obc_tensor& t) { return TensorView{t.ptr, t.stride_b, t.stride_h, t.stride_t}; }

obc_status resolve_score(const obc_score_params* p, ScoreShape* s) {
    if (!p) return OBC_ERR_NULL;
    if (p->struct_size != sizeof(obc_score_params)) return OBC_ERR_UNSUPPORTED;
    if (p->head_dim != kD) return OBC_ERR_UNSUPPORTED;
    if (p->batch < 1 || p->n_kv_heads < 1 || p->n_q_heads < 1 || p->n_q_heads % p->n_kv_heads) return OBC_ERR_SHAPE;
    if (p->window < 1 || p->max_len < 1 || (!p->mask_lens && p->window > p->max_len)) return OBC_ERR_SHAPE;
    if ((long long)p->batch * p->n_kv_heads > 65535) return OBC_ERR_SHAPE;
    const unsigned known = OBC_VAR_V | OBC_VAR_K | OBC_VAR_VK | OBC_VAR_ATTN | OBC_VAR_VATP;
    if (p->variants == 0 || (p->variants & ~known)) return OBC_ERR_UNSUPPORTED;
    if (p->path < OBC_PATH_AUTO || p->path > OBC_PATH_TC) return OBC_ERR_UNSUPPORTED;
    s->B = p->batch; s->Hq = p->n_q_heads; s->Hkv = p->n_kv_heads; s->G = s->Hq / s->Hkv;
    s->W = p->window; s->R = s->G * s->W; s->Nmax = p->max_len; s->seq_lens = p->seq_lens; s->mask_lens = p->mask_lens;
    s->scale = p->scale > 0.f ? p->scale : 1.0f / sqrtf((float)kD);
    s->causal = p->causal != 0; s->variants = p->variants;
    s->n_planes = __builtin_popcount(p->variants);
    return OBC_OK;
}

// which kernel family runs: decided from the parameters alone so that the size query and the
// launch agree.  The dtype is not known to the size query, so the workspace covers both.
bool want_tc(const obc_score_params* p, const ScoreShape& s, int dtype, const TensorView& q) {
    if (p->path == OBC_PATH_SIMT) return false;
    return tc_supported(s, dtype, q);
}

}  // namespace
}  // namespace obc

using namespace obc;

extern "C" {

obc_status obc_score_workspace(const obc_score_params* p, size_t* bytes) {
    if (!bytes) return OBC_ERR_NULL;
    ScoreShape s;
    obc_status st = resolve_score(p, &s);
    if (st != OBC_OK) return st;
    size_t need = make_simt_plan(s, s.R, false).bytes;
    if (p->path != OBC_PATH_SIMT && tc_shape_supported(s)) {
        size_t t = tc_workspace_bytes(s);
        if (t > need) need = t;
    }
    *bytes = need;
    return OBC_OK;
}

static obc_status score_impl(const obc_score_params* p, obc_tensor q, obc_tensor k, obc_tensor v,
                             const obc_tensor* o, const float* lse,
                             float* scores, void* workspace, size_t workspace_bytes, void* stream) {
    ScoreShape s;
    obc_status st = resolve_score(p, &s);
    if (st != OBC_OK) return st;
    if (!scores) return OBC_ERR_NULL;
    if ((st = check_tensor(q, true)) != OBC_OK) return st;
    if ((st = check_tensor(k, true)) != OBC_OK) return st;
    if ((st = check_tensor(v, true)) != OBC_OK) return st;
    if (q.dtype != k.dtype || k.dtype != v.dtype) return OBC_ERR_UNSUPPORTED;
    if (((uintptr_t)scores & 15) != 0) return OBC_ERR_ALIGN;
    GivenAttention given{};
    if (o) {
        if (!lse) return OBC_ERR_NULL;
        if ((st = check_tensor(*o, true)) != OBC_OK) return st;
        if (((uintptr_t)lse & 3) != 0) return OBC_ERR_ALIGN;
        given = GivenAttention{view(*o), o->dtype, lse};
    }
    size_t need = 0;
    if ((st = obc_score_workspace(p, &need)) != OBC_OK) return st;
    if (!workspace || workspace_bytes < need) return OBC_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255) != 0) return OBC_ERR_ALIGN;
    const bool tc = want_tc(p, s, q.dtype, view(q));
    if (p->path == OBC_PATH_TC && !tc) return OBC_ERR_UNSUPPORTED;
    if (tc) return launch_score_tc(s, view(q), view(k), view(v), scores, workspace, (cudaStream_t)stream, o ? &given : nullptr);
    const SimtPlan plan = make_simt_plan(s, s.R, false);
    st = o ? launch_given_prep(s, plan, given, workspace, (cudaStream_t)stream)
           : launch_simt_pass1_combine(s, plan, q.dtype, view(q), view(k), view(v), workspace, (cudaStream_t)stream);
    if (st != OBC_OK) return st;
    return launch_simt_pass2(s, plan, q.dtype, view(q), view(k), view(v), scores, workspace, (cudaStream_t)stream);
}

obc_status obc_window_attention(const obc_score_params* p, obc_tensor q, obc_tensor k, obc_tensor v,
                                float* o_out, float* lse_out,
                                void* workspace, size_t workspace_bytes, void* stream) {
    ScoreShape s;
    obc_status st = resolve_score(p, &s);
    if (st != OBC_OK) return st;
    if (!o_out || !lse_out) return OBC_ERR_NULL;
    if ((st = check_tensor(q, true)) != OBC_OK) return st;
    if ((st = check_tensor(k, true)) != OBC_OK) return st;
    if ((st = check_tensor(v, true)) != OBC_OK) return st;
    if (q.dtype != k.dtype || k.dtype != v.dtype) return OBC_ERR_UNSUPPORTED;
    if (((uintptr_t)o_out & 15) != 0 || ((uintptr_t)lse_out & 3) != 0) return OBC_ERR_ALIGN;
    size_t need = 0;
    if ((st = obc_score_workspace(p, &need)) != OBC_OK) return st;
    if (!workspace || workspace_bytes < need) return OBC_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255) != 0) return OBC_ERR_ALIGN;
    const bool tc = want_tc(p, s, q.dtype, view(q));
    if (p->path == OBC_PATH_TC && !tc) return OBC_ERR_UNSUPPORTED;
    SimtPlan plan;
    if (tc) {
        st = launch_attention_tc(s, view(q), view(k), view(v), workspace, (cudaStream_t)stream, &plan);
    } else {
        plan = make_simt_plan(s, s.R, false);
        st = launch_simt_pass1_combine(s, plan, q.dtype, view(q), view(k), view(v), workspace, (cudaStream_t)stream);
    }
    if (st != OBC_OK) return st;
    return launch_export_attention(s, plan, workspace, o_out, lse_out, (cudaStream_t)stream);
}

obc_status obc_merge_attention(int32_t n_parts, int64_t rows, int32_t head_dim,
                               const float* o_parts, const float* lse_parts,
                               float* o_out, float* lse_out, void* stream) {
    if (head_dim != kD) return OBC_ERR_UNSUPPORTED;
    if (n_parts < 1 || n_parts > 4096 || rows < 1 || rows > 0x7fffffffLL) return OBC_ERR_SHAPE;
    if (!o_parts || !lse_parts || !o_out || !lse_out) return OBC_ERR_NULL;
    if ((((uintptr_t)o_parts | (uintptr_t)o_out) & 15) != 0 || (((uintptr_t)lse_parts | (uintptr_t)lse_out) & 3) != 0) return OBC_ERR_ALIGN;
    return launch_merge_attention(n_parts, rows, o_parts, lse_parts, o_out, lse_out, (cudaStream_t)stream);
}

obc_status obc_shard_indices(int32_t batch, int32_t n_kv_heads, int32_t idx_stride, const int32_t* idx,
                             int32_t token_offset, int32_t n_local, int32_t* idx_local, int32_t* counts, void* stream) {
    if (batch < 1 || n_kv_heads < 1 || idx_stride < 1 || token_offset < 0 || n_local < 1) return OBC_ERR_SHAPE;
    if ((long long)batch * n_kv_heads > 0x7fffffffLL || (long long)token_offset + n_local > 0x7fffffffLL) return OBC_ERR_SHAPE;
    if (!idx || !idx_local || !counts) return OBC_ERR_NULL;
    if (idx == idx_local) return OBC_ERR_SHAPE;
    return launch_shard_indices(batch * n_kv_heads, idx_stride, token_offset, n_local, idx, idx_local, counts, (cudaStream_t)stream);
}

obc_status obc_score(const obc_score_params* p, obc_tensor q, obc_tensor k, obc_tensor v,
                     float* scores, void* workspace, size_t workspace_bytes, void* stream) {
    return score_impl(p, q, k, v, nullptr, nullptr, scores, workspace, workspace_bytes, stream);
}

obc_status obc_score_given(const obc_score_params* p, obc_tensor q, obc_tensor k, obc_tensor v,
                           obc_tensor o, const float* lse,
                           float* scores, void* workspace, size_t workspace_bytes, void* stream) {
    if (!lse) return OBC_ERR_NULL;
    return score_impl(p, q, k, v, &o, lse, scores, workspace, workspace_bytes, stream);
}

obc_status obc_score_status(const void* workspace, void* stream) {
    if (!workspace) return OBC_ERR_NULL;
    unsigned int word = 0;
    OBC_CUDA_TRY(cudaMemcpyAsync(&word, workspace, sizeof(word), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    OBC_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    return word == 0 ? OBC_OK : OBC_ERR_TIMEOUT;
}

obc_status obc_score_kernel_spans(void* workspace, void* stream, double* pass1_us, double* pass2_us) {
    if (!workspace || !pass1_us || !pass2_us) return OBC_ERR_NULL;
    unsigned long long w[4] = {0, 0, 0, 0};
    char* at = static_cast<char*>(workspace) + kSpanOffset;
    OBC_CUDA_TRY(cudaMemcpyAsync(w, at, sizeof(w), cudaMemcpyDeviceToHost, (cudaStream_t)stream));
    OBC_CUDA_TRY(cudaMemsetAsync(at, 0, sizeof(w), (cudaStream_t)stream));
    OBC_CUDA_TRY(cudaStreamSynchronize((cudaStream_t)stream));
    auto span_us = [](unsigned long long not_start, unsigned long long end) {
        const unsigned long long start = ~not_start;
        return (not_start == 0 || end == 0 || end < start) ? 0.0 : (double)(end - start) * 1e-3;
    };
    *pass1_us = span_us(w[0], w[1]);
    *pass2_us = span_us(w[2], w[3]);
    return OBC_OK;
}

static obc_status resolve_select(const obc_select_params* p, SelectShape* s) {
    if (!p) return OBC_ERR_NULL;
    if (p->struct_size != sizeof(obc_select_params)) return OBC_ERR_UNSUPPORTED;
    if (p->batch < 1 || p->n_kv_heads < 1 || p->max_len < 1) return OBC_ERR_SHAPE;
    if ((long long)p->batch * p->n_kv_heads > 65535) return OBC_ERR_SHAPE;      // units index gridDim.y
    if (p->n_sink < 0 || p->n_recent < 0 || p->idx_stride < 1) return OBC_ERR_SHAPE;
    if (p->pool_mode < OBC_POOL_NONE || p->pool_mode > OBC_POOL_MAX) return OBC_ERR_UNSUPPORTED;
    if (p->pool_kernel < 1 || p->pool_kernel % 2 == 0) return OBC_ERR_SHAPE;
    if (!p->budgets) {
        if (p->budget < p->n_sink + p->n_recent || p->budget > p->idx_stride) return OBC_ERR_SHAPE;
        if (!p->seq_lens && p->budget > p->max_len) return OBC_ERR_SHAPE;
    }
    if (!p->seq_lens && p->n_sink + p->n_recent > p->max_len) return OBC_ERR_SHAPE;
    *s = SelectShape{p->batch, p->n_kv_heads, p->max_len, p->seq_lens, p->budget, p->budgets,
                     p->idx_stride, p->n_sink, p->n_recent, p->pool_mode, p->pool_kernel};
    return OBC_OK;
}

obc_status obc_select_workspace(const obc_select_params* p, size_t* bytes) {
    if (!bytes) return OBC_ERR_NULL;
    SelectShape s;
    obc_status st = resolve_select(p, &s);
    if (st != OBC_OK) return st;
    *bytes = select_workspace_bytes(s.B, s.Hkv, s.Nmax);
    return OBC_OK;
}

obc_status obc_select(const obc_select_params* p, const float* scores, int32_t* idx,
                      void* workspace, size_t workspace_bytes, void* stream) {
    SelectShape s;
    obc_status st = resolve_select(p, &s);
    if (st != OBC_OK) return st;
    if (!scores || !idx) return OBC_ERR_NULL;
    if (!workspace || workspace_bytes < select_workspace_bytes(s.B, s.Hkv, s.Nmax)) return OBC_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255) != 0) return OBC_ERR_ALIGN;
    return launch_select(s, scores, idx, workspace, (cudaStream_t)stream);
}

// scored tokens every head keeps by its own ranking: floor(safeguard * n_hh), in double like the size query
static obc_status resolve_adaptive(const obc_select_params* p, float safeguard, SelectShape* s, int* n_safe) {
    obc_status st = resolve_select(p, s);
    if (st != OBC_OK) return st;
    if (p->budgets) return OBC_ERR_UNSUPPORTED;            // one budget for the whole batch
    if (!(safeguard >= 0.f && safeguard <= 1.f)) return OBC_ERR_SHAPE;
    if ((long long)s->Hkv * s->Nmax > 0x7fffffffLL || (long long)s->Hkv * s->budget > 0x7fffffffLL) return OBC_ERR_SHAPE;
    const int n_hh = s->budget - s->n_sink - s->n_recent;
    int ns = (int)floor((double)safeguard * (double)n_hh);
    if (ns > n_hh) ns = n_hh;
    *n_safe = ns;
    return OBC_OK;
}

obc_status obc_select_adaptive_workspace(const obc_select_params* p, float safeguard, size_t* bytes) {
    if (!bytes) return OBC_ERR_NULL;
    SelectShape s; int n_safe = 0;
    obc_status st = resolve_adaptive(p, safeguard, &s, &n_safe);
    if (st != OBC_OK) return st;
    *bytes = select_adaptive_workspace_bytes(s, n_safe);
    return OBC_OK;
}

obc_status obc_select_adaptive(const obc_select_params* p, float safeguard, const float* scores,
                               int32_t* idx, int32_t* counts, void* workspace, size_t workspace_bytes, void* stream) {
    SelectShape s; int n_safe = 0;
    obc_status st = resolve_adaptive(p, safeguard, &s, &n_safe);
    if (st != OBC_OK) return st;
    if (!scores || !idx || !counts) return OBC_ERR_NULL;
    if (!workspace || workspace_bytes < select_adaptive_workspace_bytes(s, n_safe)) return OBC_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255) != 0) return OBC_ERR_ALIGN;
    return launch_select_adaptive(s, n_safe, scores, idx, counts, workspace, (cudaStream_t)stream);
}

obc_status obc_select_noalloc(const obc_select_params* p, const float* scores, int32_t* idx, void* stream) {
    SelectShape s;
    obc_status st = resolve_select(p, &s);
    if (st != OBC_OK) return st;
    if (!scores || !idx) return OBC_ERR_NULL;
    return launch_select_static(s, scores, idx, (cudaStream_t)stream);
}

obc_status obc_compact(int32_t batch, int32_t n_kv_heads, int32_t head_dim, int32_t idx_stride,
                       int32_t max_len, obc_tensor k, obc_tensor v, const int32_t* idx,
                       obc_tensor k_out, obc_tensor v_out,
                       const float* scores_in, float* scores_out, void* stream) {
    if (head_dim != kD) return OBC_ERR_UNSUPPORTED;
    if (batch < 1 || n_kv_heads < 1 || idx_stride < 1 || max_len < 1) return OBC_ERR_SHAPE;
    if ((long long)batch * n_kv_heads > 65535) return OBC_ERR_SHAPE;            // units index gridDim.y
    if (!idx) return OBC_ERR_NULL;
    if ((scores_in == nullptr) != (scores_out == nullptr)) return OBC_ERR_NULL;
    obc_status st;
    if ((st = check_tensor(k, true)) != OBC_OK) return st;
    if ((st = check_tensor(v, true)) != OBC_OK) return st;
    if ((st = check_tensor(k_out, true)) != OBC_OK) return st;
    if ((st = check_tensor(v_out, true)) != OBC_OK) return st;
    if (k.dtype != v.dtype || k.dtype != k_out.dtype || k.dtype != v_out.dtype) return OBC_ERR_UNSUPPORTED;
    return launch_gather(batch, n_kv_heads, idx_stride, max_len, elem_size(k.dtype), view(k), view(v),
                         view(k_out), view(v_out), idx, scores_in, scores_out, (cudaStream_t)stream);
}

static obc_status resolve_decode(const obc_decode_params* p, DecodeShape* s) {
    if (!p) return OBC_ERR_NULL;
    if (p->struct_size != sizeof(obc_decode_params)) return OBC_ERR_UNSUPPORTED;
    if (p->head_dim != kD) return OBC_ERR_UNSUPPORTED;
    if (p->batch < 1 || p->n_kv_heads < 1 || p->n_q_heads < 1 || p->n_q_heads % p->n_kv_heads) return OBC_ERR_SHAPE;
    if (p->n_q_heads / p->n_kv_heads > 8) return OBC_ERR_UNSUPPORTED;
    if (p->capacity < 1 || p->budget < 1 || p->capacity <= p->budget) return OBC_ERR_SHAPE;
    if (p->n_sink < 0 || p->n_recent < 1 || p->n_sink + p->n_recent >= p->budget) return OBC_ERR_SHAPE;
    if (p->variant != OBC_VAR_V && p->variant != OBC_VAR_K && p->variant != OBC_VAR_VK && p->variant != OBC_VAR_ATTN)
        return OBC_ERR_UNSUPPORTED;
    if ((long long)p->batch * p->n_kv_heads > 65535) return OBC_ERR_SHAPE;
    if (p->acc_window < 0 || p->acc_window > 4096) return OBC_ERR_SHAPE;
    *s = DecodeShape{p->batch, p->n_q_heads, p->n_kv_heads, p->n_q_heads / p->n_kv_heads, p->capacity,
                     p->budget, p->n_sink, p->n_recent, p->variant,
                     p->scale > 0.f ? p->scale : 1.0f / sqrtf((float)kD),
                     p->acc_window, p->acc_window > 0 ? p->s_hist : nullptr};
    return OBC_OK;
}

obc_status obc_decode_workspace(const obc_decode_params* p, size_t* bytes) {
    if (!bytes) return OBC_ERR_NULL;
    DecodeShape s;
    obc_status st = resolve_decode(p, &s);
    if (st != OBC_OK) return st;
    *bytes = decode_workspace_bytes(s);
    return OBC_OK;
}

obc_status obc_decode_step(const obc_decode_params* p, obc_tensor q_t, obc_tensor k_t, obc_tensor v_t,
                           obc_tensor k_cache, obc_tensor v_cache, float* s_acc, int32_t* pos,
                           int32_t* state, int32_t step_pos,
                           void* workspace, size_t workspace_bytes, void* stream) {
    DecodeShape s;
    obc_status st = resolve_decode(p, &s);
    if (st != OBC_OK) return st;
    if (!s_acc || !pos || !state) return OBC_ERR_NULL;
    if (s.acc_window > 0 && !s.s_hist) return OBC_ERR_NULL;
    if (s.acc_window > 0 && ((uintptr_t)s.s_hist & 3) != 0) return OBC_ERR_ALIGN;
    const obc_tensor* ts[5] = {&q_t, &k_t, &v_t, &k_cache, &v_cache};
    for (int i = 0; i < 5; ++i) {
        if ((st = check_tensor(*ts[i], true)) != OBC_OK) return st;
        if (ts[i]->dtype != OBC_BF16) return OBC_ERR_UNSUPPORTED;
    }
    if (step_pos < 0) return OBC_ERR_SHAPE;
    if (!workspace || workspace_bytes < decode_workspace_bytes(s)) return OBC_ERR_WORKSPACE;
    if (((uintptr_t)workspace & 255) != 0) return OBC_ERR_ALIGN;
    return launch_decode(s, view(q_t), view(k_t), view(v_t), view(k_cache), view(v_cache), s_acc, pos, state,
                         step_pos, workspace, (cudaStream_t)stream);
}

obc_status obc_profile_begin(void) {
    std::lock_guard<std::mutex> lk(g_prof_mu);
    for (auto& r : g_prof) { cudaEventDestroy(r.e0); cudaEventDestroy(r.e1); }
    g_prof.clear();
    g_prof_on.store(true);
    return OBC_OK;
}

obc_status obc_profile_end(obc_kernel_time* out, int32_t max_out, int32_t* n_out) {
    if (!out || !n_out || max_out < 1) return OBC_ERR_NULL;
    g_prof_on.store(false);
    std::lock_guard<std::mutex> lk(g_prof_mu);
    int n = 0;
    obc_status st = OBC_OK;
    for (auto& r : g_prof) {
        float ms = 0.f;
        cudaError_t e = cudaEventSynchronize(r.e1);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, r.e0, r.e1);
        if (e != cudaSuccess) { set_last_cuda_error((int)e); st = OBC_ERR_CUDA; }
        int j = 0;
        for (; j < n; ++j) if (std::strcmp(out[j].name, r.name) == 0) break;
        if (j == n) {
            if (n == max_out) { cudaEventDestroy(r.e0); cudaEventDestroy(r.e1); continue; }
            std::memset(&out[n], 0, sizeof(out[n]));
            std::strncpy(out[n].name, r.name, sizeof(out[n].name) - 1);
            ++n;
        }
        out[j].launches += 1; out[j].ms_total += ms;
        cudaEventDestroy(r.e0); cudaEventDestroy(r.e1);
    }
    g_prof.clear();
    *n_out = n;
    return st;
}

const char* obc_status_string(obc_status s) {
    switch (s) {
        case OBC_OK: return "ok";
        case OBC_ERR_NULL: return "a required pointer is NULL";
        case OBC_ERR_SHAPE: return "inconsistent or out-of-range sizes";
        case OBC_ERR_UNSUPPORTED: return "unsupported head_dim, dtype, variant, mode or struct size";
        case OBC_ERR_ALIGN: return "pointer or stride not 16-byte aligned (workspace: 256-byte)";
        case OBC_ERR_WORKSPACE: return "workspace missing or too small";
        case OBC_ERR_CUDA: return "a CUDA call failed (see obc_last_cuda_error)";
        case OBC_ERR_TIMEOUT: return "a bounded device-side wait gave up";
        case OBC_ERR_CAPACITY: return "problem larger than the fixed capacity of the allocation-free entry point";
    }
    return "unknown status";
}

int obc_last_cuda_error(void) { return g_last_cuda_error; }
int obc_version(void) { return 100; }

}  // extern "C"
