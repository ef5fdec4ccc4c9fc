// Host side of the C ABI: argument validation, workspace carving and kernel launches.
// Nothing here allocates device memory or synchronises.
#include <atomic>

#include "ciar_internal.h"

namespace ciar {

namespace {
std::atomic<int64_t> g_launches{0};
// bound of the device-side waits (about a second of SM clocks) and the test hook that withholds one row's copy
std::atomic<int64_t> g_wait_cycles{2000000000ll};
std::atomic<int32_t> g_drop_cta{-1}, g_drop_k{-1};

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

inline int elem_size(int dtype) { return dtype == CIAR_F32 ? 4 : 2; }

ciar_status check_desc(const ciar_logits_desc *d, const void *logits)
{
    if (!d) return CIAR_ERR_INVALID_ARG;
    if (d->dtype != CIAR_F32 && d->dtype != CIAR_BF16) return CIAR_ERR_UNSUPPORTED;
    if (d->rows < 0 || d->vocab < 1 || d->row_stride < d->vocab) return CIAR_ERR_INVALID_ARG;
    if (d->valid_count < 1 || d->valid_begin < 0 || (int64_t)d->valid_begin + d->valid_count > d->vocab)
        return CIAR_ERR_INVALID_ARG;
    if (d->rows > 0 && !logits) return CIAR_ERR_INVALID_ARG;
    if (((uintptr_t)logits & 15u) != 0 || (d->row_stride * elem_size(d->dtype)) % 16 != 0) return CIAR_ERR_ALIGNMENT;
    return CIAR_OK;
}

ciar_status check_interval(const ciar_logits_desc *d, const ciar_interval_params *p)
{
    if (!p) return CIAR_ERR_INVALID_ARG;
    if (p->radius_mode < CIAR_RADIUS_SCALAR || p->radius_mode > CIAR_RADIUS_PER_CODE) return CIAR_ERR_INVALID_ARG;
    if (p->policy < CIAR_POLICY_INTERVAL || p->policy > CIAR_POLICY_ALL) return CIAR_ERR_INVALID_ARG;
    if (!(p->r_max > 0.f) || !(p->r_max <= 80.f)) return CIAR_ERR_INVALID_ARG;
    if (!(p->lo_cap > 0.f) || !(p->hi_cap > 0.f)) return CIAR_ERR_INVALID_ARG;
    if (p->radius_mode == CIAR_RADIUS_SCALAR && !p->radius_is_raw && !(p->r_scalar >= 0.f)) return CIAR_ERR_INVALID_ARG;
    if (p->radius_mode != CIAR_RADIUS_SCALAR && d->rows > 0 && !p->radius) return CIAR_ERR_INVALID_ARG;
    if (p->radius_mode == CIAR_RADIUS_PER_CODE && ((uintptr_t)p->radius & 15u) != 0) return CIAR_ERR_ALIGNMENT;
    if (p->policy == CIAR_POLICY_RANDOM && d->rows > 0 && !p->u_flag) return CIAR_ERR_INVALID_ARG;
    if (p->tau != p->tau) return CIAR_ERR_INVALID_ARG;
    return CIAR_OK;
}

ciar_status check_verify_params(const ciar_verify_params *vp)
{
    if (!vp) return CIAR_ERR_INVALID_ARG;
    if (vp->window < 1 || vp->window > CIAR_MAX_WINDOW) return CIAR_ERR_INVALID_ARG;
    if (vp->mode < CIAR_VERIFY_ANCHORED || vp->mode > CIAR_VERIFY_ALL) return CIAR_ERR_INVALID_ARG;
    return CIAR_OK;
}

void fill_quantify_args(QuantifyArgs &a, const ciar_logits_desc *d, const void *logits, const ciar_interval_params *p)
{
    a.logits = logits;
    a.rows = d->rows;
    a.row_stride = d->row_stride;
    a.vb = d->valid_begin;
    a.n = d->valid_count;
    a.rm.pos = nullptr;
    a.rm.seq_len = 0;
    a.rm.window = 1;
    a.radius_mode = p->radius_mode;
    a.radius_is_raw = p->radius_is_raw;
    a.radius = p->radius;
    a.r_scalar = p->r_scalar;
    a.r_max = p->r_max;
    a.lo_cap = p->lo_cap;
    a.hi_cap = p->hi_cap;
    a.policy = p->policy;
    a.tau = p->tau;
    a.u_flag = p->u_flag;
    a.wait_cycles = g_wait_cycles.load(std::memory_order_relaxed);
    a.drop_cta = g_drop_cta.load(std::memory_order_relaxed);
    a.drop_k = g_drop_k.load(std::memory_order_relaxed);
}

// Layout of the workspace: verify scratch first, then the per-step arrays of the decode loop.
struct WsLayout {
    size_t window_done, candidate, accept, tested, tq_max, tq_sum;  // verify
    size_t flag, row_max, sum_exp, first_flag, accepted_len, resampled;  // decode step
    size_t total;
};

WsLayout ws_layout(int64_t rows, int32_t window)
{
    const size_t r = (size_t)rows, nw = (size_t)(rows / window) + 1;
    WsLayout l;
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 16); return o; };
    l.window_done = take(nw * 4);
    l.candidate = take(r * 4);
    l.accept = take(r);
    l.tested = take((r + 1) * 4);
    l.tq_max = take(r * 4);
    l.tq_sum = take(r * 4);
    l.flag = take(r);
    l.row_max = take(r * 4);
    l.sum_exp = take(r * 4);
    l.first_flag = take(nw * 4);
    l.accepted_len = take(nw * 4);
    l.resampled = take(nw * 4);
    l.total = off;
    return l;
}

}  // namespace

void count_launch() { g_launches.fetch_add(1, std::memory_order_relaxed); }

int sm_count()
{
    static int cached[64] = { 0 };
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    if (cached[dev] == 0) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached[dev] = n;
    }
    return cached[dev];
}

}  // namespace ciar

using namespace ciar;

extern "C" {

const char *ciar_status_string(ciar_status s)
{
    switch (s) {
    case CIAR_OK: return "ok";
    case CIAR_ERR_INVALID_ARG: return "invalid argument";
    case CIAR_ERR_UNSUPPORTED: return "unsupported dtype or shape";
    case CIAR_ERR_ALIGNMENT: return "pointer or row stride not 16-byte aligned";
    case CIAR_ERR_WORKSPACE_TOO_SMALL: return "workspace too small";
    case CIAR_ERR_CUDA: return "CUDA error";
    case CIAR_ERR_TIMEOUT: return "device-side wait ran out";
    }
    return "unknown status";
}

int ciar_version(void) { return CIAR_VERSION; }

ciar_status ciar_test_stall(int32_t cta, int32_t row_in_walk, int64_t wait_cycles)
{
    g_drop_cta.store(cta < 0 ? -1 : cta, std::memory_order_relaxed);
    g_drop_k.store(cta < 0 ? -1 : row_in_walk, std::memory_order_relaxed);
    g_wait_cycles.store(wait_cycles > 0 ? wait_cycles : 2000000000ll, std::memory_order_relaxed);
    return CIAR_OK;
}

int64_t ciar_launch_count(void) { return g_launches.load(std::memory_order_relaxed); }

size_t ciar_workspace_bytes(int64_t rows, int32_t window)
{
    if (rows < 0 || window < 1) return 0;
    return ws_layout(rows, window).total;
}

ciar_status ciar_quantify(const ciar_logits_desc *desc, const void *draft_logits,
                          const ciar_interval_params *params, const ciar_quantify_out *out, void *stream)
{
    ciar_status s = check_desc(desc, draft_logits);
    if (s != CIAR_OK) return s;
    s = check_interval(desc, params);
    if (s != CIAR_OK) return s;
    if (!out) return CIAR_ERR_INVALID_ARG;
    if (desc->rows == 0) return CIAR_OK;
    QuantifyArgs a;
    fill_quantify_args(a, desc, draft_logits, params);
    a.out = *out;
    return launch_quantify(a, desc->dtype, (cudaStream_t)stream) == cudaSuccess ? CIAR_OK : CIAR_ERR_CUDA;
}

ciar_status ciar_verify(const ciar_logits_desc *desc, const void *draft_logits, const void *target_logits,
                        const int32_t *draft_tokens, const uint8_t *flag,
                        const float *draft_row_max, const float *draft_sum_exp,
                        const float *u_accept, const float *u_resample,
                        const ciar_verify_params *params, const ciar_verify_out *out,
                        void *ws, size_t ws_bytes, void *stream)
{
    ciar_status s = check_desc(desc, draft_logits);
    if (s != CIAR_OK) return s;
    s = check_desc(desc, target_logits);
    if (s != CIAR_OK) return s;
    s = check_verify_params(params);
    if (s != CIAR_OK) return s;
    if (!out) return CIAR_ERR_INVALID_ARG;
    if (desc->rows % params->window != 0) return CIAR_ERR_INVALID_ARG;
    if ((draft_row_max == nullptr) != (draft_sum_exp == nullptr)) return CIAR_ERR_INVALID_ARG;
    if (desc->rows == 0) return CIAR_OK;
    if (!draft_tokens || !u_accept || !u_resample) return CIAR_ERR_INVALID_ARG;
    if (params->mode != CIAR_VERIFY_ALL && !flag) return CIAR_ERR_INVALID_ARG;
    if (!ws) return CIAR_ERR_INVALID_ARG;
    if (((uintptr_t)ws & 15u) != 0) return CIAR_ERR_ALIGNMENT;
    const WsLayout l = ws_layout(desc->rows, params->window);
    if (ws_bytes < l.total) return CIAR_ERR_WORKSPACE_TOO_SMALL;

    char *w = reinterpret_cast<char *>(ws);
    VerifyArgs a;
    a.draft = draft_logits;
    a.target = target_logits;
    a.rows = desc->rows;
    a.row_stride = desc->row_stride;
    a.vocab = desc->vocab;
    a.vb = desc->valid_begin;
    a.n = desc->valid_count;
    a.rm.pos = nullptr;
    a.rm.seq_len = 0;
    a.rm.window = params->window;
    a.tokens = draft_tokens;
    a.flag = flag;
    a.draft_row_max = draft_row_max;
    a.draft_sum_exp = draft_sum_exp;
    a.u_accept = u_accept;
    a.u_resample = u_resample;
    a.window = params->window;
    a.mode = params->mode;
    a.out = *out;
    a.ws.window_done = reinterpret_cast<int32_t *>(w + l.window_done);
    a.ws.candidate = reinterpret_cast<int32_t *>(w + l.candidate);
    a.ws.accept = reinterpret_cast<uint8_t *>(w + l.accept);
    a.ws.tested = reinterpret_cast<int32_t *>(w + l.tested);
    a.ws.tq_max = reinterpret_cast<float *>(w + l.tq_max);
    a.ws.tq_sum = reinterpret_cast<float *>(w + l.tq_sum);
    cudaStream_t st = (cudaStream_t)stream;
    if (verify_stream_eligible(a, desc->dtype))
        return launch_verify_stream(a, desc->dtype, st) == cudaSuccess ? CIAR_OK : CIAR_ERR_CUDA;
    if (cudaMemsetAsync(a.ws.window_done, 0, (size_t)(desc->rows / params->window) * 4, st) != cudaSuccess)
        return CIAR_ERR_CUDA;
    return launch_verify(a, desc->dtype, st) == cudaSuccess ? CIAR_OK : CIAR_ERR_CUDA;
}

ciar_status ciar_decode_init(const ciar_decode_state *state, int32_t pos0, void *stream)
{
    if (!state || state->requests < 0 || state->seq_len < 1 || pos0 < 0 || pos0 > state->seq_len)
        return CIAR_ERR_INVALID_ARG;
    if (!state->counters || (state->requests > 0 && (!state->pos || !state->tokens_out))) return CIAR_ERR_INVALID_ARG;
    return launch_decode_init(*state, pos0, (cudaStream_t)stream) == cudaSuccess ? CIAR_OK : CIAR_ERR_CUDA;
}

ciar_status ciar_decode_step(const ciar_decode_state *state, const ciar_logits_desc *desc,
                             const void *draft_pool, const void *target_pool, const int32_t *draft_token_pool,
                             const float *u_accept_pool, const float *u_resample_pool,
                             const ciar_interval_params *params, const ciar_verify_params *vparams,
                             void *ws, size_t ws_bytes, void *stream)
{
    if (!state || state->requests < 0 || state->seq_len < 1) return CIAR_ERR_INVALID_ARG;
    if (!state->counters || (state->requests > 0 && (!state->pos || !state->tokens_out))) return CIAR_ERR_INVALID_ARG;
    ciar_status s = check_desc(desc, draft_pool);
    if (s != CIAR_OK) return s;
    s = check_desc(desc, target_pool);
    if (s != CIAR_OK) return s;
    s = check_interval(desc, params);
    if (s != CIAR_OK) return s;
    s = check_verify_params(vparams);
    if (s != CIAR_OK) return s;
    if (desc->rows != (int64_t)state->requests * state->seq_len) return CIAR_ERR_INVALID_ARG;
    if (state->requests == 0) return CIAR_OK;
    if (!draft_token_pool || !u_accept_pool || !u_resample_pool) return CIAR_ERR_INVALID_ARG;
    if (!ws) return CIAR_ERR_INVALID_ARG;
    if (((uintptr_t)ws & 15u) != 0) return CIAR_ERR_ALIGNMENT;
    const int32_t W = vparams->window;
    const int64_t step_rows = (int64_t)state->requests * W;
    const WsLayout l = ws_layout(step_rows, W);
    if (ws_bytes < l.total) return CIAR_ERR_WORKSPACE_TOO_SMALL;
    char *w = reinterpret_cast<char *>(ws);
    cudaStream_t st = (cudaStream_t)stream;

    uint8_t *flag = reinterpret_cast<uint8_t *>(w + l.flag);
    float *row_max = reinterpret_cast<float *>(w + l.row_max);
    float *sum_exp = reinterpret_cast<float *>(w + l.sum_exp);
    int32_t *first_flag = reinterpret_cast<int32_t *>(w + l.first_flag);
    int32_t *accepted_len = reinterpret_cast<int32_t *>(w + l.accepted_len);
    int32_t *resampled = reinterpret_cast<int32_t *>(w + l.resampled);

    QuantifyArgs qa;
    fill_quantify_args(qa, desc, draft_pool, params);
    qa.rows = step_rows;
    qa.rm.pos = state->pos;
    qa.rm.seq_len = state->seq_len;
    qa.rm.window = W;
    ciar_quantify_out qo = {};
    qo.row_max = row_max;
    qo.sum_exp = sum_exp;
    qo.flag = flag;
    qa.out = qo;
    if (launch_quantify(qa, desc->dtype, st) != cudaSuccess) return CIAR_ERR_CUDA;

    VerifyArgs va;
    va.draft = draft_pool;
    va.target = target_pool;
    va.rows = step_rows;
    va.row_stride = desc->row_stride;
    va.vocab = desc->vocab;
    va.vb = desc->valid_begin;
    va.n = desc->valid_count;
    va.rm = qa.rm;
    va.tokens = draft_token_pool;
    va.flag = flag;
    va.draft_row_max = row_max;
    va.draft_sum_exp = sum_exp;
    va.u_accept = u_accept_pool;
    va.u_resample = u_resample_pool;
    va.window = W;
    va.mode = vparams->mode;
    ciar_verify_out vo = {};
    vo.first_flag = first_flag;
    vo.accepted_len = accepted_len;
    vo.resampled_token = resampled;
    va.out = vo;
    va.ws.window_done = reinterpret_cast<int32_t *>(w + l.window_done);
    va.ws.candidate = reinterpret_cast<int32_t *>(w + l.candidate);
    va.ws.accept = reinterpret_cast<uint8_t *>(w + l.accept);
    va.ws.tested = reinterpret_cast<int32_t *>(w + l.tested);
    va.ws.tq_max = reinterpret_cast<float *>(w + l.tq_max);
    va.ws.tq_sum = reinterpret_cast<float *>(w + l.tq_sum);
    if (verify_stream_eligible(va, desc->dtype)) {
        if (launch_verify_stream(va, desc->dtype, st) != cudaSuccess) return CIAR_ERR_CUDA;
    } else {
        if (cudaMemsetAsync(va.ws.window_done, 0, (size_t)state->requests * 4, st) != cudaSuccess) return CIAR_ERR_CUDA;
        if (launch_verify(va, desc->dtype, st) != cudaSuccess) return CIAR_ERR_CUDA;
    }

    DecodeUpdateArgs ua;
    ua.st = *state;
    ua.window = W;
    ua.mode = vparams->mode;
    ua.tokens = draft_token_pool;
    ua.flag = flag;
    ua.first_flag = first_flag;
    ua.accepted_len = accepted_len;
    ua.resampled_token = resampled;
    return launch_decode_update(ua, st) == cudaSuccess ? CIAR_OK : CIAR_ERR_CUDA;
}

ciar_status ciar_quantify_topk(const ciar_logits_desc *desc, const void *draft_logits, int32_t k,
                               const ciar_interval_params *params, const ciar_topk_out *out, void *stream)
{
    ciar_status st = check_desc(desc, draft_logits);
    if (st != CIAR_OK) return st;
    st = check_interval(desc, params);
    if (st != CIAR_OK) return st;
    if (!out) return CIAR_ERR_INVALID_ARG;
    if (k < 1 || k > desc->valid_count) return CIAR_ERR_INVALID_ARG;
    if (params->radius_mode == CIAR_RADIUS_PER_CODE) return CIAR_ERR_UNSUPPORTED;
    if (desc->rows == 0) return CIAR_OK;
    TopkArgs a;
    a.logits = draft_logits;
    a.rows = desc->rows;
    a.row_stride = desc->row_stride;
    a.vb = desc->valid_begin;
    a.n = desc->valid_count;
    a.k = k;
    a.radius_mode = params->radius_mode;
    a.radius_is_raw = params->radius_is_raw;
    a.radius = params->radius;
    a.r_scalar = params->r_scalar;
    a.r_max = params->r_max;
    a.lo_cap = params->lo_cap;
    a.hi_cap = params->hi_cap;
    a.tau = params->tau;
    a.out = *out;
    return launch_topk(a, desc->dtype, (cudaStream_t)stream) == cudaSuccess ? CIAR_OK : CIAR_ERR_CUDA;
}

ciar_status ciar_rescore(int64_t rows, int32_t n, const float *omega, const float *sigma,
                         const ciar_score_params *params, float *score_out, uint8_t *flag_out, void *stream)
{
    if (!params || rows < 0 || n < 1) return CIAR_ERR_INVALID_ARG;
    if (params->variant < CIAR_SCORE_PRODUCT || params->variant > CIAR_SCORE_ADDITIVE) return CIAR_ERR_INVALID_ARG;
    if (params->tau != params->tau) return CIAR_ERR_INVALID_ARG;
    if (rows > 0 && (!omega || !sigma)) return CIAR_ERR_INVALID_ARG;
    return launch_rescore(rows, n, omega, sigma, *params, score_out, flag_out, (cudaStream_t)stream) == cudaSuccess
               ? CIAR_OK : CIAR_ERR_CUDA;
}

ciar_status ciar_vote(int32_t n_heads, int64_t rows, const uint8_t *flags, uint8_t *flag_out,
                      int32_t *votes_out, void *stream)
{
    if (n_heads < 1 || n_heads > CIAR_MAX_HEADS || rows < 0) return CIAR_ERR_INVALID_ARG;
    if (rows > 0 && !flags) return CIAR_ERR_INVALID_ARG;
    return launch_vote(n_heads, rows, flags, flag_out, votes_out, (cudaStream_t)stream) == cudaSuccess
               ? CIAR_OK : CIAR_ERR_CUDA;
}

ciar_status ciar_quantify_ensemble(const ciar_logits_desc *desc, const void *head_logits, int32_t n_heads,
                                   int64_t head_stride, const ciar_interval_params *params,
                                   const ciar_quantify_out *out, void *stream)
{
    ciar_status st = check_desc(desc, head_logits);
    if (st != CIAR_OK) return st;
    st = check_interval(desc, params);
    if (st != CIAR_OK) return st;
    if (!out) return CIAR_ERR_INVALID_ARG;
    if (n_heads < 1 || n_heads > CIAR_MAX_HEADS) return CIAR_ERR_INVALID_ARG;
    if (params->radius_mode == CIAR_RADIUS_PER_CODE) return CIAR_ERR_UNSUPPORTED;
    if (n_heads > 1 && head_stride < desc->rows * desc->row_stride) return CIAR_ERR_INVALID_ARG;
    if ((head_stride * elem_size(desc->dtype)) % 16 != 0) return CIAR_ERR_ALIGNMENT;
    if (out->row_max || out->sum_exp || out->lse || out->argmax || out->dense_lo || out->dense_up) return CIAR_ERR_INVALID_ARG;
    if (desc->rows == 0) return CIAR_OK;
    EnsembleArgs a;
    a.heads = head_logits;
    a.n_heads = n_heads;
    a.head_stride = head_stride;
    a.rows = desc->rows;
    a.row_stride = desc->row_stride;
    a.vb = desc->valid_begin;
    a.n = desc->valid_count;
    a.radius_mode = params->radius_mode;
    a.radius_is_raw = params->radius_is_raw;
    a.radius = reinterpret_cast<const float *>(params->radius);
    a.r_scalar = params->r_scalar;
    a.r_max = params->r_max;
    a.lo_cap = params->lo_cap;
    a.hi_cap = params->hi_cap;
    a.tau = params->tau;
    a.out = *out;
    return launch_ensemble(a, desc->dtype, (cudaStream_t)stream) == cudaSuccess ? CIAR_OK : CIAR_ERR_CUDA;
}

size_t ciar_interdro_workspace_bytes(int64_t rows) { return rows < 0 ? 0 : (size_t)rows * 7 * sizeof(double); }

ciar_status ciar_interdro_forward(const ciar_logits_desc *desc, const void *center, const void *radius,
                                  const void *cloud, const ciar_interdro_params *params,
                                  const ciar_interdro_out *out, void *workspace, size_t workspace_bytes,
                                  void *stream)
{
    ciar_status st = check_desc(desc, center);
    if (st != CIAR_OK) return st;
    if ((st = check_desc(desc, radius)) != CIAR_OK) return st;
    if ((st = check_desc(desc, cloud)) != CIAR_OK) return st;
    if (!params || !out || desc->rows < 1) return CIAR_ERR_INVALID_ARG;
    if (!(params->r_max > 0.f) || !(params->r_max <= 80.f)) return CIAR_ERR_INVALID_ARG;
    if (!workspace || ((uintptr_t)workspace & 15u) != 0) return workspace ? CIAR_ERR_ALIGNMENT : CIAR_ERR_INVALID_ARG;
    if (workspace_bytes < ciar_interdro_workspace_bytes(desc->rows)) return CIAR_ERR_WORKSPACE_TOO_SMALL;
    InterDroArgs a;
    a.center = center;
    a.radius = radius;
    a.cloud = cloud;
    a.rows = desc->rows;
    a.row_stride = desc->row_stride;
    a.vb = desc->valid_begin;
    a.n = desc->valid_count;
    a.prm = *params;
    a.out = *out;
    a.ws = reinterpret_cast<double *>(workspace);
    return launch_interdro(a, desc->dtype, (cudaStream_t)stream) == cudaSuccess ? CIAR_OK : CIAR_ERR_CUDA;
}

}  // extern "C"
