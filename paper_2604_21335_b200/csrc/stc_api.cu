// C-ABI of libstc: host-side argument validation and dispatch.  Nothing here
// allocates device memory; every launch goes to the caller's stream.
#include <nvtx3/nvToolsExt.h>

#include "common.cuh"

using namespace stc;

namespace {

int32_t make_geom(const stc_shape* s, Geom* g) {
    if (!s) return STC_ERR_INVALID_ARG;
    if (s->batch < 0 || s->n_q_heads <= 0 || s->n_kv_heads <= 0 || s->t_cap < 0 || s->reserved != 0)
        return STC_ERR_INVALID_ARG;
    if (s->n_q_heads % s->n_kv_heads != 0) return STC_ERR_INVALID_ARG;
    if (s->head_dim != kHeadDim || s->page_size != kPage) return STC_ERR_UNSUPPORTED;
    if (s->n_groups != 4 && s->n_groups != 8 && s->n_groups != 16) return STC_ERR_UNSUPPORTED;
    if (s->n_q_heads / s->n_kv_heads > 8) return STC_ERR_UNSUPPORTED;
    if ((int64_t)s->t_cap * 16 >= (int64_t)1 << 31) return STC_ERR_UNSUPPORTED;   // u32 offsets
    if ((int64_t)s->batch * s->n_kv_heads >= (int64_t)1 << 24) return STC_ERR_UNSUPPORTED;
    g->B = s->batch; g->Hq = s->n_q_heads; g->Hkv = s->n_kv_heads; g->Gq = g->Hq / g->Hkv;
    g->S = s->n_groups; g->g = kHeadDim / g->S; g->T = s->t_cap; g->P = (g->T + kPage - 1) / kPage;
    g->problems = g->B * g->Hkv;
    g->seq_len = s->seq_len;
    return STC_OK;
}

bool empty(const Geom& g) { return g.problems == 0 || g.T == 0; }

int32_t check_ws(const void* ws, size_t have, size_t need) {
    if (need == 0) return STC_OK;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255u) != 0 || have < need) return STC_ERR_WORKSPACE;
    return STC_OK;
}

int32_t cuda_rc(cudaError_t e) { return e == cudaSuccess ? STC_OK : STC_ERR_CUDA; }

// NVTX range around the host side of a call (what it enqueues shows under it in a timeline).
struct Range {
    explicit Range(const char* name) { nvtxRangePushA(name); }
    ~Range() { nvtxRangePop(); }
};

}  // namespace

namespace {
// The kernels move keys, values, queries, page metadata and scores in 16-byte pieces.
template <typename... P>
bool aligned16(P... p) { return ((reinterpret_cast<uintptr_t>(p) | ...) & 15u) == 0; }
}  // namespace

extern "C" {

const char* stc_status_string(int32_t status) {
    switch (status) {
        case STC_OK: return "ok";
        case STC_ERR_INVALID_ARG: return "invalid argument";
        case STC_ERR_UNSUPPORTED: return "unsupported shape";
        case STC_ERR_WORKSPACE: return "workspace missing, misaligned or too small";
        case STC_ERR_CAPACITY: return "packed value store too small";
        case STC_ERR_BUDGET: return "group budget below one group per routed token";
        case STC_ERR_CUDA: return "CUDA runtime error";
        case STC_ERR_TIMEOUT: return "timeout";
        case STC_ERR_SCRATCH_LIMIT: return "shape needs more than the built-in scratch array";
        default: return "unknown status";
    }
}

int32_t stc_version(void) { return 100; }

int32_t stc_workspace_bytes(const stc_shape* shape, int32_t op, int64_t arg, size_t* bytes_host) {
    Geom g;
    int32_t rc = make_geom(shape, &g);
    if (rc != STC_OK) return rc;
    if (!bytes_host) return STC_ERR_INVALID_ARG;
    if (empty(g)) { *bytes_host = 0; return STC_OK; }
    switch (op) {
        case STC_OP_QUEST_SELECT: *bytes_host = select_ws_bytes(g); break;
        case STC_OP_ROUTE_PACK: *bytes_host = route_ws_bytes(g); break;
        case STC_OP_DECODE_ATTN:
            if (arg < 0 || arg > g.P) return STC_ERR_INVALID_ARG;
            *bytes_host = attn_ws_bytes(g, (int)arg);
            break;
        default: return STC_ERR_INVALID_ARG;
    }
    return STC_OK;
}

int32_t stc_build_page_meta(const stc_shape* shape, const stc_cache* cache, int32_t page_begin,
                            int32_t page_end, void* stream) {
    Range nvtx_range("stc_build_page_meta");
    Geom g;
    int32_t rc = make_geom(shape, &g);
    if (rc != STC_OK) return rc;
    if (!cache) return STC_ERR_INVALID_ARG;
    if (empty(g)) return STC_OK;
    if (!cache->k || !cache->kmin || !cache->kmax || page_begin < 0) return STC_ERR_INVALID_ARG;
    if (!aligned16(cache->k, cache->kmin, cache->kmax)) return STC_ERR_INVALID_ARG;
    return cuda_rc(launch_page_meta(g, cache->k, cache->kmin, cache->kmax, page_begin, page_end,
                                    static_cast<cudaStream_t>(stream)));
}

int32_t stc_quest_select(const stc_shape* shape, const stc_cache* cache, const void* q,
                         int32_t token_budget, int32_t max_pages, int32_t* page_ids,
                         int32_t* n_pages, float* scores_opt, void* ws, size_t ws_bytes,
                         void* stream) {
    return stc_quest_select_window(shape, cache, q, token_budget, 0, max_pages, page_ids, n_pages, scores_opt, ws,
                                   ws_bytes, stream);
}

int32_t stc_quest_select_window(const stc_shape* shape, const stc_cache* cache, const void* q,
                                int32_t token_budget, int32_t n_recent_pages, int32_t max_pages,
                                int32_t* page_ids, int32_t* n_pages, float* scores_opt, void* ws,
                                size_t ws_bytes, void* stream) {
    Range nvtx_range("stc_quest_select_window");
    Geom g;
    int32_t rc = make_geom(shape, &g);
    if (rc != STC_OK) return rc;
    if (!cache || token_budget < 0 || max_pages < 0 || n_recent_pages < 0) return STC_ERR_INVALID_ARG;
    if (empty(g)) return STC_OK;
    if (!cache->kmin || !cache->kmax || !q || !page_ids || !n_pages) return STC_ERR_INVALID_ARG;
    if (!aligned16(cache->kmin, cache->kmax, q)) return STC_ERR_INVALID_ARG;
    const int want = token_budget / kPage < g.P ? token_budget / kPage : g.P;
    if (max_pages < want) return STC_ERR_INVALID_ARG;
    rc = check_ws(ws, ws_bytes, select_ws_bytes(g));
    if (rc != STC_OK) return rc;
    return cuda_rc(launch_quest_select(g, cache->kmin, cache->kmax, q, token_budget, n_recent_pages, max_pages,
                                       page_ids, n_pages, scores_opt, ws,
                                       static_cast<cudaStream_t>(stream)));
}

int32_t stc_pages_to_class(const stc_shape* shape, const int32_t* page_ids, const int32_t* n_pages,
                           int32_t max_pages, uint8_t* tok_class, void* stream) {
    Range nvtx_range("stc_pages_to_class");
    Geom g;
    int32_t rc = make_geom(shape, &g);
    if (rc != STC_OK) return rc;
    if (max_pages < 0) return STC_ERR_INVALID_ARG;
    if (empty(g)) return STC_OK;
    if (!tok_class || (max_pages > 0 && (!page_ids || !n_pages))) return STC_ERR_INVALID_ARG;
    return cuda_rc(launch_pages_to_class(g, page_ids, n_pages, max_pages, tok_class,
                                         static_cast<cudaStream_t>(stream)));
}

namespace {
int32_t route_pack_phases(const stc_shape* shape, const void* v, const float* scores,
                          const uint8_t* tok_class, int64_t class_head_stride, int32_t k_nominal,
                          int32_t min_per_token, int32_t mode, const stc_cache* out,
                          int64_t* total_groups, int32_t* status, void* ws, size_t ws_bytes, int phases,
                          void* stream) {
    Geom g;
    int32_t rc = make_geom(shape, &g);
    if (rc != STC_OK) return rc;
    if (!out || k_nominal < 0 || k_nominal > g.S || (min_per_token != 0 && min_per_token != 1) ||
        (mode != STC_MODE_GLOBAL && mode != STC_MODE_PER_TOKEN))
        return STC_ERR_INVALID_ARG;
    if (class_head_stride != 0 && class_head_stride != g.T) return STC_ERR_INVALID_ARG;
    if (empty(g)) return STC_OK;
    if (!out->v_mask) return STC_ERR_INVALID_ARG;
    if ((phases & 1) && (!scores || !aligned16(scores))) return STC_ERR_INVALID_ARG;
    if ((phases & 2) && !aligned16(v, out->v_packed)) return STC_ERR_INVALID_ARG;
    if ((phases & 2) && (!v || !out->v_packed || !out->v_offs || !total_groups || !status || out->cap_groups < 0))
        return STC_ERR_INVALID_ARG;
    rc = check_ws(ws, ws_bytes, route_ws_bytes(g));
    if (rc != STC_OK) return rc;
    return cuda_rc(launch_route_pack(g, v, scores, tok_class, class_head_stride, k_nominal,
                                     min_per_token, mode, out->v_packed, out->v_mask, out->v_offs,
                                     out->cap_groups, total_groups, status, ws, phases,
                                     static_cast<cudaStream_t>(stream)));
}
}  // namespace

int32_t stc_route_pack(const stc_shape* shape, const void* v, const float* scores,
                       const uint8_t* tok_class, int64_t class_head_stride, int32_t k_nominal,
                       int32_t min_per_token, int32_t mode, const stc_cache* out,
                       int64_t* total_groups, int32_t* status, void* ws, size_t ws_bytes,
                       void* stream) {
    Range nvtx_range("stc_route_pack");
    return route_pack_phases(shape, v, scores, tok_class, class_head_stride, k_nominal, min_per_token, mode,
                             out, total_groups, status, ws, ws_bytes, 3, stream);
}

int32_t stc_route_mask(const stc_shape* shape, const float* scores, const uint8_t* tok_class,
                       int64_t class_head_stride, int32_t k_nominal, int32_t min_per_token, int32_t mode,
                       const stc_cache* out, void* ws, size_t ws_bytes, void* stream) {
    Range nvtx_range("stc_route_mask");
    return route_pack_phases(shape, nullptr, scores, tok_class, class_head_stride, k_nominal, min_per_token,
                             mode, out, nullptr, nullptr, ws, ws_bytes, 1, stream);
}

int32_t stc_pack_values(const stc_shape* shape, const void* v, int32_t mode, const stc_cache* out,
                        int64_t* total_groups, int32_t* status, void* ws, size_t ws_bytes, void* stream) {
    Range nvtx_range("stc_pack_values");
    return route_pack_phases(shape, v, nullptr, nullptr, 0, 0, 0, mode, out, total_groups, status, ws,
                             ws_bytes, 2, stream);
}

int32_t stc_router_logits(const stc_shape* shape, const void* h, const void* w, const float* bias_opt,
                          int32_t d_model, float* scores, int32_t* status_word, void* stream) {
    Range nvtx_range("stc_router_logits");
    Geom g;
    int32_t rc = make_geom(shape, &g);
    if (rc != STC_OK) return rc;
    if (d_model <= 0) return STC_ERR_INVALID_ARG;
    const int n = g.Hkv * g.S;
    if (d_model % 64 != 0 || n % 16 != 0 || (n > 256 && n % 256 != 0)) return STC_ERR_UNSUPPORTED;
    if (empty(g)) return STC_OK;
    if (!h || !w || !scores || !status_word) return STC_ERR_INVALID_ARG;
    if (((reinterpret_cast<uintptr_t>(h) | reinterpret_cast<uintptr_t>(w) | reinterpret_cast<uintptr_t>(scores) |
          reinterpret_cast<uintptr_t>(bias_opt)) & 15u) != 0)
        return STC_ERR_INVALID_ARG;
    return cuda_rc(launch_router_logits(g, h, w, bias_opt, d_model, scores, status_word,
                                        static_cast<cudaStream_t>(stream)));
}

int32_t stc_query_bias(int32_t batch, int32_t q_cap, int32_t d_model, int32_t n_logits, const void* h_q,
                       const int32_t* q_len_opt, const void* w_q, float* s_q, float* bias, void* stream) {
    Range nvtx_range("stc_query_bias");
    if (batch < 0 || q_cap < 0 || d_model <= 0 || n_logits < 0 || batch > 65535) return STC_ERR_INVALID_ARG;
    if (d_model % 8 != 0) return STC_ERR_UNSUPPORTED;
    if (batch == 0) return STC_OK;
    if (!s_q || (n_logits > 0 && (!w_q || !bias)) || (q_cap > 0 && !h_q)) return STC_ERR_INVALID_ARG;
    if (((reinterpret_cast<uintptr_t>(h_q) | reinterpret_cast<uintptr_t>(w_q) | reinterpret_cast<uintptr_t>(s_q)) & 15u) != 0)
        return STC_ERR_INVALID_ARG;
    return cuda_rc(launch_query_bias(batch, q_cap, d_model, n_logits, h_q, q_len_opt, w_q, s_q, bias,
                                     static_cast<cudaStream_t>(stream)));
}

int32_t stc_append_tokens(const stc_shape* shape, const stc_cache* cache, const void* v,
                          const int32_t* old_len, int32_t max_new, int64_t* total_groups, int32_t* status,
                          void* stream) {
    Range nvtx_range("stc_append_tokens");
    Geom g;
    int32_t rc = make_geom(shape, &g);
    if (rc != STC_OK) return rc;
    if (!cache || max_new < 0) return STC_ERR_INVALID_ARG;
    if (empty(g) || max_new == 0) return STC_OK;
    if (!cache->k || !cache->kmin || !cache->kmax || !cache->v_packed || !cache->v_mask || !cache->v_offs ||
        cache->cap_groups < 0 || !v || !old_len || !total_groups || !status)
        return STC_ERR_INVALID_ARG;
    if (!aligned16(cache->k, cache->kmin, cache->kmax, cache->v_packed, v)) return STC_ERR_INVALID_ARG;
    return cuda_rc(launch_append(g, cache->k, cache->kmin, cache->kmax, v, old_len, max_new, cache->v_packed,
                                 cache->v_mask, cache->v_offs, cache->cap_groups, total_groups, status,
                                 static_cast<cudaStream_t>(stream)));
}

int32_t stc_route_new_pages(const stc_shape* shape, const stc_cache* cache, const float* scores,
                            const int32_t* first_page, int32_t k_nominal, int32_t min_per_token,
                            int32_t mode, int64_t* total_groups, int32_t* status, void* stream) {
    Range nvtx_range("stc_route_new_pages");
    Geom g;
    int32_t rc = make_geom(shape, &g);
    if (rc != STC_OK) return rc;
    if (!cache || k_nominal < 0 || k_nominal > g.S || (min_per_token != 0 && min_per_token != 1) ||
        (mode != STC_MODE_GLOBAL && mode != STC_MODE_PER_TOKEN))
        return STC_ERR_INVALID_ARG;
    if (empty(g)) return STC_OK;
    if (!cache->v_packed || !cache->v_mask || !cache->v_offs || cache->cap_groups < 0 || !scores || !first_page ||
        !total_groups || !status)
        return STC_ERR_INVALID_ARG;
    if (!aligned16(cache->v_packed, scores)) return STC_ERR_INVALID_ARG;
    return cuda_rc(launch_route_new_pages(g, scores, first_page, k_nominal, min_per_token, mode, cache->v_packed,
                                          cache->v_mask, cache->v_offs, cache->cap_groups, total_groups, status,
                                          static_cast<cudaStream_t>(stream)));
}

int32_t stc_decode_attn(const stc_shape* shape, const stc_cache* cache, const void* q,
                        const int32_t* page_ids, const int32_t* n_pages, int32_t max_pages,
                        float sm_scale, float* out, float* lse_opt, void* ws, size_t ws_bytes,
                        void* stream) {
    Range nvtx_range("stc_decode_attn");
    Geom g;
    int32_t rc = make_geom(shape, &g);
    if (rc != STC_OK) return rc;
    if (!cache || max_pages < 0 || !(sm_scale == sm_scale)) return STC_ERR_INVALID_ARG;
    if (g.problems == 0) return STC_OK;
    if (!q || !out) return STC_ERR_INVALID_ARG;
    if (page_ids && !n_pages) return STC_ERR_INVALID_ARG;
    if (!page_ids) max_pages = g.P;
    if (max_pages > g.P && !page_ids) return STC_ERR_INVALID_ARG;
    if (g.T > 0 && (!cache->k || !cache->v_packed || !cache->v_mask || !cache->v_offs || cache->cap_groups < 0))
        return STC_ERR_INVALID_ARG;
    if (!aligned16(cache->k, cache->v_packed, q, out)) return STC_ERR_INVALID_ARG;
    rc = check_ws(ws, ws_bytes, attn_ws_bytes(g, max_pages));
    if (rc != STC_OK) return rc;
    return cuda_rc(launch_decode_attn(g, cache->k, cache->v_packed, cache->v_mask, cache->v_offs,
                                      cache->cap_groups, q, page_ids, n_pages, max_pages, sm_scale,
                                      out, lse_opt, ws, static_cast<cudaStream_t>(stream)));
}

int32_t stc_decode_step(const stc_shape* shape, const stc_cache* cache, const void* q, int32_t token_budget,
                        int32_t max_pages, int32_t* page_ids, int32_t* n_pages, float sm_scale, float* out,
                        float* lse_opt, void* ws_select, size_t ws_select_bytes, void* ws_attn,
                        size_t ws_attn_bytes, void* stream) {
    Range nvtx_range("stc_decode_step");
    Geom g;
    int32_t rc = make_geom(shape, &g);
    if (rc != STC_OK) return rc;
    if (!cache || token_budget < 0 || max_pages < 0 || !(sm_scale == sm_scale)) return STC_ERR_INVALID_ARG;
    if (g.problems == 0) return STC_OK;
    if (!q || !out || !page_ids || !n_pages) return STC_ERR_INVALID_ARG;
    if (g.T == 0 || max_pages < 1) {              // nothing to select or attend: the two plain calls handle it
        rc = stc_quest_select(shape, cache, q, token_budget, max_pages, page_ids, n_pages, nullptr, ws_select,
                              ws_select_bytes, stream);
        if (rc != STC_OK) return rc;
        return stc_decode_attn(shape, cache, q, page_ids, n_pages, max_pages, sm_scale, out, lse_opt, ws_attn,
                               ws_attn_bytes, stream);
    }
    if (!cache->kmin || !cache->kmax || !cache->k || !cache->v_packed || !cache->v_mask || !cache->v_offs ||
        cache->cap_groups < 0)
        return STC_ERR_INVALID_ARG;
    if (!aligned16(cache->k, cache->v_packed, cache->kmin, cache->kmax, q, out)) return STC_ERR_INVALID_ARG;
    const int want = token_budget / kPage < g.P ? token_budget / kPage : g.P;
    if (max_pages < want || max_pages > g.P) return STC_ERR_INVALID_ARG;
    rc = check_ws(ws_select, ws_select_bytes, select_ws_bytes(g));
    if (rc == STC_OK) rc = check_ws(ws_attn, ws_attn_bytes, attn_ws_bytes(g, max_pages));
    if (rc != STC_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // both workspaces are cleared first, so that nothing stands between the two kernels
    cudaError_t e = clear_two(ws_select, quest_select_clear_bytes(g), ws_attn, decode_attn_clear_bytes(g), st);
    if (e == cudaSuccess)
        e = launch_quest_select(g, cache->kmin, cache->kmax, q, token_budget, 0, max_pages, page_ids, n_pages,
                                nullptr, ws_select, st, kLaunchNoClear);
    if (e == cudaSuccess)
        e = launch_decode_attn(g, cache->k, cache->v_packed, cache->v_mask, cache->v_offs, cache->cap_groups, q,
                               page_ids, n_pages, max_pages, sm_scale, out, lse_opt, ws_attn, st,
                               kLaunchNoClear);
    return cuda_rc(e);
}

int32_t stc_cache_bytes(int64_t n_tokens_retained, int64_t n_groups_kept, int32_t n_groups,
                        int64_t* kv_bytes_host, int64_t* index_bytes_host) {
    if (n_tokens_retained < 0 || n_groups_kept < 0 || !kv_bytes_host) return STC_ERR_INVALID_ARG;
    if (n_groups != 4 && n_groups != 8 && n_groups != 16) return STC_ERR_UNSUPPORTED;
    *kv_bytes_host = n_tokens_retained * kRowBytes + n_groups_kept * (kHeadDim / n_groups) * 2;
    if (index_bytes_host) {
        const int64_t pages = (n_tokens_retained + kPage - 1) / kPage;
        *index_bytes_host = n_tokens_retained * 2 + (n_tokens_retained + 1) * 4 + pages * 2 * kRowBytes;
    }
    return STC_OK;
}

}  // extern "C"

namespace {

struct Arena {
    char *k, *v, *scores, *cls, *q, *kmin, *kmax, *packed, *mask, *offs, *ids, *npages, *out, *total,
        *status, *ws;
    size_t ws_bytes, total_bytes;
    int max_pages;
};

size_t up256(size_t x) { return (x + 255) & ~(size_t)255; }

Arena carve_arena(const Geom& g, int64_t cap_groups, int token_budget, void* base) {
    Arena a;
    char* p = static_cast<char*>(base);
    size_t o = 0;
    auto take = [&](size_t bytes) { char* r = p + o; o += up256(bytes); return r; };
    const size_t rows = (size_t)g.problems * g.T;
    a.max_pages = token_budget < 0 ? g.P : (token_budget / kPage < g.P ? token_budget / kPage : g.P);
    if (a.max_pages < 1) a.max_pages = 1;
    a.k = take(rows * kRowBytes);
    a.v = take(rows * kRowBytes);
    a.scores = take(rows * g.S * 4);
    a.cls = take((size_t)g.B * g.T);
    a.q = take((size_t)g.B * g.Hq * kRowBytes);
    a.kmin = take((size_t)g.problems * g.P * kRowBytes);
    a.kmax = take((size_t)g.problems * g.P * kRowBytes);
    a.packed = take((size_t)g.problems * cap_groups * g.g * 2);
    a.mask = take(rows * 2);
    a.offs = take((size_t)g.problems * (g.T + 1) * 4);
    a.ids = take((size_t)g.problems * a.max_pages * 4);
    a.npages = take((size_t)g.problems * 4);
    a.out = take((size_t)g.B * g.Hq * kHeadDim * 4);
    a.total = take((size_t)g.problems * 8);
    a.status = take((size_t)g.problems * 4);
    size_t w = select_ws_bytes(g);
    if (route_ws_bytes(g) > w) w = route_ws_bytes(g);
    if (attn_ws_bytes(g, a.max_pages) > w) w = attn_ws_bytes(g, a.max_pages);
    a.ws_bytes = up256(w);
    a.ws = take(a.ws_bytes);
    a.total_bytes = o;
    return a;
}

}  // namespace

extern "C" {

int32_t stc_pass_host_arena_bytes(const stc_shape* shape, int64_t cap_groups, int32_t token_budget,
                                  size_t* bytes_host) {
    Geom g;
    int32_t rc = make_geom(shape, &g);
    if (rc != STC_OK) return rc;
    if (!bytes_host || cap_groups < 0) return STC_ERR_INVALID_ARG;
    *bytes_host = empty(g) ? 0 : carve_arena(g, cap_groups, token_budget, nullptr).total_bytes;
    return STC_OK;
}

int32_t stc_pass_host(const stc_shape* shape, const void* k_host, const void* v_host,
                      const float* scores_host, const uint8_t* tok_class_host, const void* q_host,
                      int32_t token_budget, int32_t k_nominal, int32_t min_per_token, int32_t mode,
                      float sm_scale, int64_t cap_groups, void* arena, size_t arena_bytes,
                      float* out_host, int64_t* total_groups_host, int32_t* status_host,
                      void* stream) {
    Range nvtx_range("stc_pass_host");
    Geom g;
    int32_t rc = make_geom(shape, &g);
    if (rc != STC_OK) return rc;
    if (cap_groups < 0 || !k_host || !v_host || !scores_host || !q_host || !out_host ||
        !total_groups_host || !status_host)
        return STC_ERR_INVALID_ARG;
    if (empty(g)) return STC_OK;
    const Arena a = carve_arena(g, cap_groups, token_budget, arena);
    rc = check_ws(arena, arena_bytes, a.total_bytes);
    if (rc != STC_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t rows = (size_t)g.problems * g.T;
    cudaError_t e = cudaMemcpyAsync(a.k, k_host, rows * kRowBytes, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(a.v, v_host, rows * kRowBytes, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(a.scores, scores_host, rows * g.S * 4, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess && tok_class_host)
        e = cudaMemcpyAsync(a.cls, tok_class_host, (size_t)g.B * g.T, cudaMemcpyHostToDevice, st);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(a.q, q_host, (size_t)g.B * g.Hq * kRowBytes, cudaMemcpyHostToDevice, st);
    if (e != cudaSuccess) return STC_ERR_CUDA;

    stc_cache c;
    c.k = a.k; c.kmin = a.kmin; c.kmax = a.kmax; c.v_packed = a.packed;
    c.v_mask = reinterpret_cast<uint16_t*>(a.mask);
    c.v_offs = reinterpret_cast<uint32_t*>(a.offs);
    c.cap_groups = cap_groups;
    rc = stc_build_page_meta(shape, &c, 0, -1, stream);
    if (rc != STC_OK) return rc;
    rc = stc_route_pack(shape, a.v, reinterpret_cast<const float*>(a.scores),
                        tok_class_host ? reinterpret_cast<const uint8_t*>(a.cls) : nullptr, 0, k_nominal,
                        min_per_token, mode, &c, reinterpret_cast<int64_t*>(a.total),
                        reinterpret_cast<int32_t*>(a.status), a.ws, a.ws_bytes, stream);
    if (rc != STC_OK) return rc;
    const int32_t* ids = nullptr;
    if (token_budget >= 0) {
        rc = stc_quest_select(shape, &c, a.q, token_budget, a.max_pages, reinterpret_cast<int32_t*>(a.ids),
                              reinterpret_cast<int32_t*>(a.npages), nullptr, a.ws, a.ws_bytes, stream);
        if (rc != STC_OK) return rc;
        ids = reinterpret_cast<const int32_t*>(a.ids);
    }
    rc = stc_decode_attn(shape, &c, a.q, ids, reinterpret_cast<const int32_t*>(a.npages), a.max_pages,
                         sm_scale, reinterpret_cast<float*>(a.out), nullptr, a.ws, a.ws_bytes, stream);
    if (rc != STC_OK) return rc;
    e = cudaMemcpyAsync(out_host, a.out, (size_t)g.B * g.Hq * kHeadDim * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(total_groups_host, a.total, (size_t)g.problems * 8, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess)
        e = cudaMemcpyAsync(status_host, a.status, (size_t)g.problems * 4, cudaMemcpyDeviceToHost, st);
    return cuda_rc(e);
}


namespace {
struct StepArena { char *q, *ids, *npages, *out, *ws; size_t ws_bytes, total_bytes; int max_pages; };
StepArena carve_step_arena(const Geom& g, int token_budget, void* base) {
    StepArena a;
    char* p = static_cast<char*>(base);
    size_t o = 0;
    auto take = [&](size_t bytes) { char* r = p + o; o += up256(bytes); return r; };
    a.max_pages = token_budget < 0 ? g.P : (token_budget / kPage < g.P ? token_budget / kPage : g.P);
    if (a.max_pages < 1) a.max_pages = 1;
    a.q = take((size_t)g.B * g.Hq * kRowBytes);
    a.ids = take((size_t)g.problems * a.max_pages * 4);
    a.npages = take((size_t)g.problems * 4);
    a.out = take((size_t)g.B * g.Hq * kHeadDim * 4);
    // selection and attention keep separate workspaces: the attention status word must survive
    const size_t ws_sel = up256(select_ws_bytes(g)), ws_att = up256(attn_ws_bytes(g, a.max_pages));
    a.ws_bytes = ws_att;
    a.ws = take(ws_att);
    take(ws_sel);
    a.total_bytes = o;
    return a;
}
}  // namespace

int32_t stc_decode_step_host_arena_bytes(const stc_shape* shape, int32_t token_budget, size_t* bytes_host) {
    Geom g;
    int32_t rc = make_geom(shape, &g);
    if (rc != STC_OK) return rc;
    if (!bytes_host) return STC_ERR_INVALID_ARG;
    *bytes_host = empty(g) ? 0 : carve_step_arena(g, token_budget, nullptr).total_bytes;
    return STC_OK;
}

int32_t stc_decode_step_host(const stc_shape* shape, const stc_cache* cache, const void* q_host,
                             int32_t token_budget, float sm_scale, void* arena, size_t arena_bytes,
                             float* out_host, int32_t* status_host, void* stream) {
    Range nvtx_range("stc_decode_step_host");
    Geom g;
    int32_t rc = make_geom(shape, &g);
    if (rc != STC_OK) return rc;
    if (!cache || !q_host || !out_host || !status_host) return STC_ERR_INVALID_ARG;
    if (empty(g)) return STC_OK;
    const StepArena a = carve_step_arena(g, token_budget, arena);
    rc = check_ws(arena, arena_bytes, a.total_bytes);
    if (rc != STC_OK) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (cudaMemcpyAsync(a.q, q_host, (size_t)g.B * g.Hq * kRowBytes, cudaMemcpyHostToDevice, st) != cudaSuccess)
        return STC_ERR_CUDA;
    if (token_budget >= 0) {
        rc = stc_decode_step(shape, cache, a.q, token_budget, a.max_pages, reinterpret_cast<int32_t*>(a.ids),
                             reinterpret_cast<int32_t*>(a.npages), sm_scale, reinterpret_cast<float*>(a.out), nullptr,
                             a.ws + a.ws_bytes, up256(select_ws_bytes(g)), a.ws, a.ws_bytes, stream);
    } else {
        rc = stc_decode_attn(shape, cache, a.q, nullptr, nullptr, a.max_pages, sm_scale,
                             reinterpret_cast<float*>(a.out), nullptr, a.ws, a.ws_bytes, stream);
    }
    if (rc != STC_OK) return rc;
    cudaError_t e = cudaMemcpyAsync(out_host, a.out, (size_t)g.B * g.Hq * kHeadDim * 4, cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemcpyAsync(status_host, a.ws, 4, cudaMemcpyDeviceToHost, st);
    return cuda_rc(e);
}

}  // extern "C"
