/*
 * stc -- decode attention over a two-level compressed KV cache on B200 (sm_100a).
 *
 * Level 1 keeps whole tokens: Quest-style page selection scores every 16-token
 * page of keys by a per-channel min/max bound against the query and keeps the
 * best pages up to a token budget (the paper's Stage I for LLMs, Section 3.2).
 * Level 2 keeps parts of tokens: each retained token's value vector is split
 * into S groups and only the routed groups are stored (Stage II, Section 3.3);
 * keys stay full width.  Attention is softmax(q K^T / sqrt(d)) V~ with the
 * dropped groups contributing zero (Section 3.3, attention equation).
 *
 * Conventions for every call
 *   - All tensor pointers are DEVICE pointers unless the argument name ends in
 *     _host.  Tensors are dense, row-major, in the layouts given below.
 *   - The library is stateless and never allocates or frees device memory;
 *     scratch space is a caller-provided workspace sized by
 *     stc_workspace_bytes().  Buffers stay owned by the caller.
 *   - Calls enqueue work on `stream` (a cudaStream_t passed as void*) and
 *     return without synchronising.
 *   - Argument errors are detected on the host before anything is enqueued and
 *     leave every output untouched.  Conditions only the device can see
 *     (budget too small for the routed-token count, packed-capacity overflow)
 *     are written to a caller-provided per-problem status array; kernels never
 *     trap and never read or write out of bounds because of them.
 *   - k, v, kmin, kmax, q, scores, v_packed and out must start on 16-byte
 *     boundaries (the kernels move them in 16-byte pieces); a call given one
 *     that does not returns STC_ERR_INVALID_ARG.
 *   - head_dim must be 128, page_size 16, n_groups in {4, 8, 16},
 *     n_q_heads a multiple of n_kv_heads with at most 8 query heads per KV head.
 *
 * A "problem" is one (batch, kv head) pair; problems are independent.
 *
 * Layouts (B = batch, Hq/Hkv = query / KV heads, T = t_cap, P = ceil(T/16),
 * S = n_groups, g = 128/S):
 *   k, v        bf16  [B][Hkv][T][128]
 *   kmin, kmax  bf16  [B][Hkv][P][128]
 *   q           bf16  [B][Hq][128]          query head h uses KV head h / (Hq/Hkv)
 *   scores      f32   [B][Hkv][T][S]        router logits a_{t,j}
 *   tok_class   u8    [B][Hkv or 1][T]
 *   v_mask      u16   [B][Hkv][T]           bit j set = group j kept
 *   v_offs      u32   [B][Hkv][T+1]         groups stored before token t; [len] = total
 *   v_packed    bf16  [B][Hkv][cap_groups][g]  kept groups, token-major, group-ascending
 *   page_ids    i32   [B][Hkv][max_pages];  n_pages i32 [B][Hkv]
 *   out         f32   [B][Hq][128];         lse f32 [B][Hq] (natural log)
 */
#ifndef STC_H_
#define STC_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
    STC_OK = 0,
    STC_ERR_INVALID_ARG = 1,   /* null pointer, negative size, inconsistent shape      */
    STC_ERR_UNSUPPORTED = 2,   /* head_dim != 128, page_size != 16, S not in {4,8,16}.. */
    STC_ERR_WORKSPACE = 3,     /* workspace missing, misaligned (256 B) or too small    */
    STC_ERR_CAPACITY = 4,      /* packed store too small (device status)                */
    STC_ERR_BUDGET = 5,        /* fewer kept groups than routed tokens with floor 1     */
    STC_ERR_CUDA = 6,          /* a CUDA runtime call failed                            */
    STC_ERR_TIMEOUT = 7,       /* a bounded device-side wait expired (device status)    */
    STC_ERR_SCRATCH_LIMIT = 8  /* problem needs more than the built-in scratch array    */
} stc_status;

enum { STC_CLS_DROP = 0, STC_CLS_ROUTED = 1, STC_CLS_FULL = 2 };
enum { STC_MODE_GLOBAL = 0, STC_MODE_PER_TOKEN = 1 };
enum { STC_OP_QUEST_SELECT = 1, STC_OP_ROUTE_PACK = 2, STC_OP_DECODE_ATTN = 3 };

typedef struct stc_shape {
    int32_t batch, n_q_heads, n_kv_heads;
    int32_t head_dim;          /* 128 */
    int32_t page_size;         /* 16  */
    int32_t n_groups;          /* S   */
    int32_t t_cap;             /* token capacity = row stride of k, v, scores, v_mask */
    int32_t reserved;          /* must be 0 */
    const int32_t* seq_len;    /* device [B] valid tokens per sequence (clamped to
                                  [0, t_cap] on the device); NULL = t_cap for all    */
} stc_shape;

typedef struct stc_cache {
    const void* k;             /* keys, read only                                     */
    void* kmin;                /* page metadata, written by stc_build_page_meta       */
    void* kmax;
    void* v_packed;            /* packed value store, written by stc_route_pack       */
    uint16_t* v_mask;
    uint32_t* v_offs;
    int64_t cap_groups;        /* rows of v_packed per problem                        */
} stc_cache;

const char* stc_status_string(int32_t status);
int32_t stc_version(void);

/* Bytes of workspace `op` (STC_OP_*) needs for `shape`; `arg` is max_pages for
 * STC_OP_DECODE_ATTN and ignored otherwise.  Workspaces must be 256-byte
 * aligned.  A workspace may be reused by consecutive calls on one stream;
 * calls that share a workspace must not overlap on the device. */
int32_t stc_workspace_bytes(const stc_shape* shape, int32_t op, int64_t arg, size_t* bytes_host);

/* Page metadata (Quest chunk size 16: Appendix C.1, table "LLM training
 * configuration"): for pages page_begin <= p < page_end (page_end < 0 = all)
 * and every channel c,
 *     kmin[p][c] = min_t k[t][c],  kmax[p][c] = max_t k[t][c]
 * over the valid tokens t of page p.  Exact (no rounding); -0 orders below
 * +0.  Pages at or beyond ceil(len/16) are left untouched.
 * Reads cache->k, writes cache->kmin / kmax. */
int32_t stc_build_page_meta(const stc_shape* shape, const stc_cache* cache,
                            int32_t page_begin, int32_t page_end, void* stream);

/* Query-aware page selection (Stage I with Quest, Section 3.2; the paper cites
 * the criterion, it is stated here): per problem and page
 *     U[p] = max over the query heads h of the KV head of
 *            sum_c max(q_h[c]*kmin[p][c], q_h[c]*kmax[p][c])
 * which bounds q_h.k_t from above for every token of the page (requires
 * kmin <= kmax as produced by stc_build_page_meta).  The sum is fp32 in a
 * fixed order: 16 partial sums, partial l = (sum of the even channels of
 * 8l..8l+7, ascending, from +0) + (the same over the odd channels); the
 * partials are combined pairwise at distances 8, 4, 2, 1.  The k_pg = min(ceil(len/16),
 * token_budget/16) pages with the largest U are kept, ties to the lower page
 * id; ids are written ascending to page_ids[problem][0..k_pg) and k_pg to
 * n_pages[problem]; entries past k_pg are left untouched.
 * max_pages is the row stride of page_ids and must be >=
 * min(ceil(t_cap/16), token_budget/16).
 * scores_opt (may be NULL): f32 [B][Hkv][P], receives U for the valid pages.
 * Non-finite scores are not supported (selection then is unspecified, still
 * in bounds).  ws: STC_OP_QUEST_SELECT.  The first int32 of ws is a device
 * status word the call writes: STC_OK, or STC_ERR_TIMEOUT if a bounded wait for
 * an asynchronous copy expired on the device (it never should; the page lists
 * then hold valid but unspecified ids).  It can be read after the stream has
 * been synchronised.
 * With several query heads per KV head and scores_opt == NULL the pages are
 * first scored on the tensor cores (same products, another summation order) and
 * only the pages whose approximate score lies within a rigorous error margin of
 * the k_pg-th score are re-scored in the fixed order above; the ids written are
 * the same either way. */
int32_t stc_quest_select(const stc_shape* shape, const stc_cache* cache, const void* q,
                         int32_t token_budget, int32_t max_pages, int32_t* page_ids,
                         int32_t* n_pages, float* scores_opt, void* ws, size_t ws_bytes,
                         void* stream);

/* stc_quest_select with Quest's local window (Appendix C.1, table "LLM training
 * configuration", which lists a Quest window of 64 next to the chunk of 16: read
 * as a window of the 64 most recent tokens = 4 pages): with w = min(n_recent_pages,
 * k_pg), the last w valid pages of every problem are always kept and count
 * against the budget; the other k_pg - w pages are the best-scoring of the
 * pages before them (same bound, same tie rule, ids ascending).
 * n_recent_pages = 0 is stc_quest_select.  Same arguments otherwise. */
int32_t stc_quest_select_window(const stc_shape* shape, const stc_cache* cache, const void* q,
                                int32_t token_budget, int32_t n_recent_pages, int32_t max_pages,
                                int32_t* page_ids, int32_t* n_pages, float* scores_opt, void* ws,
                                size_t ws_bytes, void* stream);

/* stc_quest_select for callers that cannot provide a workspace.  (The paper has
 * no counterpart: this is a deployment convenience of the library.)
 *
 * Who needs it: code that must select pages at a point where it cannot obtain
 * device memory -- a serving loop whose memory pool is frozen while it runs, a
 * plugin that is handed only its input and output buffers by the framework that
 * owns the GPU, a process whose device memory has all been assigned up front.
 * This call makes no allocation of any kind, on the host or on the device.
 *
 * Same operation, arguments, outputs and errors as stc_quest_select, except that
 * the scratch space (arrival counters + fp32 page scores) is an array built into
 * the library image: STC_STATIC_SCRATCH_BYTES of device memory on every GPU that
 * loads the library, held until the process exits.
 *   - Shapes whose selection workspace (stc_workspace_bytes with
 *     STC_OP_QUEST_SELECT) exceeds STC_STATIC_SCRATCH_BYTES are refused with
 *     STC_ERR_SCRATCH_LIMIT before anything is enqueued; with 16-token pages the
 *     array covers batch * n_kv_heads * ceil(t_cap/16) up to about two million
 *     pages (e.g. 16 sequences x 8 KV heads x 131072 tokens).
 *   - The first call made while a given device is current looks up the array's
 *     address on that device (a runtime query, not an allocation) and remembers
 *     it; make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the last
 *     call left in it.  Each call clears the counters it relies on as its first
 *     enqueued operation, so calls that are ordered on the device (same stream,
 *     or otherwise serialised) are independent of each other; two calls that
 *     overlap on the device race on the array and give undefined page lists. */
#define STC_STATIC_SCRATCH_BYTES (8u << 20)
int32_t stc_quest_select_static(const stc_shape* shape, const stc_cache* cache, const void* q,
                                int32_t token_budget, int32_t max_pages, int32_t* page_ids,
                                int32_t* n_pages, float* scores_opt, void* stream);

/* Token classes from a page selection, for running the two stages in the
 * paper's own order (Section 3.4 / Appendix B.1: the value-group router acts on
 * the tokens Stage I retained, with M = N*K over those N tokens):
 *     tok_class[b][hk][t] = STC_CLS_ROUTED if a listed page of problem (b, hk)
 *                           holds the valid token t, STC_CLS_DROP otherwise.
 * Feeding the result to stc_route_pack (class_head_stride = t_cap) routes and
 * packs only the selected tokens; stc_decode_attn with the same page list then
 * attends them.  page_ids / n_pages / max_pages as written by stc_quest_select
 * (ids outside the sequence are ignored).  tok_class: u8 [B][Hkv][t_cap], every
 * byte is written.  Needs no workspace. */
int32_t stc_pages_to_class(const stc_shape* shape, const int32_t* page_ids, const int32_t* n_pages,
                           int32_t max_pages, uint8_t* tok_class, void* stream);

/* Sub-token routing and packing (Section 3.3 "Routing mask"; Section 3.4 and
 * Appendix B.1 for the global budget M = N*K; the VLM per-token rule is the
 * fixed top-K of Section 3.5 / Appendix B.1).
 *   tok_class (NULL = every valid token ROUTED): DROP tokens store nothing,
 *   FULL tokens store all S groups, neither uses budget.  class_head_stride
 *   is T when classes differ per KV head and 0 when one [B][T] array serves
 *   all heads.
 *   STC_MODE_GLOBAL: with N routed tokens in the problem, M = N*k_nominal
 *   (token, group) pairs are kept.  min_per_token = 1: each routed token
 *   keeps its highest-scoring group (first maximum), then the M-N best of the
 *   remaining pairs are kept; min_per_token = 0: the M best of all pairs
 *   (tokens may end with no group, as in the paper's Fig. 1).  Ties go to
 *   the lower flat index t*S + j; -0 and +0 compare equal.
 *   STC_MODE_PER_TOKEN: every routed token keeps its k_nominal best groups
 *   (ties to the lower group).
 * Outputs: out->v_mask (0 for tokens past len), out->v_offs[0..len],
 * out->v_packed, total_groups i64 [B][Hkv], status i32 [B][Hkv] (STC_OK,
 * STC_ERR_BUDGET: nothing packed for that problem, STC_ERR_CAPACITY: groups
 * past cap_groups were not stored, or STC_ERR_TIMEOUT in every entry: a
 * bounded wait between the CTAs of the selection kernel expired and the masks
 * are not valid; all writes stay in bounds).  Non-finite scores are not
 * supported.  The selection kernel is launched cooperatively (its whole grid
 * is resident), so the device must support cooperative launches.
 * ws: STC_OP_ROUTE_PACK. */
int32_t stc_route_pack(const stc_shape* shape, const void* v, const float* scores,
                       const uint8_t* tok_class, int64_t class_head_stride, int32_t k_nominal,
                       int32_t min_per_token, int32_t mode, const stc_cache* out,
                       int64_t* total_groups, int32_t* status, void* ws, size_t ws_bytes,
                       void* stream);

/* stc_route_pack in its two halves, for callers that want the masks before the
 * values are available (or want to time them apart).  stc_route_mask is the
 * routing-mask rule of stc_route_pack (same passages, same arguments): it
 * leaves in out->v_mask the groups every token keeps for certain and, in the
 * workspace, the groups tied at the selection threshold and the per-unit
 * counts.  stc_pack_values turns that into the final masks (ties resolved to
 * the lowest flat indices), the offsets, the packed store, totals and status.
 * It must be the next use of the same workspace after stc_route_mask, with
 * the same shape, cache and mode.  The pair produces exactly the outputs of
 * stc_route_pack.  ws: STC_OP_ROUTE_PACK for both. */
int32_t stc_route_mask(const stc_shape* shape, const float* scores, const uint8_t* tok_class,
                       int64_t class_head_stride, int32_t k_nominal, int32_t min_per_token, int32_t mode,
                       const stc_cache* out, void* ws, size_t ws_bytes, void* stream);
int32_t stc_pack_values(const stc_shape* shape, const void* v, int32_t mode, const stc_cache* out,
                        int64_t* total_groups, int32_t* status, void* ws, size_t ws_bytes, void* stream);

/* Value-group router logits (Appendix B.1 "Value-Group Router": one linear
 * projection from the layer's input hidden state to S group logits per KV
 * head; Section 3.4's query-aware form g(h, s_Q) is the same projection with an
 * additive per-sequence term, passed as bias_opt):
 *     scores[b][hk][t][j] = sum_c h[b][t][c] * w[hk*S + j][c]  (+ bias_opt[b][hk*S + j])
 *   h         bf16 [B][t_cap][d_model]      hidden states
 *   w         bf16 [Hkv*S][d_model]         router weights
 *   bias_opt  f32  [B][Hkv*S] or NULL
 *   scores    f32  [B][Hkv][t_cap][S]       the layout stc_route_pack reads
 * bf16 products, fp32 accumulation on the tensor cores (tcgen05 + TMA); all
 * t_cap rows are computed.  Supported: d_model a multiple of 64; Hkv*S a
 * multiple of 16 and either <= 256 or a multiple of 256 (else
 * STC_ERR_UNSUPPORTED); h, w, bias, scores 16-byte aligned.  status_word:
 * device i32 the call writes (STC_OK, or STC_ERR_TIMEOUT if a bounded wait on
 * the device expired; scores are then unspecified).  Needs no workspace. */
int32_t stc_router_logits(const stc_shape* shape, const void* h, const void* w, const float* bias_opt,
                          int32_t d_model, float* scores, int32_t* status_word, void* stream);

/* Query summary and its router term (Section 3.4 "query-aware routing": the
 * router sees the token's hidden state and a summary s_Q of the query region;
 * the paper fixes neither the summary operator nor g -- taken here: s_Q = mean
 * of the query-region hidden states, g linear in [h ; s_Q], so the query adds
 * one term per sequence and logit, the bias_opt of stc_router_logits):
 *     s_q[b][c]  = (1 / len_b) * sum_{t < len_b} h_q[b][t][c]     (0 when len_b = 0)
 *     bias[b][n] = sum_c s_q[b][c] * w_q[n][c]
 *   h_q        bf16 [batch][q_cap][d_model]   hidden states of the query region
 *   q_len_opt  i32  [batch] or NULL (= q_cap); clamped to 0..q_cap
 *   w_q        bf16 [n_logits][d_model]       the s_Q half of the router weights
 *   s_q        f32  [batch][d_model]  (out)    bias  f32 [batch][n_logits]  (out)
 * fp32 accumulation in a fixed order (repeatable bit for bit).  d_model must be
 * a multiple of 8 (else STC_ERR_UNSUPPORTED), batch <= 65535; h_q, w_q, s_q
 * 16-byte aligned; all pointers are device pointers.  Needs no workspace. */
int32_t stc_query_bias(int32_t batch, int32_t q_cap, int32_t d_model, int32_t n_logits, const void* h_q,
                       const int32_t* q_len_opt, const void* w_q, float* s_q, float* bias, void* stream);

/* Streaming append (Section 3.4 exempts the query region from value compression:
 * the tokens generated during decoding keep all their value groups).  For every sequence
 * b the tokens old_len[b] <= t < len[b] (len = shape->seq_len AFTER the append,
 * or t_cap when seq_len is NULL) have just been added: their keys are already in
 * cache->k and their values in v (same [B][Hkv][T][128] layout as stc_route_pack;
 * only the new rows are read).  The call
 *   - stores all S groups of each new token behind the sequence's packed groups
 *     (v_mask = all ones, v_offs advanced by S per token, v_offs[len] = total),
 *   - recomputes kmin / kmax of every page that holds a new token, over all of
 *     the page's valid tokens.
 * The result equals stc_build_page_meta + stc_route_pack over the longer
 * sequence with the new tokens in class FULL.  old_len: device i32 [B];
 * max_new: upper bound of len[b] - old_len[b] (sizes the launch).
 * total_groups / status as in stc_route_pack; a sequence whose lengths are
 * inconsistent (old_len > len, or more than max_new new tokens) is left
 * untouched with status STC_ERR_INVALID_ARG.  Needs no workspace. */
int32_t stc_append_tokens(const stc_shape* shape, const stc_cache* cache, const void* v,
                          const int32_t* old_len, int32_t max_new, int64_t* total_groups, int32_t* status,
                          void* stream);

/* Routing of the pages completed during decoding (Section 3.4: the budget is global over the
 * retained tokens, M = N*K in Appendix B.1, and the query region stays uncompressed; the paper
 * does not say when a generated token leaves the query region -- reading taken: while its
 * 16-token page is still open).  For every sequence b with len = shape->seq_len[b], each complete
 * page p with first_page[b] <= p < len/16 -- stored at full width by stc_append_tokens -- is
 * routed ON ITS OWN: its 16 tokens join the routed set, the budget grows by 16*k_nominal groups
 * and they are allotted among the page's (token, group) pairs by the rule of stc_route_pack
 * (STC_MODE_GLOBAL with floor min_per_token: each token's first maximum, then the best
 * 16*k_nominal - 16 of the page's other pairs, ties to the lower flat index; STC_MODE_PER_TOKEN:
 * every token's k_nominal best groups).  The kept groups are compacted in place, the tokens of
 * the still open page stay at full width and move down behind them; v_mask, v_offs[first..len]
 * and total_groups are updated.  The result does not depend on whether pages are routed one
 * call at a time or several at once, and the routed tokens always hold exactly N*k_nominal
 * groups.
 *   scores      f32 [B][Hkv][t_cap][S], rows of the completed pages are read
 *   first_page  device i32 [B]: first page not yet routed
 * At most 8 pages per sequence and call.  status i32 [B][Hkv]: STC_OK; STC_ERR_INVALID_ARG
 * (more than 8 completed pages, or the range is not stored at full width) and STC_ERR_BUDGET
 * (k_nominal = 0 with floor 1) leave the problem untouched.  Needs no workspace. */
int32_t stc_route_new_pages(const stc_shape* shape, const stc_cache* cache, const float* scores,
                            const int32_t* first_page, int32_t k_nominal, int32_t min_per_token,
                            int32_t mode, int64_t* total_groups, int32_t* status, void* stream);

/* Routed decode attention (Section 3.3, attention equation): per query head h
 * with KV head h / (Hq/Hkv) and R = the valid tokens of the listed pages,
 *     s_t = sm_scale * q_h.k_t,  p = softmax over R of s,
 *     out[h][j*g .. (j+1)*g) = sum_{t in R} p_t * [bit j of v_mask[t]] * v_t^{(j)}
 * so a dropped group adds zero while its token still counts in the
 * normaliser.  page_ids NULL = every page of the sequence (selection off);
 * otherwise n_pages[problem] ids are read from page_ids[problem] (row stride
 * max_pages); ids outside [0, ceil(len/16)) are skipped, a page listed twice
 * counts twice.  An empty R gives out = 0 and lse = -inf.
 * bf16 inputs, fp32 accumulation, fp32 outputs; the softmax weights enter the
 * value contraction as a bf16 pair (high + residual part) when the tensor-core
 * path is used (more than one query head per KV head).  lse_opt may be NULL.
 * k and v_packed must be 16-byte aligned (pages and packed spans are moved by
 * bulk asynchronous copies).
 * ws: STC_OP_DECODE_ATTN with arg = max_pages (for page_ids NULL: ceil(T/16)).
 * The first int32 of ws is a device status word the call writes: STC_OK, or
 * STC_ERR_TIMEOUT if a bounded wait for a copy expired on the device (it never
 * should; out / lse are then unspecified).  It can be read after the stream
 * has been synchronised. */
int32_t stc_decode_attn(const stc_shape* shape, const stc_cache* cache, const void* q,
                        const int32_t* page_ids, const int32_t* n_pages, int32_t max_pages,
                        float sm_scale, float* out, float* lse_opt, void* ws, size_t ws_bytes,
                        void* stream);

/* One decode step on the device: stc_quest_select followed by stc_decode_attn over the pages it
 * selected (Stage I per step, Section 3.2, then the routed attention of Section 3.3), as one call.
 * Same operation, arguments, outputs and errors as the two calls made one after the other with
 * scores_opt = NULL; the difference is in the launch: both workspaces are cleared first, so that
 * the two kernels follow each other directly on the stream (about 2 us less per step than the two
 * calls).  ws_select: STC_OP_QUEST_SELECT; ws_attn: STC_OP_DECODE_ATTN with arg = max_pages;
 * the two must not overlap (each carries its status word).  max_pages >= min(ceil(t_cap/16),
 * token_budget/16) and <= ceil(t_cap/16). */
int32_t stc_decode_step(const stc_shape* shape, const stc_cache* cache, const void* q, int32_t token_budget,
                        int32_t max_pages, int32_t* page_ids, int32_t* n_pages, float sm_scale, float* out,
                        float* lse_opt, void* ws_select, size_t ws_select_bytes, void* ws_attn,
                        size_t ws_attn_bytes, void* stream);

/* Stored bytes of the compressed cache for the accounting of Section 3.3
 * ("Compression ratio") and Appendix C.2 ("SubToken configuration and budget"): full-width keys of the retained
 * tokens plus the packed groups (mask/offset/metadata bytes are returned
 * separately).  Host arithmetic only. */
int32_t stc_cache_bytes(int64_t n_tokens_retained, int64_t n_groups_kept, int32_t n_groups,
                        int64_t* kv_bytes_host, int64_t* index_bytes_host);

/* One whole pass from HOST memory (the end-to-end form of the calls above):
 * copies k, v, scores, tok_class and q from host buffers into a caller-provided
 * device arena, runs stc_build_page_meta, stc_route_pack (STC_MODE_* / floor as
 * given), stc_quest_select (skipped when token_budget < 0: every page attended)
 * and stc_decode_attn, and copies out [B][Hq][128], total_groups [B][Hkv] and
 * status [B][Hkv] back to host buffers.  Everything is enqueued on `stream`;
 * the host outputs are valid after the caller synchronises the stream.  Host
 * buffers should be page-locked so the copies run asynchronously.
 *   *_host       host pointers, same layouts as the device tensors;
 *                tok_class_host is [B][T] shared by heads, or NULL
 *   shape->seq_len  still a DEVICE pointer (or NULL)
 *   cap_groups   rows of the packed store per problem inside the arena
 *   arena        device memory, 256-byte aligned, at least
 *                stc_pass_host_arena_bytes() bytes; owned by the caller and
 *                reusable by the next call on the same stream
 * Operation and errors are those of the four calls it chains. */
int32_t stc_pass_host_arena_bytes(const stc_shape* shape, int64_t cap_groups, int32_t token_budget,
                                  size_t* bytes_host);
int32_t stc_pass_host(const stc_shape* shape, const void* k_host, const void* v_host,
                      const float* scores_host, const uint8_t* tok_class_host, const void* q_host,
                      int32_t token_budget, int32_t k_nominal, int32_t min_per_token, int32_t mode,
                      float sm_scale, int64_t cap_groups, void* arena, size_t arena_bytes,
                      float* out_host, int64_t* total_groups_host, int32_t* status_host,
                      void* stream);

/* One decode step from HOST memory over a cache that is resident on the device
 * (the per-step read side: Stage I selection, Section 3.2, then the routed
 * attention of Section 3.3): copies q from q_host into the arena, runs
 * stc_quest_select (skipped when token_budget < 0: every page attended) and
 * stc_decode_attn on `cache` (device pointers: k, kmin, kmax, v_packed, v_mask,
 * v_offs as left by the write-side calls), and copies out [B][Hq][128] and the
 * attention call's device status word (STC_OK or STC_ERR_TIMEOUT) to host
 * buffers.  Everything is enqueued on `stream`; the host outputs are valid after
 * the caller synchronises it.  q_host / out_host / status_host should be
 * page-locked.  arena: device memory, 256-byte aligned, at least
 * stc_decode_step_host_arena_bytes() bytes, owned by the caller, reusable by the
 * next call on the same stream.  Errors are those of the two calls it chains. */
int32_t stc_decode_step_host_arena_bytes(const stc_shape* shape, int32_t token_budget, size_t* bytes_host);
int32_t stc_decode_step_host(const stc_shape* shape, const stc_cache* cache, const void* q_host,
                             int32_t token_budget, float sm_scale, void* arena, size_t arena_bytes,
                             float* out_host, int32_t* status_host, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* STC_H_ */
