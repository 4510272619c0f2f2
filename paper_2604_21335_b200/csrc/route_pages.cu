// Routing of the pages that complete during decoding.
//
// stc_append_tokens stores every generated token at full width (the query region is exempt from
// value compression, Section 3.4).  The paper does not say when a generated token stops being
// "query region"; the reading taken here: while its 16-token page is still open.  When a page
// completes, its 16 tokens join the routed set, so the global budget M = N*K (Appendix B.1)
// grows by 16*K groups, and those are allotted among the page's own (token, group) pairs by the
// rule of stc_route_pack -- the dropped groups of older tokens no longer exist in a packed
// store, so an older decision cannot be revisited, and a page routed on its own gives a result
// that does not depend on how many pages a call happens to find completed.
//
// One CTA per (batch, kv head) problem.  The range to rewrite -- the completed pages plus the
// tokens of the open page behind them -- is at most kMaxPages pages + 15 tokens of full-width
// values, contiguous in the packed store: it is staged in shared memory, the pages are routed
// (a page has at most 16 x 16 candidate pairs, so ranking by counting is enough), and the kept
// groups are written back compacted; every byte written comes from shared memory, so the
// in-place move toward lower addresses is safe.  Scores are compared through their
// order-preserving keys (-0 == +0), ties go to the lower flat index t*S + j.
#include "common.cuh"

namespace stc {
namespace {

constexpr int kThreads = 256;
constexpr int kMaxPages = 8;
constexpr int kMaxTok = kMaxPages * kPage + kPage - 1;

template <int S>
__global__ void __launch_bounds__(kThreads)
route_new_pages_kernel(const float* __restrict__ scores, const int32_t* __restrict__ seq_len,
                       const int32_t* __restrict__ first_page, int Hkv, int T, int k_nominal,
                       int min_per_token, int mode, uint16_t* __restrict__ v_mask, uint32_t* __restrict__ v_offs,
                       uint4* __restrict__ v_packed, int64_t cap_groups, int64_t* __restrict__ total_groups,
                       int32_t* __restrict__ status) {
    constexpr int OPG = kOctets / S;               // 16-byte chunks per group
    constexpr uint32_t kAll = (1u << S) - 1u;
    __shared__ uint4 s_val[kMaxTok * kOctets];     // full-width values of the range
    __shared__ uint32_t s_key[kMaxPages * kPage * S];
    __shared__ uint16_t s_mask[kMaxTok];
    __shared__ uint32_t s_off[kMaxTok + 1];
    __shared__ int s_bad;

    const int problem = blockIdx.x, b = problem / Hkv, tid = threadIdx.x;
    const int len = clamp_len(seq_len, b, T);
    const int fp = first_page[b];
    const int t0 = fp * kPage;
    const int n_pages = len / kPage - fp;
    uint32_t* offs = v_offs + (size_t)problem * (T + 1);
    uint16_t* mask = v_mask + (size_t)problem * T;
    if (tid == 0) s_bad = 0;
    __syncthreads();
    if (fp < 0 || n_pages > kMaxPages) {           // inconsistent arguments: nothing is touched
        if (tid == 0) status[problem] = STC_ERR_INVALID_ARG;
        return;
    }
    if (n_pages <= 0 || t0 >= len) {               // no page has completed
        if (tid == 0) { status[problem] = STC_OK; total_groups[problem] = (int64_t)offs[len]; }
        return;
    }
    const int n_tok = len - t0;                    // <= kMaxTok
    const int64_t base = (int64_t)offs[t0];
    // the range must be stored at full width, inside the store
    for (int i = tid; i < n_tok; i += kThreads)
        if (mask[t0 + i] != (uint16_t)kAll || offs[t0 + i + 1] - offs[t0 + i] != (uint32_t)S) s_bad = 1;
    if (tid == 0 && base + (int64_t)n_tok * S > cap_groups) s_bad = 1;
    __syncthreads();
    if (s_bad) {
        if (tid == 0) status[problem] = STC_ERR_INVALID_ARG;
        return;
    }
    if (mode == STC_MODE_GLOBAL && min_per_token && k_nominal < 1) {
        if (tid == 0) status[problem] = STC_ERR_BUDGET;
        return;
    }
    // ---- stage the values and the score keys --------------------------------------------------
    const uint4* src = v_packed + ((size_t)problem * cap_groups + base) * OPG;   // = n_tok rows of 16 chunks
    for (int i = tid; i < n_tok * kOctets; i += kThreads) s_val[i] = src[i];
    const float* sc = scores + ((size_t)problem * T + t0) * S;
    for (int i = tid; i < n_pages * kPage * S; i += kThreads) s_key[i] = float_key(sc[i]);
    __syncthreads();

    // ---- masks: one thread per token of a completed page ---------------------------------------
    for (int i = tid; i < n_tok; i += kThreads) {
        uint32_t m = kAll;                          // tokens of the open page keep everything
        if (i < n_pages * kPage) {
            const int page = i / kPage;
            const uint32_t* pk = s_key + page * kPage * S;   // the page's [16][S] keys
            const uint32_t* mine = s_key + i * S;
            m = 0u;
            if (mode == STC_MODE_PER_TOKEN) {
#pragma unroll 1
                for (int j = 0; j < S; ++j) {
                    int rank = 0;
                    for (int o = 0; o < S; ++o) rank += (mine[o] > mine[j]) || (mine[o] == mine[j] && o < j);
                    if (rank < k_nominal) m |= 1u << j;
                }
            } else {
                // the reserved first maximum of a token, as every thread of the page needs them all
                auto reserved = [&](int tok) {
                    const uint32_t* kk = pk + tok * S;
                    int best = 0;
                    for (int j = 1; j < S; ++j) if (kk[j] > kk[best]) best = j;
                    return best;
                };
                const int tl = i - page * kPage;
                const int my_best = min_per_token ? reserved(tl) : -1;
                const int take = k_nominal * kPage - (min_per_token ? kPage : 0);
                if (my_best >= 0) m |= 1u << my_best;
#pragma unroll 1
                for (int j = 0; j < S; ++j) {
                    if (j == my_best) continue;
                    const uint32_t x = mine[j];
                    int rank = 0;                   // candidates ahead of (x, flat index) in (key desc, flat asc)
                    for (int tok = 0; tok < kPage; ++tok) {
                        const int rb = min_per_token ? reserved(tok) : -1;
                        const uint32_t* kk = pk + tok * S;
                        for (int o = 0; o < S; ++o) {
                            if (o == rb) continue;
                            rank += (kk[o] > x) || (kk[o] == x && (tok < tl || (tok == tl && o < j)));
                        }
                    }
                    if (rank < take) m |= 1u << j;
                }
            }
        }
        s_mask[i] = (uint16_t)m;
    }
    __syncthreads();
    if (tid == 0) {                                 // offsets: a short sequential walk
        uint32_t n = 0;
        for (int i = 0; i < n_tok; ++i) { s_off[i] = n; n += __popc((uint32_t)s_mask[i]); }
        s_off[n_tok] = n;
    }
    __syncthreads();
    // ---- write back: masks, offsets, the kept groups compacted ------------------------------------
    for (int i = tid; i < n_tok; i += kThreads) {
        mask[t0 + i] = s_mask[i];
        offs[t0 + i] = (uint32_t)(base + s_off[i]);
    }
    if (tid == 0) {
        const int64_t total = base + s_off[n_tok];
        offs[len] = (uint32_t)total;
        total_groups[problem] = total;
        status[problem] = STC_OK;
    }
    uint4* dst = v_packed + ((size_t)problem * cap_groups + base) * OPG;
    for (int i = tid; i < n_tok * kOctets; i += kThreads) {
        const int tok = i / kOctets, oct = i - tok * kOctets, grp = oct / OPG;
        const uint32_t m = s_mask[tok];
        if (!((m >> grp) & 1u)) continue;
        const uint32_t pos = (s_off[tok] + __popc(m & ((1u << grp) - 1u))) * OPG + (uint32_t)(oct % OPG);
        dst[pos] = s_val[i];
    }
}

}  // namespace

int route_new_pages_max() { return kMaxPages; }

cudaError_t launch_route_new_pages(const Geom& g, const float* scores, const int32_t* first_page, int k_nominal,
                                   int min_per_token, int mode, void* v_packed, uint16_t* v_mask,
                                   uint32_t* v_offs, int64_t cap_groups, int64_t* total_groups, int32_t* status,
                                   cudaStream_t st) {
    if (g.problems == 0) return cudaSuccess;
#define STC_RNP(S_)                                                                                         \
    case S_:                                                                                                \
        route_new_pages_kernel<S_><<<g.problems, kThreads, 0, st>>>(                                        \
            scores, g.seq_len, first_page, g.Hkv, g.T, k_nominal, min_per_token, mode, v_mask, v_offs,      \
            static_cast<uint4*>(v_packed), cap_groups, total_groups, status);                               \
        break;
    switch (g.S) {
        STC_RNP(4) STC_RNP(8) STC_RNP(16)
        default: return cudaErrorInvalidValue;
    }
#undef STC_RNP
    return cudaGetLastError();
}

}  // namespace stc
