// Query-aware page selection: bound scoring + per-problem top-k, one launch.
//
// Scoring streams the page metadata once (512 B per page).  A half-warp owns a
// page; lane l of the half owns channels 8l..8l+7 (one 16-byte chunk of kmin and
// of kmax), accumulates its eight terms in ascending channel order, and the 16
// partial sums are combined by an xor butterfly at distances 8, 4, 2, 1 -- the
// fixed summation order the selection is defined with.  The term
// max(q*kmin, q*kmax) is formed as fma(q+, kmax, fma(q-, kmin, acc)) with
// q+ = max(q,0), q- = min(q,0): bf16*bf16 products are exact in fp32 and one of
// the two products is zero, so each channel adds exactly one rounding, the same
// as acc + max(q*kmin, q*kmax).
//
// With more than four query heads per KV head the two halves of a warp share a
// page and split the heads (keeps the query registers of a lane at 4 heads).
//
// The CTA that finishes a problem last (atomic ticket, no waiting) selects the
// pages: 4-pass 8-bit radix select on order-preserving keys held in shared
// memory, then an ordered compaction that emits ids ascending and resolves
// ties at the threshold in favour of lower page ids.
#include "common.cuh"

namespace stc {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kPagesPerCta = 128;
constexpr int kKeysSmem = 8192;              // pages whose keys are staged in shared memory

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, int lane) {
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t o = __shfl_up_sync(0xFFFFFFFFu, v, d);
        if (lane >= d) v += o;
    }
    return v;
}

// Top-k of u[0..n) by (value descending, index ascending); ids written ascending.
// Requires 0 < k < n.  All kThreads threads of the CTA call it.
__device__ void block_topk(const float* __restrict__ u, int n, int k, int32_t* __restrict__ ids,
                           uint32_t* skeys) {
    __shared__ uint32_t hist[256];
    __shared__ uint32_t s_prefix, s_krem;
    __shared__ uint32_t s_wtot[kWarps][2];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const bool staged = n <= kKeysSmem;
    if (staged)
        for (int i = tid; i < n; i += kThreads) skeys[i] = float_key(__ldcg(u + i));
    __syncthreads();
    auto key_at = [&](int i) -> uint32_t { return staged ? skeys[i] : float_key(__ldcg(u + i)); };

    uint32_t prefix = 0, krem = (uint32_t)k;
#pragma unroll 1
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        const uint32_t hi_mask = pass == 0 ? 0u : (0xFFFFFFFFu << (shift + 8));
        hist[tid] = 0;
        __syncthreads();
        for (int i = tid; i < n; i += kThreads) {
            uint32_t key = key_at(i);
            if ((key & hi_mask) == prefix) atomicAdd(&hist[(key >> shift) & 255u], 1u);
        }
        __syncthreads();
        if (warp == 0) {
            // lane L owns digits 255-8L .. 248-8L, walked downwards
            uint32_t c[8], sum = 0;
#pragma unroll
            for (int j = 0; j < 8; ++j) { c[j] = hist[255 - 8 * lane - j]; sum += c[j]; }
            uint32_t incl = warp_incl_scan(sum, lane), run = incl - sum;
            if (run < krem && krem <= incl) {
#pragma unroll
                for (int j = 0; j < 8; ++j) {
                    if (run + c[j] >= krem) {
                        s_prefix = prefix | ((uint32_t)(255 - 8 * lane - j) << shift);
                        s_krem = krem - run;
                        break;
                    }
                    run += c[j];
                }
            }
        }
        __syncthreads();
        prefix = s_prefix;
        krem = s_krem;
    }
    const uint32_t tau = prefix;                 // krem = ties at tau still to take

    const int per = (n + kThreads - 1) / kThreads;
    const int lo = min(n, tid * per), hi = min(n, lo + per);
    uint32_t gt = 0, eq = 0;
    for (int i = lo; i < hi; ++i) { uint32_t key = key_at(i); gt += key > tau; eq += key == tau; }
    uint32_t gi = warp_incl_scan(gt, lane), ei = warp_incl_scan(eq, lane);
    if (lane == 31) { s_wtot[warp][0] = gi; s_wtot[warp][1] = ei; }
    __syncthreads();
    uint32_t gb = gi - gt, eb = ei - eq;
    for (int w = 0; w < warp; ++w) { gb += s_wtot[w][0]; eb += s_wtot[w][1]; }
    uint32_t pos = gb + min(eb, krem);
    for (int i = lo; i < hi; ++i) {
        uint32_t key = key_at(i);
        if (key > tau) ids[pos++] = i;
        else if (key == tau) { if (eb < krem) ids[pos++] = i; ++eb; }
    }
}

template <int GQ>
__global__ void __launch_bounds__(kThreads)
quest_select_kernel(const uint4* __restrict__ kmin, const uint4* __restrict__ kmax,
                    const uint4* __restrict__ q, const int32_t* __restrict__ seq_len, int Hq, int Hkv,
                    int T, int P, int token_budget, int max_pages, int32_t* __restrict__ page_ids,
                    int32_t* __restrict__ n_pages, float* __restrict__ scores, int scores_wanted,
                    unsigned* __restrict__ counters, int chunks) {
    constexpr bool kSplit = GQ > 4;            // halves of a warp share a page, split the heads
    constexpr int NH = kSplit ? 4 : GQ;        // heads per lane
    constexpr int kPagesPerIter = kWarps * (kSplit ? 1 : 2);
    constexpr int kIters = kPagesPerCta / kPagesPerIter;
    constexpr int kBatch = 4;                  // iterations whose loads are in flight together

    extern __shared__ uint32_t skeys[];
    __shared__ int s_last;

    const int problem = blockIdx.x / chunks;
    const int chunk = blockIdx.x - problem * chunks;
    const int b = problem / Hkv, hk = problem - b * Hkv;
    const int len = clamp_len(seq_len, b, T);
    const int np = (len + kPage - 1) / kPage;
    int k_pg = token_budget / kPage;
    k_pg = min(k_pg, min(np, max_pages));
    const bool trivial = (k_pg >= np) || (k_pg <= 0);
    int32_t* ids = page_ids + (size_t)problem * max_pages;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    if (trivial && chunk == 0) {
        for (int i = tid; i < k_pg; i += kThreads) ids[i] = i;
        if (tid == 0) n_pages[problem] = max(k_pg, 0);
    }
    if (trivial && !scores_wanted) return;

    // ---- bound scores for this CTA's pages --------------------------------
    const int half = lane >> 4, l = lane & 15;
    float qp[NH][8], qn[NH][8];
#pragma unroll
    for (int h = 0; h < NH; ++h) {
        int head = kSplit ? min(half * 4 + h, GQ - 1) : h;   // padding repeats a real head
        uint4 w = q[((size_t)b * Hq + (size_t)hk * GQ + head) * kOctets + l];
        float f[8] = {bf16lo(w.x), bf16hi(w.x), bf16lo(w.y), bf16hi(w.y),
                      bf16lo(w.z), bf16hi(w.z), bf16lo(w.w), bf16hi(w.w)};
#pragma unroll
        for (int c = 0; c < 8; ++c) { qp[h][c] = fmaxf(f[c], 0.f); qn[h][c] = fminf(f[c], 0.f); }
    }
    const size_t row0 = (size_t)problem * P;
    const int c0 = chunk * kPagesPerCta;
    float* urow = scores + row0;
#pragma unroll 1
    for (int it0 = 0; it0 < kIters; it0 += kBatch) {
        uint4 lo[kBatch], hi[kBatch];
        int page[kBatch];
#pragma unroll
        for (int i = 0; i < kBatch; ++i) {
            page[i] = c0 + (it0 + i) * kPagesPerIter + (kSplit ? warp : warp * 2 + half);
            if (page[i] < np) {
                lo[i] = ldg_nc16(kmin + (row0 + page[i]) * kOctets + l);
                hi[i] = ldg_nc16(kmax + (row0 + page[i]) * kOctets + l);
            } else {
                lo[i] = hi[i] = make_uint4(0, 0, 0, 0);
            }
        }
#pragma unroll
        for (int i = 0; i < kBatch; ++i) {
            const float a[8] = {bf16lo(lo[i].x), bf16hi(lo[i].x), bf16lo(lo[i].y), bf16hi(lo[i].y),
                                bf16lo(lo[i].z), bf16hi(lo[i].z), bf16lo(lo[i].w), bf16hi(lo[i].w)};
            const float z[8] = {bf16lo(hi[i].x), bf16hi(hi[i].x), bf16lo(hi[i].y), bf16hi(hi[i].y),
                                bf16lo(hi[i].z), bf16hi(hi[i].z), bf16lo(hi[i].w), bf16hi(hi[i].w)};
            float best = 0.f;
#pragma unroll
            for (int h = 0; h < NH; ++h) {
                float acc = 0.f;
#pragma unroll
                for (int c = 0; c < 8; ++c) acc = __fmaf_rn(qp[h][c], z[c], __fmaf_rn(qn[h][c], a[c], acc));
#pragma unroll
                for (int d = 8; d >= 1; d >>= 1) acc = acc + __shfl_xor_sync(0xFFFFFFFFu, acc, d);
                best = (h == 0) ? acc : fmaxf(best, acc);
            }
            if (kSplit) best = fmaxf(best, __shfl_xor_sync(0xFFFFFFFFu, best, 16));
            if (l == 0 && (!kSplit || half == 0) && page[i] < np) urow[page[i]] = best;
        }
    }
    if (trivial) return;

    // ---- last CTA of the problem selects ----------------------------------
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(&counters[problem], 1u) == (unsigned)(chunks - 1));
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    block_topk(urow, np, k_pg, ids, skeys);
    if (tid == 0) n_pages[problem] = k_pg;
}

size_t counters_bytes(const Geom& g) { return (((size_t)g.problems * 4) + 255) & ~(size_t)255; }

}  // namespace

size_t select_ws_bytes(const Geom& g) {
    return counters_bytes(g) + (size_t)g.problems * g.P * sizeof(float);
}

cudaError_t launch_quest_select(const Geom& g, const void* kmin, const void* kmax, const void* q,
                                int token_budget, int max_pages, int32_t* page_ids,
                                int32_t* n_pages, float* scores_opt, void* ws, cudaStream_t st) {
    if (g.problems == 0) return cudaSuccess;
    unsigned* counters = static_cast<unsigned*>(ws);
    float* scores = scores_opt ? scores_opt
                               : reinterpret_cast<float*>(static_cast<char*>(ws) + counters_bytes(g));
    cudaError_t e = cudaMemsetAsync(counters, 0, (size_t)g.problems * 4, st);
    if (e != cudaSuccess) return e;
    const int chunks = (g.P + kPagesPerCta - 1) / kPagesPerCta;
    const long long n_cta = (long long)chunks * g.problems;
    if (n_cta > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    const size_t smem = (size_t)min(g.P, kKeysSmem) * 4;
#define STC_SEL(GQ_)                                                                             \
    case GQ_:                                                                                    \
        quest_select_kernel<GQ_><<<(unsigned)n_cta, kThreads, smem, st>>>(                       \
            static_cast<const uint4*>(kmin), static_cast<const uint4*>(kmax),                    \
            static_cast<const uint4*>(q), g.seq_len, g.Hq, g.Hkv, g.T, g.P, token_budget,        \
            max_pages, page_ids, n_pages, scores, scores_opt != nullptr, counters, chunks);      \
        break;
    switch (g.Gq) {
        STC_SEL(1) STC_SEL(2) STC_SEL(3) STC_SEL(4) STC_SEL(5) STC_SEL(6) STC_SEL(7) STC_SEL(8)
        default: return cudaErrorInvalidValue;
    }
#undef STC_SEL
    return cudaGetLastError();
}

}  // namespace stc
