// Query-aware page selection: bound scoring + per-problem top-k, one launch.
//
// Scoring streams the page metadata once (512 B per page).  A half-warp owns a
// page; lane l of the half owns channels 8l..8l+7 (one 16-byte chunk of kmin and
// of kmax).  The fixed fp32 summation order the selection is defined with:
//   - lane l keeps two running sums, one over its even channels (8l, 8l+2, 8l+4,
//     8l+6, ascending, from +0) and one over its odd channels, then adds
//     even + odd;
//   - the 16 lane sums are combined pairwise at distances 8, 4, 2, 1.
// The two running sums are the two halves of one packed fp32x2 FMA
// (fma.rn.f32x2), which halves the issue slots of the inner product.  The term
// max(q*kmin, q*kmax) is formed as fma(q+, kmax, fma(q-, kmin, acc)) with
// q+ = max(q,0), q- = min(q,0): bf16*bf16 products are exact in fp32 and one of
// the two products is zero, so each channel adds exactly one rounding, the same
// as acc + max(q*kmin, q*kmax).
// With several heads the butterfly halves its payload at each level (a lane keeps
// the heads its lane-id bits select), so 4 heads cost 7 shuffles, not 16; the
// pairing of partial sums, and therefore every rounding, is unchanged.
//
// With more than four query heads per KV head the two halves of a warp share a
// page and split the heads (keeps the query registers of a lane at 4 heads).
//
// Work split: the pages of all problems form one flat sequence of units (one
// unit = the pages the 8 warps of a CTA reduce together); a persistent grid of
// (SM count x 2) CTAs cuts it into equal contiguous ranges, so there is no
// partial wave.  Inside a problem each lane keeps a private ring of 16-byte
// cp.async copies running kDepth units ahead; nothing waits on another thread.
// When a CTA leaves a problem it adds the units it covered to the problem's
// counter; whoever completes the count (no waiting) selects the pages: bitwise
// binary search for the k-th largest order-preserving key held in registers (no
// atomics, so hot histogram bins cannot serialise it), then an ordered
// compaction that emits ids ascending and resolves ties at the threshold in
// favour of lower page ids.
#include "common.cuh"

namespace stc {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kCtasPerSm = 2;
constexpr int kDepth = 8;                    // units in flight per lane (32 B each)
constexpr size_t kRingBytes = (size_t)kDepth * kThreads * 32;
constexpr int kKpt = 32;                     // keys per thread held in registers by the top-k
constexpr int kRegKeys = kKpt * kThreads;    // 8192 pages; longer rows take the memory path

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, int lane) {
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t o = __shfl_up_sync(0xFFFFFFFFu, v, d);
        if (lane >= d) v += o;
    }
    return v;
}

// Top-k of u[0..n) by (value descending, index ascending); ids written ascending.
// Requires 0 < k < n.  All kThreads threads of the CTA call it.  Thread t owns the
// contiguous keys [t*per, (t+1)*per); REG keeps them in registers (n <= kRegKeys).
template <bool REG>
__device__ void block_topk(const float* __restrict__ u, int n, int k, int32_t* __restrict__ ids) {
    __shared__ uint32_t s_cnt[2][kWarps];
    __shared__ uint32_t s_wtot[kWarps][2];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int per = (n + kThreads - 1) / kThreads;
    const int lo = min(n, tid * per), hi = min(n, lo + per);
    uint32_t key[REG ? kKpt : 1];
    if (REG) {
#pragma unroll
        for (int j = 0; j < kKpt; ++j) key[j] = (lo + j < hi) ? float_key(__ldcg(u + lo + j)) : 0u;
    }
    auto key_at = [&](int i) -> uint32_t { return float_key(__ldcg(u + i)); };

    // k-th largest key, one bit per step: the largest value v with #(key >= v) >= k
    uint32_t tau = 0;
#pragma unroll 1
    for (int bit = 31; bit >= 0; --bit) {
        const uint32_t cand = tau | (1u << bit);
        uint32_t c = 0;
        if (REG) {
#pragma unroll
            for (int j = 0; j < kKpt; ++j) c += key[j] >= cand;
        } else {
            for (int i = lo; i < hi; ++i) c += key_at(i) >= cand;
        }
        c = __reduce_add_sync(0xFFFFFFFFu, c);
        if (lane == 0) s_cnt[bit & 1][warp] = c;
        __syncthreads();
        uint32_t tot = 0;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) tot += s_cnt[bit & 1][w];
        if (tot >= (uint32_t)k) tau = cand;
    }

    uint32_t gt = 0, eq = 0;
    if (REG) {
#pragma unroll
        for (int j = 0; j < kKpt; ++j) { gt += key[j] > tau; eq += (lo + j < hi) && key[j] == tau; }
    } else {
        for (int i = lo; i < hi; ++i) { uint32_t x = key_at(i); gt += x > tau; eq += x == tau; }
    }
    const uint32_t gi = warp_incl_scan(gt, lane), ei = warp_incl_scan(eq, lane);
    if (lane == 31) { s_wtot[warp][0] = gi; s_wtot[warp][1] = ei; }
    __syncthreads();
    uint32_t gb = gi - gt, eb = ei - eq, g_all = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) {
        if (w < warp) { gb += s_wtot[w][0]; eb += s_wtot[w][1]; }
        g_all += s_wtot[w][0];
    }
    const uint32_t ties = (uint32_t)k - g_all;     // keys equal to tau still to take
    uint32_t pos = gb + min(eb, ties);
    if (REG) {
#pragma unroll
        for (int j = 0; j < kKpt; ++j) {
            if (lo + j < hi) {
                if (key[j] > tau) ids[pos++] = lo + j;
                else if (key[j] == tau) { if (eb < ties) ids[pos++] = lo + j; ++eb; }
            }
        }
    } else {
        for (int i = lo; i < hi; ++i) {
            const uint32_t x = key_at(i);
            if (x > tau) ids[pos++] = i;
            else if (x == tau) { if (eb < ties) ids[pos++] = i; ++eb; }
        }
    }
    __syncthreads();                               // shared scratch is reused by the next call
}

__device__ __forceinline__ uint64_t pack2(float lo, float hi) {
    uint64_t r;
    asm("mov.b64 %0, {%1,%2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ float sum2(uint64_t v) {
    float lo, hi;
    asm("mov.b64 {%0,%1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
    return lo + hi;
}
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c) {
    uint64_t d;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(d) : "l"(a), "l"(b), "l"(c));
    return d;
}

// Lane sums of NH heads -> max over heads of the 16-lane totals (pairing at
// distances 8, 4, 2, 1).  hm = the lanes of this half-warp.
template <int NH>
__device__ __forceinline__ float reduce_heads(float (&v)[NH], int l, unsigned hm) {
    static_assert(NH == 1 || NH == 2 || NH == 4, "head count is padded to a power of two");
    float x;
    if (NH == 4) {
        const bool up8 = l & 8, up4 = l & 4;
        float k0 = up8 ? v[2] : v[0], k1 = up8 ? v[3] : v[1];
        k0 += __shfl_xor_sync(hm, up8 ? v[0] : v[2], 8);
        k1 += __shfl_xor_sync(hm, up8 ? v[1] : v[3], 8);
        x = (up4 ? k1 : k0) + __shfl_xor_sync(hm, up4 ? k0 : k1, 4);
    } else if (NH == 2) {
        const bool up8 = l & 8;
        x = (up8 ? v[1] : v[0]) + __shfl_xor_sync(hm, up8 ? v[0] : v[1], 8);
        x += __shfl_xor_sync(hm, x, 4);
    } else {
        x = v[0] + __shfl_xor_sync(hm, v[0], 8);
        x += __shfl_xor_sync(hm, x, 4);
    }
    x += __shfl_xor_sync(hm, x, 2);
    x += __shfl_xor_sync(hm, x, 1);
    if (NH >= 2) x = fmaxf(x, __shfl_xor_sync(hm, x, 8));
    if (NH == 4) x = fmaxf(x, __shfl_xor_sync(hm, x, 4));
    return x;
}

template <int GQ>
__global__ void __launch_bounds__(kThreads, kCtasPerSm)
quest_select_kernel(const uint4* __restrict__ kmin, const uint4* __restrict__ kmax,
                    const uint4* __restrict__ q, const int32_t* __restrict__ seq_len, int Hq, int Hkv,
                    int T, int P, int token_budget, int max_pages, int32_t* __restrict__ page_ids,
                    int32_t* __restrict__ n_pages, float* __restrict__ scores, int scores_wanted,
                    unsigned* __restrict__ counters, int units_per_problem, long long total_units) {
    constexpr bool kSplit = GQ > 4;            // halves of a warp share a page, split the heads
    constexpr int NH = kSplit ? 4 : (GQ == 3 ? 4 : GQ);   // heads per lane, padded to 1 / 2 / 4
    constexpr int kPagesPerUnit = kWarps * (kSplit ? 1 : 2);

    extern __shared__ uint32_t ring_mem[];
    __shared__ int s_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int half = lane >> 4, l = lane & 15;
    const int sub = kSplit ? warp : warp * 2 + half;       // this half-warp's page inside a unit
    const unsigned hm = kSplit ? 0xFFFFFFFFu : (0xFFFFu << (16 * half));
    const long long x1 = total_units * (blockIdx.x + 1) / gridDim.x;
    long long x = total_units * blockIdx.x / gridDim.x;

    // ring slot: per warp 512 B of kmin chunks then 512 B of kmax chunks (conflict-free)
    const uint32_t ring = smem_u32(ring_mem) + (uint32_t)warp * 1024u + (uint32_t)lane * 16u;
    constexpr uint32_t kSlotBytes = kThreads * 32u;

#pragma unroll 1
    while (x < x1) {
        // ---- one segment: this CTA's units of one problem -------------------------
        const int problem = (int)(x / units_per_problem);
        const int u_begin = (int)(x - (long long)problem * units_per_problem);
        const int n = (int)min((long long)(units_per_problem - u_begin), x1 - x);
        x += n;
        const int b = problem / Hkv, hk = problem - b * Hkv;
        const int len = clamp_len(seq_len, b, T);
        const int np = (len + kPage - 1) / kPage;
        const int k_pg = min(token_budget / kPage, min(np, max_pages));
        const bool trivial = (k_pg >= np) || (k_pg <= 0);
        if (trivial && u_begin == 0) {             // every page kept (or none): no scores needed
            int32_t* ids = page_ids + (size_t)problem * max_pages;
            for (int i = tid; i < k_pg; i += kThreads) ids[i] = i;
            if (tid == 0) n_pages[problem] = max(k_pg, 0);
        }
        if (trivial && !scores_wanted) continue;

        const size_t row0 = (size_t)problem * P;
        auto issue = [&](int i) {                 // unit i of the segment -> slot i % kDepth
            const int page = (u_begin + i) * kPagesPerUnit + sub;
            if (i < n && page < np) {
                const uint32_t dst = ring + (uint32_t)(i % kDepth) * kSlotBytes;
                const size_t src = (row0 + page) * kOctets + l;
                cp_async16(dst, kmin + src);
                cp_async16(dst + 512u, kmax + src);
            }
            cp_async_commit();
        };
#pragma unroll
        for (int i = 0; i < kDepth; ++i) issue(i);

        uint64_t qp2[NH][4], qn2[NH][4];           // (even, odd) channel pairs of q+ and q-
#pragma unroll
        for (int h = 0; h < NH; ++h) {
            const int head = min(kSplit ? half * 4 + h : h, GQ - 1);   // padding repeats a real head
            const uint4 qw = q[((size_t)b * Hq + (size_t)hk * GQ + head) * kOctets + l];
            const uint32_t w[4] = {qw.x, qw.y, qw.z, qw.w};
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float e = bf16lo(w[i]), o = bf16hi(w[i]);
                qp2[h][i] = pack2(fmaxf(e, 0.f), fmaxf(o, 0.f));
                qn2[h][i] = pack2(fminf(e, 0.f), fminf(o, 0.f));
            }
        }
        auto score_unit = [&](int i, const uint4& lo, const uint4& hi) {
            const int page = (u_begin + i) * kPagesPerUnit + sub;
            const uint32_t wl[4] = {lo.x, lo.y, lo.z, lo.w}, wh[4] = {hi.x, hi.y, hi.z, hi.w};
            uint64_t a2[4], z2[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                a2[c] = pack2(bf16lo(wl[c]), bf16hi(wl[c]));
                z2[c] = pack2(bf16lo(wh[c]), bf16hi(wh[c]));
            }
            float v[NH];
#pragma unroll
            for (int h = 0; h < NH; ++h) {
                uint64_t acc = pack2(0.f, 0.f);
#pragma unroll
                for (int c = 0; c < 4; ++c) acc = fma2(qp2[h][c], z2[c], fma2(qn2[h][c], a2[c], acc));
                v[h] = sum2(acc);
            }
            float best = reduce_heads<NH>(v, l, hm);
            if (kSplit) best = fmaxf(best, __shfl_xor_sync(0xFFFFFFFFu, best, 16));
            if (l == 0 && (!kSplit || half == 0) && i < n && page < np) scores[row0 + page] = best;
        };

#pragma unroll 1
        for (int i = 0; i < n; i += 2) {
            cp_async_wait<kDepth - 2>();           // units i and i+1 have landed
            const uint32_t s0 = ring + (uint32_t)(i % kDepth) * kSlotBytes;
            const uint32_t s1 = ring + (uint32_t)((i + 1) % kDepth) * kSlotBytes;
            const uint4 lo0 = lds16(s0), hi0 = lds16(s0 + 512u);
            const uint4 lo1 = lds16(s1), hi1 = lds16(s1 + 512u);
            score_unit(i, lo0, hi0);
            score_unit(i + 1, lo1, hi1);
            issue(i + kDepth);                     // refill the two slots just read
            issue(i + kDepth + 1);
        }
        cp_async_wait<0>();
        if (trivial) continue;

        // ---- whoever completes the problem's unit count selects its pages ---------
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const unsigned old = atomicAdd(&counters[problem], (unsigned)n);
            s_last = (old + (unsigned)n == (unsigned)units_per_problem);
        }
        __syncthreads();
        if (s_last) {
            __threadfence();
            int32_t* ids = page_ids + (size_t)problem * max_pages;
            if (np <= kRegKeys) block_topk<true>(scores + row0, np, k_pg, ids);
            else                block_topk<false>(scores + row0, np, k_pg, ids);
            if (tid == 0) n_pages[problem] = k_pg;
        }
    }
}

size_t counters_bytes(const Geom& g) { return (((size_t)g.problems * 4) + 255) & ~(size_t)255; }

int sm_count() {
    static int n = 0;
    if (n == 0) {
        int dev = 0;
        if (cudaGetDevice(&dev) != cudaSuccess ||
            cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0)
            n = 148;
    }
    return n;
}

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
    const int pages_per_unit = kWarps * (g.Gq > 4 ? 1 : 2);
    const int units_per_problem = (g.P + pages_per_unit - 1) / pages_per_unit;
    const long long total_units = (long long)units_per_problem * g.problems;
    long long grid = (long long)sm_count() * kCtasPerSm;
    if (grid > total_units) grid = total_units;
#define STC_SEL(GQ_)                                                                                 \
    case GQ_:                                                                                        \
        cudaFuncSetAttribute(quest_select_kernel<GQ_>, cudaFuncAttributeMaxDynamicSharedMemorySize,  \
                             (int)kRingBytes);                                                       \
        quest_select_kernel<GQ_><<<(unsigned)grid, kThreads, kRingBytes, st>>>(                      \
            static_cast<const uint4*>(kmin), static_cast<const uint4*>(kmax),                        \
            static_cast<const uint4*>(q), g.seq_len, g.Hq, g.Hkv, g.T, g.P, token_budget,            \
            max_pages, page_ids, n_pages, scores, scores_opt != nullptr, counters,                   \
            units_per_problem, total_units);                                                         \
        break;
    switch (g.Gq) {
        STC_SEL(1) STC_SEL(2) STC_SEL(3) STC_SEL(4) STC_SEL(5) STC_SEL(6) STC_SEL(7) STC_SEL(8)
        default: return cudaErrorInvalidValue;
    }
#undef STC_SEL
    return cudaGetLastError();
}

}  // namespace stc
