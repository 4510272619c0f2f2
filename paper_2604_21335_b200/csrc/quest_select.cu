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
// counter; whoever completes the count (no waiting) selects the pages: radix
// select of the k-th largest order-preserving key on the bits the problem's keys
// actually differ in, then an ordered compaction that emits ids ascending and
// resolves ties at the threshold in favour of lower page ids (see block_topk).
#include "common.cuh"

namespace stc {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kCtasPerSm = 2;
constexpr int kDepth = 8;                    // (a power of two)                    // units in flight per lane (32 B each)
constexpr size_t kRingBytes = (size_t)kDepth * kThreads * 32;

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, int lane) {
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t o = __shfl_up_sync(0xFFFFFFFFu, v, d);
        if (lane >= d) v += o;
    }
    return v;
}

// Top-k of u[0..n) by (value descending, index ascending); ids written ascending.
// Requires 0 < k < n.  All kThreads threads of the CTA call it.  `skeys` is shared
// memory for kSmemKeys keys that nothing else uses during the call; `sh` is
// kTopkSmemWords words of shared scratch.
//
// Keys are the order-preserving integer images of the scores, staged once in
// shared memory (longer rows re-read the scores from L2 instead).  Warp w owns the
// contiguous index block [w*per_warp, (w+1)*per_warp); inside it lane l visits
// l, l+32, ...  The code runs once per problem, so every phase is a short rolled
// loop (straight-line code that is executed once costs an instruction-cache miss
// per line):
//   1. block min / max of the keys: the leading bits on which they agree need no
//      search (scores of one problem share sign and exponent almost always);
//   2. radix select of the k-th largest key on the bits that do vary, 8 bits per
//      pass, histogram in shared memory (the worst case, every key in one bin, is
//      32 serialised updates per warp instruction: microseconds, not more); as soon
//      as at most kRankMax candidates share the selected prefix they are gathered
//      and ranked directly, which ends the search;
//   3. ordered compaction: keys above the threshold, plus the first
//      k - #above keys equal to it in index order, ballot-ranked per warp.
constexpr int kRankMax = 64;
constexpr int kTopkSmemWords = 256 /*hist*/ + kRankMax /*candidates*/ + 2 * kWarps + 8 /*scalars*/;
constexpr int kSmemKeys = (int)(kRingBytes / 4);

__device__ __noinline__ void block_topk(const float* __restrict__ u, int n, int k, int32_t* __restrict__ ids,
                                        uint32_t* __restrict__ skeys, uint32_t* __restrict__ sh) {
    uint32_t* hist = sh;
    uint32_t* cbuf = sh + 256;
    uint32_t* sc = sh + 256 + kRankMax;         // [kWarps] warp mins, [kWarps] warp maxs / totals, then results
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // Warp w owns the index block [w*per_warp, (w+1)*per_warp); a lane visits groups of four
    // consecutive keys (one 16-byte read), group j*32 + lane in pass j.  Slots past n hold key 0,
    // which is below every real key, so it can never be selected (k < n).
    const int per_warp = ((n + kWarps * 128 - 1) / (kWarps * 128)) * 128;
    const int J = per_warp / 128;                // groups per lane
    const int padded = per_warp * kWarps;
    const unsigned lt = (1u << lane) - 1u;
    const bool staged = padded <= kSmemKeys;

    // ---- 1. stage the keys, block min / max on the way ----------------------------------------
    uint32_t kmn = 0xFFFFFFFFu, kmx = 0u;
    if (staged) {
        // up to eight groups per thread in flight (one round trip to L2 for 8192 keys)
        const bool vec = (reinterpret_cast<uintptr_t>(u) & 15u) == 0;
#pragma unroll 1
        for (int g0 = tid; g0 < padded / 4; g0 += 8 * kThreads) {
            uint4 raw[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int i = 4 * (g0 + e * kThreads);
                raw[e] = make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu);   // -NaN: key 0
                if (vec && i + 3 < n) {
                    raw[e] = __ldcg(reinterpret_cast<const uint4*>(u + i));
                } else {
                    if (i < n) raw[e].x = __float_as_uint(__ldcg(u + i));
                    if (i + 1 < n) raw[e].y = __float_as_uint(__ldcg(u + i + 1));
                    if (i + 2 < n) raw[e].z = __float_as_uint(__ldcg(u + i + 2));
                    if (i + 3 < n) raw[e].w = __float_as_uint(__ldcg(u + i + 3));
                }
            }
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int i = 4 * (g0 + e * kThreads);
                if (i >= padded) continue;
                const uint32_t w4[4] = {raw[e].x, raw[e].y, raw[e].z, raw[e].w};
                uint32_t x[4];
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    x[c] = i + c < n ? float_key(__uint_as_float(w4[c])) : 0u;
                    if (i + c < n) { kmn = min(kmn, x[c]); kmx = max(kmx, x[c]); }
                }
                *reinterpret_cast<uint4*>(skeys + i) = make_uint4(x[0], x[1], x[2], x[3]);
            }
        }
    }
    // fn(keys[4], first index) for every group of this lane; all lanes call it J times
    auto for_each = [&](auto&& fn) {
#pragma unroll 2
        for (int j = 0; j < J; ++j) {
            const int i0 = warp * per_warp + (j * 32 + lane) * 4;
            uint32_t x[4];
            if (staged) {
                const uint4 v = *reinterpret_cast<const uint4*>(skeys + i0);
                x[0] = v.x; x[1] = v.y; x[2] = v.z; x[3] = v.w;
            } else {
#pragma unroll
                for (int e = 0; e < 4; ++e) x[e] = i0 + e < n ? float_key(__ldcg(u + i0 + e)) : 0u;
            }
            fn(x, i0);
        }
    };
    if (!staged)
        for_each([&](const uint32_t (&x)[4], int i0) {
#pragma unroll
            for (int e = 0; e < 4; ++e) if (i0 + e < n) { kmn = min(kmn, x[e]); kmx = max(kmx, x[e]); }
        });
    kmn = __reduce_min_sync(0xFFFFFFFFu, kmn);
    kmx = __reduce_max_sync(0xFFFFFFFFu, kmx);
    if (lane == 0) { sc[warp] = kmn; sc[kWarps + warp] = kmx; }
    __syncthreads();
#pragma unroll
    for (int w2 = 0; w2 < kWarps; ++w2) { kmn = min(kmn, sc[w2]); kmx = max(kmx, sc[kWarps + w2]); }

    // ---- 2. k-th largest key -----------------------------------------------------------------
    int bits_left = 32 - __clz(kmn ^ kmx);       // low bits that differ somewhere (0: all keys equal)
    uint32_t fixed_mask = bits_left >= 32 ? 0u : ~((1u << bits_left) - 1u);
    uint32_t fixed_val = kmx & fixed_mask;
    uint32_t krem = (uint32_t)k, cand = (uint32_t)n;
    uint32_t tau = kmx;
    bool found = bits_left == 0;
#pragma unroll 1
    while (!found) {
        __syncthreads();                          // previous readers of hist / scalars are done
        if (cand <= (uint32_t)kRankMax) {
            // gather the candidates and rank them directly
            if (tid == 0) sc[2 * kWarps] = 0u;
            __syncthreads();
            for_each([&](const uint32_t (&x)[4], int) {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (x[e] != 0u && (x[e] & fixed_mask) == fixed_val) cbuf[atomicAdd(&sc[2 * kWarps], 1u)] = x[e];
            });
            __syncthreads();
            if ((uint32_t)tid < cand) {
                const uint32_t x = cbuf[tid];
                uint32_t g = 0, e = 0;
#pragma unroll 4
                for (uint32_t i = 0; i < cand; ++i) { const uint32_t y = cbuf[i]; g += y > x; e += y == x; }
                if (g < krem && krem <= g + e) sc[2 * kWarps + 1] = x;   // every thread that qualifies holds the same key
            }
            __syncthreads();
            tau = sc[2 * kWarps + 1];
            break;
        }
        const int nb = bits_left < 8 ? bits_left : 8, shift = bits_left - nb;
        const uint32_t dmask = (1u << nb) - 1u;
        if (tid < 256) hist[tid] = 0u;
        __syncthreads();
        for_each([&](const uint32_t (&x)[4], int) {
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (x[e] != 0u && (x[e] & fixed_mask) == fixed_val) atomicAdd(&hist[(x[e] >> shift) & dmask], 1u);
        });
        __syncthreads();
        if (warp == 0) {                          // bin holding the krem-th largest candidate
            uint32_t c8[8], sum = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) { c8[i] = hist[255 - 8 * lane - i]; sum += c8[i]; }
            const uint32_t incl = warp_incl_scan(sum, lane), excl = incl - sum;
            if (excl < krem && krem <= incl) {
                uint32_t run = excl;
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    if (run < krem && krem <= run + c8[i]) {
                        sc[2 * kWarps + 2] = 255 - 8 * lane - i; sc[2 * kWarps + 3] = krem - run; sc[2 * kWarps + 4] = c8[i];
                    }
                    run += c8[i];
                }
            }
        }
        __syncthreads();
        const uint32_t digit = sc[2 * kWarps + 2];
        krem = sc[2 * kWarps + 3]; cand = sc[2 * kWarps + 4];
        fixed_mask |= dmask << shift;
        fixed_val |= digit << shift;
        bits_left = shift;
        if (bits_left == 0) { tau = fixed_val; found = true; }
    }

    // ---- 3. ordered compaction ---------------------------------------------------------------
    // counts packed as (#above) | (#equal) << 16 : a warp holds at most 4096 keys per pass
    uint32_t gt = 0, eq = 0;
    for_each([&](const uint32_t (&x)[4], int) {
#pragma unroll
        for (int e = 0; e < 4; ++e) { gt += x[e] > tau; eq += x[e] == tau; }
    });
    gt = __reduce_add_sync(0xFFFFFFFFu, gt);
    eq = __reduce_add_sync(0xFFFFFFFFu, eq);
    __syncthreads();
    if (lane == 0) { sc[warp] = gt; sc[kWarps + warp] = eq; }
    __syncthreads();
    uint32_t run_gt = 0, run_eq = 0, all_gt = 0;
#pragma unroll
    for (int w2 = 0; w2 < kWarps; ++w2) {
        if (w2 < warp) { run_gt += sc[w2]; run_eq += sc[kWarps + w2]; }
        all_gt += sc[w2];
    }
    const uint32_t ties = (uint32_t)k - all_gt;   // keys equal to tau still to take, lowest indices first
    for_each([&](const uint32_t (&x)[4], int i0) {
        uint32_t mine = 0;                        // this lane's four keys: #above | #equal << 16
#pragma unroll
        for (int e = 0; e < 4; ++e) mine += (x[e] > tau) + ((uint32_t)(x[e] == tau) << 16);
        const uint32_t incl = warp_incl_scan(mine, lane), before = incl - mine;
        uint32_t g_before = run_gt + (before & 0xFFFFu), e_before = run_eq + (before >> 16);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (x[e] > tau) { ids[g_before + min(e_before, ties)] = i0 + e; ++g_before; }
            else if (x[e] == tau) { if (e_before < ties) ids[g_before + e_before] = i0 + e; ++e_before; }
        }
        const uint32_t tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
        run_gt += tot & 0xFFFFu; run_eq += tot >> 16;
    });
    __syncthreads();                              // the scratch may be reused by the caller
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
                    int T, int P, int token_budget, int n_recent, int max_pages, int32_t* __restrict__ page_ids,
                    int32_t* __restrict__ n_pages, float* __restrict__ scores, int scores_wanted,
                    unsigned* __restrict__ counters, int units_per_problem, long long total_units) {
    constexpr bool kSplit = GQ > 4;            // halves of a warp share a page, split the heads
    constexpr int NH = kSplit ? 4 : (GQ == 3 ? 4 : GQ);   // heads per lane, padded to 1 / 2 / 4
    constexpr int kPagesPerUnit = kWarps * (kSplit ? 1 : 2);

    extern __shared__ __align__(16) uint32_t ring_mem[];
    __shared__ uint32_t s_topk[kTopkSmemWords];
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
        // units of the segment in which this half-warp's page exists (pages advance by
        // kPagesPerUnit per unit, so validity is a prefix of the units)
        const int page0 = u_begin * kPagesPerUnit + sub;
        const int lim = max(0, min(n, (np - page0 + kPagesPerUnit - 1) / kPagesPerUnit));
        // running source pointers / ring slot of the next unit to issue (units are issued in order)
        const uint4* src_min = kmin + (row0 + page0) * kOctets + l;
        const uint4* src_max = kmax + (row0 + page0) * kOctets + l;
        uint32_t slot_off = 0;
        auto issue = [&](int i) {                 // unit i of the segment -> slot i % kDepth
            if (i < lim) {
                cp_async16(ring + slot_off, src_min);
                cp_async16(ring + slot_off + 512u, src_max);
            }
            cp_async_commit();
            src_min += kPagesPerUnit * kOctets;
            src_max += kPagesPerUnit * kOctets;
            slot_off = (slot_off + kSlotBytes) & (kDepth * kSlotBytes - 1u);
        };
        float* dst_score = scores + row0 + page0;
        const bool writer = l == 0 && (!kSplit || half == 0);
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
            if (writer && i < lim) *dst_score = best;
            dst_score += kPagesPerUnit;
        };

#pragma unroll 1
        for (int i = 0; i < n; i += 2) {
            cp_async_wait<kDepth - 2>();           // units i and i+1 have landed
            const uint32_t s0 = ring + (uint32_t)(i & (kDepth - 1)) * kSlotBytes;
            const uint32_t s1 = ring + (uint32_t)((i + 1) & (kDepth - 1)) * kSlotBytes;
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
            // the copy ring is idle here (all copies have landed): it stages the keys
            // the local window: the last w pages are kept, the rest of the budget goes to the pages before them
            const int w = min(max(n_recent, 0), k_pg);
            if (k_pg > w) block_topk(scores + row0, np - w, k_pg - w, ids, ring_mem, s_topk);
            for (int i = tid; i < w; i += kThreads) ids[k_pg - w + i] = np - w + i;
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
                                int token_budget, int n_recent_pages, int max_pages, int32_t* page_ids,
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
            n_recent_pages, max_pages, page_ids, n_pages, scores, scores_opt != nullptr, counters,                   \
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
