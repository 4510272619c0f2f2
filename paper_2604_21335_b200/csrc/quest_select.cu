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
//
// Two scan kernels share that selection code.
//   quest_select_kernel: the bound of every page in the declared fp32 order on the
//     fp32 pipes (what the caller gets when it asks for the scores, and the path for
//     a single query head per KV head).
//   quest_filter_kernel: with several query heads the bound of a tile of 16 pages is
//     one dense contraction [16 pages x 256] . [256 x heads] over [kmax | kmin] and
//     [q+ | q-] with exact bf16 products, so the tensor cores (mma.sync m16n8k16)
//     compute it while the scan stays at HBM speed; their fp32 accumulation order is
//     not the declared one, so those scores only FILTER: a second product on absolute
//     values gives a rigorous margin, pages whose approximate score lies within the
//     margin of the approximate k-th score are re-scored exactly in the declared
//     order, and the exact scores settle membership and ties (see block_topk).
#include "common.cuh"

namespace stc {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kCtasPerSm = 2;
constexpr int kDepth = 8;                    // (a power of two)                    // units in flight per lane (32 B each)
constexpr size_t kRingBytes = (size_t)kDepth * kThreads * 32;


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
constexpr int kMaxWarps = 16;                 // the selection code runs with 256 or 512 threads
constexpr int kTopkSmemWords = 256 /*hist*/ + kRankMax /*candidates*/ + 2 * kMaxWarps + 8 /*scalars*/;
constexpr int kSmemKeys = (int)(kRingBytes / 4);

// Bound of one page in the declared fp32 order, by one half-warp (lane l of the half owns
// channels 8l..8l+7), heads one after the other; all 32 lanes of the warp call it.
__device__ __forceinline__ uint64_t pack2(float lo, float hi);
__device__ __forceinline__ float sum2(uint64_t v);
__device__ __forceinline__ uint64_t fma2(uint64_t a, uint64_t b, uint64_t c);
__device__ __noinline__ float exact_page_score(const uint4* __restrict__ kmin_row, const uint4* __restrict__ kmax_row,
                                               const uint4* __restrict__ q_heads, int gq, int l, unsigned hm);

// What the filtered selection needs to settle the pages near the threshold exactly.
struct FilterCtx {
    const uint4* kmin;       // the problem's first page row
    const uint4* kmax;
    const uint4* q_heads;    // the problem's first query head
    int gq;
    float delta;             // |approximate score - declared-order score| <= delta for every page
    int32_t* amb_idx;        // shared memory: kAmbMax page indices, then kAmbMax keys
    uint32_t* amb_key;
};
constexpr int kAmbMax = 2048;

//
// With a FilterCtx the scores in u are approximations (each within f->delta of the page's
// declared-order score).  After the k-th largest approximate score t is known, a page is
// certainly selected if its approximation exceeds t + 2 delta and certainly not if it is
// below t - 2 delta (the exact k-th score lies within delta of t); the pages in between are
// scored exactly, ranked by (exact score descending, index ascending), and the best of them
// fill the remaining places.  Returns false (nothing written) when more than kAmbMax pages
// fall in between; u may be overwritten.
template <int NT>
__device__ __noinline__ bool block_topk(float* __restrict__ u, int n, int k, int32_t* __restrict__ ids,
                                        uint32_t* __restrict__ skeys, uint32_t* __restrict__ sh,
                                        const FilterCtx* __restrict__ f) {
    constexpr int NW = NT / 32;
    __syncthreads();                              // nobody still reads what an earlier selection left in the scratch
    uint32_t* hist = sh;
    uint32_t* cbuf = sh + 256;
    uint32_t* sc = sh + 256 + kRankMax;         // [NW] warp mins, [NW] warp maxs / totals, then results
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    // Warp w owns the index block [w*per_warp, (w+1)*per_warp); a lane visits groups of four
    // consecutive keys (one 16-byte read), group j*32 + lane in pass j.  Slots past n hold key 0,
    // which is below every real key, so it can never be selected (k < n).
    const int per_warp = ((n + NW * 128 - 1) / (NW * 128)) * 128;
    const int J = per_warp / 128;                // groups per lane
    const int padded = per_warp * NW;
    const unsigned lt = (1u << lane) - 1u;
    const bool staged = padded <= kSmemKeys;

    // ---- 1. stage the keys, block min / max on the way ----------------------------------------
    uint32_t kmn = 0xFFFFFFFFu, kmx = 0u;
    if (staged) {
        // up to eight groups per thread in flight (one round trip to L2 for 8192 keys)
        const bool vec = (reinterpret_cast<uintptr_t>(u) & 15u) == 0;
#pragma unroll 1
        for (int g0 = tid; g0 < padded / 4; g0 += 8 * NT) {
            uint4 raw[8];
#pragma unroll
            for (int e = 0; e < 8; ++e) {
                const int i = 4 * (g0 + e * NT);
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
                const int i = 4 * (g0 + e * NT);
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
    if (lane == 0) { sc[warp] = kmn; sc[NW + warp] = kmx; }
    __syncthreads();
#pragma unroll
    for (int w2 = 0; w2 < NW; ++w2) { kmn = min(kmn, sc[w2]); kmx = max(kmx, sc[NW + w2]); }

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
            if (tid == 0) sc[2 * NW] = 0u;
            __syncthreads();
            for_each([&](const uint32_t (&x)[4], int) {
#pragma unroll
                for (int e = 0; e < 4; ++e)
                    if (x[e] != 0u && (x[e] & fixed_mask) == fixed_val) cbuf[atomicAdd(&sc[2 * NW], 1u)] = x[e];
            });
            __syncthreads();
            if ((uint32_t)tid < cand) {
                const uint32_t x = cbuf[tid];
                uint32_t g = 0, e = 0;
#pragma unroll 4
                for (uint32_t i = 0; i < cand; ++i) { const uint32_t y = cbuf[i]; g += y > x; e += y == x; }
                if (g < krem && krem <= g + e) sc[2 * NW + 1] = x;   // every thread that qualifies holds the same key
            }
            __syncthreads();
            tau = sc[2 * NW + 1];
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
                        sc[2 * NW + 2] = 255 - 8 * lane - i; sc[2 * NW + 3] = krem - run; sc[2 * NW + 4] = c8[i];
                    }
                    run += c8[i];
                }
            }
        }
        __syncthreads();
        const uint32_t digit = sc[2 * NW + 2];
        krem = sc[2 * NW + 3]; cand = sc[2 * NW + 4];
        fixed_mask |= dmask << shift;
        fixed_val |= digit << shift;
        bits_left = shift;
        if (bits_left == 0) { tau = fixed_val; found = true; }
    }

    // ---- 2b. filtered scores: settle the pages near the threshold exactly ---------------------
    if (f) {
        const float tf = key_float(tau), pad = 2.0f * f->delta;
        const uint32_t key_hi = float_key(tf + pad), key_lo = float_key(tf - pad);
        __syncthreads();
        if (tid == 0) { sc[2 * NW] = 0u; sc[2 * NW + 1] = 0u; }
        __syncthreads();
        uint32_t n_in = 0;
        for_each([&](const uint32_t (&x)[4], int i0) {
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (x[e] > key_hi) ++n_in;
                else if (x[e] >= key_lo && x[e] != 0u) {
                    const uint32_t pos = atomicAdd(&sc[2 * NW], 1u);
                    if (pos < (uint32_t)kAmbMax) f->amb_idx[pos] = i0 + e;
                }
            }
        });
        n_in = __reduce_add_sync(0xFFFFFFFFu, n_in);
        if (lane == 0) atomicAdd(&sc[2 * NW + 1], n_in);
        __syncthreads();
        const int n_amb = (int)sc[2 * NW];
        const int need = k - (int)sc[2 * NW + 1];      // 1 <= need <= n_amb
        if (n_amb > kAmbMax) return false;
        {
            const int half = lane >> 4, l = lane & 15;
            const unsigned hm = 0xFFFFu << (16 * half);
#pragma unroll 1
            for (int e0 = 0; e0 < n_amb; e0 += 2 * NW) {
                const int e = e0 + warp * 2 + half;
                const int idx = f->amb_idx[min(e, n_amb - 1)];
                const float sx = exact_page_score(f->kmin + (size_t)idx * kOctets, f->kmax + (size_t)idx * kOctets,
                                                  f->q_heads, f->gq, l, hm);
                if (l == 0 && e < n_amb) f->amb_key[e] = float_key(sx);
            }
        }
        __syncthreads();
#pragma unroll 1
        for (int e = tid; e < n_amb; e += NT) {
            const uint32_t kx = f->amb_key[e];
            const int ix = f->amb_idx[e];
            int rank = 0;
#pragma unroll 4
            for (int o = 0; o < n_amb; ++o) {
                const uint32_t ko = f->amb_key[o];
                rank += (ko > kx) || (ko == kx && f->amb_idx[o] < ix);
            }
            const bool chosen = rank < need;
            if (staged) skeys[ix] = chosen ? 0xFFFFFFFFu : 0u;
            else u[ix] = chosen ? INFINITY : -INFINITY;
        }
        __threadfence_block();
        __syncthreads();
        tau = key_hi;                                      // selected = key above key_hi; no ties left
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
    if (lane == 0) { sc[warp] = gt; sc[NW + warp] = eq; }
    __syncthreads();
    uint32_t run_gt = 0, run_eq = 0, all_gt = 0;
#pragma unroll
    for (int w2 = 0; w2 < NW; ++w2) {
        if (w2 < warp) { run_gt += sc[w2]; run_eq += sc[NW + w2]; }
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
            // (every position is below k by construction; the comparison keeps a wrong count from ever
            // becoming a write past the caller's list)
            if (x[e] > tau) {
                const uint32_t pos = g_before + min(e_before, ties);
                if (pos < (uint32_t)k) ids[pos] = i0 + e;
                ++g_before;
            } else if (x[e] == tau) {
                if (e_before < ties && g_before + e_before < (uint32_t)k) ids[g_before + e_before] = i0 + e;
                ++e_before;
            }
        }
        const uint32_t tot = __shfl_sync(0xFFFFFFFFu, incl, 31);
        run_gt += tot & 0xFFFFu; run_eq += tot >> 16;
    });
    __syncthreads();                              // the scratch may be reused by the caller
    return true;
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

__device__ __noinline__ float exact_page_score(const uint4* __restrict__ kmin_row, const uint4* __restrict__ kmax_row,
                                               const uint4* __restrict__ q_heads, int gq, int l, unsigned hm) {
    const uint4 lo = __ldg(kmin_row + l), hi = __ldg(kmax_row + l);
    float best = -INFINITY;
#pragma unroll 1
    for (int h0 = 0; h0 < gq; h0 += 4) {          // four heads' query chunks in flight at a time
        uint4 qw[4];
#pragma unroll
        for (int i = 0; i < 4; ++i) qw[i] = __ldg(q_heads + (size_t)min(h0 + i, gq - 1) * kOctets + l);
        const uint32_t wl[4] = {lo.x, lo.y, lo.z, lo.w}, wh[4] = {hi.x, hi.y, hi.z, hi.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {              // (a repeated last head leaves the maximum unchanged)
            const uint32_t w[4] = {qw[i].x, qw[i].y, qw[i].z, qw[i].w};
            uint64_t acc = pack2(0.f, 0.f);
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                const float e = bf16lo(w[c]), o = bf16hi(w[c]);
                acc = fma2(pack2(fmaxf(e, 0.f), fmaxf(o, 0.f)), pack2(bf16lo(wh[c]), bf16hi(wh[c])),
                           fma2(pack2(fminf(e, 0.f), fminf(o, 0.f)), pack2(bf16lo(wl[c]), bf16hi(wl[c])), acc));
            }
            float x = sum2(acc);
            x += __shfl_xor_sync(hm, x, 8);
            x += __shfl_xor_sync(hm, x, 4);
            x += __shfl_xor_sync(hm, x, 2);
            x += __shfl_xor_sync(hm, x, 1);
            best = fmaxf(best, x);
        }
    }
    return best;
}

// ---- the tensor-core scan ------------------------------------------------------------------
// A warp owns a tile of 16 consecutive pages; a unit is the 16 tiles of a CTA (256 pages).
// A tile is two contiguous 4 KiB blocks (16 rows of kmax, 16 rows of kmin): lane 0 brings them
// into the warp's ring slot with two bulk asynchronous copies that signal the slot's mbarrier
// (sixteen warps per SM, so sixteen tiles are in flight or being reduced at any time), and the
// copies run on across the boundaries between problems; nothing waits on another warp.  Every wait on an mbarrier is
// bounded: a wait that expires records STC_ERR_TIMEOUT in the workspace status word and the
// warp stops issuing copies and skips its arithmetic (the page lists of the call are then
// unspecified, still valid ids).
// Lane (g = lane / 4, t = lane % 4) reads, for j = 0..3, the 16-byte chunk t + 4j of rows g and
// g + 8 of both blocks: the chunk words are A fragments of m16n8k16 as they stand (row = page,
// k = the lane's own channels; the query fragments use the same channel-to-k assignment, and a
// sum over channels does not care about their order):
//   words 0,1 of the chunks of pages g / g+8 -> a0..a3 of one mma, words 2,3 -> of the next.
// Column n of the B operand is query head n (heads past the group repeat real ones, which
// leaves the maximum unchanged): q+ against kmax and q- against kmin give
// sum_c max(q kmin, q kmax); the same products on absolute values give sum_c |term|, whose
// largest value over the problem scales the error margin of the filter.
constexpr int kFilterMinGq = 2;               // single-head problems stay on the fp32 pipes
constexpr int kFilterMinPages = 4096;         // pages per problem from which the filtered scan is the faster one
constexpr int kFilterMinPagesSplit = 1024;    // ... with more than four query heads per KV head
constexpr int kFThreads = 512;                                   // one CTA per SM, 16 warps
constexpr int kFWarps = kFThreads / 32;
constexpr int kFDepth = 1;                                       // ring slots per warp (16 tiles in flight per SM)
constexpr int kFCtasPerSm = 1;
constexpr uint32_t kFTileBytes = 16u * 512u;                     // 8 KiB per tile: kmax rows | kmin rows
constexpr size_t kFRingBytes = (size_t)kFWarps * kFDepth * kFTileBytes;  // 128 KiB
constexpr unsigned long long kFWaitLimitNs = 1000000000ull;
constexpr int kFUnitPages = kFWarps * 16;
constexpr float kMarginRel = 1.0f / 8192.0f;   // 2^-13 of sum|term|: far above the 2^-24-per-add error of either sum

// Shared memory of the selection behind the copy ring (the ring keeps streaming the next
// problem's pages while a problem is being selected), in 32-bit words.
constexpr int kHistBits = 11, kHistBins = 1 << kHistBits;
constexpr int kCandMax = 1024;
constexpr int kSelKeys = 0;                                      // keys [kSmemKeys]
constexpr int kSelHist = kSelKeys + kSmemKeys;                   // histogram [kHistBins]; block_topk: ambiguous list
constexpr int kSelCidx = kSelHist + kHistBins;                   // candidate page indices [kCandMax]
constexpr int kSelCkey = kSelCidx + kCandMax;                    // candidate keys [kCandMax]
constexpr int kSelAmb = kSelCkey + kCandMax;                     // positions of the ambiguous candidates [kCandMax]
constexpr int kSelWords = kSelAmb + kCandMax;
constexpr size_t kFSmemBytes = kFRingBytes + (size_t)kSelWords * 4;
static_assert(kSelWords >= kSmemKeys + 2 * kAmbMax, "block_topk's list of pages to settle fits behind the keys");
static_assert(kFSmemBytes <= 227 * 1024 - 2048, "ring + selection scratch fit one CTA per SM");

// The selection of a filtered problem in few passes (n <= kSmemKeys approximate scores, 0 < k < n;
// key_min / key_max bound the keys of the problem's scores and come from the scan).  Same result
// as block_topk with a FilterCtx; returns false (nothing written, u untouched) whenever a case it
// does not handle turns up, and the caller then takes block_topk.
//   A. one pass stages the keys and builds the histogram of the top kHistBits bits on which the
//      problem's keys differ; a block-wide scan of the bins finds the bin b of the k-th largest key;
//   B. one pass gathers the keys of the bins around b that can hold a key within the margin of the
//      k-th key, and counts, per warp, the keys in the bins above them;
//   C. the k-th largest key t is ranked among the candidates; candidates above t + 2 delta are
//      selected, those below t - 2 delta are not, the rest are scored exactly and ranked by
//      (exact score descending, page ascending); the decisions are written into the staged keys;
//   D. one pass writes the selected pages in ascending order (ballot ranks inside a warp's
//      contiguous block, block offsets from the per-warp counts).
template <int NT>
__device__ __noinline__ bool filter_select_fast(const float* __restrict__ u, int n, int k, int32_t* __restrict__ ids,
                                                uint32_t* __restrict__ sm, uint32_t* __restrict__ sc,
                                                uint32_t key_min, uint32_t key_max,
                                                const FilterCtx* __restrict__ f) {
    uint32_t* skeys = sm + kSelKeys;
    uint32_t* hist = sm + kSelHist;
    int32_t* cidx = reinterpret_cast<int32_t*>(sm + kSelCidx);
    uint32_t* ckey = sm + kSelCkey;
    uint32_t* amb = sm + kSelAmb;
    constexpr int NW = NT / 32, BPT = kHistBins / NT;      // warps; histogram bins per thread in the bin scan
    // scalars: sc[0..NW) warp totals of the bin scan, sc[NW..2NW) selected pages per warp block, then
    enum { kCnt = 2 * NW, kTau, kBin, kAbove, kNin, kNamb };
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int bits_left = 32 - __clz(key_min ^ key_max);
    if (bits_left == 0 || n > kSmemKeys) return false;
    const int nb = bits_left < kHistBits ? bits_left : kHistBits, shift = bits_left - nb;
    const uint32_t dmask = (1u << nb) - 1u;
    const uint32_t fixed = bits_left >= 32 ? 0u : (key_max & ~((1u << bits_left) - 1u));
    const int per_warp = ((n + NW * 128 - 1) / (NW * 128)) * 128;
    const int J = per_warp / 128;
    const unsigned lt = (1u << lane) - 1u;
    const bool vec = (reinterpret_cast<uintptr_t>(u) & 15u) == 0;

    for (int i = tid; i < kHistBins; i += NT) hist[i] = 0u;
    if (tid < 2 * NW + 8) sc[tid] = 0u;
    __syncthreads();

    // ---- A. stage + histogram --------------------------------------------------------------------
#pragma unroll 1
    for (int j0 = 0; j0 < J; j0 += 4) {
        uint4 raw[4];
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            const int i = warp * per_warp + ((j0 + e) * 32 + lane) * 4;
            raw[e] = make_uint4(0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu, 0xFFFFFFFFu);
            if (j0 + e < J) {
                if (vec && i + 3 < n) raw[e] = __ldcg(reinterpret_cast<const uint4*>(u + i));
                else {
                    if (i < n) raw[e].x = __float_as_uint(__ldcg(u + i));
                    if (i + 1 < n) raw[e].y = __float_as_uint(__ldcg(u + i + 1));
                    if (i + 2 < n) raw[e].z = __float_as_uint(__ldcg(u + i + 2));
                    if (i + 3 < n) raw[e].w = __float_as_uint(__ldcg(u + i + 3));
                }
            }
        }
#pragma unroll
        for (int e = 0; e < 4; ++e) {
            if (j0 + e >= J) continue;
            const int i = warp * per_warp + ((j0 + e) * 32 + lane) * 4;
            const uint32_t w4[4] = {raw[e].x, raw[e].y, raw[e].z, raw[e].w};
            uint32_t x[4];
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                x[c] = i + c < n ? float_key(__uint_as_float(w4[c])) : 0u;      // slots past n: key 0, never selected
                if (i + c < n) atomicAdd(&hist[(x[c] >> shift) & dmask], 1u);
            }
            *reinterpret_cast<uint4*>(skeys + i) = make_uint4(x[0], x[1], x[2], x[3]);
        }
    }
    __syncthreads();

    // ---- bin of the k-th largest key: thread t owns bins 2047 - BPT t - i, i = 0..BPT-1 (descending) ----
    {
        uint32_t c8[BPT], sum = 0;
#pragma unroll
        for (int i = 0; i < BPT; ++i) { c8[i] = hist[kHistBins - 1 - BPT * tid - i]; sum += c8[i]; }
        const uint32_t incl_w = warp_incl_scan(sum, lane);
        if (lane == 31) sc[warp] = incl_w;
        __syncthreads();
        uint32_t before = 0;
#pragma unroll
        for (int w2 = 0; w2 < NW; ++w2) if (w2 < warp) before += sc[w2];
        const uint32_t incl = before + incl_w, excl = incl - sum;
        if (excl < (uint32_t)k && (uint32_t)k <= incl) {
            uint32_t run = excl;
#pragma unroll
            for (int i = 0; i < BPT; ++i) {
                if (run < (uint32_t)k && (uint32_t)k <= run + c8[i]) { sc[kBin] = kHistBins - 1 - BPT * tid - i; sc[kAbove] = run; }
                run += c8[i];
            }
        }
        __syncthreads();
    }
    const int bin = (int)sc[kBin];
    const uint32_t above = sc[kAbove];                                   // keys in the bins above `bin`
    // The k-th key t lies in `bin`, so every key within 2 delta of it lies between (lowest value of the bin)
    // - 2 delta and (highest value of the bin) + 2 delta: the bins d_lo..d_hi of those two keys (keys outside
    // the problem's own range do not exist) hold the k-th key and the whole window around it.
    const float pad = 2.0f * f->delta;
    const uint32_t bin_lo_key = fixed | ((uint32_t)bin << shift);
    const uint32_t bin_hi_key = bin_lo_key | ((1u << shift) - 1u);
    const uint32_t k_lo = max(float_key(key_float(bin_lo_key) - pad), key_min);
    const uint32_t k_hi = min(float_key(key_float(bin_hi_key) + pad), key_max);
    const int d_lo = (int)((k_lo >> shift) & dmask), d_hi = (int)((k_hi >> shift) & dmask);
    if (d_lo > bin || d_hi < bin || d_hi - d_lo > 64) return false;      // (non-finite scores)
    uint32_t cnt_gathered = 0, cnt_up = 0;                               // keys in d_lo..d_hi; of them, above `bin`
    for (int d = d_lo; d <= d_hi; ++d) { const uint32_t c = hist[d]; cnt_gathered += c; if (d > bin) cnt_up += c; }
    if (cnt_gathered > (uint32_t)kCandMax) return false;
    const uint32_t krem = (uint32_t)k - above;                           // rank of the k-th key inside its bin

    // ---- B. gather the candidates, count the certainly selected keys per warp block ---------------
    {
        uint32_t wc = 0;
#pragma unroll 2
        for (int j = 0; j < J; ++j) {
            const int i0 = warp * per_warp + (j * 32 + lane) * 4;
            const uint4 v = *reinterpret_cast<const uint4*>(skeys + i0);
            const uint32_t x[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                if (x[e] == 0u) continue;
                const int d = (int)((x[e] >> shift) & dmask);
                if (d > d_hi) ++wc;
                else if (d >= d_lo) {
                    const uint32_t pos = atomicAdd(&sc[kCnt], 1u);
                    if (pos < (uint32_t)kCandMax) { cidx[pos] = i0 + e; ckey[pos] = x[e]; }
                }
            }
        }
        wc = __reduce_add_sync(0xFFFFFFFFu, wc);
        if (lane == 0) sc[NW + warp] = wc;
    }
    __syncthreads();
    const int ncand = (int)sc[kCnt];
    if (ncand > kCandMax) return false;                                  // (cannot happen: the bins were counted)
    // the metadata rows of the candidates are wanted in a moment by the exact re-scoring: start them towards L2
    for (int e = tid; e < 4 * ncand; e += NT) {
        const char* row = reinterpret_cast<const char*>(((e & 2) ? f->kmax : f->kmin) + (size_t)cidx[e >> 2] * kOctets);
        asm volatile("prefetch.global.L2 [%0];" ::"l"(row + 128 * (e & 1)));
    }

    // ---- C. the k-th largest approximate key, then the decision on every candidate -----------------
    for (int e = tid; e < ncand; e += NT) {
        const uint32_t x = ckey[e];
        if ((int)((x >> shift) & dmask) != bin) continue;
        uint32_t gt = 0, eq = 0;
#pragma unroll 4
        for (int o = 0; o < ncand; ++o) { const uint32_t y = ckey[o]; gt += y > x; eq += y == x; }
        gt -= cnt_up;                                                    // the gathered keys of the bins above are all larger
        if (gt < krem && krem <= gt + eq) sc[kTau] = x;                  // every thread that qualifies holds the same key
    }
    __syncthreads();
    const uint32_t tau = sc[kTau];
    const float tf = key_float(tau);
    const uint32_t key_hi = float_key(tf + pad), key_lo = float_key(tf - pad);
    // keys above hi_edge (the largest key of bin d_hi) were counted as certainly selected
    const uint32_t hi_edge = min(fixed | ((uint32_t)d_hi << shift) | ((1u << shift) - 1u), 0xFFFFFFFEu);
    for (int e = tid; e < ncand; e += NT) {
        const uint32_t x = ckey[e];
        const int ix = cidx[e];
        if (x > key_hi) {                                                // certainly selected
            skeys[ix] = 0xFFFFFFFFu;
            atomicAdd(&sc[NW + ix / per_warp], 1u);
            atomicAdd(&sc[kNin], 1u);
        } else if (x >= key_lo) {
            amb[atomicAdd(&sc[kNamb], 1u)] = (uint32_t)e;                // settled below
        } else {
            skeys[ix] = 0u;                                              // certainly not selected
        }
    }
    __syncthreads();
    const int n_amb = (int)sc[kNamb];
    const int need = k - (int)(above - cnt_up) - (int)sc[kNin];          // places left for the ambiguous pages
    if (need < 0 || need > n_amb) return false;                          // (cannot happen; u is still intact)
    {
        const int half = lane >> 4, l = lane & 15;
        const unsigned hm = 0xFFFFu << (16 * half);
#pragma unroll 1
        for (int e0 = 0; e0 < n_amb; e0 += 2 * NW) {
            const int e = e0 + warp * 2 + half;
            const int ce = (int)amb[min(e, n_amb - 1)];
            const int idx = cidx[ce];
            const float sx = exact_page_score(f->kmin + (size_t)idx * kOctets, f->kmax + (size_t)idx * kOctets,
                                              f->q_heads, f->gq, l, hm);
            if (l == 0 && e < n_amb) ckey[ce] = float_key(sx);           // the approximate key is no longer needed
        }
    }
    __syncthreads();
    for (int e = tid; e < n_amb; e += NT) {
        const uint32_t kx = ckey[amb[e]];
        const int ix = cidx[amb[e]];
        int rank = 0;
#pragma unroll 4
        for (int o = 0; o < n_amb; ++o) {
            const uint32_t ko = ckey[amb[o]];
            rank += (ko > kx) || (ko == kx && cidx[amb[o]] < ix);
        }
        const bool chosen = rank < need;
        skeys[ix] = chosen ? 0xFFFFFFFFu : 0u;
        if (chosen) atomicAdd(&sc[NW + ix / per_warp], 1u);
    }
    __syncthreads();

    // ---- D. ordered write ---------------------------------------------------------------------------
    uint32_t base = 0, all = 0;
#pragma unroll
    for (int w2 = 0; w2 < NW; ++w2) { if (w2 < warp) base += sc[NW + w2]; all += sc[NW + w2]; }
    if (all != (uint32_t)k) return false;                                // (cannot happen; u is still intact)
#pragma unroll 2
    for (int j = 0; j < J; ++j) {
        const int i0 = warp * per_warp + (j * 32 + lane) * 4;
        const uint4 v = *reinterpret_cast<const uint4*>(skeys + i0);
        const bool s0 = v.x > hi_edge, s1 = v.y > hi_edge, s2 = v.z > hi_edge, s3 = v.w > hi_edge;
        const unsigned b0 = __ballot_sync(0xFFFFFFFFu, s0), b1 = __ballot_sync(0xFFFFFFFFu, s1);
        const unsigned b2 = __ballot_sync(0xFFFFFFFFu, s2), b3 = __ballot_sync(0xFFFFFFFFu, s3);
        if ((b0 | b1 | b2 | b3) == 0u) continue;
        uint32_t pos = base + __popc(b0 & lt) + __popc(b1 & lt) + __popc(b2 & lt) + __popc(b3 & lt);
        if (s0 && pos < (uint32_t)k) ids[pos] = i0;
        pos += s0;
        if (s1 && pos < (uint32_t)k) ids[pos] = i0 + 1;
        pos += s1;
        if (s2 && pos < (uint32_t)k) ids[pos] = i0 + 2;
        pos += s2;
        if (s3 && pos < (uint32_t)k) ids[pos] = i0 + 3;
        base += __popc(b0) + __popc(b1) + __popc(b2) + __popc(b3);
    }
    __syncthreads();
    return true;
}

__device__ __forceinline__ void mma_bf16_16816(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                               uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

// Per-problem words the scan leaves for the selection (all start at zero).
struct ProblemStats {
    unsigned* counters;      // units scanned so far
    unsigned* absmax;        // largest sum|term| (bits of a non-negative float)
    unsigned* keymax;        // largest score key
    unsigned* keymin_inv;    // ~(smallest score key)
};

template <int GQ>
__global__ void __launch_bounds__(kFThreads, kFCtasPerSm)
quest_filter_kernel(const uint4* __restrict__ kmin, const uint4* __restrict__ kmax,
                    const uint4* __restrict__ q, const int32_t* __restrict__ seq_len, int Hq, int Hkv,
                    int T, int P, int token_budget, int n_recent, int max_pages, int32_t* __restrict__ page_ids,
                    int32_t* __restrict__ n_pages, float* __restrict__ scores, const ProblemStats st,
                    int32_t* __restrict__ status, int units_per_problem, long long total_units) {
    extern __shared__ __align__(128) uint32_t ring_mem[];
    __shared__ uint32_t s_topk[kTopkSmemWords];
    __shared__ __align__(8) unsigned long long s_bars[kFWarps * kFDepth];
    __shared__ int s_last;
    uint32_t* sel_mem = ring_mem + kFRingBytes / 4;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const long long x1 = total_units * (blockIdx.x + 1) / gridDim.x;
    long long x = total_units * blockIdx.x / gridDim.x;
    // this warp's ring slots and their barriers; a lane's chunk t of row g inside a 4 KiB block
    const uint32_t ring = smem_u32(ring_mem) + (uint32_t)warp * (kFDepth * kFTileBytes);
    const uint32_t bars = smem_u32(s_bars) + (uint32_t)warp * (kFDepth * 8u);
    const uint32_t frag = (uint32_t)g * 256u + (uint32_t)t * 16u;
    constexpr uint32_t kAbs = 0x7FFF7FFFu;
    if (lane == 0) {
#pragma unroll
        for (int i = 0; i < kFDepth; ++i) mbar_init(bars + 8u * i, 1);
        fence_mbar_init();
    }
    __syncthreads();

    // What a cursor over the CTA's units knows about the problem it is in.
    struct Seg {
        int problem, np, k_pg, u_begin, n;       // n units of `problem` from unit u_begin on; n = 0: past the end
        bool trivial;                            // every page kept (or none): nothing to scan
    };
    auto seg_at = [&](long long xx) {
        Seg s{0, 0, 0, 0, 0, true};
        if (xx >= x1) return s;
        s.problem = (int)(xx / units_per_problem);
        s.u_begin = (int)(xx - (long long)s.problem * units_per_problem);
        s.n = (int)min((long long)(units_per_problem - s.u_begin), x1 - xx);
        const int len = clamp_len(seq_len, s.problem / Hkv, T);
        s.np = (len + kPage - 1) / kPage;
        s.k_pg = min(token_budget / kPage, min(s.np, max_pages));
        s.trivial = (s.k_pg >= s.np) || (s.k_pg <= 0);
        return s;
    };

    // ---- the copy stream: its own cursor over the CTA's units; it skips the problems that need
    //      no scan.  A tile with no valid page issues nothing (the reader skips it the same way).
    long long xi = x;
    Seg si = seg_at(xi);
    int ui = 0;                                   // unit of si being issued
    int slot_issue = 0;
    bool dead = false;                            // a wait expired: stop copying and computing
    auto issue = [&](bool reuse) {
        while (si.n > 0 && (si.trivial || ui == si.n)) { xi += si.n; si = seg_at(xi); ui = 0; }
        if (si.n > 0) {
            const int page0 = (si.u_begin + ui) * kFUnitPages + warp * 16;
            const int nv = min(16, si.np - page0);
            if (nv > 0 && !dead && lane == 0) {
                const size_t row = (size_t)si.problem * P + page0;
                const uint32_t dst = ring + (uint32_t)slot_issue * kFTileBytes, bar = bars + 8u * slot_issue;
                (void)reuse;   // the slot's earlier reads have returned their data (the warp has used it)
                mbar_expect_tx(bar, (uint32_t)nv * 512u);
                bulk_g2s(dst, kmax + row * kOctets, (uint32_t)nv * 256u, bar);
                bulk_g2s(dst + 4096u, kmin + row * kOctets, (uint32_t)nv * 256u, bar);
            }
            ++ui;
        }
        slot_issue = slot_issue + 1 == kFDepth ? 0 : slot_issue + 1;
    };
#pragma unroll
    for (int i = 0; i < kFDepth; ++i) issue(false);
    int slot_rd = 0;
    uint32_t phase = 0;                           // bit s = parity to wait for on slot s

#pragma unroll 1
    while (x < x1) {
        // ---- one segment: this CTA's units of one problem -------------------------
        const Seg sg = seg_at(x);
        const int problem = sg.problem, n = sg.n, np = sg.np, k_pg = sg.k_pg;
        x += n;
        if (sg.trivial) {                          // no scores needed
            if (sg.u_begin == 0) {
                int32_t* ids = page_ids + (size_t)problem * max_pages;
                for (int i = tid; i < k_pg; i += kFThreads) ids[i] = i;
                if (tid == 0) n_pages[problem] = max(k_pg, 0);
            }
            continue;
        }
        const int b = problem / Hkv, hk = problem - b * Hkv;
        const size_t row0 = (size_t)problem * P;
        const uint4* q_heads = q + ((size_t)b * Hq + (size_t)hk * GQ) * kOctets;

        // ---- query fragments of column n = g: chunks t + 4j of q+ and q- ----
        uint32_t qp[4][4], qn[4][4];
        {
            const uint4* qrow = q_heads + (size_t)(g < GQ ? g : g % GQ) * kOctets;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint4 qw = __ldg(qrow + t + 4 * j);
                const uint32_t w[4] = {qw.x, qw.y, qw.z, qw.w};
#pragma unroll
                for (int c = 0; c < 4; ++c) {
                    const uint32_t neg = ((w[c] >> 15) & 0x00010001u) * 0xFFFFu;   // 0xFFFF in the negative halves
                    qn[j][c] = w[c] & neg;
                    qp[j][c] = w[c] & ~neg;
                }
            }
        }

        float amax = 0.f;
        uint32_t kmx = 0u, kmn = 0xFFFFFFFFu;        // keys of this lane's valid pages
        int pa = sg.u_begin * kFUnitPages + warp * 16 + g;
        float* dst_score = scores + row0;
#pragma unroll 1
        for (int i = 0; i < n; ++i, pa += kFUnitPages) {
            const int nv = min(16, np - (pa - g));       // valid pages of this warp's tile
            if (nv > 0 && !dead) {
                const uint32_t par = (phase >> slot_rd) & 1u;
                phase ^= 1u << slot_rd;
                if (!__all_sync(0xFFFFFFFFu, mbar_wait_bounded(bars + 8u * slot_rd, par, kFWaitLimitNs))) {
                    if (lane == 0) atomicExch(status, (int)STC_ERR_TIMEOUT);
                    dead = true;
                }
            }
            if (nv > 0 && !dead) {
                float sx[4] = {0.f, 0.f, 0.f, 0.f}, sn[4] = {0.f, 0.f, 0.f, 0.f};
                float ax[4] = {0.f, 0.f, 0.f, 0.f}, an[4] = {0.f, 0.f, 0.f, 0.f};
                const uint32_t s = ring + (uint32_t)slot_rd * kFTileBytes + frag;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint4 x0 = lds16(s + 64u * j), x8 = lds16(s + 64u * j + 2048u);
                    const uint4 n0 = lds16(s + 64u * j + 4096u), n8 = lds16(s + 64u * j + 6144u);
                    mma_bf16_16816(sx, x0.x, x8.x, x0.y, x8.y, qp[j][0], qp[j][1]);
                    mma_bf16_16816(sn, n0.x, n8.x, n0.y, n8.y, qn[j][0], qn[j][1]);
                    mma_bf16_16816(ax, x0.x & kAbs, x8.x & kAbs, x0.y & kAbs, x8.y & kAbs, qp[j][0], qp[j][1]);
                    mma_bf16_16816(an, n0.x & kAbs, n8.x & kAbs, n0.y & kAbs, n8.y & kAbs, qn[j][0] & kAbs, qn[j][1] & kAbs);
                    mma_bf16_16816(sx, x0.z, x8.z, x0.w, x8.w, qp[j][2], qp[j][3]);
                    mma_bf16_16816(sn, n0.z, n8.z, n0.w, n8.w, qn[j][2], qn[j][3]);
                    mma_bf16_16816(ax, x0.z & kAbs, x8.z & kAbs, x0.w & kAbs, x8.w & kAbs, qp[j][2], qp[j][3]);
                    mma_bf16_16816(an, n0.z & kAbs, n8.z & kAbs, n0.w & kAbs, n8.w & kAbs, qn[j][2] & kAbs, qn[j][3] & kAbs);
                }
                __syncwarp();                            // every lane has read the slot
                issue(true);                             // refills the slot just consumed
                // rows g and g + 8 of the tile: maximum over the head columns (two in this lane, the rest in the
                // quad); rows past the sequence hold whatever the slot held before and are left out
                float r0 = fmaxf(sx[0] + sn[0], sx[1] + sn[1]), r8 = fmaxf(sx[2] + sn[2], sx[3] + sn[3]);
                r0 = fmaxf(r0, __shfl_xor_sync(0xFFFFFFFFu, r0, 1));
                r8 = fmaxf(r8, __shfl_xor_sync(0xFFFFFFFFu, r8, 1));
                r0 = fmaxf(r0, __shfl_xor_sync(0xFFFFFFFFu, r0, 2));
                r8 = fmaxf(r8, __shfl_xor_sync(0xFFFFFFFFu, r8, 2));
                if (pa < np) {
                    amax = fmaxf(amax, fmaxf(ax[0] + an[0], ax[1] + an[1]));
                    const uint32_t kk = float_key(r0); kmx = max(kmx, kk); kmn = min(kmn, kk);
                    if (t == 0) dst_score[pa] = r0;
                }
                if (pa + 8 < np) {
                    amax = fmaxf(amax, fmaxf(ax[2] + an[2], ax[3] + an[3]));
                    const uint32_t kk = float_key(r8); kmx = max(kmx, kk); kmn = min(kmn, kk);
                    if (t == 0) dst_score[pa + 8] = r8;
                }
            } else {
                issue(true);                             // keeps the two cursors in step
            }
            slot_rd = slot_rd + 1 == kFDepth ? 0 : slot_rd + 1;
        }
#pragma unroll
        for (int d = 16; d >= 1; d >>= 1) amax = fmaxf(amax, __shfl_xor_sync(0xFFFFFFFFu, amax, d));
        kmx = __reduce_max_sync(0xFFFFFFFFu, kmx);
        kmn = __reduce_min_sync(0xFFFFFFFFu, kmn);
        if (lane == 0) {
            atomicMax(&st.absmax[problem], __float_as_uint(amax));   // non-negative floats order as integers
            atomicMax(&st.keymax[problem], kmx);
            atomicMax(&st.keymin_inv[problem], ~kmn);
        }

        // ---- whoever completes the problem's unit count selects its pages ---------
        __threadfence();
        __syncthreads();
        if (tid == 0) {
            const unsigned old = atomicAdd(&st.counters[problem], (unsigned)n);
            s_last = (old + (unsigned)n == (unsigned)units_per_problem);
        }
        __syncthreads();
        if (s_last) {
            __threadfence();
            int32_t* ids = page_ids + (size_t)problem * max_pages;
            const int w = min(max(n_recent, 0), k_pg);   // the local window: the last w pages are kept
            if (k_pg > w) {
                FilterCtx f;
                f.kmin = kmin + row0 * kOctets;
                f.kmax = kmax + row0 * kOctets;
                f.q_heads = q_heads;
                f.gq = GQ;
                // margin: both sums round each addition to fp32 (relative 2^-24 of a partial sum that never
                // exceeds sum|term|); 2^-13 of the problem's largest sum|term| covers several hundred such
                // roundings on each side with room to spare; the factor 1.01 covers the rounding of the
                // absolute sum itself
                f.delta = __uint_as_float(__ldcg(st.absmax + problem)) * (kMarginRel * 1.01f);
                f.amb_idx = reinterpret_cast<int32_t*>(sel_mem + kSmemKeys);
                f.amb_key = sel_mem + kSmemKeys + kAmbMax;
                float* u = scores + row0;
                const uint32_t key_max = __ldcg(st.keymax + problem), key_min = ~__ldcg(st.keymin_inv + problem);
                if (!filter_select_fast<kFThreads>(u, np - w, k_pg - w, ids, sel_mem, s_topk, key_min, key_max, &f) &&
                    !block_topk<kFThreads>(u, np - w, k_pg - w, ids, sel_mem, s_topk, &f)) {
                    // too many pages within the margin (many equal pages): score every page exactly instead
                    const int half = lane >> 4, l = lane & 15;
                    const unsigned hm = 0xFFFFu << (16 * half);
#pragma unroll 1
                    for (int p0 = 0; p0 < np - w; p0 += 2 * kFWarps) {
                        const int p = p0 + warp * 2 + half;
                        const int pc = min(p, np - w - 1);
                        const float sxp = exact_page_score(f.kmin + (size_t)pc * kOctets, f.kmax + (size_t)pc * kOctets,
                                                           q_heads, GQ, l, hm);
                        if (l == 0 && p < np - w) u[p] = sxp;
                    }
                    __threadfence_block();
                    __syncthreads();
                    block_topk<kFThreads>(u, np - w, k_pg - w, ids, sel_mem, s_topk, nullptr);
                }
            }
            for (int i = tid; i < w; i += kFThreads) ids[k_pg - w + i] = np - w + i;
            if (tid == 0) n_pages[problem] = k_pg;
        }
    }
    // (every tile issued has been waited for by the loop above, so nothing is in flight here; after a
    // timeout the copies still pending get one more bounded wait each so that none lands in the shared
    // memory of a CTA that has gone)
    if (dead) {
#pragma unroll
        for (int sl = 0; sl < kFDepth; ++sl) mbar_wait_bounded(bars + 8u * sl, (phase >> sl) & 1u, kFWaitLimitNs);
    }
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
            if (k_pg > w) block_topk<kThreads>(scores + row0, np - w, k_pg - w, ids, ring_mem, s_topk, nullptr);
            for (int i = tid; i < w; i += kThreads) ids[k_pg - w + i] = np - w + i;
            if (tid == 0) n_pages[problem] = k_pg;
        }
    }
}

// workspace: four words per problem (ProblemStats: arrival counter, largest sum|term|, largest key,
// inverted smallest key), then the page scores
size_t counters_bytes(const Geom& g) { return (((size_t)g.problems * 16) + 255) & ~(size_t)255; }

}  // namespace

size_t select_ws_bytes(const Geom& g) {
    return 256 + counters_bytes(g) + (size_t)g.problems * g.P * sizeof(float);
}

size_t quest_select_clear_bytes(const Geom& g) { return 256 + (size_t)g.problems * 16; }

cudaError_t clear_quest_select_ws(const Geom& g, void* ws, cudaStream_t st) {
    return cudaMemsetAsync(ws, 0, quest_select_clear_bytes(g), st);
}

namespace {
__global__ void clear_two_kernel(uint4* a, size_t na, uint4* b, size_t nb) {     // counts in 16-byte words
    const uint4 z = make_uint4(0u, 0u, 0u, 0u);
    for (size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x; i < na + nb; i += (size_t)gridDim.x * blockDim.x)
        if (i < na) a[i] = z; else b[i - na] = z;
}
}  // namespace

cudaError_t clear_two(void* a, size_t a_bytes, void* b, size_t b_bytes, cudaStream_t st) {
    // both ranges start on 256-byte boundaries and are rounded up to 16 bytes (the words behind them are
    // score / partial storage that the call rewrites anyway)
    const size_t na = (a_bytes + 15) / 16, nb = (b_bytes + 15) / 16;
    const unsigned blocks = (unsigned)((na + nb + 255) / 256 < 64 ? (na + nb + 255) / 256 : 64);
    clear_two_kernel<<<blocks ? blocks : 1, 256, 0, st>>>(static_cast<uint4*>(a), na, static_cast<uint4*>(b), nb);
    return cudaGetLastError();
}

cudaError_t launch_quest_select(const Geom& g, const void* kmin, const void* kmax, const void* q,
                                int token_budget, int n_recent_pages, int max_pages, int32_t* page_ids,
                                int32_t* n_pages, float* scores_opt, void* ws, cudaStream_t st, unsigned flags) {
    if (g.problems == 0) return cudaSuccess;
    // workspace: status word (its own 256 bytes), the per-problem words, the page scores
    int32_t* status = static_cast<int32_t*>(ws);
    unsigned* counters = reinterpret_cast<unsigned*>(static_cast<char*>(ws) + 256);
    ProblemStats stats{counters, counters + g.problems, counters + 2 * (size_t)g.problems, counters + 3 * (size_t)g.problems};
    float* scores = scores_opt ? scores_opt
                               : reinterpret_cast<float*>(static_cast<char*>(ws) + 256 + counters_bytes(g));
    cudaError_t e = cudaSuccess;
    if (!(flags & kLaunchNoClear)) e = clear_quest_select_ws(g, ws, st);
    if (e != cudaSuccess) return e;
    int sms = 0;
    e = device_sm_count(&sms);
    if (e != cudaSuccess) return e;
    // Several query heads per KV head, long rows of pages and no score output: the tensor-core scan
    // filters, the declared-order fp32 bound settles the pages near the threshold (one CTA per SM, a
    // heavier per-problem selection: it pays once a problem's scan outweighs that).  Otherwise every
    // page gets the declared-order bound on the fp32 pipes.
    const bool filter = scores_opt == nullptr &&
                        ((g.Gq >= kFilterMinGq && g.P >= kFilterMinPages) || (g.Gq > 4 && g.P >= kFilterMinPagesSplit));
    const int pages_per_unit = filter ? kFUnitPages : kWarps * (g.Gq > 4 ? 1 : 2);
    const int units_per_problem = (g.P + pages_per_unit - 1) / pages_per_unit;
    const long long total_units = (long long)units_per_problem * g.problems;
    long long grid = (long long)sms * (filter ? kFCtasPerSm : kCtasPerSm);
    if (grid > total_units) grid = total_units;
#define STC_SEL(GQ_)                                                                                 \
    case GQ_:                                                                                        \
        if (filter) {                                                                                \
            cudaFuncSetAttribute(quest_filter_kernel<GQ_>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                                 (int)kFSmemBytes);                                                  \
            quest_filter_kernel<GQ_><<<(unsigned)grid, kFThreads, kFSmemBytes, st>>>(                \
                static_cast<const uint4*>(kmin), static_cast<const uint4*>(kmax),                    \
                static_cast<const uint4*>(q), g.seq_len, g.Hq, g.Hkv, g.T, g.P, token_budget,        \
                n_recent_pages, max_pages, page_ids, n_pages, scores, stats, status,                 \
                units_per_problem, total_units);                                                     \
            break;                                                                                   \
        }                                                                                            \
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
