// Routed decode attention: split-K flash-decode over the selected pages, full
// width keys, values read from the packed group store and expanded in
// registers.
//
// Work split: one CTA (4 warps) per (problem, split); a warp owns one 16-token
// page at a time.  Lane (r = lane/4, c = lane%4) loads, for tokens r and r+8 of
// the page, the 16-byte chunks c, c+4, c+8, c+12 of the key row (four lanes
// cover 64 contiguous bytes) and the matching chunks of the value row.  A value
// chunk whose group was dropped is not loaded at all: the lane substitutes
// zeros, which is how a dropped group "contributes zero" while its token still
// counts in the softmax normaliser.  The address of a kept chunk comes from the
// page's first offset, a 16-lane prefix sum of the tokens' group counts and a
// popcount of the lower mask bits.
//
// One query head per KV head: dot products and the value update run on the
// fp32 pipes (2 x 64 FMAs per lane and page).
// Several query heads per KV head: Q.K^T over the grouped heads is a dense
// contraction and runs on tensor cores (mma.sync m16n8k16, heads padded to the
// 16-row operand, key chunks used directly as the col-major operand with the
// head_dim positions permuted identically on both operands); P.V uses the same
// instruction with the value chunks transposed in registers (movmatrix); the
// softmax weights enter as a bf16 high part plus a bf16 residual so the product
// keeps ~16 bits of the fp32 weight.
//
// Each CTA reduces its warps' (max, sum, acc) states in shared memory and, when
// the problem is split, writes a partial; the CTA that arrives last at the
// problem's ticket merges the partials (nobody waits on anybody).
#include "common.cuh"

namespace stc {
namespace {

constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr int kMaxGq = 8;
constexpr int kTargetCtas = 148 * 4;
static_assert(kThreads == kHeadDim, "the CTA reductions map one thread to one channel");

__device__ __forceinline__ void mma_bf16(float& d0, float& d1, float& d2, float& d3, uint32_t a0,
                                         uint32_t a1, uint32_t a2, uint32_t a3, uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(d0), "+f"(d1), "+f"(d2), "+f"(d3)
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}

__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

struct AttnArgs {
    const uint4* k;
    const uint4* v_packed;
    const uint16_t* v_mask;
    const uint32_t* v_offs;
    const uint4* q;
    const int32_t* page_ids;
    const int32_t* n_pages;
    const int32_t* seq_len;
    float* out;
    float* lse;
    float* part_acc;     // [problems][n_splits][Gq][128]
    float* part_ml;      // [problems][n_splits][Gq][2]
    unsigned* counters;  // [problems]
    int64_t cap_groups;
    int Hq, Hkv, Gq, T, max_pages, pages_per_cta, n_splits;
    float scale_log2;    // sm_scale * log2(e)
};

// Per-page token bookkeeping held by lanes 0..15 (one token each).
struct TokInfo { uint32_t mask; uint32_t base; };

template <int S, bool MMA>
__global__ void __launch_bounds__(kThreads, 3)
decode_attn_kernel(const AttnArgs a) {
    constexpr int OPG = kOctets / S;            // 16-byte chunks per value group
    constexpr int NH = MMA ? kMaxGq : 1;        // head rows reduced per CTA
    __shared__ float s_acc[kWarps][NH][kHeadDim];
    __shared__ float s_m[kWarps][NH], s_l[kWarps][NH];
    __shared__ int s_last;

    const int problem = blockIdx.x / a.n_splits, split = blockIdx.x - problem * a.n_splits;
    const int b = problem / a.Hkv, hk = problem - b * a.Hkv;
    const int len = clamp_len(a.seq_len, b, a.T);
    const int np = (len + kPage - 1) / kPage;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int r = lane >> 2, c = lane & 3;
    const int32_t* ids = a.page_ids ? a.page_ids + (size_t)problem * a.max_pages : nullptr;
    int n_list = ids ? min(max(a.n_pages[problem], 0), a.max_pages) : np;
    const int begin = split * a.pages_per_cta;
    const int end = min(n_list, begin + a.pages_per_cta);
    const int my_count = (end > begin + warp) ? (end - begin - warp + kWarps - 1) / kWarps : 0;

    const uint4* krows = a.k + (size_t)problem * a.T * kOctets;
    const uint4* vstore = a.v_packed + (size_t)problem * a.cap_groups * OPG;
    const int64_t cap_chunks = a.cap_groups * OPG;
    const uint16_t* masks = a.v_mask + (size_t)problem * a.T;
    const uint32_t* offs = a.v_offs + (size_t)problem * (a.T + 1);

    // ---- query operand ------------------------------------------------------
    // MMA: lane holds chunk c+4j of head row r (zeros past Gq) as A fragments.
    // MHA: lane holds the same chunks of the single head as floats.
    uint4 qa[4];
    {
        const int head = MMA ? r : 0;
        const bool ok = head < a.Gq;
        const uint4* qrow = a.q + ((size_t)b * a.Hq + (size_t)hk * a.Gq + (ok ? head : 0)) * kOctets;
#pragma unroll
        for (int j = 0; j < 4; ++j) qa[j] = ok ? qrow[c + 4 * j] : make_uint4(0, 0, 0, 0);
    }

    float acc[4][4][2];                          // [j][pair][e]: dims 8(c+4j) + 2*pair + e
#pragma unroll
    for (int j = 0; j < 4; ++j)
#pragma unroll
        for (int p = 0; p < 4; ++p) acc[j][p][0] = acc[j][p][1] = 0.f;
    float m_run = -INFINITY, l_run = 0.f;
    float dz0 = 0.f, dz1 = 0.f;                  // rows 8..15 of the padded head operand

    // Page ids of this warp, 32 at a time: lane i holds the id of the warp's
    // (n0+i)-th page, so the per-page lookup is a shuffle, not a dependent load.
    int pid_reg = -1;
    auto refill = [&](int n0) {
        const int n = n0 + lane;
        int p = -1;
        if (n < my_count) {
            const int i = begin + warp + n * kWarps;
            p = ids ? ids[i] : i;
            if (p < 0 || p >= np) p = -1;
        }
        pid_reg = p;
    };
    auto page_of = [&](int n) -> int {           // n-th page of this warp, -1 if none / invalid
        if ((n & 31) == 0) refill(n);
        return __shfl_sync(0xFFFFFFFFu, pid_reg, n & 31);
    };
    auto tok_info = [&](int page) -> TokInfo {
        TokInfo ti{0u, 0u};
        if (page >= 0) {
            const int t = page * kPage + lane;
            if (lane < kPage && t < len) ti.mask = masks[t];
            ti.base = offs[page * kPage];
        }
        return ti;
    };

    int page = page_of(0);
    TokInfo ti = tok_info(page);
#pragma unroll 1
    for (int n = 0; n < my_count; ++n) {
        const int page_next = page_of(n + 1);
        const TokInfo ti_next = tok_info(page_next);
        if (page >= 0) {
            const int t0 = page * kPage;
            // ---- key loads ----------------------------------------------------
            uint4 kr[2][4];
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const int t = t0 + r + 8 * hf;
                const uint4* row = krows + (size_t)t * kOctets;
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    kr[hf][j] = (t < len) ? ldg_nc16(row + c + 4 * j) : make_uint4(0, 0, 0, 0);
            }
            // ---- value loads, dropped groups become zeros ------------------------
            uint32_t cnt = __popc(ti.mask), pre = cnt;
#pragma unroll
            for (int d = 1; d < 16; d <<= 1) {
                uint32_t o = __shfl_up_sync(0xFFFFFFFFu, pre, d);
                if (lane >= d) pre += o;
            }
            pre -= cnt;                           // exclusive, lanes 0..15
            uint4 vr[2][4];
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const uint32_t m = __shfl_sync(0xFFFFFFFFu, ti.mask, r + 8 * hf);
                const uint32_t first = ti.base + __shfl_sync(0xFFFFFFFFu, pre, r + 8 * hf);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int oct = c + 4 * j, grp = oct / OPG;
                    const int64_t chunk = (int64_t)(first + __popc(m & ((1u << grp) - 1u))) * OPG + (oct % OPG);
                    vr[hf][j] = (((m >> grp) & 1u) && chunk < cap_chunks) ? ldg_nc16(vstore + chunk)
                                                                          : make_uint4(0, 0, 0, 0);
                }
            }

            if constexpr (MMA) {
                // ---- S = Q.K^T on tensor cores: rows = heads, cols = tokens -------
                float s[2][4];
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    s[hf][0] = s[hf][1] = s[hf][2] = s[hf][3] = 0.f;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        mma_bf16(s[hf][0], s[hf][1], s[hf][2], s[hf][3], qa[j].x, 0u, qa[j].y, 0u,
                                 kr[hf][j].x, kr[hf][j].y);
                        mma_bf16(s[hf][0], s[hf][1], s[hf][2], s[hf][3], qa[j].z, 0u, qa[j].w, 0u,
                                 kr[hf][j].z, kr[hf][j].w);
                    }
                }
                // lane: head r, tokens 8hf + 2c + e
                float sv[2][2], pmax = -INFINITY;
#pragma unroll
                for (int hf = 0; hf < 2; ++hf)
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const bool valid = t0 + 8 * hf + 2 * c + e < len;
                        sv[hf][e] = valid ? s[hf][e] * a.scale_log2 : -INFINITY;
                        pmax = fmaxf(pmax, sv[hf][e]);
                    }
                pmax = fmaxf(pmax, __shfl_xor_sync(0xFFFFFFFFu, pmax, 1));
                pmax = fmaxf(pmax, __shfl_xor_sync(0xFFFFFFFFu, pmax, 2));
                const float m_new = fmaxf(m_run, pmax);
                const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
                const float alpha = exp2f(m_run - m_use);
                float p[2][2];
#pragma unroll
                for (int hf = 0; hf < 2; ++hf)
#pragma unroll
                    for (int e = 0; e < 2; ++e) p[hf][e] = exp2f(sv[hf][e] - m_use);
                l_run = l_run * alpha + (p[0][0] + p[0][1]) + (p[1][0] + p[1][1]);
                m_run = m_new;
#pragma unroll
                for (int j = 0; j < 4; ++j)
#pragma unroll
                    for (int q2 = 0; q2 < 4; ++q2) { acc[j][q2][0] *= alpha; acc[j][q2][1] *= alpha; }
                // weights as bf16 high part + residual (A fragments: k = token)
                const uint32_t ph0 = pack_bf16(p[0][0], p[0][1]), ph2 = pack_bf16(p[1][0], p[1][1]);
                const uint32_t pl0 = pack_bf16(p[0][0] - bf16lo(ph0), p[0][1] - bf16hi(ph0));
                const uint32_t pl2 = pack_bf16(p[1][0] - bf16lo(ph2), p[1][1] - bf16hi(ph2));
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t v0[4] = {vr[0][j].x, vr[0][j].y, vr[0][j].z, vr[0][j].w};
                    const uint32_t v1[4] = {vr[1][j].x, vr[1][j].y, vr[1][j].z, vr[1][j].w};
#pragma unroll
                    for (int q2 = 0; q2 < 4; ++q2) {
                        const uint32_t b0 = movmatrix_trans(v0[q2]);   // tokens 0..7  x 8 dims
                        const uint32_t b1 = movmatrix_trans(v1[q2]);   // tokens 8..15 x 8 dims
                        mma_bf16(acc[j][q2][0], acc[j][q2][1], dz0, dz1, ph0, 0u, ph2, 0u, b0, b1);
                        mma_bf16(acc[j][q2][0], acc[j][q2][1], dz0, dz1, pl0, 0u, pl2, 0u, b0, b1);
                    }
                }
            } else {
                // ---- one head: fp32 pipes ----------------------------------------
                float sdot[2];
#pragma unroll
                for (int hf = 0; hf < 2; ++hf) {
                    float d = 0.f;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        d = fmaf(bf16lo(qa[j].x), bf16lo(kr[hf][j].x), d);
                        d = fmaf(bf16hi(qa[j].x), bf16hi(kr[hf][j].x), d);
                        d = fmaf(bf16lo(qa[j].y), bf16lo(kr[hf][j].y), d);
                        d = fmaf(bf16hi(qa[j].y), bf16hi(kr[hf][j].y), d);
                        d = fmaf(bf16lo(qa[j].z), bf16lo(kr[hf][j].z), d);
                        d = fmaf(bf16hi(qa[j].z), bf16hi(kr[hf][j].z), d);
                        d = fmaf(bf16lo(qa[j].w), bf16lo(kr[hf][j].w), d);
                        d = fmaf(bf16hi(qa[j].w), bf16hi(kr[hf][j].w), d);
                    }
                    d += __shfl_xor_sync(0xFFFFFFFFu, d, 1);
                    d += __shfl_xor_sync(0xFFFFFFFFu, d, 2);
                    sdot[hf] = (t0 + r + 8 * hf < len) ? d * a.scale_log2 : -INFINITY;
                }
                float pmax = fmaxf(sdot[0], sdot[1]);
                pmax = fmaxf(pmax, __shfl_xor_sync(0xFFFFFFFFu, pmax, 4));
                pmax = fmaxf(pmax, __shfl_xor_sync(0xFFFFFFFFu, pmax, 8));
                pmax = fmaxf(pmax, __shfl_xor_sync(0xFFFFFFFFu, pmax, 16));
                const float m_new = fmaxf(m_run, pmax);
                const float m_use = (m_new == -INFINITY) ? 0.f : m_new;
                const float alpha = exp2f(m_run - m_use);
                const float p0 = exp2f(sdot[0] - m_use), p1 = exp2f(sdot[1] - m_use);
                l_run = l_run * alpha + p0 + p1;   // per token-lane; summed over r at the end
                m_run = m_new;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t v0[4] = {vr[0][j].x, vr[0][j].y, vr[0][j].z, vr[0][j].w};
                    const uint32_t v1[4] = {vr[1][j].x, vr[1][j].y, vr[1][j].z, vr[1][j].w};
#pragma unroll
                    for (int q2 = 0; q2 < 4; ++q2) {
                        acc[j][q2][0] = fmaf(p1, bf16lo(v1[q2]), fmaf(p0, bf16lo(v0[q2]), acc[j][q2][0] * alpha));
                        acc[j][q2][1] = fmaf(p1, bf16hi(v1[q2]), fmaf(p0, bf16hi(v0[q2]), acc[j][q2][1] * alpha));
                    }
                }
            }
        }
        page = page_next;
        ti = ti_next;
    }

    // ---- warp state -> shared memory -----------------------------------------
    if constexpr (MMA) {
        l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 1);
        l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, 2);
#pragma unroll
        for (int j = 0; j < 4; ++j)
#pragma unroll
            for (int q2 = 0; q2 < 4; ++q2)
                *reinterpret_cast<float2*>(&s_acc[warp][r][8 * (c + 4 * j) + 2 * q2]) =
                    make_float2(acc[j][q2][0], acc[j][q2][1]);
        if (c == 0) { s_m[warp][r] = m_run; s_l[warp][r] = l_run; }
    } else {
#pragma unroll
        for (int d = 4; d < 32; d <<= 1) {
            l_run += __shfl_xor_sync(0xFFFFFFFFu, l_run, d);
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int q2 = 0; q2 < 4; ++q2) {
                    acc[j][q2][0] += __shfl_xor_sync(0xFFFFFFFFu, acc[j][q2][0], d);
                    acc[j][q2][1] += __shfl_xor_sync(0xFFFFFFFFu, acc[j][q2][1], d);
                }
        }
        if (r == 0) {
#pragma unroll
            for (int j = 0; j < 4; ++j)
#pragma unroll
                for (int q2 = 0; q2 < 4; ++q2)
                    *reinterpret_cast<float2*>(&s_acc[warp][0][8 * (c + 4 * j) + 2 * q2]) =
                        make_float2(acc[j][q2][0], acc[j][q2][1]);
            if (c == 0) { s_m[warp][0] = m_run; s_l[warp][0] = l_run; }
        }
    }
    __syncthreads();

    // ---- CTA reduction: thread = one channel, loop over heads -----------------
    const int gq = MMA ? a.Gq : 1;
    const float ln2 = 0.6931471805599453f;
    for (int h = 0; h < gq; ++h) {
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) M = fmaxf(M, s_m[w][h]);
        float L = 0.f, o = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float mw = s_m[w][h];
            const float sc = (mw == -INFINITY) ? 0.f : exp2f(mw - M);
            L = fmaf(s_l[w][h], sc, L);
            o = fmaf(s_acc[w][h][tid], sc, o);
        }
        if (a.n_splits == 1) {
            const size_t row = (size_t)b * a.Hq + (size_t)hk * a.Gq + h;
            a.out[row * kHeadDim + tid] = L > 0.f ? o / L : 0.f;
            if (a.lse && tid == 0) a.lse[row] = L > 0.f ? (M + log2f(L)) * ln2 : -INFINITY;
        } else {
            const size_t slot = ((size_t)problem * a.n_splits + split) * a.Gq + h;
            a.part_acc[slot * kHeadDim + tid] = o;
            if (tid == 0) { a.part_ml[slot * 2] = M; a.part_ml[slot * 2 + 1] = L; }
        }
    }
    if (a.n_splits == 1) return;

    // ---- last CTA of the problem merges the partials ---------------------------
    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(&a.counters[problem], 1u) == (unsigned)(a.n_splits - 1));
    __syncthreads();
    if (!s_last) return;
    __threadfence();
    for (int h = 0; h < gq; ++h) {
        const size_t slot0 = (size_t)problem * a.n_splits * a.Gq + h;
        float M = -INFINITY;
        for (int s = 0; s < a.n_splits; ++s) M = fmaxf(M, __ldcg(a.part_ml + (slot0 + (size_t)s * a.Gq) * 2));
        float L = 0.f, o = 0.f;
        for (int s = 0; s < a.n_splits; ++s) {
            const size_t slot = slot0 + (size_t)s * a.Gq;
            const float ms = __ldcg(a.part_ml + slot * 2);
            const float sc = (ms == -INFINITY) ? 0.f : exp2f(ms - M);
            L = fmaf(__ldcg(a.part_ml + slot * 2 + 1), sc, L);
            o = fmaf(__ldcg(a.part_acc + slot * kHeadDim + tid), sc, o);
        }
        const size_t row = (size_t)b * a.Hq + (size_t)hk * a.Gq + h;
        a.out[row * kHeadDim + tid] = L > 0.f ? o / L : 0.f;
        if (a.lse && tid == 0) a.lse[row] = L > 0.f ? (M + log2f(L)) * ln2 : -INFINITY;
    }
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

}  // namespace

AttnPlan attn_plan(const Geom& g, int max_pages) {
    AttnPlan p;
    max_pages = max_pages < 1 ? 1 : max_pages;
    const int problems = g.problems < 1 ? 1 : g.problems;
    int splits = (kTargetCtas + problems - 1) / problems;
    const int max_splits = (max_pages + kWarps - 1) / kWarps;
    splits = splits < 1 ? 1 : (splits > max_splits ? max_splits : splits);
    int ppc = (max_pages + splits - 1) / splits;
    ppc = (ppc + kWarps - 1) / kWarps * kWarps;
    p.pages_per_cta = ppc;
    p.n_splits = (max_pages + ppc - 1) / ppc;
    return p;
}

size_t attn_ws_bytes(const Geom& g, int max_pages) {
    const AttnPlan p = attn_plan(g, max_pages);
    const size_t slots = (size_t)g.problems * p.n_splits * g.Gq;
    return align256((size_t)g.problems * 4) + align256(slots * kHeadDim * 4) + align256(slots * 2 * 4);
}

cudaError_t launch_decode_attn(const Geom& g, const void* k, const void* v_packed,
                               const uint16_t* v_mask, const uint32_t* v_offs, int64_t cap_groups,
                               const void* q, const int32_t* page_ids, const int32_t* n_pages,
                               int max_pages, float sm_scale, float* out, float* lse, void* ws,
                               cudaStream_t st) {
    if (g.problems == 0) return cudaSuccess;
    const AttnPlan p = attn_plan(g, max_pages);
    const size_t slots = (size_t)g.problems * p.n_splits * g.Gq;
    AttnArgs a;
    char* w = static_cast<char*>(ws);
    a.counters = reinterpret_cast<unsigned*>(w);
    w += align256((size_t)g.problems * 4);
    a.part_acc = reinterpret_cast<float*>(w);
    w += align256(slots * kHeadDim * 4);
    a.part_ml = reinterpret_cast<float*>(w);
    a.k = static_cast<const uint4*>(k);
    a.v_packed = static_cast<const uint4*>(v_packed);
    a.v_mask = v_mask;
    a.v_offs = v_offs;
    a.q = static_cast<const uint4*>(q);
    a.page_ids = page_ids;
    a.n_pages = n_pages;
    a.seq_len = g.seq_len;
    a.out = out;
    a.lse = lse;
    a.cap_groups = cap_groups;
    a.Hq = g.Hq; a.Hkv = g.Hkv; a.Gq = g.Gq; a.T = g.T;
    a.max_pages = max_pages;
    a.pages_per_cta = p.pages_per_cta;
    a.n_splits = p.n_splits;
    a.scale_log2 = sm_scale * 1.4426950408889634f;
    if (p.n_splits > 1) {
        cudaError_t e = cudaMemsetAsync(a.counters, 0, (size_t)g.problems * 4, st);
        if (e != cudaSuccess) return e;
    }
    const long long n_cta = (long long)g.problems * p.n_splits;
    if (n_cta > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    const bool mma = g.Gq > 1;
#define STC_ATTN(S_)                                                                         \
    case S_:                                                                                 \
        if (mma) decode_attn_kernel<S_, true><<<(unsigned)n_cta, kThreads, 0, st>>>(a);      \
        else     decode_attn_kernel<S_, false><<<(unsigned)n_cta, kThreads, 0, st>>>(a);     \
        break;
    switch (g.S) {
        STC_ATTN(4) STC_ATTN(8) STC_ATTN(16)
        default: return cudaErrorInvalidValue;
    }
#undef STC_ATTN
    return cudaGetLastError();
}

}  // namespace stc
