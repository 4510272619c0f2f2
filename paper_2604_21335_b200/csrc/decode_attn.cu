// Routed decode attention: split-K flash-decode over the selected pages, full
// width keys, values read from the packed group store.
//
// Work split.  The (problem, listed page) pairs of the whole call form one flat
// sequence; it is cut into equal contiguous ranges, one per WARP of a grid that
// fits the machine in a single wave.  A warp is a complete worker: it streams its
// pages, keeps its own online-softmax state and, where its range ends inside a
// problem, writes a partial (max, sum, accumulator) for that problem.  Warps never
// wait on each other: a per-problem counter of covered pages tells the warp that
// completes a problem to merge the partials, in slot order, so results are
// bitwise repeatable.
//
// Data movement.  Each warp owns a ring of kStages shared-memory stages.  A stage
// holds one page: its 16 key rows (4 KiB, contiguous in HBM) and the packed value
// groups of its 16 tokens (one contiguous span of the packed store, 0..4 KiB).
// Lane 0 brings both in with two bulk asynchronous copies (cp.async.bulk, the 1-D
// TMA path) that signal the stage's mbarrier; the copies for the next kStages-1
// pages are in flight while the warp computes on the current one, which is what
// hides HBM latency (3 stages at 8 warps per SM; 6 stages at 4 warps per SM when the call is too
// small to fill a wave and per-warp latency is what counts; 2 stages at 12 warps per SM for
// the single-head path on full-size calls, where a warp's per-page arithmetic is longer than a
// copy's latency and more warps buy more than a deeper ring).  The list entry, sequence length and value
// offsets a copy needs are fetched 32 pages at a time, one page per lane.
//
// A dropped value group is never copied for its own sake and never read: the
// position of a kept group inside the span follows from the token masks (prefix
// sum of their popcounts), and a dropped group's operand is a row of zeros, which
// is how it "contributes zero" while its token still counts in the normaliser.
//
// Arithmetic.  One query head per KV head: fp32 FMAs (lane = two tokens x 32
// dims).  Several query heads per KV head: the two contractions are dense tiles
// and run on tensor cores (mma.sync m16n8k16, bf16 in, fp32 accumulate):
//   S^T[token][head] = K . Q^T      A = key chunks straight from the stage, B = Q
//   O^T[dim][head]   = V^T . P^T    A = value chunks via ldmatrix.trans with one
//                                   row address per token (zero row if dropped),
//                                   B = softmax weights as a bf16 high part plus a
//                                   bf16 residual (two mma), transposed by movmatrix
// Both operands of the first product use the same permutation of head_dim
// positions, so a lane's 16-byte chunk feeds two k-steps without any shuffle.
//
// Every wait on an mbarrier is bounded (about a second); a wait that expires
// records STC_ERR_TIMEOUT in the workspace status word and the warp stops issuing
// copies, skips its arithmetic and leaves without touching the outputs.
#include "common.cuh"

namespace stc {
namespace {

constexpr int kWarps = 4;
constexpr int kThreads = kWarps * 32;
constexpr int kStagesWide = 3;                   // two CTAs per SM (full-size calls)
constexpr int kStagesDeep = 6;                   // one CTA per SM (calls too small to fill a wave)
constexpr int kStagesLean = 2;                   // three CTAs per SM: the single-head path on full-size calls, whose
                                                 // per-page arithmetic (not the copies) sets the pace, so that
                                                 // twelve warps per SM beat eight with a deeper ring
constexpr int kMaxGq = 8;
constexpr int kCtasPerSm = 2;
constexpr int kMinPagesPerWarp = 4;
constexpr int kMaxSlots = 32;                    // partials per problem the merging warp handles (lane = slot, <= 32)
constexpr uint32_t kKeyBytes = kPage * kRowBytes;          // 4096
constexpr uint32_t kStageBytes = 2 * kKeyBytes;            // keys + worst-case value span
__host__ __device__ constexpr uint32_t ring_bytes(int stages) { return kWarps * stages * kStageBytes; }
__host__ __device__ constexpr uint32_t smem_bytes(int stages) {      // ring + zero row (padded) + mbarriers
    return ring_bytes(stages) + 64 + kWarps * stages * 8;
}
constexpr unsigned long long kWaitLimitNs = 1000000000ull;

// ---- PTX wrappers -----------------------------------------------------------------------
__device__ __forceinline__ void mma_bf16(float (&d)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                         uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, "
        "{%0,%1,%2,%3};"
        : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
        : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t movmatrix_trans(uint32_t a) {
    uint32_t d;
    asm volatile("movmatrix.sync.aligned.m8n8.trans.b16 %0, %1;" : "=r"(d) : "r"(a));
    return d;
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t& r0, uint32_t& r1, uint32_t& r2,
                                                  uint32_t& r3) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr) : "memory");
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// Bounded wait for a stage's copies.  False = gave up.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity) {
    return mbar_wait_bounded(bar, parity, kWaitLimitNs);
}

struct AttnArgs {
    const unsigned char* k;
    const unsigned char* v_packed;
    const uint16_t* v_mask;
    const uint32_t* v_offs;
    const uint4* q;
    const int32_t* page_ids;
    const int32_t* n_pages;
    const int32_t* seq_len;
    float* out;
    float* lse;
    float* part_acc;     // [problems][slots_cap][Gq][128]
    float* part_ml;      // [problems][slots_cap][Gq][2]
    unsigned* counters;  // [problems] pages covered so far
    int32_t* status;     // one word: STC_OK or STC_ERR_TIMEOUT
    int64_t cap_groups;
    long long total;     // problems * max_pages
    int n_warps;         // workers
    int slots_cap;
    int Hq, Hkv, Gq, T, max_pages;
    float scale_log2;    // sm_scale * log2(e)
};

// What a lane remembers about one page of the 32-page lookahead window.
struct PageRef {
    int page;            // page id, -1 = nothing to attend (past the list, id out of range)
    int n_valid;         // valid tokens of the page, 1..16
    uint32_t first;      // first packed group of the page (clipped to the store)
    uint32_t groups;     // packed groups of the page actually stored
};

template <int S, bool MMA, int kStages>
__global__ void __launch_bounds__(kThreads, kStages == kStagesLean ? 3 : (kStages == kStagesWide ? kCtasPerSm : 1))
decode_attn_kernel(const AttnArgs a) {
    constexpr uint32_t kRingBytes = ring_bytes(kStages);
    constexpr int OPG = kOctets / S;             // 16-byte chunks per value group
    constexpr uint32_t kGroupBytes = OPG * 16;
    extern __shared__ __align__(128) unsigned char smem[];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int r = lane >> 2, c = lane & 3;
    const uint32_t ring = smem_u32(smem) + (uint32_t)warp * kStages * kStageBytes;
    const uint32_t zero_row = smem_u32(smem) + kRingBytes;
    const uint32_t bars = smem_u32(smem) + kRingBytes + 64 + (uint32_t)warp * kStages * 8;

    if (tid < 4) reinterpret_cast<uint32_t*>(smem + kRingBytes)[tid] = 0u;
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < kStages; ++s) mbar_init(bars + 8 * s, 1);
        fence_mbar_init();
    }
    __syncthreads();                             // the only CTA-wide barrier: after it warps are independent

    const long long w = (long long)blockIdx.x * kWarps + warp;
    if (w >= a.n_warps) return;
    const long long x_lo = a.total * w / a.n_warps, x_hi = a.total * (w + 1) / a.n_warps;
    const int count = (int)(x_hi - x_lo);        // >= 1 by construction (n_warps <= total)
    const int mp = a.max_pages;

    // ---- lookahead window: lane i describes flat position win_base + i ----------------------
    PageRef win{-1, 0, 0u, 0u};
    auto fill_window = [&](long long base) {
        const long long x = base + lane;
        win = PageRef{-1, 0, 0u, 0u};
        if (x < x_hi) {
            const int p = (int)(x / mp), slot = (int)(x - (long long)p * mp);
            const int len = clamp_len(a.seq_len, p / a.Hkv, a.T);
            const int np = (len + kPage - 1) / kPage;
            int n_list = np, id = slot;
            if (a.page_ids) {
                n_list = min(max(a.n_pages[p], 0), mp);
                id = a.page_ids[(size_t)p * mp + slot];
            }
            if (slot < n_list && id >= 0 && id < np) {
                const int t0 = id * kPage, nv = min(kPage, len - t0);
                const uint32_t* o = a.v_offs + (size_t)p * (a.T + 1) + t0;
                const long long ob = min((long long)o[0], (long long)a.cap_groups);
                const long long oe = min((long long)o[nv], (long long)a.cap_groups);
                const long long ng = min(oe > ob ? oe - ob : 0LL, (long long)(kPage * S));   // never past the stage
                win = PageRef{id, nv, (uint32_t)ob, (uint32_t)ng};
            }
        }
    };

    // ---- the pages in flight: a register FIFO, oldest first (uniform across the warp except mask) ----
    struct InFlight {
        int nv;              // valid tokens; 0 = nothing to attend at this position
        uint32_t chunks;     // 16-byte chunks of the value span present in the stage
        uint32_t mask;       // lanes 0..15: group mask of token `lane`
    };
    uint32_t phase = 0;                          // bit s = parity to wait for on stage s

    long long win_base = x_lo;
    fill_window(win_base);
    long long x_issue = x_lo;                    // next flat position to bring in
    int p_issue = (int)(x_lo / mp);              // its problem
    int slot_issue = (int)(x_lo - (long long)p_issue * mp);

    auto issue = [&](int s, bool reuse) -> InFlight {   // bring position x_issue into stage s
        InFlight f{0, 0u, 0u};
        if (x_issue >= x_hi) return f;
        if (x_issue - win_base >= 32) { win_base = x_issue; fill_window(win_base); }
        const int src = (int)(x_issue - win_base);
        const int page = __shfl_sync(0xFFFFFFFFu, win.page, src);
        const int nv = __shfl_sync(0xFFFFFFFFu, win.n_valid, src);
        const uint32_t first = __shfl_sync(0xFFFFFFFFu, win.first, src);
        const uint32_t groups = __shfl_sync(0xFFFFFFFFu, win.groups, src);
        if (page >= 0) {
            const size_t row0 = (size_t)p_issue * a.T + (size_t)page * kPage;
            if (lane < nv) f.mask = a.v_mask[row0 + lane];
            f.nv = nv;
            f.chunks = groups * OPG;
            if (lane == 0) {
                const uint32_t kb = (uint32_t)nv * kRowBytes, vb = groups * kGroupBytes;
                const uint32_t bar = bars + 8 * s, dst = ring + (uint32_t)s * kStageBytes;
                if (reuse) fence_proxy_async();  // the stage's earlier reads precede the new writes
                mbar_expect_tx(bar, kb + vb);
                bulk_g2s(dst, a.k + row0 * kRowBytes, kb, bar);
                if (vb)
                    bulk_g2s(dst + kKeyBytes,
                             a.v_packed + ((size_t)p_issue * a.cap_groups + first) * kGroupBytes, vb, bar);
            }
        }
        ++x_issue;
        if (++slot_issue == mp) { slot_issue = 0; ++p_issue; }
        return f;
    };

    // ---- query operand ----------------------------------------------------------------------
    // MMA: lane (r, c) holds chunks c, c+4, c+8, c+12 of head r (zeros past Gq) = B fragments.
    // FMA: the same chunks of the single head.
    uint4 qa[4];
    auto load_q = [&](int problem) {
        const int b = problem / a.Hkv, hk = problem - b * a.Hkv;
        const int head = MMA ? r : 0;
        const bool ok = head < a.Gq;
        const uint4* qrow = a.q + ((size_t)b * a.Hq + (size_t)hk * a.Gq + (ok ? head : 0)) * kOctets;
#pragma unroll
        for (int j = 0; j < 4; ++j) qa[j] = ok ? __ldg(qrow + c + 4 * j) : make_uint4(0, 0, 0, 0);
    };

    // ---- running state of the current problem -------------------------------------------------
    // MMA: acc[dt][0..3] = (dim 16dt+r, head 2c), (16dt+r, 2c+1), (16dt+r+8, 2c), (16dt+r+8, 2c+1);
    //      m_run/l_run[e] belong to head 2c+e (l_run summed over the lane's own tokens only).
    // FMA: acc[j][2q2+e] -> dim 8(c+4j)+2q2+e, summed over the lane's own two tokens; m_run[0], l_run[0].
    float acc[8][4];
    float m_run[2], l_run[2];
    auto reset_state = [&]() {
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i][0] = acc[i][1] = acc[i][2] = acc[i][3] = 0.f;
        m_run[0] = m_run[1] = -INFINITY;
        l_run[0] = l_run[1] = 0.f;
    };

    // ---- one page -----------------------------------------------------------------------------
    auto compute = [&](int s, const InFlight& f) {
        const uint32_t kst = ring + (uint32_t)s * kStageBytes, vst = kst + kKeyBytes;
        const int nv = f.nv;
        // exclusive prefix (in groups) of the page's token masks, lanes 0..15
        const uint32_t cnt = __popc(f.mask);
        uint32_t pre = cnt;
#pragma unroll
        for (int d = 1; d < 16; d <<= 1) {
            const uint32_t o = __shfl_up_sync(0xFFFFFFFFu, pre, d);
            if (lane >= d) pre += o;
        }
        pre -= cnt;

        if constexpr (MMA) {
            // S^T = K . Q^T : rows = tokens (r, r+8), columns = heads (2c, 2c+1)
            float s0[4] = {0.f, 0.f, 0.f, 0.f}, s1[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint4 k0 = lds16(kst + (uint32_t)r * kRowBytes + (uint32_t)(c + 4 * j) * 16u);
                const uint4 k1 = lds16(kst + (uint32_t)(r + 8) * kRowBytes + (uint32_t)(c + 4 * j) * 16u);
                mma_bf16(s0, k0.x, k1.x, k0.y, k1.y, qa[j].x, qa[j].y);
                mma_bf16(s1, k0.z, k1.z, k0.w, k1.w, qa[j].z, qa[j].w);
            }
            const bool v0 = r < nv, v1 = r + 8 < nv;
            float sv[4];
            sv[0] = v0 ? (s0[0] + s1[0]) * a.scale_log2 : -INFINITY;
            sv[1] = v0 ? (s0[1] + s1[1]) * a.scale_log2 : -INFINITY;
            sv[2] = v1 ? (s0[2] + s1[2]) * a.scale_log2 : -INFINITY;
            sv[3] = v1 ? (s0[3] + s1[3]) * a.scale_log2 : -INFINITY;
            float pm0 = fmaxf(sv[0], sv[2]), pm1 = fmaxf(sv[1], sv[3]);
#pragma unroll
            for (int d = 4; d < 32; d <<= 1) {
                pm0 = fmaxf(pm0, __shfl_xor_sync(0xFFFFFFFFu, pm0, d));
                pm1 = fmaxf(pm1, __shfl_xor_sync(0xFFFFFFFFu, pm1, d));
            }
            const float mn0 = fmaxf(m_run[0], pm0), mn1 = fmaxf(m_run[1], pm1);   // finite: token 0 is valid
            const float al0 = exp2f(m_run[0] - mn0), al1 = exp2f(m_run[1] - mn1);
            const float p0 = exp2f(sv[0] - mn0), p1 = exp2f(sv[1] - mn1);
            const float p2 = exp2f(sv[2] - mn0), p3 = exp2f(sv[3] - mn1);
            l_run[0] = fmaf(l_run[0], al0, p0 + p2);
            l_run[1] = fmaf(l_run[1], al1, p1 + p3);
            m_run[0] = mn0; m_run[1] = mn1;
            // P^T as B fragments: high bf16 part and bf16 residual
            const uint32_t wh0 = pack_bf16(p0, p1), wh1 = pack_bf16(p2, p3);
            const uint32_t wl0 = pack_bf16(p0 - bf16lo(wh0), p1 - bf16hi(wh0));
            const uint32_t wl1 = pack_bf16(p2 - bf16lo(wh1), p3 - bf16hi(wh1));
            const uint32_t bh0 = movmatrix_trans(wh0), bh1 = movmatrix_trans(wh1);
            const uint32_t bl0 = movmatrix_trans(wl0), bl1 = movmatrix_trans(wl1);
            // value rows: this lane addresses token tau, chunk 2dt + hb of every dim tile
            const int tau = (lane & 7) + 8 * (lane >> 4), hb = (lane >> 3) & 1;
            const uint32_t m = __shfl_sync(0xFFFFFFFFu, f.mask, tau);
            const uint32_t base = __shfl_sync(0xFFFFFFFFu, pre, tau) * OPG;
            const uint32_t limit = f.chunks;
#pragma unroll
            for (int dt = 0; dt < 8; ++dt) {
                const int oct = 2 * dt + hb, grp = oct / OPG;
                const uint32_t idx = base + __popc(m & ((1u << grp) - 1u)) * OPG + (uint32_t)(oct % OPG);
                const bool kept = ((m >> grp) & 1u) && idx < limit;
                uint32_t a0, a1, a2, a3;
                ldmatrix_x4_trans(kept ? vst + idx * 16u : zero_row, a0, a1, a2, a3);
                acc[dt][0] *= al0; acc[dt][1] *= al1; acc[dt][2] *= al0; acc[dt][3] *= al1;
                mma_bf16(acc[dt], a0, a1, a2, a3, bh0, bh1);
                mma_bf16(acc[dt], a0, a1, a2, a3, bl0, bl1);
            }
        } else {
            // one head on the fp32 pipes: lane = tokens r, r+8 x chunks c, c+4, c+8, c+12
            float sd[2];
            uint4 kr[2][4];
#pragma unroll
            for (int hf = 0; hf < 2; ++hf)
#pragma unroll
                for (int j = 0; j < 4; ++j)
                    kr[hf][j] = lds16(kst + (uint32_t)(r + 8 * hf) * kRowBytes + (uint32_t)(c + 4 * j) * 16u);
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                float d0 = 0.f, d1 = 0.f;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    d0 = fmaf(bf16lo(qa[j].x), bf16lo(kr[hf][j].x), d0);
                    d1 = fmaf(bf16hi(qa[j].x), bf16hi(kr[hf][j].x), d1);
                    d0 = fmaf(bf16lo(qa[j].y), bf16lo(kr[hf][j].y), d0);
                    d1 = fmaf(bf16hi(qa[j].y), bf16hi(kr[hf][j].y), d1);
                    d0 = fmaf(bf16lo(qa[j].z), bf16lo(kr[hf][j].z), d0);
                    d1 = fmaf(bf16hi(qa[j].z), bf16hi(kr[hf][j].z), d1);
                    d0 = fmaf(bf16lo(qa[j].w), bf16lo(kr[hf][j].w), d0);
                    d1 = fmaf(bf16hi(qa[j].w), bf16hi(kr[hf][j].w), d1);
                }
                float d = d0 + d1;
                d += __shfl_xor_sync(0xFFFFFFFFu, d, 1);
                d += __shfl_xor_sync(0xFFFFFFFFu, d, 2);
                sd[hf] = (r + 8 * hf < nv) ? d * a.scale_log2 : -INFINITY;
            }
            float pm = fmaxf(sd[0], sd[1]);
#pragma unroll
            for (int d = 4; d < 32; d <<= 1) pm = fmaxf(pm, __shfl_xor_sync(0xFFFFFFFFu, pm, d));
            const float mn = fmaxf(m_run[0], pm);
            const float al = exp2f(m_run[0] - mn);
            const float p0 = exp2f(sd[0] - mn), p1 = exp2f(sd[1] - mn);
            l_run[0] = fmaf(l_run[0], al, p0 + p1);
            m_run[0] = mn;
            const uint32_t limit = f.chunks;
            uint4 vr[2][4];
#pragma unroll
            for (int hf = 0; hf < 2; ++hf) {
                const uint32_t m = __shfl_sync(0xFFFFFFFFu, f.mask, r + 8 * hf);
                const uint32_t base = __shfl_sync(0xFFFFFFFFu, pre, r + 8 * hf) * OPG;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const int oct = c + 4 * j, grp = oct / OPG;
                    const uint32_t idx = base + __popc(m & ((1u << grp) - 1u)) * OPG + (uint32_t)(oct % OPG);
                    const bool kept = ((m >> grp) & 1u) && idx < limit;
                    vr[hf][j] = kept ? lds16(vst + idx * 16u) : make_uint4(0, 0, 0, 0);
                }
            }
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t u0[4] = {vr[0][j].x, vr[0][j].y, vr[0][j].z, vr[0][j].w};
                const uint32_t u1[4] = {vr[1][j].x, vr[1][j].y, vr[1][j].z, vr[1][j].w};
#pragma unroll
                for (int q2 = 0; q2 < 4; ++q2) {
                    float& lo = acc[2 * j + (q2 >> 1)][2 * (q2 & 1)];
                    float& hi = acc[2 * j + (q2 >> 1)][2 * (q2 & 1) + 1];
                    lo = fmaf(p1, bf16lo(u1[q2]), fmaf(p0, bf16lo(u0[q2]), lo * al));
                    hi = fmaf(p1, bf16hi(u1[q2]), fmaf(p0, bf16hi(u0[q2]), hi * al));
                }
            }
        }
    };

    // ---- end of a problem segment: output, or partial + ticket + merge ---------------------
    const float ln2 = 0.6931471805599453f;
    auto finish = [&](int problem, int covered) {
        const int b = problem / a.Hkv, hk = problem - b * a.Hkv;
        const size_t row_base = (size_t)b * a.Hq + (size_t)hk * a.Gq;
        // totals of the normaliser over the lanes that share a head column / the single head
#pragma unroll
        for (int d = 4; d < 32; d <<= 1) {
            l_run[0] += __shfl_xor_sync(0xFFFFFFFFu, l_run[0], d);
            if (MMA) l_run[1] += __shfl_xor_sync(0xFFFFFFFFu, l_run[1], d);
        }
        if constexpr (!MMA) {
#pragma unroll
            for (int d = 4; d < 32; d <<= 1)
#pragma unroll
                for (int i = 0; i < 8; ++i)
#pragma unroll
                    for (int e = 0; e < 4; ++e) acc[i][e] += __shfl_xor_sync(0xFFFFFFFFu, acc[i][e], d);
        }
        const bool whole = covered == mp;         // this warp saw the whole problem: no partial needed
        // first / count of the workers that overlap this problem (closed forms of the equal split)
        const long long A = (long long)problem * mp;
        const long long first = ((A + 1) * a.n_warps + a.total - 1) / a.total - 1;
        const long long last = ((A + mp) * a.n_warps + a.total - 1) / a.total - 1;
        const int n_slots = (int)(last - first + 1);
        const size_t slot0 = ((size_t)problem * a.slots_cap) * a.Gq;
        const size_t slot = slot0 + (size_t)(w - first) * a.Gq;

        if constexpr (MMA) {
#pragma unroll
            for (int e = 0; e < 2; ++e) {
                const int h = 2 * c + e;
                if (h >= a.Gq) continue;
                if (whole) {
                    const float inv = l_run[e] > 0.f ? 1.f / l_run[e] : 0.f;
                    float* o = a.out + (row_base + h) * kHeadDim;
#pragma unroll
                    for (int dt = 0; dt < 8; ++dt) {
                        o[16 * dt + r] = acc[dt][e] * inv;
                        o[16 * dt + r + 8] = acc[dt][2 + e] * inv;
                    }
                    if (a.lse && r == 0)
                        a.lse[row_base + h] = l_run[e] > 0.f ? (m_run[e] + log2f(l_run[e])) * ln2 : -INFINITY;
                } else {
                    float* o = a.part_acc + (slot + h) * kHeadDim;
#pragma unroll
                    for (int dt = 0; dt < 8; ++dt) {
                        o[16 * dt + r] = acc[dt][e];
                        o[16 * dt + r + 8] = acc[dt][2 + e];
                    }
                    if (r == 0) { a.part_ml[(slot + h) * 2] = m_run[e]; a.part_ml[(slot + h) * 2 + 1] = l_run[e]; }
                }
            }
        } else {
            if (r == 0) {                          // lanes 0..3 hold the reduced 128 channels
                const float inv = l_run[0] > 0.f ? 1.f / l_run[0] : 0.f;
                float* o = whole ? a.out + row_base * kHeadDim : a.part_acc + slot * kHeadDim;
                const float sc = whole ? inv : 1.f;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    float4 lo = make_float4(acc[2 * j][0] * sc, acc[2 * j][1] * sc, acc[2 * j][2] * sc, acc[2 * j][3] * sc);
                    float4 hi = make_float4(acc[2 * j + 1][0] * sc, acc[2 * j + 1][1] * sc, acc[2 * j + 1][2] * sc,
                                            acc[2 * j + 1][3] * sc);
                    *reinterpret_cast<float4*>(o + 8 * (c + 4 * j)) = lo;
                    *reinterpret_cast<float4*>(o + 8 * (c + 4 * j) + 4) = hi;
                }
                if (c == 0) {
                    if (whole) {
                        if (a.lse) a.lse[row_base] = l_run[0] > 0.f ? (m_run[0] + log2f(l_run[0])) * ln2 : -INFINITY;
                    } else {
                        a.part_ml[slot * 2] = m_run[0];
                        a.part_ml[slot * 2 + 1] = l_run[0];
                    }
                }
            }
        }
        if (whole) return;

        // ticket: the worker that completes the problem's page count merges, in slot order
        __threadfence();
        __syncwarp();
        unsigned old = 0;
        if (lane == 0) old = atomicAdd(&a.counters[problem], (unsigned)covered);
        old = __shfl_sync(0xFFFFFFFFu, old, 0);
        if (old + (unsigned)covered != (unsigned)mp) return;
        __threadfence();
        // Heads are merged kHB at a time (head indices clamped, so no load is conditional):
        // (1) lane = slot: the (max, sum) pairs in one round of loads, then per head the
        //     global max, each slot's weight 2^(m - M) and the total of the normaliser;
        // (2) weighted sums in slot order, kSB slots' loads in flight; a lane owns 4 channels.
        constexpr int kHB = MMA ? 4 : 1, kSB = MMA ? 4 : 8;
        const int sl_mine = min(lane, n_slots - 1);
#pragma unroll 1
        for (int h0 = 0; h0 < a.Gq; h0 += kHB) {
            float wgt[kHB], M[kHB], L[kHB];
            float2 ml[kHB];
#pragma unroll
            for (int i = 0; i < kHB; ++i)
                ml[i] = __ldcg(reinterpret_cast<const float2*>(a.part_ml) + slot0 + (size_t)sl_mine * a.Gq +
                               min(h0 + i, a.Gq - 1));
#pragma unroll
            for (int i = 0; i < kHB; ++i) {
                const float m = lane < n_slots ? ml[i].x : -INFINITY;
                float mx = m;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) mx = fmaxf(mx, __shfl_xor_sync(0xFFFFFFFFu, mx, d));
                wgt[i] = (m == -INFINITY) ? 0.f : exp2f(m - mx);
                float ls = lane < n_slots ? ml[i].y * wgt[i] : 0.f;
#pragma unroll
                for (int d = 1; d < 32; d <<= 1) ls += __shfl_xor_sync(0xFFFFFFFFu, ls, d);
                M[i] = mx; L[i] = ls;
            }
            float4 o[kHB];
#pragma unroll
            for (int i = 0; i < kHB; ++i) o[i] = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll 1
            for (int sl0 = 0; sl0 < n_slots; sl0 += kSB) {
                float4 v[kSB][kHB];
#pragma unroll
                for (int j = 0; j < kSB; ++j)
#pragma unroll
                    for (int i = 0; i < kHB; ++i) {
                        const size_t ps = slot0 + (size_t)min(sl0 + j, n_slots - 1) * a.Gq + min(h0 + i, a.Gq - 1);
                        v[j][i] = __ldcg(reinterpret_cast<const float4*>(a.part_acc + ps * kHeadDim) + lane);
                    }
#pragma unroll
                for (int j = 0; j < kSB; ++j)
#pragma unroll
                    for (int i = 0; i < kHB; ++i) {
                        float sc = __shfl_sync(0xFFFFFFFFu, wgt[i], (sl0 + j) & 31);
                        if (sl0 + j >= n_slots) sc = 0.f;
                        o[i].x = fmaf(v[j][i].x, sc, o[i].x); o[i].y = fmaf(v[j][i].y, sc, o[i].y);
                        o[i].z = fmaf(v[j][i].z, sc, o[i].z); o[i].w = fmaf(v[j][i].w, sc, o[i].w);
                    }
            }
#pragma unroll
            for (int i = 0; i < kHB; ++i) {
                const int h = h0 + i;
                if (h >= a.Gq) continue;
                const float inv = L[i] > 0.f ? 1.f / L[i] : 0.f;
                reinterpret_cast<float4*>(a.out + (row_base + h) * kHeadDim)[lane] =
                    make_float4(o[i].x * inv, o[i].y * inv, o[i].z * inv, o[i].w * inv);
                if (a.lse && lane == 0) a.lse[row_base + h] = L[i] > 0.f ? (M[i] + log2f(L[i])) * ln2 : -INFINITY;
            }
        }
    };

    // ---- main loop ----------------------------------------------------------------------------
    InFlight f[kStages];                          // f[0] = oldest page in flight, in stage s
#pragma unroll
    for (int i = 0; i < kStages; ++i) f[i] = issue(i, false);

    int p_cur = (int)(x_lo / mp);
    int slot_cur = (int)(x_lo - (long long)p_cur * mp);
    int seg_begin_slot = slot_cur;
    load_q(p_cur);
    reset_state();
    int s = 0;
#pragma unroll 1
    for (int n = 0; n < count; ++n) {
        if (f[0].nv > 0) {                        // uniform across the warp
            const uint32_t par = (phase >> s) & 1u;
            phase ^= 1u << s;
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(bars + 8 * s, par))) {
                // A copy did not land in time.  Report it, give the copies still in flight
                // one more bounded wait each so they do not land in a dead CTA's memory,
                // and leave; the outputs this worker owes stay unwritten.
                if (lane == 0) atomicExch(a.status, (int)STC_ERR_TIMEOUT);
                int s2 = s;
#pragma unroll
                for (int i = 1; i < kStages; ++i) {
                    s2 = s2 + 1 == kStages ? 0 : s2 + 1;
                    if (f[i].nv > 0) mbar_wait(bars + 8 * s2, (phase >> s2) & 1u);
                }
                return;
            }
            compute(s, f[0]);
        }
        __syncwarp();
#pragma unroll
        for (int i = 0; i + 1 < kStages; ++i) f[i] = f[i + 1];
        f[kStages - 1] = issue(s, true);
        s = s + 1 == kStages ? 0 : s + 1;
        ++slot_cur;
        if (slot_cur == mp || n + 1 == count) {   // the range leaves this problem (one call site: finish is big)
            finish(p_cur, slot_cur - seg_begin_slot);
            if (slot_cur == mp) { ++p_cur; slot_cur = 0; }
            seg_begin_slot = slot_cur;
            if (n + 1 < count) { load_q(p_cur); reset_state(); }
        }
    }
}

// out = 0, lse = -inf for every head: the call has nothing to attend.
__global__ void attn_empty_kernel(float* __restrict__ out, float* __restrict__ lse, int rows) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i < rows * kHeadDim) out[i] = 0.f;
    if (lse && i < rows) lse[i] = -INFINITY;
}

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

}  // namespace

// Workers (warps) and partial slots per problem.  Sized from max_pages only, so the
// workspace query and the launch agree; independent of the device so that the
// workspace size can be asked for without one.
// The plan is sized for kPlanSms multiprocessors: the workspace size has to be computable without a
// device (stc_workspace_bytes is host arithmetic), so the plan uses the B200's count as a documented
// constant; the launch only picks the ring depth from the device it runs on.
constexpr long long kPlanSms = 148;

AttnPlan attn_plan(const Geom& g, int max_pages) {
    AttnPlan p;
    const long long mp = max_pages < 1 ? 1 : max_pages;
    const long long total = (long long)(g.problems < 1 ? 1 : g.problems) * mp;
    long long workers = (total + kMinPagesPerWarp - 1) / kMinPagesPerWarp;
    const long long wave = kPlanSms * (g.Gq == 1 ? 3 : kCtasPerSm) * kWarps;   // resident warps (see kStagesLean)
    if (workers > wave) workers = wave;
    // a call that fits one CTA per SM runs there, with the deeper ring
    if (workers > kPlanSms * kWarps && workers < kPlanSms * kWarps * 3 / 2) workers = kPlanSms * kWarps;
    // many short problems: one warp per problem, so that no problem is split and nothing is merged (long
    // single-head problems that would leave a third of the warps idle are split all the same)
    if (g.problems <= wave && 2LL * g.problems >= workers && !(g.Gq == 1 && mp >= 64 && 10LL * g.problems < 7 * wave))
        workers = g.problems;
    const long long by_slots = (long long)(kMaxSlots - 1) * (g.problems < 1 ? 1 : g.problems);
    if (workers > by_slots) workers = by_slots;  // keeps ceil(workers / problems) + 1 <= kMaxSlots
    if (workers < 1) workers = 1;
    p.n_workers = (int)workers;
    p.slots_cap = (int)((workers + g.problems - 1) / (g.problems < 1 ? 1 : g.problems)) + 1;
    return p;
}

size_t attn_ws_bytes(const Geom& g, int max_pages) {
    const AttnPlan p = attn_plan(g, max_pages);
    const size_t slots = (size_t)g.problems * p.slots_cap * g.Gq;
    return 256 + align256((size_t)g.problems * 4) + align256(slots * kHeadDim * 4) + align256(slots * 2 * 4);
}

cudaError_t launch_decode_attn(const Geom& g, const void* k, const void* v_packed,
                               const uint16_t* v_mask, const uint32_t* v_offs, int64_t cap_groups,
                               const void* q, const int32_t* page_ids, const int32_t* n_pages,
                               int max_pages, float sm_scale, float* out, float* lse, void* ws,
                               cudaStream_t st, unsigned flags) {
    if (g.problems == 0) return cudaSuccess;
    const int rows = g.B * g.Hq;
    char* wsp = static_cast<char*>(ws);
    if (max_pages < 1 || g.T == 0) {
        cudaError_t e = cudaMemsetAsync(wsp, 0, 4, st);
        if (e != cudaSuccess) return e;
        attn_empty_kernel<<<(rows * kHeadDim + 255) / 256, 256, 0, st>>>(out, lse, rows);
        return cudaGetLastError();
    }
    const AttnPlan p = attn_plan(g, max_pages);
    const size_t slots = (size_t)g.problems * p.slots_cap * g.Gq;
    AttnArgs a;
    a.status = reinterpret_cast<int32_t*>(wsp);
    a.counters = reinterpret_cast<unsigned*>(wsp + 256);
    char* w = wsp + 256 + align256((size_t)g.problems * 4);
    a.part_acc = reinterpret_cast<float*>(w);
    w += align256(slots * kHeadDim * 4);
    a.part_ml = reinterpret_cast<float*>(w);
    a.k = static_cast<const unsigned char*>(k);
    a.v_packed = static_cast<const unsigned char*>(v_packed);
    a.v_mask = v_mask;
    a.v_offs = v_offs;
    a.q = static_cast<const uint4*>(q);
    a.page_ids = page_ids;
    a.n_pages = n_pages;
    a.seq_len = g.seq_len;
    a.out = out;
    a.lse = lse;
    a.cap_groups = cap_groups;
    a.total = (long long)g.problems * max_pages;
    a.n_warps = p.n_workers;
    a.slots_cap = p.slots_cap;
    a.Hq = g.Hq; a.Hkv = g.Hkv; a.Gq = g.Gq; a.T = g.T;
    a.max_pages = max_pages;
    a.scale_log2 = sm_scale * 1.4426950408889634f;
    // status word + page counters start at zero
    cudaError_t e = cudaSuccess;
    if (!(flags & kLaunchNoClear)) e = clear_decode_attn_ws(g, ws, st);
    if (e != cudaSuccess) return e;
    const int n_cta = (p.n_workers + kWarps - 1) / kWarps;
    int sms = 0;
    e = device_sm_count(&sms);
    if (e != cudaSuccess) return e;
    const bool mma = g.Gq > 1, deep = n_cta <= sms;      // a call that fits one CTA per SM takes the deeper ring
#define STC_ATTN_LAUNCH(S_, MMA_, ST_)                                                                  \
    do {                                                                                                \
        cudaFuncSetAttribute(decode_attn_kernel<S_, MMA_, ST_>, cudaFuncAttributeMaxDynamicSharedMemorySize, \
                             (int)smem_bytes(ST_));                                                     \
        decode_attn_kernel<S_, MMA_, ST_><<<n_cta, kThreads, smem_bytes(ST_), st>>>(a);                 \
    } while (0)
#define STC_ATTN(S_)                                                                                    \
    case S_:                                                                                            \
        if (mma && deep) STC_ATTN_LAUNCH(S_, true, kStagesDeep);                                        \
        else if (mma) STC_ATTN_LAUNCH(S_, true, kStagesWide);                                           \
        else if (deep) STC_ATTN_LAUNCH(S_, false, kStagesDeep);                                         \
        else if (n_cta > 2 * sms) STC_ATTN_LAUNCH(S_, false, kStagesLean);                              \
        else STC_ATTN_LAUNCH(S_, false, kStagesWide);                                                   \
        break;
    switch (g.S) {
        STC_ATTN(4) STC_ATTN(8) STC_ATTN(16)
        default: return cudaErrorInvalidValue;
    }
#undef STC_ATTN_LAUNCH
#undef STC_ATTN
    return cudaGetLastError();
}

// status word + page counters of a call
size_t decode_attn_clear_bytes(const Geom& g) { return 256 + (size_t)g.problems * 4; }

cudaError_t clear_decode_attn_ws(const Geom& g, void* ws, cudaStream_t st) {
    return cudaMemsetAsync(ws, 0, decode_attn_clear_bytes(g), st);
}

}  // namespace stc
