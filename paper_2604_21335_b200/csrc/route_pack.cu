// Sub-token routing (write side): mask selection under a global (token, group)
// budget, prefix-sum offsets and compaction of the kept value groups.
//
// Per problem the kept set is: every routed token's best group (when the floor
// of one group per token is on) plus the `take` best remaining pairs, ties to
// the lower flat index.  `take` depends on the routed-token count, which only
// the device knows, so everything is resolved on the device:
//
//   hist pass 0/1/2  radix select (11+11+10 bits) of the take-th largest key
//                    among the candidates; each CTA histograms a 1024-token
//                    tile in shared memory and merges into the problem's
//                    global histogram; the CTA that arrives last (atomic
//                    ticket, nobody waits) picks the digit for the next pass.
//   mask             per token: definite bits (reserved, FULL, key > tau) and
//                    tie bits (key == tau); per-tile counts of both.
//   compact          per tile: exclusive scan of the counts (tile base from the
//                    preceding tiles' sums), ties kept in flat-index order
//                    until the remaining rank is used up, final mask + offsets
//                    written, kept 16-byte chunks of V copied to the store.
//
// PER_TOKEN mode skips the histogram passes (the mask is local to a token).
// HBM traffic: scores 4x (3 passes + mask; 1x in PER_TOKEN mode), kept part of
// V once in and once out.
#include "common.cuh"

namespace stc {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kTile = 1024;                   // tokens per CTA in every kernel here
constexpr int kTokPerThread = kTile / kThreads;
constexpr int kBins = 2048;

// state words per problem
enum { ST_NROUTED = 0, ST_PREFIX, ST_KREM, ST_FLAGS, ST_TICKET0, ST_TICKET1, ST_TICKET2, ST_PAD, ST_WORDS };
enum { FL_NONE = 1, FL_BUDGET = 2 };          // nothing beyond the reserved groups / budget error

struct RouteWs {
    uint32_t* state;      // [problems][ST_WORDS]
    uint32_t* hist;       // [problems][3][kBins]
    uint32_t* tile_sums;  // [problems][n_tiles][2]
    uint16_t* tie;        // [problems][T]
    size_t zero_bytes;    // leading bytes (state + hist) cleared per call
    size_t total_bytes;
};

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

RouteWs carve(const Geom& g, void* ws) {
    RouteWs r;
    char* p = static_cast<char*>(ws);
    const int n_tiles = (g.T + kTile - 1) / kTile;
    size_t o = 0;
    r.state = reinterpret_cast<uint32_t*>(p + o); o += align256((size_t)g.problems * ST_WORDS * 4);
    r.hist = reinterpret_cast<uint32_t*>(p + o);  o += align256((size_t)g.problems * 3 * kBins * 4);
    r.zero_bytes = o;
    r.tile_sums = reinterpret_cast<uint32_t*>(p + o); o += align256((size_t)g.problems * n_tiles * 2 * 4);
    r.tie = reinterpret_cast<uint16_t*>(p + o);   o += align256((size_t)g.problems * g.T * 2);
    r.total_bytes = o;
    return r;
}

__device__ __forceinline__ int pass_shift(int pass) { return pass == 0 ? 21 : (pass == 1 ? 10 : 0); }
__device__ __forceinline__ uint32_t pass_digit(uint32_t key, int pass) {
    return pass == 2 ? (key & 1023u) : ((key >> pass_shift(pass)) & 2047u);
}
__device__ __forceinline__ uint32_t pass_himask(int pass) {
    return pass == 0 ? 0u : (pass == 1 ? 0xFFE00000u : 0xFFFFFC00u);
}

__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, int lane) {
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t o = __shfl_up_sync(0xFFFFFFFFu, v, d);
        if (lane >= d) v += o;
    }
    return v;
}

// Block-wide exclusive scan of one value per thread (kThreads threads).
__device__ __forceinline__ uint32_t block_excl_scan(uint32_t v, uint32_t* s_w /*[kWarps]*/, uint32_t* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    uint32_t incl = warp_incl_scan(v, lane);
    __syncthreads();                            // s_w may still be read from a previous use
    if (lane == 31) s_w[warp] = incl;
    __syncthreads();
    uint32_t base = 0, tot = 0;
#pragma unroll
    for (int w = 0; w < kWarps; ++w) { uint32_t x = s_w[w]; if (w < warp) base += x; tot += x; }
    if (total) *total = tot;
    return base + incl - v;
}

// Raw scores of one token (S/4 16-byte loads, issued together).
template <int S>
__device__ __forceinline__ void load_raw(const float* __restrict__ row, uint4 (&raw)[S / 4]) {
    const uint4* p = reinterpret_cast<const uint4*>(row);
#pragma unroll
    for (int i = 0; i < S / 4; ++i) raw[i] = __ldg(p + i);   // L1-allocating: the row's 16-byte pieces share sectors
}
// Scores of one token -> order-preserving keys; best = first maximum (tracked by
// value, so no register array is indexed at run time).
template <int S>
__device__ __forceinline__ void make_keys(const uint4 (&raw)[S / 4], uint32_t (&key)[S], int& best) {
#pragma unroll
    for (int i = 0; i < S / 4; ++i) {
        const uint4 w = raw[i];
        key[4 * i + 0] = float_key(__uint_as_float(w.x));
        key[4 * i + 1] = float_key(__uint_as_float(w.y));
        key[4 * i + 2] = float_key(__uint_as_float(w.z));
        key[4 * i + 3] = float_key(__uint_as_float(w.w));
    }
    uint32_t bk = key[0];
    best = 0;
#pragma unroll
    for (int j = 1; j < S; ++j) {
        const bool up = key[j] > bk;
        bk = up ? key[j] : bk;
        best = up ? j : best;
    }
}

__device__ __forceinline__ int token_class(const uint8_t* cls, int t, int len) {
    if (t >= len) return STC_CLS_DROP;
    return cls ? cls[t] : STC_CLS_ROUTED;
}

// The last CTA of a pass: find the bin holding the krem-th largest candidate.
__device__ void pick_digit(const uint32_t* __restrict__ hist, int nbins, uint32_t krem,
                           uint32_t* s_w, uint32_t* s_out /*[2]: digit, new krem*/) {
    // thread t owns bins nbins-1-8t .. nbins-8-8t (descending); nbins <= 8*kThreads
    uint32_t c[8], sum = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        int bin = nbins - 1 - 8 * (int)threadIdx.x - j;
        c[j] = bin >= 0 ? __ldcg(hist + bin) : 0u;
        sum += c[j];
    }
    uint32_t excl = block_excl_scan(sum, s_w, nullptr);
    if (excl < krem && krem <= excl + sum) {
        uint32_t run = excl;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (run + c[j] >= krem) {
                s_out[0] = (uint32_t)(nbins - 1 - 8 * (int)threadIdx.x - j);
                s_out[1] = krem - run;
                break;
            }
            run += c[j];
        }
    }
    __syncthreads();
}

template <int S>
__global__ void __launch_bounds__(kThreads)
route_hist_kernel(const float* __restrict__ scores, const uint8_t* __restrict__ cls, int64_t cls_b_stride,
                  int64_t cls_h_stride, const int32_t* __restrict__ seq_len, int Hkv, int T, int n_tiles,
                  int tiles_per_cta, int k_nominal, int min_per_token, int pass,
                  uint32_t* __restrict__ state_all, uint32_t* __restrict__ hist_all) {
    __shared__ uint32_t shist[kBins];
    __shared__ uint32_t s_w[kWarps];
    __shared__ uint32_t s_pick[2];
    __shared__ int s_last;

    const int n_groups = (n_tiles + tiles_per_cta - 1) / tiles_per_cta;
    const int problem = blockIdx.x / n_groups, group = blockIdx.x - problem * n_groups;
    const int b = problem / Hkv, hk = problem - b * Hkv;
    const int len = clamp_len(seq_len, b, T);
    uint32_t* state = state_all + (size_t)problem * ST_WORDS;
    uint32_t* hist = hist_all + ((size_t)problem * 3 + pass) * kBins;
    const int tid = threadIdx.x;

    uint32_t prefix = 0;
    if (pass > 0) {
        if (__ldcg(state + ST_FLAGS) != 0u) return;      // nothing to select / budget error
        prefix = __ldcg(state + ST_PREFIX);
    }
    const uint32_t himask = pass_himask(pass);
    const int dshift = pass_shift(pass);
    const uint32_t dmask = pass == 2 ? 1023u : 2047u;
    for (int i = tid; i < kBins; i += kThreads) shist[i] = 0;
    __syncthreads();

    const uint8_t* c = cls ? cls + (size_t)b * cls_b_stride + (size_t)hk * cls_h_stride : nullptr;
    uint32_t n_routed = 0;
    // several 1024-token tiles per CTA: the shared histogram is cleared and flushed once
    const int tile_end = min(n_tiles, (group + 1) * tiles_per_cta);
#pragma unroll 1
    for (int tile = group * tiles_per_cta; tile < tile_end; ++tile) {
        if (tile * kTile >= len) break;
        uint4 raw[kTokPerThread][S / 4];          // all of the thread's loads are in flight before the first use
        bool routed[kTokPerThread];
#pragma unroll
        for (int i = 0; i < kTokPerThread; ++i) {
            const int t = tile * kTile + i * kThreads + tid;
            routed[i] = token_class(c, t, len) == STC_CLS_ROUTED;
            if (routed[i]) load_raw<S>(scores + ((size_t)problem * T + t) * S, raw[i]);
        }
#pragma unroll
        for (int i = 0; i < kTokPerThread; ++i) {
            if (!routed[i]) continue;
            ++n_routed;
            uint32_t key[S];
            int best;
            make_keys<S>(raw[i], key, best);
#pragma unroll
            const int skip = min_per_token ? best : -1;
#pragma unroll
            for (int j = 0; j < S; ++j)
                if (j != skip && (key[j] & himask) == prefix) atomicAdd(&shist[(key[j] >> dshift) & dmask], 1u);
        }
    }
    __syncthreads();
    for (int i = tid; i < kBins; i += kThreads) {
        uint32_t v = shist[i];
        if (v) atomicAdd(hist + i, v);
    }
    if (pass == 0) {
        uint32_t tot;
        block_excl_scan(n_routed, s_w, &tot);
        if (tid == 0 && tot) atomicAdd(state + ST_NROUTED, tot);
    }

    __threadfence();
    __syncthreads();
    if (tid == 0) s_last = (atomicAdd(state + ST_TICKET0 + pass, 1u) == (unsigned)(n_groups - 1));
    __syncthreads();
    if (!s_last) return;
    __threadfence();

    uint32_t krem;
    if (pass == 0) {
        const uint64_t n = __ldcg(state + ST_NROUTED);
        const uint64_t m_total = n * (uint64_t)k_nominal;
        uint32_t flags = 0;
        if (min_per_token && m_total < n) flags = FL_BUDGET;
        const uint64_t take = m_total - (min_per_token ? n : 0);
        if (!flags && take == 0) flags = FL_NONE;
        if (flags) {
            if (tid == 0) { state[ST_FLAGS] = flags; state[ST_PREFIX] = 0; state[ST_KREM] = 0; }
            return;
        }
        krem = (uint32_t)take;
    } else {
        krem = __ldcg(state + ST_KREM);
    }
    pick_digit(hist, pass == 2 ? 1024 : kBins, krem, s_w, s_pick);
    if (tid == 0) {
        state[ST_PREFIX] = prefix | (s_pick[0] << pass_shift(pass));
        state[ST_KREM] = s_pick[1];
    }
}

template <int S>
__global__ void __launch_bounds__(kThreads)
route_mask_kernel(const float* __restrict__ scores, const uint8_t* __restrict__ cls, int64_t cls_b_stride,
                  int64_t cls_h_stride, const int32_t* __restrict__ seq_len, int Hkv, int T, int n_tiles,
                  int tiles_per_cta, int k_nominal, int min_per_token, int mode,
                  const uint32_t* __restrict__ state_all, uint16_t* __restrict__ v_mask,
                  uint16_t* __restrict__ tie_all, uint32_t* __restrict__ tile_sums) {
    __shared__ uint32_t s_w[kWarps];
    const int n_groups = (n_tiles + tiles_per_cta - 1) / tiles_per_cta;
    const int problem = blockIdx.x / n_groups, group = blockIdx.x - problem * n_groups;
    const int b = problem / Hkv, hk = problem - b * Hkv;
    const int len = clamp_len(seq_len, b, T);
    const int tid = threadIdx.x;
    const uint8_t* c = cls ? cls + (size_t)b * cls_b_stride + (size_t)hk * cls_h_stride : nullptr;

    uint32_t tau = 0, flags = 0;
    if (mode == STC_MODE_GLOBAL) {
        const uint32_t* state = state_all + (size_t)problem * ST_WORDS;
        flags = __ldcg(state + ST_FLAGS);
        tau = __ldcg(state + ST_PREFIX);
    }
    const int tile_end = min(n_tiles, (group + 1) * tiles_per_cta);
#pragma unroll 1
    for (int tile = group * tiles_per_cta; tile < tile_end; ++tile) {
    uint32_t n_def = 0, n_tie = 0;
    uint4 raw[kTokPerThread][S / 4];              // loads first, arithmetic after
    int cls_of[kTokPerThread];
#pragma unroll
    for (int i = 0; i < kTokPerThread; ++i) {
        const int t = tile * kTile + i * kThreads + tid;
        cls_of[i] = t < T ? token_class(c, t, len) : STC_CLS_DROP;
        if (cls_of[i] == STC_CLS_ROUTED && !(flags & FL_BUDGET))
            load_raw<S>(scores + ((size_t)problem * T + t) * S, raw[i]);
    }
#pragma unroll
    for (int i = 0; i < kTokPerThread; ++i) {
        const int t = tile * kTile + i * kThreads + tid;
        if (t >= T) continue;
        const int cl = cls_of[i];
        uint32_t def = 0, tie = 0;
        if (flags & FL_BUDGET) {
            def = 0;
        } else if (cl == STC_CLS_FULL) {
            def = (1u << S) - 1u;
        } else if (cl == STC_CLS_ROUTED) {
            uint32_t key[S];
            int best;
            make_keys<S>(raw[i], key, best);
            if (mode == STC_MODE_PER_TOKEN) {
#pragma unroll
                for (int j = 0; j < S; ++j) {
                    int rank = 0;
#pragma unroll
                    for (int i2 = 0; i2 < S; ++i2)
                        rank += (key[i2] > key[j]) || (key[i2] == key[j] && i2 < j);
                    if (rank < k_nominal) def |= 1u << j;
                }
            } else {
#pragma unroll
                for (int j = 0; j < S; ++j) {
                    if (min_per_token && j == best) { def |= 1u << j; continue; }
                    if (flags & FL_NONE) continue;
                    if (key[j] > tau) def |= 1u << j;
                    else if (key[j] == tau) tie |= 1u << j;
                }
            }
        }
        v_mask[(size_t)problem * T + t] = (uint16_t)def;
        tie_all[(size_t)problem * T + t] = (uint16_t)tie;
        n_def += __popc(def);
        n_tie += __popc(tie);
    }
    uint32_t tot_def, tot_tie;
    block_excl_scan(n_def, s_w, &tot_def);
    block_excl_scan(n_tie, s_w, &tot_tie);
    if (tid == 0) {
        tile_sums[((size_t)problem * n_tiles + tile) * 2 + 0] = tot_def;
        tile_sums[((size_t)problem * n_tiles + tile) * 2 + 1] = tot_tie;
    }
    }
}

template <int S>
__global__ void __launch_bounds__(kThreads)
route_compact_kernel(const uint4* __restrict__ v, const int32_t* __restrict__ seq_len, int Hkv, int T,
                     int n_tiles, int mode, const uint32_t* __restrict__ state_all,
                     const uint32_t* __restrict__ tile_sums, const uint16_t* __restrict__ tie_all,
                     uint16_t* __restrict__ v_mask, uint32_t* __restrict__ v_offs,
                     uint4* __restrict__ v_packed, int64_t cap_groups, int64_t* __restrict__ total_groups,
                     int32_t* __restrict__ status) {
    constexpr int OPG = kOctets / S;            // 16-byte chunks per group
    __shared__ uint32_t s_w[kWarps];
    __shared__ uint16_t s_mask[kTile];
    __shared__ uint32_t s_offs[kTile];

    const int problem = blockIdx.x / n_tiles, tile = blockIdx.x - problem * n_tiles;
    const int b = problem / Hkv;
    const int len = clamp_len(seq_len, b, T);
    const int tid = threadIdx.x;
    const int t_begin = tile * kTile;
    const bool owns_end = (len == 0) ? (tile == 0) : ((len - 1) / kTile == tile);
    if (t_begin >= len && !owns_end) return;

    uint32_t krem = 0, flags = 0;
    if (mode == STC_MODE_GLOBAL) {
        const uint32_t* state = state_all + (size_t)problem * ST_WORDS;
        flags = __ldcg(state + ST_FLAGS);
        krem = flags ? 0u : __ldcg(state + ST_KREM);
    }
    // base counts from the preceding tiles
    uint32_t bd = 0, be = 0;
    for (int i = tid; i < tile; i += kThreads) {
        bd += __ldcg(tile_sums + ((size_t)problem * n_tiles + i) * 2 + 0);
        be += __ldcg(tile_sums + ((size_t)problem * n_tiles + i) * 2 + 1);
    }
    uint32_t base_d, base_e;
    block_excl_scan(bd, s_w, &base_d);
    block_excl_scan(be, s_w, &base_e);

    // four consecutive tokens per thread keep the scan in token order
    const int t0 = t_begin + tid * kTokPerThread;
    uint32_t def[kTokPerThread], tie[kTokPerThread], nd = 0, ne = 0;
#pragma unroll
    for (int i = 0; i < kTokPerThread; ++i) {
        const int t = t0 + i;
        def[i] = t < len ? v_mask[(size_t)problem * T + t] : 0u;
        tie[i] = t < len ? tie_all[(size_t)problem * T + t] : 0u;
        nd += __popc(def[i]);
        ne += __popc(tie[i]);
    }
    uint32_t d_before = base_d + block_excl_scan(nd, s_w, nullptr);
    uint32_t e_before = base_e + block_excl_scan(ne, s_w, nullptr);
#pragma unroll
    for (int i = 0; i < kTokPerThread; ++i) {
        const int t = t0 + i;
        uint32_t m = def[i];
        const uint32_t off = d_before + min(e_before, krem);
        uint32_t tb = tie[i];
        while (tb) {                                  // ties in ascending group order
            const int j = __ffs(tb) - 1;
            tb &= tb - 1;
            if (e_before < krem) m |= 1u << j;
            ++e_before;
        }
        d_before += __popc(def[i]);
        s_mask[tid * kTokPerThread + i] = (uint16_t)m;
        s_offs[tid * kTokPerThread + i] = off;
        if (t < len) {
            v_mask[(size_t)problem * T + t] = (uint16_t)m;
            v_offs[(size_t)problem * (T + 1) + t] = off;
        }
        if (owns_end && ((len == 0 && t == 0) || (len > 0 && t == len - 1))) {
            const uint32_t total = len == 0 ? 0u : off + __popc(m);
            v_offs[(size_t)problem * (T + 1) + len] = total;
            total_groups[problem] = (int64_t)total;
            status[problem] = (flags & FL_BUDGET) ? STC_ERR_BUDGET
                              : ((int64_t)total > cap_groups ? STC_ERR_CAPACITY : STC_OK);
        }
    }
    __syncthreads();

    // copy the kept 16-byte chunks: item = (token, chunk), a warp covers two rows
    const uint4* vrow = v + ((size_t)problem * T + t_begin) * kOctets;
    uint4* dst = v_packed + (size_t)problem * cap_groups * OPG;
    constexpr int kItems = kTile * kOctets / kThreads;   // per thread
    constexpr int kUnroll = 8;
#pragma unroll 1
    for (int it0 = 0; it0 < kItems; it0 += kUnroll) {
        uint4 val[kUnroll];
        int64_t where[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            const int idx = (it0 + u) * kThreads + tid;
            const int tl = idx >> 4, oct = idx & 15, grp = oct / OPG;
            const uint32_t m = s_mask[tl];
            where[u] = -1;
            if (t_begin + tl < len && ((m >> grp) & 1u)) {
                const int64_t slot = (int64_t)s_offs[tl] + __popc(m & ((1u << grp) - 1u));
                if (slot < cap_groups) {
                    where[u] = slot * OPG + (oct % OPG);
                    val[u] = ldg_nc16_narrow(vrow + idx);
                }
            }
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u)
            if (where[u] >= 0) dst[where[u]] = val[u];
    }
}

}  // namespace

size_t route_ws_bytes(const Geom& g) { return carve(g, nullptr).total_bytes; }

cudaError_t launch_route_pack(const Geom& g, const void* v, const float* scores,
                              const uint8_t* tok_class, int64_t class_head_stride, int k_nominal,
                              int min_per_token, int mode, void* v_packed, uint16_t* v_mask,
                              uint32_t* v_offs, int64_t cap_groups, int64_t* total_groups,
                              int32_t* status, void* ws, int phases, cudaStream_t st) {
    if (g.problems == 0) return cudaSuccess;
    const RouteWs w = carve(g, ws);
    const bool do_route = phases & 1, do_pack = phases & 2;
    const int n_tiles = (g.T + kTile - 1) / kTile;
    const long long n_cta = (long long)n_tiles * g.problems;
    if (n_cta > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    // score-scanning kernels: enough CTAs for a few waves, several tiles each beyond that
    int tpc = (int)(n_cta / (148 * 8 * 2));
    tpc = tpc < 1 ? 1 : (tpc > 16 ? 16 : tpc);
    const unsigned n_cta_scan = (unsigned)((n_tiles + tpc - 1) / tpc) * (unsigned)g.problems;
    const int64_t cls_h = class_head_stride;
    const int64_t cls_b = class_head_stride ? (int64_t)g.Hkv * class_head_stride : (int64_t)g.T;
    if (do_route) {
        cudaError_t e = cudaMemsetAsync(w.state, 0, w.zero_bytes, st);
        if (e != cudaSuccess) return e;
    }

#define STC_ROUTE(S_)                                                                               \
    case S_: {                                                                                      \
        if (do_route && mode == STC_MODE_GLOBAL)                                                    \
            for (int pass = 0; pass < 3; ++pass)                                                    \
                route_hist_kernel<S_><<<n_cta_scan, kThreads, 0, st>>>(                             \
                    scores, tok_class, cls_b, cls_h, g.seq_len, g.Hkv, g.T, n_tiles, tpc, k_nominal, \
                    min_per_token, pass, w.state, w.hist);                                          \
        if (do_route) route_mask_kernel<S_><<<n_cta_scan, kThreads, 0, st>>>(                                     \
            scores, tok_class, cls_b, cls_h, g.seq_len, g.Hkv, g.T, n_tiles, tpc, k_nominal,        \
            min_per_token, mode, w.state, v_mask, w.tie, w.tile_sums);                              \
        if (do_pack) route_compact_kernel<S_><<<(unsigned)n_cta, kThreads, 0, st>>>(                             \
            static_cast<const uint4*>(v), g.seq_len, g.Hkv, g.T, n_tiles, mode, w.state,            \
            w.tile_sums, w.tie, v_mask, v_offs, static_cast<uint4*>(v_packed), cap_groups,          \
            total_groups, status);                                                                  \
    } break;
    switch (g.S) {
        STC_ROUTE(4) STC_ROUTE(8) STC_ROUTE(16)
        default: return cudaErrorInvalidValue;
    }
#undef STC_ROUTE
    return cudaGetLastError();
}

}  // namespace stc
