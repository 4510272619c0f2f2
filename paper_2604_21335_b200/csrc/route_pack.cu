// Sub-token routing (write side): mask selection under a global (token, group)
// budget, prefix-sum offsets and compaction of the kept value groups.
//
// Per problem the kept set is: every routed token's best group (when the floor
// of one group per token is on) plus the `take` best remaining pairs, ties to
// the lower flat index.  `take` depends on the routed-token count, which only
// the device knows, so everything is resolved on the device:
//
//   GLOBAL budget, score arrays from half the L2 size on: the band kernel and the
//   settle kernel (described where they are defined, further down) find the threshold in
//   one scan of the scores plus a sampled one; the multi-pass kernel below then only
//   redoes the problems they could not settle.  Otherwise:
//
//   select kernel (one persistent cooperative launch):
//   hist pass 0/1/2  radix select (11+11+10 bits) of the take-th largest key
//                    among the candidates; each CTA histograms its units of a
//                    problem in shared memory and merges into the problem's
//                    global histogram; the CTA that arrives last (atomic
//                    ticket) picks the digit and publishes it; CTAs wait (with
//                    a time limit) for the digits of the problems they scan.
//   mask pass        per token: definite bits (reserved, FULL, key > tau) and
//                    tie bits (key == tau); per-unit counts of both.
//   compact kernel   per tile: exclusive scan of the counts (tile base from the
//                    preceding units' sums), ties kept in flat-index order
//                    until the remaining rank is used up, final mask + offsets
//                    written, kept 16-byte chunks of V copied to the store.
//
// PER_TOKEN mode skips the histogram passes (the mask is local to a token).
// HBM traffic: scores 4x in the multi-pass kernel (3 passes + mask, from L2 when they
// fit), 1x plus the sample in the band kernel, 1x in PER_TOKEN mode; kept part of V once
// in and once out.
#include <atomic>

#include "common.cuh"

namespace stc {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kTile = 512;                    // tokens per CTA of the compaction kernel
constexpr int kUnit = kThreads;               // tokens per unit of the score scans (one per thread)
constexpr int kUnitsPerTile = kTile / kUnit;
constexpr int kTokPerThread = kTile / kThreads;
constexpr int kBins = 2048;

// state words per problem
enum { ST_NROUTED = 0, ST_PREFIX, ST_KREM, ST_FLAGS, ST_TICKET0, ST_TICKET1, ST_TICKET2, ST_DONE,
       // words of the band kernel (it leaves the eight above to the multi-pass kernel, except the results
       // ST_KREM / ST_FLAGS / ST_PREFIX that the compaction reads)
       ST_PATH, ST_BLO, ST_BHI, ST_LISTN, ST_TICKETA, ST_TICKETB, ST_DONEA, ST_NROUTEDA, ST_NROUTEDB, ST_ABOVE,
       ST_SPARE0, ST_SPARE1, ST_WORDS };
enum { FL_NONE = 1, FL_BUDGET = 2 };          // nothing beyond the reserved groups / budget error
enum { PATH_OPEN = 0, PATH_BAND = 1, PATH_WIDE = 2 };   // who settles the problem: nobody yet / band kernel / multi-pass kernel
// ST_DONE = histogram passes resolved so far (3 = threshold final)
constexpr int kBins13 = 8192;                 // first digit of the band kernel: the top 13 key bits
constexpr int kShift13 = 19;

struct RouteWs {
    uint32_t* state;      // [problems][ST_WORDS]
    uint32_t* hist;       // [problems][3][kBins]
    uint32_t* hist13;     // [problems][kBins13]
    uint32_t* abort_word; // set when a bounded wait gave up; the next word: some problem is left to the multi-pass kernel
    uint2* list;          // [problems][list_cap] (score bits, flat index) of the candidates inside the band
    uint32_t list_cap;
    uint32_t* unit_sums;  // [problems][units]: definite count | tie count << 16 (the band kernel adds to zeroed words)
    uint16_t* tie;        // [problems][T]
    size_t zero_small;    // leading bytes cleared per call: state and abort word only ...
    size_t zero_bytes;    // ... or with the global histograms (problems that span several CTAs)
    size_t total_bytes;
};

size_t align256(size_t x) { return (x + 255) & ~(size_t)255; }

RouteWs carve(const Geom& g, void* ws) {
    RouteWs r;
    char* p = static_cast<char*>(ws);
    const int n_units = (g.T + kUnit - 1) / kUnit;
    size_t o = 0;
    r.state = reinterpret_cast<uint32_t*>(p + o); o += align256((size_t)g.problems * ST_WORDS * 4);
    r.abort_word = reinterpret_cast<uint32_t*>(p + o); o += 256;
    r.zero_small = o;
    r.hist = reinterpret_cast<uint32_t*>(p + o);  o += align256((size_t)g.problems * 3 * kBins * 4);
    const bool small = n_units <= 32 / g.S;       // (the one-CTA-per-problem kernel needs neither of the next two)
    r.hist13 = reinterpret_cast<uint32_t*>(p + o); o += small ? 0 : align256((size_t)g.problems * kBins13 * 4);
    r.unit_sums = reinterpret_cast<uint32_t*>(p + o); o += align256((size_t)g.problems * n_units * 4);
    r.zero_bytes = o;
    r.tie = reinterpret_cast<uint16_t*>(p + o);   o += align256((size_t)g.problems * g.T * 2);
    // a sixteenth of a problem's keys (one bin of the 13-bit digit holds a few per cent at most on smooth data)
    const size_t cap = small ? 0 : (((size_t)g.T * g.S / 16 + 4095) & ~(size_t)4095);
    r.list_cap = (uint32_t)(cap < 0x40000000u ? cap : 0x40000000u);
    r.list = reinterpret_cast<uint2*>(p + o);     o += align256((size_t)g.problems * r.list_cap * sizeof(uint2));
    r.total_bytes = o;
    return r;
}

__device__ __forceinline__ int pass_shift(int pass) { return pass == 0 ? 21 : (pass == 1 ? 10 : 0); }
__device__ __forceinline__ uint32_t pass_himask(int pass) {
    return pass == 0 ? 0u : (pass == 1 ? 0xFFE00000u : 0xFFFFFC00u);
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
// Scores of one token -> order-preserving keys.
template <int S>
__device__ __forceinline__ void make_keys(const uint4 (&raw)[S / 4], uint32_t (&key)[S]) {
#pragma unroll
    for (int i = 0; i < S / 4; ++i) {
        const uint4 w = raw[i];
        key[4 * i + 0] = float_key(__uint_as_float(w.x));
        key[4 * i + 1] = float_key(__uint_as_float(w.y));
        key[4 * i + 2] = float_key(__uint_as_float(w.z));
        key[4 * i + 3] = float_key(__uint_as_float(w.w));
    }
}
// Index of the first maximum (tracked by value, so no register array is indexed at run time).
template <int S>
__device__ __forceinline__ int first_max(const uint32_t (&key)[S]) {
    uint32_t bk = key[0];
    int best = 0;
#pragma unroll
    for (int j = 1; j < S; ++j) {
        const bool up = key[j] > bk;
        bk = up ? key[j] : bk;
        best = up ? j : best;
    }
    return best;
}

__device__ __forceinline__ int token_class(const uint8_t* cls, int t, int len) {
    if (t >= len) return STC_CLS_DROP;
    return cls ? cls[t] : STC_CLS_ROUTED;
}

// The last CTA of a pass: find the bin holding the krem-th largest candidate.
template <bool kSharedHist>
__device__ void pick_digit(const uint32_t* __restrict__ hist, int nbins, uint32_t krem,
                           uint32_t* s_w, uint32_t* s_out /*[2]: digit, new krem*/) {
    // thread t owns bins nbins-1-8t .. nbins-8-8t (descending); nbins <= 8*kThreads
    uint32_t c[8], sum = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) {
        int bin = nbins - 1 - 8 * (int)threadIdx.x - j;
        c[j] = bin >= 0 ? (kSharedHist ? hist[bin] : __ldcg(hist + bin)) : 0u;
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
__device__ __forceinline__ uint32_t max_key(const uint32_t (&key)[S]) {
    uint32_t m = key[0];
#pragma unroll
    for (int j = 1; j + 1 < S; j += 2) m = max(m, max(key[j], key[j + 1]));
    return max(m, key[S - 1]);
}

// shist[bin] += delta when `on` (a predicated reduction: no branch per key).
__device__ __forceinline__ void red_if(bool on, uint32_t shist_base, uint32_t bin, int delta) {
    asm volatile(
        "{\n\t.reg .pred p;\n\tsetp.ne.u32 p, %0, 0;\n\t@p red.shared.add.u32 [%1], %2;\n\t}"
        ::"r"((uint32_t)on), "r"(shist_base + bin * 4u), "r"((uint32_t)delta) : "memory");
}

// Histogram contribution of one routed token in one pass: its keys that still match the
// resolved prefix, except the reserved first maximum (counted, then taken back: equal
// keys share a bin, so which of them is the reserved one does not matter here).
template <int S, bool kFirstPass>
__device__ __forceinline__ void hist_token(const uint32_t (&key)[S], uint32_t himask, uint32_t prefix, int dshift,
                                           uint32_t dmask, int min_per_token, uint32_t shist_base) {
    const uint32_t bk = max_key<S>(key);
    if (kFirstPass) {                              // every key is a candidate; the digit is the top 11 bits
#pragma unroll
        for (int j = 0; j < S; ++j) red_if(true, shist_base, key[j] >> 21, 1);
        red_if(min_per_token != 0, shist_base, bk >> 21, -1);
    } else {
#pragma unroll
        for (int j = 0; j < S; ++j)
            red_if((key[j] & himask) == prefix, shist_base, (key[j] >> dshift) & dmask, 1);
        red_if(min_per_token != 0 && (bk & himask) == prefix, shist_base, (bk >> dshift) & dmask, -1);
    }
}

// Bounds, as floats, of the keys that match a resolved prefix: lo <= x <= hi is what the
// later passes test before they build any key (scores are not NaN).
__device__ __forceinline__ void prefix_bounds(uint32_t prefix, uint32_t himask, float& lo, float& hi) {
    uint32_t klo = prefix, khi = prefix | ~himask;
    klo = max(klo, 0x007FFFFFu);                   // -inf
    khi = min(khi, 0xFF800000u);                   // +inf
    if (khi == 0x7FFFFFFFu) khi = 0x7FFFFFFEu;     // the key of -0 is unused: stop below zero
    lo = key_float(klo);
    hi = key_float(khi);
}
template <int S>
__device__ __forceinline__ bool any_in_bounds(const uint4 (&raw)[S / 4], float lo, float hi) {
    bool any = false;
#pragma unroll
    for (int i = 0; i < S / 4; ++i) {
        const float x0 = __uint_as_float(raw[i].x), x1 = __uint_as_float(raw[i].y);
        const float x2 = __uint_as_float(raw[i].z), x3 = __uint_as_float(raw[i].w);
        any |= (x0 >= lo && x0 <= hi) || (x1 >= lo && x1 <= hi) || (x2 >= lo && x2 <= hi) || (x3 >= lo && x3 <= hi);
    }
    return any;
}

// Definite and tie bits of one routed token against the final threshold.
template <int S>
__device__ __forceinline__ void mask_token(const uint32_t (&key)[S], int mode, uint32_t flags, uint32_t tau,
                                           int k_nominal, int min_per_token, uint32_t& def, uint32_t& tie) {
    def = 0;
    tie = 0;
    if (mode == STC_MODE_PER_TOKEN) {
#pragma unroll
        for (int j = 0; j < S; ++j) {
            int rank = 0;
#pragma unroll
            for (int i2 = 0; i2 < S; ++i2) rank += (key[i2] > key[j]) || (key[i2] == key[j] && i2 < j);
            if (rank < k_nominal) def |= 1u << j;
        }
        return;
    }
    if (!(flags & FL_NONE)) {
        bool any_tie = false;
#pragma unroll
        for (int j = 0; j < S; ++j) {
            def |= (key[j] > tau ? 1u : 0u) << j;
            any_tie |= key[j] == tau;
        }
        if (any_tie) {
#pragma unroll
            for (int j = 0; j < S; ++j) tie |= (key[j] == tau ? 1u : 0u) << j;
        }
    }
    if (min_per_token && def == 0u) {
        // The reserved group is the token's first maximum.  With a key above the threshold it is
        // among the definite bits already; with the maximum on the threshold it is the first tie.
        uint32_t bit;
        if (tie) bit = tie & (0u - tie);
        else bit = 1u << first_max<S>(key);
        def = bit;
        tie &= ~bit;
    }
}

// Budget of a problem from its routed-token count: flags (FL_*) and the number of pairs to
// take beyond the reserved ones.
__device__ __forceinline__ uint32_t budget_of(uint64_t n_routed, int k_nominal, int min_per_token, uint32_t& flags) {
    const uint64_t m_total = n_routed * (uint64_t)k_nominal;
    flags = 0;
    if (min_per_token && m_total < n_routed) flags = FL_BUDGET;
    const uint64_t take = m_total - (min_per_token ? n_routed : 0);
    if (!flags && take == 0) flags = FL_NONE;
    return (uint32_t)take;
}

// ---- bounded cross-CTA hand-off -------------------------------------------------
constexpr uint64_t kWaitNs = 2000000000ull;   // a wait that lasts this long gives up and reports a time-out
// Launch parameters of the selection kernel that only the library's own tests change (see
// stc_test_route_select_knobs at the end of this file): the first histogram pass to run and the
// limit of a hand-off wait.
std::atomic<int> g_first_pass{0};
std::atomic<unsigned long long> g_wait_ns{kWaitNs};

__device__ __forceinline__ uint64_t globaltimer_ns() {
    uint64_t t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ uint32_t ld_acquire(const uint32_t* p) {
    uint32_t v;
    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void st_release(uint32_t* p, uint32_t v) {
    asm volatile("st.release.gpu.global.u32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}

// Wait until `need` passes of the problem are resolved, then broadcast its state:
// s_bc = {ok, flags, prefix, krem}.  False (for the whole CTA) after a time-out or when
// another CTA has already given up.
__device__ __forceinline__ bool wait_done(const uint32_t* state, uint32_t need, uint32_t* s_bc,
                                          uint32_t* abort_word, uint64_t wait_ns) {
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t ok = 1;
        if (ld_acquire(state + ST_DONE) < need) {
            const uint64_t t0 = globaltimer_ns();
            while (ld_acquire(state + ST_DONE) < need) {
                __nanosleep(100);
                if (globaltimer_ns() - t0 > wait_ns || ld_acquire(abort_word) != 0u) { ok = 0; break; }
            }
        }
        if (!ok) atomicExch(abort_word, 1u);
        s_bc[0] = ok;
        s_bc[1] = __ldcg(state + ST_FLAGS);
        s_bc[2] = __ldcg(state + ST_PREFIX);
        s_bc[3] = __ldcg(state + ST_KREM);
    }
    __syncthreads();
    return s_bc[0] != 0u;
}

// One persistent, cooperatively launched kernel (every CTA is resident, so a CTA may
// wait for a digit another CTA publishes): the three histogram passes and the mask
// pass.  Work is cut into units of 256 tokens (one per thread); a CTA owns a fixed,
// contiguous range of the flat (problem, unit) sequence in every pass, and works through
// it one segment (its units of one problem) at a time.
template <int S>
__global__ void __launch_bounds__(kThreads, 4)
route_select_kernel(const float* __restrict__ scores, const uint8_t* __restrict__ cls, int64_t cls_b_stride,
                    int64_t cls_h_stride, const int32_t* __restrict__ seq_len, int Hkv, int T, int upp,
                    int k_nominal, int min_per_token, int mode, uint32_t* __restrict__ state_all,
                    uint32_t* __restrict__ hist_all, uint32_t* __restrict__ abort_word,
                    uint16_t* __restrict__ v_mask, uint16_t* __restrict__ tie_all,
                    uint32_t* __restrict__ unit_sums, long long total_units, int first_pass,
                    unsigned long long wait_ns, int only_wide) {
    constexpr int kBatch = 32 / S;               // tokens in flight per thread (32 score registers)
    // after the band kernel: only the problems it left (PATH_WIDE) are this kernel's, usually none
    if (only_wide && __ldcg(abort_word + 1) == 0u) return;
    __shared__ uint32_t shist[kBins];
    __shared__ uint32_t s_w[kWarps];
    __shared__ uint32_t s_red[kBatch][kWarps];
    __shared__ uint32_t s_pick[2];
    __shared__ uint32_t s_bc[4];
    __shared__ int s_last;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const long long x0 = total_units * blockIdx.x / gridDim.x;
    const long long x1 = total_units * (blockIdx.x + 1) / gridDim.x;
    const int n_pass = mode == STC_MODE_GLOBAL ? 3 : 0;

#pragma unroll 1
    for (int pass = first_pass; pass < n_pass; ++pass) {
        const uint32_t himask = pass_himask(pass);
        const int dshift = pass_shift(pass);
        const uint32_t dmask = pass == 2 ? 1023u : 2047u;
#pragma unroll 1
        for (long long x = x0; x < x1;) {
            const int problem = (int)(x / upp);
            const int u0 = (int)(x - (long long)problem * upp);
            const int n = (int)min((long long)(upp - u0), x1 - x);
            x += n;
            const int b = problem / Hkv, hk = problem - b * Hkv;
            const int len = clamp_len(seq_len, b, T);
            uint32_t* state = state_all + (size_t)problem * ST_WORDS;
            if (only_wide && __ldcg(state + ST_PATH) != PATH_WIDE) continue;
            uint32_t* hist = hist_all + ((size_t)problem * 3 + pass) * kBins;
            const uint8_t* c = cls ? cls + (size_t)b * cls_b_stride + (size_t)hk * cls_h_stride : nullptr;
            uint4 raw[kBatch][S / 4];
            bool routed[kBatch];
            const float* rows = scores + (size_t)problem * T * S;
            auto load_batch = [&](int u) {               // all of the thread's loads are in flight before the first use
#pragma unroll
                for (int i = 0; i < kBatch; ++i) {
                    const int t = (u + i) * kUnit + tid;
                    routed[i] = u + i < u0 + n && token_class(c, t, len) == STC_CLS_ROUTED;
                    load_raw<S>(rows + (size_t)min(t, T - 1) * S, raw[i]);   // unconditional: no branch per token
                }
            };
            load_batch(u0);                              // in flight while the digit of the previous pass arrives
            uint32_t prefix = 0, krem_in = 0;
            if (pass > 0) {
                if (!wait_done(state, (uint32_t)pass, s_bc, abort_word, wait_ns)) return;
                if (s_bc[1] != 0u) continue;             // nothing to select / budget error: resolved in pass 0
                prefix = s_bc[2];
                krem_in = s_bc[3];
            }
            for (int i = tid; i < kBins; i += kThreads) shist[i] = 0;
            __syncthreads();
            float lo, hi;
            prefix_bounds(prefix, himask, lo, hi);
            const uint32_t shist_base = smem_u32(shist);

            uint32_t n_routed = 0;
#pragma unroll 1
            for (int u = u0; u < u0 + n; u += kBatch) {
                if (u * kUnit >= len) break;
                if (u != u0) load_batch(u);
                if (pass == 0) {
#pragma unroll
                    for (int i = 0; i < kBatch; ++i) {
                        n_routed += routed[i];
                        if (routed[i]) {
                            uint32_t key[S];
                            make_keys<S>(raw[i], key);
                            hist_token<S, true>(key, 0u, 0u, 21, 2047u, min_per_token, shist_base);
                        }
                    }
                } else {
#pragma unroll
                    for (int i = 0; i < kBatch; ++i) {
                        if (routed[i] && any_in_bounds<S>(raw[i], lo, hi)) {
                            uint32_t key[S];
                            make_keys<S>(raw[i], key);
                            hist_token<S, false>(key, himask, prefix, dshift, dmask, min_per_token, shist_base);
                        }
                    }
                }
            }
            __syncthreads();
            for (int i = tid; i < kBins; i += kThreads) {
                const uint32_t v = shist[i];
                if (v) atomicAdd(hist + i, v);
            }
            if (pass == 0) {
                uint32_t tot;
                block_excl_scan(n_routed, s_w, &tot);
                if (tid == 0 && tot) atomicAdd(state + ST_NROUTED, tot);
            }
            __threadfence();
            __syncthreads();
            if (tid == 0)
                s_last = (atomicAdd(state + ST_TICKET0 + pass, (unsigned)n) + (unsigned)n == (unsigned)upp);
            __syncthreads();
            if (!s_last) continue;
            __threadfence();

            // the CTA that completed the problem's pass picks the digit and publishes it
            uint32_t krem = krem_in, flags = 0;
            if (pass == 0) {
                krem = budget_of(__ldcg(state + ST_NROUTED), k_nominal, min_per_token, flags);
            }
            if (flags) {
                if (tid == 0) { state[ST_FLAGS] = flags; state[ST_PREFIX] = 0; state[ST_KREM] = 0; }
            } else {
                pick_digit<false>(hist, pass == 2 ? 1024 : kBins, krem, s_w, s_pick);
                if (tid == 0) {
                    state[ST_PREFIX] = prefix | (s_pick[0] << pass_shift(pass));
                    state[ST_KREM] = s_pick[1];
                }
            }
            if (tid == 0) {
                __threadfence();
                st_release(state + ST_DONE, flags ? 3u : (uint32_t)(pass + 1));
            }
        }
    }

    // ---- mask pass: definite bits, tie bits and their per-unit counts ------------------
#pragma unroll 1
    for (long long x = x0; x < x1;) {
        const int problem = (int)(x / upp);
        const int u0 = (int)(x - (long long)problem * upp);
        const int n = (int)min((long long)(upp - u0), x1 - x);
        x += n;
        const int b = problem / Hkv, hk = problem - b * Hkv;
        const int len = clamp_len(seq_len, b, T);
        if (only_wide && __ldcg(state_all + (size_t)problem * ST_WORDS + ST_PATH) != PATH_WIDE) continue;
        const uint8_t* c = cls ? cls + (size_t)b * cls_b_stride + (size_t)hk * cls_h_stride : nullptr;
        uint4 raw[kBatch][S / 4];
        int cls_of[kBatch];
        const float* rows = scores + (size_t)problem * T * S;
        auto load_batch = [&](int u) {
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                const int t = (u + i) * kUnit + tid;
                cls_of[i] = (u + i < u0 + n && t < T) ? token_class(c, t, len) : STC_CLS_DROP;
                load_raw<S>(rows + (size_t)min(t, T - 1) * S, raw[i]);
            }
        };
        load_batch(u0);                                  // in flight while the last digit arrives
        uint32_t tau = 0, flags = 0;
        if (mode == STC_MODE_GLOBAL) {
            if (!wait_done(state_all + (size_t)problem * ST_WORDS, 3u, s_bc, abort_word, wait_ns)) return;
            flags = s_bc[1];
            tau = s_bc[2];
        }
#pragma unroll 1
        for (int u = u0; u < u0 + n; u += kBatch) {
            if (u != u0) load_batch(u);
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                const int t = (u + i) * kUnit + tid;
                const int cl = cls_of[i];
                uint32_t def = 0, tie = 0;
                if (flags & FL_BUDGET) {
                    def = 0;
                } else if (cl == STC_CLS_FULL) {
                    def = (1u << S) - 1u;
                } else if (cl == STC_CLS_ROUTED) {
                    uint32_t key[S];
                    make_keys<S>(raw[i], key);
                    mask_token<S>(key, mode, flags, tau, k_nominal, min_per_token, def, tie);
                }
                if (u + i < u0 + n && t < T) {
                    v_mask[(size_t)problem * T + t] = (uint16_t)def;
                    tie_all[(size_t)problem * T + t] = (uint16_t)tie;
                }
                // a unit holds at most 256 * 16 bits of each kind: both counts fit one word
                const uint32_t cnt = __reduce_add_sync(0xFFFFFFFFu, __popc(def) | (__popc(tie) << 16));
                if (lane == 0) s_red[i][warp] = cnt;
            }
            __syncthreads();
            if (tid < kBatch && u + tid < u0 + n) {
                uint32_t tot = 0;
#pragma unroll
                for (int w2 = 0; w2 < kWarps; ++w2) tot += s_red[tid][w2];
                unit_sums[(size_t)problem * upp + u + tid] = tot;
            }
            __syncthreads();
        }
    }
}

// ---- the band kernel -----------------------------------------------------------------------
// One scan of the scores (and a fraction of another) instead of four.
//   Scan A looks at a sample of every problem (runs of four consecutive tokens, evenly spread; all
//   tokens when the problem is small) and histograms the top 13 key bits of the sample's candidates.
//   The CTA that completes a problem's sample derives a BAND of bins that holds the take-th largest
//   candidate of the whole problem with near certainty: the bins of the sample ranks
//   f m -+ (5 sqrt(m f (1 - f)) + 2), f = take / candidates = (K - floor) / (S - floor), m = sample size.
//   Scan B reads every score once: candidates above the band are kept (their definite bits are
//   written straight away and counted), those below are dropped, those inside -- a per cent or two
//   of the problem -- are appended as (key, flat index) pairs to the problem's list.  All tests are
//   float comparisons against the band's two edges; keys are only built for the list.
//   The settle kernel (next launch, one CTA per problem) settles each problem exactly: with `above`
//   pairs counted above the band, the take-th largest candidate is the (take - above)-th largest of
//   the list, provided above < take <= above + list length -- which is the check that the band was
//   right.  Radix select over the list, then one pass that sets the definite bit of every listed pair
//   above the threshold; the pairs on the threshold are ranked by flat index and the lowest are kept
//   (the rule the compaction applies to the tie bits of the multi-pass kernel), so a settled problem
//   has no tie bits and its part of the tie array is neither cleared nor read.
// A problem whose band was wrong, or holds more pairs than the list has room for (massive ties), is
// or has more than a few thousand pairs on the threshold, is marked PATH_WIDE and left to the multi-pass
// kernel that runs next; the result is the same either way.

template <bool kSharedHist>
__device__ void pick_digit_n(const uint32_t* __restrict__ hist, int nbins, int per, uint32_t krem,
                             uint32_t* s_w, uint32_t* s_out /*[3]*/) {
    const int top = nbins - 1 - per * (int)threadIdx.x;
    uint32_t sum = 0;
    // a histogram in global memory: the thread's bins are `per` consecutive words ending at `top`, read as
    // 16-byte pieces that are all in flight together (per = 32, nbins = per * kThreads)
    constexpr int kQuads = 8;
    const bool quads = !kSharedHist && per == 4 * kQuads && top - per + 1 >= 0;
    uint32_t qsum[kQuads];
    if (quads) {
        const uint4* h4 = reinterpret_cast<const uint4*>(hist + top - per + 1);
#pragma unroll
        for (int j = 0; j < kQuads; ++j) {
            const uint4 v = __ldcg(h4 + j);
            qsum[j] = v.x + v.y + v.z + v.w;
            sum += qsum[j];
        }
    } else {
#pragma unroll 4
        for (int j = 0; j < per; ++j) {
            const int bin = top - j;
            sum += bin >= 0 ? (kSharedHist ? hist[bin] : __ldcg(hist + bin)) : 0u;
        }
    }
    const uint32_t excl = block_excl_scan(sum, s_w, nullptr);
    if (excl < krem && krem <= excl + sum) {
        uint32_t run = excl;
        int j0 = 0, j1 = per;
        if (quads) {                                // first the piece (from the top one down), then the bin inside it
            int piece = 0;
            bool found = false;
#pragma unroll
            for (int q = kQuads - 1; q >= 0; --q) {
                if (!found) {
                    if (run + qsum[q] >= krem) { piece = q; found = true; }
                    else run += qsum[q];
                }
            }
            j0 = (kQuads - 1 - piece) * 4;
            j1 = j0 + 4;
        }
        for (int j = j0; j < j1; ++j) {
            const int bin = top - j;
            const uint32_t c = bin >= 0 ? (kSharedHist ? hist[bin] : __ldcg(hist + bin)) : 0u;
            if (run + c >= krem) {
                s_out[0] = (uint32_t)bin;
                s_out[1] = krem - run;
                s_out[2] = c;
                break;
            }
            run += c;
        }
    }
    __syncthreads();
}

// Sets bits of a 16-bit mask word that other threads may be updating.  word_ok: the mask array starts
// on a 4-byte boundary and a problem's masks never share a 32-bit word with another problem's, so the
// update can be a 32-bit reduction (nothing comes back, nothing waits); otherwise a 16-bit
// compare-and-swap loop.
__device__ __forceinline__ void or16(uint16_t* p, uint32_t bits, bool word_ok) {
    if (word_ok) {
        const uintptr_t a = reinterpret_cast<uintptr_t>(p);
        atomicOr(reinterpret_cast<unsigned int*>(a & ~(uintptr_t)3), bits << ((a & 2) ? 16 : 0));
    } else {
        unsigned short* q = reinterpret_cast<unsigned short*>(p);
        unsigned short old = *reinterpret_cast<volatile unsigned short*>(q), assumed;
        do {
            assumed = old;
            old = atomicCAS(q, assumed, (unsigned short)(assumed | bits));
        } while (old != assumed);
    }
}

// Wait (bounded) until the problem's band is published, then broadcast it: s_bc = {ok, path, b_lo, b_hi}.
__device__ __forceinline__ bool wait_band(const uint32_t* state, uint32_t* s_bc, uint32_t* abort_word,
                                          uint64_t wait_ns) {
    __syncthreads();
    if (threadIdx.x == 0) {
        uint32_t ok = 1;
        if (ld_acquire(state + ST_DONEA) == 0u) {
            const uint64_t t0 = globaltimer_ns();
            while (ld_acquire(state + ST_DONEA) == 0u) {
                __nanosleep(100);
                if (globaltimer_ns() - t0 > wait_ns || ld_acquire(abort_word) != 0u) { ok = 0; break; }
            }
        }
        if (!ok) atomicExch(abort_word, 1u);
        s_bc[0] = ok;
        s_bc[1] = __ldcg(state + ST_PATH);
        s_bc[2] = __ldcg(state + ST_BLO);
        s_bc[3] = __ldcg(state + ST_BHI);
    }
    __syncthreads();
    return s_bc[0] != 0u;
}

// The scores whose 13-bit digit lies in [b_lo, b_hi], as a closed float interval (scores are not NaN).
__device__ __forceinline__ void band_bounds(uint32_t b_lo, uint32_t b_hi, float& lo, float& hi) {
    uint32_t klo = b_lo << kShift13, khi = (b_hi << kShift13) | ((1u << kShift13) - 1u);
    klo = max(klo, 0x00800000u);                   // -FLT_MAX: the edges stay finite (band_token subtracts them), and an
    khi = min(khi, 0xFF7FFFFFu);                   // +FLT_MAX  infinite score is then simply below or above the band
    if (khi == 0x7FFFFFFFu) khi = 0x7FFFFFFEu;     // the key of -0 is unused: stop below zero
    lo = key_float(klo);
    hi = key_float(khi);
}

// Definite bits and list candidates of one routed token against the band, on the raw scores.  The scan is
// bound by the integer / compare pipe, so the work per score is kept to two comparisons: one against each
// edge (a candidate is at or above the lower edge and not above the upper one).  The reserved group -- the
// token's first maximum -- only has to be looked for when no score lies above the band: otherwise the
// maximum is above the band too, and it changes neither the definite bits nor the candidates.
template <int S>
__device__ __forceinline__ void band_token(const uint4 (&raw)[S / 4], bool select, float lo, float hi,
                                           int min_per_token, uint32_t& def, uint32_t& cand) {
    float x[S];
#pragma unroll
    for (int i = 0; i < S / 4; ++i) {
        x[4 * i + 0] = __uint_as_float(raw[i].x);
        x[4 * i + 1] = __uint_as_float(raw[i].y);
        x[4 * i + 2] = __uint_as_float(raw[i].z);
        x[4 * i + 3] = __uint_as_float(raw[i].w);
    }
    def = 0;
    cand = 0;
    if (select) {
        // x > hi  <=>  hi - x is negative, x >= lo  <=>  x - lo is not (a difference of two different floats is
        // never zero without flush-to-zero, which this library is not built with; equal floats give +0): the
        // subtractions run on the FMA pipe, which the scan leaves idle, and one funnel shift per score moves the
        // sign into the mask, instead of compare + select + or on the pipe the scan is bound by.  The edges are
        // finite (band_bounds), so an infinite score is simply above or below the band.
        uint32_t above = 0, below = 0;
#pragma unroll
        for (int j = S - 1; j >= 0; --j) {
            const float xj = __fadd_rn(x[j], 0.f);   // -0 -> +0, as in the keys (-0 - +0 would be -0)
            above = __funnelshift_l(__float_as_uint(__fsub_rn(hi, xj)), above, 1);
            below = __funnelshift_l(__float_as_uint(__fsub_rn(xj, lo)), below, 1);
        }
        def = above;
        cand = ~below & ~above & ((1u << S) - 1u);
    }
    if (min_per_token && def == 0u) {
        float bx = x[0];
        int best = 0;
#pragma unroll
        for (int j = 1; j < S; ++j) {
            const bool up = x[j] > bx;             // (-0 and +0 compare equal here and as keys)
            bx = up ? x[j] : bx;
            best = up ? j : best;
        }
        def = 1u << best;
        cand &= ~def;
    }
}

// ---- the settle kernel: one CTA of 1024 threads per problem, after the band kernel -------------
// Checks the band (above < take <= above + list length), finds the (take - above)-th largest key of the
// list by radix select (11 + 11 + 10 bits; the keys are staged in shared memory when they fit, else every
// pass reads the list, which sits in L2), then sets the definite bit of every listed pair above the
// threshold and of the lowest-indexed pairs on it, and adds them to the per-unit counts.
constexpr int kSettleThreads = 1024;
constexpr int kSettleWarps = kSettleThreads / 32;
constexpr int kSettleKeys = 45056;                 // keys staged in shared memory (176 KiB)
constexpr size_t kSettleSmem = (size_t)kSettleKeys * 4;

// Exclusive scan of one value per thread over a CTA of 1024 threads (the band and the settle kernel).
__device__ __forceinline__ uint32_t settle_excl_scan(uint32_t v, uint32_t* s_w /*[kSettleWarps]*/) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const uint32_t incl = warp_incl_scan(v, lane);
    __syncthreads();
    if (lane == 31) s_w[warp] = incl;
    __syncthreads();
    uint32_t base = 0;
    for (int w = 0; w < warp; ++w) base += s_w[w];
    return base + incl - v;
}
// The bin holding the krem-th largest count of a histogram (thread t owns the `per` bins nbins-1-per*t
// downwards; nbins = per * 1024; kGlobal: the histogram is in global memory and per = 8, read as two
// 16-byte pieces).  s_out = {bin, rank inside it}.
template <bool kGlobal>
__device__ __forceinline__ void settle_pick(const uint32_t* hist, int nbins, int per, uint32_t krem, uint32_t* s_w,
                                            uint32_t* s_out) {
    const int top = nbins - 1 - per * (int)threadIdx.x;
    uint32_t c[8];
    if (kGlobal) {
        const uint4 a = __ldcg(reinterpret_cast<const uint4*>(hist + top - 7));
        const uint4 b = __ldcg(reinterpret_cast<const uint4*>(hist + top - 3));
        c[7] = a.x; c[6] = a.y; c[5] = a.z; c[4] = a.w; c[3] = b.x; c[2] = b.y; c[1] = b.z; c[0] = b.w;   // c[j] = bin top - j
    } else {
#pragma unroll
        for (int j = 0; j < 8; ++j) c[j] = j < per ? hist[top - j] : 0u;
    }
    uint32_t sum = 0;
#pragma unroll
    for (int j = 0; j < 8; ++j) sum += c[j];
    const uint32_t excl = settle_excl_scan(sum, s_w);
    if (excl < krem && krem <= excl + sum) {
        uint32_t run = excl;
        bool found = false;
#pragma unroll
        for (int j = 0; j < 8; ++j) {
            if (!found && run + c[j] >= krem) { s_out[0] = (uint32_t)(top - j); s_out[1] = krem - run; found = true; }
            run += c[j];
        }
    }
    __syncthreads();
}

template <int S>
__global__ void __launch_bounds__(kSettleThreads, 1)
route_settle_kernel(uint32_t* __restrict__ state_all, uint32_t* __restrict__ abort_word,
                    const uint2* __restrict__ list_all, uint32_t list_cap, uint16_t* __restrict__ v_mask,
                    uint32_t* __restrict__ unit_sums, int T, int upp, int k_nominal, int min_per_token) {
    extern __shared__ __align__(16) uint32_t s_keys[];
    __shared__ uint32_t shist[2048];
    __shared__ uint32_t s_w[kSettleWarps];
    __shared__ uint32_t s_pick[2];
    __shared__ uint32_t s_ntie;
    constexpr int kTieRankMax = 4096;                    // pairs on the threshold that are ranked here (all-pairs count)
    const int tid = threadIdx.x;
    const int problem = blockIdx.x;
    uint32_t* state = state_all + (size_t)problem * ST_WORDS;
    if (__ldcg(abort_word) != 0u || __ldcg(state + ST_PATH) != PATH_BAND) return;   // a wait gave up: nothing is settled
    const bool select = k_nominal > (min_per_token ? 1 : 0);
    uint32_t flags = 0;
    const uint32_t take = budget_of(__ldcg(state + ST_NROUTEDB), k_nominal, min_per_token, flags);
    const uint32_t above = __ldcg(state + ST_ABOVE), n_list = __ldcg(state + ST_LISTN);
    if (flags || !select) {                              // nothing beyond the reserved groups (budget errors do not come here)
        if (tid == 0) { state[ST_FLAGS] = flags; state[ST_KREM] = 0u; state[ST_PREFIX] = 0u; }
        return;
    }
    if (!(n_list <= list_cap && above < take && take - above <= n_list)) {
        if (tid == 0) {                                  // the band missed the threshold, or the list overflowed
            state[ST_PATH] = PATH_WIDE;
            atomicExch(abort_word + 1, 1u);
        }
        return;
    }
    const uint2* list = list_all + (size_t)problem * list_cap;
    const bool word_ok = (reinterpret_cast<uintptr_t>(v_mask) & 3u) == 0 && (T & 1) == 0;
    uint16_t* mask_row = v_mask + (size_t)problem * T;
    uint32_t* sums_row = unit_sums + (size_t)problem * upp;
    constexpr int kInFlight = 8;                         // list entries a thread has in flight
    const bool staged = n_list <= (uint32_t)kSettleKeys;
    if (staged) {
#pragma unroll 1
        for (uint32_t e0 = tid; e0 < n_list; e0 += kInFlight * kSettleThreads) {
            uint32_t w[kInFlight];
#pragma unroll
            for (int i = 0; i < kInFlight; ++i) w[i] = __ldcg(&list[min(e0 + i * kSettleThreads, n_list - 1)].x);
#pragma unroll
            for (int i = 0; i < kInFlight; ++i)
                if (e0 + i * kSettleThreads < n_list) s_keys[e0 + i * kSettleThreads] = float_key(__uint_as_float(w[i]));
        }
    }
    auto key_at = [&](uint32_t e) {
        return staged ? s_keys[e] : float_key(__uint_as_float(__ldcg(&list[e].x)));
    };
    uint32_t prefix = 0, krem = take - above;
#pragma unroll 1
    for (int pass = 0; pass < 3; ++pass) {               // 11 + 11 + 10 bits
        const uint32_t himask = pass_himask(pass);
        const int dshift = pass_shift(pass);
        const int nbins = pass == 2 ? 1024 : 2048;
        for (int i = tid; i < nbins; i += kSettleThreads) shist[i] = 0u;
        __syncthreads();
#pragma unroll 4
        for (uint32_t e = tid; e < n_list; e += kSettleThreads) {
            const uint32_t k = key_at(e);
            if ((k & himask) == prefix) atomicAdd(&shist[(k >> dshift) & (uint32_t)(nbins - 1)], 1u);
        }
        __syncthreads();
        settle_pick<false>(shist, nbins, nbins / kSettleThreads, krem, s_w, s_pick);
        prefix |= s_pick[0] << dshift;
        krem = s_pick[1];
        __syncthreads();
    }
    const uint32_t tau = prefix;                         // krem: how many of the pairs on the threshold are kept
    // the per-unit counts of what is added are gathered in the histogram's words when the problem's units fit there
    const bool local_sums = upp <= 2048;
    if (local_sums) for (int i = tid; i < upp; i += kSettleThreads) shist[i] = 0u;
    if (tid == 0) s_ntie = 0u;
    uint32_t* s_ties = s_keys;                           // (the staged keys have served)
    __syncthreads();
    auto keep = [&](uint32_t flat) {                     // the pair's definite bit and its unit's count
        const uint32_t t = flat / S, j = flat - t * S;
        or16(mask_row + t, 1u << j, word_ok);
        if (local_sums) atomicAdd(&shist[t / kUnit], 1u);
        else atomicAdd(sums_row + t / kUnit, 1u);
    };
#pragma unroll 1
    for (uint32_t e0 = tid; e0 < n_list; e0 += kInFlight * kSettleThreads) {
        uint2 en[kInFlight];
#pragma unroll
        for (int i = 0; i < kInFlight; ++i) en[i] = __ldcg(&list[min(e0 + i * kSettleThreads, n_list - 1)]);
#pragma unroll
        for (int i = 0; i < kInFlight; ++i) {
            const uint32_t key = float_key(__uint_as_float(en[i].x));
            if (e0 + i * kSettleThreads >= n_list || key < tau) continue;
            if (en[i].y / S >= (uint32_t)T) continue;    // (cannot happen: the scan wrote the entry)
            if (key > tau) {
                keep(en[i].y);
            } else {                                     // on the threshold: settled below, in flat-index order
                const uint32_t at = atomicAdd(&s_ntie, 1u);
                if (at < (uint32_t)kSettleKeys) s_ties[at] = en[i].y;
            }
        }
    }
    __syncthreads();
    // The pairs on the threshold: the krem lowest flat indices are kept.  (A problem's tie array is not
    // used after this kernel -- the compaction does not read it for a settled problem -- so the scan did
    // not have to clear it.)
    const uint32_t n_tie = s_ntie;
    if (n_tie > (uint32_t)kSettleKeys || (krem < n_tie && n_tie > (uint32_t)kTieRankMax)) {   // massive ties: the multi-pass kernel redoes the problem
        if (tid == 0) {
            state[ST_PATH] = PATH_WIDE;
            atomicExch(abort_word + 1, 1u);
        }
        return;
    }
    for (uint32_t e = tid; e < n_tie; e += kSettleThreads) {
        const uint32_t flat = s_ties[e];
        uint32_t rank = 0;
        if (krem < n_tie)
            for (uint32_t o = 0; o < n_tie; ++o) rank += s_ties[o] < flat;
        if (rank < krem) keep(flat);
    }
    if (local_sums) {
        __syncthreads();
        for (int i = tid; i < upp; i += kSettleThreads) {       // (nobody else touches the problem's counts now)
            const uint32_t v = shist[i];
            if (v) sums_row[i] += v;
        }
    }
    if (tid == 0) { state[ST_FLAGS] = 0u; state[ST_PREFIX] = tau; state[ST_KREM] = 0u; }
}

// samp: a power of two up to 16 -- scan A looks at one token in `samp`.  z_tenths: the band's half-width in tenths of
// a standard deviation of the sample rank (50 in production).
// One CTA of 1024 threads per SM: the CTAs of an SM that start at different times do not advance at the
// same pace (the warp schedulers favour the older one), and with static ranges the youngest of four sets
// the kernel's time.  The warps of one CTA are of one age, and in scan B they draw their work (items of
// 32 * kBatch consecutive tokens) from a counter in shared memory, so they end a segment together.
constexpr int kBandThreads = 1024;
constexpr int kBandWarps = kBandThreads / 32;
constexpr int kBandStage = 64;                   // list entries a warp can hold back
template <int S>
constexpr size_t band_smem_bytes() {             // dynamic: the warps' staging slots, one scratch row per thread
    return (size_t)kBandWarps * kBandStage * sizeof(uint2) + (size_t)kBandThreads * S * 4;
}

template <int S>
__global__ void __launch_bounds__(kBandThreads, 1)
route_band_kernel(const float* __restrict__ scores, const uint8_t* __restrict__ cls, int64_t cls_b_stride,
                  int64_t cls_h_stride, const int32_t* __restrict__ seq_len, int Hkv, int T, int upp,
                  int k_nominal, int min_per_token, uint32_t* __restrict__ state_all,
                  uint32_t* __restrict__ hist_all, uint32_t* __restrict__ abort_word,
                  uint16_t* __restrict__ v_mask, uint32_t* __restrict__ unit_sums, uint2* __restrict__ list_all,
                  uint32_t list_cap, long long total_units, int skip_scan_a, unsigned long long wait_ns, int samp,
                  int z_tenths) {
    constexpr int kBatch = S >= 8 ? 32 / S : 4;  // tokens in flight per thread (at most 32 score registers)
    extern __shared__ __align__(16) uint32_t band_dyn[];
    __shared__ __align__(16) uint32_t shist[kBins13];
    __shared__ uint32_t s_w[kBandWarps];
    __shared__ uint32_t s_pick[2];
    __shared__ uint32_t s_bc[4];
    __shared__ uint32_t s_cnt[2];
    __shared__ uint32_t s_next;
    __shared__ int s_last;
    // scan B has no use for the histogram: its words hold the segment's per-unit counts
    constexpr int kUnitsMax = kBins13;
    uint32_t* s_units = shist;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    uint2* stage = reinterpret_cast<uint2*>(band_dyn) + warp * kBandStage;
    uint32_t* s_row = band_dyn + kBandWarps * kBandStage * 2 + tid * S;
    const long long x0 = total_units * blockIdx.x / gridDim.x;
    const long long x1 = total_units * (blockIdx.x + 1) / gridDim.x;
    const int floor_k = min_per_token ? 1 : 0;
    // nothing beyond the reserved groups is ever taken: no threshold, scan B alone
    const bool select = k_nominal > floor_k;

    // ---- scan A: histogram of the top 13 key bits of the sample's candidates ---------------------
    // the CTA covers 4 * samp units at a time: thread -> (unit du of those, sampled token sidx of the unit)
    const int per_unit = kUnit / samp;               // sampled tokens per unit
    const int du = tid / per_unit, sidx = tid - du * per_unit;
    const int group = (kBandThreads / kUnit) * samp; // units per step of a thread
#pragma unroll 1
    for (long long x = (skip_scan_a || !select) ? x1 : x0; x < x1;) {
        const int problem = (int)(x / upp);
        const int u0 = (int)(x - (long long)problem * upp);
        const int n = (int)min((long long)(upp - u0), x1 - x);
        x += n;
        const int b = problem / Hkv, hk = problem - b * Hkv;
        const int len = clamp_len(seq_len, b, T);
        uint32_t* state = state_all + (size_t)problem * ST_WORDS;
        uint32_t* hist = hist_all + (size_t)problem * kBins13;
        const uint8_t* c = cls ? cls + (size_t)b * cls_b_stride + (size_t)hk * cls_h_stride : nullptr;
        const float* rows = scores + (size_t)problem * T * S;
        for (int i = tid; i < kBins13; i += kBandThreads) shist[i] = 0;
        if (tid == 0) s_cnt[0] = 0u;
        __syncthreads();
        const uint32_t shist_base = smem_u32(shist);
        uint32_t n_routed = 0;
#pragma unroll 1
        for (int v = u0; v < u0 + n; v += group * kBatch) {
            if (v * kUnit >= len) break;
            uint4 raw[kBatch][S / 4];
            bool routed[kBatch];
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {           // all of the thread's loads are in flight before the first use
                // the thread's token of unit `unit`: run (sidx / 4) of the unit's sampled runs of four tokens;
                // the runs of a unit start every 4 * samp tokens, shifted by the unit's number
                const int unit = v + i * group + du;
                const int t = unit * kUnit + ((((sidx >> 2) * samp + (unit & (samp - 1))) << 2) | (sidx & 3));
                routed[i] = unit < u0 + n && token_class(c, t, len) == STC_CLS_ROUTED;
                load_raw<S>(rows + (size_t)min(t, T - 1) * S, raw[i]);
            }
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                n_routed += routed[i];
                if (routed[i]) {
                    uint32_t key[S];
                    make_keys<S>(raw[i], key);
#pragma unroll
                    for (int j = 0; j < S; ++j) red_if(true, shist_base, key[j] >> kShift13, 1);
                    red_if(min_per_token != 0, shist_base, max_key<S>(key) >> kShift13, -1);
                }
            }
        }
        n_routed = __reduce_add_sync(0xFFFFFFFFu, n_routed);
        if (lane == 0 && n_routed) atomicAdd(&s_cnt[0], n_routed);
        __syncthreads();
        for (int i = tid; i < kBins13; i += kBandThreads) {
            const uint32_t v = shist[i];
            if (v) atomicAdd(hist + i, v);
        }
        if (tid == 0 && s_cnt[0]) atomicAdd(state + ST_NROUTEDA, s_cnt[0]);
        __threadfence();
        __syncthreads();
        if (tid == 0)
            s_last = (atomicAdd(state + ST_TICKETA, (unsigned)n) + (unsigned)n == (unsigned)upp);
        __syncthreads();
        if (!s_last) continue;
        __threadfence();

        // the CTA that completed the problem's sample derives the band and publishes it
        const uint32_t n_s = __ldcg(state + ST_NROUTEDA);
        const uint32_t m_c = n_s * (uint32_t)(S - floor_k);           // candidates in the sample
        uint32_t b_lo = 0, b_hi = kBins13 - 1;
        if (m_c > 0) {
            float r_hi, r_lo;                                         // sample ranks (1 = largest) that bracket the threshold
            if (samp == 1) {
                r_hi = r_lo = (float)(n_s * (uint32_t)(k_nominal - floor_k));
            } else {
                const float f = (float)(k_nominal - floor_k) / (float)(S - floor_k);
                const float r = f * (float)m_c;
                const float d = 0.1f * (float)z_tenths * sqrtf((float)m_c * f * (1.f - f)) + 2.f;
                r_hi = floorf(r - d);
                r_lo = ceilf(r + d);
            }
            if (r_hi >= 1.f) {
                settle_pick<true>(hist, kBins13, kBins13 / kBandThreads, (uint32_t)r_hi, s_w, s_pick);
                b_hi = s_pick[0];
                __syncthreads();
            }
            if (r_lo <= (float)m_c) {
                settle_pick<true>(hist, kBins13, kBins13 / kBandThreads, (uint32_t)r_lo, s_w, s_pick);
                b_lo = s_pick[0];
                __syncthreads();
            }
        }
        if (tid == 0) {
            state[ST_BLO] = b_lo;
            state[ST_BHI] = b_hi;
            state[ST_PATH] = PATH_BAND;
            __threadfence();
            st_release(state + ST_DONEA, 1u);
        }
    }

    // ---- scan B: definite bits above the band, the list inside it, counts ----------------------
    constexpr int kItemTokens = 32 * kBatch;             // a warp's item: kBatch runs of 32 consecutive tokens
#pragma unroll 1
    for (long long x = x0; x < x1;) {
        const int problem = (int)(x / upp);
        const int u0 = (int)(x - (long long)problem * upp);
        const int n = (int)min((long long)min(upp - u0, kUnitsMax), x1 - x);   // (its unit counts fit the scratch)
        x += n;
        const int b = problem / Hkv, hk = problem - b * Hkv;
        const int len = clamp_len(seq_len, b, T);
        uint32_t* state = state_all + (size_t)problem * ST_WORDS;
        const uint8_t* c = cls ? cls + (size_t)b * cls_b_stride + (size_t)hk * cls_h_stride : nullptr;
        const float* rows = scores + (size_t)problem * T * S;
        uint2* list = list_all + (size_t)problem * list_cap;
        const int t_begin = u0 * kUnit, t_end = min((u0 + n) * kUnit, T);
        const int items = (t_end - t_begin + kItemTokens - 1) / kItemTokens;

        if (tid < 2) s_cnt[tid] = 0u;
        if (tid == 0) s_next = 0u;
        for (int i = tid; i < n; i += kBandThreads) s_units[i] = 0u;
        __syncthreads();
        uint4 raw[kBatch][S / 4];
        int cls_of[kBatch];
        auto grab = [&]() {                              // the warp's next item of the segment
            uint32_t it = 0;
            if (lane == 0) it = atomicAdd(&s_next, 1u);
            return (int)__shfl_sync(0xFFFFFFFFu, it, 0);
        };
        auto load_item = [&](int item) {
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                const int t = t_begin + item * kItemTokens + 32 * i + lane;
                cls_of[i] = t < t_end ? token_class(c, t, len) : STC_CLS_DROP;
                load_raw<S>(rows + (size_t)min(t, T - 1) * S, raw[i]);
            }
        };
        int item = grab();
        if (item < items) load_item(item);               // in flight while the band arrives
        float lo = 0.f, hi = 0.f;
        if (select) {
            if (!wait_band(state, s_bc, abort_word, wait_ns)) return;
            band_bounds(s_bc[2], s_bc[3], lo, hi);
        }
        uint32_t pend_n = 0, pend_base = 0;              // staged entries of the warp and (lane 31) their place in the list
        auto flush = [&]() {
            if (pend_n) {
                __syncwarp();
                const uint32_t base = __shfl_sync(0xFFFFFFFFu, pend_base, 31);
                for (uint32_t e = lane; e < pend_n; e += 32)
                    if (base + e < list_cap) list[base + e] = stage[e];
                __syncwarp();
                pend_n = 0;
            }
        };
        uint32_t n_routed = 0, n_above = 0;
#pragma unroll 1
        while (item < items) {
            const int t0 = t_begin + item * kItemTokens + lane;      // the lane's token of run 0
            // 1. everything that needs the item's scores: masks, counts, the list entries (to the staging slots)
            uint32_t defs[kBatch], cands[kBatch], c_mine = 0;
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                const int cl = cls_of[i];
                defs[i] = 0;
                cands[i] = 0;
                if (cl == STC_CLS_FULL) {
                    defs[i] = (1u << S) - 1u;
                } else if (cl == STC_CLS_ROUTED) {
                    band_token<S>(raw[i], select, lo, hi, min_per_token, defs[i], cands[i]);
                    ++n_routed;
                    n_above += __popc(defs[i]) - floor_k;
                }
                c_mine += __popc(cands[i]);
            }
            // The warp's candidates go to the list in one piece.  Its place there comes from an atomic addition
            // whose answer takes a microsecond: the entries wait in the warp's staging slots and are written out
            // one item later, when the answer has long arrived.
            flush();
            const uint32_t incl = warp_incl_scan(c_mine, lane);
            const uint32_t w_total = __shfl_sync(0xFFFFFFFFu, incl, 31);
            const bool staged = w_total <= (uint32_t)kBandStage;
            if (w_total) {
                uint32_t pos = incl - c_mine;
                if (!staged) {                           // (too many for the slots: rare; wait for the place)
                    uint32_t base = 0;
                    if (lane == 31) base = atomicAdd(state + ST_LISTN, w_total);
                    pos += __shfl_sync(0xFFFFFFFFu, base, 31);
                }
                uint2* dst = staged ? stage : list;
                const uint32_t lim = staged ? (uint32_t)kBandStage : list_cap;
#pragma unroll
                for (int i = 0; i < kBatch; ++i) {
                    uint32_t m = cands[i];
                    if (m == 0u) continue;               // (nine tokens in ten)
                    // the token's scores go to the thread's scratch row, where a score can be picked by number
#pragma unroll
                    for (int q = 0; q < S / 4; ++q) reinterpret_cast<uint4*>(s_row)[q] = raw[i][q];
                    const uint32_t flat = (uint32_t)(t0 + 32 * i) * S;
                    while (m) {
                        const int j = __ffs(m) - 1;
                        m &= m - 1;
                        if (pos < lim) dst[pos] = make_uint2(s_row[j], flat + j);   // (score bits, flat index)
                        ++pos;
                    }
                }
            }
            // 2. the scores are no longer needed: the next item's loads go out now and fly during the rest
            const int next = grab();
            if (next < items) load_item(next);
            // 3. what only needs the masks
            if (w_total && staged) {
                if (lane == 31) pend_base = atomicAdd(state + ST_LISTN, w_total);
                pend_n = w_total;
            }
#pragma unroll
            for (int i = 0; i < kBatch; ++i) {
                const int t = t0 + 32 * i;
                if (t < t_end) {
                    v_mask[(size_t)problem * T + t] = (uint16_t)defs[i];
                }
                // per-unit count of definite bits (the 32 tokens of a run lie in one unit), gathered in shared
                // memory for the whole segment
                const uint32_t cnt = __reduce_add_sync(0xFFFFFFFFu, __popc(defs[i]));
                const int run_t = t0 - lane + 32 * i;
                if (lane == 0 && cnt && run_t < t_end) atomicAdd(&s_units[run_t / kUnit - u0], cnt);
            }
            item = next;
        }
        flush();
        n_routed = __reduce_add_sync(0xFFFFFFFFu, n_routed);
        n_above = __reduce_add_sync(0xFFFFFFFFu, n_above);
        if (lane == 0) { atomicAdd(&s_cnt[0], n_routed); atomicAdd(&s_cnt[1], n_above); }
        __syncthreads();
        if (tid == 0) {
            if (s_cnt[0]) atomicAdd(state + ST_NROUTEDB, s_cnt[0]);
            if (s_cnt[1]) atomicAdd(state + ST_ABOVE, s_cnt[1]);
        }
        // (plain stores: the settle kernel, which runs after this one, adds the listed pairs it keeps)
        for (int i = tid; i < n; i += kBandThreads) unit_sums[(size_t)problem * upp + u0 + i] = s_units[i];
        __syncthreads();                                 // the scratch is reused by the next segment
    }
}

// Problems of at most kBatch units (one token per thread and unit): a CTA takes whole
// problems, keeps their keys in registers and resolves the three digits from its own
// shared-memory histogram -- no global histogram, no hand-off between CTAs.
template <int S>
__global__ void __launch_bounds__(kThreads)
route_select_small_kernel(const float* __restrict__ scores, const uint8_t* __restrict__ cls,
                          int64_t cls_b_stride, int64_t cls_h_stride, const int32_t* __restrict__ seq_len,
                          int Hkv, int T, int upp, int k_nominal, int min_per_token, int mode,
                          uint32_t* __restrict__ state_all, uint16_t* __restrict__ v_mask,
                          uint16_t* __restrict__ tie_all, uint32_t* __restrict__ unit_sums, int problems) {
    constexpr int kBatch = 32 / S;
    __shared__ uint32_t shist[kBins];
    __shared__ uint32_t s_w[kWarps];
    __shared__ uint32_t s_red[kBatch][kWarps];
    __shared__ uint32_t s_pick[2];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;

#pragma unroll 1
    for (int problem = blockIdx.x; problem < problems; problem += gridDim.x) {
        const int b = problem / Hkv, hk = problem - b * Hkv;
        const int len = clamp_len(seq_len, b, T);
        const uint8_t* c = cls ? cls + (size_t)b * cls_b_stride + (size_t)hk * cls_h_stride : nullptr;
        uint4 raw[kBatch][S / 4];
        int cls_of[kBatch];
#pragma unroll
        for (int i = 0; i < kBatch; ++i) {
            const int t = i * kUnit + tid;
            cls_of[i] = (i < upp && t < T) ? token_class(c, t, len) : STC_CLS_DROP;
            if (cls_of[i] == STC_CLS_ROUTED) load_raw<S>(scores + ((size_t)problem * T + t) * S, raw[i]);
        }
        uint32_t key[kBatch][S];
        uint32_t n_routed = 0;
#pragma unroll
        for (int i = 0; i < kBatch; ++i) {
            if (cls_of[i] == STC_CLS_ROUTED) {
                make_keys<S>(raw[i], key[i]);
                ++n_routed;
            } else {
#pragma unroll
                for (int j = 0; j < S; ++j) key[i][j] = 0u;
            }
        }
        uint32_t tau = 0, flags = 0, krem = 0;
        if (mode == STC_MODE_GLOBAL) {
            uint32_t tot;
            block_excl_scan(n_routed, s_w, &tot);
            krem = budget_of(tot, k_nominal, min_per_token, flags);
#pragma unroll 1
            for (int pass = 0; pass < 3 && !flags; ++pass) {
                for (int i = tid; i < kBins; i += kThreads) shist[i] = 0;
                __syncthreads();
#pragma unroll
                for (int i = 0; i < kBatch; ++i)
                    if (cls_of[i] == STC_CLS_ROUTED)
                        hist_token<S, false>(key[i], pass_himask(pass), tau, pass_shift(pass),
                                             pass == 2 ? 1023u : 2047u, min_per_token, smem_u32(shist));
                __syncthreads();
                pick_digit<true>(shist, pass == 2 ? 1024 : kBins, krem, s_w, s_pick);
                tau |= s_pick[0] << pass_shift(pass);
                krem = s_pick[1];
                __syncthreads();                       // s_pick and the histogram are reused by the next pass
            }
            if (tid == 0) {                            // what the compaction kernel reads
                uint32_t* state = state_all + (size_t)problem * ST_WORDS;
                state[ST_FLAGS] = flags;
                state[ST_PREFIX] = flags ? 0u : tau;
                state[ST_KREM] = flags ? 0u : krem;
            }
        }
#pragma unroll
        for (int i = 0; i < kBatch; ++i) {
            const int t = i * kUnit + tid;
            uint32_t def = 0, tie = 0;
            if (flags & FL_BUDGET) {
                def = 0;
            } else if (cls_of[i] == STC_CLS_FULL) {
                def = (1u << S) - 1u;
            } else if (cls_of[i] == STC_CLS_ROUTED) {
                mask_token<S>(key[i], mode, flags, tau, k_nominal, min_per_token, def, tie);
            }
            if (i < upp && t < T) {
                v_mask[(size_t)problem * T + t] = (uint16_t)def;
                tie_all[(size_t)problem * T + t] = (uint16_t)tie;
            }
            const uint32_t cnt = __reduce_add_sync(0xFFFFFFFFu, __popc(def) | (__popc(tie) << 16));
            if (lane == 0) s_red[i][warp] = cnt;
        }
        __syncthreads();
        if (tid < kBatch && tid < upp) {
            uint32_t tot = 0;
#pragma unroll
            for (int w2 = 0; w2 < kWarps; ++w2) tot += s_red[tid][w2];
            unit_sums[(size_t)problem * upp + tid] = tot;
        }
        __syncthreads();
    }
}

template <int S>
__global__ void __launch_bounds__(kThreads, 4)
route_compact_kernel(const uint4* __restrict__ v, const int32_t* __restrict__ seq_len, int Hkv, int T,
                     int n_tiles, int upp, int mode, const uint32_t* __restrict__ state_all,
                     const uint32_t* __restrict__ abort_word, const uint32_t* __restrict__ unit_sums,
                     const uint16_t* __restrict__ tie_all,
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
    // base counts from the preceding units
    uint32_t bd = 0, be = 0;
    for (int i = tid; i < tile * kUnitsPerTile; i += kThreads) {
        const uint32_t c = __ldcg(unit_sums + (size_t)problem * upp + i);
        bd += c & 0xFFFFu;
        be += c >> 16;
    }
    uint32_t base_d, base_e;
    block_excl_scan(bd, s_w, &base_d);
    block_excl_scan(be, s_w, &base_e);

    // consecutive tokens per thread keep the scan in token order
    const int t0 = t_begin + tid * kTokPerThread;
    uint32_t def[kTokPerThread], tie[kTokPerThread], nd = 0, ne = 0;
#pragma unroll
    for (int i = 0; i < kTokPerThread; ++i) {
        const int t = t0 + i;
        def[i] = t < len ? v_mask[(size_t)problem * T + t] : 0u;
        tie[i] = t < len ? tie_all[(size_t)problem * T + t] : 0u;
        // a problem settled by the band path has no tie bits, no cleared tie array and a remaining rank of zero:
        // whatever was read there is dropped
        tie[i] = krem ? tie[i] : 0u;
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
            status[problem] = __ldcg(abort_word) ? STC_ERR_TIMEOUT
                              : (flags & FL_BUDGET) ? STC_ERR_BUDGET
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

namespace {

// CTAs of a cooperatively launched kernel that can be resident at once.
cudaError_t coop_grid_limit(const void* fn, int threads, size_t dyn_smem, std::atomic<int>* cached /*[kMaxDevices]*/,
                            int* limit) {
    // per device: the occupancy of a kernel is a property of the kernel and the device, the
    // query is cheap next to a cooperative launch, and a process may drive several devices
    constexpr int kMaxDevices = 64;
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    int v = (dev >= 0 && dev < kMaxDevices) ? cached[dev].load() : 0;
    if (v == 0) {
        int sms = 0, per_sm = 0;
        e = cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
        if (e == cudaSuccess) e = cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, fn, threads, dyn_smem);
        if (e != cudaSuccess) return e;
        if (sms <= 0 || per_sm <= 0) return cudaErrorLaunchOutOfResources;
        v = sms * per_sm;
        if (dev >= 0 && dev < kMaxDevices) cached[dev].store(v);
    }
    *limit = v;
    return cudaSuccess;
}

template <int S>
cudaError_t launch_select(const Geom& g, const float* scores, const uint8_t* cls, int64_t cls_b, int64_t cls_h,
                          int k_nominal, int min_per_token, int mode, const RouteWs& w, uint16_t* v_mask,
                          cudaStream_t st) {
    static std::atomic<int> cached_select[64], cached_band[64];
    int upp = (g.T + kUnit - 1) / kUnit;
    long long total_units = (long long)upp * g.problems;
    const int32_t* seq_len = g.seq_len;
    int Hkv = g.Hkv, T = g.T;
    uint32_t *state = w.state, *hist = w.hist, *hist13 = w.hist13, *abort_word = w.abort_word, *unit_sums = w.unit_sums;
    uint16_t* tie = w.tie;
    uint2* list = w.list;
    uint32_t list_cap = w.list_cap;
    const int knob = g_first_pass.load();
    unsigned long long wait_ns = g_wait_ns.load();
    // The band kernel settles the global budget in two scans; the multi-pass kernel follows for the problems
    // it left (it returns at once when there is none) and does everything in PER_TOKEN mode.
    // (a floor of one group per token with a nominal budget of none is the budget error: the multi-pass kernel reports it)
    // It pays when the scores do not stay in L2 between the scans (each of the four passes of the multi-pass
    // kernel is then a trip to HBM): measured, from about half the L2 size on; smaller score arrays
    // are as quick or quicker with the multi-pass kernel.
    bool big = false;
    {
        int dev = 0, l2 = 0;
        if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&l2, cudaDevAttrL2CacheSize, dev) == cudaSuccess)
            big = (double)g.problems * g.T * g.S * 4.0 >= 0.5 * (double)l2;
    }
    const bool band = mode == STC_MODE_GLOBAL && ((knob == 0 && big) || knob >= 4) &&
                      !(min_per_token && k_nominal == 0);
    cudaError_t e;
    int limit = 0;
    if (band) {
        e = cudaFuncSetAttribute(route_band_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                 (int)band_smem_bytes<S>());
        if (e != cudaSuccess) return e;
        e = coop_grid_limit(reinterpret_cast<const void*>(route_band_kernel<S>), kBandThreads, band_smem_bytes<S>(),
                            cached_band, &limit);
        if (e != cudaSuccess) return e;
        const unsigned grid = (unsigned)(total_units < limit ? total_units : limit);
        int skip_scan_a = knob == 4;
        // scan A samples one token in `samp`, keeping at least 2^16 keys of a problem in the sample
        const long long keys = (long long)g.T * g.S;
        int samp = knob == 5 ? 1 : (keys >= (1 << 20) ? 16 : keys >= (1 << 19) ? 8 : keys >= (1 << 18) ? 4 : keys >= (1 << 17) ? 2 : 1);
        int z_tenths = knob == 6 ? 0 : 50;
        void* args[] = {&scores, &cls, &cls_b, &cls_h, &seq_len, &Hkv, &T, &upp, &k_nominal, &min_per_token,
                        &state, &hist13, &abort_word, &v_mask, &unit_sums, &list, &list_cap, &total_units,
                        &skip_scan_a, &wait_ns, &samp, &z_tenths};
        e = cudaLaunchCooperativeKernel(reinterpret_cast<void*>(route_band_kernel<S>), dim3(grid),
                                        dim3(kBandThreads), args, band_smem_bytes<S>(), st);
        if (e != cudaSuccess) return e;
        e = cudaFuncSetAttribute(route_settle_kernel<S>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSettleSmem);
        if (e != cudaSuccess) return e;
        route_settle_kernel<S><<<(unsigned)g.problems, kSettleThreads, kSettleSmem, st>>>(
            state, abort_word, list, list_cap, v_mask, unit_sums, T, upp, k_nominal, min_per_token);
        e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    e = coop_grid_limit(reinterpret_cast<const void*>(route_select_kernel<S>), kThreads, 0, cached_select, &limit);
    if (e != cudaSuccess) return e;
    const unsigned grid = (unsigned)(total_units < limit ? total_units : limit);
    int first_pass = (knob >= 1 && knob <= 3) ? knob : 0;
    int only_wide = band;
    void* args[] = {&scores, &cls, &cls_b, &cls_h, &seq_len, &Hkv, &T, &upp, &k_nominal, &min_per_token, &mode,
                    &state, &hist, &abort_word, &v_mask, &tie, &unit_sums, &total_units, &first_pass, &wait_ns,
                    &only_wide};
    return cudaLaunchCooperativeKernel(reinterpret_cast<void*>(route_select_kernel<S>), dim3(grid),
                                       dim3(kThreads), args, 0, st);
}

}  // namespace

cudaError_t launch_route_pack(const Geom& g, const void* v, const float* scores,
                              const uint8_t* tok_class, int64_t class_head_stride, int k_nominal,
                              int min_per_token, int mode, void* v_packed, uint16_t* v_mask,
                              uint32_t* v_offs, int64_t cap_groups, int64_t* total_groups,
                              int32_t* status, void* ws, int phases, cudaStream_t st) {
    if (g.problems == 0) return cudaSuccess;
    const RouteWs w = carve(g, ws);
    const bool do_route = phases & 1, do_pack = phases & 2;
    const int n_tiles = (g.T + kTile - 1) / kTile;
    const int upp = (g.T + kUnit - 1) / kUnit;
    const long long n_cta = (long long)n_tiles * g.problems;
    if (n_cta > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    const int64_t cls_h = class_head_stride;
    const int64_t cls_b = class_head_stride ? (int64_t)g.Hkv * class_head_stride : (int64_t)g.T;
    cudaError_t e = cudaSuccess;
    const bool small = upp <= 32 / g.S;            // a problem fits one CTA's registers
    if (do_route) {
        e = cudaMemsetAsync(w.state, 0, small ? w.zero_small : w.zero_bytes, st);
        if (e != cudaSuccess) return e;
    }
    int sms = 0;
    e = device_sm_count(&sms);
    if (e != cudaSuccess) return e;
    const unsigned grid_small = (unsigned)(g.problems < sms * 16 ? g.problems : sms * 16);

#define STC_ROUTE(S_)                                                                               \
    case S_: {                                                                                      \
        if (do_route && small)                                                                      \
            route_select_small_kernel<S_><<<grid_small, kThreads, 0, st>>>(                         \
                scores, tok_class, cls_b, cls_h, g.seq_len, g.Hkv, g.T, upp, k_nominal,             \
                min_per_token, mode, w.state, v_mask, w.tie, w.unit_sums, g.problems);              \
        else if (do_route)                                                                          \
            e = launch_select<S_>(g, scores, tok_class, cls_b, cls_h, k_nominal, min_per_token,     \
                                  mode, w, v_mask, st);                                             \
        if (e != cudaSuccess) return e;                                                             \
        if (do_pack) route_compact_kernel<S_><<<(unsigned)n_cta, kThreads, 0, st>>>(                \
            static_cast<const uint4*>(v), g.seq_len, g.Hkv, g.T, n_tiles, upp, mode, w.state,       \
            w.abort_word, w.unit_sums, w.tie, v_mask, v_offs, static_cast<uint4*>(v_packed),        \
            cap_groups, total_groups, status);                                                      \
    } break;
    switch (g.S) {
        STC_ROUTE(4) STC_ROUTE(8) STC_ROUTE(16)
        default: return cudaErrorInvalidValue;
    }
#undef STC_ROUTE
    return cudaGetLastError();
}

void set_route_select_knobs(int first_pass, unsigned long long wait_ns) {
    g_first_pass.store(first_pass < -1 || first_pass > 7 ? 0 : first_pass);
    g_wait_ns.store(wait_ns ? wait_ns : kWaitNs);
}

}  // namespace stc

// Test hook, not part of the public interface (not declared in stc.h).  first_pass: 0 = normal (for score
// arrays of half the L2 size and beyond the band kernel, then the multi-pass kernel for what it left; else the
// multi-pass kernel alone); -1 = the multi-pass kernel alone; 1..3 = the
// multi-pass kernel alone, starting at that histogram pass; 4 = the band kernel without its first scan;
// 5 = the band kernel with every token in its sample (the band is then exact); 6 = the band kernel with
// a band of almost no width (it misses often, and the multi-pass kernel then redoes those problems);
// 7 = the band kernel as in production, whatever the size of the call.
// wait_ns bounds the hand-off waits (0 = the default of two seconds).  With first_pass = 3 or 4 on a
// freshly cleared workspace no CTA ever publishes a digit, so every wait runs into its limit and the
// give-up path (abort word, orderly return, STC_ERR_TIMEOUT from the packing kernel) executes without
// anything hanging.
extern "C" void stc_test_route_select_knobs(int32_t first_pass, uint64_t wait_ns) {
    stc::set_route_select_knobs(first_pass, wait_ns);
}
