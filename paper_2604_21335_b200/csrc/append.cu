// Streaming append: tokens added to a sequence after its cache was routed.
//
// The method leaves query-region tokens uncompressed (Section 3.4: the tokens that
// ask the question keep their full values), and during decoding every newly
// generated token is such a token.  So an append stores all S groups of each new
// token behind the sequence's packed groups (mask = all ones, offsets advance by
// S) and refreshes the min/max metadata of the pages the new keys fall in.
// Routing the appended region later is a new stc_route_pack over the sequence.
//
// Two small kernels, both bandwidth-trivial: a 16-byte-chunk copy of the new value
// rows, and the page-metadata kernel restricted to the touched pages.
#include "common.cuh"

namespace stc {
namespace {

constexpr int kThreads = 256;


// Appended range of sequence b: [lo, hi), or an empty range with `bad` set when the
// lengths are inconsistent (shrinking sequence, more than max_new tokens).
__device__ __forceinline__ void new_range(const int32_t* seq_len, const int32_t* old_len, int b, int T,
                                          int max_new, int& lo, int& hi, bool& bad) {
    const int nl = clamp_len(seq_len, b, T);
    const int ol = old_len[b];
    bad = ol < 0 || ol > nl || nl - ol > max_new;
    lo = bad ? 0 : ol;
    hi = bad ? 0 : nl;
}

// One thread per 16-byte chunk of a new value row; 16 tokens per CTA.
template <int S>
__global__ void __launch_bounds__(kThreads)
append_values_kernel(const uint4* __restrict__ v, const int32_t* __restrict__ seq_len,
                     const int32_t* __restrict__ old_len, int Hkv, int T, int max_new, int chunks_per_problem,
                     uint16_t* __restrict__ v_mask, uint32_t* __restrict__ v_offs, uint4* __restrict__ v_packed,
                     int64_t cap_groups, int64_t* __restrict__ total_groups, int32_t* __restrict__ status) {
    constexpr int OPG = kOctets / S;
    const int problem = blockIdx.x / chunks_per_problem, part = blockIdx.x - problem * chunks_per_problem;
    const int b = problem / Hkv;
    int lo, hi;
    bool bad;
    new_range(seq_len, old_len, b, T, max_new, lo, hi, bad);
    const int i = part * (kThreads / kOctets) + (threadIdx.x >> 4);      // i-th new token
    const int oct = threadIdx.x & 15;
    const int t = lo + i;
    uint32_t* offs = v_offs + (size_t)problem * (T + 1);
    const int64_t base = offs[lo];                                        // groups stored before the append
    if (part == 0 && threadIdx.x == 0) {
        const int64_t total = base + (int64_t)(hi - lo) * S;
        if (!bad) total_groups[problem] = total;
        status[problem] = bad ? STC_ERR_INVALID_ARG : (total > cap_groups ? STC_ERR_CAPACITY : STC_OK);
    }
    if (t >= hi) return;
    const int64_t first = base + (int64_t)i * S;                          // first group of token t
    if (oct == 0) {
        v_mask[(size_t)problem * T + t] = (uint16_t)((1u << S) - 1u);
        offs[t + 1] = (uint32_t)(first + S);
    }
    const int grp = oct / OPG;
    if (first + grp < cap_groups)
        v_packed[((size_t)problem * cap_groups + first + grp) * OPG + (oct % OPG)] =
            ldg_nc16(v + ((size_t)problem * T + t) * kOctets + oct);
}

// Min / max metadata of the pages that hold appended tokens (half-warp per page).
__global__ void __launch_bounds__(kThreads)
append_meta_kernel(const uint4* __restrict__ k, uint4* __restrict__ kmin, uint4* __restrict__ kmax,
                   const int32_t* __restrict__ seq_len, const int32_t* __restrict__ old_len, int Hkv, int T,
                   int P, int max_new, int tiles) {
    const int problem = blockIdx.x / tiles, tile = blockIdx.x - problem * tiles;
    int lo, hi;
    bool bad;
    new_range(seq_len, old_len, problem / Hkv, T, max_new, lo, hi, bad);
    if (hi <= lo) return;
    const int page = lo / kPage + tile * (kThreads / 16) + (threadIdx.x >> 4);
    const int oct = threadIdx.x & 15;
    if (page > (hi - 1) / kPage) return;
    const int t0 = page * kPage, n_valid = min(kPage, hi - t0);
    const uint4* src = k + ((size_t)problem * T + t0) * kOctets + oct;
    uint4 lo4 = ldg_nc16(src), hi4 = lo4;
    for (int t = 1; t < n_valid; ++t) {
        const uint4 r = ldg_nc16(src + (size_t)t * kOctets);
        lo4.x = bmin2(lo4.x, r.x); hi4.x = bmax2(hi4.x, r.x);
        lo4.y = bmin2(lo4.y, r.y); hi4.y = bmax2(hi4.y, r.y);
        lo4.z = bmin2(lo4.z, r.z); hi4.z = bmax2(hi4.z, r.z);
        lo4.w = bmin2(lo4.w, r.w); hi4.w = bmax2(hi4.w, r.w);
    }
    const size_t dst = ((size_t)problem * P + page) * kOctets + oct;
    kmin[dst] = lo4;
    kmax[dst] = hi4;
}

}  // namespace

cudaError_t launch_append(const Geom& g, const void* k, void* kmin, void* kmax, const void* v,
                          const int32_t* old_len, int max_new, void* v_packed, uint16_t* v_mask,
                          uint32_t* v_offs, int64_t cap_groups, int64_t* total_groups, int32_t* status,
                          cudaStream_t st) {
    if (g.problems == 0 || max_new <= 0) return cudaSuccess;
    const int tokens_per_cta = kThreads / kOctets;
    const int chunks = (max_new + tokens_per_cta - 1) / tokens_per_cta;
    const long long n_cta = (long long)chunks * g.problems;
    if (n_cta > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
#define STC_APPEND(S_)                                                                               \
    case S_:                                                                                         \
        append_values_kernel<S_><<<(unsigned)n_cta, kThreads, 0, st>>>(                              \
            static_cast<const uint4*>(v), g.seq_len, old_len, g.Hkv, g.T, max_new, chunks, v_mask,   \
            v_offs, static_cast<uint4*>(v_packed), cap_groups, total_groups, status);                \
        break;
    switch (g.S) {
        STC_APPEND(4) STC_APPEND(8) STC_APPEND(16)
        default: return cudaErrorInvalidValue;
    }
#undef STC_APPEND
    const int pages_touched = max_new / kPage + 2;                 // a range of max_new tokens spans at most this
    const int tiles = (pages_touched + kThreads / 16 - 1) / (kThreads / 16);
    append_meta_kernel<<<(unsigned)(tiles * g.problems), kThreads, 0, st>>>(
        static_cast<const uint4*>(k), static_cast<uint4*>(kmin), static_cast<uint4*>(kmax), g.seq_len, old_len,
        g.Hkv, g.T, g.P, max_new, tiles);
    return cudaGetLastError();
}

}  // namespace stc
