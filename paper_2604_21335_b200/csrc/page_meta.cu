// Page metadata builder: per 16-token page and channel, the min and max key.
//
// One half-warp owns one page: lane l of the half reads the 16-byte chunk
// (channels 8l..8l+7) of each of the page's rows, so every load instruction of
// a warp covers two full 256-byte rows.  All 16 row loads of a lane are issued
// before the first compare.  HBM-bound: 4 KiB read, 512 B written per page.
#include "common.cuh"

namespace stc {
namespace {

constexpr int kThreads = 256;
constexpr int kPagesPerCta = kThreads / 16;


__global__ void __launch_bounds__(kThreads)
page_meta_kernel(const uint4* __restrict__ k, uint4* __restrict__ kmin, uint4* __restrict__ kmax,
                 const int32_t* __restrict__ seq_len, int Hkv, int T, int P, int page_begin,
                 int page_end, int tiles) {
    const int problem = blockIdx.x / tiles;
    const int tile = blockIdx.x - problem * tiles;
    const int len = clamp_len(seq_len, problem / Hkv, T);
    const int n_pages = (len + kPage - 1) / kPage;
    const int page = page_begin + tile * kPagesPerCta + (threadIdx.x >> 4);
    const int oct = threadIdx.x & 15;
    if (page >= page_end || page >= n_pages) return;

    const int t0 = page * kPage;
    const int n_valid = min(kPage, len - t0);
    const uint4* src = k + ((size_t)problem * T + t0) * kOctets + oct;

    uint4 r[kPage];
#pragma unroll
    for (int t = 0; t < kPage; ++t)
        r[t] = (t < n_valid) ? ldg_nc16(src + (size_t)t * kOctets) : make_uint4(0, 0, 0, 0);

    uint4 lo = r[0], hi = r[0];
#pragma unroll
    for (int t = 1; t < kPage; ++t) {
        if (t < n_valid) {
            lo.x = bmin2(lo.x, r[t].x); hi.x = bmax2(hi.x, r[t].x);
            lo.y = bmin2(lo.y, r[t].y); hi.y = bmax2(hi.y, r[t].y);
            lo.z = bmin2(lo.z, r[t].z); hi.z = bmax2(hi.z, r[t].z);
            lo.w = bmin2(lo.w, r[t].w); hi.w = bmax2(hi.w, r[t].w);
        }
    }
    const size_t dst = ((size_t)problem * P + page) * kOctets + oct;
    kmin[dst] = lo;
    kmax[dst] = hi;
}

}  // namespace

cudaError_t launch_page_meta(const Geom& g, const void* k, void* kmin, void* kmax, int page_begin,
                             int page_end, cudaStream_t st) {
    if (page_end < 0 || page_end > g.P) page_end = g.P;
    if (page_begin < 0) page_begin = 0;
    if (page_begin >= page_end || g.problems == 0) return cudaSuccess;
    const int tiles = (page_end - page_begin + kPagesPerCta - 1) / kPagesPerCta;
    const long long n_cta = (long long)tiles * g.problems;
    if (n_cta > 0x7FFFFFFFLL) return cudaErrorInvalidConfiguration;
    page_meta_kernel<<<(unsigned)n_cta, kThreads, 0, st>>>(static_cast<const uint4*>(k), static_cast<uint4*>(kmin),
                                               static_cast<uint4*>(kmax), g.seq_len, g.Hkv, g.T, g.P,
                                               page_begin, page_end, tiles);
    return cudaGetLastError();
}

}  // namespace stc
