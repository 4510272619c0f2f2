// Token classes from a page selection: the link between the two stages when they
// run in the paper's own order (Stage I keeps tokens, Stage II routes the value
// groups of the kept tokens only).  One thread per (problem, list slot, token of
// the page); the class array is cleared to DROP first, so a token is ROUTED exactly
// when one of the listed pages holds it.
#include "common.cuh"

namespace stc {
namespace {

__global__ void __launch_bounds__(256)
pages_to_class_kernel(const int32_t* __restrict__ page_ids, const int32_t* __restrict__ n_pages,
                      const int32_t* __restrict__ seq_len, int Hkv, int T, int max_pages,
                      long long total, uint8_t* __restrict__ tok_class) {
    const long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= total) return;
    const int t_in = (int)(i & (kPage - 1));
    const long long x = i >> 4;
    const int problem = (int)(x / max_pages), slot = (int)(x - (long long)problem * max_pages);
    const int len = clamp_len(seq_len, problem / Hkv, T);
    const int n = min(max(n_pages[problem], 0), max_pages);
    if (slot >= n) return;
    const int id = page_ids[(size_t)problem * max_pages + slot];
    const long long t = (long long)id * kPage + t_in;
    if (id < 0 || t >= len) return;
    tok_class[(size_t)problem * T + t] = (uint8_t)STC_CLS_ROUTED;
}

}  // namespace

cudaError_t launch_pages_to_class(const Geom& g, const int32_t* page_ids, const int32_t* n_pages,
                                  int max_pages, uint8_t* tok_class, cudaStream_t st) {
    cudaError_t e = cudaMemsetAsync(tok_class, STC_CLS_DROP, (size_t)g.problems * g.T, st);
    if (e != cudaSuccess || max_pages < 1) return e;
    const long long total = (long long)g.problems * max_pages * kPage;
    const long long blocks = (total + 255) / 256;
    if (blocks > 0x7FFFFFFFLL) return cudaErrorInvalidValue;
    pages_to_class_kernel<<<(unsigned)blocks, 256, 0, st>>>(page_ids, n_pages, g.seq_len, g.Hkv, g.T,
                                                            max_pages, total, tok_class);
    return cudaGetLastError();
}

}  // namespace stc
