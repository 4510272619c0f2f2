// Shared device helpers and internal launch declarations for libstc (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "stc.h"

namespace stc {

constexpr int kHeadDim = 128;
constexpr int kPage = 16;
constexpr int kRowBytes = kHeadDim * 2;        // one key / value row
constexpr int kOctets = kHeadDim / 8;          // 16-byte chunks per row

// Geometry resolved once on the host.
struct Geom {
    int B, Hq, Hkv, Gq, S, g, T, P;            // P = ceil(T/16)
    int problems;
    const int32_t* seq_len;
};

__device__ __forceinline__ int clamp_len(const int32_t* seq_len, int b, int T) {
    int n = seq_len ? seq_len[b] : T;
    return n < 0 ? 0 : (n > T ? T : n);
}

__device__ __forceinline__ float bf16lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }

__device__ __forceinline__ uint4 ldg_nc16(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

// Same, asking L2 to fetch no more than the 64-byte granule around the address: for
// gathers whose neighbours are mostly not wanted.
__device__ __forceinline__ uint4 ldg_nc16_narrow(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.L2::64B.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

// Ampere-style asynchronous 16-byte copy global -> shared (L2 only), with
// optional zero fill: src_bytes = 0 writes 16 zero bytes without reading.
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async16_zfill(uint32_t dst, const void* src, int src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ uint4 lds16(uint32_t addr) {
    uint4 r;
    asm volatile("ld.shared.v4.u32 {%0,%1,%2,%3}, [%4];" : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "r"(addr));
    return r;
}

// Order-preserving map from fp32 to uint32 (larger float -> larger key); -0 is folded
// onto +0 (by the addition) so the two compare equal.
__device__ __forceinline__ uint32_t float_key(float f) {
    const uint32_t u = __float_as_uint(__fadd_rn(f, 0.0f));
    return u ^ ((uint32_t)((int32_t)u >> 31) | 0x80000000u);               // negative: ~u, else u | sign
}
// The float whose key is k (k = 0x7FFFFFFF, the unused key of -0, gives -0).
__device__ __forceinline__ float key_float(uint32_t k) {
    return __uint_as_float((k & 0x80000000u) ? (k & 0x7FFFFFFFu) : ~k);
}

// ---- internal launchers (one per source file) -------------------------------
cudaError_t launch_page_meta(const Geom& g, const void* k, void* kmin, void* kmax, int page_begin,
                             int page_end, cudaStream_t st);

size_t select_ws_bytes(const Geom& g);
cudaError_t launch_quest_select(const Geom& g, const void* kmin, const void* kmax, const void* q,
                                int token_budget, int n_recent_pages, int max_pages, int32_t* page_ids,
                                int32_t* n_pages, float* scores_opt, void* ws, cudaStream_t st);

size_t route_ws_bytes(const Geom& g);
cudaError_t launch_route_pack(const Geom& g, const void* v, const float* scores,
                              const uint8_t* tok_class, int64_t class_head_stride, int k_nominal,
                              int min_per_token, int mode, void* v_packed, uint16_t* v_mask,
                              uint32_t* v_offs, int64_t cap_groups, int64_t* total_groups,
                              int32_t* status, void* ws, int phases /*1 = masks, 2 = pack, 3 = both*/,
                              cudaStream_t st);

cudaError_t launch_append(const Geom& g, const void* k, void* kmin, void* kmax, const void* v,
                          const int32_t* old_len, int max_new, void* v_packed, uint16_t* v_mask,
                          uint32_t* v_offs, int64_t cap_groups, int64_t* total_groups, int32_t* status,
                          cudaStream_t st);

cudaError_t launch_router_logits(const Geom& g, const void* h, const void* w, const float* bias, int d_model,
                                 float* scores, int32_t* status, cudaStream_t st);

cudaError_t launch_query_bias(int B, int Lq, int d_model, int n_logits, const void* h_q, const int32_t* q_len,
                              const void* w_q, float* s_q, float* bias, cudaStream_t st);

struct AttnPlan { int n_workers, slots_cap; };   // warps that share the pages; partial slots per problem
AttnPlan attn_plan(const Geom& g, int max_pages);
size_t attn_ws_bytes(const Geom& g, int max_pages);
cudaError_t launch_decode_attn(const Geom& g, const void* k, const void* v_packed,
                               const uint16_t* v_mask, const uint32_t* v_offs, int64_t cap_groups,
                               const void* q, const int32_t* page_ids, const int32_t* n_pages,
                               int max_pages, float sm_scale, float* out, float* lse, void* ws,
                               cudaStream_t st);

}  // namespace stc
