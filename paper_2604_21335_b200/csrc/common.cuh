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

// ---- mbarrier + 1-D bulk asynchronous copy (the untiled TMA path) ---------------------------
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
__device__ __forceinline__ unsigned long long global_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
// Bounded wait for the phase `parity` of an mbarrier.  False = gave up after limit_ns.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity, unsigned long long limit_ns) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
#pragma unroll 1
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (global_ns() - t0 > limit_ns) return false;
    }
}
// 1-D bulk copy global -> this CTA's shared memory, completion counted on `bar`.
// dst, src 16-byte aligned; bytes a positive multiple of 16.
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];"
                 ::"r"(dst), "l"(src), "r"(bytes), "r"(bar) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void fence_mbar_init() { asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory"); }

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

// Inclusive prefix sum over the lanes of a warp.
__device__ __forceinline__ uint32_t warp_incl_scan(uint32_t v, int lane) {
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t o = __shfl_up_sync(0xFFFFFFFFu, v, d);
        if (lane >= d) v += o;
    }
    return v;
}

// Packed bf16 min / max of two words.
__device__ __forceinline__ uint32_t bmin2(uint32_t a, uint32_t b) {
    __nv_bfloat162 r = __hmin2(*reinterpret_cast<__nv_bfloat162*>(&a), *reinterpret_cast<__nv_bfloat162*>(&b));
    return *reinterpret_cast<uint32_t*>(&r);
}
__device__ __forceinline__ uint32_t bmax2(uint32_t a, uint32_t b) {
    __nv_bfloat162 r = __hmax2(*reinterpret_cast<__nv_bfloat162*>(&a), *reinterpret_cast<__nv_bfloat162*>(&b));
    return *reinterpret_cast<uint32_t*>(&r);
}

// Multiprocessor count of the current device (queried per call: cheap next to a launch, and
// right on every device of a multi-GPU process).
inline cudaError_t device_sm_count(int* n) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    e = cudaDeviceGetAttribute(n, cudaDevAttrMultiProcessorCount, dev);
    if (e == cudaSuccess && *n <= 0) e = cudaErrorInvalidDevice;
    return e;
}

// Launch options of the internal launchers.
enum : unsigned {
    kLaunchNoClear = 1u    // the caller has already cleared the call's status / counter words on the stream
};

// ---- internal launchers (one per source file) -------------------------------
cudaError_t launch_page_meta(const Geom& g, const void* k, void* kmin, void* kmax, int page_begin,
                             int page_end, cudaStream_t st);

size_t select_ws_bytes(const Geom& g);
cudaError_t launch_quest_select(const Geom& g, const void* kmin, const void* kmax, const void* q,
                                int token_budget, int n_recent_pages, int max_pages, int32_t* page_ids,
                                int32_t* n_pages, float* scores_opt, void* ws, cudaStream_t st, unsigned flags = 0);
cudaError_t clear_quest_select_ws(const Geom& g, void* ws, cudaStream_t st);
size_t quest_select_clear_bytes(const Geom& g);    // leading bytes of the workspace a call needs zeroed
// One small kernel that zeroes the leading bytes of two workspaces (one graph node instead of two memsets).
cudaError_t clear_two(void* a, size_t a_bytes, void* b, size_t b_bytes, cudaStream_t st);

cudaError_t launch_pages_to_class(const Geom& g, const int32_t* page_ids, const int32_t* n_pages,
                                  int max_pages, uint8_t* tok_class, cudaStream_t st);

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

int route_new_pages_max();
cudaError_t launch_route_new_pages(const Geom& g, const float* scores, const int32_t* first_page, int k_nominal,
                                   int min_per_token, int mode, void* v_packed, uint16_t* v_mask,
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
                               cudaStream_t st, unsigned flags = 0);
cudaError_t clear_decode_attn_ws(const Geom& g, void* ws, cudaStream_t st);
size_t decode_attn_clear_bytes(const Geom& g);     // leading bytes of the workspace a call needs zeroed

}  // namespace stc
