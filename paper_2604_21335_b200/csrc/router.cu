// Value-group router logits: scores[b][hk][t][j] = sum_c h[b][t][c] * w[hk*S+j][c] (+ bias).
//
// This is the one dense contraction of the method (Appendix B.1: the router is a
// single linear projection of the layer's hidden state to S group logits), so it
// runs on the 5th-generation tensor cores: a [tokens x d_model] . [d_model x Hkv*S]
// GEMM with both operands K-major, bf16 in, fp32 accumulate.
//
// One CTA computes a 128-token x BN-logit tile (BN = all Hkv*S logits, <= 256):
//   warp 0      one lane streams 64-wide K slices of both operands into a 2..8-stage
//               shared-memory ring with TMA (cp.async.bulk.tensor, 128-byte swizzle)
//   warp 1      allocates the accumulator in tensor memory (128 lanes x BN columns);
//               one lane issues tcgen05.mma (M128 x N(BN) x K16, four per slice) and
//               commits each slice back to the producer, the last one to the epilogue
//   warps 2..5  read the accumulator with tcgen05.ld (each warp its 32 lanes = 32
//               tokens), add the per-sequence bias and write S consecutive floats
//               per (token, kv head): neighbouring lanes write neighbouring tokens,
//               which are adjacent in the [B][Hkv][T][S] score layout
// Every mbarrier wait is bounded (about a second); a wait that expires raises a
// CTA-wide abort flag and STC_ERR_TIMEOUT in the status word, the roles leave their
// loops, the producer gives its copies in flight one more bounded wait, the tensor
// memory is freed and the CTA returns.
#include <cuda.h>

#include "common.cuh"

namespace stc {
namespace {

constexpr int kBM = 128;                 // tokens per CTA
constexpr int kBK = 64;                  // K slice: 64 bf16 = one 128-byte swizzle row
constexpr int kMaxStages = 8;            // ring depth = what fits in kRingBytes, at most this
constexpr int kMaxBN = 256;
constexpr int kThreads = 192;            // 6 warps: TMA, MMA, 4 x epilogue
constexpr uint32_t kABytes = kBM * kBK * 2;              // 16 KiB
constexpr uint32_t kBBytesMax = kMaxBN * kBK * 2;        // 32 KiB
constexpr uint32_t kRingBytes = 2 * (kABytes + kBBytesMax);  // 96 KiB: two CTAs per SM; 2 stages at BN = 256, 4 at BN = 64
constexpr uint32_t kSmemBytes = kRingBytes + 1024 /* alignment slack */ + 256 /* barriers etc. */;
constexpr unsigned long long kWaitLimitNs = 1000000000ull;

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, volatile int* abort_flag) {
    if (mbar_try_wait(bar, parity)) return true;
    const unsigned long long t0 = global_ns();
#pragma unroll 1
    for (;;) {
#pragma unroll 1
        for (int i = 0; i < 64; ++i)
            if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag || global_ns() - t0 > kWaitLimitNs) return false;
    }
}
// 2-D tiled TMA load: box at element (x = k, y = row) of the tensor map -> shared memory.
// x is a multiple of 64 bf16, i.e. 128 bytes (the copy must start on a 16-byte boundary).
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(bar) : "memory");
}
__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// D[tmem] (+)= A[smem desc] . B[smem desc]; kind::f16 covers bf16 inputs with fp32 accumulation.
__device__ __forceinline__ void tc_mma(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                       uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate) : "memory");
}
// Shared-memory operand descriptor, K-major, 128-byte swizzle: rows of 128 bytes, groups
// of 8 rows 1024 bytes apart (stride byte offset), leading byte offset unused (1),
// descriptor version 1, layout type 2; addresses in units of 16 bytes.
__device__ __forceinline__ uint64_t smem_desc_sw128(uint32_t addr) {
    return (uint64_t)((addr >> 4) & 0x3FFFu) | ((uint64_t)1 << 16) | ((uint64_t)(1024 >> 4) << 32) |
           ((uint64_t)1 << 46) | ((uint64_t)2 << 61);
}

struct RouterArgs {
    const float* bias;      // [B][N] or nullptr
    float* scores;          // [B][Hkv][T][S]
    int32_t* status;        // one word
    int M, N, K, T, S, Hkv; // M = B*T tokens, N = Hkv*S logits, K = d_model
    int BN;                 // logits per CTA tile (<= 256, multiple of 16)
};

__global__ void __launch_bounds__(kThreads, 2)
router_logits_kernel(const __grid_constant__ CUtensorMap map_h, const __grid_constant__ CUtensorMap map_w,
                     const RouterArgs a) {
    extern __shared__ unsigned char smem_raw[];
    // 128-byte-swizzled tiles need 1024-byte aligned bases
    const uint32_t base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t ctrl = base + kRingBytes;                     // barriers, TMEM address, abort flag
    const uint32_t full0 = ctrl, empty0 = ctrl + 8 * kMaxStages, tmem_full = ctrl + 16 * kMaxStages;
    unsigned char* ctrl_ptr = smem_raw + (ctrl - smem_u32(smem_raw));
    volatile uint32_t* tmem_slot = reinterpret_cast<volatile uint32_t*>(ctrl_ptr + 16 * kMaxStages + 8);
    volatile int* abort_flag = reinterpret_cast<volatile int*>(ctrl_ptr + 16 * kMaxStages + 12);
    // a stage = the 128 x 64 slice of h and the BN x 64 slice of w (both multiples of 1024 bytes)
    const uint32_t kStageBytes = kABytes + (uint32_t)a.BN * kBK * 2;
    const int kStages = min(kMaxStages, (int)(kRingBytes / kStageBytes));

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int m0 = blockIdx.x * kBM, n0 = blockIdx.y * a.BN;
    const int k_tiles = a.K / kBK;
    const uint32_t b_bytes = (uint32_t)a.BN * kBK * 2;
    // tensor-memory columns: a power of two >= 32 that holds BN fp32 columns
    uint32_t tmem_cols = 32;
    while (tmem_cols < (uint32_t)a.BN) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(full0 + 8 * s, 1); mbar_init(empty0 + 8 * s, 1); }
        mbar_init(tmem_full, 1);
        *abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {                                  // whole warp: allocate the accumulator
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(ctrl + 16 * kMaxStages + 8), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_acc = *tmem_slot;

    if (warp == 0 && lane == 0) {
        // ---- TMA producer ---------------------------------------------------------------------
        int issued = 0;
        for (int kt = 0; kt < k_tiles; ++kt, ++issued) {
            const int s = kt % kStages;
            const uint32_t ph = (uint32_t)(kt / kStages) & 1u;
            if (!mbar_wait(empty0 + 8 * s, ph ^ 1u, abort_flag)) {       // slot free (fresh barrier: passes)
                *abort_flag = 1; atomicExch(a.status, (int)STC_ERR_TIMEOUT); break;
            }
            const uint32_t sa = base + (uint32_t)s * kStageBytes, sb = sa + kABytes;
            mbar_expect_tx(full0 + 8 * s, kABytes + b_bytes);
            tma_load_2d(sa, &map_h, kt * kBK, m0, full0 + 8 * s);
            tma_load_2d(sb, &map_w, kt * kBK, n0, full0 + 8 * s);
        }
        if (*abort_flag) {
            // copies still in flight: give each of the last kStages slices one more bounded wait
            int dummy = 0;
            for (int kt = max(0, issued - kStages); kt < issued; ++kt)
                mbar_wait(full0 + 8 * (kt % kStages), (uint32_t)(kt / kStages) & 1u, &dummy);
        }
    } else if (warp == 1 && lane == 0) {
        // ---- MMA issuer ------------------------------------------------------------------------
        // instruction descriptor: D = f32, A = B = bf16, both K-major, N = BN, M = 128
        const uint32_t idesc = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(a.BN >> 3) << 17) | ((kBM >> 4) << 24);
        bool ok = true;
        for (int kt = 0; kt < k_tiles && ok; ++kt) {
            const int s = kt % kStages;
            const uint32_t ph = (uint32_t)(kt / kStages) & 1u;
            if (!mbar_wait(full0 + 8 * s, ph, abort_flag)) {
                *abort_flag = 1; atomicExch(a.status, (int)STC_ERR_TIMEOUT); ok = false; break;
            }
            tc_fence_after();
            const uint32_t sa = base + (uint32_t)s * kStageBytes, sb = sa + kABytes;
            const uint64_t da = smem_desc_sw128(sa), db = smem_desc_sw128(sb);
#pragma unroll
            for (int k = 0; k < kBK / 16; ++k)          // 16 bf16 = 32 bytes = 2 descriptor units per step
                tc_mma(tmem_acc, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc, (kt | k) != 0);
            tc_commit(empty0 + 8 * s);                  // slot reusable once these MMAs have read it
        }
        if (ok) tc_commit(tmem_full);                   // accumulator complete
    } else if (warp >= 2) {
        // ---- epilogue: warp w owns TMEM lanes 32*(w%4) .. +31 = tokens m0 + 32*(w%4) + lane ---------
        const int quarter = warp & 3;
        const int m = m0 + quarter * 32 + lane;
        if (mbar_wait(tmem_full, 0u, abort_flag)) {
            tc_fence_after();
            const int b = m / a.T, t = m - b * a.T;
            for (int c0 = 0; c0 < a.BN; c0 += 16) {
                uint32_t r[16];
                const uint32_t taddr = tmem_acc + ((uint32_t)(quarter * 32) << 16) + (uint32_t)c0;
                asm volatile(
                    "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
                    "{%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                    : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                      "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                    : "r"(taddr));
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (m < a.M) {
#pragma unroll
                    for (int i = 0; i < 16; i += 4) {   // S is 4, 8 or 16: a float4 never straddles a kv head
                        const int n = n0 + c0 + i;
                        if (n >= a.N) break;
                        float4 v = make_float4(__uint_as_float(r[i]), __uint_as_float(r[i + 1]),
                                               __uint_as_float(r[i + 2]), __uint_as_float(r[i + 3]));
                        if (a.bias) {
                            const float4 bb = *reinterpret_cast<const float4*>(a.bias + (size_t)b * a.N + n);
                            v.x += bb.x; v.y += bb.y; v.z += bb.z; v.w += bb.w;
                        }
                        const int hk = n / a.S, j = n - hk * a.S;
                        *reinterpret_cast<float4*>(a.scores + (((size_t)b * a.Hkv + hk) * a.T + t) * a.S + j) = v;
                    }
                }
            }
        } else if (lane == 0) {
            *abort_flag = 1; atomicExch(a.status, (int)STC_ERR_TIMEOUT);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(tmem_cols) : "memory");
    }
}

}  // namespace

namespace {

using EncodeTiledFn = CUresult (*)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                   const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                   CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// The tensor-map encoder lives in the driver; it is looked up through the runtime so the
// library does not link against libcuda.
EncodeTiledFn encode_tiled() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

// bf16 matrix [rows][cols] (cols contiguous) -> map with a [box_rows][64] box, 128-byte swizzle,
// zero fill outside the matrix.
bool make_map(CUtensorMap* map, const void* ptr, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    EncodeTiledFn enc = encode_tiled();
    if (!enc) return false;
    const cuuint64_t dims[2] = {cols, rows};
    const cuuint64_t strides[1] = {cols * 2};
    const cuuint32_t box[2] = {(cuuint32_t)kBK, box_rows};
    const cuuint32_t elem[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, elem,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

}  // namespace

// Returns cudaErrorNotSupported for shapes the tile scheme does not cover (checked by the caller too).
cudaError_t launch_router_logits(const Geom& g, const void* h, const void* w, const float* bias, int d_model,
                                 float* scores, int32_t* status, cudaStream_t st) {
    const long long M = (long long)g.B * g.T;
    const int N = g.Hkv * g.S;
    if (M == 0) return cudaSuccess;
    const int BN = N <= kMaxBN ? N : kMaxBN;
    if (d_model <= 0 || d_model % kBK != 0 || N % 16 != 0 || N % BN != 0 || M > 0x7FFFFFFFLL)
        return cudaErrorNotSupported;
    CUtensorMap map_h, map_w;
    if (!make_map(&map_h, h, (uint64_t)M, (uint64_t)d_model, kBM) || !make_map(&map_w, w, (uint64_t)N, (uint64_t)d_model, (uint32_t)BN))
        return cudaErrorInvalidValue;
    cudaError_t e = cudaMemsetAsync(status, 0, sizeof(int32_t), st);
    if (e != cudaSuccess) return e;
    RouterArgs a;
    a.bias = bias; a.scores = scores; a.status = status;
    a.M = (int)M; a.N = N; a.K = d_model; a.T = g.T; a.S = g.S; a.Hkv = g.Hkv; a.BN = BN;
    e = cudaFuncSetAttribute(router_logits_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kSmemBytes);
    if (e != cudaSuccess) return e;
    const dim3 grid((unsigned)((M + kBM - 1) / kBM), (unsigned)(N / BN));
    router_logits_kernel<<<grid, kThreads, kSmemBytes, st>>>(map_h, map_w, a);
    return cudaGetLastError();
}

}  // namespace stc
