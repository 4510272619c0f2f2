// Query summary and its router term (Section 3.4: the value-group router sees the
// token's hidden state and a summary s_Q of the query region).  The summary operator
// and the router's g are not specified; the reading here is s_Q = mean of the
// query-region hidden states and g linear in [h ; s_Q], so the query contributes one
// additive term per sequence and logit:
//     s_q[b][c]  = (1 / q_len[b]) * sum_{t < q_len[b]} h_q[b][t][c]
//     bias[b][n] = sum_c s_q[b][c] * w_q[n][c]
// which stc_router_logits takes as bias_opt.
//
// Two small bandwidth-trivial kernels with a fixed summation order (no atomics):
//   mean: a CTA owns 256 channels of one sequence; warp w sums tokens w, w+8, ...
//         (lane = 16-byte chunk of 8 channels), the eight partial sums are added in
//         warp order.
//   bias: one warp per (sequence, logit); lanes stride over the channels, then a
//         shuffle tree.
#include "common.cuh"

namespace stc {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;
constexpr int kChanPerCta = 32 * 8;

__global__ void __launch_bounds__(kThreads)
query_mean_kernel(const uint4* __restrict__ h_q, const int32_t* __restrict__ q_len, int Lq, int d_model,
                  float* __restrict__ s_q) {
    __shared__ float part[kWarps][kChanPerCta];
    const int b = blockIdx.y, lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int oct = blockIdx.x * 32 + lane, octs = d_model / 8;
    int n_tok = q_len ? q_len[b] : Lq;
    n_tok = n_tok < 0 ? 0 : (n_tok > Lq ? Lq : n_tok);
    float acc[8] = {0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f, 0.f};
    if (oct < octs) {
        const uint4* src = h_q + (size_t)b * Lq * octs + oct;
#pragma unroll 4
        for (int t = warp; t < n_tok; t += kWarps) {
            const uint4 r = ldg_nc16(src + (size_t)t * octs);
            acc[0] += bf16lo(r.x); acc[1] += bf16hi(r.x);
            acc[2] += bf16lo(r.y); acc[3] += bf16hi(r.y);
            acc[4] += bf16lo(r.z); acc[5] += bf16hi(r.z);
            acc[6] += bf16lo(r.w); acc[7] += bf16hi(r.w);
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) part[warp][lane * 8 + i] = acc[i];
    __syncthreads();
    const int ch = blockIdx.x * kChanPerCta + threadIdx.x;
    if (ch < d_model) {
        float s = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) s += part[w][threadIdx.x];
        s_q[(size_t)b * d_model + ch] = n_tok > 0 ? s / (float)n_tok : 0.f;
    }
}

__global__ void __launch_bounds__(kThreads)
query_bias_kernel(const float4* __restrict__ s_q, const uint4* __restrict__ w_q, int d_model, int n_logits,
                  int rows, float* __restrict__ bias) {
    const int row = blockIdx.x * kWarps + (threadIdx.x >> 5), lane = threadIdx.x & 31;
    if (row >= rows) return;
    const int b = row / n_logits, n = row - b * n_logits, octs = d_model / 8;
    const float4* s = s_q + (size_t)b * octs * 2;
    const uint4* w = w_q + (size_t)n * octs;
    float acc = 0.f;
    for (int o = lane; o < octs; o += 32) {
        const uint4 r = ldg_nc16(w + o);
        const float4 s0 = s[2 * o], s1 = s[2 * o + 1];
        acc += s0.x * bf16lo(r.x); acc += s0.y * bf16hi(r.x);
        acc += s0.z * bf16lo(r.y); acc += s0.w * bf16hi(r.y);
        acc += s1.x * bf16lo(r.z); acc += s1.y * bf16hi(r.z);
        acc += s1.z * bf16lo(r.w); acc += s1.w * bf16hi(r.w);
    }
#pragma unroll
    for (int d = 16; d >= 1; d >>= 1) acc += __shfl_xor_sync(0xFFFFFFFFu, acc, d);
    if (lane == 0) bias[row] = acc;
}

}  // namespace

cudaError_t launch_query_bias(int B, int Lq, int d_model, int n_logits, const void* h_q, const int32_t* q_len,
                              const void* w_q, float* s_q, float* bias, cudaStream_t st) {
    if (B <= 0 || d_model <= 0) return cudaSuccess;
    const dim3 grid_mean((unsigned)((d_model + kChanPerCta - 1) / kChanPerCta), (unsigned)B);
    query_mean_kernel<<<grid_mean, kThreads, 0, st>>>(static_cast<const uint4*>(h_q), q_len, Lq, d_model, s_q);
    const int rows = B * n_logits;
    if (rows > 0)
        query_bias_kernel<<<(unsigned)((rows + kWarps - 1) / kWarps), kThreads, 0, st>>>(
            reinterpret_cast<const float4*>(s_q), static_cast<const uint4*>(w_q), d_model, n_logits, rows, bias);
    return cudaGetLastError();
}

}  // namespace stc
