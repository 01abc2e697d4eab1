// FP32 projection GEMM on the FP32 pipes (FFMA), for models whose weights are FP32 and whose scores have to
// match an FP32 definition to 1e-3: no TF32, no reduced-precision operands.  Same D^T[n, m] orientation and
// the same epilogues as the tensor-core kernel: one thread per output feature, 16 tokens per CTA, the
// contraction index walked in ascending order.
#pragma once

#include "ad_common.cuh"
#include "gemm_tc.cuh"   // epilogue_chunk, warp_argmax

namespace ad {
namespace simt {

constexpr int FEAT = 128;
constexpr int TOK = 16;
constexpr int KT = 32;

// grid = (ceil(N / 128), ceil(M_cap / 16)); block = 128.  x: [M_cap, K] float, w: [N, K] float.
template <int EPI>
__global__ void __launch_bounds__(128)
gemm_f32_kernel(const float* __restrict__ w, const float* __restrict__ x, const GemmParams p) {
  __shared__ float ws[KT][FEAT + 1];
  __shared__ float xs[TOK][KT];
  __shared__ float red_val[4][TOK];
  __shared__ int red_idx[4][TOK];
  __shared__ int red_cnt[4][TOK];

  pdl_launch();
  pdl_wait();
  const int M = p.M_ptr ? *p.M_ptr : p.M_host;
  const int t0 = blockIdx.y * TOK;
  if (t0 >= M) return;
  const int n0 = blockIdx.x * FEAT;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int K = p.K;

  float acc[TOK];
#pragma unroll
  for (int j = 0; j < TOK; ++j) acc[j] = 0.f;

  for (int k0 = 0; k0 < K; k0 += KT) {
#pragma unroll
    for (int i = 0; i < (FEAT * KT) / 128; ++i) {
      const int idx = i * 128 + tid;
      const int row = idx / KT, col = idx % KT;
      const int n = n0 + row, k = k0 + col;
      ws[col][row] = (n < p.N && k < K) ? w[(size_t)n * K + k] : 0.f;
    }
#pragma unroll
    for (int i = 0; i < (TOK * KT) / 128; ++i) {
      const int idx = i * 128 + tid;
      const int row = idx / KT, col = idx % KT;
      const int m = t0 + row, k = k0 + col;
      xs[row][col] = (m < M && k < K) ? x[(size_t)m * K + k] : 0.f;
    }
    __syncthreads();
#pragma unroll 8
    for (int kk = 0; kk < KT; ++kk) {
      const float wv = ws[kk][tid];
#pragma unroll
      for (int j = 0; j < TOK; ++j) acc[j] = fmaf(wv, xs[j][kk], acc[j]);
    }
    __syncthreads();
  }

  const int n = n0 + tid;
  if (EPI == EPI_ARGMAX) {
#pragma unroll
    for (int j = 0; j < TOK; ++j) {
      float v = (n < p.N) ? acc[j] : -INFINITY;
      int i = n;
      if (p.draft_val) {   // relaxed verification: features other than the draft that score strictly higher
        const bool on = t0 + j < M;
        const bool above = on && n < p.N && n != p.draft_id[t0 + j] && acc[j] > p.draft_val[t0 + j];
        const unsigned int bal = __ballot_sync(0xffffffffu, above);
        if (lane == 0) red_cnt[warp][j] = __popc(bal);
      }
      tc::warp_argmax(v, i);
      if (lane == 0) { red_val[warp][j] = v; red_idx[warp][j] = i; }
    }
    __syncthreads();
    if (tid < TOK && t0 + tid < M) {
      float v = red_val[0][tid];
      int i = red_idx[0][tid];
#pragma unroll
      for (int wq = 1; wq < 4; ++wq) {
        const float ov = red_val[wq][tid];
        const int oi = red_idx[wq][tid];
        if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
      }
      p.part_val[(size_t)(t0 + tid) * gridDim.x + blockIdx.x] = v;
      p.part_idx[(size_t)(t0 + tid) * gridDim.x + blockIdx.x] = i;
      if (p.draft_val)
        p.part_cnt[(size_t)(t0 + tid) * gridDim.x + blockIdx.x] =
            red_cnt[0][tid] + red_cnt[1][tid] + red_cnt[2][tid] + red_cnt[3][tid];
    }
  } else {
    __shared__ int slot_s[TOK];
    if (EPI == EPI_SCATTER) {
      if (tid < TOK) slot_s[tid] = (t0 + tid < M) ? p.slot[t0 + tid] : 0;
      __syncthreads();
    }
    const float b = (p.bias && n < p.N) ? p.bias[n] : 0.f;
    tc::epilogue_chunk<EPI, float>(p, n, t0, M, acc, b, p.out_f32, slot_s, 0);
  }
}

}  // namespace simt
}  // namespace ad
