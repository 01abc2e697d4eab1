// Shared device-side definitions of the verification-step kernels (sm_100a).
#pragma once

#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/aggressive_decoding.h"

namespace ad {

typedef __nv_bfloat16 bf16;

// ---------------------------------------------------------------------------------------------
// Scalar conversion helpers: activations between kernels are float (FP32 models) or bf16.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ float to_f32(float v) { return v; }
__device__ __forceinline__ float to_f32(bf16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ bf16 from_f32<bf16>(float v) { return __float2bfloat16_rn(v); }

// ---------------------------------------------------------------------------------------------
// One pass over a packed set of token rows.  A "pass" is the verification block forward, the
// drafter forward or the encoder forward; rows of the batch contribute seg_len[b] consecutive
// packed tokens starting at seg_off[b].
// ---------------------------------------------------------------------------------------------
struct PassPlan {
  int* M;          // [1] total packed tokens of this pass
  int* seg_off;    // [B] first packed token of row b
  int* seg_len;    // [B] tokens of row b (0 = row idle)
  int* key_base;   // [B] slot index of self-attention key 0 of row b
  int* tok_row;    // [Mmax] batch row of packed token m
  int* tok_pos;    // [Mmax] position fed to the positional table
  int* tok_id;     // [Mmax] input token id
  int* kv_slot;    // [Mmax] slot that receives this token's self-attention key/value
  int* att_n;      // [Mmax] number of self-attention keys the token may see (from key_base)
};

// Epilogue selector of the two GEMM kernels.
enum Epi : int {
  EPI_F32 = 0,      // out_f32[m][n] = acc (+ bias) (+ resid[m][n])
  EPI_ACT = 1,      // out_act[m][n] = act(acc + bias), optional ReLU
  EPI_SCATTER = 2,  // feature n belongs to segment n / seg_width; segment s goes to dst[s] at row
                    //   (s < n_direct ? m : slot[m]), column n % seg_width
  EPI_ARGMAX = 3    // per (feature tile, token) running (max, lowest id) partials
};

struct GemmParams {
  int K;                 // contraction length
  int N;                 // output features (rows of W)
  int ntile;             // tokens per CTA tile
  const int* M_ptr;      // device scalar: number of valid packed tokens (null: use M_host)
  int M_host;
  int M_cap;             // capacity of the token dimension of the buffers
  const float* bias;     // [N] or null
  int relu;
  // EPI_F32
  float* out_f32;        // [M_cap, N]
  const float* resid;    // [M_cap, N] or null
  // EPI_ACT
  void* out_act;         // [M_cap, N] float or bf16
  // EPI_SCATTER
  void* dst[3];
  int seg_width;
  int n_direct;
  const int* slot;       // [M_cap]
  // EPI_ARGMAX
  float* part_val;       // [n_tiles, M_cap]
  int* part_idx;         // [n_tiles, M_cap]
  int* status;           // device status word (latches AD_ERR_TIMEOUT), may be null
};

__device__ __forceinline__ void latch_error(int* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

}  // namespace ad
