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
  int* row_nk;     // [B] largest number of self-attention keys any token of row b sees
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
                    //   (s < n_direct ? m : slot[m]), column n % seg_width.  With seg_pair_stride != 0 there may be any
                    //   number of segments: segment s goes to dst[s & 1] + (s >> 1) * seg_pair_stride bytes (key / value
                    //   buffers of consecutive layers)
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
  int ksplit;            // EPI_F32 only: blockIdx.z takes K range z/ksplit and writes partial z (1 = no split)
  // EPI_F32
  float* out_f32;        // [ksplit][M_cap, N]: partial sums; the consumer adds them up
  // EPI_ACT
  void* out_act;         // [M_cap, N] float or bf16
  // EPI_SCATTER
  void* dst[3];
  size_t seg_pair_stride;
  int seg_width;
  int n_direct;
  const int* slot;       // [M_cap]
  // EPI_ARGMAX
  float* part_val;       // [M_cap, n_tiles]: per token, the best value of every 128-feature tile
  int* part_idx;         // [M_cap, n_tiles]
  // EPI_ARGMAX with the relaxed verification (null: off): per token, the drafted token and its score; the kernel
  // adds, per feature tile, how many OTHER features score strictly higher than the draft
  const float* draft_val;  // [M_cap]
  const int* draft_id;     // [M_cap] (negative: no draft at this position)
  int* part_cnt;           // [M_cap, n_tiles]
  int* status;           // device status word (latches AD_ERR_TIMEOUT), may be null
};

// Programmatic dependent launch: a kernel launched with the programmatic-serialization attribute may start
// while its predecessor in the stream is still running.  pdl_wait() blocks until the predecessor grid (and,
// transitively, everything before it) has completed and its writes are visible; everything a kernel does
// before pdl_wait() must touch only data that no kernel ever writes (weights, the kernel's own shared memory).
// pdl_launch() lets the successor begin its own pre-wait part.  Both are no-ops in an ordinary launch.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_launch() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Optional timeline tracing (compile with -DAD_TRACE): thread 0 of CTA (0,0,0) of every kernel stamps the
// global nanosecond timer at entry (phase 0), after the dependency wait (phase 1), at exit (phase 2) and at
// kernel-specific points in between (phases 3..7); the last CTA along x does the same under id + 16.
#ifdef AD_TRACE
__device__ unsigned long long g_trace_buf[1 << 15];
__device__ unsigned int g_trace_n;
__device__ __forceinline__ void trace_mark(int id, int phase) {
  const bool first = blockIdx.x == 0, last = blockIdx.x == gridDim.x - 1 && gridDim.x > 1;
#ifdef AD_TRACE_ALL_EXITS
  // every CTA stamps its exit (under id + 16 unless it is CTA (0,0,0)): shows the tail of a grid
  if (phase == 2 && threadIdx.x == 0 && !(first && blockIdx.y == 0 && blockIdx.z == 0)) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    const unsigned int i = atomicAdd(&g_trace_n, 1u);
    if (i < (1u << 15)) g_trace_buf[i] = (t & 0x00FFFFFFFFFFFFFFull) | ((unsigned long long)((id + 16) * 8 + phase) << 56);
    return;
  }
#endif
  if (threadIdx.x == 0 && (first || last) && blockIdx.y == 0 && blockIdx.z == 0) {
    if (last) id += 16;
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    const unsigned int i = atomicAdd(&g_trace_n, 1u);
    if (i < (1u << 15)) g_trace_buf[i] = (t & 0x00FFFFFFFFFFFFFFull) | ((unsigned long long)(id * 8 + phase) << 56);
  }
}
// The same from whichever thread of CTA 0 calls it (role threads of warp-specialised kernels).
__device__ __forceinline__ void trace_mark_role(int id, int phase) {
  if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0) {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    const unsigned int i = atomicAdd(&g_trace_n, 1u);
    if (i < (1u << 15)) g_trace_buf[i] = (t & 0x00FFFFFFFFFFFFFFull) | ((unsigned long long)(id * 8 + phase) << 56);
  }
}
#else
__device__ __forceinline__ void trace_mark(int, int) {}
__device__ __forceinline__ void trace_mark_role(int, int) {}
#endif
enum TraceId { TR_GEMM = 0, TR_ATTN = 8, TR_LN = 9, TR_EMBED = 10, TR_PREPARE = 11, TR_ACCEPT = 12, TR_COMMIT = 13,
               TR_PV_ISSUE = 20, TR_PV_EPI = 21, TR_PV_LOAD = 22 };

__device__ __forceinline__ void latch_error(int* status, int code) {
  if (status) atomicCAS(status, 0, code);
}

}  // namespace ad
