// Scaled dot-product attention over packed token rows with keys/values staged through shared memory and
// an online (running max / running sum) softmax reduced with warp shuffles.
//
// One kernel serves the three attention patterns of the model:
//   - block-causal self-attention of the verification pass: query i of a row sees the cached prefix and the
//     block positions up to and including its own (per-token key count),
//   - cross-attention over the cached encoder keys/values of the row's source (per-row key count, which is
//     what masks the padding of a right-padded batch),
//   - unmasked self-attention of the encoder and of the drafter (per-token key count = whole segment).
#pragma once

#include "ad_common.cuh"

namespace ad {

struct AttnParams {
  const void* q;         // [M_cap, d]
  const void* k;         // [slots, d]
  const void* v;         // [slots, d]
  void* out;             // [M_cap, d]
  const int* seg_off;    // [B]
  const int* seg_len;    // [B]
  const int* key_base;   // [B] slot of key 0 of row b
  const int* nkeys_tok;  // [M_cap] keys visible to each packed token, or null
  const int* nkeys_row;  // [B] upper bound of the keys any token of row b sees (the count itself when nkeys_tok is null)
  int d;
  int qchunks;           // query chunks per row = ceil(longest possible segment / 16)
  float scale;           // 1 / sqrt(head dim)
};

// Eight consecutive elements (16-byte aligned for bf16, 32-byte for float) as floats.
__device__ __forceinline__ void load8(const bf16* p, float* out) {
  const uint4 u = *reinterpret_cast<const uint4*>(p);
  const __nv_bfloat162* h = reinterpret_cast<const __nv_bfloat162*>(&u);
#pragma unroll
  for (int t = 0; t < 4; ++t) {
    const float2 f = __bfloat1622float2(h[t]);
    out[2 * t] = f.x;
    out[2 * t + 1] = f.y;
  }
}
__device__ __forceinline__ void load8(const float* p, float* out) {
  const float4 a = *reinterpret_cast<const float4*>(p);
  const float4 b = *reinterpret_cast<const float4*>(p + 4);
  out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w;
  out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
}

constexpr int ATT_QC = 8;    // queries per CTA: one per warp
constexpr int ATT_KT = 64;   // keys per shared-memory tile

// grid = (B * qchunks, H); block = 256 threads (8 warps, one query each).
// Global-memory round trips on the critical path: (1) the row's segment / key-range descriptors,
// (2) the queries, their key counts and the first K/V tile together, then compute and store.
template <typename ActT, int DH>
__global__ void __launch_bounds__(256)
attention_kernel(const AttnParams p) {
  constexpr int R = DH / 32;                 // output dims per lane
  __shared__ float ks[ATT_KT][DH + 1];
  __shared__ float vs[ATT_KT][DH];
  __shared__ float qs[ATT_QC][DH];
  __shared__ float ps[ATT_QC][ATT_KT];

  trace_mark(TR_ATTN, 0);
  pdl_launch();
  pdl_wait();
  trace_mark(TR_ATTN, 1);
  const int b = blockIdx.x / p.qchunks;
  const int chunk = blockIdx.x % p.qchunks;
  const int h = blockIdx.y;
  const int seg_len = p.seg_len[b];
  const int seg_off = p.seg_off[b];
  const int kbase = p.key_base[b];
  const int row_nk = p.nkeys_row[b];         // no token of this row sees more keys than this
  const int i0 = chunk * ATT_QC;
  if (i0 >= seg_len) return;
  const int nq = min(ATT_QC, seg_len - i0);
  const int m0 = seg_off + i0;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const ActT* q = reinterpret_cast<const ActT*>(p.q);
  const ActT* kk = reinterpret_cast<const ActT*>(p.k);
  const ActT* vv = reinterpret_cast<const ActT*>(p.v);
  const int d = p.d;
  const bool has_q = warp < nq;

  // this warp's query and its visible-key count
  int nk = 0;
  if (has_q) {
    nk = p.nkeys_tok ? min(p.nkeys_tok[m0 + warp], row_nk) : row_nk;
#pragma unroll
    for (int rr = 0; rr < R; ++rr)
      qs[warp][lane + 32 * rr] = to_f32(q[(size_t)(m0 + warp) * d + h * DH + lane + 32 * rr]) * p.scale;
  }

  float mx = -INFINITY, den = 0.f, acc[R];
#pragma unroll
  for (int r = 0; r < R; ++r) acc[r] = 0.f;

  for (int j0 = 0; j0 < row_nk; j0 += ATT_KT) {
    __syncthreads();   // previous tile fully consumed
    for (int idx = tid; idx < ATT_KT * (DH / 8); idx += 256) {
      const int j = idx / (DH / 8), c = (idx % (DH / 8)) * 8;
      float kf[8], vf[8];
      if (j0 + j < row_nk) {
        const size_t off = (size_t)(kbase + j0 + j) * d + h * DH + c;
        load8(kk + off, kf);
        load8(vv + off, vf);
      } else {
#pragma unroll
        for (int t = 0; t < 8; ++t) { kf[t] = 0.f; vf[t] = 0.f; }
      }
#pragma unroll
      for (int t = 0; t < 8; ++t) { ks[j][c + t] = kf[t]; vs[j][c + t] = vf[t]; }
    }
    __syncthreads();
    if (nk <= j0) continue;   // warp-uniform: no visible key in this tile (the barriers above are still reached)
    float s0 = 0.f, s1 = 0.f;
#pragma unroll 8
    for (int c = 0; c < DH; ++c) {
      const float qv = qs[warp][c];
      s0 = fmaf(qv, ks[lane][c], s0);
      s1 = fmaf(qv, ks[lane + 32][c], s1);
    }
    if (j0 + lane >= nk) s0 = -INFINITY;
    if (j0 + lane + 32 >= nk) s1 = -INFINITY;
    float tmax = fmaxf(s0, s1);
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, off));
    const float m_new = fmaxf(mx, tmax);           // finite: key j0 is visible
    const float corr = expf(mx - m_new);           // exp(-inf) = 0 on the first tile
    const float p0 = expf(s0 - m_new), p1 = expf(s1 - m_new);
    float psum = p0 + p1;
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, off);
    den = den * corr + psum;
    mx = m_new;
    ps[warp][lane] = p0;
    ps[warp][lane + 32] = p1;
    __syncwarp();
#pragma unroll
    for (int rr = 0; rr < R; ++rr) {
      float a = acc[rr] * corr;
      const int c = lane + 32 * rr;
#pragma unroll 8
      for (int j = 0; j < ATT_KT; ++j) a = fmaf(ps[warp][j], vs[j][c], a);
      acc[rr] = a;
    }
    __syncwarp();
  }

  if (has_q && nk > 0) {
    ActT* out = reinterpret_cast<ActT*>(p.out);
    const float inv = 1.f / den;
#pragma unroll
    for (int rr = 0; rr < R; ++rr)
      out[(size_t)(m0 + warp) * d + h * DH + lane + 32 * rr] = from_f32<ActT>(acc[rr] * inv);
  }
  trace_mark(TR_ATTN, 2);
}

}  // namespace ad
