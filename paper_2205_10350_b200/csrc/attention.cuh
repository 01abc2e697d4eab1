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
  const int* nkeys_row;  // [B] keys visible to every token of row b (used when nkeys_tok is null)
  int d;
  int qchunks;           // query chunks per row = ceil(longest possible segment / 16)
  float scale;           // 1 / sqrt(head dim)
};

constexpr int ATT_QC = 16;   // queries per CTA
constexpr int ATT_KT = 64;   // keys per shared-memory tile

// grid = (B * qchunks, H); block = 128 threads (4 warps, 4 queries each).
template <typename ActT, int DH>
__global__ void __launch_bounds__(128)
attention_kernel(const AttnParams p) {
  constexpr int R = DH / 32;                 // output dims per lane
  __shared__ float ks[ATT_KT][DH + 1];
  __shared__ float vs[ATT_KT][DH];
  __shared__ float qs[ATT_QC][DH];
  __shared__ float ps[4][ATT_KT];

  const int b = blockIdx.x / p.qchunks;
  const int chunk = blockIdx.x % p.qchunks;
  const int h = blockIdx.y;
  const int seg_len = p.seg_len[b];
  const int i0 = chunk * ATT_QC;
  if (i0 >= seg_len) return;
  const int nq = min(ATT_QC, seg_len - i0);
  const int m0 = p.seg_off[b] + i0;
  const int kbase = p.key_base[b];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const ActT* q = reinterpret_cast<const ActT*>(p.q);
  const ActT* kk = reinterpret_cast<const ActT*>(p.k);
  const ActT* vv = reinterpret_cast<const ActT*>(p.v);
  const int d = p.d;

  for (int idx = tid; idx < ATT_QC * DH; idx += 128) {
    const int r = idx / DH, c = idx % DH;
    qs[r][c] = (r < nq) ? to_f32(q[(size_t)(m0 + r) * d + h * DH + c]) * p.scale : 0.f;
  }

  // per-query key counts (this warp's queries are warp, warp+4, warp+8, warp+12)
  int nk[4];
  int nk_max = 0;
#pragma unroll
  for (int t = 0; t < 4; ++t) {
    const int r = warp + 4 * t;
    nk[t] = (r < nq) ? (p.nkeys_tok ? p.nkeys_tok[m0 + r] : p.nkeys_row[b]) : 0;
  }
  for (int r = 0; r < nq; ++r) nk_max = max(nk_max, p.nkeys_tok ? p.nkeys_tok[m0 + r] : p.nkeys_row[b]);

  float mx[4], den[4], acc[4][R];
#pragma unroll
  for (int t = 0; t < 4; ++t) {
    mx[t] = -INFINITY; den[t] = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) acc[t][r] = 0.f;
  }

  for (int j0 = 0; j0 < nk_max; j0 += ATT_KT) {
    __syncthreads();   // previous tile fully consumed (also orders the qs writes before the first use)
    for (int idx = tid; idx < ATT_KT * DH; idx += 128) {
      const int j = idx / DH, c = idx % DH;
      float kvl = 0.f, vvl = 0.f;
      if (j0 + j < nk_max) {
        const size_t off = (size_t)(kbase + j0 + j) * d + h * DH + c;
        kvl = to_f32(kk[off]);
        vvl = to_f32(vv[off]);
      }
      ks[j][c] = kvl;
      vs[j][c] = vvl;
    }
    __syncthreads();
#pragma unroll
    for (int t = 0; t < 4; ++t) {
      const int r = warp + 4 * t;
      if (nk[t] <= j0) continue;   // warp-uniform: no visible key in this tile
      float s0 = 0.f, s1 = 0.f;
#pragma unroll 8
      for (int c = 0; c < DH; ++c) {
        const float qv = qs[r][c];
        s0 = fmaf(qv, ks[lane][c], s0);
        s1 = fmaf(qv, ks[lane + 32][c], s1);
      }
      if (j0 + lane >= nk[t]) s0 = -INFINITY;
      if (j0 + lane + 32 >= nk[t]) s1 = -INFINITY;
      float tmax = fmaxf(s0, s1);
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, off));
      const float m_new = fmaxf(mx[t], tmax);        // finite: key j0 is visible
      const float corr = expf(mx[t] - m_new);        // exp(-inf) = 0 on the first tile
      const float p0 = expf(s0 - m_new), p1 = expf(s1 - m_new);
      float psum = p0 + p1;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, off);
      den[t] = den[t] * corr + psum;
      mx[t] = m_new;
      ps[warp][lane] = p0;
      ps[warp][lane + 32] = p1;
      __syncwarp();
#pragma unroll
      for (int rr = 0; rr < R; ++rr) {
        float a = acc[t][rr] * corr;
        const int c = lane + 32 * rr;
#pragma unroll 8
        for (int j = 0; j < ATT_KT; ++j) a = fmaf(ps[warp][j], vs[j][c], a);
        acc[t][rr] = a;
      }
      __syncwarp();
    }
  }

  ActT* out = reinterpret_cast<ActT*>(p.out);
#pragma unroll
  for (int t = 0; t < 4; ++t) {
    const int r = warp + 4 * t;
    if (r < nq && nk[t] > 0) {
      const float inv = 1.f / den[t];
#pragma unroll
      for (int rr = 0; rr < R; ++rr)
        out[(size_t)(m0 + r) * d + h * DH + lane + 32 * rr] = from_f32<ActT>(acc[t][rr] * inv);
    }
  }
}

}  // namespace ad
