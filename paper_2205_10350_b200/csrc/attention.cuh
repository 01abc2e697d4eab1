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
  // When q_part is set the queries come straight from the split-K partial sums of their projection instead:
  // q = round_to_activation_type(sum over q_nsplit partials [M_cap, d], q_stride elements apart, + q_bias).
  const float* q_part;
  const float* q_bias;   // [d] or null
  int q_nsplit;
  size_t q_stride;
  const void* k;         // [slots, d]
  const void* v;         // [slots, d]
  void* out;             // [M_cap, d]
  const int* seg_off;    // [B]
  const int* seg_len;    // [B]
  const int* key_base;   // [B] slot of key 0 of row b
  const int* nkeys_tok;  // [M_cap] keys visible to each packed token, or null
  const int* nkeys_row;  // [B] upper bound of the keys any token of row b sees (the count itself when nkeys_tok is null)
  int d;
  int qchunks;           // query chunks per row = ceil(longest possible segment / queries per CTA)
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

constexpr int ATT_WARPS = 8;   // warps per CTA
constexpr int ATT_MAX_QSPLIT = 16;   // most split-K partials a query may be summed from
constexpr int ATT_KT = 64;     // keys per shared-memory tile

template <int DH, int QPW>
constexpr size_t att_smem_bytes() {
  return sizeof(float) * (size_t)(ATT_KT * (DH + 1) + ATT_KT * DH + ATT_WARPS * QPW * DH + ATT_WARPS * QPW * ATT_KT);
}

// grid = (B * qchunks, H); block = 256 threads (8 warps, QPW queries each; a CTA covers 8 * QPW queries of one
// row and one head and stages every K/V tile once for all of them).  QPW = 1 keeps the critical path short when
// there are few queries; QPW = 8 amortises the K/V staging when there are thousands.
// Global-memory round trips on the critical path: (1) the row's segment / key-range descriptors,
// (2) the queries, their key counts and the first K/V tile together, then compute and store.
template <typename ActT, int DH, int QPW>
__global__ void __launch_bounds__(256)
attention_kernel(const AttnParams p) {
  constexpr int R = DH / 32;                 // output dims per lane
  constexpr int QC = ATT_WARPS * QPW;        // queries per CTA
  // dynamic shared memory (att_smem_bytes<DH, QPW>()): K tile (padded rows), V tile, queries, probabilities
  extern __shared__ __align__(16) float att_smem[];
  float (*ks)[DH + 1] = reinterpret_cast<float (*)[DH + 1]>(att_smem);
  float (*vs)[DH] = reinterpret_cast<float (*)[DH]>(att_smem + ATT_KT * (DH + 1));
  float (*qs)[DH] = reinterpret_cast<float (*)[DH]>(att_smem + ATT_KT * (DH + 1) + ATT_KT * DH);
  float (*ps)[ATT_KT] = reinterpret_cast<float (*)[ATT_KT]>(att_smem + ATT_KT * (DH + 1) + ATT_KT * DH + QC * DH);

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
  const int i0 = chunk * QC;
  if (i0 >= seg_len) return;
  const int nq = min(QC, seg_len - i0);
  const int m0 = seg_off + i0;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const ActT* q = reinterpret_cast<const ActT*>(p.q);
  const ActT* kk = reinterpret_cast<const ActT*>(p.k);
  const ActT* vv = reinterpret_cast<const ActT*>(p.v);
  const int d = p.d;

  // this warp's queries (warp, warp + 8, ...) and their visible-key counts
  int nk[QPW];
#pragma unroll
  for (int t = 0; t < QPW; ++t) {
    const int r = warp + ATT_WARPS * t;
    nk[t] = 0;
    if (r < nq) {
      nk[t] = p.nkeys_tok ? min(p.nkeys_tok[m0 + r], row_nk) : row_nk;
#pragma unroll
      for (int rr = 0; rr < R; ++rr) {
        const int col = h * DH + lane + 32 * rr;
        const size_t off = (size_t)(m0 + r) * d + col;
        float qv;
        if (p.q_part) {
          qv = p.q_bias ? p.q_bias[col] : 0.f;
          float part[ATT_MAX_QSPLIT];                  // all partials in one round trip
#pragma unroll
          for (int sp = 0; sp < ATT_MAX_QSPLIT; ++sp) part[sp] = sp < p.q_nsplit ? p.q_part[sp * p.q_stride + off] : 0.f;
#pragma unroll
          for (int sp = 0; sp < ATT_MAX_QSPLIT; ++sp) qv += part[sp];
          qv = to_f32(from_f32<ActT>(qv));     // the value a stored query would have had
        } else {
          qv = to_f32(q[off]);
        }
        qs[r][lane + 32 * rr] = qv * p.scale;
      }
    }
  }

  float mx[QPW], den[QPW], acc[QPW][R];
#pragma unroll
  for (int t = 0; t < QPW; ++t) {
    mx[t] = -INFINITY; den[t] = 0.f;
#pragma unroll
    for (int r = 0; r < R; ++r) acc[t][r] = 0.f;
  }

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
    // scores of this warp's QPW queries against keys lane and lane + 32: every K element read from shared
    // memory is used for all QPW queries
    float s0[QPW], s1[QPW];
#pragma unroll
    for (int t = 0; t < QPW; ++t) { s0[t] = 0.f; s1[t] = 0.f; }
#pragma unroll 4
    for (int c = 0; c < DH; ++c) {
      const float k0 = ks[lane][c], k1 = ks[lane + 32][c];
#pragma unroll
      for (int t = 0; t < QPW; ++t) {
        const float qv = qs[warp + ATT_WARPS * t][c];
        s0[t] = fmaf(qv, k0, s0[t]);
        s1[t] = fmaf(qv, k1, s1[t]);
      }
    }
    float corr[QPW];
#pragma unroll
    for (int t = 0; t < QPW; ++t) {
      float p0 = 0.f, p1 = 0.f;
      corr[t] = 1.f;
      if (nk[t] > j0) {              // warp-uniform; otherwise no key of this tile is visible to the query
        const float a0 = (j0 + lane < nk[t]) ? s0[t] : -INFINITY;
        const float a1 = (j0 + lane + 32 < nk[t]) ? s1[t] : -INFINITY;
        float tmax = fmaxf(a0, a1);
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, off));
        const float m_new = fmaxf(mx[t], tmax);        // finite: key j0 is visible
        corr[t] = expf(mx[t] - m_new);                 // exp(-inf) = 0 on the first tile
        p0 = expf(a0 - m_new);
        p1 = expf(a1 - m_new);
        float psum = p0 + p1;
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, off);
        den[t] = den[t] * corr[t] + psum;
        mx[t] = m_new;
      }
      ps[warp * QPW + t][lane] = p0;
      ps[warp * QPW + t][lane + 32] = p1;
    }
    __syncwarp();
#pragma unroll
    for (int rr = 0; rr < R; ++rr) {
      const int c = lane + 32 * rr;
      float a[QPW];
#pragma unroll
      for (int t = 0; t < QPW; ++t) a[t] = acc[t][rr] * corr[t];
      const int jn = min(ATT_KT, row_nk - j0);      // keys of this tile that exist at all
#pragma unroll 4
      for (int j = 0; j < jn; ++j) {
        const float v = vs[j][c];
#pragma unroll
        for (int t = 0; t < QPW; ++t) a[t] = fmaf(ps[warp * QPW + t][j], v, a[t]);
      }
#pragma unroll
      for (int t = 0; t < QPW; ++t) acc[t][rr] = a[t];
    }
    __syncwarp();
  }

  ActT* out = reinterpret_cast<ActT*>(p.out);
#pragma unroll
  for (int t = 0; t < QPW; ++t) {
    const int r = warp + ATT_WARPS * t;
    if (r < nq && nk[t] > 0) {
      const float inv = 1.f / den[t];
#pragma unroll
      for (int rr = 0; rr < R; ++rr)
        out[(size_t)(m0 + r) * d + h * DH + lane + 32 * rr] = from_f32<ActT>(acc[t][rr] * inv);
    }
  }
  trace_mark(TR_ATTN, 2);
}

}  // namespace ad
