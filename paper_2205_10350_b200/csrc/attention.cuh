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
  // Fused output projection (FUSE kernels only): instead of storing the attention output, the CTA of head h multiplies
  // its queries' outputs (rounded to BF16, as a stored output would be) with columns [64 h, 64 h + 64) of wo [d, d]
  // and writes o_part[h][m, :] = the head's FP32 share of the projection; the residual + LayerNorm kernel adds the
  // heads up like split-K partials.
  const bf16* wo;
  float* o_part;         // [heads][M_cap, d]
  size_t o_stride;       // M_cap * d
};

// D (16 x 8, FP32) += A (16 x 16, BF16, row-major) * B (16 x 8, BF16, column-major), warp-level.
__device__ __forceinline__ void att_mma_bf16(float (&c)[4], uint32_t a0, uint32_t a1, uint32_t a2, uint32_t a3,
                                             uint32_t b0, uint32_t b1) {
  asm volatile(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a0), "r"(a1), "r"(a2), "r"(a3), "r"(b0), "r"(b1));
}

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

// Eight consecutive elements kept as loaded (no use of the data, so the load stays in flight) and widened later.
template <typename T> struct Raw8;
template <> struct Raw8<bf16> {
  uint4 u;
  __device__ __forceinline__ void load(const bf16* p) { u = *reinterpret_cast<const uint4*>(p); }
  __device__ __forceinline__ void zero() { u = make_uint4(0u, 0u, 0u, 0u); }
  __device__ __forceinline__ void widen(float* out) const {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int t = 0; t < 4; ++t) { out[2 * t] = __uint_as_float(w[t] << 16); out[2 * t + 1] = __uint_as_float(w[t] & 0xffff0000u); }
  }
};
template <> struct Raw8<float> {
  float4 a, b;
  __device__ __forceinline__ void load(const float* p) { a = *reinterpret_cast<const float4*>(p); b = *reinterpret_cast<const float4*>(p + 4); }
  __device__ __forceinline__ void zero() { a = make_float4(0.f, 0.f, 0.f, 0.f); b = a; }
  __device__ __forceinline__ void widen(float* out) const {
    out[0] = a.x; out[1] = a.y; out[2] = a.z; out[3] = a.w; out[4] = b.x; out[5] = b.y; out[6] = b.z; out[7] = b.w;
  }
};

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
// (2) the queries, their key counts and the first K/V tile together (the tile's loads are issued first and only
// widened once the queries are in shared memory), then compute and store.
// FUSE (BF16, 64-wide heads, one query per warp): the output projection of the 8 queries is done here as well (see
// AttnParams::wo).  Warp w owns output features [w d / 8, (w + 1) d / 8); its weight fragments -- 16 rows x 64 columns
// per group of rows, read with 16-byte loads whose eight elements are consecutive in K (the contraction index is
// permuted identically for both MMA operands) -- are requested before the dependency wait, since weights never change.
// MINB = 2 (at most 128 registers, two CTAs per SM) is for grids of more CTAs than SMs -- a batch of 8 rows x 4 query
// chunks x 8 heads: measured, the second wave of such a 256-CTA grid doubled the kernel's time; grids that fit one wave
// use MINB = 1, which keeps every CTA on an SM of its own.
template <typename ActT, int DH, int QPW, bool FUSE = false, int MINB = 1>
__global__ void __launch_bounds__(256, MINB)
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
  // fused projection: first four row groups of this warp's weight fragments ([group][K chunk][row g / g + 8])
  uint4 wf[4][2][2];
  __shared__ __align__(16) bf16 a_s[ATT_WARPS][96];       // the queries' outputs; row stride 192 B: conflict-free 16-byte loads
  if (FUSE) {
    const int lane_ = threadIdx.x & 31, g_ = lane_ >> 2, t_ = lane_ & 3;
    const int nrgw = p.d >> 7;                              // row groups of 16 per warp
    const bf16* wbase = p.wo + (size_t)((threadIdx.x >> 5) * nrgw * 16 + g_) * p.d + blockIdx.y * DH + 8 * t_;
#pragma unroll
    for (int r = 0; r < 4; ++r)
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        if (r < nrgw) {
          wf[r][c][0] = __ldg(reinterpret_cast<const uint4*>(wbase + (size_t)(r * 16) * p.d + c * 32));
          wf[r][c][1] = __ldg(reinterpret_cast<const uint4*>(wbase + (size_t)(r * 16 + 8) * p.d + c * 32));
        }
      }
  }
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

  // first K/V tile: requested now, used after the queries have been staged
  constexpr int NPRE = (ATT_KT * (DH / 8) + 255) / 256;
  Raw8<ActT> kpre[NPRE], vpre[NPRE];
#pragma unroll
  for (int u = 0; u < NPRE; ++u) {
    const int idx = tid + 256 * u;
    const int j = idx / (DH / 8), c = (idx % (DH / 8)) * 8;
    if (idx < ATT_KT * (DH / 8) && j < row_nk) {
      const size_t off = (size_t)(kbase + j) * d + h * DH + c;
      kpre[u].load(kk + off);
      vpre[u].load(vv + off);
    } else {
      kpre[u].zero();
      vpre[u].zero();
    }
  }

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
    if (j0 == 0) {
#pragma unroll
      for (int u = 0; u < NPRE; ++u) {
        const int idx = tid + 256 * u;
        if (idx < ATT_KT * (DH / 8)) {
          const int j = idx / (DH / 8), c = (idx % (DH / 8)) * 8;
          float kf[8], vf[8];
          kpre[u].widen(kf);
          vpre[u].widen(vf);
#pragma unroll
          for (int t = 0; t < 8; ++t) { ks[j][c + t] = kf[t]; vs[j][c + t] = vf[t]; }
        }
      }
    }
    for (int idx = tid; j0 > 0 && idx < ATT_KT * (DH / 8); idx += 256) {
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

  if (FUSE) {
    // this warp's query (QPW == 1) as BF16 into shared memory, zeros for the chunk's missing queries
    const bool have = warp < nq && nk[0] > 0;
    const float inv = have ? 1.f / den[0] : 0.f;
#pragma unroll
    for (int rr = 0; rr < R; ++rr) a_s[warp][lane + 32 * rr] = __float2bfloat16_rn(have ? acc[0][rr] * inv : 0.f);
    __syncthreads();
    const int g = lane >> 2, t4 = lane & 3;
    const int nrgw = d >> 7;
    // B fragments: query g, K elements 8 t .. 8 t + 7 of each 32-wide chunk
    const uint4 xb0 = *reinterpret_cast<const uint4*>(&a_s[g][8 * t4]);
    const uint4 xb1 = *reinterpret_cast<const uint4*>(&a_s[g][32 + 8 * t4]);
    float* obase = p.o_part + (size_t)h * p.o_stride + (size_t)m0 * d;
    for (int r0 = 0; r0 < nrgw; r0 += 4) {
      if (r0 > 0) {                                         // wider models: the next four row groups
        const bf16* wbase = p.wo + (size_t)((warp * nrgw + r0) * 16 + g) * d + h * DH + 8 * t4;
#pragma unroll
        for (int r = 0; r < 4; ++r)
#pragma unroll
          for (int c = 0; c < 2; ++c) {
            if (r0 + r < nrgw) {
              wf[r][c][0] = __ldg(reinterpret_cast<const uint4*>(wbase + (size_t)(r * 16) * d + c * 32));
              wf[r][c][1] = __ldg(reinterpret_cast<const uint4*>(wbase + (size_t)(r * 16 + 8) * d + c * 32));
            }
          }
      }
      float o[4][4];
#pragma unroll
      for (int r = 0; r < 4; ++r) { o[r][0] = 0.f; o[r][1] = 0.f; o[r][2] = 0.f; o[r][3] = 0.f; }
      // the four MMAs of a row group share an accumulator: walk the groups in the inner loop so that dependent
      // MMAs are four instructions apart
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        const uint4 xb = c == 0 ? xb0 : xb1;
#pragma unroll
        for (int r = 0; r < 4; ++r)
          if (r0 + r < nrgw) att_mma_bf16(o[r], wf[r][c][0].x, wf[r][c][1].x, wf[r][c][0].y, wf[r][c][1].y, xb.x, xb.y);
#pragma unroll
        for (int r = 0; r < 4; ++r)
          if (r0 + r < nrgw) att_mma_bf16(o[r], wf[r][c][0].z, wf[r][c][1].z, wf[r][c][0].w, wf[r][c][1].w, xb.z, xb.w);
      }
      // o[r]: features n, n + 8 (n = first feature of the group + g) of queries 2 t, 2 t + 1
#pragma unroll
      for (int r = 0; r < 4; ++r) {
        if (r0 + r < nrgw) {
          const int n = (warp * nrgw + r0 + r) * 16 + g;
          const int q0 = 2 * t4, q1 = q0 + 1;
          if (q0 < nq) { obase[(size_t)q0 * d + n] = o[r][0]; obase[(size_t)q0 * d + n + 8] = o[r][2]; }
          if (q1 < nq) { obase[(size_t)q1 * d + n] = o[r][1]; obase[(size_t)q1 * d + n + 8] = o[r][3]; }
        }
      }
    }
  } else {
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
  }
  trace_mark(TR_ATTN, 2);
}

}  // namespace ad
