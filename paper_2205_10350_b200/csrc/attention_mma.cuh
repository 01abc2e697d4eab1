// Attention for many queries on the tensor cores (BF16, head dimension 64).
//
// Same operation and masking rules as attention_kernel (attention.cuh); used when a pass has thousands of
// queries, where the FFMA kernel is bound by its multiply-adds.  The tiles of one (row, head) pair are small
// (at most 64 queries x 64 keys x 64 dims per step), far below the 128-row atoms of the tcgen05 path and not
// worth a round trip through tensor memory, so the products run as warp-level m16n8k16 MMAs on register
// fragments: S = Q K^T, online softmax on the accumulator fragments, P (rounded to BF16) reused in place as
// the A operand of O += P V, with V read through transposing ldmatrix loads.
//
// grid = (B * qchunks, H), qchunks = ceil(longest segment / queries per CTA); block = 128 threads.
#pragma once

#include "attention.cuh"

namespace ad {

constexpr int AM_Q = 64;        // queries per CTA with one key group
constexpr int AM_KT = 64;       // keys per shared-memory tile
constexpr int AM_LD = 64 + 8;   // padded row length (bf16 elements): rows 144 bytes apart, conflict-free fragments

__device__ __forceinline__ void mma_bf16_16816(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
  asm(
      "mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, "
      "{%0, %1, %2, %3};"
      : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
      : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);   // .x = lo (low half), .y = hi
  return *reinterpret_cast<uint32_t*>(&h);
}
// Two 8x8 BF16 matrices, transposed on the way into registers: lanes 0..7 give the row addresses of the first,
// lanes 8..15 of the second.
__device__ __forceinline__ void ldmatrix_x2_trans(uint32_t& r0, uint32_t& r1, const void* row_ptr) {
  const uint32_t addr = static_cast<uint32_t>(__cvta_generic_to_shared(row_ptr));
  asm volatile("ldmatrix.sync.aligned.m8n8.x2.trans.shared.b16 {%0, %1}, [%2];" : "=r"(r0), "=r"(r1) : "r"(addr));
}

// NG = number of key groups.  With NG = 1 the CTA's four warps take 16 queries each (64 queries per CTA).  When
// rows have few queries, NG = 2 or 4 warps share a 16-query tile instead (32 or 16 queries per CTA) and split
// the keys of every K/V tile between them; their running maxima, sums and outputs are merged at the end.
template <int NG>
__global__ void __launch_bounds__(128)
attention_mma_kernel(const AttnParams p) {
  constexpr int DH = 64;
  constexpr int QT = 4 / NG;            // 16-query tiles per CTA
  constexpr int KS = AM_KT / NG;        // keys of a tile that one warp handles
  __shared__ __align__(16) bf16 kv[2][AM_KT][AM_LD];
  bf16 (*ks)[AM_LD] = kv[0];
  bf16 (*vs)[AM_LD] = kv[1];

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
  const int row_nk = p.nkeys_row[b];
  const int i0 = chunk * (16 * QT);
  if (i0 >= seg_len) return;
  const int nq = min(16 * QT, seg_len - i0);
  const int m0 = seg_off + i0;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, tq = lane & 3;           // fragment row (0..7) and column pair (0..3) of this lane
  const int qtile = warp % QT, grp = warp / QT;     // this warp's query tile and key group
  const int kofs = grp * KS;                        // first key of a tile that this warp handles
  const bool active = qtile * 16 < nq;              // otherwise the warp only helps loading
  const int d = p.d;
  const bf16* q = reinterpret_cast<const bf16*>(p.q);
  const bf16* kk = reinterpret_cast<const bf16*>(p.k);
  const bf16* vv = reinterpret_cast<const bf16*>(p.v);

  // this lane's two queries (fragment rows g and g + 8 of the warp's 16) and their visible-key counts
  const int r0 = qtile * 16 + g, r1 = r0 + 8;
  int nk0 = 0, nk1 = 0;
  if (r0 < nq) nk0 = p.nkeys_tok ? min(p.nkeys_tok[m0 + r0], row_nk) : row_nk;
  if (r1 < nq) nk1 = p.nkeys_tok ? min(p.nkeys_tok[m0 + r1], row_nk) : row_nk;
  // Q as A fragments of the four 16-wide steps along the head dimension
  uint32_t qa[DH / 16][4];
  if (p.q_part) {
    // queries straight from the split-K partial sums of their projection (+ bias), rounded like stored ones
#pragma unroll
    for (int s4 = 0; s4 < DH / 16; ++s4) {
#pragma unroll
      for (int e = 0; e < 4; ++e) {
        const int r = (e & 1) ? r1 : r0;
        const int c = h * DH + s4 * 16 + tq * 2 + (e >> 1) * 8;
        float2 acc = make_float2(0.f, 0.f);
        if (r < nq) {
          if (p.q_bias) acc = *reinterpret_cast<const float2*>(p.q_bias + c);
          const float* src = p.q_part + (size_t)(m0 + r) * d + c;
          float2 part[ATT_MAX_QSPLIT];                 // all partials in one round trip
#pragma unroll
          for (int sp = 0; sp < ATT_MAX_QSPLIT; ++sp)
            part[sp] = sp < p.q_nsplit ? *reinterpret_cast<const float2*>(src + sp * p.q_stride) : make_float2(0.f, 0.f);
#pragma unroll
          for (int sp = 0; sp < ATT_MAX_QSPLIT; ++sp) { acc.x += part[sp].x; acc.y += part[sp].y; }
        }
        qa[s4][e] = pack_bf16(acc.x, acc.y);
      }
    }
  } else {
#pragma unroll
    for (int s4 = 0; s4 < DH / 16; ++s4) {
      const int c = h * DH + s4 * 16 + tq * 2;
      const bf16* q0 = q + (size_t)(m0 + r0) * d + c;
      const bf16* q1 = q + (size_t)(m0 + r1) * d + c;
      qa[s4][0] = r0 < nq ? *reinterpret_cast<const uint32_t*>(q0) : 0u;
      qa[s4][1] = r1 < nq ? *reinterpret_cast<const uint32_t*>(q1) : 0u;
      qa[s4][2] = r0 < nq ? *reinterpret_cast<const uint32_t*>(q0 + 8) : 0u;
      qa[s4][3] = r1 < nq ? *reinterpret_cast<const uint32_t*>(q1 + 8) : 0u;
    }
  }

  float o[DH / 8][4];
#pragma unroll
  for (int t = 0; t < DH / 8; ++t) { o[t][0] = 0.f; o[t][1] = 0.f; o[t][2] = 0.f; o[t][3] = 0.f; }
  float mx0 = -INFINITY, mx1 = -INFINITY, den0 = 0.f, den1 = 0.f;   // den: this lane's share of the row sums

  // K/V tiles travel global -> registers -> shared memory; the loads of tile t + 1 are issued before the
  // arithmetic of tile t so that their latency is hidden behind it.
  constexpr int PIECES = AM_KT * (DH / 8) / 128;    // 16-byte pieces per thread, per matrix and tile
  uint4 kreg[PIECES], vreg[PIECES];
  auto fetch = [&](int j0) {
#pragma unroll
    for (int i = 0; i < PIECES; ++i) {
      const int idx = tid + 128 * i;
      const int j = idx >> 3, c = (idx & 7) * 8;
      kreg[i] = make_uint4(0u, 0u, 0u, 0u);          // keys that do not exist read as zeros
      vreg[i] = kreg[i];
      if (j0 + j < row_nk) {
        const size_t off = (size_t)(kbase + j0 + j) * d + h * DH + c;
        kreg[i] = *reinterpret_cast<const uint4*>(kk + off);
        vreg[i] = *reinterpret_cast<const uint4*>(vv + off);
      }
    }
  };
  fetch(0);
  for (int j0 = 0; j0 < row_nk; j0 += AM_KT) {
    __syncthreads();   // previous tile fully consumed
#pragma unroll
    for (int i = 0; i < PIECES; ++i) {
      const int idx = tid + 128 * i;
      const int j = idx >> 3, c = (idx & 7) * 8;
      *reinterpret_cast<uint4*>(&ks[j][c]) = kreg[i];
      *reinterpret_cast<uint4*>(&vs[j][c]) = vreg[i];
    }
    __syncthreads();
    if (j0 + AM_KT < row_nk) fetch(j0 + AM_KT);
    const int jw = j0 + kofs;                        // first key of this warp's share of the tile
    if (!active || jw >= row_nk) continue;

    // S = Q K^T for 16 queries x KS keys: KS / 8 key groups of 8, 4 steps along the head dimension
    // (the step along the head dimension is the outer loop: consecutive MMAs then go to different accumulators
    // and do not wait for one another)
    float s[KS / 8][4];
#pragma unroll
    for (int nt = 0; nt < KS / 8; ++nt) { s[nt][0] = 0.f; s[nt][1] = 0.f; s[nt][2] = 0.f; s[nt][3] = 0.f; }
#pragma unroll
    for (int s4 = 0; s4 < DH / 16; ++s4) {
      uint32_t kb0[KS / 8], kb1[KS / 8];
#pragma unroll
      for (int nt = 0; nt < KS / 8; ++nt) {
        const bf16* kp = &ks[kofs + nt * 8 + g][s4 * 16 + tq * 2];
        kb0[nt] = *reinterpret_cast<const uint32_t*>(kp);
        kb1[nt] = *reinterpret_cast<const uint32_t*>(kp + 8);
      }
#pragma unroll
      for (int nt = 0; nt < KS / 8; ++nt) mma_bf16_16816(s[nt], qa[s4], kb0[nt], kb1[nt]);
    }
    // mask, scale, online softmax; element e of group nt is key jw + nt * 8 + tq * 2 + (e & 1), query row e >> 1
    float t0 = -INFINITY, t1 = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < KS / 8; ++nt) {
      const int j = jw + nt * 8 + tq * 2;
      s[nt][0] = (j < nk0) ? s[nt][0] * p.scale : -INFINITY;
      s[nt][1] = (j + 1 < nk0) ? s[nt][1] * p.scale : -INFINITY;
      s[nt][2] = (j < nk1) ? s[nt][2] * p.scale : -INFINITY;
      s[nt][3] = (j + 1 < nk1) ? s[nt][3] * p.scale : -INFINITY;
      t0 = fmaxf(t0, fmaxf(s[nt][0], s[nt][1]));
      t1 = fmaxf(t1, fmaxf(s[nt][2], s[nt][3]));
    }
    t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, 1)); t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, 2));
    t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, 1)); t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, 2));
    const bool on0 = nk0 > jw, on1 = nk1 > jw;       // otherwise none of these keys is visible to the query
    const float m0n = on0 ? fmaxf(mx0, t0) : mx0, m1n = on1 ? fmaxf(mx1, t1) : mx1;
    const float corr0 = on0 ? __expf(mx0 - m0n) : 1.f, corr1 = on1 ? __expf(mx1 - m1n) : 1.f;   // exp(-inf) = 0 at first
    mx0 = m0n; mx1 = m1n;
    float sum0 = 0.f, sum1 = 0.f;
    uint32_t pa[KS / 16][4];
#pragma unroll
    for (int nt = 0; nt < KS / 8; ++nt) {
      const float p0 = on0 ? __expf(s[nt][0] - m0n) : 0.f, p1 = on0 ? __expf(s[nt][1] - m0n) : 0.f;
      const float p2 = on1 ? __expf(s[nt][2] - m1n) : 0.f, p3 = on1 ? __expf(s[nt][3] - m1n) : 0.f;
      sum0 += p0 + p1; sum1 += p2 + p3;
      // accumulator fragments of two neighbouring key groups are exactly one A fragment of 16 keys
      pa[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p0, p1);
      pa[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
    }
    den0 = den0 * corr0 + sum0;
    den1 = den1 * corr1 + sum1;
    // O = O * corr + P V
#pragma unroll
    for (int dt = 0; dt < DH / 8; ++dt) { o[dt][0] *= corr0; o[dt][1] *= corr0; o[dt][2] *= corr1; o[dt][3] *= corr1; }
#pragma unroll
    for (int t = 0; t < KS / 16; ++t) {
      uint32_t v0[DH / 8], v1[DH / 8];
#pragma unroll
      for (int dt = 0; dt < DH / 8; ++dt) ldmatrix_x2_trans(v0[dt], v1[dt], &vs[kofs + t * 16 + (lane & 15)][dt * 8]);
#pragma unroll
      for (int dt = 0; dt < DH / 8; ++dt) mma_bf16_16816(o[dt], pa[t], v0[dt], v1[dt]);
    }
  }

  den0 += __shfl_xor_sync(0xffffffffu, den0, 1); den0 += __shfl_xor_sync(0xffffffffu, den0, 2);
  den1 += __shfl_xor_sync(0xffffffffu, den1, 1); den1 += __shfl_xor_sync(0xffffffffu, den1, 2);
  if (NG > 1) {
    // Merge the key groups of a query tile.  Every lane of a group > 0 leaves its fragment (32 outputs, two
    // maxima, two sums) in the tile memory, value-major so that lanes hit different banks; the lane with the
    // same number in group 0 folds them in.
    float* rec = reinterpret_cast<float*>(&kv[0][0][0]);   // [36][128]
    __syncthreads();                                       // all tile reads are done
    if (grp > 0) {
#pragma unroll
      for (int dt = 0; dt < DH / 8; ++dt)
#pragma unroll
        for (int e = 0; e < 4; ++e) rec[(dt * 4 + e) * 128 + tid] = o[dt][e];
      rec[32 * 128 + tid] = mx0; rec[33 * 128 + tid] = mx1;
      rec[34 * 128 + tid] = den0; rec[35 * 128 + tid] = den1;
    }
    __syncthreads();
    if (grp > 0) return;
#pragma unroll
    for (int g2 = 1; g2 < NG; ++g2) {
      const int src = (g2 * QT + qtile) * 32 + lane;       // same query tile, same lane, key group g2
      const float om0 = rec[32 * 128 + src], om1 = rec[33 * 128 + src];
      const float n0 = fmaxf(mx0, om0), n1 = fmaxf(mx1, om1);
      // a row that saw no key at all keeps maximum -inf on both sides: factors 0, nothing to add
      const float a0 = n0 == -INFINITY ? 0.f : __expf(mx0 - n0), b0 = n0 == -INFINITY ? 0.f : __expf(om0 - n0);
      const float a1 = n1 == -INFINITY ? 0.f : __expf(mx1 - n1), b1 = n1 == -INFINITY ? 0.f : __expf(om1 - n1);
      den0 = den0 * a0 + rec[34 * 128 + src] * b0;
      den1 = den1 * a1 + rec[35 * 128 + src] * b1;
#pragma unroll
      for (int dt = 0; dt < DH / 8; ++dt) {
        o[dt][0] = o[dt][0] * a0 + rec[(dt * 4 + 0) * 128 + src] * b0;
        o[dt][1] = o[dt][1] * a0 + rec[(dt * 4 + 1) * 128 + src] * b0;
        o[dt][2] = o[dt][2] * a1 + rec[(dt * 4 + 2) * 128 + src] * b1;
        o[dt][3] = o[dt][3] * a1 + rec[(dt * 4 + 3) * 128 + src] * b1;
      }
      mx0 = n0; mx1 = n1;
    }
  }
  bf16* out = reinterpret_cast<bf16*>(p.out);
  if (r0 < nq && nk0 > 0) {
    const float inv = 1.f / den0;
    bf16* dst = out + (size_t)(m0 + r0) * d + h * DH + tq * 2;
#pragma unroll
    for (int dt = 0; dt < DH / 8; ++dt) *reinterpret_cast<uint32_t*>(dst + dt * 8) = pack_bf16(o[dt][0] * inv, o[dt][1] * inv);
  }
  if (r1 < nq && nk1 > 0) {
    const float inv = 1.f / den1;
    bf16* dst = out + (size_t)(m0 + r1) * d + h * DH + tq * 2;
#pragma unroll
    for (int dt = 0; dt < DH / 8; ++dt) *reinterpret_cast<uint32_t*>(dst + dt * 8) = pack_bf16(o[dt][2] * inv, o[dt][3] * inv);
  }
  trace_mark(TR_ATTN, 2);
}

// ---- rows with hundreds of keys ------------------------------------------------------------------------
// In the kernel above a warp walks all K/V tiles of its row one after the other; with 400 keys that is seven tiles of
// ~570 dependent-latency-bound instructions each, and a warp that is alone on its scheduler issues one instruction
// every 5-6 cycles: 14-15 us per launch however few queries there are.  Here the KEYS are spread over warps instead:
// a CTA holds QT 16-query tiles x NW key warps; warp (qtile, kw) handles the whole tiles kw, kw + NW, ... of the row
// for its 16 queries, and the NW partial results (running maximum, sum, output) of a query tile are merged through
// shared memory at the end.  All tiles of a round (NW tiles, 18 KB each) are copied asynchronously at once.
//
// grid = (B * qchunks, H), qchunks = ceil(longest segment / (16 QT)); block = 32 QT NW threads;
// dynamic shared memory = NW * AM_TILE_BYTES + AM_Q_BYTES.
constexpr int AM_TILE_BYTES = 2 * AM_KT * AM_LD * 2;   // K and V of one 64-key tile: 18 432 bytes
constexpr int AM_Q_BYTES = AM_Q * AM_LD * 2;           // staged queries of a CTA (up to 64)

// 16-byte asynchronous copy global -> shared; src_bytes = 0 writes zeros (the source address must still be valid).
__device__ __forceinline__ void am_cp_async16(void* smem_dst, const void* gmem_src, int src_bytes) {
  const uint32_t s = static_cast<uint32_t>(__cvta_generic_to_shared(smem_dst));
  asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(s), "l"(gmem_src), "r"(src_bytes) : "memory");
}

template <int QT, int NW>
__global__ void __launch_bounds__(32 * QT * NW)
attention_mma_wide_kernel(const AttnParams p) {
  constexpr int DH = 64;
  constexpr int THREADS = 32 * QT * NW;
  constexpr int KS = AM_KT;             // a warp handles whole tiles
  extern __shared__ __align__(16) uint8_t am_smem[];
  typedef bf16 (*TilePtr)[AM_LD];

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
  const int row_nk = p.nkeys_row[b];
  const int i0 = chunk * (16 * QT);
  if (i0 >= seg_len) return;
  const int nq = min(16 * QT, seg_len - i0);
  const int m0 = seg_off + i0;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int g = lane >> 2, tq = lane & 3;           // fragment row (0..7) and column pair (0..3) of this lane
  const int qtile = warp % QT, kw = warp / QT;      // this warp's query tile and key warp
  const bool active = qtile * 16 < nq;              // otherwise the warp only helps loading
  const int d = p.d;
  const bf16* q = reinterpret_cast<const bf16*>(p.q);
  const bf16* kk = reinterpret_cast<const bf16*>(p.k);
  const bf16* vv = reinterpret_cast<const bf16*>(p.v);

  // the first round of tiles does not depend on the queries: request it before they are fetched
  const int n_tiles = (row_nk + AM_KT - 1) / AM_KT;
  auto fetch_round = [&](int first_tile) {
    for (int idx = tid; idx < NW * AM_KT * (DH / 8); idx += THREADS) {
      const int tl = idx / (AM_KT * (DH / 8)), rem = idx - tl * (AM_KT * (DH / 8));
      const int j = rem >> 3, c = (rem & 7) * 8;
      const int key = (first_tile + tl) * AM_KT + j;
      if ((first_tile + tl) < n_tiles) {             // tiles past the end are never read
        const bool there = key < row_nk;             // keys that do not exist are written as zeros
        const size_t off = (size_t)(kbase + (there ? key : 0)) * d + h * DH + c;
        bf16 (*kd)[AM_LD] = reinterpret_cast<TilePtr>(am_smem + tl * AM_TILE_BYTES);
        am_cp_async16(&kd[j][c], kk + off, there ? 16 : 0);
        am_cp_async16(&kd[AM_KT + j][c], vv + off, there ? 16 : 0);
      }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
  };
  fetch_round(0);

  // this lane's two queries (fragment rows g and g + 8 of the warp's 16) and their visible-key counts
  const int r0 = qtile * 16 + g, r1 = r0 + 8;
  int nk0 = 0, nk1 = 0;
  if (r0 < nq) nk0 = p.nkeys_tok ? min(p.nkeys_tok[m0 + r0], row_nk) : row_nk;
  if (r1 < nq) nk1 = p.nkeys_tok ? min(p.nkeys_tok[m0 + r1], row_nk) : row_nk;
  // Queries that come as split-K partial sums of their projection are summed (+ bias) and rounded like stored ones by
  // the whole CTA, every thread issuing all partial loads of its elements at once: one memory round trip.  (Left to
  // the warps, each lane would walk its 16 fragment elements x q_nsplit partials in 16 dependent rounds.)
  bf16 (*qs)[AM_LD] = reinterpret_cast<TilePtr>(am_smem + NW * AM_TILE_BYTES);   // [16 QT][AM_LD]
  if (p.q_part) {
    for (int idx = tid; idx < 16 * QT * (DH / 2); idx += THREADS) {
      const int r = idx / (DH / 2), c2 = (idx - r * (DH / 2)) * 2;
      float2 acc = make_float2(0.f, 0.f);
      if (r < nq) {
        const int c = h * DH + c2;
        if (p.q_bias) acc = *reinterpret_cast<const float2*>(p.q_bias + c);
        const float* src = p.q_part + (size_t)(m0 + r) * d + c;
        float2 part[ATT_MAX_QSPLIT];
#pragma unroll
        for (int sp = 0; sp < ATT_MAX_QSPLIT; ++sp)
          part[sp] = sp < p.q_nsplit ? *reinterpret_cast<const float2*>(src + sp * p.q_stride) : make_float2(0.f, 0.f);
#pragma unroll
        for (int sp = 0; sp < ATT_MAX_QSPLIT; ++sp) { acc.x += part[sp].x; acc.y += part[sp].y; }
      }
      *reinterpret_cast<uint32_t*>(&qs[r][c2]) = pack_bf16(acc.x, acc.y);
    }
  }
  asm volatile("cp.async.wait_group 0;" ::: "memory");
  __syncthreads();                                   // first round of tiles and the staged queries are in place
  trace_mark(TR_ATTN, 3);
  // Q as A fragments of the four 16-wide steps along the head dimension
  uint32_t qa[DH / 16][4];
  if (p.q_part) {
#pragma unroll
    for (int s4 = 0; s4 < DH / 16; ++s4) {
      const int c = s4 * 16 + tq * 2;
      qa[s4][0] = *reinterpret_cast<const uint32_t*>(&qs[r0][c]);
      qa[s4][1] = *reinterpret_cast<const uint32_t*>(&qs[r1][c]);
      qa[s4][2] = *reinterpret_cast<const uint32_t*>(&qs[r0][c + 8]);
      qa[s4][3] = *reinterpret_cast<const uint32_t*>(&qs[r1][c + 8]);
    }
  } else {
#pragma unroll
    for (int s4 = 0; s4 < DH / 16; ++s4) {
      const int c = h * DH + s4 * 16 + tq * 2;
      const bf16* q0 = q + (size_t)(m0 + r0) * d + c;
      const bf16* q1 = q + (size_t)(m0 + r1) * d + c;
      qa[s4][0] = r0 < nq ? *reinterpret_cast<const uint32_t*>(q0) : 0u;
      qa[s4][1] = r1 < nq ? *reinterpret_cast<const uint32_t*>(q1) : 0u;
      qa[s4][2] = r0 < nq ? *reinterpret_cast<const uint32_t*>(q0 + 8) : 0u;
      qa[s4][3] = r1 < nq ? *reinterpret_cast<const uint32_t*>(q1 + 8) : 0u;
    }
  }

  float o[DH / 8][4];
#pragma unroll
  for (int t = 0; t < DH / 8; ++t) { o[t][0] = 0.f; o[t][1] = 0.f; o[t][2] = 0.f; o[t][3] = 0.f; }
  float mx0 = -INFINITY, mx1 = -INFINITY, den0 = 0.f, den1 = 0.f;   // den: this lane's share of the row sums

  for (int first = 0; first < n_tiles; first += NW) {
    if (first > 0) {
      __syncthreads();                               // the previous round is fully consumed
      fetch_round(first);
      asm volatile("cp.async.wait_group 0;" ::: "memory");
      __syncthreads();                               // everybody's copies have landed
    }
    const int t = first + kw;
    if (!active || t >= n_tiles) continue;
    const int jw = t * AM_KT;                        // first key of this warp's tile
    bf16 (*ks)[AM_LD] = reinterpret_cast<TilePtr>(am_smem + kw * AM_TILE_BYTES);
    bf16 (*vs)[AM_LD] = ks + AM_KT;

    // S = Q K^T for 16 queries x 64 keys (the step along the head dimension is the outer loop: consecutive MMAs go
    // to different accumulators and do not wait for one another)
    float s[KS / 8][4];
#pragma unroll
    for (int nt = 0; nt < KS / 8; ++nt) { s[nt][0] = 0.f; s[nt][1] = 0.f; s[nt][2] = 0.f; s[nt][3] = 0.f; }
#pragma unroll
    for (int s4 = 0; s4 < DH / 16; ++s4) {
      uint32_t kb0[KS / 8], kb1[KS / 8];
#pragma unroll
      for (int nt = 0; nt < KS / 8; ++nt) {
        const bf16* kp = &ks[nt * 8 + g][s4 * 16 + tq * 2];
        kb0[nt] = *reinterpret_cast<const uint32_t*>(kp);
        kb1[nt] = *reinterpret_cast<const uint32_t*>(kp + 8);
      }
#pragma unroll
      for (int nt = 0; nt < KS / 8; ++nt) mma_bf16_16816(s[nt], qa[s4], kb0[nt], kb1[nt]);
    }
    // mask, scale, online softmax; element e of group nt is key jw + nt * 8 + tq * 2 + (e & 1), query row e >> 1
    float t0 = -INFINITY, t1 = -INFINITY;
#pragma unroll
    for (int nt = 0; nt < KS / 8; ++nt) {
      const int j = jw + nt * 8 + tq * 2;
      s[nt][0] = (j < nk0) ? s[nt][0] * p.scale : -INFINITY;
      s[nt][1] = (j + 1 < nk0) ? s[nt][1] * p.scale : -INFINITY;
      s[nt][2] = (j < nk1) ? s[nt][2] * p.scale : -INFINITY;
      s[nt][3] = (j + 1 < nk1) ? s[nt][3] * p.scale : -INFINITY;
      t0 = fmaxf(t0, fmaxf(s[nt][0], s[nt][1]));
      t1 = fmaxf(t1, fmaxf(s[nt][2], s[nt][3]));
    }
    t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, 1)); t0 = fmaxf(t0, __shfl_xor_sync(0xffffffffu, t0, 2));
    t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, 1)); t1 = fmaxf(t1, __shfl_xor_sync(0xffffffffu, t1, 2));
    const bool on0 = nk0 > jw, on1 = nk1 > jw;       // otherwise none of these keys is visible to the query
    const float m0n = on0 ? fmaxf(mx0, t0) : mx0, m1n = on1 ? fmaxf(mx1, t1) : mx1;
    const float corr0 = on0 ? __expf(mx0 - m0n) : 1.f, corr1 = on1 ? __expf(mx1 - m1n) : 1.f;   // exp(-inf) = 0 at first
    mx0 = m0n; mx1 = m1n;
    float sum0 = 0.f, sum1 = 0.f;
    uint32_t pa[KS / 16][4];
#pragma unroll
    for (int nt = 0; nt < KS / 8; ++nt) {
      const float p0 = on0 ? __expf(s[nt][0] - m0n) : 0.f, p1 = on0 ? __expf(s[nt][1] - m0n) : 0.f;
      const float p2 = on1 ? __expf(s[nt][2] - m1n) : 0.f, p3 = on1 ? __expf(s[nt][3] - m1n) : 0.f;
      sum0 += p0 + p1; sum1 += p2 + p3;
      pa[nt >> 1][(nt & 1) * 2 + 0] = pack_bf16(p0, p1);
      pa[nt >> 1][(nt & 1) * 2 + 1] = pack_bf16(p2, p3);
    }
    den0 = den0 * corr0 + sum0;
    den1 = den1 * corr1 + sum1;
#pragma unroll
    for (int dt = 0; dt < DH / 8; ++dt) { o[dt][0] *= corr0; o[dt][1] *= corr0; o[dt][2] *= corr1; o[dt][3] *= corr1; }
#pragma unroll
    for (int tt = 0; tt < KS / 16; ++tt) {
      uint32_t v0[DH / 8], v1[DH / 8];
#pragma unroll
      for (int dt = 0; dt < DH / 8; ++dt) ldmatrix_x2_trans(v0[dt], v1[dt], &vs[tt * 16 + (lane & 15)][dt * 8]);
#pragma unroll
      for (int dt = 0; dt < DH / 8; ++dt) mma_bf16_16816(o[dt], pa[tt], v0[dt], v1[dt]);
    }
  }

  den0 += __shfl_xor_sync(0xffffffffu, den0, 1); den0 += __shfl_xor_sync(0xffffffffu, den0, 2);
  den1 += __shfl_xor_sync(0xffffffffu, den1, 1); den1 += __shfl_xor_sync(0xffffffffu, den1, 2);
  // Merge the key warps of a query tile.  Every lane leaves its fragment (32 outputs, two maxima, two sums) in the tile
  // memory, value-major so that lanes hit different banks.  The merge itself is spread over the key warps as well: key
  // warp kw folds the NW records for the output columns 8 dt .. 8 dt + 7 with dt = kw, kw + NW, ... and stores them
  // (folding everything in key warp 0 took longer than the attention itself).  36 * THREADS floats <= NW tiles.
  float* rec = reinterpret_cast<float*>(am_smem);          // [36][THREADS]
  trace_mark(TR_ATTN, 4);
  __syncthreads();                                         // all tile reads are done
#pragma unroll
  for (int dt = 0; dt < DH / 8; ++dt)
#pragma unroll
    for (int e = 0; e < 4; ++e) rec[(dt * 4 + e) * THREADS + tid] = o[dt][e];
  rec[32 * THREADS + tid] = mx0; rec[33 * THREADS + tid] = mx1;
  rec[34 * THREADS + tid] = den0; rec[35 * THREADS + tid] = den1;
  __syncthreads();
  trace_mark(TR_ATTN, 5);
  if (!active) return;
  float n0 = -INFINITY, n1 = -INFINITY;
#pragma unroll
  for (int g2 = 0; g2 < NW; ++g2) {
    const int src = (g2 * QT + qtile) * 32 + lane;         // same query tile, same lane, key warp g2
    n0 = fmaxf(n0, rec[32 * THREADS + src]);
    n1 = fmaxf(n1, rec[33 * THREADS + src]);
  }
  float f0[NW], f1[NW], dsum0 = 0.f, dsum1 = 0.f;
#pragma unroll
  for (int g2 = 0; g2 < NW; ++g2) {
    const int src = (g2 * QT + qtile) * 32 + lane;
    // a key warp that saw no visible key keeps maximum -inf: factor 0 (also when no warp saw any)
    const float om0 = rec[32 * THREADS + src], om1 = rec[33 * THREADS + src];
    f0[g2] = om0 == -INFINITY ? 0.f : __expf(om0 - n0);
    f1[g2] = om1 == -INFINITY ? 0.f : __expf(om1 - n1);
    dsum0 += rec[34 * THREADS + src] * f0[g2];
    dsum1 += rec[35 * THREADS + src] * f1[g2];
  }
  bf16* out = reinterpret_cast<bf16*>(p.out);
  const float inv0 = 1.f / dsum0, inv1 = 1.f / dsum1;
  for (int dt = kw; dt < DH / 8; dt += NW) {
    float a0 = 0.f, a1 = 0.f, a2 = 0.f, a3 = 0.f;
#pragma unroll
    for (int g2 = 0; g2 < NW; ++g2) {
      const int src = (g2 * QT + qtile) * 32 + lane;
      a0 += rec[(dt * 4 + 0) * THREADS + src] * f0[g2];
      a1 += rec[(dt * 4 + 1) * THREADS + src] * f0[g2];
      a2 += rec[(dt * 4 + 2) * THREADS + src] * f1[g2];
      a3 += rec[(dt * 4 + 3) * THREADS + src] * f1[g2];
    }
    if (r0 < nq && nk0 > 0)
      *reinterpret_cast<uint32_t*>(out + (size_t)(m0 + r0) * d + h * DH + tq * 2 + dt * 8) = pack_bf16(a0 * inv0, a1 * inv0);
    if (r1 < nq && nk1 > 0)
      *reinterpret_cast<uint32_t*>(out + (size_t)(m0 + r1) * d + h * DH + tq * 2 + dt * 8) = pack_bf16(a2 * inv1, a3 * inv1);
  }
  trace_mark(TR_ATTN, 2);
}


}  // namespace ad
