// The small kernels around the GEMMs and attention: block planning (which tokens are fed at which
// positions), embedding, LayerNorm, the arg-max reduction with the draft compare / first-mismatch decision,
// the commit (cache-length advance / rollback), the input-guided draft policy of Algorithm 1, and the
// planning of the drafter and encoder passes.
#pragma once

#include <cuda_device_runtime_api.h>

#include "ad_common.cuh"

namespace ad {

// Per-row decoding state and per-call block buffers, all resident in the workspace.
struct DevState {
  int* len;        // [B] accepted-prefix length = cached positions
  int* last;       // [B] last accepted token ([BOS] at the start)
  int* fin;        // [B] 1 once [EOS] was accepted or the row's cap was reached
  int* maxlen;     // [B] per-row output cap
  int* srclen;     // [B]
  int* src;        // [B, max_src]
  int* out_ids;    // [B, max_tgt]
  int* drafts;     // [B, kmax]
  int* pred;       // [B, kmax] greedy choices of the last verification
  int* n_acc;      // [B] accepted count of the last verification (0 = nothing to commit)
  int* stat_it;    // [B] iterations the row took part in
  int* stat_acc;   // [B] tokens accepted
  int* stat_off;   // [B] block sizes offered
  int* loop_it;    // [1] iterations with at least one active row
  int* status;     // [1] latched device error
  int* all_fin;    // [1] 1 when every row is finished
  int* cross_base; // [B] = b * max_src
  int* gidx;       // [B * kmax] drafter: packed token holding mask position i of row b
  int* enc_slot;   // [B * max_src] encoder: cross-K/V slot of packed source token m
  int* user_k;     // [B] staging of caller-provided k / n
  int* user_n;     // [B]
  int* user_drafts;// [B, kmax]
  unsigned int* sync_ctr;  // [128 x 32] per-stage arrival counters of the persistent decoder pass (one per 128-byte line);
                           // every planning kernel that precedes such a pass clears them
};

enum DraftSource : int {
  SRC_USER = 0,      // drafts and k come from the caller (ad_verify_block)
  SRC_OVERRIDE = 1,  // k = min(cap, remaining); drafts = position-aligned stream
  SRC_POLICY = 2,    // Algorithm 1: suffix match on the source
  SRC_SIZES = 3,     // k = min(cap, remaining); drafts left untouched (the drafter fills them)
  SRC_KEEP = 4       // k and drafts as they are (after the drafter); optional override on top
};

struct Dims {
  int B, max_src, max_tgt, kmax;
  int bos, pad, eos, mask;
  int vocab;
};

// Token ids that reach an embedding lookup come from the caller (source, drafts, override stream, forced tokens).
// An id outside [0, vocab) is never used as an index: it is replaced and AD_ERR_ARG is latched.
__device__ __forceinline__ bool id_in_vocab(int id, const Dims& dm) { return id >= 0 && id < dm.vocab; }

// ---------------------------------------------------------------------------------------------
// Suffix match of Algorithm 1, line 3, for one row, executed by one warp.
// o_0 = [BOS], o_t = out[t-1]; x_0 = [BOS], x_t = src[t-1], t <= n.  For q = 0, 1, ... counts the end
// positions i with o[j-q..j] == x[i-q..i]; a unique one is the match, none means no match, several means
// a longer suffix is tried.  Returns i or -1 (same value in every lane).
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ int tok_o(const int* out, int t, int bos) { return t == 0 ? bos : out[t - 1]; }

__device__ int warp_suffix_match(const int* out, int j, const int* src, int n, int bos, int lane) {
  for (int q = 0; q <= j; ++q) {
    int count = 0, where = -1;
    for (int i0 = q; i0 <= n; i0 += 32) {
      const int i = i0 + lane;
      bool ok = i <= n;
      for (int t = 0; ok && t <= q; ++t) ok = tok_o(out, j - t, bos) == tok_o(src, i - t, bos);
      const unsigned bal = __ballot_sync(0xffffffffu, ok);
      if (bal) { count += __popc(bal); where = i0 + 31 - __clz(bal); }
    }
    if (count == 1) return where;
    if (count == 0) return -1;
  }
  return -1;
}

// ---------------------------------------------------------------------------------------------
// Chooses every row's block (size and drafted tokens) and lays the block tokens out as packed rows.
// Decoder inputs of row b are (last accepted token, drafts[0..k-2]) at positions len .. len+k-1
// (Eq. 6 / Eq. 7); a negative draft that would be fed is replaced by [PAD].
// Executed by ALL threads of one CTA (any multiple of 32 threads); s_k / s_off: shared arrays of 256 / 257 ints.
// The per-row state is read past L1: the caller may be the last CTA of the accept kernel, reading what the other
// CTAs of that kernel have just committed.
// ---------------------------------------------------------------------------------------------
struct NextBlock {
  int source;                  // DraftSource
  int k_cap;
  const int* override_stream;
  int override_stride, override_len;
};

__device__ __forceinline__ void plan_verify_block(const DevState& st, const PassPlan& plan, const Dims& dm, const NextBlock& nb,
                                                  int* s_k, int* s_off) {
  const int tid = threadIdx.x, nthreads = blockDim.x, warp = tid >> 5, lane = tid & 31, nwarps = nthreads >> 5;
  const int B = dm.B, source = nb.source, k_cap = nb.k_cap;
  const int* override_stream = nb.override_stream;
  const int override_stride = nb.override_stride, override_len = nb.override_len;

  if (source == SRC_POLICY) {
    for (int b = warp; b < B; b += nwarps) {
      int k = 0;
      const int len = __ldcg(st.len + b);
      if (!__ldcg(st.fin + b) && len < st.maxlen[b]) {
        const int n = st.srclen[b];
        const int* src = st.src + (size_t)b * dm.max_src;
        const int i = warp_suffix_match(st.out_ids + (size_t)b * dm.max_tgt, len, src, n, dm.bos, lane);
        int* dr = st.drafts + (size_t)b * dm.kmax;
        if (i >= 0) {
          // draft = x_{i+1..n} followed by the [PAD] slot that matches nothing
          k = n - i + 1;
          k = min(k, min(k_cap, st.maxlen[b] - len));
          for (int t = lane; t < k; t += 32) dr[t] = (i + 1 + t <= n) ? src[i + t] : -1;
        } else {
          k = 1;
          if (lane == 0) dr[0] = -1;
        }
      }
      if (lane == 0) s_k[b] = k;
    }
  } else {
    for (int b = tid; b < B; b += nthreads) {
      int k;
      const int len = __ldcg(st.len + b);
      if (source == SRC_USER) {
        k = st.user_k[b];
        if (k < 0 || k > dm.kmax || len + k > dm.max_tgt) { latch_error(st.status, AD_ERR_ARG); k = 0; }
      } else if (source == SRC_KEEP) {
        k = plan.seg_len[b];
      } else {
        k = (__ldcg(st.fin + b) || len >= st.maxlen[b]) ? 0 : min(k_cap, st.maxlen[b] - len);
      }
      s_k[b] = k;
    }
  }
  __syncthreads();
  if (tid == 0) {
    int acc = 0;
    for (int b = 0; b < B; ++b) { s_off[b] = acc; acc += s_k[b]; }
    s_off[B] = acc;
    *plan.M = acc;
    st.loop_it[1] = 0;   // rows-done counter of the accept kernel: every iteration starts from zero
  }
  if (tid < 128) st.sync_ctr[tid * 32] = 0u;
  __syncthreads();
  for (int b = warp; b < B; b += nwarps) {
    const int k = s_k[b], off = s_off[b], len = __ldcg(st.len + b);
    int* dr = st.drafts + (size_t)b * dm.kmax;
    if (lane == 0) {
      plan.seg_off[b] = off;
      plan.seg_len[b] = k;
      plan.key_base[b] = b * dm.max_tgt;
      plan.row_nk[b] = len + k;
    }
    for (int i = lane; i < k; i += 32) {
      if (source == SRC_USER) dr[i] = st.user_drafts[(size_t)b * dm.kmax + i];
      if (override_stream && (source == SRC_OVERRIDE || source == SRC_KEEP))
        dr[i] = (len + i < override_len) ? override_stream[(size_t)b * override_stride + len + i] : -1;
      // a caller-provided draft beyond the vocabulary becomes a slot that matches nothing (negative = sentinel is legal)
      if (dr[i] >= dm.vocab) { latch_error(st.status, AD_ERR_ARG); dr[i] = -1; }
    }
    __syncwarp();
    for (int i = lane; i < k; i += 32) {
      const int m = off + i;
      int tok = (i == 0) ? __ldcg(st.last + b) : dr[i - 1];
      if (tok < 0 || tok >= dm.vocab) tok = dm.pad;
      plan.tok_row[m] = b;
      plan.tok_pos[m] = len + i;
      plan.tok_id[m] = tok;
      plan.kv_slot[m] = b * dm.max_tgt + len + i;
      plan.att_n[m] = len + i + 1;
    }
  }
}

// grid = 1, block = 256.
__global__ void __launch_bounds__(256)
prepare_verify_kernel(DevState st, PassPlan plan, Dims dm, int source, int k_cap, const int* override_stream,
                      int override_stride, int override_len) {
  trace_mark(TR_PREPARE, 0);
  pdl_launch();
  pdl_wait();
  trace_mark(TR_PREPARE, 1);
  __shared__ int s_k[256];
  __shared__ int s_off[257];
  NextBlock nb;
  nb.source = source; nb.k_cap = k_cap; nb.override_stream = override_stream;
  nb.override_stride = override_stride; nb.override_len = override_len;
  plan_verify_block(st, plan, dm, nb, s_k, s_off);
}

// ---------------------------------------------------------------------------------------------
// Drafter pass (Section 3.2.1): row b feeds ([BOS], accepted tokens, k x [MASK]) at positions 0 .. len+k
// with no cache and unmasked attention.  blk is the verification plan holding k per row.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
plan_draft_kernel(DevState st, PassPlan blk, PassPlan plan, Dims dm) {
  pdl_launch();
  pdl_wait();
  __shared__ int s_off[257];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int B = dm.B;
  if (tid == 0) {
    int acc = 0;
    for (int b = 0; b < B; ++b) {
      s_off[b] = acc;
      const int k = blk.seg_len[b];
      acc += k > 0 ? st.len[b] + 1 + k : 0;
    }
    s_off[B] = acc;
    *plan.M = acc;
  }
  if (tid < 128) st.sync_ctr[tid * 32] = 0u;
  __syncthreads();
  for (int b = warp; b < B; b += 8) {
    const int k = blk.seg_len[b], len = st.len[b], off = s_off[b];
    const int n = k > 0 ? len + 1 + k : 0;
    if (lane == 0) { plan.seg_off[b] = off; plan.seg_len[b] = n; plan.key_base[b] = off; plan.row_nk[b] = n; }
    for (int i = lane; i < n; i += 32) {
      const int m = off + i;
      plan.tok_row[m] = b;
      plan.tok_pos[m] = i;
      plan.tok_id[m] = (i == 0) ? dm.bos : (i <= len ? st.out_ids[(size_t)b * dm.max_tgt + i - 1] : dm.mask);
      plan.kv_slot[m] = m;
      plan.att_n[m] = n;
    }
    for (int i = lane; i < k; i += 32) st.gidx[blk.seg_off[b] + i] = off + len + 1 + i;
  }
}

// ---------------------------------------------------------------------------------------------
// Encoder pass: row b feeds its src_len[b] source tokens (padding is simply not packed, and the per-row
// key counts keep it out of every attention).  Also resets the decoding state of every row.
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
plan_encode_kernel(DevState st, PassPlan plan, Dims dm) {
  pdl_launch();
  pdl_wait();
  __shared__ int s_off[257];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int B = dm.B;
  // a device-resident src_len is checked here (the host cannot see it): out-of-range lengths are clamped
  for (int b = tid; b < B; b += 256) {
    const int n = st.srclen[b];
    if (n < 1 || n > dm.max_src) { latch_error(st.status, AD_ERR_ARG); st.srclen[b] = max(1, min(n, dm.max_src)); }
  }
  __syncthreads();
  if (tid == 0) {
    int acc = 0;
    for (int b = 0; b < B; ++b) { s_off[b] = acc; acc += st.srclen[b]; }
    *plan.M = acc;
    *st.loop_it = 0;
    st.loop_it[2] = 0;
    *st.all_fin = 0;
  }
  for (int b = tid; b < B; b += 256) {
    st.len[b] = 0; st.last[b] = dm.bos; st.fin[b] = 0; st.n_acc[b] = 0; st.maxlen[b] = dm.max_tgt;
    st.stat_it[b] = 0; st.stat_acc[b] = 0; st.stat_off[b] = 0;
    st.cross_base[b] = b * dm.max_src;
  }
  __syncthreads();
  for (int b = warp; b < B; b += 8) {
    const int n = st.srclen[b], off = s_off[b];
    if (lane == 0) { plan.seg_off[b] = off; plan.seg_len[b] = n; plan.key_base[b] = off; plan.row_nk[b] = n; }
    for (int i = lane; i < n; i += 32) {
      const int m = off + i;
      plan.tok_row[m] = b;
      plan.tok_pos[m] = i;
      int id = st.src[(size_t)b * dm.max_src + i];
      if (!id_in_vocab(id, dm)) { latch_error(st.status, AD_ERR_ARG); id = dm.pad; st.src[(size_t)b * dm.max_src + i] = id; }
      plan.tok_id[m] = id;
      plan.kv_slot[m] = m;
      plan.att_n[m] = n;
      st.enc_slot[m] = b * dm.max_src + i;
    }
  }
}

__global__ void set_maxlen_kernel(DevState st, Dims dm, const int* maxlen) {
  pdl_launch();
  pdl_wait();
  const int b = blockIdx.x * blockDim.x + threadIdx.x;
  if (b < dm.B) {
    int v = maxlen[b];
    if (v < 1 || v > dm.max_tgt) { latch_error(st.status, AD_ERR_ARG); v = max(1, min(v, dm.max_tgt)); }
    st.maxlen[b] = v;
  }
}

// ---------------------------------------------------------------------------------------------
// y = emb[token] * sqrt(d) + PE[pos]  ->  FP32 residual stream and the GEMM-operand copy.
// grid = M_cap, block = 128.
// ---------------------------------------------------------------------------------------------
template <typename WT, typename ActT>
__global__ void __launch_bounds__(128)
embed_kernel(PassPlan plan, const WT* __restrict__ emb, const float* __restrict__ pe, int d, float scale,
             float* __restrict__ y, ActT* __restrict__ yb) {
  trace_mark(TR_EMBED, 0);
  pdl_launch();
  pdl_wait();
  trace_mark(TR_EMBED, 1);
  const int m = blockIdx.x;
  if (m >= *plan.M) return;
  const int id = plan.tok_id[m], pos = plan.tok_pos[m];
  for (int i = threadIdx.x; i < d; i += blockDim.x) {
    const float v = to_f32(emb[(size_t)id * d + i]) * scale + pe[(size_t)pos * d + i];
    y[(size_t)m * d + i] = v;
    yb[(size_t)m * d + i] = from_f32<ActT>(v);
  }
}

// ---------------------------------------------------------------------------------------------
// Residual + LayerNorm:  x = sum_s pre[s][m, :] + bias + resid[m, :];  y = LN(x) (biased variance).
// pre holds the split-K partial sums of the preceding projection (nsplit <= 16 of them, split_stride floats
// apart).  One CTA per packed token; each thread owns up to two groups of four consecutive features and issues
// all of its loads (partials, residual) at once, so the kernel costs one global-memory round trip.
// y may alias resid.  d % 4 == 0, d <= 1024.  grid = M_cap, block = THREADS (128, or 256 for d > 512).
// ---------------------------------------------------------------------------------------------
template <int THREADS>
__device__ __forceinline__ float block_sum(float v, float* red) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) v += __shfl_xor_sync(0xffffffffu, v, off);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  __syncthreads();                 // red may still be read from a previous call
  if (lane == 0) red[warp] = v;
  __syncthreads();
  float t = 0.f;
#pragma unroll
  for (int w = 0; w < THREADS / 32; ++w) t += red[w];
  return t;
}
__device__ __forceinline__ float block_sum_128(float v, float* red) { return block_sum<128>(v, red); }

__device__ __forceinline__ void store4(float* p, float4 v) { *reinterpret_cast<float4*>(p) = v; }
__device__ __forceinline__ void store4(bf16* p, float4 v) {
  __nv_bfloat162 a = __floats2bfloat162_rn(v.x, v.y), b = __floats2bfloat162_rn(v.z, v.w);
  uint2 u;
  u.x = *reinterpret_cast<unsigned int*>(&a);
  u.y = *reinterpret_cast<unsigned int*>(&b);
  *reinterpret_cast<uint2*>(p) = u;
}

// THREADS = 128 for d <= 512 and 256 beyond: one 4-element group per thread, so that all partial sums of a thread are
// requested at once (with two groups per thread the second group's loads waited for the first group's sums: 2.8 us
// instead of 1.5 us per launch on a 1024-wide model with 16 partials).
template <typename ActT, int THREADS = 128>
__global__ void __launch_bounds__(THREADS)
layernorm_kernel(const int* __restrict__ M_ptr, const float* __restrict__ pre, int nsplit, size_t split_stride,
                 const float* __restrict__ bias, const float* resid, const float* __restrict__ g,
                 const float* __restrict__ bta, int d, float eps, float* y, ActT* __restrict__ yb) {
  __shared__ float red[THREADS / 32];
  constexpr int NG = 256 / THREADS;            // groups per thread: d <= 1024
  trace_mark(TR_LN, 0);
  pdl_launch();
  const int groups = d >> 2;
  const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
  // gains and biases are weights: fetch them while the previous kernel is still running
  float4 gv[NG], bv[NG], cb[NG];
#pragma unroll
  for (int i = 0; i < NG; ++i) {
    const int gi = threadIdx.x + THREADS * i;
    const bool on = gi < groups;
    gv[i] = on ? reinterpret_cast<const float4*>(g)[gi] : zero4;
    bv[i] = on ? reinterpret_cast<const float4*>(bta)[gi] : zero4;
    cb[i] = (on && bias) ? reinterpret_cast<const float4*>(bias)[gi] : zero4;
  }
  pdl_wait();
  trace_mark(TR_LN, 1);
  const int m = blockIdx.x;
  if (m >= *M_ptr) return;
  float4 xv[NG];
  float s = 0.f;
#pragma unroll
  for (int i = 0; i < NG; ++i) {
    const int gi = threadIdx.x + THREADS * i;
    float4 v = zero4;
    if (gi < groups) {
      const size_t off = (size_t)m * groups + gi;
      float4 part[16];
#pragma unroll
      for (int sp = 0; sp < 16; ++sp)
        part[sp] = (sp < nsplit) ? reinterpret_cast<const float4*>(pre + sp * split_stride)[off] : zero4;
      const float4 r = resid ? reinterpret_cast<const float4*>(resid)[off] : zero4;
      v = make_float4(cb[i].x + r.x, cb[i].y + r.y, cb[i].z + r.z, cb[i].w + r.w);
#pragma unroll
      for (int sp = 0; sp < 16; ++sp) { v.x += part[sp].x; v.y += part[sp].y; v.z += part[sp].z; v.w += part[sp].w; }
    }
    xv[i] = v;
    s += v.x + v.y + v.z + v.w;
  }
  const float mean = block_sum<THREADS>(s, red) / (float)d;
  float vs = 0.f;
#pragma unroll
  for (int i = 0; i < NG; ++i) {
    if (threadIdx.x + THREADS * i < groups) {
      const float a = xv[i].x - mean, b = xv[i].y - mean, c = xv[i].z - mean, e = xv[i].w - mean;
      vs += a * a + b * b + c * c + e * e;
    }
  }
  const float inv = rsqrtf(block_sum<THREADS>(vs, red) / (float)d + eps);
#pragma unroll
  for (int i = 0; i < NG; ++i) {
    const int gi = threadIdx.x + THREADS * i;
    if (gi < groups) {
      float4 o;
      o.x = gv[i].x * ((xv[i].x - mean) * inv) + bv[i].x;
      o.y = gv[i].y * ((xv[i].y - mean) * inv) + bv[i].y;
      o.z = gv[i].z * ((xv[i].z - mean) * inv) + bv[i].z;
      o.w = gv[i].w * ((xv[i].w - mean) * inv) + bv[i].w;
      const size_t off = ((size_t)m * groups + gi) * 4;
      store4(y + off, o);
      store4(yb + off, o);
    }
  }
  trace_mark(TR_LN, 2);
}

// The same operation for large token counts: one warp per token (no block-wide barrier), 8 tokens per CTA.
// The loads of two element groups (residual and up to four partial sums each: ten 16-byte loads per lane) are issued
// before their first use.  nsplit <= 4 here (more partials take the one-CTA-per-token kernel).
// grid = ceil(M_cap / 8), block = 256, d <= 1024 and a multiple of 128.
template <typename ActT>
__global__ void __launch_bounds__(256, 2)
layernorm_rows_kernel(const int* __restrict__ M_ptr, const float* __restrict__ pre, int nsplit, size_t split_stride,
                      const float* __restrict__ bias, const float* resid, const float* __restrict__ g,
                      const float* __restrict__ bta, int d, float eps, float* y, ActT* __restrict__ yb) {
  trace_mark(TR_LN, 0);
  pdl_launch();
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int per = d >> 7;                               // float4 groups per lane (d / 128), <= 8
  const float4 zero4 = make_float4(0.f, 0.f, 0.f, 0.f);
  pdl_wait();
  trace_mark(TR_LN, 1);
  const int m = blockIdx.x * 8 + warp;
  if (m < *M_ptr) {
    const size_t row = (size_t)m * (d >> 2);
    float4 xv[8];
    float s = 0.f;
#pragma unroll
    for (int pair = 0; pair < 4; ++pair) {
      if (pair * 2 >= per) break;
      float4 r4[2], c4[2], q4[2][4];
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int gi = pair * 2 + i;
        const size_t off = row + lane + 32 * gi;
        r4[i] = (gi < per && resid) ? reinterpret_cast<const float4*>(resid)[off] : zero4;
        c4[i] = (gi < per && bias) ? reinterpret_cast<const float4*>(bias)[lane + 32 * gi] : zero4;
#pragma unroll
        for (int sp = 0; sp < 4; ++sp)
          q4[i][sp] = (gi < per && sp < nsplit) ? reinterpret_cast<const float4*>(pre + sp * split_stride)[off] : zero4;
      }
#pragma unroll
      for (int i = 0; i < 2; ++i) {
        const int gi = pair * 2 + i;
        float4 v = r4[i];
        v.x += c4[i].x; v.y += c4[i].y; v.z += c4[i].z; v.w += c4[i].w;
#pragma unroll
        for (int sp = 0; sp < 4; ++sp) { v.x += q4[i][sp].x; v.y += q4[i][sp].y; v.z += q4[i][sp].z; v.w += q4[i][sp].w; }
        xv[gi] = v;
        s += v.x + v.y + v.z + v.w;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
    const float mean = s / (float)d;
    float vs = 0.f;
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (i < per) {
        const float a = xv[i].x - mean, b = xv[i].y - mean, c = xv[i].z - mean, e = xv[i].w - mean;
        vs += a * a + b * b + c * c + e * e;
      }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) vs += __shfl_xor_sync(0xffffffffu, vs, o);
    const float inv = rsqrtf(vs / (float)d + eps);
#pragma unroll
    for (int i = 0; i < 8; ++i) {
      if (i < per) {
        const float4 gv = reinterpret_cast<const float4*>(g)[lane + 32 * i];
        const float4 bv = reinterpret_cast<const float4*>(bta)[lane + 32 * i];
        float4 o;
        o.x = gv.x * ((xv[i].x - mean) * inv) + bv.x;
        o.y = gv.y * ((xv[i].y - mean) * inv) + bv.y;
        o.z = gv.z * ((xv[i].z - mean) * inv) + bv.z;
        o.w = gv.w * ((xv[i].w - mean) * inv) + bv.w;
        const size_t off = (row + lane + 32 * i) * 4;
        store4(y + off, o);
        store4(yb + off, o);
      }
    }
  }
  trace_mark(TR_LN, 2);
}

// dst[j, :] = src[gidx[j], :] for j < *M_ptr.  grid = M_cap, block = 128.
template <typename ActT>
__global__ void __launch_bounds__(128)
gather_rows_kernel(const int* __restrict__ M_ptr, const int* __restrict__ gidx, const ActT* __restrict__ src,
                   ActT* __restrict__ dst, int d) {
  pdl_launch();
  pdl_wait();
  const int j = blockIdx.x;
  if (j >= *M_ptr) return;
  const int s = gidx[j];
  for (int i = threadIdx.x; i < d; i += blockDim.x) dst[(size_t)j * d + i] = src[(size_t)s * d + i];
}

// ---------------------------------------------------------------------------------------------
// Commit of one row (Algorithm 1 lines 6-7): n > 0 appends pred[0..n) to the row's output, advances the cache
// length, sets the last token and the finished flag; n < 0 rolls |n| committed tokens back; n = 0 discards
// the block.  Executed by one warp.
// ---------------------------------------------------------------------------------------------
__device__ __forceinline__ void commit_row(const DevState& st, const PassPlan& blk, const Dims& dm, int b, int n,
                                           int nacc, int lane) {
  int len = st.len[b];
  if (n > nacc || (n < 0 && -n > len)) {
    if (lane == 0) latch_error(st.status, AD_ERR_ARG);
    n = 0;
  }
  __syncwarp();
  if (n > 0) {
    const int* pred = st.pred + (size_t)b * dm.kmax;
    int* out = st.out_ids + (size_t)b * dm.max_tgt;
    for (int i = lane; i < n; i += 32) out[len + i] = pred[i];
    if (lane == 0) {
      const int last = pred[n - 1];
      len += n;
      st.len[b] = len;
      st.last[b] = last;
      if (last == dm.eos || len >= st.maxlen[b]) st.fin[b] = 1;
      st.stat_acc[b] += n;
    }
  } else if (n < 0 && lane == 0) {
    len += n;
    st.len[b] = len;
    st.last[b] = len > 0 ? st.out_ids[(size_t)b * dm.max_tgt + len - 1] : dm.bos;
    st.fin[b] = 0;
  }
  if (lane == 0) {
    if (nacc > 0) {
      st.stat_it[b] += 1;
      st.stat_off[b] += blk.seg_len[b];
    }
    st.n_acc[b] = 0;
  }
}

// After every row has been committed: loop counter and the "all rows finished" word.  One thread.
// cond != 0: the iteration runs inside a device-side `while` graph node; the node repeats while its condition
// is non-zero, so it is cleared when every row has finished -- or, as a bound that does not depend on the data,
// when the iteration counter st.loop_it[2] reaches the limit st.loop_it[3] the host stored before the launch.
__device__ __forceinline__ void finish_iteration(const DevState& st, const Dims& dm, bool any_active,
                                                 unsigned long long cond) {
  int all = 1;
  for (int b = 0; b < dm.B; ++b) all &= (__ldcg(st.fin + b) != 0);
  if (any_active) *st.loop_it += 1;
  *st.all_fin = all;
  if (cond) {
    const int it = st.loop_it[2] + 1;
    st.loop_it[2] = it;
    cudaGraphSetConditional(cond, (all || it >= st.loop_it[3]) ? 0u : 1u);
  }
}

// ---------------------------------------------------------------------------------------------
// Relaxed verification (Section 3.2.3): score of every block position's drafted token,
// draft_val[m] = x[m, :] . emb[draft, :], and its id (negative: sentinel, never kept).  The projection kernel
// then counts, per position, the other tokens that score strictly higher (Eq. 8), and the accept kernel applies
// Eq. 8 and Eq. 9.  One warp per packed token; grid = ceil(M_cap / 8), block = 256.
// ---------------------------------------------------------------------------------------------
template <typename WT, typename ActT>
__global__ void __launch_bounds__(256)
draft_score_kernel(DevState st, PassPlan blk, Dims dm, const WT* __restrict__ emb, const ActT* __restrict__ x, int d,
                   float* __restrict__ draft_val, int* __restrict__ draft_id) {
  pdl_launch();
  pdl_wait();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int m = blockIdx.x * 8 + warp;
  if (m >= *blk.M) return;
  const int b = blk.tok_row[m];
  int id = st.drafts[(size_t)b * dm.kmax + (m - blk.seg_off[b])];
  if (id >= dm.vocab) id = -1;
  float acc = 0.f;
  if (id >= 0)
    for (int i = lane; i < d; i += 32) acc = fmaf(to_f32(x[(size_t)m * d + i]), to_f32(emb[(size_t)id * d + i]), acc);
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
  if (lane == 0) { draft_val[m] = acc; draft_id[m] = id; }
}

// ---------------------------------------------------------------------------------------------
// Final arg-max over the per-tile partials of the fused projection, then the draft compare:
//   c = first block position whose greedy choice differs from the draft (Section 3.1.1; definition of c
//   in Section 3.2), n = c + 1 (the bifurcation token is kept), n = k when nothing differs, cut at the
//   first accepted [EOS].  One CTA per row, one warp per block position for the reduction; warp 0 takes the
//   decision with ballots.
// beta >= 1: relaxed verification of Section 3.2.3 -- a position keeps its drafted token when fewer than beta other
//   tokens score strictly higher (Eq. 8: the draft is within the top beta) and the best score exceeds the draft's
//   by at most tau (Eq. 9; differences of log-likelihoods are differences of scores); otherwise the greedy choice.
// to_drafts != 0: drafter mode, the choices are written as the row's drafts and nothing is compared.
// auto_commit != 0: the row's n_accepted is committed right away (decode loop); the last CTA to finish
//   updates the loop counter and the all-finished word (done_ctr: rows done in the low half, active rows in
//   the high half; left at zero).
// next.source >= 0 (decode loop, small blocks): the LAST CTA to finish also chooses the next iteration's blocks
//   (plan_verify_block) and embeds their tokens (y = emb[token] * sqrt(d) + PE[pos]), so that the next iteration starts
//   at its first projection: two launches fewer per iteration.
// grid = B, block = 1024.
// ---------------------------------------------------------------------------------------------
struct NextEmbed {
  const void* emb;       // embedding matrix in the weight type
  const float* pe;
  int d;
  float scale;
  float* y;
  void* yb;              // GEMM-operand copy in the activation type
};

template <typename WT>
__global__ void __launch_bounds__(1024)
argmax_accept_kernel(DevState st, PassPlan blk, Dims dm, const float* __restrict__ part_val,
                     const int* __restrict__ part_idx, int n_tiles, int M_cap, int to_drafts, int auto_commit,
                     unsigned int* done_ctr, unsigned long long cond, int beta, float tau,
                     const float* __restrict__ draft_val, const int* __restrict__ draft_id,
                     const int* __restrict__ part_cnt, NextBlock next, NextEmbed ne) {
  __shared__ int s_k[256];
  __shared__ int s_off[257];
  __shared__ int s_last;
  trace_mark(TR_ACCEPT, 0);
  pdl_launch();
  pdl_wait();
  trace_mark(TR_ACCEPT, 1);
  const int b = blockIdx.x;
  const int k = blk.seg_len[b];
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  int* pred = (to_drafts ? st.drafts : st.pred) + (size_t)b * dm.kmax;
  if (k > 0) {
    const int off = blk.seg_off[b];
    for (int i = warp; i < k; i += 32) {
      const int m = off + i;
      float v = -INFINITY;
      int idx = 0x7fffffff;
      int higher = 0;
      const bool relaxed = beta >= 1 && !to_drafts;
      for (int t = lane; t < n_tiles; t += 32) {
        const float ov = part_val[(size_t)m * n_tiles + t];
        const int oi = part_idx[(size_t)m * n_tiles + t];
        if (ov > v || (ov == v && oi < idx)) { v = ov; idx = oi; }
        if (relaxed) higher += part_cnt[(size_t)m * n_tiles + t];
      }
#pragma unroll
      for (int o = 16; o > 0; o >>= 1) {
        const float ov = __shfl_xor_sync(0xffffffffu, v, o);
        const int oi = __shfl_xor_sync(0xffffffffu, idx, o);
        if (ov > v || (ov == v && oi < idx)) { v = ov; idx = oi; }
        higher += __shfl_xor_sync(0xffffffffu, higher, o);
      }
      if (lane == 0) {
        int choice = idx;
        if (relaxed) {
          const int did = draft_id[m];
          if (did >= 0 && higher <= beta - 1 && v - draft_val[m] <= tau) choice = did;
        }
        pred[i] = choice;
      }
    }
  }
  if (to_drafts) return;
  if (tid == 0) s_last = 0;
  __syncthreads();
  if (warp == 0) {
    int n = 0;
    if (k > 0) {
      const int* dr = st.drafts + (size_t)b * dm.kmax;
      n = k;
      bool found = false;
      for (int i0 = 0; i0 < k && !found; i0 += 32) {
        const int i = i0 + lane;
        const bool mism = (i < k) && (dr[i] < 0 || pred[i] != dr[i]);
        const unsigned bal = __ballot_sync(0xffffffffu, mism);
        if (bal) { n = i0 + __ffs(bal); found = true; }
      }
      found = false;
      for (int i0 = 0; i0 < n && !found; i0 += 32) {
        const int i = i0 + lane;
        const bool is_eos = (i < n) && (pred[i] == dm.eos);
        const unsigned bal = __ballot_sync(0xffffffffu, is_eos);
        if (bal) { n = i0 + __ffs(bal); found = true; }
      }
    }
    if (lane == 0) st.n_acc[b] = n;
    if (auto_commit) {
      __syncwarp();
      commit_row(st, blk, dm, b, n, n, lane);
      if (lane == 0) {
        __threadfence();
        const unsigned int t = atomicAdd(done_ctr, n > 0 ? 0x10001u : 1u);
        if ((t & 0xffffu) == (unsigned)dm.B - 1) {
          __threadfence();
          finish_iteration(st, dm, ((t >> 16) + (n > 0 ? 1u : 0u)) != 0, cond);
          *done_ctr = 0;
          s_last = 1;
        }
      }
    }
  }
  if (auto_commit && next.source >= 0) {
    __syncthreads();
    if (s_last) {                  // block-uniform: this CTA saw every row committed
      __threadfence();
      plan_verify_block(st, blk, dm, next, s_k, s_off);
      __syncthreads();
      // embedding of the next block's tokens (written by this CTA just above)
      const int M = s_off[dm.B], d = ne.d, groups = d >> 2;
      const WT* emb = reinterpret_cast<const WT*>(ne.emb);
      WT* yb = reinterpret_cast<WT*>(ne.yb);
      for (int idx = tid; idx < M * groups; idx += blockDim.x) {
        const int m = idx / groups, c = (idx - m * groups) * 4;
        const WT* er = emb + (size_t)blk.tok_id[m] * d + c;
        const float4 pp = *reinterpret_cast<const float4*>(ne.pe + (size_t)blk.tok_pos[m] * d + c);
        float4 v;
        v.x = to_f32(er[0]) * ne.scale + pp.x; v.y = to_f32(er[1]) * ne.scale + pp.y;
        v.z = to_f32(er[2]) * ne.scale + pp.z; v.w = to_f32(er[3]) * ne.scale + pp.w;
        *reinterpret_cast<float4*>(ne.y + (size_t)m * d + c) = v;
        store4(yb + (size_t)m * d + c, v);
      }
    }
  }
  trace_mark(TR_ACCEPT, 2);
}

// ---------------------------------------------------------------------------------------------
// Commit as a call of its own (ad_commit): cache-length advance or rollback.  n_in == null commits n_acc.
// grid = 1, block = 256 (one warp per row at a time).
// ---------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256)
commit_kernel(DevState st, PassPlan blk, Dims dm, const int* n_in) {
  __shared__ int s_active;
  trace_mark(TR_COMMIT, 0);
  pdl_launch();
  pdl_wait();
  trace_mark(TR_COMMIT, 1);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  if (threadIdx.x == 0) s_active = 0;
  __syncthreads();
  for (int b = warp; b < dm.B; b += 8) {
    const int nacc = st.n_acc[b];
    const int n = n_in ? n_in[b] : nacc;
    __syncwarp();
    commit_row(st, blk, dm, b, n, nacc, lane);
    if (lane == 0 && nacc > 0) atomicOr(&s_active, 1);
  }
  __syncthreads();
  if (threadIdx.x == 0) finish_iteration(st, dm, s_active != 0, 0ull);
}

// Teacher-forced commit: the caller supplies the accepted tokens.  grid = 1, block = 256.
__global__ void __launch_bounds__(256)
force_commit_kernel(DevState st, PassPlan blk, Dims dm, const int* tokens, const int* n_in) {
  pdl_launch();
  pdl_wait();
  for (int b = threadIdx.x; b < dm.B; b += 256) {
    const int n = n_in[b], k = blk.seg_len[b];
    const int* tk = tokens + (size_t)b * dm.kmax;
    const int* dr = st.drafts + (size_t)b * dm.kmax;
    bool ok = n >= 0 && n <= k;
    for (int i = 0; ok && i + 1 < n; ++i) ok = tk[i] == dr[i];
    for (int i = 0; ok && i < n; ++i) ok = id_in_vocab(tk[i], dm);      // the last one is fed to the next block
    if (!ok) { latch_error(st.status, AD_ERR_ARG); continue; }
    if (n > 0) {
      int len = st.len[b];
      int* out = st.out_ids + (size_t)b * dm.max_tgt;
      for (int i = 0; i < n; ++i) out[len + i] = tk[i];
      len += n;
      st.len[b] = len;
      st.last[b] = tk[n - 1];
      if (tk[n - 1] == dm.eos || len >= st.maxlen[b]) st.fin[b] = 1;
    }
    st.n_acc[b] = 0;
  }
}

// Copies the block results to caller-visible arrays (device pointers).  grid = B, block = 64.
__global__ void export_block_kernel(DevState st, Dims dm, int* argmax_out, int* n_out, int* drafts_out, int* k_out,
                                    PassPlan blk) {
  pdl_launch();
  pdl_wait();
  const int b = blockIdx.x;
  if (argmax_out)
    for (int i = threadIdx.x; i < dm.kmax; i += blockDim.x) argmax_out[(size_t)b * dm.kmax + i] = st.pred[(size_t)b * dm.kmax + i];
  if (drafts_out)
    for (int i = threadIdx.x; i < dm.kmax; i += blockDim.x) drafts_out[(size_t)b * dm.kmax + i] = st.drafts[(size_t)b * dm.kmax + i];
  if (threadIdx.x == 0) {
    if (n_out) n_out[b] = st.n_acc[b];
    if (k_out) k_out[b] = blk.seg_len[b];
  }
}

// End of ad_generate: everything the host needs, gathered into one block (device pointer of pinned, mapped host memory
// or a device buffer), so that the call ends with ONE synchronisation and no further copies:
//   block[0] = iterations the device-side loop ran, block[1] = latched status word (cleared here),
//   block[2] = iterations with an active row, block[3] = B,
//   block[4 + 4 b ..] = {row iterations, accepted, offered, output length} of row b,
//   block[4 + 4 B + b * max_tgt ..] = output ids of row b (only when out_dev is null: host-resident results).
// out_dev / out_len_dev (device pointers, may be null): the caller's result arrays when they live on the device.
// grid = B, block = 128.
__global__ void __launch_bounds__(128)
finalize_generate_kernel(DevState st, Dims dm, int* out_dev, int out_stride, int* out_len_dev, int* block) {
  pdl_launch();
  pdl_wait();
  const int b = blockIdx.x, tid = threadIdx.x;
  const int len = st.len[b];
  if (tid == 0) {
    if (b == 0) {
      block[0] = st.loop_it[2];
      block[1] = *st.status;
      *st.status = 0;
      block[2] = st.loop_it[0];
      block[3] = dm.B;
    }
    int* row = block + 4 + 4 * b;
    row[0] = st.stat_it[b]; row[1] = st.stat_acc[b]; row[2] = st.stat_off[b]; row[3] = len;
    if (out_len_dev) out_len_dev[b] = len;
  }
  const int* src = st.out_ids + (size_t)b * dm.max_tgt;
  if (out_dev) {
    const int w = min(out_stride, dm.max_tgt);
    for (int i = tid; i < w; i += 128) out_dev[(size_t)b * out_stride + i] = src[i];
  } else {
    int* dst = block + 4 + 4 * dm.B + (size_t)b * dm.max_tgt;
    for (int i = tid; i < dm.max_tgt; i += 128) dst[i] = src[i];
  }
}

// FP32 copy of an activation buffer (debug).  grid-stride.
template <typename ActT>
__global__ void to_f32_kernel(const ActT* __restrict__ src, float* __restrict__ dst, size_t n) {
  pdl_launch();
  pdl_wait();
  for (size_t i = blockIdx.x * (size_t)blockDim.x + threadIdx.x; i < n; i += (size_t)gridDim.x * blockDim.x)
    dst[i] = to_f32(src[i]);
}

}  // namespace ad
