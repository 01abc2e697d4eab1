// Persistent decoder pass: the whole decoder stack over one block of packed tokens (verification pass or drafter
// pass) and the vocabulary projection with its per-tile arg-max, as ONE kernel.
//
// Why: with a few dozen tokens a decoder layer is a chain of dependent stages whose work is tiny next to the cost
// of handing data from one set of SMs to the next.  As separate kernels every stage also pays its own prologue
// (barrier set-up, tensor-memory allocation) and fetches its weights only once it runs.  Here the CTAs stay resident,
// set up once, and -- weights never depend on activations -- a producer thread per CTA streams the weight tiles of
// FUTURE stages into a shared-memory ring while the CTA waits for the current stage's inputs.
//
// Shape of the grid: NC clusters of CS CTAs (CS = 4 or 8), one CTA per SM.  A projection stage deals its 128-row
// weight tiles to the clusters; inside a cluster the CS CTAs split the contraction (K) range of the tile, each runs
// its K blocks on the tensor cores (tcgen05.mma, accumulator in tensor memory, tokens on the MMA's N side), leaves its
// partial [tokens x 128] in shared memory, and after a cluster-scope mbarrier hand-shake every CTA sums, in rank
// order (deterministic), the partials of its share of the tokens through distributed shared memory and applies the
// stage's epilogue.  Stages are separated by grid-wide arrival counters (release-add / acquire-poll, one per stage); all
// activations between stages live in L2-resident global buffers and are read with L1-bypassing loads.
//
// LayerNorm has no stage of its own: a projection that closes a sublayer (output projection, FFN2) writes the
// pre-normalisation sum x = residual + bias + projection in FP32 together with per-token partial sums (sum x,
// sum x^2 per 128-feature tile); every consumer of the normalised value (the next projection's operand staging,
// the next residual) applies (x - mean) * rstd * gain + bias itself.
//
// Stages per layer: QKV | self-attention | Wo (+residual, statistics) | cross-Q | cross-attention | cross-Wo (+residual,
// statistics) | FFN1 (+ReLU) | FFN2 (+residual, statistics); after the last layer the vocabulary projection with
// the fused per-tile (max, id) epilogue, B operand resident, two accumulators so the epilogue of a tile overlaps the
// MMAs of the next.
//
// Every wait (mbarrier, cluster hand-shake, grid barrier) is bounded by time; on expiry AD_ERR_TIMEOUT is latched,
// the CTA stops working, drains its copies in flight, frees its tensor memory and returns.
#pragma once

#include "ad_common.cuh"
#include "gemm_tc.cuh"
#include "grid_sync.cuh"

namespace ad {
namespace mega {

constexpr int N_WORKERS = 256;               // warps 0..7: operand staging, attention, reduction, epilogues
constexpr int THREADS = 320;                 // + warp 8 (weight-tile producer) + warp 9 (MMA issuer, owns tensor memory)
constexpr int TILE_A = tc::A_STAGE_BYTES;    // one weight tile: 128 rows x 64 bf16
constexpr int MAX_RING = 10;
constexpr int NT_MAX = 64;                   // most packed tokens a pass may hold
constexpr int RED_LD = 128;                  // floats per token row of a reduction buffer
constexpr int ATT_SMEM = 4 * (64 * 65 + 64 * 64 + 8 * 64 + 8 * 64);
constexpr unsigned long long BUDGET_NS = 20ull * 1000 * 1000;
constexpr int SYNC_STRIDE = 32;              // words between the per-stage arrival counters (one 128-byte line each)
constexpr int SYNC_COUNTERS = 128;           // counters the planning kernels clear (stages per pass <= 128)

enum StageKind : int { ST_QKV = 0, ST_SATT, ST_WO, ST_CQ, ST_CATT, ST_CO, ST_FFN1, ST_FFN2, ST_PER_LAYER, ST_VOCAB = 100 };

struct LayerPtrs {
  const float *bqkv, *bo, *ln1g, *ln1b, *cbq, *cbo, *ln2g, *ln2b, *b1, *b2, *ln3g, *ln3b;
  bf16 *kself, *vself;          // self-attention keys / values of this layer: cache (verification) or scratch (drafter)
  const bf16 *kenc, *venc;      // cross-attention keys / values of this layer
};

struct Params {
  int d, H, F, V, L;
  int B, qchunks;               // attention jobs: B rows x qchunks chunks of 8 queries x H heads
  const CUtensorMap* maps;      // global memory: per layer {Wqkv, Wo, cross-Wq, cross-Wo, W1, W2}, then the embedding matrix
  const LayerPtrs* layers;      // global memory, [L]
  PassPlan plan;
  const int* cross_base;        // [B] slot of source key 0 of row b
  const int* srclen;            // [B]
  const bf16* emb;
  const float* pe;
  float emb_scale, eps, att_scale;
  float* x[2];                  // pre-normalisation residual stream, ping-pong, [M_cap, d] each
  float* stats[2];              // [d / 128][M_cap][2] partial (sum, sum of squares) of the matching x buffer
  int M_cap;
  bf16 *q, *attn, *hid;         // [M_cap, d], [M_cap, d], [M_cap, F]
  bf16* yb_out;                 // [M_cap, d]: the normalised final hidden states the projection consumed
  const int* vocab_M;           // rows the projection scores (null: all M rows of the pass)
  const int* vocab_rows;        // [vocab_M] packed row of each scored row (null: identity)
  float* part_val;              // [rows][n_vtiles]
  int* part_idx;
  int n_vtiles;
  unsigned int* sync_ctr;       // one arrival counter per stage, SYNC_STRIDE words apart, all zero when the kernel starts
  int* status;
  int ring;                     // weight-ring depth (tiles)
  int b_bytes;                  // shared-memory area of a cluster stage's B operand; the reduction buffers follow it
  int red_bytes;                // one reduction buffer: (token capacity rounded up to 16) x 128 floats
  unsigned long long* timeline; // optional: CTA 0 stamps the global timer when a stage's inputs are ready and when it has signalled
};

struct Ctl {
  uint64_t full[MAX_RING], empty[MAX_RING];
  uint64_t acc_full[2], acc_empty[2];
  uint64_t b_ready;
  uint64_t red_full[2];
  uint32_t tmem_base;
  volatile int abort_flag;
  int ok_flag;
  int M, Mv;
  float mu[NT_MAX], rs[NT_MAX];
  __align__(16) float gain[1024];   // LayerNorm gain / bias of the columns this CTA stages in the current stage
  __align__(16) float beta[1024];
  int tok[NT_MAX], pos[NT_MAX], slot[NT_MAX], vrow[NT_MAX];
  float red_val[4][NT_MAX];
  int red_idx[4][NT_MAX];
};


// ---- small PTX helpers -------------------------------------------------------------------------------------
__device__ __forceinline__ void worker_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }
// true in every worker iff ok was true in every worker
__device__ __forceinline__ bool worker_all(bool ok) {
  uint32_t n;
  asm volatile(
      "{\n\t.reg .pred q;\n\tsetp.ne.u32 q, %1, 0;\n\tbar.red.popc.u32 %0, 1, 256, q;\n\t}"
      : "=r"(n) : "r"((uint32_t)ok) : "memory");
  return n == (uint32_t)N_WORKERS;
}
__device__ __forceinline__ uint32_t cluster_rank() { uint32_t v; asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(v)); return v; }
__device__ __forceinline__ uint32_t cluster_size() { uint32_t v; asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(v)); return v; }
__device__ __forceinline__ void cluster_sync_all() {
  asm volatile("barrier.cluster.arrive.release;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
__device__ __forceinline__ uint32_t map_to_rank(uint32_t local_addr, uint32_t rank) {
  uint32_t ra;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(ra) : "r"(local_addr), "r"(rank));
  return ra;
}
__device__ __forceinline__ void mbar_arrive_local(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void mbar_arrive_remote(uint32_t local_bar, uint32_t rank) {
  const uint32_t ra = map_to_rank(local_bar, rank);
  asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(ra) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
  return ok != 0;
}
__device__ __forceinline__ float4 ld_dsmem_f4(uint32_t cluster_addr) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(cluster_addr));
  return v;
}
__device__ __forceinline__ void st_shared_u4(uint32_t addr, uint4 v) {
  asm volatile("st.shared.v4.b32 [%0], {%1, %2, %3, %4};" ::"r"(addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
  __nv_bfloat162 h = __floats2bfloat162_rn(lo, hi);
  return *reinterpret_cast<uint32_t*>(&h);
}
__device__ __forceinline__ uint4 pack8(const float* v) {
  return make_uint4(pack2(v[0], v[1]), pack2(v[2], v[3]), pack2(v[4], v[5]), pack2(v[6], v[7]));
}
__device__ __forceinline__ void unpack8(uint4 u, float* out) {
  const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
  for (int t = 0; t < 4; ++t) { out[2 * t] = __uint_as_float(w[t] << 16); out[2 * t + 1] = __uint_as_float(w[t] & 0xffff0000u); }
}

// Bounded wait on a local mbarrier phase; gives up at once when another role has already aborted.
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, Ctl* ctl, int* status, bool cluster_scope = false) {
  for (int i = 0; i < 64; ++i)
    if (cluster_scope ? mbar_try_wait_cluster(bar, parity) : tc::mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = gs::now_ns();
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (cluster_scope ? mbar_try_wait_cluster(bar, parity) : tc::mbar_try_wait(bar, parity)) return true;
    if (ctl->abort_flag) return false;
    if (gs::now_ns() - t0 > BUDGET_NS) break;
  }
  latch_error(status, AD_ERR_TIMEOUT);
  ctl->abort_flag = 1;
  return false;
}

// Where the (normalised) activation a stage consumes comes from.
enum SrcMode : int { SRC_EMBED = 0, SRC_LAZY_LN = 1, SRC_PLAIN = 2 };
struct ActSrc {
  int mode;
  const float* x;        // SRC_LAZY_LN: pre-normalisation rows [M_cap, ld]
  const float* g;        //              LayerNorm gain / bias
  const float* b;
  const bf16* plain;     // SRC_PLAIN: rows [M_cap, ld]
  int ld;
};

// Raw inputs of eight consecutive activation columns of one packed token: loaded first (so that several chunks'
// loads are in flight at once), turned into values afterwards.
struct Raw8 {
  float4 a0, a1;   // SRC_LAZY_LN: x;  SRC_EMBED: positional table
  uint4 u;         // SRC_PLAIN: the values;  SRC_EMBED: embedding row
};
__device__ __forceinline__ void raw8_load(const Params& p, const Ctl* ctl, const ActSrc& a, int row, int col, Raw8& r) {
  if (a.mode == SRC_PLAIN) {
    r.u = __ldcg(reinterpret_cast<const uint4*>(a.plain + (size_t)row * a.ld + col));
  } else if (a.mode == SRC_LAZY_LN) {
    const float* xr = a.x + (size_t)row * a.ld + col;
    r.a0 = __ldcg(reinterpret_cast<const float4*>(xr));
    r.a1 = __ldcg(reinterpret_cast<const float4*>(xr + 4));
  } else {
    r.u = __ldg(reinterpret_cast<const uint4*>(p.emb + (size_t)ctl->tok[row] * p.d + col));
    const float* pr = p.pe + (size_t)ctl->pos[row] * p.d + col;
    r.a0 = __ldg(reinterpret_cast<const float4*>(pr));
    r.a1 = __ldg(reinterpret_cast<const float4*>(pr + 4));
  }
}
// gcol: index of `col` inside the gain / bias slice held in shared memory (ctl->gain, ctl->beta)
__device__ __forceinline__ uint4 raw8_finish(const Params& p, const Ctl* ctl, const ActSrc& a, int row, int gcol, const Raw8& r) {
  if (a.mode == SRC_PLAIN) return r.u;
  float o[8];
  if (a.mode == SRC_LAZY_LN) {
    const float mu = ctl->mu[row], rs = ctl->rs[row];
    const float4 g0 = *reinterpret_cast<const float4*>(&ctl->gain[gcol]), g1 = *reinterpret_cast<const float4*>(&ctl->gain[gcol + 4]);
    const float4 b0 = *reinterpret_cast<const float4*>(&ctl->beta[gcol]), b1 = *reinterpret_cast<const float4*>(&ctl->beta[gcol + 4]);
    o[0] = g0.x * ((r.a0.x - mu) * rs) + b0.x; o[1] = g0.y * ((r.a0.y - mu) * rs) + b0.y;
    o[2] = g0.z * ((r.a0.z - mu) * rs) + b0.z; o[3] = g0.w * ((r.a0.w - mu) * rs) + b0.w;
    o[4] = g1.x * ((r.a1.x - mu) * rs) + b1.x; o[5] = g1.y * ((r.a1.y - mu) * rs) + b1.y;
    o[6] = g1.z * ((r.a1.z - mu) * rs) + b1.z; o[7] = g1.w * ((r.a1.w - mu) * rs) + b1.w;
  } else {
    float e[8];
    unpack8(r.u, e);
    o[0] = e[0] * p.emb_scale + r.a0.x; o[1] = e[1] * p.emb_scale + r.a0.y;
    o[2] = e[2] * p.emb_scale + r.a0.z; o[3] = e[3] * p.emb_scale + r.a0.w;
    o[4] = e[4] * p.emb_scale + r.a1.x; o[5] = e[5] * p.emb_scale + r.a1.y;
    o[6] = e[6] * p.emb_scale + r.a1.z; o[7] = e[7] * p.emb_scale + r.a1.w;
  }
  return pack8(o);
}

// Residual of a sublayer-closing projection, four consecutive columns: raw loads, then the value.
struct Raw4 {
  float4 x, g, b;  // SRC_LAZY_LN: x, gain, bias;  SRC_EMBED: x = positional table
  uint2 u;         // SRC_EMBED: embedding row
};
__device__ __forceinline__ void raw4_load(const Params& p, const Ctl* ctl, const ActSrc& a, int row, int col, Raw4& r) {
  if (a.mode == SRC_LAZY_LN) {
    r.x = __ldcg(reinterpret_cast<const float4*>(a.x + (size_t)row * a.ld + col));
    r.g = __ldg(reinterpret_cast<const float4*>(a.g + col));
    r.b = __ldg(reinterpret_cast<const float4*>(a.b + col));
  } else {
    r.u = __ldg(reinterpret_cast<const uint2*>(p.emb + (size_t)ctl->tok[row] * p.d + col));
    r.x = __ldg(reinterpret_cast<const float4*>(p.pe + (size_t)ctl->pos[row] * p.d + col));
  }
}
__device__ __forceinline__ float4 raw4_finish(const Params& p, const Ctl* ctl, const ActSrc& a, int row, const Raw4& r) {
  if (a.mode == SRC_LAZY_LN) {
    const float mu = ctl->mu[row], rs = ctl->rs[row];
    return make_float4(r.g.x * ((r.x.x - mu) * rs) + r.b.x, r.g.y * ((r.x.y - mu) * rs) + r.b.y,
                       r.g.z * ((r.x.z - mu) * rs) + r.b.z, r.g.w * ((r.x.w - mu) * rs) + r.b.w);
  }
  return make_float4(__uint_as_float(r.u.x << 16) * p.emb_scale + r.x.x, __uint_as_float(r.u.x & 0xffff0000u) * p.emb_scale + r.x.y,
                     __uint_as_float(r.u.y << 16) * p.emb_scale + r.x.z, __uint_as_float(r.u.y & 0xffff0000u) * p.emb_scale + r.x.w);
}

// Per-token mean and reciprocal standard deviation from the partial sums of the producing stage (four threads per
// token, one round trip for all tokens), and the LayerNorm gain / bias slice [col0, col0 + ncols) into shared memory.
// Workers only; ends with a worker barrier.  stats == null: only the barrier.
__device__ __forceinline__ void row_stats(const Params& p, Ctl* ctl, const float* stats, int M, int tid, const float* gain,
                                          const float* beta, int col0, int ncols) {
  if (stats) {
    const int m = tid >> 2, part = tid & 3, slabs = p.d >> 7;
    float s1 = 0.f, s2 = 0.f;
    if (m < M) {
      float2 v0 = make_float2(0.f, 0.f), v1 = v0;
      if (part < slabs) v0 = __ldcg(reinterpret_cast<const float2*>(stats + ((size_t)part * p.M_cap + m) * 2));
      if (part + 4 < slabs) v1 = __ldcg(reinterpret_cast<const float2*>(stats + ((size_t)(part + 4) * p.M_cap + m) * 2));
      s1 = v0.x + v1.x; s2 = v0.y + v1.y;
    }
    s1 += __shfl_xor_sync(0xffffffffu, s1, 1); s2 += __shfl_xor_sync(0xffffffffu, s2, 1);
    s1 += __shfl_xor_sync(0xffffffffu, s1, 2); s2 += __shfl_xor_sync(0xffffffffu, s2, 2);
    if (part == 0 && m < M) {
      const float mean = s1 / (float)p.d;
      const float var = fmaxf(s2 / (float)p.d - mean * mean, 0.f);
      ctl->mu[m] = mean;
      ctl->rs[m] = rsqrtf(var + p.eps);
    }
    if (gain) {
      for (int i = tid; i < (ncols >> 2); i += N_WORKERS) {
        *reinterpret_cast<float4*>(&ctl->gain[i * 4]) = __ldg(reinterpret_cast<const float4*>(gain + col0 + i * 4));
        *reinterpret_cast<float4*>(&ctl->beta[i * 4]) = __ldg(reinterpret_cast<const float4*>(beta + col0 + i * 4));
      }
    }
  }
  worker_sync();
}

// Stages the B operand of a projection: n_kb sub-tiles [ntile rows x 64 columns] starting at K block kb0, in the
// 128-byte-swizzled K-major layout the MMA descriptor expects (16-byte chunk c of row r at chunk c ^ (r & 7)).
// rows: packed row of each tile row (null: identity); rows >= n_valid are zero.  yb_out != null: the staged values
// are also written there as plain rows (the normalised hidden states, for the debug paths).
// The raw loads of the first batch of chunks are issued BEFORE the row statistics are fetched, so that both round
// trips overlap; stats / gain / beta as for row_stats (all null when nothing is normalised here or later in the stage).
constexpr int STAGE_NB = 4;      // 16-byte chunks a thread has in flight
__device__ __forceinline__ void stage_b(const Params& p, Ctl* ctl, const ActSrc& a, int kb0, int n_kb, int ntile,
                                        int n_valid, const int* rows, uint32_t b_smem, bf16* yb_out, int tid,
                                        const float* stats, int M, const float* gain, const float* beta) {
  const int per_kb = ntile * 8, total = n_kb * per_kb;
  const int n_batches = (total + N_WORKERS * STAGE_NB - 1) / (N_WORKERS * STAGE_NB);
  for (int bt = 0; bt < n_batches; ++bt) {
    Raw8 raw[STAGE_NB];
#pragma unroll
    for (int i = 0; i < STAGE_NB; ++i) {
      const int idx = (bt * STAGE_NB + i) * N_WORKERS + tid;
      if (idx < total) {
        const int kbl = idx / per_kb, rem = idx - kbl * per_kb, m = rem >> 3, c = rem & 7;
        if (m < n_valid) raw8_load(p, ctl, a, rows ? rows[m] : m, (kb0 + kbl) * 64 + c * 8, raw[i]);
      }
    }
    if (bt == 0) row_stats(p, ctl, stats, M, tid, gain, beta, kb0 * 64, n_kb * 64);
#pragma unroll
    for (int i = 0; i < STAGE_NB; ++i) {
      const int idx = (bt * STAGE_NB + i) * N_WORKERS + tid;
      if (idx < total) {
        const int kbl = idx / per_kb, rem = idx - kbl * per_kb, m = rem >> 3, c = rem & 7;
        uint4 v = make_uint4(0u, 0u, 0u, 0u);
        if (m < n_valid) {
          v = raw8_finish(p, ctl, a, rows ? rows[m] : m, kbl * 64 + c * 8, raw[i]);
          if (yb_out) *reinterpret_cast<uint4*>(yb_out + (size_t)m * a.ld + (kb0 + kbl) * 64 + c * 8) = v;
        }
        st_shared_u4(b_smem + (uint32_t)(kbl * ntile * 128 + m * 128 + ((c ^ (m & 7)) << 4)), v);
      }
    }
  }
  asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // generic-proxy writes -> visible to the MMA's reads
}

// One attention job: 8 queries (one per warp) of one row and one head against that row's keys, K/V tiles of 64 keys
// staged in shared memory as floats, online softmax with warp-shuffle reductions.  Keys and values may have been
// written by other CTAs earlier in this kernel, hence the L1-bypassing loads.
__device__ __forceinline__ void attention_job(const bf16* q, const bf16* kk, const bf16* vv, bf16* out, int d, int h,
                                              int m0, int nq, int kbase, int row_nk, const int* nk_tok, float scale,
                                              float* sm, int tid) {
  constexpr int DH = 64, KT = 64;
  float (*ks)[DH + 1] = reinterpret_cast<float (*)[DH + 1]>(sm);
  float (*vs)[DH] = reinterpret_cast<float (*)[DH]>(sm + KT * (DH + 1));
  float (*qs)[DH] = reinterpret_cast<float (*)[DH]>(sm + KT * (DH + 1) + KT * DH);
  float (*ps)[KT] = reinterpret_cast<float (*)[KT]>(sm + KT * (DH + 1) + KT * DH + 8 * DH);
  const int warp = tid >> 5, lane = tid & 31;
  int nk = 0;
  if (warp < nq) {      // this warp's query: two elements per lane, read past L1 (written earlier in this kernel)
    nk = nk_tok ? min(nk_tok[m0 + warp], row_nk) : row_nk;
    const unsigned short* qp = reinterpret_cast<const unsigned short*>(q + (size_t)(m0 + warp) * d + h * DH);
    qs[warp][lane] = __uint_as_float((uint32_t)__ldcg(qp + lane) << 16) * scale;
    qs[warp][lane + 32] = __uint_as_float((uint32_t)__ldcg(qp + lane + 32) << 16) * scale;
  }
  float mx = -INFINITY, den = 0.f, acc0 = 0.f, acc1 = 0.f;
  for (int j0 = 0; j0 < row_nk; j0 += KT) {
    worker_sync();   // previous tile (or previous job) fully consumed
    for (int idx = tid; idx < KT * (DH / 8); idx += N_WORKERS) {
      const int j = idx >> 3, c = (idx & 7) * 8;
      float kf[8], vf[8];
      if (j0 + j < row_nk) {
        const size_t off = (size_t)(kbase + j0 + j) * d + h * DH + c;
        unpack8(__ldcg(reinterpret_cast<const uint4*>(kk + off)), kf);
        unpack8(__ldcg(reinterpret_cast<const uint4*>(vv + off)), vf);
      } else {
#pragma unroll
        for (int t = 0; t < 8; ++t) { kf[t] = 0.f; vf[t] = 0.f; }
      }
#pragma unroll
      for (int t = 0; t < 8; ++t) { ks[j][c + t] = kf[t]; vs[j][c + t] = vf[t]; }
    }
    worker_sync();
    float s0 = 0.f, s1 = 0.f;
#pragma unroll 8
    for (int c = 0; c < DH; ++c) {
      const float qv = qs[warp][c];
      s0 = fmaf(qv, ks[lane][c], s0);
      s1 = fmaf(qv, ks[lane + 32][c], s1);
    }
    float p0 = 0.f, p1 = 0.f, corr = 1.f;
    if (nk > j0) {              // warp-uniform
      const float a0 = (j0 + lane < nk) ? s0 : -INFINITY;
      const float a1 = (j0 + lane + 32 < nk) ? s1 : -INFINITY;
      float tmax = fmaxf(a0, a1);
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) tmax = fmaxf(tmax, __shfl_xor_sync(0xffffffffu, tmax, off));
      const float m_new = fmaxf(mx, tmax);
      corr = expf(mx - m_new);
      p0 = expf(a0 - m_new);
      p1 = expf(a1 - m_new);
      float psum = p0 + p1;
#pragma unroll
      for (int off = 16; off > 0; off >>= 1) psum += __shfl_xor_sync(0xffffffffu, psum, off);
      den = den * corr + psum;
      mx = m_new;
    }
    ps[warp][lane] = p0;
    ps[warp][lane + 32] = p1;
    __syncwarp();
    acc0 *= corr; acc1 *= corr;
    const int jn = min(KT, row_nk - j0);
#pragma unroll 4
    for (int j = 0; j < jn; ++j) {
      const float pj = ps[warp][j];
      acc0 = fmaf(pj, vs[j][lane], acc0);
      acc1 = fmaf(pj, vs[j][lane + 32], acc1);
    }
    __syncwarp();
  }
  if (warp < nq && nk > 0) {
    const float inv = 1.f / den;
    bf16* op = out + (size_t)(m0 + warp) * d + h * DH;
    op[lane] = __float2bfloat16_rn(acc0 * inv);
    op[lane + 32] = __float2bfloat16_rn(acc1 * inv);
  }
}

struct StageInfo {
  int kind, layer;
  bool gemm;
  int N, K, map;
};
__device__ __forceinline__ StageInfo stage_info(const Params& p, int s) {
  StageInfo si;
  si.layer = s / ST_PER_LAYER;
  si.kind = s - si.layer * ST_PER_LAYER;
  si.gemm = true; si.N = p.d; si.K = p.d; si.map = 0;
  if (si.layer >= p.L) { si.kind = ST_VOCAB; si.N = p.V; si.map = 6 * p.L; return si; }
  switch (si.kind) {
    case ST_QKV: si.N = 3 * p.d; si.map = 0; break;
    case ST_WO: si.map = 1; break;
    case ST_CQ: si.map = 2; break;
    case ST_CO: si.map = 3; break;
    case ST_FFN1: si.N = p.F; si.map = 4; break;
    case ST_FFN2: si.K = p.F; si.map = 5; break;
    default: si.gemm = false; break;
  }
  si.map += 6 * si.layer;
  return si;
}

// grid = NC * CS CTAs in clusters of CS; block = 320 threads; dynamic shared memory =
//   1024 (alignment) + ring * 16 KB (weight tiles) + a work area that holds, per kind of stage, either the B operand
//   of a cluster stage (b_bytes) followed by two reduction buffers (red_bytes each), or the resident B operand of the
//   vocabulary stage, or the K/V tiles of an attention job.
__global__ void __launch_bounds__(THREADS, 1)
decoder_pass_kernel(const __grid_constant__ Params p) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(16) Ctl ctl_s;
  Ctl* ctl = &ctl_s;

  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int CS = (int)cluster_size(), r = (int)cluster_rank();
  const int G = gridDim.x, g = blockIdx.x, NC = G / CS, c = g / CS;
  const int R = p.ring;
  const int L = p.L;
  const int n_stages = ST_PER_LAYER * L + 1;
  const uint32_t smem_base = (tc::smem_u32(smem_raw) + 1023u) & ~1023u;
  const uint32_t ring_base = smem_base;
  const uint32_t b_base = smem_base + (uint32_t)R * TILE_A;
  uint8_t* flex_ptr = smem_raw + (b_base - tc::smem_u32(smem_raw));
  const uint32_t red_base = b_base + (uint32_t)p.b_bytes;
  float* red_ptr = reinterpret_cast<float*>(flex_ptr + p.b_bytes);

  if (tid == 0) {
    for (int i = 0; i < R; ++i) { tc::mbar_init(tc::smem_u32(&ctl->full[i]), 1); tc::mbar_init(tc::smem_u32(&ctl->empty[i]), 1); }
    for (int i = 0; i < 2; ++i) {
      tc::mbar_init(tc::smem_u32(&ctl->acc_full[i]), 1);
      tc::mbar_init(tc::smem_u32(&ctl->acc_empty[i]), 8);
      tc::mbar_init(tc::smem_u32(&ctl->red_full[i]), (uint32_t)CS);
    }
    tc::mbar_init(tc::smem_u32(&ctl->b_ready), 8);
    ctl->abort_flag = 0;
    ctl->M = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 9) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tc::smem_u32(&ctl->tmem_base)), "r"(128u) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  cluster_sync_all();            // every CTA of the cluster has initialised its barriers before anybody arrives remotely
  const uint32_t tmem_base = ctl->tmem_base;
  pdl_launch();

  if (warp == 8) {
    // ================================ weight-tile producer ================================
    if (lane == 0) {
      uint32_t seq = 0;
      bool ok = true, know_m = false;
      for (int s = 0; s < n_stages && ok; ++s) {
        const StageInfo si = stage_info(p, s);
        if (!si.gemm) continue;
        const CUtensorMap* map = p.maps + si.map;
        const bool vocab = si.kind == ST_VOCAB;
        const int n_tiles = (si.N + 127) >> 7;
        const int kpc = vocab ? (si.K >> 6) : (si.K >> 6) / CS;
        const int kb0 = vocab ? 0 : r * kpc;
        for (int nt = vocab ? g : c; nt < n_tiles && ok; nt += vocab ? G : NC) {
          for (int kb = 0; kb < kpc && ok; ++kb) {
            const uint32_t slot = seq % (uint32_t)R, round = seq / (uint32_t)R;
            if (round > 0) {
              if (!know_m) {           // the ring is full: from here on the tiles are only needed if there is work
                pdl_wait();
                know_m = true;
                const int M = *reinterpret_cast<const volatile int*>(p.plan.M);
                if (M <= 0 || M > NT_MAX) { ok = false; break; }
              }
              ok = wait_bar(tc::smem_u32(&ctl->empty[slot]), (round - 1) & 1, ctl, p.status);
              if (!ok) break;
            }
            const uint32_t bar = tc::smem_u32(&ctl->full[slot]);
            tc::mbar_expect_tx(bar, TILE_A);
            tc::tma_load_2d(ring_base + slot * TILE_A, map, (kb0 + kb) * 64, nt * 128, bar);
            ++seq;
          }
        }
      }
      // drain: every copy this thread has issued must have landed before the CTA may leave
      for (uint32_t i = seq > (uint32_t)R ? seq - R : 0; i < seq; ++i) {
        const uint32_t bar = tc::smem_u32(&ctl->full[i % R]);
        const unsigned long long t0 = gs::now_ns();
        while (!tc::mbar_try_wait(bar, (i / R) & 1))
          if (gs::now_ns() - t0 > BUDGET_NS) { latch_error(p.status, AD_ERR_TIMEOUT); break; }
      }
    }
  } else if (warp == 9) {
    // ================================ MMA issuer ================================
    pdl_wait();
    const int M = *reinterpret_cast<const volatile int*>(p.plan.M);
    const int ntile = max(16, (M + 15) & ~15);
    if (lane == 0 && M > 0 && M <= NT_MAX) {
      const uint32_t idesc = tc::make_idesc(128, ntile);
      uint32_t seq = 0, jc = 0, bc = 0;
      bool ok = true;
      for (int s = 0; s < n_stages && ok; ++s) {
        const StageInfo si = stage_info(p, s);
        if (!si.gemm) continue;
        const bool vocab = si.kind == ST_VOCAB;
        const int n_tiles = (si.N + 127) >> 7;
        const int kpc = vocab ? (si.K >> 6) : (si.K >> 6) / CS;
        bool b_staged = false;
        for (int nt = vocab ? g : c; nt < n_tiles && ok; nt += vocab ? G : NC) {
          const uint32_t a = jc & 1;
          if (jc >= 2) ok = wait_bar(tc::smem_u32(&ctl->acc_empty[a]), ((jc >> 1) - 1) & 1, ctl, p.status);
          if (ok && (!vocab || !b_staged)) {
            ok = wait_bar(tc::smem_u32(&ctl->b_ready), bc & 1, ctl, p.status);
            ++bc;
            b_staged = true;
          }
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint32_t acc = tmem_base + a * 64;
          for (int kb = 0; kb < kpc && ok; ++kb) {
            const uint32_t slot = seq % (uint32_t)R;
            ok = wait_bar(tc::smem_u32(&ctl->full[slot]), (seq / R) & 1, ctl, p.status);
            if (!ok) break;
            asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
            const uint64_t da = tc::make_smem_desc(ring_base + slot * TILE_A);
            const uint64_t db = tc::make_smem_desc(b_base + (uint32_t)(kb * ntile * 128));
#pragma unroll
            for (int k4 = 0; k4 < 4; ++k4) tc::umma_bf16(acc, da + 2 * k4, db + 2 * k4, idesc, (kb | k4) ? 1u : 0u);
            tc::umma_commit(tc::smem_u32(&ctl->empty[slot]));
            ++seq;
          }
          if (ok) tc::umma_commit(tc::smem_u32(&ctl->acc_full[a]));
          ++jc;
        }
      }
    }
    __syncwarp();
  } else {
    // ================================ workers ================================
    pdl_wait();
    const int M = *reinterpret_cast<const volatile int*>(p.plan.M);
    const int Mv = p.vocab_M ? min(*reinterpret_cast<const volatile int*>(p.vocab_M), M) : M;
    if (tid < NT_MAX) {
      const bool on = tid < M;
      ctl->tok[tid] = on ? p.plan.tok_id[tid] : 0;
      ctl->pos[tid] = on ? p.plan.tok_pos[tid] : 0;
      ctl->slot[tid] = on ? p.plan.kv_slot[tid] : 0;
      ctl->vrow[tid] = tid < Mv ? (p.vocab_rows ? p.vocab_rows[tid] : tid) : 0;
    }
    const int ntile = max(16, (M + 15) & ~15);
    const int quad = warp & 3, half = warp >> 2;
    uint32_t jc = 0, rc = 0;
    bool ok = M > 0 && M <= NT_MAX;
    worker_sync();

    for (int s = 0; s < n_stages && ok; ++s) {
      const StageInfo si = stage_info(p, s);
      const LayerPtrs* lp = p.layers + (si.layer < L ? si.layer : L - 1);
      const bool vocab = si.kind == ST_VOCAB;
      const int n_tiles = (si.N + 127) >> 7;
      const int att_jobs = p.B * p.qchunks * p.H;
      const bool has_work = si.gemm ? ((vocab ? g : c) < n_tiles) : (g < att_jobs);
      if (has_work) {
        if (s > 0) {           // inputs of this stage: everything all CTAs wrote in the stages before
          if (tid == 0) {
            // stage s - 1 is complete once all G CTAs have arrived on its counter (a CTA without work in a stage arrives
            // at once and runs ahead, which is why every stage has a counter of its own)
            const bool got = gs::wait_reached(p.sync_ctr + (size_t)(s - 1) * SYNC_STRIDE, (unsigned int)G, BUDGET_NS);
            if (!got) { latch_error(p.status, AD_ERR_TIMEOUT); ctl->abort_flag = 1; }
            ctl->ok_flag = got ? 1 : 0;
          }
          worker_sync();
          ok = ctl->ok_flag != 0;
          if (!ok) break;
        }
        if (p.timeline && g == 0 && tid == 0) p.timeline[2 * s] = gs::now_ns();
        // the x / statistics buffer holding this layer's input, and the other one
        const int in_buf = si.layer & 1, oth = in_buf ^ 1;

        if (!si.gemm) {
          // ---------------- attention stages ----------------
          const bool cross = si.kind == ST_CATT;
          for (int j = g; j < att_jobs; j += G) {
            const int h = j % p.H, chunk = (j / p.H) % p.qchunks, b = j / (p.H * p.qchunks);
            const int seg_len = p.plan.seg_len[b], i0 = chunk * 8;
            if (i0 >= seg_len) continue;
            const int m0 = p.plan.seg_off[b] + i0, nq = min(8, seg_len - i0);
            if (cross)
              attention_job(p.q, lp->kenc, lp->venc, p.attn, p.d, h, m0, nq, p.cross_base[b], p.srclen[b], nullptr, p.att_scale,
                            reinterpret_cast<float*>(flex_ptr), tid);
            else
              attention_job(p.q, lp->kself, lp->vself, p.attn, p.d, h, m0, nq, p.plan.key_base[b], p.plan.row_nk[b], p.plan.att_n,
                            p.att_scale, reinterpret_cast<float*>(flex_ptr), tid);
          }
        } else {
          // ---------------- projection stages ----------------
          ActSrc bsrc, rsrc;                       // B operand source; residual source (sublayer-closing projections)
          bsrc.mode = SRC_PLAIN; bsrc.x = nullptr; bsrc.g = nullptr; bsrc.b = nullptr; bsrc.plain = nullptr; bsrc.ld = p.d;
          rsrc = bsrc;
          const float* stats_in = nullptr;         // statistics needed by this stage (for the lazy LayerNorm)
          const float* bias = nullptr;
          float* x_out = nullptr; float* stats_out = nullptr;
          auto lazy = [&](ActSrc& a, int buf, const float* gg, const float* bb) {
            a.mode = SRC_LAZY_LN; a.x = p.x[buf]; a.g = gg; a.b = bb; a.ld = p.d; stats_in = p.stats[buf];
          };
          const LayerPtrs* prev = si.layer > 0 && si.layer <= L ? p.layers + si.layer - 1 : nullptr;
          switch (si.kind) {
            case ST_QKV:
              bias = lp->bqkv;
              if (si.layer == 0) bsrc.mode = SRC_EMBED; else lazy(bsrc, in_buf, prev->ln3g, prev->ln3b);
              break;
            case ST_WO:
              bias = lp->bo; bsrc.plain = p.attn;
              if (si.layer == 0) rsrc.mode = SRC_EMBED; else lazy(rsrc, in_buf, prev->ln3g, prev->ln3b);
              x_out = p.x[oth]; stats_out = p.stats[oth];
              break;
            case ST_CQ: bias = lp->cbq; lazy(bsrc, oth, lp->ln1g, lp->ln1b); break;
            case ST_CO:
              bias = lp->cbo; bsrc.plain = p.attn; lazy(rsrc, oth, lp->ln1g, lp->ln1b);
              x_out = p.x[in_buf]; stats_out = p.stats[in_buf];
              break;
            case ST_FFN1: bias = lp->b1; lazy(bsrc, in_buf, lp->ln2g, lp->ln2b); break;
            case ST_FFN2:
              bias = lp->b2; bsrc.plain = p.hid; bsrc.ld = p.F; lazy(rsrc, in_buf, lp->ln2g, lp->ln2b);
              x_out = p.x[oth]; stats_out = p.stats[oth];
              break;
            default:   // ST_VOCAB: the last layer's output sits in the buffer its FFN2 wrote
              lazy(bsrc, L & 1, p.layers[L - 1].ln3g, p.layers[L - 1].ln3b);
              break;
          }
          // LayerNorm gain / bias of the staged operand (null when the operand is not normalised here)
          const float* bg = bsrc.mode == SRC_LAZY_LN ? bsrc.g : nullptr;
          const float* bb = bsrc.mode == SRC_LAZY_LN ? bsrc.b : nullptr;

          if (vocab) {
            // B operand resident for the whole stage; tiles g, g + G, ...; epilogue of tile i under the MMAs of tile i + 1
            stage_b(p, ctl, bsrc, 0, si.K >> 6, ntile, Mv, ctl->vrow, b_base, g == 0 ? p.yb_out : nullptr, tid, stats_in, M, bg, bb);
            __syncwarp();
            if (lane == 0) mbar_arrive_local(tc::smem_u32(&ctl->b_ready));
            for (int nt = g; nt < n_tiles; nt += G) {
              const uint32_t a = jc & 1;
              ok = worker_all(wait_bar(tc::smem_u32(&ctl->acc_full[a]), (jc >> 1) & 1, ctl, p.status));
              if (!ok) break;
              asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
              const uint32_t tl = tmem_base + a * 64 + (static_cast<uint32_t>(quad * 32) << 16);
              const int n = nt * 128 + quad * 32 + lane;
              for (int c0 = half * 16; c0 < ntile && c0 < Mv; c0 += 32) {
                float acc[16];
                tc::tmem_ld16(tl + (uint32_t)c0, acc);
#pragma unroll
                for (int j = 0; j < 16; ++j) acc[j] = n < p.V ? acc[j] : -INFINITY;
                float my_v; int my_i;
                tc::warp_argmax_items16(acc, lane, my_v, my_i);
                const int t = c0 + (lane >> 1);
                if (!(lane & 1) && t < Mv) { ctl->red_val[quad][t] = my_v; ctl->red_idx[quad][t] = nt * 128 + quad * 32 + my_i; }
              }
              asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
              __syncwarp();
              if (lane == 0) mbar_arrive_local(tc::smem_u32(&ctl->acc_empty[a]));
              worker_sync();
              if (tid < Mv) {
                float v = ctl->red_val[0][tid];
                int idx = ctl->red_idx[0][tid];
#pragma unroll
                for (int w = 1; w < 4; ++w) {
                  const float ov = ctl->red_val[w][tid];
                  if (ov > v) { v = ov; idx = ctl->red_idx[w][tid]; }
                }
                p.part_val[(size_t)tid * p.n_vtiles + nt] = v;
                p.part_idx[(size_t)tid * p.n_vtiles + nt] = idx;
              }
              worker_sync();
              ++jc;
            }
          } else {
            const int kpc = (si.K >> 6) / CS;
            const int tpc = ntile / CS;                      // tokens this CTA reduces and finishes
            for (int nt = c; nt < n_tiles; nt += NC) {
              const uint32_t a = jc & 1, pb = rc & 1;
              // (the statistics are the same for every tile of the stage: fetched with the first one)
              stage_b(p, ctl, bsrc, r * kpc, kpc, ntile, M, nullptr, b_base, nullptr, tid, nt == c ? stats_in : nullptr, M, bg, bb);
              __syncwarp();
              if (lane == 0) mbar_arrive_local(tc::smem_u32(&ctl->b_ready));
              ok = worker_all(wait_bar(tc::smem_u32(&ctl->acc_full[a]), (jc >> 1) & 1, ctl, p.status));
              if (!ok) break;
              asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
              // this CTA's partial [tokens x 128 features] -> reduction buffer pb
              float* red = red_ptr + (size_t)pb * (p.red_bytes / 4);
              const uint32_t tl = tmem_base + a * 64 + (static_cast<uint32_t>(quad * 32) << 16);
              for (int ci = half; ci < (ntile >> 4); ci += 2) {
                float acc[16];
                tc::tmem_ld16(tl + (uint32_t)(ci * 16), acc);
#pragma unroll
                for (int j = 0; j < 16; ++j) red[(ci * 16 + j) * RED_LD + quad * 32 + lane] = acc[j];
              }
              asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
              __syncwarp();
              if (lane == 0) mbar_arrive_local(tc::smem_u32(&ctl->acc_empty[a]));
              worker_sync();                                 // the whole partial is in shared memory
              if (tid < CS) mbar_arrive_remote(tc::smem_u32(&ctl->red_full[pb]), (uint32_t)tid);
              ok = worker_all(wait_bar(tc::smem_u32(&ctl->red_full[pb]), (rc >> 1) & 1, ctl, p.status, true));
              if (!ok) break;
              // sum the CS partials of this CTA's tokens in rank order; lane owns features 4 lane .. 4 lane + 3
              for (int tl_ = warp; tl_ < tpc; tl_ += 8) {
                const int m = r * tpc + tl_;
                if (m >= M) continue;
                const uint32_t local = red_base + (uint32_t)pb * (uint32_t)p.red_bytes + (uint32_t)((m * RED_LD + lane * 4) * 4);
                const int n = nt * 128 + lane * 4;
                // all loads first: the CS partials, the bias and the residual's inputs are one round trip together
                float4 part[8];
#pragma unroll
                for (int q = 0; q < 8; ++q)
                  if (q < CS) part[q] = ld_dsmem_f4(map_to_rank(local, (uint32_t)q));
                const float4 bv = __ldg(reinterpret_cast<const float4*>(bias + n));
                Raw4 rr;
                if (x_out) raw4_load(p, ctl, rsrc, m, n, rr);
                float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
                for (int q = 0; q < 8; ++q)
                  if (q < CS) { v.x += part[q].x; v.y += part[q].y; v.z += part[q].z; v.w += part[q].w; }
                v.x += bv.x; v.y += bv.y; v.z += bv.z; v.w += bv.w;
                if (x_out) {
                  const float4 rv = raw4_finish(p, ctl, rsrc, m, rr);
                  v.x += rv.x; v.y += rv.y; v.z += rv.z; v.w += rv.w;
                  *reinterpret_cast<float4*>(x_out + (size_t)m * p.d + n) = v;
                  float s1 = v.x + v.y + v.z + v.w, s2 = v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
#pragma unroll
                  for (int o = 16; o > 0; o >>= 1) { s1 += __shfl_xor_sync(0xffffffffu, s1, o); s2 += __shfl_xor_sync(0xffffffffu, s2, o); }
                  if (lane == 0) *reinterpret_cast<float2*>(stats_out + ((size_t)nt * p.M_cap + m) * 2) = make_float2(s1, s2);
                } else {
                  if (si.kind == ST_FFN1) { v.x = fmaxf(v.x, 0.f); v.y = fmaxf(v.y, 0.f); v.z = fmaxf(v.z, 0.f); v.w = fmaxf(v.w, 0.f); }
                  const uint2 u = make_uint2(pack2(v.x, v.y), pack2(v.z, v.w));
                  bf16* dst;
                  if (si.kind == ST_QKV) {
                    const int seg = n / p.d, col = n - seg * p.d;
                    dst = seg == 0 ? p.q + (size_t)m * p.d + col
                                   : (seg == 1 ? lp->kself : lp->vself) + (size_t)ctl->slot[m] * p.d + col;
                  } else if (si.kind == ST_CQ) {
                    dst = p.q + (size_t)m * p.d + n;
                  } else {
                    dst = p.hid + (size_t)m * p.F + n;
                  }
                  *reinterpret_cast<uint2*>(dst) = u;
                }
              }
              worker_sync();
              ++jc; ++rc;
            }
            if (!ok) break;
          }
        }
      }
      if (!ok) break;
      // this CTA's part of stage s is done (trivially so if it had none)
#ifdef AD_MEGA_FENCE_ALL
      __threadfence();
#endif
      worker_sync();
      if (tid == 0) {
        gs::arrive_release(p.sync_ctr + (size_t)s * SYNC_STRIDE, 1u);
        if (p.timeline && g == 0) p.timeline[2 * s + 1] = gs::now_ns();
      }
    }
    if (M > NT_MAX && tid == 0) latch_error(p.status, AD_ERR_CAPACITY);
  }

  // ---- teardown: nobody leaves while a peer may still read its shared memory or arrive on its barriers ----
  __syncthreads();
  cluster_sync_all();
  if (warp == 9) {
    __syncwarp();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(128u) : "memory");
  }
}

}  // namespace mega
}  // namespace ad
