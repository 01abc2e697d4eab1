// BF16 projection GEMM on the 5th-generation tensor cores (tcgen05.mma, accumulator in tensor memory),
// operands staged in shared memory by TMA through an mbarrier ring.
//
// Computes D^T[n, m] = sum_k W[n, k] * X[m, k]  ("swap-AB"): the 128 rows of a weight tile fill the MMA's
// M side (one TMEM lane per output feature) and the packed tokens are the MMA's N side, so a block of a few
// drafted tokens still issues full-width instructions and the kernel streams every weight byte exactly once.
// Both operands are K-major (row-major [rows, K]) and land in shared memory in the 128-byte-swizzled
// canonical layout that the TMA and the MMA shared-memory descriptor agree on.
//
// Thread roles inside the 256-thread CTA: lane 0 of several warps issues TMA loads, lane 0 of warps 4..7 issues the
// MMAs (up to four issuers, each with its own accumulator region in tensor memory), then all eight warps take part
// in the epilogue: warp w reads the 32 TMEM lanes of quadrant w % 4 (tcgen05.ld 32x32b), adds the issuers' regions
// up, and the two warps of a quadrant share its token columns.  The epilogue is a chain of dependent instructions
// per thread, so halving each thread's share of it shortens the kernel.
// Every mbarrier wait is bounded in time (20 ms); on expiry the kernel latches AD_ERR_TIMEOUT, frees its TMEM and returns.
#pragma once

#include "ad_common.cuh"

namespace ad {
namespace tc {

constexpr int BLOCK_N_FEAT = 128;   // weight rows per CTA = MMA M
constexpr int BLOCK_K = 64;         // bf16 elements per 128-byte swizzle row
constexpr int THREADS = 256;        // 8 warps: two per tensor-memory lane quadrant
constexpr int UMMA_K = 16;          // K of one tcgen05.mma kind::f16
constexpr int A_STAGE_BYTES = BLOCK_N_FEAT * BLOCK_K * 2;   // 16 KiB
constexpr int MAX_STAGES = 8;
// Budget of a bounded wait in nanoseconds of the global timer (a legitimate wait lasts microseconds).
constexpr unsigned long long WAIT_BUDGET_NS = 20ull * 1000 * 1000;

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
  return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
  asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count));
}
__device__ __forceinline__ void mbar_expect_tx(uint32_t bar, uint32_t bytes) {
  asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok != 0;
}
// Non-blocking probe of a barrier phase: returns at once with 1 if the phase has completed, else 0.
__device__ __forceinline__ uint32_t mbar_test(uint32_t bar, uint32_t parity) {
  uint32_t ok;
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
      "selp.u32 %0, 1, 0, p;\n\t}"
      : "=r"(ok)
      : "r"(bar), "r"(parity)
      : "memory");
  return ok;
}
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
// Bounded wait: bounded by TIME, not by a poll count (one try_wait may itself suspend the thread for a while).
// The timer is read every 64 polls.  Returns false (after latching the error) when the phase did not complete
// within WAIT_BUDGET_NS.
__device__ __forceinline__ bool mbar_wait_budget(uint32_t bar, uint32_t parity, int* status, unsigned long long budget_ns) {
  for (int i = 0; i < 64; ++i)
    if (mbar_try_wait(bar, parity)) return true;
  const unsigned long long t0 = global_ns();
  for (;;) {
    for (int i = 0; i < 64; ++i)
      if (mbar_try_wait(bar, parity)) return true;
    if (global_ns() - t0 > budget_ns) break;
  }
  latch_error(status, AD_ERR_TIMEOUT);
  return false;
}
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, int* status) {
  return mbar_wait_budget(bar, parity, status, WAIT_BUDGET_NS);
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int c0, int c1, uint32_t bar) {
  asm volatile(
      "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
      ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(c0), "r"(c1), "r"(bar)
      : "memory");
}

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes (64 bf16) and whose 8-row
// groups are 1024 bytes apart, 128-byte swizzle: start address >> 4 in bits [0,14), leading byte offset
// (unused by swizzled K-major layouts, encoded as 1) in [16,30), stride byte offset 1024 >> 4 in [32,46),
// descriptor version 1 in [46,48), layout type 2 (SWIZZLE_128B) in [61,64).
__device__ __forceinline__ uint64_t make_smem_desc(uint32_t addr) {
  uint64_t d = 0;
  d |= static_cast<uint64_t>((addr >> 4) & 0x3FFF);
  d |= static_cast<uint64_t>(1) << 16;
  d |= static_cast<uint64_t>(1024 >> 4) << 32;
  d |= static_cast<uint64_t>(1) << 46;
  d |= static_cast<uint64_t>(2) << 61;
  return d;
}

// Instruction descriptor of kind::f16 with BF16 A and B (both K-major), FP32 accumulator:
// accumulator format 1 (F32) in bits [4,6), A format 1 (BF16) in [7,10), B format 1 in [10,13),
// N >> 3 in [17,23), M >> 4 in [24,29).
__device__ __forceinline__ uint32_t make_idesc(int mma_m, int mma_n) {
  return (1u << 4) | (1u << 7) | (1u << 10) | (static_cast<uint32_t>(mma_n >> 3) << 17) |
         (static_cast<uint32_t>(mma_m >> 4) << 24);
}

__device__ __forceinline__ void umma_bf16(uint32_t tmem_d, uint64_t desc_a, uint64_t desc_b, uint32_t idesc,
                                          uint32_t accumulate) {
  asm volatile(
      "{\n\t.reg .pred p;\n\t"
      "setp.ne.b32 p, %4, 0;\n\t"
      "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n\t}"
      ::"r"(tmem_d), "l"(desc_a), "l"(desc_b), "r"(idesc), "r"(accumulate)
      : "memory");
}
// Makes the mbarrier track completion of every MMA this thread has issued so far.
__device__ __forceinline__ void umma_commit(uint32_t bar) {
  asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar)
               : "memory");
}
// 32 consecutive accumulator columns of this thread's TMEM lane.
__device__ __forceinline__ void tmem_ld32(uint32_t taddr, float* v) {
  uint32_t r[32];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
      "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15]),
        "=r"(r[16]), "=r"(r[17]), "=r"(r[18]), "=r"(r[19]), "=r"(r[20]), "=r"(r[21]), "=r"(r[22]), "=r"(r[23]),
        "=r"(r[24]), "=r"(r[25]), "=r"(r[26]), "=r"(r[27]), "=r"(r[28]), "=r"(r[29]), "=r"(r[30]), "=r"(r[31])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 32; ++i) v[i] = __uint_as_float(r[i]);
}
__device__ __forceinline__ void tmem_ld16(uint32_t taddr, float* v) {
  uint32_t r[16];
  asm volatile(
      "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
      "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
      : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
        "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
      : "r"(taddr));
  asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
#pragma unroll
  for (int i = 0; i < 16; ++i) v[i] = __uint_as_float(r[i]);
}

// Order-preserving map from float to unsigned: a > b  <=>  key(a) > key(b) (no NaNs expected).
__device__ __forceinline__ unsigned int float_key(float v) {
  const unsigned int u = __float_as_uint(v);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float key_float(unsigned int k) {
  return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
}
// Largest value over the warp and the lowest lane holding it: one redux and one ballot.
__device__ __forceinline__ void warp_argmax_lane(float v, float& best, int& lane_of_best) {
  const unsigned int k = float_key(v);
  const unsigned int m = __reduce_max_sync(0xffffffffu, k);
  const unsigned int bal = __ballot_sync(0xffffffffu, k == m);
  best = key_float(m);
  lane_of_best = __ffs(bal) - 1;
}

// Arg-max over the 32 lanes for 32 values per lane at once.  v[j] is this lane's candidate for item j; on
// return lane L holds, for item L, the largest candidate and the lowest lane that offered it.  Each halving
// step sends one half of the items a lane still holds to its partner and keeps the other half, so that every
// item costs about one exchange instead of five.
__device__ __forceinline__ void warp_argmax_items(float (&v)[32], int lane, float& best, int& from) {
  int src[32];
#pragma unroll
  for (int j = 0; j < 32; ++j) src[j] = lane;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const bool up = (lane & o) != 0;                 // this lane keeps the upper half of its items
#pragma unroll
    for (int i = 0; i < o; ++i) {
      const float keep_v = up ? v[i + o] : v[i];
      const int keep_s = up ? src[i + o] : src[i];
      const float send_v = up ? v[i] : v[i + o];
      const int send_s = up ? src[i] : src[i + o];
      const float ov = __shfl_xor_sync(0xffffffffu, send_v, o);
      const int os = __shfl_xor_sync(0xffffffffu, send_s, o);
      const bool take = ov > keep_v || (ov == keep_v && os < keep_s);
      v[i] = take ? ov : keep_v;
      src[i] = take ? os : keep_s;
    }
  }
  best = v[0];
  from = src[0];
}
// The same for 16 items per lane: lanes 2j and 2j+1 both end up with item j.
__device__ __forceinline__ void warp_argmax_items16(float (&v)[16], int lane, float& best, int& from) {
  int src[16];
#pragma unroll
  for (int j = 0; j < 16; ++j) src[j] = lane;
#pragma unroll
  for (int o = 16; o > 1; o >>= 1) {
    const int h = o >> 1;                            // items kept after this step
    const bool up = (lane & o) != 0;
#pragma unroll
    for (int i = 0; i < h; ++i) {
      const float keep_v = up ? v[i + h] : v[i];
      const int keep_s = up ? src[i + h] : src[i];
      const float send_v = up ? v[i] : v[i + h];
      const int send_s = up ? src[i] : src[i + h];
      const float ov = __shfl_xor_sync(0xffffffffu, send_v, o);
      const int os = __shfl_xor_sync(0xffffffffu, send_s, o);
      const bool take = ov > keep_v || (ov == keep_v && os < keep_s);
      v[i] = take ? ov : keep_v;
      src[i] = take ? os : keep_s;
    }
  }
  const float ov = __shfl_xor_sync(0xffffffffu, v[0], 1);
  const int os = __shfl_xor_sync(0xffffffffu, src[0], 1);
  const bool take = ov > v[0] || (ov == v[0] && os < src[0]);
  best = take ? ov : v[0];
  from = take ? os : src[0];
}

// Best (value, lowest index) over the 32 lanes of a warp.
__device__ __forceinline__ void warp_argmax(float& v, int& i) {
#pragma unroll
  for (int off = 16; off > 0; off >>= 1) {
    float ov = __shfl_xor_sync(0xffffffffu, v, off);
    int oi = __shfl_xor_sync(0xffffffffu, i, off);
    if (ov > v || (ov == v && oi < i)) { v = ov; i = oi; }
  }
}

// Applies the epilogue to 16 consecutive tokens (m0 .. m0+15) of output feature n held by this thread.
// b is the bias of feature n (0 when there is none); slot_s holds the K/V slot of every token of the tile.
template <int EPI, typename ActT>
__device__ __forceinline__ void epilogue_chunk(const GemmParams& p, int n, int m0, int M, const float* acc, float b,
                                               float* out_f32, const int* slot_s, int j0) {
  if (n >= p.N) return;
#pragma unroll
  for (int j = 0; j < 16; ++j) {
    const int m = m0 + j;
    if (m >= M) break;
    float v = acc[j] + b;
    if (EPI == EPI_F32) {
      out_f32[(size_t)m * p.N + n] = v;
    } else if (EPI == EPI_ACT) {
      if (p.relu) v = fmaxf(v, 0.f);
      reinterpret_cast<ActT*>(p.out_act)[(size_t)m * p.N + n] = from_f32<ActT>(v);
    } else if (EPI == EPI_SCATTER) {
      const int s = n / p.seg_width, c = n - s * p.seg_width;
      const int row = (s < p.n_direct) ? m : slot_s[j0 + j];
      char* seg_base = p.seg_pair_stride ? static_cast<char*>(p.dst[s & 1]) + (size_t)(s >> 1) * p.seg_pair_stride
                                         : static_cast<char*>(p.dst[s]);
      reinterpret_cast<ActT*>(seg_base)[(size_t)row * p.seg_width + c] = from_f32<ActT>(v);
    }
  }
}

// grid = (ceil(N / 128), ceil(M_cap / ntile), ksplit); block = 256 threads;
// dynamic smem = stages * stage bytes + 1024.
//
// Order of events in a CTA (the part before pdl_wait() overlaps the previous kernel of the stream):
//   barriers, TMEM allocation, pdl_launch;  producer: weight tiles of the first ring round (token tile 0 only);
//   pdl_wait;  token count M;  producer: activation tiles, then the rest of the K loop;  MMA issue;  epilogue.
template <int EPI>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
               const GemmParams p, const int stages) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[MAX_STAGES];
  __shared__ __align__(8) uint64_t bar_empty[MAX_STAGES];
  __shared__ __align__(8) uint64_t bar_acc;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  __shared__ int slot_s[256];
  __shared__ float dval_s[256];   // relaxed verification: score and id of every token's draft
  __shared__ int did_s[256];

  trace_mark(TR_GEMM + EPI, 0);
  const int ntile = p.ntile;
  const int t0 = blockIdx.y * ntile;
  const int n0 = blockIdx.x * BLOCK_N_FEAT;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int quad = warp & 3, grp = warp >> 2;   // accumulator lane quadrant of this warp; column group in the epilogue
  const int b_stage_bytes = ntile * BLOCK_K * 2;
  const int stage_bytes = A_STAGE_BYTES + b_stage_bytes;
  const int kb_total = p.K / BLOCK_K;
  const int ksplit = (EPI == EPI_F32 && p.ksplit > 1) ? p.ksplit : 1;
  const int kb_begin = (int)(((long long)kb_total * blockIdx.z) / ksplit);
  const int kb_end = (int)(((long long)kb_total * (blockIdx.z + 1)) / ksplit);
  const int num_kb = kb_end - kb_begin;
  const int first_round = num_kb < stages ? num_kb : stages;
  const bool early = (blockIdx.y == 0);   // token tile 0 always has work (M >= 1 whenever a result is read)

  const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;   // swizzled tiles need 1024-byte alignment
  // MMA issuers.  Issuing one tcgen05.mma costs its thread 65-80 cycles whatever the tile, so with few tokens (short
  // MMAs) a single issuer, not the tensor pipe or shared memory, sets the pace of the K loop.  Up to four threads in
  // different warps therefore issue side by side: issuer j takes the K blocks j, j + n, j + 2n, ... of this CTA and
  // accumulates them in its own ntile-column region of tensor memory; the epilogue adds the regions up.
  // An issuer waits for ring phase r of a stage only after phase r - 1 has completed (a parity wait two phases ahead
  // would alias): with more than one ring round this holds when the ring depth is a multiple of the issuer count, since
  // the K block that used the stage one round earlier was then this issuer's own.
  int n_issuers = 1;
  {
    const int cap = ntile <= 64 ? 4 : (ntile <= 128 ? 2 : 1);
    for (int cand = 4; cand > 1; cand >>= 1)
      if (cand <= cap && cand <= num_kb && (num_kb <= stages || stages % cand == 0)) { n_issuers = cand; break; }
  }
  uint32_t tmem_cols = 32;
  while (tmem_cols < (uint32_t)(ntile * n_issuers)) tmem_cols <<= 1;

  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_w)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_x)) : "memory");
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    mbar_init(smem_u32(&bar_acc), (uint32_t)n_issuers);
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {   // one full warp allocates the accumulator columns
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(
                     smem_u32(&tmem_base_slot)), "r"(tmem_cols)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  trace_mark(TR_GEMM + EPI, 6);
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  trace_mark(TR_GEMM + EPI, 7);
  const uint32_t tmem_acc = tmem_base_slot;
  // Successors may start now: this CTA already owns its tensor memory, so a later kernel's allocation can
  // never starve it.
  pdl_launch();

  // TMA issue is spread over lane 0 of all eight warps: one thread's bulk-tensor copies are processed one after
  // the other, several threads' copies run side by side.  Stage i of the first ring round belongs to warp i;
  // later rounds are fed by up to four of the warps 0 .. 3.
  if (early && lane == 0) {
    // weights never change: fetch the first ring round before the previous kernel has finished
    for (int i = warp; i < first_round; i += THREADS / 32) {
      const uint32_t bar = smem_u32(&bar_full[i]);
      mbar_expect_tx(bar, (uint32_t)stage_bytes);
      tma_load_2d(smem_base + i * stage_bytes, &map_w, (kb_begin + i) * BLOCK_K, n0, bar);
    }
  }
  const int n = n0 + quad * 32 + lane;
  const float bias_n = (p.bias && n < p.N) ? p.bias[n] : 0.f;   // a weight as well: no dependency

  pdl_wait();
  trace_mark(TR_GEMM + EPI, 1);
  if (early && lane == 0) {
    // activations of the first ring round (the activation buffer is always valid memory; rows beyond M are
    // simply never stored), issued before the token count is known
    for (int i = warp; i < first_round; i += THREADS / 32)
      tma_load_2d(smem_base + i * stage_bytes + A_STAGE_BYTES, &map_x, (kb_begin + i) * BLOCK_K, t0,
                  smem_u32(&bar_full[i]));
  }
  const int M = p.M_ptr ? *p.M_ptr : p.M_host;
  const bool valid = early || (t0 < M);

  if (valid) {
    if (EPI == EPI_SCATTER) {
      for (int j = threadIdx.x; j < ntile; j += THREADS) slot_s[j] = (t0 + j < M) ? p.slot[t0 + j] : 0;
    }
    if (EPI == EPI_ARGMAX && p.draft_val) {
      for (int j = threadIdx.x; j < ntile; j += THREADS) {
        dval_s[j] = (t0 + j < M) ? p.draft_val[t0 + j] : 0.f;
        did_s[j] = (t0 + j < M) ? p.draft_id[t0 + j] : -1;
      }
    }
    if (lane == 0 && warp < 4) {
      // ---- TMA producers: everything that was not issued above ----
      // The producer count divides the ring depth, so producer pw refills the same stages (pw, pw + nprod, ...) round
      // after round and every stage is refilled by one thread only.  Its parity wait on a stage's "empty" barrier is
      // then always for the phase right after the one it waited for last time on that stage.  (With a count that does
      // not divide the depth a producer comes back to a stage only every few rounds; arriving early it would find the
      // barrier an even number of phases behind, take the stale parity for the one it waits for, overwrite a stage
      // that has not been consumed and arm its "full" barrier twice in one phase -- seen as an "unspecified launch
      // failure" with 4 stages, 3 producers and 4 ring rounds.)
      const int pw = warp;
      int nprod = 1;
      for (int cand = 4; cand > 1; --cand)
        if (stages % cand == 0) { nprod = cand; break; }
      const int begin = early ? first_round : 0;
      for (int i = begin + pw; pw < nprod && i < num_kb; i += nprod) {
        const int s = i % stages;
        const uint32_t round = i / stages;
        if (round > 0 && !mbar_wait(smem_u32(&bar_empty[s]), (round - 1) & 1, p.status)) { abort_flag = 1; break; }
        if (*reinterpret_cast<volatile int*>(&abort_flag)) break;
        const uint32_t a_dst = smem_base + s * stage_bytes;
        const uint32_t bar = smem_u32(&bar_full[s]);
        mbar_expect_tx(bar, (uint32_t)stage_bytes);
        tma_load_2d(a_dst, &map_w, (kb_begin + i) * BLOCK_K, n0, bar);
        tma_load_2d(a_dst + A_STAGE_BYTES, &map_x, (kb_begin + i) * BLOCK_K, t0, bar);
      }
      if (warp == 0) trace_mark(TR_GEMM + EPI, 3);
    } else if (warp >= 4 && warp - 4 < n_issuers && lane == 0) {
      // ---- MMA issuers (lane 0 of warps 4 .. 4 + n_issuers - 1) ----
      const int j = warp - 4;
      const uint32_t idesc = make_idesc(BLOCK_N_FEAT, ntile);
      const uint32_t acc_j = tmem_acc + (uint32_t)(j * ntile);
      const uint64_t desc_a0 = make_smem_desc(smem_base);
      const uint64_t desc_b0 = make_smem_desc(smem_base + A_STAGE_BYTES);
      const uint64_t desc_step = (uint64_t)(stage_bytes >> 4);     // stage stride in the (address >> 4) field
      bool ok = true;
      int s = j % stages;
      uint32_t parity = (uint32_t)(j / stages) & 1u;
      for (int i = j; i < num_kb; i += n_issuers) {
        ok = mbar_wait(smem_u32(&bar_full[s]), parity, p.status);
        if (!ok) { abort_flag = 1; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint64_t desc_a = desc_a0 + desc_step * (uint64_t)s, desc_b = desc_b0 + desc_step * (uint64_t)s;
#pragma unroll
        for (int k4 = 0; k4 < BLOCK_K / UMMA_K; ++k4) {
          // advancing 16 bf16 = 32 bytes along K inside the swizzle row: +2 in the (address >> 4) field
          umma_bf16(acc_j, desc_a + 2 * k4, desc_b + 2 * k4, idesc, (i != j || k4 != 0) ? 1u : 0u);
        }
        // the stage is handed back to the producers only if a later K block will land in it
        if (i + stages < num_kb) umma_commit(smem_u32(&bar_empty[s]));
        s += n_issuers;
        while (s >= stages) { s -= stages; parity ^= 1u; }
      }
      // one arrival per issuer: the accumulator barrier fires when every region is complete.  An issuer that gave
      // up still arrives (plainly), so that nobody waits for it; the abort flag tells the epilogue to do nothing.
      if (ok) umma_commit(smem_u32(&bar_acc));
      else asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(&bar_acc)) : "memory");
    }
    __syncwarp();

    // ---- epilogue: all eight warps ----
    bool ready = mbar_wait(smem_u32(&bar_acc), 0, p.status);
    if (*reinterpret_cast<volatile int*>(&abort_flag)) ready = false;
    ready = __syncthreads_and(ready) != 0;     // one decision for the CTA (also makes slot_s visible)
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    trace_mark(TR_GEMM + EPI, 4);
    // The accumulator holds one output feature per TMEM lane and one token per column.  Warp w reads lanes
    // 32 (w % 4) .. +31; the two warps of a quadrant take alternate chunks of 16 columns.  The TMA ring is free
    // once the accumulator barrier has fired and serves as staging memory.
    float* stage = reinterpret_cast<float*>(smem_raw + (smem_base - smem_u32(smem_raw)));
    constexpr int LD = 132;                                // rows stay 16-byte aligned
    const int ntok_all = min(ntile, M - t0);               // valid tokens of this tile (<= 0 only if M == 0)
    const uint32_t tlane = tmem_acc + (static_cast<uint32_t>(quad * 32) << 16);
    if (EPI == EPI_ARGMAX) {
      // No transposition: a warp reduces its 32 features for 16 tokens at a time with a halving exchange, after
      // which lanes 2j and 2j+1 hold the best of token c + j (lowest id on ties).  The four quadrants' results
      // meet in shared memory and one thread per token combines them in ascending feature order.
      float* red_val = stage;                                   // [4][ntile]
      int* red_idx = reinterpret_cast<int*>(stage + 4 * 256);   // [4][ntile]
      int* red_cnt = reinterpret_cast<int*>(stage + 8 * 256);   // [4][ntile] features scoring above the draft
      const bool relaxed = p.draft_val != nullptr;
      if (ready) {
        for (int c = grp * 16; c < ntile && c < ntok_all; c += 32) {
          float acc[16];
          tmem_ld16(tlane + static_cast<uint32_t>(c), acc);
          for (int r = 1; r < n_issuers; ++r) {              // the other issuers' shares of the K range
            float more[16];
            tmem_ld16(tlane + static_cast<uint32_t>(r * ntile + c), more);
#pragma unroll
            for (int j = 0; j < 16; ++j) acc[j] += more[j];
          }
          // columns past the last valid token hold whatever the padded activation rows produced: never stored
#pragma unroll
          for (int j = 0; j < 16; ++j) acc[j] = n < p.N ? acc[j] + bias_n : -INFINITY;
          int my_cnt = 0;
          if (relaxed) {
#pragma unroll
            for (int j = 0; j < 16; ++j) {
              const int tt = c + j;
              const bool above = tt < ntok_all && n < p.N && n != did_s[tt] && acc[j] > dval_s[tt];
              const unsigned int bal = __ballot_sync(0xffffffffu, above);
              if ((lane >> 1) == j) my_cnt = __popc(bal);
            }
          }
          float my_v;
          int my_i;
          warp_argmax_items16(acc, lane, my_v, my_i);
          const int t = c + (lane >> 1);
          if (!(lane & 1) && t < ntok_all) {
            red_val[quad * ntile + t] = my_v;
            red_idx[quad * ntile + t] = n0 + quad * 32 + my_i;
            if (relaxed) red_cnt[quad * ntile + t] = my_cnt;
          }
        }
      }
      trace_mark(TR_GEMM + EPI, 5);
      __syncthreads();
      for (int t = threadIdx.x; t < ntok_all && ready; t += THREADS) {
        float v = red_val[t];
        int idx = red_idx[t];
#pragma unroll
        for (int w = 1; w < 4; ++w) {
          const float ov = red_val[w * ntile + t];
          if (ov > v) { v = ov; idx = red_idx[w * ntile + t]; }
        }
        p.part_val[(size_t)(t0 + t) * gridDim.x + blockIdx.x] = v;
        p.part_idx[(size_t)(t0 + t) * gridDim.x + blockIdx.x] = idx;
        if (relaxed)
          p.part_cnt[(size_t)(t0 + t) * gridDim.x + blockIdx.x] =
              red_cnt[t] + red_cnt[ntile + t] + red_cnt[2 * ntile + t] + red_cnt[3 * ntile + t];
      }
    }
    // Other epilogues: the tile is transposed through shared memory into rows of 128 features per token, in
    // passes of at most 128 tokens (68 KB), so that global stores are 16 bytes per thread and whole rows per warp.
    const int sub = ntile < 128 ? ntile : 128;
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    for (int tb = 0; EPI != EPI_ARGMAX && tb < ntile && tb < ntok_all && ready; tb += sub) {
      const int ntok = min(sub, ntok_all - tb);            // valid tokens of this pass
      const int tg = t0 + tb;                              // packed index of the pass's first token
      if (tb > 0) __syncthreads();                         // previous pass has been read out
      for (int c = grp * 16; c < sub && c < ntok; c += 32) {
        float acc[16];
        tmem_ld16(tlane + static_cast<uint32_t>(tb + c), acc);
        for (int r = 1; r < n_issuers; ++r) {
          float more[16];
          tmem_ld16(tlane + static_cast<uint32_t>(r * ntile + tb + c), more);
#pragma unroll
          for (int j = 0; j < 16; ++j) acc[j] += more[j];
        }
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          if (c + j < ntok) {
            float v = acc[j] + bias_n;
            if (EPI == EPI_ACT && p.relu) v = fmaxf(v, 0.f);
            stage[(c + j) * LD + quad * 32 + lane] = v;
          }
        }
      }
      if (tb == 0) trace_mark(TR_GEMM + EPI, 5);
      __syncthreads();
      if (EPI == EPI_F32) {
        float* out = p.out_f32 + (size_t)blockIdx.z * p.M_cap * p.N;
        const int col = n0 + lane * 4;
        const bool vec = (p.N & 3) == 0;
        for (int r = warp; r < ntok; r += THREADS / 32) {
          const float4 v = *reinterpret_cast<const float4*>(stage + r * LD + lane * 4);
          float* dst = out + (size_t)(tg + r) * p.N + col;
          if (vec && col + 3 < p.N) {
            *reinterpret_cast<float4*>(dst) = v;
          } else {
            if (col < p.N) dst[0] = v.x;
            if (col + 1 < p.N) dst[1] = v.y;
            if (col + 2 < p.N) dst[2] = v.z;
            if (col + 3 < p.N) dst[3] = v.w;
          }
        }
      } else if (EPI == EPI_ACT || EPI == EPI_SCATTER) {
        // two token rows per warp pass: 16 lanes x 8 features = 128 features = 256 bytes of bf16
        const int half = lane >> 4, f0 = (lane & 15) * 8;
        int width = p.N, seg = 0, col0 = n0;
        bf16* base = reinterpret_cast<bf16*>(p.out_act);
        if (EPI == EPI_SCATTER) {           // a 128-feature tile lies inside one segment (seg_width % 128 == 0)
          width = p.seg_width;
          seg = n0 / width;
          col0 = n0 - seg * width;
          base = p.seg_pair_stride ? reinterpret_cast<bf16*>(static_cast<char*>(p.dst[seg & 1]) + (size_t)(seg >> 1) * p.seg_pair_stride)
                                   : reinterpret_cast<bf16*>(p.dst[seg]);
        }
        const bool vec = (width & 7) == 0;
        for (int r = warp * 2 + half; r < ntok; r += THREADS / 16) {
          const float* srow = stage + r * LD + f0;
          const float4 a = *reinterpret_cast<const float4*>(srow);
          const float4 b = *reinterpret_cast<const float4*>(srow + 4);
          const int grow = (EPI == EPI_SCATTER && seg >= p.n_direct) ? slot_s[tb + r] : tg + r;
          bf16* dst = base + (size_t)grow * width + col0 + f0;
          const int lim = p.N - (n0 + f0);                 // features of this lane that exist
          if (vec && lim >= 8) {
            __nv_bfloat162 h0 = __floats2bfloat162_rn(a.x, a.y), h1 = __floats2bfloat162_rn(a.z, a.w);
            __nv_bfloat162 h2 = __floats2bfloat162_rn(b.x, b.y), h3 = __floats2bfloat162_rn(b.z, b.w);
            uint4 u;
            u.x = *reinterpret_cast<unsigned int*>(&h0); u.y = *reinterpret_cast<unsigned int*>(&h1);
            u.z = *reinterpret_cast<unsigned int*>(&h2); u.w = *reinterpret_cast<unsigned int*>(&h3);
            *reinterpret_cast<uint4*>(dst) = u;
          } else {
            const float vals[8] = {a.x, a.y, a.z, a.w, b.x, b.y, b.z, b.w};
#pragma unroll
            for (int t = 0; t < 8; ++t)
              if (t < lim) dst[t] = __float2bfloat16_rn(vals[t]);
          }
        }
      }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
  }
  if (warp == 1) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(tmem_cols) : "memory");
  }
  trace_mark(TR_GEMM + EPI, 2);
}

}  // namespace tc
}  // namespace ad
