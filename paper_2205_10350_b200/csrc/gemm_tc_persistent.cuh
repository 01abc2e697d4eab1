// Output projection fused with the per-tile arg-max for passes with many tokens (hundreds to thousands of packed
// rows): a persistent, warp-specialised, token-stationary tcgen05 GEMM.
//
// Unlike gemm_tc.cuh (weights on the MMA's M side so that a handful of tokens still fill an instruction), the tokens
// are the M side here: D[token, vocabulary row] = sum_k X[token, k] * E[row, k], one token per tensor-memory lane and
// one vocabulary row per column.  The arg-max over vocabulary rows is then a scan over a thread's own columns: no
// exchange between lanes, no shared memory, no barrier.
//
// One CTA per SM owns a contiguous range of (token tile, vocabulary tile) pairs, the vocabulary tile running fastest:
// 128 tokens x 256 vocabulary rows per pair.  The token tile (128 x K BF16, K <= 512) stays in shared memory for all of
// its pairs; only vocabulary rows stream through the ring, 8 bytes of L2 traffic per output instead of 12.  Roles (512
// threads):
//   warps 8 .. 8+S-1, lane 0: producers of the vocabulary ring, one stage each (two 128-row boxes per stage);
//   warp 14, lane 0:          loads the resident token tile whenever the range moves on to the next token tile;
//   warp 15, lane 0:          MMA issuer; the accumulator alternates between two 256-column halves of tensor memory, so
//                             the K loop of pair i + 1 runs while pair i is read out;
//   warps 0-7:                read-out: warp w owns the 32 tokens of lane quadrant w % 4 and the 128 columns w / 4 of
//                             the half, i.e. one 128-row vocabulary tile of the partial arrays; each thread scans its
//                             columns in ascending row order (strict comparison: lowest id wins ties) and writes the
//                             token's (maximum, id[, rows scoring above the draft]) for that tile.
// Every mbarrier wait is bounded in time; a wait that runs out latches AD_ERR_TIMEOUT, raises the CTA's abort flag and
// every role leaves its loop.  No role waits at a block-wide barrier inside the loops.
#pragma once

#include "gemm_tc.cuh"

namespace ad {
namespace tc {

constexpr int P_THREADS = 512;
constexpr int P_TOK = 128;                       // tokens per pair = MMA M
constexpr int P_VOC = 256;                       // vocabulary rows per pair = MMA N
constexpr int P_MAX_KB = 8;                      // K <= 512
constexpr int P_MAX_STAGES = 6;
constexpr int P_A_KB_BYTES = P_TOK * BLOCK_K * 2;   // 16 KiB: one K block of the resident token tile
constexpr int P_B_STAGE_BYTES = P_VOC * BLOCK_K * 2;   // 32 KiB
constexpr int P_READ_WARPS = 8;

__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
  asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}

// Shared memory a launch needs for kb K blocks and `stages` ring stages.
inline size_t vocab_persistent_smem(int kb, int stages) {
  return (size_t)kb * P_A_KB_BYTES + (size_t)stages * P_B_STAGE_BYTES + 1024;
}

// grid = min(SMs, pairs); block = 512 threads; dynamic smem = vocab_persistent_smem(K / 64, stages).
// map_x: box of 128 token rows x 64; map_w: box of 128 vocabulary rows x 64.  p.bias must be null.
__global__ void __launch_bounds__(P_THREADS, 1)
vocab_argmax_persistent_kernel(const __grid_constant__ CUtensorMap map_w, const __grid_constant__ CUtensorMap map_x,
                               const GemmParams p, const int stages) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t bar_full[P_MAX_STAGES];
  __shared__ __align__(8) uint64_t bar_empty[P_MAX_STAGES];
  __shared__ __align__(8) uint64_t a_full, a_empty;
  __shared__ __align__(8) uint64_t acc_full[2];
  __shared__ __align__(8) uint64_t acc_empty[2];
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;

  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const int KB = p.K / BLOCK_K;
  const uint32_t a_base = (smem_u32(smem_raw) + 1023u) & ~1023u;      // resident token tile: KB blocks of 16 KiB
  const uint32_t b_base = a_base + (uint32_t)(KB * P_A_KB_BYTES);     // ring
  constexpr uint32_t TMEM_COLS = 2 * P_VOC;

  if (threadIdx.x == 0) {
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_w)) : "memory");
    asm volatile("prefetch.tensormap [%0];" ::"l"(reinterpret_cast<uint64_t>(&map_x)) : "memory");
    for (int s = 0; s < stages; ++s) {
      mbar_init(smem_u32(&bar_full[s]), 1);
      mbar_init(smem_u32(&bar_empty[s]), 1);
    }
    mbar_init(smem_u32(&a_full), 1);
    mbar_init(smem_u32(&a_empty), 1);
    for (int b = 0; b < 2; ++b) {
      mbar_init(smem_u32(&acc_full[b]), 1);
      mbar_init(smem_u32(&acc_empty[b]), P_READ_WARPS);
    }
    abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 15) {
    asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)),
                 "r"(TMEM_COLS)
                 : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
  }
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
  const uint32_t tmem_acc = tmem_base_slot;
  pdl_launch();
  pdl_wait();

  const int M = p.M_ptr ? *p.M_ptr : p.M_host;
  const int n_vt = (p.N + BLOCK_N_FEAT - 1) / BLOCK_N_FEAT;    // 128-row tiles: the layout of the partial arrays
  const int n_v2 = (p.N + P_VOC - 1) / P_VOC;                  // 256-row tiles of a pair
  const int n_tt = (M + P_TOK - 1) / P_TOK;                    // token tiles that hold tokens
  const long long n_pairs = (long long)n_tt * n_v2;
  const int q_lo = (int)((n_pairs * blockIdx.x) / gridDim.x);
  const int q_hi = (int)((n_pairs * (blockIdx.x + 1)) / gridDim.x);
  const int my_pairs = q_hi - q_lo;
  volatile int* abort_v = &abort_flag;

  if (warp >= 8 && warp < 8 + stages) {
    // ---- ring producers: producer pw owns stage pw and the K blocks pw, pw + S, ... of the CTA's whole sequence ----
    if (lane == 0) {
      const int pw = warp - 8;
      const int total_kb = my_pairs * KB;
      const uint32_t full = smem_u32(&bar_full[pw]), empty = smem_u32(&bar_empty[pw]);
      const uint32_t dst = b_base + (uint32_t)(pw * P_B_STAGE_BYTES);
      for (int g = pw; g < total_kb; g += stages) {
        const int it = g / KB, kb = g - it * KB;
        const int v2 = (q_lo + it) % n_v2;
        const uint32_t round = (uint32_t)(g / stages);
        if (round > 0 && !mbar_wait(empty, (round - 1) & 1u, p.status)) { *abort_v = 1; break; }
        if (*abort_v) break;
        if (pw == 0) trace_mark_role(TR_PV_LOAD, 0);
        mbar_expect_tx(full, (uint32_t)P_B_STAGE_BYTES);
        // a box that starts beyond the last vocabulary row is filled with zeros and still counts its bytes
        tma_load_2d(dst, &map_w, kb * BLOCK_K, v2 * P_VOC, full);
        tma_load_2d(dst + A_STAGE_BYTES, &map_w, kb * BLOCK_K, v2 * P_VOC + BLOCK_N_FEAT, full);
      }
    }
  } else if (warp == 14) {
    // ---- the resident token tile ----
    if (lane == 0) {
      int cur_t = -1;
      uint32_t uses = 0;
      for (int it = 0; it < my_pairs; ++it) {
        const int t = (q_lo + it) / n_v2;
        if (t == cur_t) continue;
        // the MMAs of the previous token tile must have read it for the last time
        if (uses > 0 && !mbar_wait(smem_u32(&a_empty), (uses - 1) & 1u, p.status)) { *abort_v = 1; break; }
        if (*abort_v) break;
        mbar_expect_tx(smem_u32(&a_full), (uint32_t)(KB * P_A_KB_BYTES));
        for (int kb = 0; kb < KB; ++kb)
          tma_load_2d(a_base + (uint32_t)(kb * P_A_KB_BYTES), &map_x, kb * BLOCK_K, t * P_TOK, smem_u32(&a_full));
        cur_t = t;
        ++uses;
      }
    }
  } else if (warp == 15) {
    // ---- MMA issuer ----
    if (lane == 0) {
      const uint32_t idesc = make_idesc(P_TOK, P_VOC);
      const uint64_t desc_a0 = make_smem_desc(a_base);
      const uint64_t desc_b0 = make_smem_desc(b_base);
      const uint64_t a_step = (uint64_t)(P_A_KB_BYTES >> 4), b_step = (uint64_t)(P_B_STAGE_BYTES >> 4);
      bool ok = true;
      int g = 0, cur_t = -1;
      uint32_t uses = 0;
      for (int it = 0; it < my_pairs && ok; ++it) {
        const int b = it & 1;
        const int t = (q_lo + it) / n_v2;
        if (t != cur_t) {
          ok = mbar_wait(smem_u32(&a_full), uses & 1u, p.status);
          cur_t = t;
          ++uses;
        }
        // the half must have been read out (pair it - 2)
        if (ok && it >= 2) ok = mbar_wait(smem_u32(&acc_empty[b]), (uint32_t)((it >> 1) - 1) & 1u, p.status);
        if (!ok || *abort_v) { ok = false; break; }
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const uint32_t acc = tmem_acc + (uint32_t)(b * P_VOC);
        trace_mark_role(TR_PV_ISSUE, 0);
        for (int kb = 0; kb < KB; ++kb, ++g) {
          const int s = g % stages;
          ok = mbar_wait(smem_u32(&bar_full[s]), (uint32_t)(g / stages) & 1u, p.status);
          if (!ok) break;
          asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
          const uint64_t desc_a = desc_a0 + a_step * (uint64_t)kb, desc_b = desc_b0 + b_step * (uint64_t)s;
#pragma unroll
          for (int k4 = 0; k4 < BLOCK_K / UMMA_K; ++k4)
            umma_bf16(acc, desc_a + 2 * k4, desc_b + 2 * k4, idesc, (kb != 0 || k4 != 0) ? 1u : 0u);
          umma_commit(smem_u32(&bar_empty[s]));
        }
        if (!ok) break;
        umma_commit(smem_u32(&acc_full[b]));
        // last pair of this token tile: once these MMAs are done the resident tile may be replaced
        if (it + 1 == my_pairs || (q_lo + it + 1) / n_v2 != t) umma_commit(smem_u32(&a_empty));
        trace_mark_role(TR_PV_ISSUE, 1);
      }
      if (!ok) {   // nobody must be left waiting for an accumulator that will not come
        *abort_v = 1;
        mbar_arrive(smem_u32(&acc_full[0]));
        mbar_arrive(smem_u32(&acc_full[1]));
      }
    }
  } else if (warp < P_READ_WARPS) {
    // ---- read-out: warps 0-7 ----
    const int quad = warp & 3, grp = warp >> 2;
    const bool relaxed = p.draft_val != nullptr;
    int cur_t = -1, did = -1;
    float dval = 0.f;
    for (int it = 0; it < my_pairs; ++it) {
      const int b = it & 1;
      const int q = q_lo + it;
      const int t = q / n_v2, v2 = q - t * n_v2;
      const int tok = t * P_TOK + quad * 32 + lane;              // this thread's token
      const int vt = v2 * 2 + grp;                               // this warp's 128-row tile of the partial arrays
      if (relaxed && t != cur_t) {
        dval = tok < M ? p.draft_val[tok] : 0.f;
        did = tok < M ? p.draft_id[tok] : -1;
      }
      cur_t = t;
      if (!mbar_wait(smem_u32(&acc_full[b]), (uint32_t)(it >> 1) & 1u, p.status)) { *abort_v = 1; break; }
      if (*abort_v) break;
      asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
      if (threadIdx.x == 0) trace_mark_role(TR_PV_EPI, 0);
      const uint32_t taddr = tmem_acc + (static_cast<uint32_t>(quad * 32) << 16) + (uint32_t)(b * P_VOC + grp * BLOCK_N_FEAT);
      const int n_base = vt * BLOCK_N_FEAT;
      float best = -INFINITY;
      int best_n = n_base, cnt = 0;
      for (int c = 0; c < BLOCK_N_FEAT; c += 16) {
        float acc[16];
        tmem_ld16(taddr + static_cast<uint32_t>(c), acc);
#pragma unroll
        for (int j = 0; j < 16; ++j) {
          const int n = n_base + c + j;
          const float val = n < p.N ? acc[j] : -INFINITY;       // rows beyond the vocabulary were zero-filled
          if (relaxed) cnt += (n != did && val > dval) ? 1 : 0;
          if (val > best) { best = val; best_n = n; }
        }
      }
      // this warp has read its share of the half: hand it back to the issuer
      asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
      __syncwarp();
      if (lane == 0) mbar_arrive(smem_u32(&acc_empty[b]));
      if (threadIdx.x == 0) trace_mark_role(TR_PV_EPI, 1);
      if (tok < M && vt < n_vt) {
        const size_t o = (size_t)tok * n_vt + vt;
        p.part_val[o] = best;
        p.part_idx[o] = best_n;
        if (relaxed) p.part_cnt[o] = cnt;
      }
    }
  }
  __syncwarp();
  asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
  __syncthreads();
  if (warp == 15) {
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_acc), "r"(TMEM_COLS) : "memory");
  }
}

}  // namespace tc
}  // namespace ad
