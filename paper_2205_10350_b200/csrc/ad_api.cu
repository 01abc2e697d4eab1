// Host side of the verification-step library: handle, workspace layout, kernel sequencing, CUDA-graph
// replay of the decode loop, and the extern "C" entry points declared in include/aggressive_decoding.h.
#include <math.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <algorithm>
#include <map>
#include <string>
#include <vector>

#include "ad_common.cuh"
#include "attention.cuh"
#include "attention_mma.cuh"
#include "gemm_simt.cuh"
#include "gemm_tc.cuh"
#include "gemm_tc_persistent.cuh"
#include "grid_sync.cuh"
#include "mega.cuh"
#include "steps.cuh"

using namespace ad;

namespace {

enum PassKind { PK_VERIFY = 0, PK_DRAFT = 1, PK_ENCODE = 2, PK_COUNT = 3 };

struct Mat {
  const void* ptr = nullptr;
  int N = 0, K = 0;
  CUtensorMap map;
};
struct ActBuf {
  void* ptr = nullptr;
  int cols = 0;
  // one map per pass kind and token tile: box rows 16, 32, 64, 128, 256 (index log2(rows) - 4), up to the pass's own tile
  CUtensorMap map[PK_COUNT][5];
  const CUtensorMap& map_for(int pk, int tile) const {
    int i = 0;
    while ((16 << i) < tile && i < 4) ++i;
    return map[pk][i];
  }
};
struct EncLayer {
  Mat wqkv, wo, w1, w2;
  const float *bqkv, *bo, *ln1g, *ln1b, *b1, *b2, *ln2g, *ln2b;
};
struct DecLayer {
  Mat wqkv, wo, cq, ckv, co, w1, w2;
  const float *bqkv, *bo, *ln1g, *ln1b, *cbq, *cbkv, *cbo, *ln2g, *ln2b, *b1, *b2, *ln3g, *ln3b;
};
struct Model {
  bool present = false;
  Mat emb;
  std::vector<EncLayer> enc;
  std::vector<DecLayer> dec;
  void* kenc = nullptr;   // [n_dec][B * max_src][d] cross-attention keys
  void* venc = nullptr;
  // the decoder layers' cross-attention key/value projections gathered into one [n_dec * 2d, d] matrix (and their
  // biases into one vector) at ad_create, so that ad_encode projects the encoder memory for all layers in one launch
  Mat ckv_all;
  void* ckv_pack = nullptr;
  float* cbkv_pack = nullptr;
};
struct PassCfg {
  int M_cap = 0;     // packed-token capacity of this pass kind
  int ntile = 16;    // tokens per GEMM tile
  int seg_max = 0;   // longest segment of one row
  int max_split = 1; // largest split-K factor this pass may use (sizes the partial-sum buffer)
  bool shrinking = false;   // set while an input-guided decode loop launches this pass: its blocks shrink every iteration
  PassPlan plan;
  // Split-K factor of a projection that feeds the LayerNorm kernel: enough CTAs to cover the SMs when the
  // token dimension alone gives only a handful of tiles (power of two, divides the K blocks, <= max_split).
  // Token tile for a projection with N output features: the pass's tile, or half of a 256-token tile when the
  // full tile would give fewer CTAs than two per SM (the K loop costs the same per CTA either way).
  // Token tile of a projection with N output features.  Up to 64 tokens: one tile (more, smaller tiles were measured
  // slower for a 40-token block).  Beyond that the pass's kernels are latency-bound and smaller tiles win -- more CTAs,
  // more MMA issuers per CTA, a shorter epilogue each -- until the grids outgrow the SMs; measured per step (base model):
  //   100 / 120 / 128 tokens: 64-token tiles 277 / 289 / 293 us against 305 / 316 / 321 us with one 128-token tile;
  //   200 / 240 tokens: 32-token tiles 331 / 305 us, 64: 344 / 311, 128: 364 / 336, 16: 372;
  //   320 / 400 / 512 tokens: 64-token tiles 366 / 357 / 389 us against 415 / 410 / 458 (128) and 383 / 380 / 410 (32);
  //   800 / 1024 tokens: 64-token tiles 455 / 468 us against 477 / 486 (128);  2048 tokens: 128-token tiles 543 us, 64: 571.
  int tile_for(int N, int n_sms) const {
    if (M_cap <= 64) return ntile;
    if (M_cap <= 128) return 64;
    if (M_cap <= 256) return 32;
    if (M_cap <= 1024) return 64;
    // Inside an input-guided decode loop a block is what is left of the sentence: the packed token count falls with
    // every iteration while the launch shapes stay those of the capacity, so up to 2048 tokens of capacity the loop
    // takes the tile of the sizes it mostly runs at (batch 32, blocks of up to 64: 364 against 382 us per iteration,
    // although one full 2048-token step costs 571 against 543 us).
    if (shrinking && M_cap <= 2048) return 64;
    if (ntile == 256 && ((N + 127) / 128) * ((M_cap + 255) / 256) < 2 * n_sms) return 128;
    return ntile;
  }
  int ksplit_for(int N, int K, int tile) const {
    const int tiles = ((N + 127) / 128) * ((M_cap + tile - 1) / tile);
    const int kb = K / 64;
    int s = 1;
    // Up to 256 tokens: at most one CTA per SM.  (With 128-token tiles a 128-CTA grid of these one-CTA-per-SM kernels ran
    // 16 of its CTAs as a second wave behind the 32 CTAs of the projection before it; with the 32- and 64-token tiles such
    // passes take now the projection before it fills the SMs itself and the full-width split is as fast or faster: big
    // model, 100 tokens, 392 against 417 us per step.)  With many tokens the grid has several waves anyway and the split
    // keeps the K loops short.
    // (a single token tile, up to 64 tokens: 112 -- the big model's 25-token pass loses 4 % with 128 one-K-block CTAs)
    const int cap = M_cap <= 64 ? 112 : (M_cap <= 256 ? 148 : 160);
    while (s * 2 <= max_split && tiles * s * 2 <= cap && kb % (s * 2) == 0) s *= 2;
    return s;
  }
};

// A second set of activation buffers (encoder-pass sized) for work that runs on the side stream.
struct ActSet {
  float *y = nullptr, *pre = nullptr, *pre2 = nullptr;
  ActBuf yb, abuf, hbuf;
  void *qbuf = nullptr, *ktmp = nullptr, *vtmp = nullptr;
};

thread_local std::string g_create_error;

}  // namespace

struct ad_handle {
  ad_model_cfg cfg;
  cudaStream_t stream = nullptr;
  bool bf16 = false;
  size_t esz = 4;            // bytes per activation / weight element
  Model ar, nar;
  PassCfg pass[PK_COUNT];
  int M_all = 0;
  Dims dims;
  DevState st;
  // activations
  float *y = nullptr, *pre = nullptr;
  float* pre2 = nullptr;     // per-head partial sums of an output projection fused into the attention kernel
  ActBuf yb, abuf, hbuf, xg;
  void *qbuf = nullptr, *ktmp = nullptr, *vtmp = nullptr, *kself = nullptr, *vself = nullptr, *encmem = nullptr;
  float* part_val = nullptr;
  int* part_idx = nullptr;
  int* part_cnt = nullptr;   // relaxed verification: per tile and token, other tokens scoring above the draft
  float* draft_val = nullptr;
  int* draft_id = nullptr;
  // The drafter's encoder does not depend on the verifier's: it runs on a side stream with its own activations.
  ActSet side;
  cudaStream_t side_stream = nullptr;
  cudaEvent_t ev_fork = nullptr, ev_join = nullptr;
  int beta = 0;              // 0: exact-match verification; >= 1: relaxed verification (Section 3.2.3)
  float tau = 0.f;
  int n_vtiles = 0;
  float* pe = nullptr;
  int max_pos = 0;
  int* ovr = nullptr;        // [B, max_tgt] staged draft-override stream
  int* host_flag = nullptr;  // pinned, mapped host memory: [0..15] flag words, then the upload area (sources, lengths, caps,
                             // override stream) and the result block of ad_generate
  int* host_flag_dev = nullptr;   // the same memory as the device sees it
  int* up_src = nullptr;     // pinned staging of host-resident inputs
  int* up_len = nullptr;
  int* up_max = nullptr;
  int* up_ovr = nullptr;
  int* down = nullptr;       // result block of finalize_generate_kernel (host view) ...
  int* down_dev = nullptr;   // ... and its device view
  bool defer_status = false; // ad_encode inside ad_generate: no synchronisation of its own
  // Decode loop with small blocks: the accept kernel of iteration i also plans and embeds the block of iteration i + 1
  // (loop_next.source >= 0), so an iteration starts at its first projection; pass_planned tells the pass being enqueued
  // that its plan and embedding already exist.
  NextBlock loop_next = {-1, 0, nullptr, 0, 0};
  bool pass_planned = false;
  bool profiling = false;    // ad_debug_profile_verify: an event in front of every launch
  std::vector<std::pair<std::string, cudaEvent_t>> prof;
  // state
  int B = 0;                 // batch of the last ad_encode
  bool encoded = false;
  int last_vocab_which = -1;
  std::string err;
  struct GraphEntry { cudaGraphExec_t exec; int launches; bool device_loop; };
  std::map<std::string, GraphEntry> graphs;
  cudaEvent_t ev0 = nullptr, ev1 = nullptr, ev2 = nullptr;
  int launches = 0;          // kernels launched by the last ad_generate (direct) or per graph replay
  // Persistent decoder pass (one kernel for the decoder stack + projection): per pass kind, whether it applies and its
  // fixed arguments; device-resident tables of tensor maps (per model) and of per-layer pointers (per pass kind).
  struct MegaPass { bool on = false; mega::Params p; };
  MegaPass mega[PK_COUNT];
  int mega_cs = 0, mega_nc = 0;
  size_t mega_smem = 0;
  CUtensorMap* mega_maps[2] = {nullptr, nullptr};          // [0] verifier, [1] drafter
  mega::LayerPtrs* mega_layers[2] = {nullptr, nullptr};    // [0] verification pass, [1] drafter pass
  float* mega_stats[2] = {nullptr, nullptr};
  unsigned long long* mega_timeline = nullptr;
  unsigned long long cond_handle = 0;   // non-zero only while the body of a device-side `while` node is captured
};

namespace {

#define AD_CUDA(h, call)                                                                      \
  do {                                                                                        \
    cudaError_t e__ = (call);                                                                 \
    if (e__ != cudaSuccess) {                                                                 \
      (h)->err = std::string(#call) + ": " + cudaGetErrorString(e__);                         \
      return AD_ERR_CUDA;                                                                     \
    }                                                                                         \
  } while (0)

int fail(ad_handle* h, int code, const std::string& msg) {
  if (h) h->err = msg; else g_create_error = msg;
  return code;
}

// Counts a kernel launch of this library and, while a profiling pass is active, drops an event in front of it (the
// time between two consecutive events is then the device time of the kernel launched after the first one).
void note_launch(ad_handle* h, const char* what) {
  h->launches++;
  if (h->profiling) {
    cudaEvent_t e = nullptr;
    if (cudaEventCreate(&e) == cudaSuccess) {
      cudaEventRecord(e, h->stream);
      h->prof.emplace_back(what, e);
    }
  }
}

// ---- TMA descriptor encoding through the driver entry point (no link-time dependency on libcuda) ----
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
  static EncodeTiledFn fn = nullptr;
  if (!fn) {
    void* p = nullptr;
    cudaDriverEntryPointQueryResult q;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
        q == cudaDriverEntryPointSuccess)
      fn = reinterpret_cast<EncodeTiledFn>(p);
  }
  return fn;
}

// Row-major bf16 [rows, cols]; box = 64 columns (one 128-byte swizzle row) x box_rows.
bool make_map(CUtensorMap* m, const void* base, int rows, int cols, int box_rows) {
  EncodeTiledFn fn = encode_fn();
  if (!fn) return false;
  cuuint64_t dims[2] = {(cuuint64_t)cols, (cuuint64_t)rows};
  cuuint64_t strides[1] = {(cuuint64_t)cols * 2};
  cuuint32_t box[2] = {64u, (cuuint32_t)box_rows};
  cuuint32_t estr[2] = {1u, 1u};
  CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                  CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                  CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  return r == CUDA_SUCCESS;
}

int pow2ceil(int v) { int p = 1; while (p < v) p <<= 1; return p; }
int clampi(int v, int lo, int hi) { return v < lo ? lo : (v > hi ? hi : v); }
size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

// ---- workspace layout: one bump allocation pass, run with base = null to size it ----
struct Bump {
  char* base;
  size_t off = 0;
  explicit Bump(void* b) : base(static_cast<char*>(b)) {}
  void* take(size_t bytes, size_t align = 1024) {
    off = align_up(off, align);
    void* p = base ? base + off : nullptr;
    off += bytes;
    return p;
  }
};

void plan_take(Bump& bp, PassPlan& pl, int B, int M_cap) {
  pl.M = (int*)bp.take(sizeof(int) * 4, 256);
  pl.seg_off = (int*)bp.take(sizeof(int) * B, 256);
  pl.seg_len = (int*)bp.take(sizeof(int) * B, 256);
  pl.key_base = (int*)bp.take(sizeof(int) * B, 256);
  pl.row_nk = (int*)bp.take(sizeof(int) * B, 256);
  pl.tok_row = (int*)bp.take(sizeof(int) * M_cap, 256);
  pl.tok_pos = (int*)bp.take(sizeof(int) * M_cap, 256);
  pl.tok_id = (int*)bp.take(sizeof(int) * M_cap, 256);
  pl.kv_slot = (int*)bp.take(sizeof(int) * M_cap, 256);
  pl.att_n = (int*)bp.take(sizeof(int) * M_cap, 256);
}

void pass_shapes(const ad_model_cfg& c, PassCfg* pass, int* M_all) {
  const int B = c.max_batch;
  pass[PK_VERIFY].seg_max = c.kmax;
  pass[PK_DRAFT].seg_max = c.max_tgt + 1;
  pass[PK_ENCODE].seg_max = c.max_src;
  int all = 0;
  for (int k = 0; k < PK_COUNT; ++k) {
    pass[k].M_cap = B * pass[k].seg_max;
    pass[k].ntile = clampi(pow2ceil(pass[k].M_cap), 16, 256);
    pass[k].max_split = pass[k].M_cap <= 256 ? 16 : 4;
    if (pass[k].M_cap > all) all = pass[k].M_cap;
  }
  if (!c.has_drafter) { /* the drafter pass is never run; keep its shapes for sizing simplicity */ }
  *M_all = all;
}

size_t layout(ad_handle* h, void* base) {
  const ad_model_cfg& c = h->cfg;
  const int B = c.max_batch, d = c.d_model, F = c.d_ffn;
  const size_t e = h->esz;
  Bump bp(base);
  pass_shapes(c, h->pass, &h->M_all);
  const int M_all = h->M_all, Mv = h->pass[PK_VERIFY].M_cap;
  const int M_tmp = std::max(h->pass[PK_DRAFT].M_cap, h->pass[PK_ENCODE].M_cap);
  h->y = (float*)bp.take(sizeof(float) * (size_t)M_all * d);
  size_t pre_elems = 0;
  for (int k = 0; k < PK_COUNT; ++k) pre_elems = std::max(pre_elems, (size_t)h->pass[k].max_split * h->pass[k].M_cap * d);
  h->pre = (float*)bp.take(sizeof(float) * pre_elems);
  if (h->bf16 && c.n_heads <= 16) h->pre2 = (float*)bp.take(sizeof(float) * (size_t)c.n_heads * M_all * d);
  h->yb.ptr = bp.take(e * (size_t)M_all * d); h->yb.cols = d;
  h->abuf.ptr = bp.take(e * (size_t)M_all * d); h->abuf.cols = d;
  h->hbuf.ptr = bp.take(e * (size_t)M_all * F); h->hbuf.cols = F;
  h->xg.ptr = bp.take(e * (size_t)M_all * d); h->xg.cols = d;
  h->qbuf = bp.take(e * (size_t)M_all * d);
  h->ktmp = bp.take(e * (size_t)M_tmp * d);
  h->vtmp = bp.take(e * (size_t)M_tmp * d);
  h->encmem = bp.take(e * (size_t)h->pass[PK_ENCODE].M_cap * d);
  const size_t self_sz = e * (size_t)c.n_dec * B * c.max_tgt * d;
  h->kself = bp.take(self_sz);
  h->vself = bp.take(self_sz);
  const size_t cross_sz = e * (size_t)c.n_dec * B * c.max_src * d;
  h->ar.kenc = bp.take(cross_sz);
  h->ar.venc = bp.take(cross_sz);
  if (c.has_drafter) {
    h->nar.kenc = bp.take(cross_sz);
    h->nar.venc = bp.take(cross_sz);
  }
  if (c.has_drafter) {
    const int Me = h->pass[PK_ENCODE].M_cap;
    ActSet& sd = h->side;
    sd.y = (float*)bp.take(sizeof(float) * (size_t)Me * d);
    sd.pre = (float*)bp.take(sizeof(float) * (size_t)h->pass[PK_ENCODE].max_split * Me * d);
    if (h->bf16 && c.n_heads <= 16) sd.pre2 = (float*)bp.take(sizeof(float) * (size_t)c.n_heads * Me * d);
    sd.yb.ptr = bp.take(e * (size_t)Me * d); sd.yb.cols = d;
    sd.abuf.ptr = bp.take(e * (size_t)Me * d); sd.abuf.cols = d;
    sd.hbuf.ptr = bp.take(e * (size_t)Me * F); sd.hbuf.cols = F;
    sd.qbuf = bp.take(e * (size_t)Me * d);
    sd.ktmp = bp.take(e * (size_t)Me * d);
    sd.vtmp = bp.take(e * (size_t)Me * d);
  }
  {
    const size_t pack = e * (size_t)c.n_dec * 2 * d * d, bpack = sizeof(float) * (size_t)c.n_dec * 2 * d;
    h->ar.ckv_pack = bp.take(pack); h->ar.cbkv_pack = (float*)bp.take(bpack);
    if (c.has_drafter) { h->nar.ckv_pack = bp.take(pack); h->nar.cbkv_pack = (float*)bp.take(bpack); }
  }
  h->n_vtiles = (c.vocab + 127) / 128;
  h->part_val = (float*)bp.take(sizeof(float) * (size_t)h->n_vtiles * Mv);
  h->part_idx = (int*)bp.take(sizeof(int) * (size_t)h->n_vtiles * Mv);
  h->part_cnt = (int*)bp.take(sizeof(int) * (size_t)h->n_vtiles * Mv);
  h->draft_val = (float*)bp.take(sizeof(float) * (size_t)Mv);
  h->draft_id = (int*)bp.take(sizeof(int) * (size_t)Mv);
  h->max_pos = std::max(c.max_src, c.max_tgt + 1);
  h->pe = (float*)bp.take(sizeof(float) * (size_t)h->max_pos * d);
  h->ovr = (int*)bp.take(sizeof(int) * (size_t)B * c.max_tgt);
  for (int i = 0; i < 2; ++i) {
    h->mega_maps[i] = (CUtensorMap*)bp.take(sizeof(CUtensorMap) * (size_t)(6 * c.n_dec + 1));
    h->mega_layers[i] = (mega::LayerPtrs*)bp.take(sizeof(mega::LayerPtrs) * (size_t)c.n_dec);
    h->mega_stats[i] = (float*)bp.take(sizeof(float) * 2 * (size_t)(d / 128 + 1) * M_all);
  }
  h->mega_timeline = (unsigned long long*)bp.take(sizeof(unsigned long long) * 2 * (size_t)(mega::ST_PER_LAYER * c.n_dec + 1));
  for (int k = 0; k < PK_COUNT; ++k) plan_take(bp, h->pass[k].plan, B, h->pass[k].M_cap);
  DevState& s = h->st;
  auto ints = [&](size_t n) { return (int*)bp.take(sizeof(int) * n, 256); };
  s.len = ints(B); s.last = ints(B); s.fin = ints(B); s.maxlen = ints(B); s.srclen = ints(B);
  s.src = ints((size_t)B * c.max_src);
  s.out_ids = ints((size_t)B * c.max_tgt);
  s.drafts = ints((size_t)B * c.kmax); s.pred = ints((size_t)B * c.kmax); s.n_acc = ints(B);
  s.stat_it = ints(B); s.stat_acc = ints(B); s.stat_off = ints(B);
  s.loop_it = ints(4); s.status = ints(4); s.all_fin = ints(4);
  s.sync_ctr = (unsigned int*)ints((size_t)mega::SYNC_COUNTERS * mega::SYNC_STRIDE);
  s.cross_base = ints(B);
  s.gidx = ints((size_t)B * c.kmax);
  s.enc_slot = ints((size_t)B * c.max_src);
  s.user_k = ints(B); s.user_n = ints(B); s.user_drafts = ints((size_t)B * c.kmax);
  return align_up(bp.off, 1024);
}

int check_cfg(const ad_model_cfg* c, std::string* why) {
  auto bad = [&](const char* m) { *why = m; return AD_ERR_ARG; };
  if (!c) return bad("cfg is null");
  if (c->d_model <= 0 || c->n_heads <= 0 || c->d_model % c->n_heads) return bad("d_model must be a positive multiple of n_heads");
  const int dh = c->d_model / c->n_heads;
  if (dh != 32 && dh != 64) return bad("head dimension must be 32 or 64");
  if (c->d_model > 1024) return bad("d_model must be at most 1024");
  if (c->d_ffn <= 0 || c->vocab <= 4 || c->n_enc < 1 || c->n_dec < 1) return bad("bad model sizes");
  if (c->dtype != AD_DTYPE_FP32 && c->dtype != AD_DTYPE_BF16) return bad("dtype must be AD_DTYPE_FP32 or AD_DTYPE_BF16");
  if (c->dtype == AD_DTYPE_BF16 && (c->d_model % 128 || c->d_ffn % 64)) return bad("BF16 needs d_model to be a multiple of 128 and d_ffn a multiple of 64");
  if (c->max_batch < 1 || c->max_batch > 256) return bad("max_batch must be 1..256");
  if (c->max_src < 1 || c->max_tgt < 1) return bad("max_src and max_tgt must be positive");
  if (c->kmax < 1 || c->kmax > 256 || c->kmax > c->max_tgt) return bad("kmax must be 1..min(256, max_tgt)");
  const int ids[4] = {c->bos, c->pad, c->eos, c->mask};
  for (int i = 0; i < 4; ++i) if (ids[i] < 0 || ids[i] >= c->vocab) return bad("special token id outside the vocabulary");
  if (!(c->ln_eps >= 0.f)) return bad("ln_eps must be non-negative");
  return AD_OK;
}

void weight_counts(const ad_model_cfg& c, size_t* mat, size_t* vec) {
  const size_t d = c.d_model, F = c.d_ffn, V = c.vocab;
  *mat = V * d + (size_t)c.n_enc * (3 * d * d + d * d + 2 * d * F) + (size_t)c.n_dec * (3 * d * d + d * d + d * d + 2 * d * d + d * d + 2 * d * F);
  *vec = (size_t)c.n_enc * (3 * d + d + 2 * d + F + d + 2 * d) + (size_t)c.n_dec * (3 * d + d + 2 * d + d + 2 * d + d + 2 * d + F + d + 2 * d);
}

int bind_model(ad_handle* h, Model& m, const ad_model_weights& w) {
  const ad_model_cfg& c = h->cfg;
  const int d = c.d_model, F = c.d_ffn;
  if (!w.matrices || !w.vectors) return fail(h, AD_ERR_ARG, "weight pointers are null");
  if (reinterpret_cast<uintptr_t>(w.matrices) % 256) return fail(h, AD_ERR_ARG, "weight matrices must be 256-byte aligned");
  const char* mp = static_cast<const char*>(w.matrices);
  const float* vp = w.vectors;
  bool ok = true;
  auto mat = [&](Mat& t, int N, int K) {
    t.ptr = mp; t.N = N; t.K = K;
    mp += (size_t)N * K * h->esz;
    if (h->bf16) ok = ok && make_map(&t.map, t.ptr, N, K, tc::BLOCK_N_FEAT);
  };
  auto vec = [&](const float*& t, int n) { t = vp; vp += n; };
  mat(m.emb, c.vocab, d);
  m.enc.resize(c.n_enc);
  m.dec.resize(c.n_dec);
  for (auto& L : m.enc) {
    mat(L.wqkv, 3 * d, d); mat(L.wo, d, d); mat(L.w1, F, d); mat(L.w2, d, F);
    vec(L.bqkv, 3 * d); vec(L.bo, d); vec(L.ln1g, d); vec(L.ln1b, d); vec(L.b1, F); vec(L.b2, d); vec(L.ln2g, d); vec(L.ln2b, d);
  }
  for (auto& L : m.dec) {
    mat(L.wqkv, 3 * d, d); mat(L.wo, d, d); mat(L.cq, d, d); mat(L.ckv, 2 * d, d); mat(L.co, d, d); mat(L.w1, F, d); mat(L.w2, d, F);
    vec(L.bqkv, 3 * d); vec(L.bo, d); vec(L.ln1g, d); vec(L.ln1b, d); vec(L.cbq, d); vec(L.cbkv, 2 * d); vec(L.cbo, d);
    vec(L.ln2g, d); vec(L.ln2b, d); vec(L.b1, F); vec(L.b2, d); vec(L.ln3g, d); vec(L.ln3b, d);
  }
  if (!ok) return fail(h, AD_ERR_CUDA, "cuTensorMapEncodeTiled failed for a weight matrix");
  m.present = true;
  return AD_OK;
}

// ---- kernel launch helpers -----------------------------------------------------------------------

bool g_use_pdl = true;       // AD_NO_PDL=1 in the environment turns programmatic dependent launch off
bool g_use_graph_encode = true;   // AD_NO_ENCODE_GRAPH=1: launch the encoder kernels directly
bool g_two_stream_encode = true;   // AD_NO_CONCURRENT_ENCODERS=1: the drafter's encoder after the verifier's, on one stream
bool g_use_devloop = true;   // AD_NO_DEVLOOP=1: one graph replay per iteration with host polling instead of a device-side loop
bool g_fuse_attn_proj = true;   // AD_NO_ATTN_PROJ=1: attention and its output projection always as separate kernels
// AD_MEGA=1: run eligible decoder passes (BF16, 64-wide heads, at most 64 packed tokens) as ONE persistent kernel
// instead of the kernel chain.  Off by default: measured on a B200 it is slower than the chain at every shape tried
// (base model: 342 / 360 / 424 / 462 us per verification step for blocks of 1 / 16 / 40 / 64 tokens against 214 / 223 /
// 247 / 258 us; big model, 25 tokens: 537 against 323 us), because a stage that hands its result to other SMs through
// L2 costs about 7 us there (operand staging 1.3-3 us, MMA hand-over 0.6, tensor-memory read-out 0.3, cluster hand-shake
// 0.8-1.2, reduction and epilogue 1-1.7, release 0.5, propagation 0.7) against about 3.7 us per kernel of the chain.
bool g_use_mega = false;

// Launches `kernel` so that it may begin while its predecessor in the stream still runs (the kernels
// themselves wait with griddepcontrol.wait before touching anything a predecessor writes).
template <typename... KArgs, typename... Args>
cudaError_t launch_k(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = g_use_pdl ? 1 : 0;
  return cudaLaunchKernelEx(&cfg, kernel, KArgs(std::forward<Args>(args))...);
}

// Per-device caches (a process may hold handles on several GPUs): SM count, and which kernels already had their
// dynamic shared-memory limit raised on that device (the attribute is per device, not per process).
constexpr int kMaxDevices = 64;
int current_device() {
  int dev = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) dev = 0;
  return dev;
}
int num_sms() {
  static int n[kMaxDevices] = {};
  const int dev = current_device();
  if (!n[dev]) {
    cudaDeviceGetAttribute(&n[dev], cudaDevAttrMultiProcessorCount, dev);
    if (n[dev] <= 0) n[dev] = 148;
  }
  return n[dev];
}

// Ring depth: as deep as ~200 KB of shared memory allows when the grid fits one wave; with more CTAs than SMs,
// half of that so that two CTAs share an SM: up to twice the SM count the whole grid is then resident at once,
// beyond that one CTA's prologue and epilogue overlap the other's K loop.
int tc_stages(int ntile, int kb, int n_ctas) {
  const int stage = tc::A_STAGE_BYTES + ntile * tc::BLOCK_K * 2;
  const int budget = n_ctas > num_sms() ? 100 * 1024 : 200 * 1024;
  int s = clampi(budget / stage, 1, tc::MAX_STAGES);
  if (s >= kb) return kb > 0 ? kb : 1;
  // several ring rounds: the kernel's producer count divides the depth, so avoid the prime depths 5 and 7
  if (s == 5 || s == 7) --s;
  return s;
}

template <int EPI>
cudaError_t launch_tc(cudaStream_t st, const CUtensorMap& mw, const CUtensorMap& mx, const GemmParams& p, int M_cap) {
  static bool attr_set[kMaxDevices] = {};
  const int dev = current_device();
  if (!attr_set[dev]) {
    cudaError_t e = cudaFuncSetAttribute(tc::gemm_tc_kernel<EPI>, cudaFuncAttributeMaxDynamicSharedMemorySize, 204 * 1024);
    if (e != cudaSuccess) return e;
    attr_set[dev] = true;
  }
  const int ksplit = (EPI == EPI_F32 && p.ksplit > 1) ? p.ksplit : 1;
  dim3 grid((p.N + 127) / 128, (M_cap + p.ntile - 1) / p.ntile, ksplit);
  const int stages = tc_stages(p.ntile, (p.K / tc::BLOCK_K) / ksplit, grid.x * grid.y * grid.z);
  // the ring doubles as the epilogue's transposition buffer (up to 128 rows of 132 floats)
  const size_t ring = (size_t)stages * (tc::A_STAGE_BYTES + p.ntile * tc::BLOCK_K * 2);
  const size_t smem = std::max(ring, (size_t)std::min(p.ntile, 128) * 132 * sizeof(float)) + 1024;
  return launch_k(tc::gemm_tc_kernel<EPI>, grid, dim3(tc::THREADS), smem, st, mw, mx, p, stages);
}

// Projection + arg-max over many tokens: the persistent token-stationary kernel (one CTA per SM, 128-token tiles
// resident in shared memory, read-out of one tile under the K loop of the next) once there are at least `min_pairs_per_sm`
// (128 token x 256 vocabulary row) pairs per SM; AD_NO_PERSISTENT_VOCAB=1 keeps the one-tile-per-CTA kernel.
bool vocab_goes_persistent(int K, int N, int M_cap, const float* bias) {
  static const bool enabled = [] { const char* e = getenv("AD_NO_PERSISTENT_VOCAB"); return !(e && e[0] == '1'); }();
  if (!enabled || bias || K % tc::BLOCK_K || K / tc::BLOCK_K > tc::P_MAX_KB) return false;
  const long pairs = (long)((N + tc::P_VOC - 1) / tc::P_VOC) * ((M_cap + tc::P_TOK - 1) / tc::P_TOK);
  return pairs >= (long)num_sms();
}
// mx128: the token operand's map with a 128-row box.
cudaError_t launch_vocab_persistent(cudaStream_t st, const CUtensorMap& mw, const CUtensorMap& mx128, const GemmParams& p, int M_cap) {
  static bool attr_set[kMaxDevices] = {};
  const int dev = current_device();
  constexpr int kSmemLimit = 227 * 1024 - 512;   // the kernel's static shared memory is a few hundred bytes
  if (!attr_set[dev]) {
    cudaError_t e = cudaFuncSetAttribute(tc::vocab_argmax_persistent_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kSmemLimit);
    if (e != cudaSuccess) return e;
    attr_set[dev] = true;
  }
  const int kb = p.K / tc::BLOCK_K;
  const int stages = clampi((kSmemLimit - 1024 - kb * tc::P_A_KB_BYTES) / tc::P_B_STAGE_BYTES, 1, tc::P_MAX_STAGES);
  const long pairs = (long)((p.N + tc::P_VOC - 1) / tc::P_VOC) * ((M_cap + tc::P_TOK - 1) / tc::P_TOK);
  const int grid = (int)std::min<long>(pairs, num_sms());
  return launch_k(tc::vocab_argmax_persistent_kernel, dim3(grid), dim3(tc::P_THREADS), tc::vocab_persistent_smem(kb, stages), st, mw, mx128, p,
                  stages);
}

template <int EPI>
cudaError_t launch_simt(cudaStream_t st, const void* w, const void* x, const GemmParams& p, int M_cap) {
  dim3 grid((p.N + 127) / 128, (M_cap + simt::TOK - 1) / simt::TOK);
  return launch_k(simt::gemm_f32_kernel<EPI>, grid, dim3(128), 0, st, (const float*)w, (const float*)x, p);
}

int gemm(ad_handle* h, int epi, const Mat& W, const ActBuf& X, int pk, const int* M_ptr, int M_cap, GemmParams p) {
  p.K = W.K; p.N = W.N; p.M_ptr = M_ptr; p.M_cap = M_cap; p.status = h->st.status;
  cudaError_t e;
  {
    static const char* epi_name[4] = {"gemm_f32_partials", "gemm_act", "gemm_scatter", "gemm_vocab_argmax"};
    char nm[64];
    snprintf(nm, sizeof(nm), "%s N%d K%d", epi_name[epi & 3], W.N, W.K);
    note_launch(h, nm);
  }
  if (h->bf16) {
    p.ntile = h->pass[pk].tile_for(W.N, num_sms());
    const CUtensorMap& mx = X.map_for(pk, p.ntile);
    if (epi != EPI_F32) p.ksplit = 1;
    switch (epi) {
      case EPI_F32: e = launch_tc<EPI_F32>(h->stream, W.map, mx, p, M_cap); break;
      case EPI_ACT: e = launch_tc<EPI_ACT>(h->stream, W.map, mx, p, M_cap); break;
      case EPI_SCATTER: e = launch_tc<EPI_SCATTER>(h->stream, W.map, mx, p, M_cap); break;
      default:
        // (a pass with a 256-token tile also has the 128-row map of its token operand)
        e = (h->pass[pk].ntile == 256 && vocab_goes_persistent(W.K, W.N, M_cap, p.bias))
                ? launch_vocab_persistent(h->stream, W.map, X.map_for(pk, tc::P_TOK), p, M_cap)
                : launch_tc<EPI_ARGMAX>(h->stream, W.map, mx, p, M_cap);
        break;
    }
  } else {
    p.ntile = simt::TOK;
    switch (epi) {
      case EPI_F32: e = launch_simt<EPI_F32>(h->stream, W.ptr, X.ptr, p, M_cap); break;
      case EPI_ACT: e = launch_simt<EPI_ACT>(h->stream, W.ptr, X.ptr, p, M_cap); break;
      case EPI_SCATTER: e = launch_simt<EPI_SCATTER>(h->stream, W.ptr, X.ptr, p, M_cap); break;
      default: e = launch_simt<EPI_ARGMAX>(h->stream, W.ptr, X.ptr, p, M_cap); break;
    }
  }
  if (e != cudaSuccess) return fail(h, AD_ERR_CUDA, std::string("GEMM launch: ") + cudaGetErrorString(e));
  return AD_OK;
}

template <typename T, int D, int Q, bool FUSE = false, int MINB = 1>
cudaError_t launch_attention(dim3 grid, dim3 block, cudaStream_t st, const AttnParams& p) {
  constexpr size_t smem = att_smem_bytes<D, Q>();
  static bool attr_set[kMaxDevices] = {};
  const int dev = current_device();
  if (!attr_set[dev] && smem > 48 * 1024) {
    cudaError_t e = cudaFuncSetAttribute(attention_kernel<T, D, Q, FUSE, MINB>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
  }
  attr_set[dev] = true;
  return launch_k(attention_kernel<T, D, Q, FUSE, MINB>, grid, block, smem, st, p);
}

int attention(ad_handle* h, const PassCfg& pc, const void* q, const void* k, const void* v, void* out,
              const int* key_base, const int* nkeys_tok, const int* nkeys_row, int max_keys,
              const float* q_bias = nullptr, int q_nsplit = 0, const Mat* wo = nullptr, bool* fused = nullptr) {
  const ad_model_cfg& c = h->cfg;
  AttnParams p;
  p.q = q; p.k = k; p.v = v; p.out = out;
  p.q_part = q_nsplit > 0 ? h->pre : nullptr; p.q_bias = q_bias; p.q_nsplit = q_nsplit;
  p.q_stride = (size_t)pc.M_cap * c.d_model;
  p.seg_off = pc.plan.seg_off; p.seg_len = pc.plan.seg_len;
  p.key_base = key_base; p.nkeys_tok = nkeys_tok; p.nkeys_row = nkeys_row;
  p.d = c.d_model;
  // one query per warp while the grid stays within a couple of waves, eight when there are many queries
  const int dh = c.d_model / c.n_heads;
  const bool many = (long long)h->dims.B * c.n_heads * ((pc.seg_max + 7) / 8) > 3LL * num_sms();
  p.scale = 1.0f / sqrtf((float)dh);
  // Tensor-core kernel when there are thousands of queries or rows may hold hundreds of keys (max_keys: the
  // capacity, known on the host); the FFMA kernel spreads few queries and few keys over more CTAs.
  if (h->bf16 && dh == 64 && max_keys >= 256) {
    // rows may hold hundreds of keys: the keys of a row are spread over the warps of a CTA (whole 64-key tiles per warp),
    // 1, 2 or 4 query tiles of 16 per CTA depending on how many queries a row can have
    const int qt = pc.seg_max <= 16 ? 1 : (pc.seg_max <= 32 ? 2 : 4);
    const int nw = qt == 4 ? 4 : 8;
    p.qchunks = (pc.seg_max + 16 * qt - 1) / (16 * qt);
    note_launch(h, "attention_mma_wide");
    const dim3 mgrid(h->dims.B * p.qchunks, c.n_heads);
    const size_t smem = (size_t)nw * AM_TILE_BYTES + AM_Q_BYTES;
    static bool attr_set[kMaxDevices] = {};
    const int dev = current_device();
    cudaError_t em = cudaSuccess;
    if (!attr_set[dev]) {
      em = cudaFuncSetAttribute(attention_mma_wide_kernel<1, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 8 * AM_TILE_BYTES + AM_Q_BYTES);
      if (em == cudaSuccess) em = cudaFuncSetAttribute(attention_mma_wide_kernel<2, 8>, cudaFuncAttributeMaxDynamicSharedMemorySize, 8 * AM_TILE_BYTES + AM_Q_BYTES);
      if (em == cudaSuccess) em = cudaFuncSetAttribute(attention_mma_wide_kernel<4, 4>, cudaFuncAttributeMaxDynamicSharedMemorySize, 4 * AM_TILE_BYTES + AM_Q_BYTES);
      if (em != cudaSuccess) return fail(h, AD_ERR_CUDA, std::string("attention attribute: ") + cudaGetErrorString(em));
      attr_set[dev] = true;
    }
    if (qt == 1) em = launch_k(attention_mma_wide_kernel<1, 8>, mgrid, dim3(256), smem, h->stream, p);
    else if (qt == 2) em = launch_k(attention_mma_wide_kernel<2, 8>, mgrid, dim3(512), smem, h->stream, p);
    else em = launch_k(attention_mma_wide_kernel<4, 4>, mgrid, dim3(512), smem, h->stream, p);
    if (em != cudaSuccess) return fail(h, AD_ERR_CUDA, std::string("attention launch: ") + cudaGetErrorString(em));
    return AD_OK;
  }
  // Tensor-core kernel when there are thousands of queries; the FFMA kernel spreads few queries and few keys over more CTAs.
  if (h->bf16 && dh == 64 && many) {
    // rows with few queries: warps share a 16-query tile and split the keys (2 or 4 key groups)
    const int ng = pc.seg_max <= 16 ? 4 : (pc.seg_max <= 32 ? 2 : 1);
    const int qcta = AM_Q / ng;
    p.qchunks = (pc.seg_max + qcta - 1) / qcta;
    note_launch(h, "attention_mma");
    const dim3 mgrid(h->dims.B * p.qchunks, c.n_heads);
    cudaError_t em;
    if (ng == 4) em = launch_k(attention_mma_kernel<4>, mgrid, dim3(128), 0, h->stream, p);
    else if (ng == 2) em = launch_k(attention_mma_kernel<2>, mgrid, dim3(128), 0, h->stream, p);
    else em = launch_k(attention_mma_kernel<1>, mgrid, dim3(128), 0, h->stream, p);
    if (em != cudaSuccess) return fail(h, AD_ERR_CUDA, std::string("attention launch: ") + cudaGetErrorString(em));
    return AD_OK;
  }
  const int qpw = many ? 8 : 1;
  p.qchunks = (pc.seg_max + 8 * qpw - 1) / (8 * qpw);
  dim3 grid(h->dims.B * p.qchunks, c.n_heads);
  const dim3 block(256);
  cudaError_t e;
#define AD_ATT(T, D, Q) launch_attention<T, D, Q>(grid, block, h->stream, p)
  // few queries, 64-wide heads: the output projection rides along (one partial sum per head for the LayerNorm kernel)
  const bool fuse = g_fuse_attn_proj && wo && fused && h->pre2 && h->bf16 && dh == 64 && !many && c.n_heads <= pc.max_split &&
                    c.n_heads <= 16 && c.d_model % 128 == 0;
  if (fused) *fused = fuse;
  note_launch(h, fuse ? "attention+out_proj" : "attention");
  if (fuse) {
    p.wo = (const bf16*)wo->ptr; p.o_part = h->pre2; p.o_stride = (size_t)pc.M_cap * c.d_model;
    // more CTAs than SMs: the two-CTAs-per-SM build, so that the grid is still one wave
    e = (long)grid.x * grid.y > num_sms() ? launch_attention<bf16, 64, 1, true, 2>(grid, block, h->stream, p)
                                           : launch_attention<bf16, 64, 1, true, 1>(grid, block, h->stream, p);
  } else if (h->bf16) {
    if (dh == 64) e = many ? AD_ATT(bf16, 64, 8) : AD_ATT(bf16, 64, 1);
    else e = many ? AD_ATT(bf16, 32, 8) : AD_ATT(bf16, 32, 1);
  } else {
    if (dh == 64) e = many ? AD_ATT(float, 64, 8) : AD_ATT(float, 64, 1);
    else e = many ? AD_ATT(float, 32, 8) : AD_ATT(float, 32, 1);
  }
#undef AD_ATT
  if (e != cudaSuccess) return fail(h, AD_ERR_CUDA, std::string("attention launch: ") + cudaGetErrorString(e));
  return AD_OK;
}

// y = LN(sum of the nsplit partial projections in `pre` + bias + y)
int layernorm(ad_handle* h, const PassCfg& pc, int nsplit, const float* bias, const float* g, const float* b,
              const float* partials = nullptr) {
  const float* pre_src = partials ? partials : h->pre;
  const int d = h->cfg.d_model;
  dim3 grid(pc.M_cap);
  const size_t stride = (size_t)pc.M_cap * d;
  note_launch(h, "residual+layernorm");
  cudaError_t e;
  // many tokens: a warp per token (measured: 1024 tokens 458 us per step with a CTA per token against 467 us, 2048 tokens 582 against 543 us)
  if (pc.M_cap >= 1536 && nsplit <= 4 && d % 128 == 0 && d <= 1024) {
    dim3 rgrid((pc.M_cap + 7) / 8);
    if (h->bf16) e = launch_k(layernorm_rows_kernel<bf16>, rgrid, dim3(256), 0, h->stream, (const int*)pc.plan.M, pre_src, nsplit, stride, bias,
                              (const float*)h->y, g, b, d, h->cfg.ln_eps, h->y, (bf16*)h->yb.ptr);
    else e = launch_k(layernorm_rows_kernel<float>, rgrid, dim3(256), 0, h->stream, (const int*)pc.plan.M, pre_src, nsplit, stride, bias,
                      (const float*)h->y, g, b, d, h->cfg.ln_eps, h->y, (float*)h->yb.ptr);
  } else if (h->bf16 && d > 512) e = launch_k(layernorm_kernel<bf16, 256>, grid, dim3(256), 0, h->stream, (const int*)pc.plan.M, pre_src, nsplit, stride, bias,
                            (const float*)h->y, g, b, d, h->cfg.ln_eps, h->y, (bf16*)h->yb.ptr);
  else if (h->bf16) e = launch_k(layernorm_kernel<bf16>, grid, dim3(128), 0, h->stream, (const int*)pc.plan.M, pre_src, nsplit, stride, bias,
                            (const float*)h->y, g, b, d, h->cfg.ln_eps, h->y, (bf16*)h->yb.ptr);
  else e = launch_k(layernorm_kernel<float>, grid, dim3(128), 0, h->stream, (const int*)pc.plan.M, pre_src, nsplit, stride, bias,
                    (const float*)h->y, g, b, d, h->cfg.ln_eps, h->y, (float*)h->yb.ptr);
  if (e != cudaSuccess) return fail(h, AD_ERR_CUDA, std::string("layernorm launch: ") + cudaGetErrorString(e));
  return AD_OK;
}

// Projection whose consumer is the residual + LayerNorm kernel: written as split-K partial sums, bias left to
// the consumer.  Returns the number of partials through *nsplit.
int gemm_to_ln(ad_handle* h, const Mat& W, const ActBuf& X, int pk, int* nsplit) {
  PassCfg& pc = h->pass[pk];
  GemmParams o = {};
  o.out_f32 = h->pre;
  o.ksplit = h->bf16 ? pc.ksplit_for(W.N, W.K, pc.tile_for(W.N, num_sms())) : 1;
  *nsplit = o.ksplit;
  return gemm(h, EPI_F32, W, X, pk, pc.plan.M, pc.M_cap, o);
}

int embed(ad_handle* h, const PassCfg& pc, const Model& m) {
  const int d = h->cfg.d_model;
  const float sc = sqrtf((float)d);
  note_launch(h, "embed");
  cudaError_t e;
  if (h->bf16) e = launch_k(embed_kernel<bf16, bf16>, dim3(pc.M_cap), dim3(128), 0, h->stream, pc.plan, (const bf16*)m.emb.ptr, (const float*)h->pe, d, sc, h->y, (bf16*)h->yb.ptr);
  else e = launch_k(embed_kernel<float, float>, dim3(pc.M_cap), dim3(128), 0, h->stream, pc.plan, (const float*)m.emb.ptr, (const float*)h->pe, d, sc, h->y, (float*)h->yb.ptr);
  if (e != cudaSuccess) return fail(h, AD_ERR_CUDA, std::string("embed launch: ") + cudaGetErrorString(e));
  return AD_OK;
}

#define AD_TRY(x) do { int rc__ = (x); if (rc__ != AD_OK) return rc__; } while (0)

// Self-attention sublayer + FFN shared by the encoder and decoder layers.
int self_attention_sublayer(ad_handle* h, int pk, const Mat& wqkv, const float* bqkv, const Mat& wo, const float* bo,
                            const float* lng, const float* lnb, void* kbuf, void* vbuf) {
  PassCfg& pc = h->pass[pk];
  GemmParams p = {};
  p.bias = bqkv; p.dst[0] = h->qbuf; p.dst[1] = kbuf; p.dst[2] = vbuf; p.seg_width = h->cfg.d_model; p.n_direct = 1;
  p.slot = pc.plan.kv_slot;
  AD_TRY(gemm(h, EPI_SCATTER, wqkv, h->yb, pk, pc.plan.M, pc.M_cap, p));
  bool fused = false;
  AD_TRY(attention(h, pc, h->qbuf, kbuf, vbuf, h->abuf.ptr, pc.plan.key_base, pc.plan.att_n, pc.plan.row_nk,
                   pk == PK_VERIFY ? h->dims.max_tgt : pc.seg_max, nullptr, 0, &wo, &fused));
  if (fused) return layernorm(h, pc, h->cfg.n_heads, bo, lng, lnb, h->pre2);
  int ns = 1;
  AD_TRY(gemm_to_ln(h, wo, h->abuf, pk, &ns));
  return layernorm(h, pc, ns, bo, lng, lnb);
}

int ffn_sublayer(ad_handle* h, int pk, const Mat& w1, const float* b1, const Mat& w2, const float* b2, const float* lng,
                 const float* lnb) {
  PassCfg& pc = h->pass[pk];
  GemmParams a = {};
  a.bias = b1; a.relu = 1; a.out_act = h->hbuf.ptr;
  AD_TRY(gemm(h, EPI_ACT, w1, h->yb, pk, pc.plan.M, pc.M_cap, a));
  int ns = 1;
  AD_TRY(gemm_to_ln(h, w2, h->hbuf, pk, &ns));
  return layernorm(h, pc, ns, b2, lng, lnb);
}


// ---- persistent decoder pass ---------------------------------------------------------------------------------

// Cluster size for the K split of the projections: the K blocks of d_model and of d_ffn must divide evenly.
int mega_cluster_size(const ad_model_cfg& c) {
  for (int cs : {8, 4}) {
    const int kd = c.d_model / 64, kf = c.d_ffn / 64;
    if (kd % cs == 0 && kf % cs == 0) return cs;
  }
  return 0;
}

// Fills the device tables and the fixed kernel arguments of the persistent decoder pass; leaves mega[pk].on false for
// pass kinds (or models, or devices) it does not apply to.  Runs once, from ad_create.
int mega_setup(ad_handle* h) {
  const ad_model_cfg& c = h->cfg;
  if (!g_use_mega || !h->bf16 || c.d_model / c.n_heads != 64 || c.d_model % 128 || c.d_ffn % 128) return AD_OK;
  if (mega::ST_PER_LAYER * c.n_dec + 1 > mega::SYNC_COUNTERS) return AD_OK;
  const int cs = mega_cluster_size(c);
  if (!cs) return AD_OK;
  // shared memory: alignment slack + weight ring + work area (see the kernel), sized for the larger of the two passes
  int max_optin = 0, dev = current_device();
  cudaDeviceGetAttribute(&max_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
  int cap = 0;
  for (int pk : {PK_VERIFY, PK_DRAFT})
    if (h->pass[pk].M_cap <= mega::NT_MAX && (pk == PK_VERIFY || c.has_drafter)) cap = std::max(cap, h->pass[pk].M_cap);
  if (cap == 0) return AD_OK;
  const int ntcap = (cap + 15) / 16 * 16;
  const int b_bytes = (std::max(c.d_model, c.d_ffn) / 64 / cs) * ntcap * 128;
  const int red_bytes = ntcap * mega::RED_LD * 4;
  const int work = std::max(std::max(b_bytes + 2 * red_bytes, (c.d_model / 64) * ntcap * 128), mega::ATT_SMEM);
  int ring = (max_optin - 1024 - work - 13 * 1024) / mega::TILE_A;     // 13 KB: the kernel's static control block
  if (ring > mega::MAX_RING) ring = mega::MAX_RING;
  if (ring < 4) return AD_OK;
  const size_t smem = 1024 + (size_t)ring * mega::TILE_A + (size_t)work;
  if (cudaFuncSetAttribute(mega::decoder_pass_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) != cudaSuccess) {
    cudaGetLastError();
    return AD_OK;
  }
  // how many clusters the device holds at once
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(cs * 64); cfg.blockDim = dim3(mega::THREADS); cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr; cfg.numAttrs = 1;
  int n_clusters = 0;
  if (cudaOccupancyMaxActiveClusters(&n_clusters, mega::decoder_pass_kernel, &cfg) != cudaSuccess || n_clusters < 2) {
    cudaGetLastError();
    return AD_OK;
  }
  h->mega_cs = cs; h->mega_nc = n_clusters; h->mega_smem = smem;

  const int d = c.d_model, L = c.n_dec;
  const size_t self_layer = (size_t)c.max_tgt * c.max_batch * d * h->esz;
  const size_t cross_layer = (size_t)c.max_src * c.max_batch * d * h->esz;
  for (int which = 0; which < 2; ++which) {          // 0: verification pass (verifier), 1: drafter pass (drafter)
    Model& m = which == 0 ? h->ar : h->nar;
    if (!m.present) continue;
    const int pk = which == 0 ? PK_VERIFY : PK_DRAFT;
    if (h->pass[pk].M_cap > mega::NT_MAX) continue;
    std::vector<CUtensorMap> maps((size_t)6 * L + 1);
    std::vector<mega::LayerPtrs> lp((size_t)L);
    for (int l = 0; l < L; ++l) {
      DecLayer& D = m.dec[l];
      const Mat* mats[6] = {&D.wqkv, &D.wo, &D.cq, &D.co, &D.w1, &D.w2};
      for (int i = 0; i < 6; ++i) maps[(size_t)6 * l + i] = mats[i]->map;
      mega::LayerPtrs& P = lp[l];
      P.bqkv = D.bqkv; P.bo = D.bo; P.ln1g = D.ln1g; P.ln1b = D.ln1b; P.cbq = D.cbq; P.cbo = D.cbo; P.ln2g = D.ln2g; P.ln2b = D.ln2b;
      P.b1 = D.b1; P.b2 = D.b2; P.ln3g = D.ln3g; P.ln3b = D.ln3b;
      P.kself = (bf16*)(which == 0 ? (char*)h->kself + l * self_layer : (char*)h->ktmp);
      P.vself = (bf16*)(which == 0 ? (char*)h->vself + l * self_layer : (char*)h->vtmp);
      P.kenc = (const bf16*)((char*)m.kenc + l * cross_layer);
      P.venc = (const bf16*)((char*)m.venc + l * cross_layer);
    }
    maps[(size_t)6 * L] = m.emb.map;
    AD_CUDA(h, cudaMemcpyAsync(h->mega_maps[which], maps.data(), sizeof(CUtensorMap) * maps.size(), cudaMemcpyHostToDevice, h->stream));
    AD_CUDA(h, cudaMemcpyAsync(h->mega_layers[which], lp.data(), sizeof(mega::LayerPtrs) * lp.size(), cudaMemcpyHostToDevice, h->stream));
    AD_CUDA(h, cudaStreamSynchronize(h->stream));     // the host vectors go out of scope
    mega::Params& p = h->mega[pk].p;
    p = mega::Params{};
    p.d = d; p.H = c.n_heads; p.F = c.d_ffn; p.V = c.vocab; p.L = L;
    p.qchunks = (h->pass[pk].seg_max + 7) / 8;
    p.maps = h->mega_maps[which]; p.layers = h->mega_layers[which];
    p.plan = h->pass[pk].plan;
    p.cross_base = h->st.cross_base; p.srclen = h->st.srclen;
    p.emb = (const bf16*)m.emb.ptr; p.pe = h->pe;
    p.emb_scale = sqrtf((float)d); p.eps = c.ln_eps; p.att_scale = 1.0f / sqrtf(64.f);
    p.x[0] = h->y; p.x[1] = h->pre;
    p.stats[0] = h->mega_stats[0]; p.stats[1] = h->mega_stats[1];
    p.M_cap = h->pass[pk].M_cap;
    p.q = (bf16*)h->qbuf; p.attn = (bf16*)h->abuf.ptr; p.hid = (bf16*)h->hbuf.ptr;
    p.yb_out = (bf16*)(which == 0 ? h->yb.ptr : h->xg.ptr);
    p.vocab_M = which == 0 ? nullptr : h->pass[PK_VERIFY].plan.M;
    p.vocab_rows = which == 0 ? nullptr : h->st.gidx;
    p.part_val = h->part_val; p.part_idx = h->part_idx; p.n_vtiles = h->n_vtiles;
    p.sync_ctr = h->st.sync_ctr; p.status = h->st.status;
    p.ring = ring; p.b_bytes = b_bytes; p.red_bytes = red_bytes;
    p.timeline = nullptr;
    h->mega[pk].on = true;
  }
  return AD_OK;
}

bool mega_applies(const ad_handle* h, int pk) {
  return h->mega[pk].on && !(pk == PK_VERIFY && h->beta >= 1);
}

// One launch: decoder stack of pass pk and the projection's per-tile arg-max partials.
int mega_launch(ad_handle* h, int pk) {
  mega::Params p = h->mega[pk].p;
  p.B = h->dims.B;
  static const bool trace = [] { const char* e = getenv("AD_MEGA_TIMELINE"); return e && e[0] == '1'; }();
  p.timeline = trace ? h->mega_timeline : nullptr;
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3(h->mega_cs * h->mega_nc); cfg.blockDim = dim3(mega::THREADS);
  cfg.dynamicSmemBytes = h->mega_smem; cfg.stream = h->stream;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = h->mega_cs; attr[0].val.clusterDim.y = 1; attr[0].val.clusterDim.z = 1;
  attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[1].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr; cfg.numAttrs = g_use_pdl ? 2 : 1;
  note_launch(h, "persistent_decoder_pass");
  cudaError_t e = cudaLaunchKernelEx(&cfg, mega::decoder_pass_kernel, p);
  if (e != cudaSuccess) return fail(h, AD_ERR_CUDA, std::string("persistent decoder pass launch: ") + cudaGetErrorString(e));
  return AD_OK;
}

// Decoder stack over the packed tokens of pass pk (verification: cached, block-causal; drafter: no cache,
// unmasked).  Leaves the final hidden states in yb.
int decoder_pass(ad_handle* h, int pk, Model& m) {
  const ad_model_cfg& c = h->cfg;
  PassCfg& pc = h->pass[pk];
  const size_t self_layer = (size_t)h->dims.max_tgt * c.max_batch * c.d_model * h->esz;
  const size_t cross_layer = (size_t)c.max_src * c.max_batch * c.d_model * h->esz;
  if (!(pk == PK_VERIFY && h->pass_planned)) AD_TRY(embed(h, pc, m));
  for (int l = 0; l < c.n_dec; ++l) {
    DecLayer& L = m.dec[l];
    void* kb = pk == PK_VERIFY ? (char*)h->kself + l * self_layer : h->ktmp;
    void* vb = pk == PK_VERIFY ? (char*)h->vself + l * self_layer : h->vtmp;
    AD_TRY(self_attention_sublayer(h, pk, L.wqkv, L.bqkv, L.wo, L.bo, L.ln1g, L.ln1b, kb, vb));
    // Query projection of the cross-attention.  With few tokens a full-K walk per CTA is the slow part of the
    // projection, so it is split along K and the attention kernel adds the partial sums (and the bias) as it
    // loads its queries.
    bool fused_x = false;
    int qs = h->bf16 && pc.M_cap <= 256 ? pc.ksplit_for(L.cq.N, L.cq.K, pc.tile_for(L.cq.N, num_sms())) : 1;
    if (qs > 1 && qs <= ATT_MAX_QSPLIT) {
      int ns_q = 1;
      AD_TRY(gemm_to_ln(h, L.cq, h->yb, pk, &ns_q));
      AD_TRY(attention(h, pc, nullptr, (char*)m.kenc + l * cross_layer, (char*)m.venc + l * cross_layer, h->abuf.ptr,
                       h->st.cross_base, nullptr, h->st.srclen, c.max_src, L.cbq, ns_q, &L.co, &fused_x));
    } else {
      GemmParams q = {};
      q.bias = L.cbq; q.out_act = h->qbuf;
      AD_TRY(gemm(h, EPI_ACT, L.cq, h->yb, pk, pc.plan.M, pc.M_cap, q));
      AD_TRY(attention(h, pc, h->qbuf, (char*)m.kenc + l * cross_layer, (char*)m.venc + l * cross_layer, h->abuf.ptr,
                       h->st.cross_base, nullptr, h->st.srclen, c.max_src, nullptr, 0, &L.co, &fused_x));
    }
    if (fused_x) {
      AD_TRY(layernorm(h, pc, c.n_heads, L.cbo, L.ln2g, L.ln2b, h->pre2));
    } else {
      int ns = 1;
      AD_TRY(gemm_to_ln(h, L.co, h->abuf, pk, &ns));
      AD_TRY(layernorm(h, pc, ns, L.cbo, L.ln2g, L.ln2b));
    }
    AD_TRY(ffn_sublayer(h, pk, L.w1, L.b1, L.w2, L.b2, L.ln3g, L.ln3b));
  }
  return AD_OK;
}

// Encoder stack + per-decoder-layer cross-attention key/value projection of the memory.
int encoder_pass(ad_handle* h, Model& m, bool keep_memory) {
  const ad_model_cfg& c = h->cfg;
  PassCfg& pc = h->pass[PK_ENCODE];
  const size_t cross_layer = (size_t)c.max_src * c.max_batch * c.d_model * h->esz;
  AD_TRY(embed(h, pc, m));
  for (int l = 0; l < c.n_enc; ++l) {
    EncLayer& L = m.enc[l];
    AD_TRY(self_attention_sublayer(h, PK_ENCODE, L.wqkv, L.bqkv, L.wo, L.bo, L.ln1g, L.ln1b, h->ktmp, h->vtmp));
    AD_TRY(ffn_sublayer(h, PK_ENCODE, L.w1, L.b1, L.w2, L.b2, L.ln2g, L.ln2b));
  }
  if (keep_memory)
    AD_CUDA(h, cudaMemcpyAsync(h->encmem, h->yb.ptr, (size_t)pc.M_cap * c.d_model * h->esz, cudaMemcpyDeviceToDevice, h->stream));
  // cross-attention keys and values of every decoder layer in one launch (segments 2l / 2l + 1 = layer l's K / V)
  GemmParams p = {};
  p.bias = m.cbkv_pack; p.dst[0] = m.kenc; p.dst[1] = m.venc; p.seg_pair_stride = cross_layer;
  p.seg_width = c.d_model; p.n_direct = 0; p.slot = h->st.enc_slot;
  AD_TRY(gemm(h, EPI_SCATTER, m.ckv_all, h->yb, PK_ENCODE, pc.plan.M, pc.M_cap, p));
  return AD_OK;
}

// Exchanges the handle's activation buffers and stream with the side set (and back, when called again).
void swap_side(ad_handle* h) {
  ActSet& sd = h->side;
  std::swap(h->y, sd.y); std::swap(h->pre, sd.pre); std::swap(h->pre2, sd.pre2);
  std::swap(h->yb, sd.yb); std::swap(h->abuf, sd.abuf); std::swap(h->hbuf, sd.hbuf);
  std::swap(h->qbuf, sd.qbuf); std::swap(h->ktmp, sd.ktmp); std::swap(h->vtmp, sd.vtmp);
  std::swap(h->stream, h->side_stream);
}

// Output projection fused with arg-max over X (yb for the verifier, the gathered mask rows for the drafter),
// then the final reduction and (verifier) the draft compare.
int vocab_stage(ad_handle* h, Model& m, const ActBuf& X, int to_drafts, int auto_commit, bool partials_ready = false) {
  PassCfg& pc = h->pass[PK_VERIFY];
  GemmParams p = {};
  p.part_val = h->part_val; p.part_idx = h->part_idx;
  const int beta = to_drafts ? 0 : h->beta;
  if (beta >= 1) {   // relaxed verification: the drafts' own scores first, then the projection counts against them
    const int d = h->cfg.d_model;
    note_launch(h, "draft_score");
    const dim3 sgrid((pc.M_cap + 7) / 8);
    if (h->bf16) AD_CUDA(h, launch_k(draft_score_kernel<bf16, bf16>, sgrid, dim3(256), 0, h->stream, h->st, pc.plan, h->dims, (const bf16*)m.emb.ptr, (const bf16*)X.ptr, d, h->draft_val, h->draft_id));
    else AD_CUDA(h, launch_k(draft_score_kernel<float, float>, sgrid, dim3(256), 0, h->stream, h->st, pc.plan, h->dims, (const float*)m.emb.ptr, (const float*)X.ptr, d, h->draft_val, h->draft_id));
    p.draft_val = h->draft_val; p.draft_id = h->draft_id; p.part_cnt = h->part_cnt;
  }
  if (!partials_ready) AD_TRY(gemm(h, EPI_ARGMAX, m.emb, X, PK_VERIFY, pc.plan.M, pc.M_cap, p));
  note_launch(h, "argmax_accept");
  NextBlock nxt = {-1, 0, nullptr, 0, 0};
  NextEmbed ne = {};
  if (auto_commit && !to_drafts && h->loop_next.source >= 0) {
    nxt = h->loop_next;
    ne.emb = m.emb.ptr; ne.pe = h->pe; ne.d = h->cfg.d_model; ne.scale = sqrtf((float)h->cfg.d_model); ne.y = h->y; ne.yb = h->yb.ptr;
  }
  if (h->bf16)
    AD_CUDA(h, launch_k(argmax_accept_kernel<bf16>, dim3(h->dims.B), dim3(1024), 0, h->stream, h->st, pc.plan, h->dims, (const float*)h->part_val, (const int*)h->part_idx, h->n_vtiles,
                        pc.M_cap, to_drafts, auto_commit, (unsigned int*)(h->st.loop_it + 1),
                        auto_commit ? h->cond_handle : 0ull, beta, h->tau, (const float*)h->draft_val, (const int*)h->draft_id,
                        (const int*)h->part_cnt, nxt, ne));
  else
    AD_CUDA(h, launch_k(argmax_accept_kernel<float>, dim3(h->dims.B), dim3(1024), 0, h->stream, h->st, pc.plan, h->dims, (const float*)h->part_val, (const int*)h->part_idx, h->n_vtiles,
                        pc.M_cap, to_drafts, auto_commit, (unsigned int*)(h->st.loop_it + 1),
                        auto_commit ? h->cond_handle : 0ull, beta, h->tau, (const float*)h->draft_val, (const int*)h->draft_id,
                        (const int*)h->part_cnt, nxt, ne));
  h->last_vocab_which = to_drafts ? 1 : 0;
  return AD_OK;
}

int prepare_verify(ad_handle* h, int source, int k_cap, const int* ovr, int ovr_len) {
  note_launch(h, "prepare_verify");
  AD_CUDA(h, launch_k(prepare_verify_kernel, dim3(1), dim3(256), 0, h->stream, h->st, h->pass[PK_VERIFY].plan, h->dims, source, k_cap, ovr,
                                                 h->cfg.max_tgt, ovr_len));
  return AD_OK;
}

// Draft substep: sizes, drafter plan, drafter decoder, gather of the mask rows, projection + arg-max.
int draft_stage(ad_handle* h, int k_cap) {
  AD_TRY(prepare_verify(h, SRC_SIZES, k_cap, nullptr, 0));
  note_launch(h, "draft_stage");
  AD_CUDA(h, launch_k(plan_draft_kernel, dim3(1), dim3(256), 0, h->stream, h->st, h->pass[PK_VERIFY].plan, h->pass[PK_DRAFT].plan, h->dims));
  if (mega_applies(h, PK_DRAFT)) {      // decoder stack, gather of the mask rows and projection in one kernel
    AD_TRY(mega_launch(h, PK_DRAFT));
    return vocab_stage(h, h->nar, h->xg, 1, 0, true);
  }
  AD_TRY(decoder_pass(h, PK_DRAFT, h->nar));
  const int d = h->cfg.d_model;
  PassCfg& pv = h->pass[PK_VERIFY];
  note_launch(h, "draft_stage");
  if (h->bf16) AD_CUDA(h, launch_k(gather_rows_kernel<bf16>, dim3(pv.M_cap), dim3(128), 0, h->stream, (const int*)pv.plan.M, (const int*)h->st.gidx, (const bf16*)h->yb.ptr, (bf16*)h->xg.ptr, d));
  else AD_CUDA(h, launch_k(gather_rows_kernel<float>, dim3(pv.M_cap), dim3(128), 0, h->stream, (const int*)pv.plan.M, (const int*)h->st.gidx, (const float*)h->yb.ptr, (float*)h->xg.ptr, d));
  return vocab_stage(h, h->nar, h->xg, 1, 0);
}

int verify_stage(ad_handle* h, int auto_commit) {
  if (mega_applies(h, PK_VERIFY)) {
    AD_TRY(mega_launch(h, PK_VERIFY));
    return vocab_stage(h, h->ar, h->yb, 0, auto_commit, true);
  }
  AD_TRY(decoder_pass(h, PK_VERIFY, h->ar));
  return vocab_stage(h, h->ar, h->yb, 0, auto_commit);
}

int commit_stage(ad_handle* h, const int* n_dev) {
  note_launch(h, "commit_stage");
  AD_CUDA(h, launch_k(commit_kernel, dim3(1), dim3(256), 0, h->stream, h->st, h->pass[PK_VERIFY].plan, h->dims, n_dev));
  return AD_OK;
}

// One iteration of the decode loop: draft -> verify -> commit, all on the device.
// Whether the loop of these options lets the accept kernel plan and embed the next block: no drafter pass in between,
// blocks small enough for one CTA to embed, kernel-chain form of the pass.
bool g_fuse_plan = true;      // AD_NO_FUSED_PLAN=1: plan and embed as kernels of their own in every iteration
bool loop_plans_ahead(const ad_handle* h, const ad_gen_opts& o) {
  return g_fuse_plan && !(o.mode == AD_MODE_GAD && o.run_drafter) && h->pass[PK_VERIFY].M_cap <= 128 && !h->mega[PK_VERIFY].on;
}

// First block of a loop that plans ahead: planned and embedded by kernels of their own, before the loop.
int plan_first_block(ad_handle* h, const ad_gen_opts& o, const int* ovr, int ovr_len) {
  AD_TRY(prepare_verify(h, (o.mode == AD_MODE_GAD || ovr) ? SRC_OVERRIDE : SRC_POLICY, o.k, ovr, ovr_len));
  return embed(h, h->pass[PK_VERIFY], h->ar);
}

int loop_iteration(ad_handle* h, const ad_gen_opts& o, const int* ovr, int ovr_len) {
  struct Shrinking {
    PassCfg& pc;
    Shrinking(PassCfg& p, bool on) : pc(p) { pc.shrinking = on; }
    ~Shrinking() { pc.shrinking = false; }
  } scope(h->pass[PK_VERIFY], o.mode == AD_MODE_IAD);
  if (loop_plans_ahead(h, o)) {
    // this iteration's plan and embedding exist already (plan_first_block, or the previous iteration's accept kernel)
    h->loop_next = NextBlock{(o.mode == AD_MODE_GAD || ovr) ? SRC_OVERRIDE : SRC_POLICY, o.k, ovr, h->cfg.max_tgt, ovr_len};
    h->pass_planned = true;
    const int rc = verify_stage(h, 1);
    h->pass_planned = false;
    h->loop_next.source = -1;
    return rc;
  }
  if (o.mode == AD_MODE_GAD) {
    if (o.run_drafter) {
      AD_TRY(draft_stage(h, o.k));
      AD_TRY(prepare_verify(h, SRC_KEEP, o.k, ovr, ovr_len));
    } else {
      AD_TRY(prepare_verify(h, SRC_OVERRIDE, o.k, ovr, ovr_len));
    }
  } else {
    AD_TRY(prepare_verify(h, ovr ? SRC_OVERRIDE : SRC_POLICY, o.k, ovr, ovr_len));
  }
  return verify_stage(h, 1);   // accept and commit in one kernel
}

int read_status(ad_handle* h) {
  int s = 0;
  AD_CUDA(h, cudaMemcpyAsync(&s, h->st.status, sizeof(int), cudaMemcpyDeviceToHost, h->stream));
  AD_CUDA(h, cudaStreamSynchronize(h->stream));
  if (s != 0) {
    int z = 0;
    cudaMemcpyAsync(h->st.status, &z, sizeof(int), cudaMemcpyHostToDevice, h->stream);
    cudaStreamSynchronize(h->stream);
    return fail(h, s, s == AD_ERR_TIMEOUT ? "a bounded device-side wait ran out" : "device-side argument check failed");
  }
  return AD_OK;
}

cudaMemcpyKind to_dev(int on_host) { return on_host ? cudaMemcpyHostToDevice : cudaMemcpyDeviceToDevice; }
cudaMemcpyKind from_dev(int on_host) { return on_host ? cudaMemcpyDeviceToHost : cudaMemcpyDeviceToDevice; }

void drop_graphs(ad_handle* h) {
  for (auto& kv : h->graphs) cudaGraphExecDestroy(kv.second.exec);
  h->graphs.clear();
}

}  // namespace

// =====================================================================================================
// extern "C"
// =====================================================================================================

extern "C" int ad_weight_counts(const ad_model_cfg* cfg, size_t* matrix_elems, size_t* vector_elems) {
  std::string why;
  if (check_cfg(cfg, &why) != AD_OK || !matrix_elems || !vector_elems) return fail(nullptr, AD_ERR_ARG, why.empty() ? "null output pointer" : why);
  weight_counts(*cfg, matrix_elems, vector_elems);
  return AD_OK;
}

extern "C" int ad_query_workspace(const ad_model_cfg* cfg, size_t* bytes) {
  std::string why;
  if (check_cfg(cfg, &why) != AD_OK || !bytes) return fail(nullptr, AD_ERR_ARG, why.empty() ? "null output pointer" : why);
  ad_handle tmp;
  tmp.cfg = *cfg;
  tmp.bf16 = cfg->dtype == AD_DTYPE_BF16;
  tmp.esz = tmp.bf16 ? 2 : 4;
  *bytes = layout(&tmp, nullptr);
  return AD_OK;
}

extern "C" const char* ad_last_error(const ad_handle* h) { return h ? h->err.c_str() : g_create_error.c_str(); }

extern "C" int ad_create(const ad_model_cfg* cfg, const ad_weights* w, void* workspace, size_t workspace_bytes,
                         void* stream, ad_handle** out) {
  std::string why;
  if (!out) return fail(nullptr, AD_ERR_ARG, "out is null");
  *out = nullptr;
  if (check_cfg(cfg, &why) != AD_OK) return fail(nullptr, AD_ERR_ARG, why);
  if (!w || !workspace) return fail(nullptr, AD_ERR_ARG, "weights or workspace is null");
  if (reinterpret_cast<uintptr_t>(workspace) % 1024) return fail(nullptr, AD_ERR_ARG, "workspace must be 1024-byte aligned");
  int dev = 0, major = 0;
  if (cudaGetDevice(&dev) != cudaSuccess || cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess)
    return fail(nullptr, AD_ERR_CUDA, "no CUDA device");
  { const char* e = getenv("AD_NO_PDL"); g_use_pdl = !(e && e[0] == '1'); }
  { const char* e = getenv("AD_NO_DEVLOOP"); g_use_devloop = !(e && e[0] == '1'); }
  { const char* e = getenv("AD_NO_ENCODE_GRAPH"); g_use_graph_encode = !(e && e[0] == '1'); }
  { const char* e = getenv("AD_NO_CONCURRENT_ENCODERS"); g_two_stream_encode = !(e && e[0] == '1'); }
  { const char* e = getenv("AD_NO_ATTN_PROJ"); g_fuse_attn_proj = !(e && e[0] == '1'); }
  { const char* e = getenv("AD_MEGA"); g_use_mega = e && e[0] == '1'; }
  { const char* e = getenv("AD_NO_FUSED_PLAN"); g_fuse_plan = !(e && e[0] == '1'); }
  if (major != 10) return fail(nullptr, AD_ERR_CUDA, "this library contains sm_100a code only; the current device is not compute capability 10.x");

  ad_handle* h = new ad_handle();
  h->cfg = *cfg;
  h->stream = static_cast<cudaStream_t>(stream);
  h->bf16 = cfg->dtype == AD_DTYPE_BF16;
  h->esz = h->bf16 ? 2 : 4;
  const size_t need = layout(h, workspace);
  auto bail = [&](int code, const std::string& msg) { g_create_error = msg; delete h; return code; };
  if (need > workspace_bytes) return bail(AD_ERR_CAPACITY, "workspace too small: need " + std::to_string(need) + " bytes");
  h->dims = Dims{cfg->max_batch, cfg->max_src, cfg->max_tgt, cfg->kmax, cfg->bos, cfg->pad, cfg->eos, cfg->mask, cfg->vocab};
  int rc = bind_model(h, h->ar, w->ar);
  if (rc == AD_OK && cfg->has_drafter) rc = bind_model(h, h->nar, w->nar);
  if (rc != AD_OK) return bail(rc, h->err);
  if (h->bf16) {
    bool ok = true;
    ActBuf* bufs[4] = {&h->yb, &h->abuf, &h->hbuf, &h->xg};
    for (ActBuf* b : bufs)
      for (int k = 0; k < PK_COUNT; ++k)
        for (int i = 0; i < 5 && (16 << i) <= h->pass[k].ntile; ++i)
          ok = ok && make_map(&b->map[k][i], b->ptr, h->M_all, b->cols, 16 << i);
    if (cfg->has_drafter) {
      const int Me = h->pass[PK_ENCODE].M_cap, nt = h->pass[PK_ENCODE].ntile;
      ActBuf* sbufs[3] = {&h->side.yb, &h->side.abuf, &h->side.hbuf};
      for (ActBuf* b : sbufs)
        for (int i = 0; i < 5 && (16 << i) <= nt; ++i)
          ok = ok && make_map(&b->map[PK_ENCODE][i], b->ptr, Me, b->cols, 16 << i);
    }
    if (!ok) return bail(AD_ERR_CUDA, "cuTensorMapEncodeTiled failed for an activation buffer");
  }
  if (cfg->has_drafter && g_two_stream_encode) {
    if (cudaStreamCreateWithFlags(&h->side_stream, cudaStreamNonBlocking) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_fork, cudaEventDisableTiming) != cudaSuccess ||
        cudaEventCreateWithFlags(&h->ev_join, cudaEventDisableTiming) != cudaSuccess)
      return bail(AD_ERR_CUDA, "creating the side stream failed");
  }
  // Cache, scratch and state start from zero so that no stale bit pattern is ever read as a number.
  if (cudaMemsetAsync(workspace, 0, need, h->stream) != cudaSuccess) return bail(AD_ERR_CUDA, "clearing the workspace failed");
  // Gather the cross-attention key/value projections of all decoder layers (see Model::ckv_all).
  for (Model* mp : {&h->ar, &h->nar}) {
    if (!mp->present) continue;
    const int d = cfg->d_model;
    const size_t one = h->esz * (size_t)2 * d * d;
    bool okc = true;
    for (int l = 0; l < cfg->n_dec; ++l) {
      okc = okc && cudaMemcpyAsync((char*)mp->ckv_pack + l * one, mp->dec[l].ckv.ptr, one, cudaMemcpyDeviceToDevice, h->stream) == cudaSuccess;
      okc = okc && cudaMemcpyAsync(mp->cbkv_pack + (size_t)l * 2 * d, mp->dec[l].cbkv, sizeof(float) * 2 * d, cudaMemcpyDeviceToDevice, h->stream) == cudaSuccess;
    }
    mp->ckv_all.ptr = mp->ckv_pack; mp->ckv_all.N = cfg->n_dec * 2 * d; mp->ckv_all.K = d;
    if (h->bf16) okc = okc && make_map(&mp->ckv_all.map, mp->ckv_pack, mp->ckv_all.N, d, tc::BLOCK_N_FEAT);
    if (!okc) return bail(AD_ERR_CUDA, "gathering the cross-attention key/value projections failed");
  }
  {
    const int rcm = mega_setup(h);
    if (rcm != AD_OK) return bail(rcm, h->err);
  }
  // Sinusoidal positional table PE(p, 2i) = sin(p / 10000^(2i/d)), PE(p, 2i+1) = cos(.), evaluated in double.
  {
    const int d = cfg->d_model;
    std::vector<float> pe((size_t)h->max_pos * d);
    for (int p = 0; p < h->max_pos; ++p)
      for (int i = 0; i < d; i += 2) {
        const double freq = exp(-log(10000.0) * (double)i / (double)d);
        pe[(size_t)p * d + i] = (float)sin(p * freq);
        if (i + 1 < d) pe[(size_t)p * d + i + 1] = (float)cos(p * freq);
      }
    if (cudaMemcpyAsync(h->pe, pe.data(), pe.size() * sizeof(float), cudaMemcpyHostToDevice, h->stream) != cudaSuccess ||
        cudaStreamSynchronize(h->stream) != cudaSuccess)
      return bail(AD_ERR_CUDA, "uploading the positional table failed");
  }
  {
    const size_t B = cfg->max_batch;
    const size_t n_up = B * cfg->max_src + 2 * B + B * cfg->max_tgt, n_down = 4 + 4 * B + B * cfg->max_tgt;
    if (cudaHostAlloc(&h->host_flag, sizeof(int) * (16 + n_up + n_down), cudaHostAllocMapped) != cudaSuccess ||
        cudaHostGetDevicePointer(&h->host_flag_dev, h->host_flag, 0) != cudaSuccess)
      return bail(AD_ERR_CUDA, "allocating pinned host memory failed");
    h->up_src = h->host_flag + 16; h->up_len = h->up_src + B * cfg->max_src; h->up_max = h->up_len + B;
    h->up_ovr = h->up_max + B; h->down = h->up_ovr + B * cfg->max_tgt;
    h->down_dev = h->host_flag_dev + (h->down - h->host_flag);
  }
  if (cudaEventCreate(&h->ev0) != cudaSuccess || cudaEventCreate(&h->ev1) != cudaSuccess || cudaEventCreate(&h->ev2) != cudaSuccess)
    return bail(AD_ERR_CUDA, "cudaEventCreate failed");
  *out = h;
  return AD_OK;
}

extern "C" int ad_destroy(ad_handle* h) {
  if (!h) return AD_ERR_ARG;
  cudaStreamSynchronize(h->stream);
  drop_graphs(h);
  if (h->host_flag) cudaFreeHost(h->host_flag);
  if (h->ev0) cudaEventDestroy(h->ev0);
  if (h->ev1) cudaEventDestroy(h->ev1);
  if (h->ev2) cudaEventDestroy(h->ev2);
  if (h->ev_fork) cudaEventDestroy(h->ev_fork);
  if (h->ev_join) cudaEventDestroy(h->ev_join);
  if (h->side_stream) { cudaStreamSynchronize(h->side_stream); cudaStreamDestroy(h->side_stream); }
  delete h;
  return AD_OK;
}

extern "C" int ad_set_acceptance(ad_handle* h, int32_t beta, float tau) {
  if (!h) return AD_ERR_ARG;
  if (beta < 0 || !(tau >= 0.f)) return fail(h, AD_ERR_ARG, "beta must be >= 0 and tau >= 0");
  h->beta = beta;
  h->tau = tau;
  return AD_OK;
}

extern "C" int ad_sync(ad_handle* h) {
  if (!h) return AD_ERR_ARG;
  return read_status(h);
}

extern "C" int ad_encode(ad_handle* h, const int32_t* src, int32_t src_stride, const int32_t* src_len, int32_t B,
                         int32_t on_host) {
  if (!h) return AD_ERR_ARG;
  const ad_model_cfg& c = h->cfg;
  if (!src || !src_len) return fail(h, AD_ERR_ARG, "src or src_len is null");
  if (B < 1 || B > c.max_batch) return fail(h, AD_ERR_CAPACITY, "B outside 1..max_batch");
  if (src_stride < 1) return fail(h, AD_ERR_ARG, "src_stride must be positive");
  if (on_host)
    for (int b = 0; b < B; ++b)
      if (src_len[b] < 1 || src_len[b] > c.max_src || src_len[b] > src_stride)
        return fail(h, src_len[b] > c.max_src ? AD_ERR_CAPACITY : AD_ERR_ARG, "src_len outside 1..min(max_src, src_stride)");
  // (captured graphs are keyed by the batch size, so a different B simply uses other entries)
  h->B = B;
  h->dims.B = B;
  h->encoded = false;
  const int w = src_stride < c.max_src ? src_stride : c.max_src;
  if (on_host) {
    // host-resident inputs go through the handle's pinned staging area (every host-array call ends synchronised, so
    // the area is free again): one truly asynchronous copy each instead of driver-staged pageable copies
    for (int b = 0; b < B; ++b) memcpy(h->up_src + (size_t)b * c.max_src, src + (size_t)b * src_stride, sizeof(int) * w);
    memcpy(h->up_len, src_len, sizeof(int) * B);
    AD_CUDA(h, cudaMemcpyAsync(h->st.src, h->up_src, sizeof(int) * (size_t)B * c.max_src, cudaMemcpyHostToDevice, h->stream));
    AD_CUDA(h, cudaMemcpyAsync(h->st.srclen, h->up_len, sizeof(int) * B, cudaMemcpyHostToDevice, h->stream));
  } else {
    AD_CUDA(h, cudaMemcpy2DAsync(h->st.src, sizeof(int) * c.max_src, src, sizeof(int) * src_stride, sizeof(int) * w, B, cudaMemcpyDeviceToDevice, h->stream));
    AD_CUDA(h, cudaMemcpyAsync(h->st.srclen, src_len, sizeof(int) * B, cudaMemcpyDeviceToDevice, h->stream));
  }
  // The encoder pass reads its inputs from fixed workspace buffers, so on a capturable stream it is captured
  // once per batch size and replayed (about fifty launches otherwise paid on the host for every sentence).
  auto enqueue = [&]() -> int {
    note_launch(h, "ad_encode");
    AD_CUDA(h, launch_k(plan_encode_kernel, dim3(1), dim3(256), 0, h->stream, h->st, h->pass[PK_ENCODE].plan, h->dims));
    if (c.has_drafter && h->side_stream) {
      // the two encoders are independent (Section 3.2: separate models): drafter's on the side stream, verifier's here
      AD_CUDA(h, cudaEventRecord(h->ev_fork, h->stream));
      AD_CUDA(h, cudaStreamWaitEvent(h->side_stream, h->ev_fork, 0));
      swap_side(h);
      const int rc_side = encoder_pass(h, h->nar, false);
      cudaError_t e_join = rc_side == AD_OK ? cudaEventRecord(h->ev_join, h->stream) : cudaSuccess;
      swap_side(h);
      if (rc_side != AD_OK) return rc_side;
      AD_CUDA(h, e_join);
      AD_TRY(encoder_pass(h, h->ar, true));
      AD_CUDA(h, cudaStreamWaitEvent(h->stream, h->ev_join, 0));
      return AD_OK;
    }
    AD_TRY(encoder_pass(h, h->ar, true));
    if (c.has_drafter) AD_TRY(encoder_pass(h, h->nar, false));
    return AD_OK;
  };
  cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
  if (h->stream != nullptr) cudaStreamIsCapturing(h->stream, &cap);
  if (h->stream != nullptr && cap == cudaStreamCaptureStatusNone && g_use_graph_encode) {
    char key[32];
    snprintf(key, sizeof(key), "encode B%d", B);
    auto it = h->graphs.find(key);
    if (it == h->graphs.end()) {
      cudaGraph_t g = nullptr;
      const int before = h->launches;
      AD_CUDA(h, cudaStreamBeginCapture(h->stream, cudaStreamCaptureModeThreadLocal));
      const int rc = enqueue();
      const cudaError_t e = cudaStreamEndCapture(h->stream, &g);
      const int n = h->launches - before;
      h->launches = before;
      if (rc != AD_OK) { if (g) cudaGraphDestroy(g); return rc; }
      if (e != cudaSuccess) return fail(h, AD_ERR_CUDA, std::string("encoder graph capture: ") + cudaGetErrorString(e));
      cudaGraphExec_t exec = nullptr;
      const cudaError_t e2 = cudaGraphInstantiate(&exec, g, 0);
      cudaGraphDestroy(g);
      if (e2 != cudaSuccess) return fail(h, AD_ERR_CUDA, std::string("encoder graph instantiate: ") + cudaGetErrorString(e2));
      it = h->graphs.emplace(key, ad_handle::GraphEntry{exec, n, false}).first;
    }
    AD_CUDA(h, cudaGraphLaunch(it->second.exec, h->stream));
    h->launches += it->second.launches;
  } else {
    AD_TRY(enqueue());
  }
  h->encoded = true;
  h->last_vocab_which = -1;
  if (on_host && !h->defer_status) return read_status(h);
  return AD_OK;
}

extern "C" int ad_verify_block(ad_handle* h, const int32_t* drafts, const int32_t* k, int32_t* argmax,
                               int32_t* n_accepted, int32_t on_host) {
  if (!h) return AD_ERR_ARG;
  if (!h->encoded) return fail(h, AD_ERR_STATE, "ad_verify_block before ad_encode");
  if (!drafts || !k) return fail(h, AD_ERR_ARG, "drafts or k is null");
  const ad_model_cfg& c = h->cfg;
  const int B = h->B;
  if (on_host)
    for (int b = 0; b < B; ++b)
      if (k[b] < 0 || k[b] > c.kmax) return fail(h, AD_ERR_ARG, "k outside 0..kmax");
  AD_CUDA(h, cudaMemcpyAsync(h->st.user_drafts, drafts, sizeof(int) * (size_t)B * c.kmax, to_dev(on_host), h->stream));
  AD_CUDA(h, cudaMemcpyAsync(h->st.user_k, k, sizeof(int) * B, to_dev(on_host), h->stream));
  AD_TRY(prepare_verify(h, SRC_USER, c.kmax, nullptr, 0));
  AD_TRY(verify_stage(h, 0));
  if (on_host) {
    if (argmax) AD_CUDA(h, cudaMemcpyAsync(argmax, h->st.pred, sizeof(int) * (size_t)B * c.kmax, cudaMemcpyDeviceToHost, h->stream));
    if (n_accepted) AD_CUDA(h, cudaMemcpyAsync(n_accepted, h->st.n_acc, sizeof(int) * B, cudaMemcpyDeviceToHost, h->stream));
    return read_status(h);
  }
  note_launch(h, "ad_verify_block");
  AD_CUDA(h, launch_k(export_block_kernel, dim3(B), dim3(64), 0, h->stream, h->st, h->dims, argmax, n_accepted, nullptr, nullptr, h->pass[PK_VERIFY].plan));
  return AD_OK;
}

extern "C" int ad_commit(ad_handle* h, const int32_t* n, int32_t on_host) {
  if (!h) return AD_ERR_ARG;
  if (!h->encoded) return fail(h, AD_ERR_STATE, "ad_commit before ad_encode");
  const int* n_dev = nullptr;
  if (n) {
    AD_CUDA(h, cudaMemcpyAsync(h->st.user_n, n, sizeof(int) * h->B, to_dev(on_host), h->stream));
    n_dev = h->st.user_n;
  }
  AD_TRY(commit_stage(h, n_dev));
  if (on_host) return read_status(h);
  return AD_OK;
}

extern "C" int ad_force_commit(ad_handle* h, const int32_t* tokens, const int32_t* n, int32_t on_host) {
  if (!h) return AD_ERR_ARG;
  if (!h->encoded) return fail(h, AD_ERR_STATE, "ad_force_commit before ad_encode");
  if (!tokens || !n) return fail(h, AD_ERR_ARG, "tokens or n is null");
  AD_CUDA(h, cudaMemcpyAsync(h->st.user_drafts, tokens, sizeof(int) * (size_t)h->B * h->cfg.kmax, to_dev(on_host), h->stream));
  AD_CUDA(h, cudaMemcpyAsync(h->st.user_n, n, sizeof(int) * h->B, to_dev(on_host), h->stream));
  note_launch(h, "ad_force_commit");
  AD_CUDA(h, launch_k(force_commit_kernel, dim3(1), dim3(256), 0, h->stream, h->st, h->pass[PK_VERIFY].plan, h->dims, h->st.user_drafts, h->st.user_n));
  if (on_host) return read_status(h);
  return AD_OK;
}

extern "C" int ad_draft_block(ad_handle* h, int32_t k_cap, int32_t* drafts, int32_t* k, int32_t on_host) {
  if (!h) return AD_ERR_ARG;
  if (!h->encoded) return fail(h, AD_ERR_STATE, "ad_draft_block before ad_encode");
  if (!h->cfg.has_drafter) return fail(h, AD_ERR_STATE, "the handle has no drafter model");
  const ad_model_cfg& c = h->cfg;
  if (k_cap < 1 || k_cap > c.kmax) return fail(h, AD_ERR_ARG, "k_cap outside 1..kmax");
  AD_TRY(draft_stage(h, k_cap));
  const int B = h->B;
  if (on_host) {
    if (drafts) AD_CUDA(h, cudaMemcpyAsync(drafts, h->st.drafts, sizeof(int) * (size_t)B * c.kmax, cudaMemcpyDeviceToHost, h->stream));
    if (k) AD_CUDA(h, cudaMemcpyAsync(k, h->pass[PK_VERIFY].plan.seg_len, sizeof(int) * B, cudaMemcpyDeviceToHost, h->stream));
    return read_status(h);
  }
  note_launch(h, "ad_draft_block");
  AD_CUDA(h, launch_k(export_block_kernel, dim3(B), dim3(64), 0, h->stream, h->st, h->dims, nullptr, nullptr, drafts, k, h->pass[PK_VERIFY].plan));
  return AD_OK;
}

extern "C" int ad_get_state(ad_handle* h, int32_t* len, int32_t* last_tok, int32_t* finished) {
  if (!h) return AD_ERR_ARG;
  if (h->B < 1) return fail(h, AD_ERR_STATE, "ad_get_state before ad_encode");
  if (len) AD_CUDA(h, cudaMemcpyAsync(len, h->st.len, sizeof(int) * h->B, cudaMemcpyDeviceToHost, h->stream));
  if (last_tok) AD_CUDA(h, cudaMemcpyAsync(last_tok, h->st.last, sizeof(int) * h->B, cudaMemcpyDeviceToHost, h->stream));
  if (finished) AD_CUDA(h, cudaMemcpyAsync(finished, h->st.fin, sizeof(int) * h->B, cudaMemcpyDeviceToHost, h->stream));
  return read_status(h);
}

extern "C" int ad_generate(ad_handle* h, const int32_t* src, int32_t src_stride, const int32_t* src_len, int32_t B,
                           const ad_gen_opts* opts, int32_t* out, int32_t out_stride, int32_t* out_len,
                           ad_stats* stats, int32_t on_host) {
  if (!h) return AD_ERR_ARG;
  const ad_model_cfg& c = h->cfg;
  if (!opts || !out || !out_len) return fail(h, AD_ERR_ARG, "opts, out or out_len is null");
  if (opts->mode != AD_MODE_IAD && opts->mode != AD_MODE_GAD) return fail(h, AD_ERR_ARG, "unknown mode");
  if (opts->k < 1 || opts->k > c.kmax) return fail(h, AD_ERR_ARG, "k outside 1..kmax");
  if (opts->mode == AD_MODE_GAD && opts->run_drafter && !c.has_drafter) return fail(h, AD_ERR_STATE, "GAD with run_drafter needs a drafter model");
  if (opts->mode == AD_MODE_GAD && !opts->run_drafter && !opts->draft_override) return fail(h, AD_ERR_ARG, "GAD without the drafter needs draft_override");
  if (opts->draft_override && opts->override_stride < 1) return fail(h, AD_ERR_ARG, "override_stride must be positive");
  if (out_stride < 1) return fail(h, AD_ERR_ARG, "out_stride must be positive");
  if (B < 1 || B > c.max_batch) return fail(h, AD_ERR_CAPACITY, "B outside 1..max_batch");
  // host-visible per-row caps are checked before any device work, so a rejected call leaves the handle untouched
  int max_iters = c.max_tgt;
  if (opts->max_len && on_host) {
    max_iters = 1;
    for (int b = 0; b < B; ++b) {
      if (opts->max_len[b] < 1 || opts->max_len[b] > c.max_tgt) return fail(h, AD_ERR_ARG, "max_len outside 1..max_tgt");
      if (opts->max_len[b] > max_iters) max_iters = opts->max_len[b];
    }
  }

  AD_CUDA(h, cudaEventRecord(h->ev0, h->stream));
  h->launches = 0;
  h->defer_status = true;       // the one synchronisation at the end of this call reports device-side errors
  const int rc_enc = ad_encode(h, src, src_stride, src_len, B, on_host);
  h->defer_status = false;
  if (rc_enc != AD_OK) return rc_enc;
  if (opts->max_len) {
    const int* ml = opts->max_len;
    if (on_host) { memcpy(h->up_max, opts->max_len, sizeof(int) * B); ml = h->up_max; }
    AD_CUDA(h, cudaMemcpyAsync(h->st.user_n, ml, sizeof(int) * B, to_dev(on_host), h->stream));
    note_launch(h, "ad_generate");
    AD_CUDA(h, launch_k(set_maxlen_kernel, dim3((B + 63) / 64), dim3(64), 0, h->stream, h->st, h->dims, h->st.user_n));
  }
  const int* ovr = nullptr;
  int ovr_len = 0;   // valid leading entries of each staged override row
  if (opts->draft_override) {
    ovr_len = opts->override_stride < c.max_tgt ? opts->override_stride : c.max_tgt;
    if (on_host) {
      for (int b = 0; b < B; ++b)
        memcpy(h->up_ovr + (size_t)b * c.max_tgt, opts->draft_override + (size_t)b * opts->override_stride, sizeof(int) * ovr_len);
      AD_CUDA(h, cudaMemcpyAsync(h->ovr, h->up_ovr, sizeof(int) * (size_t)B * c.max_tgt, cudaMemcpyHostToDevice, h->stream));
    } else {
      AD_CUDA(h, cudaMemcpy2DAsync(h->ovr, sizeof(int) * c.max_tgt, opts->draft_override, sizeof(int) * opts->override_stride,
                                   sizeof(int) * ovr_len, B, cudaMemcpyDeviceToDevice, h->stream));
    }
    ovr = h->ovr;
  }
  AD_CUDA(h, cudaEventRecord(h->ev1, h->stream));

  cudaGraphExec_t exec = nullptr;
  int per_iter_launches = 0;
  bool device_loop = false;
  if (opts->use_graph && h->stream != nullptr) {   // the legacy default stream cannot be captured
    char key[160];
    snprintf(key, sizeof(key), "B%d m%d k%d o%d v%d d%d b%d t%a", B, opts->mode, opts->k, ovr ? 1 : 0, ovr_len, opts->run_drafter,
             h->beta, (double)h->tau);
    auto it = h->graphs.find(key);
    if (it == h->graphs.end()) {
      const int before = h->launches;
      // First choice: the whole loop as one graph -- a device-side `while` node whose body is one iteration and
      // whose condition the accept/commit kernel clears; no host round trip between iterations.
      if (g_use_devloop) {
        cudaGraph_t g = nullptr;
        cudaGraphConditionalHandle ch = 0;
        bool okb = cudaGraphCreate(&g, 0) == cudaSuccess &&
                   cudaGraphConditionalHandleCreate(&ch, g, 1, cudaGraphCondAssignDefault) == cudaSuccess;
        cudaGraphNodeParams np = {cudaGraphNodeTypeConditional};
        np.conditional.handle = ch;
        np.conditional.type = cudaGraphCondTypeWhile;
        np.conditional.size = 1;
        cudaGraphNode_t node;
        okb = okb && cudaGraphAddNode(&node, g, nullptr, 0, &np) == cudaSuccess;
        if (okb) {
          cudaGraph_t body = np.conditional.phGraph_out[0];
          okb = cudaStreamBeginCaptureToGraph(h->stream, body, nullptr, nullptr, 0, cudaStreamCaptureModeThreadLocal) == cudaSuccess;
          if (okb) {
            h->cond_handle = (unsigned long long)ch;
            const int rc = loop_iteration(h, *opts, ovr, ovr_len);
            h->cond_handle = 0;
            cudaGraph_t dummy = nullptr;
            const cudaError_t e = cudaStreamEndCapture(h->stream, &dummy);
            okb = rc == AD_OK && e == cudaSuccess;
          }
        }
        per_iter_launches = h->launches - before;
        h->launches = before;
        if (okb) okb = cudaGraphInstantiate(&exec, g, 0) == cudaSuccess;
        if (g) cudaGraphDestroy(g);
        if (okb) {
          h->graphs[key] = ad_handle::GraphEntry{exec, per_iter_launches, true};
          device_loop = true;
        } else {
          exec = nullptr;
          cudaGetLastError();   // clear; fall back to one replay per iteration
        }
      }
      if (!exec) {
        cudaGraph_t g = nullptr;
        AD_CUDA(h, cudaStreamBeginCapture(h->stream, cudaStreamCaptureModeThreadLocal));
        const int rc = loop_iteration(h, *opts, ovr, ovr_len);
        cudaError_t e = cudaStreamEndCapture(h->stream, &g);
        per_iter_launches = h->launches - before;
        h->launches = before;
        if (rc != AD_OK) { if (g) cudaGraphDestroy(g); return rc; }
        if (e != cudaSuccess) return fail(h, AD_ERR_CUDA, std::string("graph capture: ") + cudaGetErrorString(e));
        e = cudaGraphInstantiate(&exec, g, 0);
        cudaGraphDestroy(g);
        if (e != cudaSuccess) return fail(h, AD_ERR_CUDA, std::string("graph instantiate: ") + cudaGetErrorString(e));
        h->graphs[key] = ad_handle::GraphEntry{exec, per_iter_launches, false};
      }
    } else {
      exec = it->second.exec;
      per_iter_launches = it->second.launches;
      device_loop = it->second.device_loop;
    }
  }

  if (loop_plans_ahead(h, *opts)) AD_TRY(plan_first_block(h, *opts, ovr, ovr_len));
  if (device_loop) {
    // one launch runs every iteration; the data-independent bound on the iteration count travels in loop_it[3]
    h->host_flag[1] = max_iters + 1;
    AD_CUDA(h, cudaMemcpyAsync(h->st.loop_it + 3, h->host_flag + 1, sizeof(int), cudaMemcpyHostToDevice, h->stream));
    AD_CUDA(h, cudaGraphLaunch(exec, h->stream));
  }
  const int sync_every = opts->sync_every > 0 ? opts->sync_every : 1;
  int iters = 0;
  volatile int* flag = h->host_flag;
  flag[0] = 0;
  while (!device_loop && iters < max_iters + sync_every) {
    for (int s = 0; s < sync_every; ++s, ++iters) {
      if (exec) {
        AD_CUDA(h, cudaGraphLaunch(exec, h->stream));
        h->launches += per_iter_launches;
      } else {
        AD_TRY(loop_iteration(h, *opts, ovr, ovr_len));
      }
    }
    AD_CUDA(h, cudaMemcpyAsync(h->host_flag, h->st.all_fin, sizeof(int), cudaMemcpyDeviceToHost, h->stream));
    AD_CUDA(h, cudaStreamSynchronize(h->stream));
    if (flag[0]) break;
  }
  AD_CUDA(h, cudaEventRecord(h->ev2, h->stream));
  // Results, statistics and the status word in one block of mapped host memory, written by one kernel: the call ends
  // with a single synchronisation (device-resident result arrays are written directly by the same kernel).
  note_launch(h, "ad_generate");
  AD_CUDA(h, launch_k(finalize_generate_kernel, dim3(B), dim3(128), 0, h->stream, h->st, h->dims, on_host ? nullptr : out, out_stride,
                      on_host ? nullptr : out_len, h->down_dev));
  AD_CUDA(h, cudaStreamSynchronize(h->stream));
  const int* blk = h->down;
  if (device_loop) h->launches += per_iter_launches * blk[0];
  if (on_host) {
    const int w = out_stride < c.max_tgt ? out_stride : c.max_tgt;
    for (int b = 0; b < B; ++b) {
      memcpy(out + (size_t)b * out_stride, blk + 4 + 4 * B + (size_t)b * c.max_tgt, sizeof(int) * w);
      out_len[b] = blk[4 + 4 * b + 3];
    }
  }
  if (stats) {
    memset(stats, 0, sizeof(*stats));
    for (int b = 0; b < B; ++b) {
      stats->row_iterations += blk[4 + 4 * b];
      stats->accepted += blk[4 + 4 * b + 1];
      stats->offered += blk[4 + 4 * b + 2];
    }
    stats->iterations = blk[2];
    cudaEventElapsedTime(&stats->encode_ms, h->ev0, h->ev1);
    cudaEventElapsedTime(&stats->device_ms, h->ev1, h->ev2);
    stats->kernel_launches = h->launches;
  }
  const int dev_status = blk[1];      // already cleared on the device by the kernel that read it
  if (dev_status != 0)
    return fail(h, dev_status, dev_status == AD_ERR_TIMEOUT ? "a bounded device-side wait ran out" : "device-side argument check failed");
  return AD_OK;
}

extern "C" int ad_debug_logits(ad_handle* h, int32_t which, float* logits, size_t capacity_elems) {
  if (!h || !logits) return AD_ERR_ARG;
  if (h->last_vocab_which != which) return fail(h, AD_ERR_STATE, "no matching projection has just run");
  PassCfg& pc = h->pass[PK_VERIFY];
  int M = 0;
  AD_CUDA(h, cudaMemcpyAsync(&M, pc.plan.M, sizeof(int), cudaMemcpyDeviceToHost, h->stream));
  AD_CUDA(h, cudaStreamSynchronize(h->stream));
  if ((size_t)M * h->cfg.vocab > capacity_elems) return fail(h, AD_ERR_CAPACITY, "logits buffer too small");
  Model& m = which == 1 ? h->nar : h->ar;
  GemmParams p = {};
  p.out_f32 = logits;
  AD_TRY(gemm(h, EPI_F32, m.emb, which == 1 ? h->xg : h->yb, PK_VERIFY, pc.plan.M, pc.M_cap, p));
  return AD_OK;
}

extern "C" int ad_debug_encoder_memory(ad_handle* h, int32_t b, float* mem, size_t capacity_elems) {
  if (!h || !mem) return AD_ERR_ARG;
  if (!h->encoded || b < 0 || b >= h->B) return fail(h, AD_ERR_STATE, "no encoded row b");
  PassPlan& pl = h->pass[PK_ENCODE].plan;
  int off = 0, len = 0;
  AD_CUDA(h, cudaMemcpyAsync(&off, pl.seg_off + b, sizeof(int), cudaMemcpyDeviceToHost, h->stream));
  AD_CUDA(h, cudaMemcpyAsync(&len, pl.seg_len + b, sizeof(int), cudaMemcpyDeviceToHost, h->stream));
  AD_CUDA(h, cudaStreamSynchronize(h->stream));
  const size_t n = (size_t)len * h->cfg.d_model;
  if (n > capacity_elems) return fail(h, AD_ERR_CAPACITY, "memory buffer too small");
  const size_t start = (size_t)off * h->cfg.d_model;
  if (h->bf16) to_f32_kernel<bf16><<<64, 256, 0, h->stream>>>((const bf16*)h->encmem + start, mem, n);
  else to_f32_kernel<float><<<64, 256, 0, h->stream>>>((const float*)h->encmem + start, mem, n);
  AD_CUDA(h, cudaGetLastError());
  return AD_OK;
}


extern "C" int ad_debug_profile_verify(ad_handle* h, const int32_t* drafts, const int32_t* k, char* names, float* us,
                                       int32_t capacity, int32_t* n_launches) {
  if (!h || !drafts || !k || !names || !us || !n_launches || capacity < 1) return AD_ERR_ARG;
  if (!h->encoded) return fail(h, AD_ERR_STATE, "ad_debug_profile_verify before ad_encode");
  const bool pdl = g_use_pdl;
  g_use_pdl = false;               // serialised launches: an event between two kernels then brackets exactly one of them
  h->profiling = true;
  h->prof.clear();
  const int rc = ad_verify_block(h, drafts, k, nullptr, nullptr, 1);
  h->profiling = false;
  g_use_pdl = pdl;
  cudaEvent_t last = nullptr;
  if (cudaEventCreate(&last) == cudaSuccess) { cudaEventRecord(last, h->stream); h->prof.emplace_back("end", last); }
  cudaStreamSynchronize(h->stream);
  int n = 0;
  for (size_t i = 0; i + 1 < h->prof.size() && n < capacity; ++i, ++n) {
    float ms = 0.f;
    cudaEventElapsedTime(&ms, h->prof[i].second, h->prof[i + 1].second);
    us[n] = ms * 1e3f;
    snprintf(names + (size_t)n * 64, 64, "%s", h->prof[i].first.c_str());
  }
  for (auto& pr : h->prof) cudaEventDestroy(pr.second);
  h->prof.clear();
  *n_launches = n;
  return rc;
}

extern "C" int ad_debug_stage_timeline(ad_handle* h, uint64_t* stamps, int32_t capacity, int32_t* n_stages) {
  if (!h || !stamps || !n_stages) return AD_ERR_ARG;
  const int n = mega::ST_PER_LAYER * h->cfg.n_dec + 1;
  if (capacity < 2 * n) return fail(h, AD_ERR_CAPACITY, "timeline buffer too small");
  AD_CUDA(h, cudaStreamSynchronize(h->stream));
  AD_CUDA(h, cudaMemcpy(stamps, h->mega_timeline, sizeof(uint64_t) * 2 * (size_t)n, cudaMemcpyDeviceToHost));
  *n_stages = n;
  return AD_OK;
}

// ---- bounded-wait self-test ---------------------------------------------------------------------------

namespace {
// One thread waits, with the given time budget, on an mbarrier phase that nothing ever completes.
__global__ void wait_probe_kernel(int* status, unsigned int budget_us, int* waited_us) {
  __shared__ __align__(8) uint64_t bar;
  if (threadIdx.x == 0) {
    tc::mbar_init(tc::smem_u32(&bar), 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    const unsigned long long t0 = tc::global_ns();
    tc::mbar_wait_budget(tc::smem_u32(&bar), 0, status, (unsigned long long)budget_us * 1000ull);
    if (waited_us) *waited_us = (int)((tc::global_ns() - t0) / 1000ull);
  }
}
}  // namespace

extern "C" int ad_debug_wait_probe(int32_t* status, int32_t budget_us, int32_t* waited_us, void* stream) {
  if (!status || budget_us < 1 || budget_us > (1 << 16)) return AD_ERR_ARG;
  wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(status, (unsigned int)budget_us, waited_us);
  return cudaGetLastError() == cudaSuccess ? AD_OK : AD_ERR_CUDA;
}

// ---- grid-barrier self-test and timing ------------------------------------------------------------------

namespace {
// Every CTA: per round, publish a word, pass the grid barrier, read the next CTA's word (bypassing L1) and check
// it.  CTA `absent` (if any) leaves at once without ever arriving, so everybody else's first wait runs out.
// result[0] = nanoseconds per barrier seen by CTA 0, result[1] = rounds CTA 0 completed, result[2] = payload
// mismatches seen by any CTA (must be 0).
__global__ void __launch_bounds__(256, 1)
grid_barrier_probe_kernel(unsigned int* ctr, unsigned int* payload, int rounds, int absent, unsigned long long budget_ns,
                          int* status, float* result, int variant) {
  extern __shared__ uint8_t probe_smem[];    // only there to hold the SM: one CTA per SM, as in the persistent kernels
  __shared__ int flag;
  const unsigned int n = gridDim.x;
  if ((int)blockIdx.x == absent) return;
  unsigned int gen = 0;
  int bad = 0, done = 0;
  if (threadIdx.x == 0) probe_smem[0] = 0;
  const unsigned long long t0 = gs::now_ns();
  for (int r = 0; r < rounds; ++r) {
    // variant bit 0: relaxed polls + one acquire fence instead of an acquire load per poll; bit 1: no payload (barrier alone)
    unsigned int* slot = payload + (size_t)(r & 1) * n;
    if (threadIdx.x == 0 && !(variant & 2)) slot[blockIdx.x] = (unsigned int)r * 4096u + blockIdx.x;
    if (!gs::grid_barrier(ctr, gen, n, budget_ns, &flag, (variant & 1) != 0)) {
      if (threadIdx.x == 0) latch_error(status, AD_ERR_TIMEOUT);
      break;
    }
    const unsigned int nb = (blockIdx.x + 1) % n;
    if (threadIdx.x == 0 && !(variant & 2) && __ldcg(slot + nb) != (unsigned int)r * 4096u + nb) bad++;
    ++done;
  }
  const unsigned long long t1 = gs::now_ns();
  if (threadIdx.x == 0) {
    if (bad) atomicAdd(reinterpret_cast<int*>(result + 2), bad);
    if (blockIdx.x == (absent == 0 ? 1 : 0)) {
      result[0] = done > 0 ? (float)(t1 - t0) / (float)done : 0.f;
      result[1] = (float)done;
    }
  }
}
constexpr int kProbeSmem = 160 * 1024;
}  // namespace

extern "C" int ad_debug_grid_barrier_probe(int32_t n_ctas, int32_t rounds, int32_t absent_cta, int32_t budget_us,
                                           void* scratch, size_t scratch_bytes, int32_t* status, float* result,
                                           void* stream) {
  int variant = 0;
  if (rounds < 0) { variant = (-rounds) & 3; rounds = (-rounds) >> 2; }   // timing variants of the probe (see the kernel)
  if (!scratch || !status || !result || rounds < 1 || rounds > (1 << 20) || budget_us < 1 || budget_us > (1 << 16))
    return fail(nullptr, AD_ERR_ARG, "ad_debug_grid_barrier_probe: bad argument");
  if (n_ctas <= 0) n_ctas = num_sms();
  if (absent_cta >= n_ctas) return fail(nullptr, AD_ERR_ARG, "ad_debug_grid_barrier_probe: absent_cta outside the grid");
  if (scratch_bytes < 256 + sizeof(unsigned int) * 2 * (size_t)n_ctas || reinterpret_cast<uintptr_t>(scratch) % 256)
    return fail(nullptr, AD_ERR_CAPACITY, "ad_debug_grid_barrier_probe: scratch too small or not 256-byte aligned");
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  if (cudaFuncSetAttribute(grid_barrier_probe_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kProbeSmem) != cudaSuccess)
    return fail(nullptr, AD_ERR_CUDA, "ad_debug_grid_barrier_probe: cudaFuncSetAttribute failed");
  int per_sm = 0;
  if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, grid_barrier_probe_kernel, 256, kProbeSmem) != cudaSuccess)
    return fail(nullptr, AD_ERR_CUDA, "ad_debug_grid_barrier_probe: occupancy query failed");
  if (n_ctas > per_sm * num_sms()) return fail(nullptr, AD_ERR_CAPACITY, "ad_debug_grid_barrier_probe: more CTAs than the device holds at once");
  unsigned int* ctr = static_cast<unsigned int*>(scratch);
  unsigned int* payload = ctr + 64;
  if (cudaMemsetAsync(scratch, 0, 256, st) != cudaSuccess || cudaMemsetAsync(result, 0, sizeof(float) * 4, st) != cudaSuccess)
    return fail(nullptr, AD_ERR_CUDA, "ad_debug_grid_barrier_probe: memset failed");
  unsigned long long budget_ns = (unsigned long long)budget_us * 1000ull;
  int absent = absent_cta;
  void* args[] = {&ctr, &payload, &rounds, &absent, &budget_ns, &status, &result, &variant};
  // cooperative launch: the runtime refuses the launch unless all CTAs can be resident at once
  cudaError_t e = cudaLaunchCooperativeKernel(reinterpret_cast<void*>(grid_barrier_probe_kernel), dim3(n_ctas), dim3(256), args,
                                              kProbeSmem, st);
  if (e != cudaSuccess) return fail(nullptr, AD_ERR_CUDA, std::string("ad_debug_grid_barrier_probe: ") + cudaGetErrorString(e));
  return AD_OK;
}

// ---- single-kernel entry points -----------------------------------------------------------------

namespace {
constexpr int kMaxOpTokens = 65536;   // operator-level entries: token rows per call (256-token tiles along grid.y)
}

extern "C" size_t ad_vocab_argmax_scratch_bytes(int32_t vocab, int32_t M) {
  const size_t tiles = (size_t)(vocab + 127) / 128;
  return align_up(tiles * (size_t)M * sizeof(float), 256) + align_up(tiles * (size_t)M * sizeof(int), 256);
}

namespace {

// Arg-max over tiles for M rows without any decoding state.  grid = M, block = 32.
__global__ void argmax_rows_kernel(const float* __restrict__ part_val, const int* __restrict__ part_idx, int n_tiles,
                                   int M_cap, int* __restrict__ out) {
  const int m = blockIdx.x, lane = threadIdx.x;
  float v = -INFINITY;
  int idx = 0x7fffffff;
  pdl_wait();   // the partials come from the kernel before this one
  for (int t = lane; t < n_tiles; t += 32) {
    const float ov = part_val[(size_t)m * n_tiles + t];
    const int oi = part_idx[(size_t)m * n_tiles + t];
    if (ov > v || (ov == v && oi < idx)) { v = ov; idx = oi; }
  }
  tc::warp_argmax(v, idx);
  if (lane == 0) out[m] = idx;
}

}  // namespace

extern "C" int ad_vocab_argmax(const void* x, const void* emb, int32_t dtype, int32_t M, int32_t d, int32_t vocab,
                               int32_t* argmax, void* scratch, size_t scratch_bytes, int32_t* status, void* stream) {
  if (!x || !emb || !scratch || M < 1 || d < 1 || vocab < 1) return AD_ERR_ARG;
  if (scratch_bytes < ad_vocab_argmax_scratch_bytes(vocab, M)) return AD_ERR_CAPACITY;
  if (reinterpret_cast<uintptr_t>(scratch) % 256) return AD_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  const int tiles = (vocab + 127) / 128;
  float* pv = static_cast<float*>(scratch);
  int* pi = reinterpret_cast<int*>(static_cast<char*>(scratch) + align_up((size_t)tiles * M * sizeof(float), 256));
  GemmParams p = {};
  p.K = d; p.N = vocab; p.M_ptr = nullptr; p.M_host = M; p.M_cap = M; p.part_val = pv; p.part_idx = pi; p.status = status;
  cudaError_t e;
  if (dtype == AD_DTYPE_BF16) {
    if (d % 64 || M > kMaxOpTokens) return AD_ERR_ARG;
    CUtensorMap mw, mx;
    p.ntile = clampi(pow2ceil(M), 16, 256);
    if (!make_map(&mw, emb, vocab, d, tc::BLOCK_N_FEAT) || !make_map(&mx, x, M, d, p.ntile)) return AD_ERR_CUDA;
    if (vocab_goes_persistent(d, vocab, M, nullptr)) {
      CUtensorMap mx128;
      if (!make_map(&mx128, x, M, d, tc::P_TOK)) return AD_ERR_CUDA;
      e = launch_vocab_persistent(st, mw, mx128, p, M);
    } else {
      e = launch_tc<EPI_ARGMAX>(st, mw, mx, p, M);
    }
  } else if (dtype == AD_DTYPE_FP32) {
    p.ntile = simt::TOK;
    e = launch_simt<EPI_ARGMAX>(st, emb, x, p, M);
  } else {
    return AD_ERR_ARG;
  }
  if (e != cudaSuccess) return AD_ERR_CUDA;
  if (!argmax) return AD_OK;   // projection kernel alone: partials stay in scratch
  e = launch_k(argmax_rows_kernel, dim3(M), dim3(32), 0, st, (const float*)pv, (const int*)pi, tiles, M, argmax);
  return e == cudaSuccess ? AD_OK : AD_ERR_CUDA;
}

extern "C" int ad_linear(const void* x, const void* W, const float* bias, int32_t dtype, int32_t M, int32_t K,
                         int32_t N, float* y, int32_t* status, void* stream) {
  if (!x || !W || !y || M < 1 || K < 1 || N < 1) return AD_ERR_ARG;
  cudaStream_t st = static_cast<cudaStream_t>(stream);
  GemmParams p = {};
  p.K = K; p.N = N; p.M_ptr = nullptr; p.M_host = M; p.M_cap = M; p.bias = bias; p.out_f32 = y; p.status = status;
  cudaError_t e;
  if (dtype == AD_DTYPE_BF16) {
    if (K % 64 || M > kMaxOpTokens) return AD_ERR_ARG;
    CUtensorMap mw, mx;
    p.ntile = clampi(pow2ceil(M), 16, 256);
    if (!make_map(&mw, W, N, K, tc::BLOCK_N_FEAT) || !make_map(&mx, x, M, K, p.ntile)) return AD_ERR_CUDA;
    e = launch_tc<EPI_F32>(st, mw, mx, p, M);
  } else if (dtype == AD_DTYPE_FP32) {
    p.ntile = simt::TOK;
    e = launch_simt<EPI_F32>(st, W, x, p, M);
  } else {
    return AD_ERR_ARG;
  }
  return e == cudaSuccess ? AD_OK : AD_ERR_CUDA;
}

// ---- projection + arg-max for callers that cannot allocate -------------------------------------------
// The scratch that ad_vocab_argmax takes from its caller is, here, a fixed array inside the library image.
// In host code the array's name is only a handle for the runtime, not a device address: the address is asked
// for once per device (cudaGetSymbolAddress with that device current) and then passed to the kernels.
static __device__ __align__(256) unsigned char g_static_scratch[AD_STATIC_SCRATCH_BYTES];

namespace {
void* g_static_scratch_addr[kMaxDevices] = {};
}  // namespace

extern "C" int ad_vocab_argmax_static(const void* x, const void* emb, int32_t dtype, int32_t M, int32_t d,
                                      int32_t vocab, int32_t* argmax, int32_t* status, void* stream) {
  if (!x || !emb || !argmax || M < 1 || d < 1 || vocab < 1) return fail(nullptr, AD_ERR_ARG, "ad_vocab_argmax_static: bad argument");
  const size_t need = ad_vocab_argmax_scratch_bytes(vocab, M);
  if (need > AD_STATIC_SCRATCH_BYTES)
    return fail(nullptr, AD_ERR_CAPACITY, "ad_vocab_argmax_static: problem needs " + std::to_string(need) +
                " bytes of scratch, the built-in array holds " + std::to_string((size_t)AD_STATIC_SCRATCH_BYTES));
  int dev = -1;
  if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices)
    return fail(nullptr, AD_ERR_CUDA, "ad_vocab_argmax_static: no current CUDA device");
  if (!g_static_scratch_addr[dev]) {   // first call on this device: resolve the array's device address
    void* p = nullptr;
    cudaError_t e = cudaGetSymbolAddress(&p, g_static_scratch);
    if (e != cudaSuccess || !p)
      return fail(nullptr, AD_ERR_CUDA, std::string("ad_vocab_argmax_static: cudaGetSymbolAddress: ") + cudaGetErrorString(e));
    g_static_scratch_addr[dev] = p;
  }
  const int rc = ad_vocab_argmax(x, emb, dtype, M, d, vocab, argmax, g_static_scratch_addr[dev], AD_STATIC_SCRATCH_BYTES, status, stream);
  if (rc != AD_OK)
    return fail(nullptr, rc, rc == AD_ERR_ARG ? "ad_vocab_argmax_static: unsupported shape or dtype (BF16 needs d % 64 == 0 and M <= 65536)"
                                              : "ad_vocab_argmax_static: encoding a TMA descriptor or launching a kernel failed");
  return AD_OK;
}

#ifdef AD_TRACE
// Timeline dump of a tracing build: copies up to cap stamps to the host and optionally clears the buffer.
extern "C" int ad_debug_trace(unsigned long long* host_buf, int cap, int reset) {
  unsigned int n = 0;
  if (cudaDeviceSynchronize() != cudaSuccess) return -1;
  if (cudaMemcpyFromSymbol(&n, g_trace_n, sizeof(n)) != cudaSuccess) return -1;
  if (n > (1u << 15)) n = 1u << 15;
  if ((int)n > cap) n = cap;
  if (n && cudaMemcpyFromSymbol(host_buf, g_trace_buf, sizeof(unsigned long long) * n) != cudaSuccess) return -1;
  if (reset) { unsigned int z = 0; cudaMemcpyToSymbol(g_trace_n, &z, sizeof(z)); }
  return (int)n;
}
#endif
