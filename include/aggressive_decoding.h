/*
 * aggressive_decoding.h -- C ABI of the B200 (sm_100a) verification-step library for
 * Aggressive Decoding (arXiv 2205.10350).
 *
 * The library runs, entirely in its own CUDA kernels, the hot path of the method: one forward pass of
 * an encoder-decoder Transformer decoder over a block of k drafted tokens on top of a key/value cache
 * of the accepted prefix and cached encoder keys/values, the greedy choice at every block position,
 * and the longest-accepted-prefix decision that keeps the output identical to greedy autoregressive
 * decoding (paper Sections 2, 3.1 and 3.2).
 *
 * General conventions
 *   - Every function returns an int status: AD_OK (0) or a negative AD_ERR_* code.  Nothing throws or
 *     aborts across this boundary.  ad_last_error() returns a static, human-readable string.
 *   - The library never allocates or frees device memory: the caller owns the weights and one workspace
 *     buffer and passes raw device pointers.  The handle itself is a host object owned by the library
 *     (ad_create / ad_destroy).
 *   - All token-id and length arrays are int32.  Batched arrays are row-major [B, stride].
 *   - `on_host` arguments say where the id/length arrays of THAT call live: 0 = device memory
 *     (the call is asynchronous on the handle's stream), 1 = host memory (the library copies through its
 *     staging area and the call returns after the stream has been synchronised).
 *   - Errors found by device code (a bounded wait that ran out, an invalid commit count) are latched in
 *     a status word and reported by the next synchronising call (on_host = 1 calls, ad_generate,
 *     ad_get_state, ad_sync).
 *   - A handle is used from one host thread at a time.
 *
 * Model (the paper names only "Transformer" with its sizes; what it leaves open is fixed here):
 *   post-LayerNorm encoder-decoder, ReLU feed-forward, biases on every projection, LayerNorm with
 *   biased variance, embedding scaled by sqrt(d_model) plus a sinusoidal positional table, one
 *   embedding matrix shared by encoder input, decoder input and output projection, no output bias,
 *   greedy ties broken toward the lowest token id.
 */
#ifndef AGGRESSIVE_DECODING_H_
#define AGGRESSIVE_DECODING_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum {
  AD_OK = 0,
  AD_ERR_ARG = -1,      /* invalid argument (null pointer, k out of range, commit count too large, ...) */
  AD_ERR_STATE = -2,    /* call order violated (verify before encode, commit without verify, ...) */
  AD_ERR_CAPACITY = -3, /* a size exceeds what the handle was created for, or the workspace is too small */
  AD_ERR_TIMEOUT = -4,  /* a bounded device-side wait ran out */
  AD_ERR_CUDA = -5      /* a CUDA runtime or driver call failed */
};

enum { AD_DTYPE_FP32 = 0, AD_DTYPE_BF16 = 1 };
enum { AD_MODE_IAD = 0, AD_MODE_GAD = 1 };

/* Plain-old-data description of one model family and of the capacities of a handle. */
typedef struct ad_model_cfg {
  int32_t d_model, n_heads, d_ffn, vocab, n_enc, n_dec;
  int32_t dtype;       /* AD_DTYPE_FP32: FP32 weights, FFMA arithmetic.  AD_DTYPE_BF16: BF16 weights and GEMM
                          operands on the tensor cores, FP32 accumulation, residual stream, LayerNorm, softmax */
  int32_t max_batch;   /* B capacity */
  int32_t max_src;     /* longest source (tokens) */
  int32_t max_tgt;     /* longest output (tokens); also the per-row cache capacity */
  int32_t kmax;        /* largest verification block */
  int32_t bos, pad, eos, mask;   /* special token ids */
  float ln_eps;
  int32_t has_drafter; /* 1: a second model (the non-autoregressive drafter of Section 3.2.1) is present */
} ad_model_cfg;

/*
 * Weights of one model, resident in device memory, borrowed for the lifetime of the handle.
 *   matrices: one contiguous array in the model dtype (float or bf16).  Every matrix is stored
 *     [out_features, in_features] row-major.  Order:
 *       emb [vocab, d]
 *       per encoder layer: Wqkv [3d, d] (q rows, then k, then v), Wo [d, d], W1 [F, d], W2 [d, F]
 *       per decoder layer: self Wqkv [3d, d], self Wo [d, d], cross Wq [d, d], cross Wkv [2d, d] (k then v),
 *                          cross Wo [d, d], W1 [F, d], W2 [d, F]
 *   vectors: one contiguous float array.  Order:
 *       per encoder layer: bqkv [3d], bo [d], ln1 gain [d], ln1 bias [d], b1 [F], b2 [d], ln2 gain, ln2 bias
 *       per decoder layer: self bqkv [3d], self bo [d], ln1 gain, ln1 bias, cross bq [d], cross bkv [2d],
 *                          cross bo [d], ln2 gain, ln2 bias, b1 [F], b2 [d], ln3 gain, ln3 bias
 * `matrices` must be 256-byte aligned.  ad_weight_counts() gives the two element counts.
 */
typedef struct ad_model_weights {
  const void* matrices;
  const float* vectors;
} ad_model_weights;

typedef struct ad_weights {
  ad_model_weights ar;   /* autoregressive verifier */
  ad_model_weights nar;  /* drafter; ignored unless cfg.has_drafter */
} ad_weights;

/* Options of ad_generate. */
typedef struct ad_gen_opts {
  int32_t mode;          /* AD_MODE_IAD: drafts are copied from the source (Algorithm 1).
                            AD_MODE_GAD: drafts come from the drafter (Section 3.2). */
  int32_t k;             /* block-size cap, 1..kmax.  k = 1 is plain greedy decoding. */
  const int32_t* max_len;        /* [B] per-row output cap, each 1..max_tgt; same memory space as src */
  const int32_t* draft_override; /* optional [B, override_stride]: position-aligned draft stream that replaces
                                    whatever the mode would have drafted (imposes an agreement rate when the
                                    weights are random); same memory space as src; NULL = none */
  int32_t override_stride;
  int32_t run_drafter;   /* GAD only: 1 = run the drafter forward every iteration (its block is then replaced by
                            draft_override when that is given); 0 = skip it (needs draft_override) */
  int32_t sync_every;    /* iterations between host checks of the device-side "all rows finished" word;
                            0 = library default (1) */
  int32_t use_graph;     /* 1 = run the loop as a CUDA graph: one launch whose device-side `while` node repeats the
                            captured iteration until every row has finished (bounded by the longest max_len); if
                            that graph cannot be built, one graph replay per iteration with host polling.
                            0 = launch kernels directly.
                            Ignored (direct launches) when the handle was created on the default stream,
                            which cannot be captured. */
} ad_gen_opts;

typedef struct ad_stats {
  int64_t iterations;      /* loop iterations in which at least one row was active */
  int64_t row_iterations;  /* sum over rows of the iterations that row took part in */
  int64_t accepted;        /* tokens accepted = output tokens produced */
  int64_t offered;         /* sum of block sizes offered */
  float device_ms;         /* device time of the decode loop (CUDA events), encoders excluded */
  float encode_ms;         /* device time of the encoder pass(es) */
  int64_t kernel_launches; /* kernels of this library launched by the call (a graph replay counts its kernel nodes) */
} ad_stats;

typedef struct ad_handle ad_handle;

/* Element counts of ad_model_weights.matrices / .vectors for cfg. */
int ad_weight_counts(const ad_model_cfg* cfg, size_t* matrix_elems, size_t* vector_elems);

/* Bytes of device workspace a handle for cfg needs (capacities max_batch, max_src, max_tgt, kmax). */
int ad_query_workspace(const ad_model_cfg* cfg, size_t* bytes);

/* Problem statement: "given model parameters Phi" (Algorithm 1, input line; Section 3.2).
 * Builds a handle over borrowed weights and workspace (device, >= ad_query_workspace bytes, 1024-byte
 * aligned).  `stream` is a cudaStream_t (NULL = default stream).  Computes the positional table on the
 * host and uploads it; encodes TMA descriptors for every weight matrix; copies the decoder layers' cross-attention
 * key/value projection matrices and biases into the workspace as one matrix (ad_encode then projects the encoder
 * memory for all layers in one launch), so a later change of those weights needs a new handle.  Synchronises the
 * stream. */
int ad_create(const ad_model_cfg* cfg, const ad_weights* w, void* workspace, size_t workspace_bytes,
              void* stream, ad_handle** out);
int ad_destroy(ad_handle* h);
const char* ad_last_error(const ad_handle* h);   /* h may be NULL: error of the last failed ad_create */

/* Encoder pass for a batch of B <= max_batch right-padded sources (Section 2; once per sentence, off the
 * per-step path).  src [B, src_stride], src_len [B] with 1 <= src_len[b] <= max_src.  Runs the encoder
 * stack of the verifier (and of the drafter if present) with padding keys masked, projects the memory to
 * per-decoder-layer cross-attention keys/values, and resets every row: cache length 0, last token [BOS],
 * not finished. */
int ad_encode(ad_handle* h, const int32_t* src, int32_t src_stride, const int32_t* src_len, int32_t B,
              int32_t on_host);

/* Verify substep (Section 3.2 "Verify", Eq. 7; Section 3.1.1, Eq. 3 / Eq. 6; Algorithm 1 lines 4-5).
 * drafts [B, kmax], k [B] (0 = row idle, else 1..kmax, and cache length + k <= max_tgt),
 * argmax [B, kmax] (out), n_accepted [B] (out).
 * Decoder inputs of row b are (last accepted token, drafts[b][0 .. k_b-2]) at positions
 * len_b .. len_b+k_b-1; drafts[b][k_b-1] is compared but never fed.  A negative draft is a slot that matches
 * nothing (the appended [PAD] of Algorithm 1); if fed it is replaced by [PAD].
 * argmax[b][i] is the greedy choice at block position i (lowest id on ties).
 * n_accepted[b] = (first i with argmax != draft) + 1, or k_b if none, cut at the first accepted [EOS];
 * always 1 <= n_accepted[b] <= k_b for active rows, 0 for idle rows.
 * Writes tentative keys/values for the block into the cache; does NOT change the cache length. */
int ad_verify_block(ad_handle* h, const int32_t* drafts, const int32_t* k, int32_t* argmax,
                    int32_t* n_accepted, int32_t on_host);

/* Cache-length advance or rollback (Section 3.1.1: predictions after the bifurcation are discarded;
 * Algorithm 1 lines 6-7).  n [B], or NULL = commit every row's n_accepted.
 *   0 <= n_b <= n_accepted_b : len_b += n_b, last token = argmax[b][n_b-1], accepted ids appended to the
 *                              row's output, row finishes on [EOS].  n_b = 0 discards the block.
 *   n_b < 0                  : roll back |n_b| committed tokens (|n_b| <= len_b); clears "finished".
 *   n_b > n_accepted_b       : AD_ERR_ARG, row unchanged.
 * No data moves on rollback: stale cache slots are overwritten by later blocks. */
int ad_commit(ad_handle* h, const int32_t* n, int32_t on_host);

/* Teacher forcing (Eq. 1: scoring with a known prefix): declares tokens[b][0 .. n_b) to be the next n_b output
 * tokens of row b after an ad_verify_block, whatever the verifier predicted.  tokens [B, kmax], n [B] with
 * 0 <= n_b <= k_b of that block.  The cache stays consistent only if the block fed exactly these tokens, so the
 * call requires tokens[b][i] == drafts[b][i] for i < n_b - 1 (else AD_ERR_ARG, row unchanged).  Sets
 * len_b += n_b and the last token to tokens[b][n_b-1]; the row finishes on [EOS] or at its cap.  Used to walk
 * the library along a reference trajectory position by position. */
int ad_force_commit(ad_handle* h, const int32_t* tokens, const int32_t* n, int32_t on_host);

/* Whole decoding loop (Algorithm 1; Section 3.2 loop "until [EOS] or the maximal length").  Encodes src,
 * then iterates draft -> verify -> commit on the device until every row has finished.  out [B, out_stride]
 * receives the tokens (an [EOS] included when produced), out_len [B] their count.  stats may be NULL.
 * Always synchronises before returning. */
int ad_generate(ad_handle* h, const int32_t* src, int32_t src_stride, const int32_t* src_len, int32_t B,
                const ad_gen_opts* opts, int32_t* out, int32_t out_stride, int32_t* out_len,
                ad_stats* stats, int32_t on_host);

/* Draft substep alone (Section 3.2 "Draft", Section 3.2.1): for every unfinished row run the drafter over
 * (accepted prefix, k x [MASK]) with bidirectional attention and no cache, and return its greedy choices
 * at the k mask positions.  k_cap 1..kmax; per row k_b = min(k_cap, max_len_b - len_b) with max_len = max_tgt
 * unless set by ad_generate.  drafts [B, kmax] (out), k [B] (out). */
int ad_draft_block(ad_handle* h, int32_t k_cap, int32_t* drafts, int32_t* k, int32_t on_host);

/* Copies the per-row state out: cache length, last accepted token, finished flag (each [B], may be NULL).
 * Synchronises; returns a latched device error if there is one (and clears it). */
int ad_get_state(ad_handle* h, int32_t* len, int32_t* last_tok, int32_t* finished);

/* Relaxed verification (Section 3.2.3, "GAD++", Eq. 8 and Eq. 9).  beta = 0 (the default) is the exact-match
 * verification of Eq. 7.  With beta >= 1, a block position keeps its DRAFTED token as the verified token when
 *   (Eq. 8) fewer than beta other vocabulary entries score strictly higher than the draft, i.e. the draft's
 *           log-likelihood is at least that of the beta-th ranked token, and
 *   (Eq. 9) the top-1 score exceeds the draft's score by at most tau (log-likelihoods of one position differ from
 *           the scores by a common constant, so the gap is taken on the scores),
 * and the greedy choice otherwise; n_accepted is then taken as before (first position whose verified token
 * differs from the draft, cut at an accepted [EOS]).  A sentinel draft (negative) never qualifies.  The output is
 * no longer bound to equal greedy decoding.  Applies to every later ad_verify_block and ad_generate of the
 * handle (host-side setting, no device work).  tau >= 0.  Errors: AD_ERR_ARG. */
int ad_set_acceptance(ad_handle* h, int32_t beta, float tau);

/* Waits for the handle's stream; returns and clears a latched device error. */
int ad_sync(ad_handle* h);

/* Debug: scores of the last ad_verify_block (or, with which = 1, of the last ad_draft_block) written out as
 * FP32 [M, vocab] (device pointer), M = sum of k_b, rows packed in row order.  This materialises what the
 * fused projection+argmax kernel never writes; for parity tests only. */
int ad_debug_logits(ad_handle* h, int32_t which, float* logits, size_t capacity_elems);

/* Debug: FP32 copy of the verifier's encoder memory of row b, [src_len_b, d_model] (device pointer). */
int ad_debug_encoder_memory(ad_handle* h, int32_t b, float* mem, size_t capacity_elems);

/* Debug: one verification block (arguments as ad_verify_block with host arrays) with a CUDA event in front of every
 * kernel launch and programmatic dependent launch switched off, so that every kernel's device time is bracketed on its
 * own.  names (host, capacity x 64 chars) and us (host, capacity floats) receive, in launch order, what was launched and
 * how long it took; *n_launches their count.  The block is verified as usual (not committed).  Synchronises. */
int ad_debug_profile_verify(ad_handle* h, const int32_t* drafts, const int32_t* k, char* names, float* us,
                            int32_t capacity, int32_t* n_launches);

/* Debug: stage timeline of the last persistent decoder pass.  The library has a second form of the decoder pass:
 * the whole decoder stack and the vocabulary projection as ONE persistent kernel (BF16 models with 64-wide heads,
 * passes of at most 64 packed tokens), selected with AD_MEGA=1 in the environment when the handle is created.  It
 * computes the same results as the default chain of kernels and is kept as a measured alternative (it is slower on a
 * B200 at every shape tried).  With AD_MEGA_TIMELINE=1 as well, CTA 0 of that kernel stamps the GPU's global nanosecond timer twice per stage: when the
 * stage's inputs have become visible, and after it has signalled its own part done.  stamps (host, >= 2 * n_stages
 * entries) receives them in stage order: per decoder layer QKV, self-attention, Wo, cross-Q, cross-attention, cross-Wo,
 * FFN1, FFN2; then the vocabulary projection.  Synchronises the stream. */
int ad_debug_stage_timeline(ad_handle* h, uint64_t* stamps, int32_t capacity, int32_t* n_stages);

/* Debug: exercises the bounded-wait mechanism that every mbarrier wait of the GEMM kernels uses (a wait gives up
 * after a time budget measured on the GPU's global timer: 20 ms in the kernels, budget_us here).  Launches one tiny
 * kernel that waits, for at most budget_us (1..65536) microseconds, on a barrier phase that nothing completes; the
 * wait runs out, AD_ERR_TIMEOUT is latched in *status (device int, must be 0 before) and the kernel returns
 * normally, leaving the context usable.  waited_us (device int, may be NULL) receives the time the wait took. */
int ad_debug_wait_probe(int32_t* status, int32_t budget_us, int32_t* waited_us, void* stream);

/* Debug: self-test and timing of the grid-wide barrier the persistent decoder kernel is built on (a monotonically
 * increasing arrival counter in global memory, release-add / acquire-poll, every wait bounded by time).  Launches,
 * cooperatively, n_ctas CTAs (0 = one per SM) of 256 threads holding 160 KB of shared memory each; per round every CTA
 * publishes a word, passes the barrier and checks the word of its neighbour.  absent_cta >= 0 names a CTA that leaves
 * without arriving: the others' first wait then runs out after budget_us (1..65536), AD_ERR_TIMEOUT is latched in
 * *status and the kernel returns normally.  scratch: device memory, 256-byte aligned, >= 256 + 8 * n_ctas bytes.
 * result (device float[4]): [0] nanoseconds per barrier, [1] rounds completed, [2] payload mismatches (must be 0).
 * A negative `rounds` = -(4 * rounds + v) selects a timing variant: v bit 0 = relaxed polls followed by one acquire fence instead of
 * one acquire load per poll, v bit 1 = the barrier alone, without the payload store and check.
 * Asynchronous on `stream`.  Errors: AD_ERR_ARG, AD_ERR_CAPACITY (more CTAs than fit at once), AD_ERR_CUDA. */
int ad_debug_grid_barrier_probe(int32_t n_ctas, int32_t rounds, int32_t absent_cta, int32_t budget_us, void* scratch,
                                size_t scratch_bytes, int32_t* status, float* result, void* stream);

/* ---- single-kernel entry points (operator-level tests and microbenchmarks) --------------------------
 * All pointers are device pointers; `stream` is a cudaStream_t.  Asynchronous. */

/* Output projection fused with the row arg-max (Eq. 3 / Eq. 7 "top-1"): for each of M rows of x [M, d]
 * (dtype as given) against emb [vocab, d], argmax[m] = lowest id with the largest score; the scores are
 * never written.  scratch: device memory for per-tile partial maxima, ad_vocab_argmax_scratch_bytes().
 * status: optional device int that latches AD_ERR_TIMEOUT.  BF16 needs d % 64 == 0 and M <= 65536 (more than
 * 256 rows run as 256-token tiles).
 * argmax == NULL runs the projection kernel alone and leaves its per-tile (maximum, id) partials in scratch
 * (values [M, tiles] FP32 first, ids [M, tiles] int32 from the next 256-byte boundary, tiles = ceil(vocab / 128)):
 * the launch a micro-benchmark times when it wants the projection without the final reduction. */
size_t ad_vocab_argmax_scratch_bytes(int32_t vocab, int32_t M);
int ad_vocab_argmax(const void* x, const void* emb, int32_t dtype, int32_t M, int32_t d, int32_t vocab,
                    int32_t* argmax, void* scratch, size_t scratch_bytes, int32_t* status, void* stream);

/* (No counterpart in the paper: this entry point exists for the sake of callers, not of the method.)
 * Same computation and arguments as ad_vocab_argmax, but the caller provides no scratch buffer: the per-tile
 * partial maxima live in a fixed array that is part of the library image itself.
 *
 * Who needs it: code that is not allowed to allocate device memory at the point of the call -- for example a
 * plug-in running inside a host application that owns the whole memory pool, a real-time or signal-handler-
 * like context where cudaMalloc's implicit synchronisation is unacceptable, or a process whose allocator has
 * already handed every byte to someone else.  Such callers still pass their inputs (x, emb) and the output
 * (argmax); the library neither calls cudaMalloc/cudaFree nor any routine that allocates on their behalf.
 *
 * Limits and rules
 *   - The built-in array is AD_STATIC_SCRATCH_BYTES (1 MiB) per GPU; every GPU that loads the library carries
 *     it until the process exits.  A problem needs ad_vocab_argmax_scratch_bytes(vocab, M) bytes; larger
 *     problems are refused with AD_ERR_CAPACITY (ad_last_error(NULL) then says how much was needed).
 *     1 MiB covers, e.g., vocab 32000 with M up to 256 rows, or vocab 65536 with M up to 256.
 *   - The first call on each device looks up the array's device address (cudaGetSymbolAddress, with that
 *     device current) and remembers it.  Make that first call before starting any stream capture.
 *   - All calls on a device share the one array and it keeps whatever the previous call left there.  Nothing in
 *     it has to start from zero (every partial that is read has been written by the same call), but two calls
 *     that overlap on the GPU -- different streams, or different host threads -- race on it.  Issue them on one
 *     stream, or order them with events. */
#define AD_STATIC_SCRATCH_BYTES (1u << 20)
int ad_vocab_argmax_static(const void* x, const void* emb, int32_t dtype, int32_t M, int32_t d, int32_t vocab,
                           int32_t* argmax, int32_t* status, void* stream);

/* y [M, N] (FP32) = x [M, K] W^T + bias, W [N, K] in `dtype` (Section 2 projections).  bias may be NULL.
 * BF16 needs K % 64 == 0 and M <= 65536. */
int ad_linear(const void* x, const void* W, const float* bias, int32_t dtype, int32_t M, int32_t K,
              int32_t N, float* y, int32_t* status, void* stream);

#ifdef __cplusplus
}
#endif
#endif /* AGGRESSIVE_DECODING_H_ */
