/*
 * tidar.h - C ABI of the TiDAR single-forward decode step for NVIDIA B200 (sm_100a).
 *
 * The library runs the decode path of "TiDAR: Think in Diffusion, Talk in
 * Autoregression" on one GPU: a first pass over the prompt (tidar_prefill) and
 * then identical-shape decode steps (tidar_step).  Each step is ONE transformer
 * forward over k*(k+1) token slots per sequence (paper, Section 3.3 footnote):
 * the k tokens proposed by the previous step, encoded causally against the
 * exact KV cache, plus k blocks of k mask tokens that pre-draft the next block
 * for every possible acceptance outcome (paper, Section 1, the description of
 * what one generation step carries; Section 3.2; figure "TiDAR Architecture").
 * After the forward the step keeps the longest prefix of drafts that agree with
 * the autoregressive prediction, picks the pre-draft that matches that outcome
 * and commits only the accepted tokens' KV (Section 3.2; Section 3.3, where the
 * KV of rejected tokens is dropped).
 *
 * Conventions
 *   - Every entry point returns TIDAR_OK (0) or a negative TIDAR_E* code.  Errors
 *     found on the host (EINVAL, ECAPACITY, ENOMEM) are reported before anything
 *     is launched and leave the context unchanged.  TIDAR_EDEVICE_TIMEOUT is
 *     different: a kernel's bounded wait ran out, the pass's results are invalid
 *     and the sequences it touched are released (they must be prefilled again).
 *     Nothing throws, aborts or traps.  tidar_last_error() gives a
 *     human-readable message for the last failure.
 *   - "host" / "device" on a pointer says where the memory lives.
 *   - Weights and the arena are BORROWED: the caller allocates them (for
 *     instance through PyTorch), keeps them alive until tidar_free and must
 *     not touch the arena while the context exists.
 *   - All work is enqueued on the CUDA stream given to tidar_init.  tidar_prefill
 *     and tidar_step synchronise that stream before they return the tokens.
 *   - A context is not synchronised between host threads: one thread at a time may call
 *     into it (different contexts are independent).
 *   - There is no CPU fallback: without a CUDA device tidar_init fails.
 */
#ifndef TIDAR_H_
#define TIDAR_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define TIDAR_OK               0
#define TIDAR_EINVAL          -1   /* bad argument or unsupported shape                 */
#define TIDAR_ECAPACITY       -2   /* sequence would outgrow max_seq_len / the KV pool   */
#define TIDAR_ENOMEM          -3   /* arena too small                                    */
#define TIDAR_ECUDA           -4   /* a CUDA call failed (message has the CUDA error)    */
#define TIDAR_EDEVICE_TIMEOUT -5   /* a bounded device-side wait gave up                 */

typedef struct tidar_ctx tidar_ctx;             /* opaque; owned by the library */

/* Model and capacity description; plain data, copied by tidar_init. */
typedef struct {
  int32_t n_layers, d_model, n_q_heads, n_kv_heads, head_dim, d_ffn, vocab;
  int32_t tie_lm_head;      /* informational: 1 if weights.lm_head == weights.embed        */
  float   rms_eps;          /* RMSNorm epsilon                                             */
  float   rope_theta;       /* RoPE base; rotate-half pairing (i, i + head_dim/2)          */
  int32_t mask_token_id;    /* id fed to every diffusion (mask) slot                       */
  int32_t k_max;            /* largest draft block length; k is chosen per prefill         */
  int32_t max_batch;        /* sequences a context can hold and step together              */
  int32_t max_seq_len;      /* per sequence; a step needs n + 2k <= max_seq_len            */
  int32_t page_size;        /* KV page length in tokens (64)                               */
  float   beta;             /* verification mix in [0, 1] (paper Section 4.4.3): a draft is checked
                               against argmax(beta * logits_ar + (1 - beta) * logits_diff).
                               1.0 (verification by the autoregressive prediction alone) is
                               the hot path and makes greedy TiDAR equal greedy AR decoding;
                               below 1 every verified position costs one more LM-head row  */
  float   temperature;      /* 0 = greedy (the hot path).  > 0: every prediction (verified
                               targets and drafts alike) is a draw from softmax(logits /
                               temperature) by the Gumbel-max rule, and a draft is accepted
                               iff it equals the drawn target (paper Section 3.2 read as
                               token match).  The noise of a draw is a pure function of
                               (sample_seed, sequence slot, predicted position, token id):
                               SplitMix64's mix of (seed, slot, position) gives a 32-bit key,
                               MurmurHash3's fmix32(key + id * 0x9E3779B9) the 24 uniform bits
                               of -ln(-ln u).  Draws therefore do not depend on how positions
                               fall into passes, and with beta = 1 the emitted sequence equals
                               one-token-per-pass sampling with the same rule                */
  uint64_t sample_seed;     /* seed of the sampling noise                                  */
  int32_t debug;            /* bit 0: keep per-layer hidden states and full logits of the
                               last pass for the tidar_debug_get_* calls (costs memory:
                               rows*vocab*4 bytes); bit 1: overwrite evicted KV slots with
                               the largest finite bf16 after each step (any use of them
                               with a non-zero weight would wreck the results); bit 2:
                               keep the split-K partial sums of the projections in bf16
                               instead of fp32 (about 4 % faster, about 20 % more rounding
                               noise in deep models; off by default); bit 3: launch the
                               kernels of a step one by one instead of replaying a captured
                               graph (A/B diagnostics)                                    */
  int32_t impl;             /* 0: tensor-core kernels (tcgen05/TMEM/TMA);
                               1: plain fp32-accumulate CUDA-core kernels ("replay"), a
                               slow diagnostic path with the same data flow               */
  int32_t prefill_rows;     /* rows one pass of the first pass (and of tidar_score) may carry;
                               0 = as many as a decode step (max_batch*k_max*(k_max+1), at
                               least 256).  With a larger value a long prompt is encoded in
                               few passes and every weight tile, once fetched, serves all row
                               blocks of the pass, so the first pass is bound by the tensor
                               cores instead of re-streaming the weights per 272 rows; costs
                               activation memory in proportion                             */
} tidar_config;

/* BORROWED device pointers.  Matrices are bf16, row-major [out_features][in_features].
 *   wqkv[l]      : [(n_q_heads + 2*n_kv_heads)*head_dim][d_model], rows = Q heads, K heads, V heads
 *   wo[l]        : [d_model][n_q_heads*head_dim]
 *   w_gate_up[l] : [2*d_ffn][d_model], row 2f = gate row f, row 2f+1 = up row f (interleaved so
 *                  that one tile of output rows holds matching gate/up pairs)
 *   w_down[l]    : [d_model][d_ffn]
 *   embed, lm_head : [vocab][d_model];  *_norm : [d_model] bf16 gains
 * The per-layer arrays are HOST arrays of n_layers device pointers.
 * Optional (NULL = absent; the paper starts from Qwen2.5 and Qwen3 decoders, Section 4.1,
 * whose attention blocks differ in these two details):
 *   bqkv[l]   : [(n_q_heads + 2*n_kv_heads)*head_dim] bf16, bias added to the QKV projection
 *   q_norm[l], k_norm[l] : [head_dim] bf16 gains of an RMSNorm (rms_eps) over the dimensions of
 *               every Q head / K head, applied before RoPE; given together or not at all   */
typedef struct {
  const void *embed, *lm_head, *final_norm;
  const void *const *attn_norm, *const *wqkv, *const *wo;
  const void *const *ffn_norm, *const *w_gate_up, *const *w_down;
  const void *const *bqkv, *const *q_norm, *const *k_norm;
} tidar_weights;

/* Bytes of device memory the context needs for cfg (KV pages, activations, scratch).
 * The caller allocates that much (256-byte aligned) and passes it to tidar_init.  */
int tidar_arena_bytes(const tidar_config *cfg, size_t *out_bytes);

/* Validate cfg, adopt the weights and the arena, build TMA descriptors, create the
 * context.  cuda_stream is a cudaStream_t (NULL = default stream).
 * Errors: EINVAL (shape not supported: head_dim must be 64 or 128, d_model and d_ffn
 * multiples of 64, page_size 64, ...), ENOMEM (arena_bytes too small), ECUDA.      */
int tidar_init(const tidar_config *cfg, const tidar_weights *weights,
               void *arena /*device*/, size_t arena_bytes, void *cuda_stream, tidar_ctx **out);

/* First pass for sequence slot `seq` (0 <= seq < max_batch), replacing whatever the
 * slot held (paper, Section 3.2, how generation begins; Appendix B, the prefill mask):
 * the prompt is encoded causally and its KV cached; one block of k mask tokens is
 * appended with bidirectional attention.  Emits the first settled token (argmax of
 * the last prompt row) to *out_first_token and stores the first draft block.
 * Needs 1 <= n_prompt, 1 <= k <= k_max, n_prompt + 2k <= max_seq_len.             */
int tidar_prefill(tidar_ctx *ctx, int32_t seq, const int32_t *prompt_ids /*host*/, int32_t n_prompt,
                  int32_t k, int32_t *out_first_token /*host*/);

/* One decode step for the listed sequences (all prefilled with the same k): paper,
 * Section 3.2 (verify the previous step's drafts against the autoregressive predictions
 * of the same pass, keep the longest agreeing prefix, hand the matching pre-draft to the
 * next step) with the slot layout of the Section 3.3 footnote and the attention mask of
 * figure "TiDAR Attention Masks".
 * forced_accept: NULL, or per sequence 0 = natural acceptance, L in [1,k] = accept
 * exactly L slots whatever the drafts were (benchmark hook; not in the paper).
 * On return out_n[i] = L_i and out_tokens[i*k_max .. i*k_max+L_i) = the L_i new tokens:
 * the accepted drafts followed by the freshly verified token.  The committed KV
 * length of sequence i grows by L_i; rejected slots are evicted.
 * Errors: EINVAL, ECAPACITY (n + 2k > max_seq_len, checked before any launch).     */
int tidar_step(tidar_ctx *ctx, const int32_t *seqs /*host,[n_seqs]*/, int32_t n_seqs,
               const int32_t *forced_accept /*host,[n_seqs] or NULL*/,
               int32_t *out_tokens /*host,[n_seqs][k_max]*/, int32_t *out_n /*host,[n_seqs]*/);

/* Same as tidar_step but returns after enqueueing; tidar_step_wait blocks until the OLDEST
 * enqueued step has finished and hands out its results.  Forced acceptance lengths are
 * required (the host must know every sequence's length to check capacity without reading
 * the device); the sequences' lengths are advanced when the step is enqueued.  A second step
 * may be enqueued while the first is still in flight (two at most), so that the device never
 * waits for the host between steps; a third, or a second one when per-step diagnostics are on
 * (debug bits 0 / 3, timing, timeline), returns TIDAR_EINVAL.  Every other entry point that
 * touches sequences returns TIDAR_EINVAL while a step is in flight.  If a step reports
 * TIDAR_EDEVICE_TIMEOUT, the sequences of the step behind it are released as well.          */
int tidar_step_async(tidar_ctx *ctx, const int32_t *seqs, int32_t n_seqs, const int32_t *forced_accept);
int tidar_step_wait(tidar_ctx *ctx, int32_t *out_tokens /*host,[n_seqs][k_max]*/, int32_t *out_n /*host*/);

/* A decode step with a block length chosen for this step (paper Section 5: the block length
 * can follow the compute profile; with B sequences the step has B*k*(k+1) token slots, and
 * those are "free" only while the pass stays memory-bound).  1 <= k <= k_max.  The step uses
 * the first k entries of each sequence's block; where a sequence holds fewer drafts than k
 * (its previous pass ran a shorter block, or it was an autoregressive step) the missing drafts
 * are fed as mask tokens and are never accepted, so such a step emits fewer tokens but leaves a
 * full block of k behind.  Everything else as tidar_step.                                 */
int tidar_step_k(tidar_ctx *ctx, const int32_t *seqs /*host,[n_seqs]*/, int32_t n_seqs, int32_t k,
                 const int32_t *forced_accept /*host or NULL*/, int32_t *out_tokens /*host,[n_seqs][k_max]*/,
                 int32_t *out_n /*host,[n_seqs]*/);

/* A decode step in which listed sequence i uses its own block length ks[i] (host, [n_seqs], each in
 * [1, k_max]); the paper's Section 5 lets the block length follow the compute profile and nothing in
 * the method ties the sequences of a batch to one length.  The pass has sum_i ks[i]*(ks[i]+1) token
 * slots, sequence after sequence.  Per sequence the results are those of tidar_step_k with that
 * sequence's length (same tokens; hidden states up to the rounding of a different row count).
 * forced_accept[i] in [0, ks[i]].  Equal lengths take tidar_step_k's path.  With beta < 1 the mixed
 * verification rows (one per verified position) follow the slots, sequence after sequence.
 * out_tokens / out_n as in tidar_step.                                                        */
int tidar_step_ks(tidar_ctx *ctx, const int32_t *seqs /*host,[n_seqs]*/, int32_t n_seqs, const int32_t *ks /*host,[n_seqs]*/,
                  const int32_t *forced_accept /*host or NULL*/, int32_t *out_tokens /*host,[n_seqs][k_max]*/,
                  int32_t *out_n /*host,[n_seqs]*/);

/* The block length that keeps a step of n_seqs sequences within row_budget token slots:
 * the largest k <= k_max with n_seqs*k*(k+1) <= row_budget (at least 1).  row_budget <= 0
 * selects 288, one row block of the projection kernels, about where the 8B-class step
 * leaves the memory-bound region on a B200 (measured ridge: 220 .. 288 rows).  Host only. */
int tidar_ridge_k(const tidar_ctx *ctx, int32_t n_seqs, int32_t row_budget);

/* Block lengths for one step of a batch under a budget of token slots (paper Section 5: the extra
 * slots are free only while the pass stays memory-bound, and a scheduler should spend them where they
 * can yield tokens).  want[i] (host, [n_seqs], or NULL) caps the block of sequence i, e.g. at the number
 * of tokens it still has to produce; out_ks[i] (host, [n_seqs]) receives a length in
 * [1, min(k_max, want[i])].  The plan maximises sum_i out_ks[i] subject to
 * sum_i out_ks[i]*(out_ks[i]+1) <= row_budget by always lengthening the shortest block that may still
 * grow (one more draft at length k costs 2(k+1) slots); when even length 1 everywhere exceeds the
 * budget every sequence gets 1.  row_budget <= 0 selects 288 as in tidar_ridge_k.  Feed the result to
 * tidar_step_ks.  Host only, needs no context or device.  TIDAR_EINVAL for a non-positive n_seqs,
 * k_max or want[i], or a null out_ks.                                                          */
int tidar_plan_ks(int32_t n_seqs, int32_t k_max, int32_t row_budget, const int32_t *want /*host or NULL*/, int32_t *out_ks /*host*/);

/* Returns a sequence slot's KV pages to the pool and marks it not prefilled, so that another prompt
 * can take the slot (sequences of a batch finish at different times; a step lists any subset of the
 * prefilled slots).  A slot that holds nothing is left as it is.  TIDAR_EINVAL while a step is in
 * flight or for a slot outside [0, max_batch).                                                   */
int tidar_release(tidar_ctx *ctx, int32_t seq);

/* One plain autoregressive step (paper Section 3.1: the model keeps a causal, chain-factorised
 * mode): a single causal slot per sequence, the settled token at position n, no mask slots.
 * Emits exactly one token per sequence (out_tokens[i]) and leaves a block that holds that
 * token alone, so a later tidar_step_k finds no drafts and accepts one token on its first
 * pass.  The baseline the paper's speed-ups are quoted against (Section 4.3).             */
int tidar_ar_step(tidar_ctx *ctx, const int32_t *seqs /*host,[n_seqs]*/, int32_t n_seqs, int32_t *out_tokens /*host,[n_seqs]*/);

/* Likelihood scoring in the autoregressive mode (paper Section 3.1, the chain-factorised joint
 * distribution; Section 4.2, likelihood tasks): one causal pass over ids[0..n) and
 * logprobs[i] = log softmax(logits at position i)[ids[i+1]] for i in [0, n-1).
 * Uses sequence slot `seq` as scratch: whatever it held is dropped and the slot is left
 * empty.  The log-sum-exp runs over vocabulary chunks; full logits are never kept.
 * Needs 2 <= n <= max_seq_len.  Synchronises the stream.                                  */
int tidar_score(tidar_ctx *ctx, int32_t seq, const int32_t *ids /*host,[n]*/, int32_t n, float *logprobs /*host,[n-1]*/);

/* Release the context (host state only; arena and weights belong to the caller). */
int tidar_free(tidar_ctx *ctx);

/* Message for the most recent error on ctx (or for the last failed tidar_init when
 * ctx is NULL).  The pointer stays valid until the next call on the same ctx.     */
const char *tidar_last_error(const tidar_ctx *ctx);

/* Committed KV length n of a sequence slot (host bookkeeping), or a negative code. */
int tidar_seq_len(const tidar_ctx *ctx, int32_t seq);

/* Number of kernels the library launched since tidar_init (for launch accounting). */
int64_t tidar_launch_count(const tidar_ctx *ctx);

/* ---- rewind / teacher forcing (parity tests) ------------------------------------ */
/* Overwrite the next step's causal section of a sequence: block[0] is the settled
 * token at position n, block[1..k) the drafts.                                      */
int tidar_debug_set_block(tidar_ctx *ctx, int32_t seq, const int32_t *block /*host,[k]*/);
int tidar_debug_get_block(tidar_ctx *ctx, int32_t seq, int32_t *block /*host,[k]*/);
/* Results of the last pass; need cfg.debug bit 0.  Row r of a decode step is slot
 * r % (k*(k+1)) of the (r / (k*(k+1)))-th listed sequence; with beta < 1 the rows that mix
 * causal slot j with the first slot of block j follow all slots (k per sequence).  For a
 * prefill the rows are the last chunk's rows (see tidar_debug_last_rows).            */
int tidar_debug_last_rows(const tidar_ctx *ctx, int32_t *n_rows, int32_t *first_row_position);
int tidar_debug_get_logits(tidar_ctx *ctx, int32_t row0, int32_t n_rows, float *out /*host,[n_rows][vocab]*/);
/* layer in [0, n_layers]: input of that layer; n_layers = input of the final norm. */
int tidar_debug_get_hidden(tidar_ctx *ctx, int32_t layer, int32_t row0, int32_t n_rows,
                           float *out /*host,[n_rows][d_model]*/);
int tidar_debug_get_argmax(tidar_ctx *ctx, int32_t row0, int32_t n_rows, int32_t *out /*host*/);
/* Cached K and V (bf16 bit patterns) of positions [pos0, pos0+npos) in canonical
 * [npos][n_kv_heads][head_dim] order, gathered from the pages.                     */
int tidar_debug_get_kv(tidar_ctx *ctx, int32_t seq, int32_t layer, int32_t pos0, int32_t npos,
                       uint16_t *k_out /*host*/, uint16_t *v_out /*host*/);
/* Per-kernel-class device time (ms) of the last pass, measured with CUDA events when
 * enabled with tidar_debug_set_timing(ctx, 1).  classes: see TIDAR_TC_* below.     */
#define TIDAR_TC_EMBED   0
#define TIDAR_TC_NORM    1
#define TIDAR_TC_GEMM    2
#define TIDAR_TC_ROPE    3
#define TIDAR_TC_ATTN    4
#define TIDAR_TC_LMHEAD  5
#define TIDAR_TC_VERIFY  6
#define TIDAR_TC_COUNT   7
int tidar_debug_set_timing(tidar_ctx *ctx, int32_t on);
/* Skipped-tile evidence for the attention kernel.  While `on`, every CTA of the tensor-core
 * attention kernel adds the number of 64-key tiles it visits to a device counter.  Each call
 * returns the count accumulated since the previous call in *visited (may be NULL), clears it
 * and sets the switch.  Synchronises the stream.  A dense mask would visit, per 128-row query
 * tile and KV head, every 64-key tile of [cache | step slots].                          */
int tidar_debug_count_attention_tiles(tidar_ctx *ctx, int32_t on, uint64_t *visited /*host*/);
/* In-kernel timeline of a decode step, for the launch mode the benchmark times (replayed
 * graph, programmatic launches), where events cannot be put between kernels without changing
 * the schedule.  While enabled, every kernel of a step records, in two device words of its
 * own, the earliest moment one of its CTAs got past the dependency on the previous kernel and
 * the latest moment one finished (%globaltimer).  After the step, class_ms[cls] is the sum of
 * (end - start) over the launches of a class (TIDAR_TC_*), *busy_ms the sum over all launches
 * and *span_ms the time from the first start to the last end.  Costs two atomics per CTA;
 * switching it on or off re-captures the step's graph.  impl 0 only.                    */
int tidar_debug_set_timeline(tidar_ctx *ctx, int32_t on);
int tidar_debug_get_timeline(tidar_ctx *ctx, float *class_ms /*host,[TIDAR_TC_COUNT]*/, float *busy_ms /*host, or NULL*/,
                             float *span_ms /*host, or NULL*/);
/* Exercises the bounded wait the tensor-core kernels are built on: enqueues a one-thread kernel
 * that waits, for at most limit_polls polls (a few milliseconds at 2^14), on a barrier that
 * nothing arrives on, gives up and sets the status word.  tidar_sync then returns
 * TIDAR_EDEVICE_TIMEOUT and the context stays usable.  impl 0 only.                       */
int tidar_debug_wait_probe(tidar_ctx *ctx, int32_t limit_polls);
/* Test hook for the error plumbing: writes `value` into the device status word that the
 * kernels set when a bounded wait gives up.  The next tidar_step / tidar_prefill /
 * tidar_sync then reports TIDAR_EDEVICE_TIMEOUT exactly as after a real timeout.  No
 * kernel is made to wait.                                                             */
int tidar_debug_force_status(tidar_ctx *ctx, int32_t value);
int tidar_debug_get_timing(tidar_ctx *ctx, float *ms /*host,[TIDAR_TC_COUNT]*/);

/* ---- structured-mask attention alone (microbenchmark and unit parity) -------------
 * The attention of one decode step under the mask of the paper's figure "TiDAR Attention
 * Masks" (Section 3.1: drafted tokens causal, each mask block bidirectional within itself
 * and blind to the other blocks), on caller-provided tensors (all DEVICE, bf16, 16-byte
 * aligned):
 *   q        [n_seqs*T][n_q_heads][head_dim], T = k*(k+1), slot order of a decode step
 *   k_pages, v_pages : page pools [n_pages][n_kv_heads][page_size][head_dim]; the
 *              cached prefix AND the k causal slots of the step (positions n..n+k-1)
 *              live there.  Whole pages may be loaded: positions a row does not see
 *              get weight zero, so they must hold finite values (not NaN/inf)
 *   page_table [n_seqs][pages_per_seq] int32, seq_len [n_seqs] int32 (= n per sequence)
 *   k_local, v_local [n_seqs*k*k][n_kv_heads][head_dim] : K/V of the mask slots
 *   out      [n_seqs*T][n_q_heads*head_dim]
 * Mask per the decode-step definition: causal slot j sees positions < n+j+1; mask
 * slot (b,i) sees positions < n+b+1 plus the k local slots of block b.
 * seq_len values are clamped to [0, pages_per_seq*page_size - k]; page indices outside
 * [0, n_pages) contribute nothing (impl 1) or zeros (impl 0: out-of-range tiles load as 0).
 * Uses ctx only for its stream, kernel implementation choice and scratch.
 * Errors: EINVAL (null or misaligned pointer, row capacity), ECUDA.                  */
int tidar_attention(tidar_ctx *ctx, const void *q, const void *k_pages, const void *v_pages,
                    int32_t n_pages, const int32_t *page_table, int32_t pages_per_seq, const int32_t *seq_len,
                    const void *k_local, const void *v_local, void *out,
                    int32_t n_seqs, int32_t k);

/* ---- one projection alone (microbenchmark and unit parity) ----------------------------
 * out[r][n] = sum_k A[r][k] * W[n][k]: the weight-streaming small-M GEMM every projection
 * of a step uses (QKV, O, gate/up, down, LM head; the step's k(k+1) token slots share one
 * pass over the weights: paper Section 1, where extra token slots cost next to nothing while
 * the pass is bound by loading the weights).
 *   A [R][K] bf16, W [N][K] bf16, out [R][N] fp32, all DEVICE, row-major, 16-byte aligned;
 *   K a multiple of 64.  splits: K splits (1..8), 0 = the library's own choice; partial
 *   sums are combined in a fixed order, so the result is deterministic.
 * Enqueued on the context's stream; does not synchronise (see tidar_sync).
 * Errors: EINVAL, ECAPACITY (R*N*splits exceeds the context's scratch), ECUDA.          */
int tidar_gemm(tidar_ctx *ctx, const void *A, const void *W, int32_t R, int32_t N, int32_t K,
               int32_t splits, float *out);

/* Wait for everything enqueued on the context's stream and report a device-side
 * timeout (TIDAR_EDEVICE_TIMEOUT) if a kernel's bounded wait gave up (results of the
 * calls since the last check are then invalid).                                        */
int tidar_sync(tidar_ctx *ctx);

/* ---- structured-mask attention for callers that cannot allocate ---------------------
 * (The paper has no counterpart: this is a packaging variant of tidar_attention.)
 * Same mask, same tensor layouts and the same result (within rounding) as
 * tidar_attention, but it needs no context and no arena: the shapes come as plain
 * arguments and the per-row visibility table, which tidar_attention keeps in the
 * caller-allocated arena, lives in a fixed table built into the library image.  It is
 * meant for hosts that hold device tensors but may not call an allocator where they need
 * attention: a server whose memory pool belongs wholly to another component, a loop that
 * must not enter the allocator (cudaMalloc may stall every stream of the device), a
 * plug-in that is handed buffers only.
 * The call performs no cudaMalloc/cudaFree and calls no allocating routine.
 *   - It always runs the plain CUDA-core kernel (one warp per row and query head, fp32
 *     accumulation, K/V re-read once per query head, no tile skipping), not the
 *     tensor-core kernel: correct and allocation-free, not fast (measured at 32 / 8 heads,
 *     k = 16: 1.1 ms against 28 us for tidar_attention with impl 0 at a thousand cached
 *     positions, 4.2 ms against 45 us at four thousand).
 *   - Limit: n_seqs * k * (k+1) <= 4352 rows (16 sequences at k = 16); beyond that the
 *     call returns TIDAR_ECAPACITY and launches nothing.  page_size is 64.
 *   - Each GPU that loads the library holds the table (85 KiB) until the process exits.
 *   - The first call on a device looks up the table's device address (with that device
 *     current); make that first call outside any stream capture.  The look-up is not
 *     synchronised between host threads: concurrent first calls are harmless (they store
 *     the same address) but not ordered.
 *   - All calls on one device share the table and each call rewrites the entries it uses,
 *     so nothing needs clearing; but two calls whose kernels may overlap on the GPU
 *     (different streams, no ordering between them) race on it.  Serialise them.
 *   - Work is enqueued on cuda_stream (a cudaStream_t, NULL = default) of the current
 *     device; the call does not synchronise.  All data pointers are DEVICE pointers,
 *     16-byte aligned (page_table, seq_len: 4-byte).  seq_len values are clamped to
 *     [0, pages_per_seq*64 - k]; keys on pages outside [0, n_pages) are skipped; a row
 *     left without any visible key gets zeros.
 * Errors: TIDAR_EINVAL, TIDAR_ECAPACITY, TIDAR_ECUDA; message via tidar_last_error(NULL). */
int tidar_attention_static(const void *q, const void *k_pages, const void *v_pages, int32_t n_pages,
                           const int32_t *page_table, int32_t pages_per_seq, const int32_t *seq_len,
                           const void *k_local, const void *v_local, void *out,
                           int32_t n_seqs, int32_t k, int32_t n_q_heads, int32_t n_kv_heads,
                           int32_t head_dim, void *cuda_stream);

#ifdef __cplusplus
}
#endif
#endif  /* TIDAR_H_ */
