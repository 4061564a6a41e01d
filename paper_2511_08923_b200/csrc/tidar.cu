// C-ABI entry points and per-step orchestration of the TiDAR decode path.
#include "../../include/tidar.h"

#include <algorithm>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <string>
#include <deque>
#include <vector>

#include "common.cuh"
#include "kernels_basic.cuh"
#include "kernels_replay.cuh"
#include "gemm_tc.cuh"
#include "attn_tc.cuh"

namespace {

std::string g_init_error;

struct SeqState {
  int n = 0;            // committed KV length
  int k = 0;            // draft block length of the sequence's last pass (entries its block holds)
  bool active = false;
  std::vector<int> pages;
};

struct TimedLaunch { int cls; cudaEvent_t a, b; };

}  // namespace

struct tidar_ctx {
  tidar_config cfg;
  cudaStream_t stream = nullptr;
  // borrowed weights
  const bf16 *embed = nullptr, *lm_head = nullptr, *final_norm = nullptr;
  std::vector<const bf16 *> attn_norm, wqkv, wo, ffn_norm, wgu, wdown;
  std::vector<const bf16 *> bqkv, q_norm, k_norm;      // optional (empty = absent)
  // geometry
  int R_head = 0;                  // rows of a pass that can get logits (the rows of a decode step)
  int head_row0 = 0;               // first row of the current pass that the LM head runs on
  int last_hidden_off = 0;         // first row of the last pass that the read-back calls address
  int R_cap = 0, T_max = 0, pages_per_seq = 0, n_pages = 0, n_qkv = 0, S_max = 4, lm_chunk = 0;
  size_t pool_stride = 0;    // elements in one layer's K (or V) pool
  size_t partial_stride = 0; // elements between split-K partial slabs
  size_t partials_cap = 0;   // floats in `partials`
  // arena carve-out (device)
  bf16 *kv = nullptr;
  RowMeta meta{};
  int32_t *d_blk_len = nullptr;    // [max_batch]: drafts a sequence's block holds (the block length of its last pass)
  // a step whose sequences use different block lengths: per listed sequence its k, first row, first local row;
  // per query tile of the attention kernel its first row and the end of its sequence's rows
  int32_t *d_step_k = nullptr, *d_step_off = nullptr, *d_step_loc = nullptr, *d_tile_row0 = nullptr, *d_tile_rend = nullptr;
  int32_t *h_lay = nullptr;        // pinned staging for those five arrays
  size_t lay_ints = 0;
  int mixed_tiles = 0;             // query tiles of the current mixed step
  float *d_run_max = nullptr, *d_run_sum = nullptr, *d_tgt_logit = nullptr, *d_logprob = nullptr;   // likelihood scoring, per row
  int32_t *d_target = nullptr;
  std::vector<CUtensorMap> tm_lm_chunks;   // the LM head in vocabulary chunks of lm_chunk rows (scoring)
  int32_t *d_seq_len = nullptr, *d_block = nullptr, *d_page_table = nullptr, *d_step_seqs = nullptr, *d_forced = nullptr,
          *d_step_n = nullptr, *d_step_L = nullptr, *d_out = nullptr, *d_prompt = nullptr, *d_arg_idx = nullptr;
  float *X = nullptr, *partials = nullptr, *rope_cos = nullptr, *rope_sin = nullptr, *d_arg_val = nullptr,
        *dbg_hidden = nullptr, *dbg_logits = nullptr;
  bf16 *A = nullptr, *Q = nullptr, *Kloc = nullptr, *Vloc = nullptr, *O = nullptr, *H = nullptr, *dbg_kv = nullptr;
  // host state
  std::vector<SeqState> seqs;
  std::vector<int> free_pages;
  int32_t *h_pinned = nullptr;     // [max_batch*(k_max+1)] results + staging
  std::string err;
  int64_t launches = 0;
  // last pass
  int last_rows = 0, last_first_pos = 0;
  // Steps that have been enqueued and not yet waited for, oldest first.  Two may be in flight when every
  // acceptance length is forced (the host then knows the lengths without reading the device): the second
  // is enqueued while the first runs, so the device never waits for the host between steps.
  struct Flight { std::vector<int> seqs, ks; int k = 0, slot = 0; bool counted = false; };
  std::deque<Flight> inflight;
  cudaEvent_t flight_done[2] = {nullptr, nullptr};
  int32_t *h_out2[2] = {nullptr, nullptr}, *h_stage2[2] = {nullptr, nullptr}, *h_status2[2] = {nullptr, nullptr};   // pinned, one set per slot
  int32_t *h_page_table = nullptr;   // pinned mirror of the page table: the source of its (asynchronous) updates
  int next_slot = 0;
  // tensor-core path
  gemm_tc::EncodeTiledFn encode = nullptr;
  std::vector<CUtensorMap> tm_wqkv, tm_wo, tm_wgu, tm_wdown;
  CUtensorMap tm_lm;
  struct AMap { const void *p; int rows, cols, box; CUtensorMap tm; };
  std::vector<AMap> amaps;
  CUtensorMap tm_q, tm_kv, tm_kloc, tm_vloc;
  float *attn_part_O = nullptr, *attn_part_ml = nullptr;
  int n_sms = 0;
  // the launches of one decode step as an executable graph, valid for one (k, n_seqs, attention split)
  struct StepGraph { int k = 0, n_seqs = 0, splits = 0, mixed_R = 0, tiles = 0, mixed_K = 0; bool ar = false, timeline = false; cudaGraphExec_t exec = nullptr; int64_t launches = 0; } sg;
  bool graphs_ok = true;
  bool slab_bf16 = false;          // split-K partial sums of the step in bf16 instead of fp32 (config debug bit 2)
  int32_t *d_status = nullptr, *cand_idx = nullptr;
  float *cand_val = nullptr;
  // in-kernel timeline (diagnostics): two words per launch of the last recorded step
  static constexpr int TL_MAX = 2048;
  unsigned long long *d_tl = nullptr;
  bool timeline = false; int tl_n = 0; std::vector<int> tl_cls;
  bool count_tiles = false;        // the attention kernel adds the key tiles it visits to d_tl[2 * TL_MAX]
  float tl_class_ms[TIDAR_TC_COUNT] = {}; float tl_span_ms = 0.f, tl_busy_ms = 0.f;
  // timing
  bool timing = false; std::vector<TimedLaunch> timed; float class_ms[TIDAR_TC_COUNT] = {};
  int cur_class = 0;
};

namespace {

int fail(tidar_ctx *c, int code, const char *fmt, ...) {
  char buf[512];
  va_list ap; va_start(ap, fmt); vsnprintf(buf, sizeof buf, fmt, ap); va_end(ap);
  if (c) c->err = buf; else g_init_error = buf;
  return code;
}

#define CUDA_TRY(c, call)                                                                     \
  do {                                                                                        \
    cudaError_t e_ = (call);                                                                  \
    if (e_ != cudaSuccess) return fail((c), TIDAR_ECUDA, "%s: %s", #call, cudaGetErrorString(e_)); \
  } while (0)

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Lays the arena out; with base == nullptr only measures.
struct Carver {
  char *base; size_t off = 0;
  explicit Carver(void *b) : base((char *)b) {}
  template <typename T> T *take(size_t n) {
    off = align_up(off, 256);
    T *p = base ? (T *)(base + off) : nullptr;
    off += n * sizeof(T);
    return p;
  }
};

int validate(const tidar_config &c, std::string &why) {
  auto bad = [&](const char *m) { why = m; return TIDAR_EINVAL; };
  if (c.n_layers < 1 || c.d_model < 64 || c.vocab < 2 || c.d_ffn < 64) return bad("n_layers, d_model, d_ffn, vocab must be positive");
  if (c.head_dim != 64 && c.head_dim != 128) return bad("head_dim must be 64 or 128");
  if (c.n_kv_heads < 1 || c.n_q_heads < 1 || c.n_q_heads % c.n_kv_heads) return bad("n_q_heads must be a positive multiple of n_kv_heads");
  if (c.n_q_heads / c.n_kv_heads > 128) return bad("at most 128 query heads per KV head (one 128-row attention tile)");
  if (c.d_model > 12288) return bad("d_model above 12288 is not supported (row buffer of the norm kernel)");
  if (c.d_model % 64 || c.d_ffn % 64) return bad("d_model and d_ffn must be multiples of 64");
  if (c.page_size != 64) return bad("page_size must be 64");
  if (c.k_max < 1 || c.k_max > 32) return bad("k_max must be in [1, 32]");
  if (c.max_batch < 1 || c.max_seq_len < 2 * c.k_max + 1) return bad("max_batch >= 1 and max_seq_len > 2*k_max required");
  if (c.mask_token_id < 0 || c.mask_token_id >= c.vocab) return bad("mask_token_id out of range");
  if (!(c.beta >= 0.0f && c.beta <= 1.0f)) return bad("beta must be in [0, 1]");
  if (!(c.temperature >= 0.0f) || c.temperature > 1e4f) return bad("temperature must be in [0, 1e4] (0 = greedy)");
  if (c.impl != 0 && c.impl != 1) return bad("impl must be 0 (tensor-core kernels) or 1 (replay kernels)");
  if (c.prefill_rows < 0 || c.prefill_rows > (1 << 16)) return bad("prefill_rows must be in [0, 65536]");
  if (!(c.rms_eps > 0.f) || !(c.rope_theta > 1.f)) return bad("rms_eps > 0 and rope_theta > 1 required");
  return TIDAR_OK;
}

void layout(tidar_ctx &x, void *arena, size_t *bytes) {
  const tidar_config &c = x.cfg;
  x.T_max = c.k_max * (c.k_max + 1);
  // rows of a pass: the step's slots, plus one mixed row per verified position when beta < 1
  x.R_head = (int)align_up((size_t)std::max(c.max_batch * (x.T_max + (c.beta < 1.0f ? c.k_max : 0)), 256), 16);
  x.R_cap = std::max(x.R_head, (int)align_up((size_t)std::max(c.prefill_rows, 0), 16));
  x.pages_per_seq = (c.max_seq_len + c.page_size - 1) / c.page_size;
  x.n_pages = x.pages_per_seq * c.max_batch;
  x.n_qkv = (c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
  x.pool_stride = (size_t)x.n_pages * c.n_kv_heads * c.page_size * c.head_dim;
  x.lm_chunk = std::min(c.vocab, 16384);
  x.S_max = c.impl == 0 ? 8 : 4;
  const size_t R = x.R_cap;
  const size_t widest = std::max<size_t>({(size_t)x.S_max * x.n_qkv, (size_t)x.S_max * c.d_model, (size_t)2 * c.d_ffn,
                                          (size_t)x.lm_chunk});
  x.partial_stride = 0;  // set per projection
  Carver cv(arena);
  x.kv = cv.take<bf16>((size_t)c.n_layers * 2 * x.pool_stride);
  x.meta.ids = cv.take<int32_t>(R); x.meta.pos = cv.take<int32_t>(R); x.meta.seq = cv.take<int32_t>(R);
  x.meta.nvis = cv.take<int32_t>(R); x.meta.loc0 = cv.take<int32_t>(R); x.meta.nloc = cv.take<int32_t>(R);
  x.meta.cache_pos = cv.take<int32_t>(R); x.meta.local_idx = cv.take<int32_t>(R);
  x.meta.skey = cv.take<uint32_t>(R);
  x.d_seq_len = cv.take<int32_t>(c.max_batch);
  x.d_blk_len = cv.take<int32_t>(c.max_batch);
  // one block, so that one copy brings the whole layout of a mixed step over (same order in h_lay)
  x.lay_ints = 3 * (size_t)(c.max_batch + 1) + 2 * (size_t)(x.R_head + c.max_batch);
  x.d_step_k = cv.take<int32_t>(x.lay_ints);
  x.d_step_off = x.d_step_k + (c.max_batch + 1); x.d_step_loc = x.d_step_off + (c.max_batch + 1);
  x.d_tile_row0 = x.d_step_loc + (c.max_batch + 1); x.d_tile_rend = x.d_tile_row0 + (x.R_head + c.max_batch);
  x.d_run_max = cv.take<float>(R); x.d_run_sum = cv.take<float>(R); x.d_tgt_logit = cv.take<float>(R); x.d_logprob = cv.take<float>(R);
  x.d_target = cv.take<int32_t>(R);
  x.d_block = cv.take<int32_t>((size_t)c.max_batch * c.k_max);
  x.d_page_table = cv.take<int32_t>((size_t)c.max_batch * x.pages_per_seq);
  x.d_step_seqs = cv.take<int32_t>(c.max_batch); x.d_forced = cv.take<int32_t>(c.max_batch);
  x.d_step_n = cv.take<int32_t>(c.max_batch); x.d_step_L = cv.take<int32_t>(c.max_batch);
  x.d_out = cv.take<int32_t>((size_t)c.max_batch * (c.k_max + 1));
  x.d_prompt = cv.take<int32_t>(c.max_seq_len);
  x.d_arg_idx = cv.take<int32_t>(R); x.d_arg_val = cv.take<float>(R);
  x.d_status = cv.take<int32_t>(64);
  x.d_tl = cv.take<unsigned long long>(2 * tidar_ctx::TL_MAX + 8);   // timeline slots, then diagnostic counters
  if (c.impl == 0) {
    x.attn_part_O = cv.take<float>((size_t)attn_tc::MAX_SPLITS * R * c.n_q_heads * c.head_dim);
    x.attn_part_ml = cv.take<float>((size_t)attn_tc::MAX_SPLITS * R * c.n_q_heads * 2);
  }
  {
    const size_t G = 4 * 256;            // (CTAs of the LM-head kernel <= SMs) x 4 lane quadrants
    x.cand_val = cv.take<float>(G * R); x.cand_idx = cv.take<int32_t>(G * R);
  }
  x.X = cv.take<float>(R * c.d_model);
  x.partials = cv.take<float>(R * widest);
  x.partials_cap = R * widest;
  x.rope_cos = cv.take<float>(R * (c.head_dim / 2)); x.rope_sin = cv.take<float>(R * (c.head_dim / 2));
  x.A = cv.take<bf16>(R * c.d_model);
  x.Q = cv.take<bf16>(R * c.n_q_heads * c.head_dim);
  x.O = cv.take<bf16>(R * c.n_q_heads * c.head_dim);
  const size_t nloc = (size_t)std::max(c.max_batch * c.k_max * c.k_max, c.k_max);
  x.Kloc = cv.take<bf16>(nloc * c.n_kv_heads * c.head_dim);
  x.Vloc = cv.take<bf16>(nloc * c.n_kv_heads * c.head_dim);
  x.H = cv.take<bf16>(R * c.d_ffn);
  x.dbg_kv = cv.take<bf16>((size_t)2 * 256 * c.n_kv_heads * c.head_dim);
  if (c.debug & 1) {
    x.dbg_hidden = cv.take<float>((size_t)(c.n_layers + 1) * R * c.d_model);
    x.dbg_logits = cv.take<float>((size_t)x.R_head * (size_t)c.vocab);
  }
  *bytes = align_up(cv.off, 256);
}

// Two ways to launch a kernel of the step.  launch_pdl: with programmatic stream serialization,
// the kernel may be scheduled while the previous kernel of the stream is still running and
// synchronises itself with pdl_wait(); only kernels that call pdl_wait() before touching
// produced data may be launched this way.  It pays for kernels with a heavy prologue (the
// projections: tensor-memory allocation, barriers, the weight ring filling; attention).
// launch_after: an ordinary dependency.  The small kernels gain nothing from starting early,
// and their CTAs waiting on the SMs only take resources from the kernel that is still
// running: a chain of small kernels in a graph costs ~1 us per kernel either way (1.5B-class
// step 2.57 -> 2.51 ms, k = 1 step 1.71 -> 1.59 ms with the small kernels launched this way).
// Their pdl_wait() / pdl_trigger() are no-ops then, apart from letting the NEXT kernel start
// early.
template <typename... KP, typename... AP>
inline void launch_with(bool programmatic, void (*kernel)(KP...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, AP &&...args) {
  cudaLaunchConfig_t cfg{};
  cfg.gridDim = grid; cfg.blockDim = block; cfg.dynamicSmemBytes = smem; cfg.stream = st;
  cudaLaunchAttribute at[1];
  at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  at[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = at; cfg.numAttrs = programmatic ? 1 : 0;
  cudaLaunchKernelEx(&cfg, kernel, KP(std::forward<AP>(args))...);
}
template <typename... KP, typename... AP>
inline void launch_pdl(void (*kernel)(KP...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, AP &&...args) {
  launch_with(true, kernel, grid, block, smem, st, std::forward<AP>(args)...);
}
template <typename... KP, typename... AP>
inline void launch_after(void (*kernel)(KP...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, AP &&...args) {
  launch_with(false, kernel, grid, block, smem, st, std::forward<AP>(args)...);
}

// ---- launch bookkeeping -----------------------------------------------------
struct Launch {
  tidar_ctx *c; int cls; cudaEvent_t a = nullptr, b = nullptr; TlSlot tl{nullptr};
  Launch(tidar_ctx *c_, int cls_) : c(c_), cls(cls_) {
    c->launches++;
    if (c->timing) { cudaEventCreate(&a); cudaEventCreate(&b); cudaEventRecord(a, c->stream); }
    if (c->timeline && c->tl_n < tidar_ctx::TL_MAX) { tl.t = c->d_tl + 2 * c->tl_n; c->tl_n++; c->tl_cls.push_back(cls); }
  }
  ~Launch() {
    if (c->timing) { cudaEventRecord(b, c->stream); c->timed.push_back({cls, a, b}); }
  }
};

void collect_timing(tidar_ctx *c) {
  for (int i = 0; i < TIDAR_TC_COUNT; ++i) c->class_ms[i] = 0.f;
  for (auto &t : c->timed) {
    float ms = 0.f; cudaEventElapsedTime(&ms, t.a, t.b);
    c->class_ms[t.cls] += ms;
    cudaEventDestroy(t.a); cudaEventDestroy(t.b);
  }
  c->timed.clear();
}

// Per class, the sum over the last step's launches of (latest CTA end - earliest CTA start);
// busy = the sum over all launches, span = first start to last end.
void collect_timeline(tidar_ctx *c) {
  std::vector<unsigned long long> h(2 * (size_t)c->tl_n);
  for (int i = 0; i < TIDAR_TC_COUNT; ++i) c->tl_class_ms[i] = 0.f;
  c->tl_span_ms = c->tl_busy_ms = 0.f;
  if (c->tl_n == 0) return;
  if (cudaMemcpy(h.data(), c->d_tl, h.size() * sizeof(unsigned long long), cudaMemcpyDeviceToHost) != cudaSuccess) { cudaGetLastError(); return; }
  unsigned long long first = ~0ull, last = 0;
  for (int i = 0; i < c->tl_n; ++i) {
    if (h[2 * i] == 0 || h[2 * i + 1] == 0) continue;          // a launch that stamped nothing
    const unsigned long long t0 = ~h[2 * i], t1 = h[2 * i + 1];
    if (t1 < t0) continue;
    const float ms = (float)((double)(t1 - t0) * 1e-6);
    c->tl_class_ms[c->tl_cls[i]] += ms; c->tl_busy_ms += ms;
    first = std::min(first, t0); last = std::max(last, t1);
  }
  if (last > first) c->tl_span_ms = (float)((double)(last - first) * 1e-6);
}

KvGeom geom(const tidar_ctx *c) {
  return KvGeom{c->cfg.n_kv_heads, c->cfg.head_dim, c->cfg.page_size, c->pages_per_seq, c->d_page_table, 0};
}

// ---- projections --------------------------------------------------------------
// Tensor map of an activation matrix [rows][cols] (bf16) with a box of `box` rows; cached.
const CUtensorMap *act_map(tidar_ctx *c, const void *p, int rows, int cols, int box) {
  for (auto &m : c->amaps) if (m.p == p && m.rows == rows && m.cols == cols && m.box == box) return &m.tm;
  tidar_ctx::AMap m{p, rows, cols, box, {}};
  if (gemm_tc::encode_2d(c->encode, &m.tm, p, (uint64_t)rows, (uint64_t)cols, (uint32_t)box) != CUDA_SUCCESS) return nullptr;
  if (c->amaps.size() > 256) c->amaps.erase(c->amaps.begin());
  c->amaps.push_back(m);
  return &c->amaps.back().tm;
}

// Tensor-core projection.  A [a_rows][K] (first R rows used), W described by tmW ([N][K]).
//   MODE_SLAB  : S split-K partial slabs of fp32 [R][N] into c->partials (S chosen here)
//   MODE_SWIGLU: bf16 c->H [R][N/2]
//   MODE_ARGMAX: candidates for argmax_merge_kernel (+ optional logits dump)
int gemm_tc_launch(tidar_ctx *c, int mode, const bf16 *A, int a_rows, const CUtensorMap &tmW, int R, int N, int K, int cls,
                   int *S_out, size_t *stride_out, float *slab_out = nullptr, int force_S = 0) {
  gemm_tc::Args a{};
  a.R = R; a.N = N; a.K = K;
  gemm_tc::plan_rows(R, a);
  a.n_tiles = (N + gemm_tc::TILE_N - 1) / gemm_tc::TILE_N;
  a.kb_total = K / gemm_tc::TILE_K;
  a.S = 1; a.fused_items = 0; a.tile_b0 = 0; a.n_tiles_b = 0;
  int rem_tiles = 0;
  if (mode == gemm_tc::MODE_SLAB) {
    a.n_tiles_b = a.n_tiles;
    a.S = force_S > 0 ? std::min(force_S, a.kb_total) : gemm_tc::plan_splits(a.n_rb * a.n_tiles, a.kb_total, c->n_sms, c->S_max, 4);
    // One row block of up to 288 rows, or two of half the rows?  Two halves fetch every weight tile
    // twice (the second time from L2: ~0.37 instead of 0.46 us per K block of an item, but twice as
    // many K blocks per item once the SMs are full), while a CTA's slab store, which its SM cannot
    // push out faster than ~42 GB/s, shrinks from 3.3 to 1.7 us and fewer slabs are left for the
    // consumer.  Halves win when an item has few K blocks (the 1.5B-class shapes: step -6.5 %), one
    // block when it has many (the 8B-class shapes: halves cost +4 %).
    if (force_S <= 0 && a.n_rb == 1 && R > gemm_tc::MAX_ROWS / 2) {
      gemm_tc::Args h = a;
      gemm_tc::plan_rows(R, h, gemm_tc::MAX_ROWS / 2);
      h.S = gemm_tc::plan_splits(h.n_rb * h.n_tiles, h.kb_total, c->n_sms, c->S_max, 4);
      auto cost = [&](const gemm_tc::Args &x, double us_per_kb, double us_store) {
        const long long items = (long long)x.n_rb * x.n_tiles * x.S;
        const long long waves = (items + c->n_sms - 1) / c->n_sms;
        return waves * ((x.kb_total + x.S - 1) / x.S * us_per_kb + 1.5) + us_store + 0.5 * x.S;
      };
      if (cost(h, 0.37, 1.7) < cost(a, 0.46, 3.3)) a = h;
    }
    a.out = slab_out ? (void *)slab_out : (void *)c->partials; a.ldo = N; a.slab_stride = (long long)R * N;
    a.slab_bf16 = (slab_out || !c->slab_bf16) ? 0 : 1;   // an explicit output buffer always gets exact fp32 slabs
  } else if (mode == gemm_tc::MODE_SWIGLU) {
    a.H = c->H; a.ldh = N / 2;
    a.fused_items = a.n_rb * a.n_tiles;
    // more tiles than SMs: whole waves of tiles finish in the fused epilogue; the tiles of the
    // last, partial wave are split along K so that they also fill the machine, and are finished
    // from fp32 slabs by swiglu_slab_kernel
    if (a.n_rb == 1 && a.n_tiles > c->n_sms && a.n_tiles % c->n_sms) {
      const int full = a.n_tiles / c->n_sms * c->n_sms;
      const int rem = a.n_tiles - full;
      const int S2 = std::min({c->n_sms / rem, a.kb_total / 4, c->S_max});
      if (S2 >= 2 && (size_t)S2 * R * rem * gemm_tc::TILE_N <= c->partials_cap) {
        rem_tiles = rem;
        a.fused_items = full; a.tile_b0 = full; a.n_tiles_b = rem; a.S = S2;
        a.out = c->partials; a.ldo = rem * gemm_tc::TILE_N; a.slab_stride = (long long)R * a.ldo; a.slab_bf16 = c->slab_bf16 ? 1 : 0;
      }
    }
  } else {
    a.fused_items = a.n_rb * a.n_tiles;
    a.cand_val = c->cand_val; a.cand_idx = c->cand_idx; a.cand_ld = c->n_sms * 4; a.dump = c->dbg_logits; a.ld_dump = c->cfg.vocab; a.col0 = 0;
    a.inv_temp = c->cfg.temperature > 0.f ? 1.0f / c->cfg.temperature : 0.f; a.skey = c->meta.skey + c->head_row0;
  }
  a.status = c->d_status;
  a.warm_epilogue = mode == gemm_tc::MODE_SWIGLU ? 1 : 0;
  const CUtensorMap *tmA = act_map(c, A, a_rows, K, a.box_rows);
  if (!tmA) return fail(c, TIDAR_ECUDA, "cuTensorMapEncodeTiled failed for an activation matrix (%d x %d, box %d)", a_rows, K, a.box_rows);
  const int items = a.total_items();
  const int grid = std::min(items, c->n_sms);
  const size_t smem = gemm_tc::smem_bytes(a);
  Launch l(c, cls);
  if (mode == gemm_tc::MODE_SLAB) launch_pdl(gemm_tc::gemm_tc_kernel<gemm_tc::MODE_SLAB>, grid, gemm_tc::THREADS, smem, c->stream, tmW, *tmA, a, l.tl);
  else if (mode == gemm_tc::MODE_SWIGLU) launch_pdl(gemm_tc::gemm_tc_kernel<gemm_tc::MODE_SWIGLU>, grid, gemm_tc::THREADS, smem, c->stream, tmW, *tmA, a, l.tl);
  else if (a.inv_temp > 0.f) launch_pdl(gemm_tc::gemm_tc_kernel<gemm_tc::MODE_SAMPLE>, grid, gemm_tc::THREADS, smem, c->stream, tmW, *tmA, a, l.tl);
  else launch_pdl(gemm_tc::gemm_tc_kernel<gemm_tc::MODE_ARGMAX>, grid, gemm_tc::THREADS, smem, c->stream, tmW, *tmA, a, l.tl);
  if (rem_tiles) {
    const int nf = (N - a.tile_b0 * gemm_tc::TILE_N) / 2;          // features of the split tiles
    const size_t n = (size_t)R * nf;
    Launch lf(c, cls);
    if (c->slab_bf16)
      launch_after(swiglu_slab_kernel<bf16>, (unsigned)((n / 2 + 255) / 256), 256, 0, c->stream, (const bf16 *)c->partials, a.S, (size_t)a.slab_stride, R, a.ldo, nf,
                                                                           a.tile_b0 * gemm_tc::TILE_N / 2, a.ldh, c->H, lf.tl);
    else
      launch_after(swiglu_slab_kernel<float>, (unsigned)((n / 2 + 255) / 256), 256, 0, c->stream, (const float *)c->partials, a.S, (size_t)a.slab_stride, R, a.ldo, nf,
                                                                           a.tile_b0 * gemm_tc::TILE_N / 2, a.ldh, c->H, lf.tl);
  }
  if (S_out) *S_out = a.S;
  if (stride_out) *stride_out = (size_t)R * N;
  return TIDAR_OK;
}

enum Proj { P_QKV, P_O, P_GU, P_DOWN };

// out = A[R][K] * W[N][K]^T as S split-K partial slabs of fp32 [R][N] (replay: S = 1).
int gemm_partials(tidar_ctx *c, const bf16 *A, int a_rows, const bf16 *W, const CUtensorMap *tmW, int R, int N, int K, float *out,
                  int *S_out, size_t *stride_out, int cls) {
  if (c->cfg.impl == 0) return gemm_tc_launch(c, gemm_tc::MODE_SLAB, A, a_rows, *tmW, R, N, K, cls, S_out, stride_out);
  Launch l(c, cls);
  dim3 grid((N + 63) / 64, (R + 63) / 64);
  gemm_replay_kernel<<<grid, 256, 0, c->stream>>>(A, K, W, K, out, N, R, N, K);
  *S_out = 1; *stride_out = (size_t)R * N;
  return TIDAR_OK;
}

// bf16 tensor maps for the attention kernel (128-byte swizzle, 64-element inner box).
bool encode_q_map(tidar_ctx *c, CUtensorMap *tm, const void *q, int rows) {
  const tidar_config &cf = c->cfg;
  const int G = cf.n_q_heads / cf.n_kv_heads, spt = 128 / G;
  cuuint64_t dims[3] = {(cuuint64_t)cf.head_dim, (cuuint64_t)cf.n_q_heads, (cuuint64_t)rows};
  cuuint64_t strides[2] = {(cuuint64_t)cf.head_dim * 2, (cuuint64_t)cf.n_q_heads * cf.head_dim * 2};
  cuuint32_t box[3] = {64, (cuuint32_t)G, (cuuint32_t)spt}, es[3] = {1, 1, 1};
  return c->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(q), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
bool encode_pages_map(tidar_ctx *c, CUtensorMap *tm, const void *pool, long long n_pages) {
  const tidar_config &cf = c->cfg;
  cuuint64_t dims[4] = {(cuuint64_t)cf.head_dim, 64, (cuuint64_t)cf.n_kv_heads, (cuuint64_t)n_pages};
  cuuint64_t strides[3] = {(cuuint64_t)cf.head_dim * 2, (cuuint64_t)64 * cf.head_dim * 2, (cuuint64_t)cf.n_kv_heads * 64 * cf.head_dim * 2};
  cuuint32_t box[4] = {64, 64, 1, 1}, es[4] = {1, 1, 1, 1};
  return c->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void *>(pool), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}
bool encode_local_map(tidar_ctx *c, CUtensorMap *tm, const void *loc, long long rows) {
  const tidar_config &cf = c->cfg;
  cuuint64_t dims[3] = {(cuuint64_t)cf.head_dim, (cuuint64_t)cf.n_kv_heads, (cuuint64_t)rows};
  cuuint64_t strides[2] = {(cuuint64_t)cf.head_dim * 2, (cuuint64_t)cf.n_kv_heads * cf.head_dim * 2};
  cuuint32_t box[3] = {64, 1, 64}, es[3] = {1, 1, 1};
  return c->encode(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void *>(loc), dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                   CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// Key-range split of the attention kernel: fill the SMs (two CTAs fit on one) without giving a
// CTA fewer than two key tiles; and once half the SMs have a CTA, not fewer than four: a CTA pays
// ~7 us of set-up, partial-result store and merge traffic whatever its key range, while a nearly
// empty machine (a one-slot step) is served best by as many CTAs as there are key tiles to hand
// out.  (8B-class heads, 1 k cached positions, 72 query-tile units: 4 splits of 4-5 tiles each
// 26.9 us per call against 29.4 with 3 splits of 6; from 4 k positions on the limit is moot.)
int attn_key_splits(const tidar_ctx *c, int units, int key_tiles_hint) {
  int splits = 2 * c->n_sms / std::max(units, 1);
  splits = std::min(splits, std::max(1, key_tiles_hint / 2));
  splits = std::max(1, std::min(splits, attn_tc::MAX_SPLITS));
  while (splits > 1 && units * splits > c->n_sms / 2 && key_tiles_hint / splits < 4) --splits;
  return splits;
}

struct AttnMaps { const CUtensorMap *q, *k, *v, *kloc, *vloc; int page_base_k, page_base_v; };

// rows_per_group: slots per sequence (k(k+1) in a step; all rows in a first-pass chunk); <= 0: the
// sequences' groups differ in size and the query tiles come from the mixed step's tile table.
// key_tiles_hint: rough number of 64-key tiles per row, to size the key split.
void launch_attention_tc(tidar_ctx *c, const AttnMaps &m, const KvGeom &g, bf16 *O, int R, int rows_per_group, int key_tiles_hint) {
  const tidar_config &cf = c->cfg;
  attn_tc::Args a{};
  a.R = R; a.rows_per_group = rows_per_group;
  a.G = cf.n_q_heads / cf.n_kv_heads; a.Hq = cf.n_q_heads; a.Hkv = cf.n_kv_heads;
  a.spt = 128 / a.G;
  if (rows_per_group > 0) {
    a.tiles_per_group = (rows_per_group + a.spt - 1) / a.spt;
    a.n_groups = (R + rows_per_group - 1) / rows_per_group;
    a.n_tiles = a.n_groups * a.tiles_per_group;
  } else {                       // groups of different sizes: the tile table of the mixed step
    a.rows_per_group = R; a.tiles_per_group = 1; a.n_groups = 1;
    a.tile_row0 = c->d_tile_row0; a.tile_rend = c->d_tile_rend; a.n_tiles = c->mixed_tiles;
  }
  const int units = a.n_tiles * a.Hkv;
  a.splits = attn_key_splits(c, units, key_tiles_hint);
  a.seq = c->meta.seq; a.nvis = c->meta.nvis; a.loc0 = c->meta.loc0; a.nloc = c->meta.nloc;
  a.page_table = g.page_table; a.pages_per_seq = g.pages_per_seq;
  a.page_base_k = m.page_base_k; a.page_base_v = m.page_base_v;
  a.scale_log2 = 1.4426950408889634f / sqrtf((float)cf.head_dim);
  a.O = O; a.part_O = c->attn_part_O; a.part_ml = c->attn_part_ml; a.status = c->d_status;
  a.tile_count = c->count_tiles ? c->d_tl + 2 * tidar_ctx::TL_MAX : nullptr;
  const int grid = units * a.splits;
  {
    Launch l(c, TIDAR_TC_ATTN);
    if (cf.head_dim == 128)
      launch_pdl(attn_tc::attn_tc_kernel<128>, grid, attn_tc::THREADS, attn_tc::Smem<128>::TOTAL, c->stream, *m.q, *m.k, *m.v, *m.kloc, *m.vloc, a, l.tl);
    else
      launch_pdl(attn_tc::attn_tc_kernel<64>, grid, attn_tc::THREADS, attn_tc::Smem<64>::TOTAL, c->stream, *m.q, *m.k, *m.v, *m.kloc, *m.vloc, a, l.tl);
  }
  if (a.splits > 1) {
    Launch l(c, TIDAR_TC_ATTN);
    const size_t threads = (size_t)R * cf.n_q_heads * (cf.head_dim / 4);
    if (cf.head_dim == 128)
      launch_after(attn_tc::attn_combine_kernel<128>, (unsigned)((threads + 255) / 256), 256, 0, c->stream, c->attn_part_O, c->attn_part_ml, a.splits, R, cf.n_q_heads, O, l.tl);
    else
      launch_after(attn_tc::attn_combine_kernel<64>, (unsigned)((threads + 255) / 256), 256, 0, c->stream, c->attn_part_O, c->attn_part_ml, a.splits, R, cf.n_q_heads, O, l.tl);
  }
}

void launch_attention(tidar_ctx *c, const bf16 *Q, const bf16 *Kp, const bf16 *Vp, const KvGeom &g, const bf16 *Kl,
                      const bf16 *Vl, bf16 *O, int R) {
  Launch l(c, TIDAR_TC_ATTN);
  const float scale = 1.0f / sqrtf((float)c->cfg.head_dim);
  dim3 grid(R, c->cfg.n_q_heads);
  if (c->cfg.head_dim == 128)
    attn_replay_kernel<128><<<grid, 32, 0, c->stream>>>(Q, Kp, Vp, g, c->meta, Kl, Vl, O, c->cfg.n_q_heads, scale);
  else
    attn_replay_kernel<64><<<grid, 32, 0, c->stream>>>(Q, Kp, Vp, g, c->meta, Kl, Vl, O, c->cfg.n_q_heads, scale);
}

// partials: split-K slabs of the previous projection, bf16 on the tensor-core path, fp32 on the replay path
void launch_norm(tidar_ctx *c, int R, const float *partials, int S, size_t stride, const bf16 *gain) {
  Launch l(c, TIDAR_TC_NORM);
  const int d = c->cfg.d_model;
  if (c->cfg.impl == 0 && c->slab_bf16)
    launch_after(rmsnorm_reduce_kernel<512, bf16>, R, 512, d * sizeof(float), c->stream, c->X, (const bf16 *)partials, S, stride, gain, c->cfg.rms_eps, d, c->A, l.tl);
  else
    launch_after(rmsnorm_reduce_kernel<512, float>, R, 512, d * sizeof(float), c->stream, c->X, partials, S, stride, gain, c->cfg.rms_eps, d, c->A, l.tl);
}

// The transformer stack over R assembled rows (metadata and X already filled).
// with_head: run final norm + LM head + per-row argmax.
// Extra LM-head input rows that mix two final-normed rows each (beta < 1; see mix_rows_kernel).
struct MixRows { int n = 0, k = 1, a0 = 0, a_seq = 0, a_j = 0, b0 = 0, b_seq = 0, b_j = 0; StepLayout lay{nullptr, nullptr, nullptr, 0}; };

// head_row0: the LM head (with_head) runs on rows [head_row0, R) only, followed by the mixed rows; the
// argmax ids and the logits dump are indexed from head_row0.
int forward_rows(tidar_ctx *c, int R, bool with_head, int rows_per_group, int key_tiles_hint, const MixRows &mix = MixRows(), int head_row0 = 0) {
  const tidar_config &cf = c->cfg;
  const int d = cf.d_model, hd = cf.head_dim, Hq = cf.n_q_heads, Hkv = cf.n_kv_heads;
  const KvGeom g = geom(c);
  {
    Launch l(c, TIDAR_TC_ROPE);
    const int n = R * (hd / 2);
    launch_after(rope_table_kernel, (n + 255) / 256, 256, 0, c->stream, c->meta.pos, R, hd / 2, (double)cf.rope_theta, c->rope_cos, c->rope_sin, l.tl);
  }
  int S = 0; size_t stride = 0;          // pending partials of the previous down projection
  const bool tc = cf.impl == 0;
  const int RA = c->R_cap;               // allocated rows of the activation buffers
  int rc;
  for (int l = 0; l < cf.n_layers; ++l) {
    bf16 *Kp = c->kv + (size_t)(2 * l) * c->pool_stride, *Vp = Kp + c->pool_stride;
    launch_norm(c, R, c->partials, S, stride, c->attn_norm[l]);
    if (c->dbg_hidden)
      CUDA_TRY(c, cudaMemcpyAsync(c->dbg_hidden + (size_t)l * c->R_cap * d, c->X, (size_t)R * d * sizeof(float),
                                  cudaMemcpyDeviceToDevice, c->stream));
    if ((rc = gemm_partials(c, c->A, RA, c->wqkv[l], tc ? &c->tm_wqkv[l] : nullptr, R, c->n_qkv, d, c->partials, &S, &stride, TIDAR_TC_GEMM))) return rc;
    {
      Launch ll(c, TIDAR_TC_ROPE);
      const int rope_chunks = ((Hq + 2 * Hkv) * (hd / 8) + 255) / 256;
      const bf16 *bias_l = c->bqkv.empty() ? nullptr : c->bqkv[l], *qn_l = c->q_norm.empty() ? nullptr : c->q_norm[l],
                 *kn_l = c->k_norm.empty() ? nullptr : c->k_norm[l];
if (tc && c->slab_bf16)
        launch_after(rope_kv_kernel<bf16>, dim3(R, rope_chunks), 256, 0, c->stream, (const bf16 *)c->partials, S, stride, Hq, Hkv, hd, c->meta, c->rope_cos,
                                                                      c->rope_sin, g, c->Q, Kp, Vp, c->Kloc, c->Vloc, bias_l, qn_l, kn_l, cf.rms_eps, ll.tl);
      else
        launch_after(rope_kv_kernel<float>, dim3(R, rope_chunks), 256, 0, c->stream, c->partials, S, stride, Hq, Hkv, hd, c->meta, c->rope_cos,
                                                                      c->rope_sin, g, c->Q, Kp, Vp, c->Kloc, c->Vloc, bias_l, qn_l, kn_l, cf.rms_eps, ll.tl);
    }
    if (tc) {
      AttnMaps am{&c->tm_q, &c->tm_kv, &c->tm_kv, &c->tm_kloc, &c->tm_vloc, (2 * l) * c->n_pages, (2 * l + 1) * c->n_pages};
      launch_attention_tc(c, am, g, c->O, R, rows_per_group, key_tiles_hint);
    } else {
      launch_attention(c, c->Q, Kp, Vp, g, c->Kloc, c->Vloc, c->O, R);
    }
    if ((rc = gemm_partials(c, c->O, RA, c->wo[l], tc ? &c->tm_wo[l] : nullptr, R, d, Hq * hd, c->partials, &S, &stride, TIDAR_TC_GEMM))) return rc;
    launch_norm(c, R, c->partials, S, stride, c->ffn_norm[l]);
    if (tc) {
      if ((rc = gemm_tc_launch(c, gemm_tc::MODE_SWIGLU, c->A, RA, c->tm_wgu[l], R, 2 * cf.d_ffn, d, TIDAR_TC_GEMM, nullptr, nullptr))) return rc;
    } else {
      if ((rc = gemm_partials(c, c->A, RA, c->wgu[l], nullptr, R, 2 * cf.d_ffn, d, c->partials, &S, &stride, TIDAR_TC_GEMM))) return rc;
      Launch ll(c, TIDAR_TC_GEMM);
      const size_t n = (size_t)R * cf.d_ffn;
      swiglu_kernel<<<(unsigned)((n + 255) / 256), 256, 0, c->stream>>>(c->partials, R, cf.d_ffn, c->H);
    }
    if ((rc = gemm_partials(c, c->H, RA, c->wdown[l], tc ? &c->tm_wdown[l] : nullptr, R, d, cf.d_ffn, c->partials, &S, &stride, TIDAR_TC_GEMM))) return rc;
  }
  launch_norm(c, R, c->partials, S, stride, c->final_norm);
  if (c->dbg_hidden)
    CUDA_TRY(c, cudaMemcpyAsync(c->dbg_hidden + (size_t)cf.n_layers * c->R_cap * d, c->X, (size_t)R * d * sizeof(float),
                                cudaMemcpyDeviceToDevice, c->stream));
  if (with_head && mix.n > 0) {            // rows R .. R + mix.n - 1 of the LM head's input
    Launch lm(c, TIDAR_TC_NORM);
    launch_after(mix_rows_kernel, mix.n, 256, 0, c->stream, c->A, d, cf.beta, mix.k, mix.a0, mix.a_seq, mix.a_j, mix.b0, mix.b_seq, mix.b_j, mix.lay, R,
                 cf.temperature > 0.f ? c->meta.skey : (uint32_t *)nullptr, lm.tl);
    R += mix.n;
  }
  const bf16 *Ah = c->A + (size_t)head_row0 * d;           // first row of the LM head's input
  c->head_row0 = head_row0;
  const float inv_temp = cf.temperature > 0.f ? 1.0f / cf.temperature : 0.f;
  const int Rh = R - head_row0;
  if (with_head && Rh > c->R_head) return fail(c, TIDAR_ECAPACITY, "%d rows for the LM head exceed the context's %d", Rh, c->R_head);
  if (with_head && tc) {
    const int G = c->n_sms * 4;          // upper bound of (CTAs of the LM-head kernel) x 4 lane quadrants
    CUDA_TRY(c, cudaMemsetAsync(c->cand_idx, 0xff, (size_t)G * Rh * sizeof(int32_t), c->stream));
    if ((rc = gemm_tc_launch(c, gemm_tc::MODE_ARGMAX, Ah, RA - head_row0, c->tm_lm, Rh, cf.vocab, d, TIDAR_TC_LMHEAD, nullptr, nullptr))) return rc;
    Launch ll(c, TIDAR_TC_LMHEAD);
    launch_after(argmax_merge_kernel, (Rh * 32 + 255) / 256, 256, 0, c->stream, c->cand_val, c->cand_idx, G, Rh, c->d_arg_val, c->d_arg_idx, ll.tl);
  } else if (with_head) {
    for (int v0 = 0; v0 < cf.vocab; v0 += c->lm_chunk) {
      const int nc = std::min(c->lm_chunk, cf.vocab - v0);
      if ((rc = gemm_partials(c, Ah, RA - head_row0, c->lm_head + (size_t)v0 * d, nullptr, Rh, nc, d, c->partials, &S, &stride, TIDAR_TC_LMHEAD))) return rc;
      Launch ll(c, TIDAR_TC_LMHEAD);
      argmax_chunk_kernel<<<Rh, 256, 0, c->stream>>>(c->partials, nc, nc, v0, v0 == 0, c->d_arg_val, c->d_arg_idx, c->dbg_logits, cf.vocab, inv_temp,
                                                     c->meta.skey + head_row0);
    }
  }
  CUDA_TRY(c, cudaGetLastError());
  return TIDAR_OK;
}

// Driver entry point for tensor-map encoding (resolved through the runtime so that the
// library has no link-time dependency on the driver), tensor maps of every weight
// matrix, kernel attributes.
int init_tensor_core_path(tidar_ctx *c) {
  const tidar_config &cf = c->cfg;
  int dev = 0;
  CUDA_TRY(c, cudaGetDevice(&dev));
  cudaDeviceProp prop;
  CUDA_TRY(c, cudaGetDeviceProperties(&prop, dev));
  if (prop.major != 10) return fail(c, TIDAR_ECUDA, "the tensor-core path needs an sm_100 device, found sm_%d%d", prop.major, prop.minor);
  c->n_sms = prop.multiProcessorCount;
  void *fn = nullptr;
  cudaDriverEntryPointQueryResult qres;
  CUDA_TRY(c, cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres));
  if (!fn || qres != cudaDriverEntryPointSuccess) return fail(c, TIDAR_ECUDA, "cuTensorMapEncodeTiled is not available in this driver");
  c->encode = (gemm_tc::EncodeTiledFn)fn;
  const int d = cf.d_model, qo = cf.n_q_heads * cf.head_dim;
  auto enc = [&](CUtensorMap *tm, const void *p, int rows, int cols) {
    return gemm_tc::encode_2d(c->encode, tm, p, (uint64_t)rows, (uint64_t)cols, gemm_tc::TILE_N) == CUDA_SUCCESS;
  };
  c->tm_wqkv.resize(cf.n_layers); c->tm_wo.resize(cf.n_layers); c->tm_wgu.resize(cf.n_layers); c->tm_wdown.resize(cf.n_layers);
  bool ok = enc(&c->tm_lm, c->lm_head, cf.vocab, d);
  c->tm_lm_chunks.resize((cf.vocab + c->lm_chunk - 1) / c->lm_chunk);
  for (size_t ci = 0; ci < c->tm_lm_chunks.size() && ok; ++ci) {
    const int v0 = (int)ci * c->lm_chunk;
    ok = enc(&c->tm_lm_chunks[ci], c->lm_head + (size_t)v0 * d, std::min(c->lm_chunk, cf.vocab - v0), d);
  }
  for (int l = 0; l < cf.n_layers && ok; ++l)
    ok = enc(&c->tm_wqkv[l], c->wqkv[l], c->n_qkv, d) && enc(&c->tm_wo[l], c->wo[l], d, qo) &&
         enc(&c->tm_wgu[l], c->wgu[l], 2 * cf.d_ffn, d) && enc(&c->tm_wdown[l], c->wdown[l], d, cf.d_ffn);
  if (!ok) return fail(c, TIDAR_ECUDA, "cuTensorMapEncodeTiled failed for a weight matrix (pointers must be 16-byte aligned)");
  {
    const size_t nloc = (size_t)std::max(cf.max_batch * cf.k_max * cf.k_max, cf.k_max);
    if (!encode_q_map(c, &c->tm_q, c->Q, c->R_cap) || !encode_pages_map(c, &c->tm_kv, c->kv, (long long)cf.n_layers * 2 * c->n_pages) ||
        !encode_local_map(c, &c->tm_kloc, c->Kloc, (long long)nloc) || !encode_local_map(c, &c->tm_vloc, c->Vloc, (long long)nloc))
      return fail(c, TIDAR_ECUDA, "cuTensorMapEncodeTiled failed for an attention operand");
    // The PV product multiplies masked keys' V rows by an exact zero, so whatever the
    // kernel may load (unwritten cache slots of a page, unwritten local rows) must be finite.
    CUDA_TRY(c, cudaMemsetAsync(c->kv, 0, (size_t)cf.n_layers * 2 * c->pool_stride * sizeof(bf16), c->stream));
    CUDA_TRY(c, cudaMemsetAsync(c->Kloc, 0, nloc * cf.n_kv_heads * cf.head_dim * sizeof(bf16), c->stream));
    CUDA_TRY(c, cudaMemsetAsync(c->Vloc, 0, nloc * cf.n_kv_heads * cf.head_dim * sizeof(bf16), c->stream));
    CUDA_TRY(c, cudaFuncSetAttribute(attn_tc::attn_tc_kernel<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_tc::Smem<128>::TOTAL));
    CUDA_TRY(c, cudaFuncSetAttribute(attn_tc::attn_tc_kernel<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, attn_tc::Smem<64>::TOTAL));
  }
  const int max_smem = gemm_tc::SMEM_BUDGET + 1024;
  CUDA_TRY(c, cudaFuncSetAttribute(gemm_tc::gemm_tc_kernel<gemm_tc::MODE_SLAB>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem));
  CUDA_TRY(c, cudaFuncSetAttribute(gemm_tc::gemm_tc_kernel<gemm_tc::MODE_SWIGLU>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem));
  CUDA_TRY(c, cudaFuncSetAttribute(gemm_tc::gemm_tc_kernel<gemm_tc::MODE_ARGMAX>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem));
  CUDA_TRY(c, cudaFuncSetAttribute(gemm_tc::gemm_tc_kernel<gemm_tc::MODE_SAMPLE>, cudaFuncAttributeMaxDynamicSharedMemorySize, max_smem));
  return TIDAR_OK;
}

// Reads the device status word (already copied to pinned memory by the caller's
// synchronised copy) and turns a device-side timeout into an error code.
int check_device_status(tidar_ctx *c) {
  if (c->cfg.impl != 0) return TIDAR_OK;
  int st = 0;
  CUDA_TRY(c, cudaMemcpyAsync(&st, c->d_status, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  if (st) {
    cudaMemsetAsync(c->d_status, 0, sizeof(int), c->stream);
    return fail(c, TIDAR_EDEVICE_TIMEOUT, "a bounded device-side wait gave up (status %d); results of this call are invalid", st);
  }
  return TIDAR_OK;
}

// Returns a sequence slot's pages to the pool and marks it as not prefilled.
void release_sequence(tidar_ctx *c, int seq) {
  SeqState &s = c->seqs[seq];
  for (int p : s.pages) c->free_pages.push_back(p);
  s.pages.clear(); s.active = false; s.n = 0;
}

int ensure_pages(tidar_ctx *c, int seq, int upto_positions) {
  SeqState &s = c->seqs[seq];
  const int need = (upto_positions + c->cfg.page_size - 1) / c->cfg.page_size;
  if (need > c->pages_per_seq) return fail(c, TIDAR_ECAPACITY, "sequence %d needs %d pages, limit %d", seq, need, c->pages_per_seq);
  if ((int)s.pages.size() >= need) return TIDAR_OK;
  // The copy reads a pinned mirror that nothing else writes at these entries until the sequence is
  // released and prefilled again (which only happens with no step in flight), so it needs no wait.
  int32_t *row = c->h_page_table + (size_t)seq * c->pages_per_seq;
  const int have = (int)s.pages.size();
  while ((int)s.pages.size() < need) {
    if (c->free_pages.empty()) return fail(c, TIDAR_ECAPACITY, "KV page pool exhausted");
    row[s.pages.size()] = c->free_pages.back();
    s.pages.push_back(c->free_pages.back());
    c->free_pages.pop_back();
  }
  CUDA_TRY(c, cudaMemcpyAsync(c->d_page_table + (size_t)seq * c->pages_per_seq + have, row + have, (size_t)(need - have) * sizeof(int),
                              cudaMemcpyHostToDevice, c->stream));
  return TIDAR_OK;
}

// Enqueues the kernels of one decode step (its inputs are already in d_step_seqs / d_forced).
// k: block length of this step; ar: plain autoregressive step (the causal section alone).
// mixed_R > 0: the listed sequences use different block lengths (layout staged in h_lay, mixed_R rows in all).
// mixed_K: the sum of those block lengths (= verified positions, one mixed row each when beta < 1).
int record_step(tidar_ctx *c, int n_seqs, int k, int key_tiles_hint, bool ar, int mixed_R = 0, int mixed_K = 0) {
  const tidar_config &cf = c->cfg;
  const int n_blocks = ar ? 0 : k;
  const int T = k * (n_blocks + 1), R = mixed_R > 0 ? mixed_R : n_seqs * T;
  StepLayout lay{nullptr, nullptr, nullptr, n_seqs};
  if (mixed_R > 0) {
    CUDA_TRY(c, cudaMemcpyAsync(c->d_step_k, c->h_lay, c->lay_ints * sizeof(int), cudaMemcpyHostToDevice, c->stream));
    lay.k = c->d_step_k; lay.off = c->d_step_off; lay.loc = c->d_step_loc;
  }
  if (c->timeline) {
    c->tl_n = 0; c->tl_cls.clear();
    CUDA_TRY(c, cudaMemsetAsync(c->d_tl, 0, 2 * tidar_ctx::TL_MAX * sizeof(unsigned long long), c->stream));
  }
  {
    Launch l(c, TIDAR_TC_EMBED);
    launch_after(assemble_step_kernel, R, 256, 0, c->stream, c->meta, c->d_step_seqs, c->d_seq_len, c->d_block, c->d_blk_len, k, n_blocks, lay, cf.k_max,
               cf.mask_token_id, c->d_step_n, c->embed, cf.d_model, c->X, cf.temperature > 0.f ? 1 : 0, (unsigned long long)cf.sample_seed, l.tl);
  }
  // beta < 1: the verified prediction of causal slot j mixes its row with the first slot of block j
  MixRows mix;
  if (cf.beta < 1.0f && !ar) {
    if (mixed_R > 0) { mix.n = mixed_K; mix.lay = lay; }
    else { mix.n = n_seqs * k; mix.k = k; mix.a0 = 0; mix.a_seq = T; mix.a_j = 1; mix.b0 = k; mix.b_seq = T; mix.b_j = k; }
  }
  if (int rc = forward_rows(c, R, true, mixed_R > 0 ? 0 : T, key_tiles_hint, mix)) return rc;
  {
    Launch l(c, TIDAR_TC_VERIFY);
    launch_after(verify_select_kernel, n_seqs, 32, 0, c->stream, c->d_arg_idx, mix.n ? c->d_arg_idx + R : (const int32_t *)nullptr, c->d_step_seqs,
               c->d_forced, k, n_blocks, lay, cf.k_max, c->d_block, c->d_blk_len, c->d_step_L, c->d_out, l.tl);
  }
  {
    Launch l(c, TIDAR_TC_VERIFY);
    launch_after(kv_commit_kernel, dim3(n_seqs, cf.n_layers), 128, 0, c->stream, c->d_step_seqs, c->d_step_n, c->d_step_L, c->d_seq_len, k, lay.k,
               (cf.debug >> 1) & 1, geom(c), c->kv, c->pool_stride, l.tl);
  }
  CUDA_TRY(c, cudaGetLastError());
  return TIDAR_OK;
}

// Every launch of a step has the same arguments from step to step (lengths, page tables, token
// blocks and, for a step of mixed block lengths, the row layout live in device memory), except
// for the grid sizes and the attention key split, so the step is captured once per (k, n_seqs,
// rows, query tiles, split) and replayed.  Per-launch timing and the debug read-backs use plain
// launches.  tiles: query tiles of the attention kernel per KV head.
int replay_or_record_step(tidar_ctx *c, int n_seqs, int k, int hint, bool ar, int mixed_R, int tiles, int mixed_K = 0) {
  const tidar_config &cf = c->cfg;
  if (cf.impl == 0 && c->graphs_ok && !c->timing && !(cf.debug & (1 | 8))) {
    const int splits = attn_key_splits(c, tiles * cf.n_kv_heads, hint);
    tidar_ctx::StepGraph &sg = c->sg;
    if (!sg.exec || sg.k != k || sg.ar != ar || sg.n_seqs != n_seqs || sg.splits != splits || sg.timeline != c->timeline ||
        sg.mixed_R != mixed_R || sg.tiles != tiles || sg.mixed_K != mixed_K) {
      if (sg.exec) {
        if (!c->inflight.empty()) CUDA_TRY(c, cudaStreamSynchronize(c->stream));    // the old graph may still be running
        cudaGraphExecDestroy(sg.exec); sg.exec = nullptr;
      }
      const int64_t l0 = c->launches;
      cudaGraph_t graph = nullptr;
      int rc = TIDAR_OK;
      cudaError_t e = cudaStreamBeginCapture(c->stream, cudaStreamCaptureModeThreadLocal);
      if (e == cudaSuccess) {
        rc = record_step(c, n_seqs, k, hint, ar, mixed_R, mixed_K);
        e = cudaStreamEndCapture(c->stream, &graph);
      }
      if (e == cudaSuccess && rc == TIDAR_OK && graph) e = cudaGraphInstantiate(&sg.exec, graph, 0);
      if (graph) cudaGraphDestroy(graph);
      if (e != cudaSuccess || rc != TIDAR_OK || !sg.exec) {
        cudaGetLastError();                         // capture is not available here: plain launches from now on
        sg.exec = nullptr; c->graphs_ok = false;
      } else {
        sg.k = k; sg.ar = ar; sg.n_seqs = n_seqs; sg.splits = splits; sg.timeline = c->timeline; sg.mixed_R = mixed_R; sg.tiles = tiles; sg.mixed_K = mixed_K;
        sg.launches = c->launches - l0;
      }
      c->launches = l0;
    }
    if (sg.exec) {
      CUDA_TRY(c, cudaGraphLaunch(sg.exec, c->stream));
      c->launches += sg.launches;
      return TIDAR_OK;
    }
  }
  return record_step(c, n_seqs, k, hint, ar, mixed_R, mixed_K);
}

// Whether one more step may be enqueued: always when none is in flight; behind a step in flight only when
// every acceptance length of both is forced (the host then knows the lengths without reading the device),
// both use one block length for all their sequences and nothing reads per-step diagnostics.
bool may_enqueue(tidar_ctx *c, bool all_forced, bool mixed) {
  if (c->inflight.empty()) return true;
  if (c->inflight.size() >= 2 || !all_forced || mixed || c->timing || c->timeline || (c->cfg.debug & (1 | 8))) return false;
  return c->inflight.front().counted && c->inflight.front().ks.empty();
}

// The step proper: its inputs from the slot's pinned staging, the kernels (replayed graph or plain
// launches), its results into the slot's pinned buffers, and the event its waiter blocks on.
int launch_step(tidar_ctx *c, int n_seqs, int k, int hint, bool ar, int mixed_R, int tiles, int slot, int mixed_K = 0) {
  const tidar_config &cf = c->cfg;
  CUDA_TRY(c, cudaMemcpyAsync(c->d_step_seqs, c->h_stage2[slot], n_seqs * sizeof(int), cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(c, cudaMemcpyAsync(c->d_forced, c->h_stage2[slot] + cf.max_batch, n_seqs * sizeof(int), cudaMemcpyHostToDevice, c->stream));
  if (int rc = replay_or_record_step(c, n_seqs, k, hint, ar, mixed_R, tiles, mixed_K)) return rc;
  CUDA_TRY(c, cudaMemcpyAsync(c->h_out2[slot], c->d_out, (size_t)n_seqs * (cf.k_max + 1) * sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaMemcpyAsync(c->h_status2[slot], c->d_status, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaEventRecord(c->flight_done[slot], c->stream));
  return TIDAR_OK;
}

// Book-keeping of an enqueued step.  With every length forced the host advances the sequences now.
void push_flight(tidar_ctx *c, const int32_t *seqs, int n_seqs, const int32_t *forced, int k, const int32_t *ks, int slot) {
  tidar_ctx::Flight f;
  f.seqs.assign(seqs, seqs + n_seqs);
  if (ks) f.ks.assign(ks, ks + n_seqs);
  f.k = k; f.slot = slot;
  f.counted = forced != nullptr;
  for (int i = 0; i < n_seqs && f.counted; ++i) f.counted = forced[i] > 0;
  if (f.counted)
    for (int i = 0; i < n_seqs; ++i) { c->seqs[seqs[i]].n += forced[i]; c->seqs[seqs[i]].k = ks ? ks[i] : k; }
  c->inflight.push_back(std::move(f));
  c->next_slot ^= 1;
}

// k_step: block length of this step (0 = the one the sequences' last pass left, which must then be
// the same for all of them); ar: plain autoregressive step (k_step is 1).
int enqueue_step(tidar_ctx *c, const int32_t *seqs, int n_seqs, const int32_t *forced, bool need_forced, int k_step = 0, bool ar = false) {
  const tidar_config &cf = c->cfg;
  if (!seqs || n_seqs < 1 || n_seqs > cf.max_batch) return fail(c, TIDAR_EINVAL, "n_seqs must be in [1, max_batch]");
  {
    bool all_forced = forced != nullptr;
    for (int i = 0; i < n_seqs && all_forced; ++i) all_forced = forced[i] > 0;
    if (!may_enqueue(c, all_forced && need_forced, false))
      return fail(c, TIDAR_EINVAL, c->inflight.size() >= 2 ? "two steps are already in flight; call tidar_step_wait first"
                                                            : "a step is in flight; call tidar_step_wait first (a second step can only follow with forced lengths, "
                                                              "one block length per step and no per-step diagnostics)");
  }
  if (k_step < 0 || k_step > cf.k_max) return fail(c, TIDAR_EINVAL, "block length %d outside [1, k_max = %d]", k_step, cf.k_max);
  int k = ar ? 1 : k_step;
  for (int i = 0; i < n_seqs; ++i) {
    const int q = seqs[i];
    if (q < 0 || q >= cf.max_batch || !c->seqs[q].active) return fail(c, TIDAR_EINVAL, "sequence %d is not prefilled", q);
    for (int j = 0; j < i; ++j) if (seqs[j] == q) return fail(c, TIDAR_EINVAL, "sequence %d listed twice", q);
    if (k == 0) k = c->seqs[q].k;
    else if (k_step == 0 && !ar && c->seqs[q].k != k)
      return fail(c, TIDAR_EINVAL, "the listed sequences hold blocks of different lengths; name the step's block length (tidar_step_k)");
    const int f = forced ? forced[i] : 0;
    if (f < 0 || f > k) return fail(c, TIDAR_EINVAL, "forced acceptance %d outside [0, %d]", f, k);
    if (need_forced && f == 0) return fail(c, TIDAR_EINVAL, "tidar_step_async needs a forced acceptance length per sequence");
    if (c->seqs[q].n + (ar ? 1 : 2 * k) > cf.max_seq_len)
      return fail(c, TIDAR_ECAPACITY, "sequence %d: n + %s = %d exceeds max_seq_len %d", q, ar ? "1" : "2k", c->seqs[q].n + (ar ? 1 : 2 * k), cf.max_seq_len);
  }
  for (int i = 0; i < n_seqs; ++i) {
    int rc = ensure_pages(c, seqs[i], c->seqs[seqs[i]].n + k);
    if (rc) return rc;
  }
  const int T = ar ? 1 : k * (k + 1), R = n_seqs * T;
  const int slot = c->next_slot;
  for (int i = 0; i < n_seqs; ++i) { c->h_stage2[slot][i] = seqs[i]; c->h_stage2[slot][cf.max_batch + i] = forced ? forced[i] : 0; }
  int min_n = 1 << 30;
  for (int i = 0; i < n_seqs; ++i) min_n = std::min(min_n, c->seqs[seqs[i]].n);
  const int hint = (min_n + k + 63) / 64;
  const int spt = 128 / (cf.n_q_heads / cf.n_kv_heads);          // slots per attention query tile
  if (int rc = launch_step(c, n_seqs, k, hint, ar, 0, n_seqs * ((T + spt - 1) / spt), slot)) return rc;
  push_flight(c, seqs, n_seqs, forced, k, nullptr, slot);
  c->last_hidden_off = 0;
  c->last_rows = R + ((cf.beta < 1.0f && !ar) ? n_seqs * k : 0); c->last_first_pos = -1;      // the mixed rows follow the slots
  // the host tracks lengths without reading the device when L is forced
  return TIDAR_OK;
}

// A step in which listed sequence i uses block length ks[i] (Section 5: the block length follows the
// compute profile; nothing in the method ties the sequences of a batch to one length).  Equal lengths
// take the ordinary path; different lengths run over R = sum k_i (k_i + 1) rows with a per-sequence
// row layout and an attention tile table (one captured graph serves every step with the same
// number of sequences, rows and query tiles).
int enqueue_step_mixed(tidar_ctx *c, const int32_t *seqs, int n_seqs, const int32_t *ks, const int32_t *forced) {
  const tidar_config &cf = c->cfg;
  if (!seqs || !ks || n_seqs < 1 || n_seqs > cf.max_batch) return fail(c, TIDAR_EINVAL, "n_seqs must be in [1, max_batch]");
  bool same = true;
  for (int i = 0; i < n_seqs; ++i) {
    if (ks[i] < 1 || ks[i] > cf.k_max) return fail(c, TIDAR_EINVAL, "block length %d of entry %d outside [1, k_max = %d]", ks[i], i, cf.k_max);
    same = same && ks[i] == ks[0];
  }
  if (same) return enqueue_step(c, seqs, n_seqs, forced, false, ks[0], false);
  if (!c->inflight.empty()) return fail(c, TIDAR_EINVAL, "a step is in flight; call tidar_step_wait first");
  for (int i = 0; i < n_seqs; ++i) {
    const int q = seqs[i], k = ks[i];
    if (q < 0 || q >= cf.max_batch || !c->seqs[q].active) return fail(c, TIDAR_EINVAL, "sequence %d is not prefilled", q);
    for (int j = 0; j < i; ++j) if (seqs[j] == q) return fail(c, TIDAR_EINVAL, "sequence %d listed twice", q);
    const int f = forced ? forced[i] : 0;
    if (f < 0 || f > k) return fail(c, TIDAR_EINVAL, "forced acceptance %d outside [0, %d]", f, k);
    if (c->seqs[q].n + 2 * k > cf.max_seq_len)
      return fail(c, TIDAR_ECAPACITY, "sequence %d: n + 2k = %d exceeds max_seq_len %d", q, c->seqs[q].n + 2 * k, cf.max_seq_len);
  }
  for (int i = 0; i < n_seqs; ++i)
    if (int rc = ensure_pages(c, seqs[i], c->seqs[seqs[i]].n + ks[i])) return rc;
  const int mb = cf.max_batch, spt = 128 / (cf.n_q_heads / cf.n_kv_heads);
  int32_t *hk = c->h_lay, *hoff = hk + (mb + 1), *hloc = hoff + (mb + 1), *ht0 = hloc + (mb + 1), *hte = ht0 + (c->R_head + mb);
  const int slot = c->next_slot;
  int R = 0, loc = 0, tiles = 0, min_nk = 1 << 30, sum_k = 0;
  for (int i = 0; i < n_seqs; ++i) {
    const int k = ks[i], T = k * (k + 1);
    hk[i] = k; hoff[i] = R; hloc[i] = loc; sum_k += k;
    for (int r0 = R; r0 < R + T; r0 += spt) { ht0[tiles] = r0; hte[tiles] = R + T; ++tiles; }
    R += T; loc += k * k;
    min_nk = std::min(min_nk, c->seqs[seqs[i]].n + k);
    c->h_stage2[slot][i] = seqs[i]; c->h_stage2[slot][mb + i] = forced ? forced[i] : 0;
  }
  hk[n_seqs] = 0; hoff[n_seqs] = R; hloc[n_seqs] = loc;
  c->mixed_tiles = tiles;
  // a mixed step's kernels take every per-sequence length from the staged layout: the nominal k is unused
  const int mixed_rows = cf.beta < 1.0f ? sum_k : 0;         // one mixed LM-head input row per verified position
  if (int rc = launch_step(c, n_seqs, 0, (min_nk + 63) / 64, false, R, tiles, slot, mixed_rows)) return rc;
  push_flight(c, seqs, n_seqs, forced, 0, ks, slot);
  c->last_hidden_off = 0;
  c->last_rows = R + mixed_rows; c->last_first_pos = -1;
  return TIDAR_OK;
}

// Waits for the oldest step in flight and hands out its results.
int finish_step(tidar_ctx *c, int32_t *out_tokens, int32_t *out_n) {
  if (c->inflight.empty()) return fail(c, TIDAR_EINVAL, "no step in flight");
  tidar_ctx::Flight f = std::move(c->inflight.front());
  c->inflight.pop_front();
  CUDA_TRY(c, cudaEventSynchronize(c->flight_done[f.slot]));
  if (c->timing) collect_timing(c);
  if (c->timeline) collect_timeline(c);
  if (c->h_status2[f.slot][0]) {
    // The step's kernels have already rewritten the device-side lengths and blocks of the listed
    // sequences from invalid results: their state is lost, and so is that of a step enqueued behind
    // it.  Release them all; a new first pass is needed.
    const int st = c->h_status2[f.slot][0];
    cudaStreamSynchronize(c->stream);
    c->h_status2[0][0] = 0; c->h_status2[1][0] = 0; cudaMemsetAsync(c->d_status, 0, sizeof(int), c->stream);
    for (int q : f.seqs) release_sequence(c, q);
    for (auto &g : c->inflight) for (int q : g.seqs) release_sequence(c, q);
    c->inflight.clear();
    return fail(c, TIDAR_EDEVICE_TIMEOUT, "a bounded device-side wait gave up during the step (status %d); its results are invalid and the "
                                          "listed sequences were released (prefill them again)", st);
  }
  const int km = c->cfg.k_max;
  const int32_t *res = c->h_out2[f.slot];
  for (size_t i = 0; i < f.seqs.size(); ++i) {
    const int L = res[i * (km + 1)];
    if (!f.counted) {
      c->seqs[f.seqs[i]].n += L;
      c->seqs[f.seqs[i]].k = f.ks.empty() ? f.k : f.ks[i];        // entries of the block the step left
    }
    if (out_n) out_n[i] = L;
    if (out_tokens) for (int j = 0; j < km; ++j) out_tokens[i * km + j] = j < L ? res[i * (km + 1) + 1 + j] : -1;
  }
  return TIDAR_OK;
}

}  // namespace

// =============================================================================
extern "C" {

int tidar_arena_bytes(const tidar_config *cfg, size_t *out_bytes) {
  if (!cfg || !out_bytes) return fail(nullptr, TIDAR_EINVAL, "null argument");
  std::string why;
  if (int rc = validate(*cfg, why)) return fail(nullptr, rc, "%s", why.c_str());
  tidar_ctx tmp; tmp.cfg = *cfg;
  layout(tmp, nullptr, out_bytes);
  return TIDAR_OK;
}

int tidar_init(const tidar_config *cfg, const tidar_weights *w, void *arena, size_t arena_bytes, void *cuda_stream,
               tidar_ctx **out) {
  if (!cfg || !w || !arena || !out) return fail(nullptr, TIDAR_EINVAL, "null argument");
  std::string why;
  if (int rc = validate(*cfg, why)) return fail(nullptr, rc, "%s", why.c_str());
  int ndev = 0;
  if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) return fail(nullptr, TIDAR_ECUDA, "no CUDA device: this library has no CPU path");
  if (!w->embed || !w->lm_head || !w->final_norm || !w->attn_norm || !w->wqkv || !w->wo || !w->ffn_norm || !w->w_gate_up || !w->w_down)
    return fail(nullptr, TIDAR_EINVAL, "null weight pointer");
  if ((uintptr_t)arena % 256) return fail(nullptr, TIDAR_EINVAL, "arena must be 256-byte aligned");
  tidar_ctx *c = new tidar_ctx;
  c->cfg = *cfg;
  c->slab_bf16 = (cfg->debug & 4) != 0;
  c->stream = (cudaStream_t)cuda_stream;
  size_t need = 0;
  layout(*c, arena, &need);
  if (need > arena_bytes) { delete c; return fail(nullptr, TIDAR_ENOMEM, "arena has %zu bytes, %zu needed", arena_bytes, need); }
  c->embed = (const bf16 *)w->embed; c->lm_head = (const bf16 *)w->lm_head; c->final_norm = (const bf16 *)w->final_norm;
  for (int l = 0; l < cfg->n_layers; ++l) {
    if (!w->attn_norm[l] || !w->wqkv[l] || !w->wo[l] || !w->ffn_norm[l] || !w->w_gate_up[l] || !w->w_down[l]) {
      delete c; return fail(nullptr, TIDAR_EINVAL, "null weight pointer in layer %d", l);
    }
    c->attn_norm.push_back((const bf16 *)w->attn_norm[l]); c->wqkv.push_back((const bf16 *)w->wqkv[l]);
    c->wo.push_back((const bf16 *)w->wo[l]); c->ffn_norm.push_back((const bf16 *)w->ffn_norm[l]);
    c->wgu.push_back((const bf16 *)w->w_gate_up[l]); c->wdown.push_back((const bf16 *)w->w_down[l]);
  }
  if ((w->q_norm != nullptr) != (w->k_norm != nullptr)) { delete c; return fail(nullptr, TIDAR_EINVAL, "q_norm and k_norm come together or not at all"); }
  for (int l = 0; l < cfg->n_layers; ++l) {
    if (w->bqkv) { if (!w->bqkv[l]) { delete c; return fail(nullptr, TIDAR_EINVAL, "null bqkv pointer in layer %d", l); } c->bqkv.push_back((const bf16 *)w->bqkv[l]); }
    if (w->q_norm) {
      if (!w->q_norm[l] || !w->k_norm[l]) { delete c; return fail(nullptr, TIDAR_EINVAL, "null q_norm / k_norm pointer in layer %d", l); }
      c->q_norm.push_back((const bf16 *)w->q_norm[l]); c->k_norm.push_back((const bf16 *)w->k_norm[l]);
    }
  }
  if (cfg->impl == 0) {
    if (int rc = init_tensor_core_path(c)) { std::string m = c->err; delete c; return fail(nullptr, rc, "%s", m.c_str()); }
  }
  c->seqs.resize(cfg->max_batch);
  // free list in a scrambled order so that page tables are never contiguous
  c->free_pages.resize(c->n_pages);
  for (int i = 0; i < c->n_pages; ++i) c->free_pages[i] = i;
  uint32_t st = 0x9e3779b9u;
  for (int i = c->n_pages - 1; i > 0; --i) { st = st * 1664525u + 1013904223u; std::swap(c->free_pages[i], c->free_pages[(st >> 8) % (i + 1)]); }
  // one pinned block: first-pass result | per slot: step results, staged inputs, status | mixed-step layout | page-table mirror
  const size_t n_out = (size_t)cfg->max_batch * (cfg->k_max + 1), n_stage = 2 * (size_t)cfg->max_batch, n_pt = (size_t)cfg->max_batch * c->pages_per_seq;
  cudaError_t e = cudaHostAlloc((void **)&c->h_pinned, (n_out + 2 * (n_out + n_stage + 16) + c->lay_ints + n_pt) * sizeof(int), cudaHostAllocDefault);
  if (e != cudaSuccess) { delete c; return fail(nullptr, TIDAR_ECUDA, "cudaHostAlloc: %s", cudaGetErrorString(e)); }
  {
    int32_t *p = c->h_pinned + n_out;
    for (int sl = 0; sl < 2; ++sl) {
      c->h_out2[sl] = p; p += n_out;
      c->h_stage2[sl] = p; p += n_stage;
      c->h_status2[sl] = p; p += 16;
      c->h_status2[sl][0] = 0;
    }
    c->h_lay = p; p += c->lay_ints;
    c->h_page_table = p;
    std::memset(c->h_page_table, 0, n_pt * sizeof(int));
  }
  for (int sl = 0; sl < 2; ++sl)
    if (cudaEventCreateWithFlags(&c->flight_done[sl], cudaEventDisableTiming) != cudaSuccess) {
      cudaFreeHost(c->h_pinned); delete c; return fail(nullptr, TIDAR_ECUDA, "cudaEventCreate failed");
    }
  e = cudaMemsetAsync(c->d_seq_len, 0, cfg->max_batch * sizeof(int), c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->d_status, 0, 64 * sizeof(int), c->stream);
  if (e == cudaSuccess) e = cudaMemsetAsync(c->d_page_table, 0, (size_t)cfg->max_batch * c->pages_per_seq * sizeof(int), c->stream);
  if (e == cudaSuccess) e = cudaStreamSynchronize(c->stream);
  if (e != cudaSuccess) { cudaFreeHost(c->h_pinned); delete c; return fail(nullptr, TIDAR_ECUDA, "arena set-up: %s", cudaGetErrorString(e)); }
  *out = c;
  return TIDAR_OK;
}

int tidar_prefill(tidar_ctx *c, int32_t seq, const int32_t *prompt, int32_t n_prompt, int32_t k, int32_t *out_first) {
  if (!c) return TIDAR_EINVAL;
  const tidar_config &cf = c->cfg;
  if (!c->inflight.empty()) return fail(c, TIDAR_EINVAL, "a step is in flight");
  if (seq < 0 || seq >= cf.max_batch) return fail(c, TIDAR_EINVAL, "seq %d out of range", seq);
  if (!prompt || n_prompt < 1) return fail(c, TIDAR_EINVAL, "empty prompt");
  if (k < 1 || k > cf.k_max) return fail(c, TIDAR_EINVAL, "k must be in [1, k_max]");
  if (n_prompt + 2 * k > cf.max_seq_len) return fail(c, TIDAR_ECAPACITY, "n_prompt + 2k = %d exceeds max_seq_len %d", n_prompt + 2 * k, cf.max_seq_len);
  for (int i = 0; i < n_prompt; ++i)
    if (prompt[i] < 0 || prompt[i] >= cf.vocab) return fail(c, TIDAR_EINVAL, "prompt id %d at %d out of range", prompt[i], i);
  SeqState &s = c->seqs[seq];
  release_sequence(c, seq);
  s.k = k;
  if (int rc = ensure_pages(c, seq, n_prompt + k)) return rc;
  CUDA_TRY(c, cudaMemcpyAsync(c->d_prompt, prompt, (size_t)n_prompt * sizeof(int), cudaMemcpyHostToDevice, c->stream));
  const int total = n_prompt + k;
  const int last_rows = std::min(total, c->R_cap - (cf.beta < 1.0f ? 1 : 0));     // the last chunk may carry one mixed row
  int row0 = 0;
  while (row0 < total) {
    const bool last = row0 >= total - last_rows;
    const int rows = last ? total - row0 : std::min(c->R_cap, total - last_rows - row0);
    {
      Launch l(c, TIDAR_TC_EMBED);
      assemble_prefill_kernel<<<rows, 256, 0, c->stream>>>(c->meta, seq, row0, n_prompt, k, cf.mask_token_id, c->d_prompt, c->embed,
                                                           cf.d_model, c->X, cf.temperature > 0.f ? 1 : 0, (unsigned long long)cf.sample_seed);
    }
    // beta < 1: the settled first token mixes the last prompt row with the first mask row
    MixRows mix;
    const int rlp = n_prompt - 1 - row0;               // the last prompt row inside this chunk
    if (last && cf.beta < 1.0f) { mix.n = 1; mix.k = 1; mix.a0 = rlp; mix.b0 = rlp + 1; }
    // logits are needed for the last prompt row and the k mask rows only; the LM head runs on the
    // trailing rows of the last chunk, as many as a decode step has (all of them for a short prompt)
    const int head_row0 = last ? std::max(0, rows + mix.n - c->R_head) : 0;
    if (int rc = forward_rows(c, rows, last, rows, (row0 + rows / 2 + 63) / 64, mix, head_row0)) return rc;
    if (last) {
      Launch l(c, TIDAR_TC_VERIFY);
      prefill_finish_kernel<<<1, 32, 0, c->stream>>>(c->d_arg_idx, rlp - head_row0, (mix.n ? rows : rlp) - head_row0, k, cf.k_max, seq, n_prompt,
                                                     c->d_block, c->d_blk_len, c->d_seq_len, c->d_out);
      c->last_rows = rows - head_row0; c->last_first_pos = row0 + head_row0; c->last_hidden_off = head_row0;
    }
    row0 += rows;
  }
  CUDA_TRY(c, cudaMemcpyAsync(c->h_pinned, c->d_out, sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  CUDA_TRY(c, cudaGetLastError());
  if (c->timing) collect_timing(c);
  if (int rc = check_device_status(c)) { release_sequence(c, seq); return rc; }
  s.n = n_prompt; s.active = true;
  if (out_first) *out_first = c->h_pinned[0];
  return TIDAR_OK;
}

int tidar_step(tidar_ctx *c, const int32_t *seqs, int32_t n_seqs, const int32_t *forced, int32_t *out_tokens, int32_t *out_n) {
  if (!c) return TIDAR_EINVAL;
  if (int rc = enqueue_step(c, seqs, n_seqs, forced, false)) return rc;
  return finish_step(c, out_tokens, out_n);
}

int tidar_step_async(tidar_ctx *c, const int32_t *seqs, int32_t n_seqs, const int32_t *forced) {
  if (!c) return TIDAR_EINVAL;
  if (!forced) return fail(c, TIDAR_EINVAL, "tidar_step_async needs forced acceptance lengths");
  return enqueue_step(c, seqs, n_seqs, forced, true);
}

int tidar_step_wait(tidar_ctx *c, int32_t *out_tokens, int32_t *out_n) {
  if (!c) return TIDAR_EINVAL;
  return finish_step(c, out_tokens, out_n);
}

int tidar_step_k(tidar_ctx *c, const int32_t *seqs, int32_t n_seqs, int32_t k, const int32_t *forced, int32_t *out_tokens, int32_t *out_n) {
  if (!c) return TIDAR_EINVAL;
  if (k < 1) return fail(c, TIDAR_EINVAL, "block length must be at least 1");
  if (int rc = enqueue_step(c, seqs, n_seqs, forced, false, k, false)) return rc;
  return finish_step(c, out_tokens, out_n);
}

int tidar_step_ks(tidar_ctx *c, const int32_t *seqs, int32_t n_seqs, const int32_t *ks, const int32_t *forced, int32_t *out_tokens, int32_t *out_n) {
  if (!c) return TIDAR_EINVAL;
  if (int rc = enqueue_step_mixed(c, seqs, n_seqs, ks, forced)) return rc;
  return finish_step(c, out_tokens, out_n);
}

int tidar_ar_step(tidar_ctx *c, const int32_t *seqs, int32_t n_seqs, int32_t *out_tokens) {
  if (!c) return TIDAR_EINVAL;
  if (int rc = enqueue_step(c, seqs, n_seqs, nullptr, false, 1, true)) return rc;
  std::vector<int32_t> toks((size_t)std::max(n_seqs, 1) * c->cfg.k_max), ls(std::max(n_seqs, 1));
  if (int rc = finish_step(c, toks.data(), ls.data())) return rc;
  if (out_tokens) for (int i = 0; i < n_seqs; ++i) out_tokens[i] = toks[(size_t)i * c->cfg.k_max];
  return TIDAR_OK;
}

int tidar_ridge_k(const tidar_ctx *c, int32_t n_seqs, int32_t row_budget) {
  if (!c || n_seqs < 1) return TIDAR_EINVAL;
  if (row_budget <= 0) row_budget = 288;       // one row block of the projections: where the 8B-class step turns tensor-bound
  int k = 1;
  while (k < c->cfg.k_max && (long long)n_seqs * (k + 1) * (k + 2) <= row_budget) ++k;
  return k;
}

int tidar_plan_ks(int32_t n_seqs, int32_t k_max, int32_t row_budget, const int32_t *want, int32_t *out_ks) {
  if (n_seqs < 1 || k_max < 1 || !out_ks) return fail(nullptr, TIDAR_EINVAL, "tidar_plan_ks: n_seqs and k_max must be positive, out_ks non-null");
  if (row_budget <= 0) row_budget = 288;
  long long rows = 0;
  for (int i = 0; i < n_seqs; ++i) {
    if (want && want[i] < 1) return fail(nullptr, TIDAR_EINVAL, "tidar_plan_ks: want[%d] = %d, must be at least 1", i, want[i]);
    out_ks[i] = 1; rows += 2;
  }
  // One more draft for a sequence at length k costs 2(k + 1) rows and can yield one more token: the cost
  // grows with k, so the shortest block that may still grow is always the best place for the next rows.
  for (;;) {
    int best = -1;
    for (int i = 0; i < n_seqs; ++i) {
      const int cap = want ? std::min(k_max, want[i]) : k_max;
      if (out_ks[i] < cap && (best < 0 || out_ks[i] < out_ks[best])) best = i;
    }
    if (best < 0 || rows + 2 * (out_ks[best] + 1) > row_budget) break;
    rows += 2 * (out_ks[best] + 1);
    out_ks[best]++;
  }
  return TIDAR_OK;
}

int tidar_release(tidar_ctx *c, int32_t seq) {
  if (!c) return TIDAR_EINVAL;
  if (!c->inflight.empty()) return fail(c, TIDAR_EINVAL, "a step is in flight");
  if (seq < 0 || seq >= c->cfg.max_batch) return fail(c, TIDAR_EINVAL, "seq %d out of range", seq);
  if (c->seqs[seq].active) release_sequence(c, seq);
  return TIDAR_OK;
}

int tidar_score(tidar_ctx *c, int32_t seq, const int32_t *ids, int32_t n, float *logprobs) {
  if (!c) return TIDAR_EINVAL;
  const tidar_config &cf = c->cfg;
  if (!c->inflight.empty()) return fail(c, TIDAR_EINVAL, "a step is in flight");
  if (seq < 0 || seq >= cf.max_batch) return fail(c, TIDAR_EINVAL, "seq %d out of range", seq);
  if (!ids || !logprobs || n < 2) return fail(c, TIDAR_EINVAL, "tidar_score needs at least two token ids");
  if (n > cf.max_seq_len) return fail(c, TIDAR_ECAPACITY, "%d tokens exceed max_seq_len %d", n, cf.max_seq_len);
  for (int i = 0; i < n; ++i)
    if (ids[i] < 0 || ids[i] >= cf.vocab) return fail(c, TIDAR_EINVAL, "token id %d at %d out of range", ids[i], i);
  release_sequence(c, seq);
  c->seqs[seq].k = 1;
  if (int rc = ensure_pages(c, seq, n)) return rc;
  CUDA_TRY(c, cudaMemcpyAsync(c->d_prompt, ids, (size_t)n * sizeof(int), cudaMemcpyHostToDevice, c->stream));
  const int d = cf.d_model;
  for (int row0 = 0; row0 < n - 1; row0 += c->R_cap) {
    const int rows = std::min(c->R_cap, n - 1 - row0);          // the last token predicts nothing that is scored
    {
      Launch l(c, TIDAR_TC_EMBED);
      assemble_prefill_kernel<<<rows, 256, 0, c->stream>>>(c->meta, seq, row0, n, 0, cf.mask_token_id, c->d_prompt, c->embed, d, c->X, 0, 0ull);
    }
    if (int rc = forward_rows(c, rows, false, rows, (row0 + rows / 2 + 63) / 64)) return rc;      // ends with the final norm in c->A
    for (int v0 = 0, ci = 0; v0 < cf.vocab; v0 += c->lm_chunk, ++ci) {
      const int nc = std::min(c->lm_chunk, cf.vocab - v0);
      int S = 1; size_t stride = 0;
      if (cf.impl == 0) {
        if (int rc = gemm_tc_launch(c, gemm_tc::MODE_SLAB, c->A, c->R_cap, c->tm_lm_chunks[ci], rows, nc, d, TIDAR_TC_LMHEAD, &S, &stride, c->partials, 1)) return rc;
      } else {
        if (int rc = gemm_partials(c, c->A, c->R_cap, c->lm_head + (size_t)v0 * d, nullptr, rows, nc, d, c->partials, &S, &stride, TIDAR_TC_LMHEAD)) return rc;
      }
      Launch ll(c, TIDAR_TC_LMHEAD);
      score_chunk_kernel<<<rows, 256, 0, c->stream>>>(c->partials, nc, nc, v0, v0 == 0, c->d_prompt + row0 + 1, c->d_run_max, c->d_run_sum, c->d_tgt_logit);
    }
    {
      Launch ll(c, TIDAR_TC_LMHEAD);
      score_finish_kernel<<<(rows + 127) / 128, 128, 0, c->stream>>>(c->d_run_max, c->d_run_sum, c->d_tgt_logit, rows, c->d_logprob);
    }
    CUDA_TRY(c, cudaMemcpyAsync(logprobs + row0, c->d_logprob, (size_t)rows * sizeof(float), cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  }
  CUDA_TRY(c, cudaGetLastError());
  if (c->timing) collect_timing(c);
  release_sequence(c, seq);                         // the slot was scratch for this call
  return check_device_status(c);
}

int tidar_free(tidar_ctx *c) {
  if (!c) return TIDAR_EINVAL;
  cudaStreamSynchronize(c->stream);
  for (auto &t : c->timed) { cudaEventDestroy(t.a); cudaEventDestroy(t.b); }
  if (c->sg.exec) cudaGraphExecDestroy(c->sg.exec);
  for (int sl = 0; sl < 2; ++sl) if (c->flight_done[sl]) cudaEventDestroy(c->flight_done[sl]);
  if (c->h_pinned) cudaFreeHost(c->h_pinned);
  delete c;
  return TIDAR_OK;
}

const char *tidar_last_error(const tidar_ctx *c) { return c ? c->err.c_str() : g_init_error.c_str(); }

int tidar_seq_len(const tidar_ctx *c, int32_t seq) {
  if (!c || seq < 0 || seq >= c->cfg.max_batch || !c->seqs[seq].active) return TIDAR_EINVAL;
  return c->seqs[seq].n;
}

int64_t tidar_launch_count(const tidar_ctx *c) { return c ? c->launches : -1; }

int tidar_debug_set_block(tidar_ctx *c, int32_t seq, const int32_t *block) {
  if (!c || !block) return TIDAR_EINVAL;
  if (seq < 0 || seq >= c->cfg.max_batch || !c->seqs[seq].active) return fail(c, TIDAR_EINVAL, "sequence %d is not prefilled", seq);
  CUDA_TRY(c, cudaMemcpyAsync(c->d_block + (size_t)seq * c->cfg.k_max, block, c->seqs[seq].k * sizeof(int), cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(c, cudaMemcpyAsync(c->d_blk_len + seq, &c->seqs[seq].k, sizeof(int), cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  return TIDAR_OK;
}

int tidar_debug_get_block(tidar_ctx *c, int32_t seq, int32_t *block) {
  if (!c || !block) return TIDAR_EINVAL;
  if (seq < 0 || seq >= c->cfg.max_batch || !c->seqs[seq].active) return fail(c, TIDAR_EINVAL, "sequence %d is not prefilled", seq);
  CUDA_TRY(c, cudaMemcpyAsync(block, c->d_block + (size_t)seq * c->cfg.k_max, c->seqs[seq].k * sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  return TIDAR_OK;
}

int tidar_debug_last_rows(const tidar_ctx *c, int32_t *n_rows, int32_t *first_pos) {
  if (!c) return TIDAR_EINVAL;
  if (n_rows) *n_rows = c->last_rows;
  if (first_pos) *first_pos = c->last_first_pos;
  return TIDAR_OK;
}

static int check_rows(tidar_ctx *c, int row0, int n) {
  if (row0 < 0 || n < 1 || row0 + n > c->last_rows) return fail(c, TIDAR_EINVAL, "rows [%d, %d) outside the last pass (%d rows)", row0, row0 + n, c->last_rows);
  return TIDAR_OK;
}

int tidar_debug_get_logits(tidar_ctx *c, int32_t row0, int32_t n, float *out) {
  if (!c || !out) return TIDAR_EINVAL;
  if (!c->dbg_logits) return fail(c, TIDAR_EINVAL, "context was created without debug bit 0");
  if (int rc = check_rows(c, row0, n)) return rc;
  CUDA_TRY(c, cudaMemcpyAsync(out, c->dbg_logits + (size_t)row0 * c->cfg.vocab, (size_t)n * c->cfg.vocab * sizeof(float), cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  return TIDAR_OK;
}

int tidar_debug_get_hidden(tidar_ctx *c, int32_t layer, int32_t row0, int32_t n, float *out) {
  if (!c || !out) return TIDAR_EINVAL;
  if (!c->dbg_hidden) return fail(c, TIDAR_EINVAL, "context was created without debug bit 0");
  if (layer < 0 || layer > c->cfg.n_layers) return fail(c, TIDAR_EINVAL, "layer out of range");
  if (int rc = check_rows(c, row0, n)) return rc;
  const size_t d = c->cfg.d_model;
  CUDA_TRY(c, cudaMemcpyAsync(out, c->dbg_hidden + ((size_t)layer * c->R_cap + c->last_hidden_off + row0) * d, (size_t)n * d * sizeof(float),
                              cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  return TIDAR_OK;
}

int tidar_debug_get_argmax(tidar_ctx *c, int32_t row0, int32_t n, int32_t *out) {
  if (!c || !out) return TIDAR_EINVAL;
  if (int rc = check_rows(c, row0, n)) return rc;
  CUDA_TRY(c, cudaMemcpyAsync(out, c->d_arg_idx + row0, (size_t)n * sizeof(int), cudaMemcpyDeviceToHost, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  return TIDAR_OK;
}

int tidar_debug_get_kv(tidar_ctx *c, int32_t seq, int32_t layer, int32_t pos0, int32_t npos, uint16_t *k_out, uint16_t *v_out) {
  if (!c || !k_out || !v_out) return TIDAR_EINVAL;
  if (seq < 0 || seq >= c->cfg.max_batch || !c->seqs[seq].active) return fail(c, TIDAR_EINVAL, "sequence %d is not prefilled", seq);
  if (layer < 0 || layer >= c->cfg.n_layers) return fail(c, TIDAR_EINVAL, "layer out of range");
  const int backed = (int)c->seqs[seq].pages.size() * c->cfg.page_size;
  if (pos0 < 0 || npos < 1 || pos0 + npos > backed) return fail(c, TIDAR_EINVAL, "positions [%d, %d) not backed by pages (%d)", pos0, pos0 + npos, backed);
  const size_t per = (size_t)c->cfg.n_kv_heads * c->cfg.head_dim;
  const bf16 *Kp = c->kv + (size_t)(2 * layer) * c->pool_stride, *Vp = Kp + c->pool_stride;
  for (int p = 0; p < npos; p += 256) {
    const int np = std::min(256, npos - p);
    bf16 *ko = c->dbg_kv, *vo = c->dbg_kv + 256 * per;
    kv_gather_kernel<<<dim3(np, c->cfg.n_kv_heads), 64, 0, c->stream>>>(Kp, Vp, geom(c), seq, pos0 + p, ko, vo);
    CUDA_TRY(c, cudaMemcpyAsync(k_out + (size_t)p * per, ko, np * per * 2, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaMemcpyAsync(v_out + (size_t)p * per, vo, np * per * 2, cudaMemcpyDeviceToHost, c->stream));
    CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  }
  return TIDAR_OK;
}

int tidar_debug_wait_probe(tidar_ctx *c, int32_t limit_polls) {
  if (!c) return TIDAR_EINVAL;
  if (c->cfg.impl != 0) return fail(c, TIDAR_EINVAL, "the bounded waits exist in the tensor-core kernels only");
  if (limit_polls < 1 || limit_polls > (1 << 20)) return fail(c, TIDAR_EINVAL, "limit_polls must be in [1, 2^20]");
  wait_probe_kernel<<<1, 32, 0, c->stream>>>((uint32_t)limit_polls, c->d_status, c->d_status + 8);
  CUDA_TRY(c, cudaGetLastError());
  return TIDAR_OK;
}

int tidar_debug_force_status(tidar_ctx *c, int32_t value) {
  if (!c) return TIDAR_EINVAL;
  CUDA_TRY(c, cudaMemcpyAsync(c->d_status, &value, sizeof(int), cudaMemcpyHostToDevice, c->stream));
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  return TIDAR_OK;
}

int tidar_debug_count_attention_tiles(tidar_ctx *c, int32_t on, uint64_t *visited) {
  if (!c) return TIDAR_EINVAL;
  if (c->cfg.impl != 0) return fail(c, TIDAR_EINVAL, "the tile counter exists for the tensor-core attention kernel only");
  unsigned long long *ctr = c->d_tl + 2 * tidar_ctx::TL_MAX;
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  if (visited) {
    unsigned long long v = 0;
    CUDA_TRY(c, cudaMemcpy(&v, ctr, sizeof v, cudaMemcpyDeviceToHost));
    *visited = v;
  }
  CUDA_TRY(c, cudaMemset(ctr, 0, sizeof(unsigned long long)));
  if ((on != 0) != c->count_tiles && c->sg.exec) { cudaGraphExecDestroy(c->sg.exec); c->sg.exec = nullptr; }   // the flag is baked into the graph
  c->count_tiles = on != 0;
  return TIDAR_OK;
}

int tidar_debug_set_timeline(tidar_ctx *c, int32_t on) {
  if (!c) return TIDAR_EINVAL;
  if (c->cfg.impl != 0) return fail(c, TIDAR_EINVAL, "the in-kernel timeline exists for the tensor-core kernels only");
  c->timeline = on != 0;
  return TIDAR_OK;
}

int tidar_debug_get_timeline(tidar_ctx *c, float *class_ms, float *busy_ms, float *span_ms) {
  if (!c || !class_ms) return TIDAR_EINVAL;
  for (int i = 0; i < TIDAR_TC_COUNT; ++i) class_ms[i] = c->tl_class_ms[i];
  if (busy_ms) *busy_ms = c->tl_busy_ms;
  if (span_ms) *span_ms = c->tl_span_ms;
  return TIDAR_OK;
}

int tidar_debug_set_timing(tidar_ctx *c, int32_t on) {
  if (!c) return TIDAR_EINVAL;
  c->timing = on != 0;
  return TIDAR_OK;
}

int tidar_debug_get_timing(tidar_ctx *c, float *ms) {
  if (!c || !ms) return TIDAR_EINVAL;
  for (int i = 0; i < TIDAR_TC_COUNT; ++i) ms[i] = c->class_ms[i];
  return TIDAR_OK;
}

int tidar_gemm(tidar_ctx *c, const void *A, const void *W, int32_t R, int32_t N, int32_t K, int32_t splits, float *out) {
  if (!c) return TIDAR_EINVAL;
  if (!A || !W || !out) return fail(c, TIDAR_EINVAL, "null argument");
  if (!c->inflight.empty()) return fail(c, TIDAR_EINVAL, "a step is in flight");
  if (R < 1 || N < 1 || K < 64 || K % 64) return fail(c, TIDAR_EINVAL, "R, N >= 1 and K a positive multiple of 64 required");
  if (((uintptr_t)A | (uintptr_t)W) % 16) return fail(c, TIDAR_EINVAL, "A and W must be 16-byte aligned");
  if (splits < 0 || splits > c->S_max) return fail(c, TIDAR_EINVAL, "splits must be in [0, %d]", c->S_max);
  const size_t need = (size_t)(splits > 0 ? splits : c->S_max) * R * N;
  if (need > c->partials_cap) return fail(c, TIDAR_ECAPACITY, "R*N*splits = %zu floats exceed the context's scratch (%zu)", need, c->partials_cap);
  int S = 1; size_t stride = 0;
  if (c->cfg.impl == 0) {
    CUtensorMap tmW;
    if (gemm_tc::encode_2d(c->encode, &tmW, W, (uint64_t)N, (uint64_t)K, gemm_tc::TILE_N) != CUDA_SUCCESS)
      return fail(c, TIDAR_ECUDA, "cuTensorMapEncodeTiled failed for W");
    if (int rc = gemm_tc_launch(c, gemm_tc::MODE_SLAB, (const bf16 *)A, R, tmW, R, N, K, TIDAR_TC_GEMM, &S, &stride, c->partials, splits)) return rc;
  } else {
    if (int rc = gemm_partials(c, (const bf16 *)A, R, (const bf16 *)W, nullptr, R, N, K, c->partials, &S, &stride, TIDAR_TC_GEMM)) return rc;
  }
  {
    Launch l(c, TIDAR_TC_GEMM);
    const size_t n = (size_t)R * N;
    slab_sum_kernel<<<(unsigned)((n + 255) / 256), 256, 0, c->stream>>>(c->partials, S, stride, n, out);
  }
  CUDA_TRY(c, cudaGetLastError());
  return TIDAR_OK;
}

int tidar_sync(tidar_ctx *c) {
  if (!c) return TIDAR_EINVAL;
  CUDA_TRY(c, cudaStreamSynchronize(c->stream));
  return check_device_status(c);
}

int tidar_attention(tidar_ctx *c, const void *q, const void *k_pages, const void *v_pages, int32_t n_pages, const int32_t *page_table,
                    int32_t pages_per_seq, const int32_t *seq_len, const void *k_local, const void *v_local, void *out,
                    int32_t n_seqs, int32_t k) {
  if (!c) return TIDAR_EINVAL;
  if (!q || !k_pages || !v_pages || !page_table || !seq_len || !k_local || !v_local || !out) return fail(c, TIDAR_EINVAL, "null argument");
  if (k < 1 || k > c->cfg.k_max || n_seqs < 1 || n_seqs * k * (k + 1) > c->R_cap) return fail(c, TIDAR_EINVAL, "n_seqs * k(k+1) exceeds the context's row capacity");
  if (n_pages < 1 || pages_per_seq < 1) return fail(c, TIDAR_EINVAL, "n_pages and pages_per_seq must be positive");
  if ((long long)pages_per_seq * c->cfg.page_size < k) return fail(c, TIDAR_EINVAL, "the page table cannot back the k causal slots");
  if (!c->inflight.empty()) return fail(c, TIDAR_EINVAL, "a step is in flight");
  if (((uintptr_t)q | (uintptr_t)k_pages | (uintptr_t)v_pages | (uintptr_t)k_local | (uintptr_t)v_local | (uintptr_t)out) % 16 ||
      ((uintptr_t)page_table | (uintptr_t)seq_len) % 4)
    return fail(c, TIDAR_EINVAL, "tensors must be 16-byte aligned (page_table and seq_len 4-byte)");
  const int R = n_seqs * k * (k + 1);
  {
    Launch l(c, TIDAR_TC_EMBED);
    attn_meta_kernel<<<(R + 127) / 128, 128, 0, c->stream>>>(c->meta, seq_len, k, R, pages_per_seq * c->cfg.page_size - k);
  }
  KvGeom g{c->cfg.n_kv_heads, c->cfg.head_dim, c->cfg.page_size, pages_per_seq, page_table, n_pages};
  if (c->cfg.impl == 0) {
    CUtensorMap tq, tk, tv, tkl, tvl;
    if (!encode_q_map(c, &tq, q, R) || !encode_pages_map(c, &tk, k_pages, n_pages) || !encode_pages_map(c, &tv, v_pages, n_pages) ||
        !encode_local_map(c, &tkl, k_local, (long long)n_seqs * k * k) || !encode_local_map(c, &tvl, v_local, (long long)n_seqs * k * k))
      return fail(c, TIDAR_ECUDA, "cuTensorMapEncodeTiled failed for an attention operand");
    AttnMaps am{&tq, &tk, &tv, &tkl, &tvl, 0, 0};
    launch_attention_tc(c, am, g, (bf16 *)out, R, k * (k + 1), pages_per_seq);
  } else {
    launch_attention(c, (const bf16 *)q, (const bf16 *)k_pages, (const bf16 *)v_pages, g, (const bf16 *)k_local, (const bf16 *)v_local,
                     (bf16 *)out, R);
  }
  CUDA_TRY(c, cudaGetLastError());
  return TIDAR_OK;
}

}  // extern "C"

// =============================================================================
// Attention without any allocation.
//
// Some hosts of this library may not allocate device memory at the moment they
// need attention: a serving process whose memory pool has been handed over
// completely to another component, a real-time loop that must not enter the
// allocator (cudaMalloc can block on every other stream of the device), or a
// plug-in that is given tensors but no allocator.  For them the per-row
// visibility table that tidar_attention keeps in the context arena lives in the
// fixed array below instead.  The array is part of the library image: every GPU
// that loads the library carries it (TIDAR_STATIC_MAX_ROWS * 5 * 4 bytes) until
// the process exits.
// =============================================================================
#define TIDAR_STATIC_MAX_ROWS 4352            /* 16 sequences of 16*17 slots */
#define TIDAR_STATIC_MAX_DEVICES 64

static __device__ __align__(256) int32_t g_static_rowmeta[5 * TIDAR_STATIC_MAX_ROWS];

namespace {
// Device address of g_static_rowmeta per device ordinal.  In host code the symbol's
// name is only a handle; the address a kernel can use comes from cudaGetSymbolAddress
// with that device current.
int32_t *g_static_ptr[TIDAR_STATIC_MAX_DEVICES] = {};
}  // namespace

extern "C" int tidar_attention_static(const void *q, const void *k_pages, const void *v_pages, int32_t n_pages, const int32_t *page_table,
                                      int32_t pages_per_seq, const int32_t *seq_len, const void *k_local, const void *v_local,
                                      void *out, int32_t n_seqs, int32_t k, int32_t n_q_heads, int32_t n_kv_heads,
                                      int32_t head_dim, void *cuda_stream) {
  if (!q || !k_pages || !v_pages || !page_table || !seq_len || !k_local || !v_local || !out)
    return fail(nullptr, TIDAR_EINVAL, "tidar_attention_static: null argument");
  if (head_dim != 64 && head_dim != 128) return fail(nullptr, TIDAR_EINVAL, "tidar_attention_static: head_dim must be 64 or 128");
  if (n_kv_heads < 1 || n_q_heads < 1 || n_q_heads % n_kv_heads)
    return fail(nullptr, TIDAR_EINVAL, "tidar_attention_static: n_q_heads must be a positive multiple of n_kv_heads");
  if (k < 1 || k > 32 || n_seqs < 1 || pages_per_seq < 1 || n_pages < 1)
    return fail(nullptr, TIDAR_EINVAL, "tidar_attention_static: bad k, n_seqs, n_pages or pages_per_seq");
  if ((long long)pages_per_seq * 64 < k) return fail(nullptr, TIDAR_EINVAL, "tidar_attention_static: the page table cannot back the k causal slots");
  // the kernel reads K/V rows with 16-byte loads
  if (((uintptr_t)q | (uintptr_t)k_pages | (uintptr_t)v_pages | (uintptr_t)k_local | (uintptr_t)v_local | (uintptr_t)out) % 16 ||
      ((uintptr_t)page_table | (uintptr_t)seq_len) % 4)
    return fail(nullptr, TIDAR_EINVAL, "tidar_attention_static: tensors must be 16-byte aligned (page_table and seq_len 4-byte)");
  const long long rows = (long long)n_seqs * k * (k + 1);
  if (rows > TIDAR_STATIC_MAX_ROWS)
    return fail(nullptr, TIDAR_ECAPACITY, "tidar_attention_static: %lld rows exceed the built-in table of %d rows; use tidar_attention",
                rows, TIDAR_STATIC_MAX_ROWS);
  int dev = -1;
  CUDA_TRY(nullptr, cudaGetDevice(&dev));
  if (dev < 0 || dev >= TIDAR_STATIC_MAX_DEVICES) return fail(nullptr, TIDAR_EINVAL, "tidar_attention_static: device ordinal %d not supported", dev);
  // First call on this device: resolve the table's device address.  Not synchronised between
  // host threads: two first calls at once both look the address up and store the same value.
  if (!g_static_ptr[dev]) {
    int32_t *p = nullptr;
    CUDA_TRY(nullptr, cudaGetSymbolAddress((void **)&p, g_static_rowmeta));
    if (!p) return fail(nullptr, TIDAR_ECUDA, "tidar_attention_static: no device address for the built-in table");
    g_static_ptr[dev] = p;
  }
  int32_t *base = g_static_ptr[dev];
  const int R = (int)rows;
  RowMeta m{};
  m.seq = base; m.pos = base + TIDAR_STATIC_MAX_ROWS; m.nvis = base + 2 * TIDAR_STATIC_MAX_ROWS;
  m.loc0 = base + 3 * TIDAR_STATIC_MAX_ROWS; m.nloc = base + 4 * TIDAR_STATIC_MAX_ROWS;
  cudaStream_t st = (cudaStream_t)cuda_stream;
  // every entry a row reads is rewritten here for rows [0, R): nothing has to start at zero
  attn_meta_kernel<<<(R + 127) / 128, 128, 0, st>>>(m, seq_len, k, R, pages_per_seq * 64 - k);
  KvGeom g{n_kv_heads, head_dim, 64, pages_per_seq, page_table, n_pages};
  const float scale = 1.0f / sqrtf((float)head_dim);
  dim3 grid(R, n_q_heads);
  if (head_dim == 128)
    attn_replay_kernel<128><<<grid, 32, 0, st>>>((const bf16 *)q, (const bf16 *)k_pages, (const bf16 *)v_pages, g, m, (const bf16 *)k_local,
                                                 (const bf16 *)v_local, (bf16 *)out, n_q_heads, scale);
  else
    attn_replay_kernel<64><<<grid, 32, 0, st>>>((const bf16 *)q, (const bf16 *)k_pages, (const bf16 *)v_pages, g, m, (const bf16 *)k_local,
                                                (const bf16 *)v_local, (bf16 *)out, n_q_heads, scale);
  CUDA_TRY(nullptr, cudaGetLastError());
  return TIDAR_OK;
}
