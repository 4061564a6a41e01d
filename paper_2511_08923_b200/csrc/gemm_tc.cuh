// Small-M weight-streaming GEMM on tcgen05 tensor cores.
//
//   out[r][n] = sum_k A[r][k] * W[n][k]      A [R][K] bf16 (activations, few rows),
//                                            W [N][K] bf16 (weights, streamed once)
//
// A decode step has only k*(k+1) token slots per sequence (paper Section 3.3 footnote),
// so every projection is a GEMM with a small row count and a weight matrix that is read
// exactly once: the regime in which, by the paper's argument, extra token slots are nearly free
// (Section 1; figure "Latency Scaling").  The kernel therefore puts the WEIGHT rows on the 128 TMEM lanes (the MMA M
// dimension) and the activation rows on the MMA N dimension (up to 288 = two instructions
// of up to 144 columns), so no tensor-core work is wasted on padding rows.
//
// Work item = (row block, 128-row weight tile, K split).  Persistent CTAs, one per SM, loop
// over items.  Warp roles:
//   warp 0      streams the weight tiles by TMA into a deep ring of shared-memory stages (a
//               tile comes from HBM and takes > 1 us to arrive);
//   warp 3      streams the wide activation tiles (from L2) into a ring of three stages;
//   warp 1      issues the MMAs into one fp32 accumulator in TMEM;
//   warp 2      watches the stages' mbarriers on behalf of warp 1, which must not touch the
//               memory pipeline between its MMAs, and releases it through hardware barriers;
//   warps 4-11  drain the accumulator into registers (which frees it for the next item at
//               once) and run the epilogue from registers while the next item's MMAs proceed.
#pragma once
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace gemm_tc {

constexpr int TILE_N = 128;         // weight rows per tile (TMEM lanes)
constexpr int TILE_K = 64;          // bf16 elements per 128-byte swizzled row
constexpr int MAX_ROWS = 288;       // activation rows per row block (2 x 144 TMEM columns)
constexpr int EPI_WARPS = 8;
constexpr int ROLE_WARPS = 4;      // warpgroup 0: weight producer, MMA issuer, stage watcher, activation producer
constexpr int THREADS = 32 * (ROLE_WARPS + EPI_WARPS);
constexpr int ROLE_REGS = 56, EPI_REGS = 224;   // registers per thread after the split: 128 * 56 + 256 * 224 <= 64 K
constexpr int W_STAGE_BYTES = TILE_N * TILE_K * 2;
constexpr int SMEM_BUDGET = 216 * 1024;   // dynamic shared memory for the rings; up to 9 KB of static shared memory come on top
constexpr int TMEM_COLS = 512;

// MODE_SAMPLE is MODE_ARGMAX with Gumbel noise added to the tempered logits (a draw per row instead of
// the argmax); it is a mode of its own so that the greedy LM head carries none of its registers.
enum Mode { MODE_SLAB = 0, MODE_SWIGLU = 1, MODE_ARGMAX = 2, MODE_SAMPLE = 3 };

struct Args {
  int R, N, K;              // activation rows in use, output features, input features
  int rb_rows;              // rows per row block: multiple of 16, 16..288
  int n_rb;                 // row blocks
  int n_tiles;              // ceil(N / 128)
  int S;                    // K splits of the split region
  int fused_items;          // items [0, fused_items) are whole tiles 0.. (no K split) finished by the mode's own epilogue;
                            // the rest are tiles tile_b0.. split S ways along K, written as fp32 slabs
  int tile_b0, n_tiles_b;   // first tile and tile count of the split region
  int kb_total;             // K / 64
  int w_stages, a_stages;   // depths of the weight ring (<= 8) and of the activation ring (<= w_stages)
  int box_rows, n_box;      // activation rows per TMA box, boxes per stage
  int n1, n2;               // MMA N of the two instructions (n2 may be 0)
  // MODE_SLAB: out[split][r][n], fp32 or (slab_bf16) bf16; strides in elements
  void *out; long long slab_stride; int ldo; int slab_bf16;
  // MODE_SWIGLU: weight rows interleave (gate f, up f); H[r][f] = silu(gate) * up, bf16
  bf16 *H; int ldh;
  // MODE_ARGMAX: per (CTA, lane quadrant) candidates, [R][cand_ld >= gridDim*4] (index -1 = none; the
  // caller pre-fills the index table with -1); optional fp32 dump [R][ld_dump]
  float *cand_val; int32_t *cand_idx; int cand_ld; float *dump; int ld_dump; int col0;
  // MODE_SAMPLE: the compared value is logit * inv_temp + Gumbel noise of (skey[row], id),
  // i.e. a draw from softmax(logits / temperature) per row (see gumbel_noise); the dump keeps the raw logits
  float inv_temp; const uint32_t *skey;
  int warm_epilogue;        // MODE_SWIGLU: walk through the epilogue once before the first accumulator is ready (see the kernel)
  int *status;              // device word set to 1 when a bounded wait gave up
  __host__ __device__ int tile_b0_or_all() const { return n_tiles_b ? tile_b0 : n_tiles; }   // tiles per row block in the fused region
  __host__ __device__ int total_items() const { return fused_items + n_rb * n_tiles_b * S; }
};

struct Item { int rb, tile, split, kb0, kb1; bool fused; };
// Item order.  With several row blocks (a long first pass) the row block varies fastest: the CTAs
// that run side by side then work on the SAME weight tile for different rows, so the tile comes
// from HBM once and from L2 for the others, and the pass is bound by the tensor cores instead of
// streaming every weight matrix once per row block.  The LM-head mode keeps a row block's tiles
// together instead (tile fastest): its epilogue carries a running argmax per row block.
template <int MODE>
__device__ __forceinline__ Item decode_item(const Args &g, int item) {
  Item w;
  if (item < g.fused_items) {
    w.fused = true; w.split = 0;
    if (MODE == MODE_ARGMAX || MODE == MODE_SAMPLE) { w.tile = item % g.tile_b0_or_all(); w.rb = item / g.tile_b0_or_all(); }
    else { w.rb = item % g.n_rb; w.tile = item / g.n_rb; }
    w.kb0 = 0; w.kb1 = g.kb_total;
  } else {
    const int j = item - g.fused_items;
    w.fused = false; w.rb = j % g.n_rb; w.split = (j / g.n_rb) % g.S; w.tile = g.tile_b0 + j / (g.n_rb * g.S);
    w.kb0 = (int)((long long)g.kb_total * w.split / g.S); w.kb1 = (int)((long long)g.kb_total * (w.split + 1) / g.S);
  }
  return w;
}

// silu(g) * u.  The fast division is exact enough for a bf16 result (2 ulp of fp32) and returns
// the right limit (-0) when exp(-g) overflows.
__device__ __forceinline__ float silu_mul(float g, float u) { return __fdividef(g, 1.f + __expf(-g)) * u; }

template <int MODE>
__global__ void __launch_bounds__(THREADS, 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmW, const __grid_constant__ CUtensorMap tmA, const Args g, const TlSlot tl) {
  extern __shared__ uint8_t smem_raw[];
  __shared__ __align__(8) uint64_t w_full[8], w_empty[8], a_full[8], a_empty[8], tmem_full_bar, tmem_empty_bar;
  __shared__ uint32_t tmem_base_slot;
  __shared__ int abort_flag;
  __shared__ __align__(16) uint16_t epi_stage[MODE == MODE_SWIGLU ? EPI_WARPS : 1][32][16];   // MODE_SWIGLU: two 16-column chunks per epilogue warp, [column][feature]

  pdl_trigger();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem0 = (sm100::smem_u32(smem_raw) + 1023u) & ~1023u;
  const int a_stage_bytes = g.rb_rows * TILE_K * 2;                 // multiple of 1024 (rb_rows % 16 == 0)
  const uint32_t smem_a0 = smem0 + (uint32_t)g.w_stages * W_STAGE_BYTES;   // activation ring behind the weight ring
  const int n_items = g.total_items();

  if (threadIdx.x == 0) {
    abort_flag = 0;
    for (int s = 0; s < 8; ++s) {
      sm100::mbar_init(sm100::smem_u32(&w_full[s]), 1); sm100::mbar_init(sm100::smem_u32(&w_empty[s]), 1);
      sm100::mbar_init(sm100::smem_u32(&a_full[s]), 1); sm100::mbar_init(sm100::smem_u32(&a_empty[s]), 1);
    }
    sm100::mbar_init(sm100::smem_u32(&tmem_full_bar), 1);
    sm100::mbar_init(sm100::smem_u32(&tmem_empty_bar), EPI_WARPS);
    sm100::fence_mbar_init();
  }
  if (warp == 1) {
    __syncwarp();
    sm100::tmem_alloc(sm100::smem_u32(&tmem_base_slot), TMEM_COLS);
    sm100::tmem_relinquish();
  }
  sm100::tc_fence_before();
  __syncthreads();
  sm100::tc_fence_after();
  const uint32_t tmem_acc = tmem_base_slot;
  volatile int *abortp = &abort_flag;

  // The epilogue warps hold the whole accumulator (144 registers per thread) next to their
  // own arithmetic; at the kernel-wide limit of 168 the compiler serialises that arithmetic to
  // save registers (SwiGLU: 1000 instead of 300 cycles per chunk) and spills in the argmax.  The
  // four role warps need few registers, so their warpgroup hands most of its share over.
  // (Each reallocation heads the code that runs under it, which is how the compiler learns
  // the register budget of that code.)

  if (warp < ROLE_WARPS) {
  sm100::setmaxnreg_dec<ROLE_REGS>();
  if (warp == 0) {
    // ===================== weight producer =====================
    if (lane == 0) {
      sm100::prefetch_tensormap(&tmW);
      const uint64_t pol_w = sm100::policy_evict_first();
      int s = 0; uint32_t ph = 0; bool ok = true;
      // Weights are never written by a kernel, so nothing here waits for the previous kernel:
      // the ring fills while that kernel is still finishing.
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
        const Item w = decode_item<MODE>(g, item);
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          if (!sm100::mbar_wait(sm100::smem_u32(&w_empty[s]), ph ^ 1u, abortp)) { ok = false; break; }
          const uint32_t fb = sm100::smem_u32(&w_full[s]);
          sm100::mbar_expect_tx(fb, (uint32_t)W_STAGE_BYTES);
          sm100::tma_load_2d(smem0 + (uint32_t)s * W_STAGE_BYTES, &tmW, fb, kb * TILE_K, w.tile * TILE_N, pol_w);
          if (++s == g.w_stages) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 3) {
    // ===================== activation producer =====================
    if (lane == 0) {
      sm100::prefetch_tensormap(&tmA);
      const uint64_t pol_a = sm100::policy_evict_last();
      int s = 0; uint32_t ph = 0; bool ok = true;
      pdl_wait();                      // the activations are the previous kernel's output
      tl_go(tl);
      for (int item = blockIdx.x; item < n_items && ok; item += gridDim.x) {
        const Item w = decode_item<MODE>(g, item);
        for (int kb = w.kb0; kb < w.kb1; ++kb) {
          if (!sm100::mbar_wait(sm100::smem_u32(&a_empty[s]), ph ^ 1u, abortp)) { ok = false; break; }
          const uint32_t fb = sm100::smem_u32(&a_full[s]);
          const uint32_t sa = smem_a0 + (uint32_t)s * a_stage_bytes;
          sm100::mbar_expect_tx(fb, (uint32_t)a_stage_bytes);
          for (int b = 0; b < g.n_box; ++b)
            sm100::tma_load_2d(sa + (uint32_t)(b * g.box_rows * TILE_K * 2), &tmA, fb, kb * TILE_K, w.rb * g.rb_rows + b * g.box_rows, pol_a);
          if (++s == g.a_stages) { s = 0; ph ^= 1u; }
        }
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    // One thread issues every MMA, and it issues them barely faster than the tensor pipe
    // retires them, so nothing else may sit in its instruction stream: a test of an mbarrier
    // (any access through the memory pipeline) completes only once the MMAs queued before it
    // have gone out, and the pipe runs dry for ~250 cycles per K block.  The watcher warp
    // therefore does the mbarrier waits and releases this warp through one hardware barrier
    // per stage.  Descriptors are built once and advanced with plain adds (the start-address
    // field counts 16-byte units and never carries out of its 14 bits inside shared memory).
    //
    // This warp and the watcher run the same (item, K block) schedule to the end whatever
    // happens elsewhere, one barrier operation each per K block, so neither can be left
    // waiting for the other; after a failed wait the MMAs read stale tiles, which is harmless,
    // and the status word reports the failure.
    const uint32_t idesc1 = sm100::make_idesc_bf16(TILE_N, g.n1), idesc2 = sm100::make_idesc_bf16(TILE_N, g.n2 ? g.n2 : 16);
    const uint64_t wdesc0 = sm100::make_desc_sw128(smem0), adesc0 = sm100::make_desc_sw128(smem_a0);   // stage 0 of each ring
    const uint64_t wstage16 = (uint64_t)(W_STAGE_BYTES >> 4), astage16 = (uint64_t)(a_stage_bytes >> 4);
    const uint64_t a2_off16 = (uint64_t)(g.n1 * 8);
    const uint32_t tmem_acc2 = tmem_acc + (uint32_t)g.n1;
    const bool two = g.n2 != 0;
    int s = 0, sa = 0;
    uint64_t wd = wdesc0, ad = adesc0;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x) {
      const Item w = decode_item<MODE>(g, item);
      const int kb0 = w.kb0, kb1 = w.kb1;
      uint32_t acc = 0u;                 // the watcher's first release of an item also says that the accumulator is free
      for (int kb = kb0; kb < kb1; ++kb) {
        sm100::named_bar_sync(1u + (uint32_t)s, 64);
        sm100::tc_fence_after();
        if (lane == 0) {
          if (two) {
            const uint64_t ad2 = ad + a2_off16;
#pragma unroll
            for (int kk = 0; kk < TILE_K / 16; ++kk) {
              sm100::mma_bf16_ss(tmem_acc, wd + 2 * kk, ad + 2 * kk, idesc1, acc);
              sm100::mma_bf16_ss(tmem_acc2, wd + 2 * kk, ad2 + 2 * kk, idesc2, acc);
              acc = 1u;
            }
          } else {
#pragma unroll
            for (int kk = 0; kk < TILE_K / 16; ++kk) {
              sm100::mma_bf16_ss(tmem_acc, wd + 2 * kk, ad + 2 * kk, idesc1, acc);
              acc = 1u;
            }
          }
          sm100::mma_commit(sm100::smem_u32(&w_empty[s]));       // both stages reusable once these MMAs have read them
          sm100::mma_commit(sm100::smem_u32(&a_empty[sa]));
        }
        __syncwarp();
        wd += wstage16; ad += astage16;
        if (++s == g.w_stages) { s = 0; wd = wdesc0; }
        if (++sa == g.a_stages) { sa = 0; ad = adesc0; }
      }
      if (lane == 0) sm100::mma_commit(sm100::smem_u32(&tmem_full_bar));
      __syncwarp();
    }
  } else if (warp == 2) {
    // ===================== stage watcher =====================
    // Waits (bounded) for the accumulator to be drained and for each stage's loads to land,
    // then arrives on the stage's hardware barrier.  A stage's barrier cannot be arrived on
    // twice before the MMA warp has passed it: the second landing needs the producer's refill,
    // which needs the MMA warp's commit for the first.  After a failed wait that argument no
    // longer holds, so from then on the watcher meets the MMA warp at every barrier instead.
    int s = 0, sa = 0; uint32_t ph = 0, pha = 0, it = 0; bool failed = false;
    for (int item = blockIdx.x; item < n_items; item += gridDim.x, ++it) {
      const Item w = decode_item<MODE>(g, item);
      if (!failed) {
        bool ok = true;
        if (lane == 0) ok = sm100::mbar_wait(sm100::smem_u32(&tmem_empty_bar), (it & 1u) ^ 1u, abortp);
        failed = !__shfl_sync(0xffffffffu, ok, 0);
      }
      for (int kb = w.kb0; kb < w.kb1; ++kb) {
        if (!failed) {
          bool ok = true;
          if (lane == 0) ok = sm100::mbar_wait(sm100::smem_u32(&w_full[s]), ph, abortp) && sm100::mbar_wait(sm100::smem_u32(&a_full[sa]), pha, abortp);
          failed = !__shfl_sync(0xffffffffu, ok, 0);
        }
        if (!failed) sm100::named_bar_arrive(1u + (uint32_t)s, 64);
        else sm100::named_bar_sync(1u + (uint32_t)s, 64);
        if (++s == g.w_stages) { s = 0; ph ^= 1u; }
        if (++sa == g.a_stages) { sa = 0; pha ^= 1u; }
      }
    }
  }
  } else {
    sm100::setmaxnreg_inc<EPI_REGS>();
    // ===================== epilogue =====================
    pdl_wait();
    const int q = warp & 3;                      // TMEM lane quadrant this warp may read
    const int half = (warp - ROLE_WARPS) >> 2;
    const int hc = ((g.rb_rows / 2 + 15) / 16) * 16;
    const int c_begin = half ? hc : 0;
    const int c_end = half ? g.rb_rows : (hc < g.rb_rows ? hc : g.rb_rows);
    const int ncols = c_end - c_begin;           // multiple of 16, <= 144
    uint32_t it = 0; bool ok = true;
    // MODE_ARGMAX: running best of column c_begin + 32*slot + lane, and the row block it belongs to
    float best_v[5]; int best_i[5]; int cur_rb = -1;
#pragma unroll
    for (int k = 0; k < 5; ++k) { best_v[k] = -INFINITY; best_i[k] = 0x7fffffff; }
    auto flush_best = [&]() {
      if (cur_rb < 0) return;
#pragma unroll
      for (int k = 0; k < 5; ++k) {
        const int cidx = k * 32 + lane;
        const int r = cur_rb * g.rb_rows + c_begin + cidx;
        if (cidx < ncols && r < g.R) {
          const long long o = (long long)r * g.cand_ld + (blockIdx.x * 4 + q);
          g.cand_val[o] = best_v[k]; g.cand_idx[o] = best_i[k] == 0x7fffffff ? -1 : best_i[k];
        }
        best_v[k] = -INFINITY; best_i[k] = 0x7fffffff;
      }
    };
    // ---- MODE_SWIGLU: two 16-column chunks of the accumulator -> bf16 rows of H ----
    // Lane pairs (2j, 2j+1) hold gate and up of feature n/2; the even lane finishes
    // column c, the odd lane column c+1, after one exchange per column pair.  The
    // results of a 16-column chunk (16 columns x 16 features per warp) are turned
    // through shared memory so that every lane stores 8 consecutive features of one
    // row with one 16-byte store: 2-byte stores from each lane took 18 us per tile.
    // All exchanges first, then sixteen independent silu chains (one chain at a time is bound by
    // instruction latency: 16 us per tile instead of 2), then the turn through shared memory.
    // c0 / c1: the two chunks (c1 only if second); row0: output row of c0's first column.
    auto swiglu_pass = [&](const uint32_t (&c0)[16], const uint32_t (&c1)[16], bool second, int row0, int R_live, int tile) {
      const bool odd = lane & 1;
      uint16_t (*stage)[16] = epi_stage[MODE == MODE_SWIGLU ? warp - ROLE_WARPS : 0];
      const int srow = lane >> 1, sf = (lane & 1) * 8;
      const int f0 = ((tile * TILE_N + q * 32) >> 1) + sf;          // first of this lane's 8 features
      const int n_feat = g.N >> 1;
      float h[2][8];
#pragma unroll
      for (int c = 0; c < 2; ++c) {
        if (c == 0 || second) {
          uint32_t recv[8];
#pragma unroll
          for (int j = 0; j < 8; ++j) recv[j] = __shfl_xor_sync(0xffffffffu, odd ? (c ? c1[2 * j] : c0[2 * j]) : (c ? c1[2 * j + 1] : c0[2 * j + 1]), 1);
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const float gate = __uint_as_float(odd ? recv[j] : (c ? c1[2 * j] : c0[2 * j]));
            const float up = __uint_as_float(odd ? (c ? c1[2 * j + 1] : c0[2 * j + 1]) : recv[j]);
            h[c][j] = silu_mul(gate, up);
          }
        }
      }
#pragma unroll
      for (int c = 0; c < 2; ++c)
        if (c == 0 || second) {
#pragma unroll
          for (int j = 0; j < 8; ++j) stage[c * 16 + 2 * j + (odd ? 1 : 0)][lane >> 1] = __bfloat16_as_ushort(__float2bfloat16(h[c][j]));
        }
      __syncwarp();
#pragma unroll
      for (int c = 0; c < 2; ++c)
        if (c == 0 || second) {
          const uint4 packed = *reinterpret_cast<const uint4 *>(&stage[c * 16 + srow][sf]);
          const int r = row0 + c * 16 + srow;
          if (r < R_live) {
            bf16 *dst = g.H + (long long)r * g.ldh + f0;
            if (f0 + 8 <= n_feat && (g.ldh & 7) == 0) {
              *reinterpret_cast<uint4 *>(dst) = packed;
            } else {
              const uint16_t *e = reinterpret_cast<const uint16_t *>(&packed);
              for (int t = 0; t < 8; ++t)
                if (f0 + t < n_feat) dst[t] = __ushort_as_bfloat16(e[t]);
            }
          }
        }
      __syncwarp();
    };
    // The epilogue below is long straight-line code that a CTA runs once or twice, and between two
    // launches of this kernel the other kernels of a layer push it out of the instruction cache: run
    // cold, next to the MMAs of the next item, one SwiGLU pass took 2 - 3.5 us instead of 0.4.  These
    // warps have nothing to do while the first item's MMAs run, so they first walk through the
    // epilogue once with every store and barrier operation switched off (dry), which
    // brings the code in; g.warm_epilogue is a run-time value so that both walks share one copy.
    // A fused item that is its CTA's last one takes a third route: nobody waits for the accumulator, so it
    // stays in tensor memory and a loop of a few hundred instructions takes 32 columns per round (the
    // 1.5B-class gate/up projection, one item per CTA, ends 4 us earlier than with the long code).
    bool dry = (MODE == MODE_SWIGLU) && g.warm_epilogue != 0 && (int)(blockIdx.x + gridDim.x) < n_items;
    for (int item = blockIdx.x; item < n_items && ok;) {
      const Item w = decode_item<MODE>(g, item);
      const int split = w.split, tile = w.tile, rb = w.rb;
      if (MODE == MODE_SWIGLU && w.fused && item + (int)gridDim.x >= n_items) {
        if (!sm100::mbar_wait(sm100::smem_u32(&tmem_full_bar), it & 1u, abortp)) { ok = false; break; }
        sm100::tc_fence_after();
        const uint32_t t0 = tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)c_begin;
        const int row_first = rb * g.rb_rows + c_begin;
#pragma unroll 1
        for (int cc = 0; cc < ncols; cc += 32) {
          uint32_t c0[16], c1[16];
          const bool second = cc + 16 < ncols;
          sm100::tmem_ld16(t0 + cc, c0);
          if (second) sm100::tmem_ld16(t0 + cc + 16, c1);
          sm100::tmem_wait_ld();
          swiglu_pass(c0, c1, second, row_first + cc, g.R, tile);
        }
        sm100::tc_fence_before();
        __syncwarp();
        if (lane == 0) sm100::mbar_arrive(sm100::smem_u32(&tmem_empty_bar));
        item += gridDim.x; ++it;
        continue;
      }
      uint32_t v[9][16];
      if (!dry) {
        if (!sm100::mbar_wait(sm100::smem_u32(&tmem_full_bar), it & 1u, abortp)) { ok = false; break; }
        sm100::tc_fence_after();
        const uint32_t t0 = tmem_acc + ((uint32_t)(q * 32) << 16) + (uint32_t)c_begin;
#pragma unroll
        for (int i = 0; i < 9; ++i)
          if (i * 16 < ncols) sm100::tmem_ld16(t0 + i * 16, v[i]);
        sm100::tmem_wait_ld();
        sm100::tc_fence_before();
        __syncwarp();
        if (lane == 0) sm100::mbar_arrive(sm100::smem_u32(&tmem_empty_bar));   // accumulator free for the next item
      }                                                  // (dry: v holds whatever the registers held; nothing of it is stored)
      const int R_live = dry ? 0 : g.R;                  // rows this walk may store

      const int n = tile * TILE_N + q * 32 + lane;       // this thread's output feature
      const int r_base = rb * g.rb_rows + c_begin;
      if (MODE == MODE_SLAB || !w.fused) {
        // split-K partial sums; columns are counted from the first tile of the split region
        const int nc = n - g.tile_b0 * TILE_N;
        const bool n_ok = n < g.N;
        if (!g.slab_bf16) {
          // One running pointer and a bound counted from this thread's first row: with the address
          // and the row test recomputed per store (r * ldo, r < R) the same 144 stores take 1.65 times
          // as long (19.5 instead of 32 bytes per cycle and SM, the rate the L2 takes stores at).
          float *p = reinterpret_cast<float *>(g.out) + (long long)split * g.slab_stride + nc + (long long)r_base * g.ldo;
          const int rows_left = n_ok ? R_live - r_base : 0;
#pragma unroll
          for (int i = 0; i < 9; ++i) {
            if (i * 16 < ncols) {
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                if (i * 16 + j < rows_left) *p = __uint_as_float(v[i][j]);
                p += g.ldo;
              }
            }
          }
        } else {
          // bf16: lane pairs (2j, 2j+1) exchange so that the even lane stores features
          // (n, n+1) of column c and the odd lane those of column c+1, 4 bytes each
          bf16 *o = reinterpret_cast<bf16 *>(g.out) + (long long)split * g.slab_stride + (nc & ~1);
          const bool odd = lane & 1;
#pragma unroll
          for (int i = 0; i < 9; ++i) {
            if (i * 16 < ncols) {
#pragma unroll
              for (int j = 0; j < 16; j += 2) {
                const uint32_t send = odd ? v[i][j] : v[i][j + 1];
                const uint32_t recv = __shfl_xor_sync(0xffffffffu, send, 1);
                const float lo = __uint_as_float(odd ? recv : v[i][j]);          // feature n & ~1
                const float hi = __uint_as_float(odd ? v[i][j + 1] : recv);      // feature n | 1
                const int r = r_base + i * 16 + j + (odd ? 1 : 0);
                if (n_ok && r < R_live) {
                  __nv_bfloat162 h2 = __floats2bfloat162_rn(lo, hi);
                  *reinterpret_cast<__nv_bfloat162 *>(o + (long long)r * g.ldo) = h2;
                }
              }
            }
          }
        }
      } else if (MODE == MODE_SWIGLU) {
        // Register-staged walk over the whole accumulator, two 16-column chunks per pass.
#pragma unroll
        for (int ip = 0; ip < 5; ++ip) {
          if (ip * 32 < ncols) {
            const bool second = (2 * ip + 1) < 9 && (2 * ip + 1) * 16 < ncols;      // warp-uniform
            swiglu_pass(v[2 * ip], v[(2 * ip + 1) < 9 ? 2 * ip + 1 : 8], second, r_base + ip * 32, R_live, tile);
          }
        }
      } else {
        // Per column: best (value, index) over the 32 features of this warp, folded into a
        // running best over all tiles this CTA processes.  The 32 lanes x 32 columns of a
        // group are reduced by recursive halving: in the step with stride h a lane keeps the
        // columns whose bit h equals its own lane bit h and hands the others to lane ^ h, so
        // after five steps lane l holds the result of column 32*g + l (31 exchanges per 32
        // columns instead of 160).  Lowest index wins ties, NaN never wins.
        if (rb != cur_rb) { flush_best(); cur_rb = rb; }
        const bool n_ok = n < g.N;
        const int my_idx = (n_ok ? g.col0 + n : 0x7fffffff);
        if (g.dump && n_ok) {
#pragma unroll
          for (int i = 0; i < 9; ++i)
            if (i * 16 < ncols) {
#pragma unroll
              for (int j = 0; j < 16; ++j) {
                const int r = r_base + i * 16 + j;
                if (r < g.R) g.dump[(long long)r * g.ld_dump + n] = __uint_as_float(v[i][j]);
              }
            }
        }
#pragma unroll
        for (int grp = 0; grp < 5; ++grp) {
          if (grp * 32 < ncols) {
            float val[32]; int idx[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) {
              const int i = grp * 2 + (j >> 4);
              float x = (i < 9 && i * 16 < ncols) ? __uint_as_float(v[i < 9 ? i : 8][j & 15]) : -INFINITY;
              if (MODE == MODE_SAMPLE) {
                const int r = r_base + grp * 32 + j;
                if (r < g.R && n_ok) x = x * g.inv_temp + gumbel_noise(g.skey[r], (uint32_t)my_idx);
              }
              const bool ok_v = n_ok && (x == x);
              val[j] = ok_v ? x : -INFINITY; idx[j] = ok_v ? my_idx : 0x7fffffff;
            }
#pragma unroll
            for (int h = 16; h >= 1; h >>= 1) {
              const bool up = lane & h;
#pragma unroll
              for (int j = 0; j < h; ++j) {
                // columns j (bit h clear) and j + h (bit h set) of the current, already folded, set
                const float sv = up ? val[j] : val[j + h];
                const int si = up ? idx[j] : idx[j + h];
                const float ov = __shfl_xor_sync(0xffffffffu, sv, h);
                const int oi = __shfl_xor_sync(0xffffffffu, si, h);
                const float mv = up ? val[j + h] : val[j];
                const int mi = up ? idx[j + h] : idx[j];
                const bool take = ov > mv || (ov == mv && oi < mi);
                val[j] = take ? ov : mv; idx[j] = take ? oi : mi;
              }
            }
            if (val[0] > best_v[grp] || (val[0] == best_v[grp] && idx[0] < best_i[grp])) { best_v[grp] = val[0]; best_i[grp] = idx[0]; }
          }
        }
      }
      if (dry) dry = false;                              // the same item again, for real
      else { item += gridDim.x; ++it; }
    }
    if (MODE == MODE_ARGMAX || MODE == MODE_SAMPLE) flush_best();
  }

  // ---- teardown ----
  sm100::tc_fence_before();
  __syncthreads();
  if (abort_flag) {
    if (threadIdx.x == 0 && g.status) atomicExch(g.status, 1);
    // give copies and MMAs that are still in flight time to land before the CTA's
    // shared and tensor memory are released
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    __syncwarp();
    sm100::tc_fence_after();
    sm100::tmem_dealloc(tmem_acc, TMEM_COLS);
  }
  if (threadIdx.x == 0) tl_end(tl);
}

// ---- host side ----------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                  const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// bf16 row-major [rows][cols] matrix, box = box_rows x 64 columns, 128-byte swizzle,
// out-of-range elements read as zero.
inline CUresult encode_2d(EncodeTiledFn fn, CUtensorMap *tm, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
  cuuint64_t dims[2] = {cols, rows};
  cuuint64_t strides[1] = {cols * 2};
  cuuint32_t box[2] = {(cuuint32_t)TILE_K, box_rows};
  cuuint32_t estr[2] = {1, 1};
  return fn(tm, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
            CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

// Row-block geometry for R activation rows.
inline void plan_rows(int R, Args &a, int max_rows = MAX_ROWS) {
  a.n_rb = (R + max_rows - 1) / max_rows;
  const int per = (R + a.n_rb - 1) / a.n_rb;
  a.rb_rows = (per + 15) / 16 * 16;
  if (a.rb_rows <= 256) { a.box_rows = a.rb_rows; a.n_box = 1; a.n1 = a.rb_rows; a.n2 = 0; }
  else { a.box_rows = a.rb_rows / 2; a.n_box = 2; a.n1 = ((a.rb_rows / 2 + 15) / 16) * 16; a.n2 = a.rb_rows - a.n1; }
  // Three activation stages keep that ring a K block ahead of the MMAs; the weight ring gets
  // the rest of the budget.  Small row blocks get equally deep rings.
  const int a_stage = a.rb_rows * TILE_K * 2;
  a.a_stages = 3;
  a.w_stages = (SMEM_BUDGET - a.a_stages * a_stage) / W_STAGE_BYTES;
  if (a.w_stages > 8) a.w_stages = 8;
  if (a.w_stages < 3) a.w_stages = 3;
  while (a.a_stages < a.w_stages && (a.a_stages + 1) * a_stage + a.w_stages * W_STAGE_BYTES <= SMEM_BUDGET) a.a_stages++;
}
inline size_t smem_bytes(const Args &a) { return (size_t)a.w_stages * W_STAGE_BYTES + (size_t)a.a_stages * (a.rb_rows * TILE_K * 2) + 1024; }

// K splits: fill the SMs with whole waves of equally sized items, keeping at least
// min_kb K blocks per item.
inline int plan_splits(int n_items_unsplit, int kb_total, int n_sms, int max_splits, int min_kb) {
  int best = 1; double best_eff = 0.0;
  for (int s = 1; s <= max_splits; ++s) {
    if (s > 1 && kb_total / s < min_kb) break;
    const long long items = (long long)n_items_unsplit * s;
    const long long waves = (items + n_sms - 1) / n_sms;
    // time ~ waves * (k blocks per item + fixed per-item cost in k-block units)
    const double per_item = (double)((kb_total + s - 1) / s) + 3.0;
    const double eff = ((double)n_items_unsplit * kb_total) / ((double)waves * n_sms * per_item);
    if (eff > best_eff + 1e-9) { best_eff = eff; best = s; }
  }
  return best;
}

}  // namespace gemm_tc
