// Structured-mask attention of one pass on tcgen05 tensor cores.
//
// A pass's rows (token slots) attend to the cached positions [0, nvis) of their sequence
// plus the nloc step-local K/V rows starting at loc0 (see RowMeta).  For a decode step this
// is the paper's decoding mask (figure "TiDAR Attention Masks"; Section 3.1): drafted
// tokens causal, every mask block bidirectional inside itself and blind to the other
// blocks.  The mask is never materialised: a query tile derives, from its rows' metadata,
// which 64-key tiles it needs (cached pages up to the largest nvis, and only the local
// rows of the blocks it contains), skips all others, and applies the per-row bound only
// on tiles that straddle it.
//
// Tiling: the G = Hq/Hkv query heads that share a KV head are packed into one 128-row
// MMA tile (floor(128/G) slots x G heads), so K/V are read once per KV head.  Per key
// tile: S = Q K^T (M 128, N 64, K hd) into TMEM (double buffered); the softmax warps read S
// (one thread per row), keep a reference max and the running sum, and write P (bf16, two keys per
// 32-bit column) back into the first half of the S buffer it came from; O += P V (M 128, N hd,
// K 64, P as the tensor-memory operand, V as the MN-major shared-memory operand) accumulates in
// TMEM over all key tiles.  P never touches shared memory: with P staged there the kernel moved
// 128 KB through shared memory per key tile (Q 32 and K 16 read by Q K^T, P 16 written and read,
// V 16, and the 32 KB the TMA writes), 1000 cycles at 128 B per cycle against 512 cycles of MMAs.
// The reference max is only raised when a tile exceeds it by more than 2^8 (P stays <= 256,
// exact enough in bf16/fp32); raising it rescales the rows of O in TMEM, which happens in the
// first tiles only.  Barriers that either side can run ahead on exist once per S buffer (a
// parity wait cannot tell two completions from none).  The CTA needs
// <= 113 KB of shared memory, 256 TMEM columns and < 170 registers per thread, so two CTAs
// share an SM and fill each other's dependency stalls.  The key range of a query tile can be
// split over several CTAs; partial (max, sum, O) results are merged by attn_combine_kernel.
#pragma once
#include "common.cuh"
#include "sm100_ptx.cuh"

namespace attn_tc {

constexpr int KT = 64;               // keys per tile (= page size)
constexpr int K_STAGES = 3, V_STAGES = 2;   // K runs a tile further ahead: Q K^T of tile i + 1 is issued before P V of tile i
constexpr int THREADS = 192;         // warp 0: TMA, warp 1: MMA, warps 2..5: softmax
constexpr int MAX_SPLITS = 8;
constexpr float RAISE_THRESHOLD = 8.f;   // log2 units

struct Args {
  int R;                    // rows (slots) of the pass
  int rows_per_group;       // slots per sequence group (k(k+1) for a step; R for a first pass)
  int tiles_per_group;      // ceil(rows_per_group / spt)
  int n_groups;
  // Groups of different sizes (a step whose sequences use different block lengths): query tile t
  // covers rows [tile_row0[t], tile_row0[t] + spt) of the group that ends at tile_rend[t]; null =
  // equal groups, derived from rows_per_group.  n_tiles = number of query tiles in either case.
  const int32_t *tile_row0, *tile_rend; int n_tiles;
  int spt;                  // slots per query tile = 128 / G
  int G, Hq, Hkv;
  int splits;
  const int32_t *seq, *nvis, *loc0, *nloc;   // per row
  const int32_t *page_table; int pages_per_seq;
  int page_base_k, page_base_v;              // offsets in the page dimension of the K / V tensor maps
  float scale_log2;                          // log2(e) / sqrt(hd)
  bf16 *O;                                   // [R][Hq*hd]
  float *part_O;                             // [splits][R][Hq][hd]  (splits > 1)
  float *part_ml;                            // [splits][R][Hq][2]
  int *status;
  unsigned long long *tile_count;            // diagnostics: += key tiles this CTA visits (null = off)
};

// Shared memory of one CTA; everything is dynamic so that the 1024-byte alignment the
// swizzled tiles need costs no padding (the kernel checks the base address).
template <int HD>
struct Smem {
  static constexpr int NH = HD / 64;                 // 64-element halves of a head
  static constexpr int Q_BYTES = 128 * HD * 2;
  static constexpr int KV_BYTES = KT * HD * 2;
  static constexpr int Q_OFF = 0;
  static constexpr int K_OFF = Q_OFF + Q_BYTES;
  static constexpr int V_OFF = K_OFF + K_STAGES * KV_BYTES;
  static constexpr int BAR_OFF = V_OFF + V_STAGES * KV_BYTES;    // mbarriers and a few words
  static constexpr int TOTAL = BAR_OFF + 256;
  static constexpr int TMEM_COLS = 256;              // 2 x 64 (S) + HD (O) <= 256
};

struct Ctl {                                         // lives at Smem::BAR_OFF
  uint64_t q_full, k_full[K_STAGES], k_empty[K_STAGES], v_full[V_STAGES], v_empty[V_STAGES], s_full[2], s_empty[2], p_full[2];
  uint32_t tmem_base;
  int abort_flag, max_nvis, loc_lo, loc_hi;
};
static_assert(sizeof(Ctl) <= 256, "control block must fit its slot");

template <int HD>
__global__ void __launch_bounds__(THREADS, 2)
attn_tc_kernel(const __grid_constant__ CUtensorMap tmQ, const __grid_constant__ CUtensorMap tmK, const __grid_constant__ CUtensorMap tmV,
               const __grid_constant__ CUtensorMap tmKloc, const __grid_constant__ CUtensorMap tmVloc, const Args a, const TlSlot tl) {
  using L = Smem<HD>;
  constexpr int NH = L::NH;
  extern __shared__ __align__(1024) uint8_t smem_raw[];
  pdl_trigger();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const uint32_t smem0 = sm100::smem_u32(smem_raw);
  if (smem0 & 1023u) {                               // cannot place swizzled tiles: report, touch nothing
    if (threadIdx.x == 0 && a.status) atomicExch(a.status, 3);
    return;
  }
  Ctl &ctl = *reinterpret_cast<Ctl *>(smem_raw + L::BAR_OFF);

  // ---- which work item ----
  int w = blockIdx.x;
  const int sp = w % a.splits; w /= a.splits;
  const int kvh = w % a.Hkv; w /= a.Hkv;
  int row0, row_end;                                                   // first slot of the tile; slots of its group end at row_end
  if (a.tile_row0) { row0 = a.tile_row0[w]; row_end = a.tile_rend[w]; }
  else {
    const int tile = w % a.tiles_per_group, grp = w / a.tiles_per_group;
    row0 = grp * a.rows_per_group + tile * a.spt;
    row_end = min((grp + 1) * a.rows_per_group, a.R);
  }
  const int rows_used = a.spt * a.G;                                   // MMA rows that carry data

  if (threadIdx.x == 0) {
    ctl.abort_flag = 0; ctl.max_nvis = 0; ctl.loc_lo = 0x7fffffff; ctl.loc_hi = 0;
    sm100::mbar_init(sm100::smem_u32(&ctl.q_full), 1);
    for (int s = 0; s < K_STAGES; ++s) { sm100::mbar_init(sm100::smem_u32(&ctl.k_full[s]), 1); sm100::mbar_init(sm100::smem_u32(&ctl.k_empty[s]), 1); }
    for (int s = 0; s < V_STAGES; ++s) { sm100::mbar_init(sm100::smem_u32(&ctl.v_full[s]), 1); sm100::mbar_init(sm100::smem_u32(&ctl.v_empty[s]), 1); }
    for (int b = 0; b < 2; ++b) { sm100::mbar_init(sm100::smem_u32(&ctl.s_full[b]), 1); sm100::mbar_init(sm100::smem_u32(&ctl.s_empty[b]), 1); }
    for (int b = 0; b < 2; ++b) sm100::mbar_init(sm100::smem_u32(&ctl.p_full[b]), 4);
    sm100::fence_mbar_init();
  }
  if (warp == 1) {
    __syncwarp();
    sm100::tmem_alloc(sm100::smem_u32(&ctl.tmem_base), L::TMEM_COLS);
    sm100::tmem_relinquish();
  }
  __syncthreads();
  pdl_wait();                 // everything below reads what earlier kernels of the pass wrote
  if (threadIdx.x == 0) tl_go(tl);

  // ---- per-row metadata (softmax threads own one MMA row each) and the tile's key range ----
  const int my_row = (warp & 3) * 32 + lane;             // MMA row = TMEM lane (softmax warps only)
  int my_slot = -1, my_nvis = 0, my_loc0 = 0, my_nloc = 0, my_head = 0;
  if (warp >= 2) {
    const int sl = my_row / a.G;
    const int pr = row0 + sl;
    if (sl < a.spt && pr < row_end) {
      my_slot = pr; my_head = kvh * a.G + my_row % a.G;
      my_nvis = a.nvis[pr]; my_nloc = a.nloc[pr]; my_loc0 = a.loc0[pr];
      atomicMax(&ctl.max_nvis, my_nvis);
      if (my_nloc > 0) { atomicMin(&ctl.loc_lo, my_loc0); atomicMax(&ctl.loc_hi, my_loc0 + my_nloc); }
    }
  }
  sm100::tc_fence_before();
  __syncthreads();
  sm100::tc_fence_after();
  const uint32_t tmem = ctl.tmem_base;
  const uint32_t tmem_S = tmem, tmem_O = tmem + 2 * KT;               // S: 2 x 64 columns, O: HD columns
  const int max_nvis = ctl.max_nvis;
  const int loc_lo = ctl.loc_lo, loc_hi = ctl.loc_hi;
  const int n_cache_tiles = (max_nvis + KT - 1) / KT;
  const int n_loc_tiles = loc_hi > loc_lo ? (loc_hi - loc_lo + KT - 1) / KT : 0;
  const int nt_all = n_cache_tiles + n_loc_tiles;
  const int t_begin = (int)((long long)nt_all * sp / a.splits), t_end = (int)((long long)nt_all * (sp + 1) / a.splits);
  const int nt = t_end - t_begin;
  const int seq = row0 < a.R ? a.seq[row0] : 0;
  volatile int *abortp = &ctl.abort_flag;
  if (threadIdx.x == 0 && a.tile_count) atomicAdd(a.tile_count, (unsigned long long)nt);

  if (warp == 0) {
    // ===================== TMA producer =====================
    if (lane == 0 && nt > 0) {
      const uint64_t pol = sm100::policy_evict_last();
      const uint32_t qb = sm100::smem_u32(&ctl.q_full);
      sm100::mbar_expect_tx(qb, (uint32_t)(NH * rows_used * 128));
      for (int h = 0; h < NH; ++h)
        sm100::tma_load_3d(smem0 + L::Q_OFF + h * (128 * 128), &tmQ, qb, h * 64, kvh * a.G, row0, pol);
      int ks = 0, vs = 0; uint32_t kph = 0, vph = 0;
      auto load_tile = [&](int t, bool is_k) -> bool {
        const bool is_cache = t < n_cache_tiles;
        const int page = is_cache ? a.page_table[(size_t)seq * a.pages_per_seq + t] : 0;
        const int lrow = loc_lo + (t - n_cache_tiles) * KT;
        const int st = is_k ? ks : vs;
        if (!sm100::mbar_wait(sm100::smem_u32(is_k ? &ctl.k_empty[st] : &ctl.v_empty[st]), (is_k ? kph : vph) ^ 1u, abortp)) return false;
        const uint32_t fb = sm100::smem_u32(is_k ? &ctl.k_full[st] : &ctl.v_full[st]);
        sm100::mbar_expect_tx(fb, (uint32_t)L::KV_BYTES);
        for (int h = 0; h < NH; ++h) {
          const uint32_t dst = smem0 + (is_k ? L::K_OFF : L::V_OFF) + st * L::KV_BYTES + h * (KT * 128);
          if (is_cache) sm100::tma_load_4d(dst, is_k ? &tmK : &tmV, fb, h * 64, 0, kvh, (is_k ? a.page_base_k : a.page_base_v) + page, pol);
          else sm100::tma_load_3d(dst, is_k ? &tmKloc : &tmVloc, fb, h * 64, kvh, lrow, pol);
        }
        if (is_k) { if (++ks == K_STAGES) { ks = 0; kph ^= 1u; } }
        else { if (++vs == V_STAGES) { vs = 0; vph ^= 1u; } }
        return true;
      };
      // K of tile t + 1 goes out before V of tile t, in the order the MMA warp consumes them
      bool ok = load_tile(t_begin, true);
      for (int t = t_begin; t < t_end && ok; ++t) {
        if (t + 1 < t_end) ok = load_tile(t + 1, true);
        if (ok) ok = load_tile(t, false);
      }
    }
  } else if (warp == 1) {
    // ===================== MMA issuer =====================
    if (lane == 0 && nt > 0) {
      const uint32_t idesc_qk = sm100::make_idesc_bf16(128, KT);
      const uint32_t idesc_pv = sm100::make_idesc_bf16(128, HD) | (1u << 16);      // B (= V) is MN-major
      bool ok = sm100::mbar_wait(sm100::smem_u32(&ctl.q_full), 0, abortp);
      sm100::tc_fence_after();
      int ks = 0; uint32_t kph = 0;          // K ring position of the next QK^T
      int vs = 0; uint32_t vph = 0;          // V ring position of the next PV
      // descriptors are built once; the issue loop only adds 16-byte-unit offsets
      const uint64_t q_desc = sm100::make_desc_sw128(smem0 + L::Q_OFF);
      const uint64_t k_desc0 = sm100::make_desc_sw128(smem0 + L::K_OFF);
      const uint64_t v_desc0 = sm100::make_desc_sw128_mn(smem0 + L::V_OFF, KT * 128);
      constexpr uint64_t KV16 = L::KV_BYTES >> 4;
      auto issue_qk = [&](int i) -> bool {   // i: tile counter of this CTA
        const int b = i & 1; const uint32_t bph = (uint32_t)(i >> 1) & 1u;
        if (!sm100::mbar_wait(sm100::smem_u32(&ctl.k_full[ks]), kph, abortp)) return false;
        if (!sm100::mbar_wait(sm100::smem_u32(&ctl.s_empty[b]), bph ^ 1u, abortp)) return false;
        sm100::tc_fence_after();
        const uint64_t kd = k_desc0 + (uint64_t)ks * KV16;
        const uint32_t d = tmem_S + b * KT;
#pragma unroll
        for (int kk = 0; kk < HD / 16; ++kk) {
          // 64-element half kk/4 of the head: Q halves are 128 rows x 128 B apart, K halves 64 rows x 128 B
          sm100::mma_bf16_ss(d, q_desc + (kk / 4) * (128 * 128 / 16) + (kk % 4) * 2, kd + (kk / 4) * (KT * 128 / 16) + (kk % 4) * 2, idesc_qk,
                             kk > 0 ? 1u : 0u);
        }
        sm100::mma_commit(sm100::smem_u32(&ctl.k_empty[ks]));
        sm100::mma_commit(sm100::smem_u32(&ctl.s_full[b]));
        if (++ks == K_STAGES) { ks = 0; kph ^= 1u; }
        return true;
      };
      if (ok) ok = issue_qk(0);
      for (int i = 0; i < nt && ok; ++i) {
        if (i + 1 < nt) { ok = issue_qk(i + 1); if (!ok) break; }
        if (!sm100::mbar_wait(sm100::smem_u32(&ctl.v_full[vs]), vph, abortp)) { ok = false; break; }
        // (one barrier per S buffer: the softmax warps may finish tile i + 1 before this thread has seen tile i,
        // and a parity wait cannot tell two completions from none)
        if (!sm100::mbar_wait(sm100::smem_u32(&ctl.p_full[i & 1]), (uint32_t)(i >> 1) & 1u, abortp)) { ok = false; break; }
        sm100::tc_fence_after();
        const uint64_t vd = v_desc0 + (uint64_t)vs * KV16;
        const uint32_t p_tmem = tmem_S + (uint32_t)((i & 1) * KT);
#pragma unroll
        for (int kk = 0; kk < KT / 16; ++kk)       // 16 keys per instruction: 8 columns of P, 16 V rows (2048 B)
          sm100::mma_bf16_ts(tmem_O, p_tmem + kk * 8, vd + kk * (16 * 128 / 16), idesc_pv, (i > 0 || kk > 0) ? 1u : 0u);
        sm100::mma_commit(sm100::smem_u32(&ctl.v_empty[vs]));
        // P consumed and O up to date through tile i: the S buffer P lived in is free for tile i + 2
        sm100::mma_commit(sm100::smem_u32(&ctl.s_empty[i & 1]));
        if (++vs == V_STAGES) { vs = 0; vph ^= 1u; }
      }
    }
  } else {
    // ===================== softmax =====================
    const uint32_t lane_addr = (uint32_t)((warp & 3) * 32) << 16;
    float m_ref = -INFINITY, l_run = 0.f;
    bool ok = true;
    for (int i = 0; i < nt && ok; ++i) {
      const int t = t_begin + i;
      const int b = i & 1; const uint32_t bph = (uint32_t)(i >> 1) & 1u;
      // a wait that gives up must take the whole warp out: the TMEM loads below are warp-collective
      if (!__all_sync(0xffffffffu, sm100::mbar_wait(sm100::smem_u32(&ctl.s_full[b]), bph, abortp))) { ok = false; break; }
      sm100::tc_fence_after();
      uint32_t sv[64];
      {
        uint32_t v0[32], v1[32];
        sm100::tmem_ld32(tmem_S + lane_addr + b * KT, v0);
        sm100::tmem_ld32(tmem_S + lane_addr + b * KT + 32, v1);
        sm100::tmem_wait_ld();
#pragma unroll
        for (int j = 0; j < 32; ++j) { sv[j] = v0[j]; sv[32 + j] = v1[j]; }
      }

      // visible keys of this tile for my row: [lo, hi) in tile-local indices
      int lo = 0, hi = 0;
      if (my_slot >= 0) {
        if (t < n_cache_tiles) { lo = 0; hi = min(KT, my_nvis - t * KT); }
        else {
          const int base = loc_lo + (t - n_cache_tiles) * KT;           // local row of key 0
          lo = max(0, my_loc0 - base); hi = my_nloc > 0 ? min(KT, my_loc0 + my_nloc - base) : 0;
        }
      }
      // Softmax of the tile in base 2.  The scores stay raw in sv: the scale is applied inside
      // one FMA per element (s * scale - m), masking is skipped for tiles that are visible in
      // full (all cached keys but the last tile of a row), and the max and the sum run as
      // four independent chains: this loop, not the MMAs, bounds the kernel.
      if (lo > 0 || hi < KT) {
#pragma unroll
        for (int j = 0; j < 64; ++j)
          if (j < lo || j >= hi) sv[j] = 0xff800000u;          // -inf
      }
      float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
      for (int j = 0; j < 64; j += 4) {
#pragma unroll
        for (int u = 0; u < 4; ++u) mx4[u] = fmaxf(mx4[u], __uint_as_float(sv[j + u]));
      }
      const float mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3])) * a.scale_log2;     // scale > 0; -inf stays -inf
      // raise the reference only when this tile exceeds it by more than the threshold
      // (-inf + threshold = -inf, so the first visible key always sets it)
      const float m_new = (mx > m_ref + RAISE_THRESHOLD) ? mx : m_ref;
      const float alpha = (m_new == m_ref) ? 1.f : exp2f(m_ref - m_new);      // m_ref = -inf gives 0
      const float neg_m = (m_new == -INFINITY) ? 0.f : -m_new;
      float sum4[4] = {0.f, 0.f, 0.f, 0.f};
      uint32_t pk[32];
#pragma unroll
      for (int j = 0; j < 64; j += 4) {
        float p[4];
#pragma unroll
        for (int u = 0; u < 4; ++u) {
          p[u] = sm100::ex2_approx(fmaf(__uint_as_float(sv[j + u]), a.scale_log2, neg_m));   // -inf -> 0
          sum4[u] += p[u];
        }
        __nv_bfloat162 h01 = __floats2bfloat162_rn(p[0], p[1]), h23 = __floats2bfloat162_rn(p[2], p[3]);
        pk[j >> 1] = *reinterpret_cast<uint32_t *>(&h01);
        pk[(j >> 1) + 1] = *reinterpret_cast<uint32_t *>(&h23);
      }
      const float sum = (sum4[0] + sum4[1]) + (sum4[2] + sum4[3]);
      l_run = l_run * alpha + sum;
      m_ref = m_new;

      if (i > 0 && __any_sync(0xffffffffu, alpha != 1.f)) {
        // O is rescaled in place, so P V of tile i - 1 must be complete: completion (i - 1) / 2 of the
        // barrier of its S buffer.  A parity wait means what it says only while the barrier is at most
        // one completion away from the one waited for, which holds although most tiles never wait
        // here: completion (i - 3) / 2 happened before the Q K^T of tile i - 1 was issued, and the
        // next one needs the P of tile i + 1.
        if (!__all_sync(0xffffffffu, sm100::mbar_wait(sm100::smem_u32(&ctl.s_empty[(i - 1) & 1]), (uint32_t)((i - 1) >> 1) & 1u, abortp))) { ok = false; break; }
        sm100::tc_fence_after();
#pragma unroll
        for (int c = 0; c < HD / 32; ++c) {
          uint32_t v[32];
          sm100::tmem_ld32(tmem_O + lane_addr + c * 32, v);
          sm100::tmem_wait_ld();
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = __float_as_uint(__uint_as_float(v[j]) * alpha);
          sm100::tmem_st32(tmem_O + lane_addr + c * 32, v);
        }
        sm100::tmem_wait_st();
        sm100::tc_fence_before();
      }
      // P -> the first 32 columns of this tile's S buffer (my row = my TMEM lane; the scores are in registers)
      sm100::tmem_st32(tmem_S + lane_addr + b * KT, pk);
      sm100::tmem_wait_st();
      sm100::tc_fence_before();
      __syncwarp();
      if (lane == 0) sm100::mbar_arrive(sm100::smem_u32(&ctl.p_full[b]));
    }
    // ---- output: O is complete once the last PV has finished ----
    // (the last two products, each on its own buffer's barrier; the bound on the distance holds as above)
    if (ok && nt > 1) ok = sm100::mbar_wait(sm100::smem_u32(&ctl.s_empty[(nt - 2) & 1]), (uint32_t)((nt - 2) >> 1) & 1u, abortp);
    if (ok && nt > 0) ok = sm100::mbar_wait(sm100::smem_u32(&ctl.s_empty[(nt - 1) & 1]), (uint32_t)((nt - 1) >> 1) & 1u, abortp);
    ok = __all_sync(0xffffffffu, ok);
    if (ok) {
      sm100::tc_fence_after();
      const float inv = (a.splits == 1) ? 1.f / l_run : 1.f;
      bf16 *o = a.O + ((size_t)max(my_slot, 0) * a.Hq + my_head) * HD;
      const size_t pidx = ((size_t)sp * a.R + max(my_slot, 0)) * a.Hq + my_head;
      float *po = a.part_O + pidx * HD;
#pragma unroll
      for (int c = 0; c < HD / 32; ++c) {
        uint32_t v[32];
        if (nt > 0) { sm100::tmem_ld32(tmem_O + lane_addr + c * 32, v); sm100::tmem_wait_ld(); }
        else {
#pragma unroll
          for (int j = 0; j < 32; ++j) v[j] = 0u;
        }
        if (my_slot >= 0) {
          if (a.splits == 1) {
#pragma unroll
            for (int j = 0; j < 32; j += 8) {
              uint4 u;
              __nv_bfloat162 h0 = __floats2bfloat162_rn(__uint_as_float(v[j]) * inv, __uint_as_float(v[j + 1]) * inv),
                             h1 = __floats2bfloat162_rn(__uint_as_float(v[j + 2]) * inv, __uint_as_float(v[j + 3]) * inv),
                             h2 = __floats2bfloat162_rn(__uint_as_float(v[j + 4]) * inv, __uint_as_float(v[j + 5]) * inv),
                             h3 = __floats2bfloat162_rn(__uint_as_float(v[j + 6]) * inv, __uint_as_float(v[j + 7]) * inv);
              u.x = *reinterpret_cast<uint32_t *>(&h0); u.y = *reinterpret_cast<uint32_t *>(&h1);
              u.z = *reinterpret_cast<uint32_t *>(&h2); u.w = *reinterpret_cast<uint32_t *>(&h3);
              *reinterpret_cast<uint4 *>(o + c * 32 + j) = u;
            }
          } else {
#pragma unroll
            for (int j = 0; j < 32; j += 4)
              *reinterpret_cast<uint4 *>(po + c * 32 + j) = make_uint4(v[j], v[j + 1], v[j + 2], v[j + 3]);
          }
        }
      }
      if (my_slot >= 0 && a.splits > 1) { a.part_ml[pidx * 2] = m_ref; a.part_ml[pidx * 2 + 1] = l_run; }
    }
  }

  // ---- teardown ----
  sm100::tc_fence_before();
  __syncthreads();
  if (ctl.abort_flag) {
    if (threadIdx.x == 0 && a.status) atomicExch(a.status, 2);
    for (int i = 0; i < 2000; ++i) __nanosleep(1000);
    __syncthreads();
  }
  if (warp == 1) {
    __syncwarp();
    sm100::tc_fence_after();
    sm100::tmem_dealloc(tmem, L::TMEM_COLS);
  }
  if (threadIdx.x == 0) tl_end(tl);
}

// Merge the per-split partial results: O = sum_s 2^(m_s - M) O_s / sum_s 2^(m_s - M) l_s.
// HD / 4 threads per (row, head), four consecutive columns each: 16-byte loads, 8-byte stores.
template <int HD>
__global__ void attn_combine_kernel(const float *__restrict__ part_O, const float *__restrict__ part_ml, int splits, int R, int Hq,
                               bf16 *__restrict__ O, TlSlot tl) {
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x == 0) tl_go(tl);
  constexpr int PER = HD / 4;
  const size_t gid = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const size_t wid = gid / PER;
  const int c4 = (int)(gid % PER);
  if (wid >= (size_t)R * Hq) { if (threadIdx.x == 0) tl_end(tl); return; }
  float M = -INFINITY;
  for (int s = 0; s < splits; ++s) M = fmaxf(M, part_ml[((size_t)s * R * Hq + wid) * 2]);
  float den = 0.f;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
  for (int s = 0; s < splits; ++s) {
    const size_t idx = (size_t)s * R * Hq + wid;
    const float m = part_ml[idx * 2], l = part_ml[idx * 2 + 1];
    const float wgt = (m == -INFINITY) ? 0.f : exp2f(m - M);
    den += wgt * l;
    const float4 v = reinterpret_cast<const float4 *>(part_O + idx * HD)[c4];
    acc.x = fmaf(wgt, v.x, acc.x); acc.y = fmaf(wgt, v.y, acc.y); acc.z = fmaf(wgt, v.z, acc.z); acc.w = fmaf(wgt, v.w, acc.w);
  }
  const float inv = 1.f / den;
  __nv_bfloat162 h0 = __floats2bfloat162_rn(acc.x * inv, acc.y * inv), h1 = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
  uint2 u; u.x = *reinterpret_cast<uint32_t *>(&h0); u.y = *reinterpret_cast<uint32_t *>(&h1);
  reinterpret_cast<uint2 *>(O + wid * HD)[c4] = u;
  if (threadIdx.x == 0) tl_end(tl);
}

}  // namespace attn_tc
