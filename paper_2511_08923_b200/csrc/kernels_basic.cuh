// Slot assembly, embedding, RMSNorm, RoPE + KV placement, SwiGLU, argmax,
// draft/verify and KV commit kernels of the TiDAR decode step.
#pragma once
#include "common.cuh"
#include "sm100_ptx.cuh"

// Four consecutive split-K partial sums starting at p (fp32 or bf16 slabs).
template <typename T> __device__ __forceinline__ float4 load4(const T *p);
template <> __device__ __forceinline__ float4 load4<float>(const float *p) { return *reinterpret_cast<const float4 *>(p); }
template <> __device__ __forceinline__ float4 load4<bf16>(const bf16 *p) {
  const uint2 u = *reinterpret_cast<const uint2 *>(p);
  const float2 a = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&u.x)), b = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&u.y));
  return make_float4(a.x, a.y, b.x, b.y);
}

// One embedding row (bf16, d a multiple of 8) -> fp32, 16-byte loads.
__device__ __forceinline__ void embed_row_to_f32(const bf16 *__restrict__ e, float *__restrict__ x, int d) {
  for (int c = threadIdx.x * 8; c < d; c += blockDim.x * 8) {
    const uint4 u = *reinterpret_cast<const uint4 *>(e + c);
    const __nv_bfloat162 *p = reinterpret_cast<const __nv_bfloat162 *>(&u);
    const float2 a = __bfloat1622float2(p[0]), b = __bfloat1622float2(p[1]), cc = __bfloat1622float2(p[2]), dd = __bfloat1622float2(p[3]);
    *reinterpret_cast<float4 *>(x + c) = make_float4(a.x, a.y, b.x, b.y);
    *reinterpret_cast<float4 *>(x + c + 4) = make_float4(cc.x, cc.y, dd.x, dd.y);
  }
}

// ---------------------------------------------------------------------------
// Slot assembly + embedding gather for a decode step.
// Slot layout per sequence (k causal slots, then n_blocks blocks of k mask slots;
// paper Section 3.3 footnote, figure "TiDAR Attention Masks"):
//   causal j       : token block[j], position n+j
//   mask (b, i)    : [MASK], position n+b+1+i (no label shift: a mask slot predicts
//                    its own position; paper Section 4.4.3)
// n_blocks = k for a TiDAR step; n_blocks = 0 for a plain autoregressive step (the
// causal section alone: paper Section 3.1, the model keeps its autoregressive mode).
// The step may use a block length k that differs from the one the previous pass left
// (blk_len[seq] valid entries): drafts the sequence does not have are fed as [MASK]
// and can never be accepted (see verify_select_kernel).
// The listed sequences may use different block lengths in one step: step_k[s] is sequence s's,
// step_off[s] its first row and step_loc[s] its first step-local K/V row (null: all use k).
// One block per row; also snapshots n into step_n for the commit kernel.
// ---------------------------------------------------------------------------
struct StepLayout { const int32_t *k, *off, *loc; int n_seqs; };     // per listed sequence; k == null: uniform

__global__ void assemble_step_kernel(RowMeta m, const int32_t *__restrict__ step_seqs, const int32_t *__restrict__ seq_len,
                                     const int32_t *__restrict__ block_ids, const int32_t *__restrict__ blk_len, int k, int n_blocks,
                                     StepLayout lay, int k_max, int mask_id,
                                     int32_t *__restrict__ step_n, const bf16 *__restrict__ embed, int d,
                                     float *__restrict__ X, int sampling, unsigned long long seed, TlSlot tl) {
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x == 0) tl_go(tl);
  const int r = blockIdx.x;
  int s, slot, loc_base;
  if (lay.k) {                                   // per-sequence block lengths: find the sequence this row belongs to
    s = 0;
    while (s + 1 < lay.n_seqs && r >= lay.off[s + 1]) ++s;
    k = lay.k[s]; n_blocks = k; slot = r - lay.off[s]; loc_base = lay.loc[s];
  } else {
    const int T = k * (n_blocks + 1);
    s = r / T; slot = r % T; loc_base = s * k * k;
  }
  const int seq = step_seqs[s];
  const int n = seq_len[seq];
  int id;
  if (slot < k && slot < blk_len[seq]) id = block_ids[seq * k_max + slot]; else id = mask_id;
  if (threadIdx.x == 0) {
    if (slot == 0) step_n[s] = n;
    m.seq[r] = seq;
    m.ids[r] = id;
    if (slot < k) {
      m.pos[r] = n + slot; m.nvis[r] = n + slot + 1; m.loc0[r] = 0; m.nloc[r] = 0;
      m.cache_pos[r] = n + slot; m.local_idx[r] = -1;
      if (sampling) m.skey[r] = position_key(seed, seq, n + slot + 1);        // a causal slot predicts the next position
    } else {
      const int b = (slot - k) / k, i = (slot - k) % k;
      m.pos[r] = n + b + 1 + i; m.nvis[r] = n + b + 1; m.loc0[r] = loc_base + b * k; m.nloc[r] = k;
      m.cache_pos[r] = -1; m.local_idx[r] = loc_base + b * k + i;
      if (sampling) m.skey[r] = position_key(seed, seq, n + b + 1 + i);       // a mask slot predicts its own position
    }
  }
  embed_row_to_f32(embed + (size_t)id * d, X + (size_t)r * d, d);
  if (threadIdx.x == 0) tl_end(tl);
}

// Prefill chunk: rows g = row0 .. row0+rows-1 of [prompt ; k mask tokens]
// (paper Section 3.2, Appendix B): prompt rows causal, mask rows see the whole
// prompt and each other.
__global__ void assemble_prefill_kernel(RowMeta m, int seq, int row0, int n_prompt, int k, int mask_id,
                                        const int32_t *__restrict__ prompt, const bf16 *__restrict__ embed, int d,
                                        float *__restrict__ X, int sampling, unsigned long long seed) {
  const int r = blockIdx.x;
  const int g = row0 + r;
  const int id = g < n_prompt ? prompt[g] : mask_id;
  if (threadIdx.x == 0) {
    m.seq[r] = seq; m.ids[r] = id; m.pos[r] = g;
    if (g < n_prompt) {
      m.nvis[r] = g + 1; m.loc0[r] = 0; m.nloc[r] = 0; m.cache_pos[r] = g; m.local_idx[r] = -1;
      if (sampling) m.skey[r] = position_key(seed, seq, g + 1);
    } else {
      m.nvis[r] = n_prompt; m.loc0[r] = 0; m.nloc[r] = k; m.cache_pos[r] = -1; m.local_idx[r] = g - n_prompt;
      if (sampling) m.skey[r] = position_key(seed, seq, g);
    }
  }
  embed_row_to_f32(embed + (size_t)id * d, X + (size_t)r * d, d);
}

// Row metadata for the stand-alone attention entry point (same slot layout as a step).
// seq_len comes from the caller: it is clamped to [0, n_max] (n_max = the positions the page
// table can back minus the k causal slots), so that no row looks past the table.
__global__ void attn_meta_kernel(RowMeta m, const int32_t *__restrict__ seq_len, int k, int R, int n_max) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r >= R) return;
  const int T = k * (k + 1);
  const int s = r / T, slot = r % T;
  const int n = min(max(seq_len[s], 0), n_max);
  m.seq[r] = s;
  if (slot < k) {
    m.pos[r] = n + slot; m.nvis[r] = n + slot + 1; m.loc0[r] = 0; m.nloc[r] = 0;
  } else {
    const int b = (slot - k) / k;
    m.pos[r] = n + b + 1 + (slot - k) % k; m.nvis[r] = n + b + 1; m.loc0[r] = s * k * k + b * k; m.nloc[r] = k;
  }
}

// cos/sin of pos * theta^(-2i/hd), evaluated in double once per pass (shared by every
// layer and head), stored as float.
__global__ void rope_table_kernel(const int32_t *__restrict__ pos, int R, int half, double theta,
                                  float *__restrict__ cs, float *__restrict__ sn, TlSlot tl) {
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x == 0) tl_go(tl);
  const int t = blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= R * half) { if (threadIdx.x == 0) tl_end(tl); return; }
  const int r = t / half, i = t % half;
  const double inv = pow(theta, -(double)i / (double)half);
  double s, c;
  sincos((double)pos[r] * inv, &s, &c);
  cs[t] = (float)c; sn[t] = (float)s;
  if (threadIdx.x == 0) tl_end(tl);
}

// ---------------------------------------------------------------------------
// Residual update + RMSNorm.  X (fp32 residual stream) += sum over the S split-K
// partial results of the previous projection (fixed order: deterministic), then
// A = bf16(X * rsqrt(mean(X^2) + eps) * gain).  One block per row.
// ---------------------------------------------------------------------------
template <int THREADS, typename SLAB>
__global__ void __launch_bounds__(THREADS)
rmsnorm_reduce_kernel(float *__restrict__ X, const SLAB *__restrict__ partials, int S, size_t partial_stride,
                      const bf16 *__restrict__ gain, float eps, int d, bf16 *__restrict__ A, TlSlot tl) {
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x == 0) tl_go(tl);
  extern __shared__ float row[];
  __shared__ float red[THREADS / 32];
  const int r = blockIdx.x;
  float ss = 0.f;
  float *xr = X + (size_t)r * d;
  for (int c = threadIdx.x * 4; c < d; c += THREADS * 4) {
    float4 v = *reinterpret_cast<const float4 *>(xr + c);
    for (int s = 0; s < S; ++s) {
      const float4 p = load4<SLAB>(partials + s * partial_stride + (size_t)r * d + c);
      v.x += p.x; v.y += p.y; v.z += p.z; v.w += p.w;
    }
    *reinterpret_cast<float4 *>(row + c) = v;
    ss += v.x * v.x + v.y * v.y + v.z * v.z + v.w * v.w;
  }
  ss = warp_sum(ss);
  if ((threadIdx.x & 31) == 0) red[threadIdx.x >> 5] = ss;
  __syncthreads();
  float tot = 0.f;
#pragma unroll
  for (int i = 0; i < THREADS / 32; ++i) tot += red[i];
  const float inv = rsqrtf(tot / (float)d + eps);
  for (int c = threadIdx.x * 4; c < d; c += THREADS * 4) {
    const float4 v = *reinterpret_cast<const float4 *>(row + c);
    if (S > 0) *reinterpret_cast<float4 *>(xr + c) = v;
    const uint2 gb = *reinterpret_cast<const uint2 *>(gain + c);
    const float2 g0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&gb.x)), g1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&gb.y));
    __nv_bfloat162 o0 = __floats2bfloat162_rn(v.x * inv * g0.x, v.y * inv * g0.y), o1 = __floats2bfloat162_rn(v.z * inv * g1.x, v.w * inv * g1.y);
    uint2 ob; ob.x = *reinterpret_cast<uint32_t *>(&o0); ob.y = *reinterpret_cast<uint32_t *>(&o1);
    *reinterpret_cast<uint2 *>(A + (size_t)r * d + c) = ob;
  }
  if (threadIdx.x == 0) tl_end(tl);
}

// ---------------------------------------------------------------------------
// RoPE + KV placement.  Input: S split-K partials of the QKV projection, fp32
// [S][R][(Hq+2Hkv)*hd].  Q heads are rotated and stored bf16 [R][Hq][hd]; K heads are
// rotated, V heads copied; both go to the paged cache at the row's cache position
// (causal slots: kept if accepted, evicted otherwise; paper Section 3.3) or to the
// step-local scratch (mask slots, never cached).  Grid (rows, unit chunks of 256).
// Optional, for checkpoints of the decoder families the paper starts from (Section 4.1):
// bias [(Hq+2Hkv)*hd] added to the projection; qn / kn [hd]: RMSNorm over each Q / K head's
// dimensions before the rotation (the hd/8 threads of a head reduce with shuffles).
// ---------------------------------------------------------------------------
template <typename SLAB>
__global__ void __launch_bounds__(256)
rope_kv_kernel(const SLAB *__restrict__ partials, int S, size_t partial_stride, int Hq, int Hkv, int hd,
               RowMeta m, const float *__restrict__ cs, const float *__restrict__ sn, KvGeom g,
               bf16 *__restrict__ Q, bf16 *__restrict__ Kpool, bf16 *__restrict__ Vpool,
               bf16 *__restrict__ Kloc, bf16 *__restrict__ Vloc,
               const bf16 *__restrict__ bias, const bf16 *__restrict__ qn, const bf16 *__restrict__ kn, float eps, TlSlot tl) {
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x == 0) tl_go(tl);
  // a work unit is 4 consecutive dims i..i+3 of the first half of one
  // head together with their rotation partners i+hd/2..
  const int r = blockIdx.x, half = hd / 2, upr = half / 4;          // units per head
  const int H = Hq + 2 * Hkv, N = H * hd;
  const int cp = m.cache_pos[r], seq = m.seq[r], li = m.local_idx[r];
  // grid (rows, ceil(units / 256)): one unit per thread, so a row's latency is one round of loads
  for (int u = blockIdx.y * blockDim.x + threadIdx.x; u < H * upr; u += gridDim.y * blockDim.x) {
    const int h = u / upr, i = (u % upr) * 4;
    const size_t base = (size_t)r * N + (size_t)h * hd + i;
    float4 x1 = make_float4(0.f, 0.f, 0.f, 0.f), x2 = x1;
    for (int s = 0; s < S; ++s) {
      const float4 a = load4<SLAB>(partials + s * partial_stride + base);
      const float4 b = load4<SLAB>(partials + s * partial_stride + base + half);
      x1.x += a.x; x1.y += a.y; x1.z += a.z; x1.w += a.w;
      x2.x += b.x; x2.y += b.y; x2.z += b.z; x2.w += b.w;
    }
    if (bias) {
      const uint2 b1 = *reinterpret_cast<const uint2 *>(bias + (size_t)h * hd + i), b2 = *reinterpret_cast<const uint2 *>(bias + (size_t)h * hd + i + half);
      const float2 p0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&b1.x)), p1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&b1.y));
      const float2 q0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&b2.x)), q1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&b2.y));
      x1.x += p0.x; x1.y += p0.y; x1.z += p1.x; x1.w += p1.y;
      x2.x += q0.x; x2.y += q0.y; x2.z += q1.x; x2.w += q1.y;
    }
    const bf16 *hn = h < Hq ? qn : (h < Hq + Hkv ? kn : nullptr);
    if (hn) {
      // the upr = hd/8 threads of this head are consecutive lanes of one warp (upr is 8 or 16 and
      // divides the unit index), and all of them are here: the loop bound is a multiple of upr
      float ss = x1.x * x1.x + x1.y * x1.y + x1.z * x1.z + x1.w * x1.w + x2.x * x2.x + x2.y * x2.y + x2.z * x2.z + x2.w * x2.w;
      const int lane = threadIdx.x & 31;
      const unsigned gmask = (upr >= 32 ? 0xffffffffu : ((1u << upr) - 1u)) << (lane & ~(upr - 1));
      for (int o = upr >> 1; o > 0; o >>= 1) ss += __shfl_xor_sync(gmask, ss, o);
      const float inv = rsqrtf(ss / (float)hd + eps);
      const uint2 g1 = *reinterpret_cast<const uint2 *>(hn + i), g2 = *reinterpret_cast<const uint2 *>(hn + i + half);
      const float2 p0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&g1.x)), p1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&g1.y));
      const float2 q0 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&g2.x)), q1 = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(&g2.y));
      x1.x *= inv * p0.x; x1.y *= inv * p0.y; x1.z *= inv * p1.x; x1.w *= inv * p1.y;
      x2.x *= inv * q0.x; x2.y *= inv * q0.y; x2.z *= inv * q1.x; x2.w *= inv * q1.y;
    }
    bf16 *dst;
    bool rotate = true;
    if (h < Hq) {
      dst = Q + ((size_t)r * Hq + h) * hd;
    } else {
      const bool isk = h < Hq + Hkv;
      const int kvh = isk ? h - Hq : h - Hq - Hkv;
      if (cp >= 0) dst = (isk ? Kpool : Vpool) + kv_row_offset(g, seq, cp, kvh);
      else dst = (isk ? Kloc : Vloc) + ((size_t)li * Hkv + kvh) * hd;
      rotate = isk;
    }
    float4 y1 = x1, y2 = x2;
    if (rotate) {
      const float4 c = *reinterpret_cast<const float4 *>(cs + r * half + i), sv = *reinterpret_cast<const float4 *>(sn + r * half + i);
      y1 = make_float4(x1.x * c.x - x2.x * sv.x, x1.y * c.y - x2.y * sv.y, x1.z * c.z - x2.z * sv.z, x1.w * c.w - x2.w * sv.w);
      y2 = make_float4(x2.x * c.x + x1.x * sv.x, x2.y * c.y + x1.y * sv.y, x2.z * c.z + x1.z * sv.z, x2.w * c.w + x1.w * sv.w);
    }
    __nv_bfloat162 a0 = __floats2bfloat162_rn(y1.x, y1.y), a1 = __floats2bfloat162_rn(y1.z, y1.w);
    __nv_bfloat162 b0 = __floats2bfloat162_rn(y2.x, y2.y), b1 = __floats2bfloat162_rn(y2.z, y2.w);
    uint2 o1, o2;
    o1.x = *reinterpret_cast<uint32_t *>(&a0); o1.y = *reinterpret_cast<uint32_t *>(&a1);
    o2.x = *reinterpret_cast<uint32_t *>(&b0); o2.y = *reinterpret_cast<uint32_t *>(&b1);
    *reinterpret_cast<uint2 *>(dst + i) = o1;
    *reinterpret_cast<uint2 *>(dst + i + half) = o2;
  }
  if (threadIdx.x == 0) tl_end(tl);
}

// SwiGLU on an fp32 [R][2*ffn] projection whose columns interleave (gate_f, up_f).
__global__ void swiglu_kernel(const float *__restrict__ GU, int R, int ffn, bf16 *__restrict__ H) {
  const size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (t >= (size_t)R * ffn) return;
  const float g = GU[2 * t], u = GU[2 * t + 1];
  H[t] = __float2bfloat16(g / (1.f + __expf(-g)) * u);
}

// SwiGLU over split-K slabs [S][R][ld] (fp32 or bf16) whose columns interleave (gate, up) and
// cover features [f0, f0 + nf): H[r][f0 + f] = silu(sum_s gate) * (sum_s up).  Two features per thread.
template <typename SLAB>
__global__ void swiglu_slab_kernel(const SLAB *__restrict__ slabs, int S, size_t stride, int R, int ld, int nf, int f0, int ldh,
                                   bf16 *__restrict__ H, TlSlot tl) {
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x == 0) tl_go(tl);
  // two features per thread; silu with the fast division of the fused epilogue (a precise
  // division costs ~170 cycles per result and was most of this kernel's time)
  const size_t t = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  const int nf2 = nf / 2;
  if (t >= (size_t)R * nf2) { if (threadIdx.x == 0) tl_end(tl); return; }
  const int r = (int)(t / nf2), f = (int)(t % nf2) * 2;
  float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);                      // gate f, up f, gate f+1, up f+1
  for (int s = 0; s < S; ++s) {
    const float4 v = load4<SLAB>(slabs + s * stride + (size_t)r * ld + 2 * f);
    acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
  }
  __nv_bfloat162 o = __floats2bfloat162_rn(__fdividef(acc.x, 1.f + __expf(-acc.x)) * acc.y, __fdividef(acc.z, 1.f + __expf(-acc.z)) * acc.w);
  *reinterpret_cast<__nv_bfloat162 *>(H + (size_t)r * ldh + f0 + f) = o;
  if (threadIdx.x == 0) tl_end(tl);
}

// Running per-row argmax over a chunk of logits [R][ncols] (fp32, leading dim ld)
// that covers vocabulary ids [col0, col0+ncols).  Lowest index wins ties; NaN never
// wins.  Optionally copies the chunk into a full [R][vocab] dump.
// With inv_temp > 0 the compared value is logit * inv_temp + Gumbel noise of (skey[r], id): a draw
// from softmax(logits / temperature) instead of the argmax; the dump always holds the raw logits.
__global__ void argmax_chunk_kernel(const float *__restrict__ L, int ld, int ncols, int col0, int first,
                                    float *__restrict__ best_val, int32_t *__restrict__ best_idx,
                                    float *__restrict__ dump, int vocab, float inv_temp, const uint32_t *__restrict__ skey) {
  const int r = blockIdx.x;
  float bv = -INFINITY; int bi = 0x7fffffff;
  const uint32_t key = inv_temp > 0.f ? skey[r] : 0u;
  for (int c = threadIdx.x; c < ncols; c += blockDim.x) {
    float v = L[(size_t)r * ld + c];
    if (dump) dump[(size_t)r * vocab + col0 + c] = v;
    if (inv_temp > 0.f) v = v * inv_temp + gumbel_noise(key, (uint32_t)(col0 + c));
    if (v > bv) { bv = v; bi = col0 + c; }
  }
  __shared__ float sv[32]; __shared__ int si[32];
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, o); const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
  }
  if ((threadIdx.x & 31) == 0) { sv[threadIdx.x >> 5] = bv; si[threadIdx.x >> 5] = bi; }
  __syncthreads();
  if (threadIdx.x == 0) {
    for (int w = 1; w < (int)(blockDim.x >> 5); ++w)
      if (sv[w] > bv || (sv[w] == bv && si[w] < bi)) { bv = sv[w]; bi = si[w]; }
    if (!first) {
      const float pv = best_val[r]; const int pi = best_idx[r];
      if (pv > bv || (pv == bv && pi < bi) || bi == 0x7fffffff) { bv = pv; bi = pi; }
    }
    if (bi == 0x7fffffff) bi = 0;
    best_val[r] = bv; best_idx[r] = bi;
  }
}

// Final argmax over the candidates [R][G] produced by the fused LM-head epilogue (one
// candidate per CTA and lane quadrant): one warp per row; a candidate index of -1 means
// "nothing valid".  Lowest index wins ties, which makes the result independent of the
// order in which candidates are combined.
__global__ void argmax_merge_kernel(const float *__restrict__ pv, const int32_t *__restrict__ pi, int G, int R,
                                    float *__restrict__ best_val, int32_t *__restrict__ best_idx, TlSlot tl) {
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x == 0) tl_go(tl);
  const int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5, lane = threadIdx.x & 31;
  if (r >= R) { if (threadIdx.x == 0) tl_end(tl); return; }
  float bv = -INFINITY; int bi = 0x7fffffff;
  for (int g = lane; g < G; g += 32) {
    const float v = pv[(size_t)r * G + g]; const int i = pi[(size_t)r * G + g];
    if (i >= 0 && (v > bv || (v == bv && i < bi))) { bv = v; bi = i; }
  }
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, o); const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (ov > bv || (ov == bv && oi < bi)) { bv = ov; bi = oi; }
  }
  if (lane == 0) { best_val[r] = bv; best_idx[r] = bi == 0x7fffffff ? 0 : bi; }
  if (threadIdx.x == 0) tl_end(tl);
}

// out[i] = sum over S slabs (fixed order) of in[s * stride + i].
__global__ void slab_sum_kernel(const float *__restrict__ in, int S, size_t stride, size_t n, float *__restrict__ out) {
  const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
  if (i >= n) return;
  float v = 0.f;
  for (int s = 0; s < S; ++s) v += in[s * stride + i];
  out[i] = v;
}

// ---------------------------------------------------------------------------
// Draft / verify / select (paper Section 3.2; Section 4.4.3).
// One warp per sequence, lane i = causal slot i:
//   target_i = verified prediction for position n+i+1: argmax of causal slot i's logits, or
//              (tgt_ids != null) the argmax of the row that mixes them with the first slot
//              of block i;
//   draft i >= 1 agrees iff the sequence had a draft there (i < blk_len) and
//              block[i] == target_{i-1};
//   L = 1 + length of the leading run of agreeing drafts (slot 0 is settled), or the
//   forced value;  emitted = block[1..L-1], target_{L-1};
//   next block = target_{L-1}, then the argmax of mask slots (L-1, 1..k-1); with no mask
//   blocks (plain autoregressive step, k = 1) the next block is target_0 alone.
// ---------------------------------------------------------------------------
__global__ void verify_select_kernel(const int32_t *__restrict__ arg_ids, const int32_t *__restrict__ tgt_ids,
                                     const int32_t *__restrict__ step_seqs,
                                     const int32_t *__restrict__ forced, int k, int n_blocks, StepLayout lay, int k_max,
                                     int32_t *__restrict__ block_ids, int32_t *__restrict__ blk_len, int32_t *__restrict__ step_L,
                                     int32_t *__restrict__ out /*[n_seqs][k_max+1]*/, TlSlot tl) {
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x == 0) tl_go(tl);
  const int s = blockIdx.x, lane = threadIdx.x;
  if (lay.k) { k = lay.k[s]; n_blocks = k; }
  const int T = k * (n_blocks + 1);
  const int seq = step_seqs[s];
  const int32_t *ids = arg_ids + (lay.k ? (size_t)lay.off[s] : (size_t)s * T);
  int32_t *blk = block_ids + (size_t)seq * k_max;
  const int valid = blk_len[seq];
  size_t tgt0 = (size_t)s * k;                    // this sequence's first verification target among the mixed rows
  if (lay.k && tgt_ids) { tgt0 = 0; for (int t = 0; t < s; ++t) tgt0 += lay.k[t]; }
  const int tgt = lane < k ? (tgt_ids ? tgt_ids[tgt0 + lane] : ids[lane]) : -1;
  const int mine = lane < k ? (lane < valid ? blk[lane] : -2) : -2;
  const int prev_tgt = __shfl_up_sync(0xffffffffu, tgt, 1);
  const bool agree = lane == 0 || (lane < k && lane < valid && mine == prev_tgt);
  const unsigned bits = __ballot_sync(0xffffffffu, agree);
  int L = __ffs(~bits) - 1;            // leading run of ones; bit 0 is always set
  if (L > k || L < 0) L = k;           // all 32 lanes agreeing gives ffs(0) = 0
  const int f = forced ? forced[s] : 0;
  if (f > 0) L = f;
  const int t_last = __shfl_sync(0xffffffffu, tgt, L - 1);
  const int next_draft = (n_blocks > 0 && lane >= 1 && lane < k) ? ids[k + (L - 1) * k + lane] : 0;
  const int shifted = __shfl_down_sync(0xffffffffu, mine, 1);     // block[lane+1]
  __syncwarp();
  if (lane < k) {
    out[(size_t)s * (k_max + 1) + 1 + lane] = lane < L - 1 ? shifted : (lane == L - 1 ? t_last : -1);
    blk[lane] = lane == 0 ? t_last : next_draft;
  }
  if (lane == 0) { out[(size_t)s * (k_max + 1)] = L; step_L[s] = L; blk_len[seq] = n_blocks > 0 ? k : 1; tl_end(tl); }
}

// Verification by a mix of the autoregressive and the diffusion prediction (paper Section 4.4.3:
// argmax(beta * logits_ar + (1 - beta) * logits_diff)).  Logits are linear in the final-normed
// hidden row, so the mix is taken there: row dst = beta * row a + (1 - beta) * row b of the LM
// head's input, one extra input row per verified position, and the LM head's argmax of that row
// is the argmax of the mixed logits.  Block i handles pair i:
//   a = a0 + (i / k) * a_seq + (i % k) * a_j,  b likewise,  dst = dst0 + i.
// With per-sequence block lengths (lay.k != null) pair i belongs to the sequence whose pairs
// (one per verified position, k_s of them) contain it: a = off_s + j, b = off_s + k_s + j * k_s.
__global__ void mix_rows_kernel(bf16 *__restrict__ A, int d, float beta, int k, int a0, int a_seq, int a_j, int b0, int b_seq, int b_j,
                                StepLayout lay, int dst0, uint32_t *__restrict__ skey, TlSlot tl) {
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x == 0) tl_go(tl);
  const int i = blockIdx.x;
  int row_a, row_b;
  if (lay.k) {
    int s = 0, p = 0;
    while (s + 1 < lay.n_seqs && i >= p + lay.k[s]) { p += lay.k[s]; ++s; }
    const int ks = lay.k[s], j = i - p;
    row_a = lay.off[s] + j; row_b = lay.off[s] + ks + j * ks;
  } else {
    const int s = i / k, j = i % k;
    row_a = a0 + s * a_seq + j * a_j; row_b = b0 + s * b_seq + j * b_j;
  }
  const bf16 *ra = A + (size_t)row_a * d, *rb = A + (size_t)row_b * d;
  bf16 *ro = A + (size_t)(dst0 + i) * d;
  if (skey && threadIdx.x == 0) skey[dst0 + i] = skey[row_a];     // the mixed row predicts what row a predicts
  for (int c = threadIdx.x * 2; c < d; c += blockDim.x * 2) {
    const float2 x = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(ra + c));
    const float2 y = __bfloat1622float2(*reinterpret_cast<const __nv_bfloat162 *>(rb + c));
    *reinterpret_cast<__nv_bfloat162 *>(ro + c) = __floats2bfloat162_rn(beta * x.x + (1.f - beta) * y.x, beta * x.y + (1.f - beta) * y.y);
  }
  if (threadIdx.x == 0) tl_end(tl);
}

// Running log-sum-exp of a row over vocabulary chunks, and the logit of the row's target id.
// L [R][ld] holds the logits of ids [col0, col0 + ncols).  (run_max, run_sum) is updated so that
// log sum_v exp(logit_v) = run_max + log(run_sum) after the last chunk; fixed reduction order.
__global__ void __launch_bounds__(256)
score_chunk_kernel(const float *__restrict__ L, int ld, int ncols, int col0, int first, const int32_t *__restrict__ target,
                   float *__restrict__ run_max, float *__restrict__ run_sum, float *__restrict__ tgt_logit) {
  __shared__ float red[8];
  __shared__ float bcast;
  const int r = blockIdx.x, warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  const float *row = L + (size_t)r * ld;
  float m = -INFINITY;
  for (int c = threadIdx.x; c < ncols; c += 256) m = fmaxf(m, row[c]);
  m = warp_max(m);
  if (lane == 0) red[warp] = m;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = red[0];
    for (int i = 1; i < 8; ++i) t = fmaxf(t, red[i]);
    bcast = first ? t : fmaxf(t, run_max[r]);
  }
  __syncthreads();
  const float M = bcast;
  float sum = 0.f;
  for (int c = threadIdx.x; c < ncols; c += 256) sum += __expf(row[c] - M);
  sum = warp_sum(sum);
  __syncthreads();
  if (lane == 0) red[warp] = sum;
  __syncthreads();
  if (threadIdx.x == 0) {
    float t = 0.f;
    for (int i = 0; i < 8; ++i) t += red[i];
    if (!first) t += run_sum[r] * __expf(run_max[r] - M);
    run_max[r] = M; run_sum[r] = t;
    const int tg = target[r] - col0;
    if (tg >= 0 && tg < ncols) tgt_logit[r] = row[tg];
  }
}

// logprob[r] = tgt_logit[r] - (run_max[r] + log(run_sum[r]))
__global__ void score_finish_kernel(const float *__restrict__ run_max, const float *__restrict__ run_sum, const float *__restrict__ tgt_logit,
                                    int R, float *__restrict__ logprob) {
  const int r = blockIdx.x * blockDim.x + threadIdx.x;
  if (r < R) logprob[r] = tgt_logit[r] - (run_max[r] + logf(run_sum[r]));
}

// First-pass finish: settled token = argmax of the last prompt row; drafts = argmax
// of mask rows 1..k-1 (paper Section 3.2, start of generation).
// row_first: the row whose argmax is the settled token (the last prompt row, or the extra row that
// mixes it with the first mask row when beta < 1).
__global__ void prefill_finish_kernel(const int32_t *__restrict__ arg_ids, int row_last_prompt, int row_first, int k, int k_max, int seq,
                                      int n_prompt, int32_t *__restrict__ block_ids, int32_t *__restrict__ blk_len,
                                      int32_t *__restrict__ seq_len, int32_t *__restrict__ out) {
  const int i = threadIdx.x;
  if (i < k) block_ids[(size_t)seq * k_max + i] = i == 0 ? arg_ids[row_first] : arg_ids[row_last_prompt + 1 + i];
  if (i == 0) { seq_len[seq] = n_prompt; blk_len[seq] = k; out[0] = arg_ids[row_first]; }
}

// ---------------------------------------------------------------------------
// KV commit / evict (paper Section 3.3): the k causal slots' K/V were written to
// the cache at positions n..n+k-1 during the pass; committing L of them is
// n <- n + L, after which positions n+L..n+k-1 are dead and get overwritten by the
// next step.  With poison != 0 the dead slots are filled, in every layer, with the
// largest finite bf16 (3.4e38), so that any later use of evicted data with a non-zero
// weight would surface as inf/NaN or a wild value.  (Not NaN itself: the tensor-core
// attention loads whole 64-position pages and multiplies the masked positions' V rows
// by an exact zero, which must stay zero.)  Grid (n_seqs, n_layers).
// ---------------------------------------------------------------------------
__global__ void kv_commit_kernel(const int32_t *__restrict__ step_seqs, const int32_t *__restrict__ step_n,
                                 const int32_t *__restrict__ step_L, int32_t *__restrict__ seq_len, int k, const int32_t *__restrict__ step_k,
                                 int poison, KvGeom g, bf16 *__restrict__ kv_base, size_t pool_stride, TlSlot tl) {
  pdl_trigger();
  pdl_wait();
  if (threadIdx.x == 0) tl_go(tl);
  const int s = blockIdx.x, l = blockIdx.y;
  if (step_k) k = step_k[s];
  const int seq = step_seqs[s];
  const int n = step_n[s], L = step_L[s];
  if (l == 0 && threadIdx.x == 0) seq_len[seq] = n + L;
  if (!poison) { if (threadIdx.x == 0) tl_end(tl); return; }
  bf16 *Kp = kv_base + (size_t)(2 * l) * pool_stride, *Vp = Kp + pool_stride;
  const int per = g.n_kv_heads * g.head_dim;
  const bf16 nanv = __ushort_as_bfloat16((unsigned short)0x7f7f);
  for (int t = threadIdx.x; t < (k - L) * per; t += blockDim.x) {
    const int p = n + L + t / per, kvh = (t % per) / g.head_dim, c = t % g.head_dim;
    const size_t off = kv_row_offset(g, seq, p, kvh) + c;
    Kp[off] = nanv; Vp[off] = nanv;
  }
  if (threadIdx.x == 0) tl_end(tl);
}

// Gather cached K/V rows into canonical [npos][Hkv][hd] order (debug read-back).
__global__ void kv_gather_kernel(const bf16 *__restrict__ Kp, const bf16 *__restrict__ Vp, KvGeom g, int seq, int pos0,
                                 bf16 *__restrict__ ko, bf16 *__restrict__ vo) {
  const int p = blockIdx.x, kvh = blockIdx.y;
  const size_t off = kv_row_offset(g, seq, pos0 + p, kvh);
  for (int c = threadIdx.x; c < g.head_dim; c += blockDim.x) {
    ko[((size_t)p * g.n_kv_heads + kvh) * g.head_dim + c] = Kp[off + c];
    vo[((size_t)p * g.n_kv_heads + kvh) * g.head_dim + c] = Vp[off + c];
  }
}

// Probe of the bounded wait every tensor-core kernel is built on: one thread waits, with a
// short limit, on an mbarrier that nothing will ever arrive on, gives up, and reports it through
// the status word, exactly as a kernel whose producer went missing would.  Nothing hangs: the
// wait is the same bounded loop, only shorter.  waited[0] receives the polls it took.
__global__ void wait_probe_kernel(uint32_t limit, int *status, int *waited) {
  __shared__ __align__(8) uint64_t bar;
  __shared__ int abort_flag;
  if (threadIdx.x == 0) {
    abort_flag = 0;
    sm100::mbar_init(sm100::smem_u32(&bar), 1);
    sm100::fence_mbar_init();
  }
  __syncthreads();
  if (threadIdx.x == 0) {
    const bool ok = sm100::mbar_wait(sm100::smem_u32(&bar), 0u, &abort_flag, limit);      // phase 0 never completes
    waited[0] = ok ? 0 : (int)limit;
    if (!ok && abort_flag) atomicExch(status, 9);
  }
}
