// Shared declarations for the TiDAR decode-step kernels (sm_100a).
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

typedef __nv_bfloat16 bf16;

// Per-row metadata of one pass (a decode step or a prefill chunk).  A "row" is one
// token slot.  Every row attends to cache positions [0, nvis) of its sequence plus
// the nloc local (never cached) K/V rows starting at loc0.  This one rule covers the
// whole structured mask of the decode step: causal slot j has its K/V written to the
// cache at position n+j before attention, so it sees nvis = n+j+1 and nothing local;
// mask slot (b,i) sees nvis = n+b+1 (the prefix plus causal slots 0..b) and the k
// local slots of its own block.
struct RowMeta {
  int32_t *ids;        // token id
  int32_t *pos;        // position id (RoPE)
  int32_t *seq;        // sequence slot
  int32_t *nvis;       // visible cache positions
  int32_t *loc0;       // first local K/V row (or 0 when nloc == 0)
  int32_t *nloc;       // number of local K/V rows visible
  int32_t *cache_pos;  // where this row's K/V go in the cache, or -1
  int32_t *local_idx;  // where this row's K/V go in the local scratch, or -1
  uint32_t *skey;      // sampling key of the position this row predicts (written when sampling is on)
};

struct KvGeom {
  int32_t n_kv_heads, head_dim, page_size, pages_per_seq;
  const int32_t *page_table;   // [max_batch][pages_per_seq]
  int32_t n_pages;             // pages in the pool; 0 = the table is the library's own and needs no check
};

__device__ __forceinline__ size_t kv_row_offset(const KvGeom &g, int seq, int position, int kvh) {
  int page = g.page_table[(size_t)seq * g.pages_per_seq + position / g.page_size];
  return (((size_t)page * g.n_kv_heads + kvh) * g.page_size + (position % g.page_size)) * (size_t)g.head_dim;
}

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// ---- seeded sampling -------------------------------------------------------------------
// A prediction is drawn from softmax(logits / temperature) by the Gumbel-max rule: the argmax of
// logits / temperature + noise(id).  The noise is a pure function of (seed, sequence slot,
// PREDICTED position, token id), so the autoregressive row of a position, the diffusion slots
// that pre-draft it and a one-token-per-pass decoder all draw with the same noise, whatever pass
// the position falls into.  mix64 is SplitMix64's output function, fmix32 MurmurHash3's 32-bit
// finaliser.
__device__ __forceinline__ unsigned long long mix64(unsigned long long z) {
  z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
  z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
  return z ^ (z >> 31);
}
__device__ __forceinline__ uint32_t fmix32(uint32_t h) {
  h ^= h >> 16; h *= 0x85EBCA6Bu; h ^= h >> 13; h *= 0xC2B2AE35u; h ^= h >> 16;
  return h;
}
__device__ __forceinline__ uint32_t position_key(unsigned long long seed, int seq, int pos) {
  return (uint32_t)(mix64(mix64(seed + 0x9E3779B97F4A7C15ull) ^ (((unsigned long long)(uint32_t)seq << 32) | (uint32_t)pos)) >> 32);
}
// Standard Gumbel noise -ln(-ln u), u = (m + 1/2) / 2^24 with m the top 24 bits of the hash.
// -ln u goes through log1p where u is close to 1 (there m + 1/2 is not a float, 2^24 - m - 1/2 is),
// so the largest draws, the ones most likely to win, are as accurate as the rest.
__device__ __forceinline__ float gumbel_noise(uint32_t key, uint32_t id) {
  const uint32_t m = fmix32(key + id * 0x9E3779B9u) >> 8;
  float e;
  if (m < (1u << 23)) e = -logf(((float)m + 0.5f) * (1.0f / 16777216.0f));
  else e = -log1pf(-((float)(16777216u - m) - 0.5f) * (1.0f / 16777216.0f));
  return -logf(e);
}

// Programmatic dependent launch.  A kernel launched with the programmatic-serialization
// attribute may start while the previous kernel of the stream is still running;
// pdl_wait() blocks until that kernel has completed and its writes are visible, so
// everything before it may only touch data no earlier kernel writes (weights, the
// kernel's own shared / tensor memory).  pdl_trigger() lets the next kernel of the stream
// be scheduled early in the same way.  Both are no-ops in a plain launch.
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }

// Optional in-kernel timeline (diagnostics; off when t is null).  Every launch of a pass gets a
// slot of two words, both zeroed before the pass: t[0] collects the bit-wise complement of the
// EARLIEST moment a CTA got past its dependency on the previous kernel (atomicMax of ~time =
// minimum of time), t[1] the LATEST moment a CTA finished.  end - start is then the time the
// launch really occupied inside a replayed graph with programmatic launches, where events
// cannot be placed without changing the schedule.  One thread per CTA calls each.
struct TlSlot { unsigned long long *t; };
__device__ __forceinline__ unsigned long long global_ns() {
  unsigned long long t;
  asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
  return t;
}
__device__ __forceinline__ void tl_go(TlSlot s) { if (s.t) atomicMax(s.t, ~global_ns()); }
__device__ __forceinline__ void tl_end(TlSlot s) { if (s.t) atomicMax(s.t + 1, global_ns()); }
