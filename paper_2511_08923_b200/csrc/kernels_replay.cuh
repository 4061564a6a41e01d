// Plain CUDA-core kernels with fp32 accumulation: the diagnostic "replay" path.
// Same data flow as the tensor-core path, none of its machinery.
#pragma once
#include "common.cuh"

// C[r][n] = sum_k A[r][k] * W[n][k];  A [R][K] bf16 (lda), W [N][K] bf16 (ldw), C fp32 (ldc).
// 64x64 tile, 16-wide K slab, 256 threads, 4x4 outputs per thread.
__global__ void __launch_bounds__(256)
gemm_replay_kernel(const bf16 *__restrict__ A, int lda, const bf16 *__restrict__ W, int ldw,
                   float *__restrict__ C, int ldc, int R, int N, int K) {
  __shared__ float As[16][64 + 4];
  __shared__ float Ws[16][64 + 4];
  const int tr = blockIdx.y * 64, tn = blockIdx.x * 64;
  const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;
  float acc[4][4] = {};
  for (int k0 = 0; k0 < K; k0 += 16) {
    for (int t = threadIdx.x; t < 64 * 16; t += 256) {
      const int row = t / 16, kk = t % 16;
      const int r = tr + row, n = tn + row, k = k0 + kk;
      As[kk][row] = (r < R && k < K) ? __bfloat162float(A[(size_t)r * lda + k]) : 0.f;
      Ws[kk][row] = (n < N && k < K) ? __bfloat162float(W[(size_t)n * ldw + k]) : 0.f;
    }
    __syncthreads();
#pragma unroll
    for (int kk = 0; kk < 16; ++kk) {
      float a[4], w[4];
#pragma unroll
      for (int i = 0; i < 4; ++i) { a[i] = As[kk][ty * 4 + i]; w[i] = Ws[kk][tx * 4 + i]; }
#pragma unroll
      for (int i = 0; i < 4; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(a[i], w[j], acc[i][j]);
    }
    __syncthreads();
  }
#pragma unroll
  for (int i = 0; i < 4; ++i)
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int r = tr + ty * 4 + i, n = tn + tx * 4 + j;
      if (r < R && n < N) C[(size_t)r * ldc + n] = acc[i][j];
    }
}

// One warp per (row, query head): online softmax over the row's visible keys
// (cache positions [0, nvis) then nloc local rows), 32 keys at a time, one key per
// lane for the scores, HD/32 output dims per lane for P*V.
template <int HD>
__global__ void __launch_bounds__(32)
attn_replay_kernel(const bf16 *__restrict__ Q, const bf16 *__restrict__ Kpool, const bf16 *__restrict__ Vpool, KvGeom g,
                   RowMeta m, const bf16 *__restrict__ Kloc, const bf16 *__restrict__ Vloc, bf16 *__restrict__ O,
                   int Hq, float scale) {
  constexpr int DPL = HD / 32;
  __shared__ float qs[HD];
  const int r = blockIdx.x, h = blockIdx.y, lane = threadIdx.x;
  const int kvh = h / (Hq / g.n_kv_heads);
  const int seq = m.seq[r], nvis = m.nvis[r], nloc = m.nloc[r], loc0 = m.loc0[r];
  const bf16 *q = Q + ((size_t)r * Hq + h) * HD;
  for (int c = lane; c < HD; c += 32) qs[c] = __bfloat162float(q[c]) * scale;
  __syncwarp();
  float mx = -INFINITY, den = 0.f, acc[DPL];
#pragma unroll
  for (int i = 0; i < DPL; ++i) acc[i] = 0.f;
  const int total = nvis + nloc;
  for (int t0 = 0; t0 < total; t0 += 32) {
    const int t = t0 + lane;
    const bf16 *kr = nullptr, *vr = nullptr;
    if (t < nvis) {
      // a caller-provided table may hold anything: a key on a page outside the pool is skipped
      const int page = g.page_table[(size_t)seq * g.pages_per_seq + t / g.page_size];
      if (g.n_pages == 0 || (unsigned)page < (unsigned)g.n_pages) {
        const size_t off = (((size_t)page * g.n_kv_heads + kvh) * g.page_size + (t % g.page_size)) * (size_t)g.head_dim;
        kr = Kpool + off; vr = Vpool + off;
      }
    } else if (t < total) {
      const size_t off = ((size_t)(loc0 + t - nvis) * g.n_kv_heads + kvh) * HD;
      kr = Kloc + off; vr = Vloc + off;
    }
    float sc = -INFINITY;
    if (kr) {
      float a = 0.f;
      const uint4 *k4 = reinterpret_cast<const uint4 *>(kr);
#pragma unroll
      for (int c = 0; c < HD / 8; ++c) {
        const uint4 u = k4[c];
        const __nv_bfloat162 *p = reinterpret_cast<const __nv_bfloat162 *>(&u);
#pragma unroll
        for (int e = 0; e < 4; ++e) {
          const float2 f = __bfloat1622float2(p[e]);
          a = fmaf(f.x, qs[c * 8 + 2 * e], a);
          a = fmaf(f.y, qs[c * 8 + 2 * e + 1], a);
        }
      }
      sc = a;
    }
    const float nmx = fmaxf(mx, warp_max(sc));
    // mx = -inf before the first visible key gives 0; a chunk without any visible key while
    // nothing has been seen yet (nmx = -inf) must leave the empty sums alone, not make them NaN
    const float corr = nmx == -INFINITY ? 1.f : __expf(mx - nmx);
    const float p = kr ? __expf(sc - nmx) : 0.f;
    den = den * corr + warp_sum(p);
#pragma unroll
    for (int i = 0; i < DPL; ++i) acc[i] *= corr;
    mx = nmx;
    const unsigned long long vaddr = (unsigned long long)vr;
    for (int j = 0; j < 32 && t0 + j < total; ++j) {
      const float pj = __shfl_sync(0xffffffffu, p, j);
      const bf16 *vj = (const bf16 *)__shfl_sync(0xffffffffu, vaddr, j);
      if (vj == nullptr) continue;                 // a skipped key (page outside the pool): weight 0, nothing to read; same for every lane
#pragma unroll
      for (int i = 0; i < DPL; ++i) acc[i] = fmaf(pj, __bfloat162float(vj[lane * DPL + i]), acc[i]);
    }
  }
  bf16 *o = O + ((size_t)r * Hq + h) * HD;
#pragma unroll
  for (int i = 0; i < DPL; ++i) o[lane * DPL + i] = __float2bfloat16(den > 0.f ? acc[i] / den : 0.f);   // no visible key: zeros
}
