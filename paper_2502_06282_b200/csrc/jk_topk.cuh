// Block-level partial top-k over one chunk of JK_TOPK_CHUNK vocabulary entries of one logits row:
// chunk maximum, sum of exp(x - max) and the k_e best (value descending, token id ascending).
// Shared by the CUDA-core path (logits read from global memory) and the tensor-core path (logits
// assembled from the GEMM's partial tiles).
//
// 1024 threads, 4 entries each.  Every warp first picks the k_e best of its own 128 entries with
// shuffles only; warp 0 then merges the 32 * k_e warp winners.  Two block barriers in total.
#pragma once

#include <limits.h>
#include <math.h>

#include "jk_common.cuh"

#define JK_TOPK_THREADS 512
#define JK_TOPK_WARPS (JK_TOPK_THREADS / 32)
#define JK_TOPK_PER (JK_TOPK_CHUNK / JK_TOPK_THREADS)

// Order-preserving map of a float (finite or -inf) to an unsigned key, and back.  -0 is folded
// into +0 first, as the comparison of the values themselves does.
__device__ __forceinline__ unsigned jk_fkey(float v) {
  const unsigned u = __float_as_uint(v + 0.f);
  return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}
__device__ __forceinline__ float jk_fkey_inv(unsigned k) {
  return __uint_as_float((k & 0x80000000u) ? (k ^ 0x80000000u) : ~k);
}
// The warp's best (value descending, index ascending) with two hardware reductions instead of a
// shuffle tree: the largest key, then the smallest index among the lanes that hold it.
__device__ __forceinline__ void jk_warp_argbest(float& v, int& i) {
  const unsigned key = jk_fkey(v);
  const unsigned kmax = __reduce_max_sync(0xffffffffu, key);
  const unsigned imin = __reduce_min_sync(0xffffffffu, key == kmax ? (unsigned)i : 0xffffffffu);
  v = jk_fkey_inv(kmax);
  i = (int)imin;
}

#define JK_TOPK_CAND 128               // candidates the short selection can hold

// JK_TOPK_THREADS threads; thread t holds entries base + t + j*JK_TOPK_THREADS in vals[j]
// (-inf past the vocabulary).
//
// Short selection: the chunk's k_e best all reach the k_e-th largest of the 16 warp maxima (the
// k_e largest warp maxima are k_e different entries), and few other entries do.  So the block
// finds that threshold, collects the entries that reach it, and one warp picks the k_e best of
// those few.  If more than JK_TOPK_CAND entries reach the threshold (many equal values) the
// full selection below does the work instead; both give the same result.
__device__ __forceinline__ void jk_topk_chunk_select_full(const float (&vals)[JK_TOPK_PER], int base,
                                                          int V, int k_e, size_t prow,
                                                          float* __restrict__ tk_val,
                                                          int32_t* __restrict__ tk_idx,
                                                          float* __restrict__ tk_ms);

__device__ __forceinline__ void jk_topk_chunk_select(const float (&vals)[JK_TOPK_PER], int base,
                                                     int V, int k_e, size_t prow,
                                                     float* __restrict__ tk_val,
                                                     int32_t* __restrict__ tk_idx,
                                                     float* __restrict__ tk_ms) {
  constexpr int NW = JK_TOPK_WARPS;
  __shared__ unsigned q_wkey[NW];
  __shared__ float q_wsum[NW];
  __shared__ unsigned q_thr;
  __shared__ int q_cnt;
  __shared__ float q_cv[JK_TOPK_CAND];
  __shared__ int q_ci[JK_TOPK_CAND];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  float lmax = -INFINITY;
#pragma unroll
  for (int j = 0; j < JK_TOPK_PER; ++j) lmax = fmaxf(lmax, vals[j]);      // (-inf past V)
  const unsigned wkey = __reduce_max_sync(0xffffffffu, jk_fkey(lmax));
  if (lane == 0) q_wkey[warp] = wkey;
  if (threadIdx.x == 0) q_cnt = 0;
  __syncthreads();
  // warp 0: the k_e-th largest warp maximum; everybody: the chunk maximum
  if (warp == 0) {
    unsigned k = lane < NW ? q_wkey[lane] : 0u;
    unsigned thr = 0u;
    for (int it = 0; it < k_e && it < NW; ++it) {
      thr = __reduce_max_sync(0xffffffffu, k);
      const unsigned who = __ballot_sync(0xffffffffu, k == thr);
      if (lane == __ffs(who) - 1) k = 0u;                                  // one holder leaves
    }
    if (lane == 0) q_thr = thr;
  }
  unsigned bkey = q_wkey[0];
#pragma unroll
  for (int w = 1; w < NW; ++w) bkey = max(bkey, q_wkey[w]);
  const float bmax = jk_fkey_inv(bkey);
  float s = 0.f;
#pragma unroll
  for (int j = 0; j < JK_TOPK_PER; ++j) {
    const int idx = base + threadIdx.x + j * JK_TOPK_THREADS;
    if (idx < V) s += expf(vals[j] - bmax);
  }
  s = jk_warp_sum(s);
  if (lane == 0) q_wsum[warp] = s;
  __syncthreads();
  const unsigned thr = q_thr;
#pragma unroll
  for (int j = 0; j < JK_TOPK_PER; ++j) {
    const int idx = base + threadIdx.x + j * JK_TOPK_THREADS;
    if (idx < V && jk_fkey(vals[j]) >= thr) {
      const int pos = atomicAdd(&q_cnt, 1);
      if (pos < JK_TOPK_CAND) { q_cv[pos] = vals[j]; q_ci[pos] = idx; }
    }
  }
  __syncthreads();
  const int cnt = q_cnt;
  if (cnt > JK_TOPK_CAND) {                     // (the same decision in every thread)
    jk_topk_chunk_select_full(vals, base, V, k_e, prow, tk_val, tk_idx, tk_ms);
    return;
  }
  if (warp != 0) return;
  if (lane == 0) {
    float bsum = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) bsum += q_wsum[w];
    tk_ms[prow * 2] = bmax;
    tk_ms[prow * 2 + 1] = bsum;
  }
  constexpr int PC = JK_TOPK_CAND / 32;
  float cv[PC];
  int ci[PC];
#pragma unroll
  for (int j = 0; j < PC; ++j) {
    const int c = lane + j * 32;
    cv[j] = c < cnt ? q_cv[c] : -INFINITY;
    ci[j] = c < cnt ? q_ci[c] : INT_MAX;
  }
  unsigned taken = 0;
  for (int it = 0; it < k_e; ++it) {
    float bv = -INFINITY;
    int bi = INT_MAX, bj = -1;
#pragma unroll
    for (int j = 0; j < PC; ++j)
      if (!(taken & (1u << j)) && ci[j] != INT_MAX && jk_better(cv[j], ci[j], bv, bi)) {
        bv = cv[j]; bi = ci[j]; bj = j;
      }
    float wv = bv;
    int wi = bi;
    jk_warp_argbest(wv, wi);
    if (wi == bi && bj >= 0) taken |= 1u << bj;
    if (lane == 0) { tk_val[prow * k_e + it] = wv; tk_idx[prow * k_e + it] = wi; }
  }
}

// The full selection: every warp picks the k_e best of its own entries, warp 0 merges them.
__device__ __forceinline__ void jk_topk_chunk_select_full(const float (&vals)[JK_TOPK_PER], int base,
                                                          int V, int k_e, size_t prow,
                                                          float* __restrict__ tk_val,
                                                          int32_t* __restrict__ tk_idx,
                                                          float* __restrict__ tk_ms) {
  constexpr int NW = JK_TOPK_WARPS;
  constexpr int MC = NW * JK_MAX_KE / 32;          // merge candidates per lane
  __shared__ float s_wmax[NW], s_wsum[NW];
  __shared__ float s_cv[NW * JK_MAX_KE];
  __shared__ int s_ci[NW * JK_MAX_KE];
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  // warp maximum and the warp's own k_e best
  float lmax = -INFINITY;
#pragma unroll
  for (int j = 0; j < JK_TOPK_PER; ++j) lmax = fmaxf(lmax, vals[j]);
  lmax = jk_warp_max(lmax);
  unsigned taken = 0;
  for (int it = 0; it < k_e; ++it) {
    float bv = -INFINITY;
    int bi = INT_MAX, bj = -1;
#pragma unroll
    for (int j = 0; j < JK_TOPK_PER; ++j) {
      const int idx = base + threadIdx.x + j * JK_TOPK_THREADS;
      if (!(taken & (1u << j)) && idx < V && jk_better(vals[j], idx, bv, bi)) {
        bv = vals[j]; bi = idx; bj = j;
      }
    }
    float wv = bv;
    int wi = bi;
    jk_warp_argbest(wv, wi);
    if (wi == bi && bj >= 0) taken |= 1u << bj;       // token ids are unique: one lane matches
    if (lane == 0) { s_cv[warp * JK_MAX_KE + it] = wv; s_ci[warp * JK_MAX_KE + it] = wi; }
  }
  if (lane == 0) s_wmax[warp] = lmax;
  __syncthreads();
  float bmax = s_wmax[0];
#pragma unroll
  for (int w = 1; w < NW; ++w) bmax = fmaxf(bmax, s_wmax[w]);
  float s = 0.f;
#pragma unroll
  for (int j = 0; j < JK_TOPK_PER; ++j) {
    const int idx = base + threadIdx.x + j * JK_TOPK_THREADS;
    if (idx < V) s += expf(vals[j] - bmax);
  }
  s = jk_warp_sum(s);
  if (lane == 0) s_wsum[warp] = s;
  __syncthreads();
  if (warp != 0) return;
  if (lane == 0) {
    float bsum = 0.f;
#pragma unroll
    for (int w = 0; w < NW; ++w) bsum += s_wsum[w];
    tk_ms[prow * 2] = bmax;
    tk_ms[prow * 2 + 1] = bsum;
  }
  // merge: lane holds warp winners lane, lane + 32, ... (NW * k_e of them)
  float cv[MC];
  int ci[MC];
#pragma unroll
  for (int j = 0; j < MC; ++j) {
    const int c = lane + j * 32;                      // candidate (warp = c / k_e, rank = c % k_e)
    const bool in = c < NW * k_e;
    cv[j] = in ? s_cv[(c / k_e) * JK_MAX_KE + c % k_e] : -INFINITY;
    ci[j] = in ? s_ci[(c / k_e) * JK_MAX_KE + c % k_e] : INT_MAX;
  }
  unsigned mtaken = 0;
  for (int it = 0; it < k_e; ++it) {
    float bv = -INFINITY;
    int bi = INT_MAX, bj = -1;
#pragma unroll
    for (int j = 0; j < MC; ++j)
      if (!(mtaken & (1u << j)) && ci[j] != INT_MAX && jk_better(cv[j], ci[j], bv, bi)) {
        bv = cv[j]; bi = ci[j]; bj = j;
      }
    float wv = bv;
    int wi = bi;
    jk_warp_argbest(wv, wi);
    if (wi == bi && bj >= 0) mtaken |= 1u << bj;
    if (lane == 0) { tk_val[prow * k_e + it] = wv; tk_idx[prow * k_e + it] = wi; }
  }
}
