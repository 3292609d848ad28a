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

// JK_TOPK_THREADS threads; thread t holds entries base + t + j*JK_TOPK_THREADS in vals[j]
// (-inf past the vocabulary).
__device__ __forceinline__ void jk_topk_chunk_select(const float (&vals)[JK_TOPK_PER], int base,
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
