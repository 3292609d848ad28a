// Block-level partial top-k over one chunk of JK_TOPK_CHUNK vocabulary entries of one logits row:
// chunk maximum, sum of exp(x - max) and the k_e best (value descending, token id ascending).
// Shared by the CUDA-core path (logits read from global memory) and the tensor-core path (logits
// assembled from the GEMM's partial tiles).
#pragma once

#include <limits.h>
#include <math.h>

#include "jk_common.cuh"

#define JK_TOPK_PER (JK_TOPK_CHUNK / 256)

// 256 threads; thread t holds entries base + t + j*256 in vals[j] (-inf past the vocabulary).
__device__ __forceinline__ void jk_topk_chunk_select(const float (&vals)[JK_TOPK_PER], int base,
                                                     int V, int k_e, size_t prow,
                                                     float* __restrict__ tk_val,
                                                     int32_t* __restrict__ tk_idx,
                                                     float* __restrict__ tk_ms) {
  __shared__ float red[33];
  __shared__ float wv[8];
  __shared__ int wi[8];
  __shared__ int win_idx;
  float lmax = -INFINITY;
#pragma unroll
  for (int j = 0; j < JK_TOPK_PER; ++j) lmax = fmaxf(lmax, vals[j]);
  const float bmax = jk_block_max(lmax, red);
  float s = 0.f;
#pragma unroll
  for (int j = 0; j < JK_TOPK_PER; ++j) {
    const int idx = base + threadIdx.x + j * 256;
    if (idx < V) s += expf(vals[j] - bmax);
  }
  const float bsum = jk_block_sum(s, red);
  if (threadIdx.x == 0) { tk_ms[prow * 2] = bmax; tk_ms[prow * 2 + 1] = bsum; }
  unsigned taken = 0;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  for (int it = 0; it < k_e; ++it) {
    float bv = -INFINITY;
    int bi = INT_MAX;
#pragma unroll
    for (int j = 0; j < JK_TOPK_PER; ++j) {
      const int idx = base + threadIdx.x + j * 256;
      if (!(taken & (1u << j)) && idx < V && jk_better(vals[j], idx, bv, bi)) { bv = vals[j]; bi = idx; }
    }
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) {
      const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
      const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
      if (jk_better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
    }
    if (lane == 0) { wv[warp] = bv; wi[warp] = bi; }
    __syncthreads();
    if (threadIdx.x == 0) {
      float fv = wv[0];
      int fi = wi[0];
      for (int w = 1; w < 8; ++w)
        if (jk_better(wv[w], wi[w], fv, fi)) { fv = wv[w]; fi = wi[w]; }
      tk_val[prow * k_e + it] = fv;
      tk_idx[prow * k_e + it] = fi;
      win_idx = fi;
    }
    __syncthreads();
    const int wsel = win_idx;
    if (wsel != INT_MAX) {
#pragma unroll
      for (int j = 0; j < JK_TOPK_PER; ++j)
        if (base + threadIdx.x + j * 256 == wsel) taken |= 1u << j;
    }
    __syncthreads();
  }
}
