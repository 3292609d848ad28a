// Shared declarations of the Jakiro CUDA library: context, workspace layout, small device helpers.
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>
#include <stdio.h>
#include <string.h>

#include "jakiro.h"

#define JK_MAX_EXPERTS 8
#define JK_MAX_KE 16
#define JK_MAX_TREE 128
#define JK_MAX_ROWS 128          // max_batch * max_frontier
#define JK_MAX_POOL 4096
#define JK_TOPK_CHUNK 4096       // vocabulary entries per partial top-k block
#define JK_ATTN_QB 64            // query rows per attention CTA
#define JK_ATTN_MAX_SPLIT 32

struct jk_ws_layout {
  size_t status;        // int32[4]: the only part of the workspace that has to start at zero
  size_t xn;            // T   [Rp, H]       normalised hidden states
  size_t probs;         // f32 [R, N]
  size_t expert;        // i32 [R, K]
  size_t gate;          // f32 [R, K]
  size_t hbuf;          // T   [N, Rp, I]    SiLU(gate)*up per (expert, row)
  size_t ybuf;          // f32 [N, Rp, H]    expert outputs
  size_t bbuf;          // T   [RKp, H]      branch features (LM-head input)
  size_t logits;        // f32 [R*K, V]      when the caller does not ask for the logits
  size_t tk_val;        // f32 [R*K, chunks, k_e]
  size_t tk_idx;        // i32 [R*K, chunks, k_e]
  size_t tk_ms;         // f32 [R*K, chunks, 2]
  size_t gemm_part;     // f32 partial tiles of the tensor-core GEMMs
  size_t attn_o;        // f32 [split, B*M*Hq, d]
  size_t attn_ml;       // f32 [split, B*M*Hq, 2]
  size_t rs_arg;        // i32 [B, M]        per tree node: top-1 token of the target row
  size_t rs_max;        // f32 [B, M]
  size_t rs_sum;        // f32 [B, M]
  size_t pbuf;          // f32 [B, 2, V]
  size_t qbuf;          // f32 [B, K, 2, V]
  size_t p_old;         // i32 [B]
  size_t qs_arg;        // i32 [B, S, K]     top-1 of every stored draft row (written, not read)
  size_t qs_max;        // f32 [B, S, K]     max of every stored draft logits row
  size_t qs_sum;        // f32 [B, S, K]     its sum of exp((x - max)/T)
  // draft pre-MoE block (Eq. 1); S = max_depth * max_frontier slots per sequence
  size_t pre_x;         // T   [Rp, 2H]      [emb(tok) ; parent feature]
  size_t pre_h;         // T   [Rp, H]       reduction layer output h
  size_t pre_qkv;       // f32 [Rp, (Hq + 2 Hkv) d]
  size_t pre_qd;        // T   [B * S, Hq d] rotated queries of the nodes expanded so far, dense
  size_t pre_par;       // i32 [B * S]       their parent slots, dense
  size_t pre_att;       // T   [B * S, Hq d] attention outputs of those nodes
  size_t pre_ao;        // T   [Rp, Hq d]    attention outputs of this pass's nodes (O-proj input)
  size_t total;
  int attn_max_split;
  size_t gemm_cnt;       // four item counters of the streaming GEMM (zero between launches)
  int topk_chunks;
  int rows_pad;         // Rp
  int rk_pad;           // RKp
  size_t gemm_part_bytes;
};

// Optional per-kernel timing: a pair of CUDA events around every launch, summed per stage.
enum jk_stage {
  JK_ST_ROUTER = 0, JK_ST_GATEUP, JK_ST_DOWN, JK_ST_BRANCH, JK_ST_LMHEAD, JK_ST_TOPK,
  JK_ST_FINISH, JK_ST_FINALIZE, JK_ST_ATTN, JK_ST_ATTN_COMBINE, JK_ST_ROWSTATS, JK_ST_WALK,
  JK_ST_COMPACT, JK_ST_GEMM_FIXUP, JK_ST_PRE_GATHER, JK_ST_PRE_GEMM, JK_ST_PRE_FIXUP,
  JK_ST_PRE_ROPE, JK_ST_PRE_ATTN, JK_ST_PRE_ATTN_COMBINE, JK_N_STAGES
};
struct jk_prof {
  cudaEvent_t* ev;        // 2 * cap events
  int* stage;             // stage of each recorded pair
  int cap, n, open;
  cudaStream_t stream;
};

struct jk_ctx {
  jk_config cfg;
  jk_ws_layout lay;
  char* ws;               // device workspace base (caller-owned)
  size_t ws_bytes;
  int tensor_path;
  int sm_count;           // filled at the first launch
  int attn_smem_set;
  int attn_sk_smem_set;
  unsigned gemm_seq;     // GEMM launches so far: picks the item counter
  int st_attn, st_combine;  // profiling stages the attention kernels are booked under
  int attn_kernel;        // 0 = by size, 1 = CTA per (query block, key slice), 2 = persistent,
                          // 3 = cluster-merged
  char cuda_err[256];
  void* tc_state;         // tensor-core path bookkeeping (tensor maps), host memory
  void* attn_tc_state;    // tensor maps of the KV caches seen by the attention kernel
  void* attn_cl_state;    // cluster-merged attention kernel: occupancy answers per cluster size
  jk_prof prof;
};

void jk_prof_begin(jk_ctx* ctx, cudaStream_t st, int stage);
void jk_prof_end(jk_ctx* ctx);
#define JK_PROF(ctx, st, stage)                                  \
  do {                                                           \
    if ((ctx)->prof.cap) jk_prof_begin(ctx, st, stage);          \
  } while (0)

static inline size_t jk_align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }
static inline int jk_elem_size(int dtype) { return dtype == JK_BF16 ? 2 : 4; }

#define JK_CUDA_CHECK(ctx, expr)                                                     \
  do {                                                                               \
    cudaError_t e_ = (expr);                                                         \
    if (e_ != cudaSuccess) {                                                         \
      snprintf((ctx)->cuda_err, sizeof((ctx)->cuda_err), "%s: %s", #expr,            \
               cudaGetErrorString(e_));                                              \
      return JK_ERR_CUDA;                                                            \
    }                                                                                \
  } while (0)

#define JK_LAUNCH_CHECK(ctx)                                                         \
  do {                                                                               \
    if ((ctx)->prof.open) jk_prof_end(ctx);                                          \
    cudaError_t e_ = cudaGetLastError();                                             \
    if (e_ != cudaSuccess) {                                                         \
      snprintf((ctx)->cuda_err, sizeof((ctx)->cuda_err), "launch at %s:%d: %s",      \
               __FILE__, __LINE__, cudaGetErrorString(e_));                          \
      return JK_ERR_CUDA;                                                            \
    }                                                                                \
  } while (0)

static inline bool jk_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

int jk_ensure_device_info(jk_ctx* ctx);

#ifdef __CUDACC__
// ---------------------------------------------------------------- programmatic dependent launch
// The kernels of one call form a chain on one stream.  Launched with the programmatic-
// serialization attribute, a kernel may start while its predecessor is still running; it must
// call jk_pdl_wait() before it reads or writes global memory that an earlier kernel of the
// stream touches, and it calls jk_pdl_trigger() only after that wait, so that at most two
// consecutive kernels overlap and everything older is complete when a kernel starts.  (One
// kernel, the SiLU fix-up between the gate/up and the down GEMM, releases its successor before
// its wait; the reasons why that is sound there are given at that call.)
__device__ __forceinline__ void jk_pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }
__device__ __forceinline__ void jk_pdl_trigger() {
  asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
}

template <typename... KArgs, typename... Args>
static inline cudaError_t jk_launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block,
                                        size_t smem, cudaStream_t st, Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// The same launch with the grid grouped into thread-block clusters of `cluster_x` blocks.
template <typename... KArgs, typename... Args>
static inline cudaError_t jk_launch_pdl_cluster(void (*kernel)(KArgs...), dim3 grid, dim3 block,
                                                unsigned cluster_x, size_t smem, cudaStream_t st,
                                                Args&&... args) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = block;
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = cluster_x;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, kernel, static_cast<KArgs>(args)...);
}

// ---------------------------------------------------------------- device helpers
__device__ __forceinline__ float jk_warp_sum(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
  return v;
}
__device__ __forceinline__ float jk_warp_max(float v) {
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) v = fmaxf(v, __shfl_xor_sync(0xffffffffu, v, o));
  return v;
}

// Block-wide sum; every thread gets the result.  `red` is shared scratch of >= 33 floats.
__device__ __forceinline__ float jk_block_sum(float v, float* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = jk_warp_sum(v);
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  if (warp == 0) {
    float t = lane < nw ? red[lane] : 0.f;
    t = jk_warp_sum(t);
    if (lane == 0) red[32] = t;
  }
  __syncthreads();
  return red[32];
}
__device__ __forceinline__ float jk_block_max(float v, float* red) {
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = (blockDim.x + 31) >> 5;
  v = jk_warp_max(v);
  __syncthreads();
  if (lane == 0) red[warp] = v;
  __syncthreads();
  if (warp == 0) {
    float t = lane < nw ? red[lane] : -INFINITY;
    t = jk_warp_max(t);
    if (lane == 0) red[32] = t;
  }
  __syncthreads();
  return red[32];
}

// "a beats b" for (value descending, index ascending) orderings
__device__ __forceinline__ bool jk_better(float va, int ia, float vb, int ib) {
  return va > vb || (va == vb && ia < ib);
}

template <typename T> struct jk_vec;   // 16-byte vector of T
template <> struct jk_vec<float> {
  static constexpr int N = 4;
  __device__ static __forceinline__ void load(const float* p, float (&o)[4]) {
    float4 v = *reinterpret_cast<const float4*>(p);
    o[0] = v.x; o[1] = v.y; o[2] = v.z; o[3] = v.w;
  }
};
template <> struct jk_vec<__nv_bfloat16> {
  static constexpr int N = 8;
  __device__ static __forceinline__ void load(const __nv_bfloat16* p, float (&o)[8]) {
    uint4 v = *reinterpret_cast<const uint4*>(p);
    const uint32_t w[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
      o[2 * i] = __uint_as_float(w[i] << 16);
      o[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
  }
};

__device__ __forceinline__ float jk_to_float(float v) { return v; }
__device__ __forceinline__ float jk_to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T jk_from_float(float v);
template <> __device__ __forceinline__ float jk_from_float<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 jk_from_float<__nv_bfloat16>(float v) {
  return __float2bfloat16_rn(v);
}

__device__ __forceinline__ void jk_set_status(int32_t* status, int code) {
  atomicCAS(status, 0, code);
}
#endif  // __CUDACC__
