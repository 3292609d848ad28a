// jk_tree_verify_attn: tree-masked attention of one target layer over the draft tree's tokens
// (arXiv 2502.06282, Sec. 2.1 step 2; mask of Fig. 4).  Split-KV: every CTA handles one
// (sequence, kv head, block of 64 query rows, slice of the key range) and writes an
// unnormalised partial (running max, sum, output); a second kernel merges the slices.
#include <math.h>

#include "jk_common.cuh"

template <int D>
struct attn_smem {
  float q[JK_ATTN_QB][D];          // pre-scaled queries
  float o[JK_ATTN_QB][D];          // running outputs
  float k[32][D + 4];              // one tile of 32 keys (padded rows: conflict-free float4 reads)
  float v[32][D];
  float m[JK_ATTN_QB];
  float l[JK_ATTN_QB];
  unsigned long long anc[JK_MAX_TREE][2];
};

// Rows of a CTA are (g, i) pairs: q-head kvh*G + g, tree node i; row index = g*M + i.
template <typename T, int D>
__global__ void __launch_bounds__(256) k_tree_attn(
    const T* __restrict__ q, const T* __restrict__ kc, const T* __restrict__ vc,
    long long stride_b, long long stride_h, int cache_rows, const int32_t* __restrict__ kv_len,
    const int32_t* __restrict__ parent, float scale, int M, int Hq, int Hkv, int n_split,
    int n_qblk, float* __restrict__ part_o, float* __restrict__ part_ml, int32_t* status) {
  extern __shared__ __align__(16) unsigned char smem_raw[];
  attn_smem<D>& S = *reinterpret_cast<attn_smem<D>*>(smem_raw);
  constexpr int VN = jk_vec<T>::N;
  constexpr int DPL = D / 32;                 // output columns per lane
  const int split = blockIdx.x % n_split, qblk = blockIdx.x / n_split;
  const int kvh = blockIdx.y, b = blockIdx.z;
  const int G = Hq / Hkv;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  const int P = kv_len[b];
  const int Ltot = P + M;
  if (P < 0 || Ltot > cache_rows) {
    if (threadIdx.x == 0) jk_set_status(status, JK_ERR_BOUNDS);
    return;
  }
  const int n_rows = G * M;
  const int row0 = qblk * JK_ATTN_QB;
  const int rows_here = min(JK_ATTN_QB, n_rows - row0);
  // ancestor bitsets from parent[] (Fig. 4)
  if (threadIdx.x < M) {
    unsigned long long lo = 0ull, hi = 0ull;
    int c = threadIdx.x;
    for (int guard = 0; c >= 0 && guard <= JK_MAX_TREE; ++guard) {
      if (c < 64) lo |= 1ull << c; else hi |= 1ull << (c - 64);
      const int p = parent[(size_t)b * M + c];
      c = (p < c) ? p : -1;
    }
    S.anc[threadIdx.x][0] = lo;
    S.anc[threadIdx.x][1] = hi;
  }
  // queries (scaled) and state
  for (int idx = threadIdx.x; idx < JK_ATTN_QB * (D / VN); idx += blockDim.x) {
    const int r = idx / (D / VN), c = (idx % (D / VN)) * VN;
    float v[VN];
    if (r < rows_here) {
      const int g = (row0 + r) / M, i = (row0 + r) % M;
      jk_vec<T>::load(q + (((size_t)b * M + i) * Hq + kvh * G + g) * D + c, v);
    } else {
#pragma unroll
      for (int t = 0; t < VN; ++t) v[t] = 0.f;
    }
#pragma unroll
    for (int t = 0; t < VN; ++t) { S.q[r][c + t] = v[t] * scale; S.o[r][c + t] = 0.f; }
  }
  if (threadIdx.x < JK_ATTN_QB) { S.m[threadIdx.x] = -INFINITY; S.l[threadIdx.x] = 0.f; }
  // key range of this split, in tiles of 32
  const int n_tiles = (Ltot + 31) / 32;
  const int tiles_per = (n_tiles + n_split - 1) / n_split;
  const int t0 = split * tiles_per, t1 = min(n_tiles, t0 + tiles_per);
  const T* kbase = kc + (size_t)b * stride_b + (size_t)kvh * stride_h;
  const T* vbase = vc + (size_t)b * stride_b + (size_t)kvh * stride_h;
  for (int tile = t0; tile < t1; ++tile) {
    __syncthreads();
    const int key0 = tile * 32;
    for (int idx = threadIdx.x; idx < 32 * (D / VN); idx += blockDim.x) {
      const int j = idx / (D / VN), c = (idx % (D / VN)) * VN;
      float kv[VN], vv[VN];
      if (key0 + j < Ltot) {
        jk_vec<T>::load(kbase + (size_t)(key0 + j) * D + c, kv);
        jk_vec<T>::load(vbase + (size_t)(key0 + j) * D + c, vv);
      } else {
#pragma unroll
        for (int t = 0; t < VN; ++t) { kv[t] = 0.f; vv[t] = 0.f; }
      }
#pragma unroll
      for (int t = 0; t < VN; ++t) { S.k[j][c + t] = kv[t]; S.v[j][c + t] = vv[t]; }
    }
    __syncthreads();
    const int key = key0 + lane;
    for (int r = warp; r < rows_here; r += 8) {
      const int i = (row0 + r) % M;
      bool vis = key < P;
      if (!vis && key < Ltot) {
        const int t = key - P;
        vis = (S.anc[i][t >> 6] >> (t & 63)) & 1ull;
      }
      float s = 0.f;
#pragma unroll 8
      for (int c = 0; c < D; c += 4) {
        const float4 qv = *reinterpret_cast<const float4*>(&S.q[r][c]);
        const float4 kv = *reinterpret_cast<const float4*>(&S.k[lane][c]);
        s = fmaf(qv.x, kv.x, s); s = fmaf(qv.y, kv.y, s);
        s = fmaf(qv.z, kv.z, s); s = fmaf(qv.w, kv.w, s);
      }
      s = vis ? s : -INFINITY;
      const float m_old = S.m[r];
      const float m_new = fmaxf(m_old, jk_warp_max(s));
      if (m_new == -INFINITY) continue;           // nothing visible yet (warp-uniform)
      const float p = vis ? __expf(s - m_new) : 0.f;
      const float corr = __expf(m_old - m_new);   // 0 when m_old = -inf
      const float psum = jk_warp_sum(p);
      float acc[DPL];
#pragma unroll
      for (int t = 0; t < DPL; ++t) acc[t] = S.o[r][lane * DPL + t] * corr;
#pragma unroll 8
      for (int j = 0; j < 32; ++j) {
        const float pj = __shfl_sync(0xffffffffu, p, j);
#pragma unroll
        for (int t = 0; t < DPL; ++t) acc[t] = fmaf(pj, S.v[j][lane * DPL + t], acc[t]);
      }
#pragma unroll
      for (int t = 0; t < DPL; ++t) S.o[r][lane * DPL + t] = acc[t];
      if (lane == 0) { S.m[r] = m_new; S.l[r] = S.l[r] * corr + psum; }
      __syncwarp();
    }
  }
  __syncthreads();
  // partial results: row index in the [B, M, Hq] order of the output
  for (int idx = threadIdx.x; idx < rows_here * D; idx += blockDim.x) {
    const int r = idx / D, c = idx % D;
    const int g = (row0 + r) / M, i = (row0 + r) % M;
    const size_t orow = ((size_t)b * M + i) * Hq + kvh * G + g;
    const size_t n_out = (size_t)gridDim.z * M * Hq;
    part_o[((size_t)split * n_out + orow) * D + c] = S.o[r][c];
    if (c == 0) {
      part_ml[((size_t)split * n_out + orow) * 2] = S.m[r];
      part_ml[((size_t)split * n_out + orow) * 2 + 1] = S.l[r];
    }
  }
}

// Merge the key-range slices: out = sum_s e^{m_s - m} o_s / sum_s e^{m_s - m} l_s.  One warp per row.
// NB slices are loaded per round: 8, 10 or 12 by the number of slices (9 at the 7B shape: a second
// round is a second trip to L2 on a call that is a chain of such trips).  Up to 10 per round the
// kernel stays within 64 registers, so that two of its blocks leave room on an SM for a CTA of
// the next call's attention kernel, which starts its prologue and its prefix copies there while
// the merge runs; 20 per round costs the occupancy that keeps the blocks in one wave.
template <typename T, int D, int NB>
__global__ void __launch_bounds__(256) k_attn_combine(
    const float* __restrict__ part_o, const float* __restrict__ part_ml, int n_split,
    size_t n_out, T* __restrict__ out) {
  jk_pdl_wait();
  jk_pdl_trigger();
  constexpr int DPL = D / 32;
  const int lane = threadIdx.x & 31;
  const size_t row = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= n_out) return;
  const float* po = part_o + row * D + lane * DPL;      // slice s is s * n_out * D further
  const size_t sstride = n_out * D;
  auto load_batch = [&](int s0, float (&v)[NB][DPL]) {  // NB independent vector loads in flight
#pragma unroll
    for (int j = 0; j < NB; ++j) {
      if (s0 + j >= n_split) continue;                  // (never read below)
      const int s = s0 + j;
      if (DPL == 4) {
        const float4 x = *reinterpret_cast<const float4*>(po + (size_t)s * sstride);
        v[j][0] = x.x; v[j][1] = x.y; v[j][DPL - 2] = x.z; v[j][DPL - 1] = x.w;
      } else {
        const float2 x = *reinterpret_cast<const float2*>(po + (size_t)s * sstride);
        v[j][0] = x.x; v[j][DPL - 1] = x.y;
      }
    }
  };
  // the first batch of partial outputs is asked for before anything waits on the (max, sum) pairs
  float v[NB][DPL];
  load_batch(0, v);
  // lane s holds (max, sum) of slice s (n_split <= 32); one load round for all slices
  float ms = -INFINITY, ls = 0.f;
  if (lane < n_split) {
    const float2 x = *reinterpret_cast<const float2*>(part_ml + ((size_t)lane * n_out + row) * 2);
    ms = x.x;
    ls = x.y;
  }
  const float m = jk_warp_max(ms);
  const float w_lane = (ms == -INFINITY) ? 0.f : __expf(ms - m);
  const float l = jk_warp_sum(w_lane * ls);
  float acc[DPL];
#pragma unroll
  for (int t = 0; t < DPL; ++t) acc[t] = 0.f;
  for (int s0 = 0; s0 < n_split; s0 += NB) {
    if (s0 > 0) load_batch(s0, v);
#pragma unroll
    for (int j = 0; j < NB; ++j) {
      const float w = __shfl_sync(0xffffffffu, w_lane, (s0 + j) & 31);
      if (s0 + j < n_split && w != 0.f) {
#pragma unroll
        for (int t = 0; t < DPL; ++t) acc[t] += w * v[j][t];
      }
    }
  }
  const float inv = 1.f / l;
#pragma unroll
  for (int t = 0; t < DPL; ++t) out[row * D + lane * DPL + t] = jk_from_float<T>(acc[t] * inv);
}

template <typename T, int D>
static int attn_impl(jk_ctx* ctx, cudaStream_t st, int B, int M, const void* q, const void* kc,
                     const void* vc, int64_t sb, int64_t sh, int cache_rows,
                     const int32_t* kv_len, const int32_t* parent, float scale, void* out) {
  const jk_config& c = ctx->cfg;
  const jk_ws_layout& L = ctx->lay;
  const int G = c.n_q_heads / c.n_kv_heads;
  const int n_qblk = (G * M + JK_ATTN_QB - 1) / JK_ATTN_QB;
  const int base_ctas = n_qblk * c.n_kv_heads * B;
  // enough slices to cover the SMs twice, each at least 2 tiles (64 keys) long
  int n_split = (2 * ctx->sm_count + base_ctas - 1) / base_ctas;
  const int max_by_len = (cache_rows / 64) > 0 ? (cache_rows / 64) : 1;
  if (n_split > max_by_len) n_split = max_by_len;
  if (n_split > L.attn_max_split) n_split = L.attn_max_split;
  if (n_split < 1) n_split = 1;
  const size_t smem = sizeof(attn_smem<D>);
  auto kern = k_tree_attn<T, D>;
  if (!ctx->attn_smem_set) {
    JK_CUDA_CHECK(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)smem));
    ctx->attn_smem_set = 1;
  }
  float* part_o = (float*)(ctx->ws + L.attn_o);
  float* part_ml = (float*)(ctx->ws + L.attn_ml);
  JK_PROF(ctx, st, ctx->st_attn);
  kern<<<dim3(n_split * n_qblk, c.n_kv_heads, B), 256, smem, st>>>(
      (const T*)q, (const T*)kc, (const T*)vc, sb, sh, cache_rows, kv_len, parent, scale, M,
      c.n_q_heads, c.n_kv_heads, n_split, n_qblk, part_o, part_ml,
      (int32_t*)(ctx->ws + L.status));
  JK_LAUNCH_CHECK(ctx);
  const size_t n_out = (size_t)B * M * c.n_q_heads;
  JK_PROF(ctx, st, ctx->st_combine);
  k_attn_combine<T, D, 8><<<(unsigned)((n_out + 7) / 8), 256, 0, st>>>(part_o, part_ml, n_split,
                                                                    n_out, (T*)out);
  JK_LAUNCH_CHECK(ctx);
  return JK_OK;
}

// tensor-core kernel (jk_attn_tc.cu)
int jk_attn_tc(jk_ctx* ctx, cudaStream_t st, int B, int M, const void* q, const void* kc,
               const void* vc, int64_t sb, int64_t sh, int cache_rows, const int32_t* kv_len,
               const int32_t* parent, float scale, void* out);
int jk_tc_available(const jk_ctx* ctx);

// Merge launch shared with the tensor-core kernel (bf16 output).
int jk_attn_combine_launch(jk_ctx* ctx, cudaStream_t st, int n_split, size_t n_out, void* out) {
  const jk_ws_layout& L = ctx->lay;
  const float* part_o = (const float*)(ctx->ws + L.attn_o);
  const float* part_ml = (const float*)(ctx->ws + L.attn_ml);
  JK_PROF(ctx, st, ctx->st_combine);
  const dim3 grid((unsigned)((n_out + 7) / 8));
#define JK_COMBINE(DD, NBB)                                                                    \
  jk_launch_pdl(k_attn_combine<__nv_bfloat16, DD, NBB>, grid, dim3(256), 0, st, part_o, part_ml, \
                n_split, n_out, (__nv_bfloat16*)out)
  if (ctx->cfg.head_dim == 128) {
    if (n_split <= 8) JK_COMBINE(128, 8);
    else if (n_split <= 10) JK_COMBINE(128, 10);
    else JK_COMBINE(128, 12);
  } else {
    if (n_split <= 8) JK_COMBINE(64, 8);
    else if (n_split <= 10) JK_COMBINE(64, 10);
    else JK_COMBINE(64, 12);
  }
#undef JK_COMBINE
  JK_LAUNCH_CHECK(ctx);
  return JK_OK;
}

int jk_attn_dispatch(jk_ctx* ctx, cudaStream_t st, int batch, int tree_size, const void* q,
                     const void* k_cache, const void* v_cache, int64_t cache_stride_b,
                     int64_t cache_stride_h, int cache_rows, const int32_t* kv_len,
                     const int32_t* parent, float softmax_scale, void* out);

extern "C" int jk_tree_verify_attn(jk_ctx* ctx, void* stream, int32_t batch, int32_t tree_size,
                                   const void* q, const void* k_cache, const void* v_cache,
                                   int64_t cache_stride_b, int64_t cache_stride_h,
                                   int32_t cache_rows, const int32_t* kv_len,
                                   const int32_t* parent, float softmax_scale, void* out) {
  if (!ctx || !q || !k_cache || !v_cache || !kv_len || !parent || !out) return JK_ERR_NULL;
  const jk_config& c = ctx->cfg;
  if (batch < 1 || tree_size < 1 || cache_rows < tree_size) return JK_ERR_SHAPE;
  if (batch > c.max_batch || tree_size > c.max_tree) return JK_ERR_CAPACITY;
  if (cache_stride_h < (int64_t)cache_rows * c.head_dim) return JK_ERR_SHAPE;
  if (!jk_aligned16(q) || !jk_aligned16(k_cache) || !jk_aligned16(v_cache) || !jk_aligned16(out))
    return JK_ERR_ALIGN;
  const int es = jk_elem_size(c.dtype);
  if ((cache_stride_b * es) % 16 || (cache_stride_h * es) % 16) return JK_ERR_ALIGN;
  if (!ctx->ws) return JK_ERR_WORKSPACE;
  int rc = jk_ensure_device_info(ctx);
  if (rc != JK_OK) return rc;
  return jk_attn_dispatch(ctx, (cudaStream_t)stream, batch, tree_size, q, k_cache, v_cache,
                          cache_stride_b, cache_stride_h, cache_rows, kv_len, parent,
                          softmax_scale, out);
}

// The kernel choice behind jk_tree_verify_attn (arguments already validated); jk_draft_pre runs
// the draft layer's own attention through it.
int jk_attn_dispatch(jk_ctx* ctx, cudaStream_t st, int batch, int tree_size, const void* q,
                     const void* k_cache, const void* v_cache, int64_t cache_stride_b,
                     int64_t cache_stride_h, int cache_rows, const int32_t* kv_len,
                     const int32_t* parent, float softmax_scale, void* out) {
  const jk_config& c = ctx->cfg;
  if (c.dtype == JK_BF16 && ctx->tensor_path && softmax_scale > 0.f && jk_tc_available(ctx))
    return jk_attn_tc(ctx, st, batch, tree_size, q, k_cache, v_cache, cache_stride_b,
                      cache_stride_h, cache_rows, kv_len, parent, softmax_scale, out);
#define JK_ATTN_CASE(T, D)                                                                \
  return attn_impl<T, D>(ctx, st, batch, tree_size, q, k_cache, v_cache, cache_stride_b,    \
                         cache_stride_h, cache_rows, kv_len, parent, softmax_scale, out)
  if (c.dtype == JK_BF16) {
    if (c.head_dim == 128) JK_ATTN_CASE(__nv_bfloat16, 128);
    JK_ATTN_CASE(__nv_bfloat16, 64);
  }
  if (c.head_dim == 128) JK_ATTN_CASE(float, 128);
  JK_ATTN_CASE(float, 64);
#undef JK_ATTN_CASE
}

// ------------------------------------------------------------------------------------------
// jk_tree_verify_attn_static: the same attention for callers that cannot allocate.
//
// Who they are: a serving process that handed every free byte of HBM to its KV-cache pool at
// start-up (a cudaMalloc for a workspace then simply fails), and a decode loop that must not
// stall, since cudaMalloc and cudaFree synchronise the whole device.  Such a caller cannot give
// this library the workspace that jk_set_workspace wants, so here the split-KV partials live in
// an array that is part of the library image itself.  Cost: every GPU that loads the library
// carries these JK_ATTN_STATIC_BYTES (+256) until the process exits, used or not.
//
// The array's name is only a handle in host code, not a device address; the address the kernels
// need comes from cudaGetSymbolAddress, asked once per device with that device current.
// ------------------------------------------------------------------------------------------
#define JK_ATTN_STATIC_BYTES (8u << 20)
#define JK_ATTN_STATIC_MAX_DEVICES 64
static __device__ __align__(256) unsigned char g_attn_static_scratch[JK_ATTN_STATIC_BYTES + 256];
static void* g_attn_static_ptr[JK_ATTN_STATIC_MAX_DEVICES];   // device address, per device

template <typename T, int D>
static int attn_static_impl(jk_ctx* ctx, cudaStream_t st, int dev, unsigned char* scratch, int B,
                            int M,
                            const void* q, const void* kc, const void* vc, int64_t sb, int64_t sh,
                            int cache_rows, const int32_t* kv_len, const int32_t* parent,
                            float scale, void* out, int32_t* status) {
  const jk_config& c = ctx->cfg;
  const int G = c.n_q_heads / c.n_kv_heads;
  const int n_qblk = (G * M + JK_ATTN_QB - 1) / JK_ATTN_QB;
  const int base_ctas = n_qblk * c.n_kv_heads * B;
  const size_t n_out = (size_t)B * M * c.n_q_heads;
  const size_t per_split = n_out * (D + 2) * sizeof(float);
  if (per_split > JK_ATTN_STATIC_BYTES) {
    snprintf(ctx->cuda_err, sizeof(ctx->cuda_err),
             "jk_tree_verify_attn_static: B*M*Hq*(d+2)*4 = %zu bytes exceeds the %u-byte scratch",
             per_split, JK_ATTN_STATIC_BYTES);
    return JK_ERR_CAPACITY;
  }
  int n_split = (2 * ctx->sm_count + base_ctas - 1) / base_ctas;
  const int max_by_len = (cache_rows / 64) > 0 ? (cache_rows / 64) : 1;
  const int max_by_mem = (int)(JK_ATTN_STATIC_BYTES / per_split);
  if (n_split > max_by_len) n_split = max_by_len;
  if (n_split > max_by_mem) n_split = max_by_mem;
  if (n_split > JK_ATTN_MAX_SPLIT) n_split = JK_ATTN_MAX_SPLIT;
  if (n_split < 1) n_split = 1;
  float* part_o = reinterpret_cast<float*>(scratch + 256);
  float* part_ml = part_o + (size_t)n_split * n_out * D;
  const size_t smem = sizeof(attn_smem<D>);
  auto kern = k_tree_attn<T, D>;
  // the shared-memory limit is a per-device property of the kernel: raised once per device
  static bool smem_set[JK_ATTN_STATIC_MAX_DEVICES];
  if (!smem_set[dev]) {
    JK_CUDA_CHECK(ctx, cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            (int)smem));
    smem_set[dev] = true;
  }
  kern<<<dim3(n_split * n_qblk, c.n_kv_heads, B), 256, smem, st>>>(
      (const T*)q, (const T*)kc, (const T*)vc, sb, sh, cache_rows, kv_len, parent, scale, M,
      c.n_q_heads, c.n_kv_heads, n_split, n_qblk, part_o, part_ml, status);
  JK_LAUNCH_CHECK(ctx);
  k_attn_combine<T, D, 8><<<(unsigned)((n_out + 7) / 8), 256, 0, st>>>(part_o, part_ml, n_split,
                                                                    n_out, (T*)out);
  JK_LAUNCH_CHECK(ctx);
  return JK_OK;
}

extern "C" int jk_tree_verify_attn_static(jk_ctx* ctx, void* stream, int32_t batch,
                                          int32_t tree_size, const void* q, const void* k_cache,
                                          const void* v_cache, int64_t cache_stride_b,
                                          int64_t cache_stride_h, int32_t cache_rows,
                                          const int32_t* kv_len, const int32_t* parent,
                                          float softmax_scale, void* out, int32_t* status) {
  // `status` is required: this call has no context workspace whose status word could record a
  // cache that is too short, and an error nobody can read is worse than an argument error.
  if (!ctx || !q || !k_cache || !v_cache || !kv_len || !parent || !out || !status)
    return JK_ERR_NULL;
  const jk_config& c = ctx->cfg;
  if (batch < 1 || tree_size < 1 || cache_rows < tree_size) return JK_ERR_SHAPE;
  if (batch > c.max_batch || tree_size > c.max_tree) return JK_ERR_CAPACITY;
  if (cache_stride_h < (int64_t)cache_rows * c.head_dim) return JK_ERR_SHAPE;
  if (!jk_aligned16(q) || !jk_aligned16(k_cache) || !jk_aligned16(v_cache) || !jk_aligned16(out))
    return JK_ERR_ALIGN;
  const int es = jk_elem_size(c.dtype);
  if ((cache_stride_b * es) % 16 || (cache_stride_h * es) % 16) return JK_ERR_ALIGN;
  if ((size_t)batch * tree_size * c.n_q_heads * (c.head_dim + 2) * sizeof(float) >
      JK_ATTN_STATIC_BYTES) {
    snprintf(ctx->cuda_err, sizeof(ctx->cuda_err),
             "jk_tree_verify_attn_static: batch*tree_size*n_q_heads*(head_dim+2)*4 exceeds the "
             "%u-byte built-in scratch", JK_ATTN_STATIC_BYTES);
    return JK_ERR_CAPACITY;
  }
  int rc = jk_ensure_device_info(ctx);
  if (rc != JK_OK) return rc;
  // once per device: turn the symbol into the device address the kernels can use
  int dev = -1;
  JK_CUDA_CHECK(ctx, cudaGetDevice(&dev));
  if (dev < 0 || dev >= JK_ATTN_STATIC_MAX_DEVICES) return JK_ERR_SHAPE;
  if (!g_attn_static_ptr[dev]) {
    void* p = nullptr;
    JK_CUDA_CHECK(ctx, cudaGetSymbolAddress(&p, g_attn_static_scratch));
    if (!p) return JK_ERR_CUDA;
    g_attn_static_ptr[dev] = p;
  }
  unsigned char* scratch = static_cast<unsigned char*>(g_attn_static_ptr[dev]);
  cudaStream_t st = (cudaStream_t)stream;
#define JK_ATTN_STATIC_CASE(T, D)                                                             \
  return attn_static_impl<T, D>(ctx, st, dev, scratch, batch, tree_size, q, k_cache, v_cache, \
                                cache_stride_b, cache_stride_h, cache_rows, kv_len, parent,   \
                                softmax_scale, out, status)
  if (c.dtype == JK_BF16) {
    if (c.head_dim == 128) JK_ATTN_STATIC_CASE(__nv_bfloat16, 128);
    JK_ATTN_STATIC_CASE(__nv_bfloat16, 64);
  }
  if (c.head_dim == 128) JK_ATTN_STATIC_CASE(float, 128);
  JK_ATTN_STATIC_CASE(float, 64);
#undef JK_ATTN_STATIC_CASE
}
