// jk_draft_pre: the draft layer in front of the MoE (arXiv 2502.06282, Sec. 3.1.2, Eq. 1 and the
// paragraph before it): token embedding and the parent's feature concatenated, the reduction
// layer h = W_fc [emb ; f_prev], then u = Attn(h) + h with the draft layer's own KV cache, the
// nodes of the partial tree attending over the committed prefix and their ancestors.
//
// The three projections run on the streaming GEMM of jk_gemm_tc.cu (bf16) or on CUDA cores
// (f32); the attention is the tree attention of jk_tree_verify_attn over the nodes expanded so
// far (their queries are kept from pass to pass, so a pass recomputes the few earlier nodes'
// outputs instead of needing a kernel whose query rows differ from its key rows).
#include <math.h>

#include "jk_common.cuh"

int jk_tc_linear(jk_ctx* ctx, cudaStream_t st, const void* W, int Mrows, int Kdim, const void* x,
                 int x_rows, int n_rows, const void* bias, const void* resid, long long resid_ld,
                 void* out_bf16, float* out_f32, long long out_ld);      // jk_gemm_tc.cu
int jk_tc_available(const jk_ctx* ctx);
int jk_attn_dispatch(jk_ctx* ctx, cudaStream_t st, int batch, int tree_size, const void* q,
                     const void* k_cache, const void* v_cache, int64_t sb, int64_t sh,
                     int cache_rows, const int32_t* kv_len, const int32_t* parent, float scale,
                     void* out);                                          // jk_attn.cu

// x[r] = [emb(tok) ; parent feature], and the node's place in the partial tree.  One block per
// node r = (b, f).  Root pass (node_gidx == NULL): tok = root_tok[b], feature = prev_feat[b].
template <typename T>
__global__ void __launch_bounds__(256) k_pre_gather(
    const T* __restrict__ emb, const T* __restrict__ prev_feat, const int32_t* __restrict__ node_gidx,
    const int32_t* __restrict__ pool_tok, long long pool_stride, const int32_t* __restrict__ root_tok,
    int F, int H, int V, int per_node, int prev_gidx_base, int prev_slot_base, int prev_frontier,
    int slot_base, long long slot_stride, T* __restrict__ x, int32_t* __restrict__ slot_parent,
    int32_t* __restrict__ slot_depth, int32_t* status) {
  jk_pdl_wait();
  jk_pdl_trigger();
  constexpr int VN = jk_vec<T>::N;
  const int r = blockIdx.x, b = r / F, f = r % F;
  int tok, prow, pslot;
  if (node_gidx) {
    const int g = node_gidx[(size_t)b * F + f];
    const int flat = g - prev_gidx_base;
    int fp = flat / per_node;
    if (flat < 0 || fp >= prev_frontier) {
      if (threadIdx.x == 0) jk_set_status(status, JK_ERR_BOUNDS);
      fp = 0;
    }
    tok = pool_tok[(size_t)b * pool_stride + (flat < 0 ? 0 : g)];
    prow = b * prev_frontier + fp;
    pslot = prev_slot_base + fp;
  } else {
    tok = root_tok[b];
    prow = b;
    pslot = -1;
  }
  if (tok < 0 || tok >= V) {
    if (threadIdx.x == 0) jk_set_status(status, JK_ERR_BOUNDS);
    tok = 0;
  }
  if (threadIdx.x == 0) {
    const size_t s = (size_t)b * slot_stride + slot_base + f;
    slot_parent[s] = pslot;
    slot_depth[s] = pslot < 0 ? 0 : slot_depth[(size_t)b * slot_stride + pslot] + 1;
  }
  const uint4* e4 = reinterpret_cast<const uint4*>(emb + (size_t)tok * H);
  const uint4* p4 = reinterpret_cast<const uint4*>(prev_feat + (size_t)prow * H);
  uint4* x4 = reinterpret_cast<uint4*>(x + (size_t)r * 2 * H);
  const int n16 = H / VN;
  for (int i = threadIdx.x; i < n16; i += blockDim.x) {
    x4[i] = e4[i];
    x4[n16 + i] = p4[i];
  }
}

// CUDA-core linear layer: out[r, m] = W[m] . x[r] (+ bias[m]) (+ resid[r, m]); one warp per
// weight row, RB activation rows at a time.
template <typename T, typename TO>
__global__ void __launch_bounds__(256) k_linear(
    const T* __restrict__ W, const T* __restrict__ x, long long x_ld, int R, int Mrows, int Kdim,
    const T* __restrict__ bias, const T* __restrict__ resid, long long resid_ld,
    TO* __restrict__ out, long long out_ld) {
  constexpr int VN = jk_vec<T>::N;
  constexpr int RB = 8;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  for (int m = blockIdx.x * nw + warp; m < Mrows; m += gridDim.x * nw) {
    const T* wr = W + (size_t)m * Kdim;
    for (int p = 0; p < R; p += RB) {
      const int nr = min(RB, R - p);
      float acc[RB];
#pragma unroll
      for (int rb = 0; rb < RB; ++rb) acc[rb] = 0.f;
      for (int k = lane * VN; k < Kdim; k += 32 * VN) {
        float wv[VN];
        jk_vec<T>::load(wr + k, wv);
#pragma unroll
        for (int rb = 0; rb < RB; ++rb) {
          if (rb < nr) {
            float xv[VN];
            jk_vec<T>::load(x + (size_t)(p + rb) * x_ld + k, xv);
#pragma unroll
            for (int i = 0; i < VN; ++i) acc[rb] = fmaf(wv[i], xv[i], acc[rb]);
          }
        }
      }
#pragma unroll
      for (int rb = 0; rb < RB; ++rb) acc[rb] = jk_warp_sum(acc[rb]);
      if (lane < nr) {
        float v = 0.f;
#pragma unroll
        for (int rb = 0; rb < RB; ++rb) if (rb == lane) v = acc[rb];
        if (bias) v += jk_to_float(bias[m]);
        if (resid) v += jk_to_float(resid[(size_t)(p + lane) * resid_ld + m]);
        out[(size_t)(p + lane) * out_ld + m] = jk_from_float<TO>(v);
      }
    }
  }
}

// Rotary positions (LLaMA convention: pair (i, i + d/2) turns by pos / theta^(2i/d), pos = prefix
// length + depth of the node), the rotated query kept per slot, K and V appended to the draft
// layer's cache at row prefix length + slot.  One block per node; the angle is formed and reduced
// in double precision (a position of several thousand times a frequency near one loses the
// tolerance in fp32).
template <typename T>
__global__ void __launch_bounds__(256) k_pre_rope_scatter(
    const float* __restrict__ qkv, int F, int Hq, int Hkv, int D, float theta,
    const int32_t* __restrict__ kv_len, const int32_t* __restrict__ slot_depth, int slot_base,
    long long slot_stride, T* __restrict__ q_slots, T* __restrict__ k_cache, T* __restrict__ v_cache,
    long long cache_sb, long long cache_sh, int cache_rows, int32_t* status) {
  // The frequencies theta^(-2j/d) in double precision, once per block and ahead of the
  // dependency wait (they depend on nothing); per pair the angle is then one double product,
  // reduced to [-pi, pi] in double, and only the sine and cosine of the small remainder are
  // taken in single precision.
  __shared__ double s_inv[64];                     // head size 64 or 128
  for (int j = threadIdx.x; j < D / 2; j += blockDim.x)
    s_inv[j] = pow((double)theta, -2.0 * (double)j / (double)D);
  __syncthreads();
  jk_pdl_wait();
  jk_pdl_trigger();
  const int r = blockIdx.x, b = r / F, f = r % F;
  const int slot = slot_base + f;
  const int P = kv_len[b];
  if (P < 0 || P + slot >= cache_rows) {
    if (threadIdx.x == 0) jk_set_status(status, JK_ERR_BOUNDS);
    return;
  }
  const int depth = slot_depth[(size_t)b * slot_stride + slot];
  const double pos = (double)(P + depth);
  const int half = D / 2;
  const float* row = qkv + (size_t)r * (Hq + 2 * Hkv) * D;
  const int n_rot = (Hq + Hkv) * half;               // rotated pairs: all q heads, then all k heads
  for (int i = threadIdx.x; i < n_rot; i += blockDim.x) {
    const int head = i / half, j = i % half;
    const double ang = pos * s_inv[j];
    const double turns = rint(ang * 0.15915494309189535);            // 1 / (2 pi)
    double red = fma(-turns, 6.283185307179586, ang);                // 2 pi, leading part
    red = fma(-turns, 2.4492935982947064e-16, red);                  // 2 pi, the rest
    float sn, cs;
    sincosf((float)red, &sn, &cs);
    const float x1 = row[head * D + j], x2 = row[head * D + half + j];
    const float o1 = x1 * cs - x2 * sn;
    const float o2 = x2 * cs + x1 * sn;
    if (head < Hq) {
      T* dst = q_slots + (((size_t)b * slot_stride + slot) * Hq + head) * D;
      dst[j] = jk_from_float<T>(o1);
      dst[half + j] = jk_from_float<T>(o2);
    } else {
      T* dst = k_cache + (size_t)b * cache_sb + (size_t)(head - Hq) * cache_sh + (size_t)(P + slot) * D;
      dst[j] = jk_from_float<T>(o1);
      dst[half + j] = jk_from_float<T>(o2);
    }
  }
  const float* vrow = row + (size_t)(Hq + Hkv) * D;
  for (int i = threadIdx.x; i < Hkv * D; i += blockDim.x) {
    const int head = i / D, j = i % D;
    v_cache[(size_t)b * cache_sb + (size_t)head * cache_sh + (size_t)(P + slot) * D + j] =
        jk_from_float<T>(vrow[i]);
  }
}

// Dense copies for the attention call: queries and parents of the M nodes expanded so far.
template <typename T>
__global__ void __launch_bounds__(256) k_pre_dense(
    const T* __restrict__ q_slots, const int32_t* __restrict__ slot_parent, long long slot_stride,
    int M, int row_elems, T* __restrict__ q_dense, int32_t* __restrict__ par_dense) {
  jk_pdl_wait();
  jk_pdl_trigger();
  constexpr int VN = jk_vec<T>::N;
  const int r = blockIdx.x, b = r / M, s = r % M;
  const uint4* src = reinterpret_cast<const uint4*>(q_slots + ((size_t)b * slot_stride + s) * row_elems);
  uint4* dst = reinterpret_cast<uint4*>(q_dense + (size_t)r * row_elems);
  for (int i = threadIdx.x; i < row_elems / VN; i += blockDim.x) dst[i] = src[i];
  if (threadIdx.x == 0) par_dense[r] = slot_parent[(size_t)b * slot_stride + s];
}

// The attention outputs of this pass's nodes, gathered as the O-projection's input rows.
template <typename T>
__global__ void __launch_bounds__(256) k_pre_pick(
    const T* __restrict__ att_dense, int M, int F, int slot_base, int row_elems, T* __restrict__ ao) {
  jk_pdl_wait();
  jk_pdl_trigger();
  constexpr int VN = jk_vec<T>::N;
  const int r = blockIdx.x, b = r / F, f = r % F;
  const uint4* src = reinterpret_cast<const uint4*>(att_dense + ((size_t)b * M + slot_base + f) * row_elems);
  uint4* dst = reinterpret_cast<uint4*>(ao + (size_t)r * row_elems);
  for (int i = threadIdx.x; i < row_elems / VN; i += blockDim.x) dst[i] = src[i];
}

template <typename T>
static int linear(jk_ctx* ctx, cudaStream_t st, bool tc, const void* W, int Mrows, int Kdim,
                  const void* x, int x_rows, int R, const void* bias, const void* resid,
                  long long resid_ld, void* out_t, float* out_f32, long long out_ld) {
  if (tc)
    return jk_tc_linear(ctx, st, W, Mrows, Kdim, x, x_rows, R, bias, resid, resid_ld, out_t, out_f32,
                        out_ld);
  const int grid = (Mrows + 7) / 8;
  JK_PROF(ctx, st, JK_ST_PRE_GEMM);
  if (out_f32)
    k_linear<T, float><<<grid, 256, 0, st>>>((const T*)W, (const T*)x, Kdim, R, Mrows, Kdim,
                                             (const T*)bias, (const T*)resid, resid_ld, out_f32,
                                             out_ld);
  else
    k_linear<T, T><<<grid, 256, 0, st>>>((const T*)W, (const T*)x, Kdim, R, Mrows, Kdim,
                                         (const T*)bias, (const T*)resid, resid_ld, (T*)out_t, out_ld);
  JK_LAUNCH_CHECK(ctx);
  return JK_OK;
}

template <typename T>
static int pre_impl(jk_ctx* ctx, cudaStream_t st, const jk_pre_weights* w, const jk_pre_state* s,
                    int B, int F, int slot_base, const int32_t* node_gidx, const jk_pool* pool,
                    int prev_gidx_base, int prev_slot_base, int prev_frontier, const void* prev_feat,
                    const int32_t* root_tok, void* k_cache, void* v_cache, int64_t sb, int64_t sh,
                    int cache_rows, const int32_t* kv_len, float theta, float scale, void* out_u) {
  const jk_config& c = ctx->cfg;
  const jk_ws_layout& L = ctx->lay;
  char* ws = ctx->ws;
  const int R = B * F, H = c.hidden, Hq = c.n_q_heads, Hkv = c.n_kv_heads, D = c.head_dim;
  const int qd = Hq * D, qkvd = (Hq + 2 * Hkv) * D;
  const int Rp = L.rows_pad;
  const int M = slot_base + F;                       // nodes expanded so far, this pass included
  int32_t* status = (int32_t*)(ws + L.status);
  T* x = (T*)(ws + L.pre_x);
  T* h = (T*)(ws + L.pre_h);
  float* qkv = (float*)(ws + L.pre_qkv);
  T* q_dense = (T*)(ws + L.pre_qd);
  int32_t* par_dense = (int32_t*)(ws + L.pre_par);
  T* att = (T*)(ws + L.pre_att);
  T* ao = (T*)(ws + L.pre_ao);
  const bool tc = ctx->tensor_path && c.dtype == JK_BF16 && jk_tc_available(ctx);

  JK_PROF(ctx, st, JK_ST_PRE_GATHER);
  jk_launch_pdl(k_pre_gather<T>, dim3(R), dim3(256), 0, st, (const T*)w->emb, (const T*)prev_feat,
                node_gidx, (const int32_t*)(pool ? pool->tok : nullptr),
                (long long)(pool ? pool->stride_b : 0), root_tok, F, H, c.vocab,
                c.top_k * c.k_per_expert, prev_gidx_base, prev_slot_base, prev_frontier, slot_base,
                (long long)s->stride_b, x, s->slot_parent, s->slot_depth, status);
  JK_LAUNCH_CHECK(ctx);
  // h = W_fc [emb ; f_prev] (+ b_fc)
  int rc = linear<T>(ctx, st, tc, w->w_fc, H, 2 * H, x, Rp, R, w->b_fc, nullptr, 0, h, nullptr, H);
  if (rc != JK_OK) return rc;
  // q, k, v = W_qkv h
  rc = linear<T>(ctx, st, tc, w->w_qkv, qkvd, H, h, Rp, R, nullptr, nullptr, 0, nullptr, qkv, qkvd);
  if (rc != JK_OK) return rc;
  JK_PROF(ctx, st, JK_ST_PRE_ROPE);
  jk_launch_pdl(k_pre_rope_scatter<T>, dim3(R), dim3(256), 0, st, (const float*)qkv, F, Hq, Hkv, D,
                theta, kv_len, (const int32_t*)s->slot_depth, slot_base, (long long)s->stride_b,
                (T*)s->q, (T*)k_cache, (T*)v_cache, (long long)sb, (long long)sh, cache_rows, status);
  JK_LAUNCH_CHECK(ctx);
  // With one sequence the slots of the nodes expanded so far already are a dense [M, Hq, d]
  // array (and their parents a dense list): the attention call reads them where they are.
  if (B == 1) {
    q_dense = (T*)s->q;
    par_dense = s->slot_parent;
  } else {
    JK_PROF(ctx, st, JK_ST_PRE_ROPE);
    jk_launch_pdl(k_pre_dense<T>, dim3(B * M), dim3(256), 0, st, (const T*)s->q,
                  (const int32_t*)s->slot_parent, (long long)s->stride_b, M, qd, q_dense, par_dense);
    JK_LAUNCH_CHECK(ctx);
  }
  // Attn over the committed prefix and each node's ancestors
  ctx->st_attn = JK_ST_PRE_ATTN;
  ctx->st_combine = JK_ST_PRE_ATTN_COMBINE;
  rc = jk_attn_dispatch(ctx, st, B, M, q_dense, k_cache, v_cache, sb, sh, cache_rows, kv_len,
                        par_dense, scale, att);
  ctx->st_attn = JK_ST_ATTN;
  ctx->st_combine = JK_ST_ATTN_COMBINE;
  if (rc != JK_OK) return rc;
  // u = W_o Attn + h.  With one sequence this pass's rows of the attention output are
  // contiguous and feed the projection where they are (rows past the last are zero-filled by
  // the copy engine: the array is declared F rows long).
  if (B == 1)
    return linear<T>(ctx, st, tc, w->w_o, H, qd, att + (size_t)slot_base * qd, F, R, nullptr, h, H,
                     out_u, nullptr, H);
  JK_PROF(ctx, st, JK_ST_PRE_ROPE);
  jk_launch_pdl(k_pre_pick<T>, dim3(R), dim3(256), 0, st, (const T*)att, M, F, slot_base, qd, ao);
  JK_LAUNCH_CHECK(ctx);
  return linear<T>(ctx, st, tc, w->w_o, H, qd, ao, Rp, R, nullptr, h, H, out_u, nullptr, H);
}

extern "C" int jk_draft_pre(jk_ctx* ctx, void* stream, const jk_pre_weights* w,
                            const jk_pre_state* state, int32_t batch, int32_t n_frontier,
                            int32_t slot_base, const int32_t* node_gidx, const jk_pool* pool,
                            int32_t prev_gidx_base, int32_t prev_slot_base, int32_t prev_frontier,
                            const void* prev_feat, const int32_t* root_tok, void* k_cache,
                            void* v_cache, int64_t cache_stride_b, int64_t cache_stride_h,
                            int32_t cache_rows, const int32_t* kv_len, float rope_theta,
                            float softmax_scale, void* out_u) {
  if (!ctx || !w || !state || !prev_feat || !k_cache || !v_cache || !kv_len || !out_u)
    return JK_ERR_NULL;
  if (!w->emb || !w->w_fc || !w->w_qkv || !w->w_o) return JK_ERR_NULL;
  if (!state->q || !state->slot_parent || !state->slot_depth) return JK_ERR_NULL;
  if (node_gidx ? (!pool || !pool->tok) : !root_tok) return JK_ERR_NULL;
  const jk_config& c = ctx->cfg;
  if (batch < 1 || n_frontier < 1 || slot_base < 0 || !(rope_theta > 0.f) || !(softmax_scale > 0.f))
    return JK_ERR_SHAPE;
  if (batch > c.max_batch || n_frontier > c.max_frontier) return JK_ERR_CAPACITY;
  const int M = slot_base + n_frontier;
  if (M > c.max_depth * c.max_frontier || M > JK_MAX_TREE || state->stride_b < M) return JK_ERR_CAPACITY;
  if (!node_gidx && (slot_base != 0 || n_frontier != 1)) return JK_ERR_SHAPE;   // the root pass
  if (node_gidx && (prev_frontier < 1 || prev_gidx_base < 0 || prev_slot_base < 0 ||
                    prev_slot_base + prev_frontier > slot_base))
    return JK_ERR_SHAPE;
  if (cache_rows < M || cache_stride_h < (int64_t)cache_rows * c.head_dim) return JK_ERR_SHAPE;
  const void* ptrs[] = {w->emb, w->w_fc, w->b_fc, w->w_qkv, w->w_o, state->q, prev_feat, k_cache,
                        v_cache, out_u};
  for (const void* p : ptrs)
    if (p && !jk_aligned16(p)) return JK_ERR_ALIGN;
  const int es = jk_elem_size(c.dtype);
  if ((cache_stride_b * es) % 16 || (cache_stride_h * es) % 16) return JK_ERR_ALIGN;
  if (!ctx->ws) return JK_ERR_WORKSPACE;
  int rc = jk_ensure_device_info(ctx);
  if (rc != JK_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  if (c.dtype == JK_BF16)
    return pre_impl<__nv_bfloat16>(ctx, st, w, state, batch, n_frontier, slot_base, node_gidx, pool,
                                   prev_gidx_base, prev_slot_base, prev_frontier, prev_feat,
                                   root_tok, k_cache, v_cache, cache_stride_b, cache_stride_h,
                                   cache_rows, kv_len, rope_theta, softmax_scale, out_u);
  return pre_impl<float>(ctx, st, w, state, batch, n_frontier, slot_base, node_gidx, pool,
                         prev_gidx_base, prev_slot_base, prev_frontier, prev_feat, root_tok,
                         k_cache, v_cache, cache_stride_b, cache_stride_h, cache_rows, kv_len,
                         rope_theta, softmax_scale, out_u);
}

// ------------------------------------------------------------------------------------------
// Verification-side steps around the tree attention of one target layer (Sec. 2.1 step 2)
// ------------------------------------------------------------------------------------------
extern "C" int jk_verify_qkv(jk_ctx* ctx, void* stream, const void* w_qkv, int32_t batch,
                             int32_t tree_size, const void* x, const int32_t* depth, void* q_out,
                             void* k_cache, void* v_cache, int64_t cache_stride_b,
                             int64_t cache_stride_h, int32_t cache_rows, const int32_t* kv_len,
                             float rope_theta) {
  if (!ctx || !w_qkv || !x || !depth || !q_out || !k_cache || !v_cache || !kv_len) return JK_ERR_NULL;
  const jk_config& c = ctx->cfg;
  if (batch < 1 || tree_size < 1 || cache_rows < tree_size || !(rope_theta > 0.f)) return JK_ERR_SHAPE;
  if (batch > c.max_batch || tree_size > c.max_tree) return JK_ERR_CAPACITY;
  if (cache_stride_h < (int64_t)cache_rows * c.head_dim) return JK_ERR_SHAPE;
  const void* ptrs[] = {w_qkv, x, q_out, k_cache, v_cache};
  for (const void* p : ptrs)
    if (!jk_aligned16(p)) return JK_ERR_ALIGN;
  const int es = jk_elem_size(c.dtype);
  if ((cache_stride_b * es) % 16 || (cache_stride_h * es) % 16) return JK_ERR_ALIGN;
  if (!ctx->ws) return JK_ERR_WORKSPACE;
  int rc = jk_ensure_device_info(ctx);
  if (rc != JK_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  const jk_ws_layout& L = ctx->lay;
  const int R = batch * tree_size, H = c.hidden, Hq = c.n_q_heads, Hkv = c.n_kv_heads, D = c.head_dim;
  const int qkvd = (Hq + 2 * Hkv) * D;
  float* qkv = (float*)(ctx->ws + L.pre_qkv);
  int32_t* status = (int32_t*)(ctx->ws + L.status);
  const bool tc = ctx->tensor_path && c.dtype == JK_BF16 && jk_tc_available(ctx);
  // the streaming GEMM takes at most 256 activation rows: larger batches of tree tokens go
  // through it in row chunks (each chunk streams W_qkv once)
  for (int r0 = 0; r0 < R; r0 += 256) {
    const int nr = R - r0 < 256 ? R - r0 : 256;
    const char* xr = (const char*)x + (size_t)r0 * H * es;
    if (c.dtype == JK_BF16)
      rc = linear<__nv_bfloat16>(ctx, st, tc, w_qkv, qkvd, H, xr, nr, nr, nullptr, nullptr, 0, nullptr,
                                 qkv + (size_t)r0 * qkvd, qkvd);
    else
      rc = linear<float>(ctx, st, false, w_qkv, qkvd, H, xr, nr, nr, nullptr, nullptr, 0, nullptr,
                         qkv + (size_t)r0 * qkvd, qkvd);
    if (rc != JK_OK) return rc;
  }
  JK_PROF(ctx, st, JK_ST_PRE_ROPE);
  if (c.dtype == JK_BF16)
    jk_launch_pdl(k_pre_rope_scatter<__nv_bfloat16>, dim3(R), dim3(256), 0, st, (const float*)qkv,
                  tree_size, Hq, Hkv, D, rope_theta, kv_len, depth, 0, (long long)tree_size,
                  (__nv_bfloat16*)q_out, (__nv_bfloat16*)k_cache, (__nv_bfloat16*)v_cache,
                  (long long)cache_stride_b, (long long)cache_stride_h, cache_rows, status);
  else
    jk_launch_pdl(k_pre_rope_scatter<float>, dim3(R), dim3(256), 0, st, (const float*)qkv, tree_size,
                  Hq, Hkv, D, rope_theta, kv_len, depth, 0, (long long)tree_size, (float*)q_out,
                  (float*)k_cache, (float*)v_cache, (long long)cache_stride_b,
                  (long long)cache_stride_h, cache_rows, status);
  JK_LAUNCH_CHECK(ctx);
  return JK_OK;
}

// out[b, 0] = hidden[b, 0]; out[b, 1 + j] = hidden[b, acc_idx[b, j]] for j < n_acc[b]; zero after.
__global__ void __launch_bounds__(256) k_gather_accepted(
    const uint4* __restrict__ hidden, const int32_t* __restrict__ n_acc,
    const int32_t* __restrict__ acc_idx, int M, int max_depth, int row16, int rows_out,
    uint4* __restrict__ out, int32_t* status) {
  jk_pdl_wait();
  jk_pdl_trigger();
  const int b = blockIdx.y, j = blockIdx.x;                 // output row j of sequence b
  const int n = n_acc[b];
  int src = -1;
  if (j == 0) src = 0;
  else if (j - 1 < n && j - 1 < max_depth) src = acc_idx[(size_t)b * max_depth + j - 1];
  if (src >= M) {
    if (threadIdx.x == 0) jk_set_status(status, JK_ERR_BOUNDS);
    src = -1;
  }
  uint4* o = out + ((size_t)b * rows_out + j) * row16;
  const uint4* h = hidden + ((size_t)b * M + (src < 0 ? 0 : src)) * row16;
  for (int i = threadIdx.x; i < row16; i += blockDim.x)
    o[i] = src < 0 ? make_uint4(0u, 0u, 0u, 0u) : h[i];
}

extern "C" int jk_gather_accepted(jk_ctx* ctx, void* stream, int32_t batch, int32_t tree_size,
                                  const void* hidden, const int32_t* n_acc, const int32_t* acc_idx,
                                  int32_t rows_out, void* out) {
  if (!ctx || !hidden || !n_acc || !acc_idx || !out) return JK_ERR_NULL;
  const jk_config& c = ctx->cfg;
  if (batch < 1 || tree_size < 1 || rows_out < 1 || rows_out > c.max_depth + 1) return JK_ERR_SHAPE;
  if (batch > c.max_batch || tree_size > c.max_tree) return JK_ERR_CAPACITY;
  if (!jk_aligned16(hidden) || !jk_aligned16(out)) return JK_ERR_ALIGN;
  if (!ctx->ws) return JK_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  const int row16 = c.hidden * jk_elem_size(c.dtype) / 16;
  JK_PROF(ctx, st, JK_ST_COMPACT);
  jk_launch_pdl(k_gather_accepted, dim3(rows_out, batch), dim3(256), 0, st, (const uint4*)hidden,
                n_acc, acc_idx, tree_size, c.max_depth, row16, rows_out, (uint4*)out,
                (int32_t*)(ctx->ws + ctx->lay.status));
  JK_LAUNCH_CHECK(ctx);
  return JK_OK;
}
