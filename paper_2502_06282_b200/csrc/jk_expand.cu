// jk_draft_expand and jk_tree_finalize: router, expert FFNs, shared LM head, per-expert top-k,
// frontier selection and tree finalisation (arXiv 2502.06282, Sec. 3.1.2, Eq. 2-5).
//
// The dense contractions have two implementations: CUDA-core kernels in this file (exact fp32
// accumulation, used for the f32 dtype and as a cross-check), and tcgen05 tensor-core kernels in
// jk_gemm_tc.cu (bf16).  Everything around them (router, activation, residuals, top-k, frontier)
// is shared.
#include <limits.h>
#include <type_traits>
#include <math.h>

#include "jk_common.cuh"
#include "jk_topk.cuh"

// tensor-core path (jk_gemm_tc.cu)
int jk_tc_ffn(jk_ctx* ctx, cudaStream_t st, const jk_draft_weights* w, int R,
              const int32_t* expert, const float* gate, const void* u, void* out_feat);
int jk_tc_lm_head(jk_ctx* ctx, cudaStream_t st, const jk_draft_weights* w, int RK, float* logits,
                  int rows_per_b, long long logits_stride_b);
int jk_tc_available(const jk_ctx* ctx);

// ------------------------------------------------------------------------------------------
// Router: RMSNorm, Eq. 2 softmax over the N centroids, Eq. 5 top-K gate.  One block per row.
// ------------------------------------------------------------------------------------------
template <typename T>
__global__ void __launch_bounds__(512) k_router(
    const T* __restrict__ u, const T* __restrict__ router, const T* __restrict__ norm_w,
    int H, int N, int K, float eps, int use_norm, T* __restrict__ xn,
    float* __restrict__ out_probs, int32_t* __restrict__ out_expert, float* __restrict__ out_gate) {
  // The weights do not depend on the kernel before: ask for this thread's pieces of them (into
  // the L2) ahead of the dependency wait, so that only u is fetched after it.
  {
    constexpr int VNP = jk_vec<T>::N;
    for (int k = threadIdx.x * VNP; k < H; k += blockDim.x * VNP) {
      if (use_norm && norm_w) asm volatile("prefetch.global.L2 [%0];" ::"l"(norm_w + k));
      for (int j = 0; j < N; ++j)
        asm volatile("prefetch.global.L2 [%0];" ::"l"(router + (size_t)j * H + k));
    }
  }
  jk_pdl_wait();
  jk_pdl_trigger();
  // One pass over the row: the sum of squares and the N centroid dot products of u * gamma are
  // accumulated together (the RMS factor is a scalar, applied to the dots afterwards).
  constexpr int VN = jk_vec<T>::N;
  __shared__ float part[16][JK_MAX_EXPERTS + 1];
  __shared__ float tot[JK_MAX_EXPERTS + 1];
  const int row = blockIdx.x;
  const T* ur = u + (size_t)row * H;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  float ss = 0.f;
  float z[JK_MAX_EXPERTS];
#pragma unroll
  for (int j = 0; j < JK_MAX_EXPERTS; ++j) z[j] = 0.f;
  for (int k = threadIdx.x * VN; k < H; k += blockDim.x * VN) {
    float v[VN];
    jk_vec<T>::load(ur + k, v);
#pragma unroll
    for (int i = 0; i < VN; ++i) ss += v[i] * v[i];
    if (use_norm && norm_w) {
      float g[VN];
      jk_vec<T>::load(norm_w + k, g);
#pragma unroll
      for (int i = 0; i < VN; ++i) v[i] *= g[i];
    }
#pragma unroll
    for (int j = 0; j < JK_MAX_EXPERTS; ++j) {
      if (j < N) {
        float e[VN];
        jk_vec<T>::load(router + (size_t)j * H + k, e);
#pragma unroll
        for (int i = 0; i < VN; ++i) z[j] += v[i] * e[i];
      }
    }
  }
  ss = jk_warp_sum(ss);
#pragma unroll
  for (int j = 0; j < JK_MAX_EXPERTS; ++j) if (j < N) z[j] = jk_warp_sum(z[j]);
  if (lane == 0) {
    part[warp][JK_MAX_EXPERTS] = ss;
#pragma unroll
    for (int j = 0; j < JK_MAX_EXPERTS; ++j) if (j < N) part[warp][j] = z[j];
  }
  __syncthreads();
  if (threadIdx.x <= JK_MAX_EXPERTS && (threadIdx.x < N || threadIdx.x == JK_MAX_EXPERTS)) {
    float t = 0.f;
    for (int w = 0; w < nw; ++w) t += part[w][threadIdx.x];
    tot[threadIdx.x] = t;
  }
  __syncthreads();
  const float rinv = use_norm ? rsqrtf(tot[JK_MAX_EXPERTS] / (float)H + eps) : 1.f;
  // normalised hidden state for the expert GEMMs
  for (int k = threadIdx.x * VN; k < H; k += blockDim.x * VN) {
    float v[VN];
    jk_vec<T>::load(ur + k, v);
    if (use_norm && norm_w) {
      float g[VN];
      jk_vec<T>::load(norm_w + k, g);
#pragma unroll
      for (int i = 0; i < VN; ++i) v[i] *= g[i];
    }
#pragma unroll
    for (int i = 0; i < VN; ++i) xn[(size_t)row * H + k + i] = jk_from_float<T>(v[i] * rinv);
  }
  if (threadIdx.x == 0) {
    float zs[JK_MAX_EXPERTS];
    float m = -INFINITY;
    for (int j = 0; j < N; ++j) { zs[j] = tot[j] * rinv; m = fmaxf(m, zs[j]); }
    float s[JK_MAX_EXPERTS], sum = 0.f;
    for (int j = 0; j < N; ++j) { s[j] = expf(zs[j] - m); sum += s[j]; }
    for (int j = 0; j < N; ++j) {
      s[j] = s[j] / sum;
      if (out_probs) out_probs[(size_t)row * N + j] = s[j];
    }
    unsigned taken = 0;
    for (int r = 0; r < K; ++r) {
      int best = -1;
      for (int j = 0; j < N; ++j) {
        if (taken & (1u << j)) continue;
        if (best < 0 || s[j] > s[best]) best = j;     // ties: lower expert id stays
      }
      taken |= 1u << best;
      out_expert[(size_t)row * K + r] = best;
      out_gate[(size_t)row * K + r] = s[best];
    }
  }
}

// ------------------------------------------------------------------------------------------
// CUDA-core contractions: one warp per weight row, RB activation rows at a time.
// ------------------------------------------------------------------------------------------
template <typename T, int RB>
__device__ __forceinline__ void warp_rows_dot(const T* __restrict__ w, const T* __restrict__ x0,
                                              size_t ldx, const int* rows, int nr, int Kdim,
                                              float (&acc)[RB]) {
  constexpr int VN = jk_vec<T>::N;
  const int lane = threadIdx.x & 31;
#pragma unroll
  for (int rb = 0; rb < RB; ++rb) acc[rb] = 0.f;
  for (int k = lane * VN; k < Kdim; k += 32 * VN) {
    float wv[VN];
    jk_vec<T>::load(w + k, wv);
#pragma unroll
    for (int rb = 0; rb < RB; ++rb) {
      if (rb < nr) {
        float xv[VN];
        jk_vec<T>::load(x0 + (size_t)rows[rb] * ldx + k, xv);
#pragma unroll
        for (int i = 0; i < VN; ++i) acc[rb] = fmaf(wv[i], xv[i], acc[rb]);
      }
    }
  }
#pragma unroll
  for (int rb = 0; rb < RB; ++rb) acc[rb] = jk_warp_sum(acc[rb]);
}

// rows routed to expert e, ascending
__device__ __forceinline__ int build_expert_rows(const int32_t* expert, int R, int K, int e,
                                                 int* list, int* count) {
  if (threadIdx.x == 0) {
    int n = 0;
    for (int r = 0; r < R; ++r)
      for (int k = 0; k < K; ++k)
        if (expert[r * K + k] == e) { list[n++] = r; break; }
    *count = n;
  }
  __syncthreads();
  return *count;
}

// h[e, r, i] = SiLU(W_gate[e, i] . x_r) * (W_up[e, i] . x_r) for the rows r routed to expert e
template <typename T>
__global__ void __launch_bounds__(256) k_gateup(
    const T* __restrict__ w_gate, const T* __restrict__ w_up, const T* __restrict__ xn,
    const int32_t* __restrict__ expert, int R, int K, int H, int I, int Rp, T* __restrict__ hbuf) {
  constexpr int RB = 4;
  __shared__ int list[JK_MAX_ROWS];
  __shared__ int count;
  const int e = blockIdx.y;
  const int n = build_expert_rows(expert, R, K, e, list, &count);
  if (n == 0) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  const int rows_per_block = 32;
  const int i0 = blockIdx.x * rows_per_block;
  for (int ii = warp; ii < rows_per_block; ii += nw) {
    const int i = i0 + ii;
    if (i >= I) break;
    const T* wg = w_gate + ((size_t)e * I + i) * H;
    const T* wu = w_up + ((size_t)e * I + i) * H;
    for (int p = 0; p < n; p += RB) {
      const int nr = min(RB, n - p);
      float ag[RB], au[RB];
      warp_rows_dot<T, RB>(wg, xn, H, list + p, nr, H, ag);
      warp_rows_dot<T, RB>(wu, xn, H, list + p, nr, H, au);
      if (lane < nr) {
        float g = 0.f, a = 0.f;
#pragma unroll
        for (int rb = 0; rb < RB; ++rb) if (rb == lane) { g = ag[rb]; a = au[rb]; }
        const float hval = g / (1.f + expf(-g)) * a;
        hbuf[((size_t)e * Rp + list[p + lane]) * I + i] = jk_from_float<T>(hval);
      }
    }
  }
}

// y[e, r, o] = W_down[e, o] . h[e, r]
template <typename T>
__global__ void __launch_bounds__(256) k_down(
    const T* __restrict__ w_down, const T* __restrict__ hbuf, const int32_t* __restrict__ expert,
    int R, int K, int H, int I, int Rp, float* __restrict__ ybuf) {
  constexpr int RB = 4;
  __shared__ int list[JK_MAX_ROWS];
  __shared__ int count;
  const int e = blockIdx.y;
  const int n = build_expert_rows(expert, R, K, e, list, &count);
  if (n == 0) return;
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  const int rows_per_block = 16;
  const int o0 = blockIdx.x * rows_per_block;
  const T* x0 = hbuf + (size_t)e * Rp * I;
  for (int oo = warp; oo < rows_per_block; oo += nw) {
    const int o = o0 + oo;
    if (o >= H) break;
    const T* wd = w_down + ((size_t)e * H + o) * I;
    for (int p = 0; p < n; p += RB) {
      const int nr = min(RB, n - p);
      float acc[RB];
      warp_rows_dot<T, RB>(wd, x0, I, list + p, nr, I, acc);
      if (lane < nr) {
        float v = 0.f;
#pragma unroll
        for (int rb = 0; rb < RB; ++rb) if (rb == lane) v = acc[rb];
        ybuf[((size_t)e * Rp + list[p + lane]) * H + o] = v;
      }
    }
  }
}

// Eq. 3 and the branch features: f = u + sum_r g_r y_r; b_r = g_r y_r (+ u)
// Contrastive mode (Eq. 6-7, K = 2): b_0 = f^moe = g_1 y_1 + g_2 y_2 (+ u), b_1 = f^const =
// beta y_1 - alpha y_2 (+ u).
template <typename T>
__global__ void __launch_bounds__(256) k_branch(
    const T* __restrict__ u, const float* __restrict__ ybuf, const int32_t* __restrict__ expert,
    const float* __restrict__ gate, int K, int H, int Rp, int branch_residual, int head_mode,
    float alpha, float beta, T* __restrict__ bbuf, T* __restrict__ out_feat) {
  const int r = blockIdx.x;
  for (int h = threadIdx.x; h < H; h += blockDim.x) {
    const float uv = jk_to_float(u[(size_t)r * H + h]);
    float f = uv;
    if (head_mode == 1) {
      const float y0 = ybuf[((size_t)expert[r * K] * Rp + r) * H + h];
      const float y1 = ybuf[((size_t)expert[r * K + 1] * Rp + r) * H + h];
      const float g0y = gate[r * K] * y0, g1y = gate[r * K + 1] * y1;
      const float fm = g0y + g1y, fc = beta * y0 - alpha * y1;
      f = (uv + g0y) + g1y;
      bbuf[((size_t)r * K) * H + h] = jk_from_float<T>(branch_residual ? fm + uv : fm);
      bbuf[((size_t)r * K + 1) * H + h] = jk_from_float<T>(branch_residual ? fc + uv : fc);
    } else {
      for (int k = 0; k < K; ++k) {
        const int e = expert[r * K + k];
        const float gy = gate[r * K + k] * ybuf[((size_t)e * Rp + r) * H + h];
        f += gy;
        bbuf[((size_t)r * K + k) * H + h] = jk_from_float<T>(branch_residual ? gy + uv : gy);
      }
    }
    out_feat[(size_t)r * H + h] = jk_from_float<T>(f);
  }
}

// offset of logits row rk = (b*F + f)*K + r when sequences are stride_b elements apart
__host__ __device__ __forceinline__ size_t logit_row_off(int rk, int rows_per_b, long long stride_b,
                                                         int V) {
  return (size_t)(rk / rows_per_b) * (size_t)stride_b + (size_t)(rk % rows_per_b) * V;
}

// logits[rk, v] = b[rk] . W_head[v]   (Eq. 4)
template <typename T>
__global__ void __launch_bounds__(256) k_lmhead(
    const T* __restrict__ lm_head, const T* __restrict__ bbuf, int RK, int H, int V,
    float* __restrict__ logits, int rows_per_b, long long stride_b) {
  constexpr int RB = 8;
  __shared__ int ident[JK_MAX_ROWS * JK_MAX_EXPERTS];
  for (int i = threadIdx.x; i < RK; i += blockDim.x) ident[i] = i;
  __syncthreads();
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, nw = blockDim.x >> 5;
  const int rows_per_block = 32;
  const int v0 = blockIdx.x * rows_per_block;
  for (int vv = warp; vv < rows_per_block; vv += nw) {
    const int v = v0 + vv;
    if (v >= V) break;
    const T* wr = lm_head + (size_t)v * H;
    for (int p = 0; p < RK; p += RB) {
      const int nr = min(RB, RK - p);
      float acc[RB];
      warp_rows_dot<T, RB>(wr, bbuf, H, ident + p, nr, H, acc);
      if (lane < nr) {
        float val = 0.f;
#pragma unroll
        for (int rb = 0; rb < RB; ++rb) if (rb == lane) val = acc[rb];
        logits[logit_row_off(p + lane, rows_per_b, stride_b, V) + v] = val;
      }
    }
  }
}

// ------------------------------------------------------------------------------------------
// Per-expert top-k over the vocabulary: partial pass per 4096-entry chunk, then a merge.
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(JK_TOPK_THREADS) k_topk_partial(
    const float* __restrict__ logits, int rows_per_b, long long stride_b, int V, int k_e,
    int chunks, float* __restrict__ tk_val, int32_t* __restrict__ tk_idx, float* __restrict__ tk_ms) {
  const int chunk = blockIdx.x, row = blockIdx.y;
  const float* lr = logits + logit_row_off(row, rows_per_b, stride_b, V);
  const int base = chunk * JK_TOPK_CHUNK;
  float vals[JK_TOPK_PER];
#pragma unroll
  for (int j = 0; j < JK_TOPK_PER; ++j) {
    const int idx = base + threadIdx.x + j * JK_TOPK_THREADS;
    vals[j] = idx < V ? lr[idx] : -INFINITY;
  }
  jk_topk_chunk_select(vals, base, V, k_e, (size_t)row * chunks + chunk, tk_val, tk_idx, tk_ms);
}

// Merge the chunk partials of every logits row of one sequence, append the children to the
// pool, then pick the next frontier (by score, or from the predefined shape's list).  One block
// per sequence.  In contrastive mode (head_mode 1) the row-1 children hang under the node's best
// row-0 child and only row-0 children can become frontier nodes.
__global__ void __launch_bounds__(1024) k_expand_finish(
    int F, int K, int k_e, int chunks, int width, int head_mode,
    const float* __restrict__ tk_val, const int32_t* __restrict__ tk_idx,
    const float* __restrict__ tk_ms, const float* __restrict__ parent_score,
    const int32_t* __restrict__ parent_gidx, int gidx_base, int slot_base,
    jk_pool pool, float* __restrict__ out_lse, int rows_per_b_lse, long long lse_stride_b,
    int32_t* __restrict__ next_frontier, float* __restrict__ next_parent_score,
    int32_t* __restrict__ next_parent_gidx, const int32_t* __restrict__ static_select,
    int32_t* status) {
  jk_pdl_wait();
  jk_pdl_trigger();
  constexpr int PER_MAX = 16;                   // candidates per lane held in registers
  __shared__ float sc[JK_MAX_POOL];             // cumulative score of every child
  __shared__ float lp[JK_MAX_POOL];             // its log-probability under its own logits row
  __shared__ int tk[JK_MAX_POOL];
  const int b = blockIdx.x;
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5, nw = blockDim.x >> 5;
  const int rows = F * K;
  const size_t pb = (size_t)b * pool.stride_b;
  const int nc = chunks * k_e;
  // One warp per logits row.  PER = candidates a lane holds (the chunks' partial winners); the
  // selection loop is instantiated for the smallest PER that covers them.
  auto merge_row = [&](auto per_tag, int lr) {
    constexpr int PER = decltype(per_tag)::value;
    const size_t row = (size_t)b * rows + lr;
    float cv[PER];
    int ci[PER];
#pragma unroll
    for (int j = 0; j < PER; ++j) {
      const int c = lane + j * 32;
      cv[j] = c < nc ? tk_val[row * nc + c] : -INFINITY;
      ci[j] = c < nc ? tk_idx[row * nc + c] : INT_MAX;
    }
    // log-sum-exp over the chunk statistics
    float m = -INFINITY;
    for (int c = lane; c < chunks; c += 32) m = fmaxf(m, tk_ms[(row * chunks + c) * 2]);
    m = jk_warp_max(m);
    float s = 0.f;
    for (int c = lane; c < chunks; c += 32)
      s += tk_ms[(row * chunks + c) * 2 + 1] * expf(tk_ms[(row * chunks + c) * 2] - m);
    s = jk_warp_sum(s);
    const float lse = m + logf(s);
    if (out_lse && lane == 0)
      out_lse[(size_t)b * (size_t)lse_stride_b + lr] = lse;
    unsigned taken = 0u;
    for (int it = 0; it < k_e; ++it) {
      float bv = -INFINITY;
      int bi = INT_MAX, bj = -1;
#pragma unroll
      for (int j = 0; j < PER; ++j)
        if (!(taken & (1u << j)) && jk_better(cv[j], ci[j], bv, bi)) { bv = cv[j]; bi = ci[j]; bj = j; }
      float wv = bv;
      int wi = bi;
      jk_warp_argbest(wv, wi);
      if (wi == bi && bj >= 0 && wi != INT_MAX) taken |= 1u << bj;
      if (lane == 0) {
        const int flat = lr * k_e + it;
        lp[flat] = wv - lse;
        tk[flat] = wi;
      }
    }
  };
  for (int lr = warp; lr < rows; lr += nw) {
    if (nc <= 64) merge_row(std::integral_constant<int, 2>{}, lr);
    else if (nc <= 128) merge_row(std::integral_constant<int, 4>{}, lr);
    else if (nc <= 256) merge_row(std::integral_constant<int, 8>{}, lr);
    else merge_row(std::integral_constant<int, PER_MAX>{}, lr);
  }
  __syncthreads();
  const int n = rows * k_e;
  const bool last_pass = width <= 0;
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    const int lr = i / k_e, f = lr / K, r = lr % K;
    const float ps = parent_score[(size_t)b * F + f];
    int pg = parent_gidx[(size_t)b * F + f];
    float base = ps;
    if (head_mode == 1 && r == 1) {
      const int best0 = (f * K) * k_e;                      // the node's best row-0 child
      base = ps + lp[best0];
      pg = gidx_base + best0;
    }
    float score = base + lp[i];
    if (head_mode == 1 && r == 1 && !last_pass) score = -INFINITY;
    const int g = gidx_base + i;
    pool.tok[pb + g] = tk[i];
    pool.score[pb + g] = score;
    pool.parent[pb + g] = pg;
    pool.qslot[pb + g] = -1;
    pool.branch[pb + g] = r;
    sc[i] = score;
  }
  __syncthreads();
  if (width <= 0 || !next_frontier) return;
  const int n_sel = head_mode == 1 ? F * k_e : n;           // children that may be expanded
  const int wsel = min(width, n_sel);
  if (static_select) {
    for (int i = threadIdx.x; i < wsel; i += blockDim.x) {
      int idx = static_select[i];
      if (idx < 0 || idx >= n || (head_mode == 1 && (idx / k_e) % K == 1)) {
        jk_set_status(status, JK_ERR_BOUNDS);
        idx = 0;
      }
      next_frontier[(size_t)b * wsel + i] = idx;
      next_parent_score[(size_t)b * wsel + i] = sc[idx];
      next_parent_gidx[(size_t)b * wsel + i] = gidx_base + idx;
      pool.qslot[pb + gidx_base + idx] = slot_base + F + i;
    }
    return;
  }
  for (int i = threadIdx.x; i < n; i += blockDim.x) {
    if (head_mode == 1 && (i / k_e) % K == 1) continue;
    const float v = sc[i];
    int rank = 0;
    for (int j = 0; j < n; ++j) {
      if (head_mode == 1 && (j / k_e) % K == 1) continue;
      rank += jk_better(sc[j], j, v, i) ? 1 : 0;
    }
    if (rank < wsel) {
      next_frontier[(size_t)b * wsel + rank] = i;
      next_parent_score[(size_t)b * wsel + rank] = v;
      next_parent_gidx[(size_t)b * wsel + rank] = gidx_base + i;
      pool.qslot[pb + gidx_base + i] = slot_base + F + rank;
    }
  }
}

// ------------------------------------------------------------------------------------------
// Tree finalisation: top (M-1) of the pool, ascending generation order, ancestor bitsets.
//
// Which candidates are kept is the rank of each under (score descending, generation index
// ascending).  Ranking all of a large pool against all of it is the long part of the kernel, so a
// pool of more than FIN_SMALL candidates is first cut down: it is divided into FIN_CHUNKS runs,
// the (M-1)-th largest of the runs' maxima is a lower bound T of the (M-1)-th largest score (the
// M-1 maxima at or above it are M-1 different candidates), everything below T is dropped unseen
// and only the candidates at or above T are ranked against one another.  If fewer than M-1 runs
// are occupied, if more than FIN_CAND candidates reach T (many equal scores) or if a score is
// NaN, every candidate is ranked against the whole pool as in a small one; the result is the
// same set either way.
// ------------------------------------------------------------------------------------------
#define FIN_SMALL 256
#define FIN_CHUNKS 128
#define FIN_CAND 256
__global__ void __launch_bounds__(1024) k_tree_finalize(
    jk_pool pool, int pool_n, const int32_t* __restrict__ root_tok, int M,
    int32_t* __restrict__ tok, int32_t* __restrict__ parent, int32_t* __restrict__ depth,
    int32_t* __restrict__ branch, int32_t* __restrict__ qslot, unsigned long long* __restrict__ anc,
    const int32_t* __restrict__ static_keep, int32_t* status) {
  jk_pdl_wait();
  jk_pdl_trigger();
  __shared__ float sc[JK_MAX_POOL];
  __shared__ short newid[JK_MAX_POOL];      // 0 = dropped, else node index
  __shared__ unsigned char keepf[JK_MAX_POOL];
  __shared__ int par_s[JK_MAX_TREE];
  __shared__ int wsum[32];
  __shared__ int keep_s[JK_MAX_TREE];
  __shared__ float cmax[FIN_CHUNKS];
  __shared__ int cand[FIN_CAND];
  __shared__ float s_thr;
  __shared__ int s_ncand, s_full;
  const int b = blockIdx.x;
  const size_t pb = (size_t)b * pool.stride_b;
  const int t = threadIdx.x, nt = blockDim.x, lane = t & 31, warp = t >> 5;
  const int m1 = M - 1;
  const int cs = (pool_n + FIN_CHUNKS - 1) / FIN_CHUNKS;      // candidates per run
  const bool cut = !static_keep && nt == FIN_CHUNKS * 8 && pool_n > FIN_SMALL &&
                   (pool_n + cs - 1) / cs >= m1 && m1 >= 1;
  if (t == 0) { s_ncand = 0; s_full = cut ? 0 : 1; s_thr = 0.f; }
  __syncthreads();
  for (int g = t; g < pool_n; g += nt) {
    const float v = pool.score[pb + g];
    sc[g] = v;
    keepf[g] = 0;
    if (v != v) s_full = 1;
  }
  if (static_keep && t < m1) {
    // the predefined shape's list: ascending generation indices inside the pool
    const int g = static_keep[t];
    const int prev = t > 0 ? static_keep[t - 1] : -1;
    if (g < 0 || g >= pool_n || g <= prev) jk_set_status(status, JK_ERR_BOUNDS);
    keep_s[t] = g;
  }
  __syncthreads();
  if (static_keep) {
    if (t < m1) {
      const int g = keep_s[t];
      if (g >= 0 && g < pool_n) keepf[g] = 1;
    }
  } else {
    if (cut) {
      // the runs' maxima, then the (M-1)-th largest of them: 8 threads rank one maximum
      for (int c = t; c < FIN_CHUNKS; c += nt) {
        float m = -INFINITY;
        for (int g = c * cs; g < min(pool_n, (c + 1) * cs); ++g) m = fmaxf(m, sc[g]);
        cmax[c] = m;
      }
      __syncthreads();
      {
        const int c = t >> 3, part = t & 7;       // 1024 threads = FIN_CHUNKS * 8
        int rank = 0;
        if (c < FIN_CHUNKS) {
          const float v = cmax[c];
          for (int j = part; j < FIN_CHUNKS; j += 8) rank += jk_better(cmax[j], j, v, c) ? 1 : 0;
        }
        rank += __shfl_xor_sync(0xffffffffu, rank, 1);
        rank += __shfl_xor_sync(0xffffffffu, rank, 2);
        rank += __shfl_xor_sync(0xffffffffu, rank, 4);
        if (c < FIN_CHUNKS && part == 0 && rank == m1 - 1) s_thr = cmax[c];
      }
      __syncthreads();
      const float thr = s_thr;
      for (int g = t; g < pool_n; g += nt) {
        if (sc[g] >= thr) {
          const int pos = atomicAdd(&s_ncand, 1);
          if (pos < FIN_CAND) cand[pos] = g;
        }
      }
      __syncthreads();
      if (s_ncand > FIN_CAND) s_full = 1;         // (every thread that sees it stores the same)
      __syncthreads();
    }
    if (!s_full) {
      // rank the candidates at or above the bound against one another: 4 threads each
      const int nc = s_ncand;
      const int i = t >> 2, part = t & 3;         // 1024 threads = FIN_CAND * 4
      int rank = 0, g = 0;
      if (i < nc) {
        g = cand[i];
        const float v = sc[g];
        for (int j = part; j < nc; j += 4) {
          const int gj = cand[j];
          rank += jk_better(sc[gj], gj, v, g) ? 1 : 0;
        }
      }
      rank += __shfl_xor_sync(0xffffffffu, rank, 1);
      rank += __shfl_xor_sync(0xffffffffu, rank, 2);
      if (i < nc && part == 0 && rank < m1) keepf[g] = 1;
    } else {
      // every candidate against the whole pool; a candidate is shared by as many threads (a
      // power of two up to 32) as the block has to spare
      int tpe = 1;
      while (tpe < 32 && pool_n * tpe * 2 <= nt) tpe <<= 1;
      for (int g0 = 0; g0 < pool_n; g0 += nt / tpe) {
        const int g = g0 + t / tpe, part = t % tpe;
        int rank = 0;
        if (g < pool_n) {
          const float v = sc[g];
          for (int j = part; j < pool_n; j += tpe) rank += jk_better(sc[j], j, v, g) ? 1 : 0;
        }
        for (int o = 1; o < tpe; o <<= 1) rank += __shfl_xor_sync(0xffffffffu, rank, o);
        if (g < pool_n && part == 0 && rank < m1) keepf[g] = 1;
      }
    }
  }
  __syncthreads();
  // each thread owns a contiguous slice so that the prefix sum runs in generation order
  const int per = (pool_n + nt - 1) / nt;
  const int g0 = t * per, g1 = min(pool_n, g0 + per);
  int cnt = 0;
  for (int g = g0; g < g1; ++g) cnt += keepf[g];
  int incl = cnt;
#pragma unroll
  for (int off = 1; off < 32; off <<= 1) {
    const int y = __shfl_up_sync(0xffffffffu, incl, off);
    if (lane >= off) incl += y;
  }
  if (lane == 31) wsum[warp] = incl;
  __syncthreads();
  if (warp == 0) {
    const int w = lane < (nt >> 5) ? wsum[lane] : 0;
    int wi = w;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const int y = __shfl_up_sync(0xffffffffu, wi, off);
      if (lane >= off) wi += y;
    }
    wsum[lane] = wi - w;                     // kept candidates before this warp
  }
  __syncthreads();
  int id = 1 + wsum[warp] + incl - cnt;
  for (int g = g0; g < g1; ++g) newid[g] = keepf[g] ? (short)(id++) : (short)0;
  __syncthreads();
  const size_t ob = (size_t)b * M;
  if (t == 0) {
    tok[ob] = root_tok[b];
    parent[ob] = -1;
    depth[ob] = 0;
    branch[ob] = 0;
    qslot[ob] = 0;
    par_s[0] = -1;
  }
  for (int g = g0; g < g1; ++g) {
    const int i = newid[g];
    if (!i) continue;
    const int pg = pool.parent[pb + g];
    int p = 0;
    if (pg >= 0) {
      p = (pg < pool_n) ? newid[pg] : 0;
      if (p == 0 || p >= i) { jk_set_status(status, JK_ERR_BOUNDS); p = 0; }
    }
    tok[ob + i] = pool.tok[pb + g];
    parent[ob + i] = p;
    par_s[i] = p;
    branch[ob + i] = pool.branch[pb + g];
    qslot[ob + i] = pool.qslot[pb + g];
  }
  __syncthreads();
  if (t < M) {
    unsigned long long lo = 0ull, hi = 0ull;
    int d = -1, c = t;
    for (int guard = 0; c >= 0 && guard <= JK_MAX_TREE; ++guard) {
      if (c < 64) lo |= 1ull << c; else hi |= 1ull << (c - 64);
      ++d;
      c = par_s[c];
    }
    depth[ob + t] = d;
    anc[(ob + t) * 2] = lo;
    anc[(ob + t) * 2 + 1] = hi;
  }
}

// ------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------
template <typename T>
static int expand_impl(jk_ctx* ctx, cudaStream_t st, const jk_draft_weights* w, int B, int F,
                       int width, const void* u, const float* parent_score,
                       const int32_t* parent_gidx, int gidx_base, int slot_base, float* out_probs,
                       int32_t* out_expert, float* out_gate, const jk_pool* pool, float* out_lse,
                       void* out_feat, float* out_logits, int64_t logits_stride_b,
                       int32_t* next_frontier, float* next_parent_score,
                       int32_t* next_parent_gidx, const int32_t* static_select) {
  const jk_config& c = ctx->cfg;
  const jk_ws_layout& L = ctx->lay;
  const int R = B * F, K = c.top_k, RK = R * K, H = c.hidden, I = c.inter, V = c.vocab;
  const int Rp = L.rows_pad;
  char* ws = ctx->ws;
  T* xn = (T*)(ws + L.xn);
  T* hbuf = (T*)(ws + L.hbuf);
  float* ybuf = (float*)(ws + L.ybuf);
  T* bbuf = (T*)(ws + L.bbuf);
  float* logits = out_logits ? out_logits : (float*)(ws + L.logits);
  const int rows_per_b = F * K;
  const long long lsb = (out_logits && logits_stride_b) ? logits_stride_b : (long long)rows_per_b * V;

  JK_PROF(ctx, st, JK_ST_ROUTER);
  jk_launch_pdl(k_router<T>, dim3(R), dim3(512), 0, st, (const T*)u, (const T*)w->router, (const T*)w->norm_weight, H,
                                 c.n_experts, K, c.rms_eps, c.use_pre_norm, xn, out_probs,
                                 out_expert, out_gate);
  JK_LAUNCH_CHECK(ctx);
  const bool tc = ctx->tensor_path && c.dtype == JK_BF16 && jk_tc_available(ctx);
  if (tc) {
    int rc = jk_tc_ffn(ctx, st, w, R, out_expert, out_gate, u, out_feat);
    if (rc != JK_OK) return rc;
    rc = jk_tc_lm_head(ctx, st, w, RK, out_logits, rows_per_b, lsb);
    if (rc != JK_OK) return rc;
  } else {
    JK_PROF(ctx, st, JK_ST_GATEUP);
    k_gateup<T><<<dim3((I + 31) / 32, c.n_experts), 256, 0, st>>>(
        (const T*)w->w_gate, (const T*)w->w_up, xn, out_expert, R, K, H, I, Rp, hbuf);
    JK_LAUNCH_CHECK(ctx);
    JK_PROF(ctx, st, JK_ST_DOWN);
    k_down<T><<<dim3((H + 15) / 16, c.n_experts), 256, 0, st>>>(
        (const T*)w->w_down, hbuf, out_expert, R, K, H, I, Rp, ybuf);
    JK_LAUNCH_CHECK(ctx);
    JK_PROF(ctx, st, JK_ST_BRANCH);
    k_branch<T><<<R, 256, 0, st>>>((const T*)u, ybuf, out_expert, out_gate, K, H, Rp,
                                   c.branch_residual, c.head_mode, c.contrast_alpha,
                                   c.contrast_beta, bbuf, (T*)out_feat);
    JK_LAUNCH_CHECK(ctx);
    JK_PROF(ctx, st, JK_ST_LMHEAD);
    k_lmhead<T><<<(V + 31) / 32, 256, 0, st>>>((const T*)w->lm_head, bbuf, RK, H, V, logits,
                                               rows_per_b, lsb);
    JK_LAUNCH_CHECK(ctx);
    JK_PROF(ctx, st, JK_ST_TOPK);
    k_topk_partial<<<dim3(L.topk_chunks, RK), JK_TOPK_THREADS, 0, st>>>(
        logits, rows_per_b, lsb, V, c.k_per_expert, L.topk_chunks, (float*)(ws + L.tk_val),
        (int32_t*)(ws + L.tk_idx), (float*)(ws + L.tk_ms));
    JK_LAUNCH_CHECK(ctx);
  }
  JK_PROF(ctx, st, JK_ST_FINISH);
  // out_lse follows the per-sequence layout of out_logits: rows slot_base.. of a [B, S, K]
  // array when the logits go to rows slot_base.. of a [B, S, K, V] one
  const long long lse_sb = (out_logits && logits_stride_b) ? logits_stride_b / V : rows_per_b;
  jk_launch_pdl(k_expand_finish, dim3(B), dim3(1024), 0, st, F, K, c.k_per_expert, L.topk_chunks, width,
                                     c.head_mode, (const float*)(ws + L.tk_val),
                                     (const int32_t*)(ws + L.tk_idx),
                                     (const float*)(ws + L.tk_ms), parent_score, parent_gidx,
                                     gidx_base, slot_base, *pool, out_lse, rows_per_b, lse_sb,
                                     next_frontier, next_parent_score, next_parent_gidx,
                                     static_select, (int32_t*)(ws + L.status));
  JK_LAUNCH_CHECK(ctx);
  return JK_OK;
}

extern "C" int jk_draft_expand(jk_ctx* ctx, void* stream, const jk_draft_weights* w,
                               int32_t batch, int32_t n_frontier, int32_t width, const void* u,
                               const float* parent_score, const int32_t* parent_gidx,
                               int32_t gidx_base, int32_t slot_base, float* out_probs,
                               int32_t* out_expert, float* out_gate, const jk_pool* pool,
                               float* out_lse, void* out_feat, float* out_logits,
                               int64_t logits_stride_b, int32_t* next_frontier,
                               float* next_parent_score, int32_t* next_parent_gidx,
                               const int32_t* static_select) {
  if (!ctx || !w || !u || !parent_score || !parent_gidx || !out_expert || !out_gate || !pool ||
      !out_feat)
    return JK_ERR_NULL;
  if (!w->router || !w->w_gate || !w->w_up || !w->w_down || !w->lm_head) return JK_ERR_NULL;
  if (!pool->tok || !pool->score || !pool->parent || !pool->qslot || !pool->branch)
    return JK_ERR_NULL;
  if (width > 0 && (!next_frontier || !next_parent_score || !next_parent_gidx)) return JK_ERR_NULL;
  const jk_config& c = ctx->cfg;
  if (batch < 1 || n_frontier < 1 || width < 0 || gidx_base < 0 || slot_base < 0)
    return JK_ERR_SHAPE;
  if (batch > c.max_batch || n_frontier > c.max_frontier) return JK_ERR_CAPACITY;
  const int n_cand = n_frontier * c.top_k * c.k_per_expert;
  if (n_cand > JK_MAX_POOL) return JK_ERR_SHAPE;
  if (pool->stride_b < (int64_t)gidx_base + n_cand) return JK_ERR_SHAPE;
  if (logits_stride_b < 0 || logits_stride_b % 4 || logits_stride_b % c.vocab ||
      (logits_stride_b && logits_stride_b < (int64_t)n_frontier * c.top_k * c.vocab))
    return JK_ERR_SHAPE;
  if (static_select && width <= 0) return JK_ERR_SHAPE;
  const void* ptrs[] = {u, w->router, w->w_gate, w->w_up, w->w_down, w->lm_head, w->norm_weight,
                        out_feat, out_logits};
  for (const void* p : ptrs)
    if (p && !jk_aligned16(p)) return JK_ERR_ALIGN;
  if (!ctx->ws) return JK_ERR_WORKSPACE;
  int rc = jk_ensure_device_info(ctx);
  if (rc != JK_OK) return rc;
  cudaStream_t st = (cudaStream_t)stream;
  if (c.dtype == JK_BF16)
    return expand_impl<__nv_bfloat16>(ctx, st, w, batch, n_frontier, width, u, parent_score,
                                      parent_gidx, gidx_base, slot_base, out_probs, out_expert,
                                      out_gate, pool, out_lse, out_feat, out_logits,
                                      logits_stride_b, next_frontier, next_parent_score,
                                      next_parent_gidx, static_select);
  return expand_impl<float>(ctx, st, w, batch, n_frontier, width, u, parent_score, parent_gidx,
                            gidx_base, slot_base, out_probs, out_expert, out_gate, pool, out_lse,
                            out_feat, out_logits, logits_stride_b, next_frontier,
                            next_parent_score, next_parent_gidx, static_select);
}

extern "C" int jk_tree_finalize(jk_ctx* ctx, void* stream, int32_t batch, const jk_pool* pool,
                                int32_t pool_n, const int32_t* root_tok, int32_t tree_size,
                                int32_t* tok, int32_t* parent, int32_t* depth, int32_t* branch,
                                int32_t* qslot, uint64_t* anc, const int32_t* static_keep) {
  if (!ctx || !pool || !root_tok || !tok || !parent || !depth || !branch || !qslot || !anc)
    return JK_ERR_NULL;
  if (!pool->tok || !pool->score || !pool->parent || !pool->qslot || !pool->branch)
    return JK_ERR_NULL;
  if (batch < 1 || tree_size < 1 || pool_n < 0) return JK_ERR_SHAPE;
  if (batch > ctx->cfg.max_batch || tree_size > ctx->cfg.max_tree) return JK_ERR_CAPACITY;
  if (pool_n > JK_MAX_POOL || pool_n < tree_size - 1 || pool->stride_b < pool_n)
    return JK_ERR_SHAPE;
  if (!ctx->ws) return JK_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  JK_PROF(ctx, st, JK_ST_FINALIZE);
  jk_launch_pdl(k_tree_finalize, dim3(batch), dim3(1024), 0, st, 
      *pool, pool_n, root_tok, tree_size, tok, parent, depth, branch, qslot,
      (unsigned long long*)anc, static_keep, (int32_t*)(ctx->ws + ctx->lay.status));
  JK_LAUNCH_CHECK(ctx);
  return JK_OK;
}
