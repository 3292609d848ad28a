// jk_accept_and_compact: per-node statistics of the target logits, the acceptance walk (greedy
// path match or speculative sampling, arXiv 2502.06282 Sec. 2.1 steps 2-3) and the compaction of
// the accepted nodes' KV rows.
#include <limits.h>
#include <math.h>

#include "jk_common.cuh"

// ------------------------------------------------------------------------------------------
// Row statistics: top-1 token (ties: lower id), max and sum exp((x - max)/T).  One block per
// row, one pass over it: every thread keeps a running (max, argmax, sum relative to that max)
// over batches of vectors that are all requested before the first one is used, and the block
// brings the partial sums onto the row maximum at the end.
// ------------------------------------------------------------------------------------------
template <typename TL>
__device__ __forceinline__ void row_stats_row(const TL* __restrict__ r, size_t row, int V,
                                              float inv_t, int32_t* __restrict__ rs_arg,
                                              float* __restrict__ rs_max,
                                              float* __restrict__ rs_sum, float* red, float* wv,
                                              int* wi) {
  constexpr int VN = jk_vec<TL>::N;
  constexpr int U = 32 / VN;                       // vectors in flight per thread (32 values)
  float bv = -INFINITY, s = 0.f;
  int bi = INT_MAX;
  const int vmain = V / VN * VN;
  const int step = blockDim.x * VN;
  for (int k0 = threadIdx.x * VN; k0 < vmain; k0 += step * U) {
    float v[U][VN];
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int k = k0 + u * step;
      if (k < vmain) {
        jk_vec<TL>::load(r + k, v[u]);
      } else {
#pragma unroll
        for (int i = 0; i < VN; ++i) v[u][i] = -INFINITY;
      }
    }
    float cv = bv;
    int ci = bi;
#pragma unroll
    for (int u = 0; u < U; ++u) {
      const int k = k0 + u * step;
      if (k < vmain) {                             // the padding takes no part in the argmax
#pragma unroll
        for (int i = 0; i < VN; ++i)
          if (jk_better(v[u][i], k + i, cv, ci)) { cv = v[u][i]; ci = k + i; }
      }
    }
    if (cv > bv) s *= expf((bv - cv) * inv_t);     // bv = -inf: s is 0 and stays 0
    bv = cv;
    bi = ci;
    if (bv > -INFINITY) {
#pragma unroll
      for (int u = 0; u < U; ++u)
#pragma unroll
        for (int i = 0; i < VN; ++i) s += expf((v[u][i] - bv) * inv_t);
    }
  }
  for (int k = vmain + threadIdx.x; k < V; k += blockDim.x) {
    const float v = jk_to_float(r[k]);
    if (jk_better(v, k, bv, bi)) {
      if (v > bv) s *= expf((bv - v) * inv_t);
      bv = v;
      bi = k;
    }
    if (bv > -INFINITY) s += expf((v - bv) * inv_t);
  }
  const float own = bv;
#pragma unroll
  for (int o = 16; o > 0; o >>= 1) {
    const float ov = __shfl_xor_sync(0xffffffffu, bv, o);
    const int oi = __shfl_xor_sync(0xffffffffu, bi, o);
    if (jk_better(ov, oi, bv, bi)) { bv = ov; bi = oi; }
  }
  const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
  if (lane == 0) { wv[warp] = bv; wi[warp] = bi; }
  __syncthreads();
  float mx = wv[0];
  int am = wi[0];
  for (int w = 1; w < (int)(blockDim.x >> 5); ++w)
    if (jk_better(wv[w], wi[w], mx, am)) { mx = wv[w]; am = wi[w]; }
  s = own > -INFINITY ? s * expf((own - mx) * inv_t) : 0.f;
  s = jk_block_sum(s, red);
  if (threadIdx.x == 0) { rs_arg[row] = am; rs_max[row] = mx; rs_sum[row] = s; }
}

// Blocks 0 .. rows-1 take the target rows, the rest (sampling mode) the stored draft rows: one
// launch for both sets.
template <typename TL>
__global__ void __launch_bounds__(512) k_row_stats(
    const TL* __restrict__ tl, int rows, const float* __restrict__ dl, int V, float inv_t,
    int32_t* __restrict__ rs_arg, float* __restrict__ rs_max, float* __restrict__ rs_sum,
    int32_t* __restrict__ qs_arg, float* __restrict__ qs_max, float* __restrict__ qs_sum) {
  jk_pdl_wait();      // (its dependent is released when this kernel's CTAs exit: measured faster)
  __shared__ float red[33];
  __shared__ float wv[16];
  __shared__ int wi[16];
  if ((int)blockIdx.x < rows) {
    const size_t row = blockIdx.x;
    row_stats_row<TL>(tl + row * V, row, V, inv_t, rs_arg, rs_max, rs_sum, red, wv, wi);
  } else {
    const size_t row = blockIdx.x - rows;
    row_stats_row<float>(dl + row * V, row, V, inv_t, qs_arg, qs_max, qs_sum, red, wv, wi);
  }
}

// ------------------------------------------------------------------------------------------
// The walk.  One block per sequence.
// ------------------------------------------------------------------------------------------
struct walk_out {
  int32_t* kv_len;
  int32_t* p_old;
  int32_t* n_acc;
  int32_t* acc_idx;
  int32_t* acc_tok;
  int32_t* bonus_tok;
};

__device__ __forceinline__ void walk_finish(const walk_out& o, int b, int max_depth, int n,
                                            const int* path, const int* path_tok, int bonus,
                                            int cache_rows, int M, int32_t* status) {
  // thread 0 only
  const int P = o.kv_len[b];
  o.p_old[b] = P;
  o.n_acc[b] = n;
  for (int j = 0; j < max_depth; ++j) {
    o.acc_idx[(size_t)b * max_depth + j] = j < n ? path[j] : -1;
    o.acc_tok[(size_t)b * max_depth + j] = j < n ? path_tok[j] : -1;
  }
  o.bonus_tok[b] = bonus;
  if (P < 0 || P + M > cache_rows) jk_set_status(status, JK_ERR_BOUNDS);
  o.kv_len[b] = P + 1 + n;
}

__global__ void __launch_bounds__(128) k_walk_greedy(
    int M, int max_depth, int V, const int32_t* __restrict__ tok,
    const int32_t* __restrict__ parent, const int32_t* __restrict__ rs_arg, walk_out o,
    int cache_rows, int32_t* status) {
  jk_pdl_wait();      // (its dependent is released when this kernel's CTAs exit: measured faster)
  __shared__ int s_next;
  __shared__ int path[16], path_tok[16];
  const int b = blockIdx.x;
  const int t = threadIdx.x;                         // one thread per tree node
  int cur = 0, n = 0;
  for (int level = 0; level < max_depth; ++level) {
    const int want = rs_arg[(size_t)b * M + cur];
    if (t == 0) s_next = INT_MAX;
    __syncthreads();
    if (t < M && t > 0 && parent[(size_t)b * M + t] == cur && tok[(size_t)b * M + t] == want)
      atomicMin(&s_next, t);                         // first matching child in child order
    __syncthreads();
    const int nxt = s_next;
    __syncthreads();
    if (nxt == INT_MAX) break;
    if (t == 0) { path[n] = nxt; path_tok[n] = want; }
    ++n;
    cur = nxt;
  }
  __syncthreads();
  if (t == 0)
    walk_finish(o, b, max_depth, n, path, path_tok, rs_arg[(size_t)b * M + cur], cache_rows, M,
                status);
}

// Sampling walk.  A thread-block cluster of WALK_CLUSTER blocks per sequence; block r of the cluster
// owns the vocabulary range [r * Vc, (r + 1) * Vc).  Every block follows the whole walk (tree
// bookkeeping, the accept / reject decisions, the path) from the same values, so all of them take
// the same branches and meet at the same cluster barriers; only the passes over the vocabulary
// (the residual after a rejection, the prefix sums of the bonus draw) are divided, and their
// per-block sums are exchanged through the blocks' shared memories and added in block order, which
// gives every block the same bits.  p and the q_r start "lazy" (read from the logits with the
// row's precomputed max and sum) and are written out to pbuf/qbuf the first time a rejection
// changes them; a value another block wrote is read from L2 after the barrier that followed the
// write.  pbuf and every q_r buffer exist twice and a rejection writes the copy it does not read:
// a block that is already in the next pass cannot overwrite the entry a slower block still has to
// read for its decision (the copy written two passes later is only reached through a barrier the
// slower block has passed after that read).  Every pass works on 4 entries per thread per step
// (16-byte loads; the host checks V % 4 == 0 for this mode).
#define WALK_CLUSTER 8                 // portable cluster size
#define WALK_THREADS 512
struct walk_vec4 { float v[4]; };

__device__ __forceinline__ uint32_t walk_cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ uint32_t walk_cluster_size() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
  return r;
}
// Release-arrive / acquire-wait on the cluster's barrier: orders the shared-memory stores into
// other blocks and the global stores made before it against the reads after it.
__device__ __forceinline__ void walk_cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// store four words into the variable at `p` (16-byte aligned) of block `rank` of the cluster
__device__ __forceinline__ void walk_st_remote(const void* p, uint32_t rank, uint32_t a, uint32_t c,
                                               uint32_t d, uint32_t e) {
  uint32_t addr;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;"
               : "=r"(addr) : "r"((uint32_t)__cvta_generic_to_shared(p)), "r"(rank));
  asm volatile("st.shared::cluster.v4.u32 [%0], {%1, %2, %3, %4};"
               ::"r"(addr), "r"(a), "r"(c), "r"(d), "r"(e) : "memory");
}

__global__ void __launch_bounds__(WALK_THREADS) k_walk_sample(
    int M, int max_depth, int V, int K, int n_slots, float inv_t,
    const void* __restrict__ tl_raw, int tl_bf16, const int32_t* __restrict__ tok,
    const int32_t* __restrict__ parent, const int32_t* __restrict__ depth,
    const int32_t* __restrict__ branch, const int32_t* __restrict__ qslot,
    const float* __restrict__ draft_logits, const float* __restrict__ u_accept,
    const float* __restrict__ u_bonus, const float* __restrict__ rs_max,
    const float* __restrict__ rs_sum, const float* __restrict__ qs_max,
    const float* __restrict__ qs_sum, float* pbuf_all, float* qbuf_all,
    walk_out o, int cache_rows, int32_t* status) {
  jk_pdl_wait();      // (its dependent is released when this kernel's CTAs exit: measured faster)
  __shared__ float red[66];
  __shared__ __align__(16) uint32_t xs[2][WALK_CLUSTER][4];  // [exchange parity][block][4 words]
  __shared__ int s_parent[JK_MAX_TREE], s_tok[JK_MAX_TREE], s_branch[JK_MAX_TREE];
  __shared__ int s_qslot[JK_MAX_TREE], s_depth[JK_MAX_TREE];
  __shared__ float s_uacc[JK_MAX_TREE], s_rmax[JK_MAX_TREE], s_risum[JK_MAX_TREE];
  __shared__ float s_qmax[JK_MAX_EXPERTS], s_qisum[JK_MAX_EXPERTS], s_qscale[JK_MAX_EXPERTS];
  __shared__ float s_fwd[2];          // the next child's token in this pass: new p, new q_r
  __shared__ int kids[JK_MAX_TREE];
  __shared__ int n_kids;
  __shared__ int path[16], path_tok[16];
  __shared__ int s_decision;
  __shared__ int s_found;
  const int C = (int)walk_cluster_size(), rank = (int)walk_cluster_rank();
  const int b = blockIdx.x / C, t = threadIdx.x, nt = blockDim.x;
  const int lane = t & 31, warp = t >> 5, nw = nt >> 5;
  const int Vc = ((V / 4 + C - 1) / C) * 4;            // this block's share of the vocabulary
  const int vlo = min(V, rank * Vc), vhi = min(V, vlo + Vc);
  float* pb2 = pbuf_all + (size_t)b * 2 * V;        // the two copies of p, V apart
  const float* tlf = (const float*)tl_raw;
  const __nv_bfloat16* tlh = (const __nv_bfloat16*)tl_raw;
  if (t < M) {                        // everything the walk reads per node, once
    const size_t i = (size_t)b * M + t;
    s_parent[t] = parent[i];
    s_tok[t] = tok[i];
    s_branch[t] = branch[i];
    s_qslot[t] = qslot[i];
    s_depth[t] = depth[i];
    s_uacc[t] = u_accept[i];
    s_rmax[t] = rs_max[i];
    s_risum[t] = 1.f / rs_sum[i];
  }
  __syncthreads();
  int cur = 0, n = 0;
  int xround = 0;                     // exchanges so far: picks the half of xs[] to use
  bool p_mat = false;                 // p lives in pbuf (scaled by p_scale) instead of the logits
  int p_par = 0;                      // which copy of pbuf holds it
  unsigned q_par = 0;                 // bit r: which copy of branch r's buffer is current
  unsigned q_mat = 0;                 // bit r: q_r lives in its buffer (scaled by s_qscale[r])
  float p_scale = 1.f, p_max = 0.f, p_isum = 1.f;
  size_t tl_row = 0;
  auto p_at = [&](int v) -> float {                // any v: another block may have written it
    if (p_mat) return __ldcg(pb2 + (size_t)p_par * V + v) * p_scale;
    const float x = tl_bf16 ? __bfloat162float(tlh[tl_row * V + v]) : tlf[tl_row * V + v];
    return expf((x - p_max) * inv_t) * p_isum;
  };
  auto p_at4 = [&](int v) -> walk_vec4 {           // v % 4 == 0, inside this block's range
    walk_vec4 r;
    if (p_mat) {
      const float4 x = *reinterpret_cast<const float4*>(pb2 + (size_t)p_par * V + v);
      r.v[0] = x.x * p_scale; r.v[1] = x.y * p_scale; r.v[2] = x.z * p_scale; r.v[3] = x.w * p_scale;
    } else {
      float x[4];
      if (tl_bf16) {
        const uint2 h = *reinterpret_cast<const uint2*>(tlh + tl_row * V + v);
        x[0] = __uint_as_float(h.x << 16); x[1] = __uint_as_float(h.x & 0xffff0000u);
        x[2] = __uint_as_float(h.y << 16); x[3] = __uint_as_float(h.y & 0xffff0000u);
      } else {
        const float4 f = *reinterpret_cast<const float4*>(tlf + tl_row * V + v);
        x[0] = f.x; x[1] = f.y; x[2] = f.z; x[3] = f.w;
      }
#pragma unroll
      for (int i = 0; i < 4; ++i) r.v[i] = expf((x[i] - p_max) * inv_t) * p_isum;
    }
    return r;
  };
  // branch r's draft probability of token v as it stands (any v)
  auto q_at = [&](int r, int v, const float* dl_r, const float* qcur_r) -> float {
    if ((q_mat >> r) & 1u) return __ldcg(qcur_r + v) * s_qscale[r];
    return expf((dl_r[v] - s_qmax[r]) * inv_t) * s_qisum[r];
  };
  // Every block hands its four words to all blocks of the cluster; after the barrier xs[half][j]
  // holds block j's words in every block.  Two halves: a block that is one exchange ahead writes
  // the other half, and it cannot get two ahead without everybody passing the barrier between.
  auto exchange = [&](uint32_t a, uint32_t c, uint32_t d, uint32_t e) -> int {
    const int half = xround & 1;
    ++xround;
    if (t < C) walk_st_remote(&xs[half][rank][0], (uint32_t)t, a, c, d, e);
    walk_cluster_sync();
    return half;
  };
  while (true) {
    tl_row = (size_t)b * M + cur;
    p_mat = false;
    q_mat = 0;
    p_max = s_rmax[cur];
    p_isum = s_risum[cur];
    const int slot = s_qslot[cur];
    const bool expandable = n < max_depth && slot >= 0 && slot < n_slots;
    // children of cur in child order (= ascending node index); the branches' (max, 1/sum)
    if (warp == 0) {
      int c = 0;
      for (int i0 = 0; i0 < M; i0 += 32) {
        const int i = i0 + lane;
        const bool k = i >= 1 && i < M && s_parent[i] == cur;
        const unsigned m = __ballot_sync(0xffffffffu, k);
        if (k) kids[c + __popc(m & ((1u << lane) - 1u))] = i;
        c += __popc(m);
      }
      if (lane == 0) n_kids = c;
    } else if (warp == 1 && lane < K && expandable) {
      const size_t qrow = ((size_t)b * n_slots + slot) * K + lane;
      s_qmax[lane] = qs_max[qrow];
      s_qisum[lane] = 1.f / qs_sum[qrow];
      s_qscale[lane] = 1.f;
    }
    __syncthreads();
    const int nk = n_kids;
    int accepted = -1;
    if (nk > 0 && expandable) {
      bool fwd = false;               // this child's decision came with the last pass's sums
      float fwd_p = 0.f, fwd_q = 0.f;
      for (int ci = 0; ci < nk; ++ci) {
        const int c = kids[ci];
        const int x = s_tok[c];
        const int r = s_branch[c];
        if (x < 0 || x >= V || r < 0 || r >= K) {
          if (t == 0) jk_set_status(status, JK_ERR_BOUNDS);
          break;
        }
        const float* dl = draft_logits + (((size_t)b * n_slots + slot) * K + r) * V;
        float* qb2 = qbuf_all + ((size_t)b * K + r) * 2 * V;
        const float* qcur = qb2 + (size_t)((q_par >> r) & 1u) * V;
        float* qnew = qb2 + (size_t)(((q_par >> r) & 1u) ^ 1u) * V;
        float* pnew = pb2 + (size_t)(p_par ^ 1) * V;
        int dec;
        if (fwd) {                    // the same arithmetic on the same values in every thread
          const float px = fwd_p, qx = fwd_q;
          dec = qx > 0.f ? (s_uacc[c] < fminf(1.f, px / qx)) : (px > 0.f);
        } else {
          if (t == 0) {
            const float px = p_at(x);
            const float qx = q_at(r, x, dl, qcur);
            s_decision = qx > 0.f ? (s_uacc[c] < fminf(1.f, px / qx)) : (px > 0.f);
          }
          __syncthreads();            // (the next write of s_decision lies behind another barrier)
          dec = s_decision;
        }
        if (dec) { accepted = c; break; }
        // rejection: p <- max(0, p - q_r) (normalised through p_scale); q_r[x] <- 0, renormalised.
        // The next child's token (xn, branch rn) is watched for in the pass: its new p and, when
        // it comes from the same branch, its new q_r travel with the sums, so that its decision
        // needs no further load.  Another branch's q is not touched by this pass: read it now.
        const bool qm = (q_mat >> r) & 1u;
        const float qmx = s_qmax[r], qis = s_qisum[r], qsc = s_qscale[r];
        int xn = -1, rn = -1;
        if (ci + 1 < nk) {
          xn = s_tok[kids[ci + 1]];
          rn = s_branch[kids[ci + 1]];
          if (xn < 0 || xn >= V || rn < 0 || rn >= K) xn = -1;
        }
        float q_other = 0.f;
        if (xn >= 0 && rn != r) {
          const float* dln = draft_logits + (((size_t)b * n_slots + slot) * K + rn) * V;
          const float* qcn = qbuf_all + (((size_t)b * K + rn) * 2 + ((q_par >> rn) & 1u)) * V;
          q_other = q_at(rn, xn, dln, qcn);
        }
        if (t == 0) { s_fwd[0] = 0.f; s_fwd[1] = 0.f; }
        __syncthreads();
        float sp = 0.f, sq = 0.f;
#pragma unroll 2
        for (int v = vlo + t * 4; v < vhi; v += nt * 4) {
          const walk_vec4 pv = p_at4(v);
          float qv[4];
          const float4 qr = *reinterpret_cast<const float4*>((qm ? qcur : dl) + v);
          if (qm) {
            qv[0] = qr.x * qsc; qv[1] = qr.y * qsc; qv[2] = qr.z * qsc; qv[3] = qr.w * qsc;
          } else {
            qv[0] = expf((qr.x - qmx) * inv_t) * qis; qv[1] = expf((qr.y - qmx) * inv_t) * qis;
            qv[2] = expf((qr.z - qmx) * inv_t) * qis; qv[3] = expf((qr.w - qmx) * inv_t) * qis;
          }
          float res[4], qn[4];
#pragma unroll
          for (int i = 0; i < 4; ++i) {
            res[i] = fmaxf(0.f, pv.v[i] - qv[i]);
            qn[i] = (v + i == x) ? 0.f : qv[i];
            sp += res[i];
            sq += qn[i];
            if (v + i == xn) { s_fwd[0] = res[i]; s_fwd[1] = qn[i]; }
          }
          *reinterpret_cast<float4*>(pnew + v) = make_float4(res[0], res[1], res[2], res[3]);
          *reinterpret_cast<float4*>(qnew + v) = make_float4(qn[0], qn[1], qn[2], qn[3]);
        }
        // sums over the block in one round, then over the cluster in block order
        sp = jk_warp_sum(sp);
        sq = jk_warp_sum(sq);
        if (lane == 0) { red[warp] = sp; red[33 + warp] = sq; }
        __syncthreads();
        if (warp == 0) {
          float a = lane < nw ? red[lane] : 0.f, y = lane < nw ? red[33 + lane] : 0.f;
          a = jk_warp_sum(a);
          y = jk_warp_sum(y);
          if (lane == 0) { red[32] = a; red[65] = y; }
        }
        __syncthreads();
        const int half = exchange(__float_as_uint(red[32]), __float_as_uint(red[65]),
                                  __float_as_uint(s_fwd[0]), __float_as_uint(s_fwd[1]));
        sp = 0.f;
        sq = 0.f;
        for (int j = 0; j < C; ++j) {
          sp += __uint_as_float(xs[half][j][0]);
          sq += __uint_as_float(xs[half][j][1]);
        }
        q_mat |= 1u << r;
        q_par ^= 1u << r;
        const float qsc_new = sq > 0.f ? 1.f / sq : 1.f;
        s_qscale[r] = qsc_new;        // every thread stores the same bits
        if (!(sp > 0.f)) {            // residual vanished: keep the node's own p for the bonus
          p_mat = false;
          break;
        }
        p_mat = true;
        p_par ^= 1;
        p_scale = 1.f / sp;
        fwd = xn >= 0;
        if (fwd) {
          const int owner = xn / Vc;  // the block whose range holds xn
          fwd_p = __uint_as_float(xs[half][owner][2]) * p_scale;
          fwd_q = rn == r ? __uint_as_float(xs[half][owner][3]) * qsc_new : q_other;
        }
      }
    }
    if (accepted >= 0) {
      if (t == 0) { path[n] = accepted; path_tok[n] = s_tok[accepted]; }
      ++n;
      cur = accepted;
      __syncthreads();
      continue;
    }
    // bonus token: inverse CDF of the current p at u_bonus[depth]; every thread owns a contiguous
    // run of `per` entries (a multiple of 4) of its block's range
    const int dcur = s_depth[cur];
    const float ub = u_bonus[(size_t)b * (max_depth + 1) + min(max(dcur, 0), max_depth)];
    const int per = ((Vc + nt - 1) / nt + 3) / 4 * 4;
    const int v0 = min(vhi, vlo + t * per), v1 = min(vhi, v0 + per);
    float loc = 0.f;
    for (int v = v0; v < v1; v += 4) {
      const walk_vec4 pv = p_at4(v);
      loc += (pv.v[0] + pv.v[1]) + (pv.v[2] + pv.v[3]);
    }
    // inclusive scan of the runs' sums: shuffles inside a warp, the warp totals by warp 0, the
    // blocks' totals in block order
    float incl = loc;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
      const float y = __shfl_up_sync(0xffffffffu, incl, off);
      if (lane >= off) incl += y;
    }
    if (t == 0) { s_found = INT_MAX; s_decision = -1; }
    __syncthreads();                       // red[] is free (the last block sum has been read)
    if (lane == 31) red[warp] = incl;
    __syncthreads();
    if (warp == 0) {
      const float w = lane < nw ? red[lane] : 0.f;
      float wi = w;
#pragma unroll
      for (int off = 1; off < 32; off <<= 1) {
        const float y = __shfl_up_sync(0xffffffffu, wi, off);
        if (lane >= off) wi += y;
      }
      red[33 + lane] = wi - w;             // what lies before this warp
      if (lane == 31) red[32] = wi;
    }
    __syncthreads();
    float base = 0.f, total = 0.f;         // what lies before this block; the whole sum
    {
      const int half = exchange(__float_as_uint(red[32]), 0u, 0u, 0u);
      for (int j = 0; j < C; ++j) {
        if (j == rank) base = total;
        total += __uint_as_float(xs[half][j][0]);
      }
    }
    incl += red[33 + warp] + base;
    const float thr = ub * total;
    // `before` is exactly the previous thread's inclusive value (for a block's first thread the
    // previous block's last, which is set to the sum of the blocks' totals up to it), so the
    // runs' intervals [before, incl) join without gaps and some run claims every threshold below
    // the total.
    if (t == nt - 1) incl = base + red[32];
    __syncthreads();                       // red[0..nw) was read above by warp 0 only
    if (lane == 31) red[warp] = incl;
    __syncthreads();
    const float up = __shfl_up_sync(0xffffffffu, incl, 1);
    const float before = lane ? up : (warp ? red[warp - 1] : base);
    // The crossing lies in this thread's run; rounding can let more than one run claim the
    // threshold (the scan need not be monotone to the last bit) and the minimum keeps the first.
    // The block's last token with p > 0 rides along: it is the answer when no run of any block
    // passed the threshold.
    const bool mine = before <= thr && incl > thr;
    if (mine) {
      float run = before;
      int last_pos = -1;
      for (int v = v0; v < v1; ++v) {
        const float pv = p_at(v);
        run += pv;
        if (pv > 0.f) last_pos = v;
        if (run > thr) { last_pos = v; break; }
      }
      // The run was first added pairwise and now one by one: rounding can leave the sequential
      // sum at or below the threshold.  The draw then belongs to this run's last token with
      // p > 0 (the pairwise sum passed the threshold, so the run has one).
      if (last_pos >= 0) atomicMin(&s_found, last_pos);
    }
    __syncthreads();
    int found;
    {
      const int half0 = exchange((uint32_t)s_found, 0u, 0u, 0u);
      found = INT_MAX;
      for (int j = 0; j < C; ++j) found = min(found, (int)xs[half0][j][0]);
    }
    if (found == INT_MAX) {
      for (int v = v1 - 1; v >= v0; --v)
        if (p_at(v) > 0.f) { atomicMax(&s_decision, v); break; }
      __syncthreads();
      const int half1 = exchange((uint32_t)s_decision, 0u, 0u, 0u);
      found = -1;
      for (int j = 0; j < C; ++j) found = max(found, (int)xs[half1][j][0]);
    }
    if (t == 0 && rank == 0)
      walk_finish(o, b, max_depth, n, path, path_tok, max(found, 0), cache_rows, M, status);
    return;
  }
}

// ------------------------------------------------------------------------------------------
// KV compaction: row P + acc_idx[j] -> row P + 1 + j.  One block per (cache, sequence, kv head);
// all source rows are loaded before any row is stored (a destination can be a later source).
// ------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(256) k_compact(
    void* const* __restrict__ k_caches, void* const* __restrict__ v_caches, int n_layers,
    long long stride_b, long long stride_h, int row_bytes, int cache_rows, int max_depth, int M,
    const int32_t* __restrict__ p_old, const int32_t* __restrict__ n_acc,
    const int32_t* __restrict__ acc_idx, int elem_size) {
  jk_pdl_wait();      // (its dependent is released when this kernel's CTAs exit: measured faster)
  const int which = blockIdx.z;                  // layer*2 + (0 = K, 1 = V)
  const int b = blockIdx.y, kvh = blockIdx.x;
  const int n = n_acc[b];
  const int P = p_old[b];
  if (n <= 0 || P < 0 || P + M > cache_rows) return;
  char* base = (char*)((which & 1) ? v_caches[which >> 1] : k_caches[which >> 1]) +
               ((size_t)b * stride_b + (size_t)kvh * stride_h) * elem_size;
  const int chunks = row_bytes / 16;
  const int total = n * chunks;
  uint4 held[2];                                 // up to 2 chunks per thread (16 rows * 32 chunks)
  int cnt = 0;
  for (int idx = threadIdx.x; idx < total && cnt < 2; idx += blockDim.x, ++cnt) {
    const int j = idx / chunks, c = idx % chunks;
    const int a = acc_idx[(size_t)b * max_depth + j];
    held[cnt] = *reinterpret_cast<const uint4*>(base + (size_t)(P + a) * row_bytes + c * 16);
  }
  __syncthreads();
  cnt = 0;
  for (int idx = threadIdx.x; idx < total && cnt < 2; idx += blockDim.x, ++cnt) {
    const int j = idx / chunks, c = idx % chunks;
    *reinterpret_cast<uint4*>(base + (size_t)(P + 1 + j) * row_bytes + c * 16) = held[cnt];
  }
}

extern "C" int jk_accept_and_compact(
    jk_ctx* ctx, void* stream, int32_t batch, int32_t tree_size, int32_t mode, float temperature,
    const void* target_logits, int32_t tl_dtype, const int32_t* tok, const int32_t* parent,
    const int32_t* depth, const int32_t* branch, const int32_t* qslot, const float* draft_logits,
    int32_t n_slots, const float* u_accept, const float* u_bonus, int32_t n_layers,
    void* const* k_caches, void* const* v_caches, int64_t cache_stride_b, int64_t cache_stride_h,
    int32_t cache_rows, int32_t* kv_len, int32_t* n_acc, int32_t* acc_idx, int32_t* acc_tok,
    int32_t* bonus_tok) {
  if (!ctx || !target_logits || !tok || !parent || !depth || !branch || !qslot || !kv_len ||
      !n_acc || !acc_idx || !acc_tok || !bonus_tok)
    return JK_ERR_NULL;
  if (mode != 0 && mode != 1) return JK_ERR_SHAPE;
  if (mode == 1 && (!draft_logits || !u_accept || !u_bonus)) return JK_ERR_NULL;
  if (mode == 1 && (!(temperature > 0.f) || n_slots < 1)) return JK_ERR_SHAPE;
  if (mode == 1 && n_slots > ctx->cfg.max_depth * ctx->cfg.max_frontier) return JK_ERR_CAPACITY;
  if (mode == 1 && ctx->cfg.vocab % 4) return JK_ERR_ALIGN;      // 16-byte rows of draft logits
  if (n_layers < 0 || (n_layers > 0 && (!k_caches || !v_caches))) return JK_ERR_NULL;
  if (tl_dtype != JK_F32 && tl_dtype != JK_BF16) return JK_ERR_DTYPE;
  const jk_config& c = ctx->cfg;
  if (batch < 1 || tree_size < 1 || cache_rows < tree_size) return JK_ERR_SHAPE;
  if (batch > c.max_batch || tree_size > c.max_tree) return JK_ERR_CAPACITY;
  if (!jk_aligned16(target_logits) || (draft_logits && !jk_aligned16(draft_logits)))
    return JK_ERR_ALIGN;
  const int es = jk_elem_size(c.dtype);
  const int row_bytes = c.head_dim * es;
  if (n_layers > 0 && ((cache_stride_b * es) % 16 || (cache_stride_h * es) % 16))
    return JK_ERR_ALIGN;
  // the vectorised row scan needs 16-byte aligned rows
  if (((size_t)c.vocab * jk_elem_size(tl_dtype)) % 16) return JK_ERR_ALIGN;
  if (!ctx->ws) return JK_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  const jk_ws_layout& L = ctx->lay;
  char* ws = ctx->ws;
  int32_t* rs_arg = (int32_t*)(ws + L.rs_arg);
  float* rs_max = (float*)(ws + L.rs_max);
  float* rs_sum = (float*)(ws + L.rs_sum);
  int32_t* status = (int32_t*)(ws + L.status);
  const float inv_t = mode == 1 ? 1.f / temperature : 1.f;
  const int rows = batch * tree_size;
  // max and sum of exp of every stored draft row too (sampling), before the serial walk
  const int q_rows = mode == 1 ? batch * n_slots * c.top_k : 0;
  JK_PROF(ctx, st, JK_ST_ROWSTATS);
  if (tl_dtype == JK_BF16)
    jk_launch_pdl(k_row_stats<__nv_bfloat16>, dim3(rows + q_rows), dim3(512), 0, st,
                  (const __nv_bfloat16*)target_logits, rows, draft_logits, c.vocab, inv_t, rs_arg,
                  rs_max, rs_sum, (int32_t*)(ws + L.qs_arg), (float*)(ws + L.qs_max),
                  (float*)(ws + L.qs_sum));
  else
    jk_launch_pdl(k_row_stats<float>, dim3(rows + q_rows), dim3(512), 0, st,
                  (const float*)target_logits, rows, draft_logits, c.vocab, inv_t, rs_arg, rs_max,
                  rs_sum, (int32_t*)(ws + L.qs_arg), (float*)(ws + L.qs_max),
                  (float*)(ws + L.qs_sum));
  JK_LAUNCH_CHECK(ctx);
  walk_out o{kv_len, (int32_t*)(ws + L.p_old), n_acc, acc_idx, acc_tok, bonus_tok};
  JK_PROF(ctx, st, JK_ST_WALK);
  if (mode == 0) {
    jk_launch_pdl(k_walk_greedy, dim3(batch), dim3(128), 0, st, tree_size, c.max_depth, c.vocab, tok, parent, rs_arg, o,
                                         cache_rows, status);
  } else {
    jk_launch_pdl_cluster(k_walk_sample, dim3(batch * WALK_CLUSTER), dim3(WALK_THREADS), WALK_CLUSTER, 0, st,
        tree_size, c.max_depth, c.vocab, c.top_k, n_slots, inv_t, target_logits,
        tl_dtype == JK_BF16, tok, parent, depth, branch, qslot, draft_logits, u_accept, u_bonus,
        rs_max, rs_sum, (const float*)(ws + L.qs_max), (const float*)(ws + L.qs_sum),
        (float*)(ws + L.pbuf), (float*)(ws + L.qbuf), o, cache_rows, status);
  }
  JK_LAUNCH_CHECK(ctx);
  if (n_layers > 0) {
    JK_PROF(ctx, st, JK_ST_COMPACT);
    jk_launch_pdl(k_compact, dim3(c.n_kv_heads, batch, 2 * n_layers), dim3(256), 0, st, 
        k_caches, v_caches, n_layers, cache_stride_b, cache_stride_h, row_bytes, cache_rows,
        c.max_depth, tree_size, (const int32_t*)(ws + L.p_old), n_acc, acc_idx, es);
    JK_LAUNCH_CHECK(ctx);
  }
  return JK_OK;
}
