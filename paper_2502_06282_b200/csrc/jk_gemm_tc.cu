// Tensor-core path of the draft layer's dense contractions (expert gate/up, expert down, LM head;
// arXiv 2502.06282 Eq. 3-4) for bf16 on sm_100a.
//
// All three are "skinny" products  out[n, m] = sum_k W[m, k] * X[n, k]  with millions of weight
// rows m but only 2..256 activation rows n, so they are bound by streaming W from HBM once.  One
// persistent kernel serves them:
//   - the weight matrix sits on the 128-row M side of tcgen05.mma, the activation rows on N
//     (padded to a multiple of 16), accumulators in tensor memory;
//   - work is cut into items: a run of k steps (a chunk, at least 128 KB of weights) of one 128-row
//     weight tile; the CTAs take items from a global counter one after the other, so an SM that
//     gets less of the memory bandwidth at some moment simply ends up with fewer items;
//   - a producer thread feeds a ring of shared-memory stages with TMA (128B swizzle), one thread
//     issues the MMAs, four warps drain finished accumulators to fp32 partial tiles in global
//     memory, one per item at a place that depends on the item alone; a small second kernel adds
//     the partials of each tile in chunk order (no atomics on data, bitwise reproducible
//     whichever CTA computed what) and applies the epilogue: SiLU * up; residual, gates and
//     branch features; or the LM head's per-chunk top-k statistics.
// Every wait on an mbarrier is bounded: after ~2 s it records JK_ERR_TIMEOUT in the status word,
// and the CTA drains its copies, frees its tensor memory and returns.
#include <cuda.h>
#include <stdlib.h>

#include "jk_common.cuh"
#include "jk_tcgen05.cuh"
#include "jk_topk.cuh"

#define TC_TILE_M 128
#define TC_BOX_K 64                  // one TMA box: 64 bf16 = the 128-byte swizzle span
// A stage holds KB boxes side by side along K.  Two (256 contiguous bytes of every weight row per
// stage) stream measurably faster than one; with many activation rows a two-box stage would leave
// too few stages in the ring, and one box is used.
#define TC_KB_WIDE_MIN_STAGES 4
#define TC_THREADS 192               // warp 0: TMA producer, warp 1: MMA issuer, warps 2-5: epilogue
#define TC_MAX_GROUPS 16
#define TC_MAX_STAGES 12
#define TC_SMEM_BUDGET (220 * 1024)

struct tc_params {
  int n_groups_max;                  // groups before filtering by active experts
  int group_expert[TC_MAX_GROUPS];   // expert whose activity gates the group, -1 = always on
  int group_amap[TC_MAX_GROUPS];     // which A tensor map (0 or 1)
  int group_arow0[TC_MAX_GROUPS];    // first row of the group in its A tensor map
  int group_brow0[TC_MAX_GROUPS];    // first row of the group's activations in the B tensor map
  int tiles_per_group;               // ceil(M_rows / 128)
  int kdim;                          // K
  int kb;                            // TMA boxes per stage along K (1 or 2)
  int kt;                            // k steps of a tile: ceil(K / (64 * kb))
  int ch;                            // k steps of a chunk
  int n_chunks;                      // chunks of a tile: ceil(kt / ch)
  int n_pad;                         // activation rows, multiple of 16
  int stages;
  int R, K_top, n_experts;           // to derive the active experts from `expert`
  int tmem_cols;
  int prefetch;                      // 1: the producer streams weight tiles before the grid-dependency wait
  int* counter;                      // next work item of this launch (zero when the kernel starts)
};

// Instruction descriptor: bf16 x bf16 -> fp32, both operands K-major, M = 128, N = n
__host__ __device__ inline uint32_t instr_desc_bf16(int n) {
  uint32_t d = 0;
  d |= 1u << 4;                      // accumulator fp32
  d |= 1u << 7;                      // A bf16
  d |= 1u << 10;                     // B bf16
  d |= (uint32_t)(n >> 3) << 17;     // N
  d |= (uint32_t)(TC_TILE_M >> 4) << 24;
  return d;
}

// ---------------------------------------------------------------------------------------------
// Work partition shared by the GEMM kernel and the fix-up kernels.  A work item is one chunk of
// the k steps of one weight tile of one active group; item i = (group, tile, chunk) in that
// order.  Its partial tile lands in slot i of the partial buffer, whichever CTA computed it, so
// the sum the fix-up kernels form (chunks in ascending order) does not depend on the dealing.
// ---------------------------------------------------------------------------------------------
struct tc_plan {
  int n_groups;                      // active groups
  int group_src[TC_MAX_GROUPS];      // index into the parameter arrays
  int total_items;
};

__device__ __forceinline__ void tc_make_plan(const tc_params& p, const int32_t* expert,
                                             tc_plan* plan) {
  // called by one whole warp; lane 0 writes the plan
  unsigned active = 0;
  for (int i = threadIdx.x & 31; i < p.R * p.K_top; i += 32) {
    const int e = __ldcg(expert + i);      // (past the L1: some callers read it before their wait)
    if (e >= 0 && e < p.n_experts) active |= 1u << e;
  }
  active = __reduce_or_sync(0xffffffffu, active);
  if ((threadIdx.x & 31) != 0) return;
  int n = 0;
  for (int g = 0; g < p.n_groups_max; ++g) {
    const int e = p.group_expert[g];
    if (e < 0 || (active >> e) & 1u) plan->group_src[n++] = g;
  }
  plan->n_groups = n;
  plan->total_items = n * p.tiles_per_group * p.n_chunks;
}

#define TC_ITEM_Q 4                  // item ids in flight between the producer and the epilogue warps
#define TC_FLAG_FIRST 1
#define TC_FLAG_LAST 2
#define TC_FLAG_END 4

struct __align__(1024) tc_smem_tail {
  uint64_t full[TC_MAX_STAGES];
  uint64_t empty[TC_MAX_STAGES];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint64_t iq_full[TC_ITEM_Q];
  uint64_t iq_empty[TC_ITEM_Q];
  uint32_t tmem_base;
  int abort_flag;
  int st_flag[TC_MAX_STAGES];        // first / last k step of its item, or the end of the work
  int q_item[TC_ITEM_Q];
  tc_plan plan;
};

// Work is dealt dynamically: a CTA asks a global counter for its next item.  The SMs do not get
// equal shares of the memory bandwidth at every moment (measured: with equal static shares the
// slowest CTA of a 110 us launch ended 20 us after the fastest), and this way a slower SM simply
// takes fewer items.
template <int TC_KB>
__global__ void __launch_bounds__(TC_THREADS, 1) k_tc_gemm(
    const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_a1,
    const __grid_constant__ CUtensorMap map_b, const tc_params p, const int32_t* __restrict__ expert,
    float* __restrict__ partial, int32_t* __restrict__ status) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  constexpr int TC_TILE_K = TC_KB * TC_BOX_K;
  const int stage_bytes = TC_TILE_M * TC_TILE_K * 2 + p.n_pad * TC_TILE_K * 2;
  tc_smem_tail& T = *reinterpret_cast<tc_smem_tail*>(smem + (size_t)p.stages * stage_bytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &T.abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(&T.full[s], 1); mbar_init(&T.empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&T.acc_full[a], 1); mbar_init(&T.acc_empty[a], 4); }
    for (int i = 0; i < TC_ITEM_Q; ++i) { mbar_init(&T.iq_full[i], 1); mbar_init(&T.iq_empty[i], 4); }
    T.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  // The plan reads the router's output.  Without prefetch the preceding kernel may be the
  // router itself, so wait for it first; with prefetch the router is at least two kernels back
  // and therefore complete (a kernel releases its successor only after its own wait).
  if (!p.prefetch) jk_pdl_wait();
  if (warp == 0) {
    __syncwarp();
    tc_make_plan(p, expert, &T.plan);
  }
  if (warp == 1) {
    tmem_alloc(&T.tmem_base, (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = T.tmem_base;
  const int total = T.plan.total_items;
  // (the whole producer warp skips this wait when it prefetches: lanes of that warp waiting here
  // would hold back the lane that issues the copies; its other lanes touch no global memory)
  if (!(p.prefetch && warp == 0)) {
    jk_pdl_wait();
    jk_pdl_trigger();
  }

  if (warp == 0 && lane == 0) {
    // ------------------------------------------------------------------ TMA producer
    bool ok = true;
    const uint64_t pol = l2_policy_evict_first();   // weight tiles are read once per call
    int s = 0, issued = 0, qn = 0;
    uint32_t ph = 0;
    // With prefetch the weights of the first item start streaming before the grid-dependency
    // wait (they do not depend on the kernel before); the activation tiles of those stages
    // follow once that kernel is done.
    bool waited = !p.prefetch;
    int pend_s[TC_MAX_STAGES], pend_k[TC_MAX_STAGES], pend_brow = 0, n_pend = 0;
    auto settle = [&]() {
      jk_pdl_wait();
      jk_pdl_trigger();
      for (int i = 0; i < n_pend; ++i) {
        unsigned char* sb = smem + (size_t)pend_s[i] * stage_bytes + TC_TILE_M * TC_TILE_K * 2;
#pragma unroll
        for (int kb = 0; kb < TC_KB; ++kb)
          tma_load_2d(sb + kb * (p.n_pad * TC_BOX_K * 2), &map_b,
                      pend_k[i] * TC_TILE_K + kb * TC_BOX_K, pend_brow, &T.full[pend_s[i]]);
      }
      n_pend = 0;
      waited = true;
    };
    // A CTA's first item is its own number (no trip to the counter before the first copies are
    // on their way); further items come from the counter, which counts from the grid size up.
    bool first_item = true;
    while (ok) {
      const int item = first_item ? (int)blockIdx.x : (int)gridDim.x + atomicAdd(p.counter, 1);
      first_item = false;
      if (item >= total) break;
      // the epilogue warps learn the item (its partial slot) through a small queue
      const int qs = qn % TC_ITEM_Q;
      if (qn >= TC_ITEM_Q)
        ok = mbar_wait(&T.iq_empty[qs], (uint32_t)(qn / TC_ITEM_Q - 1) & 1u, abort_flag, status);
      if (!ok) break;
      T.q_item[qs] = item;
      mbar_arrive(&T.iq_full[qs]);
      ++qn;
      const int c = item % p.n_chunks, tt = item / p.n_chunks;
      const int t = tt % p.tiles_per_group, g = T.plan.group_src[tt / p.tiles_per_group];
      const CUtensorMap* ma = p.group_amap[g] ? &map_a1 : &map_a0;
      const int arow = p.group_arow0[g] + t * TC_TILE_M, brow = p.group_brow0[g];
      const int k0 = c * p.ch, k1 = min(p.kt, k0 + p.ch);
      for (int k = k0; k < k1 && ok; ++k) {
        if (issued >= p.stages) ok = mbar_wait(&T.empty[s], ph ^ 1u, abort_flag, status);
        if (!ok) break;
        unsigned char* sa = smem + (size_t)s * stage_bytes;
        unsigned char* sb = sa + TC_TILE_M * TC_TILE_K * 2;
        T.st_flag[s] = (k == k0 ? TC_FLAG_FIRST : 0) | (k == k1 - 1 ? TC_FLAG_LAST : 0);
        mbar_expect_tx(&T.full[s], (uint32_t)stage_bytes);   // (an arrive: releases the flag too)
#pragma unroll
        for (int kb = 0; kb < TC_KB; ++kb)
          tma_load_2d_hint(sa + kb * (TC_TILE_M * TC_BOX_K * 2), ma, k * TC_TILE_K + kb * TC_BOX_K,
                           arow, &T.full[s], pol);
        if (waited) {
#pragma unroll
          for (int kb = 0; kb < TC_KB; ++kb)
            tma_load_2d(sb + kb * (p.n_pad * TC_BOX_K * 2), &map_b, k * TC_TILE_K + kb * TC_BOX_K,
                        brow, &T.full[s]);
        } else {
          pend_s[n_pend] = s; pend_k[n_pend] = k; pend_brow = brow; ++n_pend;
        }
        ++issued;
        if (++s == p.stages) { s = 0; ph ^= 1u; }
        if (!waited && (issued == p.stages || k == k1 - 1)) settle();
      }
    }
    if (!waited) settle();
    if (ok) {
      // the end of the work, for the epilogue warps and for the MMA thread
      const int qs = qn % TC_ITEM_Q;
      if (qn >= TC_ITEM_Q)
        ok = mbar_wait(&T.iq_empty[qs], (uint32_t)(qn / TC_ITEM_Q - 1) & 1u, abort_flag, status);
      if (ok) {
        T.q_item[qs] = -1;
        mbar_arrive(&T.iq_full[qs]);
        if (issued >= p.stages) ok = mbar_wait(&T.empty[s], ph ^ 1u, abort_flag, status);
      }
      if (ok) {
        T.st_flag[s] = TC_FLAG_END;
        mbar_arrive(&T.full[s]);
      }
    }
    if (!ok) {
      // gave up: let the copies already in flight land before the CTA's memory goes away
      const int first = issued > p.stages ? issued - p.stages : 0;
      for (int i = first; i < issued; ++i) {
        const unsigned long long t0 = global_ns();
        while (!mbar_try_wait(&T.full[i % p.stages], (uint32_t)(i / p.stages) & 1u))
          if (global_ns() - t0 > TC_WAIT_NS) break;
      }
    }
  } else if (warp == 1 && lane == 0) {
    // ------------------------------------------------------------------ MMA issuer
    const uint32_t idesc = instr_desc_bf16(p.n_pad);
    int seg = 0, s = 0, acc = 0;
    uint32_t fph = 0;
    bool ok = true, first = true;
    uint32_t d_addr = tmem_base;
    while (ok) {
      ok = mbar_wait(&T.full[s], fph, abort_flag, status);
      if (!ok) break;
      const int flag = T.st_flag[s];
      if (flag & TC_FLAG_END) break;
      if (flag & TC_FLAG_FIRST) {
        acc = seg & 1;
        if (seg >= 2)
          ok = mbar_wait(&T.acc_empty[acc], ((uint32_t)(seg >> 1) & 1u) ^ 1u, abort_flag, status);
        if (!ok) break;
        d_addr = tmem_base + (uint32_t)(acc * p.n_pad);
        first = true;
      }
      tc_fence_after();
      const uint32_t a_addr = smem_u32(smem + (size_t)s * stage_bytes);
      const uint32_t b_addr = a_addr + TC_TILE_M * TC_TILE_K * 2;
#pragma unroll
      for (int kb = 0; kb < TC_KB; ++kb) {
        const uint64_t da = smem_desc_sw128(a_addr + kb * (TC_TILE_M * TC_BOX_K * 2));
        const uint64_t db = smem_desc_sw128(b_addr + kb * (p.n_pad * TC_BOX_K * 2));
#pragma unroll
        for (int k = 0; k < TC_BOX_K / 16; ++k) {
          // 16 bf16 = 32 bytes further along K inside the swizzled row: +2 in the address field
          tc_mma_bf16(d_addr, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc,
                      (first && kb == 0 && k == 0) ? 0u : 1u);
        }
      }
      first = false;
      tc_commit(&T.empty[s]);          // the stage is free once these MMAs have read it
      if (flag & TC_FLAG_LAST) {
        tc_commit(&T.acc_full[acc]);
        ++seg;
      }
      if (++s == p.stages) { s = 0; fph ^= 1u; }
    }
  } else if (warp >= 2) {
    // ------------------------------------------------------------------ epilogue
    const int quarter = warp & 3;        // the TMEM lanes this warp may read: 32*quarter .. +31
    const int m = quarter * 32 + lane;
    int seg = 0, qn = 0;
    bool ok = true;
    while (ok) {
      const int qs = qn % TC_ITEM_Q;
      ok = mbar_wait(&T.iq_full[qs], (uint32_t)(qn / TC_ITEM_Q) & 1u, abort_flag, status);
      ok = __all_sync(0xffffffffu, ok);
      if (!ok) break;
      const int item = T.q_item[qs];
      __syncwarp();
      if (lane == 0) mbar_arrive(&T.iq_empty[qs]);
      ++qn;
      if (item < 0) break;
      const int acc = seg & 1;
      ok = mbar_wait(&T.acc_full[acc], (uint32_t)(seg >> 1) & 1u, abort_flag, status);
      ok = __all_sync(0xffffffffu, ok);          // the TMEM loads below need the whole warp
      if (!ok) break;
      tc_fence_after();
      float* dst = partial + ((size_t)item * p.n_pad) * TC_TILE_M + m;
      const uint32_t t_addr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(acc * p.n_pad);
      for (int c = 0; c < p.n_pad; c += 16) {
        uint32_t r[16];
        tmem_ld16(t_addr + (uint32_t)c, r);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 16; ++j) dst[(size_t)(c + j) * TC_TILE_M] = __uint_as_float(r[j]);
      }
      tc_fence_before();
      __syncwarp();
      if (lane == 0) mbar_arrive(&T.acc_empty[acc]);
      ++seg;
    }
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
  }
}

// ---------------------------------------------------------------------------------------------
// Fix-up kernels: every output element is the sum of the partial tiles of its tile's chunks,
// added in ascending chunk order (fixed order: bitwise reproducible), followed by the epilogue
// of the contraction.  The first thread of each also puts the launch's item counter back to zero.
// ---------------------------------------------------------------------------------------------
// tile = (index of the group among the active ones) * tiles_per_group + tile of the group
__device__ __forceinline__ float tc_tile_sum(const float* __restrict__ partial, const tc_params& p,
                                             long long tile, int n, int m) {
  const float* src = partial + (((size_t)tile * p.n_chunks) * p.n_pad + n) * TC_TILE_M + m;
  float acc = 0.f;
  for (int c = 0; c < p.n_chunks; ++c) acc += src[(size_t)c * p.n_pad * TC_TILE_M];
  return acc;
}
// NV such sums at once: the loads of two chunks of all NV sums are in flight together (a loop
// per sum would pay one trip to the L2 per chunk and sum, one after the other); every sum still
// adds its chunks in ascending order.  tiles[v] < 0: that sum is skipped (stays 0).
template <int NV>
__device__ __forceinline__ void tc_tile_sums(const float* __restrict__ partial, const tc_params& p,
                                             const long long (&tiles)[NV], int n, int m,
                                             float (&acc)[NV]) {
  const size_t stride = (size_t)p.n_pad * TC_TILE_M;
  const float* src[NV];
#pragma unroll
  for (int v = 0; v < NV; ++v) {
    acc[v] = 0.f;
    src[v] = partial + (((size_t)(tiles[v] < 0 ? 0 : tiles[v]) * p.n_chunks) * p.n_pad + n) * TC_TILE_M + m;
  }
  for (int c = 0; c < p.n_chunks; c += 2) {
    float a[NV], b[NV];
    const bool two = c + 1 < p.n_chunks;
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      a[v] = tiles[v] < 0 ? 0.f : src[v][(size_t)c * stride];
      b[v] = (tiles[v] < 0 || !two) ? 0.f : src[v][(size_t)(c + 1) * stride];
    }
#pragma unroll
    for (int v = 0; v < NV; ++v) {
      acc[v] += a[v];
      if (two) acc[v] += b[v];
    }
  }
}
__device__ __forceinline__ void tc_reset_counter(const tc_params& p) {
  if (blockIdx.x == 0 && blockIdx.y == 0 && blockIdx.z == 0 && threadIdx.x == 0) *p.counter = 0;
}

// h[e, n, i] = SiLU(gate) * up for every touched expert (Eq. 3's Expert_j, first half).
// grid (tiles over I, experts, row slices); groups come in (gate, up) pairs.
__global__ void __launch_bounds__(128) k_tc_fix_silu(const tc_params p, int I, int n_rows,
                                                     int Rp, const int32_t* __restrict__ expert,
                                                     const float* __restrict__ partial,
                                                     __nv_bfloat16* __restrict__ hbuf) {
  // The router's output is older than the GEMM this kernel follows (a kernel releases its
  // successor only after its own wait), so the plan can be made while that GEMM still runs.
  __shared__ tc_plan plan;
  if (threadIdx.x < 32) tc_make_plan(p, expert, &plan);
  __syncthreads();
  // This kernel has more blocks than fit the SMs at once, so its last blocks start late; if the
  // successor (the down GEMM) were released only after each block's wait, it would be launched
  // when this kernel is nearly over and could not stream its first weights meanwhile.  It is
  // released before the wait instead.  That is sound here: ahead of its own wait the down GEMM
  // reads only weights, the router's output (complete before the gate/up GEMM started) and its
  // own item counter, and it needs all of an SM's shared memory, so it gets onto an SM only when
  // the gate/up GEMM's CTA there has left; everything it writes comes after its wait.
  jk_pdl_trigger();
  jk_pdl_wait();
  tc_reset_counter(p);
  const int t = blockIdx.x, go = blockIdx.y, m = threadIdx.x;
  if (2 * go + 1 >= plan.n_groups) return;
  const long long tile_g = (long long)(2 * go) * p.tiles_per_group + t;
  const long long tile_u = tile_g + p.tiles_per_group;
  const int i = t * TC_TILE_M + m;
  if (i >= I) return;
  const int e = p.group_expert[plan.group_src[2 * go]];
  __nv_bfloat16* o = hbuf + (size_t)e * Rp * I + i;
#pragma unroll 4
  for (int n = blockIdx.z; n < n_rows; n += gridDim.z) {
    const long long tl[2] = {tile_g, tile_u};
    float gu[2];
    tc_tile_sums<2>(partial, p, tl, n, m, gu);
    const float g = gu[0], u = gu[1];
    o[(size_t)n * I] = __float2bfloat16_rn(g / (1.f + expf(-g)) * u);
  }
}

// y_r = W_down h for the K experts of row r, then Eq. 3 and the branch features:
//   f = u + sum_r g_r y_r,  b_r = g_r y_r (+ u).   grid (tiles over H, rows).
__global__ void __launch_bounds__(128) k_tc_fix_down_branch(
    const tc_params p, int H, const int32_t* __restrict__ expert,
    const float* __restrict__ gate, const __nv_bfloat16* __restrict__ u, int branch_residual,
    int head_mode, float alpha, float beta, const float* __restrict__ partial,
    __nv_bfloat16* __restrict__ bbuf, __nv_bfloat16* __restrict__ out_feat) {
  // Everything but the partial tiles is older than the GEMM this kernel follows (the router's
  // output, the caller's u): it is fetched, past the L1, while that GEMM still runs.
  __shared__ tc_plan plan;
  __shared__ long long tiles[JK_MAX_EXPERTS];
  __shared__ float s_gate[JK_MAX_EXPERTS];
  if (threadIdx.x < 32) tc_make_plan(p, expert, &plan);
  __syncthreads();
  const int t = blockIdx.x, r = blockIdx.y, m = threadIdx.x;
  const int K = p.K_top;
  if (threadIdx.x < K) {
    const int e = __ldcg(expert + r * K + threadIdx.x);
    int ga = 0;                       // position of expert e among the active groups
    for (int g = 0; g < plan.n_groups; ++g)
      if (p.group_expert[plan.group_src[g]] == e) ga = g;
    tiles[threadIdx.x] = (long long)ga * p.tiles_per_group + t;
    s_gate[threadIdx.x] = __ldcg(gate + r * K + threadIdx.x);
  }
  const int h = t * TC_TILE_M + m;
  const unsigned short u_bits = h < H ? __ldcg(reinterpret_cast<const unsigned short*>(u) + (size_t)r * H + h) : 0;
  __syncthreads();
  jk_pdl_wait();
  jk_pdl_trigger();
  tc_reset_counter(p);
  if (h >= H) return;
  const float uv = __uint_as_float((unsigned)u_bits << 16);
  float f = uv;
  if (head_mode == 1) {
    // contrastive heads (Eq. 6-7): b_0 = f^moe (+ u), b_1 = beta y_1 - alpha y_2 (+ u)
    const long long tl[2] = {tiles[0], tiles[1]};
    float yy[2];
    tc_tile_sums<2>(partial, p, tl, r, m, yy);
    const float y0 = yy[0], y1 = yy[1];
    const float g0y = s_gate[0] * y0, g1y = s_gate[1] * y1;
    const float fm = g0y + g1y, fc = beta * y0 - alpha * y1;
    f = (uv + g0y) + g1y;
    bbuf[((size_t)r * K) * H + h] = __float2bfloat16_rn(branch_residual ? fm + uv : fm);
    bbuf[((size_t)r * K + 1) * H + h] = __float2bfloat16_rn(branch_residual ? fc + uv : fc);
  } else {
    long long tl[JK_MAX_EXPERTS];
    float ys[JK_MAX_EXPERTS];
#pragma unroll
    for (int k = 0; k < JK_MAX_EXPERTS; ++k) tl[k] = k < K ? tiles[k] : -1;
    tc_tile_sums<JK_MAX_EXPERTS>(partial, p, tl, r, m, ys);
#pragma unroll
    for (int k = 0; k < JK_MAX_EXPERTS; ++k) {
      if (k >= K) break;
      const float y = ys[k];
      const float gy = s_gate[k] * y;
      f += gy;
      bbuf[((size_t)r * K + k) * H + h] = __float2bfloat16_rn(branch_residual ? gy + uv : gy);
    }
  }
  out_feat[(size_t)r * H + h] = __float2bfloat16_rn(f);
}

// logits = b W_head^T (Eq. 4) assembled from the partial tiles, optionally stored, and the
// per-chunk top-k statistics of jk_topk.cuh.   grid (chunks, logits rows), JK_TOPK_THREADS threads.
__global__ void __launch_bounds__(JK_TOPK_THREADS, 2) k_tc_fix_lmhead_topk(
    const tc_params p, int V, int k_e, int chunks, const float* __restrict__ partial,
    float* __restrict__ logits, int rows_per_b, long long stride_b, float* __restrict__ tk_val,
    int32_t* __restrict__ tk_idx, float* __restrict__ tk_ms) {
  jk_pdl_wait();
  jk_pdl_trigger();
  tc_reset_counter(p);
  constexpr int TILES = JK_TOPK_CHUNK / TC_TILE_M;     // 32 tiles per chunk
  const int chunk = blockIdx.x, row = blockIdx.y;
  const int base = chunk * JK_TOPK_CHUNK;
  float vals[JK_TOPK_PER];
  float* lrow = logits ? logits + (size_t)(row / rows_per_b) * (size_t)stride_b +
                             (size_t)(row % rows_per_b) * V : nullptr;
  // thread t owns entries t, t + 512, ...: the same column m of JK_TOPK_PER different tiles
  long long tl[JK_TOPK_PER];
#pragma unroll
  for (int j = 0; j < JK_TOPK_PER; ++j) {
    const int off = threadIdx.x + j * JK_TOPK_THREADS; // within the chunk
    tl[j] = base + off < V ? (long long)chunk * TILES + off / TC_TILE_M : -1;
  }
  tc_tile_sums<JK_TOPK_PER>(partial, p, tl, row, threadIdx.x % TC_TILE_M, vals);
#pragma unroll
  for (int j = 0; j < JK_TOPK_PER; ++j) {
    const int idx = base + threadIdx.x + j * JK_TOPK_THREADS;
    if (idx < V) { if (lrow) lrow[idx] = vals[j]; }
    else vals[j] = -INFINITY;
  }
  jk_topk_chunk_select(vals, base, V, k_e, (size_t)row * chunks + chunk, tk_val, tk_idx, tk_ms);
}

// ---------------------------------------------------------------------------------------------
// host side
// ---------------------------------------------------------------------------------------------
typedef CUresult (*tc_encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*,
                                 const cuuint64_t*, const cuuint64_t*, const cuuint32_t*,
                                 const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

struct tc_map_entry {
  const void* ptr;
  uint64_t rows, cols;
  uint32_t box_rows;
  CUtensorMap map;
};

struct tc_state {
  tc_encode_fn encode;
  tc_map_entry maps[32];
  int n_maps;
  int smem_set;
  int failed;
};

#define TC_MAX_GRID 192
static int tc_grid(const jk_ctx* ctx) {
  const int n = ctx->sm_count > 0 ? ctx->sm_count : 148;
  return n > TC_MAX_GRID ? TC_MAX_GRID : n;
}

static int tc_stage_bytes(int n_pad, int kb) { return (TC_TILE_M + n_pad) * kb * TC_BOX_K * 2; }

static int tc_stages(int n_pad, int kb) {
  int s = (TC_SMEM_BUDGET - (int)sizeof(tc_smem_tail) - 1024) / tc_stage_bytes(n_pad, kb);
  if (s > TC_MAX_STAGES) s = TC_MAX_STAGES;
  return s;
}

// Tiling of one contraction: boxes per stage, k steps of a tile, and the cut of a tile's k steps
// into chunks (the work items).  Chunks are at least 128 KB of weights long and as many as give
// every CTA about six items when all groups are active: more chunks balance the CTAs better but
// mean more partial tiles for the fix-up kernels to add up, and those sit on the critical path
// (measured at the 7B shape: 3-4 items per CTA 519, 6 items 532, 12 items 531, 24 items 524 steps/s).
struct tc_tiling { int kb, kt, ch, n_chunks; };
static tc_tiling tc_tile_plan(int kdim, int n_pad, long long tiles_all_groups, int n_cta) {
  tc_tiling t;
  t.kb = tc_stages(n_pad, 2) >= TC_KB_WIDE_MIN_STAGES ? 2 : 1;
  t.kt = (kdim + t.kb * TC_BOX_K - 1) / (t.kb * TC_BOX_K);
  const int ch_min = 8 / t.kb;                                  // 8 boxes of 128 x 64 bf16 = 128 KB
  long long want = (6ll * n_cta + tiles_all_groups - 1) / tiles_all_groups;
  const int most = t.kt / ch_min > 1 ? t.kt / ch_min : 1;
  if (want > most) want = most;
  if (want < 1) want = 1;
  t.ch = (t.kt + (int)want - 1) / (int)want;
  t.n_chunks = (t.kt + t.ch - 1) / t.ch;
  return t;
}

static size_t tc_partial_for(long long tiles_all_groups, int kdim, int n_pad) {
  // (the grid is the SM count, which the sizing does not know: take the chunk count of the
  // largest grid, which is the largest chunk count)
  const tc_tiling t = tc_tile_plan(kdim, n_pad, tiles_all_groups, TC_MAX_GRID);
  return (size_t)tiles_all_groups * t.n_chunks * n_pad * TC_TILE_M * sizeof(float);
}

// Worst case over the contractions.
size_t jk_tc_partial_bytes(const jk_config& c) {
  const int R = c.max_batch * c.max_frontier;
  const int np1 = (int)jk_align_up(R, 16), np2 = (int)jk_align_up((size_t)R * c.top_k, 16);
  const long long t_i = (c.inter + TC_TILE_M - 1) / TC_TILE_M, t_h = (c.hidden + TC_TILE_M - 1) / TC_TILE_M,
                  t_v = (c.vocab + TC_TILE_M - 1) / TC_TILE_M;
  size_t a = tc_partial_for(2ll * c.n_experts * t_i, c.hidden, np1);
  size_t b = tc_partial_for((long long)c.n_experts * t_h, c.inter, np1);
  size_t d = tc_partial_for(t_v, c.hidden, np2);
  // the draft layer's reduction, QKV and output projections (one group each)
  const int qd = c.n_q_heads * c.head_dim, qkvd = (c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
  const long long t_qkv = (qkvd + TC_TILE_M - 1) / TC_TILE_M;
  size_t e1 = tc_partial_for(t_h, 2 * c.hidden, np1);
  // (jk_verify_qkv sends up to 256 tree tokens at a time through the QKV projection)
  int np_v = (int)jk_align_up((size_t)c.max_batch * c.max_tree, 16);
  if (np_v > 256) np_v = 256;
  size_t e2 = tc_partial_for(t_qkv, c.hidden, np_v > np1 ? np_v : np1);
  size_t e3 = tc_partial_for(t_h, qd, np1);
  size_t m = a > b ? a : b;
  m = m > d ? m : d;
  m = m > e1 ? m : e1;
  m = m > e2 ? m : e2;
  return m > e3 ? m : e3;
}

void jk_tc_destroy(jk_ctx* ctx) {
  if (ctx && ctx->tc_state) {
    free(ctx->tc_state);
    ctx->tc_state = nullptr;
  }
}

static tc_state* tc_get_state(jk_ctx* ctx) {
  if (ctx->tc_state) return (tc_state*)ctx->tc_state;
  tc_state* s = (tc_state*)calloc(1, sizeof(tc_state));
  if (!s) return nullptr;
  void* fn = nullptr;
  cudaDriverEntryPointQueryResult q;
  if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
      q != cudaDriverEntryPointSuccess || !fn) {
    s->failed = 1;
  }
  s->encode = (tc_encode_fn)fn;
  ctx->tc_state = s;
  return s;
}

int jk_tc_available(const jk_ctx* ctx) {
  const jk_config& c = ctx->cfg;
  if (c.dtype != JK_BF16) return 0;
  const int np2 = (int)jk_align_up((size_t)c.max_batch * c.max_frontier * c.top_k, 16);
  if (np2 > 256) return 0;                       // two accumulators must fit the 512 TMEM columns
  if (tc_stages(np2, 1) < 2) return 0;
  tc_state* s = tc_get_state(const_cast<jk_ctx*>(ctx));
  return s && !s->failed;
}

extern "C" int jk_tensor_path_active(jk_ctx* ctx) {
  return (ctx && ctx->tensor_path && jk_tc_available(ctx)) ? 1 : 0;
}

// 2-D bf16 tensor map: `rows` x `cols` (cols contiguous), box = box_rows x 64, 128-byte swizzle.
static const CUtensorMap* tc_map_lookup(jk_ctx* ctx, tc_state* s, const void* ptr, uint64_t rows,
                                        uint64_t cols, uint32_t box_rows) {
  for (int i = 0; i < s->n_maps; ++i) {
    tc_map_entry& e = s->maps[i];
    if (e.ptr == ptr && e.rows == rows && e.cols == cols && e.box_rows == box_rows) return &e.map;
  }
  if (s->n_maps == 32) s->n_maps = 0;            // recycle (pointers changed often)
  tc_map_entry& e = s->maps[s->n_maps];
  const cuuint64_t gdim[2] = {cols, rows};
  const cuuint64_t gstride[1] = {cols * 2};
  const cuuint32_t box[2] = {TC_BOX_K, box_rows};
  const cuuint32_t estr[2] = {1, 1};
  CUresult r = s->encode(&e.map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(ptr), gdim,
                         gstride, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(ctx->cuda_err, sizeof(ctx->cuda_err), "cuTensorMapEncodeTiled failed (%d)", (int)r);
    return nullptr;
  }
  e.ptr = ptr; e.rows = rows; e.cols = cols; e.box_rows = box_rows;
  ++s->n_maps;
  return &e.map;
}

// The same, handed out by value: a later lookup may recycle the slot an earlier one returned.
static bool tc_map(jk_ctx* ctx, tc_state* s, const void* ptr, uint64_t rows, uint64_t cols,
                   uint32_t box_rows, CUtensorMap* out) {
  const CUtensorMap* m = tc_map_lookup(ctx, s, ptr, rows, cols, box_rows);
  if (!m) return false;
  *out = *m;
  return true;
}

// Launch the streaming GEMM; fills the launch-dependent fields of p.  Four item counters take
// turns: a launch's counter is put back to zero by its own fix-up kernel, well before the same
// counter is used again four launches later (a GEMM that prefetches reads its counter while the
// fix-up of the GEMM before it is still running, so that one cannot share it).
static int tc_launch_gemm(jk_ctx* ctx, cudaStream_t st, tc_state* s, const CUtensorMap* a0,
                          const CUtensorMap* a1, const CUtensorMap* b, tc_params& p,
                          const int32_t* expert, int stage_id) {
  const jk_ws_layout& L = ctx->lay;
  const int n_cta = tc_grid(ctx);
  const long long tiles_all = (long long)p.n_groups_max * p.tiles_per_group;
  const tc_tiling t = tc_tile_plan(p.kdim, p.n_pad, tiles_all, n_cta);
  p.kb = t.kb; p.kt = t.kt; p.ch = t.ch; p.n_chunks = t.n_chunks;
  p.stages = tc_stages(p.n_pad, p.kb);
  if (tiles_all * p.n_chunks >= (1ll << 30)) return JK_ERR_SHAPE;    // item ids are 32-bit
  int cols = 32;
  while (cols < 2 * p.n_pad) cols <<= 1;
  p.tmem_cols = cols;
  if ((size_t)tiles_all * p.n_chunks * p.n_pad * TC_TILE_M * sizeof(float) > L.gemm_part_bytes)
    return JK_ERR_WORKSPACE;
  p.counter = (int*)(ctx->ws + L.gemm_cnt) + (ctx->gemm_seq++ & 3);
  const size_t smem = (size_t)p.stages * tc_stage_bytes(p.n_pad, p.kb) + sizeof(tc_smem_tail) + 1024;
  if (!s->smem_set) {
    JK_CUDA_CHECK(ctx, cudaFuncSetAttribute(k_tc_gemm<1>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            TC_SMEM_BUDGET));
    JK_CUDA_CHECK(ctx, cudaFuncSetAttribute(k_tc_gemm<2>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            TC_SMEM_BUDGET));
    s->smem_set = 1;
  }
  JK_PROF(ctx, st, stage_id);
  if (p.kb == 2)
    jk_launch_pdl(k_tc_gemm<2>, dim3(n_cta), dim3(TC_THREADS), smem, st, *a0, *a1, *b, p, expert,
                  (float*)(ctx->ws + L.gemm_part), (int32_t*)(ctx->ws + L.status));
  else
    jk_launch_pdl(k_tc_gemm<1>, dim3(n_cta), dim3(TC_THREADS), smem, st, *a0, *a1, *b, p, expert,
                  (float*)(ctx->ws + L.gemm_part), (int32_t*)(ctx->ws + L.status));
  JK_LAUNCH_CHECK(ctx);
  return JK_OK;
}

// Expert FFNs of the draft layer (Eq. 3) on the tensor core: gate/up GEMM, SiLU * up, down GEMM,
// then the combined feature and the branch features (LM-head input).
int jk_tc_ffn(jk_ctx* ctx, cudaStream_t st, const jk_draft_weights* w, int R,
              const int32_t* expert, const float* gate, const void* u, void* out_feat) {
  tc_state* s = tc_get_state(ctx);
  if (!s || s->failed) return JK_ERR_CUDA;
  const jk_config& c = ctx->cfg;
  const jk_ws_layout& L = ctx->lay;
  const int H = c.hidden, I = c.inter, N = c.n_experts, Rp = L.rows_pad;
  const float* partial = (const float*)(ctx->ws + L.gemm_part);
  tc_params p;
  memset(&p, 0, sizeof(p));
  p.R = R; p.K_top = c.top_k; p.n_experts = N;
  const int n_pad = (int)jk_align_up(R, 16);
  // gate / up
  CUtensorMap ag, au, bx;
  if (!tc_map(ctx, s, w->w_gate, (uint64_t)N * I, H, TC_TILE_M, &ag) ||
      !tc_map(ctx, s, w->w_up, (uint64_t)N * I, H, TC_TILE_M, &au) ||
      !tc_map(ctx, s, ctx->ws + L.xn, Rp, H, n_pad, &bx))
    return JK_ERR_CUDA;
  p.n_groups_max = 2 * N;
  for (int e = 0; e < N; ++e)
    for (int h = 0; h < 2; ++h) {
      const int g = 2 * e + h;
      p.group_expert[g] = e; p.group_amap[g] = h; p.group_arow0[g] = e * I; p.group_brow0[g] = 0;
    }
  p.tiles_per_group = (I + TC_TILE_M - 1) / TC_TILE_M;
  p.kdim = H;
  p.n_pad = n_pad;
  int rc = tc_launch_gemm(ctx, st, s, &ag, &au, &bx, p, expert, JK_ST_GATEUP);
  if (rc != JK_OK) return rc;
  JK_PROF(ctx, st, JK_ST_GEMM_FIXUP);
  jk_launch_pdl(k_tc_fix_silu, dim3(p.tiles_per_group, N, R), dim3(128), 0, st, 
      p, I, R, Rp, expert, partial, (__nv_bfloat16*)(ctx->ws + L.hbuf));
  JK_LAUNCH_CHECK(ctx);
  // down
  CUtensorMap ad, bh;
  if (!tc_map(ctx, s, w->w_down, (uint64_t)N * H, I, TC_TILE_M, &ad) ||
      !tc_map(ctx, s, ctx->ws + L.hbuf, (uint64_t)N * Rp, I, n_pad, &bh))
    return JK_ERR_CUDA;
  p.n_groups_max = N;
  for (int e = 0; e < N; ++e) {
    p.group_expert[e] = e; p.group_amap[e] = 0; p.group_arow0[e] = e * H; p.group_brow0[e] = e * Rp;
  }
  p.tiles_per_group = (H + TC_TILE_M - 1) / TC_TILE_M;
  p.kdim = I;
  p.prefetch = 1;
  rc = tc_launch_gemm(ctx, st, s, &ad, &ad, &bh, p, expert, JK_ST_DOWN);
  if (rc != JK_OK) return rc;
  JK_PROF(ctx, st, JK_ST_BRANCH);
  jk_launch_pdl(k_tc_fix_down_branch, dim3(p.tiles_per_group, R), dim3(128), 0, st, 
      p, H, expert, gate, (const __nv_bfloat16*)u, c.branch_residual, c.head_mode,
      c.contrast_alpha, c.contrast_beta, partial,
      (__nv_bfloat16*)(ctx->ws + L.bbuf), (__nv_bfloat16*)out_feat);
  JK_LAUNCH_CHECK(ctx);
  return JK_OK;
}

// Shared LM head (Eq. 4) on the tensor core, with the per-chunk top-k statistics; `logits` may be
// NULL when the caller does not keep the draft distributions.
int jk_tc_lm_head(jk_ctx* ctx, cudaStream_t st, const jk_draft_weights* w, int RK, float* logits,
                  int rows_per_b, long long logits_stride_b) {
  tc_state* s = tc_get_state(ctx);
  if (!s || s->failed) return JK_ERR_CUDA;
  const jk_config& c = ctx->cfg;
  const jk_ws_layout& L = ctx->lay;
  const int H = c.hidden, V = c.vocab;
  tc_params p;
  memset(&p, 0, sizeof(p));
  p.R = 0; p.K_top = c.top_k; p.n_experts = c.n_experts;
  const int n_pad = (int)jk_align_up(RK, 16);
  CUtensorMap ah, bb;
  if (!tc_map(ctx, s, w->lm_head, V, H, TC_TILE_M, &ah) ||
      !tc_map(ctx, s, ctx->ws + L.bbuf, L.rk_pad, H, n_pad, &bb))
    return JK_ERR_CUDA;
  p.n_groups_max = 1;
  p.group_expert[0] = -1; p.group_amap[0] = 0; p.group_arow0[0] = 0; p.group_brow0[0] = 0;
  p.tiles_per_group = (V + TC_TILE_M - 1) / TC_TILE_M;
  p.kdim = H;
  p.n_pad = n_pad;
  p.prefetch = 1;
  int rc = tc_launch_gemm(ctx, st, s, &ah, &ah, &bb, p, nullptr, JK_ST_LMHEAD);
  if (rc != JK_OK) return rc;
  JK_PROF(ctx, st, JK_ST_TOPK);
  jk_launch_pdl(k_tc_fix_lmhead_topk, dim3(L.topk_chunks, RK), dim3(JK_TOPK_THREADS), 0, st, 
      p, V, c.k_per_expert, L.topk_chunks, (const float*)(ctx->ws + L.gemm_part), logits,
      rows_per_b, logits_stride_b, (float*)(ctx->ws + L.tk_val), (int32_t*)(ctx->ws + L.tk_idx),
      (float*)(ctx->ws + L.tk_ms));
  JK_LAUNCH_CHECK(ctx);
  return JK_OK;
}

// ---------------------------------------------------------------------------------------------
// Plain linear layer on the same streaming GEMM: out[r, m] = sum_k W[m, k] x[r, k] (+ bias[m])
// (+ resid[r, m]), used by the draft layer's reduction, QKV and output projections (Eq. 1).
// ---------------------------------------------------------------------------------------------
// grid (tiles over the M output features, rows); one of out_bf16 / out_f32 is written
__global__ void __launch_bounds__(128) k_tc_fix_linear(
    const tc_params p, int Mrows, const float* __restrict__ partial,
    const __nv_bfloat16* __restrict__ bias, const __nv_bfloat16* __restrict__ resid,
    long long resid_ld, __nv_bfloat16* __restrict__ out_bf16, float* __restrict__ out_f32,
    long long out_ld) {
  jk_pdl_wait();
  jk_pdl_trigger();
  tc_reset_counter(p);
  const int t = blockIdx.x, r = blockIdx.y, m = threadIdx.x;
  const int o = t * TC_TILE_M + m;
  if (o >= Mrows) return;
  float v = tc_tile_sum(partial, p, t, r, m);
  if (bias) v += __bfloat162float(bias[o]);
  if (resid) v += __bfloat162float(resid[(size_t)r * resid_ld + o]);
  if (out_bf16) out_bf16[(size_t)r * out_ld + o] = __float2bfloat16_rn(v);
  else out_f32[(size_t)r * out_ld + o] = v;
}

// x: bf16 [x_rows, Kdim] with x_rows >= n_rows (the copy's box is n_rows rounded up to 16: rows
// past x_rows are filled with zeros by the copy engine), W: bf16 [Mrows, Kdim].  The weights do not depend on the kernel before: their first ring is prefetched.
int jk_tc_linear(jk_ctx* ctx, cudaStream_t st, const void* W, int Mrows, int Kdim, const void* x,
                 int x_rows, int n_rows, const void* bias, const void* resid, long long resid_ld,
                 void* out_bf16, float* out_f32, long long out_ld) {
  tc_state* s = tc_get_state(ctx);
  if (!s || s->failed) return JK_ERR_CUDA;
  const jk_ws_layout& L = ctx->lay;
  tc_params p;
  memset(&p, 0, sizeof(p));
  p.R = 0; p.K_top = ctx->cfg.top_k; p.n_experts = ctx->cfg.n_experts;
  const int n_pad = (int)jk_align_up(n_rows, 16);
  if (n_rows > x_rows || n_pad > 256) return JK_ERR_SHAPE;   // (rows of the box past x_rows read as zero)
  CUtensorMap aw, bx;
  if (!tc_map(ctx, s, W, Mrows, Kdim, TC_TILE_M, &aw) || !tc_map(ctx, s, x, x_rows, Kdim, n_pad, &bx))
    return JK_ERR_CUDA;
  p.n_groups_max = 1;
  p.group_expert[0] = -1; p.group_amap[0] = 0; p.group_arow0[0] = 0; p.group_brow0[0] = 0;
  p.tiles_per_group = (Mrows + TC_TILE_M - 1) / TC_TILE_M;
  p.kdim = Kdim;
  p.n_pad = n_pad;
  p.prefetch = 1;
  int rc = tc_launch_gemm(ctx, st, s, &aw, &aw, &bx, p, nullptr, JK_ST_PRE_GEMM);
  if (rc != JK_OK) return rc;
  JK_PROF(ctx, st, JK_ST_PRE_FIXUP);
  jk_launch_pdl(k_tc_fix_linear, dim3(p.tiles_per_group, n_rows), dim3(128), 0, st, p, Mrows,
                (const float*)(ctx->ws + L.gemm_part), (const __nv_bfloat16*)bias,
                (const __nv_bfloat16*)resid, resid_ld, (__nv_bfloat16*)out_bf16, out_f32, out_ld);
  JK_LAUNCH_CHECK(ctx);
  return JK_OK;
}

// General bf16 tensor map with the 128-byte swizzle (used by the attention kernel): `rank` dims,
// innermost first; strides in bytes for dims 1..rank-1; box extents per dim.
int jk_tma_encode_bf16(jk_ctx* ctx, CUtensorMap* out, const void* ptr, int rank,
                       const uint64_t* dims, const uint64_t* strides_bytes, const uint32_t* box) {
  tc_state* s = tc_get_state(ctx);
  if (!s || s->failed) return JK_ERR_CUDA;
  cuuint64_t gdim[5], gstr[4];
  cuuint32_t bx[5], es[5];
  for (int i = 0; i < rank; ++i) { gdim[i] = dims[i]; bx[i] = box[i]; es[i] = 1; }
  for (int i = 0; i + 1 < rank; ++i) gstr[i] = strides_bytes[i];
  CUresult r = s->encode(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, (cuuint32_t)rank,
                         const_cast<void*>(ptr), gdim, gstr, bx, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                         CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                         CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
  if (r != CUDA_SUCCESS) {
    snprintf(ctx->cuda_err, sizeof(ctx->cuda_err), "cuTensorMapEncodeTiled failed (%d)", (int)r);
    return JK_ERR_CUDA;
  }
  return JK_OK;
}
