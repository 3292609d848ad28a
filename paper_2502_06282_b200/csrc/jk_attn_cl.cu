// Cluster-merged tensor-core kernel of jk_tree_verify_attn for bf16 (arXiv 2502.06282, Sec. 2.1
// step 2, mask of Fig. 4): the kernel for calls that are too small to keep a persistent kernel busy
// (a few key tiles per SM), where the call is a chain of latencies and every launch and every trip
// through global memory counts.
//
// One CTA = (sequence, kv head, block of 128 query rows, slice of the key range); the CTAs of the
// n_split <= 8 slices of one query block form a thread-block cluster.  Query rows are (q head of
// the group, tree node) pairs, so for GQA the heads that share a kv head share its K/V tiles.
//   - K tiles (three-deep ring) and V tiles (two-deep ring) of 128 keys arrive by TMA; all of a
//     short slice's tiles are in flight from the first instruction on.
//   - S = Q K^T on the tensor core into one of two tensor-memory buffers, so the product of tile
//     i+1 runs under the softmax of tile i.
//   - Two threads own a query row, 64 keys each: one read of S into registers, tree mask as a
//     128-bit visibility word (ancestor set shifted by the prefix length), the two halves' maxima
//     exchanged through shared memory, P = exp(S - max) packed to bf16 and stored back into tensor
//     memory over S: the second product O += P V takes P from tensor memory as its A operand
//     (no shared-memory tile, no proxy fence) and V MN-major straight from its row-major tile.
//   - The running maximum only moves when it grows by more than 2^8 (the bf16 P and the fp32 sum
//     have room for that), so O is rarely rescaled.
//   - The slices are merged inside the cluster: every CTA leaves its unnormalised (max, sum, O) in
//     its own shared memory, the CTAs meet at the cluster barrier, and CTA r combines rows
//     r, r + n_split, ... by reading all slices' copies through distributed shared memory and
//     writes the bf16 result.  No partials in global memory and no second launch.
// 1 CTA per SM (about 195 KB of shared memory, 512 tensor-memory columns).  Every mbarrier wait is
// bounded; the two cluster barriers are reached on every path, an aborting CTA included.
#include <math.h>
#include <stdlib.h>

#include "jk_common.cuh"
#include "jk_tcgen05.cuh"

#define ACL_ROWS 128
#define ACL_KEYS 128
#define ACL_THREADS 256
#define ACL_NK 3                       // K ring depth
#define ACL_NV 2                       // V ring depth
#define ACL_MAX_SPLIT 8                // portable cluster size

struct acl_tail {
  uint64_t bar_k[ACL_NK], bar_v[ACL_NV], bar_s[2], bar_o;
  uint32_t tmem_base;
  int abort_flag;
  int parent[JK_MAX_TREE];
  float xmax[2][ACL_ROWS];             // [key half][row]: that half's visible maximum of a tile
  float xsum[2][ACL_ROWS];             // [key half][row]: that half's sum of exponentials
  float pm[ACL_ROWS];                  // the slice's (max, sum) per row, read by the whole cluster
  float pl[ACL_ROWS];
};

__device__ __forceinline__ uint32_t acl_cluster_rank() {
  uint32_t r;
  asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
  return r;
}
__device__ __forceinline__ void acl_cluster_sync() {
  asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
  asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
// address of this CTA's shared variable `p` in CTA `rank` of the cluster
__device__ __forceinline__ uint32_t acl_map(const void* p, uint32_t rank) {
  uint32_t a;
  asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(a) : "r"(smem_u32(p)), "r"(rank));
  return a;
}
__device__ __forceinline__ float acl_ld_f32(uint32_t a) {
  float v;
  asm volatile("ld.shared::cluster.f32 %0, [%1];" : "=f"(v) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ float4 acl_ld_f32x4(uint32_t a) {
  float4 v;
  asm volatile("ld.shared::cluster.v4.f32 {%0, %1, %2, %3}, [%4];"
               : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "r"(a) : "memory");
  return v;
}
__device__ __forceinline__ void acl_pair_sync(int quarter) {
  // the two warps that share 32 query rows (64 threads); ids 1..4, 0 is __syncthreads
  asm volatile("bar.sync %0, 64;" ::"r"(quarter + 1) : "memory");
}

template <int D>
__global__ void __launch_bounds__(ACL_THREADS, 1) k_tree_attn_cl(
    const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
    const __nv_bfloat16* __restrict__ q, const int32_t* __restrict__ kv_len,
    const int32_t* __restrict__ parent, float scale, int M, int Hq, int Hkv, int n_split,
    int cache_rows, __nv_bfloat16* __restrict__ out, int32_t* status) {
  constexpr int KB = D / 64;                       // 64-element blocks along d
  constexpr int Q_BYTES = ACL_ROWS * D * 2;
  constexpr int KV_BYTES = ACL_KEYS * D * 2;
  constexpr uint32_t TMEM_COLS = 512;
  constexpr uint32_t O_COL = 256;
  constexpr int NC4 = D / 4;                       // 16-byte chunks of an fp32 output row
  static_assert(ACL_NK * KV_BYTES >= ACL_ROWS * D * 4, "the partial O reuses the K ring");
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* sq = smem;
  unsigned char* sk = sq + Q_BYTES;
  unsigned char* sv = sk + ACL_NK * KV_BYTES;
  acl_tail& T = *reinterpret_cast<acl_tail*>(sv + ACL_NV * KV_BYTES);
  volatile int* abort_flag = &T.abort_flag;

  const int split = (int)acl_cluster_rank();       // = blockIdx.x % n_split
  const int qblk = blockIdx.x / n_split;
  const int kvh = blockIdx.y, b = blockIdx.z;
  const int G = Hq / Hkv;
  // two threads per query row: tensor-memory lane quarter = warp % 4, key half = warp / 4
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int quarter = warp & 3, half = warp >> 2;
  const int row = quarter * 32 + lane;
  const int n_rows = G * M;
  const int row0 = qblk * ACL_ROWS;
  const int rows_here = min(ACL_ROWS, n_rows - row0);
  const bool row_valid = row < rows_here;
  const bool warp_has_rows = quarter * 32 < rows_here;
  const int node = row_valid ? (row0 + row) % M : 0;
  jk_pdl_wait();
  // The query block is asked for first: its loads need nothing from kv_len and travel while
  // thread 0 reads the prefix length and starts the K/V copies.
  constexpr int QV = ACL_ROWS * (D / 8) / ACL_THREADS;   // 16-byte vectors per thread
  uint4 qv[QV];
#pragma unroll
  for (int it = 0; it < QV; ++it) {
    const int idx = tid + it * ACL_THREADS;
    const int rr = idx / (D / 8), ch = idx % (D / 8);
    qv[it] = make_uint4(0u, 0u, 0u, 0u);
    if (rr < rows_here) {
      const int gg = (row0 + rr) / M, ii = (row0 + rr) % M;
      qv[it] = __ldg(reinterpret_cast<const uint4*>(
          q + (((size_t)b * M + ii) * Hq + kvh * G + gg) * D + ch * 8));
    }
  }
  const int par_mine = tid < M ? __ldg(parent + (size_t)b * M + tid) : -1;
  const int P = kv_len[b];
  const int Ltot = P + M;
  if (P < 0 || Ltot > cache_rows) {                // the same verdict in every CTA of the cluster
    if (tid == 0) jk_set_status(status, JK_ERR_BOUNDS);
    return;
  }
  const int tiles_total = (Ltot + ACL_KEYS - 1) / ACL_KEYS;
  // the key tiles are dealt evenly: slice s takes tiles [floor(s T / n), floor((s + 1) T / n))
  const int t0 = (split * tiles_total) / n_split;
  const int t1 = ((split + 1) * tiles_total) / n_split;
  const int n_tiles = t1 - t0;
  bool ok = true;
  float m_run = -INFINITY, l_run = 0.f;
  const float sl2 = scale * 1.4426950408889634f;

  const uint64_t pol = l2_policy_evict_first();    // the cache is read once per call
  auto issue_k = [&](int i) {                      // tile t0 + i into K stage i % ACL_NK
    uint64_t* bar = &T.bar_k[i % ACL_NK];
    unsigned char* dst = sk + (i % ACL_NK) * KV_BYTES;
    mbar_expect_tx(bar, KV_BYTES);
#pragma unroll
    for (int kb = 0; kb < KB; ++kb)
      tma_load_4d_hint(dst + kb * 16384, &map_k, kb * 64, (t0 + i) * ACL_KEYS, kvh, b, bar, pol);
  };
  auto issue_v = [&](int i) {
    uint64_t* bar = &T.bar_v[i % ACL_NV];
    unsigned char* dst = sv + (i % ACL_NV) * KV_BYTES;
    mbar_expect_tx(bar, KV_BYTES);
#pragma unroll
    for (int kb = 0; kb < KB; ++kb)
      tma_load_4d_hint(dst + kb * 16384, &map_v, kb * 64, (t0 + i) * ACL_KEYS, kvh, b, bar, pol);
  };

  if (tid == 0) {
    for (int i = 0; i < ACL_NK; ++i) mbar_init(&T.bar_k[i], 1);
    for (int i = 0; i < ACL_NV; ++i) mbar_init(&T.bar_v[i], 1);
    mbar_init(&T.bar_s[0], 1); mbar_init(&T.bar_s[1], 1); mbar_init(&T.bar_o, 1);
    T.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    for (int i = 0; i < n_tiles && i < ACL_NK; ++i) issue_k(i);
    for (int i = 0; i < n_tiles && i < ACL_NV; ++i) issue_v(i);
  }
  if (warp == 0) {
    tmem_alloc(&T.tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  uint32_t tmem_base = 0;
  if (n_tiles > 0) {
    if (tid < M) T.parent[tid] = par_mine;
    // Q block -> shared memory in the K-major 128-byte-swizzled layout the MMA reads
#pragma unroll
    for (int it = 0; it < QV; ++it) {
      const int idx = tid + it * ACL_THREADS;
      const int rr = idx / (D / 8), ch = idx % (D / 8);
      const int kb = ch >> 3, cb = ch & 7;
      *reinterpret_cast<uint4*>(sq + kb * 16384 + rr * 128 + ((cb ^ (rr & 7)) << 4)) = qv[it];
    }
    fence_proxy_async_smem();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  tmem_base = T.tmem_base;

  if (n_tiles > 0) {
    // ancestor set of this thread's node (Fig. 4), walked in shared memory
    unsigned long long anc_lo = 0ull, anc_hi = 0ull;
    if (row_valid) {
      int c = node;
      for (int guard = 0; c >= 0 && guard <= JK_MAX_TREE; ++guard) {
        if (c < 64) anc_lo |= 1ull << c; else anc_hi |= 1ull << (c - 64);
        const int pp = T.parent[c];
        c = (pp < c) ? pp : -1;
      }
    }
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const uint32_t idesc_s = instr_desc_bf16_ex(ACL_KEYS, 0);
    const uint32_t idesc_pv = instr_desc_bf16_ex(D, 1);
    const uint32_t qa = smem_u32(sq);
    auto issue_s = [&](int i) {                    // thread 0, after K tile i has arrived
      tc_fence_after();
      const uint32_t ka = smem_u32(sk + (i % ACL_NK) * KV_BYTES);
      const uint32_t sa = tmem_base + (uint32_t)(i & 1) * 128u;
#pragma unroll
      for (int kb = 0; kb < KB; ++kb)
#pragma unroll
        for (int k = 0; k < 4; ++k)
          tc_mma_bf16(sa, smem_desc_sw128(qa + kb * 16384 + k * 32),
                      smem_desc_sw128(ka + kb * 16384 + k * 32), idesc_s, (kb | k) ? 1u : 0u);
      tc_commit(&T.bar_s[i & 1]);
    };
    int s_issued = 0;                              // thread 0: S products issued so far
    if (tid == 0) {
      ok = mbar_wait(&T.bar_k[0], 0u, abort_flag, status);
      if (ok) { issue_s(0); s_issued = 1; }
    }

    for (int i = 0; i < n_tiles; ++i) {
      const int tile = t0 + i;
      const int buf = i & 1;
      // The next tile's S product is issued as early as its K tile is here and its destination
      // is free: that buffer holds the P of tile i-1 until the P V product of tile i-1 is done.
      auto try_issue_next_s = [&]() {
        if (i + 1 < n_tiles && s_issued == i + 1 &&
            mbar_try_wait(&T.bar_k[(i + 1) % ACL_NK], (uint32_t)((i + 1) / ACL_NK) & 1u)) {
          issue_s(i + 1);
          s_issued = i + 2;
        }
      };
      // visibility of this thread's 64 keys (Fig. 4): prefix keys, then the ancestor set
      unsigned long long vis = 0ull;
      if (row_valid) {
        unsigned long long vis_lo = 0ull, vis_hi = 0ull;
        const int s = P - tile * ACL_KEYS;
        if (s >= 128) { vis_lo = ~0ull; vis_hi = ~0ull; }
        else if (s >= 0) {
          if (s >= 64) { vis_lo = ~0ull; vis_hi = (s == 64) ? 0ull : ((1ull << (s - 64)) - 1ull); }
          else { vis_lo = (s == 0) ? 0ull : ((1ull << s) - 1ull); }
          unsigned long long a_lo, a_hi;
          if (s == 0) { a_lo = anc_lo; a_hi = anc_hi; }
          else if (s < 64) { a_lo = anc_lo << s; a_hi = (anc_hi << s) | (anc_lo >> (64 - s)); }
          else if (s == 64) { a_lo = 0ull; a_hi = anc_lo; }
          else { a_lo = 0ull; a_hi = anc_lo << (s - 64); }
          vis_lo |= a_lo; vis_hi |= a_hi;
        } else {
          const int t = -s;
          if (t < 64) { vis_lo = (anc_lo >> t) | (anc_hi << (64 - t)); vis_hi = anc_hi >> t; }
          else if (t < 128) { vis_lo = anc_hi >> (t - 64); vis_hi = 0ull; }
        }
        vis = half ? vis_hi : vis_lo;
      }
      const unsigned b0 = (unsigned)vis, b1 = (unsigned)(vis >> 32);
      ok = ok && mbar_wait(&T.bar_s[buf], (uint32_t)(i >> 1) & 1u, abort_flag, status);
      if (!__syncthreads_and(ok)) { ok = false; break; }
      tc_fence_after();
      // S of this tile has completed, so its K stage is free for the tile three ahead
      if (tid == 0 && i + ACL_NK < n_tiles) issue_k(i + ACL_NK);
      if (tid == 0 && i == 0) try_issue_next_s();

      // ---- this thread's half row of S, read once
      const uint32_t sa = tmem_base + lane_base + (uint32_t)buf * 128u + (uint32_t)half * 64u;
      uint32_t r0[32], r1[32];
      float mx = -INFINITY;
      if (warp_has_rows) {
        tmem_ld32(sa, r0);
        tmem_ld32(sa + 32u, r1);
        tmem_ld_wait();
#pragma unroll
        for (int j = 0; j < 32; ++j) {
          if ((b0 >> j) & 1u) mx = fmaxf(mx, __uint_as_float(r0[j]));
          if ((b1 >> j) & 1u) mx = fmaxf(mx, __uint_as_float(r1[j]));
        }
      }
      T.xmax[half][row] = mx;
      tc_fence_before();
      acl_pair_sync(quarter);                      // both halves have S in registers and xmax out
      tc_fence_after();
      mx = fmaxf(mx, T.xmax[half ^ 1][row]);
      // The reference maximum moves only when the row maximum outgrows it by more than 2^8.
      float alpha = 1.f;
      if (mx != -INFINITY && (m_run == -INFINITY || (mx - m_run) * sl2 > 8.f)) {
        alpha = (m_run == -INFINITY) ? 0.f : fast_exp2((m_run - mx) * sl2);
        m_run = mx;
      }
      const float m_use = (m_run == -INFINITY) ? 0.f : m_run;
      // ---- P = exp(S - max) as bf16, two keys per 32-bit column, back into tensor memory (this
      // tile's S buffer: the P V product of the previous tile reads the other one)
      float lsum = 0.f;
      if (warp_has_rows) {
        uint32_t pk[32];
#pragma unroll
        for (int j = 0; j < 32; j += 2) {
          const float p0 = ((b0 >> j) & 1u) ? fast_exp2((__uint_as_float(r0[j]) - m_use) * sl2) : 0.f;
          const float p1 = ((b0 >> (j + 1)) & 1u)
                               ? fast_exp2((__uint_as_float(r0[j + 1]) - m_use) * sl2) : 0.f;
          const float p2 = ((b1 >> j) & 1u) ? fast_exp2((__uint_as_float(r1[j]) - m_use) * sl2) : 0.f;
          const float p3 = ((b1 >> (j + 1)) & 1u)
                               ? fast_exp2((__uint_as_float(r1[j + 1]) - m_use) * sl2) : 0.f;
          const __nv_bfloat162 h01 = __floats2bfloat162_rn(p0, p1);
          const __nv_bfloat162 h23 = __floats2bfloat162_rn(p2, p3);
          // the sum runs over the rounded values the second product will use
          lsum += (__low2float(h01) + __high2float(h01)) + (__low2float(h23) + __high2float(h23));
          pk[j >> 1] = *reinterpret_cast<const uint32_t*>(&h01);
          pk[16 + (j >> 1)] = *reinterpret_cast<const uint32_t*>(&h23);
        }
        tmem_st32(tmem_base + lane_base + (uint32_t)buf * 128u + (uint32_t)half * 32u, pk);
      }
      if (i > 0) {
        // the previous tile's P V product has completed: O may be rescaled, its V stage refilled
        ok = mbar_wait(&T.bar_o, (uint32_t)(i - 1) & 1u, abort_flag, status);
        if (!__syncthreads_and(ok)) { ok = false; break; }
        tc_fence_after();
        if (tid == 0 && i - 1 + ACL_NV < n_tiles) issue_v(i - 1 + ACL_NV);
        if (tid == 0) try_issue_next_s();
        if (warp_has_rows && __any_sync(0xffffffffu, alpha != 1.f)) {
#pragma unroll 1
          for (int c = 0; c < D / 64; ++c) {
            uint32_t r[32];
            const uint32_t oa = tmem_base + lane_base + O_COL + (uint32_t)(half * (D / 2) + c * 32);
            tmem_ld32(oa, r);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 32; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * alpha);
            tmem_st32(oa, r);
          }
        }
      }
      if (warp_has_rows) tmem_st_wait();
      l_run = l_run * alpha + lsum;
      // Cache rows past the last live key (only the sequence's last tile has any) may hold
      // anything, NaN bit patterns included, and 0 * NaN would poison every output row: they are
      // cleared in the V tile before the second product reads it.
      const int live = Ltot - tile * ACL_KEYS;
      if (live < ACL_KEYS) {
        ok = ok && mbar_wait(&T.bar_v[i % ACL_NV], (uint32_t)(i / ACL_NV) & 1u, abort_flag, status);
        if (ok) {
          const int n16 = (ACL_KEYS - live) * 8;   // 16-byte pieces per 64-wide block
          unsigned char* vt = sv + (i % ACL_NV) * KV_BYTES;
          for (int idx = tid; idx < n16 * KB; idx += ACL_THREADS) {
            const int kb = idx / n16, rem = idx % n16;
            *reinterpret_cast<uint4*>(vt + kb * 16384 + (live + (rem >> 3)) * 128 + ((rem & 7) << 4)) =
                make_uint4(0u, 0u, 0u, 0u);
          }
        }
        fence_proxy_async_smem();
      }
      tc_fence_before();
      if (!__syncthreads_and(ok)) { ok = false; break; }
      if (tid == 0) {
        ok = mbar_wait(&T.bar_v[i % ACL_NV], (uint32_t)(i / ACL_NV) & 1u, abort_flag, status);
        if (ok) {
          tc_fence_after();
          const uint32_t pa = tmem_base + (uint32_t)buf * 128u;
          const uint32_t va = smem_u32(sv + (i % ACL_NV) * KV_BYTES);
#pragma unroll
          for (int j = 0; j < ACL_KEYS / 16; ++j)
            tc_mma_bf16_ts(tmem_base + O_COL, pa + (uint32_t)(j * 8),
                           smem_desc_mn_sw128(va + j * 2048, 16384), idesc_pv,
                           (i > 0 || j > 0) ? 1u : 0u);
          tc_commit(&T.bar_o);
          // the next tile's S product, if its K tile was not there in time to go first
          if (i + 1 < n_tiles && s_issued == i + 1) {
            ok = mbar_wait(&T.bar_k[(i + 1) % ACL_NK], (uint32_t)((i + 1) / ACL_NK) & 1u,
                           abort_flag, status);
            if (ok) { issue_s(i + 1); s_issued = i + 2; }
          }
        }
      }
    }
    if (ok) ok = mbar_wait(&T.bar_o, (uint32_t)(n_tiles - 1) & 1u, abort_flag, status);
    ok = __syncthreads_and(ok);
    tc_fence_after();
    if (ok) {
      // The unnormalised O of the slice goes to shared memory (over the K ring: every MMA has
      // completed) for the cluster to read.  16-byte chunk c of row t sits at chunk index
      // c * 128 + (t ^ (c & 31)), which the row-per-lane writes and the chunk-per-lane reads both
      // reach without bank conflicts.
      float4* so4 = reinterpret_cast<float4*>(sk);
      if (warp_has_rows) {
#pragma unroll 1
        for (int c = 0; c < D / 64; ++c) {
          uint32_t r[32];
          tmem_ld32(tmem_base + lane_base + O_COL + (uint32_t)(half * (D / 2) + c * 32), r);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int c4 = half * (NC4 / 2) + c * 8 + j;
            so4[c4 * ACL_ROWS + (row ^ (c4 & 31))] =
                make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                            __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
          }
        }
      }
    } else if (tid == 0) {
      // gave up, possibly with copies still in flight: give them a bounded time to land
      const unsigned long long ts = global_ns();
      while (global_ns() - ts < 2000000ull) { /* 2 ms: far longer than any TMA copy */ }
    }
    T.xsum[half][row] = l_run;
  }
  __syncthreads();
  if (tid < ACL_ROWS) {
    const bool have = ok && n_tiles > 0;
    T.pm[tid] = have ? m_run : -INFINITY;          // (threads 0..127 are the half-0 owners of row tid)
    T.pl[tid] = have ? T.xsum[0][tid] + T.xsum[1][tid] : 0.f;
  }
  // ---- merge inside the cluster
  acl_cluster_sync();                              // every slice's (max, sum, O) is in place
  {
    // A round trip through distributed shared memory was measured at about half a microsecond, so
    // every remote value a warp needs - (max, sum) and the O chunks of all slices, for up to two
    // rows at a time - is asked for before the first one is used.
    const float4* so4 = reinterpret_cast<const float4*>(sk);
    constexpr int RB = 2;                          // rows per batch and warp
    const int stride = n_split * (ACL_THREADS / 32);
    for (int r_first = split + warp * n_split; r_first < rows_here; r_first += RB * stride) {
      float ms[RB], ls[RB];
      float4 v[RB][ACL_MAX_SPLIT];
#pragma unroll
      for (int k = 0; k < RB; ++k) {
        const int r = r_first + k * stride;
        ms[k] = -INFINITY; ls[k] = 0.f;
        if (r < rows_here && lane < n_split) {
          ms[k] = acl_ld_f32(acl_map(&T.pm[r], (uint32_t)lane));
          ls[k] = acl_ld_f32(acl_map(&T.pl[r], (uint32_t)lane));
        }
#pragma unroll
        for (int s = 0; s < ACL_MAX_SPLIT; ++s) {
          v[k][s] = make_float4(0.f, 0.f, 0.f, 0.f);
          if (r < rows_here && lane < NC4 && s < n_split)
            v[k][s] = acl_ld_f32x4(acl_map(&so4[lane * ACL_ROWS + (r ^ (lane & 31))], (uint32_t)s));
        }
      }
#pragma unroll
      for (int k = 0; k < RB; ++k) {
        const int r = r_first + k * stride;
        if (r >= rows_here) break;                 // warp-uniform
        const float m = jk_warp_max(ms[k]);
        const float w_lane = (ms[k] == -INFINITY) ? 0.f : fast_exp2((ms[k] - m) * sl2);
        const float l = jk_warp_sum(w_lane * ls[k]);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int s = 0; s < ACL_MAX_SPLIT; ++s) {  // fixed order: bitwise reproducible
          const float w = __shfl_sync(0xffffffffu, w_lane, s);
          if (s < n_split && w != 0.f) {           // (a slice without keys or one that gave up: skipped)
            acc.x += w * v[k][s].x; acc.y += w * v[k][s].y;
            acc.z += w * v[k][s].z; acc.w += w * v[k][s].w;
          }
        }
        if (lane < NC4) {
          const float inv = 1.f / l;
          const int gg = (row0 + r) / M, ii = (row0 + r) % M;
          const size_t orow = ((size_t)b * M + ii) * Hq + kvh * G + gg;
          const __nv_bfloat162 o01 = __floats2bfloat162_rn(acc.x * inv, acc.y * inv);
          const __nv_bfloat162 o23 = __floats2bfloat162_rn(acc.z * inv, acc.w * inv);
          uint2 pkd;
          pkd.x = *reinterpret_cast<const uint32_t*>(&o01);
          pkd.y = *reinterpret_cast<const uint32_t*>(&o23);
          *reinterpret_cast<uint2*>(out + orow * D + lane * 4) = pkd;
        }
      }
    }
  }
  tc_fence_before();
  acl_cluster_sync();                              // nobody leaves while its memory is being read
  jk_pdl_trigger();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// jk_attn_tc.cu: tensor maps of the two caches
int jk_attn_tc_maps(jk_ctx* ctx, const void* kc, const void* vc, int64_t sb, int64_t sh,
                    int cache_rows, CUtensorMap* mk, CUtensorMap* mv);

static size_t acl_smem_bytes(int D) {
  return (size_t)ACL_ROWS * D * 2 + (size_t)(ACL_NK + ACL_NV) * ACL_KEYS * D * 2 +
         sizeof(acl_tail) + 1024;
}

template <int D>
static cudaError_t acl_launch(dim3 grid, int n_split, size_t smem, cudaStream_t st,
                              const CUtensorMap& mk, const CUtensorMap& mv, const void* q,
                              const int32_t* kv_len, const int32_t* parent, float scale, int M,
                              int Hq, int Hkv, int cache_rows, void* out, int32_t* status) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = grid;
  cfg.blockDim = dim3(ACL_THREADS);
  cfg.dynamicSmemBytes = smem;
  cfg.stream = st;
  cudaLaunchAttribute attr[2];
  attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
  attr[0].val.programmaticStreamSerializationAllowed = 1;
  attr[1].id = cudaLaunchAttributeClusterDimension;
  attr[1].val.clusterDim.x = (unsigned)n_split;
  attr[1].val.clusterDim.y = 1;
  attr[1].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 2;
  return cudaLaunchKernelEx(&cfg, k_tree_attn_cl<D>, mk, mv, (const __nv_bfloat16*)q, kv_len,
                            parent, scale, M, Hq, Hkv, n_split, cache_rows, (__nv_bfloat16*)out,
                            status);
}

// Clusters of `n_split` CTAs of this kernel that the device can hold at once (0 on error).
template <int D>
static int acl_max_clusters(int n_split, size_t smem) {
  cudaLaunchConfig_t cfg = {};
  cfg.gridDim = dim3((unsigned)n_split, 1, 1);
  cfg.blockDim = dim3(ACL_THREADS);
  cfg.dynamicSmemBytes = smem;
  cudaLaunchAttribute attr[1];
  attr[0].id = cudaLaunchAttributeClusterDimension;
  attr[0].val.clusterDim.x = (unsigned)n_split;
  attr[0].val.clusterDim.y = 1;
  attr[0].val.clusterDim.z = 1;
  cfg.attrs = attr;
  cfg.numAttrs = 1;
  int n = 0;
  if (cudaOccupancyMaxActiveClusters(&n, k_tree_attn_cl<D>, &cfg) != cudaSuccess) {
    cudaGetLastError();
    return 0;
  }
  return n;
}

struct acl_state {
  int smem_set;
  int max_clusters[ACL_MAX_SPLIT + 1];   // per cluster size, -1 = not asked yet
};

void jk_attn_cl_destroy(jk_ctx* ctx) {
  if (ctx && ctx->attn_cl_state) {
    free(ctx->attn_cl_state);
    ctx->attn_cl_state = nullptr;
  }
}

// The number of key slices (= cluster size) for a call: the largest one whose whole grid is
// resident at once, at most one slice per key tile.  0 if the kernel should not take the call
// (its grid would leave more than 40 % of the SMs idle or would need several waves).
int jk_attn_cl_plan(jk_ctx* ctx, int B, int M, int cache_rows) {
  const jk_config& c = ctx->cfg;
  if (!ctx->attn_cl_state) {
    acl_state* s = (acl_state*)calloc(1, sizeof(acl_state));
    if (!s) return 0;
    for (int i = 0; i <= ACL_MAX_SPLIT; ++i) s->max_clusters[i] = -1;
    ctx->attn_cl_state = s;
  }
  acl_state* s = (acl_state*)ctx->attn_cl_state;
  const int D = c.head_dim;
  const size_t smem = acl_smem_bytes(D);
  if (!s->smem_set) {
    cudaError_t e = D == 128
        ? cudaFuncSetAttribute(k_tree_attn_cl<128>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem)
        : cudaFuncSetAttribute(k_tree_attn_cl<64>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) { cudaGetLastError(); return 0; }
    s->smem_set = 1;
  }
  const int G = c.n_q_heads / c.n_kv_heads;
  const int n_qblk = (G * M + ACL_ROWS - 1) / ACL_ROWS;
  const int base = n_qblk * c.n_kv_heads * B;
  const int tiles_max = (cache_rows + ACL_KEYS - 1) / ACL_KEYS;
  for (int ns = ACL_MAX_SPLIT; ns >= 1; --ns) {
    if (ns > tiles_max && ns > 1) continue;
    if (base * ns > ctx->sm_count) continue;
    if (s->max_clusters[ns] < 0)
      s->max_clusters[ns] = D == 128 ? acl_max_clusters<128>(ns, smem) : acl_max_clusters<64>(ns, smem);
    if (s->max_clusters[ns] >= base) return ns;
  }
  return 0;
}

int jk_attn_cl(jk_ctx* ctx, cudaStream_t st, int n_split, int B, int M, const void* q,
               const void* kc, const void* vc, int64_t sb, int64_t sh, int cache_rows,
               const int32_t* kv_len, const int32_t* parent, float scale, void* out) {
  const jk_config& c = ctx->cfg;
  CUtensorMap mk, mv;
  if (jk_attn_tc_maps(ctx, kc, vc, sb, sh, cache_rows, &mk, &mv) != JK_OK) return JK_ERR_CUDA;
  const int G = c.n_q_heads / c.n_kv_heads;
  const int n_qblk = (G * M + ACL_ROWS - 1) / ACL_ROWS;
  const int D = c.head_dim;
  const dim3 grid(n_split * n_qblk, c.n_kv_heads, B);
  int32_t* status = (int32_t*)(ctx->ws + ctx->lay.status);
  JK_PROF(ctx, st, ctx->st_attn);
  if (D == 128)
    acl_launch<128>(grid, n_split, acl_smem_bytes(D), st, mk, mv, q, kv_len, parent, scale, M,
                    c.n_q_heads, c.n_kv_heads, cache_rows, out, status);
  else
    acl_launch<64>(grid, n_split, acl_smem_bytes(D), st, mk, mv, q, kv_len, parent, scale, M,
                   c.n_q_heads, c.n_kv_heads, cache_rows, out, status);
  JK_LAUNCH_CHECK(ctx);
  return JK_OK;
}
