// Tensor-core (tcgen05) kernel of jk_tree_verify_attn for bf16 (arXiv 2502.06282, Sec. 2.1 step 2,
// mask of Fig. 4).
//
// One CTA = (sequence, kv head, block of 128 query rows, slice of the key range).  Query rows are
// (q head of the group, tree node) pairs, so for GQA the heads that share a kv head share its K/V
// tiles.  Per tile of 128 keys:
//   TMA brings K [128 keys x d] and V [128 keys x d] into swizzled shared memory;
//   S = Q K^T on the tensor core into tensor memory (128 x 128 fp32);
//   two threads own one query row, 64 keys each: one read of S into registers, the tree mask (a
//   128-bit visibility word built from the node's ancestor set and the prefix length), the two
//   halves' maxima exchanged through shared memory, P = exp(S - max) packed to bf16 and stored
//   back into tensor memory over S;
//   O (+)= P V on the tensor core, P taken from tensor memory as the A operand, V MN-major straight
//   from its row-major tile; the reference maximum only moves when it is outgrown by more than
//   2^8, so O is rarely rescaled.
// The CTA writes an unnormalised partial (max, sum, O) per row; the merge kernel of jk_attn.cu
// combines the slices.  96 KB of shared memory and 256 tensor-memory columns per CTA: two CTAs
// share an SM and overlap each other's copy and math phases.  All mbarrier waits are bounded.
#include <math.h>
#include <stdlib.h>

#include "jk_common.cuh"
#include "jk_tcgen05.cuh"

#define ATC_ROWS 128
#define ATC_KEYS 128

struct atc_tail {
  uint64_t bar_k, bar_v, bar_s, bar_o;
  uint32_t tmem_base;
  int abort_flag;
  int parent[JK_MAX_TREE];
  float xmax[2][ATC_ROWS];             // [key half][row]: the half's visible maximum of a tile
  float xsum[2][ATC_ROWS];             // [key half][row]: the half's sum of exponentials
};

#define ATC_THREADS 256

template <int D>
__global__ void __launch_bounds__(ATC_THREADS, 2) k_tree_attn_tc(
    const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
    const __nv_bfloat16* __restrict__ q, const int32_t* __restrict__ kv_len,
    const int32_t* __restrict__ parent, float scale, int M, int Hq, int Hkv, int n_split,
    int n_qblk, int cache_rows, float* __restrict__ part_o, float* __restrict__ part_ml,
    __nv_bfloat16* __restrict__ out, int32_t* status) {
  constexpr int KB = D / 64;                       // 64-element blocks along d
  constexpr int Q_BYTES = ATC_ROWS * D * 2;
  constexpr int KP_BYTES = 2 * ATC_ROWS * 64 * 2;  // K tile (KB blocks) or P tile (2 blocks)
  constexpr int V_BYTES = ATC_KEYS * D * 2;
  constexpr uint32_t TMEM_COLS = 256;
  constexpr uint32_t O_COL = 128;
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* sq = smem;
  unsigned char* skp = smem + Q_BYTES;
  unsigned char* sv = skp + KP_BYTES;
  atc_tail& T = *reinterpret_cast<atc_tail*>(sv + V_BYTES);
  volatile int* abort_flag = &T.abort_flag;

  const int split = blockIdx.x % n_split, qblk = blockIdx.x / n_split;
  const int kvh = blockIdx.y, b = blockIdx.z;
  const int G = Hq / Hkv;
  // two threads per query row: tensor-memory lane quarter = warp % 4, key half = warp / 4
  const int tid = threadIdx.x, warp = tid >> 5;
  const int quarter = warp & 3, half = warp >> 2;
  const int row = quarter * 32 + (tid & 31);
  const int n_rows = G * M;
  const int row0 = qblk * ATC_ROWS;
  const bool row_valid = row0 + row < n_rows;
  const bool warp_has_rows = row0 + quarter * 32 < n_rows;
  const int g_idx = row_valid ? (row0 + row) / M : 0;
  const int node = row_valid ? (row0 + row) % M : 0;
  const size_t n_out = (size_t)gridDim.z * M * Hq;
  const size_t orow = ((size_t)b * M + node) * Hq + kvh * G + g_idx;
  // barriers and tensor memory touch no global memory: set up before the grid-dependency wait
  if (tid == 0) {
    mbar_init(&T.bar_k, 1); mbar_init(&T.bar_v, 1); mbar_init(&T.bar_s, 1); mbar_init(&T.bar_o, 1);
    T.abort_flag = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 0) {
    tmem_alloc(&T.tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  // Before the grid-dependency wait the kernel may only read what no kernel it can overlap with
  // writes.  That holds for kv_len and for the committed prefix rows of the caches (rows below
  // kv_len[b]): they are written by the acceptance call of an earlier step, whose kernels release
  // their dependents only when they exit, so they are complete before this kernel starts.  A key
  // tile that lies wholly in the prefix is therefore asked for right away and travels while the
  // kernel before (typically the previous layer's merge) is still running; the tree rows, Q and
  // parent[] are fresh and wait.
  const int P = kv_len[b];
  const int Ltot = P + M;
  const bool bad = P < 0 || Ltot > cache_rows;
  const int tiles_total = bad ? 0 : (Ltot + ATC_KEYS - 1) / ATC_KEYS;
  const int tiles_per = (tiles_total + n_split - 1) / n_split;
  const int t0 = split * tiles_per;
  const int t1 = min(tiles_total, t0 + tiles_per);
  const bool have_keys = t0 < t1;
  bool ok = true;
  uint32_t tmem_base = 0;
  float m_run = -INFINITY, l_run = 0.f;

  auto issue_k = [&](int tile) {
    const uint64_t pol = l2_policy_evict_first();   // the cache is read once per call
    mbar_expect_tx(&T.bar_k, ATC_KEYS * D * 2);
#pragma unroll
    for (int kb = 0; kb < KB; ++kb)
      tma_load_4d_hint(skp + kb * 16384, &map_k, kb * 64, tile * ATC_KEYS, kvh, b, &T.bar_k, pol);
  };
  auto issue_v = [&](int tile) {
    const uint64_t pol = l2_policy_evict_first();
    mbar_expect_tx(&T.bar_v, ATC_KEYS * D * 2);
#pragma unroll
    for (int kb = 0; kb < KB; ++kb)
      tma_load_4d_hint(sv + kb * 16384, &map_v, kb * 64, tile * ATC_KEYS, kvh, b, &T.bar_v, pol);
  };
  auto issue_kv = [&](int tile) { issue_k(tile); issue_v(tile); };
  const bool early = have_keys && (t0 + 1) * ATC_KEYS <= P;
  if (early && tid == 0) issue_kv(t0);
  jk_pdl_wait();
  if (bad && tid == 0) jk_set_status(status, JK_ERR_BOUNDS);
  // The query block is asked for first: its loads travel while thread 0 starts the K/V copies.
  constexpr int QV = ATC_ROWS * (D / 8) / ATC_THREADS;   // 16-byte vectors per thread
  uint4 qv[QV];
#pragma unroll
  for (int it = 0; it < QV; ++it) {
    const int idx = tid + it * ATC_THREADS;
    const int rr = idx / (D / 8), ch = idx % (D / 8);
    qv[it] = make_uint4(0u, 0u, 0u, 0u);
    if (row0 + rr < n_rows) {
      const int gg = (row0 + rr) / M, ii = (row0 + rr) % M;
      qv[it] = __ldg(reinterpret_cast<const uint4*>(
          q + (((size_t)b * M + ii) * Hq + kvh * G + gg) * D + ch * 8));
    }
  }
  const int par_mine = tid < M ? __ldg(parent + (size_t)b * M + tid) : -1;
  if (have_keys && !early && tid == 0) issue_kv(t0);
  if (have_keys) {
    if (tid < M) T.parent[tid] = par_mine;
    // Q block -> shared memory in the K-major 128-byte-swizzled layout the MMA reads
#pragma unroll
    for (int it = 0; it < QV; ++it) {
      const int idx = tid + it * ATC_THREADS;
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
  if (bad) ok = false;
  if (have_keys) {
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
    const uint32_t idesc_s = instr_desc_bf16_ex(ATC_KEYS, 0);
    const uint32_t idesc_pv = instr_desc_bf16_ex(D, 1);
    const float sl2 = scale * 1.4426950408889634f;

    for (int tile = t0; tile < t1; ++tile) {
      const uint32_t ph = (uint32_t)(tile - t0) & 1u;
      if (tid == 0) {
        ok = mbar_wait(&T.bar_k, ph, abort_flag, status);
        if (ok) {
          tc_fence_after();
          const uint32_t qa = smem_u32(sq), ka = smem_u32(skp);
#pragma unroll
          for (int kb = 0; kb < KB; ++kb)
#pragma unroll
            for (int k = 0; k < 4; ++k)
              tc_mma_bf16(tmem_base, smem_desc_sw128(qa + kb * 16384 + k * 32),
                          smem_desc_sw128(ka + kb * 16384 + k * 32), idesc_s, (kb | k) ? 1u : 0u);
          tc_commit(&T.bar_s);
        }
      }
      // visibility of this thread's 64 keys (Fig. 4): prefix keys, then the ancestor set
      unsigned long long vis = 0ull;
      if (row_valid) {
        unsigned long long vis_lo = 0ull, vis_hi = 0ull;
        const int s = P - tile * ATC_KEYS;
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
      ok = ok && mbar_wait(&T.bar_s, ph, abort_flag, status);
      if (!__syncthreads_and(ok)) { ok = false; break; }
      tc_fence_after();
      // S is complete, so the K tile is free: the next one travels under this tile's softmax
      if (tid == 0 && tile + 1 < t1) issue_k(tile + 1);

      // ---- this thread's half row of S, read once.  (Warps whose 32 rows all lie past the last
      // query row skip the row work: their rows of P and O are never stored.)
      const uint32_t sa = tmem_base + lane_base + (uint32_t)half * 64u;
      uint32_t r0[32], r1[32];
      float mx = -INFINITY;
      // A tile inside the prefix needs no masking at all.  The choice is made per warp (a warp
      // that ran both paths would pay for both): rows past the last live one count as fully
      // visible there, their values are finite and nobody reads them.
      const bool all_vis = __all_sync(0xffffffffu, vis == ~0ull || !row_valid);
      if (warp_has_rows) {
        tmem_ld32(sa, r0);
        tmem_ld32(sa + 32u, r1);
        tmem_ld_wait();
        if (all_vis) {
          float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            m0 = fmaxf(m0, fmaxf(__uint_as_float(r0[j]), __uint_as_float(r0[j + 1])));
            m1 = fmaxf(m1, fmaxf(__uint_as_float(r1[j]), __uint_as_float(r1[j + 1])));
          }
          mx = fmaxf(m0, m1);
        } else {
#pragma unroll
          for (int j = 0; j < 32; ++j) {
            if ((b0 >> j) & 1u) mx = fmaxf(mx, __uint_as_float(r0[j]));
            if ((b1 >> j) & 1u) mx = fmaxf(mx, __uint_as_float(r1[j]));
          }
        }
      }
      T.xmax[half][row] = mx;
      tc_fence_before();
      // the two warps that share 32 query rows meet (64 threads; barrier ids 1..4): both halves
      // have S in registers and their maximum out, so P may overwrite S
      asm volatile("bar.sync %0, 64;" ::"r"(quarter + 1) : "memory");
      tc_fence_after();
      mx = fmaxf(mx, T.xmax[half ^ 1][row]);
      // The reference maximum moves only when the row maximum outgrows it by more than 2^8.
      float alpha = 1.f;
      if (mx != -INFINITY && (m_run == -INFINITY || (mx - m_run) * sl2 > 8.f)) {
        alpha = (m_run == -INFINITY) ? 0.f : fast_exp2((m_run - mx) * sl2);
        m_run = mx;
      }
      const float m_sl2 = (m_run == -INFINITY) ? 0.f : m_run * sl2;
      // ---- P = exp2(S * c - max * c) as bf16, two keys per 32-bit column, back into tensor
      // memory over S (its only reader, this thread pair, is done with it); the row sum adds the
      // values before their rounding
      float lsum = 0.f;
      if (warp_has_rows) {
        uint32_t pk[32];
        float l0 = 0.f, l1 = 0.f;
        if (all_vis) {
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            const float p0 = fast_exp2(fmaf(__uint_as_float(r0[j]), sl2, -m_sl2));
            const float p1 = fast_exp2(fmaf(__uint_as_float(r0[j + 1]), sl2, -m_sl2));
            const float p2 = fast_exp2(fmaf(__uint_as_float(r1[j]), sl2, -m_sl2));
            const float p3 = fast_exp2(fmaf(__uint_as_float(r1[j + 1]), sl2, -m_sl2));
            const __nv_bfloat162 h01 = __floats2bfloat162_rn(p0, p1);
            const __nv_bfloat162 h23 = __floats2bfloat162_rn(p2, p3);
            l0 += p0 + p1;
            l1 += p2 + p3;
            pk[j >> 1] = *reinterpret_cast<const uint32_t*>(&h01);
            pk[16 + (j >> 1)] = *reinterpret_cast<const uint32_t*>(&h23);
          }
        } else {
#pragma unroll
          for (int j = 0; j < 32; j += 2) {
            const float p0 = ((b0 >> j) & 1u) ? fast_exp2(fmaf(__uint_as_float(r0[j]), sl2, -m_sl2)) : 0.f;
            const float p1 = ((b0 >> (j + 1)) & 1u)
                                 ? fast_exp2(fmaf(__uint_as_float(r0[j + 1]), sl2, -m_sl2)) : 0.f;
            const float p2 = ((b1 >> j) & 1u) ? fast_exp2(fmaf(__uint_as_float(r1[j]), sl2, -m_sl2)) : 0.f;
            const float p3 = ((b1 >> (j + 1)) & 1u)
                                 ? fast_exp2(fmaf(__uint_as_float(r1[j + 1]), sl2, -m_sl2)) : 0.f;
            const __nv_bfloat162 h01 = __floats2bfloat162_rn(p0, p1);
            const __nv_bfloat162 h23 = __floats2bfloat162_rn(p2, p3);
            l0 += p0 + p1;
            l1 += p2 + p3;
            pk[j >> 1] = *reinterpret_cast<const uint32_t*>(&h01);
            pk[16 + (j >> 1)] = *reinterpret_cast<const uint32_t*>(&h23);
          }
        }
        lsum = l0 + l1;
        tmem_st32(tmem_base + lane_base + (uint32_t)half * 32u, pk);
        // rescale this thread's half of the running output when some row of the warp moved its
        // reference (the previous tile's P V product has completed: the loop waits for it)
        if (tile > t0 && __any_sync(0xffffffffu, alpha != 1.f)) {
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
        tmem_st_wait();
      }
      l_run = l_run * alpha + lsum;
      // Cache rows past the last live key (only the sequence's last tile has any) may hold
      // anything, NaN bit patterns included, and 0 * NaN would poison every output row: they are
      // cleared in the V tile before the second product reads it.
      const int live = Ltot - tile * ATC_KEYS;
      if (live < ATC_KEYS) {
        ok = ok && mbar_wait(&T.bar_v, ph, abort_flag, status);
        if (ok) {
          const int n16 = (ATC_KEYS - live) * 8;               // 16-byte pieces per 64-wide block
          for (int idx = tid; idx < n16 * KB; idx += ATC_THREADS) {
            const int kb = idx / n16, rem = idx % n16;
            *reinterpret_cast<uint4*>(sv + kb * 16384 + (live + (rem >> 3)) * 128 + ((rem & 7) << 4)) =
                make_uint4(0u, 0u, 0u, 0u);
          }
        }
        fence_proxy_async_smem();
      }
      tc_fence_before();
      __syncthreads();
      if (tid == 0) {
        ok = ok && mbar_wait(&T.bar_v, ph, abort_flag, status);
        if (ok) {
          tc_fence_after();
          const uint32_t va = smem_u32(sv);
#pragma unroll
          for (int j = 0; j < ATC_KEYS / 16; ++j)
            tc_mma_bf16_ts(tmem_base + O_COL, tmem_base + (uint32_t)(j * 8),
                           smem_desc_mn_sw128(va + j * 2048, 16384), idesc_pv,
                           (tile > t0 || j > 0) ? 1u : 0u);
          tc_commit(&T.bar_o);
        }
      }
      ok = ok && mbar_wait(&T.bar_o, ph, abort_flag, status);
      if (!__syncthreads_and(ok)) { ok = false; break; }
      tc_fence_after();
      if (tid == 0 && tile + 1 < t1) issue_v(tile + 1);
    }
    if (ok) {
      // The partial O goes through shared memory (over the K and V tiles: every MMA has
      // completed) so that it leaves in whole 512-byte rows: a thread per row storing straight
      // from its registers would touch 32 different rows with every store instruction.
      // 16-byte chunk c of row t sits at chunk index c * 128 + (t ^ c), which the row-per-lane
      // writes and the chunk-per-lane reads both reach without bank conflicts.
      float4* so4 = reinterpret_cast<float4*>(skp);
      constexpr int NC4 = D / 4;                       // chunks of a row
      if (warp_has_rows) {
#pragma unroll 1
        for (int c = 0; c < D / 64; ++c) {
          uint32_t r[32];
          tmem_ld32(tmem_base + lane_base + O_COL + (uint32_t)(half * (D / 2) + c * 32), r);
          tmem_ld_wait();
#pragma unroll
          for (int j = 0; j < 8; ++j) {
            const int c4 = half * (NC4 / 2) + c * 8 + j;
            so4[c4 * ATC_ROWS + (row ^ (c4 & 31))] =
                make_float4(__uint_as_float(r[4 * j]), __uint_as_float(r[4 * j + 1]),
                            __uint_as_float(r[4 * j + 2]), __uint_as_float(r[4 * j + 3]));
          }
        }
      }
      __syncthreads();
      const int lane = tid & 31;
      const int rows_here = min(ATC_ROWS, n_rows - row0);
      if (lane < NC4) {
        for (int r = warp; r < rows_here; r += ATC_THREADS / 32) {
          const int gg = (row0 + r) / M, ii = (row0 + r) % M;
          const size_t orr = ((size_t)b * M + ii) * Hq + kvh * G + gg;
          *reinterpret_cast<float4*>(part_o + ((size_t)split * n_out + orr) * D + lane * 4) =
              so4[lane * ATC_ROWS + (r ^ (lane & 31))];
        }
      }
    } else if (tid == 0) {
      // gave up, possibly with copies still in flight: give them a bounded time to land
      const unsigned long long ts = global_ns();
      while (global_ns() - ts < 2000000ull) { /* 2 ms: far longer than any TMA copy */ }
    }
    T.xsum[half][row] = l_run;
  }
  tc_fence_before();
  __syncthreads();
  if (warp == 0) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
  if (row_valid && ok && half == 0) {
    part_ml[((size_t)split * n_out + orow) * 2] = (m_run == -INFINITY) ? -INFINITY : m_run * scale;
    part_ml[((size_t)split * n_out + orow) * 2 + 1] = have_keys ? l_run + T.xsum[1][row] : 0.f;
  }
  // Only now may the next kernel of the stream be scheduled: CTAs of a dependent grid that sit on
  // an SM in their grid-dependency wait were measured to slow the warps still working there.
  jk_pdl_trigger();
}

// jk_attn.cu
int jk_attn_combine_launch(jk_ctx* ctx, cudaStream_t st, int n_split, size_t n_out, void* out);

struct atc_map_entry {
  const void* ptr;
  int64_t sb, sh;
  int rows;
  CUtensorMap map;
};
struct atc_state {
  atc_map_entry e[256];
  int n, next;
  int smem_set;
};

static const CUtensorMap* atc_map(jk_ctx* ctx, atc_state* s, const void* ptr, int64_t sb, int64_t sh,
                                  int rows) {
  for (int i = 0; i < s->n; ++i)
    if (s->e[i].ptr == ptr && s->e[i].sb == sb && s->e[i].sh == sh && s->e[i].rows == rows)
      return &s->e[i].map;
  const int slot = s->n < 256 ? s->n++ : (s->next++ & 255);
  atc_map_entry& e = s->e[slot];
  const jk_config& c = ctx->cfg;
  const uint64_t dims[4] = {(uint64_t)c.head_dim, (uint64_t)rows, (uint64_t)c.n_kv_heads,
                            (uint64_t)c.max_batch};
  const uint64_t strides[3] = {(uint64_t)c.head_dim * 2, (uint64_t)sh * 2, (uint64_t)sb * 2};
  const uint32_t box[4] = {64, ATC_KEYS, 1, 1};
  if (jk_tma_encode_bf16(ctx, &e.map, ptr, 4, dims, strides, box) != JK_OK) {
    e.ptr = nullptr;
    return nullptr;
  }
  e.ptr = ptr; e.sb = sb; e.sh = sh; e.rows = rows;
  return &e.map;
}

void jk_attn_tc_destroy(jk_ctx* ctx) {
  if (ctx && ctx->attn_tc_state) {
    free(ctx->attn_tc_state);
    ctx->attn_tc_state = nullptr;
  }
}

// Tensor maps of a K and a V cache (cached per pointer and strides).
// The maps are handed out by value: a later lookup may recycle the slot an earlier one returned.
int jk_attn_tc_maps(jk_ctx* ctx, const void* kc, const void* vc, int64_t sb, int64_t sh,
                    int cache_rows, CUtensorMap* mk, CUtensorMap* mv) {
  if (!ctx->attn_tc_state) {
    ctx->attn_tc_state = calloc(1, sizeof(atc_state));
    if (!ctx->attn_tc_state) return JK_ERR_CUDA;
  }
  atc_state* s = (atc_state*)ctx->attn_tc_state;
  const CUtensorMap* m = atc_map(ctx, s, kc, sb, sh, cache_rows);
  if (!m) return JK_ERR_CUDA;
  *mk = *m;
  m = atc_map(ctx, s, vc, sb, sh, cache_rows);
  if (!m) return JK_ERR_CUDA;
  *mv = *m;
  return JK_OK;
}

// jk_attn_cl.cu: the cluster-merged kernel for small calls
int jk_attn_cl_plan(jk_ctx* ctx, int B, int M, int cache_rows);
int jk_attn_cl(jk_ctx* ctx, cudaStream_t st, int n_split, int B, int M, const void* q,
               const void* kc, const void* vc, int64_t sb, int64_t sh, int cache_rows,
               const int32_t* kv_len, const int32_t* parent, float scale, void* out);

// jk_attn_sk.cu: the persistent pipelined kernel
int jk_attn_sk_usable(const jk_ctx* ctx, int B, int M, int cache_rows);
int jk_attn_sk(jk_ctx* ctx, cudaStream_t st, int B, int M, const void* q, const void* kc,
               const void* vc, int64_t sb, int64_t sh, int cache_rows, const int32_t* kv_len,
               const int32_t* parent, float scale, void* out);

int jk_attn_tc(jk_ctx* ctx, cudaStream_t st, int B, int M, const void* q, const void* kc,
               const void* vc, int64_t sb, int64_t sh, int cache_rows, const int32_t* kv_len,
               const int32_t* parent, float scale, void* out) {
  const jk_config& c = ctx->cfg;
  const jk_ws_layout& L = ctx->lay;
  // The persistent kernel wins where the call is bound by streaming K and V and every SM has
  // many key tiles to walk: one query block per kv head (at most 128 (q head, node) rows share a
  // K/V tile) and at least 16 tiles per SM.  Measured, persistent against per-slice: 50 against
  // 65 us (40 heads, batch 4, prefix 2048), 261 against 410 us (batch 8, prefix 8192), but 32
  // against 30 us at 9 tiles per SM.  With several query blocks per kv head the call is bound by
  // the tensor pipe and the exponentials, and two per-slice CTAs per SM overlap those better
  // than one persistent CTA does (64 q / 8 kv heads, batch 8, prefix 8192: 218 against 228 us).
  {
    const int Gq = c.n_q_heads / c.n_kv_heads;
    const int n_qblk = (Gq * M + ATC_ROWS - 1) / ATC_ROWS;
    const long long units = (long long)B * c.n_kv_heads * n_qblk *
                            ((cache_rows + ATC_KEYS - 1) / ATC_KEYS);
    const bool want = ctx->attn_kernel == 2 ||
                      (ctx->attn_kernel == 0 && n_qblk == 1 && units >= 16ll * ctx->sm_count);
    if (want && jk_attn_sk_usable(ctx, B, M, cache_rows))
      return jk_attn_sk(ctx, st, B, M, q, kc, vc, sb, sh, cache_rows, kv_len, parent, scale, out);
  }
  // Opt-in (mode 3): the slices of a query block form a cluster and merge through distributed
  // shared memory, when a cluster size exists whose whole grid is resident at once.  It saves the
  // partials' trip through global memory and the merge launch, but with one CTA per SM its two or
  // three key tiles per CTA run one after the other, and at the benchmarked shapes it measured
  // slower than one CTA per slice (17.4 against 13.8 us at the LLaMA2-7B shape).
  if (ctx->attn_kernel == 3) {
    const int ns = jk_attn_cl_plan(ctx, B, M, cache_rows);
    if (ns > 0)
      return jk_attn_cl(ctx, st, ns, B, M, q, kc, vc, sb, sh, cache_rows, kv_len, parent, scale,
                        out);
  }
  CUtensorMap mk, mv;
  if (jk_attn_tc_maps(ctx, kc, vc, sb, sh, cache_rows, &mk, &mv) != JK_OK) return JK_ERR_CUDA;
  atc_state* s = (atc_state*)ctx->attn_tc_state;
  const int G = c.n_q_heads / c.n_kv_heads;
  const int n_qblk = (G * M + ATC_ROWS - 1) / ATC_ROWS;
  const int base = n_qblk * c.n_kv_heads * B;
  const int tiles_max = (cache_rows + ATC_KEYS - 1) / ATC_KEYS;
  // as many key slices as keep all CTAs resident at once (two per SM): one wave
  int n_split = (2 * ctx->sm_count) / base;
  if (n_split > tiles_max) n_split = tiles_max;
  if (n_split > L.attn_max_split) n_split = L.attn_max_split;
  if (n_split < 1) n_split = 1;
  const int D = c.head_dim;
  const size_t smem = (size_t)ATC_ROWS * D * 2 + 2 * ATC_ROWS * 64 * 2 + (size_t)ATC_KEYS * D * 2 +
                      sizeof(atc_tail) + 1024;
  float* part_o = (float*)(ctx->ws + L.attn_o);
  float* part_ml = (float*)(ctx->ws + L.attn_ml);
  int32_t* status = (int32_t*)(ctx->ws + L.status);
  const dim3 grid(n_split * n_qblk, c.n_kv_heads, B);
  if (!s->smem_set) {
    JK_CUDA_CHECK(ctx, cudaFuncSetAttribute(k_tree_attn_tc<128>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024));
    JK_CUDA_CHECK(ctx, cudaFuncSetAttribute(k_tree_attn_tc<64>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, 100 * 1024));
    s->smem_set = 1;
  }
  JK_PROF(ctx, st, ctx->st_attn);
  if (D == 128)
    jk_launch_pdl(k_tree_attn_tc<128>, dim3(grid), dim3(ATC_THREADS), smem, st, mk, mv, (const __nv_bfloat16*)q, kv_len, parent,
                                                 scale, M, c.n_q_heads, c.n_kv_heads, n_split,
                                                 n_qblk, cache_rows, part_o, part_ml,
                                                 (__nv_bfloat16*)out, status);
  else
    jk_launch_pdl(k_tree_attn_tc<64>, dim3(grid), dim3(ATC_THREADS), smem, st, mk, mv, (const __nv_bfloat16*)q, kv_len, parent,
                                                scale, M, c.n_q_heads, c.n_kv_heads, n_split,
                                                n_qblk, cache_rows, part_o, part_ml,
                                                (__nv_bfloat16*)out, status);
  JK_LAUNCH_CHECK(ctx);
  return jk_attn_combine_launch(ctx, st, n_split, (size_t)B * M * c.n_q_heads, out);
}
