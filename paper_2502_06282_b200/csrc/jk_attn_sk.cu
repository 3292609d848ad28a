// Persistent, pipelined tensor-core kernel of jk_tree_verify_attn for bf16 (arXiv 2502.06282,
// Sec. 2.1 step 2, mask of Fig. 4).
//
// Work is counted in units of one (sequence, kv head, block of 128 query rows, tile of 128 keys).
// The U units of a call, ordered by sequence, kv head, query block and key tile, are dealt evenly
// to one CTA per SM: CTA j takes units [floor(j U / n), floor((j + 1) U / n)).  A CTA's range is a
// list of segments, each a run of key tiles of one query block; a query block whose tiles are
// spread over several CTAs gets one unnormalised partial (max, sum, O) per CTA, numbered from the
// first CTA that touches it, and the merge kernel below combines them.
//
// Inside the CTA the roles are split across warps and every stage is buffered at least twice, so
// that the copy of tile i+2, the S product of tile i+1 and the softmax of tile i run at the same
// time:
//   warp 0      TMA producer (a ring of three K tiles and one of two or three V tiles)
//   warp 1      MMA issuer: S = Q K^T into one of three tensor-memory buffers, then O += P V with
//               P taken from tensor memory as the A operand and V MN-major straight from its
//               row-major tile.  It polls for whichever of "next S" and "this P V" has its inputs
//               first, without parking on either.
//   warps 2-9   softmax: two threads per query row, each owning 64 of the tile's 128 keys; one
//               read of S into registers, the tree mask (a visibility word built from the node's
//               ancestor set and the prefix length; a tile inside the prefix takes a path without
//               any masking, chosen per warp), the halves' maxima exchanged through shared
//               memory, P = exp2(S * c - max * c) packed to bf16 and stored over S in tensor
//               memory.  The reference maximum only moves when it is outgrown by more than 2^8, so
//               O is rarely rescaled and the softmax of a tile seldom has to wait for the tile
//               before it.  At a segment's end they request the next segment's query rows, stage
//               them as soon as the last product has completed, and only then store the partial,
//               laid out [slice][query block][16-byte piece][row] so that a warp's 32 rows write
//               512 contiguous bytes per instruction.
// 190 to 220 KB of shared memory and 512 tensor-memory columns per CTA.  All waits are bounded
// mbarrier waits (no named barriers), so a role that gives up cannot leave another one waiting
// for ever.
#include <math.h>
#include <stdlib.h>

#include "jk_common.cuh"
#include "jk_tcgen05.cuh"

#define ASK_ROWS 128
#define ASK_KEYS 128
#define ASK_THREADS 320
#define ASK_SM_THREADS 256
#define ASK_NK 3                    // K tiles in the ring
#define ASK_NV_MAX 3                // V tiles in the ring: 3 with a 64-row Q tile, else 2
#define ASK_NS 3                    // S / P buffers in tensor memory (128 columns each)
#define ASK_MAX_UNITS_X_CTAS 0x7fffffffu   // unit index * CTA count stays in 32 bits

struct ask_tail {
  uint64_t k_full[ASK_NK], v_full[ASK_NV_MAX], k_empty[ASK_NK], v_empty[ASK_NV_MAX], s_full[ASK_NS];
  uint64_t p_full[ASK_NS], p_free[ASK_NS], q_full, par_full, o_ready;
  uint64_t pair[4];                  // the two threads of a row meet here (64 arrivals)
  uint32_t tmem_base;
  int abort_flag;
  int bad;
  int parent[JK_MAX_TREE];
  int tiles[JK_MAX_ROWS];            // key tiles of every sequence
  int plen[JK_MAX_ROWS];             // prefix length of every sequence
  float xmax[ASK_NS][2][ASK_ROWS];   // [S buffer][key half][row]: tile maximum of that half
};

struct ask_plan {
  uint32_t U;       // units of the call
  uint32_t n;       // CTAs that take part
};
struct ask_seg {
  int b, kvh, qblk, tile_lo, tile_hi, slice;
};

// CTA that owns unit x when U units are dealt to n CTAs as [floor(j U / n), floor((j+1) U / n))
__device__ __forceinline__ uint32_t ask_owner(uint32_t x, const ask_plan& pl) {
  return ((x + 1u) * pl.n - 1u) / pl.U;
}
__device__ __forceinline__ uint32_t ask_range_start(uint32_t cta, const ask_plan& pl) {
  return (uint32_t)(((unsigned long long)cta * pl.U) / pl.n);
}

// U and the number of participating CTAs.  Every range is at least
// max(min_units, ceil(Tmax / (max_split - 2))) units long, so that no query block is spread over
// more than max_split - 1 CTAs.
__device__ __forceinline__ ask_plan ask_make_plan(const int* tiles, int B, int items_per_b,
                                                  int n_cta, int max_split, int min_units) {
  uint32_t U = 0;
  int tmax = 1;
  for (int b = 0; b < B; ++b) {
    U += (uint32_t)tiles[b] * (uint32_t)items_per_b;
    tmax = max(tmax, tiles[b]);
  }
  int cmin = (tmax + max_split - 3) / (max_split - 2);
  if (cmin < min_units) cmin = min_units;
  uint32_t n = U / (uint32_t)cmin;
  if (n > (uint32_t)n_cta) n = (uint32_t)n_cta;
  if (n < 1u) n = 1u;
  ask_plan p;
  p.U = U;
  p.n = n;
  return p;
}

// The segment that starts at unit x of a range that ends at x1.
__device__ __forceinline__ ask_seg ask_segment(const int* tiles, int B, int items_per_b, int n_qblk,
                                               uint32_t x, uint32_t x1, const ask_plan& pl,
                                               int cta) {
  uint32_t base = 0;
  int b = 0;
  for (; b < B - 1; ++b) {
    const uint32_t span = (uint32_t)tiles[b] * (uint32_t)items_per_b;
    if (x < base + span) break;
    base += span;
  }
  const uint32_t Tb = (uint32_t)tiles[b];
  const uint32_t rem = x - base;
  const uint32_t item = rem / Tb;
  ask_seg s;
  s.b = b;
  s.kvh = (int)(item / (uint32_t)n_qblk);
  s.qblk = (int)(item % (uint32_t)n_qblk);
  s.tile_lo = (int)(rem - item * Tb);
  const uint32_t left = x1 - x;
  s.tile_hi = (int)min(Tb, (uint32_t)s.tile_lo + left);
  s.slice = cta - (int)ask_owner(base + item * Tb, pl);
  return s;
}

// QR = rows of the Q tile kept in shared memory: 64 when a query block has at most 64 live rows
// (the product still spans 128 rows; rows 64..127 then read whatever follows the Q tile, and their
// results, which no one reads, stay in their own rows), which leaves room for a third V tile.
template <int D, int QR>
__global__ void __launch_bounds__(ASK_THREADS, 1) k_tree_attn_sk(
    const __grid_constant__ CUtensorMap map_k, const __grid_constant__ CUtensorMap map_v,
    const __nv_bfloat16* __restrict__ q, const int32_t* __restrict__ kv_len,
    const int32_t* __restrict__ parent, float scale, int B, int M, int Hq, int Hkv, int max_split,
    int min_units, int cache_rows, float* __restrict__ part_o, float* __restrict__ part_ml,
    int32_t* status) {
  constexpr int KB = D / 64;
  constexpr int ASK_NV = QR == 64 ? 3 : 2;
  constexpr int Q_BYTES = QR * D * 2;
  constexpr int Q_KB = QR * 128;                   // bytes of one 64-column block of the Q tile
  constexpr int KV_BYTES = ASK_KEYS * D * 2;
  constexpr uint32_t TMEM_COLS = 512;
  constexpr uint32_t O_COL = ASK_NS * 128;
  static_assert(O_COL + D <= TMEM_COLS, "S buffers and O must fit the tensor memory of an SM");
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  unsigned char* sq = smem;
  unsigned char* sk = sq + Q_BYTES;
  unsigned char* sv = sk + ASK_NK * KV_BYTES;
  ask_tail& T = *reinterpret_cast<ask_tail*>(sv + ASK_NV * KV_BYTES);
  volatile int* abort_flag = &T.abort_flag;

  const int G = Hq / Hkv;
  const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
  const int n_rows = G * M;
  const int n_qblk = (n_rows + ASK_ROWS - 1) / ASK_ROWS;
  const int items_per_b = Hkv * n_qblk;
  const size_t n_out = (size_t)B * M * Hq;
  if (tid == 0) {
    for (int i = 0; i < ASK_NK; ++i) { mbar_init(&T.k_full[i], 1); mbar_init(&T.k_empty[i], 1); }
    for (int i = 0; i < ASK_NV; ++i) { mbar_init(&T.v_full[i], 1); mbar_init(&T.v_empty[i], 1); }
    for (int i = 0; i < ASK_NS; ++i) {
      mbar_init(&T.s_full[i], 1); mbar_init(&T.p_free[i], 1);
      mbar_init(&T.p_full[i], ASK_SM_THREADS);
    }
    mbar_init(&T.o_ready, 1);
    mbar_init(&T.q_full, ASK_SM_THREADS);
    mbar_init(&T.par_full, ASK_SM_THREADS);
    for (int i = 0; i < 4; ++i) mbar_init(&T.pair[i], 64);
    T.abort_flag = 0;
    T.bad = 0;
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(&T.tmem_base, TMEM_COLS);
    tmem_relinquish();
  }
  __syncthreads();
  // everything above touches no global memory; kv_len may be the product of the kernel before
  jk_pdl_wait();
  for (int i = tid; i < B; i += ASK_THREADS) {
    const int P = kv_len[i];
    const bool bad = P < 0 || P + M > cache_rows;
    T.plen[i] = P;
    T.tiles[i] = bad ? 1 : (P + M + ASK_KEYS - 1) / ASK_KEYS;
    if (bad) T.bad = 1;
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = T.tmem_base;
  const bool bad = T.bad != 0;
  if (bad && blockIdx.x == 0 && tid == 0) jk_set_status(status, JK_ERR_BOUNDS);
  const ask_plan pl = ask_make_plan(T.tiles, B, items_per_b, (int)gridDim.x, max_split, min_units);
  const int cta = (int)blockIdx.x;
  uint32_t x0 = 0, x1 = 0;
  if (!bad && (uint32_t)cta < pl.n) {
    x0 = ask_range_start((uint32_t)cta, pl);
    x1 = ask_range_start((uint32_t)cta + 1u, pl);
  }
  bool ok = true;

  if (warp == 0) {
    // ------------------------------------------------------------------ TMA producer
    // K runs one tile ahead of V: the K buffer of tile g is free as soon as S of tile g - ASK_NK
    // has completed, the V buffer only after the second product of tile g - ASK_NV.
    if (lane == 0) {
      const uint64_t pol = l2_policy_evict_first();   // the cache is read once per call
      int g = 0;
      int pt = 0, pkvh = 0, pb = 0;                 // coordinates of tile g-1 (its V is still due)
      auto load_v = [&](int gv, int t, int kvh, int b) -> bool {
        const int bf = gv % ASK_NV;
        if (gv >= ASK_NV &&
            !mbar_wait(&T.v_empty[bf], (uint32_t)(gv / ASK_NV - 1) & 1u, abort_flag, status))
          return false;
        mbar_expect_tx(&T.v_full[bf], KV_BYTES);
#pragma unroll
        for (int kb = 0; kb < KB; ++kb)
          tma_load_4d_hint(sv + bf * KV_BYTES + kb * 16384, &map_v, kb * 64, t * ASK_KEYS, kvh, b,
                           &T.v_full[bf], pol);
        return true;
      };
      for (uint32_t x = x0; x < x1 && ok;) {
        const ask_seg s = ask_segment(T.tiles, B, items_per_b, n_qblk, x, x1, pl, cta);
        for (int t = s.tile_lo; t < s.tile_hi; ++t, ++g) {
          const int bf = g % ASK_NK;
          if (g >= ASK_NK)
            ok = mbar_wait(&T.k_empty[bf], (uint32_t)(g / ASK_NK - 1) & 1u, abort_flag, status);
          if (!ok) break;
          mbar_expect_tx(&T.k_full[bf], KV_BYTES);
#pragma unroll
          for (int kb = 0; kb < KB; ++kb)
            tma_load_4d_hint(sk + bf * KV_BYTES + kb * 16384, &map_k, kb * 64, t * ASK_KEYS, s.kvh,
                             s.b, &T.k_full[bf], pol);
          if (g >= 1) ok = load_v(g - 1, pt, pkvh, pb);
          if (!ok) break;
          pt = t; pkvh = s.kvh; pb = s.b;
        }
        x += (uint32_t)(s.tile_hi - s.tile_lo);
      }
      if (ok && g >= 1) ok = load_v(g - 1, pt, pkvh, pb);
    }
  } else if (warp == 1) {
    // ------------------------------------------------------------------ MMA issuer
    if (lane == 0) {
      const uint32_t idesc_s = instr_desc_bf16_ex(ASK_KEYS, 0);
      const uint32_t idesc_pv = instr_desc_bf16_ex(D, 1);
      const uint32_t qa = smem_u32(sq);
      // The S buffer of tile g holds P of tile g until the P V product of tile g has read it, so
      // S of tile g + ASK_NS (same buffer) is issued only once that product has completed, which
      // is what p_free signals (the tensor core gives no ordering between a product's operand
      // reads from tensor memory and a later product's writes there).
      auto s_ready = [&](int g) -> bool {
        const int bf = g % ASK_NS;
        const uint32_t ph = (uint32_t)(g / ASK_NS) & 1u;
        return mbar_test(&T.k_full[g % ASK_NK], (uint32_t)(g / ASK_NK) & 1u) &&
               (g < ASK_NS || mbar_test(&T.p_free[bf], ph ^ 1u));
      };
      auto issue_s = [&](int g) -> bool {
        const int bf = g % ASK_NS, kbf = g % ASK_NK;
        const uint32_t ph = (uint32_t)(g / ASK_NS) & 1u;
        if (!mbar_wait(&T.k_full[kbf], (uint32_t)(g / ASK_NK) & 1u, abort_flag, status)) return false;
        if (g >= ASK_NS && !mbar_wait(&T.p_free[bf], ph ^ 1u, abort_flag, status)) return false;
        tc_fence_after();
        const uint32_t ka = smem_u32(sk + kbf * KV_BYTES);
#pragma unroll
        for (int kb = 0; kb < KB; ++kb)
#pragma unroll
          for (int k = 0; k < 4; ++k)
            tc_mma_bf16(tmem_base + (uint32_t)bf * 128u, smem_desc_sw128(qa + kb * Q_KB + k * 32),
                        smem_desc_sw128(ka + kb * 16384 + k * 32), idesc_s, (kb | k) ? 1u : 0u);
        tc_commit(&T.s_full[bf]);
        tc_commit(&T.k_empty[kbf]);
        return true;
      };
      int g = 0, seg = 0;
      for (uint32_t x = x0; x < x1 && ok; ++seg) {
        const ask_seg s = ask_segment(T.tiles, B, items_per_b, n_qblk, x, x1, pl, cta);
        ok = mbar_wait(&T.q_full, (uint32_t)seg & 1u, abort_flag, status);
        ok = ok && issue_s(g);
        for (int t = s.tile_lo; t < s.tile_hi && ok; ++t, ++g) {
          const int bf = g % ASK_NS;
          const int vbf = g % ASK_NV;
          // The next kernel of the stream (the merge) may be scheduled once every CTA has reached
          // its last tile: its launch and its prologue then pass under the tail of this kernel,
          // while its CTAs do not sit on the SMs for long (they were measured to slow this kernel's
          // warps when they arrive early).
          // Two things are due, in whichever order their inputs arrive: S of the next tile (its K
          // tile has landed and its buffer is free) and P V of this tile (P written, V landed).
          bool s_due = t + 1 < s.tile_hi, pv_due = true;
          const long long w0 = clock64();
          for (unsigned it = 1; ok && (s_due || pv_due); ++it) {
            if (s_due && s_ready(g + 1)) {
              ok = issue_s(g + 1);
              s_due = false;
              continue;
            }
            if (pv_due && mbar_test(&T.p_full[bf], (uint32_t)(g / ASK_NS) & 1u) &&
                mbar_test(&T.v_full[vbf], (uint32_t)(g / ASK_NV) & 1u)) {
              tc_fence_after();
              const uint32_t va = smem_u32(sv + vbf * KV_BYTES);
#pragma unroll
              for (int j = 0; j < ASK_KEYS / 16; ++j)
                tc_mma_bf16_ts(tmem_base + O_COL, tmem_base + (uint32_t)bf * 128u + (uint32_t)(j * 8),
                               smem_desc_mn_sw128(va + j * 2048, 16384), idesc_pv,
                               (t > s.tile_lo || j > 0) ? 1u : 0u);
              tc_commit(&T.v_empty[vbf]);
              tc_commit(&T.p_free[bf]);
              pv_due = false;
              continue;
            }
            __nanosleep(40);               // leave the issue slots to the softmax warps of this quarter
            if ((it & 255u) == 0) {
              if (*abort_flag) ok = false;
              else if (clock64() - w0 > TC_WAIT_CYCLES) {
                *abort_flag = 1;
                jk_set_status(status, JK_ERR_TIMEOUT);
                ok = false;
              }
            }
          }
        }
        // the segment's O is complete: pass that on through a barrier this thread arrives on
        // (p_free of the last tile's buffer: the phase before it completed before that tile's S
        // was issued, so the parity cannot be mistaken for an older one)
        ok = ok && mbar_wait(&T.p_free[(g - 1) % ASK_NS], (uint32_t)((g - 1) / ASK_NS) & 1u, abort_flag,
                             status);
        if (ok) mbar_arrive(&T.o_ready);
        x += (uint32_t)(s.tile_hi - s.tile_lo);
      }
    }
  } else {
    // ------------------------------------------------------------------ softmax (2 threads / row)
    // tensor-memory lane quarter = warp % 4, key half = (warp - 2) / 4
    const int quarter = warp & 3, half = (warp - 2) >> 2;
    const int row = quarter * 32 + lane;
    const int sm_tid = tid - 64;
    const uint32_t lane_base = (uint32_t)(quarter * 32) << 16;
    const float sl2 = scale * 1.4426950408889634f;
    constexpr int QV = D / 16;                       // 16-byte vectors of half a query row
    int g = 0, seg = 0;
    uint32_t pair_uses = 0;
    auto pair_sync = [&]() -> bool {
      mbar_arrive(&T.pair[quarter]);
      const bool o = mbar_wait(&T.pair[quarter], pair_uses & 1u, abort_flag, status);
      ++pair_uses;
      return __all_sync(0xffffffffu, o);
    };
    // Per segment: where this thread's row lives.  The query rows and the tree of the NEXT segment
    // are fetched while the last product of the current one drains, and staged as soon as that
    // product has completed, so that the next segment's first S runs under this one's epilogue.
    struct seg_row { bool row_valid, warp_active; int node; size_t orow; };
    auto row_of = [&](const ask_seg& sg) -> seg_row {
      seg_row r;
      const int row0 = sg.qblk * ASK_ROWS;
      r.row_valid = row0 + row < n_rows;
      r.warp_active = row0 + quarter * 32 < n_rows;
      const int g_idx = r.row_valid ? (row0 + row) / M : 0;
      r.node = r.row_valid ? (row0 + row) % M : 0;
      r.orow = ((size_t)sg.b * M + r.node) * Hq + sg.kvh * G + g_idx;
      return r;
    };
    uint4 qv[QV];
    auto fetch_q = [&](const seg_row& r) {
#pragma unroll
      for (int c = 0; c < QV; ++c) {
        qv[c] = make_uint4(0u, 0u, 0u, 0u);
        if (r.row_valid)
          qv[c] = __ldg(reinterpret_cast<const uint4*>(q + r.orow * D + half * (D / 2) + c * 8));
      }
    };
    // (every MMA that read the Q tile has completed when this runs)
    auto stage = [&](const ask_seg& sg) {
      if (sm_tid < M) T.parent[sm_tid] = __ldg(parent + (size_t)sg.b * M + sm_tid);
      mbar_arrive(&T.par_full);
#pragma unroll
      for (int c = 0; c < QV; ++c) {
        const int ch = half * QV + c;
        if (row < QR)
          *reinterpret_cast<uint4*>(sq + (ch >> 3) * Q_KB + row * 128 + (((ch & 7) ^ (row & 7)) << 4)) =
              qv[c];
      }
      fence_proxy_async_smem();
      mbar_arrive(&T.q_full);
    };
    uint32_t x = x0;
    bool have = x < x1;
    ask_seg s{};
    if (have) {
      s = ask_segment(T.tiles, B, items_per_b, n_qblk, x, x1, pl, cta);
      fetch_q(row_of(s));
      stage(s);
    }
    for (; have; ++seg) {
      x += (uint32_t)(s.tile_hi - s.tile_lo);
      const int P = T.plen[s.b];
      const seg_row sr = row_of(s);
      const bool row_valid = sr.row_valid, warp_active = sr.warp_active;
      const int node = sr.node;
      const size_t orow = sr.orow;
      {
        const bool okp = mbar_wait(&T.par_full, (uint32_t)seg & 1u, abort_flag, status);
        ok = __all_sync(0xffffffffu, okp);
      }
      if (!ok) break;
      unsigned long long anc_lo = 0ull, anc_hi = 0ull;
      if (row_valid) {
        int c = node;
        for (int guard = 0; c >= 0 && guard <= JK_MAX_TREE; ++guard) {
          if (c < 64) anc_lo |= 1ull << c; else anc_hi |= 1ull << (c - 64);
          const int pp = T.parent[c];
          c = (pp < c) ? pp : -1;
        }
      }
      float m_run = -INFINITY, l_run = 0.f;
      for (int tile = s.tile_lo; tile < s.tile_hi; ++tile, ++g) {
        const int bf = g % ASK_NS;
        // visibility of this thread's 64 keys (Fig. 4): prefix keys, then the ancestor set
        unsigned long long vis_lo = 0ull, vis_hi = 0ull;
        if (row_valid) {
          const int sft = P - tile * ASK_KEYS;
          if (sft >= 128) { vis_lo = ~0ull; vis_hi = ~0ull; }
          else if (sft >= 0) {
            if (sft >= 64) { vis_lo = ~0ull; vis_hi = (sft == 64) ? 0ull : ((1ull << (sft - 64)) - 1ull); }
            else { vis_lo = (sft == 0) ? 0ull : ((1ull << sft) - 1ull); }
            unsigned long long a_lo, a_hi;
            if (sft == 0) { a_lo = anc_lo; a_hi = anc_hi; }
            else if (sft < 64) { a_lo = anc_lo << sft; a_hi = (anc_hi << sft) | (anc_lo >> (64 - sft)); }
            else if (sft == 64) { a_lo = 0ull; a_hi = anc_lo; }
            else { a_lo = 0ull; a_hi = anc_lo << (sft - 64); }
            vis_lo |= a_lo; vis_hi |= a_hi;
          } else {
            const int t = -sft;
            if (t < 64) { vis_lo = (anc_lo >> t) | (anc_hi << (64 - t)); vis_hi = anc_hi >> t; }
            else if (t < 128) { vis_lo = anc_hi >> (t - 64); vis_hi = 0ull; }
          }
        }
        const unsigned long long vis = half ? vis_hi : vis_lo;
        const unsigned b0 = (unsigned)vis, b1 = (unsigned)(vis >> 32);
        {
          const bool okw = mbar_wait(&T.s_full[bf], (uint32_t)(g / ASK_NS) & 1u, abort_flag, status);
          ok = __all_sync(0xffffffffu, okw);
        }
        if (!ok) break;
        tc_fence_after();
        const uint32_t sa = tmem_base + lane_base + (uint32_t)bf * 128u + (uint32_t)half * 64u;
        // this thread's half row of S, read once; the row maximum via the partner
        uint32_t r0[32], r1[32];
        float mx = -INFINITY;
        // A tile inside the prefix needs no masking at all.  The choice is made per warp (a warp
        // that ran both paths would pay for both): rows past the last live one count as fully
        // visible there, their values are finite and nobody reads them.
        const bool all_vis = __all_sync(0xffffffffu, vis == ~0ull || !row_valid);
        if (warp_active) {
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
        T.xmax[bf][half][row] = mx;
        tc_fence_before();
        ok = pair_sync();                  // both halves have S in registers: P may overwrite it
        if (!ok) break;
        tc_fence_after();
        mx = fmaxf(mx, T.xmax[bf][half ^ 1][row]);
        // The reference maximum moves only when the row maximum outgrows it by more than 2^8.
        float alpha = 1.f;
        if (mx != -INFINITY && (m_run == -INFINITY || (mx - m_run) * sl2 > 8.f)) {
          alpha = (m_run == -INFINITY) ? 0.f : fast_exp2((m_run - mx) * sl2);
          m_run = mx;
        }
        const float m_sl2 = (m_run == -INFINITY) ? 0.f : m_run * sl2;
        // P = exp2(S * scale * log2 e - max * scale * log2 e) as bf16, two keys per 32-bit column,
        // back into tensor memory over S; the row sum adds the values before their rounding
        float lsum = 0.f;
        if (warp_active) {
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
          tmem_st32(tmem_base + lane_base + (uint32_t)bf * 128u + (uint32_t)half * 32u, pk);
        }
        // O is rescaled only when some row of the warp moved its reference, and only then does
        // the softmax have to wait for the previous tile's P V product (both warps of a row pair
        // see the same rows and take the same decision)
        if (tile > s.tile_lo && __any_sync(0xffffffffu, alpha != 1.f)) {
          const bool okp = mbar_wait(&T.p_free[(g - 1) % ASK_NS], (uint32_t)((g - 1) / ASK_NS) & 1u,
                                     abort_flag, status);
          ok = __all_sync(0xffffffffu, okp);
          if (!ok) break;
          tc_fence_after();
          if (warp_active) {
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
        if (warp_active) tmem_st_wait();
        l_run = l_run * alpha + lsum;
        // Cache rows past the last live key (only a sequence's last tile has any) may hold
        // anything, NaN bit patterns included, and 0 * NaN would poison every output row: they
        // are cleared in the V tile before the second product reads it.
        const int live = P + M - tile * ASK_KEYS;
        if (live < ASK_KEYS) {
          const bool okv = mbar_wait(&T.v_full[g % ASK_NV], (uint32_t)(g / ASK_NV) & 1u, abort_flag, status);
          ok = __all_sync(0xffffffffu, okv);
          if (!ok) break;
          const int n16 = (ASK_KEYS - live) * 8;               // 16-byte pieces per 64-wide block
          unsigned char* vt = sv + (g % ASK_NV) * KV_BYTES;
          for (int idx = sm_tid; idx < n16 * KB; idx += ASK_SM_THREADS) {
            const int kb = idx / n16, rem = idx % n16;
            *reinterpret_cast<uint4*>(vt + kb * 16384 + (live + (rem >> 3)) * 128 + ((rem & 7) << 4)) =
                make_uint4(0u, 0u, 0u, 0u);
          }
        }
        fence_proxy_async_smem();
        tc_fence_before();
        mbar_arrive(&T.p_full[bf]);
      }
      if (!ok) break;
      // ---- the next segment's rows are requested now and staged once this segment's products
      //      have completed; then the segment's partial (max, sum, O) of every row
      const bool have_next = x < x1;
      ask_seg sn{};
      if (have_next) {
        sn = ask_segment(T.tiles, B, items_per_b, n_qblk, x, x1, pl, cta);
        fetch_q(row_of(sn));
      }
      {
        const bool okd = mbar_wait(&T.o_ready, (uint32_t)seg & 1u, abort_flag, status);
        ok = __all_sync(0xffffffffu, okd);
      }
      if (!ok) break;
      tc_fence_after();
      if (have_next) stage(sn);
      // The partials are laid out for this store: [slice][item][16-byte piece][row of the block],
      // so that the 32 rows of a warp write 512 contiguous bytes per instruction.  Each half row
      // stores its own sum; the merge adds the two.
      if (warp_active) {
        const size_t item = ((size_t)s.b * Hkv + s.kvh) * n_qblk + s.qblk;
        const size_t blk = (size_t)s.slice * ((size_t)B * items_per_b) + item;
        float* po = part_o + blk * ((size_t)ASK_ROWS * D) + (size_t)row * 4;
#pragma unroll 1
        for (int c = 0; c < D / 64; ++c) {
          uint32_t r[32];
          tmem_ld32(tmem_base + lane_base + O_COL + (uint32_t)(half * (D / 2) + c * 32), r);
          tmem_ld_wait();
          if (row_valid) {
#pragma unroll
            for (int j = 0; j < 32; j += 4) {
              const int piece = (half * (D / 2) + c * 32 + j) >> 2;
              *reinterpret_cast<float4*>(po + (size_t)piece * (ASK_ROWS * 4)) =
                  make_float4(__uint_as_float(r[j]), __uint_as_float(r[j + 1]),
                              __uint_as_float(r[j + 2]), __uint_as_float(r[j + 3]));
            }
          }
        }
        if (row_valid) {
          float* pm = part_ml + (blk * ASK_ROWS + row) * 4;
          if (half == 0) pm[0] = (m_run == -INFINITY) ? -INFINITY : m_run * scale;
          pm[1 + half] = l_run;
        }
      }
      tc_fence_before();
      s = sn;
      have = have_next;
    }
  }
  if (tid == 0 && *abort_flag) {
    // some role gave up, possibly with copies still in flight: give them a bounded time to land
    const unsigned long long ts = global_ns();
    while (global_ns() - ts < 2000000ull) { /* 2 ms: far longer than any TMA copy */ }
  }
  tc_fence_before();
  __syncthreads();
  jk_pdl_trigger();                  // (CTAs without work, and the ones that gave up)
  if (warp == 1) {
    tc_fence_after();
    tmem_dealloc(tmem_base, TMEM_COLS);
  }
}

// Merge of the partials of one output row (one warp per row): the number of partials of the
// row's query block follows from the same dealing of units to CTAs as in the kernel above.
template <int D>
__global__ void __launch_bounds__(256) k_attn_combine_sk(
    const float* __restrict__ part_o, const float* __restrict__ part_ml,
    const int32_t* __restrict__ kv_len, int B, int M, int Hq, int Hkv, int n_cta, int max_split,
    int min_units, int cache_rows, __nv_bfloat16* __restrict__ out) {
  __shared__ int s_tiles[JK_MAX_ROWS];
  __shared__ int s_bad;
  if (threadIdx.x == 0) s_bad = 0;
  __syncthreads();
  for (int i = threadIdx.x; i < B; i += blockDim.x) {
    const int P = kv_len[i];         // not written by the attention kernel: read before the wait
    const bool bad = P < 0 || P + M > cache_rows;
    s_tiles[i] = bad ? 1 : (P + M + ASK_KEYS - 1) / ASK_KEYS;
    if (bad) s_bad = 1;
  }
  __syncthreads();
  jk_pdl_wait();
  jk_pdl_trigger();
  if (s_bad) return;
  constexpr int DPL = D / 32;
  const int lane = threadIdx.x & 31;
  const size_t n_out = (size_t)B * M * Hq;
  const size_t row = (size_t)blockIdx.x * 8 + (threadIdx.x >> 5);
  if (row >= n_out) return;
  const int G = Hq / Hkv;
  const int n_qblk = (G * M + ASK_ROWS - 1) / ASK_ROWS;
  const int items_per_b = Hkv * n_qblk;
  const ask_plan pl = ask_make_plan(s_tiles, B, items_per_b, n_cta, max_split, min_units);
  const int head = (int)(row % Hq);
  const int node = (int)((row / Hq) % M);
  const int b = (int)(row / ((size_t)Hq * M));
  uint32_t base = 0;
  for (int i = 0; i < b; ++i) base += (uint32_t)s_tiles[i] * (uint32_t)items_per_b;
  const uint32_t Tb = (uint32_t)s_tiles[b];
  const uint32_t item = (uint32_t)((head / G) * n_qblk + ((head % G) * M + node) / ASK_ROWS);
  const uint32_t start = base + item * Tb;
  const int n_split = (int)(ask_owner(start + Tb - 1u, pl) - ask_owner(start, pl)) + 1;
  // [slice][item][16-byte piece][row of the block][4]: see the attention kernel's epilogue
  const size_t gitem = (size_t)b * items_per_b + item;
  const int lrow = ((head % G) * M + node) % ASK_ROWS;
  const size_t n_items = (size_t)B * items_per_b;
  const float* po = part_o + gitem * ((size_t)ASK_ROWS * D) +
                    ((size_t)((lane * DPL) >> 2) * ASK_ROWS + lrow) * 4 + ((lane * DPL) & 3);
  const size_t sstride = n_items * ((size_t)ASK_ROWS * D);
  auto load_batch = [&](int s0, float (&v)[4][DPL]) {   // four independent vector loads in flight
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const int s = s0 + j < n_split ? s0 + j : n_split - 1;
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
  float v[4][DPL];
  load_batch(0, v);
  // lane s holds (max, sum) of partial s (n_split < 32); one load round for all partials
  float ms = -INFINITY, ls = 0.f;
  if (lane < n_split) {
    const float4 x = *reinterpret_cast<const float4*>(
        part_ml + (((size_t)lane * n_items + gitem) * ASK_ROWS + lrow) * 4);
    ms = x.x;
    ls = x.y + x.z;
  }
  const float m = jk_warp_max(ms);
  const float w_lane = (ms == -INFINITY) ? 0.f : __expf(ms - m);
  const float l = jk_warp_sum(w_lane * ls);
  float acc[DPL];
#pragma unroll
  for (int t = 0; t < DPL; ++t) acc[t] = 0.f;
  for (int s0 = 0; s0 < n_split; s0 += 4) {
    if (s0 > 0) load_batch(s0, v);
#pragma unroll
    for (int j = 0; j < 4; ++j) {
      const float w = __shfl_sync(0xffffffffu, w_lane, (s0 + j) & 31);
      if (s0 + j < n_split && w != 0.f) {
#pragma unroll
        for (int t = 0; t < DPL; ++t) acc[t] += w * v[j][t];
      }
    }
  }
  const float inv = 1.f / l;
#pragma unroll
  for (int t = 0; t < DPL; ++t)
    out[row * D + lane * DPL + t] = __float2bfloat16_rn(acc[t] * inv);
}

// The same merge with two rows per warp (16 lanes per row, D / 16 values per lane): half as many
// warps, so that the rows of a large call (9600 at the 13B shape with batch 4, more than the
// 64 warps per SM the device holds) fit in one wave.  A lane keeps the (max, sum) of slices
// lane and lane + 16 of its row.
template <int D>
__global__ void __launch_bounds__(256, 5) k_attn_combine_sk2(
    const float* __restrict__ part_o, const float* __restrict__ part_ml,
    const int32_t* __restrict__ kv_len, int B, int M, int Hq, int Hkv, int n_cta, int max_split,
    int min_units, int cache_rows, __nv_bfloat16* __restrict__ out) {
  __shared__ int s_tiles[JK_MAX_ROWS];
  __shared__ int s_bad;
  if (threadIdx.x == 0) s_bad = 0;
  __syncthreads();
  for (int i = threadIdx.x; i < B; i += blockDim.x) {
    const int P = kv_len[i];         // not written by the attention kernel: read before the wait
    const bool bad = P < 0 || P + M > cache_rows;
    s_tiles[i] = bad ? 1 : (P + M + ASK_KEYS - 1) / ASK_KEYS;
    if (bad) s_bad = 1;
  }
  __syncthreads();
  jk_pdl_wait();
  jk_pdl_trigger();
  if (s_bad) return;
  constexpr int DPL = D / 16;        // values per lane
  constexpr int NP = DPL / 4;        // 16-byte pieces per lane
  constexpr int NBS = NP == 2 ? 3 : 4;   // slices per round of loads (48 registers a thread)
  const int lane = threadIdx.x & 31, hl = lane & 15;
  const size_t n_out = (size_t)B * M * Hq;
  const size_t row_w = (size_t)blockIdx.x * 16 + (size_t)(threadIdx.x >> 5) * 2;
  if (row_w >= n_out) return;        // both rows of the warp are past the end
  const bool live = row_w + (lane >> 4) < n_out;
  const size_t row = live ? row_w + (lane >> 4) : n_out - 1;
  const int G = Hq / Hkv;
  const int n_qblk = (G * M + ASK_ROWS - 1) / ASK_ROWS;
  const int items_per_b = Hkv * n_qblk;
  const ask_plan pl = ask_make_plan(s_tiles, B, items_per_b, n_cta, max_split, min_units);
  const int head = (int)(row % Hq);
  const int node = (int)((row / Hq) % M);
  const int b = (int)(row / ((size_t)Hq * M));
  uint32_t base = 0;
  for (int i = 0; i < b; ++i) base += (uint32_t)s_tiles[i] * (uint32_t)items_per_b;
  const uint32_t Tb = (uint32_t)s_tiles[b];
  const uint32_t item = (uint32_t)((head / G) * n_qblk + ((head % G) * M + node) / ASK_ROWS);
  const uint32_t start = base + item * Tb;
  const int n_split = (int)(ask_owner(start + Tb - 1u, pl) - ask_owner(start, pl)) + 1;
  const int n_loop = max(n_split, __shfl_xor_sync(0xffffffffu, n_split, 16));
  // [slice][item][16-byte piece][row of the block][4]: see the attention kernel's epilogue
  const size_t gitem = (size_t)b * items_per_b + item;
  const int lrow = ((head % G) * M + node) % ASK_ROWS;
  const size_t n_items = (size_t)B * items_per_b;
  const float* po = part_o + gitem * ((size_t)ASK_ROWS * D) +
                    ((size_t)(hl * NP) * ASK_ROWS + lrow) * 4;
  const size_t sstride = n_items * ((size_t)ASK_ROWS * D);
  auto load_batch = [&](int s0, float4 (&v)[NBS][NP]) {   // NBS * NP independent vector loads in flight
#pragma unroll
    for (int j = 0; j < NBS; ++j) {
      const int s = s0 + j < n_split ? s0 + j : n_split - 1;
#pragma unroll
      for (int k = 0; k < NP; ++k)
        v[j][k] = *reinterpret_cast<const float4*>(po + (size_t)s * sstride + (size_t)k * ASK_ROWS * 4);
    }
  };
  // the first batch of partial outputs is asked for before anything waits on the (max, sum) pairs
  float4 v[NBS][NP];
  load_batch(0, v);
  float ms_a = -INFINITY, ls_a = 0.f, ms_b = -INFINITY, ls_b = 0.f;
  if (hl < n_split) {
    const float4 x = *reinterpret_cast<const float4*>(
        part_ml + (((size_t)hl * n_items + gitem) * ASK_ROWS + lrow) * 4);
    ms_a = x.x;
    ls_a = x.y + x.z;
  }
  if (hl + 16 < n_split) {
    const float4 x = *reinterpret_cast<const float4*>(
        part_ml + (((size_t)(hl + 16) * n_items + gitem) * ASK_ROWS + lrow) * 4);
    ms_b = x.x;
    ls_b = x.y + x.z;
  }
  float m = fmaxf(ms_a, ms_b);
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, o));
  const float w_a = (ms_a == -INFINITY) ? 0.f : __expf(ms_a - m);
  const float w_b = (ms_b == -INFINITY) ? 0.f : __expf(ms_b - m);
  float l = w_a * ls_a + w_b * ls_b;
#pragma unroll
  for (int o = 8; o > 0; o >>= 1) l += __shfl_xor_sync(0xffffffffu, l, o);
  float acc[DPL];
#pragma unroll
  for (int t = 0; t < DPL; ++t) acc[t] = 0.f;
  for (int s0 = 0; s0 < n_loop; s0 += NBS) {
    if (s0 > 0) load_batch(s0, v);
#pragma unroll
    for (int j = 0; j < NBS; ++j) {
      const int sl = (s0 + j) & 31;
      const int src = (lane & 16) | (sl & 15);
      const float wa = __shfl_sync(0xffffffffu, w_a, src);
      const float wb = __shfl_sync(0xffffffffu, w_b, src);
      const float w = sl < 16 ? wa : wb;
      if (s0 + j < n_split && w != 0.f) {
#pragma unroll
        for (int k = 0; k < NP; ++k) {
          acc[4 * k] += w * v[j][k].x; acc[4 * k + 1] += w * v[j][k].y;
          acc[4 * k + 2] += w * v[j][k].z; acc[4 * k + 3] += w * v[j][k].w;
        }
      }
    }
  }
  if (!live) return;
  const float inv = 1.f / l;
  __nv_bfloat16* dst = out + row * D + hl * DPL;
#pragma unroll
  for (int k = 0; k < NP; ++k) {
    const __nv_bfloat162 lo = __floats2bfloat162_rn(acc[4 * k] * inv, acc[4 * k + 1] * inv);
    const __nv_bfloat162 hi = __floats2bfloat162_rn(acc[4 * k + 2] * inv, acc[4 * k + 3] * inv);
    uint2 pk;
    pk.x = *reinterpret_cast<const uint32_t*>(&lo);
    pk.y = *reinterpret_cast<const uint32_t*>(&hi);
    *reinterpret_cast<uint2*>(dst + 4 * k) = pk;
  }
}

// jk_attn_tc.cu: tensor maps of the two caches
int jk_attn_tc_maps(jk_ctx* ctx, const void* kc, const void* vc, int64_t sb, int64_t sh,
                    int cache_rows, CUtensorMap* mk, CUtensorMap* mv);

// The kernel needs room for at least three partials per query block, sequence counts that fit
// its shared arrays, and unit indices that stay in 32 bits.
int jk_attn_sk_usable(const jk_ctx* ctx, int B, int M, int cache_rows) {
  const jk_config& c = ctx->cfg;
  if (ctx->lay.attn_max_split < 4 || B > JK_MAX_ROWS || ctx->sm_count < 1) return 0;
  const int G = c.n_q_heads / c.n_kv_heads;
  const unsigned long long units = (unsigned long long)B * c.n_kv_heads *
                                   ((G * M + ASK_ROWS - 1) / ASK_ROWS) *
                                   ((cache_rows + ASK_KEYS - 1) / ASK_KEYS);
  return units * (unsigned long long)ctx->sm_count <= ASK_MAX_UNITS_X_CTAS;
}

int jk_attn_sk(jk_ctx* ctx, cudaStream_t st, int B, int M, const void* q, const void* kc,
               const void* vc, int64_t sb, int64_t sh, int cache_rows, const int32_t* kv_len,
               const int32_t* parent, float scale, void* out) {
  const jk_config& c = ctx->cfg;
  const jk_ws_layout& L = ctx->lay;
  CUtensorMap mk, mv;
  int rc = jk_attn_tc_maps(ctx, kc, vc, sb, sh, cache_rows, &mk, &mv);
  if (rc != JK_OK) return rc;
  const int D = c.head_dim;
  float* part_o = (float*)(ctx->ws + L.attn_o);
  float* part_ml = (float*)(ctx->ws + L.attn_ml);
  int32_t* status = (int32_t*)(ctx->ws + L.status);
  if (!ctx->attn_sk_smem_set) {
    const int cap = 227 * 1024;
    JK_CUDA_CHECK(ctx, cudaFuncSetAttribute(k_tree_attn_sk<128, 128>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, cap));
    JK_CUDA_CHECK(ctx, cudaFuncSetAttribute(k_tree_attn_sk<128, 64>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, cap));
    JK_CUDA_CHECK(ctx, cudaFuncSetAttribute(k_tree_attn_sk<64, 128>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, cap));
    JK_CUDA_CHECK(ctx, cudaFuncSetAttribute(k_tree_attn_sk<64, 64>,
                                            cudaFuncAttributeMaxDynamicSharedMemorySize, cap));
    ctx->attn_sk_smem_set = 1;
  }
  // a query block of at most 64 live rows keeps a 64-row Q tile and a third V tile instead
  const int G = c.n_q_heads / c.n_kv_heads;
  const int qr = (G * M <= 64) ? 64 : ASK_ROWS;
  const int nv = qr == 64 ? 3 : 2;
  const size_t smem = (size_t)qr * D * 2 + (size_t)(ASK_NK + nv) * ASK_KEYS * D * 2 +
                      sizeof(ask_tail) + 1024;
  const int n_cta = ctx->sm_count;
  const int ms = L.attn_max_split;
  const int min_units = 1;
  JK_PROF(ctx, st, ctx->st_attn);
#define ASK_LAUNCH(DD, QQ)                                                                        \
  jk_launch_pdl(k_tree_attn_sk<DD, QQ>, dim3(n_cta), dim3(ASK_THREADS), smem, st, mk, mv,         \
                (const __nv_bfloat16*)q, kv_len, parent, scale, B, M, c.n_q_heads, c.n_kv_heads,  \
                ms, min_units, cache_rows, part_o, part_ml, status)
  if (D == 128) {
    if (qr == 64) ASK_LAUNCH(128, 64); else ASK_LAUNCH(128, 128);
  } else {
    if (qr == 64) ASK_LAUNCH(64, 64); else ASK_LAUNCH(64, 128);
  }
#undef ASK_LAUNCH
  JK_LAUNCH_CHECK(ctx);
  const size_t n_out = (size_t)B * M * c.n_q_heads;
  JK_PROF(ctx, st, ctx->st_combine);
  // more rows than the device holds warps at once: two rows per warp keep the merge in one wave
  const bool two = n_out > (size_t)ctx->sm_count * 48;
  if (D == 128 && two)
    jk_launch_pdl(k_attn_combine_sk2<128>, dim3((unsigned)((n_out + 15) / 16)), dim3(256), 0, st,
                  (const float*)part_o, (const float*)part_ml, kv_len, B, M, c.n_q_heads,
                  c.n_kv_heads, n_cta, ms, min_units, cache_rows, (__nv_bfloat16*)out);
  else if (D == 64 && two)
    jk_launch_pdl(k_attn_combine_sk2<64>, dim3((unsigned)((n_out + 15) / 16)), dim3(256), 0, st,
                  (const float*)part_o, (const float*)part_ml, kv_len, B, M, c.n_q_heads,
                  c.n_kv_heads, n_cta, ms, min_units, cache_rows, (__nv_bfloat16*)out);
  else if (D == 128)
    jk_launch_pdl(k_attn_combine_sk<128>, dim3((unsigned)((n_out + 7) / 8)), dim3(256), 0, st,
                  (const float*)part_o, (const float*)part_ml, kv_len, B, M, c.n_q_heads,
                  c.n_kv_heads, n_cta, ms, min_units, cache_rows, (__nv_bfloat16*)out);
  else
    jk_launch_pdl(k_attn_combine_sk<64>, dim3((unsigned)((n_out + 7) / 8)), dim3(256), 0, st,
                  (const float*)part_o, (const float*)part_ml, kv_len, B, M, c.n_q_heads,
                  c.n_kv_heads, n_cta, ms, min_units, cache_rows, (__nv_bfloat16*)out);
  JK_LAUNCH_CHECK(ctx);
  return JK_OK;
}
