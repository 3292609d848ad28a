// Tensor-core path of the draft layer's dense contractions (expert gate/up, expert down, LM head;
// arXiv 2502.06282 Eq. 3-4) for bf16 on sm_100a.
//
// All three are "skinny" products  out[n, m] = sum_k W[m, k] * X[n, k]  with millions of weight
// rows m but only 2..256 activation rows n, so they are bound by streaming W from HBM once.  One
// persistent kernel serves them:
//   - the weight matrix sits on the 128-row M side of tcgen05.mma, the activation rows on N
//     (padded to a multiple of 16), accumulators in tensor memory;
//   - work is cut into units of one 128 x 64 weight tile; the units of all (group, tile) pairs are
//     laid end to end and every CTA takes an equal contiguous span (stream-K), so all SMs stream
//     the same number of bytes whatever the tile count is;
//   - a producer thread feeds a ring of shared-memory stages with TMA (128B swizzle), one thread
//     issues the MMAs, four warps drain finished accumulators to fp32 partial tiles in global
//     memory; a small second kernel adds the partials of each tile in a fixed order (no atomics,
//     bitwise reproducible) and applies the epilogue (SiLU * up, or a plain store).
// Every wait on an mbarrier is bounded: after ~2 s it records JK_ERR_TIMEOUT in the status word,
// and the CTA drains its copies, frees its tensor memory and returns.
#include <cuda.h>
#include <stdlib.h>

#include "jk_common.cuh"
#include "jk_tcgen05.cuh"

#define TC_TILE_M 128
#define TC_TILE_K 64
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
  int kt;                            // ceil(K / 64)
  int n_pad;                         // activation rows, multiple of 16
  int stages;
  int max_seg;                       // partial slots per CTA
  int R, K_top, n_experts;           // to derive the active experts from `expert`
  int tmem_cols;
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
// Work partition shared by the GEMM kernel and the fix-up kernel
// ---------------------------------------------------------------------------------------------
struct tc_plan {
  int n_groups;                      // active groups
  int group_src[TC_MAX_GROUPS];      // index into the parameter arrays
  long long total_units;
};

__device__ __forceinline__ void tc_make_plan(const tc_params& p, const int32_t* expert,
                                             tc_plan* plan) {
  // one thread
  unsigned active = 0;
  for (int i = 0; i < p.R * p.K_top; ++i) {
    const int e = expert[i];
    if (e >= 0 && e < p.n_experts) active |= 1u << e;
  }
  int n = 0;
  for (int g = 0; g < p.n_groups_max; ++g) {
    const int e = p.group_expert[g];
    if (e < 0 || (active >> e) & 1u) plan->group_src[n++] = g;
  }
  plan->n_groups = n;
  plan->total_units = (long long)n * p.tiles_per_group * p.kt;
}
__device__ __forceinline__ long long tc_span_start(long long total, int cta, int n_cta) {
  return total * cta / n_cta;
}

struct __align__(1024) tc_smem_tail {
  uint64_t full[TC_MAX_STAGES];
  uint64_t empty[TC_MAX_STAGES];
  uint64_t acc_full[2];
  uint64_t acc_empty[2];
  uint32_t tmem_base;
  int abort_flag;
  tc_plan plan;
};

__global__ void __launch_bounds__(TC_THREADS, 1) k_tc_gemm(
    const __grid_constant__ CUtensorMap map_a0, const __grid_constant__ CUtensorMap map_a1,
    const __grid_constant__ CUtensorMap map_b, const tc_params p, const int32_t* __restrict__ expert,
    float* __restrict__ partial, int32_t* __restrict__ status) {
  extern __shared__ unsigned char smem_raw[];
  unsigned char* smem = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
  const int stage_bytes = TC_TILE_M * TC_TILE_K * 2 + p.n_pad * TC_TILE_K * 2;
  tc_smem_tail& T = *reinterpret_cast<tc_smem_tail*>(smem + (size_t)p.stages * stage_bytes);
  const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
  volatile int* abort_flag = &T.abort_flag;

  if (threadIdx.x == 0) {
    for (int s = 0; s < p.stages; ++s) { mbar_init(&T.full[s], 1); mbar_init(&T.empty[s], 1); }
    for (int a = 0; a < 2; ++a) { mbar_init(&T.acc_full[a], 1); mbar_init(&T.acc_empty[a], 4); }
    T.abort_flag = 0;
    tc_make_plan(p, expert, &T.plan);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
  }
  if (warp == 1) {
    tmem_alloc(&T.tmem_base, (uint32_t)p.tmem_cols);
    tmem_relinquish();
  }
  tc_fence_before();
  __syncthreads();
  tc_fence_after();
  const uint32_t tmem_base = T.tmem_base;
  const long long total = T.plan.total_units;
  const long long u0 = tc_span_start(total, blockIdx.x, gridDim.x);
  const long long u1 = tc_span_start(total, blockIdx.x + 1, gridDim.x);
  const int units_per_tile = p.kt;
  const long long first_tile = u0 / units_per_tile;

  if (warp == 0 && lane == 0) {
    // ------------------------------------------------------------------ TMA producer
    int issued = 0;
    bool ok = true;
    for (long long u = u0; u < u1 && ok; ++u, ++issued) {
      const int s = issued % p.stages;
      const uint32_t ph = (uint32_t)(issued / p.stages) & 1u;
      if (issued >= p.stages) ok = mbar_wait(&T.empty[s], ph ^ 1u, abort_flag, status);
      if (!ok) break;
      const long long tile = u / units_per_tile;
      const int kt = (int)(u - tile * units_per_tile);
      const int g = T.plan.group_src[(int)(tile / p.tiles_per_group)];
      const int t = (int)(tile % p.tiles_per_group);
      unsigned char* sa = smem + (size_t)s * stage_bytes;
      unsigned char* sb = sa + TC_TILE_M * TC_TILE_K * 2;
      mbar_expect_tx(&T.full[s], (uint32_t)stage_bytes);
      tma_load_2d(sa, p.group_amap[g] ? &map_a1 : &map_a0, kt * TC_TILE_K,
                  p.group_arow0[g] + t * TC_TILE_M, &T.full[s]);
      tma_load_2d(sb, &map_b, kt * TC_TILE_K, p.group_brow0[g], &T.full[s]);
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
    int consumed = 0, seg = 0;
    bool ok = true;
    for (long long u = u0; u < u1 && ok; ++seg) {
      const long long tile = u / units_per_tile;
      const long long tile_end = (tile + 1) * units_per_tile;
      const long long ue = tile_end < u1 ? tile_end : u1;
      const int acc = seg & 1;
      if (seg >= 2) ok = mbar_wait(&T.acc_empty[acc], ((uint32_t)(seg >> 1) & 1u) ^ 1u, abort_flag, status);
      if (!ok) break;
      tc_fence_after();
      const uint32_t d_addr = tmem_base + (uint32_t)(acc * p.n_pad);
      bool first = true;
      for (; u < ue; ++u, ++consumed) {
        const int s = consumed % p.stages;
        ok = mbar_wait(&T.full[s], (uint32_t)(consumed / p.stages) & 1u, abort_flag, status);
        if (!ok) break;
        tc_fence_after();
        const uint32_t a_addr = smem_u32(smem + (size_t)s * stage_bytes);
        const uint32_t b_addr = a_addr + TC_TILE_M * TC_TILE_K * 2;
        const uint64_t da = smem_desc_sw128(a_addr), db = smem_desc_sw128(b_addr);
#pragma unroll
        for (int k = 0; k < TC_TILE_K / 16; ++k) {
          // 16 bf16 = 32 bytes further along K inside the swizzled row: +2 in the address field
          tc_mma_bf16(d_addr, da + (uint64_t)(2 * k), db + (uint64_t)(2 * k), idesc,
                      (first && k == 0) ? 0u : 1u);
        }
        first = false;
        tc_commit(&T.empty[s]);          // the stage is free once these MMAs have read it
      }
      if (ok) tc_commit(&T.acc_full[acc]);
    }
  } else if (warp >= 2) {
    // ------------------------------------------------------------------ epilogue
    const int quarter = warp & 3;        // the TMEM lanes this warp may read: 32*quarter .. +31
    const int m = quarter * 32 + lane;
    int seg = 0;
    bool ok = true;
    for (long long u = u0; u < u1 && ok; ++seg) {
      const long long tile = u / units_per_tile;
      const long long tile_end = (tile + 1) * units_per_tile;
      u = tile_end < u1 ? tile_end : u1;
      const int acc = seg & 1;
      ok = mbar_wait(&T.acc_full[acc], (uint32_t)(seg >> 1) & 1u, abort_flag, status);
      ok = __all_sync(0xffffffffu, ok);          // the TMEM loads below need the whole warp
      if (!ok) break;
      tc_fence_after();
      const int slot = blockIdx.x * p.max_seg + (int)(tile - first_tile);
      float* dst = partial + ((size_t)slot * p.n_pad) * TC_TILE_M + m;
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
// Fix-up: out[n, m] = sum over the CTAs that touched the tile, in ascending CTA order.
//   mode 0: out[(group_out0[g] + n) * ld + m]          (plain store, fp32)
//   mode 1: groups come in (gate, up) pairs: h = SiLU(gate) * up as bf16
// ---------------------------------------------------------------------------------------------
struct tc_fix_params {
  int mode;
  int m_rows;                        // valid rows of a group (I, H or V)
  int n_rows;                        // valid activation rows
  long long ld;                      // output leading dimension (elements)
  long long group_out0[TC_MAX_GROUPS];   // element offset of the group's output block (by source group)
  int n_cta;                         // grid of the GEMM kernel
  int rows_per_b;                    // mode 0 with a batch stride: n -> (n / rows_per_b, n % rows_per_b)
  long long stride_b;
};

__device__ __forceinline__ float tc_tile_sum(const float* __restrict__ partial, const tc_params& p,
                                             long long total, int n_cta, long long tile, int n,
                                             int m) {
  const long long a = tile * p.kt, b = a + p.kt;
  int c = (int)(a * n_cta / total);
  while (c + 1 < n_cta && tc_span_start(total, c + 1, n_cta) <= a) ++c;
  while (c > 0 && tc_span_start(total, c, n_cta) > a) --c;
  float acc = 0.f;
  for (; c < n_cta; ++c) {
    const long long s0 = tc_span_start(total, c, n_cta);
    if (s0 >= b) break;
    const long long s1 = tc_span_start(total, c + 1, n_cta);
    if (s1 <= a || s1 == s0) continue;                        // before the tile, or empty
    const long long first_tile = s0 / p.kt;
    const int slot = c * p.max_seg + (int)(tile - first_tile);
    acc += partial[((size_t)slot * p.n_pad + n) * TC_TILE_M + m];
  }
  return acc;
}

__global__ void __launch_bounds__(128) k_tc_fixup(const tc_params p, const tc_fix_params f,
                                                  const int32_t* __restrict__ expert,
                                                  const float* __restrict__ partial,
                                                  void* __restrict__ out) {
  __shared__ tc_plan plan;
  if (threadIdx.x == 0) tc_make_plan(p, expert, &plan);
  __syncthreads();
  const int t = blockIdx.x;                       // tile within the group
  const int go = blockIdx.y;                      // output group (a pair of groups in mode 1)
  const int m = threadIdx.x;
  const int mg = t * TC_TILE_M + m;
  const long long total = plan.total_units;
  if (f.mode == 1) {
    if (2 * go + 1 >= plan.n_groups || mg >= f.m_rows) return;
    const int src = plan.group_src[2 * go];
    const long long tile_g = (long long)(2 * go) * p.tiles_per_group + t;
    const long long tile_u = (long long)(2 * go + 1) * p.tiles_per_group + t;
    __nv_bfloat16* o = reinterpret_cast<__nv_bfloat16*>(out) + f.group_out0[src];
    for (int n = blockIdx.z; n < f.n_rows; n += gridDim.z) {
      const float g = tc_tile_sum(partial, p, total, f.n_cta, tile_g, n, m);
      const float u = tc_tile_sum(partial, p, total, f.n_cta, tile_u, n, m);
      o[(size_t)n * f.ld + mg] = __float2bfloat16_rn(g / (1.f + expf(-g)) * u);
    }
  } else {
    if (go >= plan.n_groups || mg >= f.m_rows) return;
    const int src = plan.group_src[go];
    const long long tile = (long long)go * p.tiles_per_group + t;
    float* o = reinterpret_cast<float*>(out) + f.group_out0[src];
    for (int n = blockIdx.z; n < f.n_rows; n += gridDim.z) {
      const float v = tc_tile_sum(partial, p, total, f.n_cta, tile, n, m);
      size_t off;
      if (f.rows_per_b > 0)
        off = (size_t)(n / f.rows_per_b) * (size_t)f.stride_b + (size_t)(n % f.rows_per_b) * f.ld;
      else
        off = (size_t)n * f.ld;
      o[off + mg] = v;
    }
  }
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

static int tc_grid(const jk_ctx* ctx) {
  const int n = ctx->sm_count > 0 ? ctx->sm_count : 148;
  return n > 192 ? 192 : n;
}

static int tc_stage_bytes(int n_pad) { return TC_TILE_M * TC_TILE_K * 2 + n_pad * TC_TILE_K * 2; }

static int tc_stages(int n_pad) {
  int s = (TC_SMEM_BUDGET - (int)sizeof(tc_smem_tail) - 1024) / tc_stage_bytes(n_pad);
  if (s > TC_MAX_STAGES) s = TC_MAX_STAGES;
  return s;
}

static int tc_max_seg(long long max_units, int n_cta, int kt) {
  const long long span = (max_units + n_cta - 1) / n_cta;
  return (int)((span + kt - 1) / kt) + 1;
}

// n_cta * max_seg <= tiles + 3 * n_cta for any grid size; grids are capped at TC_MAX_GRID.
#define TC_MAX_GRID 192
static size_t tc_partial_for(long long units, int, int kt, int n_pad) {
  return (size_t)(units / kt + 3 * TC_MAX_GRID) * n_pad * TC_TILE_M * sizeof(float);
}

// Worst case over the three contractions.
size_t jk_tc_partial_bytes(const jk_config& c) {
  const int n_cta = TC_MAX_GRID;
  const int R = c.max_batch * c.max_frontier;
  const int np1 = (int)jk_align_up(R, 16), np2 = (int)jk_align_up((size_t)R * c.top_k, 16);
  const int kt_h = (c.hidden + TC_TILE_K - 1) / TC_TILE_K, kt_i = (c.inter + TC_TILE_K - 1) / TC_TILE_K;
  const long long t_i = (c.inter + TC_TILE_M - 1) / TC_TILE_M, t_h = (c.hidden + TC_TILE_M - 1) / TC_TILE_M,
                  t_v = (c.vocab + TC_TILE_M - 1) / TC_TILE_M;
  size_t a = tc_partial_for(2ll * c.n_experts * t_i * kt_h, n_cta, kt_h, np1);
  size_t b = tc_partial_for((long long)c.n_experts * t_h * kt_i, n_cta, kt_i, np1);
  size_t d = tc_partial_for(t_v * kt_h, n_cta, kt_h, np2);
  size_t m = a > b ? a : b;
  return m > d ? m : d;
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
  if (tc_stages(np2) < 2) return 0;
  tc_state* s = tc_get_state(const_cast<jk_ctx*>(ctx));
  return s && !s->failed;
}

extern "C" int jk_tensor_path_active(jk_ctx* ctx) {
  return (ctx && ctx->tensor_path && jk_tc_available(ctx)) ? 1 : 0;
}

// 2-D bf16 tensor map: `rows` x `cols` (cols contiguous), box = box_rows x 64, 128-byte swizzle.
static const CUtensorMap* tc_map(jk_ctx* ctx, tc_state* s, const void* ptr, uint64_t rows,
                                 uint64_t cols, uint32_t box_rows) {
  for (int i = 0; i < s->n_maps; ++i) {
    tc_map_entry& e = s->maps[i];
    if (e.ptr == ptr && e.rows == rows && e.cols == cols && e.box_rows == box_rows) return &e.map;
  }
  if (s->n_maps == 32) s->n_maps = 0;            // recycle (pointers changed often)
  tc_map_entry& e = s->maps[s->n_maps];
  const cuuint64_t gdim[2] = {cols, rows};
  const cuuint64_t gstride[1] = {cols * 2};
  const cuuint32_t box[2] = {TC_TILE_K, box_rows};
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

static int tc_launch(jk_ctx* ctx, cudaStream_t st, tc_state* s, const CUtensorMap* a0,
                     const CUtensorMap* a1, const CUtensorMap* b, tc_params& p,
                     const tc_fix_params& f, const int32_t* expert, void* out, int out_groups,
                     int stage_id) {
  const jk_ws_layout& L = ctx->lay;
  const int n_cta = tc_grid(ctx);
  p.stages = tc_stages(p.n_pad);
  const long long max_units = (long long)p.n_groups_max * p.tiles_per_group * p.kt;
  p.max_seg = tc_max_seg(max_units, n_cta, p.kt);
  int cols = 32;
  while (cols < 2 * p.n_pad) cols <<= 1;
  p.tmem_cols = cols;
  if ((size_t)n_cta * p.max_seg * p.n_pad * TC_TILE_M * sizeof(float) > L.gemm_part_bytes)
    return JK_ERR_WORKSPACE;
  const size_t smem = (size_t)p.stages * tc_stage_bytes(p.n_pad) + sizeof(tc_smem_tail) + 1024;
  if (!s->smem_set) {
    JK_CUDA_CHECK(ctx, cudaFuncSetAttribute(k_tc_gemm, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                            TC_SMEM_BUDGET));
    s->smem_set = 1;
  }
  float* partial = (float*)(ctx->ws + L.gemm_part);
  int32_t* status = (int32_t*)(ctx->ws + L.status);
  JK_PROF(ctx, st, stage_id);
  k_tc_gemm<<<n_cta, TC_THREADS, smem, st>>>(*a0, *a1, *b, p, expert, partial, status);
  JK_LAUNCH_CHECK(ctx);
  tc_fix_params ff = f;
  ff.n_cta = n_cta;
  int zdim = 1;
  const int base = p.tiles_per_group * out_groups;
  while (zdim < ff.n_rows && base * zdim < 2 * n_cta) zdim <<= 1;
  JK_PROF(ctx, st, JK_ST_GEMM_FIXUP);
  k_tc_fixup<<<dim3(p.tiles_per_group, out_groups, zdim), 128, 0, st>>>(p, ff, expert, partial, out);
  JK_LAUNCH_CHECK(ctx);
  return JK_OK;
}

// do_lm_head = 0: h = SiLU(W_gate x) * (W_up x) and y = W_down h for every touched expert
//                 (hbuf, ybuf of the workspace);  do_lm_head = 1: logits = b W_head^T.
int jk_tc_expert_ffn(jk_ctx* ctx, cudaStream_t st, const jk_draft_weights* w, int R,
                     const int32_t* expert, int do_lm_head, float* logits, int RK, int rows_per_b,
                     long long logits_stride_b) {
  tc_state* s = tc_get_state(ctx);
  if (!s || s->failed) return JK_ERR_CUDA;
  const jk_config& c = ctx->cfg;
  const jk_ws_layout& L = ctx->lay;
  const int H = c.hidden, I = c.inter, V = c.vocab, N = c.n_experts, Rp = L.rows_pad;
  tc_params p;
  memset(&p, 0, sizeof(p));
  p.R = R; p.K_top = c.top_k; p.n_experts = N;
  tc_fix_params f;
  memset(&f, 0, sizeof(f));
  if (!do_lm_head) {
    const int n_pad = (int)jk_align_up(R, 16);
    // gate / up
    const CUtensorMap* ag = tc_map(ctx, s, w->w_gate, (uint64_t)N * I, H, TC_TILE_M);
    const CUtensorMap* au = tc_map(ctx, s, w->w_up, (uint64_t)N * I, H, TC_TILE_M);
    const CUtensorMap* bx = tc_map(ctx, s, ctx->ws + L.xn, Rp, H, n_pad);
    if (!ag || !au || !bx) return JK_ERR_CUDA;
    p.n_groups_max = 2 * N;
    for (int e = 0; e < N; ++e)
      for (int h = 0; h < 2; ++h) {
        const int g = 2 * e + h;
        p.group_expert[g] = e; p.group_amap[g] = h; p.group_arow0[g] = e * I; p.group_brow0[g] = 0;
        f.group_out0[g] = (long long)e * Rp * I;
      }
    p.tiles_per_group = (I + TC_TILE_M - 1) / TC_TILE_M;
    p.kt = (H + TC_TILE_K - 1) / TC_TILE_K;
    p.n_pad = n_pad;
    f.mode = 1; f.m_rows = I; f.n_rows = R; f.ld = I;
    int rc = tc_launch(ctx, st, s, ag, au, bx, p, f, expert, ctx->ws + L.hbuf, N, JK_ST_GATEUP);
    if (rc != JK_OK) return rc;
    // down
    const CUtensorMap* ad = tc_map(ctx, s, w->w_down, (uint64_t)N * H, I, TC_TILE_M);
    const CUtensorMap* bh = tc_map(ctx, s, ctx->ws + L.hbuf, (uint64_t)N * Rp, I, n_pad);
    if (!ad || !bh) return JK_ERR_CUDA;
    p.n_groups_max = N;
    for (int e = 0; e < N; ++e) {
      p.group_expert[e] = e; p.group_amap[e] = 0; p.group_arow0[e] = e * H; p.group_brow0[e] = e * Rp;
      f.group_out0[e] = (long long)e * Rp * H;
    }
    p.tiles_per_group = (H + TC_TILE_M - 1) / TC_TILE_M;
    p.kt = (I + TC_TILE_K - 1) / TC_TILE_K;
    f.mode = 0; f.m_rows = H; f.n_rows = R; f.ld = H; f.rows_per_b = 0;
    return tc_launch(ctx, st, s, ad, ad, bh, p, f, expert, ctx->ws + L.ybuf, N, JK_ST_DOWN);
  }
  const int n_pad = (int)jk_align_up(RK, 16);
  const CUtensorMap* ah = tc_map(ctx, s, w->lm_head, V, H, TC_TILE_M);
  const CUtensorMap* bb = tc_map(ctx, s, ctx->ws + L.bbuf, L.rk_pad, H, n_pad);
  if (!ah || !bb) return JK_ERR_CUDA;
  p.n_groups_max = 1;
  p.group_expert[0] = -1; p.group_amap[0] = 0; p.group_arow0[0] = 0; p.group_brow0[0] = 0;
  p.tiles_per_group = (V + TC_TILE_M - 1) / TC_TILE_M;
  p.kt = (H + TC_TILE_K - 1) / TC_TILE_K;
  p.n_pad = n_pad;
  f.mode = 0; f.m_rows = V; f.n_rows = RK; f.ld = V; f.group_out0[0] = 0;
  f.rows_per_b = rows_per_b; f.stride_b = logits_stride_b;
  return tc_launch(ctx, st, s, ah, ah, bb, p, f, expert, logits, 1, JK_ST_LMHEAD);
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
