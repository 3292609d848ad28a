// Context, workspace layout and status handling of the Jakiro CUDA library.
#include <stdio.h>
#include <stdlib.h>

#include "jk_common.cuh"

size_t jk_tc_partial_bytes(const jk_config& c);   // jk_gemm_tc.cu
void jk_tc_destroy(jk_ctx* ctx);                  // jk_gemm_tc.cu
static void prof_free(jk_ctx* ctx);
void jk_attn_tc_destroy(jk_ctx* ctx);             // jk_attn_tc.cu
void jk_attn_cl_destroy(jk_ctx* ctx);             // jk_attn_cl.cu

static int validate_config(const jk_config& c) {
  if (c.dtype != JK_F32 && c.dtype != JK_BF16) return JK_ERR_DTYPE;
  if (c.hidden <= 0 || c.inter <= 0 || c.vocab <= 0) return JK_ERR_SHAPE;
  if (c.hidden % 8 || c.inter % 8) return JK_ERR_SHAPE;
  if (c.n_experts < 1 || c.n_experts > JK_MAX_EXPERTS) return JK_ERR_SHAPE;
  if (c.top_k < 1 || c.top_k > c.n_experts) return JK_ERR_SHAPE;
  if (c.k_per_expert < 1 || c.k_per_expert > JK_MAX_KE || c.k_per_expert > c.vocab)
    return JK_ERR_SHAPE;
  if (c.max_tree < 1 || c.max_tree > JK_MAX_TREE) return JK_ERR_SHAPE;
  if (c.max_batch < 1 || c.max_frontier < 1 || c.max_batch * c.max_frontier > JK_MAX_ROWS)
    return JK_ERR_SHAPE;
  if (c.max_depth < 1 || c.max_depth > 16) return JK_ERR_SHAPE;
  if (c.head_dim != 64 && c.head_dim != 128) return JK_ERR_SHAPE;
  if (c.n_kv_heads < 1 || c.n_q_heads < c.n_kv_heads || c.n_q_heads % c.n_kv_heads)
    return JK_ERR_SHAPE;
  if (!(c.rms_eps >= 0.f)) return JK_ERR_SHAPE;
  if (c.head_mode != 0 && c.head_mode != 1) return JK_ERR_SHAPE;
  if (c.head_mode == 1 && c.top_k != 2) return JK_ERR_SHAPE;      // Eq. 6-7 contrast two experts
  // the top-k merge keeps chunks * k_e candidates in 16 registers per lane
  if ((size_t)((c.vocab + JK_TOPK_CHUNK - 1) / JK_TOPK_CHUNK) * c.k_per_expert > 512) return JK_ERR_SHAPE;
  return JK_OK;
}

static void build_layout(const jk_config& c, jk_ws_layout* L) {
  const size_t es = jk_elem_size(c.dtype);
  const size_t R = (size_t)c.max_batch * c.max_frontier;
  const size_t Rp = jk_align_up(R, 16);
  const size_t RK = R * c.top_k;
  const size_t RKp = jk_align_up(RK, 16);
  const size_t BM = (size_t)c.max_batch * c.max_tree;
  L->rows_pad = (int)Rp;
  L->rk_pad = (int)RKp;
  size_t off = 0;
  auto take = [&](size_t bytes) { size_t o = off; off = jk_align_up(off + bytes, 256); return o; };
  L->status = take(16);
  L->xn = take(Rp * c.hidden * es);
  L->probs = take(R * c.n_experts * 4);
  L->expert = take(R * c.top_k * 4);
  L->gate = take(R * c.top_k * 4);
  L->hbuf = take((size_t)c.n_experts * Rp * c.inter * es);
  L->ybuf = take((size_t)c.n_experts * Rp * c.hidden * 4);
  L->bbuf = take(RKp * c.hidden * es);
  L->logits = take(RK * (size_t)c.vocab * 4);
  L->topk_chunks = (c.vocab + JK_TOPK_CHUNK - 1) / JK_TOPK_CHUNK;
  L->tk_val = take(RK * L->topk_chunks * c.k_per_expert * 4);
  L->tk_idx = take(RK * L->topk_chunks * c.k_per_expert * 4);
  L->tk_ms = take(RK * L->topk_chunks * 2 * 4);
  L->gemm_part_bytes = c.dtype == JK_BF16 ? jk_tc_partial_bytes(c) : 0;
  L->gemm_part = take(L->gemm_part_bytes);
  L->gemm_cnt = take(16);
  // split-KV partials, capped at 256 MiB
  const size_t pre_nodes = (size_t)c.max_batch * c.max_depth * c.max_frontier;
  size_t rows = (BM > pre_nodes ? BM : pre_nodes) * c.n_q_heads;
  // the persistent kernel keeps its partials per 128-row query block, dead rows included
  const size_t grp = (size_t)(c.n_q_heads / c.n_kv_heads) * c.max_tree;
  const size_t rows_blk = (size_t)c.max_batch * c.n_kv_heads * ((grp + 127) / 128) * 128;
  if (rows_blk > rows) rows = rows_blk;
  const size_t per_split = rows * (c.head_dim + 4) * 4;
  int ms = JK_ATTN_MAX_SPLIT;
  while (ms > 1 && per_split * ms > ((size_t)256 << 20)) --ms;
  L->attn_max_split = ms;
  L->attn_o = take(rows * c.head_dim * 4 * ms);
  L->attn_ml = take(rows * 4 * 4 * ms);
  L->rs_arg = take(BM * 4);
  L->rs_max = take(BM * 4);
  L->rs_sum = take(BM * 4);
  L->pbuf = take((size_t)c.max_batch * 2 * c.vocab * 4);              // two copies each: a
  L->qbuf = take((size_t)c.max_batch * c.top_k * 2 * c.vocab * 4);    // rejection writes the other
  L->p_old = take((size_t)c.max_batch * 4);
  const size_t qrows = (size_t)c.max_batch * c.max_depth * c.max_frontier * c.top_k;
  L->qs_arg = take(qrows * 4);
  L->qs_max = take(qrows * 4);
  L->qs_sum = take(qrows * 4);
  const size_t S = (size_t)c.max_depth * c.max_frontier;
  const size_t qd = (size_t)c.n_q_heads * c.head_dim;
  const size_t qkvd = (size_t)(c.n_q_heads + 2 * c.n_kv_heads) * c.head_dim;
  L->pre_x = take(Rp * 2 * c.hidden * es);
  L->pre_h = take(Rp * c.hidden * es);
  const size_t vrows = jk_align_up(BM, 16);                 // jk_verify_qkv: all tree tokens
  L->pre_qkv = take((Rp > vrows ? Rp : vrows) * qkvd * 4);
  L->pre_qd = take((size_t)c.max_batch * S * qd * es);
  L->pre_par = take((size_t)c.max_batch * S * 4);
  L->pre_att = take((size_t)c.max_batch * S * qd * es);
  L->pre_ao = take(Rp * qd * es);
  L->total = off;
}

extern "C" int jk_create(jk_ctx** out, const jk_config* cfg) {
  if (!out || !cfg) return JK_ERR_NULL;
  int rc = validate_config(*cfg);
  if (rc != JK_OK) return rc;
  jk_ctx* ctx = (jk_ctx*)calloc(1, sizeof(jk_ctx));
  if (!ctx) return JK_ERR_CUDA;
  ctx->cfg = *cfg;
  build_layout(ctx->cfg, &ctx->lay);
  ctx->tensor_path = cfg->dtype == JK_BF16 ? 1 : 0;
  ctx->st_attn = JK_ST_ATTN;
  ctx->st_combine = JK_ST_ATTN_COMBINE;
  *out = ctx;
  return JK_OK;
}

extern "C" int jk_destroy(jk_ctx* ctx) {
  if (!ctx) return JK_ERR_NULL;
  jk_tc_destroy(ctx);
  jk_attn_tc_destroy(ctx);
  jk_attn_cl_destroy(ctx);
  if (ctx->prof.cap) prof_free(ctx);
  free(ctx);
  return JK_OK;
}

extern "C" size_t jk_workspace_bytes(const jk_ctx* ctx) { return ctx ? ctx->lay.total : 0; }

extern "C" int jk_set_workspace(jk_ctx* ctx, void* stream, void* dev_ptr, size_t bytes) {
  if (!ctx || !dev_ptr) return JK_ERR_NULL;
  if (reinterpret_cast<uintptr_t>(dev_ptr) & 255) return JK_ERR_ALIGN;
  if (bytes < ctx->lay.total) return JK_ERR_WORKSPACE;
  ctx->ws = (char*)dev_ptr;
  ctx->ws_bytes = bytes;
  jk_tc_destroy(ctx);   // tensor maps over an earlier workspace are stale
  JK_CUDA_CHECK(ctx, cudaMemsetAsync(ctx->ws + ctx->lay.status, 0, 16, (cudaStream_t)stream));
  JK_CUDA_CHECK(ctx, cudaMemsetAsync(ctx->ws + ctx->lay.gemm_cnt, 0, 16, (cudaStream_t)stream));
  return JK_OK;
}

extern "C" int jk_set_tensor_path(jk_ctx* ctx, int32_t enable) {
  if (!ctx) return JK_ERR_NULL;
  ctx->tensor_path = (enable && ctx->cfg.dtype == JK_BF16) ? 1 : 0;
  return JK_OK;
}

extern "C" int jk_set_attn_kernel(jk_ctx* ctx, int32_t mode) {
  if (!ctx) return JK_ERR_NULL;
  if (mode < 0 || mode > 3) return JK_ERR_SHAPE;
  ctx->attn_kernel = mode;
  return JK_OK;
}

extern "C" const char* jk_strerror(int code) {
  switch (code) {
    case JK_OK: return "ok";
    case JK_ERR_NULL: return "required pointer is NULL";
    case JK_ERR_SHAPE: return "size outside the supported range";
    case JK_ERR_ALIGN: return "pointer or stride not 16-byte aligned";
    case JK_ERR_DTYPE: return "unknown dtype";
    case JK_ERR_CAPACITY: return "more rows than the context was created for";
    case JK_ERR_WORKSPACE: return "workspace missing or too small";
    case JK_ERR_CUDA: return "CUDA runtime error";
    case JK_ERR_TIMEOUT: return "bounded device-side wait ran out";
    case JK_ERR_BOUNDS: return "input index out of range (device status)";
    default: return "unknown status";
  }
}

extern "C" const char* jk_last_cuda_error(const jk_ctx* ctx) { return ctx ? ctx->cuda_err : ""; }

extern "C" int jk_read_status(jk_ctx* ctx, void* stream, int32_t* host_status) {
  if (!ctx || !host_status) return JK_ERR_NULL;
  if (!ctx->ws) return JK_ERR_WORKSPACE;
  cudaStream_t st = (cudaStream_t)stream;
  JK_CUDA_CHECK(ctx, cudaMemcpyAsync(host_status, ctx->ws + ctx->lay.status, 4,
                                     cudaMemcpyDeviceToHost, st));
  JK_CUDA_CHECK(ctx, cudaMemsetAsync(ctx->ws + ctx->lay.status, 0, 16, st));
  JK_CUDA_CHECK(ctx, cudaStreamSynchronize(st));
  return JK_OK;
}

// ---------------------------------------------------------------- per-kernel timing
// While the stream is being captured into a graph an ordinary event record only adds a
// dependency; the "external" flavour becomes an event-record node that every replay executes,
// which is what a timing pair needs.
static cudaError_t prof_record(cudaEvent_t ev, cudaStream_t st) {
  cudaStreamCaptureStatus cs = cudaStreamCaptureStatusNone;
  if (cudaStreamIsCapturing(st, &cs) != cudaSuccess) cs = cudaStreamCaptureStatusNone;
  return cudaEventRecordWithFlags(ev, st, cs == cudaStreamCaptureStatusActive
                                              ? cudaEventRecordExternal : cudaEventRecordDefault);
}

void jk_prof_begin(jk_ctx* ctx, cudaStream_t st, int stage) {
  jk_prof& p = ctx->prof;
  if (p.n >= p.cap) return;
  p.stage[p.n] = stage;
  p.stream = st;
  if (prof_record(p.ev[2 * p.n], st) == cudaSuccess) p.open = 1;
}

void jk_prof_end(jk_ctx* ctx) {
  jk_prof& p = ctx->prof;
  p.open = 0;
  if (prof_record(p.ev[2 * p.n + 1], p.stream) == cudaSuccess) ++p.n;
}

static void prof_free(jk_ctx* ctx) {
  jk_prof& p = ctx->prof;
  for (int i = 0; i < 2 * p.cap; ++i) cudaEventDestroy(p.ev[i]);
  free(p.ev);
  free(p.stage);
  memset(&p, 0, sizeof(p));
}

extern "C" int jk_profile_enable(jk_ctx* ctx, int32_t max_launches) {
  if (!ctx) return JK_ERR_NULL;
  if (max_launches < 0 || max_launches > (1 << 20)) return JK_ERR_SHAPE;
  if (ctx->prof.cap) prof_free(ctx);
  if (max_launches == 0) return JK_OK;
  jk_prof& p = ctx->prof;
  p.ev = (cudaEvent_t*)calloc(2 * (size_t)max_launches, sizeof(cudaEvent_t));
  p.stage = (int*)calloc(max_launches, sizeof(int));
  if (!p.ev || !p.stage) return JK_ERR_CUDA;
  for (int i = 0; i < 2 * max_launches; ++i) JK_CUDA_CHECK(ctx, cudaEventCreate(&p.ev[i]));
  p.cap = max_launches;
  return JK_OK;
}

static int prof_sum(jk_ctx* ctx, void* stream, float* host_ms, int32_t* host_count, bool reset) {
  if (!ctx || !host_ms || !host_count) return JK_ERR_NULL;
  for (int s = 0; s < JK_N_STAGES; ++s) { host_ms[s] = 0.f; host_count[s] = 0; }
  jk_prof& p = ctx->prof;
  if (!p.cap) return JK_OK;
  JK_CUDA_CHECK(ctx, cudaStreamSynchronize((cudaStream_t)stream));
  for (int i = 0; i < p.n; ++i) {
    float ms = 0.f;
    JK_CUDA_CHECK(ctx, cudaEventElapsedTime(&ms, p.ev[2 * i], p.ev[2 * i + 1]));
    host_ms[p.stage[i]] += ms;
    host_count[p.stage[i]] += 1;
  }
  if (reset) p.n = 0;
  return JK_OK;
}

extern "C" int jk_profile_collect(jk_ctx* ctx, void* stream, float* host_ms, int32_t* host_count) {
  return prof_sum(ctx, stream, host_ms, host_count, true);
}

extern "C" int jk_profile_read(jk_ctx* ctx, void* stream, float* host_ms, int32_t* host_count) {
  return prof_sum(ctx, stream, host_ms, host_count, false);
}

extern "C" int32_t jk_profile_stage_count(void) { return JK_N_STAGES; }

extern "C" const char* jk_profile_stage_name(int32_t stage) {
  static const char* names[JK_N_STAGES] = {
      "router", "expert_gate_up", "expert_down", "branch_features", "lm_head", "topk_partial",
      "expand_finish", "tree_finalize", "tree_attn", "attn_combine", "row_stats", "accept_walk",
      "kv_compact", "gemm_fixup", "pre_gather", "pre_gemm", "pre_fixup", "pre_rope", "pre_attn",
      "pre_attn_combine"};
  return (stage >= 0 && stage < JK_N_STAGES) ? names[stage] : "?";
}

int jk_ensure_device_info(jk_ctx* ctx) {
  if (ctx->sm_count > 0) return JK_OK;
  int dev = 0;
  JK_CUDA_CHECK(ctx, cudaGetDevice(&dev));
  int sms = 0;
  JK_CUDA_CHECK(ctx, cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
  ctx->sm_count = sms > 0 ? sms : 148;
  return JK_OK;
}
