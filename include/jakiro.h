/*
 * jakiro.h - C interface of the Jakiro draft-and-verify step for NVIDIA B200 (sm_100a).
 *
 * One speculative-decoding step of arXiv 2502.06282 has three phases (Sec. 2.1): draft,
 * verify, refine.  This library provides the per-step kernels of each phase:
 *
 *   jk_draft_pre           the draft layer in front of the MoE: reduction layer and attention
 *                          (Sec. 3.1.2, Eq. 1)
 *   jk_draft_expand        one layer of the decoupled MoE draft head (Sec. 3.1.2, Eq. 2-5)
 *   jk_tree_finalize       rerank the drafted candidates into the verification tree and
 *                          build its attention mask (Sec. 3.1.2, Fig. 4)
 *   jk_tree_verify_attn    tree-masked attention of one target layer (Sec. 2.1 step 2)
 *   jk_accept_and_compact  acceptance walk, bonus token and KV-cache compaction
 *                          (Sec. 2.1 steps 2-3)
 *
 * Conventions that hold for every call
 *   - Returns 0 (JK_OK) or a negative jk_status.  Nothing throws or aborts.
 *   - Pointers named "host" are host memory; every other pointer is DEVICE memory on the
 *     current CUDA device, owned by the caller, 16-byte aligned.  The library allocates no
 *     device memory: scratch space is the caller-provided workspace (jk_set_workspace).
 *   - `stream` is a cudaStream_t passed as void*.  Calls enqueue work and return without
 *     synchronising.  Argument errors are reported by the return value before anything is
 *     launched; data-dependent errors found on the device (an index out of range) are
 *     recorded in a status word that jk_read_status returns.
 *   - Tensors are dense, row-major, innermost index last.  "T" below is the context's
 *     dtype (float or bfloat16).  B = batch, F = frontier nodes of this layer, H = hidden,
 *     N = experts, K = active experts per node, I = expert inner size, V = vocabulary,
 *     k_e = children per (node, expert), W = frontier width, M = tree nodes incl. root,
 *     D = tree depth, Hq/Hkv/d = attention heads and head size, L = target layers.
 *   - Same inputs give bitwise the same outputs (no floating-point atomics).
 *   - Calls on one context must not overlap on the device: they share the workspace.
 */
#ifndef JAKIRO_H_
#define JAKIRO_H_

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum {
  JK_OK = 0,
  JK_ERR_NULL = -1,       /* a required pointer is NULL                                  */
  JK_ERR_SHAPE = -2,      /* a size is outside the supported range                       */
  JK_ERR_ALIGN = -3,      /* a pointer or stride is not 16-byte aligned                  */
  JK_ERR_DTYPE = -4,      /* unknown dtype                                               */
  JK_ERR_CAPACITY = -5,   /* more rows than the context was created for                  */
  JK_ERR_WORKSPACE = -6,  /* workspace missing or too small                              */
  JK_ERR_CUDA = -7,       /* a CUDA runtime call failed (see jk_last_cuda_error)         */
  JK_ERR_TIMEOUT = -8,    /* a bounded device-side wait ran out                          */
  JK_ERR_BOUNDS = -9      /* device status: an input index was out of range              */
} jk_status;

typedef enum { JK_F32 = 0, JK_BF16 = 1 } jk_dtype;

/* Limits: top_k <= n_experts <= 8, k_per_expert <= 16, max_tree <= 128, max_depth <= 16,
 * max_batch * max_frontier <= 128, head_dim 64 or 128, hidden/inter multiples of 8,
 * ceil(vocab / 4096) * k_per_expert <= 512; a step's candidate pool holds at most 4096 entries
 * per sequence. */
typedef struct {
  int32_t hidden, n_experts, top_k, inter, vocab;
  int32_t n_q_heads, n_kv_heads, head_dim;
  int32_t max_batch, max_tree, max_depth, max_frontier, k_per_expert;
  int32_t dtype;            /* jk_dtype of weights, hidden states, Q and the KV cache    */
  float rms_eps;            /* epsilon of the pre-MoE RMSNorm                            */
  int32_t use_pre_norm;     /* 1: router and experts see RMSNorm(u) * norm_weight (the
                               normalisation Sec. 3.1.2 leaves out of Eq. 1-5); 0: u     */
  int32_t branch_residual;  /* 1: branch feature = g_r * Expert_r(x) + u; 0: g_r * Expert_r(x) */
  int32_t head_mode;        /* 0: decoupled heads, one logits row per selected expert (Eq. 4);
                               1: contrastive heads (Sec. 3.2, Eq. 6-8; needs top_k = 2): row 0 is
                               Head(f^moe), row 1 is Head(f^const), see jk_draft_expand            */
  float contrast_alpha;     /* alpha and beta of Eq. 7: f^const = beta f^top1 - alpha f^top2       */
  float contrast_beta;
} jk_config;

typedef struct jk_ctx jk_ctx;

/* Host-only bookkeeping; no CUDA call is made.  *out is owned by the caller until jk_destroy. */
int jk_create(jk_ctx** out, const jk_config* host_cfg);
int jk_destroy(jk_ctx* ctx);
/* Bytes of device scratch the context needs (a multiple of 256). */
size_t jk_workspace_bytes(const jk_ctx* ctx);
/* dev_ptr: device memory, 256-byte aligned, at least jk_workspace_bytes(ctx) bytes, owned by
 * the caller and kept alive while the context is used.  Clears the device status word on
 * `stream`. */
int jk_set_workspace(jk_ctx* ctx, void* stream, void* dev_ptr, size_t bytes);
const char* jk_strerror(int code);
/* Text of the last CUDA runtime error seen by this context ("" if none). */
const char* jk_last_cuda_error(const jk_ctx* ctx);
/* Synchronises `stream`, copies the device status word to *host_status (0 or a jk_status)
 * and clears it. */
int jk_read_status(jk_ctx* ctx, void* stream, int32_t* host_status);
/* Which kernels run the dense contractions: 0 = CUDA-core kernels, 1 = tensor-core
 * (tcgen05) kernels where the dtype allows.  Default 1 for bf16, always 0 for f32. */
int jk_set_tensor_path(jk_ctx* ctx, int32_t enable);
/* 1 if the tensor-core kernels will run the contractions of this context (bf16, enabled, rows
 * within their limit, driver entry point for tensor maps found), else 0. */
int jk_tensor_path_active(jk_ctx* ctx);
/* Which tensor-core kernel runs jk_tree_verify_attn for bf16: 0 = chosen per call from the sizes
 * (default), 1 = one CTA per (query block, key slice) with a merge kernel, 2 = the persistent
 * kernel that deals key tiles evenly to one CTA per SM, 3 = the kernel whose key slices form a
 * thread-block cluster and merge through distributed shared memory (2 and 3 fall back to 1 where
 * their limits do not hold).  All compute the operation of arXiv 2502.06282 Sec. 2.1 step 2 with
 * the mask of Fig. 4; the choice only affects speed.  Returns JK_ERR_SHAPE for another value. */
int jk_set_attn_kernel(jk_ctx* ctx, int32_t mode);

/* Diagnostics (the paper has no counterpart): with max_launches > 0 every kernel launch of this
 * context is bracketed by a pair of CUDA events on its stream (up to max_launches launches
 * between two collects); 0 switches it off.  jk_profile_collect synchronises `stream`, writes
 * the summed milliseconds and the launch count of every stage to the two host arrays of
 * jk_profile_stage_count() entries and starts over.  Event handles are host resources; no
 * device memory is allocated. */
int jk_profile_enable(jk_ctx* ctx, int32_t max_launches);
int jk_profile_collect(jk_ctx* ctx, void* stream, float* host_ms, int32_t* host_count);
/* As jk_profile_collect, but the recorded event pairs are kept.  When the calls were recorded into
 * a CUDA graph (stream capture with profiling enabled turns every event record into a graph
 * node), every replay of the graph records the same events again: read them after each replay. */
int jk_profile_read(jk_ctx* ctx, void* stream, float* host_ms, int32_t* host_count);
int32_t jk_profile_stage_count(void);
const char* jk_profile_stage_name(int32_t stage);

/* Draft weights (Sec. 3.1.1-3.1.2): device pointers, read-only, output-major. */
typedef struct {
  const void* router;       /* T [N, H]     expert centroids e_j (Eq. 2)                 */
  const void* w_gate;       /* T [N, I, H]  SiLU branch of Expert_j                      */
  const void* w_up;         /* T [N, I, H]  linear branch of Expert_j                    */
  const void* w_down;       /* T [N, H, I]  output projection of Expert_j                */
  const void* lm_head;      /* T [V, H]     the target model's LM head (shared, Eq. 4)   */
  const void* norm_weight;  /* T [H] or NULL (= ones)                                    */
} jk_draft_weights;

/* Candidate pool of one step: every child proposed by any jk_draft_expand call, in
 * generation order (layer, frontier slot, branch, rank).  Arrays are [B, *] with
 * `stride_b` elements between sequences; jk_draft_expand fills entries
 * gidx_base .. gidx_base + F*K*k_e - 1 of each sequence. */
typedef struct {
  int32_t* tok;             /* token id                                                  */
  float* score;             /* cumulative log-probability from the root                  */
  int32_t* parent;          /* generation index of the parent, -1 = root                 */
  int32_t* qslot;           /* row of the stored draft logits if the node was expanded, else -1 */
  int32_t* branch;          /* 0 = left (larger router score), 1 = right, ...            */
  int64_t stride_b;
} jk_pool;

/*
 * One draft layer for F frontier nodes per sequence (Sec. 3.1.2).
 *   x = RMSNorm(u) * norm_weight; s = softmax_N(x E^T) (Eq. 2); the K largest s keep their
 *   value as gates, larger one first = left (Eq. 5); y_r = Expert_{j_r}(x);
 *   f = sum_r g_r y_r + u (Eq. 3); branch feature b_r = g_r y_r (+ u);
 *   logits_r = b_r W_head^T (Eq. 4); per branch the k_e largest logits (ties: lower id)
 *   become children with score = parent_score + logit - logsumexp(logits_r); the W best
 *   children of the layer (ties: lower index) form the next frontier.
 * Inputs
 *   u            T   [B, F, H]   hidden state of each frontier node after draft attention (Eq. 1)
 *   parent_score f32 [B, F]      cumulative score of each frontier node (0 for the root)
 *   parent_gidx  i32 [B, F]      generation index of each frontier node (-1 for the root)
 *   gidx_base    generation index of this call's first child; slot_base: row index of this
 *                call's first node among all expanded nodes of the step (root = 0)
 * Outputs (any marked "opt" may be NULL)
 *   out_probs    f32 [B, F, N]   router scores s (opt)
 *   out_expert   i32 [B, F, K]   selected experts, left first
 *   out_gate     f32 [B, F, K]
 *   pool         children appended as described at jk_pool; qslot is set for the children
 *                chosen as next frontier (slot_base + F + position), -1 for the others
 *   out_lse      f32 [B, F, K]   logsumexp of each logits row (opt); laid out like out_logits:
 *                with logits_stride_b given, sequences are logits_stride_b / V elements apart,
 *                so that a call writes rows slot_base.. of a [B, S, K] array
 *   out_feat     T   [B, F, H]   combined feature f (Eq. 3)
 *   out_logits   f32 [B, F, K, V] (opt; needed later for sampling acceptance), with
 *                logits_stride_b elements between sequences (0 = dense, F*K*V), so that a call
 *                can write rows slot_base..slot_base+F-1 of a [B, S, K, V] buffer directly
 *   next_frontier      i32 [B, W'] flat child index (f*K + r)*k_e + j of the chosen children,
 *                      best first, W' = min(width, F*K*k_e) (opt, with the two arrays below);
 *                      width = 0 skips the selection (last layer)
 *   next_parent_score  f32 [B, W'] their scores
 *   next_parent_gidx   i32 [B, W'] their generation indices
 * Static tree policy (Sec. 3.1.2, last paragraph: the predefined tree of Eagle-1 is as usable as
 * the dynamic one): with static_select != NULL the next frontier is not chosen by score but
 * read from static_select, i32 [width] device, the flat child indices of the predefined shape in
 * frontier order, the same for every sequence; an index outside 0 .. F*K*k_e-1 sets JK_ERR_BOUNDS.
 * Contrastive mode (cfg.head_mode = 1; Sec. 3.2, Eq. 6-8): the head inputs are
 *   row 0: f^moe = g_1 y_1 + g_2 y_2 (+ u), row 1: f^const = beta y_1 - alpha y_2 (+ u).
 * The k_e best tokens of row 0 are the node's children as above.  Row 1 is the parallel-decoding
 * head: its k_e best tokens hang one level lower, under the node's best row-0 child (their pool
 * parent is that child's generation index, their score its score plus their log-probability
 * under row 1); they count only in a step's last pass (width = 0), get the score -inf in the
 * others, and are never chosen for the next frontier, so W' = min(width, F*k_e).  A step of tree
 * depth D then takes D-1 calls.
 * Errors: NULL/ALIGN/SHAPE/CAPACITY (B > max_batch, F > max_frontier)/WORKSPACE/CUDA.
 */
int jk_draft_expand(jk_ctx* ctx, void* stream, const jk_draft_weights* host_w,
                    int32_t batch, int32_t n_frontier, int32_t width,
                    const void* u, const float* parent_score, const int32_t* parent_gidx,
                    int32_t gidx_base, int32_t slot_base,
                    float* out_probs, int32_t* out_expert, float* out_gate,
                    const jk_pool* host_pool, float* out_lse, void* out_feat, float* out_logits,
                    int64_t logits_stride_b, int32_t* next_frontier, float* next_parent_score,
                    int32_t* next_parent_gidx, const int32_t* static_select);

/* Weights of the draft layer in front of the MoE (Sec. 3.1.1, 3.1.2): device pointers, read-only,
 * output-major. */
typedef struct {
  const void* emb;          /* T [V, H]      token embedding, shared with the target model      */
  const void* w_fc;         /* T [H, 2H]     reduction layer, acts on [emb(tok) ; parent feature] */
  const void* b_fc;         /* T [H] or NULL                                                     */
  const void* w_qkv;        /* T [(Hq + 2 Hkv) d, H]  rows of W_q, then W_k, then W_v           */
  const void* w_o;          /* T [H, Hq d]                                                       */
} jk_pre_weights;

/* State of the draft layer's attention over one step, caller-owned device memory: one entry per
 * expanded node ("slot": root = 0, then the frontier nodes of every pass in order), S_max =
 * stride_b slots per sequence. */
typedef struct {
  void* q;                  /* T   [B, S_max, Hq, d]  rotated query of every expanded node        */
  int32_t* slot_parent;     /* i32 [B, S_max]         parent slot, -1 for the root                */
  int32_t* slot_depth;      /* i32 [B, S_max]                                                     */
  int64_t stride_b;         /* S_max                                                              */
} jk_pre_state;

/*
 * The draft layer before the MoE for the F frontier nodes of one pass (Sec. 3.1.2, Eq. 1 and the
 * paragraph before it):
 *   h = W_fc [emb(tok) ; f_prev] (+ b_fc), with f_prev the feature f (Eq. 3, out_feat of
 *   jk_draft_expand) of the node's parent - for the root the target model's last feature;
 *   q, k, v = W_qkv h, q and k rotated (rotary positions, LLaMA pairing (i, i + d/2), base
 *   rope_theta) to position kv_len[b] + depth; k and v are appended to the draft layer's own
 *   cache at row kv_len[b] + slot; every node attends over rows 0 .. kv_len[b]-1 and the rows of
 *   itself and its ancestors; u = W_o Attn + h (Eq. 1).
 * No normalisation is applied in this block (Eq. 1-5 leave the norms out; Eagle-style drafts drop
 * the input norm of their single layer).  out_u feeds jk_draft_expand of the same pass.
 *   slot_base    slot of this pass's first node (0 for the root pass, then the running count)
 *   node_gidx    i32 [B, F] generation index of each node = next_parent_gidx of the previous
 *                jk_draft_expand; NULL in the root pass (then F = 1, the token is root_tok[b]
 *                and prev_feat is T [B, H])
 *   pool         the step's candidate pool: the nodes' tokens are pool.tok[node_gidx]
 *   prev_gidx_base, prev_slot_base, prev_frontier   gidx_base, slot_base and F of the previous
 *                pass; prev_feat T [B, prev_frontier, H] its out_feat.  A node's parent is
 *                frontier row (node_gidx - prev_gidx_base) / (K k_e) of that pass.
 *   k_cache, v_cache  T [B, Hkv, cap, d] with strides as in jk_tree_verify_attn; rows
 *                kv_len[b] .. kv_len[b] + slot_base + F - 1 are written over the passes
 *   out_u        T [B, F, H]
 * The attention runs over all slot_base + F nodes expanded so far (their queries are kept in
 * state.q), so slot_base + F <= 128 and <= max_depth * max_frontier.
 * Errors: NULL/ALIGN/SHAPE/CAPACITY/WORKSPACE/CUDA; a token or index out of range, or a cache too
 * short, sets JK_ERR_BOUNDS in the status word.
 */
int jk_draft_pre(jk_ctx* ctx, void* stream, const jk_pre_weights* host_w,
                 const jk_pre_state* host_state, int32_t batch, int32_t n_frontier,
                 int32_t slot_base, const int32_t* node_gidx, const jk_pool* host_pool,
                 int32_t prev_gidx_base, int32_t prev_slot_base, int32_t prev_frontier,
                 const void* prev_feat, const int32_t* root_tok, void* k_cache, void* v_cache,
                 int64_t cache_stride_b, int64_t cache_stride_h, int32_t cache_rows,
                 const int32_t* kv_len, float rope_theta, float softmax_scale, void* out_u);

/*
 * The target layer's own steps in front of jk_tree_verify_attn in a verification pass (Sec. 2.1
 * step 2: the target model evaluates all tree tokens in one forward pass): QKV projection of the
 * M tree tokens, rotary positions, K/V written at the tree slots.
 *   x        T [B, M, H]   the layer's (normalised) input hidden states of the tree tokens
 *   w_qkv    T [(Hq + 2 Hkv) d, H]   rows of W_q, then W_k, then W_v
 *   depth    i32 [B, M]    as written by jk_tree_finalize: node i sits at position kv_len[b] +
 *            depth[i] (nodes of one depth are alternatives for the same place in the sequence)
 *   q_out    T [B, M, Hq, d]   rotated queries (LLaMA pairing (i, i + d/2), base rope_theta)
 *   k_cache, v_cache   rotated K and V of node i go to row kv_len[b] + i
 * More than 256 tree tokens per call (B * M) go through the projection in chunks of 256 rows,
 * each streaming W_qkv once.  Errors as jk_tree_verify_attn; kv_len[b] + M > cache_rows sets
 * JK_ERR_BOUNDS.
 */
int jk_verify_qkv(jk_ctx* ctx, void* stream, const void* w_qkv, int32_t batch, int32_t tree_size,
                  const void* x, const int32_t* depth, void* q_out, void* k_cache, void* v_cache,
                  int64_t cache_stride_b, int64_t cache_stride_h, int32_t cache_rows,
                  const int32_t* kv_len, float rope_theta);

/*
 * The hidden states the next draft round starts from (Sec. 2.1 step 3 keeps the accepted path):
 *   out[b, 0] = hidden[b, 0] (the root), out[b, 1 + j] = hidden[b, acc_idx[b, j]] for
 *   j < n_acc[b]; rows after the accepted path are zero.
 *   hidden T [B, M, H]; n_acc i32 [B], acc_idx i32 [B, max_depth] as written by
 *   jk_accept_and_compact; out T [B, rows_out, H], rows_out <= max_depth + 1.
 */
int jk_gather_accepted(jk_ctx* ctx, void* stream, int32_t batch, int32_t tree_size,
                       const void* hidden, const int32_t* n_acc, const int32_t* acc_idx,
                       int32_t rows_out, void* out);

/*
 * Build the verification tree from the pool (Sec. 3.1.2; mask as in Fig. 4): node 0 is the
 * root (root_tok[b]); nodes 1..M-1 are the M-1 best pool entries by (score descending,
 * generation index ascending), listed in ascending generation index, so parent[i] < i.
 *   pool_n <= 4096 entries per sequence; tree_size = M <= max_tree, pool_n >= M-1.
 *   root_tok i32 [B]; outputs i32 [B, M]: tok, parent (-1 for the root), depth, branch, qslot
 *   (root: 0); anc u64 [B, M, 2]: bit t of the 128-bit set is 1 iff t is the node itself or
 *   one of its ancestors.
 *   static_keep  i32 [M-1] device or NULL.  Static tree policy: the generation indices of the
 *   predefined shape's nodes, ascending, the same for every sequence, kept instead of the M-1
 *   best by score; a list that is not ascending, reaches past pool_n or keeps a node without
 *   its parent sets JK_ERR_BOUNDS.
 */
int jk_tree_finalize(jk_ctx* ctx, void* stream, int32_t batch, const jk_pool* host_pool,
                     int32_t pool_n, const int32_t* root_tok, int32_t tree_size,
                     int32_t* tok, int32_t* parent, int32_t* depth, int32_t* branch,
                     int32_t* qslot, uint64_t* anc, const int32_t* static_keep);

/*
 * Tree-masked attention of one target layer over all M tree tokens (Sec. 2.1 step 2):
 *   out[b,i,h] = sum_c softmax_c(softmax_scale * q[b,i,h] . K[b,h/G,c] + mask) V[b,h/G,c],
 *   c < kv_len[b] + M, G = Hq/Hkv; column c is visible to node i iff c < kv_len[b] or
 *   c - kv_len[b] is i or an ancestor of i.
 *   q, out       T [B, M, Hq, d]
 *   k_cache, v_cache  T [B, Hkv, cap, d] addressed with cache_stride_b / cache_stride_h
 *                (elements); rows 0..kv_len[b]-1 hold the committed prefix, the caller has
 *                written the tree tokens' K/V at rows kv_len[b] .. kv_len[b]+M-1
 *   kv_len       i32 [B]; parent i32 [B, M] with parent[i] < i, -1 for the root
 *   cache_rows   rows addressable in each cache (cap); kv_len[b] + M > cap sets JK_ERR_BOUNDS
 */
int jk_tree_verify_attn(jk_ctx* ctx, void* stream, int32_t batch, int32_t tree_size,
                        const void* q, const void* k_cache, const void* v_cache,
                        int64_t cache_stride_b, int64_t cache_stride_h, int32_t cache_rows,
                        const int32_t* kv_len, const int32_t* parent, float softmax_scale,
                        void* out);

/*
 * jk_tree_verify_attn for callers that cannot allocate device memory.  (The paper has no
 * counterpart: this is a packaging variant of the call above.  It computes the same operation
 * with the CUDA-core kernel for both dtypes - fp32 products and an fp32 softmax - where
 * jk_tree_verify_attn uses the tensor-core kernels for bf16, which round the softmax weights to
 * bf16 and run several times faster; the two agree within the bf16 tolerance, not bit for bit.)
 *
 * Meant for processes that have given all free HBM to their own pools at start-up, so that a
 * later cudaMalloc for a workspace fails, and for decode loops that cannot afford the
 * device-wide synchronisation of cudaMalloc/cudaFree.  It needs no jk_set_workspace: the split-KV
 * partials go to a fixed 8 MiB (+256 B) array compiled into the library, which every GPU that
 * loads the library holds until the process exits.  The call makes no cudaMalloc/cudaFree and
 * uses no allocating library routine.
 *
 *   Arguments as jk_tree_verify_attn, plus
 *   status   i32 [1] device, required (NULL returns JK_ERR_NULL): receives JK_ERR_BOUNDS if
 *            kv_len[b] + M > cache_rows, in which case `out` is not written.  It is set by an
 *            atomic compare-and-swap on 0, so the caller clears it before the call and reads it
 *            after synchronising the stream.
 *   Limit    batch * tree_size * n_q_heads * (head_dim + 2) * 4 bytes <= 8 MiB (e.g. 60 nodes x
 *            32 heads x 128 uses 1 MiB per key slice); beyond it the call returns
 *            JK_ERR_CAPACITY, launches nothing, and jk_last_cuda_error(ctx) says why.
 *   Set-up   the first call on each device (with that device current) looks up the array's
 *            device address; make that first call before starting any stream capture.
 *   Sharing  all contexts, streams and threads of the process share the one array per GPU, and
 *            it keeps the previous call's contents.  Nothing in it has to start at zero (every
 *            partial a call reads it has written itself); but two of these calls that overlap
 *            on the same GPU race on the partials and give wrong results: run them one after
 *            the other.
 */
int jk_tree_verify_attn_static(jk_ctx* ctx, void* stream, int32_t batch, int32_t tree_size,
                               const void* q, const void* k_cache, const void* v_cache,
                               int64_t cache_stride_b, int64_t cache_stride_h, int32_t cache_rows,
                               const int32_t* kv_len, const int32_t* parent, float softmax_scale,
                               void* out, int32_t* status);

/*
 * Acceptance walk and KV compaction (Sec. 2.1 steps 2-3).
 *   mode 0 (greedy): from the root, follow the first child whose token equals the target's
 *     top-1 token (ties: lower id) at the current node; stop when none does; the bonus token
 *     is the top-1 at the stop node.
 *   mode 1 (sampling, temperature > 0): p = softmax(target/T) at the current node, q_r =
 *     softmax(draft/T) of branch r; children in order: accept iff u_accept[c] <
 *     min(1, p[x]/q_r[x]); on rejection p <- norm(max(0, p - q_r)), q_r[x] <- 0 and q_r is
 *     renormalised; if no child is accepted the bonus token is the inverse-CDF draw from p with
 *     u_bonus[depth].
 *   Then, for every layer l < n_layers and both caches, row kv_len+acc_idx[j] moves to row
 *   kv_len+1+j (j < n_acc) and kv_len[b] becomes kv_len[b] + 1 + n_acc[b].
 *   target_logits  [B, M, V] of tl_dtype (f32 or bf16)
 *   tok, parent, depth, branch, qslot   i32 [B, M] as written by jk_tree_finalize
 *   draft_logits   f32 [B, S, K, V], S = n_slots (mode 1; NULL in mode 0)
 *   u_accept       f32 [B, M], u_bonus f32 [B, max_depth+1], uniform in [0,1) (mode 1)
 *   k_caches, v_caches   device arrays of n_layers device pointers (may be NULL if n_layers = 0)
 *   outputs: n_acc i32 [B], acc_idx i32 [B, max_depth], acc_tok i32 [B, max_depth] (entries
 *   past n_acc are -1), bonus_tok i32 [B]
 */
int jk_accept_and_compact(jk_ctx* ctx, void* stream, int32_t batch, int32_t tree_size,
                          int32_t mode, float temperature,
                          const void* target_logits, int32_t tl_dtype,
                          const int32_t* tok, const int32_t* parent, const int32_t* depth,
                          const int32_t* branch, const int32_t* qslot,
                          const float* draft_logits, int32_t n_slots,
                          const float* u_accept, const float* u_bonus,
                          int32_t n_layers, void* const* k_caches, void* const* v_caches,
                          int64_t cache_stride_b, int64_t cache_stride_h, int32_t cache_rows,
                          int32_t* kv_len, int32_t* n_acc, int32_t* acc_idx, int32_t* acc_tok,
                          int32_t* bonus_tok);

#ifdef __cplusplus
}
#endif
#endif /* JAKIRO_H_ */
