"""ctypes binding of libjakiro.so: same entry points as include/jakiro.h.

Argument marshalling only.  Every arithmetic step runs in the CUDA kernels of
the library; torch is used for device memory and for the current stream.  If
the shared library has not been built the import of the library raises; there
is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, List, Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libjakiro.so")

JK_F32, JK_BF16 = 0, 1
JK_OK = 0
ERR = {"NULL": -1, "SHAPE": -2, "ALIGN": -3, "DTYPE": -4, "CAPACITY": -5, "WORKSPACE": -6,
       "CUDA": -7, "TIMEOUT": -8, "BOUNDS": -9}

EXPORTS = ["jk_create", "jk_destroy", "jk_workspace_bytes", "jk_set_workspace", "jk_strerror",
           "jk_last_cuda_error", "jk_read_status", "jk_set_tensor_path", "jk_draft_expand",
           "jk_tree_finalize", "jk_tree_verify_attn", "jk_accept_and_compact",
           "jk_profile_enable", "jk_profile_collect", "jk_profile_stage_count",
           "jk_profile_stage_name", "jk_tree_verify_attn_static", "jk_tensor_path_active",
           "jk_set_attn_kernel", "jk_profile_read", "jk_draft_pre",
           "jk_verify_qkv", "jk_gather_accepted"]


class JkConfig(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "hidden", "n_experts", "top_k", "inter", "vocab", "n_q_heads", "n_kv_heads", "head_dim",
        "max_batch", "max_tree", "max_depth", "max_frontier", "k_per_expert", "dtype")] + [
        ("rms_eps", C.c_float), ("use_pre_norm", C.c_int32), ("branch_residual", C.c_int32),
        ("head_mode", C.c_int32), ("contrast_alpha", C.c_float), ("contrast_beta", C.c_float)]


class JkDraftWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("router", "w_gate", "w_up", "w_down", "lm_head",
                                          "norm_weight")]


class JkPool(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("tok", "score", "parent", "qslot", "branch")] + [
        ("stride_b", C.c_int64)]


class JkPreWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in ("emb", "w_fc", "b_fc", "w_qkv", "w_o")]


class JkPreState(C.Structure):
    _fields_ = [("q", C.c_void_p), ("slot_parent", C.c_void_p), ("slot_depth", C.c_void_p),
                ("stride_b", C.c_int64)]


_lib = None


def lib() -> C.CDLL:
    """The loaded shared library.  Raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2502_06282_b200.build` "
                "(needs nvcc); there is no fallback implementation")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
        L.jk_create.argtypes = [C.POINTER(vp), C.POINTER(JkConfig)]
        L.jk_destroy.argtypes = [vp]
        L.jk_workspace_bytes.argtypes = [vp]
        L.jk_workspace_bytes.restype = C.c_size_t
        L.jk_set_workspace.argtypes = [vp, vp, vp, C.c_size_t]
        L.jk_strerror.argtypes = [C.c_int]
        L.jk_strerror.restype = C.c_char_p
        L.jk_last_cuda_error.argtypes = [vp]
        L.jk_last_cuda_error.restype = C.c_char_p
        L.jk_read_status.argtypes = [vp, vp, C.POINTER(i32)]
        L.jk_set_tensor_path.argtypes = [vp, i32]
        L.jk_tensor_path_active.argtypes = [vp]
        L.jk_set_attn_kernel.argtypes = [vp, i32]
        L.jk_draft_expand.argtypes = [vp, vp, C.POINTER(JkDraftWeights), i32, i32, i32, vp, vp,
                                      vp, i32, i32, vp, vp, vp, C.POINTER(JkPool), vp, vp, vp,
                                      i64, vp, vp, vp, vp]
        L.jk_tree_finalize.argtypes = [vp, vp, i32, C.POINTER(JkPool), i32, vp, i32, vp, vp, vp,
                                       vp, vp, vp, vp]
        L.jk_tree_verify_attn.argtypes = [vp, vp, i32, i32, vp, vp, vp, i64, i64, i32, vp, vp,
                                          f32, vp]
        L.jk_tree_verify_attn_static.argtypes = L.jk_tree_verify_attn.argtypes + [vp]
        L.jk_accept_and_compact.argtypes = [vp, vp, i32, i32, i32, f32, vp, i32, vp, vp, vp, vp,
                                            vp, vp, i32, vp, vp, i32, vp, vp, i64, i64, i32, vp,
                                            vp, vp, vp, vp]
        L.jk_draft_pre.argtypes = [vp, vp, C.POINTER(JkPreWeights), C.POINTER(JkPreState), i32, i32,
                                   i32, vp, C.POINTER(JkPool), i32, i32, i32, vp, vp, vp, vp, i64,
                                   i64, i32, vp, f32, f32, vp]
        L.jk_verify_qkv.argtypes = [vp, vp, vp, i32, i32, vp, vp, vp, vp, vp, i64, i64, i32, vp, f32]
        L.jk_gather_accepted.argtypes = [vp, vp, i32, i32, vp, vp, vp, i32, vp]
        L.jk_profile_enable.argtypes = [vp, i32]
        L.jk_profile_collect.argtypes = [vp, vp, C.POINTER(f32), C.POINTER(i32)]
        L.jk_profile_read.argtypes = [vp, vp, C.POINTER(f32), C.POINTER(i32)]
        L.jk_profile_stage_count.argtypes = []
        L.jk_profile_stage_name.argtypes = [i32]
        L.jk_profile_stage_name.restype = C.c_char_p
        for name in EXPORTS:
            if name not in ("jk_workspace_bytes", "jk_strerror", "jk_last_cuda_error",
                            "jk_profile_stage_name"):
                getattr(L, name).restype = C.c_int
        _lib = L
    return _lib


class JakiroError(RuntimeError):
    def __init__(self, code: int, where: str, detail: str = ""):
        self.code = code
        msg = lib().jk_strerror(code).decode()
        super().__init__(f"{where}: {msg} ({code}) {detail}".strip())


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    return None if t is None else t.data_ptr()


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def torch_dtype(dtype: str) -> torch.dtype:
    return torch.bfloat16 if dtype == "bf16" else torch.float32


class Context:
    """Owns a jk_ctx and its device workspace (a torch allocation)."""

    def __init__(self, *, hidden, n_experts, top_k, inter, vocab, n_q_heads, n_kv_heads,
                 head_dim, max_batch, max_tree, max_depth, max_frontier, k_per_expert, dtype,
                 rms_eps=1e-5, use_pre_norm=True, branch_residual=True, head_mode=0,
                 contrast_alpha=0.0, contrast_beta=1.0, device="cuda", allocate=True):
        self.cfg = JkConfig(hidden, n_experts, top_k, inter, vocab, n_q_heads, n_kv_heads,
                            head_dim, max_batch, max_tree, max_depth, max_frontier,
                            k_per_expert, JK_BF16 if dtype == "bf16" else JK_F32, rms_eps,
                            int(use_pre_norm), int(branch_residual), int(head_mode),
                            float(contrast_alpha), float(contrast_beta))
        self.dtype = dtype
        self.tdtype = torch_dtype(dtype)
        self._h = C.c_void_p()
        rc = lib().jk_create(C.byref(self._h), C.byref(self.cfg))
        if rc != JK_OK:
            self._h = C.c_void_p()
            raise JakiroError(rc, "jk_create")
        self.workspace = None
        self.device = device
        if allocate:
            n = lib().jk_workspace_bytes(self._h)
            self.workspace = torch.empty(n + 256, dtype=torch.uint8, device=device)
            base = (self.workspace.data_ptr() + 255) // 256 * 256
            self._check(lib().jk_set_workspace(self._h, _stream(), base, n), "jk_set_workspace")

    def set_workspace(self, buf: torch.Tensor, offset: int = 0):
        """jk_set_workspace on a caller-made uint8 device buffer: the workspace starts at the
        first 256-byte boundary at or after buf[offset]; the buffer must stay alive."""
        n = lib().jk_workspace_bytes(self._h)
        base = (buf.data_ptr() + offset + 255) // 256 * 256
        if base + n > buf.data_ptr() + buf.numel():
            raise ValueError("buffer too small for the workspace")
        self.workspace = buf
        self._check(lib().jk_set_workspace(self._h, _stream(), base, n), "jk_set_workspace")
        return base - buf.data_ptr()

    @classmethod
    def for_workload(cls, w, frontier_sizes=None, **kw) -> "Context":
        fs = w.frontier_sizes if frontier_sizes is None else frontier_sizes
        kw.setdefault("head_mode", getattr(w, "head_mode", 0))
        return cls(hidden=w.hidden, n_experts=w.n_experts, top_k=w.top_k, inter=w.inter,
                   vocab=w.vocab, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads,
                   head_dim=w.head_dim, max_batch=w.batch, max_tree=w.tree_size,
                   max_depth=w.depth, max_frontier=max(fs),
                   k_per_expert=w.k_per_expert, dtype=w.dtype, **kw)

    def _check(self, rc: int, where: str):
        if rc != JK_OK:
            detail = lib().jk_last_cuda_error(self._h).decode() if rc == ERR["CUDA"] else ""
            raise JakiroError(rc, where, detail)

    @property
    def workspace_bytes(self) -> int:
        return lib().jk_workspace_bytes(self._h)

    def close(self):
        if self._h:
            lib().jk_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def set_attn_kernel(self, mode: int):
        self._check(lib().jk_set_attn_kernel(self._h, int(mode)), "jk_set_attn_kernel")

    def set_tensor_path(self, enable: bool):
        self._check(lib().jk_set_tensor_path(self._h, int(enable)), "jk_set_tensor_path")

    @property
    def tensor_path_active(self) -> bool:
        return bool(lib().jk_tensor_path_active(self._h))

    def read_status(self) -> int:
        out = C.c_int32(0)
        self._check(lib().jk_read_status(self._h, _stream(), C.byref(out)), "jk_read_status")
        return out.value

    def profile_enable(self, max_launches: int):
        self._check(lib().jk_profile_enable(self._h, max_launches), "jk_profile_enable")

    def profile_collect(self, keep: bool = False) -> Dict[str, tuple]:
        """{stage name: (total ms, launches)} since the last collect; synchronises.  keep=True
        leaves the recorded event pairs in place (jk_profile_read), for graph replays."""
        n = lib().jk_profile_stage_count()
        ms = (C.c_float * n)()
        cnt = (C.c_int32 * n)()
        fn = lib().jk_profile_read if keep else lib().jk_profile_collect
        self._check(fn(self._h, _stream(), ms, cnt), "jk_profile_collect")
        return {lib().jk_profile_stage_name(i).decode(): (float(ms[i]), int(cnt[i]))
                for i in range(n) if cnt[i]}

    # ------------------------------------------------------------------ calls
    @staticmethod
    def weights_struct(w: Dict[str, torch.Tensor]) -> JkDraftWeights:
        return JkDraftWeights(_ptr(w["router"]), _ptr(w["w_gate"]), _ptr(w["w_up"]),
                              _ptr(w["w_down"]), _ptr(w["lm_head"]), _ptr(w.get("norm_weight")))

    @staticmethod
    def pool_struct(pool: Dict[str, torch.Tensor]) -> JkPool:
        return JkPool(_ptr(pool["tok"]), _ptr(pool["score"]), _ptr(pool["parent"]),
                      _ptr(pool["qslot"]), _ptr(pool["branch"]), pool["tok"].stride(0))

    def draft_expand(self, weights, batch, n_frontier, width, u, parent_score, parent_gidx,
                     gidx_base, slot_base, out_probs, out_expert, out_gate, pool, out_lse,
                     out_feat, out_logits, next_frontier, next_parent_score, next_parent_gidx,
                     static_select=None):
        ws = weights if isinstance(weights, JkDraftWeights) else self.weights_struct(weights)
        ps = pool if isinstance(pool, JkPool) else self.pool_struct(pool)
        rc = lib().jk_draft_expand(
            self._h, _stream(), C.byref(ws), batch, n_frontier, width, _ptr(u),
            _ptr(parent_score), _ptr(parent_gidx), gidx_base, slot_base, _ptr(out_probs),
            _ptr(out_expert), _ptr(out_gate), C.byref(ps), _ptr(out_lse), _ptr(out_feat),
            _ptr(out_logits), 0 if out_logits is None else out_logits.stride(0),
            _ptr(next_frontier), _ptr(next_parent_score),
            _ptr(next_parent_gidx), _ptr(static_select))
        self._check(rc, "jk_draft_expand")

    @staticmethod
    def pre_weights_struct(w: Dict[str, torch.Tensor]) -> JkPreWeights:
        return JkPreWeights(_ptr(w["emb"]), _ptr(w["w_fc"]), _ptr(w.get("b_fc")), _ptr(w["w_qkv"]),
                            _ptr(w["w_o"]))

    def draft_pre(self, pre_weights, state: JkPreState, batch, n_frontier, slot_base, node_gidx,
                  pool, prev_gidx_base, prev_slot_base, prev_frontier, prev_feat, root_tok, k_cache,
                  v_cache, kv_len, rope_theta, scale, out_u, cache_rows=None):
        ws = pre_weights if isinstance(pre_weights, JkPreWeights) else self.pre_weights_struct(pre_weights)
        ps = pool if isinstance(pool, JkPool) else self.pool_struct(pool)
        rows = k_cache.shape[2] if cache_rows is None else cache_rows
        rc = lib().jk_draft_pre(self._h, _stream(), C.byref(ws), C.byref(state), batch, n_frontier,
                                slot_base, _ptr(node_gidx), C.byref(ps), prev_gidx_base,
                                prev_slot_base, prev_frontier, _ptr(prev_feat), _ptr(root_tok),
                                _ptr(k_cache), _ptr(v_cache), k_cache.stride(0), k_cache.stride(1),
                                rows, _ptr(kv_len), float(rope_theta), float(scale), _ptr(out_u))
        self._check(rc, "jk_draft_pre")

    def verify_qkv(self, w_qkv, batch, tree_size, x, depth, q_out, k_cache, v_cache, kv_len,
                   rope_theta, cache_rows=None):
        rows = k_cache.shape[2] if cache_rows is None else cache_rows
        rc = lib().jk_verify_qkv(self._h, _stream(), _ptr(w_qkv), batch, tree_size, _ptr(x),
                                 _ptr(depth), _ptr(q_out), _ptr(k_cache), _ptr(v_cache),
                                 k_cache.stride(0), k_cache.stride(1), rows, _ptr(kv_len),
                                 float(rope_theta))
        self._check(rc, "jk_verify_qkv")

    def gather_accepted(self, batch, tree_size, hidden, n_acc, acc_idx, rows_out, out):
        rc = lib().jk_gather_accepted(self._h, _stream(), batch, tree_size, _ptr(hidden),
                                      _ptr(n_acc), _ptr(acc_idx), rows_out, _ptr(out))
        self._check(rc, "jk_gather_accepted")

    def tree_finalize(self, batch, pool, pool_n, root_tok, tree_size, tok, parent, depth, branch,
                      qslot, anc, static_keep=None):
        ps = pool if isinstance(pool, JkPool) else self.pool_struct(pool)
        rc = lib().jk_tree_finalize(self._h, _stream(), batch, C.byref(ps), pool_n,
                                    _ptr(root_tok), tree_size, _ptr(tok), _ptr(parent),
                                    _ptr(depth), _ptr(branch), _ptr(qslot), _ptr(anc),
                                    _ptr(static_keep))
        self._check(rc, "jk_tree_finalize")

    def tree_verify_attn(self, batch, tree_size, q, k_cache, v_cache, kv_len, parent, scale, out,
                         cache_rows=None):
        rows = k_cache.shape[2] if cache_rows is None else cache_rows
        rc = lib().jk_tree_verify_attn(self._h, _stream(), batch, tree_size, _ptr(q),
                                       _ptr(k_cache), _ptr(v_cache), k_cache.stride(0),
                                       k_cache.stride(1), rows, _ptr(kv_len), _ptr(parent),
                                       float(scale), _ptr(out))
        self._check(rc, "jk_tree_verify_attn")

    def tree_verify_attn_static(self, batch, tree_size, q, k_cache, v_cache, kv_len, parent,
                                scale, out, status, cache_rows=None):
        """jk_tree_verify_attn_static: the same attention without any workspace, for callers
        that cannot allocate device memory; scratch is the library's built-in 8 MiB array.
        `status` is a caller-owned int32 device word (cleared by the caller) that receives
        JK_ERR_BOUNDS when a cache is too short."""
        rows = k_cache.shape[2] if cache_rows is None else cache_rows
        rc = lib().jk_tree_verify_attn_static(self._h, _stream(), batch, tree_size, _ptr(q),
                                              _ptr(k_cache), _ptr(v_cache), k_cache.stride(0),
                                              k_cache.stride(1), rows, _ptr(kv_len),
                                              _ptr(parent), float(scale), _ptr(out),
                                              _ptr(status))
        if rc != JK_OK:
            detail = lib().jk_last_cuda_error(self._h).decode()
            raise JakiroError(rc, "jk_tree_verify_attn_static", detail)

    def accept_and_compact(self, batch, tree_size, mode, temperature, target_logits, tree,
                           draft_logits, n_slots, u_accept, u_bonus, n_layers, k_ptrs, v_ptrs,
                           cache_stride_b, cache_stride_h, cache_rows, kv_len, n_acc, acc_idx,
                           acc_tok, bonus_tok):
        tl_dtype = JK_BF16 if target_logits.dtype == torch.bfloat16 else JK_F32
        rc = lib().jk_accept_and_compact(
            self._h, _stream(), batch, tree_size, mode, float(temperature), _ptr(target_logits),
            tl_dtype, _ptr(tree["tok"]), _ptr(tree["parent"]), _ptr(tree["depth"]),
            _ptr(tree["branch"]), _ptr(tree["qslot"]), _ptr(draft_logits), n_slots,
            _ptr(u_accept), _ptr(u_bonus), n_layers, _ptr(k_ptrs), _ptr(v_ptrs), cache_stride_b,
            cache_stride_h, cache_rows, _ptr(kv_len), _ptr(n_acc), _ptr(acc_idx), _ptr(acc_tok),
            _ptr(bonus_tok))
        self._check(rc, "jk_accept_and_compact")


class StepBuffers:
    """Device buffers of one draft-and-verify step for a workload, allocated once."""

    def __init__(self, ctx: Context, w, keep_logits: bool = True, device="cuda",
                 frontier_sizes=None):
        """frontier_sizes: the expanded nodes per draft pass when they do not follow from the
        workload's width (a predefined tree shape); default w.frontier_sizes."""
        B, K, ke, V, H = w.batch, w.top_k, w.k_per_expert, w.vocab, w.hidden
        fs = list(w.frontier_sizes if frontier_sizes is None else frontier_sizes)
        self.frontier_sizes = fs
        self.pool_n = sum(f * K * ke for f in fs)
        self.n_slots = sum(fs)
        i32 = dict(dtype=torch.int32, device=device)
        f32 = dict(dtype=torch.float32, device=device)
        self.w = w
        self.pool = {"tok": torch.empty(B, self.pool_n, **i32),
                     "score": torch.empty(B, self.pool_n, **f32),
                     "parent": torch.empty(B, self.pool_n, **i32),
                     "qslot": torch.empty(B, self.pool_n, **i32),
                     "branch": torch.empty(B, self.pool_n, **i32)}
        self.pool_struct = ctx.pool_struct(self.pool)
        self.probs = [torch.empty(B, F, w.n_experts, **f32) for F in fs]
        self.expert = [torch.empty(B, F, K, **i32) for F in fs]
        self.gate = [torch.empty(B, F, K, **f32) for F in fs]
        # log-sum-exp of every stored logits row: [B, S, K], laid out like the logits (a call
        # writes rows slot_base.. of every sequence); dense per-pass arrays when no logits are kept
        self.lse_all = torch.empty(B, self.n_slots, K, **f32) if keep_logits else None
        self.lse = self.lse_views() if keep_logits else [torch.empty(B, F, K, **f32) for F in fs]
        self.feat = [torch.empty(B, F, H, dtype=ctx.tdtype, device=device) for F in fs]
        self.logits = torch.empty(B, self.n_slots, K, V, **f32) if keep_logits else None
        nxt = fs[1:] + [1]                      # nodes chosen by pass l = nodes expanded by pass l+1
        self.frontier = [torch.empty(B, n, **i32) for n in nxt]
        self.parent_score = [torch.zeros(B, 1, **f32)] + [torch.empty(B, n, **f32) for n in nxt]
        self.parent_gidx = [torch.full((B, 1), -1, **i32)] + [torch.empty(B, n, **i32) for n in nxt]
        M = w.tree_size
        self.tree = {k: torch.empty(B, M, **i32) for k in ("tok", "parent", "depth", "branch",
                                                           "qslot")}
        self.anc = torch.empty(B, M, 2, dtype=torch.int64, device=device)
        self.n_acc = torch.empty(B, **i32)
        self.acc_idx = torch.empty(B, w.depth, **i32)
        self.acc_tok = torch.empty(B, w.depth, **i32)
        self.bonus = torch.empty(B, **i32)


def _lse_views(self):
    out, s0 = [], 0
    for F in self.frontier_sizes:
        out.append(self.lse_all[:, s0:s0 + F])
        s0 += F
    return out


StepBuffers.lse_views = _lse_views


def run_draft(ctx: Context, bufs: StepBuffers, weights, u_layers: Sequence[torch.Tensor],
              root_tok: torch.Tensor, finalize: bool = True, static_plan=None):
    """One jk_draft_expand call per draft pass, then jk_tree_finalize.  The expanded nodes'
    logits are kept in bufs.logits at slot order when that buffer exists.  static_plan (from
    static_tree.plan_from_paths, with device arrays): the predefined tree shape that replaces the
    score-driven choice of frontier and final tree."""
    w = bufs.w
    fs = bufs.frontier_sizes
    B, K, ke = w.batch, w.top_k, w.k_per_expert
    gidx_base = 0
    slot_base = 0
    for l, F in enumerate(fs):
        last = l == len(fs) - 1
        out_logits = None
        if bufs.logits is not None:      # rows slot_base..slot_base+F-1 of every sequence
            out_logits = bufs.logits[:, slot_base:slot_base + F]
        width = 0 if last else fs[l + 1]
        ctx.draft_expand(weights, B, F, width, u_layers[l],
                         bufs.parent_score[l], bufs.parent_gidx[l], gidx_base, slot_base,
                         bufs.probs[l], bufs.expert[l], bufs.gate[l], bufs.pool_struct,
                         bufs.lse[l], bufs.feat[l], out_logits,
                         None if last else bufs.frontier[l],
                         None if last else bufs.parent_score[l + 1],
                         None if last else bufs.parent_gidx[l + 1],
                         None if (last or static_plan is None) else static_plan["select"][l])
        gidx_base += F * K * ke
        slot_base += F
    if finalize:
        ctx.tree_finalize(B, bufs.pool_struct, bufs.pool_n, root_tok, w.tree_size,
                          bufs.tree["tok"], bufs.tree["parent"], bufs.tree["depth"],
                          bufs.tree["branch"], bufs.tree["qslot"], bufs.anc,
                          None if static_plan is None else static_plan["keep"])


class PreBuffers:
    """Device state of the draft layer's pre-MoE block for one step: the rotated queries and the
    partial tree (parent slot, depth) of every expanded node, and the hidden states u per pass."""

    def __init__(self, ctx: Context, bufs: StepBuffers, device="cuda"):
        w = bufs.w
        S = bufs.n_slots
        self.q = torch.empty(w.batch, S, w.n_q_heads, w.head_dim, dtype=ctx.tdtype, device=device)
        self.slot_parent = torch.empty(w.batch, S, dtype=torch.int32, device=device)
        self.slot_depth = torch.empty(w.batch, S, dtype=torch.int32, device=device)
        self.state = JkPreState(_ptr(self.q), _ptr(self.slot_parent), _ptr(self.slot_depth), S)
        self.u = [torch.empty(w.batch, F, w.hidden, dtype=ctx.tdtype, device=device)
                  for F in bufs.frontier_sizes]


def run_draft_chained(ctx: Context, bufs: StepBuffers, pre: PreBuffers, weights, pre_weights,
                      root_tok: torch.Tensor, root_feat: torch.Tensor, k_cache, v_cache, kv_len,
                      rope_theta: float, scale: float, finalize: bool = True):
    """The whole draft of one step with nothing synthetic in between: per pass jk_draft_pre turns
    the frontier's tokens and their parents' features into u (Eq. 1), jk_draft_expand grows the
    tree from u (Eq. 2-5) and hands back the features the next pass starts from."""
    w = bufs.w
    fs = bufs.frontier_sizes
    B, K, ke = w.batch, w.top_k, w.k_per_expert
    gidx_base = slot_base = 0
    prev = (0, 0, 1)                       # gidx_base, slot_base, F of the previous pass
    for l, F in enumerate(fs):
        last = l == len(fs) - 1
        ctx.draft_pre(pre_weights, pre.state, B, F, slot_base,
                      None if l == 0 else bufs.parent_gidx[l], bufs.pool_struct, prev[0], prev[1],
                      prev[2], root_feat if l == 0 else bufs.feat[l - 1], root_tok, k_cache,
                      v_cache, kv_len, rope_theta, scale, pre.u[l])
        out_logits = None if bufs.logits is None else bufs.logits[:, slot_base:slot_base + F]
        ctx.draft_expand(weights, B, F, 0 if last else fs[l + 1], pre.u[l], bufs.parent_score[l],
                         bufs.parent_gidx[l], gidx_base, slot_base, bufs.probs[l], bufs.expert[l],
                         bufs.gate[l], bufs.pool_struct, bufs.lse[l], bufs.feat[l], out_logits,
                         None if last else bufs.frontier[l],
                         None if last else bufs.parent_score[l + 1],
                         None if last else bufs.parent_gidx[l + 1])
        prev = (gidx_base, slot_base, F)
        gidx_base += F * K * ke
        slot_base += F
    if finalize:
        ctx.tree_finalize(B, bufs.pool_struct, bufs.pool_n, root_tok, w.tree_size,
                          bufs.tree["tok"], bufs.tree["parent"], bufs.tree["depth"],
                          bufs.tree["branch"], bufs.tree["qslot"], bufs.anc)
