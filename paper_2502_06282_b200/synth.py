"""Seeded synthetic inputs for the Jakiro draft-and-verify step.

This module only *draws* inputs (weights, hidden states, KV caches, trees,
target logits, uniforms) and rounds them to the storage type.  It holds none
of the method's arithmetic: no router, no expert, no attention, no acceptance
rule.  Both the CPU oracle's tests and the CUDA path's tests read their inputs
from here so that the two sides see identical bits.

Shapes follow the paper's setting: one Eagle-style draft decoder layer whose
MLP is replaced by N expert FFNs with K=2 active (Sec. 3.1.2, Eq. 1-5), batch
size 1 by default (Sec. 4, "Models and tasks"), LLaMA-family target shapes.
Trained weights and the evaluation suites of Sec. 4 are not available, so all
tensors are random: weights N(0, 0.02), activations N(0, 1), token ids
uniform, and target logits with a planted agreement rate so that the accepted
length per step lands in the range the paper's tables report (3.5 to 5.9).
"""
from __future__ import annotations

from dataclasses import dataclass, replace
from typing import Dict, List, Optional, Tuple

import numpy as np


# --------------------------------------------------------------------------
# storage rounding
# --------------------------------------------------------------------------
def bf16_round(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even) and return
    them as float32, so that a later cast to bf16 is exact."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    bits = a.view(np.uint32)
    lsb = (bits >> np.uint32(16)) & np.uint32(1)
    rounded = (bits + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return rounded.view(np.float32)


def store_round(a: np.ndarray, dtype: str) -> np.ndarray:
    """Values as they are stored on the device for `dtype` ("f32" | "bf16")."""
    if dtype == "bf16":
        return bf16_round(a)
    return np.ascontiguousarray(a, dtype=np.float32)


# --------------------------------------------------------------------------
# workload configurations
# --------------------------------------------------------------------------
@dataclass(frozen=True)
class Workload:
    name: str
    hidden: int            # H
    n_q_heads: int         # Hq
    n_kv_heads: int        # Hkv
    head_dim: int          # d
    vocab: int             # V
    n_experts: int         # N
    top_k: int             # K (active experts per node, Eq. 5)
    inter: int             # I (expert inner size)
    prefix: int            # P (committed KV length)
    tree_size: int         # M (tree nodes including the root)
    depth: int             # D (draft layers = expand calls per step)
    k_per_expert: int      # k_e (children proposed per expert per node)
    width: int             # W (frontier nodes kept per layer)
    batch: int             # B
    dtype: str             # "f32" | "bf16"
    n_layers: int          # L target layers verified per step
    seed: int
    head_mode: int = 0     # 0: decoupled heads (Eq. 4); 1: contrastive heads with the hybrid
                           # schedule of Sec. 3.2 (depth D from D-1 draft passes)

    @property
    def n_passes(self) -> int:
        """jk_draft_expand calls per step."""
        return self.depth - 1 if self.head_mode == 1 else self.depth

    @property
    def frontier_sizes(self) -> List[int]:
        """F_1.. of the draft passes: the root alone, then at most W nodes per pass (in the
        contrastive mode only a node's row-0 children can be expanded)."""
        per_node = self.k_per_expert * (1 if self.head_mode == 1 else self.top_k)
        out = [1]
        for _ in range(1, self.n_passes):
            out.append(min(self.width, out[-1] * per_node))
        return out

    @property
    def pool_size(self) -> int:
        return sum(f * self.top_k * self.k_per_expert for f in self.frontier_sizes)

    @property
    def n_slots(self) -> int:
        """Expanded nodes per sequence over the whole step (rows of q kept)."""
        return sum(self.frontier_sizes)

    @property
    def kv_capacity(self) -> int:
        cap = self.prefix + self.tree_size
        return (cap + 63) // 64 * 64


WORKLOADS: Dict[str, Workload] = {
    # configs[0]: small case the oracle finishes in seconds
    "tiny": Workload("tiny", 512, 8, 8, 64, 4096, 4, 2, 1376, 128, 16, 4, 2, 4, 1,
                     "f32", 2, 1000),
    # a bf16 twin of the tiny case, used to exercise the tensor-core kernels
    "tiny_bf16": Workload("tiny_bf16", 512, 8, 8, 64, 4096, 4, 2, 1376, 128, 16, 4, 2, 4, 1,
                          "bf16", 2, 1500),
    # configs[1]: LLaMA2-7B-shaped step
    "llama2_7b": Workload("llama2_7b", 4096, 32, 32, 128, 32000, 4, 2, 11008, 1024, 60, 6,
                          5, 10, 1, "bf16", 32, 2000),
    # configs[2]: LLaMA2-13B-shaped step (batch 1 and 4)
    "llama2_13b": Workload("llama2_13b", 5120, 40, 40, 128, 32000, 4, 2, 13824, 2048, 60, 6,
                           5, 10, 1, "bf16", 40, 3000),
    "llama2_13b_b4": Workload("llama2_13b_b4", 5120, 40, 40, 128, 32000, 4, 2, 13824, 2048,
                              60, 6, 5, 10, 4, "bf16", 40, 3400),
    # configs[3]: LLaMA3-8B-shaped step (GQA, large vocabulary)
    "llama3_8b": Workload("llama3_8b", 4096, 32, 8, 128, 128256, 4, 2, 14336, 4096, 60, 6,
                          5, 10, 1, "bf16", 32, 4000),
    # configs[4]: one point of the LLaMA2-70B layer-shaped sweep
    "llama2_70b_layer": Workload("llama2_70b_layer", 8192, 64, 8, 128, 32000, 4, 2, 28672,
                                 4096, 60, 6, 5, 10, 1, "bf16", 1, 5000),
}


def scaled(w: Workload, **kw) -> Workload:
    return replace(w, **kw)


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[seed, stream]))


def _normal(rng: np.random.Generator, shape, std: float) -> np.ndarray:
    a = rng.standard_normal(size=shape, dtype=np.float32)
    if std != 1.0:
        a *= np.float32(std)
    return a


# --------------------------------------------------------------------------
# draft weights and hidden states
# --------------------------------------------------------------------------
def draft_weights(w: Workload) -> Dict[str, np.ndarray]:
    """Random-init draft layer: expert centroids, N SiLU-gated FFNs, shared LM
    head; N(0, 0.02), rounded to the storage type.  Output-major layouts:
    router [N,H], w_gate/w_up [N,I,H], w_down [N,H,I], lm_head [V,H]."""
    r = lambda s: _rng(w.seed, s)
    out = {
        "router": _normal(r(1), (w.n_experts, w.hidden), 0.02),
        "w_gate": _normal(r(2), (w.n_experts, w.inter, w.hidden), 0.02),
        "w_up": _normal(r(3), (w.n_experts, w.inter, w.hidden), 0.02),
        "w_down": _normal(r(4), (w.n_experts, w.hidden, w.inter), 0.02),
        "lm_head": _normal(r(5), (w.vocab, w.hidden), 0.02),
        "norm_weight": np.ones((w.hidden,), dtype=np.float32),
    }
    return {k: store_round(v, w.dtype) for k, v in out.items()}


def shared_weights(w: Workload) -> Dict[str, np.ndarray]:
    """The parts of draft_weights that do not grow with the expert count: expert centroids, LM
    head, norm weight (same streams as draft_weights)."""
    r = lambda s: _rng(w.seed, s)
    out = {
        "router": _normal(r(1), (w.n_experts, w.hidden), 0.02),
        "lm_head": _normal(r(5), (w.vocab, w.hidden), 0.02),
        "norm_weight": np.ones((w.hidden,), dtype=np.float32),
    }
    return {k: store_round(v, w.dtype) for k, v in out.items()}


def expert_weight(w: Workload, name: str, e: int) -> np.ndarray:
    """One expert's matrix ("w_gate" | "w_up" [I, H], "w_down" [H, I]), N(0, 0.02), from a
    stream of its own, for shapes whose whole expert set would not fit the host in fp32.  (Not
    the same numbers as draft_weights, which draws all experts of a matrix from one stream.)"""
    idx = {"w_gate": 0, "w_up": 1, "w_down": 2}[name]
    shape = (w.hidden, w.inter) if name == "w_down" else (w.inter, w.hidden)
    return store_round(_normal(_rng(w.seed, 1000 + 3 * e + idx), shape, 0.02), w.dtype)


def pre_weights(w: Workload, bias: bool = True) -> Dict[str, np.ndarray]:
    """Random-init weights of the draft layer in front of the MoE (Sec. 3.1.2, Eq. 1): token
    embedding [V, H] N(0, 1), reduction layer w_fc [H, 2H] and b_fc [H], w_qkv [(Hq + 2 Hkv) d, H]
    (W_q rows, W_k rows, W_v rows), w_o [H, Hq d], all N(0, 0.02) but the embedding."""
    r = lambda s: _rng(w.seed, s)
    qd, kvd = w.n_q_heads * w.head_dim, w.n_kv_heads * w.head_dim
    out = {
        "emb": _normal(r(21), (w.vocab, w.hidden), 1.0),
        "w_fc": _normal(r(22), (w.hidden, 2 * w.hidden), 0.02),
        "w_qkv": _normal(r(24), (qd + 2 * kvd, w.hidden), 0.02),
        "w_o": _normal(r(25), (w.hidden, qd), 0.02),
    }
    if bias:
        out["b_fc"] = _normal(r(23), (w.hidden,), 0.02)
    return {k: store_round(v, w.dtype) for k, v in out.items()}


def root_feature(w: Workload) -> np.ndarray:
    """[B, H]: the target model's feature of the last committed token (the f_{i-1} the root's
    token is paired with), N(0, 1)."""
    return store_round(_normal(_rng(w.seed, 26), (w.batch, w.hidden), 1.0), w.dtype)


def layer_hidden(w: Workload, layer: int, n_frontier: int) -> np.ndarray:
    """u [B, F, H]: post-attention hidden state of each frontier node (the
    output of Eq. 1), N(0, 1).  Stands in for the draft's reduction layer and
    self-attention, which sit before the MoE."""
    a = _normal(_rng(w.seed, 100 + layer), (w.batch, n_frontier, w.hidden), 1.0)
    return store_round(a, w.dtype)


# --------------------------------------------------------------------------
# trees (structure only)
# --------------------------------------------------------------------------
def chain_tree(m: int) -> np.ndarray:
    return np.arange(-1, m - 1, dtype=np.int32)


def star_tree(m: int) -> np.ndarray:
    p = np.zeros(m, dtype=np.int32)
    p[0] = -1
    return p


def binary_tree(m: int) -> np.ndarray:
    p = np.array([(i - 1) // 2 for i in range(m)], dtype=np.int32)
    p[0] = -1
    return p


def random_tree(m: int, max_depth: int, seed: int) -> np.ndarray:
    """Random tree built level by level: parent[i] < i, depth <= max_depth,
    nodes in non-decreasing depth order, children of one parent contiguous."""
    rng = _rng(seed, 7)
    parent = [-1]
    prev = [0]
    remaining = m - 1
    level = 1
    while remaining > 0:
        if level >= max_depth:
            n = remaining
        else:
            hi = max(1, min(remaining, 3 * len(prev)))
            n = int(rng.integers(1, hi + 1))
        picks = sorted(int(prev[int(j)]) for j in rng.integers(0, len(prev), size=n))
        first = len(parent)
        parent.extend(picks)
        prev = list(range(first, first + n))
        remaining -= n
        level += 1
    return np.asarray(parent, dtype=np.int32)


def static_paths(w: Workload) -> List[Tuple[int, ...]]:
    """A predefined tree shape of w.tree_size - 1 nodes and depth <= w.depth for the static
    policy, as rank paths (rank c of a node = its c-th candidate in child order).  Level 1 takes
    the root's candidates in order; below, the first w.width nodes of a level (in path order) are
    expanded and handed children round-robin, best left-branch rank, best right-branch rank, second
    left, second right, ..., until the node budget is spent."""
    per_node = w.top_k * w.k_per_expert
    order = []
    for j in range(w.k_per_expert):
        for r in range(w.top_k):
            order.append(r * w.k_per_expert + j)
    budget = w.tree_size - 1
    paths: List[Tuple[int, ...]] = []
    level = [(c,) for c in range(min(per_node, budget))]
    paths += level
    budget -= len(level)
    for d in range(2, w.depth + 1):
        parents = sorted(level)[:w.width]
        left = w.depth - d                       # levels still to come below this one
        here = budget if left == 0 else max(len(parents), budget // (left + 1))
        here = min(here, budget, len(parents) * per_node)
        nxt = []
        i = 0
        while len(nxt) < here:
            p = parents[i % len(parents)]
            nxt.append(p + (order[i // len(parents)],))
            i += 1
        paths += nxt
        budget -= len(nxt)
        level = nxt
        if budget <= 0 or not level:
            break
    return paths


def tree_depths(parent: np.ndarray) -> np.ndarray:
    d = np.zeros(len(parent), dtype=np.int32)
    for i in range(1, len(parent)):
        d[i] = d[parent[i]] + 1
    return d


def random_tokens(w: Workload, shape, stream: int) -> np.ndarray:
    return _rng(w.seed, stream).integers(0, w.vocab, size=shape, dtype=np.int32)


# --------------------------------------------------------------------------
# verification attention inputs
# --------------------------------------------------------------------------
def attn_inputs(w: Workload, layer: int = 0, ragged: bool = False
                ) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """Q [B,M,Hq,d], K/V caches [B,Hkv,cap,d] with the live P+M rows N(0,1)
    (prefix rows, then the tree tokens' rows at slots P..P+M-1) and the rest
    zero, kv_len [B].  One distinct cache per target layer."""
    rng = _rng(w.seed, 200 + layer)
    cap = w.kv_capacity
    q = _normal(rng, (w.batch, w.tree_size, w.n_q_heads, w.head_dim), 1.0)
    kv_len = np.full((w.batch,), w.prefix, dtype=np.int32)
    if ragged and w.batch > 1:
        lo = max(1, w.prefix // 2)
        kv_len = _rng(w.seed, 299).integers(lo, w.prefix + 1, size=w.batch).astype(np.int32)
        kv_len[0] = w.prefix
    k = np.zeros((w.batch, w.n_kv_heads, cap, w.head_dim), dtype=np.float32)
    v = np.zeros_like(k)
    for b in range(w.batch):
        live = int(kv_len[b]) + w.tree_size
        k[b, :, :live] = _normal(rng, (w.n_kv_heads, live, w.head_dim), 1.0)
        v[b, :, :live] = _normal(rng, (w.n_kv_heads, live, w.head_dim), 1.0)
    return (store_round(q, w.dtype), store_round(k, w.dtype), store_round(v, w.dtype), kv_len)


# --------------------------------------------------------------------------
# target logits with planted agreement, uniforms
# --------------------------------------------------------------------------
def target_logits(w: Workload, tok: np.ndarray, parent: np.ndarray, alpha: float,
                  stream: int = 300, boost: float = 12.0) -> np.ndarray:
    """tl [B, M, V] fp32: N(0,1) rows; at every node that has children, with
    probability alpha one child's token gets +boost (child chosen with weights
    1/2, 1/4, ... over the child order), so that a greedy walk continues with
    probability about alpha per level."""
    B, M = tok.shape
    rng = _rng(w.seed, stream)
    tl = _normal(rng, (B, M, w.vocab), 1.0)
    for b in range(B):
        for i in range(M):
            kids = [c for c in range(M) if parent[b, c] == i]
            if not kids:
                continue
            if rng.random() < alpha:
                wts = np.array([0.5 ** (j + 1) for j in range(len(kids))])
                wts /= wts.sum()
                c = kids[int(rng.choice(len(kids), p=wts))]
                tl[b, i, tok[b, c]] += np.float32(boost)
    return tl


def uniforms(w: Workload, stream: int = 400) -> Tuple[np.ndarray, np.ndarray]:
    """u_accept [B, M] and u_bonus [B, D+1], uniform in [0, 1), fp32."""
    rng = _rng(w.seed, stream)
    ua = rng.random(size=(w.batch, w.tree_size), dtype=np.float32)
    ub = rng.random(size=(w.batch, w.depth + 1), dtype=np.float32)
    return ua, ub
