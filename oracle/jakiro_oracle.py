"""CPU oracle for one Jakiro draft-and-verify step (arXiv 2502.06282).

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain definition that the
CUDA library is checked against.  It is imported by the tests, by the smoke
check and by the benchmark's CPU-baseline leg, never by the product path, and
it shares no code with the CUDA sources.  Everything is NumPy in float64, one
step of the paper after the other, with no blocking, fusion or reordering.

What each function follows:

  rmsnorm               the layer norm that Eq. 1-5 leave out (Sec. 3.1.2, the
                        note after Eq. 5); read as a LLaMA-style pre-MLP
                        RMSNorm in front of router and experts
  router_scores         Eq. 2: softmax over the N expert centroids
  topk_gate             Eq. 5: the K largest scores keep their value, the rest
                        are zero; larger score = "left" (Sec. 3.1.2)
  expert_ffn            Expert_j in Eq. 3, a SiLU-gated FFN without bias
  moe_features          Eq. 3 (combined feature) and the per-branch features
                        f^top1, f^top2 that Eq. 4 and Eq. 6 feed to the head
  head_logits           Eq. 4: the LM head shared with the target model
  branch_topk           per-expert top-k children with cumulative log-prob,
                        the Eagle-style tree growth of Sec. 3.1.2 (last
                        paragraph)
  frontier_select       dynamic-tree frontier (Sec. 3.1.2, last paragraph)
  draft_expand          one draft layer: all of the above for F frontier nodes
  grow_tree             D draft layers in sequence -> candidate pool
  tree_finalize         rerank the pool, keep the best M-1 nodes plus the root
  ancestor_mask         the tree attention mask of Fig. 4
  tree_verify_attn      verification attention (Sec. 2.1 step 2) as plain
                        masked softmax attention
  accept_greedy         strict top-1 verification (Sec. 2.1, Sec. 3.2)
  accept_sampling       min(1, p/q) acceptance with norm(max(0, p-q))
                        resampling (Sec. 2.1 steps 2-3), applied sibling by
                        sibling down the tree
  compact_kv            move the accepted nodes' KV rows behind the prefix
  grow_static_tree      the same draft layers under a predefined (Eagle-1 style)
                        tree shape instead of the score-driven one (Sec. 3.1.2,
                        last paragraph: both policies are usable)
  contrastive_features  Eq. 6-7: f^moe and f^const from the two selected
                        experts' outputs (Sec. 3.2)
  draft_expand_contrastive, grow_tree_hybrid
                        Eq. 8 and the hybrid schedule of Sec. 3.2: autoregressive
                        passes from logits^moe, and logits^const of the last pass
                        proposing one token further, so that a tree of depth D
                        costs D-1 draft passes
  verify_qkv_append, gather_accepted
                        the target layer's own steps around tree attention in a
                        verification pass (Sec. 2.1 step 2): QKV projection of
                        the tree tokens, rotary positions by depth, K/V written
                        at the tree slots; and the accepted nodes' hidden states
                        picked out for the next draft round
  rope, draft_pre_block Eq. 1 and the Eagle-style input path described before
                        it (Sec. 3.1.2): token embedding and the parent's
                        feature concatenated, the reduction layer, then
                        u = Attn(h) + h with the draft layer's own KV cache

Parity status: every function is pinned by tests/test_oracle_*.py to closed
forms, brute force or invariants, with two exceptions that stay
"parity unpinned": (1) the choice b_r = g_r * Expert_{j_r}(x) + u for the
branch feature (the printed Eq. 4 is ambiguous; only b_1 + b_2 - u = f ties it
to Eq. 3), and (2) exact losslessness of accept_sampling when the children
are deterministic top-k tokens rather than samples from q (pinned only in the
sampled-children mode).  Readings the paper leaves open in the later functions
(where the proposals of logits^const hang in the tree, no normalisation and
LLaMA-style rotary positions in the draft attention) are stated at the
functions; their arithmetic is pinned, the readings themselves cannot be.
"""
from __future__ import annotations

from typing import Dict, List, Optional, Sequence, Tuple

import numpy as np

F64 = np.float64


# --------------------------------------------------------------------------
# small pieces
# --------------------------------------------------------------------------
def softmax(z: np.ndarray, axis: int = -1) -> np.ndarray:
    z = np.asarray(z, dtype=F64)
    m = np.max(z, axis=axis, keepdims=True)
    e = np.exp(z - m)
    return e / np.sum(e, axis=axis, keepdims=True)


def logsumexp(z: np.ndarray, axis: int = -1) -> np.ndarray:
    z = np.asarray(z, dtype=F64)
    m = np.max(z, axis=axis, keepdims=True)
    return (m + np.log(np.sum(np.exp(z - m), axis=axis, keepdims=True))).squeeze(axis)


def silu(a: np.ndarray) -> np.ndarray:
    a = np.asarray(a, dtype=F64)
    return a / (1.0 + np.exp(-a))


def rmsnorm(u: np.ndarray, weight: Optional[np.ndarray], eps: float) -> np.ndarray:
    """x = u / sqrt(mean(u^2) + eps) * weight over the last axis."""
    u = np.asarray(u, dtype=F64)
    ms = np.mean(u * u, axis=-1, keepdims=True)
    x = u / np.sqrt(ms + eps)
    if weight is not None:
        x = x * np.asarray(weight, dtype=F64)
    return x


def order_desc(values: np.ndarray) -> np.ndarray:
    """Indices sorted by value descending, ties by lower index first."""
    values = np.asarray(values)
    idx = np.arange(values.shape[0])
    return np.lexsort((idx, -values))


# --------------------------------------------------------------------------
# draft layer (Eq. 2-5)
# --------------------------------------------------------------------------
def router_scores(x: np.ndarray, centroids: np.ndarray) -> np.ndarray:
    """Eq. 2: s[., j] = softmax_j(x . e_j).  x [..., H], centroids [N, H]."""
    z = np.asarray(x, dtype=F64) @ np.asarray(centroids, dtype=F64).T
    return softmax(z, axis=-1)


def topk_gate(s_row: np.ndarray, k: int) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 5 for one node: ids of the K largest scores (largest first = left
    branch, ties to the lower expert id) and their gate values, which are the
    scores themselves, not renormalised."""
    ids = order_desc(np.asarray(s_row))[:k]
    return ids.astype(np.int32), np.asarray(s_row, dtype=F64)[ids]


def expert_ffn(x: np.ndarray, w_gate: np.ndarray, w_up: np.ndarray, w_down: np.ndarray
               ) -> np.ndarray:
    """Expert_j(x) = W_down ( SiLU(W_gate x) * (W_up x) ); x [H], W_gate/W_up
    [I, H], W_down [H, I]."""
    x = np.asarray(x, dtype=F64)
    g = np.asarray(w_gate, dtype=F64) @ x
    a = np.asarray(w_up, dtype=F64) @ x
    h = silu(g) * a
    return np.asarray(w_down, dtype=F64) @ h


def moe_features(u_row: np.ndarray, x_row: np.ndarray, ids: np.ndarray, gates: np.ndarray,
                 weights: Dict[str, np.ndarray], branch_residual: bool = True
                 ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """For one node: y [K, H] expert outputs, b [K, H] branch features,
    f [H] combined feature.  f = sum_r g_r y_r + u is Eq. 3; branch r carries
    only its own expert, weighted by its score (g_r y_r), plus the residual u
    when branch_residual is set."""
    u_row = np.asarray(u_row, dtype=F64)
    K = len(ids)
    y = np.zeros((K, u_row.shape[0]), dtype=F64)
    for r in range(K):
        j = int(ids[r])
        y[r] = expert_ffn(x_row, weights["w_gate"][j], weights["w_up"][j], weights["w_down"][j])
    f = u_row.copy()
    for r in range(K):
        f = f + gates[r] * y[r]
    b = np.zeros_like(y)
    for r in range(K):
        b[r] = gates[r] * y[r]
        if branch_residual:
            b[r] = b[r] + u_row
    return y, b, f


def head_logits(b: np.ndarray, lm_head: np.ndarray) -> np.ndarray:
    """Eq. 4: logits = b . W_head^T; b [..., H], lm_head [V, H]."""
    return np.asarray(b, dtype=F64) @ np.asarray(lm_head, dtype=F64).T


def branch_topk(logits_row: np.ndarray, k_e: int, parent_score: float
                ) -> Tuple[np.ndarray, np.ndarray, float]:
    """One (node, branch): the k_e tokens with the largest logits (ties to the
    lower token id), their cumulative scores parent_score + log-softmax, and
    the row's log-sum-exp."""
    logits_row = np.asarray(logits_row, dtype=F64)
    ids = order_desc(logits_row)[:k_e]
    lse = float(logsumexp(logits_row))
    score = parent_score + (logits_row[ids] - lse)
    return ids.astype(np.int32), score, lse


def frontier_select(scores_flat: np.ndarray, width: int) -> np.ndarray:
    """Flat candidate indices of the `width` best candidates of one layer by
    (score descending, index ascending)."""
    return order_desc(np.asarray(scores_flat))[:width].astype(np.int32)


def draft_expand(u: np.ndarray, parent_score: np.ndarray, weights: Dict[str, np.ndarray],
                 k_e: int, width: int, top_k: int = 2, rms_eps: float = 1e-5,
                 use_pre_norm: bool = True, branch_residual: bool = True
                 ) -> Dict[str, np.ndarray]:
    """One draft layer for u [B, F, H] (outputs of Eq. 1) and the frontier
    nodes' cumulative scores [B, F].  Children of node f are ordered left
    branch ranks 0..k_e-1, then right branch ranks 0..k_e-1."""
    u = np.asarray(u, dtype=F64)
    B, F, H = u.shape
    N = weights["router"].shape[0]
    V = weights["lm_head"].shape[0]
    K = top_k
    x = rmsnorm(u, weights.get("norm_weight"), rms_eps) if use_pre_norm else u.copy()
    probs = router_scores(x, weights["router"])                     # [B, F, N]
    expert = np.zeros((B, F, K), dtype=np.int32)
    gate = np.zeros((B, F, K), dtype=F64)
    feat = np.zeros((B, F, H), dtype=F64)
    branch = np.zeros((B, F, K, H), dtype=F64)
    logits = np.zeros((B, F, K, V), dtype=F64)
    tok = np.zeros((B, F, K, k_e), dtype=np.int32)
    score = np.zeros((B, F, K, k_e), dtype=F64)
    lse = np.zeros((B, F, K), dtype=F64)
    for b in range(B):
        for f in range(F):
            ids, g = topk_gate(probs[b, f], K)
            expert[b, f], gate[b, f] = ids, g
            _, br, ff = moe_features(u[b, f], x[b, f], ids, g, weights, branch_residual)
            branch[b, f], feat[b, f] = br, ff
            logits[b, f] = head_logits(br, weights["lm_head"])
            for r in range(K):
                tok[b, f, r], score[b, f, r], lse[b, f, r] = branch_topk(
                    logits[b, f, r], k_e, float(parent_score[b, f]))
    n_cand = F * K * k_e
    wsel = min(width, n_cand)
    frontier = np.zeros((B, wsel), dtype=np.int32)
    for b in range(B):
        frontier[b] = frontier_select(score[b].reshape(-1), wsel)
    return {"probs": probs, "expert": expert, "gate": gate, "feat": feat, "branch": branch,
            "logits": logits, "tok": tok, "score": score, "lse": lse, "frontier": frontier,
            "x": x}


def grow_tree(u_layers: Sequence[np.ndarray], weights: Dict[str, np.ndarray], k_e: int,
              width: int, top_k: int = 2, **kw) -> Dict[str, np.ndarray]:
    """D draft layers.  u_layers[l] is [B, F_l, H] with F_1 = 1 (the root) and
    row f of layer l+1 belonging to the f-th node chosen by frontier_select in
    layer l.  Every candidate gets a generation index (gidx) in the order
    (layer, frontier slot, branch, rank).  Returns the candidate pool:
    tok/score [B, n], parent [B, n] (gidx of the parent, -1 = root), qslot
    [B, n] (row of `logits` holding the node's own draft distributions if the
    node was expanded, else -1) and logits [B, S, K, V], S = sum F_l, with the
    root in slot 0."""
    B = u_layers[0].shape[0]
    pool_tok: List[np.ndarray] = []
    pool_score: List[np.ndarray] = []
    pool_parent: List[np.ndarray] = []
    pool_qslot: List[np.ndarray] = []
    all_logits: List[np.ndarray] = []
    layers = []
    parent_score = np.zeros((B, 1), dtype=F64)
    parent_gidx = np.full((B, 1), -1, dtype=np.int32)
    gidx_base = 0
    slot_base = 0
    for u in u_layers:
        F = u.shape[1]
        assert F == parent_score.shape[1], "frontier size mismatch"
        out = draft_expand(u, parent_score, weights, k_e, width, top_k, **kw)
        layers.append(out)
        n_cand = F * top_k * k_e
        pool_tok.append(out["tok"].reshape(B, n_cand))
        pool_score.append(out["score"].reshape(B, n_cand))
        pool_parent.append(np.repeat(parent_gidx, top_k * k_e, axis=1))
        q = np.full((B, n_cand), -1, dtype=np.int32)
        wsel = out["frontier"].shape[1]
        for b in range(B):
            q[b, out["frontier"][b]] = slot_base + F + np.arange(wsel)
        pool_qslot.append(q)
        all_logits.append(out["logits"])
        parent_score = np.take_along_axis(out["score"].reshape(B, n_cand), out["frontier"], 1)
        parent_gidx = (gidx_base + out["frontier"]).astype(np.int32)
        gidx_base += n_cand
        slot_base += F
    # the last layer's frontier is never expanded: its qslot entries point
    # past the stored rows, so clear them
    pool_qslot[-1][:] = -1
    return {"tok": np.concatenate(pool_tok, 1), "score": np.concatenate(pool_score, 1),
            "parent": np.concatenate(pool_parent, 1), "qslot": np.concatenate(pool_qslot, 1),
            "logits": np.concatenate(all_logits, 1), "layers": layers}


def _tree_finalize(pool_tok, pool_score, pool_parent, pool_qslot, pool_branch, root_tok,
                   tree_size):
    n = len(pool_tok)
    m1 = tree_size - 1
    if n < m1:
        raise ValueError("candidate pool smaller than the requested tree")
    keep = np.sort(order_desc(np.asarray(pool_score))[:m1])      # ascending gidx
    new_id = {int(g): i + 1 for i, g in enumerate(keep)}
    tok = np.zeros(tree_size, dtype=np.int32)
    parent = np.full(tree_size, -1, dtype=np.int32)
    depth = np.zeros(tree_size, dtype=np.int32)
    branch = np.zeros(tree_size, dtype=np.int32)
    qslot = np.full(tree_size, -1, dtype=np.int32)
    score = np.zeros(tree_size, dtype=F64)
    tok[0] = root_tok
    qslot[0] = 0
    for i, g in enumerate(keep, start=1):
        g = int(g)
        pg = int(pool_parent[g])
        if pg >= 0 and pg not in new_id:
            raise ValueError("kept node whose parent was dropped")
        parent[i] = 0 if pg < 0 else new_id[pg]
        depth[i] = depth[parent[i]] + 1
        tok[i] = pool_tok[g]
        branch[i] = pool_branch[g]
        qslot[i] = pool_qslot[g]
        score[i] = pool_score[g]
    return {"tok": tok, "parent": parent, "depth": depth, "branch": branch, "qslot": qslot,
            "score": score, "keep": keep.astype(np.int32)}


def pool_branches(frontier_sizes: Sequence[int], top_k: int, k_e: int) -> np.ndarray:
    """Branch (0 = left, 1 = right, ...) of every pool entry in gidx order."""
    out = []
    for F in frontier_sizes:
        out.append(np.tile(np.repeat(np.arange(top_k), k_e), F))
    return np.concatenate(out).astype(np.int32)


def tree_finalize(pool_tok, pool_score, pool_parent, pool_qslot, root_tok, tree_size,
                  frontier_sizes=None, top_k=2, k_e=1, pool_branch=None):
    """One sequence.  Keep the tree_size-1 best candidates of the pool by
    (score descending, gidx ascending), list them in ascending gidx behind the
    root (node 0) and rename the parents, so that parent[i] < i and depth is
    non-decreasing.  Because log-probabilities are <= 0 a child never scores
    above its parent, and the gidx tie-break keeps a parent ahead of its
    children, so the kept set is closed under taking ancestors."""
    if pool_branch is None:
        pool_branch = pool_branches(frontier_sizes, top_k, k_e)
    return _tree_finalize(np.asarray(pool_tok), np.asarray(pool_score), np.asarray(pool_parent),
                          np.asarray(pool_qslot), np.asarray(pool_branch), root_tok, tree_size)


# --------------------------------------------------------------------------
# verification attention (Fig. 4, Sec. 2.1 step 2)
# --------------------------------------------------------------------------
def ancestor_mask(parent: np.ndarray) -> np.ndarray:
    """anc[i, t] = True iff t is i or an ancestor of i (Fig. 4)."""
    m = len(parent)
    anc = np.zeros((m, m), dtype=bool)
    for i in range(m):
        t = i
        while t >= 0:
            anc[i, t] = True
            t = int(parent[t])
    return anc


def tree_verify_attn(q: np.ndarray, k_cache: np.ndarray, v_cache: np.ndarray,
                     kv_len: np.ndarray, parent: np.ndarray, scale: float) -> np.ndarray:
    """out[b, i, h] = sum_c softmax_c(scale * q[b,i,h] . K[b,h//G,c] + mask) V[b,h//G,c]
    over cache columns c < P_b + M, where column c is visible to tree node i
    iff c < P_b (committed prefix) or c - P_b is i itself or one of its
    ancestors.  q [B, M, Hq, d]; caches [B, Hkv, cap, d] with the tree tokens'
    rows at P_b .. P_b+M-1; parent [B, M]."""
    q = np.asarray(q, dtype=F64)
    B, M, Hq, d = q.shape
    Hkv = k_cache.shape[1]
    G = Hq // Hkv
    out = np.zeros((B, M, Hq, d), dtype=F64)
    for b in range(B):
        P = int(kv_len[b])
        anc = ancestor_mask(parent[b])
        visible = np.concatenate([np.ones((M, P), dtype=bool), anc], axis=1)   # [M, P+M]
        for h in range(Hq):
            kh = np.asarray(k_cache[b, h // G, :P + M], dtype=F64)
            vh = np.asarray(v_cache[b, h // G, :P + M], dtype=F64)
            s = scale * (q[b, :, h, :] @ kh.T)                                 # [M, P+M]
            s = np.where(visible, s, -np.inf)
            out[b, :, h, :] = softmax(s, axis=-1) @ vh
    return out


# --------------------------------------------------------------------------
# acceptance (Sec. 2.1 steps 2-3)
# --------------------------------------------------------------------------
def children_of(parent: np.ndarray, i: int) -> List[int]:
    return [c for c in range(len(parent)) if parent[c] == i]


def argmax_low(row: np.ndarray) -> int:
    """argmax with ties to the lowest index."""
    return int(np.argmax(np.asarray(row)))


def accept_greedy(target_logits: np.ndarray, tok: np.ndarray, parent: np.ndarray
                  ) -> Tuple[List[int], List[int], int]:
    """One sequence, temperature 0.  Walk from the root: the target's top-1
    token at the current node must equal a child's token (first such child in
    child order); stop when none does.  Returns (accepted node indices,
    accepted tokens, bonus token = the target's top-1 at the stop node)."""
    cur = 0
    path: List[int] = []
    toks: List[int] = []
    while True:
        t_star = argmax_low(target_logits[cur])
        nxt = -1
        for c in children_of(parent, cur):
            if int(tok[c]) == t_star:
                nxt = c
                break
        if nxt < 0:
            return path, toks, t_star
        path.append(nxt)
        toks.append(int(tok[nxt]))
        cur = nxt


def inverse_cdf(p: np.ndarray, u: float) -> int:
    """Smallest v with cumsum(p)[v] > u * sum(p); the last index with p > 0
    if rounding leaves none."""
    p = np.asarray(p, dtype=F64)
    c = np.cumsum(p)
    hit = np.nonzero(c > u * c[-1])[0]
    if len(hit):
        return int(hit[0])
    return int(np.nonzero(p > 0)[0][-1])


def accept_sampling(target_logits: np.ndarray, tok: np.ndarray, parent: np.ndarray,
                    depth: np.ndarray, branch: np.ndarray, qslot: np.ndarray,
                    draft_logits: np.ndarray, u_accept: np.ndarray, u_bonus: np.ndarray,
                    temperature: float, trace: Optional[list] = None
                    ) -> Tuple[List[int], List[int], int]:
    """One sequence, temperature > 0.  At the current node p = softmax(tl/T)
    and each branch r has its own draft distribution q_r = softmax(draft
    logits / T).  The children are tried in child order: child c with token x
    from branch r is accepted iff u_accept[c] < min(1, p[x]/q_r[x]) (Sec. 2.1
    step 2).  On rejection p <- norm(max(0, p - q_r)) (step 3) and x is
    removed from q_r, which is renormalised for later siblings of the same
    branch.  When no child is accepted (or the node has none) the bonus token
    is drawn from the current p by inverse CDF with u_bonus[depth]."""
    T = float(temperature)
    cur = 0
    path: List[int] = []
    toks: List[int] = []
    while True:
        p = softmax(np.asarray(target_logits[cur], dtype=F64) / T)
        p_orig = p
        kids = children_of(parent, cur)
        nxt = -1
        if kids and qslot[cur] >= 0:
            K = draft_logits.shape[1]
            qd = [softmax(np.asarray(draft_logits[qslot[cur], r], dtype=F64) / T)
                  for r in range(K)]
            for c in kids:
                x = int(tok[c])
                q = qd[int(branch[c])]
                if q[x] > 0.0:
                    ratio = min(1.0, p[x] / q[x])
                    acc = float(u_accept[c]) < ratio
                else:
                    ratio = 1.0 if p[x] > 0.0 else 0.0
                    acc = p[x] > 0.0
                if trace is not None:
                    trace.append({"node": cur, "child": c, "tok": x, "p": float(p[x]),
                                  "q": float(q[x]), "ratio": ratio, "accepted": bool(acc)})
                if acc:
                    nxt = c
                    break
                resid = np.maximum(0.0, p - q)
                tot = resid.sum()
                if not tot > 0.0:
                    p = p_orig          # residual vanished: fall back to the node's p
                    break
                p = resid / tot
                q = q.copy()
                q[x] = 0.0
                qs = q.sum()
                if qs > 0.0:
                    q = q / qs
                qd[int(branch[c])] = q
        if nxt < 0:
            bonus = inverse_cdf(p, float(u_bonus[int(depth[cur])]))
            if trace is not None:
                trace.append({"node": cur, "bonus": bonus})
            return path, toks, bonus
        path.append(nxt)
        toks.append(int(tok[nxt]))
        cur = nxt


# --------------------------------------------------------------------------
# KV compaction
# --------------------------------------------------------------------------
def compact_kv(cache: np.ndarray, prefix_len: int, acc_idx: Sequence[int]) -> np.ndarray:
    """cache [Hkv, cap, d] of one sequence and layer.  The root's row stays at
    slot P; accepted node acc_idx[j] moves from slot P + acc_idx[j] to slot
    P + 1 + j.  Done out of place on a copy.  New length P + 1 + len(acc_idx)."""
    out = np.array(cache, copy=True)
    for j, a in enumerate(acc_idx):
        out[:, prefix_len + 1 + j, :] = cache[:, prefix_len + int(a), :]
    return out


# --------------------------------------------------------------------------
# static tree policy (Sec. 3.1.2, last paragraph)
# --------------------------------------------------------------------------
def grow_static_tree(u_of_path, weights: Dict[str, np.ndarray], paths: Sequence[Tuple[int, ...]],
                     k_e: int, root_tok: int, top_k: int = 2, **kw) -> Dict[str, np.ndarray]:
    """One sequence under a predefined tree shape.  `paths` lists the tree's
    nodes below the root as tuples of child ranks: rank c of a node is its
    c-th candidate in child order (left branch ranks 0..k_e-1, then the right
    branch), so (0,) is the root's best left-branch child and (k_e, 0) the best
    left-branch child of the root's best right-branch child.  Every prefix of
    a listed path must be listed.  A node is expanded iff it has listed
    children; which tokens fill the shape depends on the draft, the shape
    itself never does.  `u_of_path(path)` returns the hidden state u [H] of the
    node at `path` (() = root).  Nodes are numbered root first, then by
    (depth, path) ascending, which keeps parent[i] < i, depth non-decreasing
    and every node's children contiguous in child order.  Returns tok, parent,
    depth, branch, score per node and the logits [K, V] of every expanded
    node (dict keyed by path)."""
    paths = sorted(set(tuple(p) for p in paths), key=lambda p: (len(p), p))
    listed = set(paths)
    for p in paths:
        if len(p) > 1 and p[:-1] not in listed:
            raise ValueError("a listed node whose parent is not listed")
        if not 0 <= p[-1] < top_k * k_e:
            raise ValueError("child rank outside the candidate list")
    order = [()] + paths
    index = {p: i for i, p in enumerate(order)}
    n = len(order)
    tok = np.zeros(n, dtype=np.int32)
    parent = np.full(n, -1, dtype=np.int32)
    depth = np.zeros(n, dtype=np.int32)
    branch = np.zeros(n, dtype=np.int32)
    score = np.zeros(n, dtype=F64)
    tok[0] = root_tok
    logits_of = {}
    expanded = [p for p in order if any(q[:-1] == p for q in paths)]
    for p in expanded:
        u = np.asarray(u_of_path(p), dtype=F64)[None, None, :]
        out = draft_expand(u, np.array([[score[index[p]]]]), weights, k_e, 1, top_k, **kw)
        logits_of[p] = out["logits"][0, 0]
        cand_tok = out["tok"][0, 0].reshape(-1)          # child order: branch, then rank
        cand_score = out["score"][0, 0].reshape(-1)
        for q in paths:
            if q[:-1] == p:
                i = index[q]
                tok[i] = cand_tok[q[-1]]
                score[i] = cand_score[q[-1]]
                parent[i] = index[p]
                depth[i] = len(q)
                branch[i] = q[-1] // k_e
    return {"tok": tok, "parent": parent, "depth": depth, "branch": branch, "score": score,
            "logits": logits_of, "order": order}


# --------------------------------------------------------------------------
# contrastive head and hybrid parallel decoding (Sec. 3.2, Eq. 6-8)
# --------------------------------------------------------------------------
def contrastive_features(y: np.ndarray, gates: np.ndarray, alpha: float, beta: float
                         ) -> Tuple[np.ndarray, np.ndarray]:
    """Eq. 6-7 for one node.  y [2, H] are the outputs f^top1, f^top2 of the
    two selected experts (larger score first), gates their scores:
    f^moe = s^top1 f^top1 + s^top2 f^top2, f^const = beta f^top1 - alpha f^top2."""
    y = np.asarray(y, dtype=F64)
    f_moe = gates[0] * y[0] + gates[1] * y[1]
    f_const = beta * y[0] - alpha * y[1]
    return f_moe, f_const


def draft_expand_contrastive(u: np.ndarray, parent_score: np.ndarray,
                             weights: Dict[str, np.ndarray], k_e: int, width: int, alpha: float,
                             beta: float, last_pass: bool, rms_eps: float = 1e-5,
                             use_pre_norm: bool = True, branch_residual: bool = True
                             ) -> Dict[str, np.ndarray]:
    """One draft pass in the contrastive mode (Eq. 6-8) for u [B, F, H].  Row 0
    of a node's logits is Head(f^moe), row 1 is Head(f^const); with
    branch_residual the residual u is added to both head inputs, as it is in
    Eq. 3 (then row 0 is the head of the combined feature f of Eq. 3 itself).
    Children: the k_e best tokens of row 0 are the node's children, scored as
    in branch_topk.  Row 1 predicts the token after the next one (the
    parallel-decoding head of Sec. 3.2): its k_e best tokens hang under the
    node's best row-0 child, with score = that child's score + their
    log-probability under row 1.  They count only in the last pass of a step
    (score -inf otherwise) and are never expanded.  Reading: the paper does not
    say under which child the row-1 proposals hang; the best one is the choice
    that keeps the candidate count of a pass unchanged."""
    u = np.asarray(u, dtype=F64)
    B, F, H = u.shape
    V = weights["lm_head"].shape[0]
    x = rmsnorm(u, weights.get("norm_weight"), rms_eps) if use_pre_norm else u.copy()
    probs = router_scores(x, weights["router"])
    expert = np.zeros((B, F, 2), dtype=np.int32)
    gate = np.zeros((B, F, 2), dtype=F64)
    feat = np.zeros((B, F, H), dtype=F64)
    logits = np.zeros((B, F, 2, V), dtype=F64)
    tok = np.zeros((B, F, 2, k_e), dtype=np.int32)
    score = np.zeros((B, F, 2, k_e), dtype=F64)
    lse = np.zeros((B, F, 2), dtype=F64)
    for b in range(B):
        for f in range(F):
            ids, g = topk_gate(probs[b, f], 2)
            expert[b, f], gate[b, f] = ids, g
            y, _, ff = moe_features(u[b, f], x[b, f], ids, g, weights, True)
            feat[b, f] = ff                                   # Eq. 3, fed to the next pass
            f_moe, f_const = contrastive_features(y, g, alpha, beta)
            if branch_residual:
                f_moe, f_const = f_moe + u[b, f], f_const + u[b, f]
            logits[b, f] = head_logits(np.stack([f_moe, f_const]), weights["lm_head"])
            tok[b, f, 0], score[b, f, 0], lse[b, f, 0] = branch_topk(
                logits[b, f, 0], k_e, float(parent_score[b, f]))
            tok[b, f, 1], score[b, f, 1], lse[b, f, 1] = branch_topk(
                logits[b, f, 1], k_e, float(score[b, f, 0, 0]))
            if not last_pass:
                score[b, f, 1, :] = -np.inf
    n_cand = F * 2 * k_e
    wsel = min(width, F * k_e)
    frontier = np.zeros((B, wsel), dtype=np.int32)
    for b in range(B):
        # only row-0 children can be expanded: the others are masked out of the selection
        sc = score[b].copy()
        sc[:, 1, :] = -np.inf
        frontier[b] = frontier_select(sc.reshape(-1), wsel)
    return {"probs": probs, "expert": expert, "gate": gate, "feat": feat, "logits": logits,
            "tok": tok, "score": score, "lse": lse, "frontier": frontier, "n_cand": n_cand}


def grow_tree_hybrid(u_layers: Sequence[np.ndarray], weights: Dict[str, np.ndarray], k_e: int,
                     width: int, alpha: float, beta: float, **kw) -> Dict[str, np.ndarray]:
    """The hybrid schedule of Sec. 3.2: len(u_layers) = D-1 contrastive passes
    build a tree of depth up to D, because the last pass's row-1 proposals sit
    one level below its row-0 children.  Pool layout as in grow_tree; the
    parent of a row-1 candidate is the generation index of its node's best
    row-0 child."""
    B = u_layers[0].shape[0]
    tok_l, score_l, parent_l, qslot_l, branch_l, logits_l = [], [], [], [], [], []
    parent_score = np.zeros((B, 1), dtype=F64)
    parent_gidx = np.full((B, 1), -1, dtype=np.int32)
    gidx_base, slot_base = 0, 0
    for l, u in enumerate(u_layers):
        F = u.shape[1]
        last = l == len(u_layers) - 1
        out = draft_expand_contrastive(u, parent_score, weights, k_e, width, alpha, beta, last, **kw)
        n_cand = F * 2 * k_e
        par = np.zeros((B, F, 2, k_e), dtype=np.int32)
        for f in range(F):
            par[:, f, 0, :] = parent_gidx[:, f:f + 1]
            par[:, f, 1, :] = gidx_base + (f * 2 + 0) * k_e + 0
        q = np.full((B, n_cand), -1, dtype=np.int32)
        if not last:
            for b in range(B):
                q[b, out["frontier"][b]] = slot_base + F + np.arange(out["frontier"].shape[1])
        tok_l.append(out["tok"].reshape(B, n_cand))
        score_l.append(out["score"].reshape(B, n_cand))
        parent_l.append(par.reshape(B, n_cand))
        qslot_l.append(q)
        branch_l.append(np.tile(np.repeat(np.arange(2), k_e), F)[None].repeat(B, 0))
        logits_l.append(out["logits"])
        parent_score = np.take_along_axis(out["score"].reshape(B, n_cand), out["frontier"], 1)
        parent_gidx = (gidx_base + out["frontier"]).astype(np.int32)
        gidx_base += n_cand
        slot_base += F
    return {"tok": np.concatenate(tok_l, 1), "score": np.concatenate(score_l, 1),
            "parent": np.concatenate(parent_l, 1), "qslot": np.concatenate(qslot_l, 1),
            "branch": np.concatenate(branch_l, 1).astype(np.int32),
            "logits": np.concatenate(logits_l, 1)}


# --------------------------------------------------------------------------
# draft pre-MoE block (Eq. 1 and the paragraph before it)
# --------------------------------------------------------------------------
def rope(x: np.ndarray, pos: float, theta: float) -> np.ndarray:
    """Rotary position embedding of one head vector x [d] at position `pos`,
    LLaMA convention: the vector is split in halves (x1, x2), pair i is
    (x1[i], x2[i]) and rotates by pos / theta^(2 i / d)."""
    x = np.asarray(x, dtype=F64)
    d = x.shape[-1]
    half = d // 2
    ang = pos / theta ** (2.0 * np.arange(half) / d)
    c, s_ = np.cos(ang), np.sin(ang)
    x1, x2 = x[:half], x[half:]
    return np.concatenate([x1 * c - x2 * s_, x2 * c + x1 * s_])


def draft_pre_block(tok: np.ndarray, f_prev: np.ndarray, pw: Dict[str, np.ndarray],
                    k_cache: np.ndarray, v_cache: np.ndarray, prefix_len: int,
                    slots: Sequence[int], slot_parent: np.ndarray, n_q_heads: int,
                    n_kv_heads: int, theta: float, scale: float
                    ) -> Tuple[np.ndarray, np.ndarray, np.ndarray, np.ndarray]:
    """Eq. 1 for the F nodes of one draft layer of one sequence.
    tok [F]: the nodes' tokens; f_prev [F, H]: each node's parent feature (the
    f of Eq. 3 the parent's pass produced; for the root the target model's
    last feature).  pw: emb [V, H], w_fc [H, 2H], b_fc [H] or None, w_q
    [Hq d, H], w_k, w_v [Hkv d, H], w_o [H, Hq d].
      h = W_fc [emb(tok) ; f_prev] (+ b_fc)          (the reduction layer)
      q, k, v = W_q h, W_k h, W_v h per head, q and k rotated to position
      prefix_len + depth of the node; k, v are stored in the draft layer's own
      cache [Hkv, cap, d] at row prefix_len + slot (slots = the nodes' rows
      among the step's expanded nodes, root = 0);
      Attn: every node attends over the committed prefix rows and the rows of
      itself and its ancestors (slot_parent [S], -1 for the root);
      u = W_o Attn + h.
    No normalisation is applied (Eagle-style drafts drop the input norm of
    their single layer; the note after Eq. 5 leaves norms out).  Returns
    (u [F, H], h [F, H], and the updated caches)."""
    emb = np.asarray(pw["emb"], dtype=F64)
    F = len(tok)
    H = emb.shape[1]
    d = pw["w_q"].shape[0] // n_q_heads
    G = n_q_heads // n_kv_heads
    kc = np.array(k_cache, dtype=F64, copy=True)
    vc = np.array(v_cache, dtype=F64, copy=True)
    depth = np.zeros(len(slot_parent), dtype=np.int64)
    for s_ in range(1, len(slot_parent)):
        if slot_parent[s_] >= 0:
            depth[s_] = depth[slot_parent[s_]] + 1
    h = np.zeros((F, H), dtype=F64)
    qs = np.zeros((F, n_q_heads, d), dtype=F64)
    for i in range(F):
        x = np.concatenate([emb[int(tok[i])], np.asarray(f_prev[i], dtype=F64)])
        h[i] = np.asarray(pw["w_fc"], dtype=F64) @ x
        if pw.get("b_fc") is not None:
            h[i] = h[i] + np.asarray(pw["b_fc"], dtype=F64)
        pos = prefix_len + int(depth[slots[i]])
        q = (np.asarray(pw["w_q"], dtype=F64) @ h[i]).reshape(n_q_heads, d)
        k = (np.asarray(pw["w_k"], dtype=F64) @ h[i]).reshape(n_kv_heads, d)
        v = (np.asarray(pw["w_v"], dtype=F64) @ h[i]).reshape(n_kv_heads, d)
        for hh in range(n_q_heads):
            qs[i, hh] = rope(q[hh], pos, theta)
        for hh in range(n_kv_heads):
            kc[hh, prefix_len + slots[i]] = rope(k[hh], pos, theta)
            vc[hh, prefix_len + slots[i]] = v[hh]
    u = np.zeros((F, H), dtype=F64)
    for i in range(F):
        anc = []
        t = int(slots[i])
        while t >= 0:
            anc.append(t)
            t = int(slot_parent[t])
        cols = list(range(prefix_len)) + [prefix_len + a for a in sorted(anc)]
        o = np.zeros((n_q_heads, d), dtype=F64)
        for hh in range(n_q_heads):
            kk, vv = kc[hh // G, cols], vc[hh // G, cols]
            o[hh] = softmax(scale * (kk @ qs[i, hh])) @ vv
        u[i] = np.asarray(pw["w_o"], dtype=F64) @ o.reshape(-1) + h[i]
    return u, h, kc, vc


# --------------------------------------------------------------------------
# verification-side glue around the tree attention (Sec. 2.1 step 2)
# --------------------------------------------------------------------------
def verify_qkv_append(x: np.ndarray, w_q: np.ndarray, w_k: np.ndarray, w_v: np.ndarray,
                      depth: np.ndarray, k_cache: np.ndarray, v_cache: np.ndarray,
                      prefix_len: int, n_q_heads: int, n_kv_heads: int, theta: float
                      ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """One sequence, one target layer.  x [M, H] are the layer's input hidden
    states of the M tree tokens.  q_i = rope(W_q x_i), k_i = rope(W_k x_i),
    v_i = W_v x_i per head, rotated to position prefix_len + depth[i] (all
    nodes of one depth share a position: they are alternatives for the same
    place in the sequence); k_i, v_i go to cache row prefix_len + i, which is
    where jk_tree_verify_attn expects the tree tokens.  Returns (q [M, Hq, d],
    caches)."""
    x = np.asarray(x, dtype=F64)
    M = x.shape[0]
    d = w_q.shape[0] // n_q_heads
    kc = np.array(k_cache, dtype=F64, copy=True)
    vc = np.array(v_cache, dtype=F64, copy=True)
    q_out = np.zeros((M, n_q_heads, d), dtype=F64)
    for i in range(M):
        pos = prefix_len + int(depth[i])
        q = (np.asarray(w_q, dtype=F64) @ x[i]).reshape(n_q_heads, d)
        k = (np.asarray(w_k, dtype=F64) @ x[i]).reshape(n_kv_heads, d)
        v = (np.asarray(w_v, dtype=F64) @ x[i]).reshape(n_kv_heads, d)
        for hh in range(n_q_heads):
            q_out[i, hh] = rope(q[hh], pos, theta)
        for hh in range(n_kv_heads):
            kc[hh, prefix_len + i] = rope(k[hh], pos, theta)
            vc[hh, prefix_len + i] = v[hh]
    return q_out, kc, vc


def gather_accepted(hidden: np.ndarray, acc_idx: Sequence[int], rows: int) -> np.ndarray:
    """hidden [M, H] of one sequence's tree tokens -> [rows, H]: row 0 is the
    root's (always committed), row 1 + j the j-th accepted node's; rows past
    the accepted path are zero.  These are the features the next draft round
    starts from."""
    hidden = np.asarray(hidden)
    out = np.zeros((rows, hidden.shape[1]), dtype=hidden.dtype)
    out[0] = hidden[0]
    for j, a in enumerate(acc_idx):
        out[1 + j] = hidden[int(a)]
    return out
