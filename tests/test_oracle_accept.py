"""Pins for the oracle's acceptance walk and KV compaction (Sec. 2.1 steps 2-3)."""
import itertools
import math

import numpy as np
import pytest

from oracle import jakiro_oracle as orc
from paper_2502_06282_b200 import synth


# ----------------------------------------------------------------- greedy
def _all_parent_arrays(m):
    """Every tree on m nodes with parent[i] < i."""
    for tail in itertools.product(*[range(i) for i in range(1, m)]):
        yield np.array((-1,) + tail, dtype=np.int32)


def _valid_paths(tl_top1, tok, parent):
    """All root-to-node paths along which each token equals the top-1 of the node before."""
    m = len(tok)
    out = [[]]
    stack = [(0, [])]
    while stack:
        cur, path = stack.pop()
        for c in range(m):
            if parent[c] == cur and tok[c] == tl_top1[cur]:
                out.append(path + [c])
                stack.append((c, path + [c]))
    return out


def test_greedy_exhaustive_small_trees():
    V = 3
    checked = 0
    rng = np.random.default_rng(0)
    for m in range(1, 6):
        for parent in _all_parent_arrays(m):
            for _ in range(12):
                tok = rng.integers(0, V, size=m).astype(np.int32)
                top1 = rng.integers(0, V, size=m)
                tl = rng.standard_normal((m, V))
                tl[np.arange(m), top1] += 10.0
                path, toks, bonus = orc.accept_greedy(tl, tok, parent)
                depth = synth.tree_depths(parent)
                # validity: a root-to-node path whose tokens are the target's own choices
                cur = 0
                for c, t in zip(path, toks):
                    assert parent[c] == cur and tok[c] == t == top1[cur]
                    cur = c
                assert bonus == top1[cur]
                # maximality at the stop node
                assert all(tok[c] != top1[cur] for c in orc.children_of(parent, cur))
                assert len(path) <= (depth.max() if m > 1 else 0)
                # with distinct sibling tokens the walk is the unique longest valid path
                distinct = all(
                    len({int(tok[c]) for c in orc.children_of(parent, i)})
                    == len(orc.children_of(parent, i)) for i in range(m))
                if distinct:
                    longest = max(_valid_paths(top1, tok, parent), key=len)
                    assert path == longest
                checked += 1
    assert checked == 34 * 12


def test_greedy_first_matching_child_wins_and_ties_go_to_low_token():
    parent = np.array([-1, 0, 0, 1, 2], dtype=np.int32)
    tok = np.array([9, 1, 1, 2, 2], dtype=np.int32)
    tl = np.zeros((5, 4))
    tl[0, 1] = 5.0
    tl[1, 3] = 5.0          # first child (node 1) leads nowhere: its top-1 is 3
    tl[2, 2] = 5.0          # second child would have continued
    path, toks, bonus = orc.accept_greedy(tl, tok, parent)
    assert path == [1] and toks == [1] and bonus == 3
    tl = np.zeros((1, 4))   # all-equal row: top-1 is token 0
    assert orc.accept_greedy(tl, np.array([0]), np.array([-1]))[2] == 0


class _ToyTarget:
    """Embedding + position embedding -> one pre-norm attention block -> norm -> head.
    The sequence pass below is written on its own (plain causal loops over the whole
    sequence); only the tree pass calls the oracle's masked attention."""

    def __init__(self, seed, V=48, H=32, heads=4, max_pos=64):
        rng = np.random.default_rng(seed)
        self.V, self.H, self.h, self.d = V, H, heads, H // heads
        self.emb = rng.standard_normal((V, H))
        self.pos = rng.standard_normal((max_pos, H))
        self.wq, self.wk, self.wv, self.wo = (rng.standard_normal((H, H)) / math.sqrt(H)
                                              for _ in range(4))
        self.head = rng.standard_normal((V, H)) * 2.0

    def _norm(self, x):
        return x / np.sqrt((x * x).mean(-1, keepdims=True) + 1e-6)

    def hidden(self, tokens, positions):
        return self.emb[tokens] + self.pos[positions]

    def qkv(self, hid):
        n = self._norm(hid)
        shape = (-1, self.h, self.d)
        return ((n @ self.wq.T).reshape(shape), (n @ self.wk.T).reshape(shape),
                (n @ self.wv.T).reshape(shape))

    def logits_from_attn(self, hid, attn):
        x = hid + attn.reshape(-1, self.H) @ self.wo.T
        return self._norm(x) @ self.head.T

    def next_token(self, seq):
        """Plain target-only decoding step on a whole sequence."""
        n = len(seq)
        hid = self.hidden(np.array(seq), np.arange(n))
        q, k, v = self.qkv(hid)
        attn = np.zeros((self.h, self.d))
        for h in range(self.h):
            s = np.array([q[n - 1, h] @ k[j, h] for j in range(n)]) / math.sqrt(self.d)
            p = np.exp(s - s.max())
            p /= p.sum()
            attn[h] = sum(p[j] * v[j, h] for j in range(n))
        return int(np.argmax(self.logits_from_attn(hid[n - 1:n], attn[None])[0]))


@pytest.mark.parametrize("seed,planted", [(1, 0), (2, 1), (3, 3), (4, 4)])
def test_greedy_speculation_reproduces_plain_argmax_decoding(seed, planted):
    tgt = _ToyTarget(seed)
    rng = np.random.default_rng(100 + seed)
    P, M, D = 10, 16, 4
    prefix = rng.integers(0, tgt.V, size=P).tolist()
    root = int(rng.integers(0, tgt.V))
    # what the target alone would emit after prefix + root
    seq = prefix + [root]
    truth = []
    for _ in range(D + 1):
        truth.append(tgt.next_token(seq + truth))
    parent = synth.random_tree(M, D, seed)
    depth = synth.tree_depths(parent)
    tok = rng.integers(0, tgt.V, size=M).astype(np.int32)
    tok[0] = root
    # plant the true continuation along one path for `planted` levels
    cur = 0
    n_planted = 0
    for lvl in range(planted):
        kids = orc.children_of(parent, cur)
        if not kids:
            break
        c = kids[int(rng.integers(0, len(kids)))]
        tok[c] = truth[lvl]
        cur = c
        n_planted += 1
    # target pass over the tree with the tree mask
    hid_p = tgt.hidden(np.array(prefix), np.arange(P))
    _, kp, vp = tgt.qkv(hid_p)
    hid_t = tgt.hidden(tok, P + depth)
    qt, kt, vt = tgt.qkv(hid_t)
    kc = np.concatenate([kp, kt]).transpose(1, 0, 2)[None]       # [1, heads, P+M, d]
    vc = np.concatenate([vp, vt]).transpose(1, 0, 2)[None]
    attn = orc.tree_verify_attn(qt[None], kc, vc, np.array([P]), parent[None],
                                1.0 / math.sqrt(tgt.d))[0]
    tl = tgt.logits_from_attn(hid_t, attn)
    path, toks, bonus = orc.accept_greedy(tl, tok, parent)
    emitted = toks + [bonus]
    assert emitted == truth[:len(emitted)]                        # lossless (Sec. 2.1)
    assert len(path) >= n_planted
    assert len(path) <= D


# ----------------------------------------------------------------- sampling
def _chain_rule_reference(p_rows, q_rows, toks, u_acc, u_bonus):
    """Sec. 2.1 steps 2-3 for a plain chain, written directly."""
    out = []
    for i, x in enumerate(toks):
        p, q = p_rows[i], q_rows[i]
        if u_acc[i] < min(1.0, p[x] / q[x]):
            out.append(x)
            continue
        r = np.maximum(0.0, p - q)
        r /= r.sum()
        c = np.cumsum(r)
        return out, int(np.nonzero(c > u_bonus[i] * c[-1])[0][0])
    p = p_rows[len(toks)]
    c = np.cumsum(p)
    return out, int(np.nonzero(c > u_bonus[len(toks)] * c[-1])[0][0])


@pytest.mark.parametrize("seed", range(8))
def test_sampling_on_a_chain_is_the_papers_rule(seed):
    rng = np.random.default_rng(seed)
    V, M = 11, 5
    parent = synth.chain_tree(M)
    depth = synth.tree_depths(parent)
    tl = rng.standard_normal((M, V)) * 2
    dl = rng.standard_normal((M, 2, V)) * 2                       # slot = node index
    tok = rng.integers(0, V, size=M).astype(np.int32)
    branch = rng.integers(0, 2, size=M).astype(np.int32)
    qslot = np.arange(M, dtype=np.int32)
    ua, ub = rng.random(M), rng.random(M + 1)
    T = 0.8
    path, toks, bonus = orc.accept_sampling(tl, tok, parent, depth, branch, qslot, dl, ua, ub, T)
    p_rows = [orc.softmax(tl[i] / T) for i in range(M)]
    q_rows = [orc.softmax(dl[i, branch[i + 1]] / T) for i in range(M - 1)]
    ref_toks, ref_bonus = _chain_rule_reference(p_rows, q_rows, tok[1:].tolist(), ua[1:], ub)
    assert toks == ref_toks and bonus == ref_bonus
    assert path == list(range(1, len(toks) + 1))


def test_sampling_accepts_every_first_child_when_draft_equals_target():
    rng = np.random.default_rng(3)
    V, M = 9, 7
    parent = synth.binary_tree(M)
    depth = synth.tree_depths(parent)
    tl = rng.standard_normal((M, V))
    dl = np.stack([tl, tl], axis=1)                               # q == p at every node
    tok = rng.integers(0, V, size=M).astype(np.int32)
    path, toks, _ = orc.accept_sampling(tl, tok, parent, depth, np.zeros(M, np.int32),
                                        np.arange(M, dtype=np.int32), dl,
                                        rng.random(M) * 0.999999, rng.random(4), 1.0)
    assert path == [1, 3]                                         # first child at each level


def test_sampling_at_low_temperature_is_greedy():
    w = synth.scaled(synth.WORKLOADS["tiny"], vocab=50, tree_size=12)
    parent = synth.random_tree(12, 4, 5)
    depth = synth.tree_depths(parent)
    rng = np.random.default_rng(5)
    tok = rng.integers(0, 50, size=12).astype(np.int32)
    for alpha in (0.0, 0.8, 1.0):
        tl = synth.target_logits(w, tok[None], parent[None], alpha)[0]
        dl = rng.standard_normal((12, 2, 50))
        g = orc.accept_greedy(tl, tok, parent)
        s = orc.accept_sampling(tl, tok, parent, depth, rng.integers(0, 2, 12).astype(np.int32),
                                np.arange(12, dtype=np.int32), dl, rng.random(12),
                                rng.random(5), 1e-3)
        assert s[0] == g[0] and s[1] == g[1] and s[2] == g[2]


def test_sampling_is_lossless_with_sampled_children_two_branches():
    """Children drawn without replacement from each branch's own q: the first emitted token
    must follow the target's p exactly (chi-square on V = 8)."""
    rng = np.random.default_rng(7)
    V, k_e, trials = 8, 2, 30000
    tl = rng.standard_normal((1 + 2 * k_e, V)) * 1.5
    dl = rng.standard_normal((1, 2, V)) * 1.5
    p = orc.softmax(tl[0])
    q = [orc.softmax(dl[0, r]) for r in range(2)]
    M = 1 + 2 * k_e
    parent = synth.star_tree(M)
    depth = synth.tree_depths(parent)
    branch = np.array([0] + [0] * k_e + [1] * k_e, dtype=np.int32)
    qslot = np.full(M, -1, dtype=np.int32)
    qslot[0] = 0
    counts = np.zeros(V)
    for _ in range(trials):
        tok = np.zeros(M, dtype=np.int32)
        for r in range(2):
            tok[1 + r * k_e:1 + (r + 1) * k_e] = rng.choice(V, size=k_e, replace=False, p=q[r])
        path, toks, bonus = orc.accept_sampling(tl, tok, parent, depth, branch, qslot, dl,
                                                rng.random(M), rng.random(2), 1.0)
        counts[toks[0] if toks else bonus] += 1
    chi2 = float(((counts - trials * p) ** 2 / (trials * p)).sum())
    assert chi2 < 24.3            # chi-square, 7 d.o.f., p = 1e-3


def test_sampling_joint_of_two_levels_is_lossless():
    rng = np.random.default_rng(11)
    V, trials = 4, 30000
    # root with one child per branch; each child with one child per branch
    parent = np.array([-1, 0, 0, 1, 1, 2, 2], dtype=np.int32)
    depth = synth.tree_depths(parent)
    branch = np.array([0, 0, 1, 0, 1, 0, 1], dtype=np.int32)
    qslot = np.array([0, 1, 2, -1, -1, -1, -1], dtype=np.int32)
    dl = rng.standard_normal((3, 2, V))
    # the target's next-token logits depend on the token sequence so far
    tl_root = rng.standard_normal(V)
    tl_after = rng.standard_normal((V, V))
    counts = np.zeros((V, V))
    for _ in range(trials):
        tok = np.zeros(7, dtype=np.int32)
        tok[1] = rng.choice(V, p=orc.softmax(dl[0, 0]))
        tok[2] = rng.choice(V, p=orc.softmax(dl[0, 1]))
        for c, slot in ((1, 1), (2, 2)):
            tok[2 * c + 1] = rng.choice(V, p=orc.softmax(dl[slot, 0]))
            tok[2 * c + 2] = rng.choice(V, p=orc.softmax(dl[slot, 1]))
        tl = np.zeros((7, V))
        tl[0] = tl_root
        tl[1], tl[2] = tl_after[tok[1]], tl_after[tok[2]]
        path, toks, bonus = orc.accept_sampling(tl, tok, parent, depth, branch, qslot, dl,
                                                rng.random(7), rng.random(3), 1.0)
        emitted = toks + [bonus]
        t1 = emitted[0]
        if len(emitted) >= 2:
            t2 = emitted[1]
        else:       # stopped at the root: the second token comes from plain target sampling
            t2 = int(rng.choice(V, p=orc.softmax(tl_after[t1])))
        counts[t1, t2] += 1
    joint = orc.softmax(tl_root)[:, None] * orc.softmax(tl_after, axis=-1)
    chi2 = float(((counts - trials * joint) ** 2 / (trials * joint)).sum())
    assert chi2 < 37.7            # chi-square, 15 d.o.f., p = 1e-3


def test_inverse_cdf_edges():
    p = np.array([0.0, 0.25, 0.0, 0.75])
    assert orc.inverse_cdf(p, 0.0) == 1
    assert orc.inverse_cdf(p, 0.2499) == 1
    assert orc.inverse_cdf(p, 0.25) == 3
    assert orc.inverse_cdf(p, 0.999999) == 3


def test_sampling_zero_draft_probability_and_vanishing_residual():
    V = 4
    parent = synth.star_tree(2)
    depth = synth.tree_depths(parent)
    tl = np.log(np.array([[0.5, 0.5, 1e-300, 1e-300], [0.25] * 4]))
    dl = np.zeros((1, 2, V))
    dl[0, 0] = [-1e4, 0.0, 0.0, 0.0]          # q[0] underflows to exactly 0
    tok = np.array([0, 0], dtype=np.int32)
    path, _, _ = orc.accept_sampling(tl, tok, parent, depth, np.zeros(2, np.int32),
                                     np.array([0, -1], np.int32), dl, np.array([0.0, 0.999]),
                                     np.array([0.3, 0.3]), 1.0)
    assert path == [1]                         # q(x) = 0 < p(x): always accepted
    # in floating point p = (1, 1e-200) and q = (1, 1e-100): token 1 is rejected and
    # max(0, p - q) is zero everywhere, so the bonus is drawn from the node's own p
    V = 2
    tl = np.array([[0.0, math.log(1e-200)], [0.0, 0.0]])
    dl = np.zeros((1, 2, V))
    dl[0, 0] = [0.0, math.log(1e-100)]
    tr = []
    path, _, bonus = orc.accept_sampling(tl, np.array([0, 1], np.int32), parent, depth,
                                         np.zeros(2, np.int32), np.array([0, -1], np.int32), dl,
                                         np.array([0.0, 0.5]), np.array([0.6, 0.3]), 1.0, trace=tr)
    assert tr[0]["accepted"] is False and path == [] and bonus == 0


# ----------------------------------------------------------------- compaction
def test_compaction_moves_rows_and_keeps_the_rest():
    rng = np.random.default_rng(1)
    Hkv, cap, d, P = 2, 24, 4, 9
    cache = rng.standard_normal((Hkv, cap, d))
    acc = [2, 5, 11]
    out = orc.compact_kv(cache, P, acc)
    assert np.array_equal(out[:, :P + 1], cache[:, :P + 1])        # prefix and root untouched
    for j, a in enumerate(acc):
        for h in range(Hkv):
            for c in range(d):
                assert out[h, P + 1 + j, c] == cache[h, P + a, c]
    assert np.array_equal(out[:, P + 1 + len(acc):], cache[:, P + 1 + len(acc):])
    # overlapping case: destination of step 1 is the source of step 0
    out = orc.compact_kv(cache, P, [2, 3])
    assert np.array_equal(out[:, P + 1], cache[:, P + 2])
    assert np.array_equal(out[:, P + 2], cache[:, P + 3])
    # a path that already sits behind the root is a no-op, and so is the empty path
    assert np.array_equal(orc.compact_kv(cache, P, [1, 2, 3]), cache)
    assert np.array_equal(orc.compact_kv(cache, P, []), cache)
