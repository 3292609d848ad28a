"""Pins for the oracle's tree mask and verification attention (Fig. 4, Sec. 2.1 step 2)."""
import math

import numpy as np
import pytest

from oracle import jakiro_oracle as orc
from paper_2502_06282_b200 import synth


def _causal_last_row(q, ks, vs, scale):
    """Plain single-query attention over a whole sequence, pure Python."""
    s = [scale * sum(q[k] * kk[k] for k in range(len(q))) for kk in ks]
    m = max(s)
    e = [math.exp(t - m) for t in s]
    z = sum(e)
    return [sum(e[j] / z * vs[j][c] for j in range(len(ks))) for c in range(len(vs[0]))]


def _inputs(seed, B, M, Hq, Hkv, d, P, cap=None):
    rng = np.random.default_rng(seed)
    cap = cap or (P + M + 3)
    q = rng.standard_normal((B, M, Hq, d))
    k = rng.standard_normal((B, Hkv, cap, d))
    v = rng.standard_normal((B, Hkv, cap, d))
    return q, k, v, np.full(B, P, dtype=np.int32)


def test_mask_shapes():
    anc = orc.ancestor_mask(synth.chain_tree(6))
    assert np.array_equal(anc, np.tril(np.ones((6, 6), bool)))       # chain = causal
    anc = orc.ancestor_mask(synth.star_tree(5))
    for i in range(5):
        assert set(np.nonzero(anc[i])[0]) == {0, i}                  # star = root + self
    par = synth.random_tree(20, 5, 3)
    anc = orc.ancestor_mask(par)
    assert np.array_equal(anc.sum(1), synth.tree_depths(par) + 1)


def test_chain_tree_equals_dense_causal_attention():
    B, M, Hq, Hkv, d, P = 1, 5, 2, 2, 4, 6
    q, k, v, kv_len = _inputs(1, B, M, Hq, Hkv, d, P)
    par = synth.chain_tree(M)[None]
    out = orc.tree_verify_attn(q, k, v, kv_len, par, 0.5)
    for i in range(M):
        for h in range(Hq):
            n = P + i + 1                                            # causal: columns 0..P+i
            ref = _causal_last_row(q[0, i, h], k[0, h, :n], v[0, h, :n], 0.5)
            assert np.allclose(out[0, i, h], ref, atol=1e-12)


@pytest.mark.parametrize("seed", [2, 3])
def test_every_row_equals_causal_attention_on_its_own_path(seed):
    # brute force that never builds a mask: node i sees prefix + path(root..i)
    B, M, Hq, Hkv, d, P = 2, 12, 4, 2, 8, 9
    q, k, v, kv_len = _inputs(seed, B, M, Hq, Hkv, d, P)
    kv_len[1] = 5
    par = np.stack([synth.random_tree(M, 4, seed), synth.binary_tree(M)])
    out = orc.tree_verify_attn(q, k, v, kv_len, par, 1.0 / math.sqrt(d))
    G = Hq // Hkv
    for b in range(B):
        Pb = int(kv_len[b])
        for i in range(M):
            path = []
            t = i
            while t >= 0:
                path.append(t)
                t = int(par[b, t])
            cols = list(range(Pb)) + [Pb + t for t in reversed(path)]
            for h in range(Hq):
                ref = _causal_last_row(q[b, i, h], k[b, h // G, cols], v[b, h // G, cols],
                                       1.0 / math.sqrt(d))
                assert np.allclose(out[b, i, h], ref, atol=1e-12)


def test_sibling_permutation_invariance():
    B, M, Hq, Hkv, d, P = 1, 7, 2, 1, 4, 5
    q, k, v, kv_len = _inputs(4, B, M, Hq, Hkv, d, P)
    par = np.array([[-1, 0, 0, 1, 1, 2, 2]], dtype=np.int32)
    out = orc.tree_verify_attn(q, k, v, kv_len, par, 0.3)
    # swap siblings 1 <-> 2 together with their subtrees (3,4) <-> (5,6)
    perm = np.array([0, 2, 1, 5, 6, 3, 4])
    q2 = q[:, perm]
    k2, v2 = k.copy(), v.copy()
    k2[:, :, P:P + M] = k[:, :, P + perm]
    v2[:, :, P:P + M] = v[:, :, P + perm]
    out2 = orc.tree_verify_attn(q2, k2, v2, kv_len, par, 0.3)
    assert np.allclose(out2, out[:, perm], atol=1e-12)


def test_single_node_tree_is_plain_decode_attention_and_rows_are_convex():
    B, M, Hq, Hkv, d, P = 1, 1, 3, 3, 4, 10
    q, k, v, kv_len = _inputs(5, B, M, Hq, Hkv, d, P)
    out = orc.tree_verify_attn(q, k, v, kv_len, np.array([[-1]]), 0.7)
    for h in range(Hq):
        ref = _causal_last_row(q[0, 0, h], k[0, h, :P + 1], v[0, h, :P + 1], 0.7)
        assert np.allclose(out[0, 0, h], ref, atol=1e-12)
    # constant V rows: softmax weights sum to one, so the output is that row
    v[:] = np.arange(d)[None, None, None, :]
    out = orc.tree_verify_attn(q, k, v, kv_len, np.array([[-1]]), 0.7)
    assert np.allclose(out, np.arange(d), atol=1e-12)


def test_gqa_equals_mha_with_repeated_kv_heads_and_ignores_rows_past_the_tree():
    B, M, Hq, Hkv, d, P = 1, 6, 4, 2, 4, 7
    q, k, v, kv_len = _inputs(6, B, M, Hq, Hkv, d, P, cap=32)
    par = synth.binary_tree(M)[None]
    out = orc.tree_verify_attn(q, k, v, kv_len, par, 0.5)
    out_mha = orc.tree_verify_attn(q, np.repeat(k, 2, axis=1), np.repeat(v, 2, axis=1), kv_len,
                                   par, 0.5)
    assert np.allclose(out, out_mha, atol=1e-13)
    k[:, :, P + M:] = 1e6
    v[:, :, P + M:] = -1e6
    assert np.allclose(orc.tree_verify_attn(q, k, v, kv_len, par, 0.5), out, atol=1e-13)


def test_empty_prefix():
    B, M, Hq, Hkv, d, P = 1, 4, 1, 1, 4, 0
    q, k, v, kv_len = _inputs(7, B, M, Hq, Hkv, d, P)
    par = synth.star_tree(M)[None]
    out = orc.tree_verify_attn(q, k, v, kv_len, par, 1.0)
    assert np.allclose(out[0, 0, 0], v[0, 0, 0], atol=1e-13)          # root sees only itself
