"""CPU-only checks of the library boundary: it loads, exports every declared entry point,
validates configurations and arguments before touching a GPU."""
import ctypes as C
import os
import re

import pytest

from paper_2502_06282_b200 import binding as jk

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2502_06282_b200 import build
    build.build()
    return jk.lib()


def test_every_declared_symbol_is_exported(lib):
    header = open(os.path.join(ROOT, "include", "jakiro.h")).read()
    declared = set(re.findall(r"\b(jk_[a-z_]+)\s*\(", header))
    assert declared, "no declarations found"
    assert declared == set(jk.EXPORTS)
    for name in declared:
        assert hasattr(lib, name), name


def _cfg(**kw):
    base = dict(hidden=512, n_experts=4, top_k=2, inter=1376, vocab=4096, n_q_heads=8,
                n_kv_heads=8, head_dim=64, max_batch=1, max_tree=16, max_depth=4,
                max_frontier=4, k_per_expert=2, dtype="f32", allocate=False)
    base.update(kw)
    return base


def test_create_and_workspace_size(lib):
    ctx = jk.Context(**_cfg())
    n = ctx.workspace_bytes
    assert n > 0 and n % 256 == 0
    big = jk.Context(**_cfg(max_batch=2)).workspace_bytes
    assert big > n
    ctx.close()


def test_contrastive_mode_needs_two_active_experts(lib):
    with pytest.raises(jk.JakiroError) as e:
        jk.Context(**_cfg(head_mode=1, top_k=3))
    assert e.value.code == jk.ERR["SHAPE"]
    with pytest.raises(jk.JakiroError):
        jk.Context(**_cfg(head_mode=2))
    jk.Context(**_cfg(head_mode=1, contrast_alpha=0.5, contrast_beta=1.5)).close()


@pytest.mark.parametrize("bad", [dict(hidden=510), dict(inter=1377), dict(n_experts=9),
                                 dict(top_k=5), dict(k_per_expert=17), dict(max_tree=129),
                                 dict(max_batch=64, max_frontier=4), dict(head_dim=96),
                                 dict(n_q_heads=8, n_kv_heads=3), dict(vocab=0)])
def test_create_rejects_unsupported_configs(lib, bad):
    with pytest.raises(jk.JakiroError) as e:
        jk.Context(**_cfg(**bad))
    assert e.value.code == jk.ERR["SHAPE"]


def test_calls_reject_bad_arguments_before_any_launch(lib):
    ctx = jk.Context(**_cfg())
    h = ctx._h
    null = None
    # NULL context / pointers
    assert lib.jk_tree_verify_attn(h, null, 1, 16, null, null, null, 0, 0, 64, null, null,
                                   1.0, null) == jk.ERR["NULL"]
    assert lib.jk_workspace_bytes(null) == 0
    assert lib.jk_destroy(null) == jk.ERR["NULL"]
    fake = C.c_void_p(0x1000)          # aligned, never dereferenced on these paths
    odd = C.c_void_p(0x1004)
    # capacity, shape, alignment, missing workspace
    assert lib.jk_tree_verify_attn(h, null, 2, 16, fake, fake, fake, 4096, 4096, 64, fake, fake,
                                   1.0, fake) == jk.ERR["CAPACITY"]
    assert lib.jk_tree_verify_attn(h, null, 1, 17, fake, fake, fake, 4096, 4096, 64, fake, fake,
                                   1.0, fake) == jk.ERR["CAPACITY"]
    assert lib.jk_tree_verify_attn(h, null, 1, 16, fake, fake, fake, 4096, 4096, 8, fake, fake,
                                   1.0, fake) == jk.ERR["SHAPE"]
    assert lib.jk_tree_verify_attn(h, null, 1, 16, odd, fake, fake, 4096, 4096, 64, fake, fake,
                                   1.0, fake) == jk.ERR["ALIGN"]
    assert lib.jk_tree_verify_attn(h, null, 1, 16, fake, fake, fake, 4098, 4098, 64, fake, fake,
                                   1.0, fake) == jk.ERR["ALIGN"]
    assert lib.jk_tree_verify_attn(h, null, 1, 16, fake, fake, fake, 4096, 4096, 64, fake, fake,
                                   1.0, fake) == jk.ERR["WORKSPACE"]
    # accept: sampling needs uniforms, a positive temperature and draft logits
    args = [h, null, 1, 16, 1, 1.0, fake, 0, fake, fake, fake, fake, fake, null, 13, null, null,
            0, null, null, 0, 0, 64, fake, fake, fake, fake, fake]
    assert lib.jk_accept_and_compact(*args) == jk.ERR["NULL"]
    args[13] = args[15] = args[16] = fake
    args[5] = 0.0
    assert lib.jk_accept_and_compact(*args) == jk.ERR["SHAPE"]
    args[5] = 1.0
    args[4] = 3
    assert lib.jk_accept_and_compact(*args) == jk.ERR["SHAPE"]
    args[4] = 0
    assert lib.jk_accept_and_compact(*args) == jk.ERR["WORKSPACE"]
    # workspace: alignment and size
    assert lib.jk_set_workspace(h, null, C.c_void_p(0x1010), 1 << 40) == jk.ERR["ALIGN"]
    assert lib.jk_set_workspace(h, null, C.c_void_p(0x1000), 16) == jk.ERR["WORKSPACE"]
    assert lib.jk_strerror(jk.ERR["BOUNDS"]).decode().startswith("input index")
    ctx.close()


def test_expand_and_finalize_argument_checks(lib):
    ctx = jk.Context(**_cfg())
    h = ctx._h
    fake = C.c_void_p(0x1000)
    w = jk.JkDraftWeights(0x1000, 0x1000, 0x1000, 0x1000, 0x1000, None)
    pool = jk.JkPool(0x1000, 0x1000, 0x1000, 0x1000, 0x1000, 52)

    def expand(batch=1, F=1, width=4, gidx=0, wts=w, p=pool, stride=0, static=None):
        return lib.jk_draft_expand(h, None, C.byref(wts), batch, F, width, fake, fake, fake, gidx,
                                   0, None, fake, fake, C.byref(p), None, fake, None, stride,
                                   fake, fake, fake, static)
    assert expand() == jk.ERR["WORKSPACE"]          # everything else is fine
    assert expand(batch=2) == jk.ERR["CAPACITY"]
    assert expand(F=5) == jk.ERR["CAPACITY"]
    assert expand(F=0) == jk.ERR["SHAPE"]
    assert expand(gidx=50) == jk.ERR["SHAPE"]        # children would not fit the pool
    assert expand(wts=jk.JkDraftWeights(0x1000, 0, 0x1000, 0x1000, 0x1000, None)) == jk.ERR["NULL"]
    assert expand(wts=jk.JkDraftWeights(0x1008, 0x1000, 0x1000, 0x1000, 0x1000, None)) \
        == jk.ERR["ALIGN"]
    assert expand(stride=6) == jk.ERR["SHAPE"]
    assert expand(width=0, static=fake) == jk.ERR["SHAPE"]   # a static list selects nothing on the last pass

    def finalize(pool_n=52, M=16, batch=1):
        return lib.jk_tree_finalize(h, None, batch, C.byref(pool), pool_n, fake, M, fake, fake,
                                    fake, fake, fake, fake, None)
    assert finalize() == jk.ERR["WORKSPACE"]
    assert finalize(pool_n=10) == jk.ERR["SHAPE"]    # fewer candidates than tree nodes
    assert finalize(pool_n=60) == jk.ERR["SHAPE"]    # more than the pool's stride
    assert finalize(M=17) == jk.ERR["CAPACITY"]
    ctx.close()


def test_static_tree_plan_matches_the_oracles_node_order():
    """plan_from_paths (product-side index bookkeeping) against the oracle's own ordering of a
    predefined tree: same node order, parents, depths and branches."""
    import numpy as np
    from oracle import jakiro_oracle as orc
    from paper_2502_06282_b200.static_tree import plan_from_paths
    paths = [(0,), (1,), (3,), (0, 0), (0, 2), (3, 1), (0, 0, 3), (0, 0, 0), (3, 1, 1), (3, 1, 2)]
    K, ke = 2, 2
    plan = plan_from_paths(paths, K, ke)
    rng = np.random.default_rng(0)
    w = {"router": rng.standard_normal((4, 8)), "w_gate": rng.standard_normal((4, 6, 8)),
         "w_up": rng.standard_normal((4, 6, 8)), "w_down": rng.standard_normal((4, 8, 6)),
         "lm_head": rng.standard_normal((11, 8)), "norm_weight": np.ones(8)}
    t = orc.grow_static_tree(lambda p: rng.standard_normal(8), w, paths, ke, root_tok=1)
    assert plan["order"] == t["order"][1:]
    assert plan["frontier_sizes"] == [1, 2, 2]
    assert plan["keep"] == sorted(plan["keep"]) and len(plan["keep"]) == len(paths)
    # generation index -> (pass, frontier row, candidate): the parent of a kept node is the
    # node that sits at that frontier row of the pass
    bases = np.cumsum([0] + [F * K * ke for F in plan["frontier_sizes"]])
    frontier = [[()]]
    for sel, base in zip(plan["select"], bases[:-1]):
        frontier.append([plan["order"][plan["keep"].index(base + s)] for s in sel])
    for p, g in zip(plan["order"], plan["keep"]):
        l = int(np.searchsorted(bases, g, side="right") - 1)
        f, c = divmod(int(g - bases[l]), K * ke)
        assert frontier[l][f] == p[:-1] and c == p[-1]
    with pytest.raises(ValueError):
        plan_from_paths([(0,), (1, 0)], K, ke)
    with pytest.raises(ValueError):
        plan_from_paths([(4,)], K, ke)
