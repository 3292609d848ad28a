"""Host-side bookkeeping of the static (predefined, Eagle-1 style) tree policy (arXiv 2502.06282,
Sec. 3.1.2, last paragraph): turns a tree shape given as rank paths into the index lists that
jk_draft_expand (static_select) and jk_tree_finalize (static_keep) take.  Index arithmetic only;
which tokens fill the shape is decided on the device.

A path is a tuple of child ranks: rank c of a node is its c-th candidate in child order (branch
r = c // k_e, then rank j = c % k_e within the branch), so (0,) is the root's best left-branch
child.  Every prefix of a listed path must be listed.
"""
from __future__ import annotations

from typing import Dict, List, Sequence, Tuple


def plan_from_paths(paths: Sequence[Tuple[int, ...]], top_k: int, k_e: int) -> Dict[str, object]:
    """Returns
      frontier_sizes  expanded nodes per draft pass (pass l expands the listed nodes of depth l
                      that have listed children; the root alone in pass 0)
      select          per pass but the last: flat child indices (f * K + r) * k_e + j, within that
                      pass's candidates, of the nodes the next pass expands, in frontier order
      keep            generation indices of all listed nodes, ascending (the final tree)
      order           the paths in final node order behind the root (= ascending generation index)
    Frontier order within a pass is ascending path order, so a node's generation index follows
    from its parent's position in its pass."""
    per_node = top_k * k_e
    listed = sorted(set(tuple(p) for p in paths), key=lambda p: (len(p), p))
    have = set(listed)
    for p in listed:
        if not p:
            raise ValueError("the root is implied, not listed")
        if len(p) > 1 and p[:-1] not in have:
            raise ValueError(f"{p}: parent not listed")
        if not 0 <= p[-1] < per_node:
            raise ValueError(f"{p}: child rank outside 0..{per_node - 1}")
    depth = max((len(p) for p in listed), default=0)
    parents = {p[:-1] for p in listed}
    expanded: List[List[Tuple[int, ...]]] = [[()]]
    for d in range(1, depth):
        expanded.append([p for p in listed if len(p) == d and p in parents])
    gidx_of: Dict[Tuple[int, ...], int] = {}
    base = 0
    select: List[List[int]] = []
    for d, nodes in enumerate(expanded):
        pos = {p: f for f, p in enumerate(nodes)}
        for p in listed:
            if len(p) == d + 1:
                gidx_of[p] = base + pos[p[:-1]] * per_node + p[-1]
        if d + 1 < len(expanded):
            select.append([gidx_of[p] - base for p in expanded[d + 1]])
        base += len(nodes) * per_node
    order = sorted(listed, key=lambda p: gidx_of[p])
    return {"frontier_sizes": [len(n) for n in expanded], "select": select,
            "keep": [gidx_of[p] for p in order], "order": order}
