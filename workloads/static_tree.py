"""A fixed-shape draft tree as a second workload for the mask, attention and acceptance steps.

The paper contrasts its dynamic tree with the static tree of its predecessor (Section 3, the figure
that shows that tree's shape is not available), so the shape here is a declared stand-in:

    a node that is the c-th most probable child of its parent (c = 0, 1, ...) at depth l (the root
    is depth 0, c = 0) gets max(0, 4 - c - l) children; child c' of a node carries the c'-th most
    probable token of that node's draft row (ties to the lower token id).

That gives 4 + 6 + 8 + 5 = 23 nodes over four levels, with at most 5 expanded nodes per level, so the
tree embeds into the interface's candidate index space for any k >= 5 (level-l node = k + (l-2)k^2 +
j*k + c', j = the slot its parent takes among the expanded nodes of level l-1) and the acceptance
step finds every node's draft row by the same convention as for a dynamic tree.
"""
from __future__ import annotations

import numpy as np

N_LEVELS = 4  # = expansion steps D of the embedding


def shape(k: int):
    """Returns (index[n], parent_flat[n], depth[n], child_rank[n], row_of[n]) in ascending candidate
    index; row_of = draft row of the node's own children, -1 for a leaf.  Draft row 0 is the root's."""
    assert k >= 5
    nodes = []  # (index, parent_index, level, rank, n_children)
    frontier = [(-1, 0, 0)]  # (candidate index, level, rank) of the nodes expanded at this step
    slot_of = {}
    for step in range(N_LEVELS):
        nxt = []
        for j, (pidx, lvl, rank) in enumerate(frontier):
            n_children = max(0, 4 - rank - lvl)
            slot_of[pidx] = (step, j)
            for c in range(n_children):
                idx = c if step == 0 else k + (step - 1) * k * k + j * k + c
                nodes.append((idx, pidx, lvl + 1, c))
                if max(0, 4 - c - (lvl + 1)) > 0 and step + 1 < N_LEVELS:
                    nxt.append((idx, lvl + 1, c))
        assert len(nxt) <= k
        frontier = nxt
    nodes.sort()
    index = np.array([n[0] for n in nodes], np.int32)
    pos = {int(i): p for p, i in enumerate(index)}
    parent = np.array([pos.get(n[1], -1) for n in nodes], np.int32)
    depth = np.array([n[2] - 1 for n in nodes], np.int32)
    rank = np.array([n[3] for n in nodes], np.int32)
    row_of = np.full(len(nodes), -1, np.int32)
    for p, i in enumerate(index):
        if int(i) in slot_of:
            step, j = slot_of[int(i)]
            row_of[p] = 1 + (step - 1) * k + j
    return index, parent, depth, rank, row_of


def tokens(draft_rows: np.ndarray, k: int):
    """sel_token [B, n]: child c of a node = the c-th largest logit of the node's draft row."""
    index, parent, depth, rank, row_of = shape(k)
    B = draft_rows.shape[0]
    tok = np.zeros((B, len(index)), np.int32)
    for b in range(B):
        for x in range(len(index)):
            row = 0 if parent[x] < 0 else int(row_of[parent[x]])
            z = draft_rows[b, row]
            order = np.lexsort((np.arange(z.size), -z.astype(np.float64)))  # logit desc, id asc
            tok[b, x] = order[rank[x]]
    return tok
