"""Writes ``caption_shape_cycle.txt``: the oracle's results for one seeded cycle at the shape the paper's
method-figure caption describes (Section 4: the 2 best nodes of a layer are expanded, the 8 best of all
nodes form the draft; three layers here, vocabulary 50).

The figure itself is an image that is not available, so the paper prints no values for this example:
the numbers in the file are the oracle's, on inputs from the seeded generators, and serve as a stored
expectation for the device path and as a tripwire for any change in the oracle's arithmetic.  This
script calls nothing but ``oracle/`` and the input generators.  Run from the repository root:

    python tests/golden/make_caption_shape_cycle.py
"""
from __future__ import annotations

import os
import sys

import numpy as np

ROOT = os.path.dirname(os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
sys.path.insert(0, ROOT)

from oracle import ref  # noqa: E402
from workloads import generators as gen  # noqa: E402
from workloads import get_config  # noqa: E402

SEED = 2
PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "caption_shape_cycle.txt")


def config():
    return get_config("tiny", B=1, V=50, k=2, D=3, m=8, kv_len=17)


def compute() -> dict:
    cfg = config()
    draft = gen.draft_rows(cfg, SEED)
    tree = ref.build_tree(draft, cfg.V, cfg.k, cfg.D)
    sel = ref.rerank(tree.token, tree.parent, tree.value, cfg.k, cfg.D, cfg.m)
    kv_len = np.full(1, cfg.kv_len, np.int32)
    bits, _, pos, st = ref.tree_mask(sel.parent, sel.depth, sel.n_sel, kv_len, cfg.m)
    target = gen.target_rows(cfg, SEED, draft, tree.parent, sel.index)
    ua, ub = gen.uniforms(cfg, SEED)
    acc = ref.accept(target, None, sel, cfg.V, cfg.k, cfg.D, cfg.m, 0.0, ua, ub)
    return {
        "tree_token": tree.token[0].tolist(), "tree_parent": tree.parent[0].tolist(),
        "tree_value": [float(v) for v in tree.value[0]], "frontier": tree.frontier[0].tolist(),
        "sel_index": sel.index[0].tolist(), "sel_parent": sel.parent[0].tolist(),
        "sel_token": sel.token[0].tolist(), "sel_depth": sel.depth[0].tolist(), "n_sel": int(sel.n_sel[0]),
        "mask_bits": [int(x) for x in bits[0, :, 0]], "pos_ids": pos[0].tolist(),
        "acc_len": int(acc.acc_len[0]), "acc_path": acc.acc_path[0].tolist(),
        "bonus_token": int(acc.bonus_token[0]), "status": int(tree.status | sel.status | st | acc.status),
    }


def render(d: dict) -> str:
    lines = ["# oracle results, seed %d, V=50 k=2 D=3 m=8 kv_len=17, greedy acceptance" % SEED,
             "# (shape of the method figure's caption, Section 4; values are the oracle's, not the paper's)"]
    for key, val in d.items():
        if key == "tree_value":
            lines.append(key + " " + " ".join(repr(v) for v in val))
        elif isinstance(val, list):
            lines.append(key + " " + " ".join(str(v) for v in val))
        else:
            lines.append(key + " " + str(val))
    return "\n".join(lines) + "\n"


def parse(text: str) -> dict:
    out = {}
    for line in text.splitlines():
        if not line or line.startswith("#"):
            continue
        key, *vals = line.split()
        conv = float if key == "tree_value" else int
        out[key] = [conv(v) for v in vals] if key not in ("n_sel", "acc_len", "bonus_token", "status") else int(vals[0])
    return out


if __name__ == "__main__":
    with open(PATH, "w") as f:
        f.write(render(compute()))
    print("wrote", PATH)
