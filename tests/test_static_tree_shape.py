"""The fixed-shape tree workload (host side): its shape is a closed forest in topological order and
its embedding into the candidate index space agrees with the oracle's mask walk."""
import numpy as np

from oracle import ref
from workloads import static_tree

K, D = 10, static_tree.N_LEVELS


def test_shape_is_a_closed_topological_forest():
    index, parent, depth, rank, row_of = static_tree.shape(K)
    assert len(index) == 23 and (np.diff(index) > 0).all()
    assert (parent < np.arange(len(index))).all() and depth.max() == D - 1
    assert (depth[parent[parent >= 0]] + 1 == depth[parent >= 0]).all()
    has_children = np.isin(np.arange(len(index)), parent)
    assert ((row_of >= 0) == has_children).all()


def test_oracle_mask_walks_the_static_forest():
    index, parent, depth, _, _ = static_tree.shape(K)
    n = len(index)
    bits, dense, pos, st = ref.tree_mask(parent[None], depth[None], np.array([n], np.int32), np.array([100], np.int32),
                                         n, dense=True)
    assert st == 0
    for i in range(n):
        chain, j = [], i
        while j >= 0:
            chain.append(j)
            j = int(parent[j])
        assert sorted(np.nonzero(dense[0, i])[0].tolist()) == sorted(chain)
        assert int(bits[0, i, 0]) == sum(1 << c for c in chain)
        assert pos[0, i] == 100 + depth[i]
