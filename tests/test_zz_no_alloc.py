"""GPU check of ``eagle2_expand_static``, the expansion entry point for callers that cannot hand
the library a workspace (a server whose HBM is all committed to its cache pool, a loop that must
not trigger a device-wide synchronising allocation).  It runs the same kernels on a buffer that is
part of the library image, so its results must be identical to ``eagle2_expand``; two full trees in
a row show that the shared buffer carries nothing over from one call to the next.

The file name keeps this test last in collection order.
"""
import numpy as np
import pytest
import torch

import paper_2406_16858_b200 as e2
from workloads import get_config
from workloads import generators as gen

from harness import DEV, GpuTree, dev, host, new_status

pytestmark = pytest.mark.gpu


def _static_tree(draft_dev, B, V, k, D):
    N, R = k + (D - 1) * k * k, 1 + (D - 1) * k
    token = torch.full((B, N), -1, dtype=torch.int32, device=DEV)
    parent = torch.full((B, N), -2, dtype=torch.int32, device=DEV)
    value = torch.full((B, N), float("-inf"), dtype=torch.float64, device=DEV)
    frontier = torch.zeros((B, k), dtype=torch.int32, device=DEV)
    status = new_status()
    for s in range(D):
        lo = 0 if s == 0 else 1 + (s - 1) * k
        e2.expand_static(draft_dev.data_ptr() + lo * V * 4, R * V, B, V, k, D, s, token, parent, value,
                         frontier, status)
    torch.cuda.synchronize()
    return token, parent, value, frontier, status


@pytest.mark.parametrize("name,B", [("tiny", 1), ("tiny", 3), ("vicuna7b", 2), ("vicuna7b", 24)])  # the last: several tiles per block
def test_static_scratch_expansion_matches_workspace_expansion(name, B):
    cfg = get_config(name).with_(B=B)
    for seed in (3, 4):  # two trees back to back through the one shared buffer
        draft = dev(gen.draft_rows(cfg, seed))
        ref_tree = GpuTree(B, cfg.V, cfg.k, cfg.D).expand_all(draft)
        token, parent, value, frontier, status = _static_tree(draft, B, cfg.V, cfg.k, cfg.D)
        assert int(status.item()) == 0 and int(ref_tree.status.item()) == 0
        assert (host(token) == host(ref_tree.token)).all()
        assert (host(parent) == host(ref_tree.parent)).all()
        assert (host(frontier) == host(ref_tree.frontier)).all()
        got, want = host(value), host(ref_tree.value)
        assert np.abs(got - want).max() <= 1e-5 * max(1.0, np.abs(want).max())


def test_static_scratch_expansion_takes_no_device_memory():
    """What the entry point is for: its calls leave the device's free memory exactly as they found
    it.  After a first tree (whose first call looks the built-in buffer up), the free bytes the
    driver reports and the bytes torch's allocator holds are read before and after two more trees
    whose output arrays already exist; neither may move."""
    cfg = get_config("vicuna7b").with_(B=2)
    B, V, k, D = cfg.B, cfg.V, cfg.k, cfg.D
    draft = dev(gen.draft_rows(cfg, 9))
    N, R = cfg.N, cfg.R
    token = torch.full((B, N), -1, dtype=torch.int32, device=DEV)
    parent = torch.full((B, N), -2, dtype=torch.int32, device=DEV)
    value = torch.full((B, N), float("-inf"), dtype=torch.float64, device=DEV)
    frontier = torch.zeros((B, k), dtype=torch.int32, device=DEV)
    status = new_status()

    def one_tree():
        for s in range(D):
            lo = 0 if s == 0 else 1 + (s - 1) * k
            e2.expand_static(draft.data_ptr() + lo * V * 4, R * V, B, V, k, D, s, token, parent, value, frontier,
                             status)
        torch.cuda.synchronize()

    one_tree()
    free_before, _ = torch.cuda.mem_get_info()
    held_before = torch.cuda.memory_reserved()
    one_tree()
    one_tree()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    assert torch.cuda.memory_reserved() == held_before
    assert int(status.item()) == 0


def test_sizes_beyond_the_built_in_buffer_are_refused():
    cfg = get_config("llama3_8b")
    B = 2048  # 2048 sequences x 10 rows x (10 keys + statistics) exceed the 1 MiB buffer
    assert e2.workspace_bytes(e2.OP_EXPAND, B=B, V=cfg.V, k=cfg.k, D=cfg.D) > (1 << 20)
    N = cfg.N
    token = torch.zeros((B, N), dtype=torch.int32, device=DEV)
    value = torch.zeros((B, N), dtype=torch.float64, device=DEV)
    frontier = torch.zeros((B, cfg.k), dtype=torch.int32, device=DEV)
    logits = torch.zeros(16, dtype=torch.float32, device=DEV)  # never read: the call is refused first
    with pytest.raises(e2.Eagle2Error) as exc:
        e2.expand_static(logits, cfg.R * cfg.V, B, cfg.V, cfg.k, cfg.D, 1, token, token, value, frontier,
                         new_status())
    assert exc.value.code == -6
    assert "built-in" in e2.strerror(-6)
