"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the header
declares, sizes workspaces, and rejects bad arguments before launching anything."""
import ctypes as C
import os
import re

import pytest

import paper_2406_16858_b200 as e2
from paper_2406_16858_b200 import binding

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_symbols():
    text = open(os.path.join(ROOT, "include", "eagle2.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(eagle2_[a-z_0-9]+)\s*\(", text)))


def test_library_exports_every_declared_symbol():
    names = _declared_symbols()
    assert set(names) == set(binding.EXPORTS)
    h = C.CDLL(e2.lib_path())
    for n in names:
        assert getattr(h, n) is not None
    assert e2.version() >= 100
    assert "NULL" in e2.strerror(-1) and e2.strerror(0) == "ok"


def test_workspace_sizes_are_positive_and_grow_with_batch():
    a = e2.workspace_bytes(e2.OP_EXPAND, B=1, V=128256, k=10, D=6, m=60)
    b = e2.workspace_bytes(e2.OP_EXPAND, B=1024, V=128256, k=10, D=6, m=60)
    assert 0 < a < b  # (not monotone in between: larger batches cut a row into fewer segments)
    assert e2.workspace_bytes(e2.OP_ACCEPT, B=1, V=32000, k=10, D=6, m=60) > 0
    assert e2.workspace_bytes(e2.OP_TREE_ATTENTION, B=1, m=60, Hq=32, Hkv=8, d=128, max_kv_len=4096) > 0
    assert e2.workspace_bytes(e2.OP_RERANK, B=4) == 0
    assert e2.workspace_bytes(e2.OP_TREE_MASK, B=4) == 0
    assert e2.workspace_bytes(e2.OP_KV_COMPACT, B=4) == 0


def _code(fn, *args):
    with pytest.raises(e2.Eagle2Error) as exc:
        fn(*args)
    return exc.value.code


FAKE = 0x1000  # a non-NULL, 4096-aligned address; never dereferenced because validation fails first


def test_null_and_shape_errors_are_found_on_the_host():
    assert _code(e2.expand, None, 0, 1, 100, 4, 3, 0, FAKE, FAKE, FAKE, FAKE, None, FAKE) == -1
    # k > V, k > 32, s out of range, too many nodes
    assert _code(e2.expand, FAKE, 0, 1, 3, 4, 3, 0, FAKE, FAKE, FAKE, FAKE, None, FAKE) == -2
    assert _code(e2.expand, FAKE, 0, 1, 100, 33, 2, 0, FAKE, FAKE, FAKE, FAKE, None, FAKE) == -2
    assert _code(e2.expand, FAKE, 0, 1, 100, 4, 3, 3, FAKE, FAKE, FAKE, FAKE, None, FAKE) == -2
    assert _code(e2.expand, FAKE, 0, 1, 100, 32, 6, 0, FAKE, FAKE, FAKE, FAKE, None, FAKE) == -2
    # missing workspace
    assert _code(e2.expand, FAKE, 0, 1, 100, 4, 3, 0, FAKE, FAKE, FAKE, FAKE, None, FAKE) == -4
    assert _code(e2.rerank, FAKE, FAKE, FAKE, 1, 4, 3, 129, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE) == -2
    assert _code(e2.rerank, FAKE, FAKE, None, 1, 4, 3, 16, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE) == -1
    assert _code(e2.tree_mask, FAKE, FAKE, FAKE, FAKE, 1, 0, FAKE, None, FAKE, FAKE) == -2
    # attention: head_dim, group size, alignment
    att = lambda **kw: e2.tree_attention(  # noqa: E731
        kw.get("q", FAKE), FAKE, FAKE, kw.get("rows", 1024), FAKE, FAKE, FAKE, 1, 16, kw.get("Hq", 4),
        kw.get("Hkv", 4), kw.get("d", 64), 128, 0.125, FAKE, None, None, FAKE)
    assert _code(att) == -4  # two KV splits at this size: a workspace is required
    with pytest.raises(e2.Eagle2Error) as exc:
        att(d=96)
    assert exc.value.code == -2
    with pytest.raises(e2.Eagle2Error) as exc:
        att(Hq=6, Hkv=4)
    assert exc.value.code == -2
    with pytest.raises(e2.Eagle2Error) as exc:
        att(q=FAKE + 2)
    assert exc.value.code == -3
    with pytest.raises(e2.Eagle2Error) as exc:
        att(rows=100)  # the longest sequence (128 + 16 rows) does not fit in the cache
    assert exc.value.code == -2
    # accept: sampling needs the uniforms
    assert _code(e2.accept, FAKE, 0, None, 0, FAKE, FAKE, FAKE, FAKE, 1, 100, 4, 3, 16, 1.0, None, None,
                 FAKE, FAKE, FAKE, None, FAKE) == -1
    assert _code(e2.accept, FAKE, 0, None, 0, FAKE, FAKE, FAKE, FAKE, 1, 100, 4, 3, 16, -1.0, FAKE, FAKE,
                 FAKE, FAKE, FAKE, None, FAKE) == -2
    # compaction: row bytes must be a multiple of 16
    assert _code(e2.kv_compact, FAKE, FAKE, 1, FAKE, FAKE, FAKE, FAKE, 1, 16, 3, 1, 4, FAKE) == -3
    # the variants: unknown expansion flag, selection without a frontier
    assert _code(e2.expand_variant, FAKE, 0, 1, 100, 4, 3, 0, 2, FAKE, FAKE, FAKE, FAKE, None, FAKE) == -2
    assert _code(e2.expand_variant, FAKE, 0, 1, 100, 4, 3, 0, 1, FAKE, FAKE, FAKE, FAKE, None, FAKE) == -4
    assert _code(e2.rerank_skipped, FAKE, FAKE, FAKE, None, 1, 4, 3, 16, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE) == -1
    assert _code(e2.rerank_skipped, FAKE, FAKE, FAKE, FAKE, 1, 4, 3, 129, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE) == -2
    # LM head: hidden size in whole 64-column blocks, 16-byte aligned operands
    assert _code(e2.lm_head, FAKE, FAKE, 4, 96, 100, FAKE, FAKE) == -2
    assert _code(e2.lm_head, FAKE, FAKE, -1, 64, 100, FAKE, FAKE) == -2
    assert _code(e2.lm_head, FAKE + 2, FAKE, 4, 64, 100, FAKE, FAKE) == -3
    assert _code(e2.lm_head, FAKE, None, 4, 64, 100, FAKE, FAKE) == -1
    e2.lm_head(FAKE, FAKE, 0, 64, 100, FAKE, FAKE)  # no rows: nothing is launched


def test_zero_batch_is_a_no_op():
    e2.rerank(FAKE, FAKE, FAKE, 0, 4, 3, 16, FAKE, FAKE, FAKE, FAKE, FAKE, FAKE)
    e2.tree_mask(FAKE, FAKE, FAKE, FAKE, 0, 16, FAKE, None, FAKE, FAKE)


def test_ordered_attention_launch_reports_its_list():
    # 17 tiles per sequence and one block per (sequence, head): no partials, but the launch takes its
    # blocks from a device-built list, which lives in the workspace
    with_list = e2.workspace_bytes(e2.OP_TREE_ATTENTION, B=8, m=60, Hq=16, Hkv=16, d=128, max_kv_len=2100)
    without = e2.workspace_bytes(e2.OP_TREE_ATTENTION, B=8, m=60, Hq=16, Hkv=16, d=128, max_kv_len=1900)
    assert with_list >= 256 + 4 * 9 and without == 0
