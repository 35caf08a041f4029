"""The C-ABI library builds, loads without a GPU and exports every symbol include/spechub.h
declares; host-side argument checks reject bad descriptors before any CUDA call."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    src = open(os.path.join(ROOT, "include", "spechub.h")).read()
    src = re.sub(r"/\*.*?\*/", "", src, flags=re.S)
    names = re.findall(r"\b([a-z_0-9]+)\s*\(", src)
    return sorted(set(n for n in names if n.startswith(("spechub_", "rrs_", "mdsd_"))))


def test_header_declares_the_expected_entry_points():
    assert declared_functions() == sorted([
        "spechub_draft_sample", "rrs_draft_sample", "spechub_verify_tree", "rrs_verify_tree",
        "mdsd_compare_draft_sample", "mdsd_compare_verify_tree", "spechub_walk_tree",
        "spechub_shard_stats", "spechub_shard_sums", "spechub_shard_decide", "spechub_shard_draft",
        "spechub_shard_draft_finish", "spechub_verify_tree_static",
        "rrs_shard_sums", "rrs_shard_decide", "rrs_shard_draft", "rrs_shard_draft_finish",
        "spechub_draft_stats_bytes", "spechub_draft_sample_stats", "rrs_draft_sample_stats",
        "spechub_verify_tree_stats", "rrs_verify_tree_stats",
        "mdsd_compare_draft_sample_stats", "mdsd_compare_verify_tree_stats",
        "spechub_workspace_bytes", "spechub_status_string", "spechub_abi_version"])


def test_library_exports_every_declared_symbol():
    import paper_2411_05289_b200 as sh

    lib = sh.load_library()
    for name in declared_functions():
        assert hasattr(lib, name), name
    assert sh.abi_version() == 1
    assert sh.status_string(0) == "ok" and "temperature" in sh.status_string(-6)


def test_descriptor_layout_matches_header():
    from paper_2411_05289_b200.binding import _Desc, _NodeOut, _SeqOut

    # struct_size is checked by the library, so a mismatch cannot go unnoticed at run time either
    assert ctypes.sizeof(_Desc) == 88
    assert ctypes.sizeof(_NodeOut) == 6 * 8 and ctypes.sizeof(_SeqOut) == 4 * 8


def test_host_side_argument_checks_need_no_gpu():
    import paper_2411_05289_b200 as sh
    from paper_2411_05289_b200.binding import _Desc

    lib = sh.load_library()

    def desc(**kw):
        d = _Desc()
        d.struct_size = ctypes.sizeof(_Desc); d.version = 1
        d.batch, d.nodes, d.vocab, d.k, d.dtype, d.levels = 2, 3, 64, 2, 0, 2
        d.stride_seq, d.stride_node, d.temperature = 192, 64, 1.0
        for k, v in kw.items():
            setattr(d, k, v)
        return d

    fake = ctypes.c_void_p(16)  # never dereferenced: every call below is rejected on the host
    call = lambda d: lib.spechub_draft_sample(ctypes.byref(d), fake, fake, fake, None, None, None, None)
    assert call(desc(k=3)) == -3   # SpecHub takes exactly two drafts
    assert call(desc(k=9)) == -3
    assert call(desc(vocab=1)) == -3
    assert call(desc(nodes=0)) == -3
    assert call(desc(batch=-1)) == -3
    assert call(desc(dtype=5)) == -4
    assert call(desc(version=2)) == -2
    # the calls that hand draft statistics on: the record buffer is required, its size is 16 bytes a row
    assert lib.spechub_draft_stats_bytes(ctypes.byref(desc())) == 16 * 2 * 3
    assert lib.spechub_draft_sample_stats(ctypes.byref(desc()), fake, fake, fake, None, None, None, None, None) == -1
    assert lib.rrs_draft_sample_stats(ctypes.byref(desc()), fake, fake, 2, fake, None, fake, None) == -9
    odd = ctypes.c_void_p(24)   # a record buffer that is not 16-byte aligned is refused before any launch
    assert lib.spechub_draft_sample_stats(ctypes.byref(desc()), fake, fake, fake, None, None, None, odd, None) == -5
    from paper_2411_05289_b200.binding import _NodeOut

    no = _NodeOut(16, 16, None, None, None, None)   # (pointers never followed: the call is refused first)
    assert lib.spechub_verify_tree_stats(ctypes.byref(desc()), fake, fake, odd, fake, fake, ctypes.byref(no), None,
                                         None, 0, None) == -5

    assert call(desc(struct_size=8)) == -2
    assert call(desc(stride_node=63)) == -5
    assert call(desc(stride_seq=100)) == -5
    assert call(desc(temperature=float("nan"))) == -6
    assert call(desc(temperature=-1.0)) == -6
    assert lib.spechub_draft_sample(None, fake, fake, fake, None, None, None, None) == -1
    assert lib.spechub_draft_sample(ctypes.byref(desc()), None, fake, fake, None, None, None, None) == -1
    assert lib.rrs_draft_sample(ctypes.byref(desc()), fake, fake, 7, fake, None, None) == -9
    assert call(desc(batch=0)) == 0  # an empty batch is a valid no-op


def test_product_path_does_not_reach_the_oracle():
    pkg = os.path.join(ROOT, "paper_2411_05289_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower() or f == "__init__.py" and "oracle" not in text.lower(), f


def test_tree_from_parents_builds_level_ordered_child_tables():
    import numpy as np
    import paper_2411_05289_b200 as sh

    # an unbalanced binary tree: 0 -> (1, 2); 1 -> (3, 4); 2 -> (5); 3 -> (6)
    t = sh.Tree.from_parents([-1, 0, 0, 1, 1, 2, 3], device="cpu")
    assert t.levels == 4 and t.k == 2
    np.testing.assert_array_equal(t.child.numpy(), [[1, 2], [3, 4], [5, -1], [6, -1], [-1, -1], [-1, -1], [-1, -1]])
    np.testing.assert_array_equal(t.node_kind.numpy(), [0, 0, 0, 0, 1, 1, 1])
    # the complete binary tree in heap order is the special case
    h = sh.Tree.from_parents([-1] + [(c - 1) // 2 for c in range(1, 7)], leaves_sample=False, device="cpu")
    np.testing.assert_array_equal(h.child.numpy()[:3], [[1, 2], [3, 4], [5, 6]])
    assert h.node_kind is None and h.levels == 3
    for bad in ([0, 0], [-1, 1], [-1, 0, 0, 0], [-1, 0, 0, 1, 3, 2]):
        with pytest.raises(ValueError):
            sh.Tree.from_parents(bad, device="cpu")
