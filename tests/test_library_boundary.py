"""The C-ABI boundary without a GPU: the library loads, exports every symbol the header
declares, and rejects bad arguments on the host before touching the device."""
import ctypes
import os
import re

import numpy as np
import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    from paper_2512_16273_b200 import build
    build.build()
    from paper_2512_16273_b200 import tslt
    return tslt.lib()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "tslt.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(tslt_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(lib):
    names = declared_symbols()
    assert {"tslt_sparsify", "tslt_verify", "tslt_tree_verify", "tslt_version"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name
    from paper_2512_16273_b200 import tslt
    assert sorted(tslt.EXPORTS) == names


def test_version_and_status_strings(lib):
    from paper_2512_16273_b200 import tslt
    assert tslt.version() >= 100
    seen = {tslt.status_string(s) for s in (0, -1, -2, -3, -4, -5, -99)}
    assert len(seen) == 7 and tslt.status_string(0) == "ok"


def test_workspace_queries_are_host_only(lib):
    from paper_2512_16273_b200 import tslt
    a = tslt.sparsify_workspace_bytes(2048, 256000, 64, 1)
    b = tslt.sparsify_workspace_bytes(4, 32000, 64, 1)
    assert a % 256 == 0 and b % 256 == 0 and a > 0 and b > 0
    v = tslt.verify_workspace_bytes(256, 8, 256000, 64)
    # one (max, sum) pair per 2 KB chunk of every target row, plus a small header
    assert v >= 256 * 9 * (256000 * 4 // 2048) * 8
    assert tslt.tree_verify_workspace_bytes(16, 40, 151936, 64) > 0
    with pytest.raises(tslt.TsltError):
        tslt.sparsify_workspace_bytes(1, 100, 101, 1)
    with pytest.raises(tslt.TsltError):
        tslt.tree_verify_workspace_bytes(1, 5000, 1000, 8)


def test_bad_arguments_rejected_before_any_launch(lib):
    from paper_2512_16273_b200 import tslt
    fake = ctypes.c_void_p(0x1000)  # 16-byte aligned, never dereferenced on these paths
    ws = ctypes.c_void_p(0x10000)
    call = lambda **kw: lib.tslt_sparsify(kw.get("logits", fake), kw.get("dtype", 1), 1, 1, kw.get("V", 1000),
                                          kw.get("stride", 1000), kw.get("k", 8), kw.get("top_p", 1.0),
                                          kw.get("T", 1.0), 1, fake, fake, fake, fake, fake, None, None,
                                          kw.get("ws", ws), kw.get("ws_bytes", 1 << 30), None)
    assert call(dtype=7) == tslt.ERR_UNSUPPORTED
    assert call(k=0) == tslt.ERR_INVALID_ARG
    assert call(k=1001) == tslt.ERR_INVALID_ARG
    assert call(V=4000, stride=4000, k=2000) == tslt.ERR_UNSUPPORTED
    assert call(top_p=0.0) == tslt.ERR_INVALID_ARG
    assert call(T=-1.0) == tslt.ERR_INVALID_ARG
    assert call(logits=None) == tslt.ERR_INVALID_ARG
    assert call(logits=ctypes.c_void_p(0x1004)) == tslt.ERR_INVALID_ARG     # misaligned base
    assert call(V=1001, stride=1001) == tslt.ERR_INVALID_ARG                # row stride not 16-byte multiple
    assert call(stride=992) == tslt.ERR_INVALID_ARG                         # stride shorter than a row
    assert call(ws=ctypes.c_void_p(0x10010)) == tslt.ERR_INVALID_ARG        # workspace not 256-byte aligned
    assert call(ws_bytes=16) == tslt.ERR_WORKSPACE
    # zero rows is a no-op
    assert lib.tslt_sparsify(None, 1, 0, 5, 1000, 1000, 8, 1.0, 1.0, 1, None, None, None, None, None, None, None,
                             None, 0, None) == tslt.OK


def test_tree_structure_validation_on_host(lib):
    from paper_2512_16273_b200 import tslt
    fake = ctypes.c_void_p(0x1000)

    def tree(parent, ndr, max_depth, B=0):
        par = np.asarray(parent, np.int32)
        nd = np.asarray(ndr, np.int32)
        M = int((nd >= 0).sum())
        return lib.tslt_tree_verify(fake, 1, B, len(parent), 1000, 1000, par.ctypes.data_as(ctypes.c_void_p),
                                    nd.ctypes.data_as(ctypes.c_void_p), M, 8, fake, fake, fake, fake, 1.0, 1.0,
                                    fake, fake, max_depth, fake, fake, fake, ctypes.c_void_p(0x10000), 1 << 30, None)

    assert tree([-1, 0, 0, 1, 1], [0, 1, -1, -1, -1], 2) == tslt.OK           # B = 0: validated, nothing launched
    assert tree([0, 0, 0], [0, -1, -1], 2) == tslt.ERR_INVALID_ARG            # root must have parent -1
    assert tree([-1, 2, 0], [0, -1, 1], 2) == tslt.ERR_INVALID_ARG            # parent after child
    assert tree([-1, 0, 1], [0, 1, -1], 1) == tslt.ERR_INVALID_ARG            # deeper than max_depth
    assert tree([-1, 0, 0], [0, 0, -1], 2) == tslt.ERR_INVALID_ARG            # leaf with a draft row
    assert tree([-1, 0, 0], [-1, -1, -1], 2) == tslt.ERR_INVALID_ARG          # internal node without one
    assert tree([-1, 0, 0], [5, -1, -1], 2) == tslt.ERR_INVALID_ARG           # draft row out of range


def test_binding_refuses_cpu_tensors(lib):
    import torch
    from paper_2512_16273_b200 import tslt
    with pytest.raises(ValueError):
        tslt.sparsify(torch.zeros(2, 100), 4, 1.0, 1.0, torch.zeros(2, 1))


def test_payload_accounting_matches_paper_formula():
    """Section 2.2: one distribution costs |V| (b_prob + b_idx) bits with b_idx = ceil(log2 |V|);
    the sparse payload replaces |V| by the retained count."""
    from paper_2512_16273_b200 import tslt
    words, entry_bits = tslt.payload_words(320, 32000, tslt.PROB_F16)   # host-only query of the C ABI
    assert entry_bits == 16 + 15 and 320 * entry_bits == 9920
    assert words == 1 + (320 * entry_bits + 31) // 32
