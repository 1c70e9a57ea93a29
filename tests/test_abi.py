"""CPU-side checks of the boundary: the library loads, exports every declared symbol, validates arguments on
the host and refuses to run without a device (no fallback path)."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import tr_oracle as orc

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def tr():
    from paper_2408_08696_b200 import build
    build.build()
    from paper_2408_08696_b200 import binding
    return binding


def _declared(header):
    text = open(os.path.join(ROOT, "include", header)).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(trs?_[a-z0-9_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported(tr):
    names = _declared("tr.h")
    assert {"tr_init", "tr_build_tree", "tr_tree_attention", "tr_verify_update"} <= set(names)
    for n in names:
        assert hasattr(tr.lib, n), n
    for n in _declared("tr_synth.h"):
        assert hasattr(tr.lib_synth, n), n


def test_template_matches_checker(tr):
    for b, n in (((8, 4, 3, 2, 2, 1), 80), ((4, 2, 1), 15), ((3,), 7), ((10, 10), 128), ((1, 1, 1), 3)):
        p, r = tr.tr_template_from_branching(b, n)
        po, ro = orc.template_from_branching(b, n)
        assert p.tolist() == po.tolist() and r.tolist() == ro.tolist()


def test_host_side_argument_errors(tr):
    p, r = tr.tr_template_from_branching((4, 2, 1), 15)
    P32 = C.POINTER(C.c_int32)
    h = C.c_void_p()

    def init(vocab, k, parent, rank, n, batch=1, device=0):
        parent = np.ascontiguousarray(parent, dtype=np.int32)
        rank = np.ascontiguousarray(rank, dtype=np.int32)
        return tr.lib.tr_init(C.byref(h), vocab, k, parent.ctypes.data_as(P32), rank.ctypes.data_as(P32), n, batch, device)

    assert init(4, 8, p, r, 15) == tr.TR_ERR_INVALID_ARG          # vocab < k
    assert init(100, 0, p, r, 15) == tr.TR_ERR_INVALID_ARG
    assert init(100, 17, p, r, 15) == tr.TR_ERR_INVALID_ARG
    assert init(100, 8, p, r, 15, batch=0) == tr.TR_ERR_INVALID_ARG
    assert init(100, 8, p, r, 15, batch=4370) == tr.TR_ERR_UNSUPPORTED    # batch * nodes = 65550 logits rows: a grid's y limit
    assert init(100, 8, p, r, 0) == tr.TR_ERR_TEMPLATE
    assert init(100, 8, p, r, 129) == tr.TR_ERR_TEMPLATE
    bad = p.copy(); bad[3] = 7
    assert init(100, 8, bad, r, 15) == tr.TR_ERR_TEMPLATE         # parent after child
    bad = p.copy(); bad[0] = 0
    assert init(100, 8, bad, r, 15) == tr.TR_ERR_TEMPLATE
    bad = r.copy(); bad[2] = 8
    assert init(100, 8, p, bad, 15) == tr.TR_ERR_TEMPLATE         # rank >= k
    bad = np.array([-1, 0, 1, 0], dtype=np.int32)                 # depth decreases: not layer order
    assert init(100, 8, bad, np.zeros(4, np.int32), 4) == tr.TR_ERR_TEMPLATE
    assert tr.lib.tr_build_tree(None, None, None, None) == tr.TR_ERR_INVALID_ARG
    assert tr.lib.tr_tree_attention(None, None, None) == tr.TR_ERR_INVALID_ARG
    assert tr.lib.tr_verify_update(None, None, None, None, None) == tr.TR_ERR_INVALID_ARG
    assert tr.lib.tr_destroy(None) == tr.TR_ERR_INVALID_ARG
    assert tr.lib.tr_matrix_fill(None, 0, 0, None) == tr.TR_ERR_INVALID_ARG
    assert tr.lib.tr_set_update_rule(None, 0, 0) == tr.TR_ERR_INVALID_ARG
    assert tr.lib.tr_status_string(tr.TR_ERR_TEMPLATE) == b"malformed tree template"
    with pytest.raises(tr.TrError):
        tr.tr_template_from_branching((4, 2, 1), 1000)


def test_no_fallback_without_a_device(tr):
    import torch
    if torch.cuda.is_available():
        pytest.skip("a device is present")
    p, r = tr.tr_template_from_branching((4, 2, 1), 15)
    with pytest.raises(tr.TrError) as e:
        tr.tr_init(1000, 8, p, r)
    assert e.value.status == tr.TR_ERR_CUDA
