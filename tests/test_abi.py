"""The C-ABI library loads without a GPU and exports every function include/samdraft.h declares;
the binding declares a signature for each of them."""
import ctypes
import os
import re

import pytest

from paper_2411_10666_b200 import _build, binding as sd

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared():
    text = open(os.path.join(ROOT, "include", "samdraft.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(sam_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported_and_bound():
    names = _declared()
    assert len(names) >= 20
    L = ctypes.CDLL(_build.build())
    for n in names:
        assert hasattr(L, n), "missing export: " + n
        assert n in sd.SIGNATURES, "binding lacks: " + n
    assert sorted(sd.SIGNATURES) == names


def test_host_side_calls_need_no_gpu():
    L = sd.lib()
    assert b"samdraft" in L.sam_version()
    assert L.sam_strerror(0) == b"ok" and L.sam_strerror(-1) == b"invalid argument"
    o = sd.BatchOpts(64, 3072, 32, 0, 1, 32000, 0, 0, 0)
    n = sd.sam_batch_workspace_bytes(o)
    assert n > 64 * 3072 * 4 and n % 256 == 0
    for bad in (sd.BatchOpts(0, 10, 8, 0, 1, 5, 0, 0, 0), sd.BatchOpts(4, 10, 200, 0, 1, 5, 0, 0, 0),
                sd.BatchOpts(4, 10, 8, -1, 1, 5, 0, 0, 0), sd.BatchOpts(4, 10, 8, 0, 1, 5, 0, 5000, 0),
                sd.BatchOpts(4, 100000, 8, 0, 1, 5, 0, 4096, 0)):
        with pytest.raises(sd.SamError):
            sd.sam_batch_workspace_bytes(bad)
    # null handles are rejected, not dereferenced
    assert L.sam_step(None, None, 1, None, 1, None, None, None, None, None, None, None) == -1
    assert L.sam_static_info(None, None) == -1
    L.sam_static_destroy(None)
    L.sam_batch_destroy(None)


def test_package_fails_loudly_without_cuda():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    import paper_2411_10666_b200 as P
    with pytest.raises(RuntimeError):
        P.Batch(None, 2, 16, vocab=10)
