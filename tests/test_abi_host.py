"""Host-side checks that need no GPU: the library loads, exports every symbol the headers declare,
and rejects bad arguments before touching the device."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2509_23472_b200 import binding as B

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def lib():
    entry.build()
    return B.lib()


def _declared():
    names = set()
    for h in sorted(os.listdir(os.path.join(ROOT, "include"))):
        text = open(os.path.join(ROOT, "include", h)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(loract_[a-z0-9_]+)\s*\(", text))
    return names


def test_every_declared_symbol_is_exported(lib):
    declared = _declared()
    assert {"loract_compress", "loract_reconstruct", "loract_weight_grad", "loract_compress_prenorm",
            "loract_sample_indices", "loract_workspace_bytes"} <= declared
    raw = ctypes.CDLL(B.LIB_PATH)
    for name in declared:
        assert hasattr(raw, name), name
    assert set(B.EXPORTS) | set(B.DEBUG_EXPORTS) == declared


def test_descriptor_layout_matches_the_header():
    assert ctypes.sizeof(B.Desc) == 56
    assert B.Desc.rank.offset == 24 and B.Desc.seed.offset == 40 and B.Desc.call_id.offset == 48


def _desc(**kw):
    base = dict(n_tokens=1024, d=512, ldx=512, rank=64, power_iters=0, dtype=B.BF16, reserved=0, seed=1, call_id=2)
    base.update(kw)
    return B.Desc(*[base[k] for k, _ in B.Desc._fields_])


def test_workspace_query_and_invalid_descriptors(lib):
    assert B.workspace_bytes(_desc()) > 0
    assert B.workspace_bytes(_desc(dtype=B.F32)) > 0
    assert B.workspace_bytes(_desc(power_iters=2)) > 0
    bad = [dict(rank=0), dict(rank=24), dict(rank=528), dict(rank=2048, n_tokens=4096, d=4096),
           dict(n_tokens=32), dict(d=32, ldx=32), dict(ldx=256), dict(dtype=7), dict(reserved=1),
           dict(d=516, ldx=516), dict(power_iters=-1), dict(power_iters=9)]
    for kw in bad:
        assert B.workspace_bytes(_desc(**kw)) == 0, kw
    # workspace grows with the problem
    assert B.workspace_bytes(_desc(n_tokens=4096)) > B.workspace_bytes(_desc())


def test_bad_arguments_return_codes_and_launch_nothing(lib):
    before = B.kernel_launch_count()
    d = _desc()
    null = ctypes.c_void_p(0)
    one = ctypes.c_void_p(4096)       # never dereferenced: the checks below fail first
    odd = ctypes.c_void_p(4096 + 2)
    assert lib.loract_compress(ctypes.byref(d), null, one, one, null, one, 1 << 30, null) == 1
    assert lib.loract_compress(ctypes.byref(d), odd, one, one, null, one, 1 << 30, null) == 3
    assert lib.loract_compress(ctypes.byref(d), one, one, one, null, one, 16, null) == 4
    assert lib.loract_compress(ctypes.byref(_desc(rank=24)), one, one, one, null, one, 1 << 30, null) == 1
    assert lib.loract_compress(ctypes.byref(_desc(power_iters=9)), one, one, one, null, one, 1 << 30, null) == 2
    assert lib.loract_compress(ctypes.byref(_desc(d=516, ldx=516)), one, one, one, null, one, 1 << 30, null) == 3
    assert lib.loract_reconstruct(ctypes.byref(d), one, null, one, null) == 1
    assert lib.loract_weight_grad(ctypes.byref(d), one, one, one, 0, 16, one, 0, one, 1 << 30, null) == 1
    assert lib.loract_weight_grad(ctypes.byref(d), one, one, one, 300, 304, one, 0, one, 1 << 30, null) == 1
    assert lib.loract_weight_grad(ctypes.byref(d), one, one, one, 16, 12, one, 0, one, 1 << 30, null) == 1
    assert lib.loract_weight_grad(ctypes.byref(d), one, one, one, 16, 20, one, 0, one, 1 << 30, null) == 3
    assert lib.loract_weight_grad(ctypes.byref(d), one, one, one, 16, 16, one, 0, one, 64, null) == 4
    assert lib.loract_compress_prenorm(ctypes.byref(d), one, one, null, 1e-5, 5, null, one, null, one, one, null,
                                       one, 1 << 30, null) == 1
    assert lib.loract_compress_prenorm(ctypes.byref(d), one, one, null, 1e-5, B.NORM_LAYER, null, one, null, one,
                                       one, null, one, 1 << 30, null) == 1   # LayerNorm needs `mean`
    assert lib.loract_sample_indices(ctypes.byref(d), null, one, 256, null) == 1
    assert lib.loract_rsvd_workspace_bytes(ctypes.byref(d), 4) == 0          # rank + oversample not a multiple of 16
    assert lib.loract_rsvd_workspace_bytes(ctypes.byref(d), 16) > 0
    assert B.kernel_launch_count() == before
    assert B.status_string(4) == "workspace too small"


def test_binding_refuses_cpu_tensors(lib):
    import torch
    with pytest.raises(RuntimeError):
        B.compress(torch.zeros(64, 64, dtype=torch.bfloat16), 16)
