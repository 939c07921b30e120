"""Host-side checks of the C-ABI library that need no GPU: it loads, exports every symbol the
header declares, validates arguments, sizes workspaces and evaluates the normal quantile."""
import ctypes as C
import os
import re

import numpy as np
import pytest

from oracle import vattn_oracle as O
from paper_2510_05688_b200 import binding as vb
from paper_2510_05688_b200 import build as vbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    vbuild.build()


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "vattn.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(vattn_[a-z_]+)\s*\(", header))
    assert declared == set(vb.EXPORTS)
    L = vb.lib()
    for name in declared:
        assert hasattr(L, name), name


def shape(**kw):
    d = dict(batch=2, num_q_heads=8, num_kv_heads=2, head_dim=128, block_size=16, max_blocks_per_seq=8,
             num_blocks=20, max_seq_len=128, dtype=vb.DTYPE_BF16)
    d.update(kw)
    return vb.Shape(d["batch"], d["num_q_heads"], d["num_kv_heads"], d["head_dim"], d["block_size"],
                    d["max_blocks_per_seq"], d["num_blocks"], d["max_seq_len"], d["dtype"], 0, 0, 0)


def create(**kw):
    h = C.c_void_p()
    s = shape(**kw)
    return vb.lib().vattn_plan_create(C.byref(s), C.byref(h)), h


def test_plan_create_validates_shape():
    rc, h = create()
    assert rc == vb.OK and h.value
    vb.lib().vattn_plan_destroy(h)
    assert create(num_q_heads=7)[0] == vb.ERR_INVALID_ARG          # Hq % Hkv != 0
    assert create(batch=0)[0] == vb.ERR_INVALID_ARG
    assert create(head_dim=96)[0] == vb.ERR_UNSUPPORTED
    assert create(block_size=32)[0] == vb.ERR_UNSUPPORTED
    assert create(dtype=5)[0] == vb.ERR_UNSUPPORTED
    assert create(max_seq_len=129)[0] == vb.ERR_INVALID_ARG        # exceeds max_blocks_per_seq * 16
    assert create(max_seq_len=1 << 20, max_blocks_per_seq=1 << 16)[0] == vb.ERR_UNSUPPORTED
    assert create(batch=1537)[0] == vb.ERR_UNSUPPORTED             # bf16: per-row tables of the score kernel
    rc, h = create(batch=1536)
    assert rc == vb.OK
    vb.lib().vattn_plan_destroy(h)
    rc, h = create(batch=4000, dtype=vb.DTYPE_FP32)
    assert rc == vb.OK
    vb.lib().vattn_plan_destroy(h)
    assert vb.lib().vattn_plan_create(None, None) == vb.ERR_INVALID_ARG


def test_workspace_and_argument_errors_without_gpu():
    L = vb.lib()
    rc, h = create()
    need = L.vattn_workspace_bytes(h)
    assert need > 0 and need % 256 == 0
    # bigger problems need more scratch
    rc2, h2 = create(batch=4)
    assert L.vattn_workspace_bytes(h2) > need
    fake = C.c_void_p(0x10000)          # never dereferenced: every call below fails validation first
    assert L.vattn_decode(h, fake, fake, fake, fake, fake, 4, 4, 4, 0.05, 0.05, 0, fake, None) == vb.ERR_WORKSPACE
    assert L.vattn_set_workspace(h, None, need) == vb.ERR_WORKSPACE
    assert L.vattn_set_workspace(h, C.c_void_p(0x10010), need) == vb.ERR_WORKSPACE      # misaligned
    assert L.vattn_set_workspace(h, fake, need - 1) == vb.ERR_WORKSPACE                 # too small
    assert L.vattn_set_workspace(h, fake, need) == vb.OK
    bad = [dict(eps=0.0), dict(eps=1.0), dict(delta=0.0), dict(delta=1.5), dict(sink=-1), dict(window=-1), dict(k=-1)]
    for kw in bad:
        a = dict(sink=4, window=4, k=4, eps=0.05, delta=0.05)
        a.update(kw)
        rc = L.vattn_decode(h, fake, fake, fake, fake, fake, a["sink"], a["window"], a["k"], a["eps"], a["delta"], 0,
                            fake, None)
        assert rc == vb.ERR_INVALID_ARG, kw
    assert L.vattn_decode(h, None, fake, fake, fake, fake, 4, 4, 4, 0.05, 0.05, 0, fake, None) == vb.ERR_INVALID_ARG
    assert L.vattn_decode(h, C.c_void_p(0x10004), fake, fake, fake, fake, 4, 4, 4, 0.05, 0.05, 0, fake, None) \
        == vb.ERR_INVALID_ARG
    assert L.vattn_dense_decode(h, fake, fake, None, fake, fake, fake, None) == vb.ERR_INVALID_ARG
    p = vb.Params()
    p.base_rate = 1.5
    assert L.vattn_set_params(h, C.byref(p)) == vb.ERR_INVALID_ARG
    p.base_rate, p.mode = 0.05, 3
    assert L.vattn_set_params(h, C.byref(p)) == vb.ERR_INVALID_ARG
    p.mode, p.gather_mode = 1, 2
    assert L.vattn_set_params(h, C.byref(p)) == vb.ERR_INVALID_ARG
    p.gather_mode = 1
    assert L.vattn_set_params(h, C.byref(p)) == vb.OK
    assert L.vattn_set_params(h, None) == vb.OK
    assert L.vattn_strerror(vb.ERR_WORKSPACE).decode().startswith("workspace")
    assert L.vattn_set_stop_after(h, -1) == vb.ERR_INVALID_ARG
    assert L.vattn_set_stop_after(h, len(vb.KERNEL_NAMES) + 1) == vb.ERR_INVALID_ARG
    assert L.vattn_set_stop_after(h, 1) == vb.OK and L.vattn_set_stop_after(h, 0) == vb.OK
    L.vattn_plan_destroy(h)
    L.vattn_plan_destroy(h2)


def test_host_normal_quantile_matches_oracle_quantile():
    # the budget ceil() must see the same z on both sides: agree to a few ulp over the delta grid
    for delta in (0.01, 0.05, 0.1, 0.2, 0.3, float(np.float32(0.05)), 1e-6, 0.999):
        for j in range(1, 17):
            x = delta * j / 16.0
            a, b = vb.normal_quantile(x), O.z_of(x)
            assert abs(a - b) <= 4e-15 * max(1.0, abs(b)), (x, a, b)
    assert np.isnan(vb.normal_quantile(0.0)) and np.isnan(vb.normal_quantile(2.0))


def test_binding_fails_loudly_without_library(monkeypatch):
    monkeypatch.setattr(vb, "_lib", None)
    monkeypatch.setattr(vb, "LIB_PATH", "/nonexistent/libvattn.so")
    with pytest.raises(RuntimeError, match="no CPU fallback"):
        vb.lib()
