"""Host-side checks of the C ABI: the library loads, exports every declared symbol, and rejects
bad arguments before touching the GPU."""
import ctypes
import os
import re

import pytest

from paper_2506_11498_b200 import build as lib_build
from paper_2506_11498_b200 import lrsa

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def _built():
    lib_build.build()


def declared_symbols():
    text = open(os.path.join(ROOT, "include", "lrsa.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(lrsa_[a-z_0-9]+)\s*\(", text)))


def test_exports_every_declared_symbol():
    names = declared_symbols()
    assert {"lrsa_score_select", "lrsa_attn_fwd", "lrsa_attn_bwd", "lrsa_workspace_bytes"} <= set(names)
    L = ctypes.CDLL(lrsa.LIB_PATH)
    for n in names:
        assert hasattr(L, n), n


def test_status_strings():
    assert lrsa.status_string(0) == "ok"
    assert "workspace" in lrsa.status_string(3)
    assert lrsa.status_string(99) == "unknown status"


GOOD = dict(batch=1, n_q_heads=4, n_kv_heads=2, seq_len=1000, head_dim=128, lag=128, top_k=32, n_sink=4)


@pytest.mark.parametrize("change,status", [
    ({}, 0),
    ({"batch": 0}, 1), ({"n_q_heads": 3}, 1), ({"top_k": 129}, 1), ({"top_k": 0}, 1), ({"n_sink": -1}, 1),
    ({"std_ddof": 2}, 1), ({"n_dense_prev": 2}, 1), ({"softmax_scale": -1.0}, 1),
    ({"head_dim": 96}, 2), ({"chunk": 64}, 2), ({"seq_len": 3}, 2), ({"lag": 40000, "top_k": 5, "seq_len": 100000}, 2),
])
def test_parameter_validation(change, status):
    p = lrsa.Params(**{**GOOD, **change})
    if status == 0:
        a, b, c = lrsa.lrsa_workspace_bytes(p)
        assert a >= 256 and b >= 256 and c >= 256
        assert lrsa.lrsa_num_sel_windows(p) == (1000 - 4) // 128 - 1
    else:
        with pytest.raises(lrsa.LrsaError) as e:
            lrsa.lrsa_workspace_bytes(p)
        assert e.value.status == status


def test_null_and_misaligned_pointers_are_rejected_on_the_host():
    L = lrsa.lib()
    cp = lrsa.Params(**GOOD).c()
    null = ctypes.c_void_p(0)
    fake = ctypes.c_void_p(0x10000)      # never dereferenced: validation fails first
    odd = ctypes.c_void_p(0x10008)
    assert L.lrsa_score_select(ctypes.byref(cp), null, fake, fake, null, fake, 1 << 30, null) == 1
    assert L.lrsa_score_select(ctypes.byref(cp), odd, fake, fake, null, fake, 1 << 30, null) == 1
    assert L.lrsa_score_select(ctypes.byref(cp), fake, fake, fake, null, fake, 16, null) == 3
    assert L.lrsa_attn_fwd(ctypes.byref(cp), fake, fake, fake, fake, null, fake, fake, 1 << 30, null) == 1
    assert L.lrsa_attn_fwd(ctypes.byref(cp), fake, fake, fake, fake, fake, fake, fake, 0, null) == 3
    assert L.lrsa_attn_bwd(ctypes.byref(cp), fake, fake, fake, fake, fake, fake, fake, fake, fake, null, fake,
                           1 << 30, null) == 1
    assert L.lrsa_attn_bwd(ctypes.byref(cp), fake, fake, fake, fake, fake, fake, fake, fake, fake, fake, fake,
                           0, null) == 3
    assert L.lrsa_workspace_status(null, null) == 1


def test_geometry_matches_definition():
    for N, S, L, want in ((32768, 4, 1024, 30), (4096, 16, 512, 6), (9, 1, 2, 3), (300, 4, 256, 0), (516, 4, 256, 1)):
        p = lrsa.Params(1, 1, 1, N, 64, L, 1, S)
        assert lrsa.lrsa_num_sel_windows(p) == want


def test_packed_parameter_validation():
    ok = lrsa.Params(**GOOD, cu_seqlens=(0, 300, 1000))
    assert lrsa.lrsa_num_sel_windows(ok) == ((300 - 4) // 128 - 1) + ((700 - 4) // 128 - 1)
    for bad in ((1, 300, 1000), (0, 300, 900), (0, 300, 300, 1000), (0, 1200, 1000)):
        with pytest.raises(lrsa.LrsaError) as e:
            lrsa.lrsa_num_sel_windows(lrsa.Params(**GOOD, cu_seqlens=bad))
        assert e.value.status == 1
    assert lrsa.lrsa_num_sel_windows(lrsa.Params(**{**GOOD, "chunk": 256})) == (1000 - 4) // 128 - 1


def test_o_residual_must_be_16_byte_aligned():
    import ctypes
    out = ctypes.c_int32(0)
    cp = lrsa.Params(**GOOD).c()
    cp.o_residual = 4096
    assert lrsa.lib().lrsa_num_sel_windows(ctypes.byref(cp), ctypes.byref(out)) == 0
    cp.o_residual = 4096 + 8
    assert lrsa.lib().lrsa_num_sel_windows(ctypes.byref(cp), ctypes.byref(out)) == 1
