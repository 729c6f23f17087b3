"""The C-ABI library loads and exports everything include/ep.h declares; host-side
argument checks answer before anything touches a GPU."""
import ctypes
import os
import re

import pytest

import __graft_entry__ as entry
from paper_2609_40093_b200 import ep

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    entry.build()


def _declared():
    text = open(os.path.join(ROOT, "include", "ep.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ep_[a-z_0-9]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    L = ep.lib()
    names = _declared()
    assert set(names) == set(ep.EXPORTS), (names, ep.EXPORTS)
    for n in names:
        assert getattr(L, n) is not None


def test_host_side_validation_needs_no_gpu():
    L = ep.lib()
    ok = ep._shape(64, 2, 256, 8, 2)
    assert L.ep_layout_workspace_bytes(ctypes.byref(ok)) > 0
    assert L.ep_host_step_arena_bytes(ctypes.byref(ok)) > 64 * 256 * 2
    bad_shapes = [
        ep._shape(64, 0, 256, 8, 2),     # K < 1
        ep._shape(64, 33, 256, 64, 2),   # K > 32
        ep._shape(64, 2, 256, 9, 2),     # E % R != 0
        ep._shape(63, 2, 256, 8, 2),     # T % R != 0
        ep._shape(64, 2, 252, 8, 2),     # H % 8 != 0
        ep._shape(-2, 2, 256, 8, 2),     # T < 0
        ep._shape(64, 2, 256, 8192, 2),  # E too large
        ep._shape(130, 2, 256, 130, 65), # R too large
    ]
    for s in bad_shapes:
        assert L.ep_dispatch(ctypes.byref(s), None, None, None, 0, None, None) == -2
        assert L.ep_layout_workspace_bytes(ctypes.byref(s)) == 0 or s.hidden == 252
    assert L.ep_dispatch(None, None, None, None, 0, None, None) == -1
    assert L.ep_dispatch(ctypes.byref(ok), None, None, None, 0, None, None) == -1
    assert L.ep_combine(ctypes.byref(ok), None, 0, None, None, None, None, None) == -1
    assert L.ep_layout(ctypes.byref(ok), None, None, None, 0, None) == -1
    assert L.ep_dispatch(ctypes.byref(ok), ctypes.c_void_p(8), ctypes.c_void_p(16), ctypes.c_void_p(16), 4, None, None) == -2
    assert b"NULL" in L.ep_strerror(-1) and L.ep_strerror(0) == b"ok"
    assert L.ep_launch_count() == 0 or L.ep_launch_count() > 0


def test_binding_rejects_wrong_dtypes_and_strided_tensors():
    import torch
    x = torch.zeros(4, 16, dtype=torch.float32)
    slot = torch.zeros(4, 2, dtype=torch.int32)
    with pytest.raises(TypeError, match="bfloat16"):
        ep.ep_dispatch(x, slot, x, 4, 2)
    xb = torch.zeros(4, 32, dtype=torch.bfloat16)[:, ::2]
    with pytest.raises(ValueError, match="contiguous"):
        ep.ep_dispatch(xb, slot, torch.zeros(8, 16, dtype=torch.bfloat16), 4, 2)
    with pytest.raises(TypeError, match="int32"):
        ep.ep_layout(torch.zeros(4, 2, dtype=torch.int64), 4, 2)


def test_binding_refuses_to_run_without_the_library(monkeypatch, tmp_path):
    monkeypatch.setattr(ep, "_lib", None)
    monkeypatch.setattr(ep, "_LIB_PATH", str(tmp_path / "absent.so"))
    with pytest.raises(RuntimeError, match="missing"):
        ep.lib()


def test_host_staged_calls_check_their_segment_tables_before_touching_a_gpu():
    """ep_host_combine / ep_host_dispatch_per_sender validate the host copy of src_row_offsets (rows abut,
    segments run forwards, the end fits the buffers) and their flags before any CUDA call is made."""
    import numpy as np
    L = ep.lib()
    R, T, K, H, E = 4, 64, 2, 64, 8
    shape = ep._shape(T, K, H, E, R)
    p = ctypes.c_void_p(256)                                  # never dereferenced: every case fails on the host
    good = np.zeros((R, R + 1), dtype=np.int32)
    rows = np.arange(R * R + 1, dtype=np.int32) * 3           # 3 rows per segment
    for r in range(R):
        good[r] = rows[r * R:r * R + R + 1]

    def combine(so, cap=int(good[-1, -1]), flags=0, bounce=p):
        return L.ep_host_combine(ctypes.byref(shape), p, 128, p, p, p, so.ctypes.data_as(ctypes.c_void_p), p, p, cap,
                                 bounce, 0, p, flags, None, None, None, None)

    def per_sender(so, cap=int(good[-1, -1]), flags=0, timeout=0, sender_flags=None):
        return L.ep_host_dispatch_per_sender(ctypes.byref(shape), p, p, p, so.ctypes.data_as(ctypes.c_void_p), p, p, cap,
                                             p, 0, p, 128, sender_flags, 1, timeout, None, None, flags, None, None,
                                             None, None, None)

    backwards = good.copy()
    backwards[1, 2] = backwards[1, 1] - 1
    gap = good.copy()
    gap[2:] += 1                                              # rank 2 does not start where rank 1 ends
    shifted = good + 1                                        # first row is not 0
    for call in (combine, per_sender):
        assert call(backwards) == -2 and call(gap) == -2 and call(shifted) == -2
        assert call(good, cap=int(good[-1, -1]) - 1) == -3    # buffers one row short
        assert call(good, flags=8) == -2                      # unknown flag bit
    assert combine(good, bounce=None) == -1
    assert per_sender(good, sender_flags=p, timeout=0) == -2                  # a flag wait needs a time limit ...
    assert per_sender(good, sender_flags=p, timeout=3_000_000_000) == -2      # ... of at most two seconds
    assert L.ep_layout_dispatch(ctypes.byref(ep._shape(T, K, 60, E, R)), p, p, None, p, 16, p, 8, None, None) == -2
    assert L.ep_layout_dispatch(ctypes.byref(shape), None, p, None, p, 16, p, 8, None, None) == -1
    big = ep._shape(4096, 8, 64, 128, 8)                     # more than 1024 tokens: a second stream needs two workspaces
    one = L.ep_layout_workspace_bytes(ctypes.byref(big))
    lay = ep._Layout(*[256] * 11)
    assert L.ep_layout_dispatch(ctypes.byref(big), p, p, ctypes.byref(lay), p, one, p, 8, None, p) == -3


def test_workspace_sizes_follow_the_launch_plan():
    """One CTA up to 256 tokens (no scratch), then one row of E+R+1 counters per CTA of 256 tokens, at most 128 CTAs."""
    ws = ep.ep_layout_workspace_bytes
    assert ws(64, 2, 8, 2) == 16 and ws(256, 8, 256, 8) == 16
    assert ws(264, 8, 256, 8) == 2 * (256 + 8 + 1) * 4 and ws(1024, 8, 256, 8) == 4 * (256 + 8 + 1) * 4
    assert ws(2048, 8, 256, 8) == 8 * (256 + 8 + 1) * 4       # 8 CTAs of 8 warps
    assert ws(8192, 8, 256, 8) == 32 * (256 + 8 + 1) * 4
    assert ws(65536, 8, 256, 8) == 128 * (256 + 8 + 1) * 4    # 128 CTAs, two 32-token groups per warp
    assert ws(32768, 2, 4096, 64) > ep.ep_layout_static_scratch_bytes()
