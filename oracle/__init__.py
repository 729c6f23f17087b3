"""ctypes front end of the CPU oracle (test infrastructure only).

Nothing under the product package imports this module. Tests, the smoke check
and the benchmark's CPU-baseline leg do. `build()` compiles `ep_oracle.c` with
the host C compiler; no CUDA is involved.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ep_oracle.c")
_LIB = os.path.join(_HERE, "libep_oracle.so")
_lib = None

STATUS_BAD_INDEX = 1


def build(force: bool = False) -> str:
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-ffp-contract=off", "-fPIC", "-shared", "-Wall", "-Wextra",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
    return _lib


def _p(a: np.ndarray):
    return a.ctypes.data_as(ctypes.c_void_p)


@dataclass
class Layout:
    expert_counts: np.ndarray
    expert_offsets: np.ndarray
    rank_rows: np.ndarray
    rank_row_offsets: np.ndarray
    src_row_offsets: np.ndarray     # [R, R+1]
    recv_slot: np.ndarray           # [T, K]
    pair_slot: np.ndarray           # [T, K]
    recv_token: np.ndarray          # [N_recv]
    pair_row: np.ndarray            # [P]
    pair_token: np.ndarray          # [P]
    status: int

    @property
    def n_recv(self) -> int:
        return int(self.rank_row_offsets[-1])

    @property
    def n_pairs(self) -> int:
        return int(self.expert_offsets[-1])


def layout(topk_idx: np.ndarray, E: int, R: int) -> Layout:
    idx = np.ascontiguousarray(topk_idx, dtype=np.int32)
    T, K = idx.shape
    i32 = np.int32
    ec = np.zeros(E, i32); eo = np.zeros(E + 1, i32)
    rr = np.zeros(R, i32); ro = np.zeros(R + 1, i32)
    so = np.zeros((R, R + 1), i32)
    rs = np.full((T, K), -1, i32); ps = np.full((T, K), -1, i32)
    rt = np.full(max(1, T * min(K, R)), -1, i32)
    pr = np.full(max(1, T * K), -1, i32); pt = np.full(max(1, T * K), -1, i32)
    st = np.zeros(1, i32)
    rc = _load().ep_oracle_layout(T, K, E, R, _p(idx), _p(ec), _p(eo), _p(rr), _p(ro), _p(so),
                                  _p(rs), _p(ps), _p(rt), _p(pr), _p(pt), _p(st))
    if rc != 0:
        raise ValueError("oracle layout: shape outside the definitions (need E % R == 0, T % R == 0)")
    return Layout(ec, eo, rr, ro, so, rs, ps, rt[: int(ro[-1])], pr[: int(eo[-1])],
                  pt[: int(eo[-1])], int(st[0]))


def dispatch(x_bits: np.ndarray, recv_slot: np.ndarray, recv_rows: int, fill: int = 0) -> np.ndarray:
    x = np.ascontiguousarray(x_bits, dtype=np.uint16)
    slot = np.ascontiguousarray(recv_slot, dtype=np.int32)
    T, H = x.shape
    K = slot.shape[1]
    recv = np.full((recv_rows, H), fill, dtype=np.uint16)
    rc = _load().ep_oracle_dispatch(T, K, H, _p(x), _p(slot), _p(recv), ctypes.c_int64(recv_rows))
    if rc != 0:
        raise ValueError("oracle dispatch: slot beyond recv_rows")
    return recv


def dispatch_into(x_bits: np.ndarray, recv_slot: np.ndarray, recv: np.ndarray) -> None:
    """`dispatch` for a contiguous range of tokens into a receive buffer the caller owns (the
    benchmark's all-cores leg calls it once per token range; the C function is the same)."""
    assert x_bits.flags.c_contiguous and recv_slot.flags.c_contiguous and recv.flags.c_contiguous
    assert x_bits.dtype == np.uint16 and recv_slot.dtype == np.int32 and recv.dtype == np.uint16
    T, H = x_bits.shape
    rc = _load().ep_oracle_dispatch(T, recv_slot.shape[1], H, _p(x_bits), _p(recv_slot), _p(recv),
                                    ctypes.c_int64(recv.shape[0]))
    if rc != 0:
        raise ValueError("oracle dispatch: slot beyond recv_rows")


def combine_f32_into(out_bits: np.ndarray, slot: np.ndarray, w: np.ndarray, y: np.ndarray) -> None:
    """`combine_f32` for a contiguous range of tokens into rows of `y` the caller owns."""
    assert out_bits.flags.c_contiguous and slot.flags.c_contiguous and w.flags.c_contiguous and y.flags.c_contiguous
    assert out_bits.dtype == np.uint16 and slot.dtype == np.int32 and w.dtype == np.float32 and y.dtype == np.uint16
    T, K = slot.shape
    rc = _load().ep_oracle_combine_f32(T, K, out_bits.shape[1], _p(out_bits), ctypes.c_int64(out_bits.shape[0]),
                                       _p(slot), _p(w), _p(y))
    if rc != 0:
        raise ValueError("oracle combine: slot beyond out rows")


def combine_f32(out_bits: np.ndarray, slot: np.ndarray, w: np.ndarray) -> np.ndarray:
    out = np.ascontiguousarray(out_bits, dtype=np.uint16)
    s = np.ascontiguousarray(slot, dtype=np.int32)
    wt = np.ascontiguousarray(w, dtype=np.float32)
    T, K = s.shape
    H = out.shape[1]
    y = np.zeros((T, H), dtype=np.uint16)
    rc = _load().ep_oracle_combine_f32(T, K, H, _p(out), ctypes.c_int64(out.shape[0]), _p(s), _p(wt), _p(y))
    if rc != 0:
        raise ValueError("oracle combine: slot beyond out rows")
    return y


def combine_f64(out_bits: np.ndarray, slot: np.ndarray, w: np.ndarray) -> np.ndarray:
    out = np.ascontiguousarray(out_bits, dtype=np.uint16)
    s = np.ascontiguousarray(slot, dtype=np.int32)
    wt = np.ascontiguousarray(w, dtype=np.float32)
    T, K = s.shape
    H = out.shape[1]
    y = np.zeros((T, H), dtype=np.float64)
    rc = _load().ep_oracle_combine_f64(T, K, H, _p(out), ctypes.c_int64(out.shape[0]), _p(s), _p(wt), _p(y))
    if rc != 0:
        raise ValueError("oracle combine: slot beyond out rows")
    return y


def group(recv_bits: np.ndarray, pair_row: np.ndarray) -> np.ndarray:
    recv = np.ascontiguousarray(recv_bits, dtype=np.uint16)
    pr = np.ascontiguousarray(pair_row, dtype=np.int32)
    H = recv.shape[1]
    grouped = np.zeros((pr.shape[0], H), dtype=np.uint16)
    rc = _load().ep_oracle_group(ctypes.c_int64(pr.shape[0]), H, _p(recv), ctypes.c_int64(recv.shape[0]), _p(pr),
                                 _p(grouped))
    if rc != 0:
        raise ValueError("oracle group: pair_row outside the receive buffer")
    return grouped


def combine_partial(out_bits, pair_slot, recv_slot, w, recv_rows: int, fill: int = 0):
    """Two-stage combine with per-rank partial outputs; returns (partial [recv_rows,H], y [T,H])."""
    out = np.ascontiguousarray(out_bits, dtype=np.uint16)
    ps = np.ascontiguousarray(pair_slot, dtype=np.int32)
    rs = np.ascontiguousarray(recv_slot, dtype=np.int32)
    wt = np.ascontiguousarray(w, dtype=np.float32)
    T, K = ps.shape
    H = out.shape[1]
    partial = np.full((recv_rows, H), fill, dtype=np.uint16)
    y = np.zeros((T, H), dtype=np.uint16)
    rc = _load().ep_oracle_combine_partial(T, K, H, _p(out), ctypes.c_int64(out.shape[0]), _p(ps), _p(rs), _p(wt),
                                           _p(partial), ctypes.c_int64(recv_rows), _p(y))
    if rc != 0:
        raise ValueError("oracle combine_partial: slot outside its buffer")
    return partial, y


def dense_allgather(x_bits: np.ndarray, R: int) -> np.ndarray:
    x = np.ascontiguousarray(x_bits, dtype=np.uint16)
    T, H = x.shape
    g = np.zeros((R * T, H), dtype=np.uint16)
    _load().ep_oracle_dense_allgather(T, H, R, _p(x), _p(g))
    return g


def dense_reduce_scatter(topk_idx, out_bits, pair_slot, w, E: int, R: int):
    """Dense per-rank buffers ordered by source token and their R-way sum; returns (dense [R*T,H], y [T,H])."""
    idx = np.ascontiguousarray(topk_idx, dtype=np.int32)
    out = np.ascontiguousarray(out_bits, dtype=np.uint16)
    ps = np.ascontiguousarray(pair_slot, dtype=np.int32)
    wt = np.ascontiguousarray(w, dtype=np.float32)
    T, K = idx.shape
    H = out.shape[1]
    dense = np.zeros((R * T, H), dtype=np.uint16)
    y = np.zeros((T, H), dtype=np.uint16)
    rc = _load().ep_oracle_dense_reduce_scatter(T, K, H, E, R, _p(idx), _p(out), ctypes.c_int64(out.shape[0]), _p(ps),
                                                _p(wt), _p(dense), _p(y))
    if rc != 0:
        raise ValueError("oracle dense_reduce_scatter: bad shape or slot")
    return dense, y
