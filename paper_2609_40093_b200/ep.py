"""Python binding of the C-ABI CUDA library (`include/ep.h`): argument marshalling only.

Every function takes torch tensors (device memory, or pinned host memory where
the header says so), passes their addresses and the current CUDA stream to the
library, and raises `EPError` on a non-zero return. Nothing is computed here
and there is no fallback: if the library has not been built, the first call fails.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libep_b200.so")
_lib = None

STATUS_BAD_INDEX = 1
STATUS_CAPACITY = 2
STATUS_TIMEOUT = 4
PROBE_READ, PROBE_WRITE, PROBE_COPY, PROBE_MEMCPY = 0, 1, 2, 3
HOST_DUPLEX, HOST_PER_PEER, HOST_LOCAL_ON_DEVICE = 1, 2, 4

EXPORTS = [
    "ep_layout_workspace_bytes", "ep_layout", "ep_layout_ranks", "ep_layout_pairs", "ep_layout_static", "ep_layout_static_scratch_bytes", "ep_layout_dispatch", "ep_dispatch", "ep_combine", "ep_group",
    "ep_combine_partial", "ep_dense_allgather", "ep_dense_reduce_scatter",
    "ep_host_roundtrip", "ep_host_dispatch_per_sender", "ep_host_combine", "ep_wait_senders", "ep_post_flags", "ep_host_step_pipelined",
    "ep_dispatch_copy_engine", "ep_host_step_arena_bytes", "ep_host_step", "ep_status",
    "ep_probe_bandwidth", "ep_launch_count", "ep_strerror", "ep_last_cuda_error",
]


class EPError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().ep_strerror(code).decode()
        cuda = lib().ep_last_cuda_error() if code == -4 else 0
        super().__init__(f"{where}: {msg} (code {code}" + (f", cudaError {cuda})" if cuda else ")"))


class _Shape(ctypes.Structure):
    _fields_ = [("num_tokens", ctypes.c_int32), ("top_k", ctypes.c_int32), ("hidden", ctypes.c_int32),
                ("num_experts", ctypes.c_int32), ("num_ranks", ctypes.c_int32)]


_LAYOUT_FIELDS = ["expert_counts", "expert_offsets", "rank_rows", "rank_row_offsets", "src_row_offsets",
                  "recv_slot", "pair_slot", "recv_token", "pair_row", "pair_token", "status"]


class _Layout(ctypes.Structure):
    _fields_ = [(f, ctypes.c_void_p) for f in _LAYOUT_FIELDS]


def lib() -> ctypes.CDLL:
    """Opens the CUDA library; a missing build is an error, never a fallback."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise RuntimeError(f"{_LIB_PATH} is missing: build it with `python -m paper_2609_40093_b200.build`")
        L = ctypes.CDLL(_LIB_PATH)
        vp, i32, i64, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_int64, ctypes.c_size_t
        sp = ctypes.POINTER(_Shape)
        L.ep_layout_workspace_bytes.restype = sz
        L.ep_layout_workspace_bytes.argtypes = [sp]
        L.ep_layout.argtypes = [sp, vp, ctypes.POINTER(_Layout), vp, sz, vp]
        L.ep_layout_ranks.argtypes = [sp, vp, ctypes.POINTER(_Layout), vp, sz, vp]
        L.ep_layout_pairs.argtypes = [sp, vp, ctypes.POINTER(_Layout), vp, sz, vp]
        L.ep_layout_ranks.restype = i32
        L.ep_layout_pairs.restype = i32
        L.ep_layout_static.argtypes = [sp, vp, ctypes.POINTER(_Layout), vp]
        L.ep_layout_static.restype = i32
        L.ep_layout_static_scratch_bytes.restype = sz
        L.ep_dispatch.argtypes = [sp, vp, vp, vp, i64, vp, vp]
        L.ep_layout_dispatch.argtypes = [sp, vp, vp, ctypes.POINTER(_Layout), vp, sz, vp, i64, vp, vp]
        L.ep_layout_dispatch.restype = i32
        L.ep_combine.argtypes = [sp, vp, i64, vp, vp, vp, vp, vp]
        L.ep_group.argtypes = [sp, vp, i64, vp, vp, vp, i64, vp, vp]
        L.ep_combine_partial.argtypes = [sp, vp, i64, vp, vp, vp, vp, i64, vp, vp, vp]
        L.ep_dense_allgather.argtypes = [sp, vp, vp, vp]
        L.ep_dense_reduce_scatter.argtypes = [sp, vp, vp, i64, vp, vp, vp, vp, vp, vp]
        L.ep_host_roundtrip.argtypes = [sp, vp, vp, vp, vp, i64, vp, i32, vp, i32, i32, vp, vp, vp, vp]
        L.ep_host_dispatch_per_sender.argtypes = [sp, vp, vp, vp, vp, vp, vp, i64, vp, i32, vp, i64, vp, ctypes.c_uint32,
                                                  ctypes.c_uint64, vp, vp, i32, vp, vp, vp, vp, vp]
        L.ep_host_combine.argtypes = [sp, vp, i64, vp, vp, vp, vp, vp, vp, i64, vp, i32, vp, i32, vp, vp, vp, vp]
        L.ep_wait_senders.argtypes = [vp, i32, ctypes.c_uint32, ctypes.c_uint64, vp, vp, vp]
        L.ep_post_flags.argtypes = [vp, i32, i32, ctypes.c_uint32, vp]
        L.ep_dispatch_copy_engine.argtypes = [sp, vp, vp, vp, vp, i64, vp, vp, vp]
        L.ep_host_step_arena_bytes.restype = sz
        L.ep_host_step_arena_bytes.argtypes = [sp]
        L.ep_host_step.argtypes = [sp, vp, vp, vp, vp, vp, vp, sz, vp]
        L.ep_host_step_pipelined.argtypes = [sp, vp, vp, vp, vp, vp, vp, sz, i32, vp, vp, vp, i32, vp]
        L.ep_host_step_pipelined.restype = i32
        L.ep_status.argtypes = [vp, vp, vp]
        L.ep_probe_bandwidth.argtypes = [i32, vp, vp, sz, i32, vp, ctypes.POINTER(ctypes.c_double)]
        L.ep_launch_count.restype = i64
        L.ep_strerror.restype = ctypes.c_char_p
        L.ep_strerror.argtypes = [i32]
        for name in ["ep_layout", "ep_dispatch", "ep_combine", "ep_group", "ep_dispatch_copy_engine",
                     "ep_combine_partial", "ep_dense_allgather", "ep_dense_reduce_scatter",
                     "ep_host_roundtrip", "ep_host_dispatch_per_sender", "ep_host_combine", "ep_wait_senders", "ep_post_flags",
                     "ep_host_step", "ep_status", "ep_probe_bandwidth", "ep_last_cuda_error"]:
            getattr(L, name).restype = i32
        _lib = L
    return _lib


def _shape(T, K, H, E, R) -> _Shape:
    return _Shape(int(T), int(K), int(H), int(E), int(R))


def _ptr(t):
    """Address of a tensor's first element; the library sees dense row-major memory only."""
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("the EP library needs contiguous tensors")
    return ctypes.c_void_p(t.data_ptr())


def _want(t, dtype, name):
    if t.dtype != dtype:
        raise TypeError(f"{name} must be {dtype}, got {t.dtype}")


def _stream():
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def _check(rc: int, where: str):
    if rc != 0:
        raise EPError(rc, where)


@dataclass
class Layout:
    """Device tensors written by `ep_layout` (all int32)."""
    expert_counts: torch.Tensor
    expert_offsets: torch.Tensor
    rank_rows: torch.Tensor
    rank_row_offsets: torch.Tensor
    src_row_offsets: torch.Tensor
    recv_slot: torch.Tensor
    pair_slot: torch.Tensor
    recv_token: torch.Tensor
    pair_row: torch.Tensor
    pair_token: torch.Tensor
    status: torch.Tensor

    def as_struct(self) -> _Layout:
        return _Layout(*[getattr(self, f).data_ptr() for f in _LAYOUT_FIELDS])


def alloc_layout(T, K, E, R, device="cuda", fill=None) -> Layout:
    """Allocates the output arrays of `ep_layout` (torch owns the memory)."""
    def mk(*shape):
        n = 1
        for d in shape:
            n *= d
        t = torch.empty(max(1, n), dtype=torch.int32, device=device)   # never a NULL pointer, even for T == 0
        if fill is not None:
            t.fill_(fill)
        return t[:n].view(*shape)
    return Layout(mk(E), mk(E + 1), mk(R), mk(R + 1), mk(R, R + 1), mk(T, K), mk(T, K),
                  mk(T * min(K, R)), mk(T * K), mk(T * K), mk(1))


def ep_layout_workspace_bytes(T, K, E, R) -> int:
    return int(lib().ep_layout_workspace_bytes(ctypes.byref(_shape(T, K, 8, E, R))))


def ep_layout(topk_idx: torch.Tensor, E: int, R: int, out: Layout = None, workspace: torch.Tensor = None) -> Layout:
    _want(topk_idx, torch.int32, "topk_idx")
    T, K = topk_idx.shape
    if out is None:
        out = alloc_layout(T, K, E, R, device=topk_idx.device)
    if workspace is None:
        workspace = torch.empty(max(16, ep_layout_workspace_bytes(T, K, E, R)), dtype=torch.uint8, device=topk_idx.device)
    st = out.as_struct()
    _check(lib().ep_layout(ctypes.byref(_shape(T, K, 8, E, R)), _ptr(topk_idx), ctypes.byref(st), _ptr(workspace),
                           workspace.numel(), _stream()), "ep_layout")
    return out


def _layout_half(fn_name, topk_idx, E, R, out, workspace, stream):
    T, K = topk_idx.shape
    st = out.as_struct()
    sp = ctypes.c_void_p(stream.cuda_stream) if stream is not None else _stream()
    _check(getattr(lib(), fn_name)(ctypes.byref(_shape(T, K, 8, E, R)), _ptr(topk_idx), ctypes.byref(st), _ptr(workspace),
                                   workspace.numel(), sp), fn_name)
    return out


def ep_layout_ranks(topk_idx, E, R, out: Layout, workspace, stream=None) -> Layout:
    """The receive-row half of `ep_layout` (what dispatch needs)."""
    return _layout_half("ep_layout_ranks", topk_idx, E, R, out, workspace, stream)


def ep_layout_pairs(topk_idx, E, R, out: Layout, workspace, stream=None) -> Layout:
    """The pair-space half of `ep_layout` (what grouping and combine need); may run on another stream."""
    return _layout_half("ep_layout_pairs", topk_idx, E, R, out, workspace, stream)


def ep_layout_static(topk_idx: torch.Tensor, E: int, R: int, out: Layout) -> Layout:
    """`ep_layout` for callers that may not allocate device memory: the scratch is a
    fixed array inside the library, so `out` must be given and nothing is allocated
    here either. Shapes whose scratch exceeds `ep_layout_static_scratch_bytes()` raise."""
    T, K = topk_idx.shape
    st = out.as_struct()
    _check(lib().ep_layout_static(ctypes.byref(_shape(T, K, 8, E, R)), _ptr(topk_idx), ctypes.byref(st), _stream()),
           "ep_layout_static")
    return out


def ep_layout_static_scratch_bytes() -> int:
    return int(lib().ep_layout_static_scratch_bytes())


def ep_layout_dispatch(topk_idx: torch.Tensor, x: torch.Tensor, recv: torch.Tensor, E: int, R: int, out: Layout,
                       workspace: torch.Tensor, stream_pairs=None) -> Layout:
    """`ep_layout` followed by `ep_dispatch` in one call: dispatch is launched behind the layout kernels and loads
    its rows while they run; past 1024 tokens the layout's pair half runs on `stream_pairs` (a torch stream) if
    given; small batches of shapes the fastest layout kernels do not cover take a single launch."""
    _want(topk_idx, torch.int32, "topk_idx"), _want(x, torch.bfloat16, "x"), _want(recv, torch.bfloat16, "recv")
    T, K = topk_idx.shape
    st = out.as_struct()
    _check(lib().ep_layout_dispatch(ctypes.byref(_shape(T, K, x.shape[1], E, R)), _ptr(topk_idx), _ptr(x), ctypes.byref(st),
                                    _ptr(workspace), workspace.numel(), _ptr(recv), recv.shape[0], _stream(),
                                    ctypes.c_void_p(stream_pairs.cuda_stream) if stream_pairs is not None else None),
           "ep_layout_dispatch")
    return out


def ep_dispatch(x: torch.Tensor, recv_slot: torch.Tensor, recv: torch.Tensor, E: int, R: int, status=None):
    _want(x, torch.bfloat16, "x"), _want(recv, torch.bfloat16, "recv"), _want(recv_slot, torch.int32, "recv_slot")
    T, H = x.shape
    K = recv_slot.shape[1]
    _check(lib().ep_dispatch(ctypes.byref(_shape(T, K, H, E, R)), _ptr(x), _ptr(recv_slot), _ptr(recv),
                             recv.shape[0], _ptr(status), _stream()), "ep_dispatch")
    return recv


def ep_combine(out: torch.Tensor, slot: torch.Tensor, topk_weights: torch.Tensor, y: torch.Tensor, E: int, R: int,
               status=None):
    _want(out, torch.bfloat16, "out"), _want(y, torch.bfloat16, "y"), _want(slot, torch.int32, "slot")
    _want(topk_weights, torch.float32, "topk_weights")
    T, K = slot.shape
    H = out.shape[1]
    _check(lib().ep_combine(ctypes.byref(_shape(T, K, H, E, R)), _ptr(out), out.shape[0], _ptr(slot),
                            _ptr(topk_weights), _ptr(y), _ptr(status), _stream()), "ep_combine")
    return y


def ep_group(recv: torch.Tensor, lay: Layout, grouped: torch.Tensor, E: int, R: int, status=None):
    T, K = lay.recv_slot.shape
    H = recv.shape[1]
    _check(lib().ep_group(ctypes.byref(_shape(T, K, H, E, R)), _ptr(recv), recv.shape[0], _ptr(lay.pair_row),
                          _ptr(lay.expert_offsets), _ptr(grouped), grouped.shape[0], _ptr(status), _stream()),
           "ep_group")
    return grouped


def ep_combine_partial(out, lay: Layout, topk_weights, partial, y, E: int, R: int, status=None):
    """Two-stage combine: per-(token, rank) partial rows in the receive space, then their sum."""
    T, K = lay.pair_slot.shape
    H = out.shape[1]
    _check(lib().ep_combine_partial(ctypes.byref(_shape(T, K, H, E, R)), _ptr(out), out.shape[0], _ptr(lay.pair_slot),
                                    _ptr(lay.recv_slot), _ptr(topk_weights), _ptr(partial), partial.shape[0], _ptr(y),
                                    _ptr(status), _stream()), "ep_combine_partial")
    return y


def ep_dense_allgather(x, gathered, K: int, E: int, R: int):
    T, H = x.shape
    _check(lib().ep_dense_allgather(ctypes.byref(_shape(T, K, H, E, R)), _ptr(x), _ptr(gathered), _stream()),
           "ep_dense_allgather")
    return gathered


def ep_dense_reduce_scatter(topk_idx, out, pair_slot, topk_weights, dense, y, E: int, R: int, status=None):
    T, K = topk_idx.shape
    H = out.shape[1]
    _check(lib().ep_dense_reduce_scatter(ctypes.byref(_shape(T, K, H, E, R)), _ptr(topk_idx), _ptr(out), out.shape[0],
                                         _ptr(pair_slot), _ptr(topk_weights), _ptr(dense), _ptr(y), _ptr(status),
                                         _stream()), "ep_dense_reduce_scatter")
    return y


def ep_dispatch_copy_engine(x, recv_slot, staging, recv_host, E, R, rank_row_offsets_host=None, status=None):
    """rank_row_offsets_host: CPU int32 tensor [R+1] or None (one worst-case copy)."""
    T, H = x.shape
    K = recv_slot.shape[1]
    _check(lib().ep_dispatch_copy_engine(ctypes.byref(_shape(T, K, H, E, R)), _ptr(x), _ptr(recv_slot),
                                         _ptr(rank_row_offsets_host), _ptr(staging), staging.shape[0],
                                         _ptr(recv_host), _ptr(status), _stream()), "ep_dispatch_copy_engine")
    return recv_host


def _sp(stream):
    return ctypes.c_void_p(stream.cuda_stream) if stream is not None else _stream()


class HalfFreeEvents:
    """Two caller-owned CUDA events, one per half of a two-half bounce buffer, in the form the
    host-staged calls take them (an array of two cudaEvent_t). torch creates an event's handle
    when it is first recorded, so both are recorded once on the current stream here."""

    def __init__(self):
        self.events = [torch.cuda.Event(), torch.cuda.Event()]
        for e in self.events:
            e.record()
        self.array = (ctypes.c_void_p * 2)(*[ctypes.c_void_p(e.cuda_event) for e in self.events])


def _half_free(h):
    return None if h is None else ctypes.cast(h.array, ctypes.c_void_p)


def ep_host_roundtrip(x, recv_slot, rank_row_offsets_host, staging, bounce_host, recv, E, R, round=0,
                      chunks_per_rank=1, duplex=True, status=None, stream_up=None, stream_down=None,
                      half_free: HalfFreeEvents = None):
    """Pack -> upload to the pinned bounce buffer -> download into `recv`, on two streams
    (torch.cuda.Stream objects; default: the current stream for both)."""
    T, H = x.shape
    K = recv_slot.shape[1]
    _check(lib().ep_host_roundtrip(ctypes.byref(_shape(T, K, H, E, R)), _ptr(x), _ptr(recv_slot),
                                   _ptr(rank_row_offsets_host), _ptr(staging), staging.shape[0], _ptr(bounce_host),
                                   int(round), _ptr(recv), int(chunks_per_rank), int(bool(duplex)), _ptr(status),
                                   _sp(stream_up), _sp(stream_down), _half_free(half_free)),
           "ep_host_roundtrip")
    return recv


def ep_host_dispatch_per_sender(x, lay: Layout, src_row_offsets_host, staging, recv, bounce_host, grouped, E, R,
                                round=0, flags=HOST_DUPLEX | HOST_PER_PEER, sender_flags=None, epoch=0,
                                timeout_ns=0, arrived=None, stamps_ns=None, status=None, stream_up=None,
                                stream_down=None, stream_consume=None, half_free: HalfFreeEvents = None):
    """Host-staged dispatch moved sender by sender, the local grouping of each sender's pairs
    launched as that sender's rows arrive. src_row_offsets_host: CPU int32 [R, R+1]."""
    T, H = x.shape
    K = lay.recv_slot.shape[1]
    _check(lib().ep_host_dispatch_per_sender(
        ctypes.byref(_shape(T, K, H, E, R)), _ptr(x), _ptr(lay.recv_slot), _ptr(lay.pair_slot),
        _ptr(src_row_offsets_host), _ptr(staging), _ptr(recv), staging.shape[0], _ptr(bounce_host), int(round),
        _ptr(grouped), grouped.shape[0], _ptr(sender_flags), int(epoch), int(timeout_ns), _ptr(arrived),
        _ptr(stamps_ns), int(flags), _ptr(status), _sp(stream_up), _sp(stream_down), _sp(stream_consume),
        _half_free(half_free)), "ep_host_dispatch_per_sender")
    return grouped


def ep_host_combine(out, lay: Layout, topk_weights, src_row_offsets_host, partial_send, partial_recv, bounce_host, y,
                    E, R, round=0, flags=HOST_DUPLEX | HOST_PER_PEER, status=None, stream_up=None, stream_down=None,
                    half_free: HalfFreeEvents = None):
    """Host-staged combine: per-rank partial rows up to the bounce buffer, down to the owner, summed on the SMs."""
    T, K = lay.pair_slot.shape
    H = out.shape[1]
    _check(lib().ep_host_combine(
        ctypes.byref(_shape(T, K, H, E, R)), _ptr(out), out.shape[0], _ptr(lay.pair_slot), _ptr(lay.recv_slot),
        _ptr(topk_weights), _ptr(src_row_offsets_host), _ptr(partial_send), _ptr(partial_recv), partial_send.shape[0],
        _ptr(bounce_host), int(round), _ptr(y), int(flags), _ptr(status), _sp(stream_up), _sp(stream_down),
        _half_free(half_free)), "ep_host_combine")
    return y


def ep_wait_senders(flags, num_senders: int, epoch: int, timeout_ns: int, arrived=None, status=None):
    _check(lib().ep_wait_senders(_ptr(flags), num_senders, epoch, timeout_ns, _ptr(arrived), _ptr(status), _stream()),
           "ep_wait_senders")


def ep_post_flags(flags, first_sender: int, num_senders: int, epoch: int):
    _check(lib().ep_post_flags(_ptr(flags), first_sender, num_senders, epoch, _stream()), "ep_post_flags")


def ep_host_step_arena_bytes(T, K, H, E, R) -> int:
    return int(lib().ep_host_step_arena_bytes(ctypes.byref(_shape(T, K, H, E, R))))


def ep_host_step(x_host, topk_idx_host, topk_weights_host, y_host, arena, E, R, status_host=None):
    """All *_host tensors live in (pinned) host memory; arena is a device uint8 tensor."""
    T, H = x_host.shape
    K = topk_idx_host.shape[1]
    _check(lib().ep_host_step(ctypes.byref(_shape(T, K, H, E, R)), _ptr(x_host), _ptr(topk_idx_host),
                              _ptr(topk_weights_host), _ptr(y_host), _ptr(status_host), _ptr(arena), arena.numel(),
                              _stream()), "ep_host_step")
    return y_host


class StepEvents:
    """Four caller-owned CUDA events for `ep_host_step_pipelined` calls back to back on one arena (kernels done and
    downloads done, per copy of the arena's transfer buffers). torch creates an event's handle when it is first
    recorded, so all four are recorded once on the current stream here."""

    def __init__(self):
        self.events = [torch.cuda.Event() for _ in range(4)]
        for e in self.events:
            e.record()
        self.array = (ctypes.c_void_p * 4)(*[ctypes.c_void_p(e.cuda_event) for e in self.events])


def ep_host_step_pipelined(x_host, topk_idx_host, topk_weights_host, y_host, arena, E, R, chunks, stream_in,
                           stream_compute, stream_out, status_host=None, round=0, step_events: StepEvents = None):
    """`ep_host_step` with uploads, kernels and downloads of token chunks overlapping on three streams. With
    `step_events` consecutive calls (round = 0, 1, 2, ...) alternate between two copies of the arena's transfer
    buffers, so that a call's uploads overlap the previous call's downloads."""
    T, H = x_host.shape
    K = topk_idx_host.shape[1]
    _check(lib().ep_host_step_pipelined(ctypes.byref(_shape(T, K, H, E, R)), _ptr(x_host), _ptr(topk_idx_host),
                                        _ptr(topk_weights_host), _ptr(y_host), _ptr(status_host), _ptr(arena),
                                        arena.numel(), int(chunks), ctypes.c_void_p(stream_in.cuda_stream),
                                        ctypes.c_void_p(stream_compute.cuda_stream),
                                        ctypes.c_void_p(stream_out.cuda_stream), int(round),
                                        None if step_events is None else ctypes.cast(step_events.array, ctypes.c_void_p)),
           "ep_host_step_pipelined")
    return y_host


def ep_status(status: torch.Tensor) -> int:
    host = ctypes.c_int32(0)
    _check(lib().ep_status(_ptr(status), _stream(), ctypes.byref(host)), "ep_status")
    return int(host.value)


def ep_probe_bandwidth(kind: int, dst, src, nbytes: int, iters: int = 10) -> float:
    g = ctypes.c_double(0.0)
    _check(lib().ep_probe_bandwidth(kind, _ptr(dst), _ptr(src), nbytes, iters, _stream(), ctypes.byref(g)),
           "ep_probe_bandwidth")
    return float(g.value)


def ep_launch_count() -> int:
    return int(lib().ep_launch_count())
