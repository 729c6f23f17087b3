"""Helpers of the GPU parity tests: numpy bit patterns <-> device tensors."""
import numpy as np
import torch

SENTINEL = 0x7FC1           # bf16 NaN pattern that no generator emits
GUARD = 4                   # guard rows before/after every checked buffer

LAYOUT_FIELDS = ["expert_counts", "expert_offsets", "rank_rows", "rank_row_offsets", "src_row_offsets",
                 "recv_slot", "pair_slot"]


def dev_bf16(bits: np.ndarray) -> torch.Tensor:
    return torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16).cuda()


def host_bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).cpu().numpy().view(np.uint16)


def guarded(rows: int, H: int):
    """A [rows+2*GUARD, H] bf16 device buffer full of the sentinel; returns (whole, view of the middle)."""
    whole = torch.full((rows + 2 * GUARD, H), SENTINEL, dtype=torch.int16, device="cuda").view(torch.bfloat16)
    return whole, whole[GUARD:GUARD + rows]


def guards_intact(whole: torch.Tensor) -> bool:
    b = host_bits(whole)
    return bool((b[:GUARD] == SENTINEL).all() and (b[-GUARD:] == SENTINEL).all())


def assert_layout_equal(lay, ref):
    for f in LAYOUT_FIELDS:
        got = getattr(lay, f).cpu().numpy()
        np.testing.assert_array_equal(got, getattr(ref, f), err_msg=f)
    n_recv, n_pairs = ref.n_recv, ref.n_pairs
    np.testing.assert_array_equal(lay.recv_token.cpu().numpy()[:n_recv], ref.recv_token, err_msg="recv_token")
    np.testing.assert_array_equal(lay.pair_row.cpu().numpy()[:n_pairs], ref.pair_row, err_msg="pair_row")
    np.testing.assert_array_equal(lay.pair_token.cpu().numpy()[:n_pairs], ref.pair_token, err_msg="pair_token")


def within_tolerance(y_bits: np.ndarray, ref64: np.ndarray):
    """max relative error 4e-3 per element, absolute 1e-3 near zero."""
    from paper_2609_40093_b200 import inputs
    got = inputs.bf16_bits_to_f32(y_bits).astype(np.float64)
    return np.abs(got - ref64) <= np.maximum(4e-3 * np.abs(ref64), 1e-3)
