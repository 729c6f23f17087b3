"""Literal evaluation of the layout / dispatch / combine definitions on tiny inputs.

Every quantity is computed straight from its set expression with Python loops
(no counters carried along a sweep, no library sort), and the combine sum is
evaluated in exact rational arithmetic with an explicit correctly rounded
fused multiply-add. It is deliberately quadratic: use it on tiny cases only.
It shares nothing with the oracle or with the CUDA path.
"""
from fractions import Fraction

import numpy as np


def layout(idx, E, R):
    idx = np.asarray(idx)
    T, K = idx.shape
    El, Tr = E // R, T // R
    pairs = [(t, k) for t in range(T) for k in range(K)]

    def valid(t, k):
        return 0 <= idx[t, k] < E

    def rank(t, k):
        return int(idx[t, k]) // El

    def hit(t, r):
        return any(valid(t, k) and rank(t, k) == r for k in range(K))

    expert_counts = [sum(1 for (t, k) in pairs if valid(t, k) and idx[t, k] == e) for e in range(E)]
    expert_offsets = [sum(expert_counts[:e]) for e in range(E + 1)]
    rank_rows = [sum(1 for t in range(T) if hit(t, r)) for r in range(R)]
    rank_row_offsets = [sum(rank_rows[:r]) for r in range(R + 1)]
    recv_slot = -np.ones((T, K), dtype=np.int64)
    pair_slot = -np.ones((T, K), dtype=np.int64)
    for (t, k) in pairs:
        if not valid(t, k):
            continue
        r, e = rank(t, k), idx[t, k]
        recv_slot[t, k] = rank_row_offsets[r] + sum(1 for t2 in range(t) if hit(t2, r))
        pair_slot[t, k] = expert_offsets[e] + sum(
            1 for (t2, k2) in pairs if (t2, k2) < (t, k) and valid(t2, k2) and idx[t2, k2] == e)
    src_row_offsets = np.zeros((R, R + 1), dtype=np.int64)
    for r in range(R):
        for s in range(R + 1):
            src_row_offsets[r, s] = rank_row_offsets[r] + sum(
                1 for t2 in range(T) if (t2 // Tr if Tr else 0) < s and hit(t2, r))
    n_recv, n_pairs = rank_row_offsets[R], expert_offsets[E]
    recv_token = -np.ones(n_recv, dtype=np.int64)
    pair_row = -np.ones(n_pairs, dtype=np.int64)
    pair_token = -np.ones(n_pairs, dtype=np.int64)
    for (t, k) in pairs:
        if valid(t, k):
            recv_token[recv_slot[t, k]] = t
            pair_row[pair_slot[t, k]] = recv_slot[t, k]
            pair_token[pair_slot[t, k]] = t
    bad = any((idx[t, k] < -1 or idx[t, k] >= E) for (t, k) in pairs)
    return dict(expert_counts=np.array(expert_counts), expert_offsets=np.array(expert_offsets),
                rank_rows=np.array(rank_rows), rank_row_offsets=np.array(rank_row_offsets),
                src_row_offsets=src_row_offsets, recv_slot=recv_slot, pair_slot=pair_slot,
                recv_token=recv_token, pair_row=pair_row, pair_token=pair_token, status=int(bad))


def _round_fraction(q: Fraction, mant_bits: int, emin: int) -> Fraction:
    """Round an exact rational to a binary float with `mant_bits` significant bits
    (ties to even), subnormals below 2**emin; overflow is not modelled."""
    if q == 0:
        return Fraction(0)
    sign = -1 if q < 0 else 1
    a = abs(q)
    e = a.numerator.bit_length() - a.denominator.bit_length()
    if Fraction(2) ** e > a:
        e -= 1
    # now 2**e <= a < 2**(e+1)
    e = max(e, emin)
    ulp = Fraction(2) ** (e - (mant_bits - 1))
    n = a / ulp
    lo = n.numerator // n.denominator
    rem = n - lo
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and lo % 2 == 1):
        lo += 1
    return sign * lo * ulp


def round_f32(q: Fraction) -> Fraction:
    return _round_fraction(q, 24, -126)


def round_bf16(q: Fraction) -> Fraction:
    return _round_fraction(q, 8, -126)


def combine_exact(out_f32, slot, w):
    """Exact rational sum_k w*out (no rounding at all)."""
    T, K = slot.shape
    H = out_f32.shape[1]
    y = [[Fraction(0)] * H for _ in range(T)]
    for t in range(T):
        for h in range(H):
            acc = Fraction(0)
            for k in range(K):
                if slot[t, k] >= 0:
                    acc += Fraction(float(w[t, k])) * Fraction(float(out_f32[slot[t, k], h]))
            y[t][h] = acc
    return y


def combine_fma_chain(out_f32, slot, w):
    """fp32 chain acc = round_f32(w*v + acc) in ascending k from 0, then one bf16
    rounding; every rounding done on exact rationals. Returns floats."""
    T, K = slot.shape
    H = out_f32.shape[1]
    y = np.zeros((T, H), dtype=np.float64)
    for t in range(T):
        for h in range(H):
            acc = Fraction(0)
            for k in range(K):
                if slot[t, k] >= 0:
                    acc = round_f32(Fraction(float(w[t, k])) * Fraction(float(out_f32[slot[t, k], h])) + acc)
            y[t, h] = float(round_bf16(acc))
    return y
