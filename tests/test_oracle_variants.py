"""Pins of the oracle's variants: local grouping, combine with per-rank partial outputs,
and the dense all-gather / reduce-scatter formulation (Section 2.1, Section 4.2, Section 4.3)."""
from fractions import Fraction

import numpy as np
import pytest

import brute
import oracle
from paper_2609_40093_b200 import inputs


def _case(T, H, E, K, R, routing="uniform", cid=80, seed=0):
    cfg = inputs.custom_config(T, H, E, K, R, routing=routing, config_id=cid)
    d = inputs.make_inputs(cfg, seed)
    lay = oracle.layout(d["topk_idx"], E, R)
    out = inputs.make_out(cfg, max(1, lay.n_pairs), seed)
    return cfg, d["topk_idx"], d["topk_weights"], d["x"], lay, out


def _two_stage_bound(y64, partial_rows_f32):
    """Error bound of a sum of bf16-rounded partial rows, itself rounded to bf16: every
    rounding to nearest loses at most half an ulp, i.e. 2^-8 of the rounded value (fp32 noise on top)."""
    return 2.0 ** -8 * (np.abs(partial_rows_f32).sum(axis=0) + np.abs(y64)) * 1.01 + 1e-6


def test_group_is_the_gather_by_pair_row():
    cfg, idx, w, x, lay, out = _case(48, 40, 12, 3, 4)
    recv = oracle.dispatch(x, lay.recv_slot, lay.n_recv)
    grouped = oracle.group(recv, lay.pair_row)
    np.testing.assert_array_equal(grouped, recv[lay.pair_row])          # numpy fancy indexing
    np.testing.assert_array_equal(grouped, x[lay.pair_token])           # every pair row is its token's row
    # "expanded" dispatch (one physical row per pair) gives the same buffer directly
    np.testing.assert_array_equal(oracle.dispatch(x, lay.pair_slot, lay.n_pairs), grouped)
    # rows of one expert are contiguous and in token order
    for e in range(cfg.E):
        toks = lay.pair_token[lay.expert_offsets[e]:lay.expert_offsets[e + 1]]
        assert (np.diff(toks) >= 0).all()


def _partial_exact(out_f, lay_recv_slot, lay_pair_slot, w):
    """Two-stage combine on exact rationals with explicit roundings (tiny inputs)."""
    T, K = lay_recv_slot.shape
    H = out_f.shape[1]
    y = np.zeros((T, H))
    for t in range(T):
        for h in range(H):
            total = Fraction(0)
            seen = []
            for k in range(K):
                rho = lay_recv_slot[t, k]
                if rho < 0 or rho in seen:
                    continue
                seen.append(rho)
                acc = Fraction(0)
                for k2 in range(K):
                    if lay_recv_slot[t, k2] == rho:
                        acc = brute.round_f32(Fraction(float(w[t, k2])) * Fraction(float(out_f[lay_pair_slot[t, k2], h])) + acc)
                total = brute.round_f32(total + brute.round_bf16(acc))
            y[t, h] = float(brute.round_bf16(total))
    return y


@pytest.mark.parametrize("seed", [0, 1])
def test_combine_partial_against_exact_rationals(seed):
    cfg, idx, w, x, lay, out = _case(6, 8, 8, 4, 2, cid=81, seed=seed)     # 4 picks over 2 ranks: partial sums exist
    partial, y = oracle.combine_partial(out, lay.pair_slot, lay.recv_slot, w, lay.n_recv)
    want = _partial_exact(inputs.bf16_bits_to_f32(out), lay.recv_slot, lay.pair_slot, w)
    np.testing.assert_array_equal(inputs.bf16_bits_to_f32(y).astype(np.float64), want)
    y64 = oracle.combine_f64(out, lay.pair_slot, w)
    got = inputs.bf16_bits_to_f32(y)
    pf = inputs.bf16_bits_to_f32(partial)
    for t in range(cfg.T):                                              # the exact sum within the rounding bound
        rows = pf[sorted(set(lay.recv_slot[t].tolist()))]
        assert (np.abs(got[t] - y64[t]) <= _two_stage_bound(y64[t], rows)).all()


def test_combine_partial_chain_runs_in_ascending_k_inside_a_rank():
    """Three picks on one rank: big + small - big. Ascending k absorbs the small term (partial = 0);
    any other order would keep it."""
    out = inputs.to_bf16_bits(np.array([[2.0 ** 20], [2.0 ** -6], [2.0 ** 20]], dtype=np.float32))
    pair_slot = np.array([[0, 1, 2]], dtype=np.int32)
    recv_slot = np.zeros((1, 3), dtype=np.int32)
    w = np.array([[1.0, 1.0, -1.0]], dtype=np.float32)
    partial, y = oracle.combine_partial(out, pair_slot, recv_slot, w, 1)
    assert inputs.bf16_bits_to_f32(partial)[0, 0] == 0.0 and inputs.bf16_bits_to_f32(y)[0, 0] == 0.0
    w2 = np.array([[1.0, -1.0, 1.0]], dtype=np.float32)
    pair_slot2 = np.array([[0, 2, 1]], dtype=np.int32)
    partial, y = oracle.combine_partial(out, pair_slot2, recv_slot, w2, 1)
    assert inputs.bf16_bits_to_f32(y)[0, 0] == 2.0 ** -6
    # two ranks: the owner adds the partial rows in the order of their first k
    recv_slot3 = np.array([[0, 1, 0]], dtype=np.int32)          # picks 0 and 2 on one rank, pick 1 on another
    partial, y = oracle.combine_partial(out, pair_slot, recv_slot3, w, 2)
    pf = inputs.bf16_bits_to_f32(partial)
    assert pf[0, 0] == 0.0 and pf[1, 0] == 2.0 ** -6 and inputs.bf16_bits_to_f32(y)[0, 0] == 2.0 ** -6


def test_combine_partial_closed_forms():
    # one rank: the partial row IS the one-stage result, and rounding it twice changes nothing
    cfg, idx, w, x, lay, out = _case(32, 64, 16, 4, 1, cid=82)
    partial, y = oracle.combine_partial(out, lay.pair_slot, lay.recv_slot, w, lay.n_recv)
    one = oracle.combine_f32(out, lay.pair_slot, w)
    np.testing.assert_array_equal(y, one)
    np.testing.assert_array_equal(partial, one)                        # R = 1: receive row of token t is t
    # one expert per rank: every partial is a single product, w*out rounded to bf16
    cfg, idx, w, x, lay, out = _case(32, 64, 8, 3, 8, cid=83)
    partial, y = oracle.combine_partial(out, lay.pair_slot, lay.recv_slot, w, lay.n_recv)
    prod = (w.ravel()[:, None] * inputs.bf16_bits_to_f32(out)[lay.pair_slot.ravel()]).astype(np.float32)
    np.testing.assert_array_equal(partial[lay.recv_slot.ravel()], inputs.to_bf16_bits(prod))
    # one-hot weights: y is a bit copy of the chosen row (the other partials are +0)
    onehot = np.zeros_like(w)
    onehot[:, 1] = 1.0
    _, y = oracle.combine_partial(out, lay.pair_slot, lay.recv_slot, onehot, lay.n_recv)
    np.testing.assert_array_equal(y, out[lay.pair_slot[:, 1]])
    # rows nobody names stay untouched
    partial, _ = oracle.combine_partial(out, lay.pair_slot, lay.recv_slot, w, lay.n_recv + 3, fill=0x7FC1)
    assert (partial[lay.n_recv:] == 0x7FC1).all()


def test_dense_formulation_volumes_and_values():
    cfg, idx, w, x, lay, out = _case(64, 32, 16, 4, 4, cid=84)
    T, K, H, E, R = cfg.T, cfg.K, cfg.H, cfg.E, cfg.R
    g = oracle.dense_allgather(x, R)
    assert g.shape[0] == R * T >= lay.n_recv                           # dense delivers R*T rows, routed N_recv
    for r in range(R):
        np.testing.assert_array_equal(g[r * T:(r + 1) * T], x)
    # the rows a rank keeps from the gathered block are exactly its receive partition
    El = E // R
    for r in range(R):
        keep = np.array([t for t in range(T) if (idx[t] // El == r).any()])
        np.testing.assert_array_equal(g[r * T + keep], oracle.dispatch(x, lay.recv_slot, lay.n_recv)[
            lay.rank_row_offsets[r]:lay.rank_row_offsets[r + 1]])
    dense, y = oracle.dense_reduce_scatter(idx, out, lay.pair_slot, w, E, R)
    # the dense block of rank r holds the routed partial rows at their tokens and +0 elsewhere
    partial, y2 = oracle.combine_partial(out, lay.pair_slot, lay.recv_slot, w, lay.n_recv)
    hit = np.zeros((R, T), bool)
    for t in range(T):
        for k in range(K):
            r = idx[t, k] // El
            hit[r, t] = True
            np.testing.assert_array_equal(dense[r * T + t], partial[lay.recv_slot[t, k]])
    assert (dense.reshape(R, T, H)[~hit] == 0).all()
    # the reduce-scatter result is the exact sum within the bound of its R+1 roundings
    y64 = oracle.combine_f64(out, lay.pair_slot, w)
    got = inputs.bf16_bits_to_f32(y)
    df = inputs.bf16_bits_to_f32(dense).reshape(R, T, H)
    for t in range(T):
        assert (np.abs(got[t] - y64[t]) <= _two_stage_bound(y64[t], df[:, t])).all()
    # a token that reaches one rank only: dense and routed two-stage results coincide bit for bit
    single = [t for t in range(T) if hit[:, t].sum() == 1]
    np.testing.assert_array_equal(y[single], y2[single])


@pytest.mark.parametrize("N", [2, 4, 6])
def test_paper_traffic_formulas(N):
    """Section 4.2: per-GPU PCIe volume of an all-gather of shards S: ring 2(N-1)S,
    single-step N*S, ratio 2(N-1)/N (1 at N=2; 10S -> 6S at N=6); reduce-scatter with GPU
    reduction 2(N-1)S, with CPU reduction N*S. Counted on the dense oracle's buffers."""
    T, H = 12 * N, 16
    S = (T // N) * H * 2                                               # one rank's shard in bytes
    x = inputs.make_x(inputs.custom_config(T, H, N, 1, N, config_id=85))
    g = oracle.dense_allgather(x, N)
    per_rank_rows = g.shape[0] // N
    single_step = S + (per_rank_rows - T // N) * H * 2                 # upload own shard once, download the others
    assert single_step == N * S
    ring = sum(2 * S for _ in range(N - 1))                            # one upload and one download per step
    assert ring == 2 * (N - 1) * S
    assert Fraction(ring, single_step) == Fraction(2 * (N - 1), N)
    if N == 2:
        assert ring == single_step
    if N == 6:
        assert (ring // S, single_step // S) == (10, 6)
    rs_gpu = (N - 1) * S + (N - 1) * S                                 # upload N-1 blocks, download N-1 blocks
    rs_cpu = (N - 1) * S + S
    assert rs_gpu == 2 * (N - 1) * S and rs_cpu == N * S
