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


def _dense_exact(out_f, idx, pair_slot, w, E, R):
    """Dense reduce-scatter on exact rationals with explicit roundings (tiny inputs): per rank an fp32
    fma chain over the k (ascending) whose expert lives there, one bf16 rounding of what the rank places
    in its dense buffer, then the owner's fp32 sum of the R placed values in the order r = 0..R-1."""
    T, K = idx.shape
    H = out_f.shape[1]
    El = E // R
    dense = np.zeros((R, T, H))
    y = np.zeros((T, H))
    for t in range(T):
        for h in range(H):
            total = Fraction(0)
            for r in range(R):
                acc = Fraction(0)
                for k in range(K):
                    if 0 <= idx[t, k] < E and idx[t, k] // El == r:
                        acc = brute.round_f32(Fraction(float(w[t, k])) * Fraction(float(out_f[pair_slot[t, k], h])) + acc)
                placed = brute.round_bf16(acc)
                dense[r, t, h] = float(placed)
                total = brute.round_f32(total + placed)
            y[t, h] = float(brute.round_bf16(total))
    return dense, y


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_dense_reduce_scatter_against_exact_rationals(seed):
    """8 experts on 4 ranks, 4 distinct picks per token: every token reaches at least two ranks and most
    reach three or four, so the owner's sum has several terms that are not bf16 numbers before placing."""
    cfg, idx, w, x, lay, out = _case(8, 6, 8, 4, 4, cid=86, seed=seed)
    assert max(len(set((idx[t] // 2).tolist())) for t in range(cfg.T)) >= 3
    dense, y = oracle.dense_reduce_scatter(idx, out, lay.pair_slot, w, cfg.E, cfg.R)
    want_dense, want_y = _dense_exact(inputs.bf16_bits_to_f32(out), idx, lay.pair_slot, w, cfg.E, cfg.R)
    np.testing.assert_array_equal(inputs.bf16_bits_to_f32(dense).astype(np.float64).reshape(cfg.R, cfg.T, cfg.H),
                                  want_dense)
    np.testing.assert_array_equal(inputs.bf16_bits_to_f32(y).astype(np.float64), want_y)


def test_dense_reduce_scatter_sums_ranks_in_ascending_order_and_after_rounding():
    """Three ranks hold big, -big and small: summed in the order r = 0, 1, 2 the small term survives;
    any order that adds small to a big term first loses it. Then a rank whose fp32 partial is not a
    bf16 number: the owner must add what was placed (rounded), not the unrounded accumulator."""
    E, R, H = 3, 3, 1
    out = inputs.to_bf16_bits(np.array([[2.0 ** 20], [2.0 ** 20], [2.0 ** -6]], dtype=np.float32))
    w = np.array([[1.0, -1.0, 1.0]] * 3, dtype=np.float32)
    idx = np.array([[0, 1, 2]] * 3, dtype=np.int32)                 # pick k sits on rank k
    pair_slot = np.array([[0, 1, 2]] * 3, dtype=np.int32)
    dense, y = oracle.dense_reduce_scatter(idx, out, pair_slot, w, E, R)
    assert (inputs.bf16_bits_to_f32(y) == 2.0 ** -6).all()
    idx2 = np.array([[2, 1, 0]] * 3, dtype=np.int32)                # big on rank 2, -big on rank 1, small on rank 0
    w2 = np.array([[1.0, -1.0, 1.0]] * 3, dtype=np.float32)
    out2 = inputs.to_bf16_bits(np.array([[2.0 ** 20], [2.0 ** 20], [2.0 ** -6]], dtype=np.float32))
    pair2 = np.array([[0, 1, 2]] * 3, dtype=np.int32)               # k=0 -> big (rank 2), k=1 -> -big (rank 1), k=2 -> small (rank 0)
    _, y2 = oracle.dense_reduce_scatter(idx2, out2, pair2, w2, E, R)
    assert (inputs.bf16_bits_to_f32(y2) == 0.0).all()               # small + (-big) = -big; -big + big = 0
    # rank 0 holds 1 + 2^-10 in fp32 (two picks), which it places as bf16 1.0; rank 1 holds -1
    E, R = 4, 2
    out3 = inputs.to_bf16_bits(np.array([[1.0], [2.0 ** -10], [1.0]], dtype=np.float32))
    idx3 = np.array([[0, 1, 2]] * 2, dtype=np.int32)                # experts 0, 1 on rank 0; expert 2 on rank 1
    w3 = np.array([[1.0, 1.0, -1.0]] * 2, dtype=np.float32)
    pair3 = np.array([[0, 1, 2]] * 2, dtype=np.int32)
    dense3, y3 = oracle.dense_reduce_scatter(idx3, out3, pair3, w3, E, R)
    assert (inputs.bf16_bits_to_f32(dense3).ravel() == np.array([1.0, 1.0, -1.0, -1.0])).all()
    assert (inputs.bf16_bits_to_f32(y3) == 0.0).all()               # 2^-10 would survive an unrounded sum


def _ring_allgather_bytes(N, S):
    """Replays the ring schedule over a host bounce buffer (no P2P): at each of N-1 steps every GPU
    uploads the shard it obtained last and downloads the one its predecessor uploaded. Returns the
    bytes per GPU over the host link and checks that every GPU ends up holding every shard."""
    holds = [{g} for g in range(N)]
    last = list(range(N))
    moved = [0] * N
    for _ in range(N - 1):
        sent = list(last)
        for g in range(N):
            moved[g] += S                                            # upload of the shard obtained last
        for g in range(N):
            got = sent[(g - 1) % N]
            moved[g] += S                                            # download from the predecessor
            holds[g].add(got)
            last[g] = got
    assert all(h == set(range(N)) for h in holds)
    assert len(set(moved)) == 1
    return moved[0]


@pytest.mark.parametrize("N", [2, 4, 6])
def test_paper_traffic_formulas(N):
    """Section 4.2, per-GPU volume over the host link with shards of S bytes: ring all-gather 2(N-1)S,
    single-step all-gather N*S, ratio 2(N-1)/N (1 at N=2; 10S -> 6S at N=6); reduce-scatter with GPU
    reduction 2(N-1)S, with CPU reduction N*S. The single-step volumes are counted on the dense oracle's
    buffers (which rows of a rank's block come from, or go to, another rank), the ring by replaying its
    schedule; neither count uses the formula it is compared with."""
    T, H, K = 12 * N, 16, 2
    Tr = T // N
    row = 2 * H
    S = Tr * row                                                     # one rank's shard in bytes
    cfg = inputs.custom_config(T, H, 2 * N, K, N, config_id=85)
    d = inputs.make_inputs(cfg)
    x, idx, w = d["x"], d["topk_idx"], d["topk_weights"]
    g = oracle.dense_allgather(x, N).reshape(N, T, H)
    owner = np.arange(T) // Tr
    for r in range(N):
        written = np.flatnonzero((g[r] != 0).any(axis=1))            # the wrapper starts from zeros; no row of x is all zero
        remote = written[owner[written] != r]
        download = remote.size * row                                 # rows of other ranks' shards that rank r reads back
        sources = {int(s) for s in owner[remote]}
        assert sources == set(range(N)) - {r}
        upload = np.unique(x[owner == r], axis=0).shape[0] * row     # rank r's own shard goes up once, whoever reads it
        assert upload == S and download == (N - 1) * S
        assert upload + download == N * S
    ring = _ring_allgather_bytes(N, S)
    assert ring == 2 * (N - 1) * S
    assert Fraction(ring, N * S) == Fraction(2 * (N - 1), N)
    if N == 2:
        assert ring == N * S
    if N == 6:
        assert (ring // S, N * S // S) == (10, 6)
    # reduce-scatter: rank r's dense block holds one row per source token; the rows of tokens another rank
    # owns are the blocks it uploads, the rows other ranks hold for its own tokens are what it downloads
    lay = oracle.layout(idx, cfg.E, N)
    out = inputs.make_out(cfg, lay.n_pairs)
    dense, _ = oracle.dense_reduce_scatter(idx, out, lay.pair_slot, w, cfg.E, N)
    dense = dense.reshape(N, T, H)
    assert dense.shape[1] == T                                       # a full source-ordered block per rank, whatever the routing
    for r in range(N):
        up_rows = int((owner != r).sum())                            # rows of rank r's block destined for other ranks
        down_rows = sum(int((owner == r).sum()) for q in range(N) if q != r)
        assert up_rows * row == (N - 1) * S and down_rows * row == (N - 1) * S
        assert (up_rows + down_rows) * row == 2 * (N - 1) * S        # GPU reduction: same volume as the ring
        assert up_rows * row + int((owner == r).sum()) * row == N * S   # CPU reduction: one reduced block comes down
    # the routed form moves only the rows a rank needs: never more than the dense R*T, never more than T*min(K,R)
    assert lay.n_recv <= T * min(K, N) <= N * T
