"""Property tests of the oracle's layout on arbitrary small routing tables (hypothesis draws the
shapes and the ids, masked, repeated and out-of-range ones included): agreement with the literal
set definitions, and the invariants that hold for any input."""
import numpy as np
from hypothesis import given, settings, strategies as st

import brute
import oracle


@st.composite
def routing_tables(draw):
    R = draw(st.sampled_from([1, 2, 3, 4]))
    E = R * draw(st.integers(1, 4))
    K = draw(st.integers(1, 5))
    T = R * draw(st.integers(1, 6))
    ids = draw(st.lists(st.integers(-2, E + 1), min_size=T * K, max_size=T * K))
    return np.array(ids, dtype=np.int32).reshape(T, K), E, R


@settings(max_examples=120, deadline=None)
@given(routing_tables())
def test_layout_equals_the_set_definitions_on_any_table(case):
    idx, E, R = case
    T, K = idx.shape
    got = oracle.layout(idx, E, R)
    want = brute.layout(idx, E, R)
    for f in ["expert_counts", "expert_offsets", "rank_rows", "rank_row_offsets", "src_row_offsets", "recv_slot",
              "pair_slot", "recv_token", "pair_row", "pair_token"]:
        np.testing.assert_array_equal(getattr(got, f), want[f], err_msg=f)
    assert got.status == want["status"]
    valid = (idx >= 0) & (idx < E)
    # counts sum to the number of valid pairs; receive rows = distinct (token, rank) <= T*min(K, R)
    assert got.n_pairs == int(valid.sum()) == int(got.expert_counts.sum())
    El = E // R
    distinct = {(t, int(idx[t, k]) // El) for t in range(T) for k in range(K) if valid[t, k]}
    assert got.n_recv == len(distinct) <= T * min(K, R)
    # slots of valid pairs: pair slots a permutation of 0..P-1, receive slots cover 0..N_recv-1
    assert sorted(got.pair_slot[valid].tolist()) == list(range(got.n_pairs))
    assert set(got.recv_slot[valid].tolist()) == set(range(got.n_recv))
    assert (got.recv_slot[~valid] == -1).all() and (got.pair_slot[~valid] == -1).all()
    # a rank's rows are ordered by token, an expert's pairs by (token, k)
    for r in range(R):
        rows = got.recv_token[got.rank_row_offsets[r]:got.rank_row_offsets[r + 1]]
        assert (np.diff(rows) > 0).all()
    for e in range(E):
        toks = got.pair_token[got.expert_offsets[e]:got.expert_offsets[e + 1]]
        assert (np.diff(toks) >= 0).all()


@settings(max_examples=60, deadline=None)
@given(routing_tables(), st.integers(0, 2 ** 31 - 1))
def test_dispatch_then_grouping_delivers_each_pair_its_token_row(case, seed):
    idx, E, R = case
    T, K = idx.shape
    lay = oracle.layout(idx, E, R)
    x = np.random.default_rng(seed).integers(0, 2 ** 16, size=(T, 8), dtype=np.uint16)
    recv = oracle.dispatch(x, lay.recv_slot, lay.n_recv + 2, fill=0xABCD)
    assert (recv[lay.n_recv:] == 0xABCD).all()
    np.testing.assert_array_equal(recv[:lay.n_recv], x[lay.recv_token])
    np.testing.assert_array_equal(oracle.group(recv, lay.pair_row), x[lay.pair_token])
