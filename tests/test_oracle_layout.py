"""Pins of the oracle's layout: brute force, numpy library routines, closed forms."""
import itertools
import math
import os

import numpy as np
import pytest

import brute
import oracle
from paper_2609_40093_b200 import inputs

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")
FIELDS = ["expert_counts", "expert_offsets", "rank_rows", "rank_row_offsets", "src_row_offsets",
          "recv_slot", "pair_slot", "recv_token", "pair_row", "pair_token"]


def _assert_same(lay, ref):
    for f in FIELDS:
        np.testing.assert_array_equal(np.asarray(getattr(lay, f), dtype=np.int64), np.asarray(ref[f]), err_msg=f)
    assert lay.status == ref["status"]


TINY = [  # T, K, E, R
    (2, 1, 2, 2), (4, 2, 4, 2), (6, 2, 6, 3), (8, 3, 8, 4), (12, 4, 12, 3), (8, 2, 8, 1),
    (16, 2, 8, 8), (9, 3, 6, 3), (10, 5, 10, 2), (4, 4, 4, 4), (0, 2, 4, 2), (64, 2, 8, 2),
]


@pytest.mark.parametrize("T,K,E,R", TINY)
@pytest.mark.parametrize("seed", [0, 1])
def test_layout_matches_brute_force(T, K, E, R, seed):
    cfg = inputs.custom_config(T, 8, E, K, R, routing="uniform", config_id=50 + seed)
    idx = inputs.make_topk_idx(cfg, seed)
    _assert_same(oracle.layout(idx, E, R), brute.layout(idx, E, R))


@pytest.mark.parametrize("seed", range(4))
def test_layout_brute_force_with_masks_duplicates_and_bad_ids(seed):
    rng = np.random.default_rng(100 + seed)
    T, K, E, R = 12, 4, 8, 4
    idx = rng.integers(-1, E, size=(T, K)).astype(np.int32)      # duplicates and -1 masks
    if seed >= 2:
        idx[rng.integers(0, T), rng.integers(0, K)] = E + 3       # out-of-range id
        idx[rng.integers(0, T), rng.integers(0, K)] = -7
    lay, ref = oracle.layout(idx, E, R), brute.layout(idx, E, R)
    _assert_same(lay, ref)
    assert lay.status == (1 if seed >= 2 else 0)


def test_layout_all_masked_and_all_to_one_expert():
    idx = -np.ones((8, 2), np.int32)
    lay = oracle.layout(idx, 4, 2)
    assert lay.n_recv == 0 and lay.n_pairs == 0 and (lay.recv_slot == -1).all()
    idx = np.zeros((8, 1), np.int32)
    lay = oracle.layout(idx, 4, 2)
    _assert_same(lay, brute.layout(idx, 4, 2))
    assert list(lay.rank_rows) == [8, 0] and list(lay.recv_slot[:, 0]) == list(range(8))


@pytest.mark.parametrize("name", ["C1", "C2", "C3", "C4"])
def test_layout_matches_numpy_library_routines(name):
    cfg = inputs.CONFIGS[name]
    idx = inputs.make_topk_idx(cfg)
    T, K, E, R = cfg.T, cfg.K, cfg.E, cfg.R
    El, Tr = E // R, T // R
    lay = oracle.layout(idx, E, R)
    flat = idx.ravel()
    # counts and scans: bincount / cumsum
    counts = np.bincount(flat, minlength=E)
    np.testing.assert_array_equal(lay.expert_counts, counts)
    np.testing.assert_array_equal(lay.expert_offsets, np.concatenate([[0], np.cumsum(counts)]))
    assert lay.expert_counts.sum() == T * K                       # counts sum to T*k
    # pair_slot is the inverse of the stable sort by expert id
    order = np.argsort(flat, kind="stable")
    inv = np.empty_like(order)
    inv[order] = np.arange(order.size)
    np.testing.assert_array_equal(lay.pair_slot.ravel(), inv)
    np.testing.assert_array_equal(lay.pair_token, order // K)
    # hits: receive rows
    hit = np.zeros((T, R), dtype=np.int64)
    hit[np.repeat(np.arange(T), K), flat // El] = 1
    rows = hit.sum(0)
    offs = np.concatenate([[0], np.cumsum(rows)])
    np.testing.assert_array_equal(lay.rank_rows, rows)
    np.testing.assert_array_equal(lay.rank_row_offsets, offs)
    excl = np.cumsum(hit, axis=0) - hit                           # tokens t' < t hitting r
    r_of = idx // El
    np.testing.assert_array_equal(lay.recv_slot, offs[r_of] + excl[np.arange(T)[:, None], r_of])
    # unique (token, rank) pairs = receive rows; bounded by T*min(K,R)
    uniq = len(set(zip(np.repeat(np.arange(T), K).tolist(), (flat // El).tolist())))
    assert lay.n_recv == uniq <= T * min(K, R)
    # per-source segmentation
    seg = np.add.reduceat(hit, np.arange(0, T, Tr), axis=0)       # [s, r]
    want = offs[:R, None] + np.concatenate([np.zeros((R, 1), np.int64), np.cumsum(seg.T, axis=1)], axis=1)
    np.testing.assert_array_equal(lay.src_row_offsets, want)
    # inverse maps
    np.testing.assert_array_equal(lay.recv_token[lay.recv_slot.ravel()], np.repeat(np.arange(T), K))
    np.testing.assert_array_equal(lay.pair_row[lay.pair_slot.ravel()], lay.recv_slot.ravel())
    # inside a rank the rows are ordered by token
    for r in range(R):
        seg_tok = lay.recv_token[offs[r]:offs[r + 1]]
        assert (np.diff(seg_tok) > 0).all()
    # inside an expert, (t,k) increases with the slot
    key = order                                                    # flat (t,k) index per pair slot
    for e in range(E):
        s = key[lay.expert_offsets[e]:lay.expert_offsets[e + 1]]
        assert (np.diff(s) > 0).all()


def test_closed_forms_single_rank_and_one_expert_per_rank():
    cfg = inputs.custom_config(32, 8, 16, 4, 1)
    idx = inputs.make_topk_idx(cfg)
    lay = oracle.layout(idx, 16, 1)
    np.testing.assert_array_equal(lay.recv_slot, np.repeat(np.arange(32), 4).reshape(32, 4))   # R=1: row = t
    assert lay.n_recv == 32
    cfg = inputs.custom_config(32, 8, 8, 3, 8)
    idx = inputs.make_topk_idx(cfg)
    lay = oracle.layout(idx, 8, 8)
    np.testing.assert_array_equal(lay.recv_slot, lay.pair_slot)   # E=R: the two spaces coincide
    assert lay.n_recv == 32 * 3
    np.testing.assert_array_equal(lay.pair_row, np.arange(lay.n_pairs))


def _read_golden(path):
    meta, rows = {}, []
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        if ":" in line:
            rows.append([int(v) for v in line.split(":")[1].split()])
        else:
            k, v = line.split()
            meta[k] = int(v)
    return meta, np.array(rows, dtype=np.int32)


def test_figure3_caption_case():
    meta, idx = _read_golden(os.path.join(GOLDEN, "fig3_caption_case.txt"))
    T, K, E, R = meta["T"], meta["K"], meta["E"], meta["R"]
    assert idx.shape == (T, K)
    El, Tr = E // R, T // R
    for t in range(T):      # the fixture obeys the caption: one expert on each remote rank
        assert sorted(idx[t] // El) == [r for r in range(R) if r != t // Tr]
    lay = oracle.layout(idx, E, R)
    assert list(lay.rank_rows) == [2 * T // 3] * R
    assert lay.n_recv == 2 * T and lay.n_pairs == T * K
    assert lay.n_recv < R * T                                     # dense all-gather delivers R*T rows
    for r in range(R):
        seg = np.diff(lay.src_row_offsets[r])
        assert seg[r] == 0 and all(seg[s] == Tr for s in range(R) if s != r)
    _assert_same(lay, brute.layout(idx, E, R))


@pytest.mark.parametrize("name,expect", [("C1", 1.571), ("C2", 2.000), ("C4", 5.295)])
def test_generator_reaches_the_expected_number_of_ranks(name, expect):
    """Uniform routing without replacement: E[distinct ranks per token] =
    R * (1 - C(E-El, K) / C(E, K)); the burst of C4 changes it only in the 3rd digit."""
    cfg = inputs.CONFIGS[name]
    El = cfg.E // cfg.R
    closed = cfg.R * (1 - math.comb(cfg.E - El, cfg.K) / math.comb(cfg.E, cfg.K))
    assert abs(closed - expect) < 2e-3
    lay = oracle.layout(inputs.make_topk_idx(cfg), cfg.E, cfg.R)
    tol = 0.25 if cfg.T < 1000 else 0.03
    assert abs(lay.n_recv / cfg.T - closed) < tol


def test_generators_are_seeded_and_distinct_per_token():
    for name, cfg in inputs.CONFIGS.items():
        a, b = inputs.make_topk_idx(cfg), inputs.make_topk_idx(cfg)
        np.testing.assert_array_equal(a, b)
        assert a.dtype == np.int32 and a.min() >= 0 and a.max() < cfg.E
        assert all(len(set(row)) == cfg.K for row in a[:256])
        w = inputs.make_topk_weights(cfg)
        np.testing.assert_allclose(w.sum(1), 1.0, rtol=1e-6)
    c4 = inputs.CONFIGS["C4"]
    idx = inputs.make_topk_idx(c4)
    assert (idx == 0).any(axis=1).sum() >= round(0.1 * c4.T)      # the hot-expert burst
    c3 = inputs.CONFIGS["C3"]
    cnt = np.bincount(inputs.make_topk_idx(c3).ravel(), minlength=c3.E)
    assert cnt.max() > 8 * np.median(cnt)                          # Zipf skew
