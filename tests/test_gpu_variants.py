"""CUDA variants around the path vs their oracle definitions, bit for bit: expanded dispatch
(one physical row per pair), combine with per-rank partial outputs, and the dense
all-gather / reduce-scatter formulation on the same logical ranks."""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import SENTINEL, dev_bf16, guarded, guards_intact, host_bits
from paper_2609_40093_b200 import ep, inputs

pytestmark = pytest.mark.gpu

CASES = [  # T, H, E, K, R, routing
    (64, 256, 8, 2, 2, "uniform"),
    (256, 4096, 8, 2, 8, "uniform"),
    (512, 2048, 128, 8, 8, "zipf"),
    (96, 2880, 32, 4, 4, "uniform"),
    (40, 520, 16, 4, 1, "uniform"),
    (48, 72, 16, 3, 16, "uniform"),
    (320, 136, 512, 10, 8, "zipf"),
    (128, 64, 64, 32, 32, "uniform"),
    (16, 16384, 8, 2, 4, "uniform"),       # rows longer than one pass of the widest thread group
]


def _setup(T, H, E, K, R, routing, mask=False):
    cfg = inputs.custom_config(T, H, E, K, R, routing=routing, config_id=90)
    d = inputs.make_inputs(cfg)
    idx, w, x = d["topk_idx"], d["topk_weights"], d["x"]
    if mask:
        idx = idx.copy()
        idx[1, :] = -1
        idx[2, 0] = -1
        idx[3, K - 1] = idx[3, 0]              # the same expert twice
    ref = oracle.layout(idx, E, R)
    out = inputs.make_out(cfg, max(1, ref.n_pairs), seed=2)
    idx_d = torch.from_numpy(idx).cuda()
    lay = ep.ep_layout(idx_d, E, R)
    return cfg, idx, w, x, ref, out, idx_d, lay


@pytest.mark.parametrize("T,H,E,K,R,routing", CASES)
def test_expanded_dispatch_and_group(T, H, E, K, R, routing):
    cfg, idx, w, x, ref, out, idx_d, lay = _setup(T, H, E, K, R, routing)
    recv_ref = oracle.dispatch(x, ref.recv_slot, ref.n_recv)
    want = oracle.group(recv_ref, ref.pair_row)
    whole, grouped = guarded(ref.n_pairs + 2, H)
    ep.ep_dispatch(dev_bf16(x), lay.pair_slot, grouped, E, R)          # x[t] straight to its pair rows
    got = host_bits(grouped)
    np.testing.assert_array_equal(got[:ref.n_pairs], want)
    assert (got[ref.n_pairs:] == SENTINEL).all() and guards_intact(whole)


@pytest.mark.parametrize("mask", [False, True])
@pytest.mark.parametrize("T,H,E,K,R,routing", CASES)
def test_combine_partial(T, H, E, K, R, routing, mask):
    cfg, idx, w, x, ref, out, idx_d, lay = _setup(T, H, E, K, R, routing, mask)
    want_partial, want_y = oracle.combine_partial(out, ref.pair_slot, ref.recv_slot, w, ref.n_recv + 2, fill=SENTINEL)
    pwhole, partial = guarded(ref.n_recv + 2, H)
    ywhole, y = guarded(T, H)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ep.ep_combine_partial(dev_bf16(out), lay, torch.from_numpy(w).cuda(), partial, y, E, R, status=status)
    np.testing.assert_array_equal(host_bits(partial), want_partial)
    np.testing.assert_array_equal(host_bits(y), want_y)
    assert guards_intact(pwhole) and guards_intact(ywhole) and ep.ep_status(status) == 0


@pytest.mark.parametrize("mask", [False, True])
@pytest.mark.parametrize("T,H,E,K,R,routing", CASES)
def test_dense_allgather_and_reduce_scatter(T, H, E, K, R, routing, mask):
    cfg, idx, w, x, ref, out, idx_d, lay = _setup(T, H, E, K, R, routing, mask)
    gwhole, gathered = guarded(R * T, H)
    ep.ep_dense_allgather(dev_bf16(x), gathered, K, E, R)
    np.testing.assert_array_equal(host_bits(gathered), oracle.dense_allgather(x, R))
    assert guards_intact(gwhole)
    want_dense, want_y = oracle.dense_reduce_scatter(idx, out, ref.pair_slot, w, E, R)
    dwhole, dense = guarded(R * T, H)
    ywhole, y = guarded(T, H)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ep.ep_dense_reduce_scatter(idx_d, dev_bf16(out), lay.pair_slot, torch.from_numpy(w).cuda(), dense, y, E, R,
                               status=status)
    np.testing.assert_array_equal(host_bits(dense), want_dense)
    np.testing.assert_array_equal(host_bits(y), want_y)
    assert guards_intact(dwhole) and guards_intact(ywhole) and ep.ep_status(status) == 0
    assert R * T >= ref.n_recv                                          # the dense form never moves fewer rows


def test_variants_on_buffers_past_four_gib():
    """65536 tokens of 7168 elements, 8 of 256 experts on 8 ranks: the dense buffers and the pair space hold
    7.5 GB each, the partial rows 4.9 GB. Sampled tokens (those that use the last rows of every buffer among
    them) against the oracle run on the sample as a batch of its own, its slots renumbered."""
    T, H, E, K, R = 65536, 7168, 256, 8, 8
    cfg = inputs.custom_config(T, H, E, K, R, routing="burst", config_id=91)
    idx, w = inputs.make_topk_idx(cfg), inputs.make_topk_weights(cfg)
    ref = oracle.layout(idx, E, R)
    idx_d, w_d = torch.from_numpy(idx).cuda(), torch.from_numpy(w).cuda()
    lay = ep.ep_layout(idx_d, E, R)
    rng = np.random.default_rng(91)
    block_rows = 1 << 15
    block = inputs.make_out(cfg, block_rows, seed=3)
    block_d = dev_bf16(block)

    def rows_of(buf, rows):
        return host_bits(buf[torch.from_numpy(np.asarray(rows, dtype=np.int64)).cuda()])

    # dense all-gather: every rank's copy of every token
    x = block[:, :]                                                    # 32768 seeded rows, repeated twice
    x_d = block_d.repeat(T // block_rows, 1)
    big = torch.empty(R * T, H, dtype=torch.bfloat16, device="cuda")
    ep.ep_dense_allgather(x_d, big, K, E, R)
    rows = np.unique(np.concatenate([np.arange(R * T - 64, R * T), np.arange(64), rng.integers(0, R * T, 4096)]))
    np.testing.assert_array_equal(rows_of(big, rows), x[(rows % T) % block_rows])
    del x_d

    # expert outputs in the pair space: the seeded block repeated (2^32 bytes is not a whole number of rows)
    assert ref.n_pairs == R * T
    out = big
    for first in range(0, ref.n_pairs, block_rows):
        out[first:first + block_rows] = block_d
    toks = np.unique(np.concatenate([ref.pair_token[-256:], ref.recv_token[-256:], np.arange(32), np.arange(T - 32, T),
                                     rng.integers(0, T, 512)]))
    toks = toks[:len(toks) - len(toks) % R]
    used = np.unique(ref.pair_slot[toks])
    pair_c = np.searchsorted(used, ref.pair_slot[toks]).astype(np.int32)
    out_c = block[used % block_rows]
    used_recv = np.unique(ref.recv_slot[toks])
    recv_c = np.searchsorted(used_recv, ref.recv_slot[toks]).astype(np.int32)

    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    partial = torch.empty(ref.n_recv, H, dtype=torch.bfloat16, device="cuda")
    y = torch.empty(T, H, dtype=torch.bfloat16, device="cuda")
    ep.ep_combine_partial(out, lay, w_d, partial, y, E, R, status=status)
    want_partial, want_y = oracle.combine_partial(out_c, pair_c, recv_c, w[toks], len(used_recv))
    np.testing.assert_array_equal(rows_of(partial, used_recv), want_partial)
    np.testing.assert_array_equal(rows_of(y, toks), want_y)
    del partial

    dense = torch.empty(R * T, H, dtype=torch.bfloat16, device="cuda")
    y.zero_()
    ep.ep_dense_reduce_scatter(idx_d, out, lay.pair_slot, w_d, dense, y, E, R, status=status)
    want_dense, want_y = oracle.dense_reduce_scatter(idx[toks], out_c, pair_c, w[toks], E, R)
    n = len(toks)
    dense_rows = (np.arange(R)[:, None] * T + toks[None, :]).ravel()   # dense[r*T + t] <-> sample's [r*n + i]
    np.testing.assert_array_equal(rows_of(dense, dense_rows), want_dense)
    np.testing.assert_array_equal(rows_of(y, toks), want_y)
    assert ep.ep_status(status) == 0
