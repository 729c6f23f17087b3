"""CUDA path vs the CPU oracle, element by element, through the C ABI.

Integer outputs (layout, slots) and dispatched rows must be bit-exact. Combine must
be within max(4e-3*|ref|, 1e-3) of the exact (fp64) sum; it is also compared bit
for bit with the oracle's fp32 chain, which the kernel reproduces because both
use correctly rounded fused multiply-adds in the same order.
"""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import (GUARD, SENTINEL, assert_layout_equal, dev_bf16, guarded, guards_intact, host_bits,
                      within_tolerance)
from paper_2609_40093_b200 import ep, inputs

pytestmark = pytest.mark.gpu

EDGE = [  # T, H, E, K, R, routing
    (1, 8, 1, 1, 1, "uniform"),
    (2, 16, 2, 1, 2, "uniform"),
    (8, 264, 8, 2, 4, "uniform"),          # H % 8 == 0 but ragged against every thread-group size
    (96, 2880, 32, 4, 4, "uniform"),       # hidden size of a 2880-wide model: 360 vectors
    (64, 1032, 16, 1, 8, "uniform"),       # K = 1
    (40, 520, 16, 4, 1, "uniform"),        # R = 1
    (48, 72, 16, 3, 16, "uniform"),        # E = R
    (1000, 136, 512, 10, 8, "zipf"),       # 10 of 512, the finest model the paper names
    (1088, 64, 4096, 32, 64, "uniform"),   # every maximum at once: K=32, E=4096, R=64 (a 7-CTA cluster of 197 KB CTAs)
    (320, 8, 4096, 32, 64, "uniform"),     # the same limits, two CTAs
    (3200, 8, 4096, 32, 64, "uniform"),    # the same limits past the cluster: 17 CTAs, two kernels
    (40000, 8, 16, 2, 8, "uniform"),       # more than 1024*32 tokens: layout tiles of 64 tokens, 16-byte rows
    (33 * 8, 40, 24, 5, 8, "zipf_identity"),
    (65536, 8, 256, 8, 8, "burst"),        # 128 layout CTAs, tiles of 64 tokens, half a million pairs
    (2048, 24, 128, 6, 8, "zipf"),         # the largest batch that takes the one-cluster layout
    (16, 16384, 8, 2, 4, "uniform"),       # rows longer than one pass of the widest thread group
    (64, 8200, 64, 20, 4, "uniform"),      # K > 8: combine's chunked path; 1025 vectors per row
]


def _run_layout(idx, E, R, fill=-7):
    T, K = idx.shape
    lay = ep.alloc_layout(T, K, E, R, fill=fill)
    ep.ep_layout(torch.from_numpy(idx).cuda(), E, R, out=lay)
    return lay


def _full_path_check(cfg, idx, w, x, check_combine_rows=None):
    T, K, H, E, R = cfg.T, cfg.K, cfg.H, cfg.E, cfg.R
    ref = oracle.layout(idx, E, R)
    lay = _run_layout(idx, E, R)
    assert_layout_equal(lay, ref)
    assert ep.ep_status(lay.status) == ref.status

    # dispatch into a guarded buffer: rows beyond N_recv and the guards stay untouched
    x_d = dev_bf16(x)
    spare = 3
    whole, recv = guarded(ref.n_recv + spare, H)
    ep.ep_dispatch(x_d, lay.recv_slot, recv, E, R, status=lay.status)
    got = host_bits(recv)
    want = oracle.dispatch(x, ref.recv_slot, ref.n_recv + spare, fill=SENTINEL)
    np.testing.assert_array_equal(got, want)
    assert guards_intact(whole)

    # local grouping: grouped[p] = recv[pair_row[p]]
    gwhole, grouped = guarded(ref.n_pairs + spare, H)
    ep.ep_group(recv, lay, grouped, E, R, status=lay.status)
    gb = host_bits(grouped)
    np.testing.assert_array_equal(gb[:ref.n_pairs], want[ref.pair_row] if ref.n_pairs else gb[:0])
    assert (gb[ref.n_pairs:] == SENTINEL).all() and guards_intact(gwhole)

    # combine over independent expert outputs in the pair space
    out = inputs.make_out(cfg, max(1, ref.n_pairs), seed=1)
    w_d = torch.from_numpy(w).cuda()
    ywhole, y = guarded(T, H)
    ep.ep_combine(dev_bf16(out), lay.pair_slot, w_d, y, E, R, status=lay.status)
    yb = host_bits(y)
    sel = slice(None) if check_combine_rows is None else check_combine_rows
    y32 = oracle.combine_f32(out, ref.pair_slot[sel], w[sel])
    y64 = oracle.combine_f64(out, ref.pair_slot[sel], w[sel])
    assert within_tolerance(yb[sel], y64).all()
    np.testing.assert_array_equal(yb[sel], y32)          # same fma chain => same bits
    assert guards_intact(ywhole)
    assert ep.ep_status(lay.status) == ref.status
    return lay, ref


@pytest.mark.parametrize("name", ["C1", "C2", "C3"])
def test_configs_full_path(name):
    cfg = inputs.CONFIGS[name]
    d = inputs.make_inputs(cfg)
    _full_path_check(cfg, d["topk_idx"], d["topk_weights"], d["x"])


@pytest.mark.parametrize("T,H,E,K,R,routing", EDGE)
def test_edge_shapes_full_path(T, H, E, K, R, routing):
    cfg = inputs.custom_config(T, H, E, K, R, routing=routing, config_id=60)
    d = inputs.make_inputs(cfg)
    _full_path_check(cfg, d["topk_idx"], d["topk_weights"], d["x"])


def test_masked_duplicate_and_bad_ids():
    rng = np.random.default_rng(3)
    T, H, E, K, R = 256, 128, 16, 6, 4
    cfg = inputs.custom_config(T, H, E, K, R, config_id=61)
    d = inputs.make_inputs(cfg)
    idx = rng.integers(-1, E, size=(T, K)).astype(np.int32)        # duplicates inside a token, -1 masks
    idx[5, :] = -1                                                  # a token that goes nowhere
    idx[7, :] = 3                                                   # the same expert K times
    lay, ref = _full_path_check(cfg, idx, d["topk_weights"], d["x"])
    assert ref.status == 0
    idx[11, 2] = E + 5
    idx[200, 0] = -9
    lay, ref = _full_path_check(cfg, idx, d["topk_weights"], d["x"])
    assert ref.status == ep.STATUS_BAD_INDEX


def test_wide_top_k_with_masks():
    rng = np.random.default_rng(9)
    T, H, E, K, R = 96, 264, 96, 32, 8
    cfg = inputs.custom_config(T, H, E, K, R, config_id=63)
    d = inputs.make_inputs(cfg)
    idx = d["topk_idx"].copy()
    idx[rng.random((T, K)) < 0.3] = -1
    idx[0, :] = -1
    _full_path_check(cfg, idx, d["topk_weights"], d["x"])


def test_all_tokens_to_one_expert_and_all_masked():
    T, H, E, K, R = 512, 64, 8, 2, 4
    cfg = inputs.custom_config(T, H, E, K, R, config_id=62)
    d = inputs.make_inputs(cfg)
    idx = np.zeros((T, K), np.int32)
    idx[:, 1] = 1                                                   # experts 0 and 1, both on rank 0
    _full_path_check(cfg, idx, d["topk_weights"], d["x"])
    _full_path_check(cfg, -np.ones((T, K), np.int32), d["topk_weights"], d["x"])


def test_layout_on_many_random_shapes():
    """Seeded sweep over shapes that exercise the single-CTA, cluster and multi-CTA forms of the
    layout, with masked and repeated ids mixed in; every integer output against the oracle."""
    rng = np.random.default_rng(11)
    for trial in range(48):
        R = int(rng.choice([1, 2, 3, 4, 8, 16]))
        E = R * int(rng.choice([1, 2, 5, 16, 32]))
        K = int(rng.integers(1, min(8, E) + 1))
        T = R * int(rng.integers(1, [40, 300, 1200][trial % 3]))
        idx = rng.integers(0, E, size=(T, K)).astype(np.int32)
        if trial % 4 == 1:
            idx[rng.random((T, K)) < 0.15] = -1
        if trial % 8 == 3:
            idx[int(rng.integers(0, T)), int(rng.integers(0, K))] = E + 1
        ref = oracle.layout(idx, E, R)
        lay = _run_layout(idx, E, R)
        assert_layout_equal(lay, ref)
        assert ep.ep_status(lay.status) == ref.status, (trial, T, K, E, R)


def test_layout_halves_on_many_random_shapes():
    """The two halves of the layout, called one after the other on the same workspace, over batch sizes
    around every switch of the launch plan (one CTA, one cluster, many CTAs, larger tiles)."""
    rng = np.random.default_rng(12)
    sizes = [1, 30, 33, 1000, 1024, 1025, 2047, 3000, 4097, 8192, 9000, 20000, 32768, 33000, 50000]
    for trial, tokens in enumerate(sizes):
        R = int(rng.choice([1, 2, 4, 8, 64] if trial % 5 == 4 else [1, 2, 4, 8]))
        T = max(R, tokens - tokens % R)
        E = R * int(rng.choice([1, 4, 32]))
        K = int(rng.integers(1, min(8, E) + 1))
        idx = rng.integers(0, E, size=(T, K)).astype(np.int32)
        if trial % 3 == 1:
            idx[rng.random((T, K)) < 0.2] = -1
        if trial % 4 == 2:
            idx[int(rng.integers(0, T)), 0] = -5
        ref = oracle.layout(idx, E, R)
        idx_d = torch.from_numpy(idx).cuda()
        lay = ep.alloc_layout(T, K, E, R, fill=-7)
        ws = torch.empty(max(16, ep.ep_layout_workspace_bytes(T, K, E, R)), dtype=torch.uint8, device="cuda")
        ep.ep_layout_ranks(idx_d, E, R, lay, ws)
        ep.ep_layout_pairs(idx_d, E, R, lay, ws)
        assert_layout_equal(lay, ref)
        assert ep.ep_status(lay.status) == ref.status, (T, K, E, R)


@pytest.mark.parametrize("name", ["C1", "C3", "C4"])
def test_layout_halves_on_two_streams_equal_the_whole(name):
    """ep_layout_ranks and ep_layout_pairs, each on its own stream with its own workspace, fill
    disjoint fields; together they must give what ep_layout gives (and the oracle)."""
    cfg = inputs.CONFIGS[name]
    idx = inputs.make_topk_idx(cfg)
    idx[5 % cfg.T, 0] = -1
    ref = oracle.layout(idx, cfg.E, cfg.R)
    idx_d = torch.from_numpy(idx).cuda()
    lay = ep.alloc_layout(cfg.T, cfg.K, cfg.E, cfg.R, fill=-7)
    nbytes = max(16, ep.ep_layout_workspace_bytes(cfg.T, cfg.K, cfg.E, cfg.R))
    ws1, ws2 = (torch.empty(nbytes, dtype=torch.uint8, device="cuda") for _ in range(2))
    s1, s2 = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for _ in range(3):
        ep.ep_layout_pairs(idx_d, cfg.E, cfg.R, lay, ws2, stream=s2)
        ep.ep_layout_ranks(idx_d, cfg.E, cfg.R, lay, ws1, stream=s1)
    torch.cuda.synchronize()
    assert_layout_equal(lay, ref)
    assert ep.ep_status(lay.status) == ref.status


def test_whole_step_replays_from_a_cuda_graph():
    """No call of the path synchronises or allocates, so one step can be captured once and replayed
    on new routing tables and activations written into the same buffers."""
    cfg = inputs.CONFIGS["C3"]
    T, K, H, E, R = cfg.T, cfg.K, cfg.H, cfg.E, cfg.R
    idx_d = torch.zeros(T, K, dtype=torch.int32, device="cuda")
    w_d = torch.zeros(T, K, dtype=torch.float32, device="cuda")
    x_d = torch.zeros(T, H, dtype=torch.bfloat16, device="cuda")
    lay = ep.alloc_layout(T, K, E, R)
    ws = torch.empty(max(16, ep.ep_layout_workspace_bytes(T, K, E, R)), dtype=torch.uint8, device="cuda")
    recv = torch.zeros(T * min(K, R), H, dtype=torch.bfloat16, device="cuda")
    grouped = torch.zeros(T * K, H, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(T, H, dtype=torch.bfloat16, device="cuda")

    def step():
        ep.ep_layout(idx_d, E, R, out=lay, workspace=ws)
        ep.ep_dispatch(x_d, lay.recv_slot, recv, E, R, status=lay.status)
        ep.ep_group(recv, lay, grouped, E, R, status=lay.status)
        ep.ep_combine(grouped, lay.pair_slot, w_d, y, E, R, status=lay.status)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):                       # first calls (per-device set-up) outside the capture
        step()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for seed in (3, 4):
        d = inputs.make_inputs(cfg, seed)
        idx_d.copy_(torch.from_numpy(d["topk_idx"]))
        w_d.copy_(torch.from_numpy(d["topk_weights"]))
        x_d.copy_(dev_bf16(d["x"]))
        graph.replay()
        torch.cuda.synchronize()
        ref = oracle.layout(d["topk_idx"], E, R)
        want = oracle.combine_f32(oracle.dispatch(d["x"], ref.recv_slot, ref.n_recv)[ref.pair_row], ref.pair_slot,
                                  d["topk_weights"])
        np.testing.assert_array_equal(host_bits(y), want)
        assert ep.ep_status(lay.status) == 0


def test_two_stream_steps_replay_from_one_cuda_graph():
    """The form the benchmark times: three steps back to back, each one `ep_layout_dispatch` with a second
    stream (pair half of the layout beside dispatch, joined by the library's events) and a combine launched
    behind it, captured in one CUDA graph and replayed on new inputs. The last step's outputs against the oracle."""
    cfg = inputs.CONFIGS["C3"]
    T, K, H, E, R = cfg.T, cfg.K, cfg.H, cfg.E, cfg.R
    idx_d = torch.zeros(T, K, dtype=torch.int32, device="cuda")
    w_d = torch.zeros(T, K, dtype=torch.float32, device="cuda")
    x_d = torch.zeros(T, H, dtype=torch.bfloat16, device="cuda")
    out_d = torch.zeros(T * K, H, dtype=torch.bfloat16, device="cuda")
    lay = ep.alloc_layout(T, K, E, R)
    ws = torch.empty(2 * ep.ep_layout_workspace_bytes(T, K, E, R) + 256, dtype=torch.uint8, device="cuda")
    recv = torch.zeros(T * min(K, R), H, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(T, H, dtype=torch.bfloat16, device="cuda")
    pairs_stream = torch.cuda.Stream()

    def step():
        ep.ep_layout_dispatch(idx_d, x_d, recv, E, R, lay, ws, stream_pairs=pairs_stream)
        ep.ep_combine(out_d, lay.pair_slot, w_d, y, E, R, status=lay.status)

    warm = torch.cuda.Stream()
    with torch.cuda.stream(warm):
        step()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        for _ in range(3):
            step()
    for seed in (5, 6):
        d = inputs.make_inputs(cfg, seed)
        out = inputs.make_out(cfg, T * K, seed=seed)
        idx_d.copy_(torch.from_numpy(d["topk_idx"]))
        w_d.copy_(torch.from_numpy(d["topk_weights"]))
        x_d.copy_(dev_bf16(d["x"]))
        out_d.copy_(dev_bf16(out))
        recv.zero_(), y.zero_()
        graph.replay()
        torch.cuda.synchronize()
        ref = oracle.layout(d["topk_idx"], E, R)
        assert_layout_equal(lay, ref)
        np.testing.assert_array_equal(host_bits(recv)[:ref.n_recv], oracle.dispatch(d["x"], ref.recv_slot, ref.n_recv))
        np.testing.assert_array_equal(host_bits(y), oracle.combine_f32(out, ref.pair_slot, d["topk_weights"]))
        assert ep.ep_status(lay.status) == 0


def test_empty_batch():
    E, R, K, H = 8, 2, 2, 64
    lay = ep.alloc_layout(0, K, E, R, fill=-7)
    ep.ep_layout(torch.empty(0, K, dtype=torch.int32, device="cuda"), E, R, out=lay)
    assert (lay.expert_counts.cpu() == 0).all() and (lay.rank_row_offsets.cpu() == 0).all()
    assert (lay.expert_offsets.cpu() == 0).all() and (lay.src_row_offsets.cpu() == 0).all()
    assert ep.ep_status(lay.status) == 0
    x = torch.empty(0, H, dtype=torch.bfloat16, device="cuda")
    recv = torch.empty(1, H, dtype=torch.bfloat16, device="cuda")
    ep.ep_dispatch(x, lay.recv_slot, recv, E, R)
    ep.ep_combine(recv, lay.recv_slot, torch.empty(0, K, device="cuda"), x, E, R)


def test_identity_expert_roundtrip_and_one_hot_weights():
    cfg = inputs.CONFIGS["C2"]
    d = inputs.make_inputs(cfg)
    idx, w, x = d["topk_idx"], d["topk_weights"], d["x"]
    lay = _run_layout(idx, cfg.E, cfg.R)
    n_recv = int(lay.rank_row_offsets[-1])
    x_d = dev_bf16(x)
    recv = torch.zeros(n_recv, cfg.H, dtype=torch.bfloat16, device="cuda")
    ep.ep_dispatch(x_d, lay.recv_slot, recv, cfg.E, cfg.R)
    y = torch.zeros_like(x_d)
    ep.ep_combine(recv, lay.recv_slot, torch.from_numpy(w).cuda(), y, cfg.E, cfg.R)
    assert within_tolerance(host_bits(y), inputs.bf16_bits_to_f32(x).astype(np.float64)).all()
    for kstar in range(cfg.K):                                     # one-hot weights: a bit copy of the chosen row
        onehot = torch.zeros(cfg.T, cfg.K, device="cuda")
        onehot[:, kstar] = 1.0
        ep.ep_combine(recv, lay.recv_slot, onehot, y, cfg.E, cfg.R)
        np.testing.assert_array_equal(host_bits(y), x)


def test_combine_uses_fused_multiply_add():
    """acc = -c, then w*v = c + c*2^-23: one rounding leaves c*2^-23, a rounded product 2^-23."""
    c = 1.0078125                                           # 1 + 2^-7, a bf16 number
    out = inputs.to_bf16_bits(np.full((2, 64), c, dtype=np.float32))
    slot = np.tile(np.array([[0, 1]], dtype=np.int32), (4, 1))
    w = np.tile(np.array([[-1.0, 1.0 + 2.0 ** -23]], dtype=np.float32), (4, 1))
    y = torch.zeros(4, 64, dtype=torch.bfloat16, device="cuda")
    ep.ep_combine(dev_bf16(out), torch.from_numpy(slot).cuda(), torch.from_numpy(w).cuda(), y, 4, 4)
    got = inputs.bf16_bits_to_f32(host_bits(y))
    assert (got == np.float32(c * 2.0 ** -23)).all()
    np.testing.assert_array_equal(host_bits(y), oracle.combine_f32(out, slot, w))


def test_capacity_overflow_is_skipped_and_flagged():
    cfg = inputs.CONFIGS["C1"]
    d = inputs.make_inputs(cfg)
    idx, w, x = d["topk_idx"], d["topk_weights"], d["x"]
    ref = oracle.layout(idx, cfg.E, cfg.R)
    lay = _run_layout(idx, cfg.E, cfg.R)
    cap = ref.n_recv - 10
    whole, recv = guarded(cap, cfg.H)
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    ep.ep_dispatch(dev_bf16(x), lay.recv_slot, recv, cfg.E, cfg.R, status=status)
    assert ep.ep_status(status) == ep.STATUS_CAPACITY
    assert guards_intact(whole)
    np.testing.assert_array_equal(host_bits(recv), oracle.dispatch(x, ref.recv_slot, ref.n_recv)[:cap])
    # combine: slots beyond out_rows contribute nothing
    out = inputs.make_out(cfg, ref.n_pairs)
    status.zero_()
    y = torch.zeros(cfg.T, cfg.H, dtype=torch.bfloat16, device="cuda")
    short = ref.n_pairs - 7
    ep.ep_combine(dev_bf16(out[:short]), lay.pair_slot, torch.from_numpy(w).cuda(), y, cfg.E, cfg.R, status=status)
    assert ep.ep_status(status) == ep.STATUS_CAPACITY
    masked = np.where(ref.pair_slot >= short, -1, ref.pair_slot).astype(np.int32)
    np.testing.assert_array_equal(host_bits(y), oracle.combine_f32(out[:short], masked, w))


def test_results_are_run_to_run_identical():
    cfg = inputs.CONFIGS["C3"]
    idx = inputs.make_topk_idx(cfg)
    a = _run_layout(idx, cfg.E, cfg.R)
    b = _run_layout(idx, cfg.E, cfg.R)
    for f in ["recv_slot", "pair_slot", "recv_token", "pair_row", "pair_token"]:
        n = int(a.rank_row_offsets[-1]) if f == "recv_token" else None
        assert torch.equal(getattr(a, f).flatten()[:n], getattr(b, f).flatten()[:n]), f


def test_host_step_matches_oracle():
    cfg = inputs.CONFIGS["C3"]
    d = inputs.make_inputs(cfg)
    idx, w, x = d["topk_idx"], d["topk_weights"], d["x"]
    xh = torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).pin_memory()
    ih, wh = torch.from_numpy(idx).pin_memory(), torch.from_numpy(w).pin_memory()
    yh = torch.zeros(cfg.T, cfg.H, dtype=torch.bfloat16).pin_memory()
    sh = torch.full((1,), -1, dtype=torch.int32).pin_memory()
    arena = torch.empty(ep.ep_host_step_arena_bytes(cfg.T, cfg.K, cfg.H, cfg.E, cfg.R), dtype=torch.uint8, device="cuda")
    ep.ep_host_step(xh, ih, wh, yh, arena, cfg.E, cfg.R, status_host=sh)
    torch.cuda.synchronize()
    assert int(sh[0]) == 0
    ref = oracle.layout(idx, cfg.E, cfg.R)
    recv = oracle.dispatch(x, ref.recv_slot, ref.n_recv)
    want = oracle.combine_f32(recv[ref.pair_row], ref.pair_slot, w)
    np.testing.assert_array_equal(yh.view(torch.int16).numpy().view(np.uint16), want)


@pytest.mark.parametrize("chunks", [1, 3, 8])
def test_pipelined_host_step_matches_oracle(chunks):
    """Uploads, kernels and downloads of token chunks overlap on three streams; the result is the
    same as the one-stream step, also when two calls follow each other without a synchronisation."""
    cfg = inputs.CONFIGS["C3"]
    ref_y = []
    hosts = []
    for seed in (0, 1):
        d = inputs.make_inputs(cfg, seed)
        idx, w, x = d["topk_idx"], d["topk_weights"], d["x"]
        ref = oracle.layout(idx, cfg.E, cfg.R)
        recv = oracle.dispatch(x, ref.recv_slot, ref.n_recv)
        ref_y.append(oracle.combine_f32(recv[ref.pair_row], ref.pair_slot, w))
        hosts.append((torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).pin_memory(),
                      torch.from_numpy(idx).pin_memory(), torch.from_numpy(w).pin_memory(),
                      torch.zeros(cfg.T, cfg.H, dtype=torch.bfloat16).pin_memory(),
                      torch.full((1,), -1, dtype=torch.int32).pin_memory()))
    arena = torch.empty(ep.ep_host_step_arena_bytes(cfg.T, cfg.K, cfg.H, cfg.E, cfg.R), dtype=torch.uint8, device="cuda")
    s_in, s_comp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for xh, ih, wh, yh, sh in hosts:                    # back to back, same arena, no synchronisation between
        ep.ep_host_step_pipelined(xh, ih, wh, yh, arena, cfg.E, cfg.R, chunks, s_in, s_comp, s_out, status_host=sh)
    torch.cuda.synchronize()
    for (xh, ih, wh, yh, sh), want in zip(hosts, ref_y):
        assert int(sh[0]) == 0
        np.testing.assert_array_equal(yh.view(torch.int16).numpy().view(np.uint16), want)


@pytest.mark.parametrize("chunks", [1, 4])
def test_pipelined_host_steps_alternate_between_two_copies_of_the_transfer_buffers(chunks):
    """Five different batches back to back with caller-owned step events and no synchronisation: call n uses
    copy n & 1 of x / topk_idx / topk_weights / y / status and waits only for call n - 2. Every result and
    every status word (one batch carries an id outside [-1, E)) against the oracle."""
    cfg = inputs.CONFIGS["C3"]
    hosts, wants = [], []
    for seed in range(5):
        d = inputs.make_inputs(cfg, seed)
        idx, w, x = d["topk_idx"].copy(), d["topk_weights"], d["x"]
        if seed == 2:
            idx[17, 3] = cfg.E + 5
        ref = oracle.layout(idx, cfg.E, cfg.R)
        recv = oracle.dispatch(x, ref.recv_slot, ref.n_recv)
        wants.append((oracle.combine_f32(recv[ref.pair_row], ref.pair_slot, w), ref.status))
        hosts.append((torch.from_numpy(x.view(np.int16)).view(torch.bfloat16).pin_memory(),
                      torch.from_numpy(idx).pin_memory(), torch.from_numpy(w).pin_memory(),
                      torch.zeros(cfg.T, cfg.H, dtype=torch.bfloat16).pin_memory(),
                      torch.full((1,), -1, dtype=torch.int32).pin_memory()))
    arena = torch.empty(ep.ep_host_step_arena_bytes(cfg.T, cfg.K, cfg.H, cfg.E, cfg.R), dtype=torch.uint8, device="cuda")
    s_in, s_comp, s_out = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    events = ep.StepEvents()
    torch.cuda.synchronize()
    for n, (xh, ih, wh, yh, sh) in enumerate(hosts):
        ep.ep_host_step_pipelined(xh, ih, wh, yh, arena, cfg.E, cfg.R, chunks, s_in, s_comp, s_out, status_host=sh,
                                  round=n, step_events=events)
    torch.cuda.synchronize()
    for (xh, ih, wh, yh, sh), (want, status) in zip(hosts, wants):
        assert int(sh[0]) == status
        np.testing.assert_array_equal(yh.view(torch.int16).numpy().view(np.uint16), want)
    assert wants[2][1] == ep.STATUS_BAD_INDEX


def test_host_staged_dispatch_both_arms():
    """Receive buffer in mapped pinned host memory: kernel stores and the copy-engine arm."""
    cfg = inputs.CONFIGS["C5"]
    d = inputs.make_inputs(cfg)
    idx, x = d["topk_idx"], d["x"]
    ref = oracle.layout(idx, cfg.E, cfg.R)
    want = oracle.dispatch(x, ref.recv_slot, ref.n_recv)
    lay = _run_layout(idx, cfg.E, cfg.R)
    x_d = dev_bf16(x)
    # (i) the dispatch kernel stores straight into pinned host memory
    recv_h = torch.zeros(ref.n_recv, cfg.H, dtype=torch.bfloat16).pin_memory()
    ep.ep_dispatch(x_d, lay.recv_slot, recv_h, cfg.E, cfg.R)
    torch.cuda.synchronize()
    np.testing.assert_array_equal(recv_h.view(torch.int16).numpy().view(np.uint16), want)
    # (ii) pack on the device, then one copy-engine transfer per destination rank
    staging = torch.zeros(ref.n_recv, cfg.H, dtype=torch.bfloat16, device="cuda")
    for offsets in (lay.rank_row_offsets.cpu(), None):
        recv_h.zero_()
        ep.ep_dispatch_copy_engine(x_d, lay.recv_slot, staging, recv_h, cfg.E, cfg.R, rank_row_offsets_host=offsets)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(recv_h.view(torch.int16).numpy().view(np.uint16), want)


def test_largest_config_in_full():
    """C4 in the launch configuration the benchmark times: integer outputs, the dispatched buffer,
    the grouped buffer and all 8192 combined rows against the oracle."""
    cfg = inputs.CONFIGS["C4"]
    d = inputs.make_inputs(cfg)
    _full_path_check(cfg, d["topk_idx"], d["topk_weights"], d["x"])


FUSED = [  # T, H, E, K, R, routing: ep_layout_dispatch on batches that take its one-launch form (K = 9 or above 10,
           # or R > 32, up to 1024 tokens), on batches the lean layout kernels take instead, and on larger ones
    (64, 256, 8, 2, 2, "uniform"),         # C1: lean main kernel alone + dependent dispatch
    (256, 4096, 8, 2, 8, "uniform"),       # C2: the same, a full CTA
    (1, 8, 1, 1, 1, "uniform"),
    (2, 16, 2, 1, 2, "uniform"),
    (8, 264, 8, 2, 4, "uniform"),
    (96, 2880, 32, 4, 4, "uniform"),
    (40, 520, 16, 4, 1, "uniform"),        # R = 1, 40 tokens: a ragged last group
    (48, 72, 16, 3, 16, "uniform"),
    (1000, 136, 512, 10, 8, "zipf"),       # 10 of 512: four CTAs of the lean kernel pair
    (1024, 7168, 256, 8, 8, "burst"),      # four CTAs of the lean kernel pair, long rows
    (520, 72, 64, 6, 8, "zipf"),           # three CTAs of the lean kernel pair, the last one ragged
    (1023 - 1023 % 3, 40, 24, 5, 3, "zipf_identity"),
    (1024, 7168, 256, 9, 8, "uniform"),    # one launch: the largest batch of that form, long rows
    (96, 2880, 36, 9, 4, "uniform"),       # one launch, 360 vectors per row
    (512, 264, 48, 12, 16, "zipf"),        # one launch, K = 12
    (40, 520, 16, 11, 1, "uniform"),       # one launch, R = 1, a ragged last group
    (64, 8, 64, 16, 64, "uniform"),        # one launch, one token per rank
    (320, 64, 4096, 4, 64, "uniform"),     # one launch, E and R at their maxima
    (64, 64, 64, 32, 32, "uniform"),       # one launch, K at its maximum
    (1088, 64, 4096, 32, 64, "uniform"),   # does not fit one launch: falls back to the general kernels
    (2048, 24, 128, 6, 8, "zipf"),         # more than 1024 tokens
]


@pytest.mark.parametrize("T,H,E,K,R,routing", FUSED)
def test_layout_and_dispatch_in_one_call(T, H, E, K, R, routing):
    cfg = inputs.custom_config(T, H, E, K, R, routing=routing, config_id=64)
    d = inputs.make_inputs(cfg)
    idx, x = d["topk_idx"].copy(), d["x"]
    if T >= 8:                                             # masked, repeated and out-of-range ids
        idx[1, :] = -1
        idx[2, 0] = -1
        idx[3, K - 1] = idx[3, 0]
        idx[5, 0] = E + 3
    ref = oracle.layout(idx, E, R)
    lay = ep.alloc_layout(T, K, E, R, fill=-7)
    ws = torch.empty(max(16, ep.ep_layout_workspace_bytes(T, K, E, R)), dtype=torch.uint8, device="cuda")
    spare = 3
    whole, recv = guarded(ref.n_recv + spare, H)
    ep.ep_layout_dispatch(torch.from_numpy(idx).cuda(), dev_bf16(x), recv, E, R, lay, ws)
    assert_layout_equal(lay, ref)
    assert ep.ep_status(lay.status) == ref.status
    np.testing.assert_array_equal(host_bits(recv), oracle.dispatch(x, ref.recv_slot, ref.n_recv + spare, fill=SENTINEL))
    assert guards_intact(whole)
    # a receive buffer that is too small: rows beyond it are skipped, the status says so
    if ref.n_recv > 4:
        cap = ref.n_recv - 3
        whole, recv = guarded(cap, H)
        ep.ep_layout_dispatch(torch.from_numpy(idx).cuda(), dev_bf16(x), recv, E, R, lay, ws)
        assert ep.ep_status(lay.status) == ref.status | ep.STATUS_CAPACITY
        np.testing.assert_array_equal(host_bits(recv), oracle.dispatch(x, ref.recv_slot, ref.n_recv)[:cap])
        assert guards_intact(whole)


def test_small_step_with_the_fused_call_replays_from_a_cuda_graph():
    """layout+dispatch in one call, combine launched with programmatic stream serialisation behind it:
    captured once, replayed on new inputs."""
    cfg = inputs.CONFIGS["C2"]
    T, K, H, E, R = cfg.T, cfg.K, cfg.H, cfg.E, cfg.R
    idx_d = torch.zeros(T, K, dtype=torch.int32, device="cuda")
    w_d = torch.zeros(T, K, dtype=torch.float32, device="cuda")
    x_d = torch.zeros(T, H, dtype=torch.bfloat16, device="cuda")
    lay = ep.alloc_layout(T, K, E, R)
    ws = torch.empty(16, dtype=torch.uint8, device="cuda")
    recv = torch.zeros(T * min(K, R), H, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(T, H, dtype=torch.bfloat16, device="cuda")

    def step():
        ep.ep_layout_dispatch(idx_d, x_d, recv, E, R, lay, ws)
        ep.ep_combine(recv, lay.recv_slot, w_d, y, E, R, status=lay.status)

    side = torch.cuda.Stream()
    with torch.cuda.stream(side):
        step()
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        step()
    for seed in (5, 6):
        d = inputs.make_inputs(cfg, seed)
        idx_d.copy_(torch.from_numpy(d["topk_idx"]))
        w_d.copy_(torch.from_numpy(d["topk_weights"]))
        x_d.copy_(dev_bf16(d["x"]))
        graph.replay()
        torch.cuda.synchronize()
        ref = oracle.layout(d["topk_idx"], E, R)
        want = oracle.combine_f32(oracle.dispatch(d["x"], ref.recv_slot, ref.n_recv), ref.recv_slot, d["topk_weights"])
        np.testing.assert_array_equal(host_bits(y), want)
        assert ep.ep_status(lay.status) == 0


@pytest.mark.parametrize("name", ["C3", "C4"])
def test_layout_and_dispatch_in_one_call_with_a_second_stream(name):
    """Prefill-size batches: the receive-row half and the dispatch kernel (launched behind it with programmatic
    stream serialisation) on the main stream, the pair half on a second stream, everything ordered on the main
    stream when the call returns. Three calls back to back on changing inputs, then the oracle's answers."""
    cfg = inputs.CONFIGS[name]
    T, K, H, E, R = cfg.T, cfg.K, cfg.H, cfg.E, cfg.R
    one = max(16, ep.ep_layout_workspace_bytes(T, K, E, R))
    ws = torch.empty(2 * one + 256, dtype=torch.uint8, device="cuda")
    side = torch.cuda.Stream()
    lay = ep.alloc_layout(T, K, E, R, fill=-7)
    recv = torch.zeros(T * min(K, R), H, dtype=torch.bfloat16, device="cuda")
    y = torch.zeros(T, H, dtype=torch.bfloat16, device="cuda")
    idx_d = torch.zeros(T, K, dtype=torch.int32, device="cuda")
    x_d = torch.zeros(T, H, dtype=torch.bfloat16, device="cuda")
    for seed in (0, 1, 2):
        d = inputs.make_inputs(cfg, seed)
        idx = d["topk_idx"].copy()
        idx[seed, 0] = -1
        idx_d.copy_(torch.from_numpy(idx))
        x_d.copy_(dev_bf16(d["x"]))
        ep.ep_layout_dispatch(idx_d, x_d, recv, E, R, lay, ws, stream_pairs=side)
        ep.ep_combine(recv, lay.recv_slot, torch.from_numpy(d["topk_weights"]).cuda(), y, E, R, status=lay.status)
    torch.cuda.synchronize()
    ref = oracle.layout(idx, E, R)
    assert_layout_equal(lay, ref)
    assert ep.ep_status(lay.status) == 0
    want = oracle.dispatch(d["x"], ref.recv_slot, ref.n_recv)
    np.testing.assert_array_equal(host_bits(recv)[:ref.n_recv], want)
    np.testing.assert_array_equal(host_bits(y), oracle.combine_f32(want, ref.recv_slot, d["topk_weights"]))
    with pytest.raises(ep.EPError) as err:                    # a second stream needs room for both halves' scratch
        ep.ep_layout_dispatch(idx_d, x_d, recv, E, R, lay, ws[:one], stream_pairs=side)
    assert err.value.code == -3


LEAN_TOP_K = [1, 2, 3, 4, 5, 6, 7, 8, 10]


@pytest.mark.parametrize("K", LEAN_TOP_K)
def test_receive_row_half_on_the_lean_kernels(K):
    """ep_layout_ranks with K in 1..8 or 10 takes kernels of its own (picks in registers, vector loads and
    stores where K is even): alone as one CTA up to 256 tokens, as a pair beyond. Ragged batch ends, masked /
    repeated / out-of-range ids, a batch too large for them (falls back), and a routing table that is not
    16-byte aligned (falls back)."""
    rng = np.random.default_rng(20 + K)
    cases = [(T, 8, 64) for T in (8, 200, 256, 264, 520, 1000, 1032, 2048, 4096 + 8, 8192, 32768, 40000)]
    cases += [(64, 64, 64), (192, 64, 128), (1024, 64, 256), (8192, 64, 256), (2000, 40, 80), (4096, 32, 64), (33 * 70, 33, 66)]
    for T, R, E in cases:
        idx = rng.integers(0, E, size=(T, K)).astype(np.int32)
        idx[rng.random((T, K)) < 0.1] = -1
        idx[7, :] = idx[7, 0]
        idx[T - 1, K - 1] = E + 2
        ref = oracle.layout(idx, E, R)
        ws = torch.empty(max(16, ep.ep_layout_workspace_bytes(T, K, E, R)), dtype=torch.uint8, device="cuda")
        for shift in (0, 1):                               # shift 1: the table starts 4 bytes past a 16-byte boundary
            store = torch.zeros(T * K + 4, dtype=torch.int32, device="cuda")
            idx_d = store[shift:shift + T * K].view(T, K)
            idx_d.copy_(torch.from_numpy(idx))
            lay = ep.alloc_layout(T, K, E, R, fill=-7)
            ep.ep_layout_ranks(idx_d, E, R, lay, ws)
            for f in ["rank_rows", "rank_row_offsets", "src_row_offsets", "recv_slot"]:
                np.testing.assert_array_equal(getattr(lay, f).cpu().numpy(), getattr(ref, f), err_msg=f"{f} T={T} shift={shift}")
            np.testing.assert_array_equal(lay.recv_token.cpu().numpy()[:ref.n_recv], ref.recv_token)
            assert ep.ep_status(lay.status) == ep.STATUS_BAD_INDEX
            assert (lay.pair_slot.cpu().numpy() == -7).all()   # the pair half is not this call's business


@pytest.mark.parametrize("K", LEAN_TOP_K)
def test_whole_layout_and_pair_half_on_the_lean_kernels(K):
    """ep_layout and ep_layout_pairs with K in 1..8 or 10 and E <= 1024 take the lean kernels too. Ragged batch
    ends, masked / repeated / out-of-range ids, 1024 experts, a batch and an expert count too large for them
    (fall back), and a routing table that is not 16-byte aligned (falls back)."""
    rng = np.random.default_rng(40 + K)
    for T, E, R in ((8, 8, 8), (96, 1024, 32), (256, 64, 8), (264, 64, 8), (520, 256, 8), (1000, 40, 5), (1032, 64, 8),
                    (64, 64, 64), (192, 128, 64), (512, 256, 64), (8192, 256, 64), (4096 + 64, 1024, 64), (4800, 96, 48), (33 * 70, 66, 33), (2048, 8, 8), (4096 + 8, 128, 8), (8192, 256, 8), (32768, 1024, 8), (40000, 64, 8),
                    (2048, 2048, 8), (3000, 30, 1), (3000, 30, 2), (4098, 63, 3), (2052, 12, 4), (2051 * 5 // 5 * 5, 35, 5),
                    (4200, 49, 7), (2048, 48, 16), (4096 + 32, 1024, 32), (6144, 96, 24), (2048, 128, 64)):
        T -= T % R
        idx = rng.integers(0, E, size=(T, K)).astype(np.int32)
        idx[rng.random((T, K)) < 0.1] = -1
        idx[7, :] = idx[7, 0]
        idx[T - 1, K - 1] = E + 2
        ref = oracle.layout(idx, E, R)
        ws = torch.empty(max(16, ep.ep_layout_workspace_bytes(T, K, E, R)), dtype=torch.uint8, device="cuda")
        for shift in (0, 1):
            store = torch.zeros(T * K + 4, dtype=torch.int32, device="cuda")
            idx_d = store[shift:shift + T * K].view(T, K)
            idx_d.copy_(torch.from_numpy(idx))
            lay = ep.alloc_layout(T, K, E, R, fill=-7)
            ep.ep_layout(idx_d, E, R, out=lay, workspace=ws)
            assert_layout_equal(lay, ref)
            assert ep.ep_status(lay.status) == ep.STATUS_BAD_INDEX
            half = ep.alloc_layout(T, K, E, R, fill=-7)
            ep.ep_layout_pairs(idx_d, E, R, half, ws)
            for f in ["expert_counts", "expert_offsets", "pair_slot"]:
                np.testing.assert_array_equal(getattr(half, f).cpu().numpy(), getattr(ref, f), err_msg=f"{f} T={T} E={E}")
            np.testing.assert_array_equal(half.pair_row.cpu().numpy()[:ref.n_pairs], ref.pair_row)
            np.testing.assert_array_equal(half.pair_token.cpu().numpy()[:ref.n_pairs], ref.pair_token)
            assert (half.recv_slot.cpu().numpy() == -7).all() and int(half.status[0]) == -7   # not the pair half's business


def test_layout_stays_inside_its_workspace():
    """The scratch a layout call uses is exactly what ep_layout_workspace_bytes asks for: guard bytes on both
    sides of a workspace of that size survive every form of the layout (one CTA, cluster, two kernels, lean
    kernels alone and as a pair, with fewer ranks than they were compiled for, large expert counts)."""
    rng = np.random.default_rng(77)
    guard = 4096
    for T, K, E, R in [(512, 2, 8, 8), (2048, 6, 128, 8), (1536, 3, 12, 4), (3000, 2, 30, 1), (4098, 2, 63, 3), (8192, 8, 256, 8),
                       (4096, 4, 1024, 8), (4096, 8, 2048, 8), (40000, 2, 16, 8), (3200, 32, 4096, 64), (4200, 6, 49, 7),
                       (4096, 8, 256, 16), (8192, 4, 64, 32), (3000, 6, 60, 20),
                       (200, 8, 256, 8), (256, 2, 8, 8), (264, 6, 1024, 8), (1000, 4, 64, 8), (1024, 8, 256, 32),
                       (4096, 8, 256, 64), (320, 4, 128, 64), (2400, 5, 96, 48)]:
        T -= T % R
        idx = rng.integers(-1, E, size=(T, K)).astype(np.int32)
        ref = oracle.layout(idx, E, R)
        need = max(16, ep.ep_layout_workspace_bytes(T, K, E, R))
        need_pad = (need + 15) // 16 * 16
        buf = torch.full((guard + need_pad + guard,), 0x5A, dtype=torch.uint8, device="cuda")
        ws = buf[guard:guard + need]
        idx_d = torch.from_numpy(idx).cuda()
        for call in ("whole", "ranks", "pairs"):
            lay = ep.alloc_layout(T, K, E, R, fill=-7)
            if call == "whole":
                ep.ep_layout(idx_d, E, R, out=lay, workspace=ws)
                assert_layout_equal(lay, ref)
            elif call == "ranks":
                ep.ep_layout_ranks(idx_d, E, R, lay, ws)
                np.testing.assert_array_equal(lay.recv_slot.cpu().numpy(), ref.recv_slot)
            else:
                ep.ep_layout_pairs(idx_d, E, R, lay, ws)
                np.testing.assert_array_equal(lay.pair_slot.cpu().numpy(), ref.pair_slot)
            torch.cuda.synchronize()
            b = buf.cpu().numpy()
            assert (b[:guard] == 0x5A).all() and (b[guard + need:] == 0x5A).all(), (T, K, E, R, call)


def _guarded_layout(T, K, E, R, guard=64, sentinel=-77):
    """All output arrays of a layout carved from one buffer with `guard` sentinel words between them
    (every array starts on a 16-byte boundary)."""
    sizes = [E, E + 1, R, R + 1, R * (R + 1), T * K, T * K, T * min(K, R), T * K, T * K, 1]
    starts, pos = [], guard
    for n in sizes:
        starts.append(pos)
        pos += (max(1, n) + 3) // 4 * 4 + guard
    buf = torch.full((pos,), sentinel, dtype=torch.int32, device="cuda")
    shapes = [(E,), (E + 1,), (R,), (R + 1,), (R, R + 1), (T, K), (T, K), (T * min(K, R),), (T * K,), (T * K,), (1,)]
    views = [buf[s:s + n].view(*shape) for s, n, shape in zip(starts, sizes, shapes)]
    keep = torch.ones(pos, dtype=torch.bool)
    for s, n in zip(starts, sizes):
        keep[s:s + n] = False
    return ep.Layout(*views), buf, keep.cuda(), sentinel


def test_layout_writes_nothing_outside_its_output_arrays():
    """Every form of the layout (one CTA, cluster, two general kernels, lean kernels alone and as a pair, the one-launch
    layout + dispatch) with its outputs carved from one guarded buffer: the words between the arrays and
    the entries past N_recv / P keep their sentinel."""
    rng = np.random.default_rng(78)
    for T, K, E, R, H in [(96, 3, 12, 4, 64), (1000, 10, 512, 8, 64), (2048, 5, 40, 8, 8), (4096, 8, 128, 8, 8),
                          (3000, 2, 30, 1, 8), (4098, 6, 63, 3, 8), (9000, 7, 64, 4, 8), (40000, 2, 16, 8, 8),
                          (4096, 8, 256, 16, 8), (8192, 4, 64, 32, 8),
                          (200, 8, 64, 8, 8), (256, 2, 8, 8, 64), (1000, 4, 64, 8, 8), (1024, 8, 256, 32, 8),
                          (4096, 8, 256, 64, 8), (320, 4, 128, 64, 8), (2400, 5, 96, 48, 8)]:
        T -= T % R
        idx = rng.integers(-1, E, size=(T, K)).astype(np.int32)
        ref = oracle.layout(idx, E, R)
        idx_d = torch.from_numpy(idx).cuda()
        ws = torch.empty(max(16, ep.ep_layout_workspace_bytes(T, K, E, R)), dtype=torch.uint8, device="cuda")
        calls = ["whole", "halves"] + (["one_launch"] if T <= 1024 else [])
        for call in calls:
            lay, buf, keep, sentinel = _guarded_layout(T, K, E, R)
            if call == "whole":
                ep.ep_layout(idx_d, E, R, out=lay, workspace=ws)
            elif call == "halves":
                ep.ep_layout_ranks(idx_d, E, R, lay, ws)
                ep.ep_layout_pairs(idx_d, E, R, lay, ws)
            else:
                x_d = torch.zeros(T, H, dtype=torch.bfloat16, device="cuda")
                recv = torch.zeros(max(1, ref.n_recv), H, dtype=torch.bfloat16, device="cuda")
                ep.ep_layout_dispatch(idx_d, x_d, recv, E, R, lay, ws)
            torch.cuda.synchronize()
            assert_layout_equal(lay, ref)
            assert bool((buf[keep] == sentinel).all()), (T, K, E, R, call)
            assert bool((lay.recv_token[ref.n_recv:] == sentinel).all()) and bool((lay.pair_row[ref.n_pairs:] == sentinel).all())
            assert bool((lay.pair_token[ref.n_pairs:] == sentinel).all())


def test_buffers_past_four_gib():
    """Row buffers whose byte offsets do not fit 32 bits (receive space 4.9 GB, pair space 7.5 GB):
    65536 tokens of 7168 elements, 8 of 256 experts on 8 ranks. The layout is compared in full; the
    moved and combined rows on samples that include the last rows of every buffer. x holds random
    bit patterns (NaNs included: dispatch and grouping move bits), `out` is a block of 2^15 seeded
    rows repeated: 2^32 bytes is not a whole number of rows, so a truncated offset cannot land on
    an equal row."""
    T, H, E, K, R = 65536, 7168, 256, 8, 8
    cfg = inputs.custom_config(T, H, E, K, R, routing="burst", config_id=61)
    idx, w = inputs.make_topk_idx(cfg), inputs.make_topk_weights(cfg)
    ref = oracle.layout(idx, E, R)
    assert ref.n_recv * H * 2 > 1 << 32 and ref.n_pairs * H * 2 > 1 << 32
    lay = _run_layout(idx, E, R)
    assert_layout_equal(lay, ref)
    rng = np.random.default_rng(61)
    x = rng.integers(0, 1 << 16, size=(T, H), dtype=np.uint16)
    x_d = dev_bf16(x)

    def rows_of(buf, rows):
        return host_bits(buf[torch.from_numpy(np.asarray(rows, dtype=np.int64)).cuda()])

    def guards_ok(whole):
        return bool((whole[:GUARD].view(torch.int16) == SENTINEL).all()) and \
            bool((whole[-GUARD:].view(torch.int16) == SENTINEL).all())

    # dispatch: the highest receive rows, rows around the 4 GiB mark, and a random sample
    spare = 2
    whole, recv = guarded(ref.n_recv + spare, H)
    ep.ep_dispatch(x_d, lay.recv_slot, recv, E, R, status=lay.status)
    mark = (1 << 32) // (2 * H)
    rows = np.unique(np.concatenate([np.arange(ref.n_recv - 64, ref.n_recv), np.arange(mark - 32, mark + 32),
                                     np.arange(64), rng.integers(0, ref.n_recv, 2048)]))
    np.testing.assert_array_equal(rows_of(recv, rows), x[ref.recv_token[rows]])
    assert (rows_of(recv, np.arange(ref.n_recv, ref.n_recv + spare)) == SENTINEL).all() and guards_ok(whole)
    assert ep.ep_status(lay.status) == 0

    # local grouping into the pair space, then (same buffer) independent expert outputs for combine
    pwhole, pair_rows = guarded(ref.n_pairs, H)
    ep.ep_group(recv, lay, pair_rows, E, R, status=lay.status)
    pmark = mark
    prows = np.unique(np.concatenate([np.arange(ref.n_pairs - 64, ref.n_pairs), np.arange(pmark - 32, pmark + 32),
                                      np.arange(64), rng.integers(0, ref.n_pairs, 2048)]))
    np.testing.assert_array_equal(rows_of(pair_rows, prows), x[ref.pair_token[prows]])
    assert guards_ok(pwhole)
    del recv, whole

    block_rows = 1 << 15
    block = inputs.make_out(cfg, block_rows, seed=2)
    block_d = dev_bf16(block)
    for first in range(0, ref.n_pairs, block_rows):
        n = min(block_rows, ref.n_pairs - first)
        pair_rows[first:first + n] = block_d[:n]
    ywhole, y = guarded(T, H)
    ep.ep_combine(pair_rows, lay.pair_slot, torch.from_numpy(w).cuda(), y, E, R, status=lay.status)
    last_pairs = ref.pair_token[np.arange(ref.n_pairs - 256, ref.n_pairs)]      # tokens that read the last rows
    toks = np.unique(np.concatenate([last_pairs, np.arange(32), np.arange(T - 32, T), rng.integers(0, T, 512)]))
    used = np.unique(ref.pair_slot[toks])
    used = used[used >= 0]
    compact = np.searchsorted(used, ref.pair_slot[toks]).astype(np.int32)        # the sampled tokens' rows, renumbered
    out_c = block[used % block_rows]
    yb = rows_of(y, toks)
    np.testing.assert_array_equal(yb, oracle.combine_f32(out_c, compact, w[toks]))
    assert within_tolerance(yb, oracle.combine_f64(out_c, compact, w[toks])).all()
    assert guards_ok(ywhole) and guards_ok(pwhole)
    assert ep.ep_status(lay.status) == 0
