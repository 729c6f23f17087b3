"""Per-sender completion flags with bounded polling, and the two-stream host round trip.

No test here makes a GPU wait on another kernel: flags are written either earlier on the
same stream or by the host, and every wait gives up after its time limit and reports it
in a status word, after which the context must still work."""
import os
import time

import numpy as np
import pytest
import torch

import oracle
from gpu_util import dev_bf16, host_bits
from paper_2609_40093_b200 import ep, inputs

pytestmark = pytest.mark.gpu
EPOCH = 7

# with blocking launches the host cannot post a flag while the kernel that waits for it is in flight
needs_async_launches = pytest.mark.skipif(os.environ.get("CUDA_LAUNCH_BLOCKING") == "1",
                                          reason="the host posts flags while the waiting kernel runs")


def _dev_i32(n, fill=0):
    return torch.full((n,), fill, dtype=torch.int32, device="cuda")


def test_flags_already_posted_on_the_same_stream():
    flags, arrived, status = _dev_i32(8), _dev_i32(8), _dev_i32(1)
    ep.ep_post_flags(flags, 0, 5, EPOCH)
    ep.ep_post_flags(flags, 5, 3, EPOCH)
    ep.ep_wait_senders(flags, 8, EPOCH, 50_000_000, arrived=arrived, status=status)
    torch.cuda.synchronize()
    assert ep.ep_status(status) == 0 and (arrived.cpu() == EPOCH).all()


def test_wait_gives_up_after_its_limit_and_the_context_survives():
    flags, arrived, status = _dev_i32(6), _dev_i32(6), _dev_i32(1)
    flags[:2] = EPOCH                                   # senders 0 and 1 are done, the others never post
    flags[2] = EPOCH - 1                                # a flag of the previous round does not count
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    ep.ep_wait_senders(flags, 6, EPOCH, 5_000_000, arrived=arrived, status=status)   # 5 ms limit
    torch.cuda.synchronize()
    elapsed = time.perf_counter() - t0
    assert 0.004 < elapsed < 1.0
    assert ep.ep_status(status) == ep.STATUS_TIMEOUT
    assert arrived.cpu().tolist() == [EPOCH, EPOCH, 0, 0, 0, 0]
    # the stream and the context still work
    cfg = inputs.CONFIGS["C1"]
    idx = inputs.make_topk_idx(cfg)
    lay = ep.ep_layout(torch.from_numpy(idx).cuda(), cfg.E, cfg.R)
    assert int(lay.expert_offsets[-1]) == cfg.T * cfg.K


@needs_async_launches
def test_host_written_flags_in_pinned_memory():
    """The flags sit in mapped pinned host memory, as the paper's do; the host posts them one
    by one while the kernel polls over the host link."""
    n = 8
    flags_h = torch.zeros(n, dtype=torch.int32).pin_memory()
    arrived, status = _dev_i32(n), _dev_i32(1)
    ep.ep_wait_senders(flags_h, n, EPOCH, 1_500_000_000, arrived=arrived, status=status)
    view = flags_h.numpy()
    for s in range(n):                                  # host-made delays between senders
        time.sleep(0.001)
        view[s] = EPOCH
    torch.cuda.synchronize()
    assert ep.ep_status(status) == 0 and (arrived.cpu() == EPOCH).all()


def test_argument_checks():
    flags = _dev_i32(4)
    for bad in [dict(num_senders=0), dict(num_senders=65), dict(timeout_ns=0), dict(timeout_ns=3_000_000_000)]:
        kw = dict(num_senders=4, epoch=1, timeout_ns=1000)
        kw.update(bad)
        with pytest.raises(ep.EPError):
            ep.ep_wait_senders(flags, kw["num_senders"], kw["epoch"], kw["timeout_ns"])


@pytest.mark.parametrize("duplex,chunks", [(False, 1), (True, 1), (True, 4)])
def test_host_roundtrip_is_the_identity_on_the_receive_rows(duplex, chunks):
    cfg = inputs.CONFIGS["C5"]
    d = inputs.make_inputs(cfg)
    idx, x = d["topk_idx"], d["x"]
    ref = oracle.layout(idx, cfg.E, cfg.R)
    want = oracle.dispatch(x, ref.recv_slot, ref.n_recv)
    lay = ep.ep_layout(torch.from_numpy(idx).cuda(), cfg.E, cfg.R)
    cap = ref.n_recv + 5
    staging = torch.zeros(cap, cfg.H, dtype=torch.bfloat16, device="cuda")
    recv = torch.zeros(cap, cfg.H, dtype=torch.bfloat16, device="cuda")
    bounce = torch.zeros(2 * cap, cfg.H, dtype=torch.bfloat16).pin_memory()
    offs = lay.rank_row_offsets.cpu()
    up, down = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for rnd in (0, 1):
        recv.zero_()
        torch.cuda.synchronize()
        ep.ep_host_roundtrip(dev_bf16(x), lay.recv_slot, offs, staging, bounce, recv, cfg.E, cfg.R, round=rnd,
                             chunks_per_rank=chunks, duplex=duplex, stream_up=up, stream_down=down)
        down.synchronize()
        np.testing.assert_array_equal(host_bits(recv)[:ref.n_recv], want)
        half = bounce.view(torch.int16).numpy().view(np.uint16)[rnd * cap:rnd * cap + ref.n_recv]
        np.testing.assert_array_equal(half, want)       # the bounce buffer of this round holds the rows
    torch.cuda.synchronize()


def _c5_case(seed=0, small=False):
    cfg = inputs.custom_config(512, 264, 32, 4, 4, routing="zipf", config_id=70) if small else inputs.CONFIGS["C5"]
    d = inputs.make_inputs(cfg, seed)
    idx, w, x = d["topk_idx"], d["topk_weights"], d["x"]
    ref = oracle.layout(idx, cfg.E, cfg.R)
    out = inputs.make_out(cfg, ref.n_pairs, seed)
    lay = ep.ep_layout(torch.from_numpy(idx).cuda(), cfg.E, cfg.R)
    return cfg, idx, w, x, ref, out, lay


ALL_FLAG_SETS = [0, ep.HOST_DUPLEX, ep.HOST_PER_PEER, ep.HOST_DUPLEX | ep.HOST_PER_PEER,
                 ep.HOST_DUPLEX | ep.HOST_LOCAL_ON_DEVICE, ep.HOST_DUPLEX | ep.HOST_PER_PEER | ep.HOST_LOCAL_ON_DEVICE,
                 ep.HOST_LOCAL_ON_DEVICE]


@pytest.mark.parametrize("flags", ALL_FLAG_SETS)
def test_host_combine_return_leg_matches_the_two_stage_oracle(flags):
    """Partial rows up to the bounce buffer, down to the owner, summed on the SMs: the downloaded
    partial rows and y are bit for bit those of the oracle's combine with partial outputs, for every
    schedule (serial / duplex, one reduction or one per owner, local blocks over the link or not)."""
    cfg, idx, w, x, ref, out, lay = _c5_case()
    want_partial, want_y = oracle.combine_partial(out, ref.pair_slot, ref.recv_slot, w, ref.n_recv)
    cap = ref.n_recv + 3
    send = torch.zeros(cap, cfg.H, dtype=torch.bfloat16, device="cuda")
    got = torch.zeros(cap, cfg.H, dtype=torch.bfloat16, device="cuda")
    bounce = torch.zeros(2 * cap, cfg.H, dtype=torch.bfloat16).pin_memory()
    y = torch.zeros(cfg.T, cfg.H, dtype=torch.bfloat16, device="cuda")
    status = _dev_i32(1)
    so = lay.src_row_offsets.cpu()
    out_d, w_d = dev_bf16(out), torch.from_numpy(w).cuda()
    up, down = torch.cuda.Stream(), torch.cuda.Stream()
    torch.cuda.synchronize()
    for rnd in (0, 1):
        got.zero_(), y.zero_()
        torch.cuda.synchronize()
        ep.ep_host_combine(out_d, lay, w_d, so, send, got, bounce, y, cfg.E, cfg.R, round=rnd, flags=flags,
                           status=status, stream_up=up, stream_down=down)
        down.synchronize()
        np.testing.assert_array_equal(host_bits(got)[:ref.n_recv], want_partial)
        np.testing.assert_array_equal(host_bits(y), want_y)
        assert (host_bits(got)[ref.n_recv:] == 0).all()
        if not flags & ep.HOST_LOCAL_ON_DEVICE:             # every block went through this round's half
            half = bounce.view(torch.int16).numpy().view(np.uint16)[rnd * cap:rnd * cap + ref.n_recv]
            np.testing.assert_array_equal(half, want_partial)
    torch.cuda.synchronize()
    assert ep.ep_status(status) == 0


def test_local_blocks_stay_off_the_host_link():
    cfg, idx, w, x, ref, out, lay = _c5_case(small=True)
    cap = ref.n_recv
    send, got = (torch.zeros(cap, cfg.H, dtype=torch.bfloat16, device="cuda") for _ in range(2))
    bounce = torch.full((2 * cap, cfg.H), -1, dtype=torch.int16).view(torch.bfloat16).pin_memory()
    y = torch.zeros(cfg.T, cfg.H, dtype=torch.bfloat16, device="cuda")
    so = lay.src_row_offsets.cpu()
    ep.ep_host_combine(dev_bf16(out), lay, torch.from_numpy(w).cuda(), so, send, got, bounce, y, cfg.E, cfg.R,
                       flags=ep.HOST_DUPLEX | ep.HOST_PER_PEER | ep.HOST_LOCAL_ON_DEVICE)
    torch.cuda.synchronize()
    want_partial, want_y = oracle.combine_partial(out, ref.pair_slot, ref.recv_slot, w, ref.n_recv)
    np.testing.assert_array_equal(host_bits(y), want_y)
    half = bounce.view(torch.int16).numpy().view(np.uint16)[:cap]
    son = ref.src_row_offsets
    for r in range(cfg.R):
        for s in range(cfg.R):
            seg = half[son[r, s]:son[r, s + 1]]
            if r == s:
                assert (seg == 0xFFFF).all()                # untouched: the block never left the device
            else:
                np.testing.assert_array_equal(seg, want_partial[son[r, s]:son[r, s + 1]])


def test_rounds_overlap_through_caller_events_and_stay_correct():
    """Four rounds of dispatch round trip + combine return leg queued back to back with no host
    synchronisation; the two halves alternate and a half is reused only behind its event. Each
    round has its own inputs and outputs, all checked at the end."""
    cases = [_c5_case(seed, small=True) for seed in range(4)]
    cfg = cases[0][0]
    cap = max(c[4].n_recv for c in cases) + 1
    staging, send = (torch.zeros(cap, cfg.H, dtype=torch.bfloat16, device="cuda") for _ in range(2))
    bounce_d = torch.zeros(2 * cap, cfg.H, dtype=torch.bfloat16).pin_memory()
    bounce_c = torch.zeros(2 * cap, cfg.H, dtype=torch.bfloat16).pin_memory()
    up, down = torch.cuda.Stream(), torch.cuda.Stream()
    free_d, free_c = ep.HalfFreeEvents(), ep.HalfFreeEvents()
    results = []
    dev_in = [(dev_bf16(c[3]), dev_bf16(c[5]), torch.from_numpy(c[2]).cuda(), c[6].src_row_offsets.cpu(),
               c[6].rank_row_offsets.cpu()) for c in cases]
    bufs = [(torch.zeros(cap, cfg.H, dtype=torch.bfloat16, device="cuda"),
             torch.zeros(cap, cfg.H, dtype=torch.bfloat16, device="cuda"),
             torch.zeros(cfg.T, cfg.H, dtype=torch.bfloat16, device="cuda")) for _ in cases]
    torch.cuda.synchronize()
    for rnd, (c, (x_d, out_d, w_d, so, ro)) in enumerate(zip(cases, dev_in)):
        lay = c[6]
        recv, got, y = bufs[rnd]
        ep.ep_host_roundtrip(x_d, lay.recv_slot, ro, staging, bounce_d, recv, cfg.E, cfg.R, round=rnd,
                             chunks_per_rank=2, duplex=True, stream_up=up, stream_down=down, half_free=free_d)
        ep.ep_host_combine(out_d, lay, w_d, so, send, got, bounce_c, y, cfg.E, cfg.R, round=rnd,
                           flags=ep.HOST_DUPLEX | ep.HOST_PER_PEER, stream_up=up, stream_down=down, half_free=free_c)
        results.append((recv, got, y))
    torch.cuda.synchronize()
    for (cfg, idx, w, x, ref, out, lay), (recv, got, y) in zip(cases, results):
        np.testing.assert_array_equal(host_bits(recv)[:ref.n_recv], oracle.dispatch(x, ref.recv_slot, ref.n_recv))
        want_partial, want_y = oracle.combine_partial(out, ref.pair_slot, ref.recv_slot, w, ref.n_recv)
        np.testing.assert_array_equal(host_bits(got)[:ref.n_recv], want_partial)
        np.testing.assert_array_equal(host_bits(y), want_y)


@pytest.mark.parametrize("flags", ALL_FLAG_SETS)
def test_dispatch_with_one_consumer_per_sender(flags):
    """The receive rows travel segment by segment, sender by sender; the local grouping of a
    sender's pairs runs behind that sender's rows (or, global policy, behind everything).
    Whatever the schedule: recv is the oracle's dispatch, grouped the oracle's grouping."""
    cfg, idx, w, x, ref, out, lay = _c5_case()
    want_recv = oracle.dispatch(x, ref.recv_slot, ref.n_recv)
    want_grouped = oracle.group(want_recv, ref.pair_row)
    cap = ref.n_recv + 2
    staging, recv = (torch.zeros(cap, cfg.H, dtype=torch.bfloat16, device="cuda") for _ in range(2))
    grouped = torch.zeros(ref.n_pairs + 2, cfg.H, dtype=torch.bfloat16, device="cuda")
    bounce = torch.zeros(2 * cap, cfg.H, dtype=torch.bfloat16).pin_memory()
    stamps = torch.zeros(cfg.R + 1, dtype=torch.int64, device="cuda")
    status = _dev_i32(1)
    so = lay.src_row_offsets.cpu()
    up, down, cons = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    x_d = dev_bf16(x)
    torch.cuda.synchronize()
    for rnd in (0, 1):
        recv.zero_(), grouped.zero_()
        torch.cuda.synchronize()
        ep.ep_host_dispatch_per_sender(x_d, lay, so, staging, recv, bounce, grouped, cfg.E, cfg.R, round=rnd,
                                       flags=flags, stamps_ns=stamps, status=status, stream_up=up,
                                       stream_down=down, stream_consume=cons)
        torch.cuda.synchronize()
        np.testing.assert_array_equal(host_bits(recv)[:ref.n_recv], want_recv)
        np.testing.assert_array_equal(host_bits(grouped)[:ref.n_pairs], want_grouped)
        assert (host_bits(grouped)[ref.n_pairs:] == 0).all()
        st = stamps.cpu().numpy()
        assert (np.diff(st) > 0).all()                      # start < sender 0 consumed < ... < last sender consumed
        first, last = st[1] - st[0], st[-1] - st[0]
        if flags & ep.HOST_PER_PEER and flags & ep.HOST_DUPLEX:
            assert first < 0.6 * last                       # the first sender's rows are in use long before the last arrive
    assert ep.ep_status(status) == 0


@needs_async_launches
def test_consumers_gated_by_host_posted_sender_flags():
    """The consumer of each sender additionally waits (bounded) for that sender's completion flag in
    pinned host memory, which the host posts one by one with delays; then the same with flags that
    never come: every wait runs out, the status says so, and the rows are still grouped."""
    cfg, idx, w, x, ref, out, lay = _c5_case(small=True)
    want_recv = oracle.dispatch(x, ref.recv_slot, ref.n_recv)
    want_grouped = oracle.group(want_recv, ref.pair_row)
    cap = ref.n_recv
    staging, recv = (torch.zeros(cap, cfg.H, dtype=torch.bfloat16, device="cuda") for _ in range(2))
    grouped = torch.zeros(ref.n_pairs, cfg.H, dtype=torch.bfloat16, device="cuda")
    bounce = torch.zeros(2 * cap, cfg.H, dtype=torch.bfloat16).pin_memory()
    flags_h = torch.zeros(cfg.R, dtype=torch.int32).pin_memory()
    arrived, status = _dev_i32(cfg.R), _dev_i32(1)
    so = lay.src_row_offsets.cpu()
    up, down, cons = torch.cuda.Stream(), torch.cuda.Stream(), torch.cuda.Stream()
    x_d = dev_bf16(x)
    torch.cuda.synchronize()
    ep.ep_host_dispatch_per_sender(x_d, lay, so, staging, recv, bounce, grouped, cfg.E, cfg.R, sender_flags=flags_h,
                                   epoch=EPOCH, timeout_ns=1_500_000_000, arrived=arrived, status=status,
                                   stream_up=up, stream_down=down, stream_consume=cons)
    view = flags_h.numpy()
    for s in range(cfg.R):
        time.sleep(0.002)
        view[s] = EPOCH
    torch.cuda.synchronize()
    assert ep.ep_status(status) == 0 and (arrived.cpu() == EPOCH).all()
    np.testing.assert_array_equal(host_bits(grouped), want_grouped)
    # flags of a round nobody posts: each wait gives up after 2 ms, nothing hangs
    grouped.zero_()
    t0 = time.perf_counter()
    ep.ep_host_dispatch_per_sender(x_d, lay, so, staging, recv, bounce, grouped, cfg.E, cfg.R, round=1,
                                   sender_flags=flags_h, epoch=EPOCH + 1, timeout_ns=2_000_000, status=status,
                                   stream_up=up, stream_down=down, stream_consume=cons)
    torch.cuda.synchronize()
    assert time.perf_counter() - t0 < 2.0
    assert ep.ep_status(status) == ep.STATUS_TIMEOUT
    np.testing.assert_array_equal(host_bits(grouped), want_grouped)


def test_segment_offsets_are_checked_on_the_host():
    cfg, idx, w, x, ref, out, lay = _c5_case(small=True)
    cap = ref.n_recv
    a, b = (torch.zeros(cap, cfg.H, dtype=torch.bfloat16, device="cuda") for _ in range(2))
    bounce = torch.zeros(2 * cap, cfg.H, dtype=torch.bfloat16).pin_memory()
    y = torch.zeros(cfg.T, cfg.H, dtype=torch.bfloat16, device="cuda")
    so = lay.src_row_offsets.cpu().clone()
    so[1, 2] = so[1, 1] - 1                                  # a segment that runs backwards
    with pytest.raises(ep.EPError):
        ep.ep_host_combine(dev_bf16(out), lay, torch.from_numpy(w).cuda(), so, a, b, bounce, y, cfg.E, cfg.R)
    so = lay.src_row_offsets.cpu().clone()
    with pytest.raises(ep.EPError) as err:                    # buffers one row short
        ep.ep_host_combine(dev_bf16(out), lay, torch.from_numpy(w).cuda(), so, a[:-1], b[:-1], bounce, y, cfg.E, cfg.R)
    assert err.value.code == -3
    torch.cuda.synchronize()
