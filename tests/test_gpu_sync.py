"""Per-sender completion flags with bounded polling, and the two-stream host round trip.

No test here makes a GPU wait on another kernel: flags are written either earlier on the
same stream or by the host, and every wait gives up after its time limit and reports it
in a status word, after which the context must still work."""
import time

import numpy as np
import pytest
import torch

import oracle
from gpu_util import dev_bf16, host_bits
from paper_2609_40093_b200 import ep, inputs

pytestmark = pytest.mark.gpu
EPOCH = 7


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
