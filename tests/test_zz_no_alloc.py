"""The allocation-free layout entry point against the ordinary one.

`ep_layout_static` serves callers that cannot allocate device memory when they need
a layout (a plugin inside an engine that owns all of the GPU's memory, code that is
not allowed to call cudaMalloc). It keeps its scratch in a fixed array inside the
library, which every call on the device shares and which still holds whatever the
previous call wrote. The test therefore runs two different routing tables back to
back through the C ABI and requires, for each, exactly the integers `ep_layout`
produces: leftovers of the first call must not leak into the second. This file
sorts last so that a run that stops at the first failure has already covered
everything else; it does not depend on any other test having run.
"""
import numpy as np
import pytest
import torch

import oracle
from gpu_util import assert_layout_equal
from paper_2609_40093_b200 import ep, inputs

pytestmark = pytest.mark.gpu

FIELDS = ["expert_counts", "expert_offsets", "rank_rows", "rank_row_offsets", "src_row_offsets",
          "recv_slot", "pair_slot", "status"]


def _same(a: ep.Layout, b: ep.Layout):
    for f in FIELDS:
        assert torch.equal(getattr(a, f), getattr(b, f)), f
    n_recv, n_pairs = int(a.rank_row_offsets[-1]), int(a.expert_offsets[-1])
    assert torch.equal(a.recv_token[:n_recv], b.recv_token[:n_recv])
    assert torch.equal(a.pair_row[:n_pairs], b.pair_row[:n_pairs])
    assert torch.equal(a.pair_token[:n_pairs], b.pair_token[:n_pairs])


def test_static_scratch_layout_matches_ep_layout_on_two_calls_in_a_row():
    assert ep.ep_layout_static_scratch_bytes() == 1 << 20
    # two workloads of different shape and routing, so stale scratch would show
    # (the 40000-token batch is past the single-cluster size, so its layout really uses the scratch)
    big = inputs.custom_config(40000, 8, 16, 2, 8, config_id=78)
    big2 = inputs.custom_config(65536, 8, 64, 4, 8, routing="zipf", config_id=79)
    for cfg in (big, inputs.CONFIGS["C4"], big2, big, inputs.CONFIGS["C3"]):
        idx = torch.from_numpy(inputs.make_topk_idx(cfg)).cuda()
        want = ep.alloc_layout(cfg.T, cfg.K, cfg.E, cfg.R, fill=-3)
        ep.ep_layout(idx, cfg.E, cfg.R, out=want)
        got = ep.alloc_layout(cfg.T, cfg.K, cfg.E, cfg.R, fill=-5)        # all memory is the caller's
        assert ep.ep_layout_workspace_bytes(cfg.T, cfg.K, cfg.E, cfg.R) <= ep.ep_layout_static_scratch_bytes()
        ep.ep_layout_static(idx, cfg.E, cfg.R, out=got)
        torch.cuda.synchronize()
        _same(got, want)
        assert_layout_equal(got, oracle.layout(inputs.make_topk_idx(cfg), cfg.E, cfg.R))
    # a table with masked and out-of-range ids: the status word travels the same way
    cfg = inputs.custom_config(512, 8, 64, 4, 8, config_id=77)
    idx_h = inputs.make_topk_idx(cfg)
    idx_h[3, 1], idx_h[100, 0], idx_h[9, :] = -1, 64 + 9, -1
    idx = torch.from_numpy(idx_h).cuda()
    want, got = (ep.alloc_layout(512, 4, 64, 8, fill=-3) for _ in range(2))
    ep.ep_layout(idx, 64, 8, out=want)
    ep.ep_layout_static(idx, 64, 8, out=got)
    _same(got, want)
    assert ep.ep_status(got.status) == ep.STATUS_BAD_INDEX


def test_static_scratch_rejects_shapes_beyond_its_limit():
    # E = 4096 experts and R = 64 ranks over 32768 tokens: 128 CTAs x 4161 counters x 4 bytes, about
    # 2.1 MB of scratch, twice what the fixed array holds: refused, nothing enqueued
    T, K, E, R = 32768, 2, 4096, 64
    assert ep.ep_layout_workspace_bytes(T, K, E, R) > ep.ep_layout_static_scratch_bytes()
    idx = torch.zeros(T, K, dtype=torch.int32, device="cuda")
    out = ep.alloc_layout(T, K, E, R, fill=-5)
    with pytest.raises(ep.EPError, match="more scratch") as err:
        ep.ep_layout_static(idx, E, R, out=out)
    assert err.value.code == -5
    torch.cuda.synchronize()
    assert int(out.expert_offsets[-1]) == -5 and int(out.status[0]) == -5      # outputs untouched


def test_static_scratch_calls_allocate_nothing_and_may_follow_each_other_without_a_sync():
    """What the entry point is for: after the first call on the device (which looks the array up) no
    call changes the amount of free device memory, and two calls on different routing tables queued
    on one stream with no host synchronisation between them both come out right (the second call
    reuses the scratch the first one left behind; stream order is all that separates them)."""
    a = inputs.custom_config(40000, 8, 16, 2, 8, config_id=78)
    b = inputs.custom_config(24000, 8, 64, 4, 8, routing="zipf", config_id=76)
    tables = [torch.from_numpy(inputs.make_topk_idx(c)).cuda() for c in (a, b)]
    outs = [ep.alloc_layout(c.T, c.K, c.E, c.R, fill=-5) for c in (a, b)]
    ep.ep_layout_static(tables[0], a.E, a.R, out=outs[0])                # first call: address look-up
    torch.cuda.synchronize()
    free_before, _ = torch.cuda.mem_get_info()
    for _ in range(3):
        for c, idx, out in zip((a, b), tables, outs):
            ep.ep_layout_static(idx, c.E, c.R, out=out)                   # no synchronisation in between
    torch.cuda.synchronize()
    free_after, _ = torch.cuda.mem_get_info()
    assert free_after == free_before
    for c, out in zip((a, b), outs):
        assert_layout_equal(out, oracle.layout(inputs.make_topk_idx(c), c.E, c.R))
        assert ep.ep_status(out.status) == 0
