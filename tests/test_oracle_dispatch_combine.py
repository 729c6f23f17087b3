"""Pins of the oracle's dispatch and combine: definitions, exact rationals, closed forms."""
from fractions import Fraction

import numpy as np
import pytest
import torch

import brute
import oracle
from paper_2609_40093_b200 import inputs

SENTINEL = 0x7FC1  # a bf16 NaN pattern no generator produces


def _case(T, H, E, K, R, routing="uniform", cid=70, seed=0):
    cfg = inputs.custom_config(T, H, E, K, R, routing=routing, config_id=cid)
    d = inputs.make_inputs(cfg, seed)
    return cfg, d["topk_idx"], d["topk_weights"], d["x"]


@pytest.mark.parametrize("T,H,E,K,R", [(64, 256, 8, 2, 2), (48, 40, 12, 3, 4), (32, 8, 16, 4, 1), (512, 64, 128, 8, 8)])
def test_dispatch_definition(T, H, E, K, R):
    cfg, idx, w, x = _case(T, H, E, K, R)
    lay = oracle.layout(idx, E, R)
    guard = 3
    recv = oracle.dispatch(x, lay.recv_slot, lay.n_recv + guard, fill=SENTINEL)
    for t in range(T):
        for k in range(K):
            assert (recv[lay.recv_slot[t, k]] == x[t]).all()
    np.testing.assert_array_equal(recv[:lay.n_recv], x[lay.recv_token])      # every row is its token's row
    assert (recv[lay.n_recv:] == SENTINEL).all()                             # nothing beyond N_recv is touched
    if R == 1:
        np.testing.assert_array_equal(recv[:T], x)


def test_dispatch_skips_masked_pairs():
    cfg, idx, w, x = _case(16, 8, 8, 2, 4)
    idx = idx.copy()
    idx[3, :] = -1
    idx[5, 1] = -1
    lay = oracle.layout(idx, 8, 4)
    recv = oracle.dispatch(x, lay.recv_slot, lay.n_recv, fill=SENTINEL)
    assert 3 not in set(lay.recv_token.tolist())
    np.testing.assert_array_equal(recv, x[lay.recv_token])


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_combine_fma_chain_against_exact_rational_arithmetic(seed):
    """The fp32 chain and both roundings, redone on exact rationals."""
    cfg, idx, w, x = _case(6, 8, 8, 4, 2, cid=71, seed=seed)
    idx = idx.copy()
    idx[1, 2] = -1                                                  # a masked pair in the middle of a chain
    lay = oracle.layout(idx, 8, 2)
    out = inputs.make_out(cfg, lay.n_pairs, seed)
    out_f = inputs.bf16_bits_to_f32(out)
    y = inputs.bf16_bits_to_f32(oracle.combine_f32(out, lay.pair_slot, w))
    want = brute.combine_fma_chain(out_f, lay.pair_slot, w)
    np.testing.assert_array_equal(y.astype(np.float64), want)
    # the fp64 evaluation agrees with the exact sum to fp64 rounding
    y64 = oracle.combine_f64(out, lay.pair_slot, w)
    exact = brute.combine_exact(out_f, lay.pair_slot, w)
    for t in range(6):
        for h in range(8):
            e = float(exact[t][h])
            assert abs(y64[t, h] - e) <= 4 * np.finfo(np.float64).eps * max(1.0, abs(e))
            # and the path's result obeys the stated tolerance against it
            assert abs(y[t, h] - e) <= max(4e-3 * abs(e), 1e-3)


def test_combine_order_of_k_matters_and_is_ascending():
    """A chain whose value depends on the order of accumulation: big + small - big."""
    out_f = np.array([[2.0 ** 20], [2.0 ** -6], [2.0 ** 20]], dtype=np.float32)
    out = inputs.to_bf16_bits(out_f)
    slot = np.array([[0, 1, 2]], dtype=np.int32)
    w = np.array([[1.0, 1.0, -1.0]], dtype=np.float32)
    y = inputs.bf16_bits_to_f32(oracle.combine_f32(out, slot, w))
    assert y[0, 0] == 0.0                                          # ascending k: the small term is absorbed
    slot2 = np.array([[0, 2, 1]], dtype=np.int32)
    w2 = np.array([[1.0, -1.0, 1.0]], dtype=np.float32)
    y2 = inputs.bf16_bits_to_f32(oracle.combine_f32(out, slot2, w2))
    assert y2[0, 0] == 2.0 ** -6
    assert oracle.combine_f64(out, slot, w)[0, 0] == 2.0 ** -6     # the exact sum keeps it


def test_combine_keeps_the_product_unrounded_inside_the_chain():
    """A fused multiply-add rounds once: with acc = -c, w*v = c + c*2^-23 leaves c*2^-23 exactly,
    whereas a rounded product (c + 2^-23) would leave 2^-23. c = 1 + 2^-7 is a bf16 number."""
    c = 1.0078125
    out = inputs.to_bf16_bits(np.array([[c], [c]], dtype=np.float32))
    slot = np.array([[0, 1]], dtype=np.int32)
    w = np.array([[-1.0, 1.0 + 2.0 ** -23]], dtype=np.float32)
    y = inputs.bf16_bits_to_f32(oracle.combine_f32(out, slot, w))
    assert y[0, 0] == np.float32(c * 2.0 ** -23) != np.float32(2.0 ** -23)
    assert oracle.combine_f64(out, slot, w)[0, 0] == c * 2.0 ** -23


def test_combine_single_rounding_of_the_product_matches_torch_cast():
    """K = 1: y = bf16(fp32(w * v)); numpy's fp32 multiply is the correctly rounded
    product and torch's CPU cast is the narrowing."""
    rng = np.random.default_rng(5)
    H = 4096
    out = inputs.to_bf16_bits(rng.standard_normal((4, H), dtype=np.float32))
    slot = np.arange(4, dtype=np.int32).reshape(4, 1)
    w = rng.standard_normal((4, 1)).astype(np.float32)
    y = oracle.combine_f32(out, slot, w)
    prod = (w * inputs.bf16_bits_to_f32(out)).astype(np.float32)
    np.testing.assert_array_equal(y, inputs.to_bf16_bits(prod))
    # ties: products exactly half way between two bf16 numbers go to the even one
    ties = np.array([[1.00390625], [1.01171875], [-1.00390625], [1.0078125]], dtype=np.float32)  # 1+2^-8, 1+3*2^-8, ., 1+2^-7
    got = oracle.combine_f32(inputs.to_bf16_bits(np.ones((1, 2), np.float32)), np.zeros((4, 1), np.int32), ties)
    assert inputs.bf16_bits_to_f32(got)[:, 0].tolist() == [1.0, 1.015625, -1.0, 1.0078125]


def test_combine_closed_forms():
    cfg, idx, w, x = _case(64, 256, 8, 2, 2, cid=72)
    T, K, H = cfg.T, cfg.K, cfg.H
    lay = oracle.layout(idx, cfg.E, cfg.R)
    out = inputs.make_out(cfg, lay.n_pairs)
    # one-hot weights: y[t] is bit for bit the selected row
    for kstar in range(K):
        onehot = np.zeros((T, K), np.float32)
        onehot[:, kstar] = 1.0
        y = oracle.combine_f32(out, lay.pair_slot, onehot)
        np.testing.assert_array_equal(y, out[lay.pair_slot[:, kstar]])
    # K = 1, w = 1: a bit copy
    y = oracle.combine_f32(out, lay.pair_slot[:, :1], np.ones((T, 1), np.float32))
    np.testing.assert_array_equal(y, out[lay.pair_slot[:, 0]])
    # constant rows c: y = bf16(chain of w*c), the same in every column
    c = 1.5
    const = inputs.to_bf16_bits(np.full((lay.n_pairs, H), c, np.float32))
    y = inputs.bf16_bits_to_f32(oracle.combine_f32(const, lay.pair_slot, w))
    acc = np.zeros(T, np.float32)
    for k in range(K):
        acc = (acc.astype(np.float64) + w[:, k].astype(np.float64) * c).astype(np.float32)  # exact in fp64: c has 2 bits
    np.testing.assert_array_equal(y, np.repeat(inputs.bf16_bits_to_f32(inputs.to_bf16_bits(acc))[:, None], H, 1))
    # all pairs masked: +0
    y = oracle.combine_f32(out, -np.ones((T, K), np.int32), w)
    assert (y == 0).all()
    # linearity of the exact sum in the weights
    w2 = inputs.make_topk_weights(cfg, seed=3)
    a = oracle.combine_f64(out, lay.pair_slot, w)
    b = oracle.combine_f64(out, lay.pair_slot, w2)
    ab = oracle.combine_f64(out, lay.pair_slot, (w.astype(np.float64) + w2).astype(np.float32))
    np.testing.assert_allclose(ab, a + b, rtol=0, atol=1e-5)


@pytest.mark.parametrize("name", ["C1", "C2", "C3"])
def test_dispatch_then_identity_expert_combine_returns_x(name):
    """Weights sum to 1 and the expert is the identity, so combine over the receive
    rows reproduces x up to the rounding of the chain."""
    cfg = inputs.CONFIGS[name]
    d = inputs.make_inputs(cfg)
    idx, w, x = d["topk_idx"], d["topk_weights"], d["x"]
    if name == "C3":                                               # keep the CPU suite short
        idx, w, x = idx[:512], w[:512], x[:512]
    lay = oracle.layout(idx, cfg.E, cfg.R)
    recv = oracle.dispatch(x, lay.recv_slot, lay.n_recv)
    y = inputs.bf16_bits_to_f32(oracle.combine_f32(recv, lay.recv_slot, w))
    xf = inputs.bf16_bits_to_f32(x)
    assert (np.abs(y - xf) <= np.maximum(4e-3 * np.abs(xf), 1e-3)).all()
    y64 = oracle.combine_f64(recv, lay.recv_slot, w)
    np.testing.assert_allclose(y64, xf, rtol=1e-6, atol=1e-6)     # exact sum: x * (sum of fp32 weights)
    # the same through the pair space: out[p] = recv[pair_row[p]] is the local grouping step
    y2 = oracle.combine_f32(recv[lay.pair_row], lay.pair_slot, w)
    np.testing.assert_array_equal(inputs.bf16_bits_to_f32(y2), y)
