"""Pins of the oracle's fake-quantization forward (Q(W) in fp32) and straight-through backward against
things that do not call them: torch autograd through clamp (a library routine), central differences of
Clamp away from its kinks, the all-inside closed form, and the forward's grid / error / idempotence
properties."""
import numpy as np
import torch

import oracle
from paper_1909_05840_b200 import synth


def test_forward_lands_on_the_group_grid_within_half_a_step():
    N, K, G = 48, 256, 8
    w = synth.weights(N, K, seed=3)
    for bits in (2, 3, 4, 8):
        st, q, delta, q0 = oracle.fake_quantize_weights(w, bits, G)
        assert st == oracle.OK
        R = N // G
        for g in range(G):
            blk, qb_ = w[g * R:(g + 1) * R].astype(np.float64), q[g * R:(g + 1) * R].astype(np.float64)
            assert q0[g] == w[g * R:(g + 1) * R].min()
            j = (qb_ - q0[g]) / delta[g]                      # grid index of every output
            assert np.all(np.abs(j - np.rint(j)) < 1e-3) and j.min() >= -1e-3 and j.max() <= 2**bits - 1 + 1e-3
            assert np.all(np.abs(blk - qb_) <= 0.5 * delta[g] * (1 + 2.0**-18) + 2 * np.spacing(np.abs(blk).astype(np.float32)))
        # idempotent under its own ranges: quantizing Q(W) with (q0, q0 + L Delta) returns Q(W)
        hi = np.array([np.float32(np.float32(delta[g]) * np.float32(2**bits - 1) + np.float32(q0[g])) for g in range(G)], dtype=np.float32)
        st2, q2, _, _ = oracle.fake_quantize_weights(q, bits, G, q0, np.maximum(hi, q.reshape(G, -1).max(1)))
        assert np.allclose(q2, q, rtol=0, atol=float(delta.max()) * 1e-3)


def test_backward_equals_torch_autograd_through_clamp():
    rng = np.random.default_rng(11)
    N, K, G = 24, 128, 6
    w = synth.weights(N, K, seed=5)
    grad = rng.standard_normal((N, K)).astype(np.float32)
    lo = np.quantile(w.reshape(G, -1), 0.05, axis=1).astype(np.float32)
    hi = np.quantile(w.reshape(G, -1), 0.95, axis=1).astype(np.float32)
    ours = oracle.ste_backward(grad, w, G, lo, hi)
    tw = torch.from_numpy(w.copy()).requires_grad_(True)
    R = N // G
    tl = torch.from_numpy(lo).repeat_interleave(R)[:, None]
    th = torch.from_numpy(hi).repeat_interleave(R)[:, None]
    torch.clamp(tw, min=tl, max=th).backward(torch.from_numpy(grad))
    assert np.array_equal(ours, tw.grad.numpy())
    assert 0 < (ours == 0).sum() < ours.size      # the clipped ranges really cut some elements off


def test_backward_is_the_slope_of_clamp_and_identity_inside():
    rng = np.random.default_rng(12)
    N, K, G = 8, 128, 2
    w = rng.standard_normal((N, K)).astype(np.float32)
    grad = rng.standard_normal((N, K)).astype(np.float32)
    lo = np.array([-0.5, -1.0], dtype=np.float32)
    hi = np.array([0.7, 0.2], dtype=np.float32)
    ours = oracle.ste_backward(grad, w, G, lo, hi)
    R = N // G
    L = np.repeat(lo, R)[:, None].astype(np.float64)
    H = np.repeat(hi, R)[:, None].astype(np.float64)
    h = 1e-4
    x = w.astype(np.float64)
    slope = (np.clip(x + h, L, H) - np.clip(x - h, L, H)) / (2 * h)
    away = (np.abs(x - L) > 2 * h) & (np.abs(x - H) > 2 * h)
    assert np.allclose(ours[away], (slope * grad)[away], rtol=1e-6, atol=0)
    # both ends of the range count as inside
    w2 = w.copy(); w2[0, 0] = lo[0]; w2[0, 1] = hi[0]
    o2 = oracle.ste_backward(grad, w2, G, lo, hi)
    assert o2[0, 0] == grad[0, 0] and o2[0, 1] == grad[0, 1]
    # default range [min, max] of each group: every element inside, gradient unchanged
    mn = w.reshape(G, -1).min(1); mx = w.reshape(G, -1).max(1)
    assert np.array_equal(oracle.ste_backward(grad, w, G, mn, mx), grad)
