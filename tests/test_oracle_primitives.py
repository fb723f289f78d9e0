"""Pins for the oracle's primitives: each against a library routine or a closed form that
is not the oracle's own code path (the oracle is plain C loops; the references here are
numpy / torch float64 library calls, textbook identities and hand values)."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import decoder as od
from paper_2311_04951_b200 import synth

RNG = np.random.default_rng(1234)


def test_linear_matches_matmul_and_is_not_transposed():
    x = RNG.standard_normal((3, 37)).astype(np.float32)
    W = RNG.standard_normal((11, 37)).astype(np.float32)
    b = RNG.standard_normal(11).astype(np.float32)
    y = od.linear(x, W, b)
    ref = x.astype(np.float64) @ W.astype(np.float64).T + b
    np.testing.assert_allclose(y, ref, rtol=0, atol=2e-6)
    # hand case: W = [[1,2],[3,4],[5,6]] (N=3,Kd=2), x=[1,10] -> [21, 43, 65]
    y = od.linear(np.array([[1.0, 10.0]]), np.array([[1, 2], [3, 4], [5, 6]], np.float32))
    assert y.tolist() == [[21.0, 43.0, 65.0]]


def test_linear_bf16_weights_widen_exactly():
    x = RNG.standard_normal((2, 64)).astype(np.float32)
    Wf = RNG.standard_normal((5, 64)).astype(np.float32)
    Wb = synth.f32_to_bf16_bits(Wf)
    Wt = torch.from_numpy(Wf).bfloat16().double().numpy()  # torch's own RNE rounding
    y = od.linear(x, Wb, None, dtype=1)
    np.testing.assert_allclose(y, x.astype(np.float64) @ Wt.T, rtol=0, atol=2e-6)


def test_round_bf16_matches_torch_including_ties():
    vals = np.concatenate([RNG.standard_normal(2000).astype(np.float32) * 3,
                           np.array([1.00390625, 1.01171875, -1.00390625, 0.0, 3.0e38, 1e-40], np.float32)])
    got = np.array([od.round_bf16(float(v)) for v in vals], np.float32)
    ref = torch.from_numpy(vals).bfloat16().float().numpy()
    assert np.array_equal(got, ref)
    # 1 + 2^-8 is a tie between 1 and 1 + 2^-7: even mantissa wins (1.0); 1 + 3*2^-8 ties up to 1+2^-6
    assert od.round_bf16(1.00390625) == 1.0 and od.round_bf16(1.01171875) == 1.015625


def test_layernorm_matches_torch_and_has_unit_statistics():
    x = (RNG.standard_normal((4, 96)) * 3 + 1.5).astype(np.float32)
    g = RNG.standard_normal(96).astype(np.float32)
    b = RNG.standard_normal(96).astype(np.float32)
    y = od.norm(x, g, b, 0, 1e-5)
    ref = F.layer_norm(torch.from_numpy(x).double(), (96,), torch.from_numpy(g).double(),
                       torch.from_numpy(b).double(), 1e-5).numpy()
    np.testing.assert_allclose(y, ref, rtol=0, atol=3e-6)
    y1 = od.norm(x, np.ones(96, np.float32), np.zeros(96, np.float32), 0, 0.0)
    np.testing.assert_allclose(y1.mean(axis=1), 0, atol=1e-6)
    np.testing.assert_allclose(y1.var(axis=1), 1, atol=1e-5)


def test_rmsnorm_matches_torch_and_scale_invariance():
    x = (RNG.standard_normal((3, 80)) * 2).astype(np.float32)
    g = (1 + 0.1 * RNG.standard_normal(80)).astype(np.float32)
    y = od.norm(x, g, None, 1, 1e-5)
    ref = F.rms_norm(torch.from_numpy(x).double(), (80,), torch.from_numpy(g).double(), 1e-5).numpy()
    np.testing.assert_allclose(y, ref, rtol=0, atol=3e-6)
    # eps = 0: scaling the input leaves the output unchanged, and mean(y^2) = 1 for unit gain
    y2 = od.norm(x * 4, np.ones(80, np.float32), None, 1, 0.0)
    y3 = od.norm(x, np.ones(80, np.float32), None, 1, 0.0)
    np.testing.assert_allclose(y2, y3, atol=1e-6)
    np.testing.assert_allclose((y3.astype(np.float64) ** 2).mean(axis=1), 1, atol=1e-6)


def test_gelu_is_erf_form_and_silu():
    for v in [-6.0, -2.5, -1.0, -0.1, 0.0, 0.3, 1.0, 2.0, 5.0]:
        t = torch.tensor(v, dtype=torch.float64)
        assert abs(od.gelu(v) - F.gelu(t).item()) < 1e-7 * max(1, abs(v))  # torch default = erf form
        assert abs(od.silu(v) - F.silu(t).item()) < 1e-7 * max(1, abs(v))
    # the erf form differs measurably from the tanh approximation: make sure we pinned the right one
    assert abs(od.gelu(2.0) - F.gelu(torch.tensor(2.0, dtype=torch.float64), approximate="tanh").item()) > 5e-5
    assert abs(od.gelu(1.0) - 0.5 * (1 + math.erf(1 / math.sqrt(2)))) < 1e-7


def test_rotary_is_the_half_split_rotation():
    rd = 8
    v = np.arange(1, rd + 1, dtype=np.float32)
    # position 0 is the identity
    assert np.array_equal(od.rotary(v, rd, 0), v)
    # pair (0, rd/2) turns by exactly pos radians (frequency base^0 = 1)
    out = od.rotary(v, rd, 1)
    c, s = math.cos(1.0), math.sin(1.0)
    assert abs(out[0] - (v[0] * c - v[4] * s)) < 1e-6 and abs(out[4] - (v[0] * s + v[4] * c)) < 1e-6
    # pair (j, j + rd/2) turns by pos * base^(-2j/rd): j=2, rd=8, base 10000 -> 10000^-0.5 = 0.01
    out = od.rotary(v, rd, 50)
    c, s = math.cos(0.5), math.sin(0.5)
    assert abs(out[2] - (v[2] * c - v[6] * s)) < 1e-5 and abs(out[6] - (v[2] * s + v[6] * c)) < 1e-5
    # rotations preserve the norm, and q.k depends only on the position difference
    q = RNG.standard_normal(rd).astype(np.float32)
    k = RNG.standard_normal(rd).astype(np.float32)
    assert abs(np.linalg.norm(od.rotary(q, rd, 77)) - np.linalg.norm(q)) < 1e-5
    d1 = float(od.rotary(q, rd, 13) @ od.rotary(k, rd, 5))
    d2 = float(od.rotary(q, rd, 108) @ od.rotary(k, rd, 100))
    assert abs(d1 - d2) < 1e-5
    # partial rotary: dims beyond rotary_dim untouched
    v16 = RNG.standard_normal(16).astype(np.float32)
    out = od.rotary(v16, 8, 9)
    assert np.array_equal(out[8:], v16[8:]) and not np.array_equal(out[:8], v16[:8])


def test_attend_matches_sdpa_and_uniform_case():
    n, Dh = 13, 16
    q = RNG.standard_normal(Dh).astype(np.float32)
    k = RNG.standard_normal((n, Dh)).astype(np.float32)
    v = RNG.standard_normal((n, Dh)).astype(np.float32)
    out = od.attend(q, k, v)
    ref = F.scaled_dot_product_attention(torch.from_numpy(q).double()[None, None, None],
                                         torch.from_numpy(k).double()[None, None],
                                         torch.from_numpy(v).double()[None, None])[0, 0, 0].numpy()
    np.testing.assert_allclose(out, ref, atol=2e-6)
    # identical keys -> uniform weights -> mean of values
    out = od.attend(q, np.tile(k[:1], (n, 1)), v)
    np.testing.assert_allclose(out, v.astype(np.float64).mean(axis=0), atol=2e-6)


def test_attention_rows_is_causal_sdpa_per_head():
    H, Dh, S, ln, m = 3, 8, 20, 9, 4
    kv = RNG.standard_normal((2, H, S, Dh)).astype(np.float32)
    q = RNG.standard_normal((m, H * Dh)).astype(np.float32)
    o = od.attention_rows(q, kv, ln, m)
    for r in range(m):
        for h in range(H):
            n = ln + r + 1
            ref = F.scaled_dot_product_attention(
                torch.from_numpy(q[r, h * Dh:(h + 1) * Dh]).double()[None, None, None],
                torch.from_numpy(kv[0, h, :n]).double()[None, None],
                torch.from_numpy(kv[1, h, :n]).double()[None, None])[0, 0, 0].numpy()
            np.testing.assert_allclose(o[r, h * Dh:(h + 1) * Dh], ref, atol=2e-6)
