"""Pins for the oracle's FP8 activation quantiser (the activation half of W8A8, Sec. 3.4 "System integration"): the
e4m3 rounding against the format's definition and torch's own cast, the per-token scale on hand-worked rows, and a
whole W8A8 micro forward against a torch restatement that quantises with torch's cast."""
import math

import numpy as np
import pytest
import torch

from oracle import fdvlm_oracle as orc
from paper_2604_06832_b200 import inputs as I

MICRO = I.ModelShape(n_layers=2, hidden=32, n_q_heads=4, n_kv_heads=2, head_dim=8, intermediate=48,
                     vocab=64, mask_id=63, tie_embeddings=False, dtype=I.FP8)


def test_every_finite_e4m3_code_is_a_fixed_point_and_midpoints_go_to_even():
    codes = np.array([c for c in range(256) if (c & 0x7F) != 0x7F], dtype=np.uint8)
    vals = orc.decode_e4m3(codes)
    assert np.array_equal(orc.round_e4m3(vals.astype(np.float32)), vals)
    pos = np.sort(vals[vals >= 0])
    mid = (pos[:-1] + pos[1:]) / 2                      # exactly representable in float32
    got = orc.round_e4m3(mid.astype(np.float32))
    for lo, hi, g in zip(pos[:-1], pos[1:], got):
        # the neighbour whose mantissa code is even: codes of the positive values ascend with the value
        lo_code = int(np.flatnonzero(orc.decode_e4m3(np.arange(128, dtype=np.uint8)) == lo)[0])
        assert g == (lo if lo_code % 2 == 0 else hi), (lo, hi, g)
    # a hair off the midpoint goes to the nearer side; beyond the largest value saturates
    assert orc.round_e4m3(np.float32([1.0625 - 1e-4, 1.0625 + 1e-4, 500.0, -1e9]))[[0, 1, 2, 3]].tolist() == [1.0, 1.125, 448.0, -448.0]


def test_rounding_matches_torch_cast():
    g = torch.Generator().manual_seed(0)
    x = torch.randn(100000, generator=g) * torch.exp(3 * torch.randn(100000, generator=g))
    ref = x.clamp(-448, 448).to(torch.float8_e4m3fn).double().numpy()
    assert np.array_equal(orc.round_e4m3(x.numpy()), ref)


def test_per_token_scale_by_hand():
    a = np.array([[1.0, -448.0, 3.0, 0.0],             # max 448 -> scale 1: every entry already on the grid
                  [0.1, 0.2, -0.05, 0.0],              # scale 0.2/448: 0.1 -> 224, 0.05 -> 112, both on the grid
                  [0.0, 0.0, 0.0, 0.0],                # an all-zero row stays zero (scale 1)
                  [8.0, 1.0, 0.26, 0.0]])              # scale 8/448 = 1/56: 1.0 -> 56, 0.26 -> 14.56 -> 15 (spacing 1)
    q = orc.quantize_rows_e4m3(a)
    assert np.array_equal(q[0], a[0]) and np.array_equal(q[2], a[2])
    s1 = np.float32(0.2) / np.float32(448)
    assert np.allclose(q[1], [224 * float(s1), 448 * float(s1), -112 * float(s1), 0.0], rtol=0, atol=0)
    assert np.array_equal(q[3], [8.0, 1.0, 15.0 / 56.0 * 1.0, 0.0]) or np.allclose(q[3], [8.0, 1.0, 15.0 / 56.0, 0.0], rtol=1e-7)
    # one scale per ROW: scaling a single row by a power of two scales only that row's result
    b = a.copy()
    b[3] *= 4.0
    qb = orc.quantize_rows_e4m3(b)
    assert np.array_equal(qb[:3], q[:3]) and np.allclose(qb[3], 4.0 * q[3], rtol=1e-7)


def test_quantiser_properties():
    rng = np.random.default_rng(1)
    a = rng.standard_normal((7, 200)) * np.exp(rng.standard_normal((7, 1)) * 2)
    q = orc.quantize_rows_e4m3(a)
    assert np.allclose(orc.quantize_rows_e4m3(q), q, rtol=1e-6)                   # idempotent up to the float32 scale
    amax = np.abs(a).max(axis=1, keepdims=True)
    assert np.allclose(np.abs(q).max(axis=1, keepdims=True), amax, rtol=1e-6)    # the row maximum is kept
    big = np.abs(a) >= amax * 2.0 ** -6                                            # normal range of the scaled value
    assert (np.abs(q - a)[big] <= np.abs(a)[big] * 2.0 ** -4 * 1.001).all()      # half a spacing = 2^-4 relative
    assert (np.abs(q - a) <= amax / 448 * 2.0 ** -10 * 1.001 + np.abs(a) * 2.0 ** -4 * 1.001).all()


def _torch_q(x):
    """per-row e4m3 quantisation with torch's own cast, float32 decisions"""
    x32 = x.float()
    amax = x32.abs().amax(dim=-1, keepdim=True)
    scale = torch.where(amax > 0, amax / 448.0, torch.ones_like(amax))
    return (x32 / scale).to(torch.float8_e4m3fn).double() * scale.double()


def _torch_w8a8_logits(w, toks):
    s = MICRO
    deq = lambda m, sc: m.view(torch.float8_e4m3fn).double() * sc.double()[:, None]
    h = w["embed"].double()[toks]
    T = len(toks)
    pos = torch.arange(T, dtype=torch.float64)
    half = s.head_dim // 2
    inv = s.rope_theta ** (-torch.arange(half, dtype=torch.float64) * 2 / s.head_dim)
    cos, sin = torch.cos(pos[:, None] * inv), torch.sin(pos[:, None] * inv)
    rot = lambda x: torch.cat([x[..., :half] * cos[:, None] - x[..., half:] * sin[:, None],
                               x[..., half:] * cos[:, None] + x[..., :half] * sin[:, None]], -1)
    norm = lambda x: x / torch.sqrt((x * x).mean(-1, keepdim=True) + s.rms_eps)
    for lw in w["layers"]:
        a = _torch_q(norm(h))
        q = rot((a @ deq(lw["wq"], lw["s_q"]).T).view(T, s.n_q_heads, s.head_dim))
        k = rot((a @ deq(lw["wk"], lw["s_k"]).T).view(T, s.n_kv_heads, s.head_dim))
        v = (a @ deq(lw["wv"], lw["s_v"]).T).view(T, s.n_kv_heads, s.head_dim)
        rep = s.n_q_heads // s.n_kv_heads
        att = torch.nn.functional.scaled_dot_product_attention(q.transpose(0, 1), k.repeat_interleave(rep, 1).transpose(0, 1),
                                                               v.repeat_interleave(rep, 1).transpose(0, 1), is_causal=True)
        h = h + _torch_q(att.transpose(0, 1).reshape(T, -1)) @ deq(lw["wo"], lw["s_o"]).T
        m = _torch_q(norm(h))
        act = _torch_q(torch.nn.functional.silu(m @ deq(lw["w_gate"], lw["s_gate"]).T) * (m @ deq(lw["w_up"], lw["s_up"]).T))
        h = h + act @ deq(lw["w_down"], lw["s_down"]).T
    return (norm(h) * w["g_final"].double()) @ deq(w["lm_head"], w["s_lm_head"]).T


def test_w8a8_micro_forward_against_torch_restatement():
    w = I.make_weights(MICRO, 4, std=0.3)
    o = orc.Oracle(MICRO, I.weights_to_numpy(w), act_fp8=True)
    toks = torch.tensor([3, 9, 27, 5, 11, 40])
    got = o.prefill(None, toks.numpy())
    want = _torch_w8a8_logits(w, toks)[-1].numpy()
    assert np.abs(got - want).max() < 1e-9
    # and the quantiser is really in the path: the same model without it gives visibly different logits
    plain = orc.Oracle(MICRO, I.weights_to_numpy(w)).prefill(None, toks.numpy())
    assert np.abs(plain - got).max() > 1e-3


def test_planted_scale_per_column_fails_the_pins(monkeypatch):
    def bad(a):
        a32 = np.asarray(a, dtype=np.float32)
        amax = np.max(np.abs(a32), axis=0, keepdims=True)          # per input channel instead of per token
        scale = np.where(amax > 0, amax / np.float32(448.0), np.float32(1.0)).astype(np.float32)
        return orc.round_e4m3(a32 / scale) * scale.astype(np.float64)
    monkeypatch.setattr(orc, "quantize_rows_e4m3", bad)
    for pin in (test_per_token_scale_by_hand, test_w8a8_micro_forward_against_torch_restatement):
        try:
            pin()
        except AssertionError:
            continue
        raise AssertionError(f"{pin.__name__} did not notice the planted error")


def test_planted_truncation_instead_of_nearest_fails_the_pins(monkeypatch):
    good = orc.round_e4m3

    def bad(v):
        v = np.asarray(v, dtype=np.float32)
        r = good(v)
        over = np.abs(r) > np.abs(v)                                # rounded away from zero: step back one spacing
        _, ex = np.frexp(np.abs(r))
        quantum = np.ldexp(1.0, np.clip(ex - 1, -6, 8) - 3)
        return np.where(over, r - np.sign(r) * quantum, r)
    monkeypatch.setattr(orc, "round_e4m3", bad)
    with pytest.raises(AssertionError):
        test_rounding_matches_torch_cast()
