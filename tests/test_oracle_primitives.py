"""Pins for the oracle's layer primitives: closed forms, invariants and library routines."""
import math

import numpy as np
import pytest
import torch
import torch.nn.functional as F

from oracle import d3_oracle as o

RNG = np.random.default_rng(7)


# ----------------------------------------------------------------------------- softmax statistics
def test_softmax_rows_sum_to_one_and_mask_excluded():
    lg = RNG.normal(0, 5, size=(9, 37))
    p, conf, tok, ent = o.softmax_stats(lg, mask_id=36)
    assert np.allclose(p.sum(-1), 1.0, atol=1e-14)
    assert np.all(p[:, 36] == 0.0)
    assert np.all(tok != 36)
    assert np.allclose(conf, p.max(-1))


def test_softmax_uniform_closed_form():
    V = 50
    lg = np.full((3, V), 1.7)
    _, conf, tok, ent = o.softmax_stats(lg, mask_id=V - 1)
    assert np.allclose(conf, 1.0 / (V - 1), rtol=1e-14)
    assert np.allclose(ent, math.log(V - 1), rtol=1e-13)
    assert np.all(tok == 0)  # all equal -> lowest index


def test_softmax_dominant_logit():
    lg = np.zeros((2, 20))
    lg[0, 5] = 60.0
    lg[1, 11] = 45.0
    _, conf, tok, ent = o.softmax_stats(lg, mask_id=19)
    assert list(tok) == [5, 11]
    assert np.all(conf > 1 - 1e-15) and np.all(ent < 1e-15) and np.all(ent >= 0)


def test_softmax_mask_token_never_wins_even_if_largest():
    lg = np.zeros((1, 8))
    lg[0, 7] = 100.0  # the mask token's own logit
    lg[0, 2] = 1.0
    _, conf, tok, _ = o.softmax_stats(lg, mask_id=7)
    assert tok[0] == 2
    assert np.isclose(conf[0], math.e / (math.e + 6.0))


def test_softmax_tie_takes_lower_index():
    lg = np.array([[0.0, 3.0, -1.0, 3.0, 2.0, 0.0]])
    _, conf, tok, ent = o.softmax_stats(lg, mask_id=5)
    assert tok[0] == 1


def test_two_point_entropy_closed_form():
    # two live tokens with log-odds a: p = sigmoid(a); H = binary entropy
    a = 1.3
    lg = np.array([[a, 0.0, -np.inf, -np.inf, 0.0]])
    _, conf, tok, ent = o.softmax_stats(lg, mask_id=4)
    p = 1 / (1 + math.exp(-a))
    assert np.isclose(conf[0], p)
    assert np.isclose(ent[0], -(p * math.log(p) + (1 - p) * math.log(1 - p)))


def test_softmax_stats_against_torch():
    lg = RNG.normal(0, 8, size=(6, 101))
    p, conf, tok, ent = o.softmax_stats(lg, mask_id=100)
    t = torch.tensor(lg)
    t[:, 100] = -float("inf")
    tp = torch.softmax(t, -1)
    assert np.allclose(p, tp.numpy(), atol=1e-15)
    assert np.allclose(ent, torch.special.entr(tp).sum(-1).numpy(), atol=1e-13)
    assert np.array_equal(tok, tp.argmax(-1).numpy())


# ----------------------------------------------------------------------------- RMSNorm / SiLU
def test_rms_norm_unit_rms_and_torch():
    x = RNG.normal(0, 3, size=(5, 64))
    y = o.rms_norm(x, np.ones(64), 0.0)
    assert np.allclose(np.sqrt((y * y).mean(-1)), 1.0, atol=1e-13)
    g = RNG.normal(1, 0.1, size=64)
    y = o.rms_norm(x, g, 1e-5)
    ty = F.rms_norm(torch.tensor(x), (64,), torch.tensor(g), 1e-5).numpy()
    assert np.allclose(y, ty, atol=1e-13)


def test_rms_norm_eps_inside_root():
    x = np.zeros((1, 8))
    x[0, 0] = 1e-3
    y = o.rms_norm(x, np.ones(8), 1e-5)
    assert np.isclose(y[0, 0], 1e-3 / math.sqrt(1e-6 / 8 + 1e-5))


def test_silu():
    assert o.silu(np.array([0.0]))[0] == 0.0
    x = RNG.normal(0, 4, size=100)
    assert np.allclose(o.silu(x), F.silu(torch.tensor(x)).numpy(), atol=1e-14)


# ----------------------------------------------------------------------------- RoPE
def test_rope_position_zero_is_identity_and_norm_preserved():
    x = RNG.normal(size=(4, 3, 16))
    cos, sin = o.rope_tables(np.zeros(4), 16, 1e4)
    assert np.array_equal(o.apply_rope(x, cos, sin), x)
    cos, sin = o.rope_tables(np.array([1, 7, 100, 4095]), 16, 1e4)
    y = o.apply_rope(x, cos, sin)
    assert np.allclose(np.linalg.norm(y, axis=-1), np.linalg.norm(x, axis=-1), rtol=1e-13)


def test_rope_is_relative():
    q = RNG.normal(size=(1, 1, 32))
    k = RNG.normal(size=(1, 1, 32))

    def dot(m, n):
        cq, sq = o.rope_tables(np.array([m]), 32, 1e4)
        ck, sk = o.rope_tables(np.array([n]), 32, 1e4)
        return float(np.sum(o.apply_rope(q, cq, sq) * o.apply_rope(k, ck, sk)))

    assert np.isclose(dot(5, 2), dot(103, 100), rtol=1e-10)
    assert np.isclose(dot(17, 17), dot(0, 0), rtol=1e-12)
    assert not np.isclose(dot(5, 2), dot(2, 5), rtol=1e-3)  # sign of the angle matters


def test_rope_matches_complex_rotation():
    # pair (k, k + dh/2) is the complex number x_k + i x_{k+dh/2}, rotated by pos * theta^(-2k/dh)
    dh, theta = 8, 1e4
    x = RNG.normal(size=(3, 2, dh))
    pos = np.array([3, 11, 200])
    cos, sin = o.rope_tables(pos, dh, theta)
    y = o.apply_rope(x, cos, sin)
    for n in range(3):
        for k in range(dh // 2):
            ang = pos[n] * theta ** (-2.0 * k / dh)
            z = (x[n, :, k] + 1j * x[n, :, k + dh // 2]) * np.exp(1j * ang)
            assert np.allclose(y[n, :, k], z.real) and np.allclose(y[n, :, k + dh // 2], z.imag)


def test_rope_frequency_spectrum():
    cos, sin = o.rope_tables(np.array([1.0]), 64, 1e4)
    assert np.isclose(cos[0, 0], math.cos(1.0)) and np.isclose(sin[0, 0], math.sin(1.0))
    assert np.isclose(sin[0, 31], math.sin(1e4 ** (-62 / 64)))


# ----------------------------------------------------------------------------- attention
def test_attention_equals_torch_sdpa_noncausal():
    n, L, hq, dh = 5, 13, 4, 16
    q = RNG.normal(size=(n, hq, dh))
    k = RNG.normal(size=(L, hq, dh))
    v = RNG.normal(size=(L, hq, dh))
    out = o.attention(q, k, v)
    tq, tk, tv = (torch.tensor(a).permute(1, 0, 2)[None] for a in (q, k, v))
    ref = F.scaled_dot_product_attention(tq, tk, tv, is_causal=False)[0].permute(1, 0, 2).numpy()
    assert np.allclose(out, ref, atol=1e-13)


def test_attention_gqa_equals_replicated_mha():
    n, L, hq, hkv, dh = 4, 9, 6, 2, 8
    q = RNG.normal(size=(n, hq, dh))
    k = RNG.normal(size=(L, hkv, dh))
    v = RNG.normal(size=(L, hkv, dh))
    out = o.attention(q, k, v)
    ref = o.attention(q, np.repeat(k, hq // hkv, axis=1), np.repeat(v, hq // hkv, axis=1))
    assert np.allclose(out, ref, atol=1e-14)
    # kv head of query head h is h // group: head 2 must read kv head 0, head 3 kv head 1
    k2 = k.copy()
    k2[:, 1] += RNG.normal(size=k2[:, 1].shape)
    out2 = o.attention(q, k2, v)
    assert np.allclose(out2[:, :3], out[:, :3]) and not np.allclose(out2[:, 3:], out[:, 3:])


def test_attention_visibility_mask():
    n, L, dh = 3, 6, 4
    q = RNG.normal(size=(n, 1, dh))
    k = RNG.normal(size=(L, 1, dh))
    v = RNG.normal(size=(L, 1, dh))
    vis = np.ones((n, L), dtype=bool)
    vis[:, 4:] = False
    assert np.allclose(o.attention(q, k, v, vis), o.attention(q, k[:4], v[:4]), atol=1e-14)


def test_attention_single_key_returns_value():
    q = RNG.normal(size=(2, 1, 4))
    k = RNG.normal(size=(1, 1, 4))
    v = RNG.normal(size=(1, 1, 4))
    assert np.allclose(o.attention(q, k, v), np.broadcast_to(v, (2, 1, 4)))


# ----------------------------------------------------------------------------- number formats
def test_bf16_rounding_ties_to_even():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7 + 2 ** -8, 1.0 + 2 ** -8 + 2 ** -20], dtype=np.float32)
    r = o.round_to_bf16(x)
    assert list(r) == [1.0, 1.0, 1.0 + 2 ** -6, 1.0 + 2 ** -7]
    t = torch.tensor(RNG.normal(size=1000).astype(np.float32))
    assert np.array_equal(o.round_to_bf16(t.numpy()), t.to(torch.bfloat16).float().numpy())
    bits = t.to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(o.bf16_bits_to_float(bits), t.to(torch.bfloat16).float().numpy())
