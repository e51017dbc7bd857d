"""Pins for the oracle's operators: closed forms, brute force on tiny inputs,
invariants, and torch CPU float64 library routines.  None of these re-type the
oracle's own formula: a dropped term, wrong sign, wrong index or transposed
operand in the oracle fails at least one of them."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import oracle as O

RNG = np.random.default_rng(1234)


# ------------------------------------------------------------------ RMSNorm --
def test_rmsnorm_constant_row_closed_form():
    c, eps = 3.0, 1e-5
    gamma = RNG.normal(1.0, 0.1, size=16)
    y = O.rmsnorm(np.full((2, 16), c), gamma, eps)
    np.testing.assert_allclose(y, np.broadcast_to(gamma * c / math.sqrt(c * c + eps), (2, 16)), rtol=1e-14)


def test_rmsnorm_unit_gain_gives_unit_rms():
    x = RNG.normal(size=(5, 64)) * 7.0
    y = O.rmsnorm(x, np.ones(64), 0.0)
    np.testing.assert_allclose(np.sqrt(np.mean(y * y, axis=-1)), 1.0, rtol=1e-13)


def test_rmsnorm_scale_invariance_and_no_mean_subtraction():
    x = RNG.normal(size=(3, 32)) + 5.0          # non-zero mean: LayerNorm would differ
    g = RNG.normal(1.0, 0.1, size=32)
    np.testing.assert_allclose(O.rmsnorm(4.0 * x, g, 0.0), O.rmsnorm(x, g, 0.0), rtol=1e-13)
    # sign is kept (no centring): every output has the sign of x*g
    assert np.all(np.sign(O.rmsnorm(x, g, 0.0)) == np.sign(x * g))


def test_rmsnorm_matches_torch_library():
    x = RNG.normal(size=(4, 7, 48))
    g = RNG.normal(1.0, 0.2, size=48)
    ref = torch.nn.functional.rms_norm(torch.from_numpy(x), (48,), torch.from_numpy(g), eps=1e-5)
    np.testing.assert_allclose(O.rmsnorm(x, g, 1e-5), ref.numpy(), rtol=1e-12, atol=1e-14)


def test_rmsnorm_eps_is_inside_the_root():
    x = np.zeros((1, 8))
    x[0, 0] = 1e-3
    eps = 1e-5
    y = O.rmsnorm(x, np.ones(8), eps)
    assert y[0, 0] == pytest.approx(1e-3 / math.sqrt(1e-6 / 8 + eps), rel=1e-13)


# --------------------------------------------------------------------- RoPE --
def test_rope_position_zero_is_identity():
    y = RNG.normal(size=(3, 2, 16))
    np.testing.assert_array_equal(O.rope(y, np.zeros((3, 2)), 10000.0), y)


def test_rope_two_dim_is_plain_rotation():
    # head_dim 2: theta_0 = 1, so position p rotates the pair by p radians.
    y = np.array([[1.0, 0.0], [0.0, 1.0], [2.0, -3.0]])
    p = 0.75
    out = O.rope(y, np.full((3,), p), 10000.0)
    c, s = math.cos(p), math.sin(p)
    expect = np.array([[c, s], [-s, c], [2 * c + 3 * s, -3 * c + 2 * s]])
    np.testing.assert_allclose(out, expect, rtol=1e-14, atol=1e-15)


def test_rope_frequencies_follow_base_and_pair_index():
    # a unit vector in pair j at position 1 is rotated by base**(-2j/d)
    d, base = 8, 10000.0
    for j in range(d // 2):
        y = np.zeros(d)
        y[2 * j] = 1.0
        out = O.rope(y[None, :], np.array([1.0]), base)[0]
        ang = base ** (-2.0 * j / d)
        assert out[2 * j] == pytest.approx(math.cos(ang), rel=1e-14)
        assert out[2 * j + 1] == pytest.approx(math.sin(ang), rel=1e-14)
        assert np.count_nonzero(out) <= 2          # pairs do not mix


def test_rope_preserves_pair_norms_and_composes():
    y = RNG.normal(size=(6, 32))
    a = O.rope(y, np.full((6,), 37.0), 10000.0)
    np.testing.assert_allclose(a[:, 0::2] ** 2 + a[:, 1::2] ** 2, y[:, 0::2] ** 2 + y[:, 1::2] ** 2, rtol=1e-12)
    b = O.rope(O.rope(y, np.full((6,), 5.0), 10000.0), np.full((6,), 32.0), 10000.0)
    np.testing.assert_allclose(a, b, rtol=1e-11, atol=1e-12)


def test_rope_relative_position_invariance():
    q = RNG.normal(size=(1, 64))
    k = RNG.normal(size=(1, 64))
    def dot(m, n):
        return float((O.rope(q, np.array([m]), 10000.0) @ O.rope(k, np.array([n]), 10000.0).T)[0, 0])
    assert dot(9.0, 4.0) == pytest.approx(dot(109.0, 104.0), rel=1e-10)
    assert dot(9.0, 4.0) != pytest.approx(dot(9.0, 5.0), rel=1e-6)


def test_rope_matches_complex_multiplication():
    # "complex number rotation": (y_2j + i y_2j+1) * exp(i pos theta_j)
    d, base = 16, 500.0
    y = RNG.normal(size=(4, d))
    pos = np.array([0.0, 1.0, 17.0, 300.0])
    z = (y[:, 0::2] + 1j * y[:, 1::2]) * np.exp(1j * pos[:, None] * base ** (-2.0 * np.arange(d // 2) / d))
    out = O.rope(y, pos, base)
    np.testing.assert_allclose(out[:, 0::2], z.real, rtol=1e-12, atol=1e-13)
    np.testing.assert_allclose(out[:, 1::2], z.imag, rtol=1e-12, atol=1e-13)


# ------------------------------------------------------------------- Linear --
def test_linear_triple_loop():
    x = RNG.normal(size=(3, 5))
    w = RNG.normal(size=(4, 5))
    ref = np.zeros((3, 4))
    for r in range(3):
        for n in range(4):
            for k in range(5):
                ref[r, n] += x[r, k] * w[n, k]
    np.testing.assert_allclose(O.linear(x, w), ref, rtol=1e-13)


def test_linear_one_hot_rows_select_columns_of_x():
    x = RNG.normal(size=(2, 6))
    w = np.zeros((3, 6))
    w[0, 4] = 1.0
    w[1, 0] = 2.0
    w[2, 5] = -1.0
    np.testing.assert_allclose(O.linear(x, w), np.stack([x[:, 4], 2 * x[:, 0], -x[:, 5]], axis=1))


def test_linear_takes_fp16_bits_exactly():
    x = RNG.normal(size=(2, 8)).astype(np.float16)
    w = RNG.normal(size=(3, 8)).astype(np.float16)
    np.testing.assert_allclose(O.linear(x, w), x.astype(np.float64) @ w.astype(np.float64).T, rtol=0, atol=0)


# ------------------------------------------------------------------- SwiGLU --
def test_silu_closed_forms():
    assert O.silu(np.array([0.0]))[0] == 0.0
    z = RNG.normal(size=50) * 3
    np.testing.assert_allclose(O.silu(z) - O.silu(-z), z, rtol=1e-12, atol=1e-14)
    assert O.silu(np.array([40.0]))[0] == pytest.approx(40.0, rel=1e-15)
    np.testing.assert_allclose(O.silu(z), torch.nn.functional.silu(torch.from_numpy(z)).numpy(), rtol=1e-13)


def test_swiglu_is_silu_of_gate_times_up():
    g = np.array([1.0, -2.0, 0.0])
    u = np.array([3.0, 5.0, 7.0])
    expect = np.array([1.0 / (1 + math.exp(-1.0)) * 3.0, -2.0 / (1 + math.exp(2.0)) * 5.0, 0.0])
    np.testing.assert_allclose(O.swiglu(g, u), expect, rtol=1e-14)
    # not symmetric in its arguments: swapping gate and up changes the result
    assert not np.allclose(O.swiglu(g, u), O.swiglu(u, g))


# ---------------------------------------------------------------- Attention --
def _brute_causal(q, k, v):
    hq, s_len, d = q.shape
    g = hq // k.shape[0]
    out = np.zeros((s_len, hq * d))
    for h in range(hq):
        for i in range(s_len):
            sc = [sum(q[h, i, c] * k[h // g, t, c] for c in range(d)) / math.sqrt(d) for t in range(i + 1)]
            m = max(sc)
            e = [math.exp(s - m) for s in sc]
            z = sum(e)
            for c in range(d):
                out[i, h * d + c] = sum(e[t] / z * v[h // g, t, c] for t in range(i + 1))
    return out


@pytest.mark.parametrize("hq,hkv", [(2, 2), (4, 2), (4, 1)])
def test_causal_attention_brute_force(hq, hkv):
    q = RNG.normal(size=(hq, 9, 4))
    k = RNG.normal(size=(hkv, 9, 4))
    v = RNG.normal(size=(hkv, 9, 4))
    np.testing.assert_allclose(O.causal_attention(q, k, v), _brute_causal(q, k, v), rtol=1e-11, atol=1e-13)


def test_causal_attention_matches_torch_sdpa():
    hq, s_len, d = 3, 12, 8
    q, k, v = (RNG.normal(size=(hq, s_len, d)) for _ in range(3))
    ref = torch.nn.functional.scaled_dot_product_attention(
        torch.from_numpy(q)[None], torch.from_numpy(k)[None], torch.from_numpy(v)[None], is_causal=True)[0]
    ref = ref.permute(1, 0, 2).reshape(s_len, hq * d).numpy()
    np.testing.assert_allclose(O.causal_attention(q, k, v), ref, rtol=1e-10, atol=1e-12)


def test_causal_attention_first_row_and_identical_keys():
    hq, s_len, d = 2, 7, 4
    q = RNG.normal(size=(hq, s_len, d))
    v = RNG.normal(size=(hq, s_len, d))
    k = np.broadcast_to(RNG.normal(size=(hq, 1, d)), (hq, s_len, d))   # identical keys
    out = O.causal_attention(q, k, v).reshape(s_len, hq, d)
    np.testing.assert_allclose(out[0], v[:, 0, :], rtol=1e-13)         # row 0 sees only v_0
    running_mean = np.cumsum(v, axis=1) / np.arange(1, s_len + 1)[None, :, None]
    np.testing.assert_allclose(out, running_mean.transpose(1, 0, 2), rtol=1e-12)


def test_causal_attention_never_looks_ahead():
    hq, s_len, d = 2, 6, 4
    q, k, v = (RNG.normal(size=(hq, s_len, d)) for _ in range(3))
    base = O.causal_attention(q, k, v)
    k2, v2 = k.copy(), v.copy()
    k2[:, 4:], v2[:, 4:] = 99.0, -99.0
    np.testing.assert_array_equal(O.causal_attention(q, k2, v2)[:4], base[:4])


def test_attention_dominant_key_selects_its_value():
    d = 4
    q = np.zeros((1, d)); q[0, 0] = 1.0
    k = np.zeros((1, 5, d)); k[0, 3, 0] = 200.0
    v = RNG.normal(size=(1, 5, d))
    np.testing.assert_allclose(O.decode_attention(q, k, v), v[0, 3], rtol=1e-12)


def test_decode_attention_is_last_row_of_causal_and_permutation_invariant():
    hq, hkv, t, d = 4, 2, 11, 8
    q = RNG.normal(size=(hq, t, d))
    k = RNG.normal(size=(hkv, t, d))
    v = RNG.normal(size=(hkv, t, d))
    full = O.causal_attention(q, k, v)
    last = O.decode_attention(q[:, -1, :], k, v)
    np.testing.assert_allclose(last, full[-1], rtol=1e-12, atol=1e-14)
    perm = RNG.permutation(t)
    np.testing.assert_allclose(O.decode_attention(q[:, -1, :], k[:, perm], v[:, perm]), last, rtol=1e-12, atol=1e-14)


def test_gqa_equals_mha_with_replicated_kv_heads():
    hq, hkv, s_len, d = 6, 2, 5, 4
    q = RNG.normal(size=(hq, s_len, d))
    k = RNG.normal(size=(hkv, s_len, d))
    v = RNG.normal(size=(hkv, s_len, d))
    rep = lambda a: np.repeat(a, hq // hkv, axis=0)
    np.testing.assert_allclose(O.causal_attention(q, k, v), O.causal_attention(q, rep(k), rep(v)), rtol=1e-13)


def test_scale_is_one_over_sqrt_head_dim():
    # two keys, scores differ by exactly sqrt(d)*ln(3) -> weights 3/4 and 1/4
    d = 16
    q = np.zeros((1, d)); q[0, 0] = math.sqrt(d) * math.log(3.0)
    k = np.zeros((1, 2, d)); k[0, 0, 0] = 1.0
    v = np.zeros((1, 2, d)); v[0, 0, 0] = 1.0; v[0, 1, 1] = 1.0
    out = O.decode_attention(q, k, v)
    assert out[0] == pytest.approx(0.75, rel=1e-13) and out[1] == pytest.approx(0.25, rel=1e-13)


# ------------------------------------------------------------------- argmax --
def test_argmax_takes_lowest_index_on_ties():
    logits = np.array([[0.0, 5.0, 5.0, 1.0], [7.0, 7.0, 7.0, 7.0]])
    np.testing.assert_array_equal(O.argmax_lowest(logits), [1, 0])


# ------------------------------------------- the paper's printed arithmetic --
def _golden():
    path = os.path.join(os.path.dirname(__file__), "golden", "paper_roofline.txt")
    out = {}
    for line in open(path):
        if line.startswith("#") or not line.strip():
            continue
        name, val = line.split("--")[0].split()
        out[name] = float(val)
    return out


def test_paper_roofline_numbers():
    g = _golden()
    assert O.gemm_intensity_mac_per_byte(128, 128, 768, 4) == pytest.approx(g["intensity_128x128x768_fp32"], rel=1e-12)
    assert O.gemm_intensity_mac_per_byte(128, 128, 768, 4) == pytest.approx(192 / 13, rel=1e-12)
    assert O.intensity_threshold(4.05e12, 30e9) == pytest.approx(g["intensity_threshold_fp32"], rel=1e-12)
    assert O.attainable(4.05e12, 30e9, 192 / 13) == pytest.approx(30e9 * 192 / 13)
    assert O.attainable(4.05e12, 30e9, 1000.0) == 4.05e12
    assert O.linear_gmacs(8192, 4096, 4096, g["linear_fp16_best_ms"]) == pytest.approx(g["linear_fp16_best_gmacs"], rel=2e-4)
    assert O.linear_gmacs(8192, 4096, 4096, g["linear_fp32_best_ms"]) == pytest.approx(g["linear_fp32_best_gmacs"], rel=2e-4)
    # utilisation figures imply the per-cluster peaks: FP32 4050, FP16 twice that
    assert g["linear_fp32_best_gmacs"] / g["linear_fp32_best_util"] == pytest.approx(g["cluster_fp32_peak_gmacs"], rel=1e-3)
    assert g["linear_fp16_best_gmacs"] / g["linear_fp16_best_util"] == pytest.approx(2 * g["cluster_fp32_peak_gmacs"], rel=1e-3)
