"""Pins for the oracle's rotation (Eq. 2) and re-positioning (Eq. 5)."""
import numpy as np
import pytest

import oracle
from oracle import ROPE_HALF, ROPE_INTERLEAVED

LAYOUTS = [ROPE_HALF, ROPE_INTERLEAVED]


def _rng(seed):
    return np.random.default_rng(seed)


def _complex_rope(x, pos, theta, layout):
    """Independent statement of rotary encoding: each slice is a complex number multiplied
    by exp(i * pos * theta^(-2p/D))."""
    d = x.shape[-1]
    freq = np.array([theta ** (-2.0 * p / d) for p in range(d // 2)])
    if layout == ROPE_HALF:
        z = x[..., : d // 2] + 1j * x[..., d // 2:]
    else:
        z = x[..., 0::2] + 1j * x[..., 1::2]
    z = z * np.exp(1j * np.asarray(pos, dtype=np.float64)[..., None] * freq)
    y = np.empty_like(x)
    if layout == ROPE_HALF:
        y[..., : d // 2], y[..., d // 2:] = z.real, z.imag
    else:
        y[..., 0::2], y[..., 1::2] = z.real, z.imag
    return y


def test_quarter_turn_sign_convention():
    # Eq. 2 with r = pi/2 maps (1, 0) to (0, 1) and (0, 1) to (-1, 0).  With D = 2 the only
    # frequency is theta^0 = 1, so delta = pi/2 is exactly that angle.
    for layout in LAYOUTS:
        y = oracle.rope_rotate(np.array([1.0, 0.0]), np.pi / 2, 10000.0, layout)
        assert np.allclose(y, [0.0, 1.0], atol=1e-15)
        y = oracle.rope_rotate(np.array([0.0, 1.0]), np.pi / 2, 10000.0, layout)
        assert np.allclose(y, [-1.0, 0.0], atol=1e-15)


def test_frequencies_closed_form():
    f = oracle.rope_inv_freq(10000.0, 128)
    assert f.shape == (64,)
    assert f[0] == 1.0
    assert np.isclose(f[32], 10000.0 ** -0.5)          # p = D/4 -> theta^(-1/2)
    assert np.isclose(f[63], 10000.0 ** (-126.0 / 128.0))
    assert np.all(np.diff(f) < 0)


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("d,theta", [(64, 1e4), (128, 1e4), (128, 1e6)])
def test_rotation_group_laws(layout, d, theta):
    x = _rng(1).standard_normal((5, 3, d))
    a, b = 37.0, -1234.0
    ya = oracle.rope_rotate(x, np.full((5, 3), a), theta, layout)
    yab = oracle.rope_rotate(ya, np.full((5, 3), b), theta, layout)
    direct = oracle.rope_rotate(x, np.full((5, 3), a + b), theta, layout)
    assert np.allclose(yab, direct, atol=1e-11)          # R(a) R(b) = R(a+b)
    assert np.array_equal(oracle.rope_rotate(x, np.zeros((5, 3)), theta, layout), x)   # R(0) = I
    back = oracle.rope_rotate(ya, np.full((5, 3), -a), theta, layout)
    assert np.allclose(back, x, atol=1e-12)              # R(-a) R(a) = I (transpose = inverse)


@pytest.mark.parametrize("layout", LAYOUTS)
def test_slice_norms_preserved_and_slices_do_not_mix(layout):
    d = 64
    x = _rng(2).standard_normal((7, d))
    y = oracle.rope_rotate(x, np.arange(7) * 13.0, 1e4, layout)
    if layout == ROPE_HALF:
        nx = x[:, : d // 2] ** 2 + x[:, d // 2:] ** 2
        ny = y[:, : d // 2] ** 2 + y[:, d // 2:] ** 2
    else:
        nx = x[:, 0::2] ** 2 + x[:, 1::2] ** 2
        ny = y[:, 0::2] ** 2 + y[:, 1::2] ** 2
    assert np.allclose(nx, ny, rtol=1e-13)
    # a vector supported on one slice stays on that slice
    e = np.zeros(d)
    idx = (5, 5 + d // 2) if layout == ROPE_HALF else (10, 11)
    e[idx[0]] = 1.0
    r = oracle.rope_rotate(e, 3.0, 1e4, layout)
    mask = np.ones(d, bool)
    mask[list(idx)] = False
    assert np.all(r[mask] == 0.0)


@pytest.mark.parametrize("layout", LAYOUTS)
@pytest.mark.parametrize("theta", [1e4, 1e6])
def test_matches_complex_formulation(layout, theta):
    x = _rng(3).standard_normal((11, 2, 128))
    pos = _rng(4).integers(-4000, 32768, size=(11, 2)).astype(np.float64)
    assert np.allclose(oracle.rope_rotate(x, pos, theta, layout), _complex_rope(x, pos, theta, layout),
                       atol=1e-9)


@pytest.mark.parametrize("layout", LAYOUTS)
def test_reposition_equals_encoding_at_target(layout):
    # Eq. 5: a key cached at position i, re-positioned by (j - i), equals the raw key encoded at j.
    theta, d, hkv = 1e4, 64, 2
    lens = [5, 9, 3]
    off = np.concatenate([[0], np.cumsum(lens)])
    raw = _rng(5).standard_normal((off[-1], hkv, d))
    src = [0, 0, 7]
    dst = [100, 17, 2]
    cached = np.empty_like(raw)
    target = np.empty_like(raw)
    for i, n in enumerate(lens):
        t = np.arange(n, dtype=np.float64)[:, None] * np.ones((1, hkv))
        cached[off[i]:off[i + 1]] = _complex_rope(raw[off[i]:off[i + 1]], src[i] + t, theta, layout)
        target[off[i]:off[i + 1]] = _complex_rope(raw[off[i]:off[i + 1]], dst[i] + t, theta, layout)
    moved = oracle.reposition_keys(cached, off, src, dst, [0, 1, 2], theta, layout)
    assert np.allclose(moved, target, atol=1e-10)
    # documents not kept are returned untouched
    partial = oracle.reposition_keys(cached, off, src, dst, [1], theta, layout)
    assert np.array_equal(partial[off[0]:off[1]], cached[off[0]:off[1]])
    assert np.array_equal(partial[off[2]:off[3]], cached[off[2]:off[3]])
    assert np.allclose(partial[off[1]:off[2]], target[off[1]:off[2]], atol=1e-10)


def test_relative_position_property():
    # q_j^T k_i depends only on j - i (text after Eq. 2).
    d, theta = 64, 1e4
    q0, k0 = _rng(6).standard_normal(d), _rng(7).standard_normal(d)
    ref = oracle.rope_rotate(q0, 50.0, theta) @ oracle.rope_rotate(k0, 20.0, theta)
    for shift in (1.0, 333.0, -20.0):
        val = oracle.rope_rotate(q0, 50.0 + shift, theta) @ oracle.rope_rotate(k0, 20.0 + shift, theta)
        assert np.isclose(val, ref, atol=1e-10)
    other = oracle.rope_rotate(q0, 51.0, theta) @ oracle.rope_rotate(k0, 20.0, theta)
    assert not np.isclose(other, ref, atol=1e-6)


def test_a_planted_sign_error_is_caught():
    """A transposed rotation (sin with the wrong sign) must break the complex-number pin."""
    x = _rng(8).standard_normal((4, 64))
    wrong = oracle.rope_rotate(x, -np.arange(4.0) - 1.0, 1e4)      # what a sign slip would compute
    right = _complex_rope(x, np.arange(4.0) + 1.0, 1e4, ROPE_HALF)
    assert not np.allclose(wrong, right, atol=1e-3)


def test_round_to_bf16_matches_the_format_definition():
    """Against a library conversion, and on hand-picked ties: 1 + 2^-8 is halfway between 1 and 1 + 2^-7
    (ties to even: down), 1 + 3 * 2^-8 halfway between 1 + 2^-7 and 1 + 2^-6 (up)."""
    import torch
    rng = np.random.default_rng(0)
    x = np.concatenate([rng.standard_normal(4096) * 10.0 ** rng.integers(-6, 6, 4096), [0.0, -0.0, 1.0, -3.5]])
    want = torch.from_numpy(x).to(torch.float32).to(torch.bfloat16).to(torch.float64).numpy()
    assert np.array_equal(oracle.round_to_bf16(x), want)
    assert oracle.round_to_bf16(np.array([1.0 + 2.0 ** -8]))[0] == 1.0
    assert oracle.round_to_bf16(np.array([1.0 + 3 * 2.0 ** -8]))[0] == 1.0 + 2.0 ** -6
    assert oracle.round_to_bf16(np.array([1.0 + 2.0 ** -8 + 2.0 ** -20]))[0] == 1.0 + 2.0 ** -7
