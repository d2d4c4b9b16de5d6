"""Pins of the quantised-cache oracle (oracle/stief_quant_oracle.py) against what the mathematics fixes: the
round-trip error bound of a uniform quantiser, exactness on the grid, the clamp outside a calibrated range,
the group structure (64 channels; key parameters shared over positions, value parameters per token), literal
attention on the dequantised reconstructions == absorbed integer-code form, convergence to unquantised attention
as the bit width grows, brute force on tiny inputs, and planted mistakes."""
import math

import numpy as np
import pytest
import torch

from oracle import stief_oracle as O
from oracle import stief_quant_oracle as Q
from paper_2601_21686_b200 import inputs as I


def _basis(seed, r):
    return I.stiefel_basis_f64(seed, I.TAG_UK, 0, 0, r)


def _rows(seed, n, r, scale=1.0):
    return (I.normal_f64(I.stream_key(seed, I.TAG_K, 0, 0, 7), n * r).numpy().reshape(n, r) * scale).astype(np.float32)


def test_groups_are_64_consecutive_channels():
    assert Q.groups_of(64) == [(0, 64)] and Q.groups_of(128) == [(0, 64), (64, 128)]
    assert Q.groups_of(96) == [(0, 64), (64, 96)] and Q.groups_of(48) == [(0, 48)]


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("r", [64, 96, 128])
def test_value_roundtrip_error_is_at_most_half_a_step(bits, r):
    V = _rows(1, 200, r, 3.0)
    codes, s, z = Q.quantize_values(V, bits)
    assert codes.min() >= 0 and codes.max() <= 2 ** bits - 1
    Vh = Q.dequant_values(codes, s, z)
    for g, (lo, hi) in enumerate(Q.groups_of(r)):
        err = np.abs(Vh[:, lo:hi] - V[:, lo:hi].astype(np.float64))
        assert np.all(err <= 0.5 * s[:, g:g + 1] * (1 + 1e-5) + 1e-6)
        # the extremes of every row group are hit exactly: min -> code 0, max -> top code
        assert np.all(codes[:, lo:hi].min(axis=1) == 0) and np.all(codes[:, lo:hi].max(axis=1) == 2 ** bits - 1)
        # scale and zero are what a uniform asymmetric quantiser must use
        assert np.allclose(z[:, g], V[:, lo:hi].min(axis=1)) and np.allclose(s[:, g] * (2 ** bits - 1), V[:, lo:hi].max(axis=1) - V[:, lo:hi].min(axis=1), rtol=1e-6)


def test_values_on_the_grid_survive_exactly_and_constant_groups_too():
    # rows built as zero + code * scale with power-of-two scale: quantisation must return the codes
    rng = np.random.default_rng(0)
    codes = rng.integers(0, 256, size=(50, 128))
    codes[:, 0], codes[:, 1], codes[:, 64], codes[:, 65] = 0, 255, 0, 255       # every group spans the full range
    V = (codes * 0.0625 - 3.0).astype(np.float32)
    c2, s, z = Q.quantize_values(V, 8)
    assert np.array_equal(c2, codes) and np.all(s == np.float32(0.0625)) and np.all(z == np.float32(-3.0))
    assert np.array_equal(Q.dequant_values(c2, s, z), V.astype(np.float64))
    const = np.full((3, 64), 1.25, dtype=np.float32)
    c3, s3, z3 = Q.quantize_values(const, 8)
    assert np.all(c3 == 0) and np.all(s3 == 1) and np.array_equal(Q.dequant_values(c3, s3, z3), const.astype(np.float64))


def test_key_parameters_are_shared_over_positions_and_clamp_outside_the_calibrated_range():
    K = _rows(2, 300, 128)
    s, z = Q.key_params_from_calibration(K[:200], 8)
    assert s.shape == (2,) and z.shape == (2,)
    codes = Q.quantize_keys(K, s, z, 8)
    Kh = Q.dequant_keys(codes, s, z)
    for g, (lo, hi) in enumerate(Q.groups_of(128)):
        inside = (K[:, lo:hi] >= z[g]) & (K[:, lo:hi] <= z[g] + 255 * s[g])
        err = np.abs(Kh[:, lo:hi] - K[:, lo:hi])
        assert np.all(err[inside] <= 0.5 * s[g] * (1 + 1e-5) + 1e-6)
        below, above = K[:, lo:hi] < z[g], K[:, lo:hi] > z[g] + 255 * s[g]
        assert np.all(codes[:, lo:hi][below] == 0) and np.all(codes[:, lo:hi][above] == 255)
    # quantising a single later row gives the same codes as quantising it inside the batch: nothing depends on position
    assert np.array_equal(Q.quantize_keys(K[250:251], s, z, 8), codes[250:251])


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("r_k,r_v", [(64, 64), (128, 64), (96, 128)])
def test_literal_and_absorbed_forms_agree(bits, r_k, r_v):
    n = 150
    Uk, Uv = _basis(3, r_k), I.stiefel_basis_f64(3, I.TAG_UV, 0, 0, r_v)
    K = I.normal_f64(I.stream_key(3, I.TAG_K), n * 128).numpy().reshape(n, 128)
    V = I.normal_f64(I.stream_key(3, I.TAG_V), n * 128).numpy().reshape(n, 128)
    q = I.normal_f64(I.stream_key(3, I.TAG_Q), 128).numpy()
    Kd, Vd = Q.project_f32(K, Uk), Q.project_f32(V, Uv)
    ks, kz = Q.key_params_from_calibration(Kd, bits)
    Kc = Q.quantize_keys(Kd, ks, kz, bits)
    Vc, vs, vz = Q.quantize_values(Vd, bits)
    oa, la = Q.attend_quantized_path_a(q, Kc, ks, kz, Vc, vs, vz, Uk, Uv)
    ob, lb = Q.attend_quantized_path_b(q, Kc, ks, kz, Vc, vs, vz, Uk, Uv)
    assert np.abs(oa - ob).max() < 1e-11 and abs(la - lb) < 1e-11


def test_more_bits_converge_to_the_unquantised_compressed_attention():
    n, r = 200, 64
    Uk, Uv = _basis(4, r), I.stiefel_basis_f64(4, I.TAG_UV, 0, 0, r)
    K = I.normal_f64(I.stream_key(4, I.TAG_K), n * 128).numpy().reshape(n, 128)
    V = I.normal_f64(I.stream_key(4, I.TAG_V), n * 128).numpy().reshape(n, 128)
    q = I.normal_f64(I.stream_key(4, I.TAG_Q), 128).numpy()
    Kd, Vd = Q.project_f32(K, Uk), Q.project_f32(V, Uv)
    ref, _ = O.attend_path_b(q, Kd.astype(np.float64), Vd.astype(np.float64), Uk, Uv)
    errs = []
    for bits in (4, 8, 12, 16):
        ks, kz = Q.key_params_from_calibration(Kd, bits)
        Vc, vs, vz = Q.quantize_values(Vd, bits)
        out, _ = Q.attend_quantized_path_b(q, Q.quantize_keys(Kd, ks, kz, bits), ks, kz, Vc, vs, vz, Uk, Uv)
        errs.append(np.abs(out - ref).max())
    assert errs[0] > errs[1] > errs[2] > errs[3] and errs[3] < 2e-5 and errs[1] < 2e-2


def test_bruteforce_tiny():
    # d_h = 4, r = 2, three tokens, hand-written loops
    Uk = np.array([[1, 0], [0, 1], [0, 0], [0, 0]], dtype=np.float64)
    Uv = np.array([[0, 0], [1, 0], [0, 1], [0, 0]], dtype=np.float64)
    Kc = np.array([[0, 3], [2, 1], [5, 5]])
    Vc = np.array([[1, 0], [0, 7], [3, 3]])
    ks, kz = np.array([0.5], dtype=np.float32), np.array([-1.0], dtype=np.float32)
    vs = np.array([[0.25], [1.0], [2.0]], dtype=np.float32)
    vz = np.array([[0.0], [-2.0], [1.0]], dtype=np.float32)
    q = np.array([1.0, -2.0, 0.3, 0.7])
    scores, vals = [], []
    for t in range(3):
        k_hat = [Kc[t][j] * 0.5 - 1.0 for j in range(2)]
        k_full = [k_hat[0], k_hat[1], 0.0, 0.0]                      # K_tilde = K_hat Uk^T
        scores.append(sum(q[i] * k_full[i] for i in range(4)) / math.sqrt(4))
        v_hat = [Vc[t][j] * float(vs[t, 0]) + float(vz[t, 0]) for j in range(2)]
        vals.append([0.0, v_hat[0], v_hat[1], 0.0])                  # V_tilde = V_hat Uv^T
    m = max(scores)
    w = [math.exp(s - m) for s in scores]
    ref = [sum(w[t] * vals[t][i] for t in range(3)) / sum(w) for i in range(4)]
    for fn in (Q.attend_quantized_path_a, Q.attend_quantized_path_b):
        out, lse = fn(q, Kc, ks, kz, Vc, vs, vz, Uk, Uv, d_h=4)
        assert np.allclose(out, ref, atol=1e-14) and abs(lse - (m + math.log(sum(w)))) < 1e-14


def test_project_f32_against_hand_loops():
    # Eq. 1 by explicit loops in exact rational arithmetic on bf16-valued inputs, then ONE rounding to fp32
    from fractions import Fraction
    g = np.random.default_rng(5)
    X = O.rnd_bf16(g.standard_normal((3, 6)))
    Ub = O.rnd_bf16(g.standard_normal((6, 4)))
    got = Q.project_f32(X, Ub)
    assert got.dtype == np.float32 and got.shape == (3, 4)
    for t in range(3):
        for j in range(4):
            exact = sum(Fraction(float(X[t, i])) * Fraction(float(Ub[i, j])) for i in range(6))
            # nearest fp32 to the exact sum: the candidates are the fp32 neighbours of its double approximation
            c = np.float32(float(exact))
            cands = [c, np.nextafter(c, np.float32(np.inf)), np.nextafter(c, np.float32(-np.inf))]
            best = min(cands, key=lambda v: abs(Fraction(float(v)) - exact))
            assert got[t, j] == best
    # a sum whose fp32-accumulated value differs from the correctly rounded one: 1 + 2^-24 + 2^-24 -> 1 + 2^-23
    Xs = np.array([[1.0, 2.0 ** -24, 2.0 ** -24]])
    assert Q.project_f32(Xs, np.ones((3, 1)))[0, 0] == np.float32(1 + 2.0 ** -23)
    # transposed operand, wrong axis: a non-square case with distinct entries catches both
    Xn = np.array([[1.0, 2.0, 3.0]])
    Un = np.array([[1.0, 10.0], [100.0, 1000.0], [10000.0, 100000.0]])
    assert list(Q.project_f32(Xn, Un)[0]) == [30201.0, 302010.0]
    # no basis: rows pass through (a side whose projection is folded into the linear layer), rounded to fp32
    assert np.array_equal(Q.project_f32(Xs, None), Xs.astype(np.float32))


def test_byte_accounting():
    assert Q.quantized_cache_bytes(64, 64, 8) == 136 and Q.quantized_cache_bytes(128, 128, 8) == 272
    assert Q.quantized_cache_bytes(64, 64, 4) == 72


def test_planted_mistakes_fail_these_pins(monkeypatch):
    V = _rows(9, 40, 64, 2.0)
    good = Q.quantize_values(V, 8)
    # (1) symmetric instead of asymmetric (zero-point dropped)
    def sym(x, bits):
        s = (np.abs(x).max(axis=1) / (2 ** (bits - 1) - 1)).astype(np.float32)
        return np.clip(np.rint(x / s[:, None]) + 2 ** (bits - 1), 0, 2 ** bits - 1).astype(np.int32), s[:, None], np.zeros_like(s)[:, None]
    bad = sym(V, 8)
    assert not np.array_equal(bad[0], good[0])
    # (2) truncation instead of rounding breaks the half-step bound
    codes_trunc = np.clip(np.floor((V - good[2]) / good[1]), 0, 255).astype(np.int32)
    err = np.abs(Q.dequant_values(codes_trunc, good[1], good[2]) - V)
    assert np.any(err > 0.5 * good[1] * (1 + 1e-5) + 1e-6)
    # (3) one parameter pair per row instead of per 64-channel group changes a rank-128 result
    V2 = _rows(10, 20, 128, 1.0)
    V2[:, 64:] *= 8.0
    c, s, z = Q.quantize_values(V2, 8)
    assert np.all(s[:, 1] > 4 * s[:, 0])
    # (4) forgetting the key zero-point in the absorbed form changes lse but not the output
    n = 30
    Uk = _basis(11, 64)
    Kd = _rows(11, n, 64)
    ks, kz = Q.key_params_from_calibration(Kd, 8)
    Kc = Q.quantize_keys(Kd, ks, kz, 8)
    q = I.normal_f64(I.stream_key(11, I.TAG_Q), 128).numpy()
    o1, l1 = Q.attend_quantized_path_b(q, Kc, ks, kz, good[0][:n], good[1][:n], good[2][:n], Uk, None)
    o2, l2 = Q.attend_quantized_path_b(q, Kc, ks, np.zeros_like(kz), good[0][:n], good[1][:n], good[2][:n], Uk, None)
    assert np.abs(o1 - o2).max() < 1e-12 and abs(l1 - l2) > 1e-3
