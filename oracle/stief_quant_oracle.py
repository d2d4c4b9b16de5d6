"""CPU oracle for the integer-quantised compressed KV cache (the paper's Sec. 4.3, "Compatibility with KV cache
quantization", and the caption of its quantisation figure).

TEST INFRASTRUCTURE ONLY: imported by the tests (and nothing in the product).  Plain numpy; shares no code with the
CUDA path.

What the paper fixes: asymmetric integer quantisation of the compressed cache tensors K_down = K P_K and
V_down = V P_V, group size 64; keys use group-wise scales shared across batch and sequence positions within each
KV head, values use token-wise group scales.  Readings taken where it is silent (also listed in the design notes):

* a group is 64 consecutive channels of the compressed dimension (the last group is shorter when the rank is not a
  multiple of 64);
* b-bit codes are 0 .. 2^b - 1 and a code c stands for c * scale + zero, with scale = (max - min) / (2^b - 1) and
  zero = min over the group's values (scale = 1 when max == min);
* key parameters: one (scale, zero) per KV head and channel group, fixed ahead of time from calibration rows and
  shared by every sequence and position; a later value outside the calibrated range is clamped;
* value parameters: one (scale, zero) per token, KV head and channel group, computed from that row when it is written;
* the quantiser sees the projection in fp32 (not rounded to bf16 first) and takes its decision in fp32:
  inv = 1 / scale, code = clamp(rint((x - zero) * inv)) with ties to even; parameters are stored in fp32.

Attention on the quantised cache is ordinary attention (Eq. 18) on the reconstructions of the DEQUANTISED cache
(Eq. 7); as in the unquantised case it is written out twice, literally (path A) and in the absorbed form the GPU
uses (path B: the key scale folds into the projected query, the key zero-point adds the same constant to every
score of a row, the value scale folds into the probabilities and the value zero-point adds p . zero per group).
"""
from __future__ import annotations

import math

import numpy as np

GROUP = 64
F32 = np.float32


def groups_of(r: int):
    """Channel ranges [lo, hi) of the quantisation groups of a rank-r row."""
    return [(lo, min(lo + GROUP, r)) for lo in range(0, r, GROUP)]


def minmax_params(lo_vals: np.ndarray, hi_vals: np.ndarray, bits: int):
    """(scale, zero) in fp32 from group minima / maxima (fp32 arithmetic, one division)."""
    mn = np.asarray(lo_vals, dtype=F32)
    mx = np.asarray(hi_vals, dtype=F32)
    levels = F32(2 ** bits - 1)
    scale = ((mx - mn) / levels).astype(F32)
    scale = np.where(mx > mn, scale, F32(1.0)).astype(F32)
    return scale, mn


def codes_from(x32: np.ndarray, scale: np.ndarray, zero: np.ndarray, bits: int) -> np.ndarray:
    """Quantiser decision in fp32: clamp(rint((x - zero) * (1 / scale)))."""
    inv = (F32(1.0) / scale).astype(F32)
    y = ((x32 - zero).astype(F32) * inv).astype(F32)
    return np.clip(np.rint(y), 0, 2 ** bits - 1).astype(np.int32)


def project_f32(X: np.ndarray, U: np.ndarray | None) -> np.ndarray:
    """X U (Eq. 1) in fp64, rounded once to fp32: what the quantiser sees."""
    X = np.asarray(X, dtype=np.float64)
    return (X if U is None else X @ np.asarray(U, dtype=np.float64)).astype(F32)


def key_params_from_calibration(K_down32: np.ndarray, bits: int):
    """Static key parameters of one KV head: per channel group, min / max over all calibration rows [n, r_k].
    Returns (scale [ng], zero [ng]) fp32."""
    r = K_down32.shape[1]
    mn = np.array([K_down32[:, lo:hi].min() for lo, hi in groups_of(r)], dtype=F32)
    mx = np.array([K_down32[:, lo:hi].max() for lo, hi in groups_of(r)], dtype=F32)
    return minmax_params(mn, mx, bits)


def quantize_keys(K_down32: np.ndarray, scale: np.ndarray, zero: np.ndarray, bits: int) -> np.ndarray:
    """Codes [n, r_k] of key rows under the head's static parameters (values outside the range clamp)."""
    out = np.empty(K_down32.shape, dtype=np.int32)
    for g, (lo, hi) in enumerate(groups_of(K_down32.shape[1])):
        out[:, lo:hi] = codes_from(K_down32[:, lo:hi], scale[g], zero[g], bits)
    return out


def quantize_values(V_down32: np.ndarray, bits: int):
    """Token-wise group quantisation of value rows [n, r_v]: returns (codes [n, r_v], scale [n, ng], zero [n, ng])."""
    n, r = V_down32.shape
    gs = groups_of(r)
    codes = np.empty((n, r), dtype=np.int32)
    scale = np.empty((n, len(gs)), dtype=F32)
    zero = np.empty((n, len(gs)), dtype=F32)
    for g, (lo, hi) in enumerate(gs):
        blk = V_down32[:, lo:hi]
        s, z = minmax_params(blk.min(axis=1), blk.max(axis=1), bits)
        scale[:, g], zero[:, g] = s, z
        codes[:, lo:hi] = codes_from(blk, s[:, None], z[:, None], bits)
    return codes, scale, zero


def dequant_keys(codes: np.ndarray, scale: np.ndarray, zero: np.ndarray) -> np.ndarray:
    """fp64 rows code * scale + zero with per-group key parameters [ng]."""
    out = np.empty(codes.shape, dtype=np.float64)
    for g, (lo, hi) in enumerate(groups_of(codes.shape[1])):
        out[:, lo:hi] = codes[:, lo:hi].astype(np.float64) * np.float64(scale[g]) + np.float64(zero[g])
    return out


def dequant_values(codes: np.ndarray, scale: np.ndarray, zero: np.ndarray) -> np.ndarray:
    """fp64 rows with per-token group parameters [n, ng]."""
    out = np.empty(codes.shape, dtype=np.float64)
    for g, (lo, hi) in enumerate(groups_of(codes.shape[1])):
        out[:, lo:hi] = codes[:, lo:hi].astype(np.float64) * scale[:, g:g + 1].astype(np.float64) + zero[:, g:g + 1].astype(np.float64)
    return out


def _softmax_row(s: np.ndarray):
    m = np.max(s)
    e = np.exp(s - m)
    z = np.sum(e)
    return e / z, m + math.log(z)


def attend_quantized_path_a(q, Kc, k_scale, k_zero, Vc, v_scale, v_zero, U_k, U_v, d_h: int = 128):
    """Literal form: dequantise, reconstruct K_tilde, V_tilde in the original dimension (Eq. 7), run Eq. 18."""
    q = np.asarray(q, dtype=np.float64)
    if Kc.shape[0] == 0:
        return np.zeros(d_h), -math.inf
    Kd = dequant_keys(Kc, k_scale, k_zero)
    Vd = dequant_values(Vc, v_scale, v_zero)
    K_t = Kd if U_k is None else Kd @ np.asarray(U_k, dtype=np.float64).T
    V_t = Vd if U_v is None else Vd @ np.asarray(U_v, dtype=np.float64).T
    p, lse = _softmax_row((K_t @ q) / math.sqrt(d_h))
    return p @ V_t, lse


def attend_quantized_path_b(q, Kc, k_scale, k_zero, Vc, v_scale, v_zero, U_k, U_v, d_h: int = 128):
    """Absorbed form: integer codes are contracted directly.  scores = (q' * scale_g) . codes + q' . zero_g;
    mix = sum_t (p_t * scale_tg) codes_t + sum_t p_t zero_tg per group; back-projection once."""
    q = np.asarray(q, dtype=np.float64)
    n = Kc.shape[0]
    if n == 0:
        return np.zeros(d_h), -math.inf
    qp = q if U_k is None else q @ np.asarray(U_k, dtype=np.float64)
    s = np.zeros(n)
    for g, (lo, hi) in enumerate(groups_of(Kc.shape[1])):
        s += Kc[:, lo:hi].astype(np.float64) @ (qp[lo:hi] * np.float64(k_scale[g])) + np.float64(k_zero[g]) * qp[lo:hi].sum()
    p, lse = _softmax_row(s / math.sqrt(d_h))
    o_down = np.zeros(Vc.shape[1])
    for g, (lo, hi) in enumerate(groups_of(Vc.shape[1])):
        o_down[lo:hi] = (p * v_scale[:, g].astype(np.float64)) @ Vc[:, lo:hi].astype(np.float64) + p @ v_zero[:, g].astype(np.float64)
    out = o_down if U_v is None else o_down @ np.asarray(U_v, dtype=np.float64).T
    return out, lse


def quantized_cache_bytes(r_k: int, r_v: int, bits: int, meta_bytes: int = 8) -> float:
    """Bytes one (token, KV head) occupies: packed codes of both sides plus the value row's (scale, zero) pairs."""
    return (r_k + r_v) * bits / 8.0 + len(groups_of(r_v)) * meta_bytes
