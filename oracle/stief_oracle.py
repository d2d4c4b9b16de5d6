"""CPU oracle for decode attention over a rank-compressed KV cache (StiefAttention inference path).

TEST INFRASTRUCTURE ONLY.  This file is the plain, slow, fp64 statement of what the GPU library
must compute.  Only the tests, the smoke check and the benchmark's CPU-baseline leg may import it;
the product never does.  It shares no code with the CUDA path and imports nothing from the package.

Notation follows the paper: a key matrix K in R^{n x d_h} of one KV head, a column-orthonormal
basis P_K in R^{d_h x r_K} (here ``U_k``), the cached projection K_down = K P_K (Eq. 1), the
reconstruction K_tilde = K_down P_K^T used inside attention (Eq. 2 / Eq. 7), the same for values,
and per-head attention softmax(Q K^T / sqrt(d_h)) V (Eq. 18) with a single query row at decode.

Two evaluation orders of the same function are written out independently:

* Path A (literal):   rebuild K_tilde, V_tilde in the original dimension, run textbook attention.
* Path B (absorbed):  q' = q P_K, scores q' K_down^T, mix p V_down, back-project by P_V^T.

They agree to rounding because q K_tilde^T = (q P_K) K_down^T and p V_tilde = (p V_down) P_V^T.

Storage: the cache holds bf16.  ``rnd_bf16`` rounds an fp64 value once, to nearest-even, straight to
bf16 (no intermediate fp32 rounding).  Everything else is fp64.

Pins (tests/test_oracle_pins.py): U^T U = I; r = d_h gives exact softmax attention (checked against
torch's scaled_dot_product_attention in fp64); attention on explicitly reconstructed K U U^T, V U U^T
through that same library routine; brute-force loops on tiny inputs; closed forms (zero query ->
mean of V_tilde rows, constant V, one dominating key); span invariance U -> U O; the combine against
scipy's logsumexp and against the unsplit result; the cache address formula against a tagged pattern;
the paper's 16 GB sizing example and Eq. 3.  No function here is "parity unpinned".
"""
from __future__ import annotations

import math

import numpy as np

D_HEAD = 128
PAGE = 64


# --------------------------------------------------------------------------------------
# bf16 storage rounding
# --------------------------------------------------------------------------------------

def rnd_bf16(x: np.ndarray) -> np.ndarray:
    """Round fp64 values to the nearest bf16 value (ties to even); returned as fp64.

    bf16 has 8 significant bits, exponent range of fp32.  For |x| in [2^(e-1), 2^e) the spacing is
    2^(e-8); below the smallest normal (2^-126) the spacing stays 2^-133.  Values that round to
    2^128 or beyond become infinity.
    """
    x = np.asarray(x, dtype=np.float64)
    _, e = np.frexp(x)                                  # x = m * 2^e, 0.5 <= |m| < 1
    e = np.maximum(e, -125)                             # subnormal range shares the last normal spacing
    q = np.ldexp(1.0, e - 8)
    y = np.rint(x / q) * q                              # rint: ties to even; scaling by 2^k is exact
    y = np.where(np.abs(y) >= 2.0 ** 128, np.copysign(np.inf, y), y)
    return np.where(np.isfinite(x), y, x)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of values that are already exactly representable in bf16."""
    f32 = np.asarray(x, dtype=np.float64).astype(np.float32)
    return (f32.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


def bf16_from_bits(b: np.ndarray) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def bf16_ordinal(bits: np.ndarray) -> np.ndarray:
    """Map bf16 bit patterns to integers that increase with the value (ulp distance = difference)."""
    b = np.asarray(bits, dtype=np.uint16).astype(np.int32)
    return np.where(b & 0x8000, -(b & 0x7FFF), b)


def bf16_ulp(x: np.ndarray) -> np.ndarray:
    """Spacing of bf16 numbers around x: 2^(e-8) for |x| in [2^(e-1), 2^e), and 2^-133 from the smallest
    normal (2^-126) down to and including zero."""
    x = np.asarray(x, dtype=np.float64)
    _, e = np.frexp(x)
    e = np.where(x == 0.0, -125, e)                     # frexp(0) reports exponent 0; zero sits in the subnormal range
    return np.ldexp(1.0, np.maximum(e, -125) - 8)


# --------------------------------------------------------------------------------------
# Eq. 1: the cached projection; Eq. 2 / Eq. 7: the reconstruction
# --------------------------------------------------------------------------------------

def compress(X: np.ndarray, U: np.ndarray | None, storage: bool = True) -> np.ndarray:
    """X_down = X U  (Eq. 1), X [n, d_h], U [d_h, r].  ``U is None`` keeps the rows full rank
    (Algorithm 2: a layer may keep keys or values uncompressed).  With ``storage`` the result is
    rounded once to bf16, as the cache stores it."""
    X = np.asarray(X, dtype=np.float64)
    Y = X if U is None else X @ np.asarray(U, dtype=np.float64)
    return rnd_bf16(Y) if storage else Y


def reconstruct(X_down: np.ndarray, U: np.ndarray | None) -> np.ndarray:
    """X_tilde = X_down U^T  (Eq. 2 / Eq. 7)."""
    X_down = np.asarray(X_down, dtype=np.float64)
    return X_down if U is None else X_down @ np.asarray(U, dtype=np.float64).T


# --------------------------------------------------------------------------------------
# Eq. 18 with a single query row (decode)
# --------------------------------------------------------------------------------------

def _softmax_row(s: np.ndarray):
    """Max-subtracted softmax of one score row; returns (p, lse).  Empty row -> (empty, -inf)."""
    if s.size == 0:
        return s, -math.inf
    m = np.max(s)
    e = np.exp(s - m)
    z = np.sum(e)
    return e / z, m + math.log(z)


def attend_path_a(q: np.ndarray, K_down: np.ndarray, V_down: np.ndarray, U_k, U_v, d_h: int = D_HEAD):
    """Literal form: attention of query row q [d_h] on K_tilde, V_tilde.  Returns (out [d_h], lse)."""
    q = np.asarray(q, dtype=np.float64)
    K_t = reconstruct(K_down, U_k)                      # [n, d_h]
    V_t = reconstruct(V_down, U_v)                      # [n, d_h]
    if K_t.shape[0] == 0:
        return np.zeros(d_h), -math.inf
    s = (K_t @ q) / math.sqrt(d_h)                      # scale is 1/sqrt(d_h) of the ORIGINAL dimension
    p, lse = _softmax_row(s)
    return p @ V_t, lse


def attend_path_b(q: np.ndarray, K_down: np.ndarray, V_down: np.ndarray, U_k, U_v, d_h: int = D_HEAD):
    """Absorbed form: project the query (the projection that compressing keys induces on queries,
    Sec. 2.2), score and mix in the compressed space, back-project once.  Returns (out [d_h], lse)."""
    q = np.asarray(q, dtype=np.float64)
    K_down = np.asarray(K_down, dtype=np.float64)
    V_down = np.asarray(V_down, dtype=np.float64)
    if K_down.shape[0] == 0:
        return np.zeros(d_h), -math.inf
    qp = q if U_k is None else q @ np.asarray(U_k, dtype=np.float64)         # [r_k]
    s = (K_down @ qp) / math.sqrt(d_h)
    p, lse = _softmax_row(s)
    o_down = p @ V_down                                                       # [r_v]
    out = o_down if U_v is None else o_down @ np.asarray(U_v, dtype=np.float64).T
    return out, lse


def attend_rows_causal(Q: np.ndarray, K_down: np.ndarray, V_down: np.ndarray, U_k, U_v, q_start: int, path: str = "b",
                       d_h: int = D_HEAD):
    """Several query rows of one head against one cache (App. A.1: during prefilling Q has one row per prefix token;
    Eq. 18 per row).  Row i sits at absolute position q_start + i and, the layer being a decoder layer, attends the
    cached positions 0 .. q_start + i only (its own key/value row is in the cache).  Each row is the single-row
    definition applied to that prefix.  Returns (out [n_q, d_out], lse [n_q])."""
    fn = attend_path_a if path == "a" else attend_path_b
    outs, lses = [], []
    for i in range(Q.shape[0]):
        n = q_start + i + 1
        o, l = fn(Q[i], K_down[:n], V_down[:n], U_k, U_v, d_h)
        outs.append(o)
        lses.append(l)
    return np.stack(outs), np.array(lses)


def attend_compressed_partial(q, K_down, V_down, U_k, d_h: int = D_HEAD):
    """One T-chunk of Path B without the back-projection: (o_down [r_v] normalised within the chunk, lse)."""
    K_down = np.asarray(K_down, dtype=np.float64)
    V_down = np.asarray(V_down, dtype=np.float64)
    if K_down.shape[0] == 0:
        return np.zeros(V_down.shape[1]), -math.inf
    q = np.asarray(q, dtype=np.float64)
    qp = q if U_k is None else q @ np.asarray(U_k, dtype=np.float64)
    p, lse = _softmax_row((K_down @ qp) / math.sqrt(d_h))
    return p @ V_down, lse


# --------------------------------------------------------------------------------------
# split-T combine: exact re-association of Eq. 18 over chunks of the prefix
# --------------------------------------------------------------------------------------

def split_combine(partial_o: np.ndarray, partial_lse: np.ndarray):
    """Merge S chunk results.  partial_o [S, c] are chunk-normalised outputs, partial_lse [S] their
    log-sum-exp.  out = sum_s w_s o_s with w_s = exp(lse_s - lse), lse = log sum_s exp(lse_s).
    Chunks with lse = -inf (no tokens) weigh nothing; if all are empty the result is zeros, lse -inf."""
    partial_o = np.asarray(partial_o, dtype=np.float64)
    partial_lse = np.asarray(partial_lse, dtype=np.float64)
    live = partial_lse > -math.inf
    if not np.any(live):
        return np.zeros(partial_o.shape[1]), -math.inf
    m = np.max(partial_lse[live])
    w = np.where(live, np.exp(np.where(live, partial_lse, m) - m), 0.0)
    z = np.sum(w)
    out = (w[:, None] * np.where(live[:, None], partial_o, 0.0)).sum(axis=0) / z
    return out, m + math.log(z)


# --------------------------------------------------------------------------------------
# paged cache layout
# --------------------------------------------------------------------------------------

def pool_offset(block_table: np.ndarray, b: int, t: int, h: int, Hkv: int, r: int) -> int:
    """Element offset of (sequence b, token t, KV head h, column 0) in a pool laid out
    [num_pages][Hkv][PAGE][r]."""
    page = int(block_table[b, t // PAGE])
    return ((page * Hkv + h) * PAGE + t % PAGE) * r


def write_cache_rows(pool: np.ndarray, block_table, b: int, h: int, t0: int, rows: np.ndarray, Hkv: int):
    """Store ``rows`` [n, r] (values) for tokens t0.. of (b, h) into the flat fp64 pool image."""
    r = rows.shape[1]
    for i in range(rows.shape[0]):
        off = pool_offset(block_table, b, t0 + i, h, Hkv, r)
        pool[off:off + r] = rows[i]


def read_cache_rows(pool: np.ndarray, block_table, b: int, h: int, n: int, Hkv: int, r: int) -> np.ndarray:
    out = np.empty((n, r), dtype=np.float64)
    for t in range(n):
        off = pool_offset(block_table, b, t, h, Hkv, r)
        out[t] = pool[off:off + r]
    return out


# --------------------------------------------------------------------------------------
# whole-layer drivers (loops over sequences, KV heads and the query heads of each group)
# --------------------------------------------------------------------------------------

def basis_of(U: np.ndarray | None, h: int):
    """Basis of KV head h from a stack [Hkv or 1, d_h, r]; one shared key basis is a stack of one."""
    if U is None:
        return None
    return U[h if U.shape[0] > 1 else 0]


def compress_layer(K: np.ndarray, V: np.ndarray, U_k, U_v, seq_lens):
    """K, V [B, T, Hkv, d_h] -> lists over b of K_down [n_b, Hkv, r_k], V_down [n_b, Hkv, r_v] (bf16 values)."""
    B, _, Hkv, _ = K.shape
    Kd, Vd = [], []
    for b in range(B):
        n = int(seq_lens[b])
        Kd.append(np.stack([compress(K[b, :n, h], basis_of(U_k, h)) for h in range(Hkv)], axis=1))
        Vd.append(np.stack([compress(V[b, :n, h], basis_of(U_v, h)) for h in range(Hkv)], axis=1))
    return Kd, Vd


def decode_layer(q: np.ndarray, Kd, Vd, U_k, U_v, path: str = "b"):
    """q [B, Hq, d_h]; Kd/Vd lists over b of [n_b, Hkv, r].  Query head g reads KV head g // (Hq/Hkv)
    (GQA: several query heads share one KV head; contiguous groups).  Returns out [B, Hq, d_h], lse [B, Hq]."""
    B, Hq, d_h = q.shape
    Hkv = Kd[0].shape[1]
    G = Hq // Hkv
    fn = attend_path_a if path == "a" else attend_path_b
    out = np.zeros((B, Hq, d_h))
    lse = np.full((B, Hq), -math.inf)
    for b in range(B):
        for g in range(Hq):
            h = g // G
            out[b, g], lse[b, g] = fn(q[b, g], Kd[b][:, h], Vd[b][:, h], basis_of(U_k, h), basis_of(U_v, h), d_h)
    return out, lse


def decode_layer_split(q, Kd, Vd, U_k, U_v, chunk_tokens: int):
    """Same result as decode_layer, evaluated chunk by chunk and merged with split_combine, the
    back-projection applied once after the merge (it is linear)."""
    B, Hq, d_h = q.shape
    Hkv = Kd[0].shape[1]
    G = Hq // Hkv
    out = np.zeros((B, Hq, d_h))
    lse = np.full((B, Hq), -math.inf)
    for b in range(B):
        n = Kd[b].shape[0]
        for g in range(Hq):
            h = g // G
            po, pl = [], []
            for t0 in range(0, max(n, 1), chunk_tokens):
                o, l = attend_compressed_partial(q[b, g], Kd[b][t0:t0 + chunk_tokens, h],
                                                 Vd[b][t0:t0 + chunk_tokens, h], basis_of(U_k, h), d_h)
                po.append(o)
                pl.append(l)
            o_down, lse[b, g] = split_combine(np.stack(po), np.array(pl))
            Uv = basis_of(U_v, h)
            out[b, g] = o_down if Uv is None else o_down @ np.asarray(Uv, dtype=np.float64).T
    return out, lse


# --------------------------------------------------------------------------------------
# byte accounting (Eq. 3 and the Introduction's sizing example)
# --------------------------------------------------------------------------------------

def cache_ratio(r_k: int, r_v: int, d_h: int = D_HEAD) -> float:
    """CR = (r_K + r_V) / (2 d_h)  (Eq. 3)."""
    return (r_k + r_v) / (2.0 * d_h)


def kv_cache_bytes(n_layers: int, Hkv: int, T: int, B: int, ranks=None, d_h: int = D_HEAD, bytes_per_el: int = 2) -> int:
    """Bytes of a half-precision KV cache; ``ranks`` = per-layer (r_k, r_v), None = uncompressed."""
    if ranks is None:
        ranks = [(d_h, d_h)] * n_layers
    return sum((rk + rv) * Hkv * T * B * bytes_per_el for rk, rv in ranks)
