"""Seeded synthetic inputs for the compressed-cache decode path.

This module only *makes inputs*: random tensors, orthonormal bases, rank
profiles, sequence lengths and block tables.  It holds none of the method's
arithmetic (no projection, no attention, no cache rounding), so both the CUDA
path and the CPU oracle can be fed from it without sharing any computation.

Every tensor is a pure function of ``(seed, stream id, flat index)`` through a
counter-based SplitMix64 generator written with torch int64 ops, so it runs
unchanged on CPU and on a CUDA device and any slice can be regenerated alone.
Values are drawn in fp64 (Box-Muller) and then rounded to bf16; a test that
generates on the device copies the very tensors it used back to the host for the
oracle, so both sides always see the same bits.

Shapes follow Llama3-8B attention (32 query heads, 8 KV heads, head dim 128, 32
layers), the model the paper sizes its 16 GB cache example on (Introduction).
"""
from __future__ import annotations

import math
from dataclasses import dataclass

import numpy as np
import torch

D_HEAD = 128
PAGE = 64
RANK_SET = (32, 48, 64, 96, 128)

_M64 = (1 << 64) - 1
_GOLDEN = 0x9E3779B97F4A7C15
_C1 = 0xBF58476D1CE4E5B9
_C2 = 0x94D049BB133111EB

# stream tags
TAG_Q, TAG_K, TAG_V, TAG_UK, TAG_UV, TAG_A, TAG_BM, TAG_KNEW, TAG_VNEW = 1, 2, 3, 4, 5, 6, 7, 8, 9
TAG_LENS, TAG_PERM, TAG_PROFILE = 10, 11, 12


def _s64(x: int) -> int:
    """Python int (mod 2^64) -> the signed value torch.int64 holds for the same bits."""
    x &= _M64
    return x - (1 << 64) if x >= (1 << 63) else x


def _mix_int(z: int) -> int:
    z = (z + _GOLDEN) & _M64
    z = ((z ^ (z >> 30)) * _C1) & _M64
    z = ((z ^ (z >> 27)) * _C2) & _M64
    return z ^ (z >> 31)


def stream_key(seed: int, tag: int, layer: int = 0, b: int = 0, h: int = 0) -> int:
    """64-bit key of one named stream; distinct (tag, layer, b, h) give unrelated streams."""
    sid = (tag << 48) | (layer << 32) | (b << 16) | h
    return _mix_int(_mix_int(seed & _M64) ^ sid)


def _lsr(z: torch.Tensor, s: int) -> torch.Tensor:
    """Logical shift right on int64 (torch's >> is arithmetic)."""
    return (z >> s) & ((1 << (64 - s)) - 1)


def splitmix64(key: int, idx: torch.Tensor) -> torch.Tensor:
    """SplitMix64 output number ``idx`` (int64 tensor, >= 0) of the stream ``key``; int64 bit patterns."""
    z = idx * _s64(_GOLDEN) + _s64(key + _GOLDEN)
    z = (z ^ _lsr(z, 30)) * _s64(_C1)
    z = (z ^ _lsr(z, 27)) * _s64(_C2)
    return z ^ _lsr(z, 31)


def uniform_bits53(key: int, idx: torch.Tensor) -> torch.Tensor:
    """53 random bits per index as int64 in [0, 2^53)."""
    return _lsr(splitmix64(key, idx), 11)


def normal_f64(key: int, n: int, device="cpu", start: int = 0, chunk: int = 1 << 24) -> torch.Tensor:
    """``n`` standard normals (fp64) number ``start .. start+n`` of stream ``key`` (Box-Muller, one per index)."""
    out = torch.empty(n, dtype=torch.float64, device=device)
    two53 = float(1 << 53)
    for c0 in range(0, n, chunk):
        c1 = min(n, c0 + chunk)
        i = torch.arange(start + c0, start + c1, dtype=torch.int64, device=device)
        u1 = (uniform_bits53(key, 2 * i).to(torch.float64) + 1.0) / two53        # (0, 1]
        u2 = uniform_bits53(key, 2 * i + 1).to(torch.float64) / two53            # [0, 1)
        out[c0:c1] = torch.sqrt(-2.0 * torch.log(u1)) * torch.cos((2.0 * math.pi) * u2)
    return out


def normal_bf16(key: int, shape, device="cpu", scale: float = 1.0) -> torch.Tensor:
    n = int(np.prod(shape))
    x = normal_f64(key, n, device=device)
    if scale != 1.0:
        x = x * scale
    return x.to(torch.float32).to(torch.bfloat16).reshape(shape)


def randint(key: int, n: int, lo: int, hi: int) -> np.ndarray:
    """``n`` integers uniform in [lo, hi] (host)."""
    i = torch.arange(n, dtype=torch.int64)
    bits = uniform_bits53(key, i).numpy().astype(np.uint64)
    return (lo + (bits % np.uint64(hi - lo + 1))).astype(np.int64)


def permutation(key: int, n: int) -> np.ndarray:
    """A seeded permutation of range(n): argsort of n random 53-bit keys (ties broken by index)."""
    i = torch.arange(n, dtype=torch.int64)
    bits = uniform_bits53(key, i).numpy()
    return np.argsort(bits, kind="stable").astype(np.int64)


# --------------------------------------------------------------------------------------
# bases, rank profile
# --------------------------------------------------------------------------------------

def stiefel_basis_f64(seed: int, tag: int, layer: int, h: int, r: int, d: int = D_HEAD) -> np.ndarray:
    """Leading ``r`` columns of the Q factor of a seeded d x d Gaussian, fp64, diag(R) > 0.

    Truncating a full orthonormal matrix to its leading columns is how the paper cuts a
    rank-r basis (Eq. 6); because thin QR nests, this is also the Q factor of the seeded
    d x r Gaussian made of the first r columns.
    """
    a = normal_f64(stream_key(seed, tag, layer, 0, h), d * d).numpy().reshape(d, d)
    qf, rf = np.linalg.qr(a)
    sgn = np.sign(np.diag(rf))
    sgn[sgn == 0] = 1.0
    return np.ascontiguousarray((qf * sgn[None, :])[:, :r])


def stiefel_bases(seed: int, layer: int, Hkv: int, r_k: int, r_v: int, d: int = D_HEAD, shared_key_basis=False):
    """(U_k, U_v) as bf16 tensors [Hkv or 1, d, r]; keys may share one basis per layer (Sec. 3.3, head sharing)."""
    nk = 1 if shared_key_basis else Hkv
    uk = np.stack([stiefel_basis_f64(seed, TAG_UK, layer, h, r_k, d) for h in range(nk)])
    uv = np.stack([stiefel_basis_f64(seed, TAG_UV, layer, h, r_v, d) for h in range(Hkv)])
    to = lambda a: torch.from_numpy(a).to(torch.float32).to(torch.bfloat16).contiguous()
    return to(uk), to(uv)


def rank_profile(seed: int, n_layers: int = 32, rank_set=RANK_SET):
    """Per-layer (r_k, r_v), each drawn independently from ``rank_set`` by a seeded stream."""
    draws = randint(stream_key(seed, TAG_PROFILE), 2 * n_layers, 0, len(rank_set) - 1)
    return [(rank_set[int(draws[2 * l])], rank_set[int(draws[2 * l + 1])]) for l in range(n_layers)]


# --------------------------------------------------------------------------------------
# activations
# --------------------------------------------------------------------------------------

def gaussian_kv(seed: int, tag: int, layer: int, B: int, T: int, Hkv: int, d: int = D_HEAD, device="cpu"):
    """[B, T, Hkv, d] bf16 ~ N(0,1)."""
    out = torch.empty(B, T, Hkv, d, dtype=torch.bfloat16, device=device)
    for b in range(B):
        out[b] = normal_bf16(stream_key(seed, tag, layer, b, 0), (T, Hkv, d), device=device)
    return out


def lowrank_keys(seed: int, layer: int, B: int, T: int, Hkv: int, rank: int = 48, noise: float = 0.1,
                 d: int = D_HEAD, device="cpu"):
    """[B, T, Hkv, d] bf16 keys: (A @ Bm)/sqrt(rank) + noise * N(0,1), A [T,rank], Bm [rank,d] per (b, h).

    Real key activations concentrate in a low-dimensional subspace (the premise of head-dimension
    compression, Sec. 2.1); this gives unit-variance entries with that structure.
    """
    out = torch.empty(B, T, Hkv, d, dtype=torch.bfloat16, device=device)
    for b in range(B):
        for h in range(Hkv):
            a = normal_f64(stream_key(seed, TAG_A, layer, b, h), T * rank, device=device).reshape(T, rank)
            bm = normal_f64(stream_key(seed, TAG_BM, layer, b, h), rank * d, device=device).reshape(rank, d)
            nz = normal_f64(stream_key(seed, TAG_K, layer, b, h), T * d, device=device).reshape(T, d)
            out[b, :, h, :] = ((a @ bm) / math.sqrt(rank) + noise * nz).to(torch.float32).to(torch.bfloat16)
    return out


def queries(seed: int, layer: int, B: int, Hq: int, d: int = D_HEAD, scale: float = 1.0, device="cpu", step: int = 0):
    return normal_bf16(stream_key(seed, TAG_Q, layer, step, 0), (B, Hq, d), device=device, scale=scale)


def new_token_kv(seed: int, layer: int, B: int, Hkv: int, d: int = D_HEAD, device="cpu", step: int = 0):
    k = normal_bf16(stream_key(seed, TAG_KNEW, layer, step, 0), (B, Hkv, d), device=device)
    v = normal_bf16(stream_key(seed, TAG_VNEW, layer, step, 0), (B, Hkv, d), device=device)
    return k, v


# --------------------------------------------------------------------------------------
# paging
# --------------------------------------------------------------------------------------

@dataclass
class Paging:
    block_table: np.ndarray     # [B, max_pages_per_seq] int32 page ids (unused slots hold -1)
    seq_lens: np.ndarray        # [B] int32
    num_pages: int              # pages in the pool


def make_paging(seed: int, seq_lens, reserve_tokens: int = 0, extra_pages: int = 0, shuffled: bool = True) -> Paging:
    """Hand pages of a pool to sequences from a seeded permutation, so block tables are non-contiguous.

    Each sequence gets ceil((len + reserve_tokens)/PAGE) pages (room to append ``reserve_tokens``).
    """
    seq_lens = np.asarray(seq_lens, dtype=np.int64)
    need = [(int(n) + reserve_tokens + PAGE - 1) // PAGE for n in seq_lens]
    mpp = max(1, max(need))
    num_pages = int(sum(need)) + extra_pages
    order = permutation(stream_key(seed, TAG_PERM), num_pages) if shuffled else np.arange(num_pages)
    bt = np.full((len(seq_lens), mpp), -1, dtype=np.int32)
    pos = 0
    for b, k in enumerate(need):
        bt[b, :k] = order[pos:pos + k]
        pos += k
    return Paging(bt, seq_lens.astype(np.int32), num_pages)


def ragged_lengths(seed: int, B: int, lo: int = 1024, hi: int = 16384) -> np.ndarray:
    return randint(stream_key(seed, TAG_LENS), B, lo, hi).astype(np.int32)


# --------------------------------------------------------------------------------------
# error surfaces for the rank selector (inputs only: the selector's arithmetic is not here)
# --------------------------------------------------------------------------------------

TAG_SURFACE = 13


def error_surfaces(seed: int, n_layers: int, cand_k=RANK_SET, cand_v=RANK_SET, d: int = D_HEAD) -> np.ndarray:
    """Synthetic layer-output error tables [L][len(cand_k)][len(cand_v)] (fp64) with the qualitative shape the paper
    reports for its measured ones: zero at the full-rank pair, growing as either rank drops, values costlier to
    compress than keys, early and late layers more sensitive than the middle ones, plus seeded per-entry jitter."""
    u = uniform_bits53(stream_key(seed, TAG_SURFACE), torch.arange(n_layers * (2 + len(cand_k) * len(cand_v)), dtype=torch.int64)).numpy()
    out = np.zeros((n_layers, len(cand_k), len(cand_v)))
    pos = 0
    for l in range(n_layers):
        x = l / max(n_layers - 1, 1)
        bowl = 0.35 + 1.2 * (2.0 * x - 1.0) ** 2 + (0.6 if x > 0.8 else 0.0)
        a_k = bowl * (0.6 + 0.8 * u[pos]); a_v = 1.8 * bowl * (0.6 + 0.8 * u[pos + 1]); pos += 2
        for i, rk in enumerate(cand_k):
            for j, rv in enumerate(cand_v):
                lost_k, lost_v = max(0.0, 1.0 - rk / d), max(0.0, 1.0 - rv / d)
                base = a_k * lost_k ** 1.5 + a_v * lost_v ** 1.5 + 0.5 * a_k * a_v * lost_k * lost_v
                out[l, i, j] = 0.0 if (rk == d and rv == d) else base * (0.9 + 0.2 * u[pos])
                pos += 1
    return out
