"""Shared helpers of the GPU parity tests: build a seeded case, run the oracle on it, compare."""
from __future__ import annotations

import math
from dataclasses import dataclass
from typing import List, Optional

import numpy as np
import torch

import paper_2601_21686_b200 as S
from oracle import stief_oracle as O
from paper_2601_21686_b200 import inputs as I

NAN_BITS = 0x7FC1  # a bf16 NaN: what "unspecified" cache rows hold in these tests


@dataclass
class Case:
    B: int
    Hq: int
    Hkv: int
    r_k: int
    r_v: int
    seq_lens: np.ndarray
    paging: I.Paging
    K: torch.Tensor                  # [B, T, Hkv, 128] bf16 (cpu)
    V: torch.Tensor
    q: torch.Tensor                  # [B, Hq, 128] bf16 (cpu)
    U_k: Optional[torch.Tensor]      # [Hkv or 1, 128, r_k] bf16 (cpu) or None
    U_v: Optional[torch.Tensor]
    # device side
    layer: S.Layer = None
    batch: S.Batch = None
    status: torch.Tensor = None


def make_case(seed, B, Hq, Hkv, r_k, r_v, seq_lens, shared_key_basis=False, full_rank_k=False, full_rank_v=False,
              reserve=2, lowrank=False, q_scale=1.0, device="cuda") -> Case:
    seq_lens = np.asarray(seq_lens, dtype=np.int32)
    T = max(int(seq_lens.max()), 1)
    gen_k = (lambda: I.lowrank_keys(seed, 0, B, T, Hkv)) if lowrank else (lambda: I.gaussian_kv(seed, I.TAG_K, 0, B, T, Hkv))
    K = gen_k()
    V = I.gaussian_kv(seed, I.TAG_V, 0, B, T, Hkv)
    q = I.queries(seed, 0, B, Hq, scale=q_scale)
    U_k, U_v = I.stiefel_bases(seed, 0, Hkv, r_k, r_v, shared_key_basis=shared_key_basis)
    if full_rank_k:
        U_k = None
    if full_rank_v:
        U_v = None
    pg = I.make_paging(seed, seq_lens, reserve_tokens=reserve, extra_pages=1)
    c = Case(B, Hq, Hkv, r_k, r_v, seq_lens, pg, K, V, q, U_k, U_v)
    if device is not None:
        to_device(c, device)
    return c


def to_device(c: Case, device="cuda"):
    nanpool = lambda r: torch.full((c.paging.num_pages, c.Hkv, 64, r), NAN_BITS, dtype=torch.int16, device=device).view(torch.bfloat16)
    c.layer = S.Layer(c.Hq, c.Hkv, c.r_k, c.r_v,
                      None if c.U_k is None else c.U_k.to(device), None if c.U_v is None else c.U_v.to(device),
                      nanpool(c.r_k), nanpool(c.r_v))
    bt = np.where(c.paging.block_table < 0, 0, c.paging.block_table).astype(np.int32)
    c.batch = S.Batch(torch.from_numpy(bt).to(device), torch.from_numpy(c.seq_lens.copy()).to(device))
    c.status = torch.zeros(1, dtype=torch.int32, device=device)


def f64(t: Optional[torch.Tensor]):
    return None if t is None else t.double().cpu().numpy()


def oracle_cache(c: Case, lens=None):
    """Oracle's storage-faithful compressed cache: lists over b of [n_b, Hkv, r] fp64 (bf16 values)."""
    lens = c.seq_lens if lens is None else lens
    return O.compress_layer(f64(c.K), f64(c.V), f64(c.U_k), f64(c.U_v), lens)


def oracle_decode(c: Case, Kd, Vd, q=None):
    return O.decode_layer(f64(c.q if q is None else q), Kd, Vd, f64(c.U_k), f64(c.U_v), "b")


def gpu_cache_rows(c: Case, pool: torch.Tensor, b: int, n: int) -> np.ndarray:
    """Rows [n, Hkv, r] of sequence b gathered from a device pool by the block table (host-side indexing)."""
    p = pool.cpu()
    bt = c.paging.block_table
    out = torch.empty(n, c.Hkv, p.shape[-1], dtype=torch.bfloat16)
    for t0 in range(0, n, 64):
        k = min(64, n - t0)
        out[t0:t0 + k] = p[int(bt[b, t0 // 64]), :, :k, :].permute(1, 0, 2)
    return out


def bits(t: torch.Tensor) -> np.ndarray:
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)


def check_cache(gpu_rows: torch.Tensor, X: np.ndarray, U: Optional[np.ndarray], oracle_rows: np.ndarray):
    """gpu_rows [n, r] bf16 against the oracle's rounded projection [n, r].  An element passes if its bf16
    pattern is within one unit in the last place of the oracle's, or if it is a correct rounding of some
    value inside the fp32 accumulation error bound around the exact product.  Returns (#elements that needed
    the second clause, max ulp distance)."""
    gb = bits(gpu_rows)
    ob = O.bf16_bits(oracle_rows)
    dist = np.abs(O.bf16_ordinal(gb) - O.bf16_ordinal(ob))
    bad = dist > 1
    n_second = 0
    if bad.any():
        exact = X if U is None else X @ U
        g = O.bf16_from_bits(gb)
        acc_err = 128 * 2.0 ** -24 * (np.abs(X) @ np.abs(U) if U is not None else np.abs(X))
        bound = 0.5 * np.maximum(O.bf16_ulp(exact), O.bf16_ulp(g)) + acc_err
        ok2 = np.abs(g - exact) <= bound * (1 + 1e-9)
        n_second = int(bad.sum())
        assert np.all(ok2[bad]), f"cache mismatch: {int((bad & ~ok2).sum())} elements, max ulp distance {int(dist.max())}"
    return n_second, int(dist.max())


def check_out(gpu_out: torch.Tensor, ref: np.ndarray, max_abs=1e-2, rel_l2=5e-3):
    g = gpu_out.double().cpu().numpy()
    assert np.all(np.isfinite(g)), "non-finite output"
    ea = np.abs(g - ref).max()
    rl = np.linalg.norm(g - ref) / max(np.linalg.norm(ref), 1e-30)
    assert ea <= max_abs and rl <= rel_l2, f"max-abs {ea:.3e} (<= {max_abs}), rel-L2 {rl:.3e} (<= {rel_l2})"
    return ea, rl


def workspace_for(c: Case, num_parts: int) -> torch.Tensor:
    n = S.stief_decode_workspace_bytes(c.B, c.Hq, c.Hkv, c.r_v, num_parts)
    ws = torch.full((n // 4,), float("nan"), dtype=torch.float32, device="cuda")
    S.stief_decode_workspace_init(ws)          # the one-time clearing the library asks for
    return ws


def upload_cache(c: Case, Kd, Vd):
    """Write the oracle's cache rows into the device pools through the block table (host-side indexing)."""
    kp = c.layer.k_pool.cpu()
    vp = c.layer.v_pool.cpu()
    bt = c.paging.block_table
    for b in range(c.B):
        n = Kd[b].shape[0]
        for t0 in range(0, n, 64):
            k = min(64, n - t0)
            pg = int(bt[b, t0 // 64])
            kp[pg, :, :k, :] = torch.from_numpy(Kd[b][t0:t0 + k]).to(torch.bfloat16).permute(1, 0, 2)
            vp[pg, :, :k, :] = torch.from_numpy(Vd[b][t0:t0 + k]).to(torch.bfloat16).permute(1, 0, 2)
    c.layer.k_pool.copy_(kp)
    c.layer.v_pool.copy_(vp)
