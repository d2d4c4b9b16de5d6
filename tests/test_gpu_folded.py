"""Sides whose projection has been folded into the model's linear layers (paper Sec. 3.3, "Overheads"): the library is
handed compressed rows directly (q', k', K' with r_k elements per head; v', V' with r_v) and, on the value side, returns
the attention output in the compressed space [B, Hq, r_v] for a U_v^T W_O layer to consume.  The oracle for this is the
absorbed form with no basis (identity in the side's own dimension); the identity that ties it to the unfolded method
(same result after back-projection) is pinned on the CPU in tests/test_oracle_pins.py."""
import numpy as np
import pytest
import torch

import paper_2601_21686_b200 as S
from oracle import stief_oracle as O
from paper_2601_21686_b200 import inputs as I
from tests import _util as U

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _bf16(x64):
    return torch.from_numpy(np.asarray(x64, dtype=np.float64)).to(torch.float32).to(torch.bfloat16)


@pytest.mark.parametrize("fold_k,fold_v,r_k,r_v", [(True, True, 64, 48), (True, False, 32, 96), (False, True, 96, 128), (True, True, 128, 64)])
def test_folded_sides_prefill_append_decode(fold_k, fold_v, r_k, r_v):
    seed, B, Hq, Hkv = 700 + r_k + r_v, 2, 8, 2
    lens = np.array([300, 129], dtype=np.int32)
    T = int(lens.max())
    K, V = I.lowrank_keys(seed, 0, B, T, Hkv), I.gaussian_kv(seed, I.TAG_V, 0, B, T, Hkv)
    q = I.queries(seed, 0, B, Hq)
    k_new, v_new = I.new_token_kv(seed, 0, B, Hkv)
    U_k, U_v = I.stiefel_bases(seed, 0, Hkv, r_k, r_v)
    Uk, Uv = U.f64(U_k), U.f64(U_v)
    G = Hq // Hkv
    # what the model's folded layers would hand over: compressed rows, rounded to bf16 like any activation
    Kin = _bf16(np.einsum("bthd,hdr->bthr", U.f64(K), Uk)) if fold_k else K
    kin = _bf16(np.einsum("bhd,hdr->bhr", U.f64(k_new), Uk)) if fold_k else k_new
    qin = _bf16(np.stack([[U.f64(q)[b, g] @ Uk[g // G] for g in range(Hq)] for b in range(B)])) if fold_k else q
    Vin = _bf16(np.einsum("bthd,hdr->bthr", U.f64(V), Uv)) if fold_v else V
    vin = _bf16(np.einsum("bhd,hdr->bhr", U.f64(v_new), Uv)) if fold_v else v_new
    pg = I.make_paging(seed, lens, reserve_tokens=2, extra_pages=1)
    nan = lambda r: torch.full((pg.num_pages, Hkv, 64, r), U.NAN_BITS, dtype=torch.int16, device=DEV).view(torch.bfloat16)
    layer = S.Layer(Hq, Hkv, r_k, r_v, None if fold_k else U_k.to(DEV), None if fold_v else U_v.to(DEV), nan(r_k), nan(r_v))
    bt = np.where(pg.block_table < 0, 0, pg.block_table).astype(np.int32)
    batch = S.Batch(torch.from_numpy(bt).to(DEV), torch.from_numpy(lens.copy()).to(DEV))
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    S.stief_prefill_compress(layer, batch, Kin.to(DEV), Vin.to(DEV), status=status)
    ws = torch.full((S.stief_decode_workspace_bytes(B, Hq, Hkv, r_v, 3) // 4,), float("nan"), dtype=torch.float32, device=DEV)
    S.stief_decode_workspace_init(ws)
    d_out = r_v if fold_v else 128
    outs = {}
    for mode in ("fused", "separate"):
        out = torch.full((B, Hq, d_out), float("nan"), dtype=torch.bfloat16, device=DEV)
        if mode == "fused":
            S.stief_decode_step(layer, batch, qin.to(DEV), kin.to(DEV), vin.to(DEV), ws, out, num_parts=3, status=status)
        else:
            S.stief_append(layer, batch, kin.to(DEV), vin.to(DEV), status=status)
            S.stief_decode_attention(layer, batch, qin.to(DEV), ws, 3, out, len_add=1, status=status)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        outs[mode] = out
    assert torch.equal(outs["fused"], outs["separate"])
    # oracle: the stored rows are the given rows (bit for bit on a folded side), attention in the side's own dimension
    kp, vp = layer.k_pool.cpu(), layer.v_pool.cpu()
    ref = np.zeros((B, Hq, d_out))
    for b in range(B):
        n = int(lens[b]) + 1
        idx = torch.arange(n)
        pages = torch.from_numpy(pg.block_table[b].astype(np.int64))[idx // 64]
        Kst, Vst = kp[pages, :, idx % 64], vp[pages, :, idx % 64]                 # [n, Hkv, r]
        if fold_k:
            assert torch.equal(Kst[:-1].view(torch.int16), Kin[b, :n - 1].view(torch.int16)) and torch.equal(Kst[-1].view(torch.int16), kin[b].view(torch.int16))
        if fold_v:
            assert torch.equal(Vst[:-1].view(torch.int16), Vin[b, :n - 1].view(torch.int16)) and torch.equal(Vst[-1].view(torch.int16), vin[b].view(torch.int16))
        for g in range(Hq):
            h = g // G
            ref[b, g], _ = O.attend_path_b(U.f64(qin)[b, g], U.f64(Kst)[:, h], U.f64(Vst)[:, h],
                                           None if fold_k else Uk[h], None if fold_v else Uv[h], d_h=128)
    U.check_out(outs["fused"], ref)
    # rows the calls were not asked to write still hold the fill
    used = np.zeros((pg.num_pages, 64), dtype=bool)
    for b in range(B):
        for t in range(int(lens[b]) + 1):
            used[pg.block_table[b, t // 64], t % 64] = True
    for pool in (kp, vp):
        assert np.all(U.bits(pool)[~used[:, None, :].repeat(Hkv, 1)] == U.NAN_BITS)
