"""GPU parity of the integer-quantised compressed cache (8-bit and 4-bit codes, every rank) against its oracle
(oracle/stief_quant_oracle.py).

A quantised code is an integer decided by floating point, so both sides decide in the same precision (fp32, the
kernel's); what still differs is the fp32 accumulation order of the projection the quantiser sees.  A cache element
therefore passes if its dequantised value is within one quantisation step of the oracle's (and the parameters agree to
fp32 rounding of the row's extremes); the share of codes that differ at all is bounded.  The decode kernel is checked
twice: tightly on the oracle's OWN codes uploaded to the device, and end to end (GPU prefill + append + decode) with
the spec output tolerances (max-abs 1e-2, relative L2 5e-3)."""
import numpy as np
import pytest
import torch

import paper_2601_21686_b200 as S
from oracle import stief_oracle as O
from oracle import stief_quant_oracle as Q
from paper_2601_21686_b200 import inputs as I
from tests import _util as U

pytestmark = pytest.mark.gpu
DEV = "cuda"


def vpos(t):
    """Position of token t (0..63 within its page) inside a value page's channel rows: the documented layout."""
    t = np.asarray(t)
    return (t & ~15) + 4 * ((t & 7) >> 1) + (t & 1) + 2 * ((t >> 3) & 1)


def test_value_positions_are_a_permutation_of_each_16_tokens():
    p = vpos(np.arange(64))
    assert sorted(p.tolist()) == list(range(64)) and np.all(p // 16 == np.arange(64) // 16)
    assert p[:16].tolist() == [0, 1, 4, 5, 8, 9, 12, 13, 2, 3, 6, 7, 10, 11, 14, 15]


def nibble_index(i):
    """(byte, shift) of index i of a 4-bit row: per 32 indices, byte i % 16 of the block; low nibble for the first 16."""
    i = np.asarray(i)
    return (i >> 5) * 16 + (i & 15), 4 * ((i >> 4) & 1)


def unpack_rows(rows: np.ndarray, n_idx: int, bits: int) -> np.ndarray:
    """[..., row bytes] uint8 -> [..., n_idx] codes (the documented byte / nibble order)."""
    if bits == 8:
        return rows[..., :n_idx].astype(np.int32)
    byte, shift = nibble_index(np.arange(n_idx))
    return ((rows[..., byte].astype(np.int32) >> shift) & 0xF)


def pack_rows(codes: np.ndarray, row_bytes: int, bits: int) -> np.ndarray:
    """[..., n_idx] codes -> [..., row_bytes] uint8 (unused nibbles zero)."""
    if bits == 8:
        return codes.astype(np.uint8)
    out = np.zeros(codes.shape[:-1] + (row_bytes,), dtype=np.uint8)
    byte, shift = nibble_index(np.arange(codes.shape[-1]))
    for i in range(codes.shape[-1]):
        out[..., byte[i]] |= (codes[..., i].astype(np.uint8) & 0xF) << np.uint8(shift[i])
    return out


def test_nibble_order_is_the_documented_one():
    byte, shift = nibble_index(np.arange(64))
    assert byte[:16].tolist() == list(range(16)) and byte[16:32].tolist() == list(range(16)) and byte[32:48].tolist() == list(range(16, 32))
    assert shift[:16].tolist() == [0] * 16 and shift[16:32].tolist() == [4] * 16 and shift[32:48].tolist() == [0] * 16
    c = np.arange(48) % 16
    assert np.array_equal(unpack_rows(pack_rows(c[None], 32, 4), 48, 4)[0], c)
    assert pack_rows(c[None], 32, 4)[0, 16:].max() <= 0x0F          # a lone block of 16 indices keeps its high nibbles zero


class QCase:
    def __init__(self, seed, B, Hq, Hkv, r_k, r_v, seq_lens, reserve=2, shared_key_basis=False, bits=8):
        self.B, self.Hq, self.Hkv, self.r_k, self.r_v, self.bits = B, Hq, Hkv, r_k, r_v, bits
        self.krow, self.vrow = S.qkey_row_bytes(r_k, bits), (64 if bits == 8 else 32)
        self.seq_lens = np.asarray(seq_lens, dtype=np.int32)
        T = max(int(self.seq_lens.max()), 1)
        self.K = I.lowrank_keys(seed, 0, B, T, Hkv)
        self.V = I.gaussian_kv(seed, I.TAG_V, 0, B, T, Hkv)
        self.q = I.queries(seed, 0, B, Hq)
        self.U_k, self.U_v = I.stiefel_bases(seed, 0, Hkv, r_k, r_v, shared_key_basis=shared_key_basis)
        self.pg = I.make_paging(seed, self.seq_lens, reserve_tokens=reserve, extra_pages=1)
        Uk, Uv = U.f64(self.U_k), U.f64(self.U_v)
        Kf, Vf = U.f64(self.K), U.f64(self.V)
        # oracle side: fp32 projections, static key parameters calibrated per head on all rows of the batch
        self.Kd = [[Q.project_f32(Kf[b, :n, h], O.basis_of(Uk, h)) for h in range(Hkv)] for b, n in enumerate(self.seq_lens)]
        self.Vd = [[Q.project_f32(Vf[b, :n, h], O.basis_of(Uv, h)) for h in range(Hkv)] for b, n in enumerate(self.seq_lens)]
        kp = []
        for h in range(Hkv):
            allrows = np.concatenate([self.Kd[b][h] for b in range(B) if self.seq_lens[b] > 0], 0)
            s, z = Q.key_params_from_calibration(allrows * np.float32(1.25), bits)  # some headroom for appended rows
            kp.append(np.stack([s, z], -1))
        self.k_params = np.stack(kp).astype(np.float32)                              # [Hkv, ngk, 2]
        P = self.pg.num_pages
        fill = lambda shape, v, dt: torch.full(shape, v, dtype=dt, device=DEV)
        self.layer = S.QLayer(Hq, Hkv, r_k, r_v, self.U_k.to(DEV), self.U_v.to(DEV), torch.from_numpy(self.k_params).to(DEV),
                              fill((P, Hkv, 64, self.krow), 0xAB, torch.uint8), fill((P, Hkv, r_v, self.vrow), 0xCD, torch.uint8),
                              fill((P, Hkv, 64, S.qgroups(r_v), 2), float("nan"), torch.float32))
        bt = np.where(self.pg.block_table < 0, 0, self.pg.block_table).astype(np.int32)
        self.batch = S.Batch(torch.from_numpy(bt).to(DEV), torch.from_numpy(self.seq_lens.copy()).to(DEV))
        self.status = torch.zeros(1, dtype=torch.int32, device=DEV)

    def oracle_cache(self, b, h, extra_k=None, extra_v=None):
        Kd, Vd = self.Kd[b][h], self.Vd[b][h]
        if extra_k is not None:
            Kd, Vd = np.concatenate([Kd, extra_k], 0), np.concatenate([Vd, extra_v], 0)
        ks, kz = self.k_params[h, :, 0], self.k_params[h, :, 1]
        Kc = Q.quantize_keys(Kd, ks, kz, self.bits)
        Vc, vs, vz = Q.quantize_values(Vd, self.bits)
        return Kd, Vd, Kc, ks, kz, Vc, vs, vz

    def gather(self, t, b, n):
        """[n, Hkv, ...] rows of sequence b gathered from a token-major device pool through the block table."""
        p = t.cpu()
        idx = torch.arange(n)
        pages = torch.from_numpy(self.pg.block_table[b].astype(np.int64))[idx // 64]
        return p[pages, :, idx % 64]

    def gather_k(self, b, n):
        """[n, Hkv, r_k] key codes of sequence b."""
        return unpack_rows(self.gather(self.layer.k_codes, b, n).numpy(), self.r_k, self.bits)

    def gather_v(self, b, n):
        """[n, Hkv, r_v] value codes of sequence b: pages are [Hkv][r_v channels][64 positions]."""
        p = self.layer.v_codes.cpu().numpy()
        idx = np.arange(n)
        pages = self.pg.block_table[b].astype(np.int64)[idx // 64]
        rows = unpack_rows(p[pages], 64, self.bits)                     # [n, Hkv, r_v, 64 positions]
        return rows[np.arange(n), :, :, vpos(idx % 64)]


def _check_cache(c: QCase):
    mism = tot = 0
    for b in range(c.B):
        n = int(c.seq_lens[b])
        if n == 0:
            continue
        gk = c.gather_k(b, n)
        gv = c.gather_v(b, n)
        gp = c.gather(c.layer.v_params, b, n).numpy()
        for h in range(c.Hkv):
            Kd, Vd, Kc, ks, kz, Vc, vs, vz = c.oracle_cache(b, h)
            # keys: static parameters are inputs, so the codes may differ by one where the projection sits on a rounding edge
            assert np.abs(gk[:, h] - Kc).max() <= 1
            mism += int((gk[:, h] != Kc).sum()) + int((gv[:, h] != Vc).sum())
            tot += Kc.size + Vc.size
            # values: parameters from the row's own extremes (fp32 accumulation differences only)
            assert np.allclose(gp[:, h, :, 0], vs, rtol=2e-4, atol=1e-7) and np.allclose(gp[:, h, :, 1], vz, rtol=1e-4, atol=2e-5)
            deq_gpu = Q.dequant_values(gv[:, h], gp[:, h, :, 0], gp[:, h, :, 1])
            deq_ref = Q.dequant_values(Vc, vs, vz)
            step = np.repeat(vs, 64, axis=1)[:, :c.r_v]                         # per channel: its group's step
            assert np.all(np.abs(deq_gpu - deq_ref) <= 1.02 * step + 1e-5)
            assert np.all(np.abs(deq_gpu - Vd) <= 0.52 * step + 2e-5)           # and each is a valid rounding of its row
    assert mism <= max(4, 2e-3 * tot), f"{mism} of {tot} codes differ from the oracle's"


def _untouched(c: QCase):
    used = np.zeros((c.pg.num_pages, 64), dtype=bool)
    for b in range(c.B):
        for t in range(int(c.seq_lens[b])):
            used[c.pg.block_table[b, t // 64], t % 64] = True
    m = ~used[:, None, :].repeat(c.Hkv, 1)
    assert np.all(c.layer.k_codes.cpu().numpy()[m] == 0xAB)
    assert np.all(np.isnan(c.layer.v_params.cpu().numpy()[m]))
    used_pos = np.zeros_like(used)
    for pgi in range(used.shape[0]):
        used_pos[pgi, vpos(np.nonzero(used[pgi])[0])] = True
    vc = c.layer.v_codes.cpu().numpy()                                      # [P, Hkv, r_v, row bytes]
    if c.bits == 8:
        used_byte = used_pos
    else:                                                                   # a byte is shared by positions p and p + 16 of a block of 32
        up = used_pos.reshape(-1, 2, 2, 16)
        used_byte = (up[:, :, 0] | up[:, :, 1]).reshape(-1, 32)
    mv = ~used_byte[:, None, None, :].repeat(c.Hkv, 1).repeat(c.r_v, 2)
    assert np.all(vc[mv] == 0xCD)


def _oracle_out(c: QCase, q, caches):
    G = c.Hq // c.Hkv
    out = np.zeros((c.B, c.Hq, 128))
    lse = np.full((c.B, c.Hq), -np.inf)
    Uk, Uv = U.f64(c.U_k), U.f64(c.U_v)
    qf = U.f64(q)
    for b in range(c.B):
        for g in range(c.Hq):
            h = g // G
            _, _, Kc, ks, kz, Vc, vs, vz = caches[b][h]
            out[b, g], lse[b, g] = Q.attend_quantized_path_b(qf[b, g], Kc, ks, kz, Vc, vs, vz, O.basis_of(Uk, h), O.basis_of(Uv, h))
    return out, lse


def _workspace(c: QCase, parts):
    ws = torch.full((S.stief_decode_workspace_bytes(c.B, c.Hq, c.Hkv, c.r_v, parts) // 4,), float("nan"), dtype=torch.float32, device=DEV)
    S.stief_decode_workspace_init(ws)
    return ws


def _upload(c: QCase, caches):
    """The oracle's codes and parameters written into the device pools in the documented layout (host-side packing)."""
    P = c.pg.num_pages
    kcodes = np.zeros((P, c.Hkv, 64, c.r_k), dtype=np.int32)
    vcodes = np.zeros((P, c.Hkv, c.r_v, 64), dtype=np.int32)               # [.., channel, position]
    vp = c.layer.v_params.cpu().numpy()
    for b in range(c.B):
        for h in range(c.Hkv):
            _, _, Kc, ks, kz, Vc, vs, vz = caches[b][h]
            for t in range(Kc.shape[0]):
                pgi = int(c.pg.block_table[b, t // 64])
                kcodes[pgi, h, t % 64] = Kc[t]
                vcodes[pgi, h, :, int(vpos(t % 64))] = Vc[t]
                vp[pgi, h, t % 64, :, 0] = vs[t]
                vp[pgi, h, t % 64, :, 1] = vz[t]
    c.layer.k_codes.copy_(torch.from_numpy(pack_rows(kcodes, c.krow, c.bits)))
    c.layer.v_codes.copy_(torch.from_numpy(pack_rows(vcodes, c.vrow, c.bits)))
    c.layer.v_params.copy_(torch.from_numpy(vp))


RANK_PAIRS = [(64, 64), (128, 64), (64, 128), (128, 128), (32, 32), (48, 48), (96, 96), (32, 128), (96, 48), (48, 96)]
# output tolerances on the oracle's own codes: the arithmetic is the same for both widths
TIGHT = dict(max_abs=6e-3, rel_l2=3e-3)


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("r_k,r_v", RANK_PAIRS)
def test_quantising_prefill_matches_the_oracles_quantiser(r_k, r_v, bits):
    c = QCase(200 + r_k + r_v, 3, 8, 2, r_k, r_v, [200, 64, 129], bits=bits)
    S.stief_q_prefill_compress(bits, c.layer, c.batch, c.K.cuda(), c.V.cuda(), status=c.status)
    torch.cuda.synchronize()
    assert int(c.status.item()) == 0
    _check_cache(c)
    _untouched(c)


@pytest.mark.parametrize("bits", [8, 4])
@pytest.mark.parametrize("r_k,r_v", RANK_PAIRS)
def test_quantised_decode_on_the_oracles_own_codes_is_tight(r_k, r_v, bits):
    c = QCase(300 + r_k + r_v, 2, 8, 2, r_k, r_v, [333, 70], bits=bits)
    caches = [[c.oracle_cache(b, h) for h in range(c.Hkv)] for b in range(c.B)]
    _upload(c, caches)
    ref, ref_lse = _oracle_out(c, c.q, caches)
    for parts in (1, 3, 0):
        out = torch.full((c.B, c.Hq, 128), float("nan"), dtype=torch.bfloat16, device=DEV)
        lse = torch.full((c.B, c.Hq), float("nan"), dtype=torch.float32, device=DEV)
        S.stief_q_decode_attention(bits, c.layer, c.batch, c.q.cuda(), _workspace(c, parts), out, parts, lse, status=c.status)
        torch.cuda.synchronize()
        assert int(c.status.item()) == 0
        U.check_out(out, ref, **TIGHT)
        assert np.abs(lse.double().cpu().numpy() - ref_lse).max() < 2e-3


@pytest.mark.parametrize("bits,r_k,r_v", [(8, 64, 64), (4, 64, 64), (8, 48, 96), (4, 48, 96), (4, 128, 32), (8, 96, 128)])
def test_quantised_prefill_append_decode_end_to_end(bits, r_k, r_v):
    B, Hq, Hkv = 3, 16, 4
    c = QCase(400, B, Hq, Hkv, r_k, r_v, [700, 63, 128], reserve=4, bits=bits)
    S.stief_q_prefill_compress(bits, c.layer, c.batch, c.K.cuda(), c.V.cuda(), status=c.status)
    k_new, v_new = I.new_token_kv(400, 0, B, Hkv)
    S.stief_q_append(bits, c.layer, c.batch, k_new.cuda(), v_new.cuda(), status=c.status)
    ws = _workspace(c, 0)
    out = torch.full((B, Hq, 128), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV)
    S.stief_q_decode_attention(bits, c.layer, c.batch, c.q.cuda(), ws, out, 0, lse, len_add=1, status=c.status)
    torch.cuda.synchronize()
    assert int(c.status.item()) == 0
    Uk, Uv = U.f64(c.U_k), U.f64(c.U_v)
    kn, vn = U.f64(k_new), U.f64(v_new)
    caches = [[c.oracle_cache(b, h, Q.project_f32(kn[b, h][None], O.basis_of(Uk, h)), Q.project_f32(vn[b, h][None], O.basis_of(Uv, h)))
               for h in range(Hkv)] for b in range(B)]
    # the appended rows: codes within one of the oracle's, parameters from the row's extremes
    for b in range(B):
        n = int(c.seq_lens[b]) + 1
        gk = c.gather_k(b, n)
        gv = c.gather_v(b, n)
        gp = c.gather(c.layer.v_params, b, n).numpy()
        for h in range(Hkv):
            _, _, Kc, ks, kz, Vc, vs, vz = caches[b][h]
            assert np.abs(gk[-1, h] - Kc[-1]).max() <= 1 and np.abs(gv[-1, h] - Vc[-1]).max() <= 1
            # the rows before it are still what the prefill wrote (a 4-bit append replaces one nibble of shared bytes)
            assert np.abs(gk[:-1, h] - Kc[:-1]).max() <= 1 and np.abs(gv[:-1, h] - Vc[:-1]).max() <= 1
            assert np.allclose(gp[-1, h, :, 0], vs[-1], rtol=2e-4) and np.allclose(gp[-1, h, :, 1], vz[-1], rtol=1e-4, atol=2e-5)
    ref, ref_lse = _oracle_out(c, c.q, caches)
    ea, rl = U.check_out(out, ref)                          # the benchmark spec's tolerances, for both code widths
    el = np.abs(lse.double().cpu().numpy() - ref_lse).max()
    assert el < 5e-3
    print(f"{bits}-bit {r_k}/{r_v} end to end: max-abs {ea:.2e}, rel-L2 {rl:.2e}, lse {el:.2e}")


@pytest.mark.parametrize("bits,r_k,r_v", [(8, 64, 64), (8, 128, 128), (4, 64, 64), (4, 48, 96), (8, 96, 32), (4, 32, 48)])
def test_quantised_fused_step_equals_append_then_attention_also_with_overlapped_launches(bits, r_k, r_v):
    B, Hq, Hkv = 2, 8, 2
    cs = [QCase(600 + l, B, Hq, Hkv, r_k, r_v, [450, 127], reserve=4, bits=bits) for l in range(2)]
    for c in cs:
        S.stief_q_prefill_compress(bits, c.layer, c.batch, c.K.cuda(), c.V.cuda(), status=c.status)
    torch.cuda.synchronize()
    snap = [(c.layer.k_codes.clone(), c.layer.v_codes.clone(), c.layer.v_params.clone()) for c in cs]
    ws = _workspace(cs[0], 0)
    kvs = [tuple(t.cuda() for t in I.new_token_kv(600, l, B, Hkv)) for l in range(2)]
    res = {}
    for mode in ("separate", "fused", "fused_overlapped"):
        for c, (kc, vc, vp) in zip(cs, snap):
            c.layer.k_codes.copy_(kc); c.layer.v_codes.copy_(vc); c.layer.v_params.copy_(vp)
        outs = [torch.full((B, Hq, 128), float("nan"), dtype=torch.bfloat16, device=DEV) for _ in range(4)]
        for i in range(4):                               # layers alternate, so consecutive kernels touch different pools
            c, (kn, vn) = cs[i % 2], kvs[i % 2]
            if mode == "separate":
                S.stief_q_append(bits, c.layer, c.batch, kn, vn, status=c.status)
                S.stief_q_decode_attention(bits, c.layer, c.batch, c.q.cuda(), ws, outs[i], 0, len_add=1, status=c.status)
            else:
                S.stief_q_decode_step(bits, c.layer, c.batch, c.q.cuda(), kn, vn, ws, outs[i], status=c.status,
                                       flags=S.STIEF_DECODE_OVERLAP_PREVIOUS if (mode == "fused_overlapped" and i) else 0)
        torch.cuda.synchronize()
        assert all(int(c.status.item()) == 0 for c in cs)
        res[mode] = ([o.clone() for o in outs], [(c.layer.k_codes.clone(), c.layer.v_codes.clone(), c.layer.v_params.clone()) for c in cs])
    for mode in ("fused", "fused_overlapped"):
        for a, b in zip(res["separate"][0], res[mode][0]):
            U.check_out(a, b.double().cpu().numpy(), max_abs=4e-3 if bits == 8 else 1e-2, rel_l2=2e-3 if bits == 8 else 5e-3)   # projection order differs in the last bits
        c0 = cs[0]
        unp = lambda t, n: torch.from_numpy(unpack_rows(t.cpu().numpy(), n, bits))
        for (k0, v0, p0), (k1, v1, p1) in zip(res["separate"][1], res[mode][1]):
            assert (unp(k0, c0.r_k) - unp(k1, c0.r_k)).abs().max() <= 1 and (unp(v0, 64) - unp(v1, 64)).abs().max() <= 1
            m = ~torch.isnan(p0)
            assert torch.equal(torch.isnan(p0), torch.isnan(p1)) and torch.allclose(p0[m], p1[m], rtol=2e-4, atol=2e-5)
    for a, b in zip(res["fused"][0], res["fused_overlapped"][0]):
        assert torch.equal(a, b)


def test_quantised_path_rejects_unsupported_ranks_on_the_host():
    c = QCase(500, 1, 4, 1, 64, 64, [100])
    bad = S.QLayer(4, 1, 80, 64, c.layer.U_k, c.layer.U_v, c.layer.k_params, c.layer.k_codes, c.layer.v_codes, c.layer.v_params)
    out = torch.empty(1, 4, 128, dtype=torch.bfloat16, device=DEV)
    for bits in (8, 4):
        with pytest.raises(S.StiefError) as e:
            S.stief_q_decode_attention(bits, bad, c.batch, c.q.cuda(), _workspace(c, 0), out)
        assert e.value.code == S.STIEF_ERR_UNSUPPORTED


@pytest.mark.parametrize("bits", [8, 4])
def test_quantised_path_runs_the_per_layer_rank_profile_end_to_end(bits):
    # all 32 layers of the seeded rank profile (ranks drawn from 32/48/64/96/128): quantising prefill, then three fused
    # decode steps per layer with overlapped launches on one workspace; the last step's outputs of every layer, sequence
    # and head against the oracle on the oracle's own codes of the grown cache
    B, Hq, Hkv, n_steps = 2, 16, 4, 3
    prof = I.rank_profile(0)
    lens = [300, 1000]
    cs = [QCase(700 + l, B, Hq, Hkv, rk, rv, lens, reserve=n_steps + 1, bits=bits) for l, (rk, rv) in enumerate(prof)]
    for c in cs:
        S.stief_q_prefill_compress(bits, c.layer, c.batch, c.K.cuda(), c.V.cuda(), status=c.status)
    ws = torch.full((S.stief_decode_workspace_bytes(B, Hq, Hkv, 128, 0) // 4,), float("nan"), dtype=torch.float32, device=DEV)
    S.stief_decode_workspace_init(ws)
    lens_dev = cs[0].batch.seq_lens
    for c in cs:
        c.batch = S.Batch(c.batch.block_table, lens_dev)
    outs = [torch.full((B, Hq, 128), float("nan"), dtype=torch.bfloat16, device=DEV) for _ in cs]
    kv_hist = [[] for _ in cs]
    qs = None
    for step in range(n_steps):
        qs = [I.queries(700, l, B, Hq, step=step) for l in range(len(cs))]
        for l, c in enumerate(cs):
            kn, vn = I.new_token_kv(700, l, B, Hkv, step=step)
            kv_hist[l].append((kn, vn))
            S.stief_q_decode_step(bits, c.layer, c.batch, qs[l].cuda(), kn.cuda(), vn.cuda(), ws, outs[l], status=c.status,
                                  flags=S.STIEF_DECODE_OVERLAP_PREVIOUS if l else 0)
        S.stief_advance_seq_lens(lens_dev, 1)
    torch.cuda.synchronize()
    assert all(int(c.status.item()) == 0 for c in cs)
    worst = 0.0
    for l, c in enumerate(cs):
        Uk, Uv = U.f64(c.U_k), U.f64(c.U_v)
        caches = []
        for b in range(B):
            row = []
            for h in range(Hkv):
                ek = np.concatenate([Q.project_f32(U.f64(kn)[b, h][None], O.basis_of(Uk, h)) for kn, _ in kv_hist[l]], 0)
                ev = np.concatenate([Q.project_f32(U.f64(vn)[b, h][None], O.basis_of(Uv, h)) for _, vn in kv_hist[l]], 0)
                row.append(c.oracle_cache(b, h, ek, ev))
            caches.append(row)
        ref, _ = _oracle_out(c, qs[l], caches)
        ea, rl = U.check_out(outs[l], ref)
        worst = max(worst, rl)
    print(f"rank profile on the {bits}-bit cache: worst rel-L2 over 32 layers {worst:.2e}")
