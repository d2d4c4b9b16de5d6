"""More GPU parity at the sizes and in the launch configurations bench.py times: the bf16 decode kernel with the rank
pairs NAMED (so that both page-lane layouts and both tile forms are reached on purpose), the 8-bit quantised path at the
config-2 shape with overlapped launches, and a scaled-down twin of the 32-layer decode loop (all layers, all 128 steps,
one captured graph replayed) compared in full."""
import numpy as np
import pytest
import torch

import paper_2601_21686_b200 as S
from oracle import stief_oracle as O
from oracle import stief_quant_oracle as Q
from paper_2601_21686_b200 import inputs as I
from tests import _util as U
from tests.test_gpu_fullsize import DEV, DevCase, check_edge_pages, check_pair, decode_full, sync_ok, workspace
from tests.test_gpu_quant import unpack_rows, vpos

pytestmark = pytest.mark.gpu


# 128/128, 128/96, 96/128: two page lanes x two warps (tiles above 24 KiB); 96/96, 32/32, 48/48, 32/128: four lanes x one warp;
# 64 and 128 use boxed tiles, 32 and 96 the linear forms, 48 the unswizzled bulk copy
@pytest.mark.parametrize("r_k,r_v", [(128, 128), (128, 96), (96, 128), (96, 96), (32, 32), (48, 48), (32, 128), (64, 48)])
def test_config2_shape_with_named_rank_pairs(r_k, r_v):
    c = DevCase(40 + r_k + 3 * r_v, 0, 4, 32, 8, r_k, r_v, [32768] * 4)
    S.stief_prefill_compress(c.layer, c.batch, c.K, c.V, status=c.status)
    q = I.queries(40, 0, 4, 32, scale=1.0 / np.sqrt(128.0), device=DEV)
    kn, vn = I.new_token_kv(40, 0, 4, 8, device=DEV)
    out = decode_full(c, q, kn, vn)
    sync_ok(c)
    check_edge_pages(c)
    for b, h in ((0, 7), (2, 3)):
        check_pair(c, b, h, q, out, new_kv=[(kn, vn)], lens=c.seq_lens + 1)


def test_overlapped_chain_of_long_and_short_kernels_matches_serial_launches():
    # Layers of very different ranks chained with the overlap flag on ONE workspace, as a 32-layer step does: a short
    # kernel (32/32) that follows a long one (128/128) has CTAs that are done long before the long kernel is, and they
    # leave without waiting for it, so three and more kernels are in flight and the workspace sections, the epochs in its
    # control words and the "last CTA waits" rule all get used.  Every step must equal the serial run bit for bit, and
    # sampled pairs the oracle.
    ranks = [(128, 128), (32, 32), (96, 128), (48, 32)]
    pg = I.make_paging(7, [32768] * 4, reserve_tokens=2, extra_pages=1)
    cs = [DevCase(70 + l, l, 4, 32, 8, rk, rv, [32768] * 4, paging=pg) for l, (rk, rv) in enumerate(ranks)]
    for i, c in enumerate(cs):
        S.stief_prefill_compress(c.layer, c.batch, c.K, c.V, status=c.status, flags=S.STIEF_PREFILL_OVERLAP_PREVIOUS if i else 0)
    sync_ok(*cs)
    ws = workspace(cs[0], r_v=128)
    n_steps = 14
    order = [0, 1, 2, 3, 1, 0, 3, 2, 0, 1, 1, 2, 0, 3]          # long -> short, short -> long, and a layer twice in a row
    qs = [I.queries(7, order[i], 4, 32, scale=1.0 / np.sqrt(128.0), device=DEV, step=i) for i in range(n_steps)]
    # a layer that comes up again within the run appends the same rows (else which rows the pool keeps is not defined)
    kvs = [I.new_token_kv(7, order[i], 4, 8, device=DEV, step=0) for i in range(n_steps)]
    res = {}
    for flags in (0, S.STIEF_DECODE_OVERLAP_PREVIOUS):
        outs = [torch.full((4, 32, 128), float("nan"), dtype=torch.bfloat16, device=DEV) for _ in range(n_steps)]
        lses = [torch.full((4, 32), float("nan"), dtype=torch.float32, device=DEV) for _ in range(n_steps)]
        for i in range(n_steps):
            c = cs[order[i]]
            S.stief_decode_step(c.layer, c.batch, qs[i], kvs[i][0], kvs[i][1], ws, outs[i], out_lse=lses[i], status=c.status,
                                flags=flags if i else 0)
        sync_ok(*cs)
        res[flags] = (outs, lses)
    for i in range(n_steps):
        assert torch.equal(res[0][0][i], res[1][0][i]), f"step {i}: outputs differ from the serial run"
        assert torch.equal(res[0][1][i], res[1][1][i]), f"step {i}: log-sum-exps differ from the serial run"
    # the workspace is clean for whoever comes next: 32 control words (four epochs, four unit counts that must be zero
    # again), then the arrival counters of the four sections (32 units each here), all zero
    ctrl = ws[:32 + 4 * 32].view(torch.int32).cpu().numpy()
    assert ctrl[:4].all() and not ctrl[4:].any()
    last_of = {l: max(i for i in range(n_steps) if order[i] == l) for l in range(len(cs))}
    for l, (b, h) in zip(range(len(cs)), ((0, 1), (1, 6), (2, 3), (3, 4))):
        i = last_of[l]                                            # every step of a layer rewrites the same appended row
        check_pair(cs[l], b, h, qs[i], res[1][0][i], new_kv=[kvs[i]], lens=cs[l].seq_lens + 1)


class QDevCase:
    """One layer of the quantised cache at full size: inputs generated on the device, static key parameters calibrated
    on the host (oracle arithmetic) from sequence 0 only, so rows of the other sequences also meet the clamp."""

    def __init__(self, seed, layer, B, Hq, Hkv, r_k, r_v, T, paging, bits=8):
        self.B, self.Hq, self.Hkv, self.r_k, self.r_v, self.T, self.bits = B, Hq, Hkv, r_k, r_v, T, bits
        self.K = I.lowrank_keys(seed, layer, B, T, Hkv, device=DEV)
        self.V = I.gaussian_kv(seed, I.TAG_V, layer, B, T, Hkv, device=DEV)
        self.U_k, self.U_v = I.stiefel_bases(seed, layer, Hkv, r_k, r_v)
        self.pg = paging
        Uk = U.f64(self.U_k)
        kp = []
        for h in range(Hkv):
            rows = Q.project_f32(self.K[0, :, h].double().cpu().numpy(), O.basis_of(Uk, h))
            s, z = Q.key_params_from_calibration(rows, bits)
            kp.append(np.stack([s, z], -1))
        self.k_params = np.stack(kp).astype(np.float32)
        P = paging.num_pages
        fill = lambda shape, v, dt: torch.full(shape, v, dtype=dt, device=DEV)
        self.layer = S.QLayer(Hq, Hkv, r_k, r_v, self.U_k.to(DEV), self.U_v.to(DEV), torch.from_numpy(self.k_params).to(DEV),
                              fill((P, Hkv, 64, S.qkey_row_bytes(r_k, bits)), 0xAB, torch.uint8),
                              fill((P, Hkv, r_v, 64 if bits == 8 else 32), 0xCD, torch.uint8),
                              fill((P, Hkv, 64, S.qgroups(r_v), 2), float("nan"), torch.float32))
        bt = np.where(paging.block_table < 0, 0, paging.block_table).astype(np.int32)
        self.batch = S.Batch(torch.from_numpy(bt).to(DEV), torch.from_numpy(paging.seq_lens.copy()).to(DEV))
        self.status = torch.zeros(1, dtype=torch.int32, device=DEV)

    def pair(self, b, h, n):
        """GPU codes and parameters of the first n tokens of (b, h): key codes [n, r_k], value codes [n, r_v], params [n, ng, 2]."""
        t = torch.arange(n, device=DEV)
        pages = torch.from_numpy(self.pg.block_table[b].astype(np.int64)).to(DEV)[t // 64]
        kc = unpack_rows(self.layer.k_codes[pages, h, t % 64, :].cpu().numpy(), self.r_k, self.bits)
        vrows = unpack_rows(self.layer.v_codes[pages, h].cpu().numpy(), 64, self.bits)          # [n, r_v, 64 positions]
        vc = vrows[np.arange(n), :, vpos(np.arange(n) % 64)]
        vp = self.layer.v_params[pages, h, t % 64].cpu().numpy()
        return kc, vc, vp


@pytest.mark.parametrize("bits,r_k,r_v", [(8, 64, 64), (8, 128, 128), (4, 64, 64), (4, 96, 48)])
def test_quantised_config2_shape_prefill_and_overlapped_steps(bits, r_k, r_v):
    # the `bench.py --q8` launch pattern: quantising prefill of two layer caches, then fused steps alternating over
    # them with overlapped launches on one workspace; every CTA's ring wraps many times (512 pages per (b, h))
    B, Hq, Hkv, T = 4, 32, 8, 32768
    pg = I.make_paging(60, [T] * B, reserve_tokens=2, extra_pages=1)
    cs = [QDevCase(60 + r_k, l, B, Hq, Hkv, r_k, r_v, T, pg, bits=bits) for l in range(2)]
    for i, c in enumerate(cs):
        S.stief_q_prefill_compress(bits, c.layer, c.batch, c.K, c.V, status=c.status, flags=S.STIEF_PREFILL_OVERLAP_PREVIOUS if i else 0)
    ws = torch.full((S.stief_decode_workspace_bytes(B, Hq, Hkv, r_v, 0) // 4,), float("nan"), dtype=torch.float32, device=DEV)
    S.stief_decode_workspace_init(ws)
    n_steps = 4
    qs = [I.queries(60, 0, B, Hq, scale=1.0 / np.sqrt(128.0), device=DEV, step=i) for i in range(n_steps)]
    # a layer cache that comes up again within the flagged run appends the same rows (the contract of the flag)
    kvs = [I.new_token_kv(60, 0, B, Hkv, device=DEV, step=i % 2) for i in range(n_steps)]
    outs = [torch.full((B, Hq, 128), float("nan"), dtype=torch.bfloat16, device=DEV) for _ in range(n_steps)]
    lses = [torch.full((B, Hq), float("nan"), dtype=torch.float32, device=DEV) for _ in range(n_steps)]
    for i in range(n_steps):
        c = cs[i % 2]
        S.stief_q_decode_step(bits, c.layer, c.batch, qs[i], kvs[i][0], kvs[i][1], ws, outs[i], out_lse=lses[i], status=c.status,
                               flags=S.STIEF_DECODE_OVERLAP_PREVIOUS if i else 0)
    torch.cuda.synchronize()
    assert all(int(c.status.item()) == 0 for c in cs)
    G = Hq // Hkv
    worst = dict(abs=0.0, rel=0.0, lse=0.0, codes=0.0)
    for step, (b, h) in ((2, (0, 0)), (3, (3, 5)), (3, (1, 2))):     # the last step of each layer cache (and one more pair)
        c = cs[step % 2]
        Uk, Uv = O.basis_of(U.f64(c.U_k), h), O.basis_of(U.f64(c.U_v), h)
        kn, vn = kvs[step]
        Kh = np.concatenate([c.K[b, :, h].double().cpu().numpy(), kn[b, h].double().cpu().numpy()[None]], 0)
        Vh = np.concatenate([c.V[b, :, h].double().cpu().numpy(), vn[b, h].double().cpu().numpy()[None]], 0)
        Kd, Vd = Q.project_f32(Kh, Uk), Q.project_f32(Vh, Uv)
        ks, kz = c.k_params[h, :, 0], c.k_params[h, :, 1]
        Kc = Q.quantize_keys(Kd, ks, kz, bits)
        Vc, vs, vz = Q.quantize_values(Vd, bits)
        gk, gv, gp = c.pair(b, h, T + 1)
        assert np.abs(gk - Kc).max() <= 1 and np.abs(gv - Vc).max() <= 1
        frac = (int((gk != Kc).sum()) + int((gv != Vc).sum())) / (Kc.size + Vc.size)
        assert frac <= 2e-3, f"{frac:.2e} of the codes differ from the oracle's"
        assert np.allclose(gp[:, :, 0], vs, rtol=2e-4, atol=1e-7) and np.allclose(gp[:, :, 1], vz, rtol=1e-4, atol=2e-5)
        qf = qs[step].double().cpu().numpy()
        ref = [Q.attend_quantized_path_b(qf[b, g], Kc, ks, kz, Vc, vs, vz, Uk, Uv) for g in range(h * G, (h + 1) * G)]
        ref_out = np.stack([r[0] for r in ref])
        ref_lse = np.array([r[1] for r in ref])
        ea, rl = U.check_out(outs[step][b, h * G:(h + 1) * G], ref_out)
        el = np.abs(lses[step][b, h * G:(h + 1) * G].double().cpu().numpy() - ref_lse).max()
        assert el < 5e-3
        worst = dict(abs=max(worst["abs"], ea), rel=max(worst["rel"], rl), lse=max(worst["lse"], el), codes=max(worst["codes"], frac))
    print(f"q{bits} {r_k}/{r_v} full size: worst max-abs {worst['abs']:.2e}, rel-L2 {worst['rel']:.2e}, lse {worst['lse']:.2e}, "
          f"share of differing codes {worst['codes']:.2e}")


def test_config3_twin_all_layers_all_steps_graph_replay():
    # The 32-layer decode loop of config 3 at T = 2048: every layer of the seeded rank profile, 128 steps, each step ONE
    # replay of a captured graph (32 fused append + attention launches, overlapped after the first, then the length
    # update), which is how bench.py --workload config3 launches it.  Compared in full: every row appended by every step
    # in every layer, and every output of the first and of the last step.
    B, Hq, Hkv, T, L, n_steps = 4, 32, 8, 2048, 32, 128
    prof = I.rank_profile(0)[:L]
    pg = I.make_paging(33, [T] * B, reserve_tokens=n_steps + 1, extra_pages=1)
    cs = [DevCase(33, l, B, Hq, Hkv, prof[l][0], prof[l][1], [T] * B, paging=pg) for l in range(L)]
    for c in cs:
        S.stief_prefill_compress(c.layer, c.batch, c.K, c.V, status=c.status)
    lens_dev = cs[0].batch.seq_lens
    for c in cs:
        c.batch = S.Batch(c.batch.block_table, lens_dev)
    status = cs[0].status
    ws = workspace(cs[0], r_v=128)
    # all steps' inputs, generated up front; the graph reads fixed buffers that are refilled before every replay
    q_all = torch.stack([torch.stack([I.queries(33, l, B, Hq, scale=1.0 / np.sqrt(128.0), device=DEV, step=s) for l in range(L)]) for s in range(n_steps)])
    kv = [[I.new_token_kv(33, l, B, Hkv, device=DEV, step=s) for l in range(L)] for s in range(n_steps)]
    k_all = torch.stack([torch.stack([kv[s][l][0] for l in range(L)]) for s in range(n_steps)])     # [steps, L, B, Hkv, 128]
    v_all = torch.stack([torch.stack([kv[s][l][1] for l in range(L)]) for s in range(n_steps)])
    q_buf, k_buf, v_buf = q_all[0].clone(), k_all[0].clone(), v_all[0].clone()
    out_buf = torch.full((L, B, Hq, 128), float("nan"), dtype=torch.bfloat16, device=DEV)
    ov = S.STIEF_DECODE_OVERLAP_PREVIOUS

    def decode_step():
        for l, c in enumerate(cs):
            S.stief_decode_step(c.layer, c.batch, q_buf[l], k_buf[l], v_buf[l], ws, out_buf[l], status=status, flags=ov if l else 0)
        S.stief_advance_seq_lens(lens_dev, 1)

    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    cap = torch.cuda.Stream()
    cap.wait_stream(torch.cuda.current_stream())
    snap = [(c.layer.k_pool.clone(), c.layer.v_pool.clone()) for c in cs]
    with torch.cuda.stream(cap):
        with torch.cuda.graph(graph, stream=cap):
            decode_step()
    torch.cuda.synchronize()
    # capturing does not run anything; put lengths and pools back anyway so the replays start from the prefilled state
    lens_dev.copy_(torch.from_numpy(pg.seq_lens).to(DEV))
    for c, (kp, vp) in zip(cs, snap):
        c.layer.k_pool.copy_(kp); c.layer.v_pool.copy_(vp)
    del snap
    first_out = None
    for s in range(n_steps):
        q_buf.copy_(q_all[s]); k_buf.copy_(k_all[s]); v_buf.copy_(v_all[s])
        graph.replay()
        if s == 0:
            first_out = out_buf.clone()
    torch.cuda.synchronize()
    assert int(status.item()) == 0
    assert np.array_equal(lens_dev.cpu().numpy(), np.full(B, T + n_steps, dtype=np.int32))
    last_out = out_buf
    worst = dict(abs=0.0, rel=0.0, second=0)
    qf_first, qf_last = q_all[0].double().cpu().numpy(), q_all[n_steps - 1].double().cpu().numpy()
    kf, vf = k_all.double().cpu().numpy(), v_all.double().cpu().numpy()
    G = Hq // Hkv
    for l, c in enumerate(cs):
        Ukf, Uvf = U.f64(c.U_k), U.f64(c.U_v)
        for b in range(B):
            for h in range(Hkv):
                Uk, Uv = O.basis_of(Ukf, h), O.basis_of(Uvf, h)
                Kh = np.concatenate([c.K[b, :, h].double().cpu().numpy(), kf[:, l, b, h]], 0)        # prompt rows, then one per step
                Vh = np.concatenate([c.V[b, :, h].double().cpu().numpy(), vf[:, l, b, h]], 0)
                Kd, Vd = O.compress(Kh, Uk), O.compress(Vh, Uv)
                n = T + n_steps
                sk, _ = U.check_cache(c.rows(c.layer.k_pool, b, h, 0, n), Kh, Uk, Kd)               # every row, appended ones included
                sv, _ = U.check_cache(c.rows(c.layer.v_pool, b, h, 0, n), Vh, Uv, Vd)
                worst["second"] += sk + sv
                for qf, out, m in ((qf_first, first_out, T + 1), (qf_last, last_out, n)):
                    ref = np.stack([O.attend_path_b(qf[l, b, g], Kd[:m], Vd[:m], Uk, Uv)[0] for g in range(h * G, (h + 1) * G)])
                    ea, rl = U.check_out(out[l, b, h * G:(h + 1) * G], ref)
                    worst["abs"], worst["rel"] = max(worst["abs"], ea), max(worst["rel"], rl)
    total = sum(B * Hkv * (T + n_steps) * (rk + rv) for rk, rv in prof)
    assert worst["second"] <= 1e-3 * total
    print(f"config-3 twin: worst max-abs {worst['abs']:.2e}, rel-L2 {worst['rel']:.2e}; {worst['second']} of {total} cache elements "
          "needed the accumulation-bound clause")
