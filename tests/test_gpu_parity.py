"""GPU parity: the CUDA path (through the C-ABI library) against the fp64 CPU oracle, element by element,
on the same seeded inputs.  Tolerances: cache layout/indexing bit-exact; cache values within 1 bf16 ulp of
the oracle's rounded projection (or a correct rounding inside the fp32 accumulation bound); attention outputs
max-abs <= 1e-2 and relative-L2 <= 5e-3."""
import math

import numpy as np
import pytest
import torch

import paper_2601_21686_b200 as S
from oracle import stief_oracle as O
from paper_2601_21686_b200 import inputs as I
from tests import _util as U

pytestmark = pytest.mark.gpu

RANKS = (32, 48, 64, 96, 128)


def _sync_status(c):
    torch.cuda.synchronize()
    return int(c.status.item())


def _prefill_and_check(c: U.Case):
    S.stief_prefill_compress(c.layer, c.batch, c.K.cuda(), c.V.cuda(), status=c.status)
    assert _sync_status(c) == 0
    Kd, Vd = U.oracle_cache(c)
    Kf, Vf = U.f64(c.K), U.f64(c.V)
    Uk, Uv = U.f64(c.U_k), U.f64(c.U_v)
    second = 0
    for b in range(c.B):
        n = int(c.seq_lens[b])
        if n == 0:
            continue
        gk = U.gpu_cache_rows(c, c.layer.k_pool, b, n)
        gv = U.gpu_cache_rows(c, c.layer.v_pool, b, n)
        for h in range(c.Hkv):
            s1, _ = U.check_cache(gk[:, h], Kf[b, :n, h], O.basis_of(Uk, h), Kd[b][:, h])
            s2, _ = U.check_cache(gv[:, h], Vf[b, :n, h], O.basis_of(Uv, h), Vd[b][:, h])
            second += s1 + s2
    total = sum(int(n) for n in c.seq_lens) * c.Hkv * (c.r_k + c.r_v)
    assert second <= max(2, 1e-3 * total), f"{second} of {total} cache elements needed the accumulation-bound clause"
    return Kd, Vd


def _untouched_rows_still_nan(c: U.Case):
    """Layout check from the other side: everything the prefill was not asked to write still holds the NaN fill."""
    used = np.zeros((c.paging.num_pages, 64), dtype=bool)
    for b in range(c.B):
        for t in range(int(c.seq_lens[b])):
            used[c.paging.block_table[b, t // 64], t % 64] = True
    for pool in (c.layer.k_pool, c.layer.v_pool):
        pb = U.bits(pool.cpu())                                   # [pages, Hkv, 64, r]
        untouched = pb[~used[:, None, :].repeat(c.Hkv, 1)]
        assert np.all(untouched == U.NAN_BITS)
        assert not np.any(pb[used[:, None, :].repeat(c.Hkv, 1)] == U.NAN_BITS)


def _decode(c: U.Case, num_splits, len_add=0, q=None):
    ws = U.workspace_for(c, num_splits)
    out = torch.full((c.B, c.Hq, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((c.B, c.Hq), float("nan"), dtype=torch.float32, device="cuda")
    S.stief_decode_attention(c.layer, c.batch, (c.q if q is None else q).cuda(), ws, num_splits, out, lse, len_add=len_add,
                             status=c.status)
    assert _sync_status(c) == 0
    return out, lse


def test_config1_prefill_then_decode():
    # B=1, Hq=4, Hkv=1, T=512, r=64/64, seed 0
    c = U.make_case(0, 1, 4, 1, 64, 64, [512])
    Kd, Vd = _prefill_and_check(c)
    _untouched_rows_still_nan(c)
    ref, ref_lse = U.oracle_decode(c, Kd, Vd)
    for ns in (1, 2, 8, 0):
        out, lse = _decode(c, ns)
        U.check_out(out, ref)
        assert np.abs(lse.double().cpu().numpy() - ref_lse).max() < 2e-3


@pytest.mark.parametrize("r_k", RANKS)
@pytest.mark.parametrize("r_v", RANKS)
def test_every_rank_pair_ragged(r_k, r_v):
    c = U.make_case(100 + r_k + 7 * r_v, 3, 8, 2, r_k, r_v, [200, 64, 129])
    Kd, Vd = _prefill_and_check(c)
    ref, ref_lse = U.oracle_decode(c, Kd, Vd)
    for ns in (1, 3):
        out, lse = _decode(c, ns)
        U.check_out(out, ref)
        assert np.abs(lse.double().cpu().numpy() - ref_lse).max() < 2e-3


def test_decode_on_the_oracles_own_cache_is_tight():
    # same cache bits on both sides: what is left is fp32 accumulation, the two-word bf16 operands and the
    # bf16 rounding of the output (2^-9 relative per element)
    c = U.make_case(5, 2, 8, 2, 64, 96, [700, 333], lowrank=True)
    Kd, Vd = U.oracle_cache(c)
    U.upload_cache(c, Kd, Vd)
    ref, ref_lse = U.oracle_decode(c, Kd, Vd)
    for ns in (1, 4, 11):
        out, lse = _decode(c, ns)
        ea, rl = U.check_out(out, ref, max_abs=4e-3, rel_l2=2.5e-3)
        assert np.abs(lse.double().cpu().numpy() - ref_lse).max() < 2e-4


def test_sharp_softmax_large_scores():
    # queries 8x larger: scores of magnitude ~10, one or two tokens dominate
    c = U.make_case(6, 1, 4, 1, 64, 64, [1000], lowrank=True, q_scale=8.0)
    Kd, Vd = _prefill_and_check(c)
    ref, ref_lse = U.oracle_decode(c, Kd, Vd)
    out, lse = _decode(c, 5)
    U.check_out(out, ref)
    assert np.abs(lse.double().cpu().numpy() - ref_lse).max() < 5e-3


@pytest.mark.parametrize("lens", [[1], [63], [64], [65], [0, 5], [128, 0, 1, 640]])
def test_edge_lengths(lens):
    c = U.make_case(7 + len(lens) + lens[0], len(lens), 4, 1, 48, 64, lens)
    Kd, Vd = _prefill_and_check(c)
    _untouched_rows_still_nan(c)
    ref, ref_lse = U.oracle_decode(c, Kd, Vd)
    out, lse = _decode(c, 2)
    U.check_out(out, ref)
    g = lse.cpu().numpy()
    for b, n in enumerate(lens):
        if n == 0:
            assert np.all(out[b].float().cpu().numpy() == 0) and np.all(np.isneginf(g[b]))
        else:
            assert np.abs(g[b] - ref_lse[b]).max() < 2e-3


@pytest.mark.parametrize("Hq,Hkv", [(4, 4), (6, 2), (16, 2), (32, 2), (8, 1)])
def test_group_sizes(Hq, Hkv):
    # G = 1 (MHA), 3, 8, 16 (two query tiles), 8 with a single KV head
    c = U.make_case(20 + Hq, 2, Hq, Hkv, 64, 32, [150, 90])
    Kd, Vd = _prefill_and_check(c)
    ref, _ = U.oracle_decode(c, Kd, Vd)
    out, _ = _decode(c, 2)
    U.check_out(out, ref)


def test_shared_key_basis_and_full_rank_sides():
    # one key basis per layer shared by all heads (head stride 0)
    c = U.make_case(30, 2, 8, 2, 64, 64, [100, 260], shared_key_basis=True)
    Kd, Vd = _prefill_and_check(c)
    ref, _ = U.oracle_decode(c, Kd, Vd)
    U.check_out(_decode(c, 3)[0], ref)
    # keys kept full rank (no basis), values compressed; then the reverse; then nothing compressed
    for fk, fv, rk, rv in ((True, False, 128, 48), (False, True, 96, 128), (True, True, 128, 128)):
        c = U.make_case(31, 2, 8, 2, rk, rv, [100, 260], full_rank_k=fk, full_rank_v=fv)
        Kd, Vd = _prefill_and_check(c)
        if fk:   # rows stored unprojected must be bit-identical to the input rows
            assert np.array_equal(U.bits(U.gpu_cache_rows(c, c.layer.k_pool, 1, 260)), U.bits(c.K[1, :260]))
        ref, _ = U.oracle_decode(c, Kd, Vd)
        U.check_out(_decode(c, 2)[0], ref)


def test_rank_128_with_orthogonal_basis_is_exact_attention():
    # r = d_h: compressed attention equals plain softmax attention on K, V (up to the bf16 cache rounding)
    c = U.make_case(32, 1, 4, 1, 128, 128, [300])
    _prefill_and_check(c)
    out, _ = _decode(c, 2)
    q, K, V = U.f64(c.q), U.f64(c.K), U.f64(c.V)
    ref, _ = O.decode_layer(q, [K[0, :300]], [V[0, :300]], None, None, "a")
    # U is orthogonal only to bf16 precision (|U^T U - I| ~ 1e-3), so this is looser than oracle parity
    U.check_out(out, ref, max_abs=3e-2, rel_l2=2e-2)


@pytest.mark.parametrize("num_parts", [0, 5])
def test_maximum_batch_of_tiny_sequences_fused_step(num_parts):
    # B = 1024 (the limit of one call) with lengths 0 .. 130, many of them 0, 63, 64, 65: every CTA walks dozens of
    # segments (its list of noted arrivals fills and is settled several times), empty sequences get their zero rows, and
    # the appended row lands on and beside page boundaries.  One KV head, two query heads.
    B, Hq, Hkv = 1024, 2, 1
    special = [0, 1, 63, 64, 65, 127, 128, 129]
    lens = [special[b % 8] if b % 3 else int(I.randint(I.stream_key(41, I.TAG_LENS), B, 0, 130)[b]) for b in range(B)]
    c = U.make_case(41, B, Hq, Hkv, 32, 48, lens, reserve=2)
    Kd, Vd = U.oracle_cache(c)
    S.stief_prefill_compress(c.layer, c.batch, c.K.cuda(), c.V.cuda(), status=c.status)
    k_new, v_new = I.new_token_kv(41, 0, B, Hkv)
    ws = U.workspace_for(c, num_parts)
    out = torch.full((B, Hq, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
    lse = torch.full((B, Hq), float("nan"), dtype=torch.float32, device="cuda")
    S.stief_decode_step(c.layer, c.batch, c.q.cuda(), k_new.cuda(), v_new.cuda(), ws, out, num_parts=num_parts, out_lse=lse,
                        status=c.status)
    assert _sync_status(c) == 0
    Uk, Uv = U.f64(c.U_k), U.f64(c.U_v)
    kn, vn = U.f64(k_new), U.f64(v_new)
    for b in range(B):
        Kd[b] = np.concatenate([Kd[b], O.compress(kn[b, 0][None], O.basis_of(Uk, 0))[None]], 0)
        Vd[b] = np.concatenate([Vd[b], O.compress(vn[b, 0][None], O.basis_of(Uv, 0))[None]], 0)
    ref, ref_lse = O.decode_layer(U.f64(c.q), Kd, Vd, Uk, Uv, "b")
    U.check_out(out, ref)
    assert np.abs(lse.double().cpu().numpy() - ref_lse).max() < 2e-3
    # B = 1025 is refused on the host
    big = S.Batch(torch.zeros(1025, 4, dtype=torch.int32, device="cuda"), torch.zeros(1025, dtype=torch.int32, device="cuda"))
    with pytest.raises(S.StiefError) as e:
        S.stief_decode_attention(c.layer, big, c.q.cuda(), ws, num_parts, out)
    assert e.value.code == S.STIEF_ERR_INVALID_ARG


def test_append_and_decode_step_across_a_page_boundary():
    B, Hq, Hkv = 2, 8, 2
    c = U.make_case(40, B, Hq, Hkv, 48, 96, [62, 127], reserve=8)
    Kd, Vd = _prefill_and_check(c)
    Uk, Uv = U.f64(c.U_k), U.f64(c.U_v)
    lens = c.seq_lens.copy()
    ws = U.workspace_for(c, 4)
    out = torch.empty(B, Hq, 128, dtype=torch.bfloat16, device="cuda")
    for step in range(5):
        k_new, v_new = I.new_token_kv(40, 0, B, Hkv, step=step)
        q = I.queries(40, 0, B, Hq, step=step + 1)
        if step % 2 == 0:      # fused step
            S.stief_decode_step(c.layer, c.batch, q.cuda(), k_new.cuda(), v_new.cuda(), ws, out, num_parts=4, status=c.status)
        else:                  # the same thing as separate calls
            S.stief_append(c.layer, c.batch, k_new.cuda(), v_new.cuda(), status=c.status)
            S.stief_decode_attention(c.layer, c.batch, q.cuda(), ws, 4, out, len_add=1, status=c.status)
        S.stief_advance_seq_lens(c.batch.seq_lens, 1)
        assert _sync_status(c) == 0
        kn, vn = U.f64(k_new), U.f64(v_new)
        for b in range(B):
            Kd[b] = np.concatenate([Kd[b], np.stack([O.compress(kn[b, h][None], O.basis_of(Uk, h))[0] for h in range(Hkv)])[None]], 0)
            Vd[b] = np.concatenate([Vd[b], np.stack([O.compress(vn[b, h][None], O.basis_of(Uv, h))[0] for h in range(Hkv)])[None]], 0)
        lens += 1
        assert np.array_equal(c.batch.seq_lens.cpu().numpy(), lens)
        # appended rows: 1 ulp; position: the row must be where the address formula says
        for b in range(B):
            n = int(lens[b])
            gk = U.gpu_cache_rows(c, c.layer.k_pool, b, n)
            gv = U.gpu_cache_rows(c, c.layer.v_pool, b, n)
            for h in range(Hkv):
                U.check_cache(gk[n - 1:, h], kn[b, h][None], O.basis_of(Uk, h), Kd[b][n - 1:, h])
                U.check_cache(gv[n - 1:, h], vn[b, h][None], O.basis_of(Uv, h), Vd[b][n - 1:, h])
        ref, _ = O.decode_layer(U.f64(q), Kd, Vd, Uk, Uv, "b")
        U.check_out(out, ref)


def test_split_count_invariance_and_span():
    c = U.make_case(50, 1, 8, 2, 64, 48, [2000])
    _prefill_and_check(c)
    outs = [_decode(c, ns)[0].float().cpu().numpy() for ns in (1, 2, 7, 32)]
    for o in outs[1:]:
        assert np.abs(o - outs[0]).max() < 4e-3
    # output lies in span(U_v) up to the bf16 rounding of out and of U_v
    Uv = U.f64(c.U_v)
    o = outs[0][0].astype(np.float64)
    for g in range(8):
        P = Uv[g // 4] @ Uv[g // 4].T
        assert np.linalg.norm(o[g] - o[g] @ P) <= 1e-2 * np.linalg.norm(o[g])


def test_separate_combine_call_matches_fused_call():
    c = U.make_case(51, 2, 8, 2, 64, 64, [500, 131])
    _prefill_and_check(c)
    ws = U.workspace_for(c, 6)
    out1 = torch.empty(2, 8, 128, dtype=torch.bfloat16, device="cuda")
    out2 = torch.empty_like(out1)
    S.stief_decode_attention(c.layer, c.batch, c.q.cuda(), ws, 6, out1, status=c.status)
    S.stief_decode_attention(c.layer, c.batch, c.q.cuda(), ws, 6, None, status=c.status)
    S.stief_split_combine(c.layer, c.batch, ws, 6, out2)
    assert _sync_status(c) == 0
    assert torch.equal(out1, out2)


def test_overlapped_launches_match_serial_ones():
    # decode steps of two layers enqueued back to back with STIEF_DECODE_OVERLAP_PREVIOUS, all sharing ONE
    # workspace: every kernel may start while its predecessor still runs, but must not touch the workspace
    # or its output before the predecessor is done.  Results must equal the serially launched ones bit for bit.
    B, Hq, Hkv = 3, 8, 2
    cs = [U.make_case(90, B, Hq, Hkv, 64, 64, [900, 300, 1500], reserve=8),
          U.make_case(91, B, Hq, Hkv, 64, 64, [900, 300, 1500], reserve=8)]
    for c in cs:
        _prefill_and_check(c)
    ws = U.workspace_for(cs[0], 0)
    n_steps = 8
    qs = [I.queries(90, 0, B, Hq, step=i).cuda() for i in range(n_steps)]
    # a layer that comes up again within one flagged run appends the same rows every time (which call's rows the pool
    # keeps is otherwise not defined); the queries differ from step to step
    kvs = [tuple(t.cuda() for t in I.new_token_kv(90, 0, B, Hkv, step=i % 2)) for i in range(n_steps)]
    pools0 = [(c.layer.k_pool.clone(), c.layer.v_pool.clone()) for c in cs]
    res = {}
    for flags in (0, S.STIEF_DECODE_OVERLAP_PREVIOUS):
        for c, (kp, vp) in zip(cs, pools0):
            c.layer.k_pool.copy_(kp)
            c.layer.v_pool.copy_(vp)
        torch.cuda.synchronize()
        outs = [torch.full((B, Hq, 128), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(n_steps)]
        for i in range(n_steps):
            c = cs[i % 2]
            S.stief_decode_step(c.layer, c.batch, qs[i], kvs[i][0], kvs[i][1], ws, outs[i], status=c.status, flags=flags)
        torch.cuda.synchronize()
        assert int(cs[0].status.item()) == 0 and int(cs[1].status.item()) == 0
        res[flags] = [o.clone() for o in outs]
    for a, b in zip(res[0], res[S.STIEF_DECODE_OVERLAP_PREVIOUS]):
        assert torch.equal(a, b)
    # and the last step against the oracle (step 7 appended the row that steps 1, 3, 5 had appended before it)
    c = cs[1]
    Kd, Vd = U.oracle_cache(c)
    Uk, Uv = U.f64(c.U_k), U.f64(c.U_v)
    kn, vn = U.f64(kvs[7][0]), U.f64(kvs[7][1])
    for b in range(B):
        Kd[b] = np.concatenate([Kd[b], np.stack([O.compress(kn[b, h][None], O.basis_of(Uk, h))[0] for h in range(Hkv)])[None]], 0)
        Vd[b] = np.concatenate([Vd[b], np.stack([O.compress(vn[b, h][None], O.basis_of(Uv, h))[0] for h in range(Hkv)])[None]], 0)
    ref, _ = O.decode_layer(U.f64(qs[7]), Kd, Vd, Uk, Uv, "b")
    U.check_out(res[1][7], ref)


@pytest.mark.parametrize("num_parts", [3, 16])
def test_flagged_chain_with_few_parts_over_two_caches_matches_serial(num_parts):
    # A grid below the SM count would let a THIRD kernel of a flagged chain start while the first still streams:
    # step i+2 works on the same cache as step i and rewrites the row step i appended.  The library serialises such
    # launches, so every step must see exactly its own appended row: bit-equal to the serial run, step by step.
    B, Hq, Hkv = 2, 8, 2
    cs = [U.make_case(92 + j, B, Hq, Hkv, 64, 64, [4000, 2500], reserve=8, lowrank=True) for j in range(2)]
    for c in cs:
        S.stief_prefill_compress(c.layer, c.batch, c.K.cuda(), c.V.cuda(), status=c.status)
    ws = U.workspace_for(cs[0], num_parts)
    n_steps = 12
    qs = [I.queries(92, 0, B, Hq, step=i).cuda() for i in range(n_steps)]
    # the new token's key is made large so that whichever appended row a step reads dominates its output
    kvs = [tuple((t * (8.0 if j == 0 else 1.0)).to(torch.bfloat16).cuda() for j, t in enumerate(I.new_token_kv(92, 0, B, Hkv, step=i)))
           for i in range(n_steps)]
    torch.cuda.synchronize()
    pools0 = [(c.layer.k_pool.clone(), c.layer.v_pool.clone()) for c in cs]
    res = {}
    for flags in (0, S.STIEF_DECODE_OVERLAP_PREVIOUS):
        for c, (kp, vp) in zip(cs, pools0):
            c.layer.k_pool.copy_(kp)
            c.layer.v_pool.copy_(vp)
        torch.cuda.synchronize()
        outs = [torch.full((B, Hq, 128), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(n_steps)]
        for i in range(n_steps):
            c = cs[i % 2]
            S.stief_decode_step(c.layer, c.batch, qs[i], kvs[i][0], kvs[i][1], ws, outs[i], num_parts=num_parts, status=c.status,
                                flags=flags)
        torch.cuda.synchronize()
        assert int(cs[0].status.item()) == 0 and int(cs[1].status.item()) == 0
        res[flags] = outs
    for i, (a, b) in enumerate(zip(res[0], res[S.STIEF_DECODE_OVERLAP_PREVIOUS])):
        assert torch.equal(a, b), f"step {i}"


def test_flagged_chains_when_the_library_cannot_know_the_workspace_history():
    # The overlap flag lets a kernel skip the wait for its predecessor when the library knows who used its workspace
    # section last; where it cannot know, it must fall back to waiting.  Here: a captured graph of an ODD number of
    # launches, all flagged (the first too), replayed several times, eager flagged launches in between (so the epochs
    # baked into the graph are stale), and launches made from another host thread (whose record of the workspace is
    # empty).  Every output must equal that of plain serial launches bit for bit.
    import threading
    B, Hq, Hkv = 3, 8, 2
    ranks = [(128, 128), (32, 32), (64, 96)]
    cs = [U.make_case(120 + l, B, Hq, Hkv, rk, rv, [2100, 700, 1300], reserve=8) for l, (rk, rv) in enumerate(ranks)]
    for c in cs:
        _prefill_and_check(c)
    ws = U.workspace_for(cs[0], 0)                       # sized for r_v = 128, the largest of the three
    ov = S.STIEF_DECODE_OVERLAP_PREVIOUS
    qs = [I.queries(120, l, B, Hq).cuda() for l in range(3)]
    kvs = [tuple(t.cuda() for t in I.new_token_kv(120, l, B, Hkv)) for l in range(3)]
    mk = lambda: [torch.full((B, Hq, 128), float("nan"), dtype=torch.bfloat16, device="cuda") for _ in range(3)]

    def step(outs, flags):
        for l, c in enumerate(cs):
            S.stief_decode_step(c.layer, c.batch, qs[l], kvs[l][0], kvs[l][1], ws, outs[l], status=c.status, flags=flags)

    ref = mk()
    step(ref, 0)
    torch.cuda.synchronize()
    g_out = mk()
    graph = torch.cuda.CUDAGraph()
    cap = torch.cuda.Stream()
    cap.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(cap):
        with torch.cuda.graph(graph, stream=cap):
            step(g_out, ov)
    torch.cuda.synchronize()
    for rep in range(3):
        for o in g_out:
            o.fill_(float("nan"))
        graph.replay()
        graph.replay()
        e_out = mk()
        step(e_out, ov)                                   # eager, flagged, right behind a replay
        t_out = mk()
        th = threading.Thread(target=step, args=(t_out, ov))   # same stream, another host thread
        th.start()
        th.join()
        graph.replay()
        torch.cuda.synchronize()
        assert all(int(c.status.item()) == 0 for c in cs)
        for l in range(3):
            assert torch.equal(g_out[l], ref[l]), f"replayed graph, round {rep}, layer {l}"
            assert torch.equal(e_out[l], ref[l]), f"eager launch after a replay, round {rep}, layer {l}"
            assert torch.equal(t_out[l], ref[l]), f"launch from another thread, round {rep}, layer {l}"


def test_flagged_chain_with_empty_sequences_and_wide_groups_matches_serial():
    # attention only (no append) over layers whose batches hold empty sequences (their units are zero-filled, which
    # also counts towards a kernel's finalised units), groups of 16 query heads per KV head (two units per pair) and a
    # batch that is empty altogether: the section bookkeeping must come out right for all of them, chained with the flag
    ov = S.STIEF_DECODE_OVERLAP_PREVIOUS
    specs = [(8, 2, 64, 64, [700, 0, 1300]), (32, 2, 128, 32, [0, 2500, 0]), (8, 2, 48, 96, [0, 0, 0]), (32, 2, 32, 128, [64, 1, 0])]
    cs = [U.make_case(130 + i, 3, Hq, Hkv, rk, rv, lens) for i, (Hq, Hkv, rk, rv, lens) in enumerate(specs)]
    for c in cs:
        _prefill_and_check(c)
    n_ws = max(S.stief_decode_workspace_bytes(3, c.Hq, c.Hkv, c.r_v, 0) for c in cs)
    ws = torch.full((n_ws // 4,), float("nan"), dtype=torch.float32, device="cuda")
    S.stief_decode_workspace_init(ws)
    order = [0, 1, 2, 3, 2, 1, 0, 3, 3, 2]
    res = {}
    for flags in (0, ov):
        outs = [torch.full((3, cs[l].Hq, 128), float("nan"), dtype=torch.bfloat16, device="cuda") for l in order]
        lses = [torch.full((3, cs[l].Hq), float("nan"), dtype=torch.float32, device="cuda") for l in order]
        for i, l in enumerate(order):
            c = cs[l]
            S.stief_decode_attention(c.layer, c.batch, c.q.cuda(), ws, 0, outs[i], out_lse=lses[i], status=c.status, flags=flags if i else 0)
        torch.cuda.synchronize()
        assert all(int(c.status.item()) == 0 for c in cs)
        res[flags] = (outs, lses)
    for i, l in enumerate(order):
        assert torch.equal(res[0][0][i], res[ov][0][i]) and torch.equal(res[0][1][i], res[ov][1][i]), f"launch {i} (layer {l})"
        empty = np.asarray(specs[l][4]) == 0
        o = res[ov][0][i].float().cpu().numpy()
        assert not np.isnan(o).any() and not o[empty].any()                   # zero rows for empty sequences
        assert np.isneginf(res[ov][1][i].cpu().numpy()[empty]).all()


def test_overlapped_prefill_launches_match_serial_ones():
    # the per-layer prefill launches of one prompt, enqueued back to back with STIEF_PREFILL_OVERLAP_PREVIOUS
    B, Hq, Hkv = 2, 8, 2
    ranks = [(64, 64), (32, 128), (96, 48), (128, 32)]
    cs = [U.make_case(95 + l, B, Hq, Hkv, rk, rv, [1000, 333]) for l, (rk, rv) in enumerate(ranks)]
    Kd = [c.K.cuda() for c in cs]
    Vd = [c.V.cuda() for c in cs]
    pools = {}
    for flags in (0, S.STIEF_PREFILL_OVERLAP_PREVIOUS):
        for c in cs:
            c.layer.k_pool.view(torch.int16).fill_(U.NAN_BITS)
            c.layer.v_pool.view(torch.int16).fill_(U.NAN_BITS)
        torch.cuda.synchronize()
        for c, K, V in zip(cs, Kd, Vd):
            S.stief_prefill_compress(c.layer, c.batch, K, V, status=c.status, flags=flags)
        torch.cuda.synchronize()
        assert all(int(c.status.item()) == 0 for c in cs)
        pools[flags] = [(c.layer.k_pool.clone(), c.layer.v_pool.clone()) for c in cs]
    for (k0, v0), (k1, v1) in zip(pools[0], pools[1]):
        assert torch.equal(k0.view(torch.int16), k1.view(torch.int16)) and torch.equal(v0.view(torch.int16), v1.view(torch.int16))
    for c in cs:                         # and the overlapped result against the oracle
        Kr, Vr = U.oracle_cache(c)
        for b in range(B):
            n = int(c.seq_lens[b])
            gk = U.gpu_cache_rows(c, c.layer.k_pool, b, n)
            for h in range(Hkv):
                U.check_cache(gk[:, h], U.f64(c.K)[b, :n, h], O.basis_of(U.f64(c.U_k), h), Kr[b][:, h])
        _untouched_rows_still_nan(c)


def test_host_staged_step():
    # host buffers pinned and mapped: the kernel reads and writes them directly; pageable buffers: staged copies
    B, Hq, Hkv = 2, 8, 2
    c = U.make_case(60, B, Hq, Hkv, 64, 64, [100, 70], reserve=4)
    Kd, Vd = _prefill_and_check(c)
    k_new, v_new = I.new_token_kv(60, 0, B, Hkv)
    staging = torch.empty(S.stief_host_staging_bytes(B, Hq, Hkv), dtype=torch.uint8, device="cuda")
    ws = U.workspace_for(c, 2)
    out_d = torch.empty(B, Hq, 128, dtype=torch.bfloat16, device="cuda")
    S.stief_decode_step(c.layer, c.batch, c.q.cuda(), k_new.cuda(), v_new.cuda(), ws, out_d, num_parts=2, status=c.status)
    assert _sync_status(c) == 0
    for pinned in (True, False):
        mk = (lambda t: t.clone().pin_memory()) if pinned else (lambda t: t.clone())
        q, kh, vh = mk(c.q), mk(k_new), mk(v_new)
        out_h = mk(torch.full((B, Hq, 128), float("nan"), dtype=torch.bfloat16))
        staging.fill_(0xFF)
        S.stief_decode_step_host(c.layer, c.batch, q, kh, vh, staging, ws, out_h, num_parts=2, status=c.status)
        assert _sync_status(c) == 0
        assert torch.equal(out_h, out_d.cpu())
        # the pinned route must not have touched the staging buffer, the pageable one must have
        assert bool((staging == 0xFF).all()) == pinned


def test_errors_are_reported_not_trapped():
    c = U.make_case(70, 1, 4, 1, 64, 64, [100])
    ws = U.workspace_for(c, 2)
    out = torch.empty(1, 4, 128, dtype=torch.bfloat16, device="cuda")
    # host-visible problems come back as return codes
    bad = S.Layer(4, 1, 40, 64, c.layer.U_k, c.layer.U_v, c.layer.k_pool, c.layer.v_pool)
    with pytest.raises(S.StiefError) as e:
        S.stief_decode_attention(bad, c.batch, c.q.cuda(), ws, 2, out)
    assert e.value.code == S.STIEF_ERR_UNSUPPORTED
    with pytest.raises(S.StiefError) as e:
        S.stief_decode_attention(c.layer, c.batch, c.q.cuda(), ws[:64], 2, out)
    assert e.value.code == S.STIEF_ERR_WORKSPACE
    with pytest.raises(S.StiefError) as e:
        S.stief_decode_attention(c.layer, c.batch, c.q.cuda().view(-1)[1:513], ws, 2, out)      # misaligned q
    assert e.value.code == S.STIEF_ERR_INVALID_ARG
    bad = S.Layer(5, 2, 64, 64, c.layer.U_k, c.layer.U_v, c.layer.k_pool, c.layer.v_pool)       # Hq % Hkv != 0
    with pytest.raises(S.StiefError) as e:
        S.stief_decode_attention(bad, c.batch, c.q.cuda(), ws, 2, out)
    assert e.value.code == S.STIEF_ERR_INVALID_ARG
    # a page id outside the pool: the kernels redirect the access, finish, and flag the status word
    S.stief_prefill_compress(c.layer, c.batch, c.K.cuda(), c.V.cuda(), status=c.status)
    bt = c.batch.block_table.clone()
    bt[0, 1] = c.paging.num_pages + 5
    badb = S.Batch(bt, c.batch.seq_lens)
    S.stief_decode_attention(c.layer, badb, c.q.cuda(), ws, 2, out, status=c.status)
    assert _sync_status(c) == S.STIEF_ERR_BOUNDS
    c.status.zero_()
    S.stief_prefill_compress(c.layer, badb, c.K.cuda(), c.V.cuda(), status=c.status)
    assert _sync_status(c) == S.STIEF_ERR_BOUNDS
    c.status.zero_()
    # a sequence longer than its block table
    long = S.Batch(c.batch.block_table, torch.tensor([64 * c.batch.block_table.shape[1] + 3], dtype=torch.int32, device="cuda"))
    S.stief_decode_attention(c.layer, long, c.q.cuda(), ws, 2, out, status=c.status)
    assert _sync_status(c) == S.STIEF_ERR_BOUNDS
    c.status.zero_()
    k_new, v_new = I.new_token_kv(70, 0, 1, 1)
    S.stief_append(c.layer, long, k_new.cuda(), v_new.cuda(), status=c.status)
    assert _sync_status(c) == S.STIEF_ERR_BOUNDS
    # and the context is still healthy
    c.status.zero_()
    S.stief_decode_attention(c.layer, c.batch, c.q.cuda(), ws, 2, out, status=c.status)
    assert _sync_status(c) == 0
