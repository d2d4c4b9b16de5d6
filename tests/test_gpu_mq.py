"""Several causal query rows per head over the compressed cache (chunked prefill / speculative decode) against the
oracle's row-by-row definition (App. A.1, Eq. 18 per row), on the cache rows the GPU itself stored."""
import numpy as np
import pytest
import torch

import paper_2601_21686_b200 as S
from oracle import stief_oracle as O
from paper_2601_21686_b200 import inputs as I
from tests import _util as U

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _queries(seed, B, n_q, Hq, d=128, scale=1.0):
    return I.normal_bf16(I.stream_key(seed, I.TAG_Q, 77), (B, n_q, Hq, d), scale=scale)


def _run(c, q, q_lens=None, lse=True):
    B, n_q, Hq = q.shape[:3]
    d_out = 128 if c.U_v is not None else c.r_v
    out = torch.full((B, n_q, Hq, d_out), float("nan"), dtype=torch.bfloat16, device=DEV)
    out_lse = torch.full((B, n_q, Hq), float("nan"), dtype=torch.float32, device=DEV) if lse else None
    ql = None if q_lens is None else torch.tensor(q_lens, dtype=torch.int32, device=DEV)
    S.stief_mq_attention(c.layer, c.batch, q.to(DEV), out, q_lens=ql, out_lse=out_lse, status=c.status)
    torch.cuda.synchronize()
    return out, out_lse


def _reference(c, q, q_lens):
    """Oracle rows on the cache the GPU holds: returns (ref [B, n_q, Hq, d_out] with NaN where no row is due, lse)."""
    B, n_q, Hq = q.shape[:3]
    G = Hq // c.Hkv
    d_out = 128 if c.U_v is not None else c.r_v
    ref = np.full((B, n_q, Hq, d_out), np.nan)
    lse = np.full((B, n_q, Hq), np.nan)
    Uk, Uv = U.f64(c.U_k), U.f64(c.U_v)
    for b in range(B):
        n, ql = int(c.seq_lens[b]), int(q_lens[b])
        if ql == 0:
            continue
        Kd = U.f64(U.gpu_cache_rows(c, c.layer.k_pool, b, n))
        Vd = U.f64(U.gpu_cache_rows(c, c.layer.v_pool, b, n))
        for g in range(Hq):
            h = g // G
            o, l = O.attend_rows_causal(U.f64(q)[b, :ql, g], Kd[:, h], Vd[:, h], O.basis_of(Uk, h), O.basis_of(Uv, h), n - ql)
            ref[b, :ql, g], lse[b, :ql, g] = o, l
    return ref, lse


def _compare(out, out_lse, ref, lse):
    due = ~np.isnan(ref[..., 0])
    g = out.double().cpu().numpy()
    assert np.all(np.isnan(g[~due])), "rows beyond q_lens were written"
    # the absolute bound of the decode tests (1e-2) presumes outputs of order one; a bf16 output of magnitude x is
    # spaced 2^-8 x apart, so for peaked attention (outputs near single value rows, |x| up to 4) it scales with x
    bound = max(1e-2, 2.0 ** -7 * np.abs(ref[due]).max())
    ea, rl = U.check_out(out[torch.from_numpy(due)], ref[due], max_abs=bound)
    msg = f"multi-query parity: max-abs {ea:.2e} (bound {bound:.2e}; the decode bound is 1e-2), rel-L2 {rl:.2e} (bound 5e-3)"
    if out_lse is not None:
        gl = out_lse.double().cpu().numpy()
        # q' is rounded to bf16 (relative 2^-9 per element), so a score, and with it the LSE, carries an error of up to
        # about 2^-9 of its own magnitude on top of the fp32 arithmetic
        el, lb = np.abs(gl[due] - lse[due]).max(), 2e-2 + 2.0 ** -8 * np.abs(lse[due]).max()
        assert np.all(np.isnan(gl[~due])) and el < lb
        msg += f", lse {el:.2e} (bound {lb:.2e})"
    print(msg)                                              # the margin, visible with pytest -s


@pytest.mark.parametrize("r_k,r_v", [(64, 64), (128, 128), (32, 48), (96, 32), (48, 96), (64, 128), (128, 64)])
def test_chunk_of_queries_all_rank_pairs(r_k, r_v):
    c = U.make_case(900 + r_k + r_v, 2, 8, 2, r_k, r_v, [300, 200], lowrank=True)
    S.stief_prefill_compress(c.layer, c.batch, c.K.to(DEV), c.V.to(DEV), status=c.status)
    q = _queries(1, 2, 70, 8, scale=1.5)
    q_lens = [70, 33]
    out, out_lse = _run(c, q, q_lens)
    assert int(c.status.item()) == 0
    _compare(out, out_lse, *_reference(c, q, q_lens))


@pytest.mark.parametrize("Hq,Hkv", [(2, 2), (16, 2), (8, 1)])
def test_group_sizes(Hq, Hkv):
    c = U.make_case(77 + Hq, 2, Hq, Hkv, 64, 64, [257, 129])
    S.stief_prefill_compress(c.layer, c.batch, c.K.to(DEV), c.V.to(DEV), status=c.status)
    n_q = 150 if Hq == Hkv else 40
    q = _queries(2, 2, n_q, Hq)
    q_lens = [n_q, min(n_q, 129)]
    out, out_lse = _run(c, q, q_lens)
    assert int(c.status.item()) == 0
    _compare(out, out_lse, *_reference(c, q, q_lens))


def test_whole_prompt_as_queries_and_single_rows():
    # q_len = seq_len (plain causal prefill attention, first row sees one position); q_len = 1 (decode); q_len = 0
    c = U.make_case(5, 3, 8, 2, 64, 64, [130, 64, 90])
    S.stief_prefill_compress(c.layer, c.batch, c.K.to(DEV), c.V.to(DEV), status=c.status)
    q = _queries(3, 3, 130, 8)
    q_lens = [130, 1, 0]
    out, out_lse = _run(c, q, q_lens)
    assert int(c.status.item()) == 0
    ref, lse = _reference(c, q, q_lens)
    _compare(out, out_lse, ref, lse)
    # the single row of sequence 1 is what the decode kernel returns for the same query
    ws = U.workspace_for(c, 2)
    dq = torch.zeros(3, 8, 128, dtype=torch.bfloat16)
    dq[1] = q[1, 0]
    dout = torch.zeros(3, 8, 128, dtype=torch.bfloat16, device=DEV)
    S.stief_decode_attention(c.layer, c.batch, dq.to(DEV), ws, 2, dout, status=c.status)
    torch.cuda.synchronize()
    assert np.abs(dout[1].double().cpu().numpy() - out[1, 0].double().cpu().numpy()).max() < 1e-2


def test_growing_scores_force_the_accumulator_rescale():
    # keys aligned with the queries and growing with the position: every page raises the row maxima by far more than
    # the lazy-rescale threshold, so the TMEM accumulator is rescaled page after page
    B, Hq, Hkv, T, n_q = 1, 4, 1, 520, 40
    c = U.make_case(41, B, Hq, Hkv, 64, 64, [T])
    Uk = U.f64(c.U_k)[0]
    direction = Uk[:, 0] / np.linalg.norm(Uk[:, 0])                       # lies in the key basis: survives the projection
    ramp = np.linspace(0.0, 60.0, T)[:, None] * direction[None, :]
    K = torch.from_numpy(ramp + 0.05 * U.f64(c.K)[0, :, 0]).to(torch.bfloat16)[None, :, None, :]
    c.K = K.contiguous()
    S.stief_prefill_compress(c.layer, c.batch, c.K.to(DEV), c.V.to(DEV), status=c.status)
    q = torch.from_numpy(np.tile(12.0 * direction, (B, n_q, Hq, 1)) + 0.1 * U.f64(_queries(4, B, n_q, Hq))).to(torch.bfloat16)
    out, out_lse = _run(c, q, [n_q])
    assert int(c.status.item()) == 0
    ref, lse = _reference(c, q, [n_q])
    # the spread of scores is ~ 60 * 12 / sqrt(128) = 64 nats over the sequence: far beyond the threshold
    assert lse[0, -1, 0] - lse[0, 0, 0] > 1.0
    _compare(out, out_lse, ref, lse)


@pytest.mark.parametrize("fold_k,fold_v", [(True, True), (True, False), (False, True)])
def test_folded_sides(fold_k, fold_v):
    r_k, r_v, B, Hq, Hkv = 64, 96, 2, 8, 2
    c = U.make_case(123, B, Hq, Hkv, r_k, r_v, [200, 140])
    S.stief_prefill_compress(c.layer, c.batch, c.K.to(DEV), c.V.to(DEV), status=c.status)     # cache built with the bases
    q = _queries(6, B, 50, Hq)
    Uk = U.f64(c.U_k)
    G = Hq // Hkv
    q_in = q
    if fold_k:      # what a folded W_Q hands over: q' rounded to bf16
        qp = np.stack([np.stack([U.f64(q)[b, :, g] @ Uk[g // G] for g in range(Hq)], axis=1) for b in range(B)])
        q_in = torch.from_numpy(qp).to(torch.float32).to(torch.bfloat16)
        c.layer.U_k, c.U_k = None, None
    if fold_v:
        c.layer.U_v, c.U_v = None, None
    out, out_lse = _run(c, q_in, [50, 50])
    assert int(c.status.item()) == 0 and out.shape[-1] == (r_v if fold_v else 128)
    _compare(out, out_lse, *_reference(c, q_in, [50, 50]))


def test_strided_tensors_and_untouched_padding():
    c = U.make_case(9, 2, 8, 2, 64, 64, [190, 100])
    S.stief_prefill_compress(c.layer, c.batch, c.K.to(DEV), c.V.to(DEV), status=c.status)
    n_q = 37
    q = _queries(8, 2, n_q, 8)
    qbig = torch.zeros(2, n_q + 3, 8 * 128 + 64, dtype=torch.bfloat16, device=DEV)
    qv = torch.as_strided(qbig, (2, n_q, 8, 128), (qbig.stride(0), qbig.stride(1), 128, 1))
    qv.copy_(q.to(DEV))
    obig = torch.full((2, n_q + 1, 8 * 128 + 8), float("nan"), dtype=torch.bfloat16, device=DEV)
    ov = torch.as_strided(obig, (2, n_q, 8, 128), (obig.stride(0), obig.stride(1), 128, 1))
    S.stief_mq_attention(c.layer, c.batch, qv, ov, status=c.status)
    torch.cuda.synchronize()
    assert int(c.status.item()) == 0
    ref, _ = _reference(c, q, [n_q, n_q])
    U.check_out(ov.contiguous(), ref)
    assert torch.isnan(obig[:, n_q:]).all() and torch.isnan(obig[:, :, 8 * 128:]).all()


def test_more_queries_than_cached_tokens_is_reported():
    c = U.make_case(10, 2, 8, 2, 64, 64, [100, 20])
    S.stief_prefill_compress(c.layer, c.batch, c.K.to(DEV), c.V.to(DEV), status=c.status)
    q = _queries(9, 2, 40, 8)
    out, _ = _run(c, q, [40, 40], lse=False)
    assert int(c.status.item()) == S.STIEF_ERR_BOUNDS
    assert torch.isnan(out[1]).all() and not torch.isnan(out[0]).any()


def test_unsupported_group_size_and_bad_arguments():
    c = U.make_case(11, 1, 6, 2, 64, 64, [100])          # G = 3 does not divide 128
    q = _queries(10, 1, 8, 6)
    out = torch.zeros(1, 8, 6, 128, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(S.StiefError) as e:
        S.stief_mq_attention(c.layer, c.batch, q.to(DEV), out, status=c.status)
    assert e.value.code == S.STIEF_ERR_UNSUPPORTED
    c = U.make_case(12, 1, 8, 2, 64, 64, [100])
    q = _queries(10, 1, 8, 8)
    out = torch.zeros(1, 8, 8, 128, dtype=torch.bfloat16, device=DEV)
    with pytest.raises(S.StiefError) as e:
        S.stief_mq_attention(c.layer, c.batch, q.to(DEV), out, status=c.status, flags=4)
    assert e.value.code == S.STIEF_ERR_INVALID_ARG


def test_chunked_prefill_end_to_end():
    # A prompt processed in chunks of 96 tokens: every chunk is projected and stored behind the cache (stief_append_chunk),
    # then attends causally to everything cached so far (stief_mq_attention).  All rows together are plain causal
    # attention of the whole prompt; the cache must equal the oracle's projection of the whole prompt.
    B, Hq, Hkv, r_k, r_v, chunk = 2, 8, 2, 64, 96, 96
    final = np.array([300, 170], dtype=np.int32)
    c = U.make_case(321, B, Hq, Hkv, r_k, r_v, final, lowrank=True)
    T = int(final.max())
    q = _queries(12, B, T, Hq)
    c.batch.seq_lens.zero_()
    outs = torch.full((B, T, Hq, 128), float("nan"), dtype=torch.bfloat16, device=DEV)
    Kd, Vd, qd = c.K.to(DEV), c.V.to(DEV), q.to(DEV)
    done = np.zeros(B, dtype=np.int32)
    step = 0
    while (done < final).any():
        lens = np.minimum(chunk, final - done).astype(np.int32)
        lens_d = torch.from_numpy(lens).to(DEV)
        # gather each sequence's next rows into a [B, chunk] batch (rows beyond lens are never read into the cache)
        Kc = torch.zeros(B, chunk, Hkv, 128, dtype=torch.bfloat16, device=DEV)
        Vc, qc = torch.zeros_like(Kc), torch.zeros(B, chunk, Hq, 128, dtype=torch.bfloat16, device=DEV)
        for b in range(B):
            n = int(lens[b])
            Kc[b, :n], Vc[b, :n], qc[b, :n] = Kd[b, done[b]:done[b] + n], Vd[b, done[b]:done[b] + n], qd[b, done[b]:done[b] + n]
        oc = torch.full((B, chunk, Hq, 128), float("nan"), dtype=torch.bfloat16, device=DEV)
        if step % 2 == 0:      # both position conventions
            S.stief_append_chunk(c.layer, c.batch, Kc, Vc, chunk_lens=lens_d, status=c.status)
            c.batch.seq_lens += lens_d
        else:
            c.batch.seq_lens += lens_d
            S.stief_append_chunk(c.layer, c.batch, Kc, Vc, chunk_lens=lens_d, ends_at_len=True, status=c.status)
        S.stief_mq_attention(c.layer, c.batch, qc, oc, q_lens=lens_d, status=c.status)
        torch.cuda.synchronize()
        assert int(c.status.item()) == 0
        for b in range(B):
            n = int(lens[b])
            outs[b, done[b]:done[b] + n] = oc[b, :n]
            assert torch.isnan(oc[b, n:]).all()
        done += lens
        step += 1
    assert np.array_equal(c.batch.seq_lens.cpu().numpy(), final)
    Kd_o, Vd_o = U.oracle_cache(c)
    for b in range(B):
        n = int(final[b])
        gk, gv = U.gpu_cache_rows(c, c.layer.k_pool, b, n), U.gpu_cache_rows(c, c.layer.v_pool, b, n)
        for h in range(Hkv):
            U.check_cache(gk[:, h], U.f64(c.K)[b, :n, h], U.f64(c.U_k)[h], Kd_o[b][:, h])
            U.check_cache(gv[:, h], U.f64(c.V)[b, :n, h], U.f64(c.U_v)[h], Vd_o[b][:, h])
    ref, _ = _reference(c, q, final)
    _compare(outs, None, ref, None)


def test_chunk_rows_have_the_bits_of_single_token_append():
    c1 = U.make_case(55, 2, 4, 2, 48, 128, [70, 3], full_rank_v=True)
    c2 = U.make_case(55, 2, 4, 2, 48, 128, [70, 3], full_rank_v=True)
    n_new = 5
    Kn = I.gaussian_kv(8, I.TAG_K, 3, 2, n_new, 2)
    Vn = I.gaussian_kv(8, I.TAG_V, 3, 2, n_new, 2)
    S.stief_append_chunk(c1.layer, c1.batch, Kn.to(DEV), Vn.to(DEV), status=c1.status)
    for i in range(n_new):
        S.stief_append(c2.layer, c2.batch, Kn[:, i].contiguous().to(DEV), Vn[:, i].contiguous().to(DEV), status=c2.status)
        S.stief_advance_seq_lens(c2.batch.seq_lens, 1)
    torch.cuda.synchronize()
    assert int(c1.status.item()) == 0 and int(c2.status.item()) == 0
    assert torch.equal(c1.layer.k_pool.view(torch.int16), c2.layer.k_pool.view(torch.int16))
    assert torch.equal(c1.layer.v_pool.view(torch.int16), c2.layer.v_pool.view(torch.int16))
    # positions without a page are reported, not written
    c3 = U.make_case(56, 1, 4, 2, 64, 64, [60], reserve=2)
    big = I.gaussian_kv(9, I.TAG_K, 3, 1, 200, 2)
    S.stief_append_chunk(c3.layer, c3.batch, big.to(DEV), big.to(DEV), status=c3.status)
    torch.cuda.synchronize()
    assert int(c3.status.item()) == S.STIEF_ERR_BOUNDS


@pytest.mark.parametrize("num_splits", [2, 4, 13])
@pytest.mark.parametrize("fold_v", [False, True])
def test_split_page_ranges_for_few_query_rows(num_splits, fold_v):
    # speculative-decode shape: a handful of query tokens over a long cache, the page range cut into parts (13 parts
    # against 5 pages of the short sequence leaves some parts empty); masked-out parts of a row must drop out
    c = U.make_case(77, 2, 8, 2, 64, 48, [700, 300], lowrank=True)
    S.stief_prefill_compress(c.layer, c.batch, c.K.to(DEV), c.V.to(DEV), status=c.status)
    if fold_v:
        c.layer.U_v, c.U_v = None, None
    q = _queries(13, 2, 6, 8, scale=1.5)
    q_lens = [6, 3]
    d_out = 48 if fold_v else 128
    ws = torch.full((S.stief_mq_workspace_bytes(2, 6, 8, 48, num_splits) // 4,), float("nan"), dtype=torch.float32, device=DEV)
    out = torch.full((2, 6, 8, d_out), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((2, 6, 8), float("nan"), dtype=torch.float32, device=DEV)
    S.stief_mq_attention(c.layer, c.batch, q.to(DEV), out, q_lens=torch.tensor(q_lens, dtype=torch.int32, device=DEV),
                         out_lse=lse, status=c.status, workspace=ws, num_splits=num_splits)
    torch.cuda.synchronize()
    assert int(c.status.item()) == 0
    _compare(out, lse, *_reference(c, q, q_lens))
    one, _ = _run(c, q, q_lens)                                  # unsplit: same rows up to the rounding of the merge
    due = ~torch.isnan(one[..., 0])
    assert (out[due].float() - one[due].float()).abs().max() < 2e-2


def test_split_across_a_page_boundary_masks_whole_parts():
    # 8 query tokens ending at position 64*5 + 2: the first rows sit on page 4, the last on page 5, so the part that holds
    # only page 5 is entirely masked for the early rows
    c = U.make_case(78, 1, 4, 1, 64, 64, [64 * 5 + 3])
    S.stief_prefill_compress(c.layer, c.batch, c.K.to(DEV), c.V.to(DEV), status=c.status)
    q = _queries(14, 1, 8, 4)
    ws = torch.empty(S.stief_mq_workspace_bytes(1, 8, 4, 64, 6) // 4, dtype=torch.float32, device=DEV)
    out = torch.full((1, 8, 4, 128), float("nan"), dtype=torch.bfloat16, device=DEV)
    S.stief_mq_attention(c.layer, c.batch, q.to(DEV), out, status=c.status, workspace=ws, num_splits=6)
    torch.cuda.synchronize()
    assert int(c.status.item()) == 0
    ref, _ = _reference(c, q, [8])
    _compare(out, None, ref, None)


def test_split_planning_and_workspace_errors():
    assert S.stief_mq_num_splits(4, 2048, 32, 8, 513) == 1                      # a chunk fills the GPU by itself
    s = S.stief_mq_num_splits(4, 8, 32, 8, 513)
    assert 2 <= s <= 32 and 32 * s <= 148
    assert S.stief_mq_num_splits(1, 4, 32, 8, 8) <= 2                          # never more parts than a quarter of the pages
    assert S.stief_mq_workspace_bytes(4, 8, 32, 64, 1) == 0
    assert S.stief_mq_workspace_bytes(4, 8, 32, 64, 4) >= 4 * 8 * 32 * 2 * 4 * 66 * 4
    c = U.make_case(79, 1, 8, 2, 64, 64, [200])
    q = _queries(15, 1, 4, 8)
    out = torch.zeros(1, 4, 8, 128, dtype=torch.bfloat16, device=DEV)
    small = torch.empty(64, dtype=torch.float32, device=DEV)
    with pytest.raises(S.StiefError) as e:
        S.stief_mq_attention(c.layer, c.batch, q.to(DEV), out, status=c.status, workspace=small, num_splits=3)
    assert e.value.code == S.STIEF_ERR_WORKSPACE
    with pytest.raises(S.StiefError) as e:
        S.stief_mq_attention(c.layer, c.batch, q.to(DEV), out, status=c.status, num_splits=3)
    assert e.value.code == S.STIEF_ERR_INVALID_ARG


def test_shared_key_basis_and_wide_groups():
    # one key basis for all heads (the paper's head sharing: uk_head_stride = 0), and a group of 32 query heads per KV
    # head (a 128-row tile then holds 4 tokens)
    c = U.make_case(88, 2, 8, 2, 48, 64, [260, 131], shared_key_basis=True)
    assert c.U_k.shape[0] == 1
    S.stief_prefill_compress(c.layer, c.batch, c.K.to(DEV), c.V.to(DEV), status=c.status)
    q = _queries(21, 2, 45, 8)
    out, lse = _run(c, q, [45, 20])
    assert int(c.status.item()) == 0
    _compare(out, lse, *_reference(c, q, [45, 20]))
    c = U.make_case(89, 1, 32, 1, 64, 64, [200])
    S.stief_prefill_compress(c.layer, c.batch, c.K.to(DEV), c.V.to(DEV), status=c.status)
    q = _queries(22, 1, 11, 32)
    out, lse = _run(c, q, [11])
    assert int(c.status.item()) == 0
    _compare(out, lse, *_reference(c, q, [11]))


def test_split_ranges_with_two_row_tiles():
    # more than 128 rows per (sequence, KV head): both tiles have rows of their own, so parts are plain page ranges
    c = U.make_case(90, 2, 8, 2, 64, 64, [500, 260], lowrank=True)
    S.stief_prefill_compress(c.layer, c.batch, c.K.to(DEV), c.V.to(DEV), status=c.status)
    q = _queries(23, 2, 50, 8)
    q_lens = [50, 37]
    ws = torch.full((S.stief_mq_workspace_bytes(2, 50, 8, 64, 3) // 4,), float("nan"), dtype=torch.float32, device=DEV)
    out = torch.full((2, 50, 8, 128), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((2, 50, 8), float("nan"), dtype=torch.float32, device=DEV)
    S.stief_mq_attention(c.layer, c.batch, q.to(DEV), out, q_lens=torch.tensor(q_lens, dtype=torch.int32, device=DEV),
                         out_lse=lse, status=c.status, workspace=ws, num_splits=3)
    torch.cuda.synchronize()
    assert int(c.status.item()) == 0
    _compare(out, lse, *_reference(c, q, q_lens))
