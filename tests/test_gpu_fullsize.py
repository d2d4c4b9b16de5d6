"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration bench.py times
(one CTA per SM, overlapped launches where bench.py overlaps them).  The inputs are generated on the device by
the seeded generators; sampled (sequence, KV head) slices are copied back and pushed through the fp64 oracle:
for each sampled pair the WHOLE compressed cache of that pair is compared row by row (1 bf16 ulp, layout
bit-exact through the block table) and the outputs of all query heads of its group are compared with the
spec tolerances (max-abs 1e-2, relative L2 5e-3).  The first and the last page of every pair are
compared as well, so an indexing slip anywhere in the batch shows."""
import numpy as np
import pytest
import torch

import paper_2601_21686_b200 as S
from oracle import stief_oracle as O
from paper_2601_21686_b200 import inputs as I
from tests import _util as U

pytestmark = pytest.mark.gpu
DEV = "cuda"


class DevCase:
    """One layer's inputs on the device: K, V [B, Tmax, Hkv, 128], bases, paging, NaN-filled pools."""

    def __init__(self, seed, layer, B, Hq, Hkv, r_k, r_v, seq_lens, reserve=2, paging=None, lowrank=True):
        self.B, self.Hq, self.Hkv, self.r_k, self.r_v = B, Hq, Hkv, r_k, r_v
        self.seq_lens = np.asarray(seq_lens, dtype=np.int32)
        T = int(self.seq_lens.max())
        self.K = (I.lowrank_keys(seed, layer, B, T, Hkv, device=DEV) if lowrank
                  else I.gaussian_kv(seed, I.TAG_K, layer, B, T, Hkv, device=DEV))
        self.V = I.gaussian_kv(seed, I.TAG_V, layer, B, T, Hkv, device=DEV)
        self.U_k, self.U_v = I.stiefel_bases(seed, layer, Hkv, r_k, r_v)
        self.paging = paging or I.make_paging(seed, self.seq_lens, reserve_tokens=reserve, extra_pages=1)
        nanpool = lambda r: torch.full((self.paging.num_pages, Hkv, 64, r), U.NAN_BITS, dtype=torch.int16, device=DEV).view(torch.bfloat16)
        self.layer = S.Layer(Hq, Hkv, r_k, r_v, self.U_k.to(DEV), self.U_v.to(DEV), nanpool(r_k), nanpool(r_v))
        bt = np.where(self.paging.block_table < 0, 0, self.paging.block_table).astype(np.int32)
        self.batch = S.Batch(torch.from_numpy(bt).to(DEV), torch.from_numpy(self.seq_lens.copy()).to(DEV))
        self.status = torch.zeros(1, dtype=torch.int32, device=DEV)

    def rows(self, pool, b, h, t0, t1):
        """Cache rows [t0, t1) of (b, h) gathered on the device through the block table -> cpu bf16 [n, r]."""
        t = torch.arange(t0, t1, device=DEV)
        pages = torch.from_numpy(self.paging.block_table[b].astype(np.int64)).to(DEV)[t // 64]
        return pool[pages, h, t % 64, :].cpu()


def check_pair(c: DevCase, b, h, q, out, new_kv=None, lens=None):
    """Whole cache of (b, h) and the outputs of its query group against the oracle.  new_kv = (k_new, v_new)
    device tensors [B, Hkv, 128] appended after the prefilled rows (a list of such pairs for several steps)."""
    n = int((c.seq_lens if lens is None else lens)[b])
    Kh = c.K[b, :int(c.seq_lens[b]), h].double().cpu().numpy()
    Vh = c.V[b, :int(c.seq_lens[b]), h].double().cpu().numpy()
    for kn, vn in (new_kv or []):
        Kh = np.concatenate([Kh, kn[b, h].double().cpu().numpy()[None]], 0)
        Vh = np.concatenate([Vh, vn[b, h].double().cpu().numpy()[None]], 0)
    assert Kh.shape[0] == n
    Uk, Uv = O.basis_of(U.f64(c.U_k), h), O.basis_of(U.f64(c.U_v), h)
    Kd, Vd = O.compress(Kh, Uk), O.compress(Vh, Uv)
    sk, _ = U.check_cache(c.rows(c.layer.k_pool, b, h, 0, n), Kh, Uk, Kd)
    sv, _ = U.check_cache(c.rows(c.layer.v_pool, b, h, 0, n), Vh, Uv, Vd)
    assert sk + sv <= max(2, 1e-3 * n * (c.r_k + c.r_v))
    G = c.Hq // c.Hkv
    qf = q.double().cpu().numpy()
    ref = np.stack([O.attend_path_b(qf[b, g], Kd, Vd, Uk, Uv)[0] for g in range(h * G, (h + 1) * G)])
    U.check_out(out[b, h * G:(h + 1) * G], ref)


def check_edge_pages(c: DevCase, lens=None):
    """First and last page of every (b, h): rounded projection of the matching input rows (prefilled rows only)."""
    lens = c.seq_lens if lens is None else lens
    for b in range(c.B):
        n = int(min(lens[b], c.seq_lens[b]))
        if n == 0:
            continue
        for t0, t1 in {(0, min(64, n)), ((n - 1) // 64 * 64, n)}:
            for h in range(c.Hkv):
                Kh = c.K[b, t0:t1, h].double().cpu().numpy()
                Uk = O.basis_of(U.f64(c.U_k), h)
                U.check_cache(c.rows(c.layer.k_pool, b, h, t0, t1), Kh, Uk, O.compress(Kh, Uk))


def decode_full(c: DevCase, q, k_new=None, v_new=None, flags=0, ws=None):
    ws = ws if ws is not None else workspace(c)
    out = torch.full((c.B, c.Hq, 128), float("nan"), dtype=torch.bfloat16, device=DEV)
    if k_new is None:
        S.stief_decode_attention(c.layer, c.batch, q, ws, 0, out, status=c.status, flags=flags)
    else:
        S.stief_decode_step(c.layer, c.batch, q, k_new, v_new, ws, out, status=c.status, flags=flags)
    return out


def workspace(c: DevCase, r_v=None):
    n = S.stief_decode_workspace_bytes(c.B, c.Hq, c.Hkv, r_v or c.r_v, 0)
    ws = torch.full((n // 4,), float("nan"), dtype=torch.float32, device=DEV)
    S.stief_decode_workspace_init(ws)
    return ws


def sync_ok(*cases):
    torch.cuda.synchronize()
    for c in cases:
        assert int(c.status.item()) == 0


def test_config2_llama3_8b_layer_decode():
    # B=4, Hq=32, Hkv=8, T=32768, r=64/64: prefill, then one decode step (append + attention) as bench.py runs it
    c = DevCase(0, 0, 4, 32, 8, 64, 64, [32768] * 4)
    S.stief_prefill_compress(c.layer, c.batch, c.K, c.V, status=c.status)
    q = I.queries(0, 0, 4, 32, scale=1.0 / np.sqrt(128.0), device=DEV)
    kn, vn = I.new_token_kv(0, 0, 4, 8, device=DEV)
    out = decode_full(c, q, kn, vn)
    sync_ok(c)
    check_edge_pages(c)
    for b, h in ((0, 0), (3, 7), (1, 4)):
        check_pair(c, b, h, q, out, new_kv=[(kn, vn)], lens=c.seq_lens + 1)


def test_config4a_single_long_sequence():
    # B=1, T=131072, r_k=48, r_v=64: 8 (sequence, head) pairs split over all SMs
    c = DevCase(1, 0, 1, 32, 8, 48, 64, [131072])
    S.stief_prefill_compress(c.layer, c.batch, c.K, c.V, status=c.status)
    q = I.queries(1, 0, 1, 32, scale=1.0 / np.sqrt(128.0), device=DEV)
    out = decode_full(c, q)
    sync_ok(c)
    check_edge_pages(c)
    for b, h in ((0, 0), (0, 5)):
        check_pair(c, b, h, q, out)


def test_config4b_ragged_batch():
    # B=16, lengths uniform in [1024, 16384], 64-token pages, r=64/64
    lens = I.ragged_lengths(2, 16)
    c = DevCase(2, 0, 16, 32, 8, 64, 64, lens)
    S.stief_prefill_compress(c.layer, c.batch, c.K, c.V, status=c.status)
    q = I.queries(2, 0, 16, 32, scale=1.0 / np.sqrt(128.0), device=DEV)
    kn, vn = I.new_token_kv(2, 0, 16, 8, device=DEV)
    out = decode_full(c, q, kn, vn)
    sync_ok(c)
    check_edge_pages(c)
    order = np.argsort(lens)
    for b, h in ((int(order[0]), 1), (int(order[-1]), 6), (int(order[8]), 3)):   # shortest, longest, a middle one
        check_pair(c, b, h, q, out, new_kv=[(kn, vn)], lens=lens + 1)


def test_config5_prefill_layers_then_first_decode():
    # B=2, T=32768, per-layer ranks from the seeded profile: overlapped per-layer prefill launches, then the first
    # decode step of every layer with overlapped launches (four layers of the 32 are enough to mix ranks)
    prof = I.rank_profile(0)
    picks = [0, 2, 5, 31]
    pg = I.make_paging(5, [32768] * 2, reserve_tokens=2, extra_pages=1)
    cs = [DevCase(5, l, 2, 32, 8, prof[l][0], prof[l][1], [32768] * 2, paging=pg) for l in picks]
    for i, c in enumerate(cs):
        S.stief_prefill_compress(c.layer, c.batch, c.K, c.V, status=c.status,
                                 flags=S.STIEF_PREFILL_OVERLAP_PREVIOUS if i else 0)
    ws = workspace(cs[0], r_v=128)
    qs = [I.queries(5, l, 2, 32, scale=1.0 / np.sqrt(128.0), device=DEV) for l in picks]
    kvs = [I.new_token_kv(5, l, 2, 8, device=DEV) for l in picks]
    outs = [decode_full(c, q, kn, vn, flags=S.STIEF_DECODE_OVERLAP_PREVIOUS if i else 0, ws=ws)
            for i, (c, q, (kn, vn)) in enumerate(zip(cs, qs, kvs))]
    sync_ok(*cs)
    for c, q, kv, out in zip(cs, qs, kvs, outs):
        check_edge_pages(c)
        check_pair(c, 1, 3, q, out, new_kv=[kv], lens=c.seq_lens + 1)


def test_config3_steps_with_per_layer_ranks():
    # the 32-layer decode loop of config 3 on three of its layers and three steps at full T: each step appends one
    # token per layer and attends; layers after the first of a step are launched overlapped, as bench.py does
    prof = I.rank_profile(0)
    picks = [1, 7, 20]
    pg = I.make_paging(3, [32768] * 4, reserve_tokens=8, extra_pages=1)
    cs = [DevCase(3, l, 4, 32, 8, prof[l][0], prof[l][1], [32768] * 4, paging=pg) for l in picks]
    for c in cs:
        S.stief_prefill_compress(c.layer, c.batch, c.K, c.V, status=c.status)
    # one seq_lens tensor shared by all layers, advanced on the device after every step
    lens_dev = cs[0].batch.seq_lens
    for c in cs:
        c.batch = S.Batch(c.batch.block_table, lens_dev)
    ws = workspace(cs[0], r_v=128)
    hist = [[] for _ in cs]
    n_steps = 3
    for step in range(n_steps):
        outs, qs = [], []
        for i, (c, l) in enumerate(zip(cs, picks)):
            q = I.queries(3, l, 4, 32, scale=1.0 / np.sqrt(128.0), device=DEV, step=step)
            kn, vn = I.new_token_kv(3, l, 4, 8, device=DEV, step=step)
            hist[i].append((kn, vn))
            qs.append(q)
            outs.append(decode_full(c, q, kn, vn, flags=S.STIEF_DECODE_OVERLAP_PREVIOUS if i else 0, ws=ws))
        S.stief_advance_seq_lens(lens_dev, 1)
    sync_ok(*cs)
    assert np.array_equal(lens_dev.cpu().numpy(), np.full(4, 32768 + n_steps, dtype=np.int32))
    for i, c in enumerate(cs):              # last step's outputs against the oracle on the grown cache
        check_pair(c, 2, 5, qs[i], outs[i], new_kv=hist[i], lens=c.seq_lens + n_steps)


def _mq_sample_check(c: DevCase, q, out, lse, n_q, samples):
    """Sampled rows (b, query token i, query head g) of a multi-query call against the oracle's single-row definition
    on the cache rows the GPU holds: row i sits at position seq_len - n_q + i and attends positions 0 .. that."""
    G = c.Hq // c.Hkv
    worst = 0.0
    cache = {}
    for b, i, g in samples:
        h = g // G
        if (b, h) not in cache:
            n = int(c.seq_lens[b])
            cache[(b, h)] = (c.rows(c.layer.k_pool, b, h, 0, n).double().numpy(), c.rows(c.layer.v_pool, b, h, 0, n).double().numpy())
        Kd, Vd = cache[(b, h)]
        p = int(c.seq_lens[b]) - n_q + i
        ref, ref_lse = O.attend_path_b(q[b, i, g].double().cpu().numpy(), Kd[:p + 1], Vd[:p + 1],
                                       O.basis_of(U.f64(c.U_k), h), O.basis_of(U.f64(c.U_v), h))
        got = out[b, i, g].double().cpu().numpy()
        assert np.all(np.isfinite(got))
        err = np.abs(got - ref).max()
        rl = np.linalg.norm(got - ref) / np.linalg.norm(ref)
        assert err <= max(1e-2, 2.0 ** -7 * np.abs(ref).max()) and rl <= 5e-3, (b, i, g, err, rl)
        if lse is not None:
            assert abs(float(lse[b, i, g]) - ref_lse) < 2e-2 + 2.0 ** -8 * abs(ref_lse), (b, i, g)
        worst = max(worst, rl)
    return worst


@pytest.mark.parametrize("r_k,r_v", [(64, 64), (128, 128)])
def test_mq_chunk_at_bench_size(r_k, r_v):
    # the `bench.py --mq` workload: a 2048-token chunk at the end of the 32768-token config-2 cache; every CTA works
    # through about 14 units, which the small cases never do
    B, Hq, Hkv, T, n_q = 4, 32, 8, 32768, 2048
    c = DevCase(21, 0, B, Hq, Hkv, r_k, r_v, [T] * B, reserve=1)
    S.stief_prefill_compress(c.layer, c.batch, c.K, c.V, status=c.status)
    del c.K, c.V
    q = I.normal_bf16(I.stream_key(21, I.TAG_Q, 100), (B, n_q, Hq, 128), device=DEV)
    out = torch.full((B, n_q, Hq, 128), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, n_q, Hq), float("nan"), dtype=torch.float32, device=DEV)
    for _ in range(2):                                   # twice: the second launch finds every barrier phase advanced
        S.stief_mq_attention(c.layer, c.batch, q, out, out_lse=lse, status=c.status)
    torch.cuda.synchronize()
    assert int(c.status.item()) == 0
    assert not torch.isnan(out).any() and not torch.isnan(lse).any()
    idx = I.randint(I.stream_key(21, I.TAG_PERM, 7), 3 * 40, 0, 2 ** 20)
    samples = [(int(idx[3 * k]) % B, int(idx[3 * k + 1]) % n_q, int(idx[3 * k + 2]) % Hq) for k in range(40)]
    samples += [(0, 0, 0), (B - 1, n_q - 1, Hq - 1), (1, 63, 5), (2, 64, 9), (3, 1023, 31), (0, 1024, 16)]   # tile and unit edges
    _mq_sample_check(c, q, out, lse, n_q, samples)


def test_mq_few_rows_at_bench_size_split_ranges():
    # the speculative-decode shape of `bench.py --mq --n-q 8`: page ranges cut as the library proposes, merged by the
    # combine kernel; every row is checked
    B, Hq, Hkv, T, n_q = 4, 32, 8, 32768, 8
    c = DevCase(22, 0, B, Hq, Hkv, 64, 64, [T] * B, reserve=1)
    S.stief_prefill_compress(c.layer, c.batch, c.K, c.V, status=c.status)
    del c.K, c.V
    q = I.normal_bf16(I.stream_key(22, I.TAG_Q, 100), (B, n_q, Hq, 128), device=DEV)
    n_split = S.stief_mq_num_splits(B, n_q, Hq, Hkv, c.batch.block_table.shape[1])
    assert n_split > 1
    ws = torch.full((S.stief_mq_workspace_bytes(B, n_q, Hq, 64, n_split) // 4,), float("nan"), dtype=torch.float32, device=DEV)
    out = torch.full((B, n_q, Hq, 128), float("nan"), dtype=torch.bfloat16, device=DEV)
    lse = torch.full((B, n_q, Hq), float("nan"), dtype=torch.float32, device=DEV)
    S.stief_mq_attention(c.layer, c.batch, q, out, out_lse=lse, status=c.status, workspace=ws, num_splits=n_split)
    torch.cuda.synchronize()
    assert int(c.status.item()) == 0 and not torch.isnan(out).any()
    samples = [(b, i, g) for b in (0, 3) for i in range(n_q) for g in (0, 13, 31)]
    _mq_sample_check(c, q, out, lse, n_q, samples)
