"""Pins of the CPU oracle against things other than itself: library routines (torch SDPA, scipy
logsumexp), closed forms, invariants the method fixes, brute-force loops on tiny inputs, and the
one figure the paper prints (cache sizing).  CPU only."""
import math
import os

import numpy as np
import pytest
import torch
from scipy.special import logsumexp, softmax

from oracle import stief_oracle as O
from paper_2601_21686_b200 import inputs as I

D = 128


def _sdpa(q, K, V, Hkv):
    """Library attention in fp64: q [Hq,d], K/V [n,Hkv,d] -> [Hq,d] (default scale 1/sqrt(d))."""
    Hq = q.shape[0]
    G = Hq // Hkv
    qt = torch.from_numpy(q).reshape(1, Hq, 1, -1)
    kt = torch.from_numpy(K).permute(1, 0, 2).repeat_interleave(G, dim=0).unsqueeze(0)
    vt = torch.from_numpy(V).permute(1, 0, 2).repeat_interleave(G, dim=0).unsqueeze(0)
    return torch.nn.functional.scaled_dot_product_attention(qt, kt, vt).reshape(Hq, -1).numpy()


def _case(seed, n, Hq, Hkv, r_k, r_v, storage=True, bf16_U=True):
    K = I.gaussian_kv(seed, I.TAG_K, 0, 1, n, Hkv).double().numpy()
    V = I.gaussian_kv(seed, I.TAG_V, 0, 1, n, Hkv).double().numpy()
    q = I.queries(seed, 0, 1, Hq).double().numpy()
    if bf16_U:
        uk, uv = I.stiefel_bases(seed, 0, Hkv, r_k, r_v)
        uk, uv = uk.double().numpy(), uv.double().numpy()
    else:
        uk = np.stack([I.stiefel_basis_f64(seed, I.TAG_UK, 0, h, r_k) for h in range(Hkv)])
        uv = np.stack([I.stiefel_basis_f64(seed, I.TAG_UV, 0, h, r_v) for h in range(Hkv)])
    Kd = [np.stack([O.compress(K[0, :, h], uk[h], storage) for h in range(Hkv)], 1)]
    Vd = [np.stack([O.compress(V[0, :, h], uv[h], storage) for h in range(Hkv)], 1)]
    return q, K, V, uk, uv, Kd, Vd


# ---------------------------------------------------------------- bf16 rounding

def test_rnd_bf16_matches_torch_on_fp32_inputs():
    # For inputs that are exactly fp32 numbers there is no double rounding, so torch's fp32->bf16
    # conversion (round to nearest even) is an independent implementation of the same map.
    g = torch.Generator().manual_seed(1)
    x = torch.randn(200000, generator=g) * torch.exp(torch.randn(200000, generator=g) * 8)
    x = torch.cat([x, torch.tensor([0.0, -0.0, 1.0, 1.00390625, 1.01171875, 3.3895e38, 1e-40, -1e-39, 2.0 ** -133, 2.0 ** -134])])
    ref = x.to(torch.bfloat16).double().numpy()
    got = O.rnd_bf16(x.double().numpy())
    assert np.array_equal(ref, got)


def test_rnd_bf16_ties_to_even_and_single_rounding():
    # halfway between 1 and 1+2^-7 -> even mantissa (1.0); between 1+2^-7 and 1+2^-6 -> 1+2^-6
    assert O.rnd_bf16(np.array([1 + 2.0 ** -8]))[0] == 1.0
    assert O.rnd_bf16(np.array([1 + 2.0 ** -7 + 2.0 ** -8]))[0] == 1 + 2.0 ** -6
    # just above a tie by less than fp32 resolution must round up (a route through fp32 would tie down)
    assert O.rnd_bf16(np.array([1 + 2.0 ** -8 + 2.0 ** -40]))[0] == 1 + 2.0 ** -7
    b = O.bf16_bits(np.array([1.0, -2.0, 0.0]))
    assert list(b) == [0x3F80, 0xC000, 0x0000]
    assert np.array_equal(O.bf16_from_bits(b), [1.0, -2.0, 0.0])
    assert list(O.bf16_ordinal(np.array([0x0000, 0x0001, 0x8001, 0x3F80, 0x3F81], dtype=np.uint16))) == [0, 1, -1, 0x3F80, 0x3F81]


def test_bf16_ulp_against_fixed_spacings():
    # bf16 keeps 8 significant bits: numbers in [2^(e-1), 2^e) are 2^(e-8) apart.  The values below are
    # written out by hand from that rule, not computed by the function under test.
    cases = {1.0: 2.0 ** -7, 1.5: 2.0 ** -7, 1.9921875: 2.0 ** -7, 2.0: 2.0 ** -6, 0.75: 2.0 ** -8, 0.5: 2.0 ** -8,
             0.49999: 2.0 ** -9, 3.0: 2.0 ** -6, 100.0: 2.0 ** -1, 255.0: 1.0, 256.0: 2.0, 1e-6: 2.0 ** -27,
             2.0 ** -126: 2.0 ** -133,            # smallest normal
             2.0 ** -130: 2.0 ** -133,            # subnormal range keeps the last normal spacing
             2.0 ** -133: 2.0 ** -133, 0.0: 2.0 ** -133}
    for x, want in cases.items():
        assert O.bf16_ulp(np.array([x]))[0] == want, x
        assert O.bf16_ulp(np.array([-x]))[0] == want, -x            # the spacing does not depend on the sign
    # the spacing is what separates neighbouring bit patterns: bits -> value, next pattern -> value, difference
    pat = np.array([0x3F80, 0x3F00, 0x4000, 0x0080, 0x0001, 0x42C8, 0x7F00], dtype=np.uint16)
    gap = O.bf16_from_bits(pat + np.uint16(1)) - O.bf16_from_bits(pat)
    assert np.array_equal(O.bf16_ulp(O.bf16_from_bits(pat)), gap)
    # and torch's own bf16 neighbours agree (nextafter on the bf16 grid), on random magnitudes
    g = torch.Generator().manual_seed(7)
    x = (torch.randn(4096, generator=g) * torch.exp(torch.randn(4096, generator=g) * 6)).to(torch.bfloat16)
    up = torch.nextafter(x.abs(), torch.full_like(x, float("inf")))
    assert np.array_equal(O.bf16_ulp(x.double().numpy()), (up.double() - x.abs().double()).numpy())


# ---------------------------------------------------------------- bases

@pytest.mark.parametrize("r", [32, 48, 64, 96, 128])
def test_basis_is_on_the_stiefel_manifold(r):
    U = I.stiefel_basis_f64(3, I.TAG_UK, 1, 2, r)
    assert U.shape == (D, r)
    assert np.abs(U.T @ U - np.eye(r)).max() < 1e-12
    Ub = torch.from_numpy(U).to(torch.float32).to(torch.bfloat16).double().numpy()
    assert np.abs(Ub.T @ Ub - np.eye(r)).max() < 1e-2


def test_truncation_nests():
    # Eq. 6: a rank-r basis is the leading r columns of the full one
    U128 = I.stiefel_basis_f64(5, I.TAG_UV, 0, 0, 128)
    U48 = I.stiefel_basis_f64(5, I.TAG_UV, 0, 0, 48)
    assert np.array_equal(U128[:, :48], U48)
    # and it equals the Q factor of the first 48 columns of the same Gaussian
    a = I.normal_f64(I.stream_key(5, I.TAG_UV, 0, 0, 0), D * D).numpy().reshape(D, D)
    q, r = np.linalg.qr(a[:, :48])
    q = q * np.sign(np.diag(r))[None, :]
    assert np.abs(q - U48).max() < 1e-10


# ---------------------------------------------------------------- projection (Eq. 1, Eq. 2)

def test_compress_bruteforce_tiny():
    rng = np.random.default_rng(0)
    X = rng.standard_normal((5, 6))
    U = rng.standard_normal((6, 3))
    ref = np.zeros((5, 3))
    for t in range(5):
        for j in range(3):
            acc = 0.0
            for c in range(6):
                acc += X[t, c] * U[c, j]
            ref[t, j] = acc
    assert np.abs(O.compress(X, U, storage=False) - ref).max() < 1e-14


def test_rows_inside_the_span_survive_exactly():
    # K = C U^T lies in span(U): K U = C and K U U^T = K
    U = I.stiefel_basis_f64(7, I.TAG_UK, 0, 0, 48)
    C = np.random.default_rng(1).standard_normal((33, 48))
    K = C @ U.T
    Kd = O.compress(K, U, storage=False)
    assert np.abs(Kd - C).max() < 1e-12
    assert np.abs(O.reconstruct(Kd, U) - K).max() < 1e-12


def test_identity_basis_keeps_rows_bit_for_bit():
    K = I.gaussian_kv(2, I.TAG_K, 0, 1, 40, 1).double().numpy()[0, :, 0]
    assert np.array_equal(O.compress(K, np.eye(D)), K)
    assert np.array_equal(O.compress(K, None), K)


def test_reconstruction_is_the_orthogonal_projector():
    # K_tilde = K P P^T: idempotent, symmetric, and K - K_tilde is orthogonal to span(P)
    U = I.stiefel_basis_f64(8, I.TAG_UK, 0, 0, 64)
    K = np.random.default_rng(2).standard_normal((20, D))
    Kt = O.reconstruct(O.compress(K, U, storage=False), U)
    Ktt = O.reconstruct(O.compress(Kt, U, storage=False), U)
    assert np.abs(Kt - Ktt).max() < 1e-12
    assert np.abs((K - Kt) @ U).max() < 1e-12


# ---------------------------------------------------------------- attention (Eq. 18)

def test_attention_bruteforce_tiny_d4():
    # toy head dimension 4, rank 2, n = 5: explicit loops on the reconstructed tensors
    rng = np.random.default_rng(3)
    d, r, n = 4, 2, 5
    U, _ = np.linalg.qr(rng.standard_normal((d, r)))
    W, _ = np.linalg.qr(rng.standard_normal((d, r)))
    K, V, q = rng.standard_normal((n, d)), rng.standard_normal((n, d)), rng.standard_normal(d)
    Kd, Vd = O.compress(K, U, False), O.compress(V, W, False)
    Kt = [[sum(sum(K[t, c] * U[c, j] for c in range(d)) * U[e, j] for j in range(r)) for e in range(d)] for t in range(n)]
    Vt = [[sum(sum(V[t, c] * W[c, j] for c in range(d)) * W[e, j] for j in range(r)) for e in range(d)] for t in range(n)]
    s = [sum(q[e] * Kt[t][e] for e in range(d)) / math.sqrt(d) for t in range(n)]
    z = sum(math.exp(x) for x in s)
    ref = [sum(math.exp(s[t]) / z * Vt[t][e] for t in range(n)) for e in range(d)]
    for fn in (O.attend_path_a, O.attend_path_b):
        out, lse = fn(q, Kd, Vd, U, W, d_h=d)
        assert np.abs(out - np.array(ref)).max() < 1e-13
        assert abs(lse - math.log(z)) < 1e-13


@pytest.mark.parametrize("r_k,r_v", [(64, 64), (32, 96), (48, 64), (128, 32)])
def test_compressed_attention_is_full_attention_on_reconstructed_kv(r_k, r_v):
    # library SDPA on explicitly formed K U U^T, V U U^T; its default scale is 1/sqrt(128) because the
    # tensors it sees have the original head dimension -> pins the scale at r < d_h
    Hq, Hkv, n = 8, 2, 77
    q, K, V, uk, uv, Kd, Vd = _case(11, n, Hq, Hkv, r_k, r_v, storage=False, bf16_U=False)
    Kt = np.stack([K[0, :, h] @ uk[h] @ uk[h].T for h in range(Hkv)], 1)
    Vt = np.stack([V[0, :, h] @ uv[h] @ uv[h].T for h in range(Hkv)], 1)
    ref = _sdpa(q[0], Kt, Vt, Hkv)
    for path in ("a", "b"):
        out, _ = O.decode_layer(q, Kd, Vd, uk, uv, path)
        assert np.abs(out[0] - ref).max() < 1e-12


def test_full_rank_equals_exact_attention():
    # r = d_h with an orthogonal basis: zero error (the full-rank pair of Algorithm 2 has Delta = 0)
    Hq, Hkv, n = 4, 1, 130
    q, K, V, uk, uv, Kd, Vd = _case(12, n, Hq, Hkv, 128, 128, storage=False, bf16_U=False)
    ref = _sdpa(q[0], K[0], V[0], Hkv)
    for path in ("a", "b"):
        out, lse = O.decode_layer(q, Kd, Vd, uk, uv, path)
        assert np.abs(out[0] - ref).max() < 1e-12
    s = (K[0, :, 0] @ q[0, 1]) / math.sqrt(D)
    assert abs(lse[0, 1] - logsumexp(s)) < 1e-12
    # no basis at all (keys and values kept full rank) is the same thing
    out, _ = O.decode_layer(q, [K[0]], [V[0]], None, None, "b")
    assert np.abs(out[0] - ref).max() < 1e-12


def test_path_a_equals_path_b_storage_faithful():
    # with bf16 U and a bf16 cache the two association orders still agree to fp64 rounding
    q, K, V, uk, uv, Kd, Vd = _case(13, 300, 8, 2, 48, 96)
    oa, la = O.decode_layer(q, Kd, Vd, uk, uv, "a")
    ob, lb = O.decode_layer(q, Kd, Vd, uk, uv, "b")
    assert np.abs(oa - ob).max() < 1e-12 and np.abs(la - lb).max() < 1e-12


def test_softmax_matches_scipy():
    s = np.random.default_rng(4).standard_normal(50) * 10
    p, lse = O._softmax_row(s)
    assert np.abs(p - softmax(s)).max() < 1e-15 and abs(lse - logsumexp(s)) < 1e-13


def test_zero_query_gives_mean_of_reconstructed_values():
    q, K, V, uk, uv, Kd, Vd = _case(14, 50, 4, 1, 64, 64)
    out, lse = O.decode_layer(np.zeros_like(q), Kd, Vd, uk, uv, "b")
    ref = (Vd[0][:, 0] @ uv[0].T).mean(axis=0)
    assert np.abs(out[0] - ref[None, :]).max() < 1e-13
    assert np.abs(lse - math.log(50)).max() < 1e-13


def test_constant_values_give_projected_value():
    q, K, V, uk, uv, Kd, _ = _case(15, 40, 4, 1, 64, 32, storage=False, bf16_U=False)
    v = np.random.default_rng(5).standard_normal(D)
    Vd = [np.stack([O.compress(np.tile(v, (40, 1)), uv[0], False)], 1)]
    out, _ = O.decode_layer(q, Kd, Vd, uk, uv, "b")
    assert np.abs(out[0] - (v @ uv[0] @ uv[0].T)[None, :]).max() < 1e-12


def test_dominating_key_selects_its_value_row():
    q, K, V, uk, uv, _, Vd = _case(16, 30, 4, 1, 64, 64, storage=False, bf16_U=False)
    K = K.copy()
    K[0, 17, 0] = 1e3 * (q[0, 2] @ uk[0] @ uk[0].T)          # aligned with query head 2, inside span(U_k)
    Kd = [np.stack([O.compress(K[0, :, 0], uk[0], False)], 1)]
    out, _ = O.decode_layer(q, Kd, Vd, uk, uv, "a")
    assert np.abs(out[0, 2] - Vd[0][17, 0] @ uv[0].T).max() < 1e-9


def test_output_lies_in_span_of_value_basis():
    q, K, V, uk, uv, Kd, Vd = _case(17, 64, 8, 2, 64, 48, storage=True, bf16_U=False)
    out, _ = O.decode_layer(q, Kd, Vd, uk, uv, "b")
    for g in range(8):
        U = uv[g // 4]
        assert np.abs(out[0, g] - out[0, g] @ U @ U.T).max() < 1e-12


def test_only_the_span_matters():
    # replacing U by U O (O orthogonal r x r) changes the cache but not the output (QR's R factor is irrelevant)
    q, K, V, uk, uv, Kd, Vd = _case(18, 90, 4, 1, 48, 64, storage=False, bf16_U=False)
    rng = np.random.default_rng(6)
    Ok, _ = np.linalg.qr(rng.standard_normal((48, 48)))
    Ov, _ = np.linalg.qr(rng.standard_normal((64, 64)))
    uk2, uv2 = uk @ Ok, uv @ Ov
    Kd2 = [np.stack([O.compress(K[0, :, 0], uk2[0], False)], 1)]
    Vd2 = [np.stack([O.compress(V[0, :, 0], uv2[0], False)], 1)]
    o1, _ = O.decode_layer(q, Kd, Vd, uk, uv, "b")
    o2, _ = O.decode_layer(q, Kd2, Vd2, uk2, uv2, "b")
    assert np.abs(o1 - o2).max() < 1e-12


def test_gqa_group_map_is_contiguous():
    # V rows constant per KV head (value = head index + 1): query head g must return KV head g//G's constant
    Hq, Hkv, n = 8, 4, 10
    q, K, V, _, _, _, _ = _case(19, n, Hq, Hkv, 128, 128)
    Vc = np.zeros_like(V)
    for h in range(Hkv):
        Vc[0, :, h, :] = h + 1
    out, _ = O.decode_layer(q, [K[0]], [Vc[0]], None, None, "b")
    for g in range(Hq):
        assert np.allclose(out[0, g], g // 2 + 1)


def test_shared_key_basis_is_broadcast_over_heads():
    q, K, V, uk, uv, _, _ = _case(20, 33, 8, 2, 64, 64)
    uk1 = uk[:1]
    Kd, Vd = O.compress_layer(K, V, uk1, uv, [33])
    Kd_ref = O.compress(K[0, :, 1], uk[0])
    assert np.array_equal(Kd[0][:, 1], Kd_ref)
    o1, _ = O.decode_layer(q, Kd, Vd, uk1, uv, "b")
    o2, _ = O.decode_layer(q, Kd, Vd, np.stack([uk[0], uk[0]]), uv, "a")
    assert np.abs(o1 - o2).max() < 1e-12


def test_empty_sequence():
    out, lse = O.attend_path_b(np.ones(D), np.zeros((0, 64)), np.zeros((0, 64)), np.zeros((D, 64)), np.zeros((D, 64)))
    assert np.all(out == 0) and lse == -math.inf
    out, lse = O.attend_path_a(np.ones(D), np.zeros((0, 64)), np.zeros((0, 64)), np.zeros((D, 64)), np.zeros((D, 64)))
    assert np.all(out == 0) and lse == -math.inf


# ---------------------------------------------------------------- combine

def test_combine_single_split_is_identity():
    o = np.random.default_rng(7).standard_normal((1, 64))
    out, lse = O.split_combine(o, np.array([0.7]))
    assert np.array_equal(out, o[0]) and lse == 0.7


def test_combine_matches_unsplit_and_scipy():
    q, K, V, uk, uv, Kd, Vd = _case(21, 333, 8, 2, 64, 96)
    ref, ref_lse = O.decode_layer(q, Kd, Vd, uk, uv, "a")
    for chunk in (64, 128, 1000):
        out, lse = O.decode_layer_split(q, Kd, Vd, uk, uv, chunk)
        assert np.abs(out - ref).max() < 1e-12 and np.abs(lse - ref_lse).max() < 1e-12
    pl = np.array([0.3, -2.0, 5.0, -math.inf])
    po = np.random.default_rng(8).standard_normal((4, 16))
    out, lse = O.split_combine(po, pl)
    assert abs(lse - logsumexp(pl)) < 1e-13
    w = softmax(pl)
    assert np.abs(out - (w[:, None] * po).sum(0)).max() < 1e-13
    # permutation invariance, empty splits weigh nothing even if their payload is garbage
    po[3] = np.nan
    perm = np.array([3, 1, 0, 2])
    out2, lse2 = O.split_combine(po[perm], pl[perm])
    assert np.abs(out2 - out).max() < 1e-13 and abs(lse2 - lse) < 1e-13
    out3, lse3 = O.split_combine(po[3:], pl[3:])
    assert np.all(out3 == 0) and lse3 == -math.inf


# ---------------------------------------------------------------- cache layout

def test_pool_address_formula_with_tagged_pattern():
    Hkv, r = 2, 48
    pg = I.make_paging(9, [130, 64, 1], reserve_tokens=1)
    assert sorted(pg.block_table[pg.block_table >= 0].tolist()) == list(range(pg.num_pages))
    pool = np.full(pg.num_pages * Hkv * 64 * r, -1.0)
    for b, n in enumerate(pg.seq_lens):
        for h in range(Hkv):
            rows = np.array([[((b * 1000 + t) * 4 + h) * 128 + j for j in range(r)] for t in range(n)], dtype=np.float64)
            O.write_cache_rows(pool, pg.block_table, b, h, 0, rows, Hkv)
    img = pool.reshape(pg.num_pages, Hkv, 64, r)
    for b, n in enumerate(pg.seq_lens):
        for t in (0, n // 2, n - 1):
            for h in range(Hkv):
                page = pg.block_table[b, t // 64]
                assert img[page, h, t % 64, 5] == ((b * 1000 + t) * 4 + h) * 128 + 5
        got = O.read_cache_rows(pool, pg.block_table, b, 1, int(n), Hkv, r)
        assert got[-1, 0] == ((b * 1000 + n - 1) * 4 + 1) * 128
    # every written element is distinct, everything else untouched
    written = pool[pool >= 0]
    assert written.size == sum(int(n) for n in pg.seq_lens) * Hkv * r == np.unique(written).size


# ---------------------------------------------------------------- byte accounting

def test_paper_sizing_example_and_cache_ratio():
    path = os.path.join(os.path.dirname(__file__), "golden", "kv_cache_sizing.txt")
    row = [l for l in open(path) if not l.startswith("#")][0].split()
    L, Hkv, d, T, B, bpe, gib = map(int, row)
    assert O.kv_cache_bytes(L, Hkv, T, B, None, d, bpe) == gib * 2 ** 30
    assert O.cache_ratio(64, 64) == 0.5 and O.cache_ratio(128, 128) == 1.0 and O.cache_ratio(48, 64) == 112 / 256
    prof = I.rank_profile(0)
    comp = O.kv_cache_bytes(L, Hkv, T, B, prof, d, bpe)
    assert abs(comp / (gib * 2 ** 30) - np.mean([O.cache_ratio(a, b) for a, b in prof])) < 1e-15


# ---------------------------------------------------------------- planted mistakes must be caught

def test_folding_the_projections_into_the_linear_layers_changes_nothing():
    # Sec. 3.3 "Overheads": with q' = q P_K handed over by a folded W_Q and the output left in the compressed space for a
    # folded P_V^T W_O, the attention is the same function: out = out_down P_V^T, lse unchanged
    n, r_k, r_v = 90, 48, 96
    Uk = I.stiefel_basis_f64(21, I.TAG_UK, 0, 0, r_k)
    Uv = I.stiefel_basis_f64(21, I.TAG_UV, 0, 0, r_v)
    K = I.normal_f64(I.stream_key(21, I.TAG_K), n * 128).numpy().reshape(n, 128)
    V = I.normal_f64(I.stream_key(21, I.TAG_V), n * 128).numpy().reshape(n, 128)
    q = I.normal_f64(I.stream_key(21, I.TAG_Q), 128).numpy()
    Kd, Vd = O.compress(K, Uk, storage=False), O.compress(V, Uv, storage=False)
    out, lse = O.attend_path_b(q, Kd, Vd, Uk, Uv)
    out_down, lse_f = O.attend_path_b(q @ Uk, Kd, Vd, None, None)
    assert out_down.shape == (r_v,) and abs(lse - lse_f) < 1e-12
    assert np.abs(out_down @ Uv.T - out).max() < 1e-12


def test_causal_rows_against_library_attention():
    # full rank, the whole sequence as queries: the textbook causal attention of a decoder, here torch's own routine
    # in fp64; then a chunk of queries at an offset, with the mask written out (True = may attend)
    import torch
    n, d = 70, 128
    K = I.normal_f64(I.stream_key(31, I.TAG_K), n * d).numpy().reshape(n, d)
    V = I.normal_f64(I.stream_key(31, I.TAG_V), n * d).numpy().reshape(n, d)
    Q = I.normal_f64(I.stream_key(31, I.TAG_Q), n * d).numpy().reshape(n, d)
    tq, tk, tv = (torch.from_numpy(x)[None, None] for x in (Q, K, V))
    want = torch.nn.functional.scaled_dot_product_attention(tq, tk, tv, is_causal=True)[0, 0].numpy()
    for path in ("a", "b"):
        got, lse = O.attend_rows_causal(Q, K, V, None, None, 0, path=path)
        assert np.abs(got - want).max() < 1e-12
    assert abs(lse[0] - (K[0] @ Q[0]) / np.sqrt(d)) < 1e-12                  # one visible position: lse = its score
    start, nq = 41, 29
    mask = torch.arange(n)[None, :] <= (start + torch.arange(nq))[:, None]
    want = torch.nn.functional.scaled_dot_product_attention(tq[:, :, start:], tk, tv, attn_mask=mask)[0, 0].numpy()
    got, _ = O.attend_rows_causal(Q[start:], K, V, None, None, start)
    assert got.shape == (nq, d) and np.abs(got - want).max() < 1e-12


def test_causal_rows_with_bases_and_causality():
    n, r_k, r_v, start = 90, 48, 96, 60
    Uk = I.stiefel_basis_f64(32, I.TAG_UK, 0, 0, r_k)
    Uv = I.stiefel_basis_f64(32, I.TAG_UV, 0, 0, r_v)
    K = I.normal_f64(I.stream_key(32, I.TAG_K), n * 128).numpy().reshape(n, 128)
    V = I.normal_f64(I.stream_key(32, I.TAG_V), n * 128).numpy().reshape(n, 128)
    Q = I.normal_f64(I.stream_key(32, I.TAG_Q), (n - start) * 128).numpy().reshape(n - start, 128)
    Kd, Vd = O.compress(K, Uk), O.compress(V, Uv)
    a, la = O.attend_rows_causal(Q, Kd, Vd, Uk, Uv, start, path="a")
    b, lb = O.attend_rows_causal(Q, Kd, Vd, Uk, Uv, start, path="b")
    assert np.abs(a - b).max() < 1e-12 and np.abs(la - lb).max() < 1e-12
    # the last row is plain decode attention over the whole cache
    o, l = O.attend_path_b(Q[-1], Kd, Vd, Uk, Uv)
    assert np.array_equal(o, b[-1]) and l == lb[-1]
    # a cache row at position p influences rows at positions >= p and no earlier one
    p = start + 10
    Kd2 = Kd.copy(); Kd2[p] += 1.0
    c, _ = O.attend_rows_causal(Q, Kd2, Vd, Uk, Uv, start)
    changed = np.abs(c - b).max(axis=1) > 0
    assert not changed[:10].any() and changed[10:].all()


def test_planted_mistakes_fail_the_pins():
    """Sanity of the pins themselves: a wrong softmax scale or a wrong query-head -> KV-head map is
    detected by the reconstructed-KV library check (the mistakes are planted here, on the CPU)."""
    Hq, Hkv, n = 8, 2, 77
    q, K, V, uk, uv, Kd, Vd = _case(11, n, Hq, Hkv, 64, 64, storage=False, bf16_U=False)
    Kt = np.stack([K[0, :, h] @ uk[h] @ uk[h].T for h in range(Hkv)], 1)
    Vt = np.stack([V[0, :, h] @ uv[h] @ uv[h].T for h in range(Hkv)], 1)
    ref = _sdpa(q[0], Kt, Vt, Hkv)
    # 1/sqrt(r_k) instead of 1/sqrt(d_h)
    bad = np.stack([O.attend_path_b(q[0, g], Kd[0][:, g // 4], Vd[0][:, g // 4], uk[g // 4], uv[g // 4], d_h=64)[0]
                    for g in range(Hq)])
    assert np.abs(bad - ref).max() > 1e-3
    # interleaved instead of contiguous groups
    bad = np.stack([O.attend_path_b(q[0, g], Kd[0][:, g % 2], Vd[0][:, g % 2], uk[g % 2], uv[g % 2])[0] for g in range(Hq)])
    assert np.abs(bad - ref).max() > 1e-3
    # value basis of the wrong head
    bad = np.stack([O.attend_path_b(q[0, g], Kd[0][:, g // 4], Vd[0][:, g // 4], uk[g // 4], uv[1 - g // 4])[0] for g in range(Hq)])
    assert np.abs(bad - ref).max() > 1e-3
