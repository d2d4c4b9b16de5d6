"""The workspace-free decode entry point against the ordinary one.

stief_decode_attention_static serves callers that cannot allocate device memory themselves (a plug-in
inside an engine that has taken all of it for its own pool; a loop where cudaMalloc's device-wide
synchronisation is not allowed): its split-T scratch is a fixed array inside the library.  It must give
what stief_decode_attention gives with a caller-allocated workspace, call after call, although every call
reuses the same array with the previous call's contents still in it.

This file sorts last on purpose, so that a run which stops at the first failure has already run every
other test."""
import pytest
import torch

import paper_2601_21686_b200 as S
from tests import _util as U

pytestmark = pytest.mark.gpu


def test_static_workspace_matches_caller_workspace_twice_in_a_row():
    # two shapes back to back: the second call finds the first call's partials and counters in the array
    cases = [U.make_case(81, 3, 8, 2, 64, 96, [700, 64, 333], lowrank=True),
             U.make_case(82, 2, 16, 2, 48, 128, [1500, 129])]
    for c in cases:
        S.stief_prefill_compress(c.layer, c.batch, c.K.cuda(), c.V.cuda(), status=c.status)
    for rep in range(2):
        for c, parts in zip(cases, (5, 0)):
            ws = U.workspace_for(c, parts)
            ref = torch.full((c.B, c.Hq, 128), float("nan"), dtype=torch.bfloat16, device="cuda")
            ref_lse = torch.full((c.B, c.Hq), float("nan"), dtype=torch.float32, device="cuda")
            S.stief_decode_attention(c.layer, c.batch, c.q.cuda(), ws, parts, ref, ref_lse, status=c.status)
            out = torch.full_like(ref, float("nan"))
            lse = torch.full_like(ref_lse, float("nan"))
            S.stief_decode_attention_static(c.layer, c.batch, c.q.cuda(), out, parts, lse, status=c.status)
            torch.cuda.synchronize()
            assert int(c.status.item()) == 0
            # same kernel, same partition, same merge order: only the scratch address differs, so not one bit may
            assert torch.equal(out, ref)
            assert torch.equal(lse, ref_lse)
            # ... and both are inside the parity tolerance of the oracle-checked entry point (max-abs 1e-2, rel-L2 5e-3)
            U.check_out(out, ref.double().cpu().numpy())


def test_static_workspace_rejects_shapes_beyond_its_size():
    # 512 (sequence, KV head) pairs with r_v = 128 need more than the built-in 2 MiB: refused on the host
    assert S.stief_decode_workspace_bytes(64, 32, 8, 128, 0) > S.STATIC_WORKSPACE_BYTES
    c = U.make_case(83, 64, 32, 8, 32, 128, [1] * 64)
    out = torch.empty(64, 32, 128, dtype=torch.bfloat16, device="cuda")
    with pytest.raises(S.StiefError) as e:
        S.stief_decode_attention_static(c.layer, c.batch, c.q.cuda(), out)
    assert e.value.code == S.STIEF_ERR_WORKSPACE
    with pytest.raises(S.StiefError) as e:       # the partials cannot be handed out, so `out` is required
        S._check(S.lib().stief_decode_attention_static(None, None, None, 0, 0, None, None, None, None), "static")
    assert e.value.code == S.STIEF_ERR_INVALID_ARG
