"""The give-up branch of the kernels' bounded waits, reached on purpose.

Every device-side wait of the library polls a limited number of times, then raises the CTA's abort flag, reports
STIEF_ERR_TIMEOUT through the status word and lets the kernel run to its normal end.  In a healthy run that branch
never executes, so stief_selftest_wait_limit exists to execute it: a barrier nobody completes, waited on with a small
poll limit.  Nothing here faults or waits without bound."""
import pytest
import torch

import paper_2601_21686_b200 as S
from tests import _util as U

pytestmark = pytest.mark.gpu


def test_a_wait_that_nobody_satisfies_runs_out_and_the_context_stays_usable():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rep = torch.full((8,), -1, dtype=torch.int32, device="cuda")
    S.stief_selftest_wait_limit(status, rep, poll_limit=64)
    torch.cuda.synchronize()
    r = rep.cpu().tolist()
    assert int(status.item()) == S.STIEF_ERR_TIMEOUT
    assert S.status_string(S.STIEF_ERR_TIMEOUT) == "bounded device-side wait ran out"
    assert r[0] == 0 and r[2] == 1, r                 # the first wait gave up and raised the abort flag
    assert r[3] == 0 and r[5] == 0, r                 # the later waits were not satisfied either ...
    assert r[7] == 0x600D, r                          # ... and the kernel still reached its end
    # the later waits carry the kernels' full limit (2^24 and 2^26 polls): only the abort flag can have ended them
    # after their first few thousand polls.  Allow a generous 50 ms of SM cycles; the full limits would take seconds.
    assert 0 < r[4] < 100_000_000 and 0 < r[6] < 100_000_000, r
    print(f"wait of 64 polls gave up after {r[1]} cycles; aborted waits returned after {r[4]} and {r[6]} cycles")

    # first error wins: a second run does not overwrite the word; a cleared word is set again
    S.stief_selftest_wait_limit(status, rep, poll_limit=1)
    torch.cuda.synchronize()
    assert int(status.item()) == S.STIEF_ERR_TIMEOUT

    # the context is healthy: an ordinary decode call afterwards is correct
    c = U.make_case(71, 2, 8, 2, 64, 64, [300, 77])
    S.stief_prefill_compress(c.layer, c.batch, c.K.cuda(), c.V.cuda(), status=c.status)
    ws = U.workspace_for(c, 0)
    out = torch.empty(c.B, c.Hq, 128, dtype=torch.bfloat16, device="cuda")
    S.stief_decode_attention(c.layer, c.batch, c.q.cuda(), ws, 0, out, status=c.status)
    torch.cuda.synchronize()
    assert int(c.status.item()) == 0
    Kd, Vd = U.oracle_cache(c)
    ref, _ = U.oracle_decode(c, Kd, Vd)
    U.check_out(out, ref)


def test_bad_arguments_are_refused_on_the_host():
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    rep = torch.zeros(8, dtype=torch.int32, device="cuda")
    for lim in (0, -1, (1 << 20) + 1):
        with pytest.raises(S.StiefError) as e:
            S.stief_selftest_wait_limit(status, rep, poll_limit=lim)
        assert e.value.code == S.STIEF_ERR_INVALID_ARG
