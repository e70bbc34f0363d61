"""A bounded wait inside the lookup-table kernel that runs out: the kernel must return by itself, the
library must report it, and the next product on the same stream must be right again.

Nothing here faults or hangs the GPU.  The test-only plan bits of include/bcq.h shorten every wait's
limit to about a millisecond and make the table builders keep the second window's table to themselves;
the consumer warps that wait for it give up, every copy that was started still lands, the blocks return.
"""
import numpy as np
import pytest
import torch

import oracle
from helpers import TOL, make_layer, rel_err
from paper_2407_02891_b200 import binding as bq

pytestmark = pytest.mark.gpu
DEV = "cuda"


def _dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


@pytest.mark.parametrize("group", [128, 0])
def test_wait_that_runs_out_is_reported_and_the_next_call_is_correct(group):
    N, K, q = 1024, 2048, 3                      # four windows in one K split
    p, codes, alpha, z, x = make_layer(f"timeout/{group}", N, K, q, group)
    L = bq.pack_layer(N, K, q, group, bq.LAYOUT_TILED, _dev(codes), _dev(alpha), _dev(z))
    xd = _dev(x.reshape(-1))
    y = torch.zeros(N, dtype=torch.float16, device=DEV)
    bq.poll_status()                             # clean before the experiment
    starve = bq.Plan(1, 2, 1, bq.PLAN_TEST_SHORT_WAITS | bq.PLAN_TEST_WITHHOLD_TABLE)
    bq.gemv_plan(L.d, starve, L.packed, L.alpha, L.z, xd, y, None)
    with pytest.raises(bq.BcqError) as e:
        bq.poll_status()
    assert e.value.status == bq.ERR_TIMEOUT
    bq.poll_status()                             # the report clears the status word
    # the same stream, the same operands, an ordinary plan: correct again
    y.fill_(float("nan"))
    bq.gemv_plan(L.d, bq.Plan(1, 2, 1, 0), L.packed, L.alpha, L.z, xd, y, None)
    torch.cuda.synchronize()
    bq.poll_status()
    ref = oracle.forward_planes(p, alpha, z, x, group)[0]
    assert rel_err(y.cpu().numpy(), ref) <= TOL


def test_short_waits_alone_change_nothing():
    N, K, q, group = 1024, 2048, 3, 128
    p, codes, alpha, z, x = make_layer("timeout/short", N, K, q, group)
    L = bq.pack_layer(N, K, q, group, bq.LAYOUT_TILED, _dev(codes), _dev(alpha), _dev(z))
    y = torch.zeros(N, dtype=torch.float16, device=DEV)
    bq.gemv_plan(L.d, bq.Plan(1, 2, 1, bq.PLAN_TEST_SHORT_WAITS), L.packed, L.alpha, L.z, _dev(x.reshape(-1)), y, None)
    torch.cuda.synchronize()
    bq.poll_status()
    ref = oracle.forward_planes(p, alpha, z, x, group)[0]
    assert rel_err(y.cpu().numpy(), ref) <= TOL


def test_unknown_plan_bits_are_rejected():
    d = bq.desc(1024, 2048, 3, 128, bq.LAYOUT_TILED)
    t = torch.zeros(64, dtype=torch.float16, device=DEV)
    with pytest.raises(bq.BcqError) as e:
        bq.gemv_plan(d, bq.Plan(1, 2, 1, 4), t, None, None, t, t, None)
    assert e.value.status == bq.ERR_INVALID_ARG
