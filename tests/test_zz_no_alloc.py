"""bcq_gemv_noalloc: the product for callers that cannot allocate device memory.

Some users of the library run where no device allocation is possible when the product is
needed (a plugin inside an application that owns all GPU memory, a serving loop that must not
stall on an allocation).  For them the library carries a fixed scratch array and this entry
point uses it instead of a caller-provided workspace.  The test checks that it gives what
bcq_gemv gives with a real workspace, on two calls in a row (the second call meets the scratch
as the first one left it), and that a product too large for the array is refused cleanly.

This file sorts last on purpose: a run that stops at the first failure has then already run
every other test.
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


@pytest.mark.parametrize("N,K,q", [(1024, 1024, 3), (4096, 4096, 3), (2048, 8192, 2)])
def test_noalloc_matches_gemv_twice_in_a_row(N, K, q):
    group = 128
    p, codes, alpha, z, x = make_layer(f"noalloc/{N}x{K}", N, K, q, group, B=2)
    L = bq.pack_layer(N, K, q, group, bq.LAYOUT_TILED, _dev(codes), _dev(alpha), _dev(z))
    plan = bq.plan_default(L.d)
    assert plan.k_splits > 1, "the case must exercise the scratch array"
    assert bq.workspace_bytes(L.d, 1, plan) <= bq.NOALLOC_SCRATCH_BYTES
    ws = bq.new_workspace(L.d, 1)
    for call in range(2):                       # two different activations, back to back
        xd = _dev(x[call])
        want = torch.zeros(N, dtype=torch.float16, device=DEV)
        got = torch.full((N,), float("nan"), dtype=torch.float16, device=DEV)
        bq.gemv(L.d, L.packed, L.alpha, L.z, xd, want, ws)
        bq.gemv_noalloc(L.d, L.packed, L.alpha, L.z, xd, got)
        torch.cuda.synchronize()
        w, g = want.cpu().numpy(), got.cpu().numpy()
        assert rel_err(g, w.astype(np.float64)) <= TOL
        ref = oracle.forward_planes(p, alpha, z, x[call:call + 1], group)[0]
        assert rel_err(g, ref) <= TOL


def test_noalloc_refuses_products_beyond_its_scratch():
    cand = [(393216, 16384), (524288, 32768), (262144, 4096), (65536, 32768), (32768, 65536), (131072, 16384), (262144, 16384)]   # 8 bytes of scratch per row
    for N, K in cand:
        d = bq.desc(N, K, 3, 128, bq.LAYOUT_TILED)
        if bq.workspace_bytes(d, 1) > bq.NOALLOC_SCRATCH_BYTES:
            t = torch.zeros(64, dtype=torch.float16, device=DEV)   # never touched: refused on the host
            with pytest.raises(bq.BcqError) as e:
                bq.gemv_noalloc(d, t, t, t, t, t)
            assert e.value.status == bq.ERR_SCRATCH_LIMIT
            return
    pytest.skip("no candidate shape needs more than the built-in scratch on this GPU")
