"""A seeded random sweep: shapes, plane counts, scaling units, column counts and explicit decompositions of the
products, and shapes, bit widths, token counts and scale-factor counts of the search, against the fp64 oracle."""
import random

import numpy as np
import pytest

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("needs a GPU", allow_module_level=True)

import oracle
from helpers import TOL, rel_err
from paper_2407_02891_b200 import binding as bq
from paper_2407_02891_b200 import synth

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda", 0)


def _to(a):
    return torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_products_match_the_oracle(seed):
    rng = random.Random(seed)
    for case in range(16):
        q = rng.choice([1, 2, 2, 3, 3, 4])
        group = rng.choice([0, 128, 128, 64, 32])
        N = 8 * rng.choice([1, 5, 23, 64, 184, 185, 368, 369, 500, 896])        # 184 row units: the most one block takes
        K = 512 * rng.choice([1, 2, 3, 4, 7, 8, 14, 18, 33])
        name = f"random/{seed}/{case}"
        planes = synth.planes(name, N, K, q)
        alpha, z = synth.scale_rows(name, N, K, q, group)
        L = bq.pack_layer(N, K, q, group, bq.LAYOUT_TILED, _to(synth.codes_from_planes(planes)), _to(alpha), _to(z))
        B = rng.choice([1, 1, 1, 2, 3, 4, 8, 16])
        X = synth.activations(name, B, K)
        plan = bq.plan_default(L.d, B)
        if B == 1 and plan.kernel == 1 and rng.random() < 0.6:                   # a decomposition the planner would not pick
            U, W = N // 8, K // 512
            ks = rng.randint(1, min(W, 64))
            while -(-W // ks) > 32:
                ks += 1
            rb_min = -(-U // 184)
            rb = rng.randint(rb_min, max(rb_min, min(U, 148 // ks)))
            plan = bq.Plan(1, rb, ks, 0)
        ws = bq.new_workspace(L.d, B, plan)
        Y = torch.full((B * N,), float("nan"), dtype=torch.float16, device=DEV)
        xd = _to(X.reshape(-1))
        for _ in range(2):                                                       # the second call meets the workspace as the first left it
            if B == 1:
                bq.gemv_plan(L.d, plan, L.packed, L.alpha, L.z, xd, Y, ws)
            else:
                bq.gemm_smallbatch(L.d, L.packed, L.alpha, L.z, xd, Y, B, ws)
        torch.cuda.synchronize()
        assert bq.lib().bcq_poll_status() == bq.OK, (case, N, K, q, group, B)
        ref = oracle.forward_planes(planes, alpha, z, X, group)
        assert rel_err(Y.cpu().numpy().reshape(B, N), ref) <= TOL, (case, N, K, q, group, B, plan.row_blocks, plan.k_splits)


def test_random_searches_match_the_oracle():
    rng = random.Random(21)
    for case in range(24):
        n_bits = rng.choice([2, 3, 4, 4, 5])
        q = rng.randint(1, min(n_bits, 4))
        N = rng.choice([8, 64, 128, 136, 200, 256, 392])
        K = 64 * rng.choice([1, 2, 4, 8, 9, 16])
        group = rng.choice([g for g in (0, 64, 128, 192, 256) if g == 0 or K % g == 0])
        T = 16 * rng.choice([1, 2, 3, 4, 8, 11, 16, 17, 20])
        n_scales = rng.choice([1, 2, 3, 9])
        name = f"random/search/{case}"
        W = (0.05 * synth.normal(name + "/W", 0, N * K)).reshape(N, K).astype(np.float16)
        X = synth.activations(name + "/X", T, K)
        parts, s = bq.partitions(n_bits, q), bq.reexplore_factors(n_bits, n_scales)
        err, rows, best = bq.grid_search(N, K, q, group, _to(W), _to(X), n_bits, parts, s)
        torch.cuda.synchronize()
        assert bq.lib().bcq_poll_status() == bq.OK
        ref_rows, ref_err, _ = oracle.grid_search(W, X, group, n_bits, list(parts), s)
        got = rows.cpu().numpy().astype(np.float64)
        assert np.abs(got - ref_rows).max() <= 5e-3 * np.abs(ref_rows).max(), (case, N, K, q, group, n_bits, T, n_scales)
        np.testing.assert_allclose(err.cpu().numpy(), ref_err, rtol=5e-3)
