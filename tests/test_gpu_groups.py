"""Groups of 64 and 32 weights per scale in the tiled layout: the lookup-table kernel against the oracle,
the quantiser into that layout, several columns (column by column), and what does not exist for them."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("needs a GPU", allow_module_level=True)

import oracle
from helpers import TOL, rel_err, tiled_operands
from paper_2407_02891_b200 import binding as bq
from paper_2407_02891_b200 import synth

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda", 0)


def _layer(name, N, K, q, group):
    planes = synth.planes(name, N, K, q)
    alpha, z = synth.scale_rows(name, N, K, q, group)
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    L = bq.pack_layer(N, K, q, group, bq.LAYOUT_TILED, to(synth.codes_from_planes(planes)), to(alpha), to(z))
    return planes, alpha, z, L


@pytest.mark.parametrize("group", [64, 32])
@pytest.mark.parametrize("N,K,q", [(1024, 1024, 3), (64, 512, 1), (4096, 2048, 2), (2048, 4096, 4), (7168, 7168, 3), (8, 512, 3),
                                   (1496, 3584, 3)])
def test_gemv_small_groups_matches_the_oracle(N, K, q, group):
    name = f"groups/{N}x{K}/{q}/{group}"
    planes, alpha, z, L = _layer(name, N, K, q, group)
    x = synth.activations(name, 1, K)
    plan = bq.plan_default(L.d, 1)
    assert plan.kernel == 1                                  # the lookup-table kernel, not the generic one
    ws = bq.new_workspace(L.d, 1)
    y = torch.full((N,), float("nan"), dtype=torch.float16, device=DEV)
    xd = torch.from_numpy(x.reshape(-1)).to(DEV)
    for _ in range(2):                                       # the second call meets the workspace as the first left it
        bq.gemv(L.d, L.packed, L.alpha, L.z, xd, y, ws)
    torch.cuda.synchronize()
    ref = oracle.forward_planes(planes, alpha, z, x, group)[0]
    assert rel_err(y.cpu().numpy(), ref) <= TOL
    assert bq.lib().bcq_poll_status() == bq.OK


@pytest.mark.parametrize("group", [64, 32])
def test_small_groups_structured_inputs(group):
    # scales that differ strongly between neighbouring units and unit activations: a unit's scale applied to
    # another unit's weights, or a chunk looked up in the wrong column, shows at once
    N, K, q = 64, 1024, 2
    name = f"groups/struct/{group}"
    planes = synth.planes(name, N, K, q)
    G = K // group
    alpha = np.zeros((q, N, G), np.float16)
    alpha[0] = (1.0 + np.arange(G)[None, :] + 0.25 * (np.arange(N)[:, None] % 4)).astype(np.float16)
    alpha[1] = (0.5 * alpha[0].astype(np.float64)).astype(np.float16)
    z = (0.125 * (np.arange(G)[None, :] % 7) - 0.25 + 0.0 * np.arange(N)[:, None]).astype(np.float16)
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    L = bq.pack_layer(N, K, q, group, bq.LAYOUT_TILED, to(synth.codes_from_planes(planes)), to(alpha), to(z))
    ws = bq.new_workspace(L.d, 1)
    Wd = oracle.dequant(synth.codes_from_planes(planes), alpha, z, group)
    y = torch.zeros(N, dtype=torch.float16, device=DEV)
    for k in [0, 7, 8, 31, 32, 63, 64, 100, 127, 128, 511, 512, 777, 1023]:
        e = np.zeros(K, np.float16)
        e[k] = 1.0
        bq.gemv(L.d, L.packed, L.alpha, L.z, to(e), y, ws)
        torch.cuda.synchronize()
        assert np.abs(y.cpu().numpy().astype(np.float64) - Wd[:, k]).max() <= 2.0 ** -10 * np.abs(Wd[:, k]).max(), k


@pytest.mark.parametrize("group,B", [(64, 2), (32, 5), (64, 16)])
def test_small_groups_several_columns_and_explicit_plans(group, B):
    N, K, q = 1024, 2048, 3
    name = f"groups/batch/{group}/{B}"
    planes, alpha, z, L = _layer(name, N, K, q, group)
    X = synth.activations(name, B, K)
    plan = bq.plan_default(L.d, B)
    assert plan.kernel == 1                                  # column by column: no pair tables, no tensor-core kernel here
    ws = bq.new_workspace(L.d, B)
    Y = torch.full((B * N,), float("nan"), dtype=torch.float16, device=DEV)
    bq.gemm_smallbatch(L.d, L.packed, L.alpha, L.z, torch.from_numpy(X.reshape(-1)).to(DEV), Y, B, ws)
    torch.cuda.synchronize()
    ref = oracle.forward_planes(planes, alpha, z, X, group)
    assert rel_err(Y.cpu().numpy().reshape(B, N), ref) <= TOL
    with pytest.raises(bq.BcqError):                         # the tensor-core kernel takes groups of 128 or one scale per row
        bq.gemm_smallbatch_plan(L.d, bq.Plan(2, 8, 2, 0), L.packed, L.alpha, L.z, torch.from_numpy(X.reshape(-1)).to(DEV), Y, B, ws)
    # explicit decompositions of the single product
    x = torch.from_numpy(X[0]).to(DEV)
    for rb, ks in [(1, 1), (3, 2), (16, 4), (128, 1)]:
        p = bq.Plan(1, rb, ks, 0)
        w2 = bq.new_workspace(L.d, 1, p)
        y = torch.full((N,), float("nan"), dtype=torch.float16, device=DEV)
        bq.gemv_plan(L.d, p, L.packed, L.alpha, L.z, x, y, w2)
        torch.cuda.synchronize()
        assert rel_err(y.cpu().numpy(), ref[0]) <= TOL, (rb, ks)


@pytest.mark.parametrize("group", [64, 32])
def test_quantise_into_small_groups(group):
    # bcq_quantize_rtn straight into the tiled layout: bit-identical to the oracle's quantise -> merge -> pack,
    # laid out as the header describes
    N, K, q, n_bits = 64, 1024, 3, 4
    W = (0.05 * synth.normal(f"groups/quant/{group}", 0, N * K)).reshape(N, K).astype(np.float16)
    b2p = np.array([0, 1, 1, 2], np.uint8)
    w_int, S, qb = oracle.quantize_rtn(W, group, n_bits, 1.0)
    codes, alpha, z = oracle.merge_linear(w_int, S, qb, group, n_bits, b2p)
    want, _, _ = tiled_operands(oracle.pack_canonical(codes, q), alpha, z, group)
    d = bq.desc(N, K, q, group, bq.LAYOUT_TILED)
    packed, a, zz = bq.empty_operands(d, DEV)
    G = K // group
    Sd = torch.zeros(N * G, dtype=torch.float16, device=DEV)
    qd = torch.zeros(N * G, dtype=torch.float16, device=DEV)
    rc = bq.lib().bcq_quantize_rtn(__import__("ctypes").byref(d), bq._ptr(torch.from_numpy(W).to(DEV)), n_bits,
                                   b2p.ctypes.data_as(__import__("ctypes").c_void_p), 1.0, bq._ptr(Sd), bq._ptr(qd), None,
                                   bq._ptr(packed), None, None, bq._stream())
    assert rc == bq.OK
    torch.cuda.synchronize()
    assert np.array_equal(packed.cpu().numpy(), want)
