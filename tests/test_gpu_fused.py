"""bcq_gemv_fused: y = act(W x + bias) + residual against the fp64 oracle product followed by the plain
definitions of the three steps."""
import numpy as np
import pytest

torch = pytest.importorskip("torch")
if not torch.cuda.is_available():
    pytest.skip("needs a GPU", allow_module_level=True)
from scipy.special import erf

import oracle
from helpers import TOL, rel_err
from paper_2407_02891_b200 import binding as bq
from paper_2407_02891_b200 import synth

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda", 0)

ACTS = {
    bq.ACT_NONE: lambda v: v,
    bq.ACT_RELU: lambda v: np.maximum(v, 0.0),
    bq.ACT_GELU: lambda v: 0.5 * v * (1.0 + erf(v / np.sqrt(2.0))),
    bq.ACT_SILU: lambda v: v / (1.0 + np.exp(-v)),
}


def _layer(name, N, K, q, group):
    planes = synth.planes(name, N, K, q)
    alpha, z = synth.scale_rows(name, N, K, q, group)
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    L = bq.pack_layer(N, K, q, group, bq.LAYOUT_TILED, to(synth.codes_from_planes(planes)), to(alpha), to(z))
    return planes, alpha, z, L


@pytest.mark.parametrize("N,K,q,group", [(1024, 1024, 3, 128), (4096, 2048, 2, 0), (64, 512, 3, 128), (2048, 8192, 4, 128)])
@pytest.mark.parametrize("act", [bq.ACT_NONE, bq.ACT_RELU, bq.ACT_GELU, bq.ACT_SILU])
def test_fused_epilogue_matches_the_definitions(N, K, q, group, act):
    name = f"fused/{N}x{K}/{q}/{group}"
    planes, alpha, z, L = _layer(name, N, K, q, group)
    x = synth.activations(name, 1, K)
    bias = (0.5 * synth.normal(name + "/bias", 0, N)).astype(np.float16)
    res = synth.normal(name + "/res", 0, N).astype(np.float16)
    xd = torch.from_numpy(x.reshape(-1)).to(DEV)
    ws = bq.new_workspace(L.d, 1)
    ref = oracle.forward_planes(planes, alpha, z, x, group)[0]
    for use_bias, use_res in [(True, True), (True, False), (False, True), (False, False)]:
        y = torch.full((N,), float("nan"), dtype=torch.float16, device=DEV)
        bq.gemv_fused(L.d, L.packed, L.alpha, L.z, xd, y, torch.from_numpy(bias).to(DEV) if use_bias else None,
                      torch.from_numpy(res).to(DEV) if use_res else None, act, ws)
        torch.cuda.synchronize()
        want = ACTS[act](ref + (bias.astype(np.float64) if use_bias else 0.0)) + (res.astype(np.float64) if use_res else 0.0)
        assert rel_err(y.cpu().numpy(), want) <= TOL


def test_fused_without_steps_is_the_plain_product_and_residual_may_be_y():
    N, K, q, group = 1024, 2048, 3, 128
    planes, alpha, z, L = _layer("fused/plain", N, K, q, group)
    x = synth.activations("fused/plain", 1, K)
    xd = torch.from_numpy(x.reshape(-1)).to(DEV)
    ws = bq.new_workspace(L.d, 1)
    a = torch.zeros(N, dtype=torch.float16, device=DEV)
    b = torch.zeros(N, dtype=torch.float16, device=DEV)
    bq.gemv(L.d, L.packed, L.alpha, L.z, xd, a, ws)
    bq.gemv_fused(L.d, L.packed, L.alpha, L.z, xd, b, None, None, bq.ACT_NONE, ws)
    torch.cuda.synchronize()
    assert torch.equal(a, b)
    # y += W x: the residual is the output buffer itself
    res = synth.normal("fused/plain/res", 0, N).astype(np.float16)
    y = torch.from_numpy(res.copy()).to(DEV)
    bq.gemv_fused(L.d, L.packed, L.alpha, L.z, xd, y, None, y, bq.ACT_NONE, ws)
    torch.cuda.synchronize()
    ref = oracle.forward_planes(planes, alpha, z, x, group)[0] + res.astype(np.float64)
    assert rel_err(y.cpu().numpy(), ref) <= TOL
    # the generic kernel has no fused form
    dc = bq.desc(N, K, q, group, bq.LAYOUT_CANONICAL)
    with pytest.raises(bq.BcqError):
        bq.gemv_fused(dc, L.packed, L.alpha, L.z, xd, y, None, None, bq.ACT_RELU, None)
