"""bcq_gemv_bf16: bfloat16 activations and outputs against the oracle's dequantised weights (fp64) times the
exact values of the bfloat16 activations."""
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


def _bf16(a64):
    """Round fp64 values to bfloat16 (torch does the rounding: a library conversion, not the kernel's)."""
    return torch.from_numpy(np.asarray(a64, np.float32)).to(torch.bfloat16)


@pytest.mark.parametrize("N,K,q,group", [(1024, 1024, 3, 128), (4096, 2048, 2, 0), (64, 512, 3, 128), (7168, 7168, 3, 128)])
def test_bf16_gemv_matches_the_oracle(N, K, q, group):
    name = f"bf16/{N}x{K}/{q}/{group}"
    planes = synth.planes(name, N, K, q)
    alpha, z = synth.scale_rows(name, N, K, q, group)
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    L = bq.pack_layer(N, K, q, group, bq.LAYOUT_TILED, to(synth.codes_from_planes(planes)), to(alpha), to(z))
    xb = _bf16(3.0 * synth.normal(name + "/x", 0, K))                  # values fp16 cannot all hold exactly
    x64 = xb.to(torch.float64).numpy()
    Wd = oracle.dequant(synth.codes_from_planes(planes), alpha, z, group)
    ref = Wd @ x64
    ws = bq.new_workspace(L.d, 1)
    y = torch.full((N,), float("nan"), dtype=torch.bfloat16, device=DEV)
    bq.gemv_bf16(L.d, L.packed, L.alpha, L.z, xb.to(DEV), y, workspace=ws)
    torch.cuda.synchronize()
    assert rel_err(y.to(torch.float64).cpu().numpy(), ref) <= TOL      # 2^-9 of the output rounding + the tables' 3e-4
    # with bias, ReLU and a residual, all bfloat16
    bias, res = _bf16(0.5 * synth.normal(name + "/b", 0, N)), _bf16(synth.normal(name + "/r", 0, N))
    bq.gemv_bf16(L.d, L.packed, L.alpha, L.z, xb.to(DEV), y, bias.to(DEV), res.to(DEV), bq.ACT_RELU, ws)
    torch.cuda.synchronize()
    want = np.maximum(ref + bias.to(torch.float64).numpy(), 0.0) + res.to(torch.float64).numpy()
    assert rel_err(y.to(torch.float64).cpu().numpy(), want) <= TOL


def test_bf16_rounding_of_the_result_is_to_nearest_even():
    # an 8 x 512 layer whose product is exact in fp32: all planes +1, alpha = 1, z = 0: y = sum of x
    N, K, q, group = 8, 512, 1, 0
    planes = np.full((q, N, K // 8), 0xFF, np.uint8)
    alpha = np.ones((q, N, 1), np.float16)
    z = np.zeros((N, 1), np.float16)
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    L = bq.pack_layer(N, K, q, group, bq.LAYOUT_TILED, to(synth.codes_from_planes(planes)), to(alpha), to(z))
    for extra, want in ((1.0, 256.0), (3.0, 260.0), (2.0, 258.0), (5.0, 260.0), (7.0, 264.0)):
        # 256 + extra: bfloat16 steps by 2 here; 257, 259, 261, 263 are ties and go to the even significand
        x = np.zeros(K, np.float32)
        x[0], x[9] = 256.0, extra
        y = torch.zeros(N, dtype=torch.bfloat16, device=DEV)
        bq.gemv_bf16(L.d, L.packed, L.alpha, L.z, torch.from_numpy(x).to(torch.bfloat16).to(DEV), y)
        torch.cuda.synchronize()
        assert torch.equal(y.cpu().to(torch.float32), torch.full((N,), want))
