"""bcq_gemv_dequant (the ablation without lookup tables: every weight dequantised to fp16, then multiplied)
against the fp64 oracle."""
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


@pytest.mark.parametrize("N,K,q,group", [(1024, 1024, 3, 128), (4096, 2048, 2, 0), (64, 512, 1, 128), (2048, 8192, 4, 128),
                                         (7168, 7168, 3, 128), (512, 3584, 3, 0)])
def test_dequant_gemv_matches_the_oracle(N, K, q, group):
    name = f"dequant/{N}x{K}/{q}/{group}"
    planes = synth.planes(name, N, K, q)
    alpha, z = synth.scale_rows(name, N, K, q, group)
    x = synth.activations(name, 1, K)
    to = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    L = bq.pack_layer(N, K, q, group, bq.LAYOUT_TILED, to(synth.codes_from_planes(planes)), to(alpha), to(z))
    y = torch.full((N,), float("nan"), dtype=torch.float16, device=DEV)
    bq.gemv_dequant(L.d, L.packed, L.alpha, L.z, to(x.reshape(-1)), y)
    torch.cuda.synchronize()
    ref = oracle.forward_planes(planes, alpha, z, x, group)[0]
    assert rel_err(y.cpu().numpy(), ref) <= TOL
    # the weights it forms are those of the oracle's dequantisation, rounded to fp16: unit activations return columns
    e = np.zeros((1, K), np.float16)
    e[0, 5] = 1.0
    bq.gemv_dequant(L.d, L.packed, L.alpha, L.z, to(e.reshape(-1)), y)
    torch.cuda.synchronize()
    col = oracle.dequant(synth.codes_from_planes(planes), alpha, z, group)[:, 5]
    assert np.abs(y.cpu().numpy().astype(np.float64) - col).max() <= 2.0 ** -9 * np.abs(col).max()


def test_dequant_gemv_needs_the_tiled_layout():
    d = bq.desc(64, 512, 3, 128, bq.LAYOUT_CANONICAL)
    t = torch.zeros(64 * 512, dtype=torch.float16, device=DEV)
    with pytest.raises(bq.BcqError):
        bq.gemv_dequant(d, t, t, t, t, t)
