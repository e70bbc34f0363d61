"""bcq_gemv_multi: several packed layers that read the same activation, one launch, separate outputs.

Checked per operand against the CPU oracle, and bit for bit against bcq_gemv_plan on each operand alone
with the same K splits and the same row blocks (the same sums in the same order)."""
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


def _layers(tag, Ns, K, q, group):
    out = []
    for o, N in enumerate(Ns):
        p, codes, alpha, z, _ = make_layer(f"multi/{tag}/{o}", N, K, q, group)
        L = bq.pack_layer(N, K, q, group, bq.LAYOUT_TILED, _dev(codes), _dev(alpha), _dev(z))
        out.append((L, p, alpha, z))
    return out


@pytest.mark.parametrize("Ns,K,q,group,rb,ks", [
    ((1024, 1024, 1024), 2048, 3, 128, 6, 2),      # q / k / v of equal size
    ((2048, 512), 4096, 3, 128, 5, 4),             # a query projection and a smaller fused k/v
    ((1024, 1024), 1536, 2, 0, 4, 3),              # one scale per row
    ((520, 8, 264, 1024), 1024, 4, 128, 9, 1),     # four operands, ragged, no K split
    ((1472,), 1024, 3, 128, 1, 2),                 # a single operand is bcq_gemv
])
def test_multi_matches_oracle_and_single_products_bit_for_bit(Ns, K, q, group, rb, ks):
    layers = _layers(f"{Ns}x{K}", Ns, K, q, group)
    x = make_layer("multi/x", 8, K, q, group)[4]
    xd = _dev(x.reshape(-1))
    d = bq.desc(sum(Ns), K, q, group, bq.LAYOUT_TILED)
    plan = bq.Plan(1, rb, ks, 0)
    shares = bq.multi_row_blocks(d, plan, Ns)
    assert sum(shares) == rb and min(shares) >= 1
    ys = [torch.full((N,), float("nan"), dtype=torch.float16, device=DEV) for N in Ns]
    ws = bq.new_workspace(d, 1, plan)
    for _ in range(2):                              # the second call finds the counters as the first left them
        bq.gemv_multi(d, [L for (L, _, _, _) in layers], xd, ys, ws, plan)
    torch.cuda.synchronize()
    bq.poll_status()
    for (L, p, alpha, z), y, share in zip(layers, ys, shares):
        got = y.cpu().numpy()
        assert rel_err(got, oracle.forward_planes(p, alpha, z, x, group)[0]) <= TOL
        single = bq.Plan(1, share, ks, 0)
        y1 = torch.zeros_like(y)
        bq.gemv_plan(L.d, single, L.packed, L.alpha, L.z, xd, y1, bq.new_workspace(L.d, 1, single))
        torch.cuda.synchronize()
        assert np.array_equal(got.view(np.uint16), y1.cpu().numpy().view(np.uint16))


@pytest.mark.parametrize("Ns,K,q,group", [((7168, 7168, 7168), 7168, 3, 128), ((8192, 2048), 8192, 3, 128),
                                          ((9216, 9216, 9216), 9216, 2, 0)])
def test_multi_default_plan_at_decoder_sizes(Ns, K, q, group):
    layers = _layers(f"full/{Ns}x{K}", Ns, K, q, group)
    x = make_layer("multi/xfull", 8, K, q, group)[4]
    d = bq.desc(sum(Ns), K, q, group, bq.LAYOUT_TILED)
    ys = [torch.full((N,), float("nan"), dtype=torch.float16, device=DEV) for N in Ns]
    bq.gemv_multi(d, [L for (L, _, _, _) in layers], _dev(x.reshape(-1)), ys, bq.new_workspace(d, 1))
    torch.cuda.synchronize()
    bq.poll_status()
    for (L, p, alpha, z), y in zip(layers, ys):
        assert rel_err(y.cpu().numpy(), oracle.forward_planes(p, alpha, z, x, group)[0]) <= TOL


def test_multi_argument_checks():
    K, q, group = 1024, 3, 128
    layers = _layers("args", (512, 512), K, q, group)
    Ls = [L for (L, _, _, _) in layers]
    x = torch.zeros(K, dtype=torch.float16, device=DEV)
    ys = [torch.zeros(512, dtype=torch.float16, device=DEV) for _ in Ls]
    good = bq.desc(1024, K, q, group, bq.LAYOUT_TILED)
    for d, plan in ((bq.desc(1536, K, q, group, bq.LAYOUT_TILED), bq.Plan(1, 2, 1, 0)),     # rows do not add up
                    (good, bq.Plan(0, 2, 1, 0)), (good, bq.Plan(2, 2, 1, 0)),               # only the lookup-table kernel
                    (good, bq.Plan(1, 1, 1, 0)),                                            # fewer row blocks than operands
                    (bq.desc(1024, K, q, group, bq.LAYOUT_CANONICAL), bq.Plan(1, 2, 1, 0))):
        with pytest.raises(bq.BcqError) as e:
            bq.gemv_multi(d, Ls, x, ys, None, plan)
        assert e.value.status == bq.ERR_INVALID_ARG
    with pytest.raises(bq.BcqError) as e:                                                   # split K without a workspace
        bq.gemv_multi(good, Ls, x, ys, None, bq.Plan(1, 2, 2, 0))
    assert e.value.status == bq.ERR_INVALID_ARG
