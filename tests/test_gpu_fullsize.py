"""Parity at the full sizes of the benchmark workloads, in the launch configuration bench.py times:
bit-planes generated on the device (integer-only generator), re-laid-out by bcq_repack, default plan.
The oracle cannot run a whole 28672 x 7168 layer per test, so it recomputes a seeded sample of
output rows from inputs regenerated on the host (never from anything the CUDA path produced)."""
import numpy as np
import pytest
import torch

import oracle
from helpers import TOL
from paper_2407_02891_b200 import binding as bq
from paper_2407_02891_b200 import synth

pytestmark = pytest.mark.gpu
DEV = torch.device("cuda")

CASES = [
    # name, N, K, q, group
    ("opt30b/attn", 7168, 7168, 3, 128),
    ("opt30b/fc1", 28672, 7168, 3, 128),
    ("opt30b/fc2", 7168, 28672, 3, 128),
    ("opt30b/attn_q2", 7168, 7168, 2, 128),
    ("opt6.7b/fc1", 16384, 4096, 3, 128),
    ("opt66b/fc2_q2", 9216, 36864, 2, 128),
    ("opt66b/attn_q2_row", 9216, 9216, 2, 0),
    ("llama70b/kv", 2048, 8192, 3, 128),
    ("llama70b/down", 8192, 28672, 3, 128),
    ("llama70b/gate", 28672, 8192, 3, 128),
    ("llama70b/q", 8192, 8192, 3, 128),
    ("opt6.7b/fc2", 4096, 16384, 3, 128),
    ("opt66b/fc1_q2_row", 36864, 9216, 2, 0),        # the paper's own granularity at the largest shapes
    ("opt66b/fc2_q2_row", 9216, 36864, 2, 0),
    ("opt66b/fc1_q2", 36864, 9216, 2, 128),
]


def _build(name, N, K, q, group):
    dc = bq.desc(N, K, q, group, bq.LAYOUT_CANONICAL)
    dt = dc.with_layout(bq.LAYOUT_TILED)
    canon = synth.planes_device(name, N, K, q, DEV).reshape(-1)
    alpha, z = synth.scale_rows(name, N, K, q, group)
    ad, zd = torch.from_numpy(alpha).to(DEV), torch.from_numpy(z).to(DEV)
    packed, at, zt = bq.empty_operands(dt, DEV)
    bq.repack(dc, canon, ad, zd, dt, packed, at, zt)
    return dt, packed, at, zt, alpha, z


def _sample_rows(name, N, count=48):
    r = synth.u64(name + "/rows", 0, count) % np.uint64(N)
    rows = np.unique(np.concatenate([r.astype(np.int64), [0, N - 1]]))
    return rows


@pytest.mark.parametrize("name,N,K,q,group", CASES)
def test_fullsize_gemv_sampled_rows(name, N, K, q, group):
    dt, packed, at, zt, alpha, z = _build(name, N, K, q, group)
    x = synth.activations(name, 1, K)
    y = torch.full((N,), float("nan"), dtype=torch.float16, device=DEV)
    ws = bq.new_workspace(dt, 1)
    bq.gemv(dt, packed, at, zt, torch.from_numpy(x.reshape(-1)).to(DEV), y, ws)
    torch.cuda.synchronize()
    bq.poll_status()
    yh = y.cpu().numpy().astype(np.float64)
    assert np.isfinite(yh).all()
    rows = _sample_rows(name, N)
    p_rows = synth.plane_rows(name, N, K, q, rows)
    ref = oracle.forward_planes(p_rows, alpha[:, rows], z[rows], x, group)[0]
    # tolerance relative to the largest output of the layer (estimated from the sample: it only
    # makes the bound tighter than the one over all rows)
    assert np.abs(yh[rows] - ref).max() <= TOL * np.abs(ref).max()
    # second call on the same workspace: bit-identical (deterministic combine, counters reset)
    y2 = torch.zeros_like(y)
    bq.gemv(dt, packed, at, zt, torch.from_numpy(x.reshape(-1)).to(DEV), y2, ws)
    torch.cuda.synchronize()
    assert torch.equal(y.view(torch.int16), y2.view(torch.int16))


def test_fullsize_repack_round_trip_sampled():
    """canonical -> tiled -> canonical on a full-size layer returns the generator's bytes."""
    name, N, K, q, group = "opt30b/fc1", 28672, 7168, 3, 128
    dt, packed, at, zt, alpha, z = _build(name, N, K, q, group)
    dc = dt.with_layout(bq.LAYOUT_CANONICAL)
    back, a2, z2 = bq.empty_operands(dc, DEV)
    bq.repack(dt, packed, None, None, dc, back, a2, z2)
    torch.cuda.synchronize()
    rows = _sample_rows(name, N)
    got = back.view(q, N, K // 8)[:, torch.from_numpy(rows).to(DEV)].cpu().numpy()
    assert np.array_equal(got, synth.plane_rows(name, N, K, q, rows))
    assert np.array_equal(a2.view(q, N, -1).cpu().numpy().view(np.uint16), alpha.view(np.uint16))
    assert np.array_equal(z2.view(N, -1).cpu().numpy().view(np.uint16), z.view(np.uint16))


@pytest.mark.parametrize("name,N,K,B", [
    ("llama70b/kv", 2048, 8192, 2), ("llama70b/kv", 2048, 8192, 16),
    ("llama70b/gate", 28672, 8192, 2), ("llama70b/gate", 28672, 8192, 3), ("llama70b/gate", 28672, 8192, 4),
    ("llama70b/gate", 28672, 8192, 8), ("llama70b/gate", 28672, 8192, 16),
    ("llama70b/down", 8192, 28672, 4), ("llama70b/down", 8192, 28672, 9),
    ("llama70b/q", 8192, 8192, 8),
])
def test_fullsize_smallbatch_sampled_rows(name, N, K, B):
    """Every small-batch path at the sizes of the Llama-2-70B-shaped layer: column pairs through the
    lookup-table kernel (B = 2, 3), the tensor-core kernel with one and with two MMAs per step (B <= 8, B > 8)."""
    q, group = 3, 128
    dt, packed, at, zt, alpha, z = _build(name, N, K, q, group)
    X = synth.activations(name, B, K)
    Y = torch.full((B, N), float("nan"), dtype=torch.float16, device=DEV)
    bq.gemm_smallbatch(dt, packed, at, zt, torch.from_numpy(X).to(DEV), Y, B, bq.new_workspace(dt, B))
    torch.cuda.synchronize()
    bq.poll_status()
    Yh = Y.cpu().numpy().astype(np.float64)
    assert np.isfinite(Yh).all()
    rows = _sample_rows(name, N)
    ref = oracle.forward_planes(synth.plane_rows(name, N, K, q, rows), alpha[:, rows], z[rows], X, group)
    assert np.abs(Yh[:, rows] - ref).max() <= TOL * np.abs(ref).max()
