"""Shared test helpers: synthetic layers as numpy arrays, and the tiled layout restated from
the documentation in include/bcq.h (numpy index arithmetic, independent of the library)."""
import numpy as np

from paper_2407_02891_b200 import synth

TOL = 5e-3   # max|y_gpu - y_ref| <= TOL * max|y_ref|  (fp16 I/O, fp32 accumulation)


def make_layer(name, N, K, q, group, B=1):
    """Canonical numpy operands of a synthetic layer: planes, codes, alpha, z, x."""
    p = synth.planes(name, N, K, q)
    alpha, z = synth.scale_rows(name, N, K, q, group)
    x = synth.activations(name, B, K)
    return p, synth.codes_from_planes(p), alpha, z, x


def tile_step(sub, j, cc):
    """Byte position s (0..15) in a lane's 16 bytes of a plane at which row j of a unit finds chunk cc of its
    128-weight segment, as the layout comment of include/bcq.h states it.  sub = scaling units per segment
    (1 for groups of 128 and for one scale per row, 2 for groups of 64, 4 for groups of 32)."""
    if sub <= 1:
        return (cc - 2 * j) % 16
    cps, wps = 16 // sub, 8 // sub                     # chunks / 4-byte table columns per scaling unit
    col = cc // 2
    sg, cw = col // wps, col % wps                      # the unit of the chunk, its column inside the unit
    ph = (sg - j // wps) % sub                          # the phase in which row j walks that unit
    th = (cw - j % wps) % wps
    return ph * cps + 2 * th + cc % 2


def tiled_operands(planes, alpha, z, group):
    """canonical planes uint8 [q,N,K/8], alpha f16 [q,N,G], z f16 [N,G] -> (packed bytes, alpha, z) of
    the tiled layout, per the layout comment of include/bcq.h.  alpha and z come back as None when
    the scales live inside the tiles (groups of 128, 64, 32)."""
    q, N, KB = planes.shape
    U, W = N // 8, KB // 64
    sub = 128 // group if group else 0
    T = q * 512 + sub * (q + 1) * 64
    out = np.zeros(U * W * T, np.uint8)
    i, n, kb = np.meshgrid(np.arange(q), np.arange(N), np.arange(KB), indexing="ij")
    w, c = kb // 64, kb % 64
    g, cc = c // 16, c % 16
    u, j = n // 8, n % 8
    s = tile_step(sub, j, cc)
    lane = 8 * g + j
    off = (w * U + u) * T + i * 512 + lane * 16 + s
    out[off.ravel()] = planes.ravel()
    G = alpha.shape[2]
    i, n, g = np.meshgrid(np.arange(q), np.arange(N), np.arange(G), indexing="ij")
    u, r = n // 8, n % 8
    if group == 0:
        a_out = np.empty(alpha.size, alpha.dtype)
        z_out = np.empty(z.size, z.dtype)
        a_out[((u * q + i) * 8 + r).ravel()] = alpha.ravel()
        z_out[(u[0] * 8 + r[0]).ravel()] = z.ravel()
        return out, a_out, z_out
    # scales of a lane: [phase][alpha_0 .. alpha_{q-1}, z]; the phase-th set belongs to the unit the lane walks then
    w, gi, sg = g // (4 * sub), (g % (4 * sub)) // sub, g % sub
    ph = (sg - r // (8 // sub)) % sub if sub > 1 else 0 * sg
    lane = 8 * gi + r
    a_off = (w * U + u) * T + q * 512 + 2 * ((lane * sub + ph) * (q + 1) + i)
    z_off = (w[0] * U + u[0]) * T + q * 512 + 2 * ((lane[0] * sub + ph[0]) * (q + 1) + q)
    ab = alpha.view(np.uint8).reshape(q, N, G, 2)
    zb = z.view(np.uint8).reshape(N, G, 2)
    for byte in range(2):
        out[(a_off + byte).ravel()] = ab[..., byte].ravel()
        out[(z_off + byte).ravel()] = zb[..., byte].ravel()
    return out, None, None


def rel_err(y_gpu, y_ref):
    y_ref = np.asarray(y_ref, np.float64)
    return float(np.abs(np.asarray(y_gpu, np.float64) - y_ref).max() / np.abs(y_ref).max())


def lut_max_units(q, group, B=1):
    """Row units (8 rows) one block of the lookup-table kernel takes, as include/bcq.h states the limit:
    184, or 160 for q = 4 when two columns share a launch (group 128 with B >= 2)."""
    return 160 if (q == 4 and group != 0 and B >= 2) else 184
