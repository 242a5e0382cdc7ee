"""GPU-vs-oracle parity of the power-iteration support sweeps (Sec. 3.2), through the C ABI."""
import numpy as np
import pytest
import torch

import paper_2508_16905_b200 as ta
from oracle import oracle as orc

pytestmark = pytest.mark.gpu


def _table():
    lengths = [1, 33, 129, 4097, 70001, 250000]
    table, off = [], 3
    for j, n in enumerate(lengths):
        off += (0, 5, 1, 7)[j % 4]
        table.append((off, n))
        off += n
    return table, (off + 7) // 4 * 4


def _check(table, got_u, got_lam, got_nrm, ref_u, ref_lam, ref_nrm):
    assert np.allclose(got_lam, ref_lam, rtol=1e-5, atol=1e-30)
    assert np.allclose(got_nrm, ref_nrm, rtol=1e-5, atol=1e-30)
    for off, n in table:
        scale = float(np.abs(ref_u[off:off + n]).max())
        assert np.abs(got_u[off:off + n] - ref_u[off:off + n]).max() <= 1e-5 * scale + 1e-30


@pytest.mark.parametrize("m", [0, 1, 5])
def test_power_iterate_matches_oracle(m):
    table, n_total = _table()
    L = len(table)
    rng = np.random.default_rng(m)
    u = rng.standard_normal(n_total).astype(np.float32)
    d = np.exp(rng.uniform(-3, 1, n_total)).astype(np.float32)
    hu = (d * u + 0.1 * np.roll(u, 1)).astype(np.float32)
    v = lam_v = None
    if m:
        v = rng.standard_normal((m, n_total)).astype(np.float32)
        for off, n in table:                                    # unit vectors per layer
            v[:, off:off + n] /= np.maximum(np.linalg.norm(v[:, off:off + n], axis=1, keepdims=True), 1e-30)
        lam_v = rng.uniform(0.5, 3.0, (m, L)).astype(np.float32)
    ref_u, ref_lam, ref_nrm = orc.power_iterate(table, n_total, u, hu, v, lam_v)

    h = ta.ta_create(table, n_total)
    dev = lambda a: torch.from_numpy(a).cuda() if a is not None else None
    out = torch.full((n_total,), 7.0, device="cuda")
    lam = torch.zeros(L, device="cuda")
    nrm = torch.zeros(L, device="cuda")
    ta.ta_power_iterate(h, dev(u), dev(hu), dev(v), dev(lam_v), m, out, lam, nrm)
    got = out.cpu().numpy()
    _check(table, got, lam.cpu().numpy(), nrm.cpu().numpy(), ref_u, ref_lam, ref_nrm)
    inside = np.zeros(n_total, dtype=bool)
    for off, n in table:
        inside[off:off + n] = True
    assert np.all(got[~inside] == 7.0)                          # gaps are never written
    # twice the same call: bit-identical (fixed summation order)
    out2, lam2 = torch.empty_like(out), torch.empty_like(lam)
    ta.ta_power_iterate(h, dev(u), dev(hu), dev(v), dev(lam_v), m, out2, lam2, None)
    assert torch.equal(out2[torch.from_numpy(inside).cuda()], out[torch.from_numpy(inside).cuda()]) and torch.equal(lam, lam2)


def test_power_iteration_converges_and_feeds_the_step_size():
    # H = diag(D): the top eigenvalue of each layer is max D; feed it to the optimizer pass as lambda_l
    table, n_total = [(0, 5000), (5000, 300)], 5304
    rng = np.random.default_rng(3)
    D = rng.uniform(0.1, 1.0, n_total).astype(np.float32)
    D[17], D[5100] = 3.0, 2.0
    Dd = torch.from_numpy(D).cuda()
    h = ta.ta_create(table, n_total, alpha=1.0, eta0=0.5)
    u = torch.from_numpy(rng.standard_normal(n_total).astype(np.float32)).cuda()
    lam = torch.zeros(2, device="cuda")
    for _ in range(60):
        ta.ta_power_iterate(h, u, Dd * u, None, None, 0, u, lam, None)
    assert lam.cpu().numpy() == pytest.approx([3.0, 2.0], rel=1e-4)
    ta.ta_set_curvature(h, lam.cpu().numpy())
    w = torch.zeros(n_total, device="cuda")
    c = torch.zeros(n_total, dtype=torch.int16, device="cuda")
    ta.ta_step(h, w, torch.ones(n_total, device="cuda"), None, c, 0, 1)
    stats, _ = ta.ta_stats(h)
    for s, l in zip(stats, lam.cpu().numpy()):
        assert s.lambda_max == l and s.eta_scale == np.float32(1) / (np.float32(1) + np.float32(l))
    assert float(w[0]) == pytest.approx(-0.5 / (1 + float(lam[0])), rel=1e-6)
