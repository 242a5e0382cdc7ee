"""Pins for the oracle's moments, casts, curvature signal and mask (CPU only)."""
from fractions import Fraction

import numpy as np
import pytest
import torch

from oracle import oracle as orc


# ---------------------------------------------------------------- moments (Sec. 3.1, Var[grad])

@pytest.mark.parametrize("n", [1, 2, 3, 31, 32, 33, 1000])
def test_moments_exact_rational_brute_force(n):
    rng = np.random.default_rng(n)
    x = (rng.standard_normal(n) * 1e-3 + 0.25).astype(np.float32)   # mean far from zero: cancellation case
    fx = [Fraction(float(v)) for v in x]
    mu = sum(fx) / n
    var = sum((v - mu) ** 2 for v in fx) / n
    m, v = orc.moments(x)
    assert m == pytest.approx(float(mu), rel=1e-13, abs=0)
    if n == 1:
        assert v == 0.0
    else:
        assert v == pytest.approx(float(var), rel=1e-9, abs=0)


def test_moments_constant_and_scaling():
    m, v = orc.moments(np.full(777, 0.3, dtype=np.float32))
    assert v == 0.0 and m == float(np.float32(0.3))
    x = np.random.default_rng(0).standard_normal(5000).astype(np.float32)
    m1, v1 = orc.moments(x)
    m2, v2 = orc.moments(x * np.float32(8.0))
    assert m2 == 8.0 * m1 and v2 == 64.0 * v1          # exact for a power-of-two factor
    # population form: two values +-a give exactly a^2
    assert orc.moments(np.array([0.5, -0.5], dtype=np.float32)) == (0.0, 0.25)


# ---------------------------------------------------------------- casts (round to nearest even)

def _rounding_classes():
    # every pattern of the upper 24 bits with the low byte in {00, 01, ff}: the low byte only
    # ever acts as a sticky bit for both 16-bit targets, so this covers every rounding case
    hi = np.arange(1 << 24, dtype=np.uint32) << np.uint32(8)
    return [hi | np.uint32(lo) for lo in (0x00, 0x01, 0xFF)]


def test_cast_bf16_against_torch_all_rounding_classes():
    for bits in _rounding_classes():
        x = bits.view(np.float32)
        got = orc.cast(x, to_bf16=True)
        ref = torch.from_numpy(x.copy()).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
        nan = np.isnan(x)
        assert np.array_equal(got[~nan], ref[~nan])
        assert np.all((got[nan] & 0x7F80) == 0x7F80) and np.all((got[nan] & 0x007F) != 0)


def test_cast_f16_against_numpy_all_rounding_classes():
    for bits in _rounding_classes():
        x = bits.view(np.float32)
        got = orc.cast(x, to_bf16=False)
        with np.errstate(over="ignore"):
            ref = x.astype(np.float16).view(np.uint16)
        nan = np.isnan(x)
        assert np.array_equal(got[~nan], ref[~nan])
        assert np.all((got[nan] & 0x7C00) == 0x7C00) and np.all((got[nan] & 0x03FF) != 0)


def test_cast_f16_named_cases():
    def h(v):
        return int(orc.cast(np.array([v], dtype=np.float32), to_bf16=False)[0])
    assert h(65504.0) == 0x7BFF and h(65519.99) == 0x7BFF and h(65520.0) == 0x7C00   # overflow to inf, no saturation
    assert h(2.0 ** -24) == 0x0001 and h(2.0 ** -25) == 0x0000 and h(np.float32(2.0 ** -25) * np.float32(1.0000001)) == 0x0001
    assert h(-0.0) == 0x8000 and h(1.0) == 0x3C00
    assert h(1.0 + 2.0 ** -11) == 0x3C00 and h(1.0 + 3 * 2.0 ** -11) == 0x3C02      # ties to even


# ---------------------------------------------------------------- Hutchinson signal

@pytest.mark.parametrize("P", [1, 2, 4, 8])
def test_diagonal_hessian_recovered_exactly(P):
    # Hz = D*z  =>  sum_p z*Hz = P*D exactly (z*z = 1, pairwise sums of equal terms are exact)
    n_total, off, n = 10000, 136, 9000
    rng = np.random.default_rng(P)
    D = np.exp(rng.uniform(np.log(1e-5), 0.0, n_total)).astype(np.float32)
    hz = np.concatenate([D * orc.probe(11, 5, p, 0, n_total) for p in range(P)])
    a = orc.hutchinson_abs(hz, n_total, P, 11, 5, off, n)
    assert np.array_equal(a / np.float32(P), D[off:off + n])


def test_dense_symmetric_hessian_probe_products():
    # dense H on a tiny layer: the oracle's sum_p z_i (Hz)_i against a float64 recomputation;
    # a transposed probe stride, a wrong sign or an index slip all fail here
    n, P = 12, 8
    rng = np.random.default_rng(3)
    A = rng.standard_normal((n, n))
    H = (A + A.T) / 2
    zs = [orc.probe(9, 2, p, 0, n).astype(np.float64) for p in range(P)]
    hz = np.concatenate([(H @ z).astype(np.float32) for z in zs])
    a = orc.hutchinson_abs(hz, n, P, 9, 2, 0, n)
    ref = np.abs(sum(z * (H @ z).astype(np.float32).astype(np.float64) for z in zs))
    assert np.allclose(a, ref, rtol=1e-6, atol=1e-6)


def test_hutchinson_mean_converges_to_diagonal():
    # E_z[z * (Hz)] = diag(H): many steps' probes on a dense symmetric H
    n, T = 8, 4000
    rng = np.random.default_rng(4)
    A = rng.standard_normal((n, n))
    H = (A + A.T) / 2
    acc = np.zeros(n)
    for t in range(1, T + 1):
        z = orc.probe(1, t, 0, 0, n).astype(np.float64)
        acc += z * (H @ z)
    off_diag_sd = np.sqrt((H ** 2).sum(1) - np.diag(H) ** 2)
    assert np.all(np.abs(acc / T - np.diag(H)) <= 5 * off_diag_sd / np.sqrt(T))


def test_pairwise_order_of_probe_sum():
    # four probes with magnitudes chosen so that ((a+b)+(c+d)) differs from left-to-right in float
    n_total, P = 8, 4
    mags = np.array([1.0, 2.0 ** -24, 2.0 ** -24, 2.0 ** -24], dtype=np.float32)
    hz = np.concatenate([mags[p] * orc.probe(0, 1, p, 0, n_total) for p in range(P)])
    a = orc.hutchinson_abs(hz, n_total, P, 0, 1, 0, n_total)
    f = np.float32
    tree = f(f(mags[0] + mags[1]) + f(mags[2] + mags[3]))
    serial = f(f(f(mags[0] + mags[1]) + mags[2]) + mags[3])
    assert tree != serial
    assert np.all(a == tree)


# ---------------------------------------------------------------- mask

def _run_mask(a_layers, ppm, P=1, gaps=3):
    """Builds Hz = a*z so that |S| = a, runs one oracle step, returns (oracle, table)."""
    table, off = [], gaps
    for a in a_layers:
        table.append((off, len(a)))
        off += len(a) + gaps
    n_total = (off + 7) // 8 * 8
    hz1 = np.zeros(n_total, dtype=np.float32)
    for (o, n), a in zip(table, a_layers):
        hz1[o:o + n] = a
    hz = np.concatenate([hz1 * orc.probe(2, 1, p, 0, n_total) for p in range(P)])
    o = orc.Oracle(table, n_total, topk_ppm=ppm, num_probes=P)
    w = np.zeros(n_total, dtype=np.float32)
    g = np.zeros(n_total, dtype=np.float32)
    c = np.zeros(n_total, dtype=np.uint16)
    assert o.step(w, g, hz, c, 2, 1) is False
    return o, table, n_total


def _bits(mask, off, n):
    idx = np.arange(off, off + n)
    return (mask[idx >> 5] >> (idx & 31).astype(np.uint32)) & 1


@pytest.mark.parametrize("ppm", [1, 100000, 333333, 999999])
def test_mask_matches_full_sort(ppm):
    rng = np.random.default_rng(ppm)
    layers = [np.exp(rng.uniform(-10, 0, n)).astype(np.float32) for n in [1, 2, 7, 64, 1000, 4097]]
    layers[4][::7] = layers[4][3]          # plant ties around the threshold
    o, table, n_total = _run_mask(layers, ppm)
    mask = o.mask()
    assert int(sum(bin(int(x)).count("1") for x in mask)) == sum(int(ly.k) for ly in o.layers())
    for (off, n), a, ly in zip(table, layers, o.layers()):
        k = max(1, (n * ppm + 999999) // 1000000)
        assert ly.k == k
        order = np.lexsort((np.arange(n), -a.astype(np.float64)))   # value descending, index ascending
        want = np.zeros(n, dtype=np.uint32)
        want[order[:k]] = 1
        got = _bits(mask, off, n)
        assert np.array_equal(got, want)
        assert ly.topk_threshold == a[order[k - 1]]
        assert a[got == 1].min() >= ly.topk_threshold >= (a[got == 0].max() if k < n else 0)
        assert ly.lambda_max == a.max()
        assert ly.topk_mass == pytest.approx(a[got == 1].astype(np.float64).sum() / a.astype(np.float64).sum(), rel=1e-12)


def test_mask_all_equal_layer_takes_lowest_indices():
    o, table, _ = _run_mask([np.full(100, 0.5, dtype=np.float32)], 250000)
    (off, n), = table
    assert np.array_equal(_bits(o.mask(), off, n), (np.arange(n) < 25).astype(np.uint32))


def test_mask_dense_is_all_ones_and_gaps_stay_zero():
    rng = np.random.default_rng(0)
    layers = [rng.uniform(0.1, 1, n).astype(np.float32) for n in [5, 70, 33]]
    o, table, n_total = _run_mask(layers, 1000000, P=4)
    mask = o.mask()
    inside = np.zeros(n_total, dtype=bool)
    for (off, n), a, ly in zip(table, layers, o.layers()):
        inside[off:off + n] = True
        assert ly.k == n and ly.topk_mass == 1.0
        assert ly.topk_threshold == np.float32(4) * a.min()          # k-th largest of |S| = P*a
        assert ly.lambda_max == a.max()                              # max|S| / P
    assert np.array_equal(_bits(mask, 0, n_total).astype(bool), inside)


# ---------------------------------------------------------------- power iteration (Sec. 3.2)

def _sym_blocks(sizes, seed):
    rng = np.random.default_rng(seed)
    table, off, mats = [], 3, []
    for n in sizes:
        A = rng.standard_normal((n, n))
        # well separated spectrum so that a few dozen iterations converge
        Q, _ = np.linalg.qr(A)
        ev = np.concatenate([[10.0, -7.0, 4.0], rng.uniform(-1, 1, max(0, n - 3))])[:n]
        mats.append((Q * ev) @ Q.T)
        table.append((off, n))
        off += n + 5
    return table, (off + 7) // 8 * 8, mats


def _apply(table, mats, u):
    hu = np.zeros_like(u)
    for (off, n), H in zip(table, mats):
        hu[off:off + n] = (H @ u[off:off + n].astype(np.float64)).astype(np.float32)
    return hu


def test_power_iteration_finds_top_eigenvalues_with_deflation():
    table, n_total, mats = _sym_blocks([6, 17, 40], seed=1)
    rng = np.random.default_rng(2)
    L = len(table)
    found_v, found_lam = [], []
    for k in range(3):                                   # top-3 by magnitude, one after the other
        u = rng.standard_normal(n_total).astype(np.float32)
        v = np.stack(found_v) if found_v else None
        lam_v = np.stack(found_lam) if found_lam else None
        for _ in range(200):
            u, lam, nrm = orc.power_iterate(table, n_total, u, _apply(table, mats, u), v, lam_v)
        found_v.append(u.copy())
        found_lam.append(lam.copy())
        for l, ((off, n), H) in enumerate(zip(table, mats)):
            ev = np.linalg.eigvalsh(H)
            want = sorted(ev, key=abs, reverse=True)[k]
            assert lam[l] == pytest.approx(want, rel=1e-4), (k, l)
            assert np.linalg.norm(u[off:off + n]) == pytest.approx(1.0, rel=1e-5)
            assert nrm[l] == pytest.approx(abs(want), rel=1e-3)


def test_power_iteration_rayleigh_quotient_closed_form():
    # an exact eigenvector gives its eigenvalue; H = diag(d) and u = e_i make every quantity exact
    n = 16
    d = np.arange(1, n + 1, dtype=np.float32)
    u = np.zeros(n, dtype=np.float32); u[4] = 2.0
    out, lam, nrm = orc.power_iterate([(0, n)], n, u, d * u)
    assert lam[0] == 5.0 and nrm[0] == 10.0 and out[4] == 1.0 and np.count_nonzero(out) == 1
    # general u: float64 recomputation
    rng = np.random.default_rng(0)
    u = rng.standard_normal(n).astype(np.float32)
    hu = (d * u).astype(np.float32)
    out, lam, nrm = orc.power_iterate([(0, n)], n, u, hu)
    assert lam[0] == pytest.approx(float((u.astype(np.float64) * hu).sum() / (u.astype(np.float64) ** 2).sum()), rel=1e-6)
    assert np.allclose(out, hu / np.linalg.norm(hu.astype(np.float64)), rtol=1e-6)
    # zero vector: defined as zeros
    out, lam, nrm = orc.power_iterate([(0, n)], n, np.zeros(n, dtype=np.float32), np.zeros(n, dtype=np.float32))
    assert lam[0] == 0.0 and nrm[0] == 0.0 and not out.any()
