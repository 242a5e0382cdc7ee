"""Size limits and odd tables on the GPU: index arithmetic beyond 2^31, thousands of tiny layers."""
import numpy as np
import pytest
import torch

import paper_2508_16905_b200 as ta
from oracle import oracle as orc
from tests.parity import ParityRun, oracle_hz

pytestmark = pytest.mark.gpu


def test_layer_longer_than_two_to_the_31():
    # one layer of 2^31 + 4099 elements behind a small one: every flat index above 2^31 must be reached once.
    # Checked through closed forms (the oracle would need minutes): g = +a on even, -a on odd flat indices.
    n_big = (1 << 31) + 4099
    table = [(8, 1000), (1016, n_big)]
    n_total = (1016 + n_big + 7) // 8 * 8
    a = 2.0 ** -10
    h = ta.ta_create(table, n_total, beta=0.0, tau_low=1.0, tau_high=2.0, tau_curv=10.0, alpha=0.0, eta0=0.5)   # everything FP16
    w = torch.zeros(n_total, device="cuda")
    g = torch.empty(n_total, device="cuda")
    g[0::2] = a
    g[1::2] = -a
    c = torch.full((n_total,), 0x5A5A, dtype=torch.int16, device="cuda")
    hz = torch.ones(n_total, device="cuda")
    hz[n_total - 9] = 3.0                                  # the layer's largest |S| sits in its last vector
    ta.ta_step(h, w, g, hz, c, 0, 1)
    stats, status = ta.ta_stats(h)
    assert status.skipped == 0
    s = stats[1]
    mean = (a / n_big) if n_big % 2 else 0.0               # odd count: one unpaired element (the layer starts on an even index: +a)
    assert s.grad_mean == pytest.approx(mean, abs=1e-12)
    assert s.grad_var == pytest.approx(a * a - mean * mean, rel=1e-6)
    assert s.lambda_max == 3.0 and s.topk_threshold == 1.0 and s.code == ta.TA_CODE_FP16
    # w = -eta * g exactly; check the head, the tail beyond 2^31 and the gap
    for lo, hi in [(1016, 1016 + 4096), (n_total - 8192, 1016 + n_big)]:
        assert torch.equal(w[lo:hi], -0.5 * g[lo:hi])
        want = (-0.5 * g[lo:hi]).to(torch.float16).view(torch.int16)
        assert torch.equal(c[lo:hi], want)
    assert float(w[1008:1016].abs().max()) == 0.0 and bool((c[1008:1016] == 0x5A5A).all())
    assert float(w[1016 + n_big:].abs().max()) == 0.0
    # every element was updated exactly once: the sum of |w| is n * eta * a (exact in float64)
    total = float(w[1016:1016 + n_big].abs().sum(dtype=torch.float64))
    assert total == pytest.approx(n_big * 0.5 * a, rel=1e-12)


@pytest.mark.parametrize("ppm,P", [(1000000, 1), (300000, 2)])
def test_thousands_of_tiny_layers(ppm, P):
    # more layers than the one-launch path keeps in shared memory: the three-kernel path with a ragged table
    rng = np.random.default_rng(P)
    lengths = rng.integers(1, 40, 6000).tolist() + [5000, 70000]
    table, off = [], 1
    for j, n in enumerate(lengths):
        off += int(j % 3 == 0)
        table.append((off, int(n)))
        off += int(n)
    n_total = (off + 7) // 4 * 4
    hp = dict(beta=0.5, tau_low=3e-7, tau_high=3e-6, tau_curv=0.5, topk_ppm=ppm, num_probes=P)
    run = ParityRun(table, n_total, hp, torch.from_numpy((rng.standard_normal(n_total) * 0.05).astype(np.float32)))
    D = np.exp(rng.uniform(np.log(1e-3), 0.0, n_total)).astype(np.float32)
    for t in (1, 2):
        g = torch.from_numpy((rng.standard_normal(n_total) * 1e-3).astype(np.float32)).cuda()
        run.step(t, g, oracle_hz(D, P, 5, t), 5)


def test_hundred_thousand_tiny_layers_one_launch():
    # dense, so the one-launch path: with 120,000 layers of one to three elements a block of its grid touches
    # several hundred layers (more than it has threads) and a warp walks dozens of runs
    from paper_2508_16905_b200 import binding as B
    rng = np.random.default_rng(11)
    lengths = rng.integers(1, 4, 120000).tolist()
    table, off = [], 2
    for j, n in enumerate(lengths):
        off += int(j % 5 == 0)
        table.append((off, int(n)))
        off += int(n)
    n_total = (off + 7) // 4 * 4
    runs, used, max_rows = B.ta_plan_one_launch(table, 148 * 24)
    per_block = {}
    for _, _, layer, warp in runs:
        per_block.setdefault(warp // 8, set()).add(layer)
    assert max(len(v) for v in per_block.values()) > 256
    hp = dict(beta=0.5, tau_low=3e-7, tau_high=3e-6, tau_curv=0.5, num_probes=1)
    run = ParityRun(table, n_total, hp, torch.from_numpy((rng.standard_normal(n_total) * 0.05).astype(np.float32)))
    D = np.exp(rng.uniform(np.log(1e-3), 0.0, n_total)).astype(np.float32)
    for t in (1, 2, 3):
        g = torch.from_numpy((rng.standard_normal(n_total) * 1e-3).astype(np.float32)).cuda()
        run.step(t, g, oracle_hz(D, 1, 5, t) if t != 2 else None, 5)
    if ta.ta_path(run.h) != "two dependent launches":
        pytest.skip("this device's grid sent the table to the three-kernel path")


@pytest.mark.parametrize("seed", range(40))
def test_random_tables(seed):
    # random tables, gaps, probe counts, mask fractions and gradient types: planner and kernels against the oracle
    rng = np.random.default_rng(1000 + seed)
    L = int(rng.integers(1, 40))
    lengths = [int(rng.integers(1, 300)) if rng.random() < 0.7 else int(rng.integers(300, 30000)) for _ in range(L)]
    table, off = [], int(rng.integers(0, 9))
    for n in lengths:
        off += int(rng.integers(0, 4)) * int(rng.random() < 0.5)
        table.append((off, n))
        off += n
    n_total = (off + int(rng.integers(0, 9)) + 3) // 4 * 4
    P = int(rng.choice([1, 2, 4, 8]))
    ppm = 1000000 if rng.random() < 0.4 else int(rng.integers(1, 999999))
    grad_dtype = "bf16" if rng.random() < 0.4 else "f32"
    hp = dict(beta=float(rng.choice([0.0, 0.5, 0.9])), tau_low=3e-7, tau_high=3e-6, tau_curv=0.5, alpha=float(rng.choice([0.0, 1.0, 3.0])),
              eta0=0.05, topk_ppm=ppm, num_probes=P, t_ctrl=int(rng.choice([1, 2])), grad_dtype=grad_dtype,
              momentum=float(rng.choice([0.0, 0.0, 0.9])), weight_decay=float(rng.choice([0.0, 0.0, 1e-3])))
    run = ParityRun(table, n_total, hp, torch.from_numpy((rng.standard_normal(n_total) * 0.05).astype(np.float32)))
    D = np.exp(rng.uniform(np.log(1e-4), 0.5, n_total)).astype(np.float32)
    if rng.random() < 0.5:
        D = np.round(D * 8) / 8 + np.float32(0.125)          # few distinct values: many ties at the threshold
    sigma = 10.0 ** rng.uniform(-4.5, -2.0, L)
    for t in (1, 2, 3):
        g = np.zeros(n_total, dtype=np.float32)
        for (o, n), s in zip(table, sigma):
            g[o:o + n] = rng.standard_normal(n) * s
        g_dev = torch.from_numpy(g).cuda()
        if grad_dtype == "bf16":
            g_dev = g_dev.to(torch.bfloat16)
        run.step(t, g_dev, oracle_hz(D, P, seed, t) if t != 2 else None, seed)


@pytest.mark.parametrize("seed", range(16))
def test_random_tables_with_large_layers_and_drifting_curvature(seed):
    # layers up to 700,000 elements; curvature that stays, drifts by a few per cent, is absent on a step and jumps by
    # a factor of eight; inputs with few distinct values, with exact zeros (pruned weights) or with every value equal:
    # the sweep's window of bins, its candidate lists, the second sweep and the resolve step against the oracle
    rng = np.random.default_rng(5000 + seed)
    L = int(rng.integers(1, 12))
    lengths = []
    for _ in range(L):
        r = rng.random()
        lengths.append(int(rng.integers(1, 300)) if r < 0.3 else int(rng.integers(300, 30000)) if r < 0.7 else int(rng.integers(30000, 700000)))
    table, off = [], int(rng.integers(0, 9))
    for n in lengths:
        off += int(rng.integers(0, 4)) * int(rng.random() < 0.5)
        table.append((off, n))
        off += n
    n_total = (off + int(rng.integers(0, 9)) + 3) // 4 * 4
    P = int(rng.choice([1, 2, 4, 8]))
    ppm = int(rng.choice([1000, 100000, 500000, 900000])) if rng.random() < 0.8 else 1000000
    grad_dtype = "bf16" if rng.random() < 0.4 else "f32"
    hp = dict(beta=0.9, tau_low=3e-7, tau_high=3e-6, tau_curv=0.5, alpha=1.0, eta0=0.05, topk_ppm=ppm, num_probes=P,
              t_ctrl=int(rng.choice([1, 2])), grad_dtype=grad_dtype)
    run = ParityRun(table, n_total, hp, torch.from_numpy((rng.standard_normal(n_total) * 0.05).astype(np.float32)))
    D0 = np.exp(rng.uniform(np.log(1e-4), 0.5, n_total)).astype(np.float32)
    mode = int(rng.integers(0, 4))
    if mode == 1:
        D0 = np.round(D0 * 8) / 8 + np.float32(0.125)
    elif mode == 2:
        D0[rng.random(n_total) < 0.6] = 0.0
    elif mode == 3:
        D0[:] = np.float32(0.5)
    sigma = 10.0 ** rng.uniform(-4.5, -2.0, L)
    for t, f in enumerate([1.0, 1.02, None, 0.97, 8.0, 1.0], start=1):
        g = np.zeros(n_total, dtype=np.float32)
        for (o, n), s in zip(table, sigma):
            g[o:o + n] = rng.standard_normal(n) * s
        g_dev = torch.from_numpy(g).cuda()
        if grad_dtype == "bf16":
            g_dev = g_dev.to(torch.bfloat16)
        run.step(t, g_dev, oracle_hz(D0 * np.float32(f), P, seed, t) if f is not None else None, seed)
