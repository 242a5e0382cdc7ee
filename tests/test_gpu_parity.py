"""GPU-vs-oracle parity of the fused optimizer pass, through the C ABI (needs a B200)."""
import numpy as np
import pytest
import torch

import paper_2508_16905_b200 as ta
from paper_2508_16905_b200 import workloads as W
from oracle import oracle as orc
from tests.parity import ParityRun, oracle_hz, to_host_bits, ulp_f32, ulp_16

pytestmark = pytest.mark.gpu


def run_workload(wl, steps, hz_every=1, layers=None, check_every=1, threads=1):
    w0 = W.make_weights(wl, "cuda")
    D = W.make_curvature(wl, "cuda").cpu().numpy()
    run = ParityRun(wl.table, wl.n_total, wl.hparams(), w0, layers=layers, threads=threads)
    for t in range(1, steps + 1):
        g = W.make_grads(wl, t, "cuda")
        hz = oracle_hz(D, wl.num_probes, wl.probe_seed, t) if (t - 1) % hz_every == 0 else None
        run.step(t, g, hz, wl.probe_seed, check=(t % check_every == 0 or t == steps))
    run.report(wl.name)
    return run


# ---------------------------------------------------------------- probes

@pytest.mark.parametrize("seed,t,p", [(0, 1, 0), (0xDEADBEEFCAFE, 77, 3), (2 ** 63 + 5, 2 ** 32 - 1, 7)])
def test_probe_bits_match_oracle(seed, t, p):
    n_total = 3 * 4096 + 520
    h = ta.ta_create([(0, n_total)], n_total, num_probes=8)
    z = torch.empty(n_total, device="cuda")
    ta.ta_probe(h, seed, t, p, z)
    assert np.array_equal(z.cpu().numpy(), orc.probe(seed, t, p, 0, n_total))


# ---------------------------------------------------------------- the five configurations

def test_mlp_tiny_all_steps():
    wl = W.get("mlp_tiny")
    run = run_workload(wl, wl.steps)
    codes = set(int(c) for c in run.o.codes())
    assert len(codes) >= 2            # the thresholds of this configuration separate the layers


def test_mlp_tiny_unpadded_offsets():
    run_workload(W.get("mlp_tiny", align=1), 4)


def test_resnet18_cifar_all_steps():
    wl = W.get("resnet18_cifar")
    run = run_workload(wl, wl.steps, check_every=10, threads=8)
    assert set(int(c) for c in run.o.codes()) == {0, 1, 2}    # FP16, BF16 and FP32 layers all occur


def test_efficientnet_b0_all_steps():
    wl = W.get("efficientnet_b0_cifar")
    run_workload(wl, wl.steps, check_every=10, threads=8)


@pytest.mark.parametrize("name", ["mlp_tiny", "efficientnet_b0_cifar", "resnet18_cifar"])
def test_small_models_as_one_cooperative_launch(name):
    wl = W.get(name)
    w0 = W.make_weights(wl, "cuda")
    D = W.make_curvature(wl, "cuda").cpu().numpy()
    run = ParityRun(wl.table, wl.n_total, dict(wl.hparams(), flags=ta.TA_FLAG_COOPERATIVE_LAUNCH), w0, threads=8)
    for t in range(1, 6):
        run.step(t, W.make_grads(wl, t, "cuda"), oracle_hz(D, 1, wl.probe_seed, t) if t != 3 else None, wl.probe_seed)
    assert ta.ta_path(run.h) == "one cooperative launch" and ta.ta_launch_count(run.h) == 5


def test_efficientnet_b0_unpadded_offsets():
    run_workload(W.get("efficientnet_b0_cifar", align=1), 3)


def test_resnet50_topk_full_size_all_steps():
    # all 50 steps at full size; the oracle runs one instance per host thread over a share of the layers
    wl = W.get("resnet50_topk")
    run_workload(wl, wl.steps, check_every=5, threads=16)


def test_resnet50_topk_quarter_width_curvature_every_third_step():
    wl = W.get("resnet50_topk", shapes=W.resnet50_shapes(width=16))
    run_workload(wl, 12, hz_every=3, check_every=2)


def test_gpt_1p3b_all_steps_sampled_layers():
    # full-size run on the GPU for all 20 steps; the oracle follows a sample of layers (independent of the rest):
    # the embedding, the first block, a middle block and the last block.  Curvature arrives on every fourth step
    # only, so that lambda_l is held over between refreshes at full size.
    wl = W.get("gpt_1p3b")
    L = len(wl.table)
    mid = 1 + 6 * 12
    layers = list(range(0, 7)) + list(range(mid, mid + 6)) + list(range(L - 6, L))
    w0 = W.make_weights(wl, "cuda")
    D_dev = W.make_curvature(wl, "cuda")
    D_host = {l: D_dev[wl.table[l][0]:wl.table[l][0] + wl.table[l][1]].cpu().numpy() for l in layers}
    run = ParityRun(wl.table, wl.n_total, wl.hparams(), w0, layers=layers, threads=16)
    del w0
    z = torch.empty(wl.n_total, device="cuda")
    for t in range(1, wl.steps + 1):
        g = W.make_grads(wl, t, "cuda")
        hz_dev = hz_host = None
        if (t - 1) % 4 == 0:
            ta.ta_probe(run.h, wl.probe_seed, t, 0, z)
            hz_dev = D_dev * z
            # oracle-side Hz is built from the oracle's own probe on the sampled layers, and only there
            hz_host = np.zeros(wl.n_total, dtype=np.float32)
            for l in layers:
                off, n = wl.table[l]
                zo = orc.probe(wl.probe_seed, t, 0, off, n)
                if t == 1:
                    assert np.array_equal(zo, z[off:off + n].cpu().numpy())
                hz_host[off:off + n] = D_host[l] * zo
        run.step(t, g, hz_host, wl.probe_seed, hz_dev=hz_dev, check=(t in (1, 2, 5, 10, 15, 20)))
        del hz_dev, hz_host, g
    run.report(wl.name + " (19 of 145 layers)")
    # every layer, not only the sampled ones, must have produced finite statistics and a code
    stats, status = ta.ta_stats(run.h)
    assert status.skipped == 0 and status.nonfinite_count == 0
    assert all(np.isfinite(s.grad_var) and s.grad_var > 0 and s.code in (0, 1, 2) for s in stats)


# ---------------------------------------------------------------- edge cases

RAGGED = [1, 2, 3, 31, 32, 33, 127, 128, 129, 500, 4095, 4096, 4097, 9000, 70000]


def ragged_table(lengths, gap_pattern=(0, 1, 3, 5, 0, 7, 2)):
    table, off = [], 5
    for j, n in enumerate(lengths):
        off += gap_pattern[j % len(gap_pattern)]
        table.append((off, n))
        off += n
    return table, (off + 11) // 4 * 4


@pytest.mark.parametrize("grad_dtype", ["f32", "bf16"])
@pytest.mark.parametrize("P,ppm", [(1, 1000000), (2, 1000000), (4, 1000000), (8, 1000000), (4, 100000), (8, 500000), (1, 1)])
def test_ragged_segments_odd_offsets(grad_dtype, P, ppm):
    table, n_total = ragged_table(RAGGED)
    rng = np.random.default_rng(P * 7 + ppm % 13)
    hp = dict(beta=0.5, tau_low=3e-7, tau_high=3e-6, tau_curv=0.5, alpha=2.0, eta0=0.05, topk_ppm=ppm,
              num_probes=P, t_ctrl=2, grad_dtype=grad_dtype)
    w0 = torch.from_numpy((rng.standard_normal(n_total) * 0.05).astype(np.float32))
    run = ParityRun(table, n_total, hp, w0)
    D = np.exp(rng.uniform(np.log(1e-4), 0.0, n_total)).astype(np.float32)
    D[table[5][0]:table[5][0] + 50] = D[table[5][0]]          # ties inside a layer
    for t in range(1, 7):
        scale = np.repeat(1e-3 * 3.0 ** np.arange(len(table)) / 3.0 ** 7, [n for _, n in table])
        g = np.zeros(n_total, dtype=np.float32)
        inside = np.concatenate([np.arange(o, o + n) for o, n in table])
        g[inside] = (rng.standard_normal(inside.size) * scale).astype(np.float32)
        g_dev = torch.from_numpy(g).cuda()
        if grad_dtype == "bf16":
            g_dev = g_dev.to(torch.bfloat16)
        hz = oracle_hz(D, P, 9, t) if t in (1, 2, 4, 5) else None       # curvature only on some steps
        run.step(t, g_dev, hz, 9)


def test_tie_breaks_lower_index_first():
    # every |S| equal in layer 0; half of layer 1 equal to its threshold value
    table, n_total = [(3, 70000), (70010, 5000)], 75012
    hp = dict(topk_ppm=250000, num_probes=2)
    run = ParityRun(table, n_total, hp, torch.zeros(n_total))
    D = np.full(n_total, 0.25, dtype=np.float32)
    D[70010:70010 + 5000:2] = 0.75
    g = torch.zeros(n_total, device="cuda")
    idx = np.arange(3, 3 + 70000)
    # step 1 has no window yet (every layer is swept a second time with the exact bin); steps 2 and 3 select inside
    # the window, where every element of layer 0 is a candidate: the warps' candidate stages fill and empty all the time
    for t in (1, 2, 3):
        run.step(t, g, oracle_hz(D, 2, 4, t), 4)
        m = ta.ta_masks_to_host(run.h)
        bits = (m[idx >> 5] >> (idx & 31).astype(np.uint32)) & 1
        assert np.array_equal(bits, (np.arange(70000) < 17500).astype(np.uint32))
    assert ta.ta_launch_count(run.h) == 3 * 4


@pytest.mark.parametrize("P", [1, 4])
def test_topk_selection_window_hits_drifts_and_misses(P):
    # the sweep selects inside a window of bins around the bin that held the k-th largest |S| at the last curvature
    # step; the curvature of the layers stays, drifts by a few per cent (inside the window), jumps up and down by
    # large factors (outside: the layer is swept again), and some steps bring no curvature at all
    table, n_total = ragged_table([70000, 5000, 129, 300000, 33, 2048])
    rng = np.random.default_rng(21 + P)
    hp = dict(topk_ppm=100000, num_probes=P, tau_curv=0.5, alpha=2.0, eta0=0.05)
    run = ParityRun(table, n_total, hp, torch.from_numpy((rng.standard_normal(n_total) * 0.05).astype(np.float32)))
    D0 = np.exp(rng.uniform(np.log(1e-4), 0.0, n_total)).astype(np.float32)
    factors = [1.0, 1.0, 1.04, 16.0, None, 16.0, 0.01, 0.0104, 1.0]
    for t, f in enumerate(factors, start=1):
        g = torch.from_numpy((rng.standard_normal(n_total) * 1e-3).astype(np.float32)).cuda()
        hz = None
        if f is not None:
            D = D0 * np.float32(f)
            if t == 6:
                D[table[3][0]:table[3][0] + 300000] = D0[table[3][0]:table[3][0] + 300000]      # one layer stays where it was
            hz = oracle_hz(D, P, 3, t)
        run.step(t, g, hz, 3)
    assert ta.ta_launch_count(run.h) == 4 * 8 + 3          # sweep, decisions, second sweep, resolve + update; 3 kernels without curvature


def test_zero_gradient_step_is_identity():
    wl = W.get("mlp_tiny")
    w0 = W.make_weights(wl, "cuda")
    h = ta.ta_create(wl.table, wl.n_total, **wl.hparams())
    w = w0.clone()
    c = torch.zeros(wl.n_total, dtype=torch.int16, device="cuda")
    ta.ta_step(h, w, torch.zeros(wl.n_total, device="cuda"), None, c, 0, 1)
    assert torch.equal(w.view(torch.int32), w0.view(torch.int32))
    stats, _ = ta.ta_stats(h)
    assert all(s.grad_var == 0.0 and s.grad_mean == 0.0 and s.code == ta.TA_CODE_FP16 for s in stats)
    for off, n in wl.table:
        want = orc.cast(w0[off:off + n].cpu().numpy(), to_bf16=False)
        assert np.array_equal(to_host_bits(c[off:off + n]), want)


def test_constant_gradient_has_zero_variance():
    n = 100000
    h = ta.ta_create([(0, n)], n, beta=0.0)
    w = torch.zeros(n, device="cuda")
    c = torch.zeros(n, dtype=torch.int16, device="cuda")
    ta.ta_step(h, w, torch.full((n,), 0.3, device="cuda"), None, c, 0, 1)
    s = ta.ta_stats(h)[0][0]
    assert s.grad_mean == pytest.approx(float(np.float32(0.3)), rel=1e-6)
    assert s.grad_var == 0.0          # differences from the pivot are all zero


@pytest.mark.parametrize("path", ["two dependent launches", "one cooperative launch", "separate kernels"])
@pytest.mark.parametrize("grad_dtype", ["f32", "bf16"])
@pytest.mark.parametrize("ratio", [1e3, 1e5])
def test_moments_of_gradients_with_a_large_mean(path, grad_dtype, ratio):
    # |mean| / std of 1e3 and 1e5 on layers of 1.5 M, 70 k and 1 k elements (bias-like gradients with a DC component):
    # the variance must still agree with the oracle's two-pass value to 1e-5 relative
    table, n_total = ragged_table([1500000, 70000, 1000, 33])
    rng = np.random.default_rng(int(ratio) + len(path))
    hp = dict(beta=0.5, eta0=1e-3, grad_dtype=grad_dtype, tau_low=1e-12, tau_high=1e-7)
    hp["flags"] = {"two dependent launches": 0, "one cooperative launch": ta.TA_FLAG_COOPERATIVE_LAUNCH,
                   "separate kernels": ta.TA_FLAG_NO_ONE_LAUNCH}[path]
    run = ParityRun(table, n_total, hp, torch.from_numpy((rng.standard_normal(n_total) * 0.05).astype(np.float32)))
    D = rng.uniform(0.1, 1.0, n_total).astype(np.float32)
    means = np.repeat([1.0, -0.37, 3e-3, 250.0], [n for _, n in table])
    inside = np.concatenate([np.arange(o, o + n) for o, n in table])
    for t in range(1, 4):
        g = np.zeros(n_total, dtype=np.float32)
        g[inside] = (means * (1.0 + rng.standard_normal(inside.size) / ratio)).astype(np.float32)
        g_dev = torch.from_numpy(g).cuda()
        if grad_dtype == "bf16":
            g_dev = g_dev.to(torch.bfloat16)
        run.step(t, g_dev, oracle_hz(D, 1, 5, t) if t != 2 else None, 5)
    assert ta.ta_path(run.h) == path
    assert ta.ta_launch_count(run.h) == {"two dependent launches": 6, "one cooperative launch": 3, "separate kernels": 9}[path]


def test_non_finite_input_skips_the_whole_step():
    table, n_total = ragged_table([5000, 300, 70000])
    rng = np.random.default_rng(0)
    hp = dict(topk_ppm=200000, num_probes=2)
    run = ParityRun(table, n_total, hp, torch.from_numpy(rng.standard_normal(n_total).astype(np.float32)))
    D = rng.uniform(0.1, 1.0, n_total).astype(np.float32)
    g = torch.from_numpy((rng.standard_normal(n_total) * 1e-3).astype(np.float32)).cuda()
    run.step(1, g, oracle_hz(D, 2, 0, 1), 0)
    before = (run.w_dev.clone(), run.c_dev.clone(), ta.ta_masks_to_host(run.h), ta.ta_stats(run.h)[0])
    cases = [("g", table[2][0] + 69999, float("inf")), ("hz", table[0][0] + 17, float("nan")), ("g", table[1][0], float("-inf"))]
    for t, (which, pos, val) in enumerate(cases, start=2):
        g2 = g.clone()
        hz = oracle_hz(D, 2, 0, t)
        if which == "g":
            g2[pos] = val
        else:
            hz[n_total + pos] = val            # second probe
        assert run.step(t, g2, hz, 0) is True
        _, status = ta.ta_stats(run.h)
        assert status.skipped == 1 and status.nonfinite_count == 1
        assert torch.equal(run.w_dev.view(torch.int32), before[0].view(torch.int32)) and torch.equal(run.c_dev, before[1])
        assert np.array_equal(ta.ta_masks_to_host(run.h), before[2])
    # a value outside every segment (a gap) is never read
    g3 = g.clone()
    g3[0] = float("nan")
    assert run.step(9, g3, oracle_hz(D, 2, 0, 9), 0) is False
    assert ta.ta_stats(run.h)[1].skipped == 0


@pytest.mark.parametrize("flags,per_step", [(0, 2), (ta.TA_FLAG_COOPERATIVE_LAUNCH, 1)])
def test_non_finite_input_skips_the_whole_step_small_model(flags, per_step):
    """Small dense model, as two dependent launches and as one cooperative launch: bad values in a one-element layer, on
    the partial last row of a layer and in two layers at once; the exact count is reported, nothing changes, and the
    next clean step matches."""
    table, n_total = ragged_table([1, 33, 5000, 2, 300, 70000, 129, 7])
    rng = np.random.default_rng(3)
    hp = dict(num_probes=1, tau_low=3e-7, tau_high=3e-6, flags=flags)
    run = ParityRun(table, n_total, hp, torch.from_numpy((rng.standard_normal(n_total) * 0.05).astype(np.float32)))
    D = rng.uniform(0.1, 1.0, n_total).astype(np.float32)

    def grad(t):
        return torch.from_numpy((np.random.default_rng(100 + t).standard_normal(n_total) * 1e-3).astype(np.float32)).cuda()

    assert run.step(1, grad(1), oracle_hz(D, 1, 0, 1), 0) is False
    cases = [[("g", table[0][0], float("nan"))],
             [("hz", table[5][0] + 69999, float("inf"))],
             [("g", table[3][0] + 1, float("-inf")), ("hz", table[2][0], float("nan")), ("g", table[7][0] + 6, float("nan"))],
             [("g", table[6][0] + 128, float("inf"))]]
    t = 1
    for bad in cases:
        before = (run.w_dev.clone(), run.c_dev.clone(), ta.ta_stats(run.h)[0])
        t += 1
        g2, hz = grad(t), oracle_hz(D, 1, 0, t)
        for which, pos, val in bad:
            if which == "g":
                g2[pos] = val
            else:
                hz[pos] = val
        assert run.step(t, g2, hz, 0) is True
        stats, status = ta.ta_stats(run.h)
        assert status.skipped == 1 and status.nonfinite_count == len(bad)
        assert torch.equal(run.w_dev.view(torch.int32), before[0].view(torch.int32)) and torch.equal(run.c_dev, before[1])
        assert all(a.ema_var == b.ema_var and a.code == b.code and a.lambda_max == b.lambda_max for a, b in zip(stats, before[2]))
        t += 1
        assert run.step(t, grad(t), oracle_hz(D, 1, 0, t) if t % 4 else None, 0) is False       # and the pass goes on
    assert ta.ta_launch_count(run.h) == per_step * t


def test_runs_are_bit_reproducible():
    wl = W.get("efficientnet_b0_cifar")
    outs = []
    for _ in range(2):
        h = ta.ta_create(wl.table, wl.n_total, **wl.hparams())
        w = W.make_weights(wl, "cuda")
        c = torch.zeros(wl.n_total, dtype=torch.int16, device="cuda")
        D = W.make_curvature(wl, "cuda")
        z = torch.empty(wl.n_total, device="cuda")
        for t in range(1, 6):
            ta.ta_probe(h, 0, t, 0, z)
            ta.ta_step(h, w, W.make_grads(wl, t, "cuda"), D * z, c, 0, t)
        stats, _ = ta.ta_stats(h)
        outs.append((w.clone(), c.clone(), [(s.grad_mean, s.grad_var, s.ema_var, s.ema_mean, s.code) for s in stats]))
    assert torch.equal(outs[0][0].view(torch.int32), outs[1][0].view(torch.int32))
    assert torch.equal(outs[0][1], outs[1][1]) and outs[0][2] == outs[1][2]


def test_state_save_load_continues_bit_identically():
    wl = W.get("resnet50_topk", shapes=W.resnet50_shapes(width=8))
    D = W.make_curvature(wl, "cuda")
    z = torch.empty(4 * wl.n_total, device="cuda")

    def hz(h, t):
        for p in range(4):
            ta.ta_probe(h, 1, t, p, z[p * wl.n_total:(p + 1) * wl.n_total])
        return z * D.repeat(4)

    a = ta.ta_create(wl.table, wl.n_total, **wl.hparams())
    wa = W.make_weights(wl, "cuda")
    ca = torch.zeros(wl.n_total, dtype=torch.int16, device="cuda")
    for t in (1, 2, 3):
        ta.ta_step(a, wa, W.make_grads(wl, t, "cuda"), hz(a, t), ca, 1, t)
    blob = ta.ta_state_save(a)
    b = ta.ta_create(wl.table, wl.n_total, **wl.hparams())
    ta.ta_state_load(b, blob)
    wb, cb = wa.clone(), ca.clone()
    for t in (4, 5):
        g = W.make_grads(wl, t, "cuda")
        use_hz = t == 5
        ta.ta_step(a, wa, g, hz(a, t) if use_hz else None, ca, 1, t)
        ta.ta_step(b, wb, g, hz(b, t) if use_hz else None, cb, 1, t)
        assert torch.equal(wa.view(torch.int32), wb.view(torch.int32)) and torch.equal(ca, cb)
        assert np.array_equal(ta.ta_masks_to_host(a), ta.ta_masks_to_host(b))
        sa, sb = ta.ta_stats(a)[0], ta.ta_stats(b)[0]
        assert [(s.ema_var, s.lambda_max, s.code, s.topk_threshold) for s in sa] == \
               [(s.ema_var, s.lambda_max, s.code, s.topk_threshold) for s in sb]
    with pytest.raises(ta.TriAccelError):
        ta.ta_state_load(ta.ta_create(wl.table, wl.n_total, **dict(wl.hparams(), beta=0.5)), blob)


def test_step_host_matches_device_step():
    wl = W.get("mlp_tiny")
    D = W.make_curvature(wl, "cuda")
    z = torch.empty(wl.n_total, device="cuda")
    a = ta.ta_create(wl.table, wl.n_total, **wl.hparams())
    b = ta.ta_create(wl.table, wl.n_total, **wl.hparams())
    w = W.make_weights(wl, "cuda")
    c = torch.full((wl.n_total,), 0x1111, dtype=torch.int16, device="cuda")
    wh = w.cpu().pin_memory()
    ch = c.cpu().pin_memory()
    for t in range(1, 5):
        g = W.make_grads(wl, t, "cuda")
        ta.ta_probe(a, 0, t, 0, z)
        hz = D * z
        ta.ta_step(a, w, g, hz, c, 0, t)
        ta.ta_step_host(b, wh, g.cpu().pin_memory(), hz.cpu().pin_memory(), ch, 0, t)
        assert torch.equal(w.cpu().view(torch.int32), wh.view(torch.int32))
        assert torch.equal(c.cpu(), ch)


def test_step_host_pipelined_matches_device_step():
    # large dense models take the pipelined host path (statistics first, weights in chunks with overlapped
    # copy-back); force it on a mid-size model by switching the one-launch path off
    wl = W.get("resnet18_cifar", align=1)                  # odd offsets: chunk edges fall inside vectors
    D = W.make_curvature(wl, "cuda")
    z = torch.empty(wl.n_total, device="cuda")
    a = ta.ta_create(wl.table, wl.n_total, **wl.hparams(), flags=ta.TA_FLAG_NO_ONE_LAUNCH)
    b = ta.ta_create(wl.table, wl.n_total, **wl.hparams(), flags=ta.TA_FLAG_NO_ONE_LAUNCH)
    w = W.make_weights(wl, "cuda")
    c = torch.full((wl.n_total,), 0x1111, dtype=torch.int16, device="cuda")
    wh = w.cpu().pin_memory()
    ch = c.cpu().pin_memory()
    for t in range(1, 5):
        g = W.make_grads(wl, t, "cuda")
        if t == 3:
            g[wl.table[10][0] + 3] = float("nan")           # a skipped step copies nothing back
        ta.ta_probe(a, 0, t, 0, z)
        hz = D * z if t != 2 else None
        ta.ta_step(a, w, g, hz, c, 0, t)
        ta.ta_step_host(b, wh, g.cpu().pin_memory(), hz.cpu().pin_memory() if hz is not None else None, ch, 0, t)
        assert torch.equal(w.cpu().view(torch.int32), wh.view(torch.int32)), t
        assert torch.equal(c.cpu(), ch), t
        sa, sb = ta.ta_stats(a), ta.ta_stats(b)
        assert sa[1].skipped == sb[1].skipped == (1 if t == 3 else 0)
        assert [(s.ema_var, s.code) for s in sa[0]] == [(s.ema_var, s.code) for s in sb[0]]


def test_argument_errors_enqueue_nothing():
    n = 4096
    h = ta.ta_create([(0, n)], n)
    w = torch.ones(n + 4, device="cuda")
    g = torch.ones(n + 4, device="cuda")
    c = torch.zeros(n + 8, dtype=torch.int16, device="cuda")
    with pytest.raises(ta.TriAccelError) as e:
        ta.ta_step(h, w[1:n + 1], g[:n], None, c[:n], 0, 1)
    assert e.value.code == ta.TA_ERR_ALIGN
    ta.ta_step(h, w[:n], g[:n], None, c[:n], 0, 5)
    with pytest.raises(ta.TriAccelError) as e:
        ta.ta_step(h, w[:n], g[:n], None, c[:n], 0, 5)
    assert e.value.code == ta.TA_ERR_STATE
    with pytest.raises(ta.TriAccelError) as e:
        ta.ta_step(h, w[:n], g[:n], None, c[:n], 0, 2 ** 32)
    assert e.value.code == ta.TA_ERR_ARG
    torch.cuda.synchronize()
    assert torch.all(w[:n] == 1.0 - 0.1)          # exactly one step was applied
    assert ta.ta_stats(h)[1].step == 5


def test_learning_rate_schedule_and_control_interval():
    table, n_total = ragged_table([3000, 40000])
    rng = np.random.default_rng(1)
    hp = dict(t_ctrl=3, beta=0.0, tau_low=1e-8, tau_high=1e-4)
    run = ParityRun(table, n_total, hp, torch.zeros(n_total))
    D = rng.uniform(0.1, 3.0, n_total).astype(np.float32)
    for t in range(1, 8):
        lr = 0.1 * t
        ta.ta_set_lr(run.h, lr)
        run.o.set_lr(lr)
        sigma = 1e-5 if t < 4 else 1.0
        g = torch.from_numpy((rng.standard_normal(n_total) * sigma).astype(np.float32)).cuda()
        run.step(t, g, oracle_hz(D, 1, 3, t) if t != 2 else None, 3)


def test_bounded_wait_runs_out_without_hanging():
    # the one-launch path waits at grid barriers; a wait that cannot be satisfied must end by itself,
    # leave everything untouched, be reported once, and leave the handle usable
    wl = W.get("mlp_tiny")
    g1, g2 = W.make_grads(wl, 1, "cuda"), W.make_grads(wl, 2, "cuda")
    hs, ws, cs = [], [], []
    for _ in range(2):
        hs.append(ta.ta_create(wl.table, wl.n_total, **wl.hparams(), flags=ta.TA_FLAG_COOPERATIVE_LAUNCH))
        ws.append(W.make_weights(wl, "cuda"))
        cs.append(torch.zeros(wl.n_total, dtype=torch.int16, device="cuda"))
        ta.ta_step(hs[-1], ws[-1], g1, None, cs[-1], 0, 1)
    ta.ta_stats(hs[0])
    before = (ws[0].clone(), cs[0].clone(), [(s.ema_var, s.code) for s in ta.ta_stats(hs[0])[0]])
    ta.ta_test_expire_next_wait(hs[0])
    ta.ta_step(hs[0], ws[0], g2, None, cs[0], 0, 2)              # every block gives up at the first barrier
    with pytest.raises(ta.TriAccelError) as e:
        ta.ta_stats(hs[0])
    assert e.value.code == ta.TA_ERR_CUDA and "wait ran out" in str(e.value)
    assert torch.equal(ws[0].view(torch.int32), before[0].view(torch.int32)) and torch.equal(cs[0], before[1])
    assert [(s.ema_var, s.code) for s in ta.ta_stats(hs[0])[0]] == before[2]      # reported once; state untouched
    # both handles now take the same next step and must agree bit for bit
    ta.ta_step(hs[0], ws[0], g2, None, cs[0], 0, 3)
    ta.ta_step(hs[1], ws[1], g2, None, cs[1], 0, 3)
    assert torch.equal(ws[0].view(torch.int32), ws[1].view(torch.int32)) and torch.equal(cs[0], cs[1])
    assert ta.ta_stats(hs[0])[1].skipped == 0


@pytest.mark.parametrize("momentum,wd,grad_dtype", [(0.9, 0.0, "f32"), (0.0, 5e-4, "f32"), (0.9, 5e-4, "bf16")])
def test_momentum_and_weight_decay(momentum, wd, grad_dtype):
    table, n_total = ragged_table(RAGGED)
    rng = np.random.default_rng(11)
    hp = dict(beta=0.5, tau_low=3e-7, tau_high=3e-6, eta0=0.05, momentum=momentum, weight_decay=wd, grad_dtype=grad_dtype)
    run = ParityRun(table, n_total, hp, torch.from_numpy((rng.standard_normal(n_total) * 0.05).astype(np.float32)))
    D = np.exp(rng.uniform(np.log(1e-4), 0.0, n_total)).astype(np.float32)
    for t in range(1, 9):
        g = torch.from_numpy((rng.standard_normal(n_total) * 1e-3).astype(np.float32)).cuda()
        if grad_dtype == "bf16":
            g = g.to(torch.bfloat16)
        if t == 5:
            g[table[3][0]] = float("inf")             # skipped: weights AND momentum buffer stay as they are
        run.step(t, g, oracle_hz(D, 1, 2, t) if t % 2 else None, 2)


def test_momentum_state_is_checkpointed():
    wl = W.get("mlp_tiny")
    hp = dict(wl.hparams(), momentum=0.9, weight_decay=1e-4)
    a = ta.ta_create(wl.table, wl.n_total, **hp)
    wa = W.make_weights(wl, "cuda")
    ca = torch.zeros(wl.n_total, dtype=torch.int16, device="cuda")
    for t in (1, 2, 3):
        ta.ta_step(a, wa, W.make_grads(wl, t, "cuda"), None, ca, 0, t)
    blob = ta.ta_state_save(a)
    b = ta.ta_create(wl.table, wl.n_total, **hp)
    ta.ta_state_load(b, blob)
    wb, cb = wa.clone(), ca.clone()
    for t in (4, 5):
        g = W.make_grads(wl, t, "cuda")
        ta.ta_step(a, wa, g, None, ca, 0, t)
        ta.ta_step(b, wb, g, None, cb, 0, t)
        assert torch.equal(wa.view(torch.int32), wb.view(torch.int32)) and torch.equal(ca, cb)
