"""The layer-pipelined pass (TA_FLAG_INPUTS_FINITE on models beyond the one-launch path) against the oracle, through
the C ABI: steps with decisions (sweep tasks, per-layer decisions by the block that finishes a layer, update tasks that
wait for them) and steps between decisions (single pass), with and without curvature."""
import numpy as np
import pytest
import torch

import paper_2508_16905_b200 as ta
from paper_2508_16905_b200 import workloads as W
from tests.parity import ParityRun, oracle_hz
from tests.test_gpu_parity import RAGGED, ragged_table

pytestmark = pytest.mark.gpu

PIPE = ta.TA_FLAG_INPUTS_FINITE | ta.TA_FLAG_NO_ONE_LAUNCH


@pytest.mark.parametrize("grad_dtype", ["f32", "bf16"])
@pytest.mark.parametrize("P,t_ctrl", [(1, 1), (1, 4), (2, 3), (4, 1), (8, 2)])
def test_ragged_segments_pipelined(grad_dtype, P, t_ctrl):
    table, n_total = ragged_table(RAGGED + [40000, 2048, 16384, 16385, 100000])
    rng = np.random.default_rng(P * 11 + t_ctrl)
    hp = dict(beta=0.5, tau_low=3e-7, tau_high=3e-6, tau_curv=0.5, alpha=2.0, eta0=0.05, num_probes=P, t_ctrl=t_ctrl,
              grad_dtype=grad_dtype, flags=PIPE)
    run = ParityRun(table, n_total, hp, torch.from_numpy((rng.standard_normal(n_total) * 0.05).astype(np.float32)))
    D = np.exp(rng.uniform(np.log(1e-4), 0.0, n_total)).astype(np.float32)
    inside = np.concatenate([np.arange(o, o + n) for o, n in table])
    scale = np.repeat(1e-3 * 3.0 ** (np.arange(len(table)) % 9) / 3.0 ** 7, [n for _, n in table])
    for t in range(1, 10):
        g = np.zeros(n_total, dtype=np.float32)
        g[inside] = (rng.standard_normal(inside.size) * scale).astype(np.float32)
        g_dev = torch.from_numpy(g).cuda()
        if grad_dtype == "bf16":
            g_dev = g_dev.to(torch.bfloat16)
        hz = oracle_hz(D, P, 9, t) if t in (1, 2, 4, 5, 8) else None       # curvature only on some steps
        run.step(t, g_dev, hz, 9)
    assert ta.ta_launch_count(run.h) == 9          # one launch per step
    run.report("ragged, pipelined")


@pytest.mark.parametrize("t_ctrl", [1, 4])
def test_two_block_decoder_pipelined(t_ctrl):
    # 33.6 M parameters in 13 tensors of 1024 ... 8.4 M elements: layers of many batches, whose update tasks wait for
    # the block that finishes their sweep; curvature on every fourth step as in the paper's schedule
    wl = W.get("gpt_1p3b", shapes=W.gpt_shapes(layers=2, d=1024, vocab=8192), t_ctrl=t_ctrl)
    w0 = W.make_weights(wl, "cuda")
    D = W.make_curvature(wl, "cuda").cpu().numpy()
    run = ParityRun(wl.table, wl.n_total, dict(wl.hparams(), flags=ta.TA_FLAG_INPUTS_FINITE), w0, threads=8)
    for t in range(1, 9):
        g = W.make_grads(wl, t, "cuda")
        hz = oracle_hz(D, 1, wl.probe_seed, t) if (t - 1) % 4 == 0 else None
        run.step(t, g, hz, wl.probe_seed)
    assert ta.ta_launch_count(run.h) == 8
    run.report(f"two-block decoder, pipelined, t_ctrl {t_ctrl}")


def test_pipelined_pass_reports_non_finite_values_without_skipping():
    table, n_total = ragged_table([5000, 300, 70000])
    rng = np.random.default_rng(0)
    h = ta.ta_create(table, n_total, flags=PIPE)
    w = torch.from_numpy(rng.standard_normal(n_total).astype(np.float32)).cuda()
    c = torch.zeros(n_total, dtype=torch.int16, device="cuda")
    g = torch.from_numpy((rng.standard_normal(n_total) * 1e-3).astype(np.float32)).cuda()
    g[table[1][0] + 7] = float("inf")
    g[0] = float("nan")                   # in a gap: never read
    w0 = w.clone()
    ta.ta_step(h, w, g, None, c, 0, 1)
    stats, status = ta.ta_stats(h)
    assert status.skipped == 0 and status.nonfinite_count == 1 and status.step == 1
    # the layers that held only finite values are updated as usual
    for l in (0, 2):
        off, n = table[l]
        assert torch.isfinite(w[off:off + n]).all() and not torch.equal(w[off:off + n], w0[off:off + n])
        assert np.isfinite(stats[l].grad_var)


def test_flag_is_accepted_where_the_pipelined_pass_does_not_apply():
    # small dense model (one-launch path), top-k, momentum: the flag changes nothing
    wl = W.get("mlp_tiny")
    outs = []
    for flags in (0, ta.TA_FLAG_INPUTS_FINITE):
        h = ta.ta_create(wl.table, wl.n_total, **wl.hparams(), flags=flags)
        w = W.make_weights(wl, "cuda")
        c = torch.zeros(wl.n_total, dtype=torch.int16, device="cuda")
        for t in (1, 2):
            ta.ta_step(h, w, W.make_grads(wl, t, "cuda"), None, c, 0, t)
        outs.append((w, c, ta.ta_launch_count(h)))
    assert torch.equal(outs[0][0].view(torch.int32), outs[1][0].view(torch.int32)) and torch.equal(outs[0][1], outs[1][1])
    assert outs[0][2] == outs[1][2] == 4           # two dependent launches per step either way
    with pytest.raises(ta.TriAccelError):
        ta.ta_create(wl.table, wl.n_total, flags=16)
