"""A model spread over ranks by flat ranges, proven on one GPU: three handles hold the thirds of one flat buffer (cuts
inside layers), exchange their per-layer records, and must arrive at the codes, step sizes, weights and copies of the
oracle (and of one handle over the whole model, bit for bit)."""
import numpy as np
import pytest
import torch

import paper_2508_16905_b200 as ta
from paper_2508_16905_b200 import dist as D
from oracle import oracle as orc
from tests.parity import compare_stats, oracle_hz, to_host_bits, ulp_f32, ulp_16
from tests.test_gpu_parity import ragged_table

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("grad_dtype,P", [("f32", 1), ("bf16", 2)])
def test_three_shards_match_the_oracle_and_the_whole_model(grad_dtype, P):
    table, n_total = ragged_table([70000, 1, 5000, 129, 300000, 33, 2048, 90000])
    world = 3
    ranges = D.shard_ranges(n_total, world)
    assert ranges[0][0] == 0 and ranges[-1][1] >= n_total and all(a % 128 == 0 and b % 128 == 0 for a, b in ranges)
    hp = dict(beta=0.5, tau_low=3e-7, tau_high=3e-6, tau_curv=0.5, alpha=2.0, eta0=0.05, num_probes=P, t_ctrl=2, grad_dtype=grad_dtype)
    rng = np.random.default_rng(5)
    w0 = (rng.standard_normal(n_total) * 0.05).astype(np.float32)
    D_h = np.exp(rng.uniform(np.log(1e-4), 0.0, n_total)).astype(np.float32)
    L = len(table)
    n_pad = ranges[-1][1]                       # the last range may reach past n_total: pad the local buffers

    def local(x, r, fill=0):
        a, b = ranges[r]
        out = np.full(b - a, fill, dtype=x.dtype)
        out[:min(b, x.size) - a] = x[a:min(b, x.size)]
        return out

    whole = ta.ta_create(table, n_total, **hp, flags=ta.TA_FLAG_NO_ONE_LAUNCH)
    o = orc.Oracle(table, n_total, **hp)
    shards = [ta.ta_create_shard(table, n_total, a, b, **hp) for a, b in ranges]
    w_whole = torch.from_numpy(w0).cuda()
    c_whole = torch.full((n_total,), 0x5A5A, dtype=torch.int16, device="cuda")
    w_host, c_host = w0.copy(), np.full(n_total, 0x5A5A, dtype=np.uint16)
    w_loc = [torch.from_numpy(local(w0, r)).cuda() for r in range(world)]
    c_loc = [torch.full((b - a,), 0x5A5A, dtype=torch.int16, device="cuda") for a, b in ranges]
    rec = [torch.empty(L * ta.RECORD_BYTES, dtype=torch.uint8, device="cuda") for _ in range(world)]
    inside = np.concatenate([np.arange(off, off + n) for off, n in table])
    for t in range(1, 7):
        g = np.zeros(n_total, dtype=np.float32)
        g[inside] = (rng.standard_normal(inside.size) * 1e-3 * (1 + t % 3)).astype(np.float32)
        if t == 5:
            g[table[4][0] + 250000] = np.inf          # on the last rank only: every rank must skip the step
        hz = oracle_hz(D_h, P, 9, t) if t != 3 else None
        g_t = torch.from_numpy(g).cuda()
        if grad_dtype == "bf16":
            g_t = g_t.to(torch.bfloat16)
        g_np = to_host_bits(g_t)
        hz_t = torch.from_numpy(hz).cuda() if hz is not None else None
        ta.ta_step(whole, w_whole, g_t, hz_t, c_whole, 9, t)
        skipped = o.step(w_host, g_np, hz, c_host, 9, t)
        assert skipped == (t == 5)
        # the ranks, one after the other on this GPU: sweep, exchange through one concatenated buffer, apply
        g_loc, hz_loc = [], []
        for r, (a, b) in enumerate(ranges):
            g_loc.append(torch.from_numpy(local(g_np, r)).cuda().view(torch.bfloat16 if grad_dtype == "bf16" else torch.float32))
            hz_loc.append(None if hz is None else torch.from_numpy(np.concatenate([local(hz[p * n_total:(p + 1) * n_total], r) for p in range(P)])).cuda())
            ta.ta_shard_sweep(shards[r], g_loc[r], hz_loc[r], 9, t, rec[r])
        everyone = torch.cat(rec)
        for r in range(world):
            ta.ta_shard_apply(shards[r], w_loc[r], g_loc[r], c_loc[r], everyone, world)
        stats_whole, status_whole = ta.ta_stats(whole)
        w_cat = torch.cat(w_loc)[:n_total]
        c_cat = torch.cat(c_loc)[:n_total]
        for r in range(world):
            stats, status = ta.ta_stats(shards[r])
            assert (status.step, status.skipped, status.nonfinite_count) == (t, int(t == 5), int(t == 5))
            for l, (s, sw, ol) in enumerate(zip(stats, stats_whole, o.layers())):
                compare_stats(s, ol, where=f"step {t} rank {r} layer {l}", n=table[l][1])
                assert (s.code, s.eta_scale, s.lambda_max, s.ema_var, s.ema_mean) == (sw.code, sw.eta_scale, sw.lambda_max, sw.ema_var, sw.ema_mean)
        assert torch.equal(w_cat.view(torch.int32), w_whole.view(torch.int32)) and torch.equal(c_cat, c_whole)
        assert int(ulp_f32(w_cat.cpu().numpy()[inside], w_host[inside]).max()) <= 2
        assert int(ulp_16(to_host_bits(c_cat)[inside], c_host[inside]).max()) <= 1
    # the padding of the last range and the gaps were never written
    gaps = np.ones(n_total, dtype=bool)
    gaps[inside] = False
    assert np.all(to_host_bits(torch.cat(c_loc))[:n_total][gaps] == 0x5A5A) and np.all(to_host_bits(c_loc[-1])[n_total - ranges[-1][0]:] == 0x5A5A)


def test_shard_handles_refuse_what_they_cannot_do():
    table, n_total = [(0, 4096)], 4096
    with pytest.raises(ta.TriAccelError):
        ta.ta_create_shard(table, n_total, 0, 100)                      # not on the 128-element grid
    with pytest.raises(ta.TriAccelError):
        ta.ta_create_shard(table, n_total, 0, 2048, topk_ppm=100000)    # no mask on a sharded model
    h = ta.ta_create_shard(table, n_total, 0, 2048)
    x = torch.zeros(2048, device="cuda")
    c = torch.zeros(2048, dtype=torch.int16, device="cuda")
    with pytest.raises(ta.TriAccelError) as e:
        ta.ta_step(h, x, x, None, c, 0, 1)
    assert e.value.code == ta.TA_ERR_STATE
    with pytest.raises(ta.TriAccelError) as e:
        ta.ta_shard_apply(h, x, x, c, torch.zeros(40, dtype=torch.uint8, device="cuda"), 1)       # no sweep before it
    assert e.value.code == ta.TA_ERR_STATE
