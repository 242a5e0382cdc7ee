"""CPU-only checks of the boundary: the library loads, exports what the header declares, and the
host-only parts (batch rule, argument validation that needs no device, replica bookkeeping) work."""
import ctypes as C
import os
import re
import subprocess
import sys

import numpy as np
import pytest
import torch

import paper_2508_16905_b200 as ta
from paper_2508_16905_b200 import binding, dist as D_mod, workloads as W

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    text = open(os.path.join(ROOT, "include", "triaccel.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(ta_[a-z_0-9]+)\s*\(", text)) - {"ta_mem_reader"})


def test_library_exports_every_declared_symbol():
    L = binding.lib()
    names = declared_functions()
    assert len(names) >= 15
    for n in names:
        assert hasattr(L, n), n
    assert sorted(binding.EXPORTS) == names


def test_struct_layouts_match_the_header():
    assert C.sizeof(binding.ta_hparams) == 56
    assert C.sizeof(binding.ta_layer_stats) == 48
    assert C.sizeof(binding.ta_step_status) == 24
    assert C.sizeof(binding.ta_segment) == 16


def test_create_rejects_bad_arguments_before_touching_a_device():
    bad = [
        dict(table=[], n_total=8),
        dict(table=[(0, 8), (4, 8)], n_total=16),                 # overlap
        dict(table=[(8, 8), (0, 8)], n_total=16),                 # not ascending
        dict(table=[(0, 0)], n_total=8),                          # empty layer
        dict(table=[(0, 9)], n_total=8),                          # beyond n_total
        dict(table=[(0, 6)], n_total=6),                          # n_total not a multiple of 4
        dict(table=[(0, 8)], n_total=8, num_probes=3),
        dict(table=[(0, 8)], n_total=8, topk_ppm=0),
        dict(table=[(0, 8)], n_total=8, beta=1.0),
        dict(table=[(0, 8)], n_total=8, t_ctrl=0),
        dict(table=[(0, 8)], n_total=8, momentum=1.0),
        dict(table=[(0, 8)], n_total=8, weight_decay=-1.0),
        dict(table=[(0, 8)], n_total=8, flags=16),               # unknown flag bit
        dict(table=[(0, 8)], n_total=8, tau_low=2.0, tau_high=1.0),
    ]
    for kw in bad:
        table, n_total = kw.pop("table"), kw.pop("n_total")
        with pytest.raises(ta.TriAccelError) as e:
            ta.ta_create(table, n_total, **kw)
        assert e.value.code == ta.TA_ERR_ARG, kw


@pytest.mark.skipif(torch.cuda.is_available(), reason="checks the no-GPU failure mode")
def test_no_device_means_a_loud_error_not_a_fallback():
    with pytest.raises(ta.TriAccelError) as e:
        ta.ta_create([(0, 8)], 8)
    assert e.value.code == ta.TA_ERR_CUDA


def _ctrl(B, free, total, budget=0, **kw):
    state = {"calls": 0}

    @binding.ta_mem_reader
    def reader(user, free_p, total_p):
        state["calls"] += 1
        if free is None:
            return 1
        free_p[0], total_p[0] = free, total
        return 0
    args = dict(B=B, delta_up=8, delta_down=16, B_min=8, B_max=128, rho_low=0.7, rho_high=0.9)
    args.update(kw)
    bc = binding.ta_batch_ctrl(args["B"], args["delta_up"], args["delta_down"], args["B_min"], args["B_max"],
                               args["rho_low"], args["rho_high"], budget, reader, None)
    return bc, reader


def test_batch_rule_truth_table_with_fake_reader():
    # Sec. 3.3: usage = total - free
    for B, used, want in [(96, 50, 104), (96, 95, 80), (96, 80, 96), (96, 70, 96), (96, 90, 96), (124, 10, 128), (16, 99, 8)]:
        bc, keep = _ctrl(B, free=100 - used, total=100)
        assert ta.ta_batch_next(bc) == want and bc.B == want
    # a caller budget replaces the device total as MemMax
    bc, keep = _ctrl(96, free=50, total=100, budget=50)       # usage 50 > 0.9 * 50
    assert ta.ta_batch_next(bc) == 80
    # the initial batch size of the paper's experiments grows while memory is free
    bc, keep = _ctrl(96, free=90, total=100)
    assert [ta.ta_batch_next(bc) for _ in range(5)] == [104, 112, 120, 128, 128]


def test_batch_rule_errors():
    bc, keep = _ctrl(96, free=None, total=0)
    with pytest.raises(ta.TriAccelError) as e:
        ta.ta_batch_next(bc)
    assert e.value.code == ta.TA_ERR_CUDA and bc.B == 96
    for kw in [dict(rho_low=0.95), dict(B_min=200), dict(delta_up=-1)]:
        bc, keep = _ctrl(96, free=50, total=100, **kw)
        with pytest.raises(ta.TriAccelError) as e:
            ta.ta_batch_next(bc)
        assert e.value.code == ta.TA_ERR_ARG


def test_workload_tables_have_the_published_parameter_counts():
    want = {"mlp_tiny": (4, 203530), "resnet18_cifar": (62, 11173962), "efficientnet_b0_cifar": (213, 4020358),
            "resnet50_topk": (161, 25557032), "gpt_1p3b": (145, 1311080448)}
    for name, (L, n) in want.items():
        wl = W.get(name)
        assert (len(wl.table), wl.num_params) == (L, n)
        assert all(off % 8 == 0 for off, _ in wl.table) and wl.n_total % 8 == 0
        ends = [o + n for o, n in wl.table]
        assert all(wl.table[i + 1][0] >= ends[i] for i in range(L - 1)) and ends[-1] <= wl.n_total
    small = [n for _, n in W.get("efficientnet_b0_cifar").table if n <= 1024]
    assert (len(small), sum(small)) == (121, 33030)


def test_generators_are_seeded_and_have_the_stated_distributions():
    wl = W.get("mlp_tiny")
    g1, g2 = W.make_grads(wl, 3), W.make_grads(wl, 3)
    assert torch.equal(g1, g2) and not torch.equal(g1, W.make_grads(wl, 4))
    for l, (off, n) in enumerate(wl.table[:3]):
        assert float(g1[off:off + n].std()) == pytest.approx(1e-3 * 2 ** l, rel=0.2 if n < 1000 else 0.02)
    D = W.make_curvature(wl)
    assert float(D.min()) >= 1e-4 * 0.999 and float(D.max()) <= 1.0
    assert float(torch.log(D).mean()) == pytest.approx(0.5 * torch.log(torch.tensor(1e-4)).item(), rel=0.02)
    assert float(W.make_weights(wl).std()) == pytest.approx(0.05, rel=0.02)
    heavy = W.get("resnet50_topk", shapes=W.resnet50_shapes(width=8))
    g = W.make_grads(heavy, 1)
    assert float((g.abs() > 8e-3).float().mean()) > 1e-4          # the Student-t(2) tail is present
    assert W.make_grads(W.get("gpt_1p3b", shapes=W.gpt_shapes(layers=1, d=64, vocab=128)), 1).dtype == torch.bfloat16


def test_pipeline_queues_cover_every_layer_once():
    rng = np.random.default_rng(5)
    tables = [W.get("gpt_1p3b").table, W.get("resnet18_cifar", align=1).table]
    off, t = 3, []
    for _ in range(60):
        n = int(rng.choice([1, 7, 2048, 2049, 14336, 14337, 50000, 3000000]))
        off += int(rng.integers(0, 9))
        t.append((off, n))
        off += n
    tables.append(t)
    for table in tables:
        hold = ta.ta_plan_pipeline(table, False)
        both = ta.ta_plan_pipeline(table, True)
        assert all(k == 2 for k, _, _, _ in hold) and len(both) == 2 * len(hold)
        # the batches tile every layer exactly, in buffer order, on a grid of 2048-element cells
        pos = {l: off for l, (off, n) in enumerate(table)}
        for _, l, b, n in hold:
            assert b == pos[l] and 0 < n <= 14336 and (b + n == table[l][0] + table[l][1] or (b + n) % 2048 == 0)
            pos[l] += n
        assert all(pos[l] == off + n for l, (off, n) in enumerate(table))
        sweeps, applies = both[:len(hold)], both[len(hold):]
        assert all(k == 0 for k, _, _, _ in sweeps) and all(k == 1 for k, _, _, _ in applies)
        assert [x[1:] for x in sweeps] == [x[1:] for x in hold]
        # update tasks: layer by layer, a layer's last batch first
        assert [l for _, l, _, _ in applies] == sorted(l for _, l, _, _ in applies)
        for l in range(len(table)):
            mine = [x[1:] for x in applies if x[1] == l]
            assert mine == [x[1:] for x in sweeps if x[1] == l][::-1]


def test_replica_bookkeeping_world_size_2_gloo(tmp_path):
    script = r"""
import os, sys
sys.path.insert(0, %r)
from paper_2508_16905_b200 import dist as D
rank, local_rank, world = D.init("gloo")
assert world == 2
D.barrier()
ms, units = D.aggregate(10.0 + 5.0 * rank, 1000.0 * (rank + 1))
assert (ms, units) == (15.0, 3000.0), (ms, units)
D.barrier()
D.shutdown()
print("rank", rank, "ok")
""" % ROOT
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="1")
    path = tmp_path / "ranks.py"
    path.write_text(script)
    res = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29571", str(path)],
                         capture_output=True, text=True, env=env, timeout=240)
    assert res.returncode == 0, res.stderr[-2000:]
    assert res.stdout.count("ok") == 2


def test_shard_ranges_and_record_exchange_world_size_2_gloo(tmp_path):
    # the ranges tile the buffer on the 128-element grid; the exchange returns every rank's records in rank order,
    # identical on all ranks (which is what makes every rank take the same decisions)
    for n_total, world in [(4096, 2), (1000, 3), (1311080448, 8), (128, 4)]:
        r = D_mod.shard_ranges(n_total, world)
        assert r[0][0] == 0 and r[-1][1] >= n_total and all(a % 128 == 0 and b % 128 == 0 and a <= b for a, b in r)
        assert all(r[i][1] == r[i + 1][0] for i in range(world - 1))
    script = r"""
import os, sys
sys.path.insert(0, %r)
import torch
from paper_2508_16905_b200 import dist as D
rank, local_rank, world = D.init("gloo")
L = 5
mine = torch.full((L * 40,), rank + 1, dtype=torch.uint8)
mine[::40] = torch.arange(L, dtype=torch.uint8) + 10 * (rank + 1)
out = D.gather_records(mine)
assert out.numel() == world * L * 40
for r in range(world):
    part = out[r * L * 40:(r + 1) * L * 40]
    assert torch.equal(part[::40], torch.arange(L, dtype=torch.uint8) + 10 * (r + 1)) and int(part[1]) == r + 1
D.shutdown()
print("rank", rank, "ok")
""" % ROOT
    path = tmp_path / "ranks.py"
    path.write_text(script)
    env = dict(os.environ, MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="1")
    res = subprocess.run([sys.executable, "-m", "torch.distributed.run", "--nnodes=1", "--nproc-per-node=2",
                          "--master-addr", "127.0.0.1", "--master-port", "29573", str(path)],
                         capture_output=True, text=True, env=env, timeout=240)
    assert res.returncode == 0, res.stderr[-2000:]
    assert res.stdout.count("ok") == 2


def test_reference_arm_of_the_benchmark_runs_on_cpu():
    # `bench.py --impl reference` times the CPU checker; it must work without a GPU and print one JSON line
    import json
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference", "--config", "mlp_tiny",
                          "--steps", "2", "--warmup", "1"], capture_output=True, text=True, timeout=300,
                         env=dict(os.environ, CUDA_VISIBLE_DEVICES=""))
    assert res.returncode == 0, res.stderr[-1500:]
    line = json.loads(res.stdout.strip().splitlines()[-1])
    assert line["impl"] == "reference" and line["unit"] == "params/s" and line["value"] > 0
    assert line["cpu_baseline"]["kind"] == "oracle" and line["cpu_baseline"]["cores"] == 1
    assert line["e2e"]["h2d_bytes_per_step"] == 0 and line["config"]["workload"] == "mlp_tiny"


# ---------------------------------------------------------------- plan of the one-launch path (host logic)

def _check_plan(table, warps):
    from paper_2508_16905_b200 import binding as B
    runs, used, max_rows = B.ta_plan_one_launch(table, warps)
    # the runs tile every layer exactly, in buffer order, and interior cuts lie on the 128-element row grid
    by_layer = {}
    for begin, length, layer, warp in runs:
        assert length > 0
        by_layer.setdefault(layer, []).append((begin, length))
    assert sorted(by_layer) == list(range(len(table)))
    for l, (off, n) in enumerate(table):
        pos = off
        for begin, length in by_layer[l]:
            assert begin == pos
            pos += length
            if pos != off + n:
                assert pos % 128 == 0
        assert pos == off + n
    # warps get consecutive runs; no warp index beyond the request; about equal cost
    warps_seen = [w for *_, w in runs]
    assert warps_seen == sorted(warps_seen) and warps_seen[-1] < max(8, -(-warps // 8) * 8)
    assert used == len(set(warps_seen))
    cost, rows = {}, {}
    for begin, length, layer, w in runs:
        cost[w] = cost.get(w, 0) + length
        rows[w] = rows.get(w, 0) + (begin + length - 1) // 128 - begin // 128 + 1
    n_layers_cost = 256 * len(table)
    total = sum(n for _, n in table) + n_layers_cost
    n_warps = max(8, -(-min(warps, -(-total // 512)) // 8) * 8)
    target = total / n_warps
    assert max(cost.values()) <= target + 128 + 64, (max(cost.values()), target)
    assert max_rows == max(rows.values())
    return runs, used, max_rows


def test_one_launch_plan_on_the_benchmark_tables():
    from paper_2508_16905_b200 import workloads as W
    for name in ("mlp_tiny", "resnet18_cifar", "efficientnet_b0_cifar"):
        wl = W.get(name)
        for warps in (8, 148 * 8, 148 * 24, 148 * 32):
            _check_plan(wl.table, warps)
    # the EfficientNet-B0 mix on a full B200 grid: every warp has work and walks a dozen rows at most
    wl = W.get("efficientnet_b0_cifar")
    runs, used, max_rows = _check_plan(wl.table, 148 * 24)
    assert used == 148 * 24 and max_rows <= 14


def test_one_launch_plan_on_random_tables():
    import numpy as np
    rng = np.random.default_rng(7)
    for trial in range(60):
        L = int(rng.integers(1, 400))
        lens = np.where(rng.random(L) < 0.6, rng.integers(1, 300, L), rng.integers(300, 200000, L))
        gaps = rng.integers(0, 50, L) * (rng.random(L) < 0.5)
        table, pos = [], 0
        for n, gap in zip(lens, gaps):
            pos += int(gap)
            table.append((pos, int(n)))
            pos += int(n)
        _check_plan(table, int(rng.choice([8, 64, 1184, 3552, 4736])))


def test_one_launch_plan_rejects_bad_tables():
    from paper_2508_16905_b200 import binding as B
    with pytest.raises(B.TriAccelError):
        B.ta_plan_one_launch([(0, 10), (5, 10)], 64)          # overlapping
    with pytest.raises(B.TriAccelError):
        B.ta_plan_one_launch([(0, 0)], 64)                    # empty segment


def _check_items(table, sm_count, topk):
    items, elems = ta.ta_plan_items(table, sm_count, topk)
    assert elems in (512, 1024, 2048, 4096, 8192, 16384)
    pos = {l: off for l, (off, n) in enumerate(table)}
    last_layer = 0
    for i, (b, n, l, warp, one_layer) in enumerate(items):
        assert warp == i % 8
        if n == 0:
            assert topk                      # padding in front of a layer that starts on a batch boundary
            continue
        assert l >= last_layer               # buffer order
        last_layer = l
        # consecutive pieces of the layer, cut on the global grid of `elems` elements
        assert b == pos[l] and (b + n == table[l][0] + table[l][1] or (b + n) % elems == 0) and n <= elems
        pos[l] += n
    assert all(pos[l] == off + n for l, (off, n) in enumerate(table))       # every element exactly once
    for bt in range(0, len(items), 8):
        batch = items[bt:bt + 8]
        layers = {l for _, n, l, _, _ in batch if n}
        assert all(flag == (1 if len(layers) <= 1 else 0) for _, _, _, _, flag in batch)
    if topk:
        # a layer of at least eight items owns its batches
        for l, (off, n) in enumerate(table):
            mine = [i for i, it in enumerate(items) if it[2] == l and it[1]]
            if len(mine) >= 8 and l > 0:
                assert mine[0] % 8 == 0
                assert all(items[i][4] == 1 for i in mine[: len(mine) // 8 * 8])
    return items, elems


def test_item_plan_of_the_multi_kernel_pass():
    import numpy as np
    from paper_2508_16905_b200 import workloads as W
    items, elems = _check_items(W.get("resnet50_topk").table, 148, True)
    assert elems == 4096 and len(items) < 8000
    _check_items(W.get("resnet50_topk").table, 148, False)
    items, elems = _check_items(W.get("gpt_1p3b").table, 148, False)
    assert elems == 16384
    rng = np.random.default_rng(11)
    for trial in range(40):
        L = int(rng.integers(1, 200))
        lens = np.where(rng.random(L) < 0.6, rng.integers(1, 300, L), rng.integers(300, 300000, L))
        gaps = rng.integers(0, 50, L) * (rng.random(L) < 0.5)
        table, p = [], int(rng.integers(0, 9))
        for n, gap in zip(lens, gaps):
            p += int(gap)
            table.append((p, int(n)))
            p += int(n)
        _check_items(table, int(rng.choice([1, 16, 148])), bool(trial % 2))
    with pytest.raises(ta.TriAccelError):
        ta.ta_plan_items([(0, 10), (5, 10)], 148, False)
