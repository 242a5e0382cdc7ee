"""Benchmark of the fused Tri-Accel optimizer pass.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--config NAME] [--impl ours|reference]

Prints ONE JSON line.  `value` is parameters per second of the whole job (N replicas), inputs
resident in HBM; `e2e` is the same metric through ta_step_host with pinned HOST buffers
(copies inside the timed region); `roofline` describes the dominant kernel against the measured HBM copy rate
(and, under `step`, the whole step against that rate and the 8 TB/s nominal peak, with the targets);
`configs` carries the same figures for all five configurations and `paths` those of the passes a caller
can opt into; `cpu_baseline` is the CPU checker timed on a bounded sample of the same workload.
`--impl reference` times the CPU checker alone.
"""
import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fused Tri-Accel step params/sec"
UNIT = "params/s"
FALLBACK_HBM_GBS = 6650.0


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def kernel_source_hash():
    h = hashlib.sha256()
    csrc = os.path.join(ROOT, "paper_2508_16905_b200", "csrc")
    for name in sorted(os.listdir(csrc)):
        with open(os.path.join(csrc, name), "rb") as f:
            h.update(f.read())
    return h.hexdigest()[:16]


class ClockSampler:
    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, uuid):
        self.proc = None
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", uuid, f"--query-gpu={self.QUERY}",
                                          "--format=csv,noheader,nounits", "-lms", "20"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
        except Exception:
            self.proc = None

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.15)
        self.proc.terminate()
        try:
            out, _ = self.proc.communicate(timeout=5)
        except Exception:
            self.proc.kill()
            out = ""
        sm, mx, reasons = [], [], set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for line in out.splitlines():
            parts = [p.strip() for p in line.split(",")]
            if len(parts) < 7:
                continue
            try:
                sm.append(float(parts[0]))
                mx.append(float(parts[1]))
            except ValueError:
                continue
            for name, val in zip(names, parts[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        return {"sm_mhz": statistics.median(sm) if sm else None, "sm_max_mhz": max(mx) if mx else None,
                "samples": len(sm), "reasons": sorted(reasons)}


def oracle_sample(wl, max_params):
    """A run of whole layers of `wl` (after the first, to skip the embedding of the GPT workload when
    it alone exceeds the budget) with at most max_params parameters."""
    layers, total = [], 0
    for l, (off, n) in enumerate(wl.table):
        if n > max_params:
            continue
        if total + n > max_params:
            break
        layers.append(l)
        total += n
    return layers, total


def time_oracle(wl, steps, warmup, budget_s, torch_device, all_cores=False):
    """Times the CPU checker, as it stands, on a bounded sample of layers; returns a dict."""
    import numpy as np
    import torch
    from oracle import oracle as orc
    from paper_2508_16905_b200 import workloads as W

    # calibrate on a small sample, then size the sample so that all steps fit the budget
    per_param_guess = 120e-9 * (1 + 0.5 * wl.num_probes) * (3.0 if wl.topk_ppm < 1000000 else 1.0)
    max_params = int(max(2e5, min(wl.num_params, budget_s / max(1, steps + warmup) / per_param_guess)))
    layers, n_sample = oracle_sample(wl, max_params)
    if not layers:
        layers, n_sample = [0], wl.table[0][1]
    sub = [wl.table[l] for l in layers]
    end = (sub[-1][0] + sub[-1][1] + 7) // 8 * 8
    dev = torch_device
    gen_total = wl.n_total

    def host(t):
        return t[:end].cpu().numpy() if t.dtype != torch.bfloat16 else t[:end].view(torch.int16).cpu().numpy().view(np.uint16)

    w = host(W.make_weights(wl, dev)).copy()
    D = host(W.make_curvature(wl, dev))
    c = np.zeros(end, dtype=np.uint16)
    o = orc.Oracle(sub, end, **wl.hparams())
    times = []
    for t in range(1, steps + warmup + 1):
        g = host(W.make_grads(wl, t, dev))
        hz = np.concatenate([D * orc.probe(wl.probe_seed, t, p, 0, end) for p in range(wl.num_probes)])
        t0 = time.perf_counter()
        o.step(w, g, hz, c, wl.probe_seed, t)
        dt = time.perf_counter() - t0
        if t > warmup:
            times.append(dt)
    del gen_total
    sec = sum(times) / len(times)
    out = {"value": n_sample / sec, "unit": UNIT, "cores": 1, "kind": "oracle",
           "sample": f"{len(layers)} layers ({n_sample} params) of {wl.name}, {len(times)} timed steps of the single-threaded C oracle",
           "ms_per_step": sec * 1e3, "sample_params": n_sample}
    # the same oracle on all host cores: layers are independent, so each thread runs its own instance over a share of
    # the layers (the C call releases the interpreter lock); one more step of the same sample
    cores = os.cpu_count() or 1
    if all_cores and cores > 1 and len(sub) > 1:
        from concurrent.futures import ThreadPoolExecutor
        shares = [[] for _ in range(min(cores, len(sub)))]
        load = [0] * len(shares)
        for seg in sorted(sub, key=lambda x: -x[1]):            # longest layer first, to the least loaded thread
            k = load.index(min(load))
            shares[k].append(seg)
            load[k] += seg[1]
        oracles = [orc.Oracle(sorted(sh), end, **wl.hparams()) for sh in shares]
        t_next = steps + warmup + 1
        g = host(W.make_grads(wl, t_next, dev))
        hz = np.concatenate([D * orc.probe(wl.probe_seed, t_next, p, 0, end) for p in range(wl.num_probes)])
        with ThreadPoolExecutor(len(oracles)) as pool:
            t0 = time.perf_counter()
            list(pool.map(lambda o_: o_.step(w, g, hz, c, wl.probe_seed, t_next), oracles))
            dt = time.perf_counter() - t0
        out["all_cores"] = {"value": n_sample / dt, "unit": UNIT, "cores": len(oracles),
                            "how": "one oracle instance per thread over a share of the sample's layers, one step"}
    return out


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import torch
    from paper_2508_16905_b200 import workloads as W
    wl = W.get(args.config)
    dev = "cuda" if torch.cuda.is_available() else "cpu"
    steps, warmup = max(1, args.steps), max(0, args.warmup)
    r = time_oracle(wl, steps, warmup, budget_s=150.0, torch_device=dev)
    line = {"impl": "reference", "metric": METRIC, "value": r["value"], "unit": UNIT, "n_gpus": args.gpus,
            "steps": steps, "warmup": warmup, "ms_per_step": r["ms_per_step"], "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": wl.name, "params": wl.num_params, "layers": len(wl.table), "sample": r["sample"]},
            "cpu_baseline": {"value": r["value"], "unit": UNIT, "cores": 1, "kind": "oracle", "sample": r["sample"]},
            "e2e": {"value": r["value"], "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line))
    return 0


TARGETS = {"gpt_1p3b": 0.75, "efficientnet_b0_cifar": 0.50}     # whole-step algorithmic GB/s over the 8 TB/s nominal peak


def algorithmic_bytes(wl, codes, momentum=False):
    """What the method itself must move per step, by kernel: (sweep, update, whole step)."""
    g_b = 2 if wl.grad_dtype == "bf16" else 4
    P, n = wl.num_probes, wl.num_params
    topk = wl.topk_ppm < 1000000
    copy_params = sum(m for (_, m), cd in zip(wl.table, codes) if cd < 2)
    mom_b = 8 if momentum else 0
    sweep = n * (g_b + 4 * P) + (4 * n if topk else 0)                       # top-k: |S| is written for the selection
    update_reads, update_writes = n * (4 + g_b + mom_b // 2), n * (4 + mom_b // 2) + 2 * copy_params
    step = n * (4 + g_b + 4 * P + 4 + mom_b) + 2 * copy_params + (n / 8 if topk else 0)
    return {"sweep": sweep, "update": update_reads + update_writes, "update_writes": update_writes, "step": step,
            "step_writes": 4 * n + 2 * copy_params + (n / 8 if topk else 0) + (4 * n if momentum else 0)}


def measure(wl, hp, steps, warmup, dev, props, sample_clocks):
    """Times `steps` optimizer passes of workload `wl` (inputs resident in HBM, rotating buffer sets where one step's
    data would fit in L2), then the same number once more with the library's per-phase events.  Returns a dict."""
    import torch
    import paper_2508_16905_b200 as ta
    from paper_2508_16905_b200 import dist as D
    from paper_2508_16905_b200 import workloads as W

    P, N = wl.num_probes, wl.n_total
    l2_bytes = props.L2_cache_size
    bytes_in_per_set = N * ((2 if wl.grad_dtype == "bf16" else 4) + 4 * P)
    state_bytes = N * 6
    # rotate over R buffer sets so that consecutive steps never find their inputs in L2
    R = 1 if (bytes_in_per_set + state_bytes) > 4 * l2_bytes else max(2, -(-6 * l2_bytes // (bytes_in_per_set + state_bytes)))
    h = ta.ta_create(wl.table, N, **hp)
    path = ta.ta_path(h)
    curv = W.make_curvature(wl, dev)
    sets = []
    z = torch.empty(N, device=dev)

    def probe_products(t):
        hz = torch.empty(P * N, device=dev)
        for p in range(P):
            ta.ta_probe(h, wl.probe_seed, t, p, z)
            torch.mul(curv, z, out=hz[p * N:(p + 1) * N])
        return hz

    for r in range(R):
        g = W.make_grads(wl, r + 1, dev)
        sets.append((W.make_weights(wl, dev), g, probe_products(r + 1), torch.zeros(N, dtype=torch.int16, device=dev)))
    # With one probe |z h| = |h| whatever the sign, so a buffer of probe products serves every step.  With several, the
    # probes of step t are the ones the products must have been taken with, or the signs no longer cancel and |S| takes
    # the values {0, 2D, 4D}: every step of the run then gets its own products (as a training loop would supply them),
    # when the device has room for them.
    total_steps = warmup + 2 * steps
    per_step_hz = None
    if P > 1 and total_steps * P * N * 4 <= 0.4 * props.total_memory:
        per_step_hz = [probe_products(t) for t in range(1, total_steps + 1)]
    del z, curv
    torch.cuda.synchronize()
    stream = torch.cuda.current_stream()
    # the step of a small model takes a few microseconds: addresses and stream are marshalled once, not per call
    import ctypes
    stream_arg = ctypes.c_void_p(stream.cuda_stream)
    ptrs = [tuple(ta.dev_ptr(x) for x in one) for one in sets]
    hz_ptrs = [ta.dev_ptr(x) for x in per_step_hz] if per_step_hz is not None else None

    def one_step(t):
        w, g, hz, c = ptrs[t % R]
        if hz_ptrs is not None:
            hz = hz_ptrs[t - 1]
        ta.ta_step(h, w, g, hz, c, wl.probe_seed, t, stream_arg)

    t = 0
    for _ in range(warmup):
        t += 1
        one_step(t)
    torch.cuda.synchronize()
    D.barrier()
    uuid = str(props.uuid)
    sampler = ClockSampler(uuid if uuid.startswith("GPU-") else "GPU-" + uuid) if sample_clocks else None
    launches0 = ta.ta_launch_count(h)
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    torch.cuda.synchronize()
    e0.record(stream)
    for _ in range(steps):
        t += 1
        one_step(t)
    e1.record(stream)
    torch.cuda.synchronize()
    D.barrier()
    ms_local = e0.elapsed_time(e1)
    launches = ta.ta_launch_count(h) - launches0
    # the same K steps once more with the library's per-phase CUDA events switched on: kernel durations for
    # the roofline (kept out of the headline region: four event records per step cost ~10 us)
    ta.ta_timing_begin(h, steps)
    for _ in range(steps):
        t += 1
        one_step(t)
    ms_sweep, ms_decide, ms_update, n_timed = ta.ta_timing_end(h)
    clocks = sampler.stop() if sampler else None
    stats, status = ta.ta_stats(h)
    assert status.skipped == 0, "a benchmark step was skipped (non-finite synthetic input?)"
    n_timed = max(1, n_timed)
    del per_step_hz
    out = {"probe_signs": "one probe: any buffer serves" if P <= 1 else ("products taken with each step's own probes" if hz_ptrs is not None else
                          "products of other steps' probes (no room for one buffer per step): |S| in {0, 2D, 4D}"),
           "ms_local": ms_local, "launches": int(launches), "path": path, "codes": [s.code for s in stats], "clocks": clocks, "R": R,
           "bytes_in_per_set": bytes_in_per_set, "state_bytes": state_bytes, "l2_bytes": l2_bytes, "sets": sets,
           "phases": {"sweep": ms_sweep / n_timed, "decide_select": ms_decide / n_timed, "update": ms_update / n_timed}}
    ta.ta_destroy(h)
    return out


def recorded_reads(workload):
    """DRAM bytes read per parameter by each kernel of this workload, from the committed ncu captures; None when there
    is no capture or a kernel source changed since."""
    try:
        with open(os.path.join(ROOT, "profiles", "ncu_traffic.json")) as f:
            rec = json.load(f)
        if rec.get("sources_sha256_16") != kernel_source_hash():
            return None
        return rec["workloads"][workload]
    except Exception:
        return None


def describe(wl, m, steps, ms, peak, peak_kind, momentum=False, pipelined=False):
    """Throughput and roofline figures of one measured workload."""
    ab = algorithmic_bytes(wl, m["codes"], momentum)
    ms_step = ms / steps
    # small dense models (one cooperative launch, or two dependent launches that overlap from step to step) and the
    # pipelined launch are taken as one unit of work per step
    one_launch = m["path"] in ("one cooperative launch", "two dependent launches", "pipelined launch")
    ph = m["phases"]
    if one_launch:
        name, k_bytes, k_writes, k_ms = f"whole step ({m['path']})", ab["step"], ab["step_writes"], ms_step
    elif ph["sweep"] > ph["update"]:                      # e.g. four probes + top-k: the sweep is the longest kernel
        name, k_bytes, k_writes, k_ms = "k_sweep (statistics + Hutchinson sums)", ab["sweep"], (4 * wl.num_params if wl.topk_ppm < 1000000 else 0), ph["sweep"]
    else:
        name, k_bytes, k_writes, k_ms = "k_apply (master update + cast)", ab["update"], ab["update_writes"], ph["update"]
    achieved = k_bytes / (k_ms * 1e-3) / 1e9
    step_gbs = ab["step"] / (ms_step * 1e-3) / 1e9
    # measured DRAM traffic of the dominant kernel: its reads per parameter from an ncu capture of a workload small
    # enough to replay, times this workload's parameters; its writes are taken as the algorithmic writes of this run's
    # own code mix (lines still dirty in L2 at the end of a captured launch are a constant, not a share)
    traffic = None
    rec = recorded_reads(wl.name)
    key = ("k_pipe" if pipelined else "k_fused") if one_launch else ("k_sweep" if ph["sweep"] > ph["update"] else "k_apply")
    if rec and key in rec.get("dram_read_bytes_per_param", {}):
        traffic = max(rec["dram_read_bytes_per_param"][key] * wl.num_params + k_writes, k_bytes)
    codes = m["codes"]
    R = m["R"]
    per_set = (m["bytes_in_per_set"] + m["state_bytes"]) / 1e6
    l2 = (f"inputs of one step ({per_set:.0f} MB) exceed L2 ({m['l2_bytes'] / 1e6:.0f} MB)" if R == 1 else
          f"{R} rotating buffer sets ({R * per_set:.0f} MB) exceed L2 ({m['l2_bytes'] / 1e6:.0f} MB)")
    roofline = {"bound": "hbm", "kernel": name, "achieved": achieved, "peak": peak, "unit": "GB/s", "frac": achieved / peak,
                "peak_kind": peak_kind, "traffic": traffic, "algorithmic_bytes_per_launch": k_bytes, "ms_per_launch": k_ms,
                "phases_ms_per_step": None if one_launch else ph,
                "sweep_achieved_gbs": None if one_launch else ab["sweep"] / (ph["sweep"] * 1e-3) / 1e9,
                "step": {"algorithmic_bytes": ab["step"], "achieved_gbs": step_gbs, "frac_of_peak": step_gbs / peak,
                         "frac_of_8tbs_nominal": step_gbs / 8000.0}}
    if wl.name in TARGETS:
        roofline["step"]["target_frac_of_8tbs_nominal"] = TARGETS[wl.name]
        roofline["step"]["target_met"] = step_gbs / 8000.0 >= TARGETS[wl.name]
    summary = {"ms_per_step": ms_step, "params_per_s": wl.num_params / (ms_step * 1e-3), "params": wl.num_params,
               "layers": len(wl.table), "algorithmic_bytes": ab["step"], "hbm_gbs_algorithmic": step_gbs,
               "frac_of_measured": step_gbs / peak, "frac_of_8tbs_nominal": step_gbs / 8000.0,
               "codes": {"fp16": codes.count(0), "bf16": codes.count(1), "fp32": codes.count(2)},
               "launches_per_step": m["launches"] / steps, "path": m["path"], "l2": l2, "probe_signs": m["probe_signs"],
               "clocks": m["clocks"]}
    if wl.name in TARGETS:
        summary["target_frac_of_8tbs_nominal"] = TARGETS[wl.name]
        summary["target_met"] = summary["frac_of_8tbs_nominal"] >= TARGETS[wl.name]
    return roofline, summary, l2


def run_ours(args):
    import torch
    import paper_2508_16905_b200 as ta
    from paper_2508_16905_b200 import dist as D
    from paper_2508_16905_b200 import workloads as W

    if args.gpus > 1 and "WORLD_SIZE" not in os.environ:
        # started by hand for several GPUs: become one rank per GPU (one replica each)
        os.execvp(sys.executable, [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={args.gpus}",
                                   "--master-addr", "127.0.0.1", "--master-port", str(29500 + os.getpid() % 500),
                                   os.path.abspath(__file__)] + sys.argv[1:])
    rank, local_rank, world = D.init("nccl")
    torch.cuda.set_device(local_rank if world > 1 else 0)
    dev = torch.device("cuda", torch.cuda.current_device())
    props = torch.cuda.get_device_properties(dev)
    over = {"t_ctrl": args.t_ctrl} if args.t_ctrl else {}
    wl = W.get(args.config, **over)
    steps, warmup = max(1, args.steps), max(3, args.warmup)
    P, N = wl.num_probes, wl.n_total
    flags = ta.TA_FLAG_INPUTS_FINITE if args.inputs_finite else 0
    hp = dict(wl.hparams(), momentum=args.momentum, weight_decay=args.weight_decay, flags=flags)
    peak, peak_kind = measured_peak()

    m = measure(wl, hp, steps, warmup, dev, props, sample_clocks=(rank == 0))
    ms, units = D.aggregate(m["ms_local"], wl.num_params * steps, device=dev)
    sets = m.pop("sets")

    # ---- end to end through the C ABI with HOST buffers (pinned), copies inside the timed region
    e2e = None
    if not args.no_e2e:
        e2e_steps = max(1, min(steps, args.e2e_steps))
        w_d, g_d, hz_d, c_d = sets[0]
        wh, gh, hzh, ch = (x.cpu().pin_memory() for x in (w_d, g_d, hz_d, c_d))
        h2 = ta.ta_create(wl.table, N, **hp)
        ta.ta_step_host(h2, wh, gh, hzh, ch, wl.probe_seed, 1)          # warm-up: allocates the staging buffers
        torch.cuda.synchronize()
        D.barrier()
        t0 = time.perf_counter()
        for s in range(e2e_steps):
            ta.ta_step_host(h2, wh, gh, hzh, ch, wl.probe_seed, 2 + s)
        torch.cuda.synchronize()
        dt_ms = (time.perf_counter() - t0) * 1e3
        D.barrier()
        codes2 = ta.ta_precision_codes(h2)
        copy_params = sum(n for (_, n), cd in zip(wl.table, codes2) if cd < 2)
        span = wl.table[-1][0] + wl.table[-1][1] - wl.table[0][0]
        ms2, units2 = D.aggregate(dt_ms, wl.num_params * e2e_steps, device=dev)
        e2e = {"value": units2 / (ms2 / 1e3), "unit": UNIT, "steps": e2e_steps, "ms_per_step": ms2 / e2e_steps,
               "h2d_bytes_per_step": int(m["bytes_in_per_set"] + 4 * N), "d2h_bytes_per_step": int(4 * span + 2 * copy_params),
               "api": "ta_step_host (pinned host tensors in, new weights and 16-bit copies out)"}
        del wh, gh, hzh, ch
        ta.ta_destroy(h2)
    del sets
    torch.cuda.empty_cache()

    # ---- one replica only: the other configurations, and the paths a caller can opt into
    configs, paths = None, None
    if world == 1 and not args.headline_only:
        roofline0, summary0, _ = describe(wl, m, steps, ms, peak, peak_kind, bool(args.momentum))
        configs = {wl.name: summary0}
        for name in W.NAMES:
            if name == wl.name:
                continue
            w2 = W.get(name)
            k = max(steps, 50) if w2.num_params < 5e7 else steps
            m2 = measure(w2, w2.hparams(), k, warmup, dev, props, sample_clocks=True)
            m2.pop("sets")
            torch.cuda.empty_cache()
            configs[name] = describe(w2, m2, k, m2["ms_local"], peak, peak_kind)[1]
        big_dense = wl.topk_ppm == 1000000 and wl.num_params > (16 << 20) and not args.momentum and not args.weight_decay
        if big_dense and not args.inputs_finite:
            # TA_FLAG_INPUTS_FINITE: the caller vouches for finite inputs; a step with decisions (this workload decides at
            # every step) and a step between decisions (T_ctrl beyond the run: the single pass)
            paths = {"flag": "TA_FLAG_INPUTS_FINITE"}
            for label, extra in (("step_with_decisions", {}), ("step_between_decisions", {"t_ctrl": 1000000})):
                w3 = W.get(args.config, **dict(over, **extra))
                for which, fl in (("default", 0), ("inputs_finite", ta.TA_FLAG_INPUTS_FINITE)):
                    if label == "step_with_decisions" and which == "default":
                        paths.setdefault(label, {})[which] = summary0
                        continue
                    m3 = measure(w3, dict(w3.hparams(), flags=fl), steps, warmup, dev, props, sample_clocks=True)
                    m3.pop("sets")
                    torch.cuda.empty_cache()
                    paths.setdefault(label, {})[which] = describe(w3, m3, steps, m3["ms_local"], peak, peak_kind, pipelined=bool(fl))[1]

    if rank != 0:
        D.shutdown()
        return 0

    roofline, summary, l2 = describe(wl, m, steps, ms, peak, peak_kind, bool(args.momentum), pipelined=bool(flags))
    cpu = None
    if world == 1 and not args.no_cpu_baseline:
        cpu = time_oracle(wl, steps=2, warmup=0, budget_s=20.0, torch_device=dev, all_cores=True)
        cpu = {k: cpu[k] for k in ("value", "unit", "cores", "kind", "sample", "all_cores") if k in cpu}

    codes = m["codes"]
    line = {"metric": METRIC, "value": units / (ms / 1e3), "unit": UNIT, "n_gpus": world, "steps": steps, "warmup": warmup,
            "ms_per_step": ms / steps, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f32", "data": "synthetic",
            "config": {"workload": wl.name, "params": wl.num_params, "layers": len(wl.table), "grad_dtype": wl.grad_dtype,
                       "num_probes": P, "topk_ppm": wl.topk_ppm, "t_ctrl": wl.t_ctrl, "momentum": args.momentum,
                       "weight_decay": args.weight_decay, "flags": flags, "parallelism": f"replicas x{world}", "l2": l2, "probe_signs": m["probe_signs"],
                       "codes": {"fp16": codes.count(0), "bf16": codes.count(1), "fp32": codes.count(2)}},
            "hbm_gbs_algorithmic": roofline["step"]["achieved_gbs"],
            "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": m["launches"], "clocks": m["clocks"],
            "configs": configs, "paths": paths}
    print(json.dumps(line))
    D.shutdown()
    return 0


def run_power(args):
    """Times ta_power_iterate (Sec. 3.2 support sweeps) on the workload's layer table; one JSON line."""
    import torch
    import paper_2508_16905_b200 as ta
    from paper_2508_16905_b200 import workloads as W
    torch.cuda.set_device(0)
    wl = W.get(args.config)
    N, L, m = wl.n_total, len(wl.table), args.deflate
    h = ta.ta_create(wl.table, N, **wl.hparams())
    gen = torch.Generator(device="cuda").manual_seed(1)
    u = torch.randn(N, generator=gen, device="cuda")
    hu = torch.randn(N, generator=gen, device="cuda")
    V = torch.randn(max(m, 1) * N, generator=gen, device="cuda") if m else None
    lam_v = torch.rand(max(m, 1) * L, generator=gen, device="cuda") if m else None
    out, lam = torch.empty(N, device="cuda"), torch.empty(L, device="cuda")
    steps, warmup = max(1, args.steps), max(3, args.warmup)
    flush = torch.empty(64 << 20, dtype=torch.float32, device="cuda")       # 256 MB > L2, written between iterations
    for _ in range(warmup):
        ta.ta_power_iterate(h, u, hu, V, lam_v, m, out, lam)
    times = []
    for _ in range(steps):
        flush.fill_(1.0)
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        ta.ta_power_iterate(h, u, hu, V, lam_v, m, out, lam)
        e1.record()
        torch.cuda.synchronize()
        times.append(e0.elapsed_time(e1))
    ms = sum(times) / len(times)
    # algorithmic bytes: projections read u and m vectors; dots read u, Hu and m vectors; the write pass reads Hu and
    # m vectors and writes u_next
    bytes_alg = wl.num_params * 4 * ((1 + m if m else 0) + (2 + m) + (1 + m) + 1)
    peak, kind = measured_peak()
    print(json.dumps({"metric": "power-iteration step params/sec", "value": wl.num_params / (ms * 1e-3), "unit": UNIT,
                      "n_gpus": 1, "steps": steps, "warmup": warmup, "ms_per_step": ms, "higher_is_better": True,
                      "dtype": "f32", "data": "synthetic",
                      "config": {"workload": wl.name, "params": wl.num_params, "layers": L, "deflated_vectors": m,
                                 "l2": "256 MB written between iterations"},
                      "roofline": {"bound": "hbm", "achieved": bytes_alg / (ms * 1e-3) / 1e9, "peak": peak, "unit": "GB/s",
                                   "frac": bytes_alg / (ms * 1e-3) / 1e9 / peak, "peak_kind": kind, "traffic": None,
                                   "algorithmic_bytes": bytes_alg}}))
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--config", default="gpt_1p3b")
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--headline-only", action="store_true", help="skip the other configurations and the opt-in paths")
    ap.add_argument("--momentum", type=float, default=0.0)
    ap.add_argument("--weight-decay", type=float, default=0.0)
    ap.add_argument("--t-ctrl", type=int, default=0, help="override the workload's control interval T_ctrl")
    ap.add_argument("--inputs-finite", action="store_true", help="create the handle with TA_FLAG_INPUTS_FINITE")
    ap.add_argument("--op", default="step", choices=["step", "power"], help="step: the optimizer pass (default); power: ta_power_iterate")
    ap.add_argument("--deflate", type=int, default=0, help="--op power: number of deflated eigenvectors")
    args = ap.parse_args()
    if args.op == "power":
        return run_power(args)
    if args.impl == "reference":
        return run_reference(args)
    return run_ours(args)


if __name__ == "__main__":
    sys.exit(main())
