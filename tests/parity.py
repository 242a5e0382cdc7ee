"""Shared harness of the GPU parity tests: runs the CUDA library (through its C ABI binding) and the
CPU oracle on the same seeded inputs and compares them element by element.

Tolerances (the bar the method's specification sets):
  codes, masks, k          bit-exact, except layers that either side flags as within 1e-5 relative
                           of a decision threshold (those are returned as a list)
  lambda_max, threshold,   bit-exact (the probe sums are exact sign flips added in one fixed order)
  eta_scale
  variance, EMA variance   1e-5 relative (+ the oracle's own rounding bound, var_tolerance)
  mean, EMA mean           1e-5 * max(|mean|, sqrt(var + mean^2))
  master weights           <= 2 ulp (float);  16-bit copies <= 1 ulp of their format
"""
import os
from concurrent.futures import ThreadPoolExecutor

import numpy as np
import torch

import paper_2508_16905_b200 as ta
from oracle import oracle as orc


def ulp_f32(a, b):
    ia = a.view(np.int32).astype(np.int64)
    ib = b.view(np.int32).astype(np.int64)
    ia = np.where(ia < 0, -(ia & 0x7FFFFFFF), ia)
    ib = np.where(ib < 0, -(ib & 0x7FFFFFFF), ib)
    return np.abs(ia - ib)


def ulp_16(a, b):
    ia = a.astype(np.int64)
    ib = b.astype(np.int64)
    ia = np.where(ia >= 0x8000, -(ia & 0x7FFF), ia)
    ib = np.where(ib >= 0x8000, -(ib & 0x7FFF), ib)
    return np.abs(ia - ib)


def to_host_bits(t):
    """torch tensor -> numpy; bfloat16 / float16 as uint16 bit patterns."""
    if t.dtype in (torch.bfloat16, torch.float16):
        return t.view(torch.int16).cpu().numpy().view(np.uint16)
    if t.dtype == torch.int16:
        return t.cpu().numpy().view(np.uint16)
    return t.cpu().numpy()


def segment_mask(table, n_total):
    inside = np.zeros(n_total, dtype=bool)
    for off, n in table:
        inside[off:off + n] = True
    return inside


def oracle_hz(D_host, P, seed, t):
    """Hz = D * z with the ORACLE's probes, [P * n_total] float32 on the host."""
    n = D_host.size
    return np.concatenate([D_host * orc.probe(seed, t, p, 0, n) for p in range(P)])


def var_tolerance(var, mean, n):
    """1e-5 relative, plus what the ORACLE's two-pass variance can be off by when the variance is (next to) zero:
    its mean is a sequential double sum, wrong by at most n * 2^-53 * |mean|, and the square of that error is
    what it reports for a constant layer.  (The CUDA side sums differences from a pivot and reports exactly 0.)"""
    return 1e-5 * var + (n * 1.2e-16 * mean) ** 2 + 1e-37


def compare_stats(gl, ol, where="", n=1):
    """gl: ta_layer_stats, ol: oracle Layer.  Returns True when the layer is flagged near a threshold."""
    mu, var = ol.grad_mean, ol.grad_var
    scale = max(abs(mu), float(np.sqrt(var + mu * mu)))
    assert abs(gl.grad_mean - mu) <= 1e-5 * scale + 1e-30, (where, "grad_mean", gl.grad_mean, mu)
    assert abs(gl.grad_var - var) <= var_tolerance(var, mu, n), (where, "grad_var", gl.grad_var, var)
    em, ev = ol.ema_mean, ol.ema_var
    assert abs(gl.ema_var - ev) <= 1e-5 * abs(ev) + (n * 1.2e-16 * em) ** 2 + 1e-37, (where, "ema_var", gl.ema_var, ev)
    assert abs(gl.ema_mean - em) <= 1e-5 * max(abs(em), float(np.sqrt(abs(ev) + em * em))) + 1e-30, (where, "ema_mean")
    assert np.float32(gl.lambda_max) == np.float32(ol.lambda_max), (where, "lambda_max", gl.lambda_max, ol.lambda_max)
    assert np.float32(gl.topk_threshold) == np.float32(ol.topk_threshold), (where, "threshold", gl.topk_threshold, ol.topk_threshold)
    assert gl.k == ol.k or ol.k == 0, (where, "k", gl.k, ol.k)
    assert abs(gl.topk_mass - ol.topk_mass) <= 1e-5 * max(ol.topk_mass, 1e-30) or ol.k == 0, (where, "topk_mass", gl.topk_mass, ol.topk_mass)
    near = bool(gl.near_threshold or ol.near_threshold)
    if not near:
        assert gl.code == ol.code, (where, "code", gl.code, ol.code)
        assert np.float32(gl.eta_scale) == np.float32(ol.eta_scale), (where, "eta_scale", gl.eta_scale, ol.eta_scale)
    return near


class ShardedOracle:
    """Several oracle instances, each over a share of the layers, stepped on one host thread each (layers are
    independent and the C call releases the interpreter lock), behind the interface of one oracle.  Only for
    finite inputs: a step that one share would skip is a whole-step skip for a single oracle, so it is refused here."""

    def __init__(self, table, n_total, threads, **hp):
        order = sorted(range(len(table)), key=lambda j: -table[j][1])
        shares, load = [[] for _ in range(max(1, min(threads, len(table))))], [0] * max(1, min(threads, len(table)))
        for j in order:                                   # longest layer first, to the least loaded share
            k = load.index(min(load))
            shares[k].append(j)
            load[k] += table[j][1]
        self.shares = [sorted(sh) for sh in shares if sh]
        self.parts = [orc.Oracle([table[j] for j in sh], n_total, **hp) for sh in self.shares]
        self.where = {j: (k, i) for k, sh in enumerate(self.shares) for i, j in enumerate(sh)}
        self.n_layers = len(table)
        self.pool = ThreadPoolExecutor(len(self.parts))

    def set_lr(self, eta0):
        for o in self.parts:
            o.set_lr(eta0)

    def step(self, w, g, hz, c, seed, t):
        skipped = list(self.pool.map(lambda o: o.step(w, g, hz, c, seed, t), self.parts))
        assert not any(skipped), "sharded oracle: non-finite input (use a single oracle for skip semantics)"
        return False

    def layers(self):
        per = [o.layers() for o in self.parts]
        return [per[self.where[j][0]][self.where[j][1]] for j in range(self.n_layers)]

    def status(self):
        st = [o.status() for o in self.parts]
        out = st[0]
        out.nonfinite_count = sum(s.nonfinite_count for s in st)
        out.near_threshold_count = sum(s.near_threshold_count for s in st)
        return out

    def mask(self):
        m = self.parts[0].mask()
        for o in self.parts[1:]:
            m |= o.mask()
        return m

    def codes(self):
        return np.array([ly.code for ly in self.layers()], dtype=np.uint8)


class ParityRun:
    """One workload on both sides.  `layers` restricts the oracle (and the comparison) to a subset of
    the layers: layers are independent, so the oracle of a subset equals the full oracle on that subset."""

    def __init__(self, table, n_total, hp, w0, layers=None, threads=1):
        self.table, self.n_total, self.hp = list(table), int(n_total), dict(hp)
        self.layers = list(range(len(table))) if layers is None else list(layers)
        self.sub_table = [self.table[l] for l in self.layers]
        # every workspace of the library between guard words, checked after each compared step
        self.h = ta.ta_create(self.table, self.n_total, **dict(self.hp, flags=self.hp.get("flags", 0) | ta.TA_FLAG_GUARD_WORKSPACES))
        threads = min(int(threads), os.cpu_count() or 1)
        ohp = {k: v for k, v in self.hp.items() if k != "flags"}      # flags choose among CUDA paths; the method is the same
        self.o = (orc.Oracle(self.sub_table, self.n_total, **ohp) if threads <= 1 else
                  ShardedOracle(self.sub_table, self.n_total, threads, **ohp))
        self.w_dev = w0.to("cuda").clone()
        self.c_dev = torch.full((self.n_total,), 0x5A5A, dtype=torch.int16, device="cuda")
        self.w_host = to_host_bits(w0).copy()
        self.c_host = np.full(self.n_total, 0x5A5A, dtype=np.uint16)
        self.w_start = self.w_host.copy()
        self.inside_all = segment_mask(self.table, self.n_total)
        self.inside_sub = segment_mask(self.sub_table, self.n_total)
        self.near_list = []
        self.layer_steps = 0
        self.max_w_ulp = 0
        self.max_c_ulp = 0

    def step(self, t, g_dev, hz_host, seed, hz_dev=None, check=True):
        """hz_host: oracle-side Hz (numpy [P*n_total]) or None; hz_dev defaults to a copy of hz_host."""
        if hz_host is not None and hz_dev is None:
            hz_dev = torch.from_numpy(hz_host).to("cuda")
        ta.ta_step(self.h, self.w_dev, g_dev, hz_dev, self.c_dev, seed, t)
        skipped = self.o.step(self.w_host, to_host_bits(g_dev), hz_host, self.c_host, seed, t)
        if check:
            self.check(t)
        return skipped

    def check(self, t):
        stats, status = ta.ta_stats(self.h)
        ta.ta_test_check_guards(self.h)
        ost = self.o.status()
        full = len(self.layers) == len(self.table)
        if full:
            assert (status.step, status.skipped, status.nonfinite_count) == (ost.step, ost.skipped, ost.nonfinite_count)
        olayers = self.o.layers()
        codes_gpu = ta.ta_precision_codes(self.h)
        near_now = set()
        self.layer_steps += len(self.layers)
        for j, l in enumerate(self.layers):
            if compare_stats(stats[l], olayers[j], where=f"step {t} layer {l}", n=self.table[l][1]):
                near_now.add(l)
                self.near_list.append((t, l, stats[l].code, olayers[j].code))
            assert codes_gpu[l] == stats[l].code
        w_gpu = self.w_dev.cpu().numpy()
        c_gpu = to_host_bits(self.c_dev)
        # gaps are never touched
        assert np.array_equal(w_gpu[~self.inside_all].view(np.uint32), self.w_start[~self.inside_all].view(np.uint32))
        assert np.all(c_gpu[~self.inside_all] == 0x5A5A)
        for j, l in enumerate(self.layers):
            off, n = self.table[l]
            du = ulp_f32(w_gpu[off:off + n], self.w_host[off:off + n])
            m = int(du.max())
            self.max_w_ulp = max(self.max_w_ulp, m)
            if stats[l].code != olayers[j].code or np.float32(stats[l].eta_scale) != np.float32(olayers[j].eta_scale):
                assert l in near_now
                # a listed near-threshold layer took another branch: resynchronise the oracle side to the GPU
                self.w_host[off:off + n] = w_gpu[off:off + n]
                self.c_host[off:off + n] = c_gpu[off:off + n]
                continue
            assert m <= 2, (t, l, "master weights differ by", m, "ulp")
            dc = ulp_16(c_gpu[off:off + n], self.c_host[off:off + n])
            mc = int(dc.max())
            self.max_c_ulp = max(self.max_c_ulp, mc)
            assert mc <= 1, (t, l, "16-bit copy differs by", mc, "ulp")
        # masks
        ppm = self.hp.get("topk_ppm", 1000000)
        if ppm < 1000000:
            mg = ta.ta_masks_to_host(self.h)
            mo = self.o.mask()
            if full:
                assert np.array_equal(mg, mo), (t, "mask words differ", int((mg != mo).sum()))
            else:
                idx = np.flatnonzero(self.inside_sub)
                bg = (mg[idx >> 5] >> (idx & 31).astype(np.uint32)) & 1
                bo = (mo[idx >> 5] >> (idx & 31).astype(np.uint32)) & 1
                assert np.array_equal(bg, bo)
        else:
            assert ta.ta_masks(self.h) == (None, 0)

    def report(self, name, max_fraction=0.01):
        """Lists the near-threshold exceptions of the run (layer-steps where either side flagged a statistic within
        1e-5 relative of a decision threshold, the only place where codes may differ) and bounds their number."""
        print(f"{name}: {self.layer_steps} layer-steps compared, {len(self.near_list)} near a threshold; "
              f"max distance master weights {self.max_w_ulp} ulp, 16-bit copies {self.max_c_ulp} ulp")
        for t, l, code_gpu, code_oracle in self.near_list:
            print(f"  near threshold: step {t} layer {l} code gpu {code_gpu} oracle {code_oracle}")
        assert len(self.near_list) <= max(1, int(max_fraction * self.layer_steps)), "too many near-threshold layer-steps"
