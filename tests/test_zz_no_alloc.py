"""ta_grad_moments_static: the entry point for callers that must not allocate device memory.

Some users of this library run where cudaMalloc is off limits at the moment the statistics are
needed: a plug-in inside an application that owns and has already handed out all device memory, a
callback running under an allocator lock, a job whose pool was sized up front.  For them the library
offers the per-layer gradient moments through a call whose scratch is a fixed array inside the
library image.  This test calls it through the C ABI twice in a row (the array is shared between
calls and keeps old contents, so the second call must not be disturbed by the first) and checks
each result against ta_step + ta_stats on the same gradient and against the CPU oracle's moments,
within the tolerances of the other parity tests.  After the warm-up call (which is when the CUDA
runtime loads the library's device code) a call must leave the free device memory exactly as it
found it.  It is collected last on purpose and needs no state from other tests.
"""
import numpy as np
import pytest
import torch

import paper_2508_16905_b200 as ta
from oracle import oracle as orc
from tests.parity import to_host_bits, var_tolerance

pytestmark = pytest.mark.gpu


def _table():
    # ragged layers, odd offsets, gaps, one layer spanning several 16384-element tiles
    lengths = [1, 33, 4097, 70001, 16384, 129, 250000]
    table, off = [], 3
    for j, n in enumerate(lengths):
        off += (0, 5, 1, 7)[j % 4]
        table.append((off, n))
        off += n
    return table, (off + 7) // 4 * 4


@pytest.mark.parametrize("grad_dtype", ["f32", "bf16"])
def test_static_moments_match_the_allocating_path_twice_in_a_row(grad_dtype):
    table, n_total = _table()
    L = len(table)
    h = ta.ta_create(table, n_total, grad_dtype=grad_dtype)
    w = torch.zeros(n_total, device="cuda")
    c = torch.zeros(n_total, dtype=torch.int16, device="cuda")
    mean_var = torch.full((2 * L,), float("nan"), dtype=torch.float64, device="cuda")
    bad = torch.full((L,), -1, dtype=torch.int32, device="cuda")
    gen = torch.Generator(device="cuda").manual_seed(7)
    for call, (shift, scale) in enumerate([(0.25, 1e-3), (-3e-4, 2e-2)], start=1):
        g = torch.randn(n_total, generator=gen, device="cuda") * scale + shift
        if grad_dtype == "bf16":
            g = g.to(torch.bfloat16)
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        ta.ta_grad_moments_static(table, g, grad_dtype, mean_var, bad)
        torch.cuda.synchronize()
        if call > 1:       # the first call on a device is the documented warm-up; later ones allocate nothing
            assert torch.cuda.mem_get_info()[0] == free_before
        ta.ta_step(h, w, g, None, c, 0, call)
        stats, status = ta.ta_stats(h)
        got = mean_var.cpu().numpy()
        assert status.skipped == 0 and np.all(bad.cpu().numpy() == 0)
        for l in range(L):
            mu, var = got[2 * l], got[2 * l + 1]
            ref_mu, ref_var = stats[l].grad_mean, stats[l].grad_var
            scale_l = max(abs(ref_mu), float(np.sqrt(ref_var + ref_mu * ref_mu)))
            assert abs(mu - ref_mu) <= 1e-5 * scale_l + 1e-30, (call, l, mu, ref_mu)
            assert abs(var - ref_var) <= 1e-5 * ref_var + 1e-37, (call, l, var, ref_var)
            # and against the oracle's two-pass moments of the same values
            off, n = table[l]
            gl = g[off:off + n].float().cpu().numpy()
            o_mu, o_var = orc.moments(gl)
            assert abs(mu - o_mu) <= 1e-5 * max(abs(o_mu), float(np.sqrt(o_var + o_mu * o_mu))) + 1e-30, (call, l, mu, o_mu)
            assert abs(var - o_var) <= var_tolerance(o_var, o_mu, n), (call, l, var, o_var)


def test_static_moments_count_non_finite_values_and_reject_oversize_tables():
    table, n_total = _table()
    g = torch.ones(n_total, device="cuda")
    g[table[3][0] + 5] = float("inf")
    g[table[3][0] + 6] = float("nan")
    g[0] = float("nan")                                   # in a gap: never read
    mean_var = torch.zeros(2 * len(table), dtype=torch.float64, device="cuda")
    bad = torch.zeros(len(table), dtype=torch.int32, device="cuda")
    ta.ta_grad_moments_static(table, g, "f32", mean_var, bad)
    assert bad.cpu().tolist() == [0, 0, 0, 2, 0, 0, 0]
    assert mean_var.cpu().numpy()[0] == 1.0 and mean_var.cpu().numpy()[1] == 0.0
    # beyond the fixed scratch: a clear error, nothing launched
    with pytest.raises(ta.TriAccelError) as e:
        ta.ta_grad_moments_static([(0, 16384 * 32768 + 1)], g, "f32", mean_var, None)
    assert e.value.code == ta.TA_ERR_ARG and "TA_STATIC_MAX_TILES" in str(e.value)
    with pytest.raises(ta.TriAccelError) as e:
        ta.ta_grad_moments_static([(8 * i, 8) for i in range(129)], g, "f32", mean_var, None)
    assert e.value.code == ta.TA_ERR_ARG
