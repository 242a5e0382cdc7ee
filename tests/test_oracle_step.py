"""Pins for the oracle's step: EMAs, precision codes, step size, update and cast (CPU only)."""
import numpy as np
import pytest
import torch

from oracle import oracle as orc

F = np.float32


def _mk(table, n_total, **hp):
    o = orc.Oracle(table, n_total, **hp)
    w = np.zeros(n_total, dtype=F)
    c = np.full(n_total, 0xABCD, dtype=np.uint16)
    return o, w, c


def _hz_for(D, P, seed, t):
    n = D.size
    return np.concatenate([D * orc.probe(seed, t, p, 0, n) for p in range(P)])


# ---------------------------------------------------------------- EMAs (Sec. 3.1 recurrence)

def test_ema_closed_form_for_constant_input():
    n, beta = 4096, 0.9
    rng = np.random.default_rng(1)
    g = (rng.standard_normal(n) * 1e-2 + 3e-3).astype(F)
    mu, var = orc.moments(g)
    o, w, c = _mk([(0, n)], n, beta=beta)
    b = float(F(beta))
    for t in range(1, 31):
        o.step(w, g, None, c, 0, t)
        ly = o.layers()[0]
        assert ly.grad_mean == mu and ly.grad_var == var
        assert ly.ema_var == pytest.approx((1 - b ** t) * var, rel=5e-6)     # float state, t roundings
        assert ly.ema_mean == pytest.approx((1 - b ** t) * mu, rel=5e-6)


def test_ema_beta_zero_is_current_moment():
    n = 1000
    o, w, c = _mk([(0, n)], n, beta=0.0)
    for t in range(1, 4):
        g = (np.random.default_rng(t).standard_normal(n) * 10.0 ** -t).astype(F)
        o.step(w, g, None, c, 0, t)
        mu, var = orc.moments(g)
        ly = o.layers()[0]
        assert ly.ema_var == F(var) and ly.ema_mean == F(mu)


# ---------------------------------------------------------------- precision codes (Sec. 3.1 cases, Sec. 3.2 promotion)

def _code_for(var_exact, lam, tau_low, tau_high, tau_curv):
    # two elements +-a give Var = a^2 exactly; beta = 0 makes v = Var; Hz = lam*z makes lambda = lam
    a = np.sqrt(var_exact)
    g = np.array([a, -a, 0, 0, 0, 0, 0, 0], dtype=F)[:2]
    n_total = 8
    gg = np.zeros(n_total, dtype=F); gg[:2] = g
    o, w, c = _mk([(0, 2)], n_total, beta=0.0, tau_low=tau_low, tau_high=tau_high, tau_curv=tau_curv)
    hz = None
    if lam is not None:
        hz = _hz_for(np.full(n_total, lam, dtype=F), 1, 0, 1)
    o.step(w, gg, hz, c, 0, 1)
    ly = o.layers()[0]
    assert ly.ema_var == F(var_exact)
    return ly.code


def test_code_boundaries_are_as_printed():
    lo, hi = 2.0 ** -20, 2.0 ** -16
    assert _code_for(2.0 ** -22, None, lo, hi, 0.9) == orc.FP16      # v < tau_low
    assert _code_for(2.0 ** -20, None, lo, hi, 0.9) == orc.BF16      # v == tau_low  -> BF16
    assert _code_for(2.0 ** -18, None, lo, hi, 0.9) == orc.BF16
    assert _code_for(2.0 ** -16, None, lo, hi, 0.9) == orc.FP32      # v == tau_high -> FP32
    assert _code_for(2.0 ** -14, None, lo, hi, 0.9) == orc.FP32


def test_promotion_is_strict_and_one_level():
    lo, hi = 2.0 ** -20, 2.0 ** -16
    assert _code_for(2.0 ** -22, 0.5, lo, hi, 0.5) == orc.FP16       # lambda == tau_curv: no promotion
    assert _code_for(2.0 ** -22, 0.75, lo, hi, 0.5) == orc.BF16      # FP16 -> BF16
    assert _code_for(2.0 ** -18, 0.75, lo, hi, 0.5) == orc.FP32      # BF16 -> FP32
    assert _code_for(2.0 ** -14, 0.75, lo, hi, 0.5) == orc.FP32      # stays FP32


def test_code_monotonicity():
    lo, hi = 2.0 ** -20, 2.0 ** -16
    vs = [2.0 ** e for e in range(-26, -8, 2)]
    for lam in [None, 0.1, 0.9]:
        codes = [_code_for(v, lam, lo, hi, 0.5) for v in vs]
        assert codes == sorted(codes)                                # non-decreasing in v
    for v in vs:
        codes = [_code_for(v, lam, lo, hi, 0.5) for lam in [0.1, 0.4, 0.5, 0.6, 2.0]]
        assert codes == sorted(codes)                                # non-decreasing in lambda
        codes = [_code_for(v, None, lo * s, hi * s, 0.5) for s in [0.25, 1, 4, 64]]
        assert codes == sorted(codes, reverse=True)                  # non-increasing in the thresholds


def test_default_code_and_control_interval():
    n = 64
    rng = np.random.default_rng(0)
    o, w, c = _mk([(0, n)], n, beta=0.0, tau_low=1e-3, tau_high=1e-2, t_ctrl=3)
    small = (rng.standard_normal(n) * 1e-4).astype(F)     # -> FP16 once a decision is taken
    big = rng.standard_normal(n).astype(F)                # -> FP32
    seen = []
    for t, g in zip(range(1, 8), [small, small, small, big, big, big, small]):
        o.step(w, g, None, c, 0, t)
        seen.append(int(o.layers()[0].code))
    #        t = 1        2        3 (ctrl)  4         5         6 (ctrl)  7
    assert seen == [orc.BF16, orc.BF16, orc.FP16, orc.FP16, orc.FP16, orc.FP32, orc.FP32]


def test_near_threshold_listing():
    lo = 2.0 ** -20
    a = np.sqrt(lo) * (1 + 2e-6)
    gg = np.zeros(8, dtype=F); gg[:2] = [a, -a]
    o, w, c = _mk([(0, 2)], 8, beta=0.0, tau_low=lo, tau_high=1.0)
    o.step(w, gg, None, c, 0, 1)
    assert o.layers()[0].near_threshold == 1 and o.status().near_threshold_count == 1


# ---------------------------------------------------------------- step size (Sec. 3.2)

def test_step_size_closed_form():
    n = 8
    g = np.arange(1, n + 1, dtype=F)
    for alpha, lam in [(1.0, 0.0), (0.0, 0.7), (1.0, 0.7), (3.5, 1e-3), (0.25, 123.0)]:
        o, w, c = _mk([(0, n)], n, alpha=alpha, eta0=0.1)
        hz = _hz_for(np.full(n, lam, dtype=F), 1, 3, 1) if lam else None
        o.step(w, g, hz, c, 3, 1)
        s = o.layers()[0].eta_scale
        assert s == F(1.0) / (F(1.0) + F(alpha) * F(lam))            # three float roundings
        if lam == 0.0 or alpha == 0.0:
            assert s == 1.0
        eta = F(F(0.1) * s)
        want = (0.0 - np.float64(eta) * g.astype(np.float64)).astype(F)
        assert np.array_equal(w, want)


def test_step_size_decreases_with_curvature_and_alpha():
    def scale(alpha, lam):
        o, w, c = _mk([(0, 8)], 8, alpha=alpha)
        o.step(w, np.ones(8, dtype=F), _hz_for(np.full(8, lam, dtype=F), 1, 0, 1), c, 0, 1)
        return o.layers()[0].eta_scale
    s = [scale(1.0, lam) for lam in [0.01, 0.1, 1, 10]]
    assert s == sorted(s, reverse=True) and 0 < min(s) and max(s) <= 1
    s = [scale(al, 0.5) for al in [0.0, 0.5, 1, 2]]
    assert s == sorted(s, reverse=True)


def test_curvature_is_reused_when_hz_is_absent():
    n = 128
    D = np.linspace(0.1, 2.0, n).astype(F)
    o, w, c = _mk([(0, n)], n, topk_ppm=500000)
    g = np.ones(n, dtype=F)
    o.step(w, g, _hz_for(D, 1, 0, 1), c, 0, 1)
    before, mask = o.layers()[0], o.mask().copy()
    o.step(w, g, None, c, 0, 2)
    after = o.layers()[0]
    assert (after.lambda_max, after.topk_threshold, after.k, after.eta_scale) == \
           (before.lambda_max, before.topk_threshold, before.k, before.eta_scale)
    assert np.array_equal(mask, o.mask())


# ---------------------------------------------------------------- update and cast

def test_zero_gradient_is_identity_and_copy_is_the_cast():
    table, n_total = [(0, 100), (104, 50), (160, 1)], 168
    rng = np.random.default_rng(0)
    w0 = (rng.standard_normal(n_total) * 0.05).astype(F)
    for tau_low, tau_high, code in [(1.0, 2.0, orc.FP16), (-1.0, 2.0, orc.BF16), (-2.0, -1.0, orc.FP32)]:
        o = orc.Oracle(table, n_total, tau_low=tau_low, tau_high=tau_high)
        w, c = w0.copy(), np.full(n_total, 0xABCD, dtype=np.uint16)
        o.step(w, np.zeros(n_total, dtype=F), None, c, 0, 1)
        assert np.array_equal(w.view(np.uint32), w0.view(np.uint32))
        inside = np.zeros(n_total, dtype=bool)
        for off, n in table:
            inside[off:off + n] = True
        assert np.all(c[~inside] == 0xABCD)                              # gaps never touched
        if code == orc.FP32:
            assert np.all(c == 0xABCD)                                   # FP32 layers keep no 16-bit copy
        elif code == orc.FP16:
            assert np.array_equal(c[inside], w0[inside].astype(np.float16).view(np.uint16))
        else:
            ref = torch.from_numpy(w0).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
            assert np.array_equal(c[inside], ref[inside])
        assert list(o.codes()) == [code] * 3


def test_update_exact_on_small_integers():
    n = 64
    rng = np.random.default_rng(1)
    w0 = rng.integers(-100, 100, n).astype(F)
    g = rng.integers(-100, 100, n).astype(F)
    o = orc.Oracle([(0, n)], n, eta0=0.25, alpha=0.0)
    w, c = w0.copy(), np.zeros(n, dtype=np.uint16)
    o.step(w, g, None, c, 0, 1)
    assert np.array_equal(w, w0 - F(0.25) * g)


def test_bf16_gradients_are_widened_exactly():
    n = 256
    rng = np.random.default_rng(2)
    g32 = (rng.standard_normal(n) * 1e-3).astype(F)
    gb = torch.from_numpy(g32).to(torch.bfloat16)
    g_bits = gb.view(torch.int16).numpy().view(np.uint16)
    g_wide = gb.to(torch.float32).numpy()
    a = orc.Oracle([(0, n)], n, grad_dtype="bf16")
    b = orc.Oracle([(0, n)], n)
    wa, wb = np.ones(n, dtype=F), np.ones(n, dtype=F)
    ca, cb = np.zeros(n, dtype=np.uint16), np.zeros(n, dtype=np.uint16)
    a.step(wa, g_bits, None, ca, 0, 1)
    b.step(wb, g_wide, None, cb, 0, 1)
    assert np.array_equal(wa, wb) and np.array_equal(ca, cb)
    assert a.layers()[0].grad_var == b.layers()[0].grad_var


def test_non_finite_input_skips_the_whole_step():
    table, n_total = [(0, 40), (40, 24)], 64
    rng = np.random.default_rng(3)
    D = rng.uniform(0.1, 1, n_total).astype(F)
    o = orc.Oracle(table, n_total)
    w = rng.standard_normal(n_total).astype(F)
    c = np.zeros(n_total, dtype=np.uint16)
    g = rng.standard_normal(n_total).astype(F)
    o.step(w, g, _hz_for(D, 1, 0, 1), c, 0, 1)
    w1, c1, ly1, m1 = w.copy(), c.copy(), [(l.ema_var, l.ema_mean, l.lambda_max, l.code) for l in o.layers()], o.mask()
    for poison_g, poison_h in [(np.inf, None), (None, np.nan), (-np.inf, np.inf)]:
        g2, hz2 = g.copy(), _hz_for(D, 1, 0, 2)
        n_bad = 0
        if poison_g is not None:
            g2[50] = poison_g; n_bad += 1
        if poison_h is not None:
            hz2[7] = poison_h; n_bad += 1
        assert o.step(w, g2, hz2, c, 0, 2) is True
        st = o.status()
        assert st.skipped == 1 and st.nonfinite_count == n_bad
        assert np.array_equal(w, w1) and np.array_equal(c, c1) and np.array_equal(o.mask(), m1)
        assert [(l.ema_var, l.ema_mean, l.lambda_max, l.code) for l in o.layers()] == ly1


# ---------------------------------------------------------------- batch rule (Sec. 3.3)

def test_batch_rule_truth_table():
    args = dict(delta_up=8, delta_down=16, rho_low=0.7, rho_high=0.9, mem_max=100.0, B_min=8, B_max=128)
    assert orc.batch_next(96, mem_usage=50.0, **args) == 104       # below rho_low * max: grow
    assert orc.batch_next(96, mem_usage=95.0, **args) == 80        # above rho_high * max: shrink
    assert orc.batch_next(96, mem_usage=80.0, **args) == 96        # in the band: hold
    assert orc.batch_next(96, mem_usage=70.0, **args) == 96        # boundaries are strict
    assert orc.batch_next(96, mem_usage=90.0, **args) == 96
    assert orc.batch_next(124, mem_usage=10.0, **args) == 128      # clamps
    assert orc.batch_next(16, mem_usage=99.0, **args) == 8


# ---------------------------------------------------------------- momentum and weight decay (Sec. 4.1 SGD)

@pytest.mark.parametrize("momentum,wd", [(0.9, 0.0), (0.0, 5e-4), (0.9, 5e-4)])
def test_momentum_and_weight_decay_follow_torch_sgd(momentum, wd):
    # an independent implementation of the same update rule: torch.optim.SGD (no dampening, no Nesterov)
    n = 3000
    rng = np.random.default_rng(0)
    w0 = rng.standard_normal(n).astype(F)
    o = orc.Oracle([(0, n)], n, alpha=0.0, eta0=0.05, momentum=momentum, weight_decay=wd, tau_low=-2.0, tau_high=-1.0)
    w, c = w0.copy(), np.zeros(n, dtype=np.uint16)
    p = torch.nn.Parameter(torch.from_numpy(w0.copy()))
    opt = torch.optim.SGD([p], lr=0.05, momentum=momentum, weight_decay=wd)
    for t in range(1, 9):
        g = (rng.standard_normal(n) * 0.1).astype(F)
        o.step(w, g, None, c, 0, t)
        p.grad = torch.from_numpy(g.copy())
        opt.step()
        assert np.allclose(w, p.detach().numpy(), rtol=2e-6, atol=1e-7), t
    if momentum:
        buf = opt.state[p]["momentum_buffer"].numpy()
        assert np.allclose(o.momentum_buffer(), buf, rtol=2e-6, atol=1e-6)


def test_momentum_buffer_untouched_by_a_skipped_step():
    n = 64
    o = orc.Oracle([(0, n)], n, momentum=0.9)
    w, c = np.ones(n, dtype=F), np.zeros(n, dtype=np.uint16)
    g = np.full(n, 0.5, dtype=F)
    o.step(w, g, None, c, 0, 1)
    before = (w.copy(), o.momentum_buffer())
    g2 = g.copy(); g2[3] = np.nan
    assert o.step(w, g2, None, c, 0, 2) is True
    assert np.array_equal(w, before[0]) and np.array_equal(o.momentum_buffer(), before[1])
    assert np.all(before[1] == 0.5)
