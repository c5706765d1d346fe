"""GPU parity at the benchmark configurations' full sizes, in the launch
configuration bench.py times (whole shape buckets in one context).

The oracle is too slow to run on every matrix of a full bucket, so each test
compares sampled matrices with it one by one (the sampled inputs are copied
from the device, so both sides see the same bits) and checks properties that
hold for all matrices: status word clear, finite positive norms, every weight
changed.  Shapes too large for the oracle's matmul chain are pinned through the
closed form instead: for G = U diag(s) V^T the step must produce
U diag(f^5(s/||s||)) V^T (Sec. 2.1: the iteration is an odd polynomial, so it
acts on the singular values only), with U, V Householder reflectors so that
the expectation costs O(rows*cols).
"""

import math

import numpy as np
import pytest
import torch

from oracle import muon_oracle as orc
from paper_2502_16982_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL_FP32 = 1e-5
TOL_NS = 2e-2


def _binding():
    from paper_2502_16982_b200 import binding
    return binding


def rel(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    n = np.linalg.norm(b)
    return np.linalg.norm(a - b) / n if n > 0 else np.linalg.norm(a - b)


def f64(t):
    return t.detach().cpu().to(torch.float64).numpy()


def bf16_ulp_ok_fraction(got_bf16, expect_f64, slack):
    exp_t = torch.from_numpy(expect_f64).to(torch.float64)
    got = got_bf16.detach().cpu().to(torch.float64)
    ulp = torch.clamp(exp_t.abs(), min=1e-30).log2().floor().exp2() * 2.0 ** -7
    return float(((got - exp_t).abs() <= ulp * 1.0001 + slack).double().mean())


def to_orc(hp):
    return orc.Hyper(lr=hp.lr, wd=hp.wd, mu=hp.mu, nesterov=hp.nesterov, ns_steps=hp.ns_steps,
                     a=hp.a, b=hp.b, c=hp.c, eps=hp.eps, rms_scale=hp.rms_scale)


class DeviceCase:
    """A configuration drawn on the device, as bench.py does."""

    def __init__(self, specs, seed):
        self.b = _binding()
        self.specs = specs
        self.state = [wl.make_group(sp, seed + gi, "cuda") for gi, sp in enumerate(specs)]
        self.ctx = self.b.MuonContext([(wl.views(W), wl.views(G), wl.views(M)) for (W, G, M) in self.state])
        self.first = np.cumsum([0] + [sp.count for sp in specs])

    def sample_snapshot(self, picks):
        return {(gi, i): tuple(f64(t[i]) for t in self.state[gi]) for (gi, i) in picks}

    def step_and_check(self, hp, picks, check_changed=True):
        snap = self.sample_snapshot(picks)
        w_before = [W.clone() for (W, G, M) in self.state] if check_changed else None
        self.ctx.muon_step(hp)
        status, which = self.ctx.muon_status()
        assert status == 0, (status, which)
        norms = np.array(self.ctx.muon_get_norms())
        assert np.all(np.isfinite(norms)) and np.all(norms > 0)
        rms = np.array(self.ctx.muon_get_update_rms())
        # Lemma 1 / Sec. 2.2: a full-rank update scaled by 0.2*sqrt(max(rows, cols)) has RMS near 0.2
        assert np.all(rms > 0.1) and np.all(rms < 0.3), (rms.min(), rms.max())
        if check_changed:
            for gi, (W, G, M) in enumerate(self.state):
                changed = (W != w_before[gi]).flatten(1).any(dim=1)
                assert bool(changed.all()), ("unchanged weight in group", gi)
            del w_before
        ohp = to_orc(hp)
        for (gi, i), (W0, G0, M0) in snap.items():
            W, G, M = self.state[gi]
            ref = orc.muon_step(W0, G0, M0, ohp)
            assert rel(f64(M[i]), ref["M"]) <= TOL_FP32, ("M", gi, i)
            nu = norms[self.first[gi] + i]
            assert abs(nu - ref["nu"]) <= TOL_FP32 * ref["nu"], ("nu", gi, i)
            assert abs(rms[self.first[gi] + i] - ref["rms"]) <= TOL_NS * ref["rms"], ("rms", gi, i)
            upd_rms = float(np.sqrt(np.mean((ref["W"] - W0 + hp.lr * hp.wd * W0) ** 2)))
            frac = bf16_ulp_ok_fraction(W[i], ref["W"], slack=4 * TOL_NS * upd_rms)
            assert frac >= 0.999, ("W ulp", gi, i, frac)
            # the update itself, recovered from the bf16 weights at a step size
            # large enough to show above their rounding
            if hp.lr >= 1e-2:
                d_gpu = f64(W[i]) - W0
                d_ref = ref["W"] - W0
                assert rel(d_gpu, d_ref) <= TOL_NS + 2.0 ** -8 * np.linalg.norm(ref["W"]) / np.linalg.norm(d_ref), \
                    ("dW", gi, i, rel(d_gpu, d_ref))

    def new_grads(self, seed):
        for gi, sp in enumerate(self.specs):
            gen = torch.Generator(device="cuda")
            gen.manual_seed(seed + gi)
            self.state[gi][1].copy_(wl.make_grads(sp, gen, "cuda"))

    def close(self):
        self.ctx.muon_destroy()
        self.state = None
        torch.cuda.empty_cache()


def test_config3_full_expert_bucket_sampled():
    """198 matrices of 2048x1408 / 1408x2048 in one bucket (the benchmark's
    workload); first step from zero momentum, second step with fresh gradients."""
    specs = wl.config_groups(3)
    case = DeviceCase(specs, seed=3000)
    try:
        hp = _binding().Hyper(lr=4.2e-4, wd=0.1)
        case.step_and_check(hp, [(0, 0), (0, 131), (1, 0), (1, 65)])
        case.new_grads(3500)
        case.step_and_check(hp, [(0, 77), (1, 33)])
    finally:
        case.close()


def test_config2_dense_shapes_sampled():
    """The dense-transformer buckets at their real shapes (two layers' worth)."""
    specs = wl.config_groups(2, layers=2)
    case = DeviceCase(specs, seed=2000)
    try:
        hp = _binding().Hyper(lr=2e-2, wd=0.1)  # a step large enough to check delta W in bf16
        case.step_and_check(hp, [(0, 0), (0, 7), (1, 3), (2, 1)])
    finally:
        case.close()


def test_config5_moonlight_shapes_sampled():
    """Every shape bucket of the Moonlight-shaped set (two layers: attention
    projections, the dense MLP, one MoE layer's experts) in one context."""
    specs = wl.config_groups(5, layers=2)
    case = DeviceCase(specs, seed=5000)
    try:
        hp = _binding().Hyper(lr=4.2e-4, wd=0.1)
        picks = [(gi, sp.count - 1) for gi, sp in enumerate(specs)]
        case.step_and_check(hp, picks)
    finally:
        case.close()


def test_config5_full_moonlight_set_sampled():
    """The whole Moonlight-shaped set in one context, as bench.py --config 5
    times it: 5286 matrices, 15.3 G parameters, 123 GB of weights, gradients
    and momentum; the 5148-matrix expert bucket runs in twelve chunks that
    reuse the workspace.  Sampled matrices include both sides of a chunk
    boundary and the last matrix of every group."""
    free, _ = torch.cuda.mem_get_info()
    if free < 150e9:
        pytest.skip("needs about 140 GB of free device memory")
    specs = wl.config_groups(5)
    case = DeviceCase(specs, seed=5000)
    try:
        hp = _binding().Hyper(lr=4.2e-4, wd=0.1)
        picks = [(gi, sp.count - 1) for gi, sp in enumerate(specs)]
        picks += [(7, 0), (7, 440), (7, 441), (8, 0)]
        case.step_and_check(hp, picks, check_changed=False)
    finally:
        case.close()


def householder_pair(rows, cols, s, rng):
    """G = U [diag(s) 0] V and a function giving U [diag(t) 0] V for any t, with
    U = I - 2 u u^T, V = I - 2 v v^T (m = min(rows, cols) singular values; the
    matrix is built short side first and transposed when rows > cols)."""
    m, n = min(rows, cols), max(rows, cols)
    u = rng.standard_normal(m)
    u /= np.linalg.norm(u)
    v = rng.standard_normal(n)
    v /= np.linalg.norm(v)

    def build(t):
        D = np.zeros((m, n))
        D[np.arange(m), np.arange(m)] = t
        D -= 2.0 * np.outer(u, u @ D)       # U D
        D -= 2.0 * np.outer(D @ v, v)       # (U D) V
        return D if rows <= cols else np.ascontiguousarray(D.T)

    return build(s), build


@pytest.mark.parametrize("rows,cols", [(4096, 4096), (8192, 8192), (4096, 16384), (16384, 4096)])
def test_config4_large_shapes_closed_form(rows, cols):
    """Shape-sweep matrices the oracle cannot finish in seconds."""
    b = _binding()
    rng = np.random.default_rng(rows + cols)
    m = min(rows, cols)
    s = rng.uniform(0.5, 1.5, size=m)
    G, build = householder_pair(rows, cols, s, rng)
    Gd = torch.from_numpy(G).to(torch.float32).cuda()[None]
    del G
    W = torch.zeros((1, rows, cols), dtype=torch.bfloat16, device="cuda")
    M = torch.zeros((1, rows, cols), dtype=torch.float32, device="cuda")
    ctx = b.MuonContext([(wl.views(W), wl.views(Gd), wl.views(M))])
    try:
        hp = b.Hyper(lr=1e-2, wd=0.0)
        ctx.muon_step(hp)
        status, which = ctx.muon_status()
        assert status == 0, (status, which)
        nu = ctx.muon_get_norms()[0]
        assert abs(nu - 1.95 * np.linalg.norm(s)) <= 1e-4 * np.linalg.norm(s)  # U = (mu + 1) G at step 1

        x = s / np.linalg.norm(s)
        for _ in range(5):
            x = 3.4445 * x - 4.7750 * x ** 3 + 2.0315 * x ** 5
        expect = -hp.lr * 0.2 * math.sqrt(max(rows, cols)) * build(x)
        got = W[0].double().cpu().numpy()
        # W starts at zero, so it is the update rounded once to bf16
        assert rel(got, expect) <= TOL_NS, rel(got, expect)
    finally:
        ctx.muon_destroy()
