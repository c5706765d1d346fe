"""GPU parity: the CUDA path, called through the C ABI, against the CPU fp64
oracle on the same seeded inputs.

Tolerances (relative Frobenius error), the one rule of this suite:
  * fp32 element-wise parts (momentum, norm):            <= 1e-5
  * bf16 Newton-Schulz path (A, B, X stages, O, delta W): <= 2e-2 (TOL_NS), on
    every input shaped and distributed like the benchmark configurations and on
    every Gaussian test input, for the paper's N = 5 and fewer iterations.
  * stress inputs only (more than five iterations; max/min in the thousands;
    spectra spanning orders of magnitude): bf16 storage, the precision the
    paper fixes (Sec. 2.3), by itself moves the result more than 2e-2 from the
    float64 iteration there.  ``ns_bound`` then measures that distance with the
    oracle's storage model (exact arithmetic, only the stored X, A and B, or
    B + a*I from 16 rows up, rounded; pinned by a hand-derived example) and
    allows max(2e-2, 1.1 x that distance): the CUDA path may be at most a tenth worse than bf16 storage
    alone.  The pair (GPU distance, model distance) is printed.
For bf16 weights the per-step change is about one bf16 ulp of the weight, so
the weight itself is compared element-wise with the oracle's result: >= 99.9 %
of elements within one bf16 ulp plus the Newton-Schulz tolerance expressed per
element (4 * 2e-2 * RMS of the oracle's update).
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
STRESS_SLACK = 1.10


def ns_bound(U, eps, ns_steps, o_ref=None):
    """(bound, model distance) for a stress input U (the Newton-Schulz input in
    float64): the larger of TOL_NS and STRESS_SLACK x the distance of the bf16
    storage model from the float64 iteration on this very input.  The model is
    taken in the reading the library documents for the size: from 16 rows
    (short side) up the stored polynomial is B + a*I."""
    if o_ref is None:
        o_ref = orc.newton_schulz(orc.frobenius_normalise(U, eps)[1], ns_steps)
    o_model = orc.newton_schulz_bf16_storage(U, eps, ns_steps, fold_identity=min(U.shape) >= 16)
    model = rel(o_model, o_ref)
    return max(TOL_NS, STRESS_SLACK * model), model


def _binding():
    from paper_2502_16982_b200 import binding
    return binding


def rel(a, b):
    a = np.asarray(a, dtype=np.float64)
    b = np.asarray(b, dtype=np.float64)
    d = np.linalg.norm(a - b)
    n = np.linalg.norm(b)
    return d / n if n > 0 else d


def f64(t):
    return t.detach().cpu().to(torch.float64).numpy()


SCALE_MODES = {0: "adjusted_lr", 1: "fixed_dim", 2: "update_norm"}


def to_orc(hp):
    return orc.Hyper(lr=hp.lr, wd=hp.wd, mu=hp.mu, nesterov=hp.nesterov, ns_steps=hp.ns_steps,
                     a=hp.a, b=hp.b, c=hp.c, eps=hp.eps, rms_scale=hp.rms_scale,
                     scale_mode=SCALE_MODES[hp.scale_mode], scale_dim=hp.scale_dim,
                     coeffs=None if hp.coeffs is None else [tuple(t) for t in hp.coeffs])


def bf16_ulp_ok_fraction(got_bf16, expect_f64, slack=0.0):
    """Fraction of elements of a bf16 tensor within one bf16 ulp (+ slack) of
    the float64 expectation."""
    exp_t = torch.from_numpy(expect_f64).to(torch.float64)
    got = got_bf16.detach().cpu().to(torch.float64)
    ulp = torch.clamp(exp_t.abs(), min=1e-30).log2().floor().exp2() * 2.0 ** -7
    return float(((got - exp_t).abs() <= ulp * 1.0001 + slack).double().mean())


class Case:
    """Device tensors of some groups plus host snapshots for the oracle."""

    def __init__(self, specs, seed, zero_momentum=True):
        b = _binding()
        self.b = b
        self.specs = specs
        self.dev = []
        for gi, sp in enumerate(specs):
            W, G, M = wl.make_group(sp, seed + gi, "cpu", zero_momentum=zero_momentum)
            self.dev.append((W.cuda(), G.cuda(), M.cuda()))
        self.ctx = b.MuonContext([(wl.views(W), wl.views(G), wl.views(M)) for (W, G, M) in self.dev])

    def snapshot(self):
        return [(f64(W), f64(G), f64(M)) for (W, G, M) in self.dev]

    def step(self, hp):
        self.ctx.muon_step(hp)
        return self.ctx.muon_status()

    def close(self):
        self.ctx.muon_destroy()


def check_step(case, hp, check_w=True, check_o=False):
    """Runs one step and compares every matrix with the oracle.  With
    ``check_o`` the last iteration also stores O (test tap) and O itself is
    compared."""
    before = case.snapshot()
    case.ctx.muon_debug_keep(bool(check_o))
    status, which = case.step(hp)
    assert status == 0, (status, which)
    norms = case.ctx.muon_get_norms()
    rms = case.ctx.muon_get_update_rms()
    gidx = 0
    ohp = to_orc(hp)
    for gi, sp in enumerate(case.specs):
        W, G, M = case.dev[gi]
        W0, G0, M0 = before[gi]
        for i in range(sp.count):
            ref = orc.muon_step(W0[i], G0[i], M0[i], ohp)
            tol_ns = TOL_NS
            if hp.ns_steps > 5:  # a stress input: see the module docstring
                U = ref["X0"] * (ref["nu"] + hp.eps)
                tol_ns, model = ns_bound(U, hp.eps, hp.ns_steps, ref["O"])
                print("N=%d %dx%d: bf16 storage model %.3e from the float64 iteration, bound %.3e"
                      % (hp.ns_steps, sp.rows, sp.cols, model, tol_ns))
            assert rel(f64(M[i]), ref["M"]) <= TOL_FP32, ("M", gi, i)
            assert abs(norms[gidx] - ref["nu"]) <= TOL_FP32 * ref["nu"] + 1e-30, ("nu", gi, i)
            # update RMS returned for logging (Algorithm 1): follows O, so the Newton-Schulz tolerance
            assert abs(rms[gidx] - ref["rms"]) <= tol_ns * ref["rms"] + 1e-30, ("rms", gi, i, rms[gidx], ref["rms"])
            if check_o and hp.ns_steps > 0:
                m, n = min(sp.rows, sp.cols), max(sp.rows, sp.cols)
                o_gpu = f64(case.ctx.muon_debug_read(gidx, case.b.MUON_TAP_X, m, n))
                o_ref = ref["O"].T if sp.rows > sp.cols else ref["O"]
                assert rel(o_gpu, o_ref) <= tol_ns, ("O", gi, i, rel(o_gpu, o_ref))
            if check_w:
                dW_ref = ref["W"] - W0[i]
                if sp.w_dtype == torch.float32:
                    assert rel(f64(W[i]) - W0[i], dW_ref) <= tol_ns, ("dW", gi, i, rel(f64(W[i]) - W0[i], dW_ref))
                else:
                    upd_rms = float(np.sqrt(np.mean((dW_ref + hp.lr * hp.wd * W0[i]) ** 2)))
                    frac = bf16_ulp_ok_fraction(W[i], ref["W"], slack=4 * tol_ns * upd_rms)
                    assert frac >= 0.999, ("W ulp", gi, i, frac)
            gidx += 1


HP = None


def default_hp(**kw):
    b = _binding()
    return b.Hyper(**kw)


# ---------------------------------------------------------------------------
def test_config1_full_step():
    specs = wl.config_groups(1)
    case = Case(specs, seed=0)
    try:
        check_step(case, default_hp(lr=2e-2, wd=0.1, mu=0.95, nesterov=True, ns_steps=5))
    finally:
        case.close()


@pytest.mark.parametrize("wdt", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("rows,cols", [(128, 256), (256, 128), (320, 704), (576, 200), (64, 96), (120, 72), (12, 40)])
def test_stagewise_one_iteration(rows, cols, wdt):
    """X0, A, B, X of a single Newton-Schulz iteration against the oracle's.
    From 16 rows (short side) up the kernels keep B + a*I instead of B."""
    sp = wl.GroupSpec(rows, cols, 2, wdt, torch.float32, 0.02, 1.0)
    case = Case([sp], seed=42)
    try:
        case.ctx.muon_debug_keep(True)
        hp = default_hp(ns_steps=1)
        before = case.snapshot()
        assert case.step(hp)[0] == 0
        m, n = min(rows, cols), max(rows, cols)
        for i in range(sp.count):
            W0, G0, M0 = (x[i] for x in before[0])
            ref = orc.muon_step(W0, G0, M0, to_orc(hp), trace=True)
            A, B, X1 = ref["stages"][0]
            U = ref["X0"] * (ref["nu"] + hp.eps)
            U = U.T if rows > cols else U
            b = case.b
            x0 = f64(case.ctx.muon_debug_read(i, b.MUON_TAP_X0, m, n))
            assert rel(x0, U) <= 4e-3  # one bf16 rounding of U
            a_gpu = f64(case.ctx.muon_debug_read(i, b.MUON_TAP_A, m, m))
            b_gpu = f64(case.ctx.muon_debug_read(i, b.MUON_TAP_B, m, m))
            x_gpu = f64(case.ctx.muon_debug_read(i, b.MUON_TAP_X, m, n))
            assert rel(a_gpu, A) <= TOL_NS, rel(a_gpu, A)
            if m >= 16:
                # off the diagonal it is B; on it, B_ii + a rounded once to bf16
                off = ~np.eye(m, dtype=bool)
                assert rel(b_gpu[off], B[off]) <= TOL_NS, rel(b_gpu[off], B[off])
                d_ref = np.diag(B) + hp.a
                assert np.all(np.abs(np.diag(b_gpu) - d_ref) <= 2.0 ** -8 * np.abs(d_ref) + TOL_NS * np.abs(np.diag(B)))
            else:
                assert rel(b_gpu, B) <= TOL_NS, rel(b_gpu, B)
            assert rel(x_gpu, X1) <= TOL_NS, rel(x_gpu, X1)
            # the diagonal blocks are computed in full: A and B symmetric bit for bit
            assert np.array_equal(a_gpu, a_gpu.T)
            assert np.array_equal(b_gpu, b_gpu.T)
    finally:
        case.close()


RAGGED = [(1, 300), (300, 1), (129, 257), (257, 129), (8, 8), (130, 130), (64, 1000), (1000, 72), (333, 515)]


@pytest.mark.parametrize("rows,cols", RAGGED)
@pytest.mark.parametrize("wdt", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("tile_mode", [1, 5])
def test_ragged_shapes(rows, cols, wdt, tile_mode):
    """Three matrices of an awkward shape.  So small a bucket is cut into finer
    tiles by default (tile mode 1: every row block on its own); mode 5 switches
    that off, so that the tiles a large bucket takes - row pairs, tiles shared
    by two matrices, a dropped block - meet the same ragged edges."""
    prev = _binding().muon_debug_set_tile_mode(tile_mode)
    try:
        sp = wl.GroupSpec(rows, cols, 3, wdt, wdt, 0.02, 1.0)
        case = Case([sp], seed=rows * 7 + cols)
    finally:
        _binding().muon_debug_set_tile_mode(prev)
    try:
        check_step(case, default_hp(lr=4.2e-4, wd=0.05), check_o=True)
        check_step(case, default_hp(lr=4.2e-4, wd=0.05))
    finally:
        case.close()


def test_mixed_orientation_bucket_and_multi_step():
    """Two orientations of one (m, n) share a bucket; three steps with fresh
    gradients exercise non-zero momentum."""
    specs = [wl.GroupSpec(384, 200, 3, torch.bfloat16, torch.bfloat16, 0.02, 1e-3, lognormal_scale=True),
             wl.GroupSpec(200, 384, 2, torch.bfloat16, torch.bfloat16, 0.02, 1e-3, lognormal_scale=True),
             wl.GroupSpec(256, 256, 2, torch.float32, torch.bfloat16, 0.02, 1e-3),
             wl.GroupSpec(200, 384, 2, torch.float32, torch.bfloat16, 0.02, 1e-3),
             wl.GroupSpec(384, 200, 1, torch.float32, torch.bfloat16, 0.02, 1e-3)]
    case = Case(specs, seed=5)
    try:
        hp = default_hp(lr=4.2e-4, wd=0.1)
        gen = torch.Generator().manual_seed(99)
        for step in range(3):
            if step:
                for gi, sp in enumerate(specs):
                    case.dev[gi][1].copy_(wl.make_grads(sp, gen, "cpu"))
            check_step(case, hp)
    finally:
        case.close()


def test_one_bucket_two_orientations_with_taps():
    """Both stored orientations of one (m, n) batched together; O is read
    through the tap at step 1 and step 3."""
    specs = [wl.GroupSpec(384, 200, 3, torch.bfloat16, torch.bfloat16, 0.02, 1e-3, lognormal_scale=True),
             wl.GroupSpec(200, 384, 2, torch.bfloat16, torch.bfloat16, 0.02, 1e-3, lognormal_scale=True)]
    case = Case(specs, seed=6)
    try:
        hp = default_hp(lr=4.2e-4, wd=0.1)
        gen = torch.Generator().manual_seed(77)
        for step in range(3):
            if step:
                for gi, sp in enumerate(specs):
                    case.dev[gi][1].copy_(wl.make_grads(sp, gen, "cpu"))
            check_step(case, hp, check_o=(step != 1))
    finally:
        case.close()


@pytest.mark.parametrize("wdt", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("ns_steps", [0, 1, 2, 10])
def test_ns_step_counts(ns_steps, wdt):
    sp = wl.GroupSpec(192, 320, 2, wdt, torch.float32, 0.02, 1.0)
    case = Case([sp], seed=3)
    try:
        check_step(case, default_hp(ns_steps=ns_steps, nesterov=(ns_steps != 2)))
    finally:
        case.close()


@pytest.mark.parametrize("off", [1, 8])
@pytest.mark.parametrize("rows,cols", [(264, 392), (392, 264)])
def test_column_slices_of_wider_buffers(rows, cols, off):
    """W, G and M that are column slices of wider buffers.  Starting one
    element in there is no 16-byte alignment, so the scalar momentum path and
    the separate weight-update kernel run; starting eight elements in, the
    vector and TMA paths run with a row pitch larger than the row.  Either way
    nothing outside the slices may change."""
    b = _binding()
    gen = torch.Generator().manual_seed(11)
    big = {}
    for name, dt, std in (("W", torch.bfloat16, 0.02), ("G", torch.bfloat16, 1.0), ("M", torch.float32, 0.0)):
        t = (torch.randn(2, rows, cols + 16, generator=gen) * std).to(dt).cuda()
        big[name] = t
    Wv = [big["W"][i][:, off:off + cols] for i in range(2)]
    Gv = [big["G"][i][:, off:off + cols] for i in range(2)]
    Mv = [big["M"][i][:, off:off + cols] for i in range(2)]
    W0 = [f64(t) for t in Wv]
    G0 = [f64(t) for t in Gv]
    guard = big["W"].clone()
    ctx = b.MuonContext([(Wv, Gv, Mv)])
    try:
        hp = default_hp(lr=1e-2, wd=0.1)
        ctx.muon_step(hp)
        assert ctx.muon_status()[0] == 0
        for i in range(2):
            ref = orc.muon_step(W0[i], G0[i], np.zeros_like(G0[i]), to_orc(hp))
            assert rel(f64(Mv[i]), ref["M"]) <= TOL_FP32
            upd_rms = float(np.sqrt(np.mean((ref["W"] - W0[i] + hp.lr * hp.wd * W0[i]) ** 2)))
            assert bf16_ulp_ok_fraction(Wv[i], ref["W"], slack=4 * TOL_NS * upd_rms) >= 0.999
        # the columns outside the views are untouched
        assert torch.equal(big["W"][:, :, :off], guard[:, :, :off])
        assert torch.equal(big["W"][:, :, off + cols:], guard[:, :, off + cols:])
        assert torch.count_nonzero(big["M"][:, :, :off]) == 0
        assert torch.count_nonzero(big["M"][:, :, off + cols:]) == 0
    finally:
        ctx.muon_destroy()


@pytest.mark.parametrize("rows,cols", [(16, 65536), (65536, 16), (48, 16400)])
def test_extreme_aspect_ratios(rows, cols):
    """The largest supported dimension with a tiny short side: one row pair,
    512 column tiles, a 1024-block contraction in the Gram product.

    With max/min this large the singular values are nearly equal and sit where
    the quintic map is steep, so the bf16 storage the paper prescribes moves the
    result further from the float64 iteration than elsewhere: a CPU model that
    only rounds the stored X, A, B to bf16 (exact arithmetic otherwise) is
    2.6e-2 away at 48x16400.  A stress input: the bound is ``ns_bound``'s, still
    measured against the float64 oracle."""
    sp = wl.GroupSpec(rows, cols, 2, torch.bfloat16, torch.bfloat16, 0.02, 1e-3)
    case = Case([sp], seed=rows + cols)
    try:
        hp = default_hp(lr=4.2e-4, wd=0.1)
        W, G, M = case.dev[0]
        G0 = f64(G)
        case.ctx.muon_debug_keep(True)
        assert case.step(hp)[0] == 0
        m, n = min(rows, cols), max(rows, cols)
        for i in range(sp.count):
            U = (hp.mu + 1.0) * G0[i]  # Nesterov-style input at step 1 from zero momentum
            o_ref = orc.newton_schulz(orc.frobenius_normalise(U, hp.eps)[1], hp.ns_steps)
            bound, model = ns_bound(U, hp.eps, hp.ns_steps, o_ref)
            o_gpu = f64(case.ctx.muon_debug_read(i, case.b.MUON_TAP_X, m, n))
            o_gpu = o_gpu.T if rows > cols else o_gpu
            print("%dx%d matrix %d: GPU %.3e, bf16 storage model %.3e from the float64 iteration (bound %.3e)"
                  % (rows, cols, i, rel(o_gpu, o_ref), model, bound))
            assert rel(o_gpu, o_ref) <= bound, (i, rel(o_gpu, o_ref), model, bound)
            assert rel(f64(M[i]), G0[i]) <= TOL_FP32
    finally:
        case.close()


@pytest.mark.parametrize("rows,cols", [(256, 512), (192, 320)])
@pytest.mark.parametrize("spectrum", ["one_over_k", "one_over_sqrt_k", "rank8_on_a_floor"])
def test_decaying_and_low_rank_spectra(rows, cols, spectrum):
    """Gradients with a wide range of singular values (the Gaussian test inputs
    have a narrow one): power-law decays and eight directions on a 1e-3 floor.
    Small singular values sit near the rounding noise of bf16 storage, which the
    iteration amplifies up to a^5, so here the bf16 model itself is 1e-2 to
    1.6e-1 from the float64 iteration: stress inputs, bounded by ``ns_bound`` as
    the extreme aspect ratios are.  256 x 512 takes its first two iterations as
    a pair, 192 x 320 the plain sequence."""
    b = _binding()
    rng = np.random.default_rng(rows + len(spectrum))
    m = min(rows, cols)
    k = np.arange(1, m + 1, dtype=np.float64)
    sig = {"one_over_k": 1.0 / k, "one_over_sqrt_k": 1.0 / np.sqrt(k),
           "rank8_on_a_floor": np.where(k <= 8, 1.0, 1e-3)}[spectrum]
    Qm, _ = np.linalg.qr(rng.standard_normal((rows, m)))
    Qn, _ = np.linalg.qr(rng.standard_normal((cols, m)))
    Gf = (Qm * sig) @ Qn.T
    G = torch.from_numpy(Gf / np.abs(Gf).max()).to(torch.bfloat16)[None].cuda()
    W = torch.zeros((1, rows, cols), dtype=torch.bfloat16, device="cuda")
    M = torch.zeros((1, rows, cols), dtype=torch.float32, device="cuda")
    ctx = b.MuonContext([(wl.views(W), wl.views(G), wl.views(M))])
    try:
        hp = default_hp(lr=1e-2, wd=0.0)
        ctx.muon_debug_keep(True)
        ctx.muon_step(hp)
        assert ctx.muon_status()[0] == 0
        U = (hp.mu + 1.0) * f64(G[0])
        o_ref = orc.newton_schulz(orc.frobenius_normalise(U, hp.eps)[1], hp.ns_steps)
        bound, model = ns_bound(U, hp.eps, hp.ns_steps, o_ref)
        o_gpu = f64(ctx.muon_debug_read(0, b.MUON_TAP_X, m, max(rows, cols)))
        print("%s %dx%d: GPU %.3e, bf16 storage model %.3e from the float64 iteration (bound %.3e)"
              % (spectrum, rows, cols, rel(o_gpu, o_ref), model, bound))
        assert rel(o_gpu, o_ref) <= bound, (rel(o_gpu, o_ref), model, bound)
    finally:
        ctx.muon_destroy()


def test_dimensions_above_the_limit_are_rejected():
    b = _binding()
    with pytest.raises(b.MuonError) as e:
        b.muon_workspace_bytes(b.shape_only_groups([(65537, 8, 1, b.MUON_DTYPE_BF16, b.MUON_DTYPE_BF16)]), 1)
    assert e.value.code == b.MUON_ERR_UNSUPPORTED


@pytest.mark.parametrize("m,n", [(200, 264), (264, 384)])
def test_chunked_bucket_matches_the_oracle(m, n):
    """A bucket larger than the chunk limit is processed in several chunks that
    reuse the workspace (as the 3432-matrix expert buckets of the full
    Moonlight-shaped set are): 7 matrices, 3 per chunk, both orientations; the
    second shape takes its first two iterations as a pair (four symmetric
    buffers per matrix)."""
    b = _binding()
    specs = [wl.GroupSpec(n, m, 4, torch.bfloat16, torch.bfloat16, 0.02, 1e-3, lognormal_scale=True),
             wl.GroupSpec(m, n, 3, torch.bfloat16, torch.bfloat16, 0.02, 1e-3, lognormal_scale=True)]
    alg, planned = b.muon_plan_flops([(m, n, 1)], 5)
    n_sym = 4 if planned < alg else 2
    assert n_sym == (4 if m >= 256 else 2)
    pad = lambda v: (v + 63) // 64 * 64
    per_matrix = (2 * m * pad(n) + n_sym * m * pad(m)) * 2  # X buffers and symmetric buffers, bf16, padded pitches
    prev = b.muon_debug_set_chunk_bytes(3 * per_matrix + 64)
    try:
        case = Case(specs, seed=31)
    finally:
        b.muon_debug_set_chunk_bytes(prev)
    try:
        assert case.ctx.workspace_bytes < 5 * per_matrix  # really chunked: room for 3 matrices, not 7
        hp = default_hp(lr=4.2e-4, wd=0.1)
        check_step(case, hp)
        gen = torch.Generator().manual_seed(32)
        for gi, sp in enumerate(specs):
            case.dev[gi][1].copy_(wl.make_grads(sp, gen, "cpu"))
        check_step(case, hp)
    finally:
        case.close()


@pytest.mark.parametrize("wdt", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("mode,dim", [(1, 1024.0), (2, 0.0)])
def test_update_scale_variants(mode, dim, wdt):
    """Sec. 3.1: "Baseline" 0.2*sqrt(H) and "Update Norm" 0.2/RMS(O), both
    orientations, two steps."""
    specs = [wl.GroupSpec(328, 200, 2, wdt, torch.bfloat16, 0.02, 1e-3),
             wl.GroupSpec(200, 328, 2, wdt, torch.bfloat16, 0.02, 1e-3)]
    case = Case(specs, seed=41)
    try:
        hp = default_hp(lr=1e-2, wd=0.1, scale_mode=mode, scale_dim=dim)
        check_step(case, hp)
        check_step(case, hp)
        if mode == 2:
            assert all(abs(r - 0.2) < 1e-6 for r in case.ctx.muon_get_update_rms())
    finally:
        case.close()


def test_coefficient_schedule():
    """One (a, b, c) per Newton-Schulz step instead of a single triple."""
    sched = [(3.4445, -4.7750, 2.0315), (3.0, -3.5, 1.2), (2.0, -1.5, 0.5)]
    specs = [wl.GroupSpec(328, 200, 2, torch.bfloat16, torch.bfloat16, 0.02, 1e-3),
             wl.GroupSpec(192, 320, 2, torch.float32, torch.float32, 0.02, 1.0)]
    case = Case(specs, seed=43)
    try:
        check_step(case, default_hp(lr=1e-2, ns_steps=3, coeffs=sched))
    finally:
        case.close()
    # a wide bucket takes the first two steps as a pair: each keeps its own triple
    case = Case([wl.GroupSpec(256, 768, 2, torch.bfloat16, torch.bfloat16, 0.02, 1e-3)], seed=47)
    try:
        assert _binding().muon_plan_flops([(256, 768, 2)], 3)[1] < _binding().muon_plan_flops([(256, 768, 2)], 3)[0]
        check_step(case, default_hp(lr=1e-2, ns_steps=3, coeffs=sched), check_o=True)
    finally:
        case.close()
    with pytest.raises(_binding().MuonError):
        default_hp(ns_steps=5, coeffs=sched).to_c()


def test_fp32_master_weights_with_bf16_shadow():
    """fp32 master weights plus a bf16 copy written by the step (Sec. 2.3's
    distributed variant keeps fp32 parameters)."""
    b = _binding()
    sp = wl.GroupSpec(264, 392, 2, torch.float32, torch.bfloat16, 0.02, 1e-3)
    W, G, M = wl.make_group(sp, 51, "cpu")
    Wd, Gd, Md = W.cuda(), G.cuda(), M.cuda()
    shadow = torch.zeros((2, 264, 392), dtype=torch.bfloat16, device="cuda")
    ctx = b.MuonContext([(wl.views(Wd), wl.views(Gd), wl.views(Md), wl.views(shadow))])
    try:
        hp = default_hp(lr=1e-2, wd=0.1)
        ctx.muon_step(hp)
        assert ctx.muon_status()[0] == 0
        for i in range(2):
            ref = orc.muon_step(f64(W[i]), f64(G[i]), f64(M[i]), to_orc(hp))
            assert rel(f64(Wd[i]) - f64(W[i]), ref["W"] - f64(W[i])) <= TOL_NS
            # the shadow is the new fp32 weight rounded once to bf16
            assert torch.equal(shadow[i], Wd[i].to(torch.bfloat16))
    finally:
        ctx.muon_destroy()
    with pytest.raises(b.MuonError):  # a shadow needs fp32 weights
        Wb = Wd.to(torch.bfloat16)
        b.MuonContext([(wl.views(Wb), wl.views(Gd), wl.views(Md), wl.views(shadow))])


@pytest.mark.parametrize("rows,cols", [(200, 332), (332, 200), (384, 1028)])
@pytest.mark.parametrize("with_shadow", [False, True])
def test_fp32_weights_updated_in_the_last_epilogue(rows, cols, with_shadow):
    """fp32 weights that TMA can address (16-byte aligned rows) are updated in the
    last combine's epilogue like bf16 ones, the bf16 copy written from the same
    registers.  Column counts that are a multiple of 4 but not of 8 or 64 leave
    a ragged last box and a scalar tail in the copy; the copy's rows are padded
    so that its pitch is a multiple of 8.  The launch count shows that no
    separate update pass ran; a second step checks the path from non-zero
    momentum."""
    b = _binding()
    sp = wl.GroupSpec(rows, cols, 2, torch.float32, torch.bfloat16, 0.02, 1e-3, lognormal_scale=True)
    W, G, M = wl.make_group(sp, rows + cols, "cpu")
    Wd, Gd, Md = W.cuda(), G.cuda(), M.cuda()
    groups = [wl.views(Wd), wl.views(Gd), wl.views(Md)]
    pitch = (cols + 7) // 8 * 8
    backing = torch.full((2, rows, pitch), 7.0, dtype=torch.bfloat16, device="cuda")
    shadow = backing[:, :, :cols]
    if with_shadow:
        groups.append([shadow[i] for i in range(2)])
    ctx = b.MuonContext([tuple(groups)])
    try:
        hp = default_hp(lr=1e-2, wd=0.1)
        gen = torch.Generator().manual_seed(5)
        Wc, Mc = W.clone(), M.clone()
        for step in range(2):
            if step:
                G = wl.make_grads(sp, gen, "cpu")
                Gd.copy_(G)
            ctx.muon_step(hp)
            assert ctx.muon_status()[0] == 0
            alg, planned = b.muon_plan_flops([(rows, cols, 2)], hp.ns_steps)
            products = 3 * hp.ns_steps + (2 if planned < alg else 0)  # a leading pair: 7 products + 1 helper for 6
            assert ctx.muon_last_launch_count() == 2 + products + 1
            for i in range(2):
                ref = orc.muon_step(f64(Wc[i]), f64(G[i]), f64(Mc[i]), to_orc(hp))
                assert rel(f64(Wd[i]) - f64(Wc[i]), ref["W"] - f64(Wc[i])) <= TOL_NS
                assert rel(f64(Md[i]), ref["M"]) <= TOL_FP32
                if with_shadow:
                    assert torch.equal(shadow[i], Wd[i].to(torch.bfloat16))
            Wc, Mc = Wd.cpu().clone(), Md.cpu().clone()
        # the padding columns of the copy's rows were never written
        assert bool((backing[:, :, cols:] == 7.0).all())
    finally:
        ctx.muon_destroy()


def test_owner_computes_shards_give_the_single_context_bits():
    """Sec. 2.3: each matrix is stepped by its owner rank alone.  A matrix's
    result must not depend on which other matrices share its launch, so the
    union of two ranks' shards equals the single-context result bit for bit."""
    b = _binding()
    specs = [wl.GroupSpec(328, 200, 5, torch.bfloat16, torch.bfloat16, 0.02, 1e-3, lognormal_scale=True),
             wl.GroupSpec(200, 328, 3, torch.bfloat16, torch.bfloat16, 0.02, 1e-3),
             wl.GroupSpec(256, 256, 2, torch.bfloat16, torch.bfloat16, 0.02, 1e-3)]
    owners, _ = b.muon_partition([(sp.rows, sp.cols, sp.count) for sp in specs], 2)
    hp = default_hp(lr=1e-2)
    single = Case(specs, seed=61)
    shard = Case(specs, seed=61)  # same bits; stepped by two "ranks", each over its own matrices
    try:
        for _ in range(2):
            assert single.step(hp)[0] == 0
        ctxs = []
        for rank in range(2):
            groups, k = [], 0
            for gi, sp in enumerate(specs):
                idx = [i for i in range(sp.count) if owners[k + i] == rank]
                k += sp.count
                if idx:
                    W, G, M = shard.dev[gi]
                    groups.append(([W[i] for i in idx], [G[i] for i in idx], [M[i] for i in idx]))
            assert groups
            ctxs.append(b.MuonContext(groups))
        for _ in range(2):
            for c in ctxs:
                c.muon_step(hp)
                assert c.muon_status()[0] == 0
        for gi in range(len(specs)):
            assert torch.equal(single.dev[gi][0], shard.dev[gi][0])
            assert torch.equal(single.dev[gi][2], shard.dev[gi][2])
        for c in ctxs:
            c.muon_destroy()
    finally:
        single.close()
        shard.close()


@pytest.fixture
def pair_fold_knob():
    b = _binding()
    prev = b.muon_debug_set_pair_fold(0)
    yield b
    b.muon_debug_set_pair_fold(prev)


@pytest.mark.parametrize("wdt", [torch.float32, torch.bfloat16])
@pytest.mark.parametrize("mode", [0, 3])
@pytest.mark.parametrize("rows,cols,ns_steps", [(256, 512, 5), (512, 256, 5), (264, 1000, 5), (1100, 392, 5),
                                               (256, 640, 4), (640, 256, 2), (392, 1100, 3), (384, 520, 5)])
def test_iterations_taken_in_pairs_match_the_oracle(rows, cols, ns_steps, mode, wdt, pair_fold_knob):
    """Two iterations per pass over X (A' = B'^2 A, X'' = B'' B' X; Eq. 2
    rearranged), for the first two iterations (the default from 256 rows) and for
    every pair (mode 3, wide matrices): same tolerance against the plain fp64
    iteration, for both orientations, ragged sizes, an odd and an even number of
    iterations (the last one alone, or the last two as a pair that updates W in
    its epilogue), with the tap on O and without."""
    b = pair_fold_knob
    b.muon_debug_set_pair_fold(mode)
    alg, planned = b.muon_plan_flops([(rows, cols, 3)], ns_steps)
    assert planned < alg  # these shapes are paired in both modes
    sp = wl.GroupSpec(rows, cols, 3, wdt, torch.bfloat16, 0.02, 1e-3, lognormal_scale=True)
    case = Case([sp], seed=rows + 3 * cols)
    try:
        hp = default_hp(lr=1e-2, wd=0.05, ns_steps=ns_steps)
        check_step(case, hp, check_o=True)
        plain_launches = 2 + 3 * ns_steps + 3   # momentum, norm, three products per iteration, two-pass update
        assert case.ctx.muon_last_launch_count() > plain_launches
        check_step(case, hp)
    finally:
        case.close()


def test_paired_and_plain_sequences_agree_within_tolerance(pair_fold_knob):
    """The same bucket stepped with the pairing off and forced on for every pair: both within
    the Newton-Schulz tolerance of the oracle, hence of each other twice over."""
    b = pair_fold_knob
    sp = wl.GroupSpec(320, 704, 2, torch.bfloat16, torch.bfloat16, 0.02, 1e-3)
    outs = []
    for mode in (1, 4):
        b.muon_debug_set_pair_fold(mode)
        case = Case([sp], seed=44)
        try:
            check_step(case, default_hp(lr=1e-2), check_o=True)
            outs.append(f64(case.ctx.muon_debug_read(0, b.MUON_TAP_X, 320, 704)))
        finally:
            case.close()
    assert 0 < rel(outs[1], outs[0]) <= 2 * TOL_NS


@pytest.mark.parametrize("mode", [4, 5, 6, 7, 1, 3])
def test_every_tile_mode_matches_the_oracle(mode):
    """Half-height tiles, tiles shared by two matrices, and full tiles whose
    second CTA works beyond the matrix are different ways of cutting the same
    products (muon_debug_set_tile_mode; 1 is the default).  Modes 4 to 7 are 0 to
    3 with the finer cut of small buckets switched off, so that these few small
    matrices take the tiles of a large bucket; modes 1 and 3 cut them finer.
    Each must meet the oracle on its own: odd and even numbers of row blocks,
    both orientations, an odd number of matrices (one is left without a partner
    in the modes that pair matrices), bf16 and fp32 weights, two steps, with the
    tap on O and with the update fused into the last epilogue."""
    b = _binding()
    specs = [wl.GroupSpec(328, 704, 2, torch.bfloat16, torch.bfloat16, 0.02, 1e-3, lognormal_scale=True),
             wl.GroupSpec(704, 328, 1, torch.bfloat16, torch.bfloat16, 0.02, 1e-3),
             wl.GroupSpec(256, 640, 3, torch.float32, torch.bfloat16, 0.02, 1e-3),
             wl.GroupSpec(100, 72, 2, torch.bfloat16, torch.bfloat16, 0.02, 1e-3)]
    hp = default_hp(lr=1e-2, wd=0.1)
    prev = b.muon_debug_set_tile_mode(mode)
    try:
        for one in specs:  # the tap needs a context with a single bucket
            case = Case([one], seed=19)
            try:
                check_step(case, hp, check_o=True)
            finally:
                case.close()
        case = Case(specs, seed=19)
        try:
            check_step(case, hp)
            gen = torch.Generator().manual_seed(20)
            for gi, sp in enumerate(specs):
                case.dev[gi][1].copy_(wl.make_grads(sp, gen, "cpu"))
            check_step(case, hp)
        finally:
            case.close()
    finally:
        b.muon_debug_set_tile_mode(prev)


def test_bucket_by_bucket_step_gives_muon_step_bits():
    """muon_step_bucket over every bucket, in reverse order, is one muon_step:
    buckets are independent, and the numbering is muon_plan_buckets' (the two
    orientations of 328 x 200 share a bucket, so three groups make two buckets)."""
    b = _binding()
    specs = [wl.GroupSpec(328, 200, 3, torch.bfloat16, torch.bfloat16, 0.02, 1e-3),
             wl.GroupSpec(256, 256, 2, torch.bfloat16, torch.bfloat16, 0.02, 1e-3),
             wl.GroupSpec(200, 328, 2, torch.bfloat16, torch.bfloat16, 0.02, 1e-3)]
    bucket_of, n_buckets = b.muon_plan_buckets(
        [(sp.rows, sp.cols, sp.count, b.MUON_DTYPE_BF16, b.MUON_DTYPE_BF16) for sp in specs])
    assert n_buckets == 2 and bucket_of == [0, 0, 0, 1, 1, 0, 0]
    hp = default_hp(lr=1e-2)
    whole = Case(specs, seed=71)
    parts = Case(specs, seed=71)
    try:
        for _ in range(2):
            assert whole.step(hp)[0] == 0
            for bk in reversed(range(n_buckets)):
                parts.ctx.muon_step_bucket(hp, bk)
            assert parts.ctx.muon_status()[0] == 0
        for gi in range(len(specs)):
            assert torch.equal(whole.dev[gi][0], parts.dev[gi][0])
            assert torch.equal(whole.dev[gi][2], parts.dev[gi][2])
        assert whole.ctx.muon_get_norms() == parts.ctx.muon_get_norms()
        assert whole.ctx.muon_get_update_rms() == parts.ctx.muon_get_update_rms()
        with pytest.raises(b.MuonError):
            parts.ctx.muon_step_bucket(hp, n_buckets)
    finally:
        whole.close()
        parts.close()


def test_distributed_wrapper_single_rank_steps_bucket_by_bucket():
    """The data-parallel wrapper with one rank owns every matrix and must give
    the plain context's bits (its momentum starts at zero like the plain one's);
    its matrices are views into the flat per-bucket storage."""
    b = _binding()
    from paper_2502_16982_b200.distributed import DistributedMuon
    specs = [wl.GroupSpec(328, 200, 3, torch.bfloat16, torch.bfloat16, 0.02, 1e-3),
             wl.GroupSpec(200, 328, 2, torch.bfloat16, torch.bfloat16, 0.02, 1e-3),
             wl.GroupSpec(128, 384, 2, torch.float32, torch.float32, 0.02, 1.0)]
    hp = default_hp(lr=1e-2)
    plain = Case(specs, seed=73)
    dm = DistributedMuon([(sp.rows, sp.cols, sp.count, sp.w_dtype, sp.g_dtype) for sp in specs], "cuda")
    try:
        assert dm.n_units == 2
        for gi, sp in enumerate(specs):
            for i in range(sp.count):
                dm.weights[gi][i].copy_(plain.dev[gi][0][i])
                dm.grads[gi][i].copy_(plain.dev[gi][1][i])
        for _ in range(2):
            assert plain.step(hp)[0] == 0
            dm.step(hp)
        assert dm.status()[0] == 0
        for gi, sp in enumerate(specs):
            for i in range(sp.count):
                assert torch.equal(plain.dev[gi][0][i], dm.weights[gi][i])
    finally:
        dm.close()
        plain.close()


def test_step_captured_in_a_cuda_graph_replays_the_eager_bits():
    """muon_step only enqueues kernels on the caller's stream (no allocation, no
    host synchronisation), so it can be captured once and replayed: two replays
    with fresh gradients give the bits of two eager steps."""
    specs = [wl.GroupSpec(328, 200, 3, torch.bfloat16, torch.bfloat16, 0.02, 1e-3),
             wl.GroupSpec(256, 384, 2, torch.float32, torch.float32, 0.02, 1.0)]
    hp = default_hp(lr=1e-2)
    eager = Case(specs, seed=91)
    graphed = Case(specs, seed=91)
    try:
        side = torch.cuda.Stream()
        side.wait_stream(torch.cuda.current_stream())
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.stream(side):
            graph.capture_begin()
            graphed.ctx.muon_step(hp, stream=side)
            graph.capture_end()
        torch.cuda.current_stream().wait_stream(side)
        # capture enqueues nothing: weights and momentum are untouched so far
        fresh = Case(specs, seed=91)
        for gi in range(len(specs)):
            assert torch.equal(graphed.dev[gi][0], fresh.dev[gi][0])
            assert torch.equal(graphed.dev[gi][2], fresh.dev[gi][2])
        fresh.close()
        for step in range(2):
            if step:
                for gi, sp in enumerate(specs):
                    gen = torch.Generator().manual_seed(900 + gi)
                    g_new = wl.make_grads(sp, gen, "cpu").cuda()
                    eager.dev[gi][1].copy_(g_new)
                    graphed.dev[gi][1].copy_(g_new)
            assert eager.step(hp)[0] == 0
            graph.replay()
            assert graphed.ctx.muon_status()[0] == 0
        for gi in range(len(specs)):
            assert torch.equal(eager.dev[gi][0], graphed.dev[gi][0])
            assert torch.equal(eager.dev[gi][2], graphed.dev[gi][2])
        assert eager.ctx.muon_get_norms() == graphed.ctx.muon_get_norms()
        del graph
    finally:
        eager.close()
        graphed.close()


def test_bitwise_reproducible():
    specs = [wl.GroupSpec(448, 640, 4, torch.bfloat16, torch.bfloat16, 0.02, 1e-3)]
    outs = []
    for _ in range(2):
        case = Case(specs, seed=17)
        try:
            hp = default_hp(lr=1e-2)
            for _ in range(2):
                assert case.step(hp)[0] == 0
            W, G, M = case.dev[0]
            outs.append((W.cpu().view(torch.int16).clone(), M.cpu().view(torch.int32).clone()))
        finally:
            case.close()
    assert torch.equal(outs[0][0], outs[1][0])
    assert torch.equal(outs[0][1], outs[1][1])


def test_zero_gradient_only_decays():
    sp = wl.GroupSpec(128, 192, 1, torch.float32, torch.float32, 0.02, 1.0)
    case = Case([sp], seed=1)
    try:
        W, G, M = case.dev[0]
        G.zero_()
        W0 = W.clone()
        hp = default_hp(lr=0.1, wd=0.5)
        assert case.step(hp)[0] == 0
        assert torch.allclose(W, W0 * (1 - 0.05), rtol=1e-6, atol=0)
        assert torch.count_nonzero(M) == 0
    finally:
        case.close()


def test_nonfinite_gradient_reports_and_keeps_weight():
    b = _binding()
    sp = wl.GroupSpec(128, 256, 3, torch.float32, torch.float32, 0.02, 1.0)
    case = Case([sp], seed=2)
    try:
        W, G, M = case.dev[0]
        G[1, 5, 7] = float("inf")
        W0 = W.clone()
        status, which = case.step(default_hp())
        assert status == b.MUON_ERR_NONFINITE and which == 1
        assert torch.equal(W[1], W0[1])
        assert not torch.equal(W[0], W0[0]) and not torch.equal(W[2], W0[2])
        # the status word was cleared by the read
        assert case.ctx.muon_status()[0] == 0
    finally:
        case.close()


def test_closed_form_medium_size_on_gpu():
    """G = U diag(s) V^T with chosen singular values: the result must equal
    U diag(f^5(s/||s||)) V^T (Sec. 2.1: the iteration is an odd polynomial, so
    it acts on singular values only).  Pins the CUDA path without the oracle."""
    rows, cols = 512, 768
    rng = np.random.default_rng(0)
    Q1, _ = np.linalg.qr(rng.standard_normal((rows, rows)))
    Q2, _ = np.linalg.qr(rng.standard_normal((cols, rows)))
    s = rng.uniform(0.5, 1.5, size=rows)
    G = (Q1 * s) @ Q2.T
    sp = wl.GroupSpec(rows, cols, 1, torch.float32, torch.float32, 0.02, 1.0)
    case = Case([sp], seed=8)
    try:
        W, Gd, M = case.dev[0]
        Gd[0].copy_(torch.from_numpy(G).to(torch.float32))
        W0 = f64(W[0])
        hp = default_hp(lr=1e-2, wd=0.0)
        assert case.step(hp)[0] == 0

        def f(x):
            return 3.4445 * x - 4.7750 * x ** 3 + 2.0315 * x ** 5

        x = s / np.linalg.norm(s)
        for _ in range(5):
            x = f(x)
        O = (Q1 * x) @ Q2.T
        dW = -hp.lr * 0.2 * math.sqrt(cols) * O
        assert rel(f64(W[0]) - W0, dW) <= TOL_NS
    finally:
        case.close()


def test_host_buffer_entry_point():
    """muon_step_host: gradients from pinned host memory, weights read back."""
    specs = [wl.GroupSpec(256, 384, 2, torch.bfloat16, torch.bfloat16, 0.02, 1e-3)]
    case = Case(specs, seed=23)
    ref = Case(specs, seed=23)
    try:
        gen = torch.Generator().manual_seed(5)
        g_new = wl.make_grads(specs[0], gen, "cpu")
        g_host = [[g_new[i].contiguous().pin_memory() for i in range(2)]]
        w_host = [[torch.empty(256, 384, dtype=torch.bfloat16).pin_memory() for _ in range(2)]]
        hp = default_hp(lr=1e-2)
        case.ctx.muon_step_host(hp, g_host, w_host)
        assert case.ctx.muon_status()[0] == 0
        ref.dev[0][1].copy_(g_new)
        assert ref.step(hp)[0] == 0
        for i in range(2):
            assert torch.equal(w_host[0][i], ref.dev[0][0][i].cpu())
            assert torch.equal(case.dev[0][0][i], ref.dev[0][0][i])
    finally:
        case.close()
        ref.close()


def test_expired_device_wait_is_reported_and_the_context_survives():
    """Failure detection without a fault: a bounded wait that nothing satisfies
    runs out after its limit, the status word carries MUON_ERR_TIMEOUT and the
    matrix named, and the next step on the same context is correct."""
    b = _binding()
    sp = wl.GroupSpec(128, 256, 3, torch.float32, torch.float32, 0.02, 1.0)
    case = Case([sp], seed=9)
    try:
        case.ctx.muon_debug_wait_expiry(2, limit_ms=20)
        status, which = case.ctx.muon_status()
        assert status == b.MUON_ERR_TIMEOUT and which == 2
        assert case.ctx.muon_status()[0] == 0  # cleared by the read
        check_step(case, default_hp())
    finally:
        case.close()


def test_host_buffer_entry_point_pipelines_several_buckets():
    """muon_step_host cuts every bucket into slices whose uploads, kernels and
    downloads overlap on three streams; the result must be the bits of
    muon_step on device-resident gradients (two buckets, nine matrices each,
    two steps so that a second call follows the first on the same stream)."""
    specs = [wl.GroupSpec(264, 200, 9, torch.bfloat16, torch.bfloat16, 0.02, 1e-3),
             wl.GroupSpec(136, 392, 9, torch.bfloat16, torch.float32, 0.02, 1e-3)]
    case = Case(specs, seed=71)
    ref = Case(specs, seed=71)
    try:
        hp = default_hp(lr=1e-2)
        gen = torch.Generator().manual_seed(72)
        for step in range(2):
            g_new = [wl.make_grads(sp, gen, "cpu") for sp in specs]
            g_host = [[g[i].contiguous().pin_memory() for i in range(sp.count)] for g, sp in zip(g_new, specs)]
            w_host = [[torch.empty(sp.rows, sp.cols, dtype=torch.bfloat16).pin_memory() for _ in range(sp.count)]
                      for sp in specs]
            case.ctx.muon_step_host(hp, g_host, w_host)
            assert case.ctx.muon_status()[0] == 0
            for gi in range(2):
                ref.dev[gi][1].copy_(g_new[gi])
            assert ref.step(hp)[0] == 0
            for gi, sp in enumerate(specs):
                for i in range(sp.count):
                    assert torch.equal(w_host[gi][i], ref.dev[gi][0][i].cpu()), (step, gi, i)
                assert torch.equal(case.dev[gi][0], ref.dev[gi][0]) and torch.equal(case.dev[gi][2], ref.dev[gi][2])
        assert case.ctx.muon_get_norms() == ref.ctx.muon_get_norms()
    finally:
        case.close()
        ref.close()


def test_invalid_descriptors_are_rejected_on_the_host():
    b = _binding()
    W = torch.zeros(2, 64, 64, device="cuda")
    G = torch.zeros(2, 64, 64, device="cuda")
    M = torch.zeros(2, 64, 64, device="cuda")
    with pytest.raises(b.MuonError) as e:
        b.MuonContext([([W[0]], [W[0]], [M[0]])])  # W aliases G
    assert e.value.code == b.MUON_ERR_INVALID_ARG
    ctx = b.MuonContext([([W[0]], [G[0]], [M[0]])])
    with pytest.raises(b.MuonError):
        ctx.muon_step(b.Hyper(ns_steps=-1))
    ctx.muon_destroy()
