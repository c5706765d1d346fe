"""muon_momentum_norm_static: the entry point for callers that cannot hand the
library a workspace (for example a hook running in a process whose framework
pool already owns all device memory, so that neither a raw cudaMalloc nor a new
torch tensor is available to it).  It keeps its per-tile partial sums in an
array built into the library instead.

The check: on the same seeded gradients, two optimizer steps in a row through
muon_step (workspace path; momentum and ||U||_F read back through
muon_get_norms) and two calls in a row of the no-workspace entry point must give
the same momentum and the same norm, within the fp32 tolerance of the GPU parity
tests; both are also held against the CPU oracle's momentum update and
Frobenius norm directly.  Two calls matter because the built-in array still
holds the first call's partial sums when the second one starts.  The cases
cover the kernel's four load paths: 16-byte vector loads and element-wise loads,
each for bf16 and for fp32 gradients.

This file sorts last on purpose, so a run that stops at the first failure has
already been through every other test.
"""

import numpy as np
import pytest
import torch

from oracle import muon_oracle as orc
from paper_2502_16982_b200 import workloads as wl

pytestmark = pytest.mark.gpu

TOL_FP32 = 1e-5


def _rel(a, b):
    a, b = a.double(), b.double()
    n = float(b.norm())
    return float((a - b).norm()) / n if n > 0 else float((a - b).norm())


@pytest.mark.parametrize("rows,cols,gdt,nesterov", [
    (320, 704, torch.bfloat16, True),     # several tiles, bf16 vector loads
    (256, 512, torch.float32, True),      # fp32 vector loads
    (200, 331, torch.float32, False),     # ragged: fp32 element-wise loads, partial tiles
    (136, 203, torch.bfloat16, False),    # ragged: bf16 element-wise loads, partial tiles
    (1408, 2048, torch.bfloat16, True),   # an expert-sized matrix: 352 tiles
])
def test_static_scratch_matches_workspace_path_twice(rows, cols, gdt, nesterov):
    from paper_2502_16982_b200 import binding as b

    spec = wl.GroupSpec(rows, cols, 1, torch.float32, gdt, 0.02, 1.0)
    W, G, M = wl.make_group(spec, 77, "cpu")
    gen = torch.Generator().manual_seed(78)
    G2 = wl.make_grads(spec, gen, "cpu")

    # existing entry point: ns_steps = 0 keeps the step to momentum, norm and update
    Wd, Gd, Md = W.cuda(), G.cuda(), M.cuda()
    ctx = b.MuonContext([(wl.views(Wd), wl.views(Gd), wl.views(Md))])
    hp = b.Hyper(mu=0.95, nesterov=nesterov, ns_steps=0)
    # the new entry point's own tensors, all created before its first call
    Gs, Ms = G.cuda()[0].contiguous(), M.cuda()[0].contiguous()
    norm_out = torch.zeros(1, dtype=torch.float32, device="cuda")
    m_oracle = M[0].double().numpy()

    for step, grad in enumerate((G, G2)):
        Gd.copy_(grad)
        ctx.muon_step(hp)
        status, which = ctx.muon_status()
        assert status == 0, (status, which)
        nu_ref = ctx.muon_get_norms()[0]

        Gs.copy_(grad[0])
        b.muon_momentum_norm_static(Gs, Ms, 0.95, nesterov, norm_out)
        torch.cuda.synchronize()
        nu = float(norm_out.item())
        assert abs(nu - nu_ref) <= TOL_FP32 * nu_ref, (step, nu, nu_ref)
        assert _rel(Ms, Md[0]) <= TOL_FP32, (step, _rel(Ms, Md[0]))

        # first hand: the oracle's momentum update, Newton-Schulz input and its Frobenius norm
        g64 = grad[0].double().numpy()
        m_oracle = orc.momentum_update(m_oracle, g64, 0.95)
        nu_oracle, _ = orc.frobenius_normalise(orc.newton_schulz_input(m_oracle, g64, 0.95, nesterov), 0.0)
        assert abs(nu - nu_oracle) <= TOL_FP32 * nu_oracle, (step, nu, nu_oracle)
        m_gpu = Ms.double().cpu().numpy()
        assert np.linalg.norm(m_gpu - m_oracle) <= TOL_FP32 * np.linalg.norm(m_oracle), step
    ctx.muon_destroy()


def test_static_scratch_rejects_oversized_and_bad_arguments():
    from paper_2502_16982_b200 import binding as b

    L = b.lib()
    import ctypes as C
    dummy = torch.zeros(8, dtype=torch.float32, device="cuda")
    p = C.c_void_p(dummy.data_ptr())
    # 65536 x 262144 would need 2 Mi tiles: beyond the built-in array, nothing is launched
    rc = L.muon_momentum_norm_static(p, p, 65536, 262144, 262144, 262144, b.MUON_DTYPE_FP32,
                                     0.95, 1, p, 0, None)
    assert rc == b.MUON_ERR_UNSUPPORTED
    assert "tiles" in b.muon_last_error()
    rc = L.muon_momentum_norm_static(None, p, 8, 8, 8, 8, b.MUON_DTYPE_FP32, 0.95, 1, p, 0, None)
    assert rc == b.MUON_ERR_INVALID_ARG
    rc = L.muon_momentum_norm_static(p, p, 8, 8, 4, 8, b.MUON_DTYPE_FP32, 0.95, 1, p, 0, None)
    assert rc == b.MUON_ERR_INVALID_ARG
    torch.cuda.synchronize()
