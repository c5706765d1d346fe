"""GPU parity of the fused AdamW step (the optimizer of the parameters Muon
does not handle) against the fp64 oracle: fp32 element-wise arithmetic, so the
bound is 1e-5 relative on the moments and on fp32 parameters; bf16 parameters
are compared with the oracle's result rounded to bf16 (one ulp)."""

import numpy as np
import pytest
import torch

from oracle import adamw_oracle as aw

pytestmark = pytest.mark.gpu
TOL = 1e-5


def f64(t):
    return t.detach().cpu().to(torch.float64).numpy()


def rel(a, b):
    n = np.linalg.norm(b)
    return np.linalg.norm(a - b) / n if n > 0 else np.linalg.norm(a - b)


def make(shape, pdt, gdt, seed, offset=0):
    gen = torch.Generator().manual_seed(seed)
    n = int(np.prod(shape))
    def buf(dt, std):
        t = (torch.randn(n + offset, generator=gen) * std).to(dt).cuda()
        return t[offset:].view(shape)
    p, g = buf(pdt, 0.02), buf(gdt, 1e-2)
    m = torch.zeros(n + offset, device="cuda")[offset:].view(shape)
    v = torch.zeros(n + offset, device="cuda")[offset:].view(shape)
    return p, g, m, v


@pytest.mark.parametrize("pdt,gdt", [(torch.bfloat16, torch.bfloat16), (torch.float32, torch.float32),
                                     (torch.float32, torch.bfloat16)])
def test_adamw_three_steps_many_tensors(pdt, gdt):
    from paper_2502_16982_b200 import binding as b

    shapes = [(2048,), (1000, 64), (7,), (333, 129), (1,)] + [(64,)] * 50  # more than one launch's worth
    tensors = [make(s, pdt, gdt, 100 + i, offset=(1 if i == 3 else 0)) for i, s in enumerate(shapes)]
    ref = [(f64(p), f64(m), f64(v)) for (p, g, m, v) in tensors]
    gen = torch.Generator().manual_seed(9)
    for step in (1, 2, 3):
        for i, (p, g, m, v) in enumerate(tensors):
            if step > 1:
                g.copy_((torch.randn(g.shape, generator=gen) * 1e-2).to(g.dtype))
        b.muon_adamw_step([t[0] for t in tensors], [t[1] for t in tensors], [t[2] for t in tensors],
                          [t[3] for t in tensors], step, lr=1e-3, wd=0.1)
        torch.cuda.synchronize()
        for i, (p, g, m, v) in enumerate(tensors):
            p0, m0, v0 = ref[i]
            # the oracle continues from the state the GPU holds (its own rounding of p for bf16)
            pr, mr, vr = aw.adamw_step(p0, f64(g), m0, v0, step, lr=1e-3, wd=0.1, beta1=0.9, beta2=0.95, eps=1e-8)
            assert rel(f64(m), mr) <= TOL and rel(f64(v), vr) <= TOL, (step, i)
            if pdt == torch.float32:
                # relative Frobenius error of the parameter and of the step it took
                assert rel(f64(p), pr) <= TOL, (step, i)
                assert rel(f64(p) - p0, pr - p0) <= TOL, (step, i, rel(f64(p) - p0, pr - p0))
            else:
                expect = torch.from_numpy(pr).to(torch.bfloat16).to(torch.float64).numpy()
                ulp = 2.0 ** (np.floor(np.log2(np.maximum(np.abs(pr), 1e-30))) - 7)
                assert np.all(np.abs(f64(p) - expect) <= ulp * 1.0001), (step, i)
            ref[i] = (f64(p), f64(m), f64(v))


def test_adamw_rejects_bad_arguments():
    from paper_2502_16982_b200 import binding as b

    p, g, m, v = make((64,), torch.float32, torch.float32, 1)
    with pytest.raises(b.MuonError):
        b.muon_adamw_step([p], [g], [m], [v], 0, lr=1e-3, wd=0.0)  # step counts from 1
    with pytest.raises(b.MuonError):
        b.muon_adamw_step([p], [g], [m], [v], 1, lr=1e-3, wd=0.0, beta1=1.0)
