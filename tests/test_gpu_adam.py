"""The Adam step on the device against the fp64 oracle (three steps in a row), and its bf16
copy against round-to-nearest-even of the device's own fp32 master weight."""
import numpy as np
import pytest
import torch

from oracle import sapo_oracle as orc
from paper_2509_08721_b200 import binding as B
from paper_2509_08721_b200 import inputs as gen

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("rows,cols", [(1000, 64), (333, 896)])
def test_adam_steps_match_the_oracle(rows, cols):
    rng = np.random.default_rng(4)
    theta0 = (rng.normal(size=(rows, cols)) * 0.02).astype(np.float32)
    master = torch.from_numpy(theta0.copy()).cuda()
    m = torch.zeros_like(master)
    v = torch.zeros_like(master)
    w16 = torch.empty(rows, cols, dtype=torch.bfloat16, device="cuda")
    th, mo, vo = theta0.astype(np.float64), np.zeros((rows, cols)), np.zeros((rows, cols))
    for step in range(1, 4):
        g = (rng.normal(size=(rows, cols)) * 10.0 ** (-2 - step)).astype(np.float32)
        g[0, :8] = 0.0                                           # zero gradient: weight must not move at step 1
        B.sapo_adam_step(master, m, v, torch.from_numpy(g).cuda(), w16, step)
        f = lambda x: float(np.float32(x))                       # the hyper-parameters as the ABI's floats carry them
        th, mo, vo = orc.adam_step(th, g, mo, vo, step, f(1e-3), f(0.9), f(0.999), f(1e-8))
        torch.cuda.synchronize()
        got = master.cpu().numpy().astype(np.float64)
        assert np.max(np.abs(got - th)) <= 2e-6 * 1e-3 + 1e-6 * np.abs(th).max()   # a step is ~lr = 1e-3
        # fp32 rounding of sums that may cancel: absolute, at 1e-6 of the largest moment
        assert np.max(np.abs(m.cpu().numpy() - mo)) <= 1e-6 * np.abs(mo).max()
        assert np.max(np.abs(v.cpu().numpy() - vo)) <= 1e-6 * np.abs(vo).max()
        bits = w16.view(torch.int16).cpu().numpy().view(np.uint16)
        assert np.array_equal(bits, gen.f32_to_bf16_bits(master.cpu().numpy()))
        if step == 1:        # zero gradient and zero moments: the weight stays bit for bit
            assert np.array_equal(master.cpu().numpy()[0, :8], theta0[0, :8])


def test_adam_rejects_bad_arguments():
    x = torch.zeros(4, 6, device="cuda")                          # cols % 4 != 0
    with pytest.raises(B.SapoError):
        B.sapo_adam_step(x, x.clone(), x.clone(), x.clone(), None, 1)
    y = torch.zeros(4, 8, device="cuda")
    with pytest.raises(B.SapoError):
        B.sapo_adam_step(y, y.clone(), y.clone(), y.clone(), None, 0)     # steps count from 1
