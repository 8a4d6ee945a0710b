"""t5_adamw_update through the C ABI against the oracle's AdamW, element by element, over several steps (bias
correction changes with the step) on the tiny model's flat parameter buffer, in both storage types."""
import numpy as np
import pytest
import torch

from oracle import t5_oracle as O
from paper_2203_17189_b200 import binding as Bd
from paper_2203_17189_b200 import workloads as WL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_adamw_matches_oracle_over_steps(dtype):
    dims = WL.model_dims("tiny")
    h = Bd.Handle(Bd.make_config(dims, 4, 64, 32, dtype))
    n = h.t5_param_count()
    man = h.t5_param_manifest()
    rng = np.random.default_rng(3)
    theta0 = (rng.standard_normal(n) * 0.05).astype(np.float32)
    master = torch.from_numpy(theta0).to(DEV)
    params = master.to(h.torch_dtype)
    m = torch.zeros(n, dtype=torch.float32, device=DEV)
    v = torch.zeros(n, dtype=torch.float32, device=DEV)
    # which elements decay: everything that belongs to a tensor of two or more dimensions
    decay = np.zeros(n, dtype=bool)
    covered = np.zeros(n, dtype=bool)
    for name, off, shape in man:
        sz = int(np.prod(shape))
        covered[off:off + sz] = True
        decay[off:off + sz] = len(shape) > 1
    th, mo, vo = theta0.astype(np.float64), np.zeros(n), np.zeros(n)
    lr, b1, b2, eps, wd, gs = 3e-3, 0.9, 0.98, 1e-7, 0.05, 0.5
    for step in range(1, 4):
        g = (rng.standard_normal(n) * 0.1).astype(np.float32)
        g[~covered] = 0.0                      # padding between tensors carries zero gradient
        h.t5_adamw_update(params, master, m, v, torch.from_numpy(g).to(DEV), step, lr, b1, b2, eps, wd, gs)
        t_d, m_d, v_d = O.adamw_update(th, mo, vo, g, step, lr, b1, b2, eps, wd, gs)
        t_n, _, _ = O.adamw_update(th, mo, vo, g, step, lr, b1, b2, eps, 0.0, gs)
        th, mo, vo = np.where(decay, t_d, t_n), m_d, v_d
    torch.cuda.synchronize()
    got = master.cpu().numpy().astype(np.float64)
    assert np.abs(got - th)[covered].max() <= 2e-6 * np.abs(th).max()
    assert np.abs(m.cpu().numpy() - mo)[covered].max() <= 1e-6 * np.abs(mo).max()
    assert np.abs(v.cpu().numpy() - vo)[covered].max() <= 1e-6 * np.abs(vo).max()
    # the operand-dtype copy is the master weight rounded
    assert torch.equal(params, master.to(h.torch_dtype))


def test_adamw_argument_errors():
    dims = WL.model_dims("tiny")
    h = Bd.Handle(Bd.make_config(dims, 4, 64, 32, "f32"))
    n = h.t5_param_count()
    t = torch.zeros(n, dtype=torch.float32, device=DEV)
    with pytest.raises(Bd.T5Error) as e:
        h.t5_adamw_update(t, t, t, t, t, 0, 1e-3)
    assert e.value.code == -8
    with pytest.raises(Bd.T5Error) as e:
        h.t5_adamw_update(t, None, t, t, t, 1, 1e-3)
    assert e.value.code == -1
