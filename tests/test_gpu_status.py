"""The status word through which a bounded device-side wait reports that it ran out.

Every wait of the tensor-core kernels on a TMA or MMA barrier has a limit; a wait that runs out writes a code into
the first word of the workspace instead of spinning, and t5_device_status turns a non-zero word into
T5_ERR_DEVICE_TIMEOUT.  The test plants the word from the host side (nothing is launched that could wait) and
checks the mapping both ways."""
import pytest
import torch

from paper_2203_17189_b200 import binding as Bd
from paper_2203_17189_b200 import workloads as WL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def test_status_word_maps_to_timeout_error_and_clears():
    dims = WL.model_dims("tiny")
    h = Bd.Handle(Bd.make_config(dims, 4, 64, 32, "bf16"))
    ws = torch.zeros(h.t5_workspace_bytes(), dtype=torch.uint8, device=DEV)
    h.t5_device_status(ws)                                  # clean workspace: no error
    ws[:4].view(torch.int32)[0] = 8                         # the code the GEMM's MMA warp leaves when a stage never fills
    torch.cuda.synchronize()
    with pytest.raises(Bd.T5Error) as e:
        h.t5_device_status(ws)
    assert e.value.code == -7
    assert "code 8" in str(e.value)
    ws[:4].zero_()
    torch.cuda.synchronize()
    h.t5_device_status(ws)                                  # cleared: usable again


def test_step_clears_a_stale_status_word():
    """A step starts by zeroing the word, so an old code does not outlive the call that caused it."""
    dims = WL.model_dims("tiny")
    h = Bd.Handle(Bd.make_config(dims, 4, 64, 32, "bf16"))
    n = h.t5_param_count()
    params = torch.empty(n, dtype=torch.bfloat16, device=DEV)
    h.t5_init_params(params, 3, 0.02)
    ws = torch.zeros(h.t5_workspace_bytes(), dtype=torch.uint8, device=DEV)
    ws[:4].view(torch.int32)[0] = 3
    grads = torch.empty(n, dtype=torch.float32, device=DEV)
    loss4 = torch.zeros(4, dtype=torch.float32, device=DEV)
    batch = {k: (None if v is None else torch.from_numpy(v).to(DEV)) for k, v in WL.make_batch("tiny").items()}
    h.t5_train_step_fwd_bwd(params, batch, grads, loss4, ws)
    torch.cuda.synchronize()
    h.t5_device_status(ws)
    assert torch.isfinite(loss4).all()
