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


def test_bounded_wait_gives_up_and_reports():
    """The kernels' wait routine on a barrier nothing arrives at: it must give up after its limit, leave its code
    in the status word and return normally (no trap, no hang); the context stays usable afterwards."""
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    Bd.t5_selftest_bounded_wait(status, 2_000_000)          # about a millisecond of SM cycles
    torch.cuda.synchronize()
    assert int(status.item()) == 99
    with pytest.raises(Bd.T5Error):
        Bd.t5_selftest_bounded_wait(status, 0)
    # the device still works: a tensor-core GEMM through the kernel-level entry point, with a status word attached
    status.zero_()
    Bd.t5_kernel_status_word(status)
    try:
        a = torch.randn(256, 128, device=DEV).to(torch.bfloat16)
        b = torch.randn(384, 128, device=DEV).to(torch.bfloat16)
        d = torch.empty(256, 384, dtype=torch.bfloat16, device=DEV)
        Bd.t5_gemm(1, 256, 384, 128, 1.0, a, 128, True, b, 128, True, d, 384)
        torch.cuda.synchronize()
        assert int(status.item()) == 0
        ref = a.float() @ b.float().T
        assert (d.float() - ref).abs().max() <= 2e-2 * ref.abs().max()
    finally:
        Bd.t5_kernel_status_word(None)
