"""The gradient-ready hook of the training step and the reducer it drives, on one GPU.

With one rank the all-reduce is the identity, so the hooked step must reproduce the plain step; what the test pins
is everything around the collective: the ranges reported from inside the backward pass are disjoint and cover the
gradient buffer, each range really is final when the reducer's stream reaches it (a range scaled too early would be
overwritten by a later kernel and come out unscaled, or be scaled twice), and the W_r weighting and the final
division cancel.  The process group is a one-rank NCCL group when NCCL can be initialised, else none."""
import os
import socket

import numpy as np
import pytest
import torch
import torch.distributed as dist

from paper_2203_17189_b200 import binding as Bd
from paper_2203_17189_b200 import data_parallel as DP
from paper_2203_17189_b200 import workloads as WL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@pytest.fixture(scope="module")
def one_rank_group():
    made = False
    if not dist.is_initialized():
        with socket.socket() as s:
            s.bind(("127.0.0.1", 0))
            port = s.getsockname()[1]
        os.environ["MASTER_ADDR"] = "127.0.0.1"
        os.environ["MASTER_PORT"] = str(port)
        try:
            torch.cuda.set_device(0)
            dist.init_process_group("nccl", rank=0, world_size=1)
            made = True
        except Exception:
            made = False
    yield
    if made:
        dist.destroy_process_group()


@pytest.mark.parametrize("workload,flags", [("tiny", 0), ("small", 0), ("small", 16)])
def test_hooked_step_equals_plain_step(one_rank_group, workload, flags):
    dims = WL.model_dims(workload)
    dims = dict(dims, n_enc_layers=min(dims["n_enc_layers"], 3), n_dec_layers=min(dims["n_dec_layers"], 3))
    B = min(dims["batch"], 4)
    batch = WL.make_batch(dims, batch=B)
    h = Bd.Handle(Bd.make_config(dims, B, dims["enc_len"], dims["dec_len"], "f32" if workload == "tiny" else "bf16", flags=flags))
    n = h.t5_param_count()
    params = torch.empty(n, dtype=h.torch_dtype, device=DEV)
    h.t5_init_params(params, 7, 0.02)
    ws = torch.empty(h.t5_workspace_bytes(), dtype=torch.uint8, device=DEV)
    dbatch = {k: (None if v is None else torch.from_numpy(v).to(DEV)) for k, v in batch.items()}

    def step(grads, loss4):
        h.t5_train_step_fwd_bwd(params, dbatch, grads, loss4, ws)

    g_plain = torch.empty(n, dtype=torch.float32, device=DEV)
    g_again = torch.empty(n, dtype=torch.float32, device=DEV)
    l_plain = torch.zeros(4, dtype=torch.float32, device=DEV)
    step(g_again, l_plain)
    step(g_plain, l_plain)
    torch.cuda.synchronize()
    h.t5_device_status(ws)
    # two plain runs differ a little in bfloat16 mode (float atomics in the row statistics, the bias and the
    # embedding gradients): that spread is the yardstick for "equal"
    noise = (g_plain - g_again).abs().cpu().numpy()

    g_hook = torch.full((n,), float("nan"), dtype=torch.float32, device=DEV)
    l_hook = torch.zeros(4, dtype=torch.float32, device=DEV)
    red = DP.OverlappedReducer(g_hook).attach(h)
    try:
        step(g_hook, l_hook)
        W, covered = red.finish(l_hook)
    finally:
        h.t5_set_grad_hook(None)
    torch.cuda.synchronize()
    h.t5_device_status(ws)
    pos = 0
    for off, cnt in covered:         # disjoint, gap-free cover of the buffer
        assert off == pos, (off, pos)
        pos += cnt
    assert pos == n
    assert len(covered) >= dims["n_enc_layers"] + dims["n_dec_layers"] + 2
    assert W == float(l_plain[3].item()) > 0
    gp, gh = g_plain.cpu().numpy(), g_hook.cpu().numpy()
    assert np.isfinite(gh).all()
    # multiplying by W_r and dividing by W again costs two float32 roundings; a range handled at the wrong time
    # would be off by a factor of W_r (hundreds) or hold NaN
    man = h.t5_param_manifest()
    for name, off, shape in man:
        cnt = int(np.prod(shape))
        a, b = gp[off:off + cnt], gh[off:off + cnt]
        scale = max(np.abs(a).max(), 1e-30)
        assert np.abs(a - b).max() <= 1e-5 * scale + 4 * noise[off:off + cnt].max(), name
    assert np.abs(l_plain.cpu().numpy() - l_hook.cpu().numpy()).max() <= 1e-5 * abs(float(l_plain[0].item()))
    # without a hook the step is the plain one again
    step(g_hook, l_hook)
    torch.cuda.synchronize()
