"""Data-parallel combination on two gloo ranks (CPU): each rank takes half of a batch through the oracle, the
combined loss and gradients must equal the oracle's on the whole batch - which holds only with the W_r / W
weighting, since the halves carry different numbers of non-pad targets."""
import os
import socket

import numpy as np
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

from oracle import t5_oracle as O
from paper_2203_17189_b200 import data_parallel as DP
from paper_2203_17189_b200 import workloads as WL


def _inputs():
    cfg = O.T5Config(arch=0, n_enc_layers=1, n_dec_layers=1, d_model=32, n_heads=2, d_kv=8, d_ff=48, vocab=40)
    rng = np.random.default_rng(0)
    enc = rng.integers(1, cfg.vocab, size=(4, 9)).astype(np.int32)
    dec = rng.integers(1, cfg.vocab, size=(4, 7)).astype(np.int32)
    dec[0, 3:] = 0          # uneven target counts: 3 + 7 on rank 0, 7 + 5 on rank 1
    dec[3, 5:] = 0
    params = WL.make_params(O.param_shapes(cfg), 1, stddev=0.2, scale_jitter=0.2)
    return cfg, params, enc, dec


def _flat(grads):
    return np.concatenate([np.asarray(grads[k], dtype=np.float64).reshape(-1) for k in sorted(grads)])


def _worker(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg, params, enc, dec = _inputs()
    rows = slice(2 * rank, 2 * rank + 2)
    loss4, grads = O.t5_train_step(cfg, params, enc[rows], None, dec[rows], None)
    g = torch.from_numpy(_flat(grads).astype(np.float32))
    l4 = torch.from_numpy(loss4.astype(np.float32))
    W = DP.combine(g, l4, bucket_elements=1000)      # several buckets
    if rank == 0:
        out.put((g.numpy(), l4.numpy(), W))
    dist.destroy_process_group()


def test_two_ranks_equal_the_whole_batch():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    g, l4, W = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    cfg, params, enc, dec = _inputs()
    loss4, grads = O.t5_train_step(cfg, params, enc, None, dec, None)
    assert W == loss4[3] == 22
    assert np.abs(l4[:3] - loss4[:3]).max() <= 1e-6 * abs(loss4[0])
    ref = _flat(grads)
    assert np.abs(g - ref).max() <= 1e-6 * np.abs(ref).max()
    # the plain mean of the two ranks' gradients is NOT the answer here (different target counts)
    assert (3 + 7) != (7 + 5)


def test_bucket_ranges_cover_the_buffer_back_to_front():
    r = DP.bucket_ranges(10, 4)
    assert r == [(6, 10), (2, 6), (0, 2)]
    assert DP.bucket_ranges(0, 4) == []


def _worker_overlapped(rank, world, port, out):
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    cfg, params, enc, dec = _inputs()
    rows = slice(2 * rank, 2 * rank + 2)
    loss4, grads = O.t5_train_step(cfg, params, enc[rows], None, dec[rows], None)
    g = torch.from_numpy(_flat(grads).astype(np.float32))
    l4 = torch.from_numpy(loss4.astype(np.float32))
    red = DP.OverlappedReducer(g)
    # the ranges arrive the way the library reports them: from the end of the buffer towards its start, ragged sizes
    n, hi = g.numel(), g.numel()
    for size in (977, 1500, 3, 10 ** 9):
        lo = max(0, hi - size)
        red.reduce_range(lo, hi - lo, l4[3:4].clone())
        hi = lo
    W, covered = red.finish(l4)
    if rank == 0:
        out.put((g.numpy(), l4.numpy(), W, covered, n))
    dist.destroy_process_group()


def test_overlapped_reducer_equals_the_whole_batch():
    """The reducer the gradient-ready hook drives: every range scaled by W_r, summed over the ranks as it arrives,
    everything divided by W at the end - the whole-batch loss and gradients again."""
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    out = ctx.Queue()
    procs = [ctx.Process(target=_worker_overlapped, args=(r, 2, port, out)) for r in range(2)]
    for p in procs:
        p.start()
    g, l4, W, covered, n = out.get(timeout=120)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    cfg, params, enc, dec = _inputs()
    loss4, grads = O.t5_train_step(cfg, params, enc, None, dec, None)
    assert W == loss4[3] == 22
    assert np.abs(l4[:3] - loss4[:3]).max() <= 1e-6 * abs(loss4[0])
    ref = _flat(grads)
    assert np.abs(g - ref).max() <= 1e-6 * np.abs(ref).max()
    pos = 0
    for off, cnt in covered:         # disjoint, gap-free cover of the buffer
        assert off == pos
        pos += cnt
    assert pos == n
