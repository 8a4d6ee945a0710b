"""Incremental decoding with the key / value cache: fed the teacher-forced inputs one position at a time,
t5_decode_step must reproduce row t of the teacher-forced logits (the library's own t5_decode_logits and the oracle's),
for the encoder-decoder and the decoder-only model, float32 (SIMT kernels) and bfloat16 (tcgen05 kernels)."""
import numpy as np
import pytest
import torch

from oracle import t5_oracle as O
from paper_2203_17189_b200 import binding as Bd
from paper_2203_17189_b200 import workloads as WL
from tests import parity as PR

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def to_dev(a):
    return None if a is None else torch.from_numpy(np.ascontiguousarray(a)).to(DEV)


@pytest.mark.parametrize("arch,dtype,d_kv", [(0, "f32", 32), (0, "bf16", 64), (1, "bf16", 64), (1, "f32", 32)])
def test_decode_steps_reproduce_teacher_forced_logits(arch, dtype, d_kv):
    if arch == 0:
        dims = WL.model_dims("small", n_enc_layers=2, n_dec_layers=2, vocab=512, d_model=128, n_heads=2, d_kv=d_kv,
                             d_ff=256, enc_len=40, dec_len=21, batch=3, padding=0.2)
    else:
        dims = WL.model_dims("declm", n_dec_layers=2, vocab=512, d_model=128, n_heads=2, d_kv=d_kv, d_ff=256,
                             dec_len=33, batch=3, packed=False)
    batch = WL.make_batch(dims, seed=5)
    B, Td, V = dims["batch"], dims["dec_len"], dims["vocab"]
    Te = dims["enc_len"] if arch == 0 else 0
    h = Bd.Handle(Bd.make_config(dims, B, max(Te, 1), Td, dtype))
    man, n = h.t5_param_manifest(), h.t5_param_count()
    named = WL.make_params(PR.oracle_shapes_from_manifest(man), 6, stddev=0.05, scale_jitter=0.05)
    params = torch.from_numpy(PR.pack_params(man, n, named)).to(DEV).to(h.torch_dtype)
    named = PR.unpack(man, params.float().cpu().numpy())
    ws = torch.empty(h.t5_workspace_bytes(), dtype=torch.uint8, device=DEV)
    dev_batch = {k: to_dev(v) for k, v in batch.items()}
    tdt = h.torch_dtype
    enc_out = None
    if arch == 0:
        enc_out = torch.empty(B, Te, dims["d_model"], dtype=tdt, device=DEV)
        h.t5_encode(params, dev_batch, enc_out, ws)
    full = torch.empty(B, Td, V, dtype=tdt, device=DEV)
    h.t5_decode_logits(params, dev_batch, enc_out, full, ws)
    # decoder inputs: targets shifted right (one example per row)
    tgt = batch["dec_targets"]
    dec_in = np.zeros_like(tgt)
    dec_in[:, 1:] = tgt[:, :-1]
    cache = torch.empty(h.t5_decode_cache_bytes(B, Te, Td), dtype=torch.uint8, device=DEV)
    sws = torch.empty(h.t5_decode_step_workspace_bytes(B), dtype=torch.uint8, device=DEV)
    h.t5_decode_begin(params, B, Te, Td, dev_batch.get("enc_tokens"), enc_out, cache)
    steps = torch.empty(B, Td, V, dtype=tdt, device=DEV)
    for t in range(Td):
        logits_t = torch.empty(B, V, dtype=tdt, device=DEV)
        h.t5_decode_step(params, cache, B, Te, Td, t, to_dev(dec_in[:, t].astype(np.int32)), logits_t, sws)
        steps[:, t] = logits_t
    torch.cuda.synchronize()
    h.t5_device_status(sws)
    got, ref = steps.float().cpu().numpy(), full.float().cpu().numpy()
    assert np.isfinite(got).all()
    # rows at padded target positions are outside the contract of the teacher-forced call (padding queries)
    valid = tgt != 0
    tol = 1e-4 if dtype == "f32" else 2e-2
    assert np.abs(got - ref)[valid].max() <= tol * np.abs(ref).max()
    ocfg = O.T5Config(**{k: dims[k] for k in WL.MODEL_KEYS})
    oe = None if arch else O.t5_encode(ocfg, named, batch["enc_tokens"], None)
    ol = O.t5_decode_logits(ocfg, named, oe, batch["enc_tokens"], None, tgt, None)
    # against the oracle the bfloat16 run also carries the rounding of every stored activation of a narrow model
    # whose logits are small (|logit| <= 0.2): twice the bar of the step-against-full comparison
    assert np.abs(got - ol)[valid].max() <= (tol if dtype == "f32" else 4e-2) * np.abs(ol).max()


def test_decode_argument_errors():
    dims = WL.model_dims("tiny")
    h = Bd.Handle(Bd.make_config(dims, 4, 64, 32, "f32"))
    t = torch.zeros(1024, dtype=torch.uint8, device=DEV)
    p = torch.zeros(h.t5_param_count(), dtype=torch.float32, device=DEV)
    with pytest.raises(Bd.T5Error) as e:
        h.t5_decode_begin(p, 4, 64, 32, torch.zeros(4, 64, dtype=torch.int32, device=DEV),
                          torch.zeros(4, 64, 128, dtype=torch.float32, device=DEV), t)
    assert e.value.code == -5
    with pytest.raises(Bd.T5Error) as e:
        h.t5_decode_step(p, t, 4, 64, 32, 40, torch.zeros(4, dtype=torch.int32, device=DEV), t, t)
    assert e.value.code == -3
