"""Members of the model family beside T5.1.1 ("Example Models" section of the paper): T5 v1.0's ReLU FFN, the
exact (erf) GELU, a separate output head, and the prefix-LM mask of the decoder-only model - each a configuration
field on both sides, GPU step against the oracle at the usual bars."""
import numpy as np
import pytest

from paper_2203_17189_b200 import workloads as WL
from tests.test_gpu_parity import check_step

pytestmark = pytest.mark.gpu

VARIANTS = {
    "relu": (dict(ffn_act=1), dict(ffn_act="relu")),
    "gelu-erf": (dict(ffn_act=2), dict(ffn_act="gated-gelu-erf")),
    "untied": (dict(untied_head=1), dict(tied_embedding=False)),
}


def small_dims(**kw):
    base = dict(n_enc_layers=2, n_dec_layers=2, vocab=1000, d_model=192, n_heads=2, d_ff=320, enc_len=75,
                dec_len=40, batch=4, padding=0.2)
    base.update(kw)
    return WL.model_dims("small", **base)


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("variant", list(VARIANTS))
def test_step_variant(variant, dtype):
    gpu_kw, oracle_kw = VARIANTS[variant]
    dims = small_dims()
    check_step(dims, WL.make_batch(dims, seed=31), dtype, floor=True, gpu_kw=gpu_kw, oracle_kw=oracle_kw)


def test_step_variants_combined_xl_width_bf16():
    """ReLU FFN and separate head together at the XL width (the tensor-core GEMMs with the plain epilogues),
    attention logits of order one.  ReLU's kink turns operand rounding into sign flips of pre-activations: the
    oracle's own bfloat16-operand floor is 5e-2 here, so the bar is twice that floor."""
    dims = WL.model_dims("xl", batch=2, n_enc_layers=1, n_dec_layers=1)
    check_step(dims, WL.make_batch(dims), "bf16", attn_scale=dims["d_kv"] ** -0.5, floor=True,
               gpu_kw=dict(ffn_act=1, untied_head=1), oracle_kw=dict(ffn_act="relu", tied_embedding=False))


def prefix_batch(dims, seed):
    """Packed decoder-only rows; the first third (at least one position) of every document is its given prefix."""
    batch = WL.make_batch(dims, seed=seed)
    seg = batch["dec_segment_ids"]
    pre = np.zeros_like(seg)
    for b in range(seg.shape[0]):
        for s in np.unique(seg[b]):
            if s == 0:
                continue
            idx = np.nonzero(seg[b] == s)[0]
            pre[b, idx[:max(1, len(idx) // 3)]] = 1
    batch["dec_prefix"] = pre.astype(np.int32)
    return batch


@pytest.mark.parametrize("dtype,d_kv,dec_len", [("f32", 32, 70), ("bf16", 64, 150), ("bf16", 128, 300)])
def test_step_prefix_lm(dtype, d_kv, dec_len):
    dims = WL.model_dims("declm", n_dec_layers=2, vocab=2000, d_model=256, n_heads=2, d_kv=d_kv, d_ff=384,
                         dec_len=dec_len, batch=2)
    batch = prefix_batch(dims, seed=9)
    assert batch["dec_prefix"].sum() > 0
    for flags in ((0,) if dtype == "f32" else (0, 1 << 17)):
        check_step(dims, batch, dtype, flags=flags, floor=True)


def test_prefix_lm_without_flags_is_the_causal_model():
    dims = WL.model_dims("declm", n_dec_layers=1, vocab=512, d_model=128, n_heads=2, d_kv=64, d_ff=256,
                         dec_len=100, batch=2)
    batch = WL.make_batch(dims, seed=4)
    _, _, loss_a, grads_a = check_step(dims, batch, "bf16", floor=True)
    batch["dec_prefix"] = np.zeros_like(batch["dec_targets"])
    _, _, loss_b, grads_b = check_step(dims, batch, "bf16", floor=True)
    assert abs(loss_a[0] - loss_b[0]) <= 1e-6 * abs(loss_a[0])
