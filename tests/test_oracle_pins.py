"""Pins for the CPU oracle: each test ties a part of oracle/t5_oracle.py to
something that is not the oracle (hand-derived tables, closed forms, finite
differences, an autograd restatement, invariances)."""
import math
import os

import numpy as np
import pytest
import torch

from oracle import t5_oracle as O
from paper_2203_17189_b200 import workloads as WL

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def tiny_cfg(**kw):
    base = dict(arch=0, n_enc_layers=2, n_dec_layers=2, d_model=32, n_heads=2, d_kv=8, d_ff=48,
                vocab=40)
    base.update(kw)
    return O.T5Config(**base)


def tiny_inputs(cfg, B=2, Te=9, Td=7, seed=0, pad=True, stddev=0.3):
    rng = np.random.default_rng(seed)
    enc = rng.integers(1, cfg.vocab, size=(B, Te)).astype(np.int32)
    dec = rng.integers(1, cfg.vocab, size=(B, Td)).astype(np.int32)
    if pad:
        enc[0, Te - 2:] = 0
        dec[0, Td - 3:] = 0
    params = WL.make_params(O.param_shapes(cfg), seed + 1, stddev=stddev, scale_jitter=0.2)
    return params, enc, dec


# ------------------------------------------------------------------ buckets
def _read_thresholds():
    th = {"bidir": [], "unidir": []}
    for line in open(os.path.join(GOLD, "bucket_thresholds.txt")):
        if line.startswith("#") or not line.strip():
            continue
        mode, n, b = line.split()
        th[mode].append((int(n), int(b)))
    return th


def test_bucket_against_hand_table():
    th = _read_thresholds()
    for mode, bid in (("bidir", True), ("unidir", False)):
        starts = th[mode]
        for n in range(0, 2048):
            want = max(b for (s, b) in starts if s <= n)
            assert O.relative_position_bucket(-n, bid) == want, (mode, n)
            if bid and n > 0:
                assert O.relative_position_bucket(n, bid) == want + 16
            if not bid and n > 0:
                assert O.relative_position_bucket(n, bid) == 0


def test_bucket_hand_picked_distances():
    bi = {0: 0, 1: 1, 7: 7, 8: 8, 11: 8, 12: 9, 15: 9, 16: 10, 22: 10, 23: 11, 31: 11, 32: 12,
          45: 12, 46: 13, 63: 13, 64: 14, 90: 14, 91: 15, 127: 15, 128: 15, 2047: 15}
    for n, b in bi.items():
        assert O.relative_position_bucket(-n, True) == b
        if n:
            assert O.relative_position_bucket(n, True) == b + 16
    uni = {0: 0, 15: 15, 16: 16, 18: 16, 19: 17, 45: 23, 46: 24, 98: 29, 99: 30, 112: 30,
           113: 31, 128: 31, 2047: 31}
    for n, b in uni.items():
        assert O.relative_position_bucket(-n, False) == b
    assert O.relative_position_bucket(1, False) == 0
    assert O.relative_position_bucket(500, False) == 0


def test_bucket_matches_float_log_away_from_integers():
    """Independent evaluation with floating logarithms wherever the real value
    is not within 1e-9 of an integer (where rounding could decide)."""
    for bid, nb in ((True, 16), (False, 32)):
        me = nb // 2
        for n in range(me, 3000):
            t = math.log(n / me) / math.log(128 / me) * (nb - me)
            if abs(t - round(t)) < 1e-9:
                continue
            want = min(nb - 1, me + int(math.floor(t)))
            assert O.relative_position_bucket(-n, bid) == want


def test_bucket_structure():
    for bid in (True, False):
        prev = -1
        for n in range(0, 500):
            b = O.relative_position_bucket(-n, bid)
            assert b >= prev
            prev = b
    assert all(O.relative_position_bucket(-n, True) != 16 for n in range(-300, 300))
    m = O.bucket_matrix(5, 7, True, 32, 128)
    assert m[2, 2] == 0 and m[0, 6] == 16 + 6 and m[4, 0] == 4


# ------------------------------------------------------- elementwise pieces
def test_gelu_printed_values_and_derivative():
    for line in open(os.path.join(GOLD, "closed_forms.txt")):
        if line.startswith("gelu "):
            _, u, v = line.split()
            assert abs(float(O.gelu_tanh(np.float64(u))) - float(v)) < 1e-6
    u = np.linspace(-4, 4, 41)
    h = 1e-6
    fd = (O.gelu_tanh(u + h) - O.gelu_tanh(u - h)) / (2 * h)
    assert np.allclose(O.gelu_tanh_grad(u), fd, atol=1e-8)
    # against the library's own tanh-GELU
    tg = torch.nn.functional.gelu(torch.tensor(u), approximate="tanh").numpy()
    assert np.allclose(O.gelu_tanh(u), tg, atol=1e-12)


def test_rmsnorm_definition_and_orthogonality():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((5, 16))
    g = 1 + 0.1 * rng.standard_normal(16)
    y, r = O.rms_norm(x, g, 1e-6)
    for i in range(5):
        ms = sum(v * v for v in x[i]) / 16
        assert np.allclose(y[i], x[i] / math.sqrt(ms + 1e-6) * g)
    dy = rng.standard_normal((5, 16))
    dx, dg = O.rms_norm_bwd(dy, x, g, r)
    # d/dx of a scale-invariant function is orthogonal to x (eps -> 0)
    assert np.all(np.abs(np.sum(dx * x, axis=-1)) < 1e-5)
    tx = torch.tensor(x, requires_grad=True)
    tg_ = torch.tensor(g, requires_grad=True)
    ty = tx * torch.rsqrt((tx * tx).mean(-1, keepdim=True) + 1e-6) * tg_
    ty.backward(torch.tensor(dy))
    assert np.allclose(dx, tx.grad.numpy(), atol=1e-12)
    assert np.allclose(dg, tg_.grad.numpy(), atol=1e-12)


def test_softmax_rows_masks_uniform():
    rng = np.random.default_rng(0)
    s = rng.standard_normal((6, 9)) * 3
    code_q = np.array([1, 1, 1, 2, 2, 0])
    code_k = np.array([1, 1, 1, 2, 2, 2, 0, 0, 1])
    m = O.attention_mask(code_q, code_k, causal=False)
    p = O.masked_softmax(s, m)
    assert np.allclose(p[:5].sum(-1), 1.0, atol=1e-12)
    assert np.all(p[~m] == 0.0)
    assert np.all(p[5] == 0.0)                      # padding query: no valid key
    mc = O.attention_mask(np.ones(6, int), np.ones(6, int), causal=True)
    pc = O.masked_softmax(rng.standard_normal((6, 6)), mc)
    assert np.all(np.triu(pc, 1) == 0.0) and np.allclose(pc.sum(-1), 1.0)
    pu = O.masked_softmax(np.zeros((6, 9)), m)
    for i in range(5):
        assert np.allclose(pu[i][m[i]], 1.0 / m[i].sum())


def test_shift_right_and_codes():
    t = np.array([5, 6, 7, 8, 9, 0, 0])
    assert list(O.shift_right(t, None)) == [0, 5, 6, 7, 8, 9, 0]
    seg = np.array([1, 1, 2, 2, 2, 0, 0])
    assert list(O.shift_right(t, seg)) == [0, 5, 0, 7, 8, 0, 0]
    assert list(O.position_codes(t, seg)) == [1, 1, 2, 2, 2, 0, 0]
    assert list(O.position_codes(t, None)) == [1, 1, 1, 1, 1, 0, 0]


# ------------------------------------------------------------- loss closed form
@pytest.mark.parametrize("V", [512, 32128])
def test_zloss_closed_form_zero_embedding(V):
    want = None
    for line in open(os.path.join(GOLD, "closed_forms.txt")):
        if line.startswith("zloss") and int(line.split()[1]) == V:
            want = float(line.split()[2])
    cfg = O.T5Config(arch=0, n_enc_layers=1, n_dec_layers=1, d_model=16, n_heads=2, d_kv=8, d_ff=16,
                     vocab=V)
    params = WL.make_params(O.param_shapes(cfg), 5)
    params["token_embed"][:] = 0
    rng = np.random.default_rng(1)
    enc = rng.integers(1, V, size=(2, 5)).astype(np.int32)
    dec = rng.integers(1, V, size=(2, 4)).astype(np.int32)
    dec[1, 3] = 0
    loss4, _ = O.t5_train_step(cfg, params, enc, None, dec, None)
    assert abs(loss4[0] - want) < 1e-8
    assert abs(loss4[1] - math.log(V)) < 1e-9
    assert loss4[3] == 7


def test_dlogits_row_sum_identity():
    cfg = tiny_cfg()
    params, enc, dec = tiny_inputs(cfg)
    loss4, g, aux = O.t5_train_step(cfg, params, enc, None, dec, None, return_aux=True)
    W = loss4[3]
    for b in range(2):
        logits = aux["logits"][b]
        lse = np.log(np.exp(logits).sum(-1))
        w = (dec[b] != 0)
        assert np.allclose(aux["dlogits"][b].sum(-1), w / W * 2 * cfg.z_loss * lse, atol=1e-12)


# ------------------------------------------------------------- gradients
def _fd_check(cfg, params, enc, eseg, dec, dseg, n_coord=24, all_of=("relbias",), seed=0, dec_prefix=None,
              h_rel=2e-4):
    loss4, g = O.t5_train_step(cfg, params, enc, eseg, dec, dseg, dtype=np.float64, dec_prefix=dec_prefix)
    rng = np.random.default_rng(seed)
    worst = 0.0
    p64 = {k: np.array(v, dtype=np.float64) for k, v in params.items()}
    for name, arr in p64.items():
        n = arr.size
        if any(s in name for s in all_of):
            idxs = range(n)
        else:
            idxs = rng.choice(n, size=min(n_coord, n), replace=False)
        flat = arr.reshape(-1)
        for i in idxs:
            old = flat[i]
            h = h_rel * max(1.0, abs(old))
            f = {}
            for mlt in (-2, -1, 1, 2):
                flat[i] = old + mlt * h
                f[mlt] = O.t5_loss_only(cfg, p64, enc, eseg, dec, dseg, dec_prefix=dec_prefix)
            flat[i] = old
            fd = (8 * (f[1] - f[-1]) - (f[2] - f[-2])) / (12 * h)     # 4th-order central difference
            an = g[name].reshape(-1)[i]
            err = abs(fd - an) / max(1e-3, abs(fd), abs(an))
            worst = max(worst, err)
            assert err < 1e-5, (name, i, fd, an)
    return worst


def test_finite_differences_encdec():
    cfg = tiny_cfg()
    params, enc, dec = tiny_inputs(cfg, stddev=0.12)
    _fd_check(cfg, params, enc, None, dec, None)


def test_finite_differences_packed_and_deconly():
    cfg = tiny_cfg(n_enc_layers=1, n_dec_layers=1)
    params, enc, dec = tiny_inputs(cfg, pad=False, stddev=0.12)
    eseg = np.array([[1, 1, 1, 1, 2, 2, 2, 0, 0], [1, 1, 2, 2, 2, 2, 3, 3, 3]], dtype=np.int32)
    dseg = np.array([[1, 1, 1, 2, 2, 0, 0], [1, 2, 2, 2, 3, 3, 3]], dtype=np.int32)
    enc = np.where(eseg == 0, 0, enc)
    dec = np.where(dseg == 0, 0, dec)
    _fd_check(cfg, params, enc, eseg, dec, dseg, n_coord=12)
    cfg1 = tiny_cfg(arch=1, n_enc_layers=0, n_dec_layers=2)
    params1 = WL.make_params(O.param_shapes(cfg1), 9, stddev=0.12, scale_jitter=0.2)
    _fd_check(cfg1, params1, None, None, dec, dseg, n_coord=12)


# --------------------------------------------- independent autograd restatement
def _torch_bucket(rel, bidirectional, nb=32, md=128):
    """Same closed form by a different route: float64 logs with a guard
    against landing a hair below an integer."""
    rel = rel.to(torch.int64)
    off = torch.zeros_like(rel)
    if bidirectional:
        nb //= 2
        off = (rel > 0).to(torch.int64) * nb
        n = rel.abs()
    else:
        n = (-rel).clamp(min=0)
    me = nb // 2
    big = me + torch.floor(torch.log(n.clamp(min=1).double() / me) / math.log(md / me) * (nb - me)
                           + 1e-9).to(torch.int64)
    big = big.clamp(max=nb - 1)
    return off + torch.where(n < me, n, big)


def _torch_model_loss(cfg, P, enc, eseg, dec, dseg):
    """Batched T5.1.1 loss with library ops and autograd, written separately
    from the oracle (different structure: batched, additive -inf masks)."""
    F = torch.nn.functional
    H, k = cfg.n_heads, cfg.d_kv

    def rms(x, g):
        return x * torch.rsqrt(x.pow(2).mean(-1, keepdim=True) + cfg.rms_eps) * g

    def codes(tok, seg):
        c = (tok != 0).long()
        return c if seg is None else c * seg.long()

    def attn(pref, xq, ykv, table, bidir, cq, ck, causal):
        yq = rms(xq, P[pref + ".norm"])
        src = yq if ykv is None else ykv
        B, Tq, _ = yq.shape
        Tk = src.shape[1]
        q = (yq @ P[pref + ".q"]).view(B, Tq, H, k).transpose(1, 2)
        kk = (src @ P[pref + ".k"]).view(B, Tk, H, k).transpose(1, 2)
        v = (src @ P[pref + ".v"]).view(B, Tk, H, k).transpose(1, 2)
        s = cfg.attn_scale * q @ kk.transpose(-1, -2)
        if table is not None:
            rel = torch.arange(Tk)[None, :] - torch.arange(Tq)[:, None]
            s = s + table[_torch_bucket(rel, bidir, cfg.rel_buckets, cfg.rel_max_distance)].permute(2, 0, 1)[None]
        m = (ck[:, None, :] != 0) & (cq[:, :, None] == ck[:, None, :])
        if causal:
            m = m & (torch.arange(Tk)[None, None, :] <= torch.arange(Tq)[None, :, None])
        m = m[:, None]
        s = s.masked_fill(~m, float("-inf"))
        anyv = m.any(-1, keepdim=True)
        p = torch.softmax(torch.where(anyv, s, torch.zeros_like(s)), -1) * anyv
        c = (p @ v).transpose(1, 2).reshape(B, Tq, H * k)
        return xq + c @ P[pref + ".o"]

    def ffn(pref, x):
        y = rms(x, P[pref + ".norm"])
        return x + (F.gelu(y @ P[pref + ".wi0"], approximate="tanh") * (y @ P[pref + ".wi1"])) @ P[pref + ".wo"]

    E = P["token_embed"]
    dec_t = torch.as_tensor(dec).long()
    dsg = None if dseg is None else torch.as_tensor(dseg)
    cd = codes(dec_t, dsg)
    ey = ce = None
    if cfg.arch == 0:
        enc_t = torch.as_tensor(enc).long()
        esg = None if eseg is None else torch.as_tensor(eseg)
        ce = codes(enc_t, esg)
        x = E[enc_t]
        for l in range(cfg.n_enc_layers):
            x = attn(f"enc.L{l}.attn", x, None, P["enc.relbias"], True, ce, ce, False)
            x = ffn(f"enc.L{l}.ffn", x)
        ey = rms(x, P["enc.final_norm"])
    u = torch.zeros_like(dec_t)
    u[:, 1:] = dec_t[:, :-1]
    if dsg is not None:
        same = torch.zeros_like(dec_t, dtype=torch.bool)
        same[:, 1:] = dsg[:, 1:] == dsg[:, :-1]
        u = u * same
    x = E[u]
    for l in range(cfg.n_dec_layers):
        x = attn(f"dec.L{l}.self", x, None, P["dec.relbias"], False, cd, cd, True)
        if cfg.arch == 0:
            x = attn(f"dec.L{l}.cross", x, ey, None, False, cd, ce, False)
        x = ffn(f"dec.L{l}.ffn", x)
    z = rms(x, P["dec.final_norm"])
    logits = cfg.logit_scale * z @ E.T
    lse = torch.logsumexp(logits, -1)
    nll = F.cross_entropy(logits.reshape(-1, cfg.vocab), dec_t.reshape(-1), reduction="none").view_as(lse)
    w = (dec_t != 0).double()
    return (w * (nll + cfg.z_loss * lse ** 2)).sum() / w.sum()


@pytest.mark.parametrize("arch,packed", [(0, False), (0, True), (1, True)])
def test_against_autograd_restatement(arch, packed):
    cfg = tiny_cfg(arch=arch, n_enc_layers=0 if arch else 2)
    params, enc, dec = tiny_inputs(cfg, B=3, Te=40, Td=37, seed=4, pad=not packed)
    eseg = dseg = None
    if packed:
        rng = np.random.default_rng(2)
        eseg = np.sort(rng.integers(0, 4, size=enc.shape), axis=1)[:, ::-1].astype(np.int32)
        eseg = np.where(eseg == 0, 0, 4 - eseg)          # 1,1,..,2,..,3,..,0,0
        dseg = np.sort(rng.integers(0, 4, size=dec.shape), axis=1)[:, ::-1].astype(np.int32)
        dseg = np.where(dseg == 0, 0, 4 - dseg)
        enc = np.where(eseg == 0, 0, enc)
        dec = np.where(dseg == 0, 0, dec)
    if arch == 1:
        enc = eseg = None
    loss4, g = O.t5_train_step(cfg, params, enc, eseg, dec, dseg, dtype=np.float64)
    P = {k_: torch.tensor(v, dtype=torch.float64, requires_grad=True) for k_, v in params.items()}
    L = _torch_model_loss(cfg, P, enc, eseg, dec, dseg)
    L.backward()
    assert abs(float(L.detach()) - loss4[0]) < 1e-10
    for name in params:
        ref = P[name].grad.numpy()
        assert np.allclose(g[name], ref, rtol=1e-8, atol=1e-11), name


# ------------------------------------------------------------- invariances
def test_bias_table_gradient_sums_to_zero_per_head():
    cfg = tiny_cfg()
    params, enc, dec = tiny_inputs(cfg)
    _, g = O.t5_train_step(cfg, params, enc, None, dec, None)
    for name in ("enc.relbias", "dec.relbias"):
        assert np.all(np.abs(g[name].sum(0)) < 1e-12)
        assert np.abs(g[name]).max() > 1e-6
    # bucket 16 never occurs in the encoder; future buckets never in the decoder
    assert np.all(g["enc.relbias"][16] == 0)


def test_padding_extension_and_row_permutation():
    cfg = tiny_cfg()
    params, enc, dec = tiny_inputs(cfg)
    l0, g0 = O.t5_train_step(cfg, params, enc, None, dec, None)
    enc2 = np.concatenate([enc, np.zeros((2, 3), np.int32)], 1)
    dec2 = np.concatenate([dec, np.zeros((2, 2), np.int32)], 1)
    l1, g1 = O.t5_train_step(cfg, params, enc2, None, dec2, None)
    l2, g2 = O.t5_train_step(cfg, params, enc[::-1], None, dec[::-1], None)
    assert np.allclose(l0, l1, atol=1e-12) and np.allclose(l0, l2, atol=1e-12)
    for k_ in g0:
        assert np.allclose(g0[k_], g1[k_], atol=1e-12), k_
        assert np.allclose(g0[k_], g2[k_], atol=1e-12), k_


def test_packed_equals_unpacked():
    cfg = tiny_cfg()
    rng = np.random.default_rng(7)
    params = WL.make_params(O.param_shapes(cfg), 3, stddev=0.3, scale_jitter=0.2)
    eA, eB = rng.integers(1, 40, 5), rng.integers(1, 40, 6)
    dA, dB = rng.integers(1, 40, 4), rng.integers(1, 40, 3)
    enc_p = np.concatenate([eA, eB, [0, 0]])[None].astype(np.int32)
    eseg = np.array([[1] * 5 + [2] * 6 + [0, 0]], np.int32)
    dec_p = np.concatenate([dA, dB, [0]])[None].astype(np.int32)
    dseg = np.array([[1] * 4 + [2] * 3 + [0]], np.int32)
    lp, gp = O.t5_train_step(cfg, params, enc_p, eseg, dec_p, dseg)
    enc_u = np.zeros((2, 6), np.int32); enc_u[0, :5] = eA; enc_u[1] = eB
    dec_u = np.zeros((2, 4), np.int32); dec_u[0] = dA; dec_u[1, :3] = dB
    lu, gu = O.t5_train_step(cfg, params, enc_u, None, dec_u, None)
    assert np.allclose(lp, lu, atol=1e-12)
    for k_ in gp:
        assert np.allclose(gp[k_], gu[k_], atol=1e-12), k_


def test_teacher_forcing_causality_and_inference_methods():
    cfg = tiny_cfg()
    params, enc, dec = tiny_inputs(cfg, pad=False)
    eo = O.t5_encode(cfg, params, enc, None)
    lg = O.t5_decode_logits(cfg, params, eo, enc, None, dec, None)
    dec2 = dec.copy()
    dec2[:, 4] = (dec2[:, 4] % 38) + 1
    lg2 = O.t5_decode_logits(cfg, params, eo, enc, None, dec2, None)
    assert np.allclose(lg[:, :5], lg2[:, :5], atol=1e-12)      # target_4 first enters at position 5
    assert not np.allclose(lg[:, 5:], lg2[:, 5:], atol=1e-6)
    _, _, aux = O.t5_train_step(cfg, params, enc, None, dec, None, return_aux=True)
    assert np.allclose(np.stack(aux["logits"]), lg, atol=1e-12)
    assert np.allclose(np.stack(aux["enc_out"]), eo, atol=1e-12)


def test_textbook_single_head_attention():
    """H=1, zero table, no padding: the attention sub-layer is plain softmax
    attention (checked against the library routine)."""
    cfg = tiny_cfg(n_heads=1, d_kv=8)
    rng = np.random.default_rng(11)
    p = WL.make_params(O.param_shapes(cfg), 2, stddev=0.3)
    p = {k_: v.astype(np.float64) for k_, v in p.items()}
    p["enc.relbias"][:] = 0
    x = rng.standard_normal((6, cfg.d_model))
    code = np.ones(6, np.int32)
    out, _ = O._attn_fwd(cfg, p, "enc.L0.attn", x, None, p["enc.relbias"], True, code, code, False)
    y = x / np.sqrt((x * x).mean(-1, keepdims=True) + 1e-6) * p["enc.L0.attn.norm"]
    q, k_, v = (torch.tensor(y @ p["enc.L0.attn." + n]) for n in "qkv")
    ref = torch.nn.functional.scaled_dot_product_attention(q[None], k_[None], v[None], scale=1.0)[0].numpy()
    assert np.allclose(out, x + ref @ p["enc.L0.attn.o"], atol=1e-12)


def test_fp32_mode_close_to_fp64():
    cfg = tiny_cfg()
    params, enc, dec = tiny_inputs(cfg)
    l64, g64 = O.t5_train_step(cfg, params, enc, None, dec, None, dtype=np.float64)
    l32, g32 = O.t5_train_step(cfg, params, enc, None, dec, None, dtype=np.float32)
    assert abs(l64[0] - l32[0]) < 1e-5
    for k_ in g64:
        assert g32[k_].dtype == np.float32
        assert np.abs(g64[k_] - g32[k_]).max() <= 1e-4 * max(1e-3, np.abs(g64[k_]).max()), k_


def test_bf16_operand_rounding_floor():
    """What rounding ONLY the operands of the oracle's matrix products to bfloat16 costs.
    At the small model's width the gradients stay within the 2e-2 / 0.999 bars; at the XL width
    (attention logits of standard deviation ~6 at N(0, 0.02) initialisation) they do not, even for one
    layer and short sequences: that distance is a property of bfloat16 operands, not of an implementation."""
    from tests import parity as PR
    out = {}
    for name, kw in (("small", dict(d_model=512, n_heads=6, d_kv=64, d_ff=1024)),
                     ("xl", dict(d_model=2048, n_heads=32, d_kv=64, d_ff=5120))):
        dims = WL.model_dims("xl", n_enc_layers=1, n_dec_layers=1, vocab=2048, enc_len=96, dec_len=48, batch=2, **kw)
        batch = WL.make_batch(dims)
        cfg = O.T5Config(**{k: dims[k] for k in WL.MODEL_KEYS})
        params = WL.make_params(O.param_shapes(cfg), 3, round_bf16=True)
        _, g0 = O.t5_train_step(cfg, params, batch["enc_tokens"], None, batch["dec_targets"], None)
        cfg.operand_bf16 = True
        _, g1 = O.t5_train_step(cfg, params, batch["enc_tokens"], None, batch["dec_targets"], None)
        m = {k: PR.tensor_metrics(g1[k], g0[k]) for k in g0}
        out[name] = (min(v[0] for v in m.values()), max(v[1] for v in m.values()))
    assert out["small"][0] > 0.9995 and out["small"][1] < 3e-2
    assert out["xl"][1] > 3e-2          # beyond the bar already
    assert out["xl"][0] > 0.99          # yet still the same gradient
    # rounding helper itself: exact on representable values, ties to even
    a = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 2 ** -7, -3.140625, 1e-30], dtype=np.float64)
    r = O.round_bf16(a)
    assert r[0] == 1.0 and r[1] == 1.0 and r[2] == 1.0 + 2 ** -7 and r[3] == -3.140625
    assert np.all(r == WL.round_to_bf16(a.astype(np.float32)).astype(np.float64))


# ------------------------------------------------------------------ model-family variants
def test_erf_gelu_printed_values_and_derivative():
    """u Phi(u) at a few points from the standard normal table (Phi(1) = 0.8413447, Phi(2) = 0.9772499) and the
    derivative against a central difference."""
    for line in open(os.path.join(GOLD, "closed_forms.txt")):
        f = line.split()
        if f and f[0] == "gelu_erf":
            assert abs(float(O.gelu_erf(np.float64(f[1]))) - float(f[2])) < 1e-6
    assert abs(float(O.gelu_erf(np.float64(1.0))) - 0.8413447) < 1e-6
    u = np.linspace(-4, 4, 81)
    h = 1e-6
    fd = (O.gelu_erf(u + h) - O.gelu_erf(u - h)) / (2 * h)
    assert np.abs(fd - O.gelu_erf_grad(u)).max() < 1e-8
    # the tanh form approximates it to a few 1e-4 (that is why the two are different configurations)
    assert 1e-5 < np.abs(O.gelu_erf(u) - O.gelu_tanh(u)).max() < 1e-3


def test_relu_ffn_is_a_plain_mlp():
    """T5 v1.0's FFN: relu(y Wi) Wo - no gate, no second input matrix; against the definition written out."""
    cfg = tiny_cfg(ffn_act="relu")
    shapes = O.param_shapes(cfg)
    assert not any(k.endswith(".wi1") for k in shapes)
    rng = np.random.default_rng(0)
    p = {k: rng.standard_normal(v) * 0.3 for k, v in shapes.items()}
    x = rng.standard_normal((5, cfg.d_model))
    out, _ = O._ffn_fwd(cfg, p, "enc.L0.ffn", x)
    g = p["enc.L0.ffn.norm"]
    y = np.array([row / math.sqrt(np.mean(row ** 2) + cfg.rms_eps) * g for row in x])
    want = x + np.maximum(y @ p["enc.L0.ffn.wi0"], 0.0) @ p["enc.L0.ffn.wo"]
    assert np.abs(out - want).max() < 1e-12


def test_prefix_lm_mask_hand_case_and_limits():
    code = np.array([1, 1, 1, 1, 2, 2, 0], dtype=np.int32)
    pre = np.array([1, 1, 0, 0, 1, 0, 0], dtype=np.int32)
    m = O.attention_mask(code, code, True, pre, pre)
    want = np.zeros((7, 7), dtype=bool)
    for i, j in [(0, 0), (0, 1), (1, 0), (1, 1),             # the prefix of example 1 sees itself in full
                 (2, 0), (2, 1), (2, 2), (3, 0), (3, 1), (3, 2), (3, 3),   # its continuation stays causal
                 (4, 4), (5, 4), (5, 5)]:                    # example 2: one prefix position, one target
        want[i, j] = True
    assert np.array_equal(m, want)
    # no flags: plain causal mask; all flagged: the bidirectional mask of the same codes
    none = np.zeros(7, dtype=np.int32)
    assert np.array_equal(O.attention_mask(code, code, True, none, none), O.attention_mask(code, code, True))
    allp = np.ones(7, dtype=np.int32)
    assert np.array_equal(O.attention_mask(code, code, True, allp, allp), O.attention_mask(code, code, False))
    # prefix positions carry no loss
    tgt = np.array([5, 6, 7, 8, 9, 3, 0])
    assert O.loss_weights(tgt, pre).tolist() == [False, False, True, True, False, True, False]
    assert O.loss_weights(tgt).tolist() == [True] * 6 + [False]


@pytest.mark.parametrize("variant", ["relu", "gated-gelu-erf", "untied", "prefix"])
def test_finite_differences_variants(variant):
    kw = {}
    if variant in ("relu", "gated-gelu-erf"):
        kw["ffn_act"] = variant
    if variant == "untied":
        kw["tied_embedding"] = False
    pre = None
    if variant == "prefix":
        cfg = tiny_cfg(arch=1, n_enc_layers=0, n_dec_layers=2)
        params = WL.make_params(O.param_shapes(cfg), 5, stddev=0.12, scale_jitter=0.2)
        rng = np.random.default_rng(3)
        dec = rng.integers(1, cfg.vocab, size=(2, 9)).astype(np.int32)
        dseg = np.array([[1, 1, 1, 1, 1, 2, 2, 2, 0], [1, 1, 1, 1, 1, 1, 1, 1, 1]], dtype=np.int32)
        dec = np.where(dseg == 0, 0, dec)
        pre = np.array([[1, 1, 1, 0, 0, 1, 0, 0, 0], [1, 1, 1, 1, 0, 0, 0, 0, 0]], dtype=np.int32)
        _fd_check(cfg, params, None, None, dec, dseg, n_coord=12, dec_prefix=pre)
        return
    cfg = tiny_cfg(n_enc_layers=1, n_dec_layers=1, **kw)
    params, enc, dec = tiny_inputs(cfg, stddev=0.12)
    if variant == "untied":
        assert cfg.logit_scale == 1.0 and O.param_shapes(cfg)["lm_head"] == (cfg.d_model, cfg.vocab)
    # relu has kinks: a step small enough that no pre-activation changes sign inside the stencil
    _fd_check(cfg, params, enc, None, dec, None, n_coord=12, h_rel=1e-6 if variant == "relu" else 2e-4)


def test_untied_head_with_the_embedding_copied_equals_tied():
    """lm_head = token_embed^T with the tied logit scale gives the tied model's loss; the tied embedding gradient
    is the sum of the two untied pieces."""
    cfg_t = tiny_cfg(n_enc_layers=1, n_dec_layers=1)
    params, enc, dec = tiny_inputs(cfg_t, stddev=0.2)
    cfg_u = tiny_cfg(n_enc_layers=1, n_dec_layers=1, tied_embedding=False, logit_scale=cfg_t.logit_scale)
    pu = dict(params)
    pu["lm_head"] = params["token_embed"].T.copy()
    lt, gt = O.t5_train_step(cfg_t, params, enc, None, dec, None)
    lu, gu = O.t5_train_step(cfg_u, pu, enc, None, dec, None)
    assert abs(lt[0] - lu[0]) < 1e-12
    assert np.abs(gt["token_embed"] - (gu["token_embed"] + gu["lm_head"].T)).max() < 1e-12


def test_prefix_lm_all_flagged_equals_bidirectional_attention_output():
    """With every position flagged the decoder's self-attention mask is the encoder's (bidirectional) one, so the
    logits at position t depend on later inputs; with no flags they do not (teacher-forcing causality)."""
    cfg = tiny_cfg(arch=1, n_enc_layers=0, n_dec_layers=1)
    params = WL.make_params(O.param_shapes(cfg), 2, stddev=0.3)
    rng = np.random.default_rng(1)
    dec = rng.integers(1, cfg.vocab, size=(1, 8)).astype(np.int32)
    dec2 = dec.copy()
    dec2[0, 6] = (dec[0, 6] % (cfg.vocab - 1)) + 1            # changes decoder input 7 only
    none, allp = np.zeros((1, 8), dtype=np.int32), np.ones((1, 8), dtype=np.int32)
    a = O.t5_decode_logits(cfg, params, None, None, None, dec, None, dec_prefix=none)
    b = O.t5_decode_logits(cfg, params, None, None, None, dec2, None, dec_prefix=none)
    assert np.abs(a[0, :7] - b[0, :7]).max() == 0.0
    a = O.t5_decode_logits(cfg, params, None, None, None, dec, None, dec_prefix=allp)
    b = O.t5_decode_logits(cfg, params, None, None, None, dec2, None, dec_prefix=allp)
    assert np.abs(a[0, :7] - b[0, :7]).max() > 1e-6


# ------------------------------------------------------------------ optimizer step
def test_adamw_first_step_closed_form_and_quadratic_descent():
    """From zero moments the bias-corrected first step is lr (g / (|g| + eps) + wd theta) whatever the betas; on
    f(theta) = |theta - c|^2 / 2 the iterates approach c; weight decay alone shrinks theta geometrically."""
    rng = np.random.default_rng(0)
    th, g = rng.standard_normal(50), rng.standard_normal(50)
    t1, m1, v1 = O.adamw_update(th, np.zeros(50), np.zeros(50), g, 1, 1e-2, 0.8, 0.95, 1e-8, 0.1)
    assert np.abs(t1 - (th - 1e-2 * (g / (np.abs(g) + 1e-8) + 0.1 * th))).max() < 1e-12
    assert np.allclose(m1, 0.2 * g) and np.allclose(v1, 0.05 * g * g)
    c = rng.standard_normal(8)
    th, m, v = np.zeros(8), np.zeros(8), np.zeros(8)
    for t in range(1, 2001):
        th, m, v = O.adamw_update(th, m, v, th - c, t, 5e-3)
    assert np.abs(th - c).max() < 2e-2
    th = np.ones(4)
    for t in range(1, 11):
        th, _, _ = O.adamw_update(th, np.zeros(4), np.zeros(4), np.zeros(4), t, 0.1, weight_decay=0.5)
    assert np.allclose(th, 0.95 ** 10)
