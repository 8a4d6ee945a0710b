"""CPU oracle for one training step (forward + backward) of a T5.1.1-style Transformer.

TEST INFRASTRUCTURE ONLY.  This file is the slow, plain statement of what the
GPU library must compute.  Only the test-suite, the smoke check and the
benchmark's CPU-baseline leg may import it; the product path never does, and
this file imports nothing from the product.

What it follows: the paper's "Example Models" section names the models (T5,
T5.1.1 and a decoder-only configuration) and its "Model Implementation"
section says a model exposes a loss, an evaluation and an inference method.
The paper prints no equation for any of it, so every formula below is the
public T5.1.1 definition under the readings listed in the design notes
(scale-only RMSNorm, bias-free projections, bucketed relative-position bias
shared by the layers of a stack, tanh-GELU gated FFN, tied embedding with a
d_model^-1/2 logit scale, mean cross-entropy plus z-loss over non-pad
targets).

Style: numpy, one batch row at a time, one attention matrix per (row, head)
materialised in full, backward written out by hand with the chain rule.  A
matmul is the only library primitive used as a step.  `dtype` selects the
arithmetic (float64 for parity and finite differences, float32 for timing).

Weight convention here is the mathematical one: a projection is `y @ W` with
W of shape [in, out].

Pins (see tests/test_oracle_pins.py): bucket table against hand-derived
thresholds and an independent floating evaluation; tanh-GELU printed values;
softmax row sums / causal zeros / uniform rows; ln V + z ln^2 V closed form;
sum_v dlogits identity; central finite differences in float64 on every
parameter tensor; an independent autograd restatement; packing, padding and
row-permutation invariances; sum over buckets of the bias-table gradient = 0.
Parity unpinned TO THE PAPER for the convention choices the paper does not
print (attention scale 1, logit scale, tanh GELU, eps, mean normalisation):
they are pinned by the benchmark spec and public convention only.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field

import numpy as np


@dataclass
class T5Config:
    arch: int = 0                 # 0 encoder-decoder, 1 decoder-only
    n_enc_layers: int = 2
    n_dec_layers: int = 2
    d_model: int = 128
    n_heads: int = 4
    d_kv: int = 32
    d_ff: int = 256
    vocab: int = 512
    rel_buckets: int = 32
    rel_max_distance: int = 128
    z_loss: float = 1e-4
    rms_eps: float = 1e-6
    attn_scale: float = 1.0
    logit_scale: float = field(default=-1.0)   # <0 -> d_model ** -0.5
    operand_bf16: bool = False    # round BOTH operands of every matrix product to bfloat16 first
                                  # (the "bf16 operands, float32 accumulate" precision the larger
                                  # workloads are stated in); everything else stays in `dtype`
    # Members of the model family the paper's "Example Models" section lists beside T5.1.1:
    ffn_act: str = "gated-gelu-tanh"   # "gated-gelu-tanh" (default): (gelu_tanh(y Wi0) * (y Wi1)) Wo;
                                       # "gated-gelu-erf": the same with the exact (erf) GELU;
                                       # "relu": T5 v1.0's FFN, relu(y Wi0) Wo, no gate and no Wi1
    tied_embedding: bool = True        # False: the logits use a separate matrix "lm_head" [d, V]
                                       # (released T5.1.1) and logit_scale defaults to 1

    def __post_init__(self):
        if self.logit_scale < 0:
            self.logit_scale = float(self.d_model) ** -0.5 if self.tied_embedding else 1.0
        if self.ffn_act not in ("gated-gelu-tanh", "gated-gelu-erf", "relu"):
            raise ValueError(f"unknown ffn_act {self.ffn_act!r}")

    @property
    def inner(self):
        return self.n_heads * self.d_kv


# ----------------------------------------------------------------------------
# Relative-position bucket: closed form evaluated in exact integer arithmetic.
# ----------------------------------------------------------------------------
def relative_position_bucket(rel: int, bidirectional: bool, num_buckets: int = 32,
                             max_distance: int = 128) -> int:
    """Bucket of the signed distance rel = key_position - query_position.

    Bidirectional (encoder): half the buckets per sign; positive distances use
    the upper half.  Unidirectional (decoder): only keys at or before the
    query get distinct buckets, n = max(-rel, 0).  The first half of the
    available buckets is exact (bucket = n); beyond that the bucket index is
    me + floor(log(n/me) / log(max_distance/me) * (nb - me)), capped at nb-1.
    The floor of the logarithm ratio is taken exactly: the largest q with
    (max_distance/me)^q <= (n/me)^(nb-me), compared as integers.
    """
    nb = num_buckets
    offset = 0
    if bidirectional:
        nb //= 2
        if rel > 0:
            offset = nb
        n = abs(rel)
    else:
        n = max(-rel, 0)
    me = nb // 2
    if n < me:
        return offset + n
    p = nb - me
    q = 0
    # (n/me)^p >= (MD/me)^(q+1)   <=>   n^p * me^(q+1) >= MD^(q+1) * me^p
    while q < nb and (n ** p) * (me ** (q + 1)) >= (max_distance ** (q + 1)) * (me ** p):
        q += 1
    return offset + min(nb - 1, me + q)


def bucket_matrix(tq: int, tk: int, bidirectional: bool, num_buckets: int,
                  max_distance: int) -> np.ndarray:
    """[tq, tk] int32 matrix of bucket(j - i)."""
    lut = {}
    out = np.empty((tq, tk), dtype=np.int32)
    for i in range(tq):
        for j in range(tk):
            r = j - i
            if r not in lut:
                lut[r] = relative_position_bucket(r, bidirectional, num_buckets, max_distance)
            out[i, j] = lut[r]
    return out


# ----------------------------------------------------------------------------
# Matrix product with optional bfloat16 operand rounding
# ----------------------------------------------------------------------------
def round_bf16(a):
    """Nearest bfloat16 (ties to even) of each element, returned in a's dtype."""
    f = np.ascontiguousarray(a, dtype=np.float32)
    u = f.view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    out = ((u + r) & np.uint32(0xFFFF0000)).astype(np.uint32).view(np.float32)
    return out.reshape(np.shape(a)).astype(np.asarray(a).dtype)


def mm(cfg, a, b):
    """a @ b; with cfg.operand_bf16 both operands are rounded to bfloat16 and the
    products are accumulated in the working precision."""
    if cfg.operand_bf16:
        return round_bf16(a) @ round_bf16(b)
    return a @ b


# ----------------------------------------------------------------------------
# Elementwise pieces
# ----------------------------------------------------------------------------
_GELU_C = math.sqrt(2.0 / math.pi)
_GELU_A = 0.044715


def gelu_tanh(u):
    """0.5 u (1 + tanh( sqrt(2/pi) (u + 0.044715 u^3) ))."""
    return 0.5 * u * (1.0 + np.tanh(_GELU_C * (u + _GELU_A * u ** 3)))


def gelu_tanh_grad(u):
    t = np.tanh(_GELU_C * (u + _GELU_A * u ** 3))
    dinner = _GELU_C * (1.0 + 3.0 * _GELU_A * u ** 2)
    return 0.5 * (1.0 + t) + 0.5 * u * (1.0 - t * t) * dinner


def gelu_erf(u):
    """u Phi(u) = 0.5 u (1 + erf(u / sqrt 2)), Phi the standard normal distribution function."""
    from scipy.special import erf
    return 0.5 * u * (1.0 + erf(u / math.sqrt(2.0)))


def gelu_erf_grad(u):
    """Phi(u) + u phi(u), phi the standard normal density."""
    from scipy.special import erf
    return 0.5 * (1.0 + erf(u / math.sqrt(2.0))) + u * np.exp(-0.5 * u * u) / math.sqrt(2.0 * math.pi)


def ffn_activation(cfg, a):
    """(act(a), act'(a)) of the configured FFN non-linearity."""
    if cfg.ffn_act == "relu":
        return np.maximum(a, 0), (a > 0).astype(a.dtype)
    if cfg.ffn_act == "gated-gelu-erf":
        return gelu_erf(a), gelu_erf_grad(a)
    return gelu_tanh(a), gelu_tanh_grad(a)


def rms_norm(x, g, eps):
    """y = x * (mean(x^2) + eps)^-1/2 * g ; returns (y, r)."""
    r = 1.0 / np.sqrt(np.mean(x * x, axis=-1) + x.dtype.type(eps))
    return x * r[:, None] * g[None, :], r


def rms_norm_bwd(dy, x, g, r):
    """Returns (dx, dg) for y = x * r * g."""
    dyg = dy * g[None, :]
    dg = np.sum(dy * x * r[:, None], axis=0)
    m = np.mean(dyg * x, axis=-1)
    dx = r[:, None] * dyg - x * (r ** 3)[:, None] * m[:, None]
    return dx, dg


def masked_softmax(s, mask):
    """Row softmax over entries with mask=True; masked entries are exactly 0;
    a row with no valid entry is all zeros."""
    neg = np.where(mask, s, -np.inf)
    mx = np.max(neg, axis=-1, keepdims=True)
    mx = np.where(np.isfinite(mx), mx, 0.0)
    e = np.where(mask, np.exp(neg - mx), 0.0)
    den = np.sum(e, axis=-1, keepdims=True)
    return np.where(den > 0, e / np.where(den > 0, den, 1.0), 0.0).astype(s.dtype)


# ----------------------------------------------------------------------------
# Input preparation
# ----------------------------------------------------------------------------
def position_codes(tokens_row, seg_row):
    """code = 0 for padding (token id 0), else the segment id (1 if unpacked).
    Query i may attend key j iff code_k[j] != 0 and code_q[i] == code_k[j]."""
    tok = np.asarray(tokens_row)
    if seg_row is None:
        return (tok != 0).astype(np.int32)
    return np.where(tok != 0, np.asarray(seg_row), 0).astype(np.int32)


def shift_right(targets_row, seg_row):
    """Decoder input u_t = target_{t-1} inside a segment, 0 at a row or segment start."""
    t = np.asarray(targets_row)
    u = np.zeros_like(t)
    for i in range(1, len(t)):
        if seg_row is None or seg_row[i] == seg_row[i - 1]:
            u[i] = t[i - 1]
    return u


def attention_mask(code_q, code_k, causal, prefix_q=None, prefix_k=None):
    """Query i may attend key j iff both carry the same non-zero code and, when causal, j <= i.
    Prefix LM: positions flagged in prefix_* form a fully visible prefix, so a causal pair is also
    allowed when query and key are both flagged."""
    m = (code_k[None, :] != 0) & (code_q[:, None] == code_k[None, :])
    if causal:
        tq, tk = m.shape
        allowed = np.arange(tk)[None, :] <= np.arange(tq)[:, None]
        if prefix_q is not None:
            allowed = allowed | ((np.asarray(prefix_q)[:, None] != 0) & (np.asarray(prefix_k)[None, :] != 0))
        m &= allowed
    return m


def loss_weights(targets_row, prefix_row=None):
    """w_t = 1 for a non-pad target outside the prefix (the prefix is given, not predicted), else 0."""
    w = np.asarray(targets_row) != 0
    if prefix_row is not None:
        w = w & (np.asarray(prefix_row) == 0)
    return w


# ----------------------------------------------------------------------------
# Parameter inventory (oracle naming; shapes in the [in, out] convention)
# ----------------------------------------------------------------------------
def param_shapes(cfg: T5Config):
    d, I, F, V, H, NB = cfg.d_model, cfg.inner, cfg.d_ff, cfg.vocab, cfg.n_heads, cfg.rel_buckets
    s = {"token_embed": (V, d)}

    def attn(prefix):
        s[prefix + ".norm"] = (d,)
        s[prefix + ".q"] = (d, I)
        s[prefix + ".k"] = (d, I)
        s[prefix + ".v"] = (d, I)
        s[prefix + ".o"] = (I, d)

    def ffn(prefix):
        s[prefix + ".norm"] = (d,)
        s[prefix + ".wi0"] = (d, F)
        if cfg.ffn_act != "relu":
            s[prefix + ".wi1"] = (d, F)
        s[prefix + ".wo"] = (F, d)

    if cfg.arch == 0:
        s["enc.relbias"] = (NB, H)
        for l in range(cfg.n_enc_layers):
            attn(f"enc.L{l}.attn")
            ffn(f"enc.L{l}.ffn")
        s["enc.final_norm"] = (d,)
    s["dec.relbias"] = (NB, H)
    for l in range(cfg.n_dec_layers):
        attn(f"dec.L{l}.self")
        if cfg.arch == 0:
            attn(f"dec.L{l}.cross")
        ffn(f"dec.L{l}.ffn")
    s["dec.final_norm"] = (d,)
    if not cfg.tied_embedding:
        s["lm_head"] = (d, V)
    return s


# ----------------------------------------------------------------------------
# Sub-layers, one batch row at a time.  Each forward returns (output, cache).
# ----------------------------------------------------------------------------
def _attn_fwd(cfg, p, prefix, x_q, y_kv, table, bidirectional, code_q, code_k, causal, lm_prefix=None):
    """x_q: residual stream [Tq, d].  y_kv: None for self-attention (keys and
    values come from the normed x_q) or the already-normed encoder output.
    lm_prefix: flags of the fully visible prefix of a prefix LM (causal self-attention only)."""
    H, k = cfg.n_heads, cfg.d_kv
    dt = x_q.dtype
    yq, r = rms_norm(x_q, p[prefix + ".norm"], cfg.rms_eps)
    ykv = yq if y_kv is None else y_kv
    Q = mm(cfg, yq, p[prefix + ".q"])
    K = mm(cfg, ykv, p[prefix + ".k"])
    Vv = mm(cfg, ykv, p[prefix + ".v"])
    tq, tk = Q.shape[0], K.shape[0]
    mask = attention_mask(code_q, code_k, causal, lm_prefix, lm_prefix)
    bk = None
    if table is not None:
        bk = bucket_matrix(tq, tk, bidirectional, cfg.rel_buckets, cfg.rel_max_distance)
    P = np.zeros((H, tq, tk), dtype=dt)
    C = np.zeros((tq, H * k), dtype=dt)
    for h in range(H):
        sl = slice(h * k, (h + 1) * k)
        S = dt.type(cfg.attn_scale) * mm(cfg, Q[:, sl], K[:, sl].T)
        if table is not None:
            S = S + table[bk, h]
        P[h] = masked_softmax(S, mask)
        C[:, sl] = mm(cfg, P[h], Vv[:, sl])
    out = x_q + mm(cfg, C, p[prefix + ".o"])
    cache = dict(x=x_q, r=r, yq=yq, ykv=ykv, Q=Q, K=K, V=Vv, P=P, C=C, bk=bk,
                 self_attn=(y_kv is None))
    return out, cache


def _attn_bwd(cfg, p, g, gtable, prefix, dout, c):
    """dout: gradient wrt the sub-layer output.  Accumulates parameter grads
    into g (and the bias-table gradient into gtable); returns (dx_q, dy_kv)
    where dy_kv is None for self-attention."""
    H, k = cfg.n_heads, cfg.d_kv
    dt = dout.dtype
    s = dt.type(cfg.attn_scale)
    g[prefix + ".o"] += mm(cfg, c["C"].T, dout)
    dC = mm(cfg, dout, p[prefix + ".o"].T)
    dQ = np.zeros_like(c["Q"])
    dK = np.zeros_like(c["K"])
    dV = np.zeros_like(c["V"])
    for h in range(H):
        sl = slice(h * k, (h + 1) * k)
        P = c["P"][h]
        dP = mm(cfg, dC[:, sl], c["V"][:, sl].T)
        dV[:, sl] = mm(cfg, P.T, dC[:, sl])
        dS = P * (dP - np.sum(dP * P, axis=-1, keepdims=True))
        if gtable is not None:
            np.add.at(gtable[:, h], c["bk"].ravel(), dS.ravel())
        dQ[:, sl] = s * mm(cfg, dS, c["K"][:, sl])
        dK[:, sl] = s * mm(cfg, dS.T, c["Q"][:, sl])
    g[prefix + ".q"] += mm(cfg, c["yq"].T, dQ)
    g[prefix + ".k"] += mm(cfg, c["ykv"].T, dK)
    g[prefix + ".v"] += mm(cfg, c["ykv"].T, dV)
    dyq = mm(cfg, dQ, p[prefix + ".q"].T)
    dykv = mm(cfg, dK, p[prefix + ".k"].T) + mm(cfg, dV, p[prefix + ".v"].T)
    if c["self_attn"]:
        dyq = dyq + dykv
        dykv = None
    dxn, dg = rms_norm_bwd(dyq, c["x"], p[prefix + ".norm"], c["r"])
    g[prefix + ".norm"] += dg
    return dout + dxn, dykv


def _ffn_fwd(cfg, p, prefix, x):
    y, r = rms_norm(x, p[prefix + ".norm"], cfg.rms_eps)
    a = mm(cfg, y, p[prefix + ".wi0"])
    act, _ = ffn_activation(cfg, a)
    if cfg.ffn_act == "relu":            # T5 v1.0: no gate
        b, hg = None, act
    else:
        b = mm(cfg, y, p[prefix + ".wi1"])
        hg = act * b
    out = x + mm(cfg, hg, p[prefix + ".wo"])
    return out, dict(x=x, r=r, y=y, a=a, b=b, hg=hg)


def _ffn_bwd(cfg, p, g, prefix, dout, c):
    g[prefix + ".wo"] += mm(cfg, c["hg"].T, dout)
    dhg = mm(cfg, dout, p[prefix + ".wo"].T)
    act, dact = ffn_activation(cfg, c["a"])
    if cfg.ffn_act == "relu":
        da = dhg * dact
        g[prefix + ".wi0"] += mm(cfg, c["y"].T, da)
        dy = mm(cfg, da, p[prefix + ".wi0"].T)
    else:
        da = dhg * c["b"] * dact
        db = dhg * act
        g[prefix + ".wi0"] += mm(cfg, c["y"].T, da)
        g[prefix + ".wi1"] += mm(cfg, c["y"].T, db)
        dy = mm(cfg, da, p[prefix + ".wi0"].T) + mm(cfg, db, p[prefix + ".wi1"].T)
    dxn, dg = rms_norm_bwd(dy, c["x"], p[prefix + ".norm"], c["r"])
    g[prefix + ".norm"] += dg
    return dout + dxn


def _encoder_fwd(cfg, p, tokens_row, seg_row):
    code = position_codes(tokens_row, seg_row)
    x = p["token_embed"][np.asarray(tokens_row)]
    caches = []
    for l in range(cfg.n_enc_layers):
        x, ca = _attn_fwd(cfg, p, f"enc.L{l}.attn", x, None, p["enc.relbias"], True, code, code, False)
        x, cf = _ffn_fwd(cfg, p, f"enc.L{l}.ffn", x)
        caches.append((ca, cf))
    y, r = rms_norm(x, p["enc.final_norm"], cfg.rms_eps)
    return y, dict(code=code, layers=caches, x_final=x, r_final=r, tokens=np.asarray(tokens_row))


def _encoder_bwd(cfg, p, g, dy, c):
    dx, dg = rms_norm_bwd(dy, c["x_final"], p["enc.final_norm"], c["r_final"])
    g["enc.final_norm"] += dg
    for l in reversed(range(cfg.n_enc_layers)):
        ca, cf = c["layers"][l]
        dx = _ffn_bwd(cfg, p, g, f"enc.L{l}.ffn", dx, cf)
        dx, _ = _attn_bwd(cfg, p, g, g["enc.relbias"], f"enc.L{l}.attn", dx, ca)
    np.add.at(g["token_embed"], c["tokens"], dx)


def _out_embedding(cfg, p):
    """[V, d] matrix of the logits: the input embedding when tied, else the separate head (stored [d, V])."""
    return p["token_embed"] if cfg.tied_embedding else p["lm_head"].T


def _decoder_fwd(cfg, p, targets_row, dseg_row, enc_y, enc_code, lm_prefix=None):
    code = position_codes(targets_row, dseg_row)
    u = shift_right(targets_row, dseg_row)
    x = p["token_embed"][u]
    caches = []
    for l in range(cfg.n_dec_layers):
        x, cs = _attn_fwd(cfg, p, f"dec.L{l}.self", x, None, p["dec.relbias"], False, code, code, True, lm_prefix)
        cc = None
        if cfg.arch == 0:
            x, cc = _attn_fwd(cfg, p, f"dec.L{l}.cross", x, enc_y, None, False, code, enc_code, False)
        x, cf = _ffn_fwd(cfg, p, f"dec.L{l}.ffn", x)
        caches.append((cs, cc, cf))
    z, r = rms_norm(x, p["dec.final_norm"], cfg.rms_eps)
    logits = x.dtype.type(cfg.logit_scale) * mm(cfg, z, _out_embedding(cfg, p).T)
    return logits, dict(u=u, layers=caches, x_final=x, r_final=r, z=z)


def _decoder_bwd(cfg, p, g, dlogits, c, enc_y):
    dt = dlogits.dtype
    ls = dt.type(cfg.logit_scale)
    if cfg.tied_embedding:
        g["token_embed"] += ls * mm(cfg, dlogits.T, c["z"])
    else:
        g["lm_head"] += ls * mm(cfg, c["z"].T, dlogits)
    dz = ls * mm(cfg, dlogits, _out_embedding(cfg, p))
    dx, dg = rms_norm_bwd(dz, c["x_final"], p["dec.final_norm"], c["r_final"])
    g["dec.final_norm"] += dg
    denc = None if enc_y is None else np.zeros_like(enc_y)
    for l in reversed(range(cfg.n_dec_layers)):
        cs, cc, cf = c["layers"][l]
        dx = _ffn_bwd(cfg, p, g, f"dec.L{l}.ffn", dx, cf)
        if cc is not None:
            dx, dkv = _attn_bwd(cfg, p, g, None, f"dec.L{l}.cross", dx, cc)
            denc += dkv
        dx, _ = _attn_bwd(cfg, p, g, g["dec.relbias"], f"dec.L{l}.self", dx, cs)
    np.add.at(g["token_embed"], c["u"], dx)
    return denc


def xent_zloss_row(logits, targets_row, weights_row, z):
    """Per position: lse = log sum_v exp(logit); returns (ce_t, zl_t, lse_t, p)
    with ce_t = lse - logit[target], zl_t = z lse^2 (unweighted)."""
    mx = np.max(logits, axis=-1, keepdims=True)
    e = np.exp(logits - mx)
    se = np.sum(e, axis=-1, keepdims=True)
    lse = (np.log(se) + mx)[:, 0]
    prob = e / se
    tl = logits[np.arange(logits.shape[0]), np.asarray(targets_row)]
    return lse - tl, logits.dtype.type(z) * lse * lse, lse, prob


# ----------------------------------------------------------------------------
# Public entry points
# ----------------------------------------------------------------------------
def _cast_params(params, dtype):
    return {k: np.asarray(v, dtype=dtype) for k, v in params.items()}


def t5_train_step(cfg: T5Config, params, enc_tokens, enc_segment_ids, dec_targets,
                  dec_segment_ids, dtype=np.float64, return_aux=False, dec_prefix=None):
    """Loss and gradients of one batch.

    dec_prefix ([B, Td] 0/1, optional): prefix-LM flags of the decoder positions - flagged positions see each
    other in full (inside their segment), the rest stay causal, and flagged positions carry no loss.

    Returns (loss4, grads): loss4 = [L, ce, zl, W] with
      W  = number of non-pad targets,
      ce = (1/W) sum_t w_t (lse_t - logit_t[target_t]),
      zl = (1/W) sum_t w_t z lse_t^2,  L = ce + zl   (all zero when W = 0),
    grads = dict of dL/dtheta in the shapes of param_shapes(cfg).
    """
    dtype = np.dtype(dtype)
    p = _cast_params(params, dtype)
    g = {k: np.zeros(v.shape, dtype=dtype) for k, v in p.items()}
    dec_targets = np.asarray(dec_targets)
    B = dec_targets.shape[0]
    dec_prefix = None if dec_prefix is None else np.asarray(dec_prefix)
    W = int(np.sum(loss_weights(dec_targets, dec_prefix)))
    ce_sum = 0.0
    zl_sum = 0.0
    aux = dict(enc_out=[], logits=[], dlogits=[])
    for b in range(B):
        eseg = None if enc_segment_ids is None else np.asarray(enc_segment_ids)[b]
        dseg = None if dec_segment_ids is None else np.asarray(dec_segment_ids)[b]
        if cfg.arch == 0:
            enc_y, ec = _encoder_fwd(cfg, p, np.asarray(enc_tokens)[b], eseg)
            enc_code = ec["code"]
        else:
            enc_y, ec, enc_code = None, None, None
        pre = None if dec_prefix is None else dec_prefix[b]
        logits, dc = _decoder_fwd(cfg, p, dec_targets[b], dseg, enc_y, enc_code, pre)
        w = loss_weights(dec_targets[b], pre).astype(dtype)
        ce_t, zl_t, lse, prob = xent_zloss_row(logits, dec_targets[b], w, cfg.z_loss)
        ce_sum += float(np.sum(w * ce_t))
        zl_sum += float(np.sum(w * zl_t))
        if return_aux:
            aux["enc_out"].append(enc_y)
            aux["logits"].append(logits)
        if W == 0:
            continue
        # dL/dlogits = (w/W) (p (1 + 2 z lse) - onehot(target))
        dlogits = prob * (1.0 + 2.0 * dtype.type(cfg.z_loss) * lse)[:, None]
        dlogits[np.arange(len(lse)), dec_targets[b]] -= 1.0
        dlogits *= (w / dtype.type(W))[:, None]
        if return_aux:
            aux["dlogits"].append(dlogits)
        denc = _decoder_bwd(cfg, p, g, dlogits, dc, enc_y)
        if cfg.arch == 0:
            _encoder_bwd(cfg, p, g, denc, ec)
    if W == 0:
        loss4 = np.zeros(4, dtype=np.float64)
    else:
        loss4 = np.array([(ce_sum + zl_sum) / W, ce_sum / W, zl_sum / W, W], dtype=np.float64)
    if return_aux:
        return loss4, g, aux
    return loss4, g


def t5_loss_only(cfg, params, enc_tokens, enc_segment_ids, dec_targets, dec_segment_ids,
                 dtype=np.float64, dec_prefix=None):
    """Forward only: the scalar L (used by finite differences)."""
    dtype = np.dtype(dtype)
    p = _cast_params(params, dtype)
    dec_targets = np.asarray(dec_targets)
    dec_prefix = None if dec_prefix is None else np.asarray(dec_prefix)
    W = int(np.sum(loss_weights(dec_targets, dec_prefix)))
    if W == 0:
        return 0.0
    tot = 0.0
    for b in range(dec_targets.shape[0]):
        eseg = None if enc_segment_ids is None else np.asarray(enc_segment_ids)[b]
        dseg = None if dec_segment_ids is None else np.asarray(dec_segment_ids)[b]
        enc_y, enc_code = None, None
        if cfg.arch == 0:
            enc_y, ec = _encoder_fwd(cfg, p, np.asarray(enc_tokens)[b], eseg)
            enc_code = ec["code"]
        pre = None if dec_prefix is None else dec_prefix[b]
        logits, _ = _decoder_fwd(cfg, p, dec_targets[b], dseg, enc_y, enc_code, pre)
        w = loss_weights(dec_targets[b], pre).astype(dtype)
        ce_t, zl_t, _, _ = xent_zloss_row(logits, dec_targets[b], w, cfg.z_loss)
        tot += float(np.sum(w * (ce_t + zl_t)))
    return tot / W


def t5_encode(cfg, params, enc_tokens, enc_segment_ids, dtype=np.float64):
    """Encoder output after the final norm, [B, Te, d]."""
    p = _cast_params(params, np.dtype(dtype))
    outs = []
    for b in range(np.asarray(enc_tokens).shape[0]):
        eseg = None if enc_segment_ids is None else np.asarray(enc_segment_ids)[b]
        y, _ = _encoder_fwd(cfg, p, np.asarray(enc_tokens)[b], eseg)
        outs.append(y)
    return np.stack(outs)


def t5_decode_logits(cfg, params, enc_out, enc_tokens, enc_segment_ids, dec_targets,
                     dec_segment_ids, dtype=np.float64, dec_prefix=None):
    """Teacher-forced decoder logits [B, Td, V] given the encoder output
    (enc_out is ignored for the decoder-only architecture)."""
    dtype = np.dtype(dtype)
    p = _cast_params(params, dtype)
    outs = []
    dec_targets = np.asarray(dec_targets)
    for b in range(dec_targets.shape[0]):
        dseg = None if dec_segment_ids is None else np.asarray(dec_segment_ids)[b]
        ey, ecode = None, None
        if cfg.arch == 0:
            eseg = None if enc_segment_ids is None else np.asarray(enc_segment_ids)[b]
            ey = np.asarray(enc_out[b], dtype=dtype)
            ecode = position_codes(np.asarray(enc_tokens)[b], eseg)
        pre = None if dec_prefix is None else np.asarray(dec_prefix)[b]
        logits, _ = _decoder_fwd(cfg, p, dec_targets[b], dseg, ey, ecode, pre)
        outs.append(logits)
    return np.stack(outs)


# ----------------------------------------------------------------------------
# Optimizer step (the training loop of the paper's "Overall structure" section continues past the gradients;
# the paper prints no update rule - this is the public AdamW definition with decoupled weight decay).
# ----------------------------------------------------------------------------
def adamw_update(theta, m, v, g, step, lr, beta1=0.9, beta2=0.999, eps=1e-8, weight_decay=0.0, grad_scale=1.0):
    """One AdamW step on arrays of equal shape; returns (theta, m, v) after it.
      g' = grad_scale g;  m = b1 m + (1 - b1) g';  v = b2 v + (1 - b2) g'^2;
      theta = theta - lr ( (m / (1 - b1^t)) / (sqrt(v / (1 - b2^t)) + eps) + weight_decay theta ),  t = step >= 1."""
    theta, m, v, g = (np.asarray(a, dtype=np.float64) for a in (theta, m, v, g))
    g = grad_scale * g
    m = beta1 * m + (1.0 - beta1) * g
    v = beta2 * v + (1.0 - beta2) * g * g
    mhat = m / (1.0 - beta1 ** step)
    vhat = v / (1.0 - beta2 ** step)
    theta = theta - lr * (mhat / (np.sqrt(vhat) + eps) + weight_decay * theta)
    return theta, m, v
