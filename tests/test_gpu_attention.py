"""Attention kernels (SIMT and tcgen05) through the C ABI against the oracle's
attention arithmetic on the same seeded inputs."""
import numpy as np
import pytest
import torch

from oracle import t5_oracle as O
from paper_2203_17189_b200 import binding as Bd
from paper_2203_17189_b200 import workloads as WL

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def make_codes(rng, B, T, mode):
    """mode: 'full', 'pad' (trailing padding) or 'packed' (segments + padded tail)."""
    c = np.ones((B, T), dtype=np.int32)
    for b in range(B):
        if mode == "pad":
            n = int(rng.integers(max(1, T // 2), T + 1))
            c[b, n:] = 0
        elif mode == "packed":
            pos, sid = 0, 1
            while pos < T:
                n = int(rng.integers(max(2, T // 8), max(3, T // 2)))
                c[b, pos:pos + n] = sid
                pos += n
                sid += 1
            c[b, T - int(rng.integers(0, max(1, T // 6))):] = 0
    return c


def make_cross_codes(rng, B, Tq, Tk, mode):
    """Packed rows with different query and key lengths (cross-attention of packed examples): the same
    examples, in the same order, on both sides, each side with its own lengths.
    'xpacked': ids 1.. in order;  'xmiss0': the queries hold only the later examples, so the first key tiles
    contain no key any query row may attend;  'xnonmono': example ids are not increasing along the row."""
    cq = np.zeros((B, Tq), dtype=np.int32)
    ck = np.zeros((B, Tk), dtype=np.int32)
    for b in range(B):
        n = int(rng.integers(3, 6))
        ids = np.arange(1, n + 1)
        if mode == "xnonmono":
            ids = rng.permutation(ids) + int(rng.integers(0, 3))

        def cut(T, frac_used):
            edges = np.sort(rng.choice(np.arange(1, int(T * frac_used)), size=n - 1, replace=False))
            return np.concatenate([[0], edges, [int(T * frac_used)]])
        ek, eq = cut(Tk, 0.93), cut(Tq, 0.9)
        for s in range(n):
            ck[b, ek[s]:ek[s + 1]] = ids[s]
        if mode == "xmiss0":
            # queries: only the last two examples, spread over the whole used part of the row
            half = eq[-1] // 2
            cq[b, :half] = ids[n - 2]
            cq[b, half:eq[-1]] = ids[n - 1]
        else:
            for s in range(n):
                cq[b, eq[s]:eq[s + 1]] = ids[s]
    return cq, ck


def reference(q, k, v, do, code_q, code_k, bias_delta, causal, scale, H, dk):
    """Oracle arithmetic per (b, h): masked softmax attention and its gradients (float64)."""
    B, Tq = code_q.shape
    Tk = code_k.shape[1]
    out = np.zeros_like(q)
    lse = np.zeros((B, H, Tq))
    dq, dk_, dv = np.zeros_like(q), np.zeros_like(k), np.zeros_like(v)
    dbias = np.zeros((H, Tq + Tk - 1))
    idx = np.arange(Tk)[None, :] - np.arange(Tq)[:, None] + Tq - 1
    for b in range(B):
        mask = O.attention_mask(code_q[b], code_k[b], causal)
        for h in range(H):
            sl = slice(h * dk, (h + 1) * dk)
            Q, K, V, dO = q[b, :, sl], k[b, :, sl], v[b, :, sl], do[b, :, sl]
            S = scale * (Q @ K.T)
            if bias_delta is not None:
                S = S + bias_delta[h][idx]
            P = O.masked_softmax(S, mask)
            out[b, :, sl] = P @ V
            with np.errstate(divide="ignore"):
                mx = np.where(mask, S, -np.inf).max(-1)
                lse[b, h] = np.where(np.isfinite(mx), np.log(np.where(mask, np.exp(S - np.where(np.isfinite(mx), mx, 0)[:, None]), 0).sum(-1)) + mx, -np.inf)
            dP = dO @ V.T
            dv[b, :, sl] = P.T @ dO
            dS = P * (dP - (dP * P).sum(-1, keepdims=True))
            dq[b, :, sl] = scale * (dS @ K)
            dk_[b, :, sl] = scale * (dS.T @ Q)
            np.add.at(dbias[h], idx.ravel(), dS.ravel())
    return out, lse, dq, dk_, dv, dbias


CASES = [
    # B, H, Tq, Tk, dk, causal, bias, mode
    (2, 3, 128, 128, 64, False, True, "full"),
    (2, 2, 200, 200, 64, True, True, "pad"),
    (3, 2, 114, 512, 64, False, False, "pad"),
    (2, 2, 75, 75, 64, False, True, "pad"),
    (1, 2, 300, 300, 128, True, True, "packed"),
    (2, 1, 512, 512, 64, False, True, "packed"),
    (1, 2, 130, 70, 128, False, False, "full"),
]


# impl 2: tcgen05 forward, then the one-pass backward entry point (dS goes through a scratch buffer)
@pytest.mark.parametrize("impl", [0, 1, 2])
@pytest.mark.parametrize("B,H,Tq,Tk,dk,causal,use_bias,mode", CASES + [
    (1, 2, 640, 640, 64, True, True, "packed"),
    (2, 2, 50, 330, 64, False, True, "pad"),
    # degenerate extents: one query, one key
    (1, 1, 1, 40, 64, False, True, "full"),
    (1, 2, 129, 1, 64, False, False, "full"),
    # large scores (scale 1): row maxima move by more than the forward kernel's lazy-rescale threshold between tiles
    (1, 2, 448, 448, 64, False, True, "full_hot"),
    # packed rows with different query / key lengths and several examples on both sides
    (3, 2, 114, 512, 64, False, False, "xpacked"),
    (2, 2, 114, 512, 64, False, False, "xmiss0"),
    (2, 2, 300, 700, 64, False, True, "xnonmono"),
    (1, 2, 260, 520, 128, False, False, "xmiss0"),
])
def test_attention_forward_backward(impl, B, H, Tq, Tk, dk, causal, use_bias, mode):
    rng = np.random.default_rng(B * 1000 + Tq + Tk + dk)
    I = H * dk
    hot = mode.endswith("_hot")
    mode = mode[:-4] if hot else mode
    bf = torch.bfloat16

    def rnd(*shape, s=1.0):
        return torch.from_numpy((rng.standard_normal(shape) * s).astype(np.float32)).to(DEV).to(bf)
    # q, k, v live as column slices of one wide buffer when Tq == Tk (the fused projection layout)
    if Tq == Tk:
        qkv = rnd(B * Tq, 3 * I, s=0.7)
        q, k, v = qkv[:, :I], qkv[:, I:2 * I], qkv[:, 2 * I:]
    else:
        q = rnd(B * Tq, I, s=0.7)
        kv = rnd(B * Tk, 2 * I, s=0.7)
        k, v = kv[:, :I], kv[:, I:]
    do = rnd(B * Tq, I)
    if mode.startswith("x"):
        code_q, code_k = make_cross_codes(rng, B, Tq, Tk, mode)
    else:
        code_k = make_codes(rng, B, Tk, mode)
        code_q = code_k if Tq == Tk else make_codes(rng, B, Tq, "pad" if mode != "full" else "full")
        if mode == "packed" and Tq != Tk:
            code_q = np.minimum(code_q, 1)
    bias = (rng.standard_normal((H, Tq + Tk - 1)) * 0.5).astype(np.float32) if use_bias else None
    scale = 1.0 if hot else (0.25 if dk == 64 else 0.2)
    # one-pass backward with a saturated bias: constant beyond +-far, whose dS mass is then booked at +-far
    far = 48 if (impl == 2 and use_bias and Tq >= 200) else 0
    if far:
        c = Tq - 1
        bias[:, c + far:] = bias[:, c + far:c + far + 1]
        bias[:, :c - far] = bias[:, c - far:c - far + 1]

    o = torch.full((B * Tq, I), float("nan"), dtype=bf, device=DEV)
    lse = torch.empty(B, H, Tq, dtype=torch.float32, device=DEV)
    dq = torch.full((B * Tq, I), float("nan"), dtype=bf, device=DEV)
    dkv = torch.full((B * Tk, 2 * I), float("nan"), dtype=bf, device=DEV)
    dk_t, dv_t = dkv[:, :I], dkv[:, I:]
    delta = torch.empty(B, H, Tq, dtype=torch.float32, device=DEV)
    dbias = torch.zeros(H, Tq + Tk - 1, dtype=torch.float32, device=DEV) if use_bias else None
    cq_d = torch.from_numpy(code_q).to(DEV)
    ck_d = torch.from_numpy(code_k).to(DEV)
    bias_d = None if bias is None else torch.from_numpy(bias).to(DEV)
    o32 = torch.full((B * Tq, I), float("nan"), dtype=torch.float32, device=DEV) if B != 3 else None
    Bd.t5_attention(min(impl, 1), False, B, H, Tq, Tk, dk, causal, scale, q, k, v, o, lse, cq_d, ck_d, bias_d, o32=o32)
    if impl == 2:
        nbytes = Bd.t5_attention_ds_scratch_bytes(B, H, Tq, Tk)
        scratch = torch.full((nbytes // 2,), float("nan"), dtype=bf, device=DEV)
        Bd.t5_attention_backward_onepass(B, H, Tq, Tk, dk, causal, scale, q, k, v, o, o32, lse, cq_d, ck_d, bias_d,
                                         do, dq, dk_t, dv_t, delta, dbias, far, scratch)
    else:
        Bd.t5_attention(impl, True, B, H, Tq, Tk, dk, causal, scale, q, k, v, o, lse, cq_d, ck_d, bias_d,
                        do=do, dq=dq, dk=dk_t, dv=dv_t, delta=delta, dbias_delta=dbias, o32=o32)
    torch.cuda.synchronize()

    f64 = lambda t, T: t.float().cpu().numpy().astype(np.float64).reshape(B, T, I)
    ro, rlse, rdq, rdk, rdv, rdb = reference(f64(q, Tq), f64(k, Tk), f64(v, Tk), f64(do, Tq), code_q, code_k,
                                             None if bias is None else bias.astype(np.float64), causal, scale, H, dk)
    qvalid = (code_q != 0)
    got_o = f64(o, Tq)
    assert np.isfinite(got_o[qvalid]).all()
    assert np.abs(got_o - ro)[qvalid].max() <= 1.5e-2 * np.abs(ro).max()
    got_lse = lse.cpu().numpy().transpose(0, 2, 1)           # [B,Tq,H]
    ref_lse = rlse.transpose(0, 2, 1)
    fin = np.isfinite(ref_lse)
    assert np.array_equal(np.isfinite(got_lse), fin)
    assert np.abs(got_lse[fin] - ref_lse[fin]).max() <= 2e-2
    for name, got, ref, T in (("dq", dq, rdq, Tq), ("dk", dk_t, rdk, Tk), ("dv", dv_t, rdv, Tk)):
        g = f64(got, T)
        assert np.isfinite(g).all(), name
        # with a single key the softmax is the constant 1 and dS, dq, dk are identically zero in exact arithmetic:
        # what the kernels leave there is the float32 rounding residue of dP - delta, far below the inputs' scale
        floor = 1e-4 if Tk == 1 else 0.0
        assert np.abs(g - ref).max() <= 2e-2 * np.abs(ref).max() + floor, (name, np.abs(g - ref).max(), np.abs(ref).max())
    if use_bias:
        g = dbias.cpu().numpy()
        if far:
            c = Tq - 1
            # blocks wholly beyond +-far are booked at +-far, straddling blocks at each distance: compare folded
            for a in (rdb, g):
                a[:, c + far] = a[:, c + far:].sum(axis=1)
                a[:, c + far + 1:] = 0
                a[:, c - far] = a[:, :c - far + 1].sum(axis=1)
                a[:, :c - far] = 0
        assert np.abs(g - rdb).max() <= 2e-2 * np.abs(rdb).max()


def test_onepass_backward_rejects_bad_scratch():
    """The one-pass backward refuses a scratch buffer that is too small or a head width it does not cover,
    before anything is launched."""
    B, H, Tq, Tk, dk = 1, 2, 128, 128, 64
    I = H * dk
    bf = torch.bfloat16
    t = torch.zeros(B * Tq, I, dtype=bf, device=DEV)
    f32 = torch.zeros(B * Tq, I, dtype=torch.float32, device=DEV)
    lse = torch.zeros(B, H, Tq, dtype=torch.float32, device=DEV)
    codes = torch.ones(B, Tq, dtype=torch.int32, device=DEV)
    need = Bd.t5_attention_ds_scratch_bytes(B, H, Tq, Tk)
    assert need == B * H * 128 * 128 * 2
    small = torch.zeros(need // 2 - 64, dtype=bf, device=DEV)
    with pytest.raises(Bd.T5Error):
        Bd.t5_attention_backward_onepass(B, H, Tq, Tk, dk, False, 1.0, t, t, t, t, f32, lse, codes, codes, None,
                                         t, t, t, t, lse, None, 0, small)
    ok = torch.zeros(need // 2, dtype=bf, device=DEV)
    with pytest.raises(Bd.T5Error):
        Bd.t5_attention_backward_onepass(B, H, Tq, Tk, 32, False, 1.0, t, t, t, t, f32, lse, codes, codes, None,
                                         t, t, t, t, lse, None, 0, ok)
