"""Times the attention entry points of the C ABI on their own (CUDA events, seeded synthetic inputs):

    python -m paper_2203_17189_b200.bench_attention [--reps 10] [--cases enc,cross,self,declm]

For each problem it prints the forward call, the backward as two kernels that each recompute the scores
(`t5_attention`, backward = 1) and the one-pass backward (`t5_attention_backward_onepass`: delta, then
dK / dV / dS, then dQ from the stored dS).  Shapes are those of the XL workload's encoder, cross- and decoder
self-attention and of the decoder-only workload."""
import argparse

import torch

from . import binding as Bd

DEV = "cuda:0"
CASES = {
    # B, H, Tq, Tk, d_kv, causal, bias
    "enc": (32, 32, 512, 512, 64, False, True),
    "cross": (32, 32, 114, 512, 64, False, False),
    "self": (32, 32, 114, 114, 64, True, True),
    "declm": (8, 16, 2048, 2048, 128, True, True),
}


def time_us(fn, reps):
    for _ in range(2):
        fn()
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    for _ in range(reps):
        fn()
    e1.record()
    torch.cuda.synchronize()
    return e0.elapsed_time(e1) / reps * 1e3


def run(name, reps):
    B, H, Tq, Tk, dk, causal, use_bias = CASES[name]
    I, bf = H * dk, torch.bfloat16
    g = torch.Generator(device=DEV)
    g.manual_seed(1)

    def rnd(*shape, s=1.0):
        return (torch.randn(*shape, device=DEV, generator=g) * s).to(bf)
    if Tq == Tk:      # q, k, v as column blocks of one projection output, like the model's layout
        qkv, dqkv = rnd(B * Tq, 3 * I, s=0.7), torch.empty(B * Tq, 3 * I, dtype=bf, device=DEV)
        q, k, v = qkv[:, :I], qkv[:, I:2 * I], qkv[:, 2 * I:]
        dq, dk_, dv = dqkv[:, :I], dqkv[:, I:2 * I], dqkv[:, 2 * I:]
    else:
        q, kv = rnd(B * Tq, I, s=0.7), rnd(B * Tk, 2 * I, s=0.7)
        k, v = kv[:, :I], kv[:, I:]
        dq, dkv = torch.empty_like(q), torch.empty_like(kv)
        dk_, dv = dkv[:, :I], dkv[:, I:]
    do = rnd(B * Tq, I)
    cq = torch.ones(B, Tq, dtype=torch.int32, device=DEV)
    ck = torch.ones(B, Tk, dtype=torch.int32, device=DEV)
    bias, far = None, 0
    if use_bias:      # constant beyond +-91, like a bias expanded from 32 buckets with maximum distance 128
        bias = torch.randn(H, Tq + Tk - 1, device=DEV, generator=g) * 0.5
        c = Tq - 1
        if c - 91 > 0:
            far = 91
            bias[:, c + far:] = bias[:, c + far:c + far + 1]
            bias[:, :c - far] = bias[:, c - far:c - far + 1]
    o = torch.empty(B * Tq, I, dtype=bf, device=DEV)
    o32 = torch.empty(B * Tq, I, dtype=torch.float32, device=DEV)
    lse = torch.empty(B, H, Tq, dtype=torch.float32, device=DEV)
    delta = torch.empty_like(lse)
    dbias = torch.zeros(H, Tq + Tk - 1, dtype=torch.float32, device=DEV) if use_bias else None
    scratch = torch.empty(Bd.t5_attention_ds_scratch_bytes(B, H, Tq, Tk) // 2, dtype=bf, device=DEV)
    scale = 0.125

    def fwd():
        Bd.t5_attention(1, False, B, H, Tq, Tk, dk, causal, scale, q, k, v, o, lse, cq, ck, bias, o32=o32)

    def two():
        Bd.t5_attention(1, True, B, H, Tq, Tk, dk, causal, scale, q, k, v, o, lse, cq, ck, bias, do=do, dq=dq, dk=dk_,
                        dv=dv, delta=delta, dbias_delta=dbias, o32=o32)

    def one():
        Bd.t5_attention_backward_onepass(B, H, Tq, Tk, dk, causal, scale, q, k, v, o, o32, lse, cq, ck, bias, do, dq,
                                         dk_, dv, delta, dbias, far, scratch)
    fwd()
    t_f, t_2, t_1 = time_us(fwd, reps), time_us(two, reps), time_us(one, reps)
    flops = 4.0 * B * H * Tq * Tk * dk * (0.5 if causal else 1.0)
    print(f"{name:6s} B{B} H{H} {Tq}x{Tk} d_kv {dk} causal {int(causal)} bias {int(use_bias)}: "
          f"forward {t_f:.0f} us ({flops / t_f / 1e6:.0f} TFLOP/s), backward two-kernel {t_2:.0f} us, one-pass {t_1:.0f} us")


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--reps", type=int, default=10)
    ap.add_argument("--cases", default="enc,cross,self")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("needs a CUDA device; there is no CPU fallback")
    for name in args.cases.split(","):
        run(name, args.reps)


if __name__ == "__main__":
    main()
