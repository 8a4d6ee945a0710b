#!/usr/bin/env python
"""Benchmark of the T5.1.1 training step (forward + backward) on B200.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl ours|reference]

One step = one call of t5_train_step_fwd_bwd on one synthetic batch.  Prints one
JSON line: whole-job train tokens/s (inputs resident in device memory), the
same through host buffers (`e2e`), model-FLOPs utilisation, a roofline entry
for the dominant kernel (the tcgen05 GEMM) from live per-launch CUDA-event
timings, the CPU oracle timed on this host (`cpu_baseline`), GPU clocks sampled
during the timed region and the number of kernels launched.

With --gpus N > 1 (under torchrun) every rank runs an independent replica on
its own batch: the step has no exchange between batch rows, so there is no
collective on the data path; ranks only agree on the slowest time.
"""
from __future__ import annotations

import argparse
import json
import os
import statistics
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2203_17189_b200 import workloads as WL  # noqa: E402

NOMINAL_BF16_TFLOPS = 2250.0
FALLBACK_PEAKS = {"hbm_gbs": 6650.0, "bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0}


def step_flops(c, B=None):
    """Algorithmic FLOPs of one step (2mnk per GEMM, backward = 2x forward, causal
    self-attention counted at half, padding not discounted, recomputation not counted)."""
    B = c["batch"] if B is None else B
    d, H, k, F, V = c["d_model"], c["n_heads"], c["d_kv"], c["d_ff"], c["vocab"]
    I = H * k
    Te, Td = c["enc_len"], c["dec_len"]
    Ne, Nd = B * Te, B * Td
    if c["arch"] == 0:
        fwd = c["n_enc_layers"] * (2 * Ne * (4 * d * I + 3 * d * F) + 4 * B * H * Te * Te * k)
        fwd += c["n_dec_layers"] * (2 * Nd * (4 * d * I + 2 * d * I + 3 * d * F) + 2 * Ne * 2 * d * I
                                    + 2 * B * H * Td * Td * k + 4 * B * H * Td * Te * k)
    else:
        fwd = c["n_dec_layers"] * (2 * Nd * (4 * d * I + 3 * d * F) + 2 * B * H * Td * Td * k)
    fwd += 2 * Nd * d * V
    return 3.0 * fwd


def attention_flops(c, B=None):
    """The attention share of step_flops: the QK^T and PV contractions, forward + backward (2x forward)."""
    B = c["batch"] if B is None else B
    H, k, Te, Td = c["n_heads"], c["d_kv"], c["enc_len"], c["dec_len"]
    if c["arch"] == 0:
        fwd = c["n_enc_layers"] * 4 * B * H * Te * Te * k + c["n_dec_layers"] * (2 * B * H * Td * Td * k
                                                                                     + 4 * B * H * Td * Te * k)
    else:
        fwd = c["n_dec_layers"] * 2 * B * H * Td * Td * k
    return 3.0 * fwd


# DRAM bytes (dram__bytes_read.sum + dram__bytes_write.sum) of the GEMM launches of one XL step, from the ncu
# capture summarised in profiles/gemm_family_dram_traffic_xl_width.md: a 1+1-layer step was captured (the full
# step holds 46 GB and 795 GEMM launches), its launches grouped into encoder-layer, decoder-layer and logits GEMMs,
# and the groups scaled by the layer counts (every layer launches the same shapes).  Valid only for the kernel
# source the capture ran: keyed by the SHA-1 of csrc/gemm_tcgen05.cu, anything else reports null.
GEMM_DRAM_TRAFFIC = {
    # "sha1 of gemm_tcgen05.cu": {"xl": bytes per launch averaged over the 795 GEMM launches of a step}
    "45b35e45ff2aa93c561dcf57cd08107b73f57855": {"xl": 290.1e6},
}


def gemm_traffic_per_launch(workload):
    import hashlib
    src = os.path.join(ROOT, "paper_2203_17189_b200", "csrc", "gemm_tcgen05.cu")
    try:
        with open(src, "rb") as f:
            key = hashlib.sha1(f.read()).hexdigest()
    except OSError:
        return None
    return GEMM_DRAM_TRAFFIC.get(key, {}).get(workload)


def write_launch_table(path, records, steps, title):
    """Per distinct (kernel call, shape): launches per step, time per step, share, and the GEMMs' TFLOP/s."""
    agg = {}
    for what, fam, M, N, K, ms in records:
        a = agg.setdefault((what, M, N, K), [0, 0.0, fam])
        a[0] += 1
        a[1] += ms
    total = sum(a[1] for a in agg.values())
    with open(path, "w") as f:
        f.write(f"# {title}\n\n| call | M | N | K | launches/step | ms/step | share | avg us | TFLOP/s |\n|---|---|---|---|---|---|---|---|---|\n")
        for (what, M, N, K), (n, ms, fam) in sorted(agg.items(), key=lambda kv: -kv[1][1]):
            tf = f"{2.0 * M * N * K * n / (ms * 1e-3) / 1e12:.0f}" if M and ms > 0 else "-"
            f.write(f"| {what} | {M or '-'} | {N or '-'} | {K or '-'} | {n / steps:g} | {ms / steps:.3f} | "
                    f"{ms / total:.3f} | {1e3 * ms / n:.1f} | {tf} |\n")
        f.write(f"\ntotal {total / steps:.2f} ms per step (sum of per-launch CUDA-event times, {steps} step(s))\n")


# ---- the attention entry points on their own (--attention-cases): forward, the backward as two kernels that each
# recompute the scores (t5_attention, backward = 1) and the one-pass backward (t5_attention_backward_onepass), on the
# shapes of the XL workload's encoder, cross- and decoder self-attention and of the decoder-only workload
ATTN_CASES = {
    # B, H, Tq, Tk, d_kv, causal, bias
    "enc": (32, 32, 512, 512, 64, False, True),
    "cross": (32, 32, 114, 512, 64, False, False),
    "self": (32, 32, 114, 114, 64, True, True),
    "declm": (8, 16, 2048, 2048, 128, True, True),
}


def attn_time_us(torch, fn, reps):
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


def run_attention_case(name, reps):
    import torch
    from paper_2203_17189_b200 import binding as Bd
    DEV = "cuda:0"
    B, H, Tq, Tk, dk, causal, use_bias = ATTN_CASES[name]
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
    t_f, t_2, t_1 = attn_time_us(torch, fwd, reps), attn_time_us(torch, two, reps), attn_time_us(torch, one, reps)
    flops = 4.0 * B * H * Tq * Tk * dk * (0.5 if causal else 1.0)
    print(f"{name:6s} B{B} H{H} {Tq}x{Tk} d_kv {dk} causal {int(causal)} bias {int(use_bias)}: "
          f"forward {t_f:.0f} us ({flops / t_f / 1e6:.0f} TFLOP/s), backward two-kernel {t_2:.0f} us, one-pass {t_1:.0f} us")



def load_peaks():
    p = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(p):
        with open(p) as f:
            d = json.load(f)
        return d, "measured"
    return dict(FALLBACK_PEAKS), "fallback"


class ClockSampler:
    """nvidia-smi clock/throttle samples while the timed region runs."""
    Q = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
         "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index):
        self.gpu = gpu_index
        self.proc = None
        self.lines = []

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", "-i", str(self.gpu), "--query-gpu=" + self.Q,
                                          "--format=csv,noheader,nounits", "-lms", "100"],
                                         stdout=subprocess.PIPE, stderr=subprocess.DEVNULL, text=True)
            self.t = threading.Thread(target=self._read, daemon=True)
            self.t.start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.lines.append(line.strip())

    def stop(self):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons, power = [], [], set(), []
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for ln in self.lines:
            f = [x.strip() for x in ln.split(",")]
            if len(f) < 9:
                continue
            try:
                sm.append(float(f[1])); mx.append(float(f[2])); power.append(float(f[3]))
            except ValueError:
                continue
            for n, v in zip(names, f[5:9]):
                if v.lower().startswith("active"):
                    reasons.add(n)
        if not sm:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["no samples"]}
        return {"sm_mhz": statistics.median(sm), "sm_max_mhz": max(mx), "reasons": sorted(reasons),
                "power_w_max": max(power), "samples": len(sm)}


class OracleSample:
    """`rows` batch rows of the workload run through the CPU oracle (full model)."""

    def __init__(self, cfg, rows, dtype=np.float32):
        from oracle import t5_oracle as O
        self.O = O
        self.cfg = cfg
        self.rows = rows
        self.dtype = dtype
        self.ocfg = O.T5Config(**{k: cfg[k] for k in WL.MODEL_KEYS})
        self.batch = WL.make_batch(cfg, batch=rows)
        params = WL.make_params(O.param_shapes(self.ocfg), cfg["seed"], round_bf16=(cfg["dtype"] == "bf16"))
        self.params = {k: np.asarray(v, dtype=dtype) for k, v in params.items()}
        self.tokens = rows * (cfg["enc_len"] + cfg["dec_len"])

    def run(self):
        """One oracle step on the sample; returns seconds."""
        b = self.batch
        t0 = time.perf_counter()
        self.O.t5_train_step(self.ocfg, self.params, b["enc_tokens"], b["enc_segment_ids"], b["dec_targets"],
                             b["dec_segment_ids"], dtype=self.dtype)
        return time.perf_counter() - t0


def max_over_ranks(ms, dist=None, device=None):
    """The job's time is the slowest rank's: all-reduce MAX of the per-rank device time (no-op on one rank)."""
    if dist is None:
        return float(ms)
    import torch
    t = torch.tensor([float(ms)], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_value(tokens_per_rank_step, world, ms_total, steps):
    """tokens/s of all ranks together (every rank runs an independent replica on its own batch)."""
    return world * tokens_per_rank_step / (ms_total * 1e-3 / steps)


def cpu_threads():
    try:
        from threadpoolctl import threadpool_info
        n = [p.get("num_threads", 0) for p in threadpool_info() if p.get("user_api") == "blas"]
        if n:
            return max(n)
    except Exception:
        pass
    return os.cpu_count() or 1


def run_reference(args, cfg):
    """The oracle as it stands, timed on the host cores; each step is a bounded sample."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    rows = args.ref_rows
    smp = OracleSample(cfg, rows)
    for _ in range(args.warmup):
        smp.run()
    t0 = time.perf_counter()
    for _ in range(args.steps):
        smp.run()
    dt = (time.perf_counter() - t0) / args.steps
    toks = rows * (cfg["enc_len"] + cfg["dec_len"])
    value = toks / dt
    sample = f"{rows} of {cfg['batch']} batch rows per step, full model, float32"
    out = {"impl": "reference", "metric": "train_tokens_per_sec", "value": value, "unit": "tokens/s",
           "n_gpus": args.gpus, "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt * 1e3,
           "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
           "config": {"workload": args.workload, "sample": sample},
           "cpu_baseline": {"value": value, "unit": "tokens/s", "cores": cpu_threads(), "kind": "oracle",
                            "sample": sample},
           "e2e": {"value": value, "unit": "tokens/s", "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(out))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=10)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="xl", choices=list(WL.CONFIGS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--batch", type=int, default=None, help="override the workload's batch rows")
    ap.add_argument("--enc-layers", type=int, default=None, help="reduced depth (small profiling captures only)")
    ap.add_argument("--dec-layers", type=int, default=None)
    ap.add_argument("--ref-rows", type=int, default=1)
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--flags", type=int, default=0)
    ap.add_argument("--recompute", type=int, default=0, choices=[0, 1],
                    help="activation policy (0 keeps everything; the reported number uses 0)")
    ap.add_argument("--attention-cases", default=None, metavar="enc,cross,self,declm",
                    help="instead of the step, time the attention calls of the C ABI on these shapes and print a table")
    ap.add_argument("--launch-table", default=None, metavar="PATH",
                    help="also write a per-call, per-shape table of the profiled steps' device times (markdown)")
    args = ap.parse_args()
    cfg = WL.model_dims(args.workload)
    if args.batch:
        cfg["batch"] = args.batch
    if args.enc_layers is not None:
        cfg["n_enc_layers"] = args.enc_layers
    if args.dec_layers is not None:
        cfg["n_dec_layers"] = args.dec_layers
    if args.impl == "reference":
        run_reference(args, cfg)
        return
    if args.attention_cases:
        import torch
        if not torch.cuda.is_available():
            raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
        for name in args.attention_cases.split(","):
            run_attention_case(name, max(args.steps, 1))
        return

    import torch
    from paper_2203_17189_b200 import binding as Bd

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU fallback")
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    dist = None
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=dev)

    Bd.lib()   # fails loudly if the CUDA library is missing
    B, Te, Td = cfg["batch"], cfg["enc_len"], cfg["dec_len"]
    h = Bd.Handle(Bd.make_config(cfg, B, Te, Td, cfg["dtype"], flags=args.flags, recompute=args.recompute))
    n = h.t5_param_count()
    params = torch.empty(n, dtype=h.torch_dtype, device=dev)
    h.t5_init_params(params, 1234 + rank, 0.02)
    ws_bytes = h.t5_workspace_bytes()
    ws = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
    grads = torch.empty(n, dtype=torch.float32, device=dev)
    loss4 = torch.zeros(4, dtype=torch.float32, device=dev)
    host_batch = WL.make_batch(cfg, seed=cfg["seed"] + 1000 * rank)
    pinned = {k: (None if v is None else torch.from_numpy(v).pin_memory()) for k, v in host_batch.items()}
    dbatch = {k: (None if v is None else v.to(dev)) for k, v in pinned.items()}
    tokens_per_step = B * (Te + Td)
    nonpad = int(sum((v != 0).sum() for k, v in host_batch.items() if v is not None and "segment" not in k))
    flops = step_flops(cfg)

    def step():
        h.t5_train_step_fwd_bwd(params, dbatch, grads, loss4, ws)

    def barrier():
        torch.cuda.synchronize()
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()

    def timed(fn, steps):
        barrier()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(steps):
            fn()
        e1.record()
        barrier()
        return max_over_ranks(e0.elapsed_time(e1), dist, dev)

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    h.t5_device_status(ws)

    sampler = ClockSampler(local)
    sampler.start()
    ms = timed(step, args.steps)
    clocks = sampler.stop()
    launches = h.t5_launch_count()
    loss_dev = loss4.cpu().numpy().tolist()
    h.t5_device_status(ws)

    # end to end: token arrays start in pinned host memory, the loss comes back to the host, every step
    loss_host = torch.zeros(4, dtype=torch.float32).pin_memory()
    h2d = sum(v.numel() * v.element_size() for v in pinned.values() if v is not None)

    def e2e_step():
        for k, v in pinned.items():
            if v is not None:
                dbatch[k].copy_(v, non_blocking=True)
        step()
        loss_host.copy_(loss4, non_blocking=True)
        torch.cuda.current_stream().synchronize()

    e2e_step()
    ms_e2e = timed(e2e_step, args.steps)

    # per-kernel-family device time (event pair around every launch) for the roofline entry
    h.t5_profile_enable(True)
    step()
    torch.cuda.synchronize()
    h.t5_profile_read()
    prof_steps = max(1, min(args.steps, 3))
    for _ in range(prof_steps):
        step()
    torch.cuda.synchronize()
    if args.launch_table and rank == 0:
        write_launch_table(args.launch_table, h.t5_profile_launches(), prof_steps,
                           f"per-launch CUDA-event times, workload {args.workload}, layers "
                           f"{cfg['n_enc_layers']}+{cfg['n_dec_layers']}, batch {B}")
    prof = h.t5_profile_read()
    h.t5_profile_enable(False)
    gemm_ms, gemm_flops, gemm_launches = prof["gemm"]
    total_prof_ms = sum(v[0] for v in prof.values())

    peaks, peak_kind = load_peaks()
    # the GEMM kernel runs inside a long step: compare with the sustained figure
    peak_tf = float(peaks.get("bf16_tflops_sustained") or peaks.get("bf16_tflops"))
    if cfg["dtype"] != "bf16":
        peak_tf = peak_tf / 16.0     # float32 SIMT validation path: not a tensor-core contraction
    achieved_tf = gemm_flops / (gemm_ms * 1e-3) / 1e12 if gemm_ms > 0 else 0.0
    attn_ms = prof["attn_fwd"][0] + prof["attn_bwd"][0]
    attn_launches = prof["attn_fwd"][2] + prof["attn_bwd"][2]
    attn_tf = attention_flops(cfg) * prof_steps / (attn_ms * 1e-3) / 1e12 if attn_ms > 0 else 0.0

    sec = ms * 1e-3 / args.steps
    value = whole_job_value(tokens_per_step, world, ms, args.steps)
    sec_e2e = ms_e2e * 1e-3 / args.steps
    out = {
        "metric": "train_tokens_per_sec", "value": value, "unit": "tokens/s", "n_gpus": world,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": sec * 1e3, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": cfg["dtype"], "data": "synthetic",
        "config": {"workload": args.workload, "layers": [cfg["n_enc_layers"], cfg["n_dec_layers"]], "batch_rows": B, "enc_len": Te, "dec_len": Td,
                   "tokens_per_step": tokens_per_step, "nonpad_tokens_per_step": nonpad,
                   "l2": f"working set {ws_bytes / 1e9:.1f} GB of activations >> 126 MB L2; no explicit flush",
                   "parallelism": "replicas only" if world > 1 else "single GPU",
                   "activation_recomputation": bool(args.recompute)},
        "mfu": {"step_tflop": flops / 1e12, "achieved_tflops": flops / sec / 1e12,
                "vs_nominal_2250": flops / sec / 1e12 / NOMINAL_BF16_TFLOPS,
                "vs_measured_burst": flops / sec / 1e12 / float(peaks.get("bf16_tflops", 1590.0)),
                "vs_measured_sustained": flops / sec / 1e12 / float(peaks.get("bf16_tflops_sustained", 1400.0))},
        "loss": loss_dev,
        "e2e": {"value": world * tokens_per_step / sec_e2e, "unit": "tokens/s", "h2d_bytes_per_step": h2d,
                "d2h_bytes_per_step": 16},
        "gpu_launches": launches * args.steps,
        "clocks": clocks,
        "roofline": {"kernel": "gemm_tc2_kernel (tcgen05.mma.cta_group::2, CTA pairs; the few shapes it does not "
                               "take run gemm_tc_kernel)" if cfg["dtype"] == "bf16" else "gemm_simt_kernel",
                     "bound": "tensor", "achieved": achieved_tf,
                     "peak": peak_tf, "unit": "TFLOP/s", "frac": achieved_tf / peak_tf if peak_tf else None,
                     "peak_kind": f"{peak_kind} sustained bf16 matmul",
                     "traffic": gemm_traffic_per_launch(args.workload),
                     "traffic_unit": "DRAM bytes per launch (ncu, 1+1-layer capture scaled by layer counts)",
                     "algorithmic_per_launch": gemm_flops / max(gemm_launches, 1),
                     "launches_per_step": gemm_launches / prof_steps,
                     "avg_launch_ms": gemm_ms / max(gemm_launches, 1),
                     "share_of_step": gemm_ms / total_prof_ms if total_prof_ms else None},
        # the attention family (forward, delta, dK/dV/dS, dQ kernels): QK^T and PV FLOPs as in step_flops
        "roofline_attention": {"kernel": "attn_fwd_tc / attn_bwd_kvf_tc / attn_bwd_dq_ds_tc / attn_delta_tc",
                               "bound": "tensor", "achieved": attn_tf, "peak": peak_tf, "unit": "TFLOP/s",
                               "frac": attn_tf / peak_tf if peak_tf else None,
                               "peak_kind": f"{peak_kind} sustained bf16 matmul", "traffic": None,
                               "launches_per_step": attn_launches / prof_steps,
                               "share_of_step": attn_ms / total_prof_ms if total_prof_ms else None},
        "kernel_ms_per_step": {k: v[0] / prof_steps for k, v in prof.items()},
    }
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        rows = args.ref_rows
        smp = OracleSample(cfg, rows)
        dt = smp.run()
        rate = smp.tokens / dt
        out["cpu_baseline"] = {"value": rate, "unit": "tokens/s", "cores": cpu_threads(), "kind": "oracle",
                               "sample": f"{rows} of {B} batch rows, full model, float32, {dt:.1f} s"}
    if rank == 0:
        print(json.dumps(out))
    if dist is not None:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
