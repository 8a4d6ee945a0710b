"""Seeded synthetic inputs shaped like the paper's workloads.

The paper feeds its models with batches produced by seqio feature converters
("Task-based API" section): fixed-length integer arrays of input and target
token ids, id 0 for padding, optionally several examples packed into one row
with segment ids.  No dataset ships with this repository, so the generators
below draw such arrays from a seeded numpy PCG64 stream.

This module holds no model arithmetic.  It serves both the CPU oracle's tests
and the GPU library's tests/benchmark, which is why it imports neither.
"""
from __future__ import annotations

import numpy as np

# Model dimensions of the five workloads (names follow the paper's model list).
CONFIGS = {
    "tiny": dict(arch=0, n_enc_layers=2, n_dec_layers=2, d_model=128, n_heads=4, d_kv=32,
                 d_ff=256, vocab=512, batch=4, enc_len=64, dec_len=32, dtype="f32",
                 tokens="uniform", padding=0.0, packed=False, seed=1234),
    "small": dict(arch=0, n_enc_layers=8, n_dec_layers=8, d_model=512, n_heads=6, d_kv=64,
                  d_ff=1024, vocab=32128, batch=64, enc_len=512, dec_len=114, dtype="bf16",
                  tokens="zipf", padding=0.1, packed=False, seed=1235),
    "base": dict(arch=0, n_enc_layers=12, n_dec_layers=12, d_model=768, n_heads=12, d_kv=64,
                 d_ff=2048, vocab=32128, batch=128, enc_len=512, dec_len=114, dtype="bf16",
                 tokens="zipf", padding=0.0, packed=True, seed=1236),
    "xl": dict(arch=0, n_enc_layers=24, n_dec_layers=24, d_model=2048, n_heads=32, d_kv=64,
               d_ff=5120, vocab=32128, batch=32, enc_len=512, dec_len=114, dtype="bf16",
               tokens="zipf", padding=0.0, packed=False, seed=1237),
    "declm": dict(arch=1, n_enc_layers=0, n_dec_layers=24, d_model=2048, n_heads=16, d_kv=128,
                  d_ff=5120, vocab=32128, batch=8, enc_len=0, dec_len=2048, dtype="bf16",
                  tokens="zipf", padding=0.0, packed=True, seed=1238),
}

MODEL_KEYS = ("arch", "n_enc_layers", "n_dec_layers", "d_model", "n_heads", "d_kv", "d_ff", "vocab")


def model_dims(name_or_dict, **overrides):
    c = dict(CONFIGS[name_or_dict]) if isinstance(name_or_dict, str) else dict(name_or_dict)
    c.update(overrides)
    return c


def _zipf_sampler(rng, vocab, a=1.1):
    """Bounded Zipf over ranks 1..vocab-1 (p(r) ~ r^-a) through the inverse CDF;
    rank -> token id by a seeded permutation of 1..vocab-1."""
    ranks = np.arange(1, vocab, dtype=np.float64)
    cdf = np.cumsum(ranks ** (-a))
    cdf /= cdf[-1]
    perm = rng.permutation(vocab - 1) + 1

    def draw(shape):
        u = rng.random(shape)
        r = np.searchsorted(cdf, u, side="left")
        r = np.minimum(r, vocab - 2)
        return perm[r].astype(np.int32)
    return draw


def _uniform_sampler(rng, vocab):
    def draw(shape):
        return rng.integers(1, vocab, size=shape, dtype=np.int64).astype(np.int32)
    return draw


def _segment_lengths(rng, total, mean_len, lo):
    """Lengths of consecutive examples packed into one row of `total` slots."""
    out = []
    used = 0
    while used < total:
        n = int(rng.geometric(1.0 / max(mean_len - lo + 1, 1))) + lo - 1
        n = max(lo, min(n, total - used))
        out.append(n)
        used += n
    return out


def make_batch(cfg, seed=None, batch=None):
    """Returns dict(enc_tokens, enc_segment_ids, dec_targets, dec_segment_ids);
    int32 arrays [B, T]; the segment arrays are None for unpacked rows and
    enc_* are None for the decoder-only architecture."""
    c = model_dims(cfg)
    rng = np.random.Generator(np.random.PCG64(c["seed"] if seed is None else seed))
    B = c["batch"] if batch is None else batch
    Te, Td, V = c["enc_len"], c["dec_len"], c["vocab"]
    draw = _zipf_sampler(rng, V) if c["tokens"] == "zipf" else _uniform_sampler(rng, V)
    dec_only = c["arch"] == 1
    enc = None if dec_only else draw((B, Te))
    dec = draw((B, Td))
    eseg = dseg = None
    if c["packed"]:
        dseg = np.zeros((B, Td), dtype=np.int32)
        if not dec_only:
            eseg = np.zeros((B, Te), dtype=np.int32)
        for b in range(B):
            if dec_only:
                # documents with log-uniform lengths in [64, Td], packed until the row is full
                pos, sid = 0, 1
                while pos < Td:
                    n = int(round(np.exp(rng.uniform(np.log(min(64, Td)), np.log(Td)))))
                    n = min(n, Td - pos)
                    if Td - pos - n < 8 and rng.random() < 0.5:   # leave a ragged padded tail sometimes
                        dec[b, pos + n:] = 0
                        dseg[b, pos:pos + n] = sid
                        pos = Td
                        break
                    dseg[b, pos:pos + n] = sid
                    pos += n
                    sid += 1
            else:
                # paired examples: encoder pieces of mean Te/4, decoder pieces of mean Td/4
                el = _segment_lengths(rng, Te, max(Te // 4, 2), 2)
                n_ex = len(el)
                ep, dp = 0, 0
                for s in range(n_ex):
                    dl = max(1, int(round(el[s] * Td / Te * rng.uniform(0.7, 1.2))))
                    if dp + dl > Td or s >= 250:
                        break
                    eseg[b, ep:ep + el[s]] = s + 1
                    dseg[b, dp:dp + dl] = s + 1
                    ep += el[s]
                    dp += dl
                enc[b, eseg[b] == 0] = 0
                dec[b, dseg[b] == 0] = 0
    elif c["padding"] > 0:
        for b in range(B):
            if not dec_only:
                le = int(rng.integers(int(np.ceil((1 - 2 * c["padding"]) * Te)), Te + 1))
                enc[b, le:] = 0
            ld = int(rng.integers(max(1, int(np.ceil((1 - 2 * c["padding"]) * Td))), Td + 1))
            dec[b, ld:] = 0
    return dict(enc_tokens=enc, enc_segment_ids=eseg, dec_targets=dec, dec_segment_ids=dseg)


def make_params(shapes, seed, stddev=0.02, scale_jitter=0.02, round_bf16=False):
    """N(0, stddev) for matrices and bias tables; norm scales (1-D) are
    1 + N(0, scale_jitter) so that their gradients are exercised.
    `shapes`: ordered mapping name -> shape.  With round_bf16 the values are
    rounded to the nearest bfloat16 (ties to even) and returned as float32."""
    rng = np.random.Generator(np.random.PCG64(seed))
    out = {}
    for name, shp in shapes.items():
        if len(shp) == 1:
            a = 1.0 + scale_jitter * rng.standard_normal(shp)
        else:
            a = stddev * rng.standard_normal(shp)
        a = a.astype(np.float32)
        if round_bf16:
            a = round_to_bf16(a)
        out[name] = a
    return out


def round_to_bf16(a):
    """float32 -> nearest bfloat16 (ties to even), returned as float32."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    r = ((u >> 16) & 1) + np.uint32(0x7FFF)
    u2 = ((u + r) & np.uint32(0xFFFF0000)).astype(np.uint32)
    return u2.view(np.float32).reshape(a.shape)
