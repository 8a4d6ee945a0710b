"""Helpers shared by the GPU parity tests, the smoke check and the benchmark's
checks: conversion between the library's flat parameter buffer and the
oracle's named tensors, and the comparison metrics."""
import numpy as np

DENSE_SUFFIXES = (".q", ".k", ".v", ".o", ".wi0", ".wi1", ".wo", "lm_head")


def is_dense(name):
    return name.endswith(DENSE_SUFFIXES)


def oracle_shapes_from_manifest(manifest):
    """name -> shape in the oracle's [in, out] convention."""
    out = {}
    for name, _, shape in manifest:
        out[name] = tuple(reversed(shape)) if is_dense(name) else tuple(shape)
    return out


def pack_params(manifest, n_params, named):
    """Oracle-convention named tensors -> flat float32 array in the library's layout."""
    flat = np.zeros(n_params, dtype=np.float32)
    for name, off, shape in manifest:
        a = np.asarray(named[name], dtype=np.float32)
        if is_dense(name):
            a = a.T
        assert a.shape == tuple(shape), (name, a.shape, shape)
        flat[off:off + a.size] = a.reshape(-1)
    return flat


def unpack(manifest, flat):
    """Flat array in the library's layout -> oracle-convention named tensors."""
    out = {}
    for name, off, shape in manifest:
        n = int(np.prod(shape))
        a = np.asarray(flat[off:off + n]).reshape(shape)
        out[name] = a.T.copy() if is_dense(name) else a.copy()
    return out


def tensor_metrics(got, ref):
    """(cosine, max-abs-normalised error) of one gradient tensor."""
    g = np.asarray(got, dtype=np.float64).reshape(-1)
    r = np.asarray(ref, dtype=np.float64).reshape(-1)
    rmax = np.abs(r).max()
    if rmax == 0:
        # an identically-zero reference (e.g. dS with a single key): only rounding residue may remain
        return (1.0 if np.abs(g).max() <= 1e-7 else 0.0), float(np.abs(g).max())
    cos = float(g @ r / (np.linalg.norm(g) * np.linalg.norm(r) + 1e-300))
    return cos, float(np.abs(g - r).max() / rmax)


def compare_grads(manifest, flat_grads, oracle_grads):
    """Per-tensor metrics; returns (worst_cos, worst_maxrel, table)."""
    named = unpack(manifest, flat_grads)
    table = {}
    for name in named:
        table[name] = tensor_metrics(named[name], oracle_grads[name])
    worst_cos = min(v[0] for v in table.values())
    worst_rel = max(v[1] for v in table.values())
    return worst_cos, worst_rel, table
