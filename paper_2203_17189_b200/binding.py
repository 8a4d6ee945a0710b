"""ctypes binding of libt5b200.so: argument marshalling only.

Every function here has the name of the C entry point it wraps (see
include/t5_b200.h) and does no arithmetic of its own.  torch is used for
device buffers and the current stream.  Loading fails loudly when the library
has not been built; there is no fallback path.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libt5b200.so")

T5_ABI_VERSION = 2
ERR_NAMES = {0: "T5_OK", -1: "T5_ERR_NULL", -2: "T5_ERR_CONFIG", -3: "T5_ERR_SHAPE", -4: "T5_ERR_ALIGN",
             -5: "T5_ERR_WORKSPACE", -6: "T5_ERR_CUDA", -7: "T5_ERR_DEVICE_TIMEOUT", -8: "T5_ERR_ARG"}


class t5_config(C.Structure):
    _fields_ = [("abi_version", C.c_int32), ("arch", C.c_int32),
                ("n_enc_layers", C.c_int32), ("n_dec_layers", C.c_int32),
                ("d_model", C.c_int32), ("n_heads", C.c_int32), ("d_kv", C.c_int32),
                ("d_ff", C.c_int32), ("vocab", C.c_int32),
                ("rel_buckets", C.c_int32), ("rel_max_distance", C.c_int32),
                ("max_batch", C.c_int32), ("max_enc_len", C.c_int32), ("max_dec_len", C.c_int32),
                ("z_loss", C.c_float), ("rms_eps", C.c_float), ("attn_scale", C.c_float),
                ("logit_scale", C.c_float),
                ("dtype", C.c_int32), ("recompute", C.c_int32), ("flags", C.c_int32),
                ("ffn_act", C.c_int32), ("untied_head", C.c_int32)]


class t5_batch(C.Structure):
    _fields_ = [("B", C.c_int32), ("Te", C.c_int32), ("Td", C.c_int32),
                ("d_enc_tokens", C.c_void_p), ("d_enc_segment_ids", C.c_void_p),
                ("d_dec_targets", C.c_void_p), ("d_dec_segment_ids", C.c_void_p), ("d_dec_prefix", C.c_void_p)]


class t5_profile_launch(C.Structure):
    _fields_ = [("what", C.c_char * 40), ("family", C.c_int32), ("M", C.c_int32), ("N", C.c_int32),
                ("K", C.c_int32), ("ms", C.c_float)]


# void hook(void* user, int64 offset, int64 count, const float* d_rank_weight, void* stream)
GRAD_HOOK = C.CFUNCTYPE(None, C.c_void_p, C.c_int64, C.c_int64, C.c_void_p, C.c_void_p)

EXPORTS = ["t5_create", "t5_destroy", "t5_last_error", "t5_param_count", "t5_param_tensors",
           "t5_param_manifest", "t5_workspace_bytes", "t5_init_params", "t5_train_step_fwd_bwd",
           "t5_encode", "t5_decode_logits", "t5_device_status", "t5_profile_enable", "t5_profile_read",
           "t5_profile_launches", "t5_adamw_update", "t5_decode_cache_bytes", "t5_decode_step_workspace_bytes",
           "t5_decode_begin", "t5_decode_step",
           "t5_launch_count", "t5_relpos_buckets", "t5_xent_zloss",
           "t5_gemm", "t5_attention", "t5_attention_backward_noalloc",
           "t5_attention_ds_scratch_bytes", "t5_attention_backward_onepass",
           "t5_kernel_status_word", "t5_selftest_bounded_wait", "t5_set_grad_hook"]

_lib = None


class T5Error(RuntimeError):
    def __init__(self, code, msg=""):
        super().__init__(f"{ERR_NAMES.get(code, code)}: {msg}")
        self.code = code


def lib():
    """The loaded shared library (raises if it was not built)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2203_17189_b200.build` "
                               "(or __graft_entry__.build()) first; there is no fallback path")
        L = C.CDLL(LIB_PATH)
        vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
        L.t5_create.argtypes = [C.POINTER(t5_config), C.POINTER(vp)]
        L.t5_destroy.argtypes = [vp]
        L.t5_last_error.argtypes = [vp]
        L.t5_last_error.restype = C.c_char_p
        L.t5_param_count.argtypes = [vp, C.POINTER(i64)]
        L.t5_param_tensors.argtypes = [vp, C.POINTER(i32)]
        L.t5_param_manifest.argtypes = [vp, i32, C.c_char_p, C.POINTER(i64), C.POINTER(i32 * 4), C.POINTER(i32)]
        L.t5_workspace_bytes.argtypes = [vp, C.POINTER(i64)]
        L.t5_init_params.argtypes = [vp, vp, C.c_uint64, f32, vp]
        L.t5_train_step_fwd_bwd.argtypes = [vp, vp, C.POINTER(t5_batch), vp, vp, vp, i64, vp]
        L.t5_adamw_update.argtypes = [vp, vp, vp, vp, vp, vp, i64, f32, f32, f32, f32, f32, f32, vp]
        L.t5_decode_cache_bytes.argtypes = [vp, i32, i32, i32, C.POINTER(i64)]
        L.t5_decode_step_workspace_bytes.argtypes = [vp, i32, C.POINTER(i64)]
        L.t5_decode_begin.argtypes = [vp, vp, i32, i32, i32, vp, vp, vp, i64, vp]
        L.t5_decode_step.argtypes = [vp, vp, vp, i64, i32, i32, i32, i32, vp, vp, vp, i64, vp]
        L.t5_encode.argtypes = [vp, vp, C.POINTER(t5_batch), vp, vp, i64, vp]
        L.t5_decode_logits.argtypes = [vp, vp, C.POINTER(t5_batch), vp, vp, vp, i64, vp]
        L.t5_device_status.argtypes = [vp, vp, vp]
        L.t5_set_grad_hook.argtypes = [vp, GRAD_HOOK, vp]
        L.t5_kernel_status_word.argtypes = [vp]
        L.t5_selftest_bounded_wait.argtypes = [vp, i64, vp]
        L.t5_profile_enable.argtypes = [vp, i32]
        L.t5_profile_read.argtypes = [vp, C.POINTER(C.c_double * 8), C.POINTER(C.c_double * 8),
                                      C.POINTER(i64 * 8)]
        L.t5_profile_launches.argtypes = [vp, C.POINTER(t5_profile_launch), i32, C.POINTER(i32)]
        L.t5_launch_count.argtypes = [vp, C.POINTER(i64)]
        L.t5_relpos_buckets.argtypes = [i32, i32, i32, i32, i32, vp, vp]
        L.t5_xent_zloss.argtypes = [i32, vp, vp, i32, i32, f32, vp, vp, vp, vp]
        L.t5_gemm.argtypes = [i32, i32, i32, i32, i32, f32, vp, i32, i32, vp, i32, i32, vp, i32, i32, i32, vp, vp]
        L.t5_attention.argtypes = ([i32] * 9 + [f32] + [vp, i32] * 3 + [vp, i32, vp, vp, vp, vp, vp]
                                   + [vp, i32] * 4 + [vp, vp, vp])
        L.t5_attention_backward_noalloc.argtypes = ([i32] * 8 + [f32] + [vp, i32] * 4 + [vp] * 5
                                                    + [vp, i32] * 4 + [vp, vp])
        L.t5_attention_ds_scratch_bytes.argtypes = [i32] * 4 + [C.POINTER(i64)]
        L.t5_attention_backward_onepass.argtypes = ([i32] * 6 + [f32] + [vp, i32] * 4 + [vp] * 5
                                                    + [vp, i32] * 4 + [vp, vp, i32, vp, i64, vp])
        for n in EXPORTS:
            if n != "t5_last_error":
                getattr(L, n).restype = C.c_int
        _lib = L
    return _lib


def _stream():
    return C.c_void_p(torch.cuda.current_stream().cuda_stream)


def _ptr(t):
    return C.c_void_p(0 if t is None else t.data_ptr())


def _check(rc, h=None):
    if rc != 0:
        msg = lib().t5_last_error(h)
        raise T5Error(rc, msg.decode() if msg else "")


def make_config(dims, max_batch, max_enc_len, max_dec_len, dtype, *, z_loss=1e-4, rms_eps=1e-6,
                attn_scale=1.0, logit_scale=None, rel_buckets=32, rel_max_distance=128,
                recompute=0, flags=0, ffn_act=0, untied_head=0):
    """dims: mapping with arch, n_enc_layers, n_dec_layers, d_model, n_heads, d_kv, d_ff, vocab.
    dtype: 'f32' or 'bf16'.  ffn_act: 0 gated GELU (tanh), 1 ReLU, 2 gated GELU (erf).  logit_scale defaults to
    d_model^-1/2 with the tied embedding and to 1 with a separate head."""
    c = t5_config()
    c.abi_version = T5_ABI_VERSION
    for k in ("arch", "n_enc_layers", "n_dec_layers", "d_model", "n_heads", "d_kv", "d_ff", "vocab"):
        setattr(c, k, int(dims[k]))
    c.rel_buckets, c.rel_max_distance = rel_buckets, rel_max_distance
    c.max_batch, c.max_enc_len, c.max_dec_len = max_batch, max_enc_len, max_dec_len
    c.z_loss, c.rms_eps, c.attn_scale = z_loss, rms_eps, attn_scale
    if logit_scale is None:
        logit_scale = 1.0 if untied_head else float(dims["d_model"]) ** -0.5
    c.logit_scale = logit_scale
    c.ffn_act, c.untied_head = ffn_act, untied_head
    c.dtype = {"f32": 0, "bf16": 1}[dtype]
    c.recompute, c.flags = recompute, flags
    return c


class Handle:
    """Owns a t5_handle*; methods are the C calls with torch tensors as buffers."""

    def __init__(self, cfg: t5_config):
        self.cfg = cfg
        self._h = C.c_void_p()
        rc = lib().t5_create(C.byref(cfg), C.byref(self._h))
        if rc != 0:
            msg = lib().t5_last_error(None)
            raise T5Error(rc, msg.decode() if msg else "")
        self.torch_dtype = torch.float32 if cfg.dtype == 0 else torch.bfloat16

    def close(self):
        if self._h:
            lib().t5_destroy(self._h)
            self._h = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def t5_param_count(self):
        n = C.c_int64()
        _check(lib().t5_param_count(self._h, C.byref(n)), self._h)
        return n.value

    def t5_param_manifest(self):
        """List of (name, offset, shape)."""
        n = C.c_int32()
        _check(lib().t5_param_tensors(self._h, C.byref(n)), self._h)
        out = []
        for i in range(n.value):
            name = C.create_string_buffer(64)
            off = C.c_int64()
            shape = (C.c_int32 * 4)()
            nd = C.c_int32()
            _check(lib().t5_param_manifest(self._h, i, name, C.byref(off), C.byref(shape), C.byref(nd)), self._h)
            out.append((name.value.decode(), off.value, tuple(shape[:nd.value])))
        return out

    def t5_workspace_bytes(self):
        n = C.c_int64()
        _check(lib().t5_workspace_bytes(self._h, C.byref(n)), self._h)
        return n.value

    def t5_init_params(self, params, seed, stddev):
        _check(lib().t5_init_params(self._h, _ptr(params), C.c_uint64(seed), stddev, _stream()), self._h)

    def _batch(self, batch):
        b = t5_batch()
        dec = batch["dec_targets"]
        b.B, b.Td = dec.shape
        enc = batch.get("enc_tokens")
        b.Te = 0 if enc is None else enc.shape[1]
        b.d_enc_tokens = None if enc is None else enc.data_ptr()
        es = batch.get("enc_segment_ids")
        ds = batch.get("dec_segment_ids")
        b.d_enc_segment_ids = None if es is None else es.data_ptr()
        b.d_dec_targets = dec.data_ptr()
        b.d_dec_segment_ids = None if ds is None else ds.data_ptr()
        pre = batch.get("dec_prefix")
        b.d_dec_prefix = None if pre is None else pre.data_ptr()
        return b

    def t5_train_step_fwd_bwd(self, params, batch, grads, loss4, workspace):
        b = self._batch(batch)
        _check(lib().t5_train_step_fwd_bwd(self._h, _ptr(params), C.byref(b), _ptr(grads), _ptr(loss4),
                                           _ptr(workspace), workspace.numel() * workspace.element_size(),
                                           _stream()), self._h)

    def t5_adamw_update(self, params, master, m, v, grads, step, lr, beta1=0.9, beta2=0.999, eps=1e-8,
                        weight_decay=0.0, grad_scale=1.0):
        _check(lib().t5_adamw_update(self._h, _ptr(params), _ptr(master), _ptr(m), _ptr(v), _ptr(grads), step, lr,
                                     beta1, beta2, eps, weight_decay, grad_scale, _stream()), self._h)

    def t5_decode_cache_bytes(self, B, Te, Tmax):
        n = C.c_int64()
        _check(lib().t5_decode_cache_bytes(self._h, B, Te, Tmax, C.byref(n)), self._h)
        return n.value

    def t5_decode_step_workspace_bytes(self, B):
        n = C.c_int64()
        _check(lib().t5_decode_step_workspace_bytes(self._h, B, C.byref(n)), self._h)
        return n.value

    def t5_decode_begin(self, params, B, Te, Tmax, enc_tokens, enc_out, cache):
        _check(lib().t5_decode_begin(self._h, _ptr(params), B, Te, Tmax, _ptr(enc_tokens), _ptr(enc_out), _ptr(cache),
                                     cache.numel() * cache.element_size(), _stream()), self._h)

    def t5_decode_step(self, params, cache, B, Te, Tmax, t, tokens, logits, workspace):
        _check(lib().t5_decode_step(self._h, _ptr(params), _ptr(cache), cache.numel() * cache.element_size(), B, Te, Tmax,
                                    t, _ptr(tokens), _ptr(logits), _ptr(workspace),
                                    workspace.numel() * workspace.element_size(), _stream()), self._h)

    def t5_encode(self, params, batch, enc_out, workspace):
        b = self._batch(batch)
        _check(lib().t5_encode(self._h, _ptr(params), C.byref(b), _ptr(enc_out), _ptr(workspace),
                               workspace.numel() * workspace.element_size(), _stream()), self._h)

    def t5_decode_logits(self, params, batch, enc_out, logits, workspace):
        b = self._batch(batch)
        _check(lib().t5_decode_logits(self._h, _ptr(params), C.byref(b), _ptr(enc_out), _ptr(logits),
                                      _ptr(workspace), workspace.numel() * workspace.element_size(),
                                      _stream()), self._h)

    def t5_profile_enable(self, on):
        _check(lib().t5_profile_enable(self._h, int(on)), self._h)

    def t5_profile_read(self):
        """{family: (ms, flops, launches)}"""
        ms, fl, ln = (C.c_double * 8)(), (C.c_double * 8)(), (C.c_int64 * 8)()
        _check(lib().t5_profile_read(self._h, C.byref(ms), C.byref(fl), C.byref(ln)), self._h)
        names = ["gemm", "attn_fwd", "attn_bwd", "rmsnorm", "geglu", "xent", "embed", "other"]
        return {n: (ms[i], fl[i], ln[i]) for i, n in enumerate(names)}

    def t5_profile_launches(self):
        """[(what, family, M, N, K, ms)] of the profiled launches since the last t5_profile_read, in launch order"""
        n = C.c_int32()
        _check(lib().t5_profile_launches(self._h, None, 0, C.byref(n)), self._h)
        buf = (t5_profile_launch * max(n.value, 1))()
        _check(lib().t5_profile_launches(self._h, buf, n.value, C.byref(n)), self._h)
        return [(r.what.decode(), r.family, r.M, r.N, r.K, r.ms) for r in buf[:n.value]]

    def t5_launch_count(self):
        n = C.c_int64()
        _check(lib().t5_launch_count(self._h, C.byref(n)), self._h)
        return n.value

    def t5_set_grad_hook(self, fn):
        """fn(offset, count, rank_weight_ptr, stream_ptr) is called from inside t5_train_step_fwd_bwd as ranges of the
        gradient buffer become final; None removes the hook.  The wrapper object is kept alive by the handle."""
        if fn is None:
            self._grad_hook = GRAD_HOOK()
        else:
            self._grad_hook = GRAD_HOOK(lambda user, off, cnt, w, st: fn(off, cnt, w, st))
        _check(lib().t5_set_grad_hook(self._h, self._grad_hook, None), self._h)

    def t5_device_status(self, workspace):
        _check(lib().t5_device_status(self._h, _ptr(workspace), _stream()), self._h)


def t5_relpos_buckets(bidirectional, num_buckets, max_distance, rel_lo, out):
    _check(lib().t5_relpos_buckets(int(bidirectional), num_buckets, max_distance, rel_lo, out.numel(),
                                   _ptr(out), _stream()))


def t5_xent_zloss(logits, targets, z_loss, W, sums, lse):
    dtype = 0 if logits.dtype == torch.float32 else 1
    n, v = logits.shape
    _check(lib().t5_xent_zloss(dtype, _ptr(logits), _ptr(targets), n, v, z_loss, _ptr(W), _ptr(sums),
                               _ptr(lse), _stream()))


def t5_gemm(impl, M, N, K, alpha, A, lda, a_kmajor, B, ldb, b_kmajor, D, ldd, accumulate=False, sk_flags=None):
    dtype = 0 if A.dtype == torch.float32 else 1
    out_f32 = int(D.dtype == torch.float32)
    _check(lib().t5_gemm(dtype, impl, M, N, K, alpha, _ptr(A), lda, int(a_kmajor), _ptr(B), ldb,
                         int(b_kmajor), _ptr(D), ldd, out_f32, int(accumulate), _ptr(sk_flags), _stream()))


def t5_attention(impl, backward, B, H, Tq, Tk, d_kv, causal, scale, q, k, v, o, lse, code_q, code_k, bias_delta,
                 do=None, dq=None, dk=None, dv=None, delta=None, dbias_delta=None, o32=None):
    """q/k/v/o/do/dq/dk/dv: 2-D tensors (possibly column-sliced views) with rows = tokens."""
    dtype = 0 if q.dtype == torch.float32 else 1

    def ld(t):
        return 0 if t is None else t.stride(0)
    _check(lib().t5_attention(dtype, impl, int(backward), B, H, Tq, Tk, d_kv, int(causal), scale,
                              _ptr(q), ld(q), _ptr(k), ld(k), _ptr(v), ld(v), _ptr(o), ld(o), _ptr(o32), _ptr(lse),
                              _ptr(code_q), _ptr(code_k), _ptr(bias_delta), _ptr(do), ld(do), _ptr(dq), ld(dq),
                              _ptr(dk), ld(dk), _ptr(dv), ld(dv), _ptr(delta), _ptr(dbias_delta), _stream()))


def t5_attention_ds_scratch_bytes(B, H, Tq, Tk):
    n = C.c_int64()
    _check(lib().t5_attention_ds_scratch_bytes(B, H, Tq, Tk, C.byref(n)))
    return n.value


def t5_attention_backward_onepass(B, H, Tq, Tk, d_kv, causal, scale, q, k, v, o, o32, lse, code_q, code_k,
                                  bias_delta, do, dq, dk, dv, delta, dbias_delta, bias_far, ds_scratch):
    """Attention backward that visits the scores once (dK, dV and a stored dS, then dQ from it)."""
    _check(lib().t5_attention_backward_onepass(B, H, Tq, Tk, d_kv, int(causal), scale,
                                               _ptr(q), q.stride(0), _ptr(k), k.stride(0), _ptr(v), v.stride(0),
                                               _ptr(o), o.stride(0), _ptr(o32), _ptr(lse), _ptr(code_q),
                                               _ptr(code_k), _ptr(bias_delta), _ptr(do), do.stride(0),
                                               _ptr(dq), dq.stride(0), _ptr(dk), dk.stride(0), _ptr(dv),
                                               dv.stride(0), _ptr(delta), _ptr(dbias_delta), int(bias_far),
                                               _ptr(ds_scratch), ds_scratch.numel() * ds_scratch.element_size(),
                                               _stream()))


def t5_attention_backward_noalloc(impl, B, H, Tq, Tk, d_kv, causal, scale, q, k, v, o, o32, lse, code_q, code_k,
                                  bias_delta, do, dq, dk, dv, dbias_delta=None):
    """Attention backward whose scratch is built into the library: for callers that cannot allocate
    device memory around the call.  Nothing in this call allocates."""
    dtype = 0 if q.dtype == torch.float32 else 1
    _check(lib().t5_attention_backward_noalloc(dtype, impl, B, H, Tq, Tk, d_kv, int(causal), scale,
                                               _ptr(q), q.stride(0), _ptr(k), k.stride(0), _ptr(v), v.stride(0),
                                               _ptr(o), o.stride(0), _ptr(o32), _ptr(lse), _ptr(code_q),
                                               _ptr(code_k), _ptr(bias_delta), _ptr(do), do.stride(0),
                                               _ptr(dq), dq.stride(0), _ptr(dk), dk.stride(0), _ptr(dv),
                                               dv.stride(0), _ptr(dbias_delta), _stream()))


def t5_kernel_status_word(status):
    """Hands the kernel-level entry points (t5_attention, ..., t5_gemm) a device int32 for their bounded waits
    to report into; None switches reporting off."""
    _check(lib().t5_kernel_status_word(_ptr(status)))


def t5_selftest_bounded_wait(status, limit_cycles):
    """One CTA waits, with the kernels' own bounded wait, on a barrier nothing arrives at; it gives up after
    limit_cycles and leaves code 99 in `status` (device int32)."""
    _check(lib().t5_selftest_bounded_wait(_ptr(status), int(limit_cycles), _stream()))
