"""ctypes binding of the CPU oracle.  TEST INFRASTRUCTURE, NOT PRODUCT.

Argument marshalling only; every number comes out of oracle/dmtd_oracle.c.
"""
import ctypes as C
import os

import numpy as np
import torch

from .build import build

_DT = {"f32": 0, "bf16": 1}


class _Shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "hidden", "n_q_heads", "n_kv_heads",
                                         "head_dim", "intermediate", "vocab")] + \
               [("rope_theta", C.c_double), ("rms_eps", C.c_double), ("weight_dtype", C.c_int32)]


_LAYER_FIELDS = ("input_norm", "q_proj", "k_proj", "v_proj", "q_norm", "k_norm", "o_proj",
                 "post_norm", "gate_proj", "up_proj", "down_proj")


class _LayerW(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _LAYER_FIELDS]


class _Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("final_norm", C.c_void_p), ("layers", C.POINTER(_LayerW))]


class _State(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_known", "lo_len", "up_len", "cycle", "slot",
                                         "n_emitted", "tau", "L_d")]


class _PassRec(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("kind", "lo_begin", "lo_end", "up_begin", "up_end",
                                         "cycle")]


_dp = np.ctypeslib.ndpointer(dtype=np.float64, flags="C_CONTIGUOUS")
_ip = np.ctypeslib.ndpointer(dtype=np.int32, flags="C_CONTIGUOUS")


class OracleLib:
    def __init__(self):
        self.dll = C.CDLL(build())
        d = self.dll
        d.oracle_rmsnorm.argtypes = [_dp, _dp, C.c_double, C.c_int, C.c_int, _dp]
        d.oracle_rmsnorm.restype = None
        d.oracle_rope.argtypes = [_dp, C.c_int, C.c_int, C.c_double]
        d.oracle_rope.restype = None
        d.oracle_attention.argtypes = [_dp, _dp, _dp] + [C.c_int] * 5 + [_dp]
        d.oracle_attention.restype = None
        d.oracle_linear.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, _dp, C.c_int, _dp]
        d.oracle_linear.restype = None
        d.oracle_silu.argtypes = [C.c_double]
        d.oracle_silu.restype = C.c_double
        d.oracle_plt.argtypes = [C.c_int] * 3
        d.oracle_plt.restype = C.c_double
        d.oracle_k_cache.restype = C.POINTER(C.c_double)
        d.oracle_v_cache.restype = C.POINTER(C.c_double)
        d.oracle_k_cache.argtypes = [C.c_void_p, C.c_int32, C.c_int32]
        d.oracle_v_cache.argtypes = [C.c_void_p, C.c_int32, C.c_int32]

    # ---- unit functions
    def rmsnorm(self, x, w, eps):
        x = np.ascontiguousarray(x, np.float64)
        w = np.ascontiguousarray(w, np.float64)
        y = np.empty_like(x)
        rows = x.size // x.shape[-1]
        self.dll.oracle_rmsnorm(x, w, eps, rows, x.shape[-1], y)
        return y

    def rope(self, v, pos, theta):
        v = np.array(v, np.float64, order="C")
        self.dll.oracle_rope(v, v.shape[-1], pos, theta)
        return v

    def attention(self, q, k, v, pos0):
        q = np.ascontiguousarray(q, np.float64)
        k = np.ascontiguousarray(k, np.float64)
        v = np.ascontiguousarray(v, np.float64)
        R, nq, d = q.shape
        nkv = k.shape[1]
        assert k.shape[0] == pos0 + R and v.shape == k.shape
        out = np.empty_like(q)
        self.dll.oracle_attention(q, k, v, R, pos0, nq, nkv, d, out)
        return out

    def linear(self, W, x):
        """W: torch tensor [out, in] fp32 or bf16; x: [rows, in] float64."""
        Wp, dt, keep = _tensor_ptr(W)
        x = np.ascontiguousarray(x, np.float64)
        rows = x.shape[0]
        y = np.empty((rows, W.shape[0]), np.float64)
        self.dll.oracle_linear(Wp, dt, W.shape[0], W.shape[1], x, rows, y)
        return y

    def silu(self, t):
        return self.dll.oracle_silu(float(t))

    def anchor_mask(self, p, P, tau):
        return int(self.dll.oracle_anchor_mask(int(p), int(P), int(tau)))

    def plt(self, L, L_d, tau):
        return self.dll.oracle_plt(L, L_d, tau)

    def philox(self, ctr, key):
        c = (C.c_uint32 * 4)(*ctr)
        k = (C.c_uint32 * 2)(*key)
        out = (C.c_uint32 * 4)()
        self.dll.oracle_philox4x32(c, k, out)
        return [int(v) for v in out]

    def sample_token(self, z, temperature, seed, position, sequence):
        z = np.ascontiguousarray(z, np.float64)
        self.dll.oracle_sample_token.argtypes = [_dp, C.c_int, C.c_double, C.c_uint64, C.c_int32, C.c_int32]
        self.dll.oracle_sample_token.restype = C.c_int32
        return int(self.dll.oracle_sample_token(z, z.size, float(temperature), int(seed), int(position), int(sequence)))


_lib = None


def lib() -> OracleLib:
    global _lib
    if _lib is None:
        _lib = OracleLib()
    return _lib


def _tensor_ptr(t: torch.Tensor):
    assert t.device.type == "cpu" and t.is_contiguous()
    if t.dtype == torch.bfloat16:
        return C.c_void_p(t.data_ptr()), 1, t
    if t.dtype == torch.float32:
        return C.c_void_p(t.data_ptr()), 0, t
    raise TypeError(t.dtype)


def _pack(shape, weights):
    """Build the C structs; returns (shape_struct, weights_struct, keepalive)."""
    s = _Shape(shape.n_layers, shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
               shape.intermediate, shape.vocab, shape.rope_theta, shape.rms_eps,
               _DT[shape.dtype])
    keep = []
    want = {"f32": torch.float32, "bf16": torch.bfloat16}[shape.dtype]

    def p(t):
        assert t.dtype == want, (t.dtype, want)
        t = t.contiguous()
        keep.append(t)
        return t.data_ptr()

    n = len(weights["layers"])
    arr = (_LayerW * n)()
    for i, lw in enumerate(weights["layers"]):
        for f in _LAYER_FIELDS:
            setattr(arr[i], f, p(lw[f]))
    w = _Weights(p(weights["embed"]), p(weights["final_norm"]), arr)
    keep.append(arr)
    return s, w, keep


class Oracle:
    """One oracle context (Section 2.2's schedule on the CPU)."""

    def __init__(self, shape, weights, L_d, tau, max_batch=1, max_seq=256, literal_sum=False, L_e=0):
        self.lib = lib()
        self.shape = shape
        self._s, self._w, self._keep = _pack(shape, weights)
        self._ctx = C.c_void_p()
        rc = self.lib.dll.oracle_create(C.byref(self._s), L_d, tau, max_batch, max_seq,
                                        C.byref(self._w), C.byref(self._ctx))
        if rc:
            raise ValueError(f"oracle_create failed: {rc}")
        self.max_seq, self.max_batch = max_seq, max_batch
        self.B = 0
        if literal_sum:
            self.lib.dll.oracle_set_literal_sum(self._ctx, 1)
        if L_e:
            rc = self.lib.dll.oracle_set_encoding_layers(self._ctx, L_e)
            if rc:
                raise ValueError(f"oracle_set_encoding_layers failed: {rc}")

    def close(self):
        if self._ctx:
            self.lib.dll.oracle_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def reset(self):
        self.lib.dll.oracle_reset(self._ctx)

    def set_tau(self, tau):
        return self.lib.dll.oracle_set_tau(self._ctx, tau)

    def set_sampling(self, temperature, seed):
        self.lib.dll.oracle_set_sampling.argtypes = [C.c_void_p, C.c_double, C.c_uint64]
        return self.lib.dll.oracle_set_sampling(self._ctx, float(temperature), int(seed))

    def prefill(self, prompt, forced_first=None, want_logits=True):
        prompt = np.ascontiguousarray(prompt, np.int32)
        B, P = prompt.shape
        self.B = B
        tok = np.zeros(B, np.int32)
        logits = np.empty((B, self.shape.vocab), np.float64) if want_logits else None
        ff = None if forced_first is None else np.ascontiguousarray(forced_first, np.int32)
        rc = self.lib.dll.oracle_prefill(
            self._ctx, prompt.ctypes.data_as(C.c_void_p), B, P,
            None if ff is None else ff.ctypes.data_as(C.c_void_p),
            tok.ctypes.data_as(C.c_void_p),
            None if logits is None else logits.ctypes.data_as(C.c_void_p))
        if rc:
            raise RuntimeError(f"oracle_prefill: {rc}")
        return tok, logits

    def decode_cycle(self, max_new, want_logits=True):
        tau = self.state()["tau"]
        toks = np.zeros((self.B, tau), np.int32)
        n_out = C.c_int32(0)
        logits = np.empty((tau, self.B, self.shape.vocab), np.float64) if want_logits else None
        rc = self.lib.dll.oracle_decode_cycle(
            self._ctx, max_new, toks.ctypes.data_as(C.c_void_p), C.byref(n_out),
            None if logits is None else logits.ctypes.data_as(C.c_void_p))
        n = n_out.value
        return rc, toks[:, :n], (None if logits is None else logits[:n])

    def decode_forced(self, forced, want_logits=True):
        forced = np.ascontiguousarray(forced, np.int32)
        B, n = forced.shape
        assert B == self.B
        logits = np.empty((n, B, self.shape.vocab), np.float64) if want_logits else None
        am = np.zeros((n, B), np.int32)
        rc = self.lib.dll.oracle_decode_forced(
            self._ctx, forced.ctypes.data_as(C.c_void_p), n,
            None if logits is None else logits.ctypes.data_as(C.c_void_p),
            am.ctypes.data_as(C.c_void_p))
        if rc:
            raise RuntimeError(f"oracle_decode_forced: {rc}")
        return logits, am

    def step_layers(self, l0, l1, hidden, pos0):
        hidden = np.array(hidden, np.float64, order="C")
        B, R, _ = hidden.shape
        rc = self.lib.dll.oracle_step_layers(self._ctx, l0, l1,
                                             hidden.ctypes.data_as(C.c_void_p), B, R, pos0)
        if rc:
            raise RuntimeError(f"oracle_step_layers: {rc}")
        return hidden

    def state(self):
        s = _State()
        self.lib.dll.oracle_get_state(self._ctx, C.byref(s))
        return {n: getattr(s, n) for n, _ in _State._fields_}

    def trace(self):
        n = self.lib.dll.oracle_get_trace(self._ctx, None, 0)
        arr = (_PassRec * max(n, 1))()
        self.lib.dll.oracle_get_trace(self._ctx, arr, n)
        return [{f: getattr(arr[i], f) for f, _ in _PassRec._fields_} for i in range(n)]

    def layer_counters(self):
        L = self.shape.n_layers
        calls = np.zeros(L, np.int64)
        rows = np.zeros(L, np.int64)
        self.lib.dll.oracle_get_layer_counters(self._ctx, calls.ctypes.data_as(C.c_void_p),
                                               rows.ctypes.data_as(C.c_void_p))
        return calls, rows

    def kv_cache(self, layer, b, n_pos):
        """(K, V) of one layer and sequence as float64 [n_pos, nkv, d] copies."""
        nkv, d = self.shape.n_kv_heads, self.shape.head_dim
        out = []
        for fn in (self.lib.dll.oracle_k_cache, self.lib.dll.oracle_v_cache):
            ptr = fn(self._ctx, layer, b)
            a = np.ctypeslib.as_array(ptr, shape=(self.max_seq, nkv, d))
            out.append(a[:n_pos].copy())
        return out


def _set_kv(self, layer, b, k, v):
    """Overwrite the first positions of one layer's cache of sequence b: k, v [n_pos, nkv, d]."""
    nkv, d = self.shape.n_kv_heads, self.shape.head_dim
    for fn, src in ((self.lib.dll.oracle_k_cache, k), (self.lib.dll.oracle_v_cache, v)):
        a = np.ctypeslib.as_array(fn(self._ctx, layer, b), shape=(self.max_seq, nkv, d))
        a[: src.shape[0]] = src


Oracle.set_kv = _set_kv


def vanilla_generate(shape, weights, prompt, n_new, forced=None):
    """Plain full-recompute autoregressive decoding of one sequence.
    Returns (tokens [P+n_new], logits [n_new, V], argmax [n_new])."""
    l = lib()
    s, w, keep = _pack(shape, weights)
    prompt = np.asarray(prompt, np.int32).reshape(-1)
    P = prompt.size
    toks = np.zeros(P + n_new, np.int32)
    toks[:P] = prompt
    logits = np.empty((n_new, shape.vocab), np.float64)
    am = np.zeros(n_new, np.int32)
    f = None if forced is None else np.ascontiguousarray(forced, np.int32)
    rc = l.dll.oracle_vanilla_generate(
        C.byref(s), C.byref(w), toks.ctypes.data_as(C.c_void_p), P, n_new,
        None if f is None else f.ctypes.data_as(C.c_void_p),
        logits.ctypes.data_as(C.c_void_p), am.ctypes.data_as(C.c_void_p))
    if rc:
        raise RuntimeError(f"oracle_vanilla_generate: {rc}")
    del keep
    return toks, logits, am


def masked_parallel_forward(shape, weights, L_d, tau, tokens, P, literal_sum=False, L_e=0):
    """Eq. 1-5 in one pass over `tokens`; logits at positions P-1 .. n-1."""
    l = lib()
    s, w, keep = _pack(shape, weights)
    tokens = np.ascontiguousarray(tokens, np.int32).reshape(-1)
    n = tokens.size
    out = np.empty((n - (P - 1), shape.vocab), np.float64)
    rc = l.dll.oracle_masked_parallel_forward_exdy(
        C.byref(s), C.byref(w), L_e, L_d, tau, tokens.ctypes.data_as(C.c_void_p), n, P,
        1 if literal_sum else 0, out.ctypes.data_as(C.c_void_p))
    if rc:
        raise RuntimeError(f"oracle_masked_parallel_forward: {rc}")
    del keep
    return out
