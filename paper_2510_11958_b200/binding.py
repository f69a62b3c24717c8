"""ctypes binding of libdmtd_b200.so (see include/dmtd.h for the contract of every call).

torch is used for device memory and the CUDA stream only; every step of the decode path
runs inside the library's kernels.
"""
import ctypes as C
import os
import re

import torch

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(HERE)
_DT = {"f32": 0, "bf16": 1, "f16": 2}


class DmtdError(RuntimeError):
    def __init__(self, status, message):
        super().__init__(f"dmtd status {status}: {message}")
        self.status = status


class _Shape(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_layers", "hidden", "n_q_heads", "n_kv_heads",
                                         "head_dim", "intermediate", "vocab")] + \
               [("rope_theta", C.c_float), ("rms_eps", C.c_float)] + \
               [(n, C.c_int32) for n in ("weight_dtype", "kv_dtype", "tied_lm_head")]


_LAYER_FIELDS = ("input_norm", "q_proj", "k_proj", "v_proj", "q_norm", "k_norm", "o_proj",
                 "post_norm", "gate_proj", "up_proj", "down_proj")


class _LayerW(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in _LAYER_FIELDS]


class _Weights(C.Structure):
    _fields_ = [("embed", C.c_void_p), ("final_norm", C.c_void_p), ("lm_head", C.c_void_p),
                ("layers", C.POINTER(_LayerW))]


class _State(C.Structure):
    _fields_ = [(n, C.c_int32) for n in ("n_known", "lo_len", "up_len", "cycle", "slot",
                                         "n_emitted", "tau", "L_d")]


STATUS = {"OK": 0, "INVALID_ARG": -1, "SHAPE": -2, "STATE": -3, "CAPACITY": -4, "CUDA": -5,
          "TIMEOUT": -6, "UNSUPPORTED": -7}


def library_path() -> str:
    return os.path.join(HERE, "libdmtd_b200.so")


def declared_symbols():
    """Names of the functions include/dmtd.h declares."""
    text = open(os.path.join(ROOT, "include", "dmtd.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(dmtd_[a-z_0-9]+)\s*\(", text)))


_dll = None


def load_library():
    """Load the CUDA library; raises if it has not been built (no fallback exists)."""
    global _dll
    if _dll is not None:
        return _dll
    path = library_path()
    if not os.path.exists(path):
        raise DmtdError(STATUS["UNSUPPORTED"],
                        f"{path} not found: build it with `python -m paper_2510_11958_b200.build`")
    d = C.CDLL(path)
    vp, i32, i64 = C.c_void_p, C.c_int32, C.c_int64
    sig = {
        "dmtd_create": [C.POINTER(_Shape), i32, i32, i32, i32, C.POINTER(_Weights), vp, C.POINTER(vp)],
        "dmtd_reset": [vp],
        "dmtd_prefill": [vp, vp, i32, i32, vp, vp, vp],
        "dmtd_decode_cycle": [vp, i32, vp, C.POINTER(i32)],
        "dmtd_decode_forced": [vp, vp, i32, vp, vp],
        "dmtd_step_layers": [vp, i32, i32, vp, i32, i32, i32],
        "dmtd_masked_forward": [vp, vp, i32, i32, i32, vp],
        "dmtd_prefill_host": [vp, vp, i32, i32, vp],
        "dmtd_decode_cycle_host": [vp, i32, vp, C.POINTER(i32)],
        "dmtd_get_state": [vp, C.POINTER(_State)],
        "dmtd_get_device_state": [vp, C.POINTER(_State)],
        "dmtd_set_tau": [vp, i32],
        "dmtd_set_option": [vp, C.c_char_p, i64],
        "dmtd_get_kv": [vp, i32, C.POINTER(vp), C.POINTER(vp)],
        "dmtd_get_launch_count": [vp, C.POINTER(i64)],
        "dmtd_debug_set_error_word": [vp, i32],
        "dmtd_attention_decode": [vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, i32, vp, C.c_size_t, vp, vp],
        "dmtd_attention_decode_static": [vp, vp, vp, i32, i32, i32, i32, i32, i32, i32, i32, vp, vp],
    }
    for name, args in sig.items():
        fn = getattr(d, name)
        fn.argtypes = args
        fn.restype = C.c_int
    d.dmtd_attention_scratch_bytes.argtypes = [i32, i32, i32, i32, i32]
    d.dmtd_attention_scratch_bytes.restype = C.c_size_t
    d.dmtd_destroy.argtypes = [vp]
    d.dmtd_destroy.restype = None
    d.dmtd_status_str.argtypes = [C.c_int]
    d.dmtd_status_str.restype = C.c_char_p
    d.dmtd_last_error.argtypes = [vp]
    d.dmtd_last_error.restype = C.c_char_p
    _dll = d
    return d


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


class Dmtd:
    """One decode context on the current CUDA device and torch's current stream."""

    def __init__(self, shape, weights, L_d, tau, max_batch=1, max_seq=1024, kv_dtype=None):
        self._ctx = C.c_void_p()
        self.dll = load_library()
        if not torch.cuda.is_available():
            raise DmtdError(STATUS["CUDA"], "no CUDA device: the DMTD decode path runs only on a GPU")
        self.shape = shape
        kv_dtype = kv_dtype or shape.dtype
        s = _Shape(shape.n_layers, shape.hidden, shape.n_q_heads, shape.n_kv_heads, shape.head_dim,
                   shape.intermediate, shape.vocab, shape.rope_theta, shape.rms_eps,
                   _DT[shape.dtype], _DT[kv_dtype], 1)
        want = {"f32": torch.float32, "bf16": torch.bfloat16}[shape.dtype]

        def p(t):
            assert t.is_cuda and t.dtype == want and t.is_contiguous(), (t.device, t.dtype)
            return t.data_ptr()

        n = len(weights["layers"])
        arr = (_LayerW * n)()
        for i, lw in enumerate(weights["layers"]):
            for f in _LAYER_FIELDS:
                setattr(arr[i], f, p(lw[f]))
        w = _Weights(p(weights["embed"]), p(weights["final_norm"]), None, arr)
        self.stream = torch.cuda.current_stream()
        rc = self.dll.dmtd_create(C.byref(s), L_d, tau, max_batch, max_seq, C.byref(w),
                                  C.c_void_p(self.stream.cuda_stream), C.byref(self._ctx))
        if rc:
            msg = self.dll.dmtd_last_error(None).decode()
            self._ctx = C.c_void_p()
            raise DmtdError(rc, msg)
        self.max_batch, self.max_seq, self.B = max_batch, max_seq, 0
        self.device = weights["embed"].device

    # -- helpers
    def _check(self, rc, allow=()):
        if rc and rc not in allow:
            raise DmtdError(rc, self.dll.dmtd_last_error(self._ctx).decode())
        return rc

    def close(self):
        if getattr(self, "_ctx", None):
            self.dll.dmtd_destroy(self._ctx)
            self._ctx = C.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # -- the calls of include/dmtd.h
    def reset(self):
        self._check(self.dll.dmtd_reset(self._ctx))

    def prefill(self, prompt, forced_first=None, want_logits=False):
        """prompt: cuda int32 [B, P].  Returns (token [B] int32, logits [B, V] float32 or None)."""
        assert prompt.is_cuda and prompt.dtype == torch.int32 and prompt.is_contiguous()
        B, P = prompt.shape
        tok = torch.empty(B, dtype=torch.int32, device=prompt.device)
        logits = torch.empty(B, self.shape.vocab, dtype=torch.float32, device=prompt.device) if want_logits else None
        self._check(self.dll.dmtd_prefill(self._ctx, _ptr(prompt), B, P, _ptr(forced_first), _ptr(tok), _ptr(logits)))
        self.B = B
        return tok, logits

    def decode_cycle(self, max_new, out_tokens=None, allow_capacity=False):
        """Returns (status, n_out, out_tokens [B, tau] with the first n_out columns valid)."""
        tau = self.state()["tau"]
        if out_tokens is None:
            out_tokens = torch.zeros(self.B, tau, dtype=torch.int32, device=self.device)
        n = C.c_int32(0)
        rc = self._check(self.dll.dmtd_decode_cycle(self._ctx, max_new, _ptr(out_tokens), C.byref(n)),
                         allow=(STATUS["CAPACITY"],) if allow_capacity else ())
        return rc, n.value, out_tokens

    def decode_forced(self, forced, want_logits=True):
        """forced: cuda int32 [B, n].  Returns (logits [n, B, V] or None, argmax [n, B])."""
        assert forced.is_cuda and forced.dtype == torch.int32 and forced.is_contiguous()
        B, n = forced.shape
        logits = torch.empty(n, B, self.shape.vocab, dtype=torch.float32, device=forced.device) if want_logits else None
        am = torch.empty(n, B, dtype=torch.int32, device=forced.device)
        self._check(self.dll.dmtd_decode_forced(self._ctx, _ptr(forced), n, _ptr(logits), _ptr(am)))
        return logits, am

    def step_layers(self, l0, l1, hidden, pos0):
        """hidden: cuda float32 [B, R, H], updated in place."""
        assert hidden.is_cuda and hidden.dtype == torch.float32 and hidden.is_contiguous()
        B, R, _ = hidden.shape
        self._check(self.dll.dmtd_step_layers(self._ctx, l0, l1, _ptr(hidden), B, R, pos0))
        return hidden

    def masked_forward(self, tokens, P):
        """tokens: cuda int32 [B, n].  Returns logits [B, n - (P-1), V] of positions P-1 .. n-1."""
        assert tokens.is_cuda and tokens.dtype == torch.int32 and tokens.is_contiguous()
        B, n = tokens.shape
        out = torch.empty(B, n - (P - 1), self.shape.vocab, dtype=torch.float32, device=tokens.device)
        self._check(self.dll.dmtd_masked_forward(self._ctx, _ptr(tokens), B, n, P, _ptr(out)))
        return out

    def prefill_host(self, prompt_host):
        """prompt_host: CPU int32 [B, P] (pinned for speed).  Returns the first tokens as a CPU tensor."""
        assert not prompt_host.is_cuda and prompt_host.dtype == torch.int32 and prompt_host.is_contiguous()
        B, P = prompt_host.shape
        out = torch.empty(B, dtype=torch.int32)
        self._check(self.dll.dmtd_prefill_host(self._ctx, _ptr(prompt_host), B, P, _ptr(out)))
        self.B = B
        return out

    def decode_cycle_host(self, max_new, out_host):
        """out_host: CPU int32 [B, tau] (pinned for speed).  Returns n_out."""
        n = C.c_int32(0)
        self._check(self.dll.dmtd_decode_cycle_host(self._ctx, max_new, _ptr(out_host), C.byref(n)))
        return n.value

    def state(self):
        s = _State()
        self._check(self.dll.dmtd_get_state(self._ctx, C.byref(s)))
        return {n: getattr(s, n) for n, _ in _State._fields_}

    def device_state(self):
        s = _State()
        self._check(self.dll.dmtd_get_device_state(self._ctx, C.byref(s)))
        return {n: getattr(s, n) for n, _ in _State._fields_}

    def set_tau(self, tau):
        self._check(self.dll.dmtd_set_tau(self._ctx, tau))

    def set_sampling(self, temperature, seed):
        self.dll.dmtd_set_sampling.argtypes = [C.c_void_p, C.c_float, C.c_uint64]
        self.dll.dmtd_set_sampling.restype = C.c_int
        self._check(self.dll.dmtd_set_sampling(self._ctx, float(temperature), int(seed)))

    def set_option(self, name, value):
        self._check(self.dll.dmtd_set_option(self._ctx, name.encode(), int(value)))

    def kv(self, layer):
        """(K, V) of one layer as torch views [max_batch, n_kv_heads, max_seq, head_dim]."""
        k, v = C.c_void_p(), C.c_void_p()
        self._check(self.dll.dmtd_get_kv(self._ctx, layer, C.byref(k), C.byref(v)))
        return k.value, v.value

    def debug_set_error_word(self, word):
        self._check(self.dll.dmtd_debug_set_error_word(self._ctx, int(word)))

    def memory_info(self):
        """Device bytes held by the context: weights (two layouts), KV cache, workspace."""
        class _Mem(C.Structure):
            _fields_ = [(n, C.c_size_t) for n in ("weight_stream_bytes", "weight_block_bytes", "kv_cache_bytes",
                                                  "workspace_bytes")]
        m = _Mem()
        self.dll.dmtd_get_memory_info.argtypes = [C.c_void_p, C.POINTER(_Mem)]
        self.dll.dmtd_get_memory_info.restype = C.c_int
        self._check(self.dll.dmtd_get_memory_info(self._ctx, C.byref(m)))
        return {n: getattr(m, n) for n, _ in _Mem._fields_}

    def launch_count(self):
        n = C.c_int64(0)
        self._check(self.dll.dmtd_get_launch_count(self._ctx, C.byref(n)))
        return n.value


def _kv_code(t):
    return {torch.float32: 0, torch.bfloat16: 1, torch.float16: 2}[t.dtype]


def attention_decode(q, k, v, pos0, scratch=None):
    """Split-KV attention of the R new rows of each sequence (dmtd_attention_decode).

    q: cuda float32 [B, R, nq, D]; k, v: cuda [B, nkv, max_seq, D] float32 or bfloat16, with the
    new rows' K and V already at positions pos0 .. pos0+R-1.  Returns out [B, R, nq, D] float32.
    `scratch` is a cuda uint8 tensor of at least attention_scratch_bytes(...) bytes; one is
    allocated through torch if none is given.
    """
    dll = load_library()
    assert q.is_cuda and q.dtype == torch.float32 and q.is_contiguous()
    assert k.is_cuda and v.is_cuda and k.is_contiguous() and v.is_contiguous() and k.dtype == v.dtype
    B, R, nq, D = q.shape
    _, nkv, max_seq, _ = k.shape
    need = dll.dmtd_attention_scratch_bytes(B, R, nq, D, pos0 + R)
    if scratch is None:
        scratch = torch.empty(max(need, 256), dtype=torch.uint8, device=q.device)
    out = torch.empty_like(q)
    rc = dll.dmtd_attention_decode(_ptr(q), _ptr(k), _ptr(v), _kv_code(k), B, R, nq, nkv, D, max_seq, pos0,
                                   _ptr(scratch), scratch.numel(), _ptr(out),
                                   C.c_void_p(torch.cuda.current_stream().cuda_stream))
    if rc:
        raise DmtdError(rc, dll.dmtd_last_error(None).decode())
    return out


ATTENTION_STATIC_SCRATCH_BYTES = 4 << 20


def attention_decode_static(q, k, v, pos0, out):
    """dmtd_attention_decode_static: the same attention for callers that cannot allocate.

    Nothing is allocated here or in the library: the caller passes `out` (cuda float32, shape of
    q) and the partial results use the library's built-in array of ATTENTION_STATIC_SCRATCH_BYTES
    bytes, shared by every call in the process.  Raises DmtdError (CAPACITY) if the problem
    needs more scratch than that.
    """
    dll = load_library()
    assert q.is_cuda and q.dtype == torch.float32 and q.is_contiguous()
    assert out.is_cuda and out.dtype == torch.float32 and out.is_contiguous() and out.shape == q.shape
    assert k.is_cuda and v.is_cuda and k.is_contiguous() and v.is_contiguous() and k.dtype == v.dtype
    B, R, nq, D = q.shape
    _, nkv, max_seq, _ = k.shape
    rc = dll.dmtd_attention_decode_static(_ptr(q), _ptr(k), _ptr(v), _kv_code(k), B, R, nq, nkv, D, max_seq, pos0,
                                          _ptr(out), C.c_void_p(torch.cuda.current_stream().cuda_stream))
    if rc:
        raise DmtdError(rc, dll.dmtd_last_error(None).decode())
    return out
