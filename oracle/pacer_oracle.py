"""ctypes front-end of the CPU oracle (``pacer_oracle.c``).

TEST INFRASTRUCTURE: only the tests, the smoke check and the benchmark's
cpu-baseline leg may import this.  It imports nothing from the CUDA package.
Weights are handed over as torch CPU tensors (bf16 or fp32); every result comes
back as a numpy array of float64 / int32.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess
from typing import Dict, Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "pacer_oracle.c")
_LIB = os.path.join(_HERE, "libpacer_oracle.so")


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP).  Returns the library path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-fopenmp", "-fPIC", "-shared", "-std=c11", "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


class Model(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32),
                ("n_kv_heads", C.c_int32), ("d_ffn", C.c_int32), ("vocab", C.c_int32),
                ("rope_theta", C.c_float), ("rms_eps", C.c_float),
                ("wdtype", C.c_int32), ("n_posemb", C.c_int32),
                ("embed", C.c_void_p), ("wqkv", C.c_void_p), ("wo", C.c_void_p), ("wgate", C.c_void_p),
                ("wup", C.c_void_p), ("wdown", C.c_void_p), ("norm1", C.c_void_p), ("norm2", C.c_void_p),
                ("normf", C.c_void_p), ("head", C.c_void_p), ("head_b", C.c_void_p), ("posemb", C.c_void_p),
                ("succ", C.c_void_p), ("succ_bias", C.c_float), ("pad_", C.c_int32)]


class Params(C.Structure):
    _fields_ = [("b", C.c_int32), ("gamma_cap", C.c_int32), ("t0", C.c_float), ("rho", C.c_float),
                ("criterion", C.c_int32), ("mode", C.c_int32), ("seed", C.c_uint64),
                ("seq_id", C.c_int32), ("use_posemb", C.c_int32), ("scope", C.c_int32), ("pad_", C.c_int32)]


class Stats(C.Structure):
    _fields_ = [("n_draft_fwd", C.c_int64), ("n_mb_calls", C.c_int64), ("n_target_fwd", C.c_int64),
                ("n_steps", C.c_int64), ("min_margin_target", C.c_double), ("min_margin_draft", C.c_double),
                ("min_margin_stop", C.c_double), ("min_margin_accept", C.c_double)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


_lib = None


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        L = _lib
        L.orc_cache_new.restype = C.c_void_p
        L.orc_cache_new.argtypes = [C.POINTER(Model), C.c_int]
        L.orc_cache_free.argtypes = [C.c_void_p]
        L.orc_cache_len.argtypes = [C.c_void_p]
        L.orc_cache_truncate.argtypes = [C.c_void_p, C.c_int]
        L.orc_forward.argtypes = [C.POINTER(Model), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int,
                                  C.c_void_p, C.c_void_p]
        L.orc_forward_scoped.argtypes = [C.POINTER(Model), C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int,
                                         C.c_void_p, C.c_void_p]
        L.orc_linear.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_void_p, C.c_int, C.c_void_p]
        L.orc_philox4x32_10.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_uniform.restype = C.c_double
        L.orc_uniform.argtypes = [C.c_uint64, C.c_uint32, C.c_uint32, C.c_uint32, C.c_uint32]
        L.orc_accept_rule.argtypes = [C.c_void_p, C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_uint64,
                                      C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p]
        L.orc_new.restype = C.c_void_p
        L.orc_new.argtypes = [C.POINTER(Model), C.POINTER(Model), C.POINTER(Model), C.c_int, C.POINTER(Params)]
        L.orc_free.argtypes = [C.c_void_p]
        L.orc_prefill.argtypes = [C.c_void_p, C.c_void_p, C.c_int]
        L.orc_draft_block.argtypes = [C.c_void_p]
        L.orc_preverify.restype = C.c_double
        L.orc_preverify.argtypes = [C.c_void_p]
        L.orc_verify.argtypes = [C.c_void_p]
        L.orc_accept.argtypes = [C.c_void_p]
        L.orc_generate_pacer.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.POINTER(Stats)]
        L.orc_generate_sd.argtypes = [C.POINTER(Model), C.POINTER(Model), C.c_void_p, C.c_int, C.c_int, C.c_int,
                                      C.c_int, C.c_uint64, C.c_int, C.c_int, C.c_void_p, C.c_void_p, C.c_void_p,
                                      C.POINTER(Stats)]
        L.orc_generate_sched.argtypes = [C.POINTER(Model), C.POINTER(Model), C.c_void_p, C.c_int, C.c_int, C.c_void_p,
                                         C.c_int, C.c_int, C.c_uint64, C.c_int, C.c_int, C.c_void_p, C.c_void_p,
                                         C.c_void_p, C.POINTER(Stats)]
        L.orc_generate_ar.argtypes = [C.POINTER(Model), C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_uint64,
                                      C.c_int, C.c_int, C.c_void_p, C.c_void_p]
        for name in ("orc_get_P", "orc_get_gamma", "orc_get_drafting", "orc_get_last_n", "orc_get_last_next",
                     "orc_get_n_pend"):
            getattr(L, name).argtypes = [C.c_void_p]
        L.orc_get_t_k.restype = C.c_float
        L.orc_get_t_k.argtypes = [C.c_void_p]
        L.orc_get_len.argtypes = [C.c_void_p, C.c_int]
        for name in ("orc_get_x", "orc_get_y", "orc_get_alpha", "orc_get_plogits", "orc_get_qlogits",
                     "orc_get_hpend"):
            getattr(L, name).restype = C.c_void_p
            getattr(L, name).argtypes = [C.c_void_p]
        L.orc_get_stats.argtypes = [C.c_void_p, C.POINTER(Stats)]
        L.orc_set_seed.argtypes = [C.c_void_p, C.c_uint64, C.c_int]
        L.orc_set_alpha_override.argtypes = [C.c_void_p, C.c_void_p, C.c_int]
        L.orc_get_cache.restype = C.c_void_p
        L.orc_get_cache.argtypes = [C.c_void_p, C.c_int]
        L.orc_cache_k.restype = C.c_void_p
        L.orc_cache_k.argtypes = [C.c_void_p]
        L.orc_cache_v.restype = C.c_void_p
        L.orc_cache_v.argtypes = [C.c_void_p]
    return _lib


def _ptr(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


class OracleModel:
    """Owns host copies of one model's tensors and the C struct that points at them.

    `shape` is any object with n_layers, d_model, n_heads, n_kv_heads, d_ffn,
    vocab, rope_theta, rms_eps.  `tensors` maps names to torch CPU tensors, all
    bf16 or all fp32."""

    def __init__(self, shape, tensors: Dict[str, torch.Tensor], succ: Optional[torch.Tensor] = None,
                 succ_bias: float = 0.0):
        self.shape = shape
        dts = {t.dtype for t in tensors.values()}
        assert len(dts) == 1, "one dtype per model"
        dt = dts.pop()
        self.keep = {}
        for k, t in tensors.items():
            t = t.detach().cpu().contiguous()
            if dt == torch.bfloat16:
                self.keep[k] = t.view(torch.int16).numpy()
            elif dt == torch.float32:
                self.keep[k] = t.numpy()
            else:
                raise TypeError(dt)
        self.succ = None if succ is None else np.ascontiguousarray(succ.cpu().numpy().astype(np.int32))
        m = Model()
        m.n_layers, m.d_model, m.n_heads = shape.n_layers, shape.d_model, shape.n_heads
        m.n_kv_heads, m.d_ffn, m.vocab = shape.n_kv_heads, shape.d_ffn, shape.vocab
        m.rope_theta, m.rms_eps = shape.rope_theta, shape.rms_eps
        m.wdtype = 1 if dt == torch.bfloat16 else 0
        for k in ("embed", "wqkv", "wo", "wgate", "wup", "wdown", "norm1", "norm2", "normf", "head", "head_b",
                  "posemb"):
            setattr(m, k, _ptr(self.keep.get(k)))
        m.n_posemb = 0 if "posemb" not in self.keep else self.keep["posemb"].shape[0]
        m.succ = _ptr(self.succ)
        m.succ_bias = succ_bias
        self.c = m

    def ref(self):
        return C.byref(self.c)


class Cache:
    def __init__(self, model: OracleModel, max_ctx: int):
        self.model = model
        self.max_ctx = max_ctx
        self.h = lib().orc_cache_new(model.ref(), max_ctx)

    def __del__(self):
        if getattr(self, "h", None) and _lib is not None:
            _lib.orc_cache_free(self.h)
            self.h = None

    @property
    def len(self):
        return lib().orc_cache_len(self.h)

    def truncate(self, n):
        lib().orc_cache_truncate(self.h, n)

    def kv(self):
        """(k, v) float64 views [L][max_ctx][Hkv*hd] of the cache memory."""
        s = self.model.shape
        shp = (s.n_layers, self.max_ctx, s.n_kv_heads * (s.d_model // s.n_heads))
        n = int(np.prod(shp))
        k = np.ctypeslib.as_array(C.cast(lib().orc_cache_k(self.h), C.POINTER(C.c_double)), (n,)).reshape(shp)
        v = np.ctypeslib.as_array(C.cast(lib().orc_cache_v(self.h), C.POINTER(C.c_double)), (n,)).reshape(shp)
        return k, v


def forward(model: OracleModel, cache: Cache, tokens=None, x_in=None, pos0: Optional[int] = None,
            want_hidden=True, want_logits=True, key_start: int = 0):
    """Decoder forward on n new rows; returns (hidden [n][d], logits [n][V]).  key_start > 0 restricts the
    attention context to the cache positions key_start.. (a row before key_start sees itself only)."""
    if tokens is not None:
        tok = np.ascontiguousarray(np.asarray(tokens, dtype=np.int32))
        n = tok.shape[0]
        xin = None
    else:
        xin = np.ascontiguousarray(np.asarray(x_in, dtype=np.float64))
        n = xin.shape[0]
        tok = None
    if pos0 is None:
        pos0 = cache.len
    s = model.shape
    hid = np.empty((n, s.d_model), np.float64) if want_hidden else None
    lg = np.empty((n, s.vocab), np.float64) if (want_logits and model.c.head) else None
    if key_start:
        lib().orc_forward_scoped(model.ref(), cache.h, _ptr(tok), _ptr(xin), n, pos0, key_start, _ptr(hid), _ptr(lg))
    else:
        lib().orc_forward(model.ref(), cache.h, _ptr(tok), _ptr(xin), n, pos0, _ptr(hid), _ptr(lg))
    return hid, lg


def linear(w: torch.Tensor, x: np.ndarray) -> np.ndarray:
    """y[r][o] = sum_k w[o][k] x[r][k] with the oracle's weight decoding."""
    w = w.detach().cpu().contiguous()
    if w.dtype == torch.bfloat16:
        wn, dt = w.view(torch.int16).numpy(), 1
    else:
        wn, dt = w.float().numpy(), 0
    x = np.ascontiguousarray(x, dtype=np.float64)
    N, K = wn.shape
    y = np.empty((x.shape[0], N), np.float64)
    lib().orc_linear(_ptr(wn), dt, N, K, _ptr(x), x.shape[0], _ptr(y))
    return y


def philox(ctr, key):
    c = np.asarray(ctr, dtype=np.uint32)
    k = np.asarray(key, dtype=np.uint32)
    o = np.zeros(4, np.uint32)
    lib().orc_philox4x32_10(_ptr(c), _ptr(k), _ptr(o))
    return o


def uniform(seed, v, pos, seq, tag):
    return lib().orc_uniform(seed, v, pos, seq, tag)


def accept_rule(plog, qlog, y, mode, seed=0, pos_first=0, seq=0):
    """Eq. 5 on explicit logits.  Returns (n, next, margin_target, margin_accept)."""
    plog = np.ascontiguousarray(plog, dtype=np.float64)
    gamma, V = plog.shape[0] - 1, plog.shape[1]
    qlog = np.ascontiguousarray(qlog, dtype=np.float64).reshape(gamma, V)
    y = np.ascontiguousarray(y, dtype=np.int32)
    nxt = C.c_int32(0)
    mt, ma = C.c_double(0), C.c_double(0)
    n = lib().orc_accept_rule(_ptr(plog), _ptr(qlog), _ptr(y), gamma, V, mode, seed, pos_first, seq,
                              C.byref(nxt), C.byref(mt), C.byref(ma))
    return n, nxt.value, mt.value, ma.value


class Pacer:
    """Algorithm 1 with access to every stage (for stage-by-stage comparisons)."""

    def __init__(self, T: OracleModel, D: OracleModel, B: Optional[OracleModel], max_ctx: int, b=4, gamma_cap=8,
                 t0=0.5, rho=1.05, criterion=0, mode=0, seed=0, seq_id=0, use_posemb=1, scope=0):
        self.T, self.D, self.B, self.max_ctx = T, D, B, max_ctx
        self.prm = Params(b, gamma_cap, t0, rho, criterion, mode, seed, seq_id, use_posemb, scope, 0)
        self.h = lib().orc_new(T.ref(), D.ref(), B.ref() if B else None, max_ctx, C.byref(self.prm))
        self._override = None

    def __del__(self):
        if getattr(self, "h", None) and _lib is not None:
            _lib.orc_free(self.h)
            self.h = None

    # stages
    def prefill(self, prompt):
        p = np.ascontiguousarray(np.asarray(prompt, dtype=np.int32))
        lib().orc_prefill(self.h, _ptr(p), p.shape[0])

    def draft_block(self):
        lib().orc_draft_block(self.h)

    def preverify(self) -> float:
        return lib().orc_preverify(self.h)

    def verify(self):
        lib().orc_verify(self.h)

    def accept(self) -> int:
        return lib().orc_accept(self.h)

    def set_alpha_override(self, values):
        self._override = np.ascontiguousarray(values, dtype=np.float64)
        lib().orc_set_alpha_override(self.h, _ptr(self._override), self._override.shape[0])

    def set_seed(self, seed, seq_id=0):
        lib().orc_set_seed(self.h, seed, seq_id)

    # state
    @property
    def P(self): return lib().orc_get_P(self.h)
    @property
    def gamma(self): return lib().orc_get_gamma(self.h)
    @property
    def drafting(self): return lib().orc_get_drafting(self.h)
    @property
    def t_k(self): return lib().orc_get_t_k(self.h)
    @property
    def last_n(self): return lib().orc_get_last_n(self.h)
    @property
    def last_next(self): return lib().orc_get_last_next(self.h)
    @property
    def n_pend(self): return lib().orc_get_n_pend(self.h)

    def cache_len(self, which: int) -> int:
        return lib().orc_get_len(self.h, which)

    def _arr(self, fn, ctype, shape):
        n = int(np.prod(shape))
        if n == 0:
            return np.zeros(shape, dtype=np.float64 if ctype is C.c_double else np.int32)
        p = C.cast(getattr(lib(), fn)(self.h), C.POINTER(ctype))
        return np.ctypeslib.as_array(p, (n,)).reshape(shape).copy()

    def x(self): return self._arr("orc_get_x", C.c_int32, (self.P,))
    def y(self): return self._arr("orc_get_y", C.c_int32, (self.gamma,))
    def alpha(self): return self._arr("orc_get_alpha", C.c_double, (self.gamma,))
    def plogits(self, rows): return self._arr("orc_get_plogits", C.c_double, (rows, self.T.shape.vocab))
    def qlogits(self, rows): return self._arr("orc_get_qlogits", C.c_double, (rows, self.T.shape.vocab))
    def hpend(self): return self._arr("orc_get_hpend", C.c_double, (self.n_pend, self.D.shape.d_model))

    def cache_kv(self, which: int):
        model = (self.T, self.D, self.B)[which]
        s = model.shape
        shp = (s.n_layers, self.max_ctx, s.n_kv_heads * (s.d_model // s.n_heads))
        n = int(np.prod(shp))
        ch = lib().orc_get_cache(self.h, which)
        k = np.ctypeslib.as_array(C.cast(lib().orc_cache_k(ch), C.POINTER(C.c_double)), (n,)).reshape(shp)
        v = np.ctypeslib.as_array(C.cast(lib().orc_cache_v(ch), C.POINTER(C.c_double)), (n,)).reshape(shp)
        return k, v

    def stats(self) -> dict:
        st = Stats()
        lib().orc_get_stats(self.h, C.byref(st))
        return st.as_dict()

    # whole loop
    def generate(self, prompt, max_new):
        p = np.ascontiguousarray(np.asarray(prompt, dtype=np.int32))
        out = np.zeros(max_new, np.int32)
        dl = np.full(max_new, -1, np.int32)
        al = np.full(max_new, -1, np.int32)
        st = Stats()
        steps = lib().orc_generate_pacer(self.h, _ptr(p), p.shape[0], max_new, _ptr(out), _ptr(dl), _ptr(al),
                                         C.byref(st))
        return out, dl[:steps], al[:steps], st.as_dict()


def generate_sd(T: OracleModel, D: OracleModel, prompt, max_new, gamma, mode=0, seed=0, seq=0, max_ctx=None):
    p = np.ascontiguousarray(np.asarray(prompt, dtype=np.int32))
    if max_ctx is None:
        max_ctx = p.shape[0] + max_new + gamma + 2
    out = np.zeros(max_new, np.int32)
    dl = np.full(max_new, -1, np.int32)
    al = np.full(max_new, -1, np.int32)
    st = Stats()
    steps = lib().orc_generate_sd(T.ref(), D.ref(), _ptr(p), p.shape[0], max_new, gamma, mode, seed, seq, max_ctx,
                                  _ptr(out), _ptr(dl), _ptr(al), C.byref(st))
    return out, dl[:steps], al[:steps], st.as_dict()


def generate_sched(T: OracleModel, D: OracleModel, prompt, max_new, windows, mode=0, seed=0, seq=0, max_ctx=None):
    """Speculative decoding with the window of every step prescribed (Section 3.1's gamma* when the windows are the
    accepted lengths of a large-window run).  Returns (tokens, draft_len, accept_len, stats)."""
    p = np.ascontiguousarray(np.asarray(prompt, dtype=np.int32))
    w = np.ascontiguousarray(np.asarray(windows, dtype=np.int32))
    assert w.ndim == 1 and w.shape[0] >= 1 and w.min() >= 0
    if max_ctx is None:
        max_ctx = p.shape[0] + max_new + int(w.max()) + 2
    out = np.zeros(max_new, np.int32)
    dl = np.full(max_new, -1, np.int32)
    al = np.full(max_new, -1, np.int32)
    st = Stats()
    steps = lib().orc_generate_sched(T.ref(), D.ref(), _ptr(p), p.shape[0], max_new, _ptr(w), w.shape[0], mode, seed,
                                     seq, max_ctx, _ptr(out), _ptr(dl), _ptr(al), C.byref(st))
    return out, dl[:steps], al[:steps], st.as_dict()


def generate_ar(T: OracleModel, prompt, max_new, mode=0, seed=0, seq=0, max_ctx=None):
    p = np.ascontiguousarray(np.asarray(prompt, dtype=np.int32))
    if max_ctx is None:
        max_ctx = p.shape[0] + max_new + 1
    out = np.zeros(max_new, np.int32)
    mm = C.c_double(0)
    lib().orc_generate_ar(T.ref(), _ptr(p), p.shape[0], max_new, mode, seed, seq, max_ctx, _ptr(out), C.byref(mm))
    return out, mm.value
