"""Thin ctypes binding of ``libpacer.so`` (C ABI declared in ``include/pacer.h``).

Argument marshalling only: every step of the decoding loop runs in the CUDA
library.  PyTorch is used for device memory (the workspace and the weights are
torch tensors owned by the caller) and for the stream.  Importing this module
fails loudly when the library has not been built; there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os
from typing import Dict, Optional

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libpacer.so")

if not os.path.exists(LIB_PATH):
    raise ImportError(
        f"{LIB_PATH} is missing: build it with `python -m paper_2602_01274_b200.build` "
        "(nvcc, sm_100a). There is no fallback path.")

_lib = C.CDLL(LIB_PATH)

PACER_TARGET, PACER_DRAFT, PACER_PREVERIFY = 0, 1, 2
PACER_GREEDY, PACER_SAMPLE = 0, 1
(BUF_TOKENS, BUF_DRAFTS, BUF_ALPHA, BUF_VERIFY_LOGITS, BUF_DRAFT_LOGITS, BUF_HPEND, BUF_DRAFT_LEN, BUF_ACCEPT_LEN,
 BUF_KCACHE_T, BUF_VCACHE_T, BUF_KCACHE_D, BUF_VCACHE_D, BUF_KCACHE_B, BUF_VCACHE_B, BUF_PHASE_NS) = range(15)


class ModelCfg(C.Structure):
    _fields_ = [("n_layers", C.c_int32), ("d_model", C.c_int32), ("n_heads", C.c_int32), ("n_kv_heads", C.c_int32),
                ("d_ffn", C.c_int32), ("vocab", C.c_int32), ("rope_theta", C.c_float), ("rms_eps", C.c_float)]


class Cfg(C.Structure):
    _fields_ = [("target", ModelCfg), ("draft", ModelCfg), ("max_batch", C.c_int32), ("max_ctx", C.c_int32),
                ("gamma_cap", C.c_int32), ("block_b", C.c_int32), ("rho", C.c_float), ("criterion", C.c_int32),
                ("succ_bias", C.c_float), ("use_posemb", C.c_int32), ("mb_scope", C.c_int32)]


class Tensor(C.Structure):
    _fields_ = [("name", C.c_char_p), ("dev_ptr", C.c_void_p), ("numel", C.c_int64)]


class Stats(C.Structure):
    _fields_ = [("n_draft_fwd", C.c_int64), ("n_mb_calls", C.c_int64), ("n_target_fwd", C.c_int64),
                ("n_steps", C.c_int64), ("n_generated", C.c_int64), ("n_kernel_launches", C.c_int64),
                ("ms_prefill", C.c_float), ("ms_decode", C.c_float)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


class SeqState(C.Structure):
    _fields_ = [("P", C.c_int32), ("len_T", C.c_int32), ("len_D", C.c_int32), ("len_B", C.c_int32),
                ("gamma", C.c_int32), ("k_round", C.c_int32), ("t_k", C.c_float), ("drafting", C.c_int32),
                ("finished", C.c_int32), ("n_steps", C.c_int32), ("last_n", C.c_int32), ("last_next", C.c_int32),
                ("n_pend", C.c_int32), ("err", C.c_int32), ("n_draft_fwd", C.c_int64), ("n_mb_calls", C.c_int64),
                ("n_target_fwd", C.c_int64)]

    def as_dict(self):
        return {k: getattr(self, k) for k, _ in self._fields_}


_P = C.c_void_p
_lib.pacer_strerror.restype = C.c_char_p
_lib.pacer_strerror.argtypes = [C.c_int]
_lib.pacer_last_error.restype = C.c_char_p
_lib.pacer_last_error.argtypes = [_P]
_lib.pacer_workspace_bytes.restype = C.c_size_t
_lib.pacer_workspace_bytes.argtypes = [C.POINTER(Cfg)]
_lib.pacer_create.argtypes = [C.POINTER(Cfg), _P, C.c_size_t, _P, C.POINTER(_P)]
_lib.pacer_destroy.argtypes = [_P]
_lib.pacer_load_weights.argtypes = [_P, C.c_int, C.POINTER(Tensor), C.c_int, _P]
_lib.pacer_prefill.argtypes = [_P, _P, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float, C.c_int, C.c_uint64]
for _n in ("pacer_draft_step", "pacer_preverify", "pacer_verify", "pacer_accept_rollback"):
    getattr(_lib, _n).argtypes = [_P]
_lib.pacer_debug_set_device_status.argtypes = [_P, C.c_int, C.c_int, C.c_int, C.c_int]
_lib.pacer_read_state.argtypes = [_P, C.POINTER(SeqState), C.c_int]
_lib.pacer_read_buffer.argtypes = [_P, C.c_int, _P, C.c_size_t]
_lib.pacer_generate.argtypes = [_P, _P, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float, C.c_int, C.c_uint64,
                                _P, _P, _P, _P, C.POINTER(Stats)]
_lib.pacer_generate_sched.argtypes = [_P, _P, C.c_int, C.c_int, C.c_int, _P, C.c_int, C.c_int, C.c_uint64,
                                      _P, _P, _P, _P, C.POINTER(Stats)]
_lib.pacer_generate_ar.argtypes = [_P, _P, C.c_int, C.c_int, C.c_int, C.c_int, C.c_uint64, _P, C.POINTER(Stats)]
_lib.pacer_profile_begin.argtypes = [_P]
_lib.pacer_profile_end.argtypes = [_P, C.POINTER(C.c_double), C.POINTER(C.c_double), C.POINTER(C.c_int64)]
_lib.pacer_linear_scratch_bytes.restype = C.c_size_t
_lib.pacer_linear_scratch_bytes.argtypes = [C.c_int, C.c_int, C.c_int]
_lib.pacer_linear.argtypes = [_P, _P, _P, C.c_int, C.c_int, C.c_int, _P, C.c_size_t, _P]
_lib.pacer_linear_static.argtypes = [_P, _P, _P, C.c_int, C.c_int, C.c_int, _P]
PACER_LINEAR_STATIC_BYTES = 4 << 20


class PacerError(RuntimeError):
    pass


def exported_symbols():
    """The C entry points this binding resolved (all declared in pacer.h)."""
    return ["pacer_strerror", "pacer_last_error", "pacer_workspace_bytes", "pacer_create", "pacer_destroy",
            "pacer_load_weights", "pacer_prefill", "pacer_draft_step", "pacer_preverify", "pacer_verify",
            "pacer_accept_rollback", "pacer_read_state", "pacer_read_buffer", "pacer_generate", "pacer_generate_sched",
            "pacer_generate_ar", "pacer_debug_set_device_status",
            "pacer_profile_begin", "pacer_profile_end", "pacer_linear_scratch_bytes", "pacer_linear", "pacer_linear_static"]


def _model_cfg(s) -> ModelCfg:
    return ModelCfg(s.n_layers, s.d_model, s.n_heads, s.n_kv_heads, s.d_ffn, s.vocab, s.rope_theta, s.rms_eps)


def make_cfg(target, draft, max_batch, max_ctx, gamma_cap, block_b=4, rho=1.05, criterion=0, succ_bias=8.0,
             use_posemb=1, mb_scope=0) -> Cfg:
    """target/draft: objects with n_layers, d_model, n_heads, n_kv_heads, d_ffn, vocab, rope_theta, rms_eps."""
    return Cfg(_model_cfg(target), _model_cfg(draft), max_batch, max_ctx, gamma_cap, block_b, rho, criterion,
               succ_bias, use_posemb, mb_scope)


def pacer_workspace_bytes(cfg: Cfg) -> int:
    return _lib.pacer_workspace_bytes(C.byref(cfg))


def _i32(a) -> np.ndarray:
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


class Context:
    """One pacer_ctx.  Methods carry the names of the C entry points."""

    def __init__(self, cfg: Cfg, device="cuda:0", stream: Optional[torch.cuda.Stream] = None):
        self.cfg = cfg
        self.device = torch.device(device)
        nbytes = pacer_workspace_bytes(cfg)
        if nbytes == 0:
            raise PacerError("bad configuration")
        with torch.cuda.device(self.device):
            self.workspace = torch.empty(nbytes + 256, dtype=torch.uint8, device=self.device)
            base = self.workspace.data_ptr()
            self._ws_ptr = (base + 255) // 256 * 256
            # a stream of its own (the legacy default stream cannot be captured into the per-step CUDA graph)
            self.stream = stream if stream is not None else torch.cuda.Stream(self.device)
            h = _P()
            rc = _lib.pacer_create(C.byref(cfg), self._ws_ptr, nbytes, self.stream.cuda_stream, C.byref(h))
        self._h = h
        self._keep = []
        self._check(rc)

    def _check(self, rc):
        if rc != 0:
            msg = _lib.pacer_last_error(self._h if self._h else None)
            raise PacerError(f"{_lib.pacer_strerror(rc).decode()} ({rc}): {msg.decode() if msg else ''}")

    def close(self):
        if getattr(self, "_h", None):
            _lib.pacer_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def pacer_load_weights(self, which: int, tensors: Dict[str, torch.Tensor], succ: Optional[torch.Tensor] = None):
        arr = (Tensor * len(tensors))()
        for i, (k, t) in enumerate(tensors.items()):
            assert t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous(), k
            arr[i] = Tensor(k.encode(), t.data_ptr(), t.numel())
            self._keep.append(t)
        sp = None
        if succ is not None:
            assert succ.is_cuda and succ.dtype == torch.int32 and succ.is_contiguous()
            self._keep.append(succ)
            sp = succ.data_ptr()
        with torch.cuda.device(self.device):
            self.stream.wait_stream(torch.cuda.current_stream(self.device))     # the tensors may still be being written
            self._check(_lib.pacer_load_weights(self._h, which, arr, len(tensors), sp))
            torch.cuda.current_stream(self.device).wait_stream(self.stream)     # later torch work sees the copy done

    def pacer_prefill(self, prompt, max_new, gamma_max, threshold, mode=PACER_GREEDY, seed=0):
        p = _i32(prompt)
        if p.ndim == 1:
            p = p[None]
        with torch.cuda.device(self.device):
            self._check(_lib.pacer_prefill(self._h, p.ctypes.data, p.shape[0], p.shape[1], max_new, gamma_max,
                                           threshold, mode, seed))

    def pacer_draft_step(self):
        with torch.cuda.device(self.device):
            self._check(_lib.pacer_draft_step(self._h))

    def pacer_preverify(self):
        with torch.cuda.device(self.device):
            self._check(_lib.pacer_preverify(self._h))

    def pacer_verify(self):
        with torch.cuda.device(self.device):
            self._check(_lib.pacer_verify(self._h))

    def pacer_accept_rollback(self):
        with torch.cuda.device(self.device):
            self._check(_lib.pacer_accept_rollback(self._h))

    def pacer_debug_set_device_status(self, code, block=0, warp=0, detail=0):
        with torch.cuda.device(self.device):
            self._check(_lib.pacer_debug_set_device_status(self._h, code, block, warp, detail))

    def pacer_read_state(self, batch=1):
        arr = (SeqState * batch)()
        with torch.cuda.device(self.device):
            self._check(_lib.pacer_read_state(self._h, arr, batch))
        return [a.as_dict() for a in arr]

    def pacer_read_buffer(self, which: int, dtype, count: int) -> np.ndarray:
        out = np.empty(count, dtype=dtype)
        with torch.cuda.device(self.device):
            self._check(_lib.pacer_read_buffer(self._h, which, out.ctypes.data, out.nbytes))
        return out

    def pacer_profile_begin(self):
        self._check(_lib.pacer_profile_begin(self._h))

    def pacer_profile_end(self):
        """Returns (summed GEMM device ms, weight bytes streamed, launches)."""
        ms, by, n = C.c_double(0), C.c_double(0), C.c_int64(0)
        with torch.cuda.device(self.device):
            self._check(_lib.pacer_profile_end(self._h, C.byref(ms), C.byref(by), C.byref(n)))
        return ms.value, by.value, n.value

    def pacer_generate(self, prompt, max_new, gamma_max, threshold, mode=PACER_GREEDY, seed=0):
        """Returns (tokens [batch][max_new], n_steps [batch], draft_len, accept_len [batch][max_new], stats dict)."""
        p = _i32(prompt)
        if p.ndim == 1:
            p = p[None]
        B = p.shape[0]
        tok = np.zeros((B, max_new), np.int32)
        ns = np.zeros(B, np.int32)
        dl = np.zeros((B, max_new), np.int32)
        al = np.zeros((B, max_new), np.int32)
        st = Stats()
        with torch.cuda.device(self.device):
            self._check(_lib.pacer_generate(self._h, p.ctypes.data, B, p.shape[1], max_new, gamma_max, threshold, mode,
                                            seed, tok.ctypes.data, ns.ctypes.data, dl.ctypes.data, al.ctypes.data,
                                            C.byref(st)))
        return tok, ns, dl, al, st.as_dict()

    def pacer_generate_sched(self, prompt, max_new, windows, mode=PACER_GREEDY, seed=0):
        """Speculative decoding with prescribed windows (int32 [batch][n_windows] or [n_windows]); returns like
        pacer_generate."""
        p = _i32(prompt)
        if p.ndim == 1:
            p = p[None]
        w = _i32(windows)
        if w.ndim == 1:
            w = w[None]
        B = p.shape[0]
        assert w.shape[0] == B
        tok = np.zeros((B, max_new), np.int32)
        ns = np.zeros(B, np.int32)
        dl = np.zeros((B, max_new), np.int32)
        al = np.zeros((B, max_new), np.int32)
        st = Stats()
        with torch.cuda.device(self.device):
            self._check(_lib.pacer_generate_sched(self._h, p.ctypes.data, B, p.shape[1], max_new, w.ctypes.data,
                                                  w.shape[1], mode, seed, tok.ctypes.data, ns.ctypes.data,
                                                  dl.ctypes.data, al.ctypes.data, C.byref(st)))
        return tok, ns, dl, al, st.as_dict()

    def pacer_generate_ar(self, prompt, max_new, mode=PACER_GREEDY, seed=0):
        p = _i32(prompt)
        if p.ndim == 1:
            p = p[None]
        tok = np.zeros((p.shape[0], max_new), np.int32)
        st = Stats()
        with torch.cuda.device(self.device):
            self._check(_lib.pacer_generate_ar(self._h, p.ctypes.data, p.shape[0], p.shape[1], max_new, mode, seed,
                                               tok.ctypes.data, C.byref(st)))
        return tok, st.as_dict()


def pacer_linear(x: torch.Tensor, w: torch.Tensor) -> torch.Tensor:
    """y = x @ w.T through the library's skinny GEMM. x bf16 [rows<=32][K], w bf16 [N][K] -> f32 [rows][N]."""
    assert x.is_cuda and w.is_cuda and x.dtype == torch.bfloat16 and w.dtype == torch.bfloat16
    x, w = x.contiguous(), w.contiguous()
    rows, K = x.shape
    N = w.shape[0]
    nbytes = _lib.pacer_linear_scratch_bytes(rows, N, K)
    if nbytes == 0:
        raise PacerError("pacer_linear: unsupported shape")
    scratch = torch.empty(nbytes + 256, dtype=torch.uint8, device=x.device)
    sp = (scratch.data_ptr() + 255) // 256 * 256
    y = torch.empty(rows, N, dtype=torch.float32, device=x.device)
    with torch.cuda.device(x.device):
        rc = _lib.pacer_linear(x.data_ptr(), w.data_ptr(), y.data_ptr(), rows, N, K, sp, nbytes,
                               torch.cuda.current_stream(x.device).cuda_stream)
    if rc != 0:
        raise PacerError(f"pacer_linear: {_lib.pacer_strerror(rc).decode()}: {_lib.pacer_last_error(None).decode()}")
    return y


def pacer_linear_static(x: torch.Tensor, w: torch.Tensor, out: torch.Tensor) -> torch.Tensor:
    """y = x @ w.T written into the caller's `out` (f32 [rows][N]) with the library's built-in scratch: the call
    itself allocates nothing on the device, for callers whose device memory is all spoken for.  Shapes that need
    more than PACER_LINEAR_STATIC_BYTES of scratch raise PacerError.  Calls on one device share the scratch, so
    they must not overlap on the GPU."""
    assert x.is_cuda and w.is_cuda and out.is_cuda and x.dtype == torch.bfloat16 and w.dtype == torch.bfloat16
    assert x.is_contiguous() and w.is_contiguous() and out.is_contiguous() and out.dtype == torch.float32
    rows, K = x.shape
    N = w.shape[0]
    assert tuple(out.shape) == (rows, N)
    with torch.cuda.device(x.device):
        rc = _lib.pacer_linear_static(x.data_ptr(), w.data_ptr(), out.data_ptr(), rows, N, K,
                                      torch.cuda.current_stream(x.device).cuda_stream)
    if rc != 0:
        raise PacerError(f"pacer_linear_static: {_lib.pacer_strerror(rc).decode()}: {_lib.pacer_last_error(None).decode()}")
    return out


def load_pair(ctx: Context, pair: dict):
    """Registers the three models of a synthetic pair (tensors already on the context's device)."""
    ctx.pacer_load_weights(PACER_TARGET, pair["target"], pair["succ_T"])
    ctx.pacer_load_weights(PACER_DRAFT, pair["draft"], pair["succ_D"])
    ctx.pacer_load_weights(PACER_PREVERIFY, pair["preverify"])
