"""Thin ctypes binding of libdisco.so (include/disco.h).  Argument marshalling only.

Every step of the path runs inside the CUDA library.  There is no fallback: if the library has
not been built, loading raises.  Tensors are torch CUDA tensors (torch is used for device memory
and streams only); the ``*_host`` calls take CPU tensors (pinned for asynchronous copies).
"""
from __future__ import annotations

import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libdisco.so")

TOPK = 10
NFEAT = 12

OK = 0
ERR_INVALID_ARG = -1
ERR_UNSUPPORTED_SHAPE = -2
ERR_WORKSPACE = -3
ERR_CUDA = -4
ERR_TIMEOUT = -5
ERR_STATIC_LIMIT = -6
STATIC_MAX_BATCH = 4

EXPORTS = [
    "disco_create", "disco_destroy", "disco_strerror", "disco_last_device_status", "disco_launch_count",
    "disco_set_kernel_path", "disco_draft_step", "disco_verify", "disco_verify_ragged",
    "disco_draft_step_host", "disco_verify_ragged_host", "disco_draft_step_static", "disco_draft_step_ppl",
    "disco_draft_step_sample", "disco_verify_sample_ragged", "disco_extract_features",
    "disco_draft_loop", "disco_verify_sl", "disco_iteration", "disco_iteration_host", "disco_test_hooks",
]


class DiscoError(RuntimeError):
    def __init__(self, code: int, what: str):
        self.code = code
        super().__init__(f"{what}: {strerror(code)} (code {code})")


class _Clf(ctypes.Structure):
    _fields_ = [("W1", ctypes.c_void_p), ("b1", ctypes.c_void_p), ("w2", ctypes.c_void_p),
                ("b2", ctypes.c_void_p), ("H", ctypes.c_int)]


_lib = None


def load() -> ctypes.CDLL:
    """Load libdisco.so; raises if it is missing (build it with paper_2405_04304_b200/build.py)."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: the CUDA library has not been built "
                           "(python paper_2405_04304_b200/build.py); there is no fallback path")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, cf = ctypes.c_void_p, ctypes.c_int, ctypes.c_float
    lib.disco_create.argtypes = [ctypes.POINTER(vp), ci, ci, ci, ci, ci, ci, ci]
    lib.disco_destroy.argtypes = [vp]
    lib.disco_strerror.argtypes = [ci]
    lib.disco_strerror.restype = ctypes.c_char_p
    lib.disco_last_device_status.argtypes = [vp, ctypes.POINTER(ci)]
    lib.disco_launch_count.argtypes = [vp, ctypes.POINTER(ctypes.c_longlong)]
    lib.disco_set_kernel_path.argtypes = [vp, ci]
    lib.disco_test_hooks.argtypes = [vp, ctypes.c_longlong, ci]
    lib.disco_draft_step.argtypes = [vp, vp, vp, ci, vp, vp, vp, ctypes.POINTER(_Clf), cf, ci,
                                     vp, vp, vp, vp, vp, vp]
    lib.disco_draft_step_ppl.argtypes = [vp, vp, vp, ci, vp, vp, vp, cf, ci, vp, vp, vp, vp]
    lib.disco_draft_step_sample.argtypes = [vp, vp, vp, ci, vp, vp, vp, ctypes.POINTER(_Clf), cf, ci, vp,
                                            vp, vp, vp, vp, vp, vp, vp]
    lib.disco_verify_sample_ragged.argtypes = [vp, vp, vp, vp, vp, vp, ci, ci, vp, vp, vp, vp, vp, vp, vp]
    lib.disco_extract_features.argtypes = [vp, vp, vp, vp, vp, vp, ci, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.disco_verify.argtypes = [vp, vp, vp, vp, ci, ci, vp, vp, vp, vp]
    lib.disco_verify_ragged.argtypes = [vp, vp, vp, vp, vp, ci, ci, vp, vp, vp, vp]
    lib.disco_draft_step_host.argtypes = [vp, vp, vp, ci, vp, vp, vp, ctypes.POINTER(_Clf), cf, ci,
                                          vp, vp, vp, vp, vp]
    lib.disco_verify_ragged_host.argtypes = [vp, vp, vp, vp, vp, ci, ci, vp, vp, vp, vp]
    lib.disco_draft_step_static.argtypes = [ci, ci, vp, vp, ci, vp, vp, vp, ctypes.POINTER(_Clf), cf, ci,
                                            vp, vp, vp, vp, vp]
    sz, ll = ctypes.c_size_t, ctypes.c_longlong
    lib.disco_draft_loop.argtypes = [vp, vp, sz, vp, ci, vp, ctypes.POINTER(_Clf), cf, ci, vp, vp, vp, vp, vp, vp, vp]
    lib.disco_verify_sl.argtypes = [vp, vp, vp, vp, ll, ll, vp, ci, ci, vp, vp, vp, vp, vp, vp, vp]
    lib.disco_iteration.argtypes = [vp, vp, sz, vp, vp, vp, ci, vp, ctypes.POINTER(_Clf), cf, ci, vp, vp,
                                    vp, vp, vp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.disco_iteration_host.argtypes = [vp, vp, sz, vp, vp, vp, ci, vp, ctypes.POINTER(_Clf), cf, ci, vp, vp,
                                         vp, vp, vp, vp, vp, vp, vp, vp]
    _lib = lib
    return lib


def strerror(code: int) -> str:
    return load().disco_strerror(int(code)).decode()


def _ptr(t, dtype=None, cuda=True):
    """Address of a contiguous tensor of the expected dtype and device kind (None -> NULL), as an integer."""
    if t is None:
        return None
    if (dtype is not None and t.dtype is not dtype) or t.is_cuda is not cuda or not t.is_contiguous():
        if dtype is not None and t.dtype != dtype:
            raise TypeError(f"expected {dtype}, got {t.dtype}")
        if t.is_cuda != cuda:
            raise ValueError("tensor is on the wrong device kind for this call")
        raise ValueError("tensor must be contiguous")
    return t.data_ptr()


def _stream(stream) -> int:
    s = stream if stream is not None else torch.cuda.current_stream()
    return s.cuda_stream


class Classifier:
    """Device-resident parameters of the halt classifier (fp32)."""

    def __init__(self, W1: torch.Tensor, b1: torch.Tensor, w2: torch.Tensor, b2: torch.Tensor):
        for t in (W1, b1, w2, b2):
            if not t.is_cuda or t.dtype != torch.float32:
                raise TypeError("classifier parameters must be fp32 CUDA tensors")
        self.W1, self.b1, self.w2, self.b2 = (t.contiguous() for t in (W1, b1, w2, b2))
        self.H = int(W1.shape[0])
        if tuple(W1.shape) != (self.H, NFEAT) or b1.numel() != self.H or w2.numel() != self.H or b2.numel() != 1:
            raise ValueError("classifier shapes must be [H,12], [H], [H], [1]")
        self._c = _Clf(self.W1.data_ptr(), self.b1.data_ptr(), self.w2.data_ptr(), self.b2.data_ptr(), self.H)


def draft_step_static(W_D, h_D, pos, n_drafted, clf: "Classifier", tau: float, sl_max: int, token, conf, halt,
                      active=None, feats=None, stream=None) -> None:
    """disco_draft_step_static: the draft step for hosts that may not allocate device memory.

    Needs no Context (creating one calls cudaMalloc).  The cross-block scratch is a fixed array inside
    libdisco.so, shared by every call on the device, so calls must not overlap on the GPU.  At most
    STATIC_MAX_BATCH sequences; larger requests raise DiscoError(ERR_STATIC_LIMIT).  The first call on a
    device also does the one-time set-up and should come before any stream capture."""
    V, d = int(W_D.shape[0]), int(W_D.shape[1])
    B = int(h_D.shape[0])
    rc = load().disco_draft_step_static(
        V, d, _ptr(W_D, torch.bfloat16), _ptr(h_D, torch.bfloat16), B, _ptr(pos, torch.int32),
        _ptr(n_drafted, torch.int32), _ptr(active, torch.uint8), ctypes.byref(clf._c), float(tau), int(sl_max),
        _ptr(token, torch.int32), _ptr(conf, torch.float32), _ptr(halt, torch.uint8), _ptr(feats, torch.float32),
        _stream(stream))
    if rc != OK:
        raise DiscoError(rc, "disco_draft_step_static")


class Context:
    """disco_ctx: scratch for one (V, d_draft, d_target) configuration on the current device."""

    def __init__(self, V: int, d_draft: int, d_target: int, max_batch: int = 1, max_rows: int = 32,
                 clf_hidden: int = 64):
        self._lib = load()
        self._h = ctypes.c_void_p()
        rc = self._lib.disco_create(ctypes.byref(self._h), V, d_draft, d_target, max_batch, max_rows, TOPK,
                                    clf_hidden)
        if rc != OK:
            self._h = ctypes.c_void_p()
            raise DiscoError(rc, "disco_create")
        self.V, self.d_draft, self.d_target = V, d_draft, d_target
        self.max_batch, self.max_rows = max_batch, max_rows

    def close(self):
        if getattr(self, "_h", None) and self._h.value:
            self._lib.disco_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ---------------------------------------------------------------- bookkeeping
    def device_status(self) -> int:
        out = ctypes.c_int()
        rc = self._lib.disco_last_device_status(self._h, ctypes.byref(out))
        if rc != OK:
            raise DiscoError(rc, "disco_last_device_status")
        return int(out.value)

    def launch_count(self) -> int:
        out = ctypes.c_longlong()
        self._lib.disco_launch_count(self._h, ctypes.byref(out))
        return int(out.value)

    def test_hooks(self, wait_budget_clocks: int = 0, withhold_records: bool = False) -> None:
        rc = self._lib.disco_test_hooks(self._h, int(wait_budget_clocks), int(bool(withhold_records)))
        if rc != OK:
            raise DiscoError(rc, "disco_test_hooks")

    def set_kernel_path(self, which: int) -> None:
        rc = self._lib.disco_set_kernel_path(self._h, int(which))
        if rc != OK:
            raise DiscoError(rc, "disco_set_kernel_path")

    # ---------------------------------------------------------------- device-resident calls
    def draft_step(self, W_D, h_D, pos, n_drafted, clf: Classifier, tau: float, sl_max: int,
                   token, conf, halt, active=None, feats=None, probs=None, stream=None) -> None:
        B = int(h_D.shape[0])
        rc = self._lib.disco_draft_step(
            self._h, _ptr(W_D, torch.bfloat16), _ptr(h_D, torch.bfloat16), B, _ptr(pos, torch.int32),
            _ptr(n_drafted, torch.int32), _ptr(active, torch.uint8), ctypes.byref(clf._c), float(tau),
            int(sl_max), _ptr(token, torch.int32), _ptr(conf, torch.float32), _ptr(halt, torch.uint8),
            _ptr(feats, torch.float32), _ptr(probs, torch.float32), _stream(stream))
        if rc != OK:
            raise DiscoError(rc, "disco_draft_step")

    def draft_step_ppl(self, W_D, h_D, n_drafted, nll_sum, ppl_max: float, sl_max: int, token, ppl, halt,
                       active=None, stream=None) -> None:
        B = int(h_D.shape[0])
        rc = self._lib.disco_draft_step_ppl(
            self._h, _ptr(W_D, torch.bfloat16), _ptr(h_D, torch.bfloat16), B, _ptr(n_drafted, torch.int32),
            _ptr(active, torch.uint8), _ptr(nll_sum, torch.float32), float(ppl_max), int(sl_max),
            _ptr(token, torch.int32), _ptr(ppl, torch.float32), _ptr(halt, torch.uint8), _stream(stream))
        if rc != OK:
            raise DiscoError(rc, "disco_draft_step_ppl")

    def draft_step_sample(self, W_D, h_D, pos, n_drafted, clf: Classifier, tau: float, sl_max: int, u,
                          token, conf, halt, probs, p_token=None, active=None, feats=None, stream=None) -> None:
        B = int(h_D.shape[0])
        rc = self._lib.disco_draft_step_sample(
            self._h, _ptr(W_D, torch.bfloat16), _ptr(h_D, torch.bfloat16), B, _ptr(pos, torch.int32),
            _ptr(n_drafted, torch.int32), _ptr(active, torch.uint8), ctypes.byref(clf._c), float(tau),
            int(sl_max), _ptr(u, torch.float32), _ptr(token, torch.int32), _ptr(p_token, torch.float32),
            _ptr(conf, torch.float32), _ptr(halt, torch.uint8), _ptr(feats, torch.float32),
            _ptr(probs, torch.float32), _stream(stream))
        if rc != OK:
            raise DiscoError(rc, "disco_draft_step_sample")

    def verify_sample_ragged(self, W_T, H_T, draft_ids, draft_probs, row_off, B: int, R: int, u_accept,
                             u_sample, n_accept, next_token, y_T, target_ids=None, stream=None) -> None:
        rc = self._lib.disco_verify_sample_ragged(
            self._h, _ptr(W_T, torch.bfloat16), _ptr(H_T, torch.bfloat16), _ptr(draft_ids, torch.int32),
            _ptr(draft_probs, torch.float32), _ptr(row_off, torch.int32), int(B), int(R),
            _ptr(u_accept, torch.float32), _ptr(u_sample, torch.float32), _ptr(n_accept, torch.int32),
            _ptr(next_token, torch.int32), _ptr(y_T, torch.float32), _ptr(target_ids, torch.int32),
            _stream(stream))
        if rc != OK:
            raise DiscoError(rc, "disco_verify_sample_ragged")

    def extract_features(self, W_D, H_D, W_T, H_T, pos, feats_D, feats_T, tv, label, token_D, token_T, y_D, y_T,
                         stream=None) -> None:
        N = int(H_D.shape[0])
        rc = self._lib.disco_extract_features(
            self._h, _ptr(W_D, torch.bfloat16), _ptr(H_D, torch.bfloat16), _ptr(W_T, torch.bfloat16),
            _ptr(H_T, torch.bfloat16), _ptr(pos, torch.int32), N, _ptr(feats_D, torch.float32),
            _ptr(feats_T, torch.float32), _ptr(tv, torch.float32), _ptr(label, torch.uint8),
            _ptr(token_D, torch.int32), _ptr(token_T, torch.int32), _ptr(y_D, torch.float32),
            _ptr(y_T, torch.float32), _stream(stream))
        if rc != OK:
            raise DiscoError(rc, "disco_extract_features")

    def verify(self, W_T, H_T, draft_ids, B: int, SL: int, n_accept, bonus, target_ids=None,
               stream=None) -> None:
        rc = self._lib.disco_verify(
            self._h, _ptr(W_T, torch.bfloat16), _ptr(H_T, torch.bfloat16), _ptr(draft_ids, torch.int32),
            int(B), int(SL), _ptr(n_accept, torch.int32), _ptr(bonus, torch.int32),
            _ptr(target_ids, torch.int32), _stream(stream))
        if rc != OK:
            raise DiscoError(rc, "disco_verify")

    def verify_ragged(self, W_T, H_T, draft_ids, row_off, B: int, R: int, n_accept, bonus,
                      target_ids=None, stream=None) -> None:
        rc = self._lib.disco_verify_ragged(
            self._h, _ptr(W_T, torch.bfloat16), _ptr(H_T, torch.bfloat16), _ptr(draft_ids, torch.int32),
            _ptr(row_off, torch.int32), int(B), int(R), _ptr(n_accept, torch.int32),
            _ptr(bonus, torch.int32), _ptr(target_ids, torch.int32), _stream(stream))
        if rc != OK:
            raise DiscoError(rc, "disco_verify_ragged")

    # ---------------------------------------------------------------- device-resident iteration
    def draft_loop(self, W_D, h_D, pos0, clf: Classifier, tau: float, sl_max: int, token, conf, halt, sl,
                   sl_forced=None, feats=None, w_step_stride: int = 0, stream=None) -> None:
        """disco_draft_loop: h_D [sl_max, B, d]; token/conf/halt [sl_max, B]; sl [B]."""
        B = int(h_D.shape[1])
        rc = self._lib.disco_draft_loop(
            self._h, _ptr(W_D, torch.bfloat16), int(w_step_stride), _ptr(h_D, torch.bfloat16), B,
            _ptr(pos0, torch.int32), ctypes.byref(clf._c), float(tau), int(sl_max), _ptr(sl_forced, torch.int32),
            _ptr(token, torch.int32), _ptr(conf, torch.float32), _ptr(halt, torch.uint8),
            _ptr(feats, torch.float32), _ptr(sl, torch.int32), _stream(stream))
        if rc != OK:
            raise DiscoError(rc, "disco_draft_loop")

    def verify_sl(self, W_T, H_T, draft_ids, ids_stride_b: int, ids_stride_j: int, sl, B: int, sl_max: int,
                  n_accept, bonus, target_ids=None, row_off=None, pos0=None, pos_next=None, stream=None) -> None:
        """disco_verify_sl: H_T [B, sl_max + 1, d]; sl [B] on the device."""
        rc = self._lib.disco_verify_sl(
            self._h, _ptr(W_T, torch.bfloat16), _ptr(H_T, torch.bfloat16), _ptr(draft_ids, torch.int32),
            int(ids_stride_b), int(ids_stride_j), _ptr(sl, torch.int32), int(B), int(sl_max),
            _ptr(n_accept, torch.int32), _ptr(bonus, torch.int32), _ptr(target_ids, torch.int32),
            _ptr(row_off, torch.int32), _ptr(pos0, torch.int32), _ptr(pos_next, torch.int32), _stream(stream))
        if rc != OK:
            raise DiscoError(rc, "disco_verify_sl")

    def iteration(self, W_D, h_D, W_T, H_T, pos0, clf: Classifier, tau: float, sl_max: int, token, conf, halt, sl,
                  n_accept, bonus, sl_forced=None, draft_ids=None, feats=None, target_ids=None, row_off=None,
                  pos_next=None, w_step_stride: int = 0, stream=None) -> None:
        """disco_iteration: the draft phase and the verification of one iteration in one call."""
        B = int(h_D.shape[1])
        rc = self._lib.disco_iteration(
            self._h, _ptr(W_D, torch.bfloat16), int(w_step_stride), _ptr(h_D, torch.bfloat16),
            _ptr(W_T, torch.bfloat16), _ptr(H_T, torch.bfloat16), B, _ptr(pos0, torch.int32), ctypes.byref(clf._c),
            float(tau), int(sl_max), _ptr(sl_forced, torch.int32), _ptr(draft_ids, torch.int32),
            _ptr(token, torch.int32), _ptr(conf, torch.float32), _ptr(halt, torch.uint8), _ptr(feats, torch.float32),
            _ptr(sl, torch.int32), _ptr(n_accept, torch.int32), _ptr(bonus, torch.int32),
            _ptr(target_ids, torch.int32), _ptr(row_off, torch.int32), _ptr(pos_next, torch.int32), _stream(stream))
        if rc != OK:
            raise DiscoError(rc, "disco_iteration")

    def iteration_host(self, W_D, h_D, W_T, H_T, pos0, clf: Classifier, tau: float, sl_max: int, token, conf, halt,
                       sl, n_accept, bonus, sl_forced=None, draft_ids=None, pos_next=None, w_step_stride: int = 0,
                       stream=None) -> None:
        """disco_iteration_host: LM heads on the device, everything else CPU tensors."""
        B = int(h_D.shape[1])
        h = lambda t, dt: _ptr(t, dt, cuda=False)
        rc = self._lib.disco_iteration_host(
            self._h, _ptr(W_D, torch.bfloat16), int(w_step_stride), h(h_D, torch.bfloat16), _ptr(W_T, torch.bfloat16),
            h(H_T, torch.bfloat16), B, h(pos0, torch.int32), ctypes.byref(clf._c), float(tau), int(sl_max),
            h(sl_forced, torch.int32), h(draft_ids, torch.int32), h(token, torch.int32), h(conf, torch.float32),
            h(halt, torch.uint8), h(sl, torch.int32), h(n_accept, torch.int32), h(bonus, torch.int32),
            h(pos_next, torch.int32), _stream(stream))
        if rc != OK:
            raise DiscoError(rc, "disco_iteration_host")

    # ---------------------------------------------------------------- host-buffer calls
    def draft_step_host(self, W_D, h_D, pos, n_drafted, clf: Classifier, tau: float, sl_max: int,
                        token, conf, halt, active=None, feats=None, stream=None) -> None:
        B = int(h_D.shape[0])
        rc = self._lib.disco_draft_step_host(
            self._h, _ptr(W_D, torch.bfloat16), _ptr(h_D, torch.bfloat16, cuda=False), B,
            _ptr(pos, torch.int32, cuda=False), _ptr(n_drafted, torch.int32, cuda=False),
            _ptr(active, torch.uint8, cuda=False), ctypes.byref(clf._c), float(tau), int(sl_max),
            _ptr(token, torch.int32, cuda=False), _ptr(conf, torch.float32, cuda=False),
            _ptr(halt, torch.uint8, cuda=False), _ptr(feats, torch.float32, cuda=False), _stream(stream))
        if rc != OK:
            raise DiscoError(rc, "disco_draft_step_host")

    def verify_ragged_host(self, W_T, H_T, draft_ids, row_off, B: int, R: int, n_accept, bonus,
                           target_ids=None, stream=None) -> None:
        rc = self._lib.disco_verify_ragged_host(
            self._h, _ptr(W_T, torch.bfloat16), _ptr(H_T, torch.bfloat16, cuda=False),
            _ptr(draft_ids, torch.int32, cuda=False), _ptr(row_off, torch.int32, cuda=False), int(B),
            int(R), _ptr(n_accept, torch.int32, cuda=False), _ptr(bonus, torch.int32, cuda=False),
            _ptr(target_ids, torch.int32, cuda=False), _stream(stream))
        if rc != OK:
            raise DiscoError(rc, "disco_verify_ragged_host")
