"""ctypes front end of the CPU oracle (oracle/disco_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests/, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this package, and this package never imports them.

Arrays are numpy.  bf16 tensors are passed as uint16 bit patterns
(``torch_tensor.view(torch.uint16).numpy()``).  All floating-point results are
float64.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "disco_oracle.cpp")
_LIB = os.path.join(_HERE, "liboracle.so")

K_TOP = 10  # Eq. 2 footnote: k = 10 in all of the paper's experiments


def build(force: bool = False) -> str:
    """Compile liboracle.so with the host C++ compiler (no CUDA involved)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-pthread", "-o", _LIB, _SRC]
        subprocess.run(cmd, check=True)
    return _LIB


_lib = None


def lib() -> ctypes.CDLL:
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def hardware_threads() -> int:
    return int(lib().oracle_hardware_threads())


# --------------------------------------------------------------------------- helpers
def _p(a, ctype):
    if a is None:
        return None
    return a.ctypes.data_as(ctypes.POINTER(ctype))


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    if a.dtype != np.uint16:
        raise TypeError("bf16 data must be passed as uint16 bit patterns")
    return a


def _check(rc: int, what: str) -> None:
    if rc != 0:
        raise ValueError(f"{what}: oracle rejected its arguments (rc={rc})")


# --------------------------------------------------------------------------- steps
def project(W: np.ndarray, H: np.ndarray, nthreads: int = 1) -> np.ndarray:
    """z[r, v] = sum_j W[v, j] H[r, j] in float64; W [V,d], H [R,d] (bf16 bits)."""
    W, H = _u16(W), _u16(H)
    V, d = W.shape
    R = H.shape[0]
    assert H.shape[1] == d
    z = np.empty((R, V), dtype=np.float64)
    _check(lib().oracle_project(_p(W, ctypes.c_uint16), _p(H, ctypes.c_uint16), V, d, R,
                                _p(z, ctypes.c_double), nthreads), "project")
    return z


def argmax(z: np.ndarray):
    """(lowest index of the maximum, gap between the two largest values)."""
    z = np.ascontiguousarray(z, dtype=np.float64)
    best = ctypes.c_int32()
    gap = ctypes.c_double()
    _check(lib().oracle_argmax(_p(z, ctypes.c_double), z.shape[0], ctypes.byref(best),
                               ctypes.byref(gap)), "argmax")
    return int(best.value), float(gap.value)


def softmax(z: np.ndarray) -> np.ndarray:
    z = np.ascontiguousarray(z, dtype=np.float64)
    y = np.empty_like(z)
    _check(lib().oracle_softmax(_p(z, ctypes.c_double), z.shape[0], _p(y, ctypes.c_double)),
           "softmax")
    return y


def topk(y: np.ndarray, k: int = K_TOP):
    y = np.ascontiguousarray(y, dtype=np.float64)
    vals = np.empty(k, dtype=np.float64)
    ids = np.empty(k, dtype=np.int32)
    _check(lib().oracle_topk(_p(y, ctypes.c_double), y.shape[0], k, _p(vals, ctypes.c_double),
                             _p(ids, ctypes.c_int32)), "topk")
    return vals, ids


def entropy(y: np.ndarray) -> float:
    y = np.ascontiguousarray(y, dtype=np.float64)
    e = ctypes.c_double()
    _check(lib().oracle_entropy(_p(y, ctypes.c_double), y.shape[0], ctypes.byref(e)), "entropy")
    return float(e.value)


def features(y: np.ndarray, pos: int, k: int = K_TOP) -> np.ndarray:
    y = np.ascontiguousarray(y, dtype=np.float64)
    x = np.empty(k + 2, dtype=np.float64)
    _check(lib().oracle_features(_p(y, ctypes.c_double), y.shape[0], k, int(pos),
                                 _p(x, ctypes.c_double)), "features")
    return x


@dataclass
class Classifier:
    """Parameters of the 2-layer halt classifier: nfeat -> H (ReLU) -> 1 (logistic)."""
    W1: np.ndarray  # [H, nfeat] float32
    b1: np.ndarray  # [H]
    w2: np.ndarray  # [H]
    b2: np.ndarray  # [1]

    def __post_init__(self):
        self.W1 = np.ascontiguousarray(self.W1, dtype=np.float32)
        self.b1 = np.ascontiguousarray(self.b1, dtype=np.float32)
        self.w2 = np.ascontiguousarray(self.w2, dtype=np.float32)
        self.b2 = np.ascontiguousarray(self.b2, dtype=np.float32).reshape(1)

    @property
    def H(self) -> int:
        return int(self.W1.shape[0])


def classifier(x: np.ndarray, clf: Classifier) -> float:
    x = np.ascontiguousarray(x, dtype=np.float64)
    C = ctypes.c_double()
    assert clf.W1.shape[1] == x.shape[0]
    _check(lib().oracle_classifier(_p(x, ctypes.c_double), x.shape[0], _p(clf.W1, ctypes.c_float),
                                   _p(clf.b1, ctypes.c_float), _p(clf.w2, ctypes.c_float),
                                   _p(clf.b2, ctypes.c_float), clf.H, ctypes.byref(C)),
           "classifier")
    return float(C.value)


def accept_prefix(draft, target):
    draft = np.ascontiguousarray(draft, dtype=np.int32)
    target = np.ascontiguousarray(target, dtype=np.int32)
    SL = draft.shape[0]
    assert target.shape[0] == SL + 1
    n = ctypes.c_int32()
    bonus = ctypes.c_int32()
    _check(lib().oracle_accept_prefix(_p(draft, ctypes.c_int32) if SL else None,
                                      _p(target, ctypes.c_int32), SL, ctypes.byref(n),
                                      ctypes.byref(bonus)), "accept_prefix")
    return int(n.value), int(bonus.value)


# --------------------------------------------------------------------------- whole calls
@dataclass
class DraftStepResult:
    token: np.ndarray      # [B] int32
    conf: np.ndarray       # [B] float64
    halt: np.ndarray       # [B] uint8
    feats: np.ndarray      # [B, k+2] float64
    gap: np.ndarray        # [B] float64, top-2 logit gap
    topk_ids: np.ndarray   # [B, k] int32
    probs: np.ndarray | None  # [B, V] float64


def draft_step(W_D, h_D, pos, n_drafted, clf: Classifier, tau: float, sl_max: int,
               active=None, want_probs: bool = False, k: int = K_TOP,
               nthreads: int = 1) -> DraftStepResult:
    W_D, h_D = _u16(W_D), _u16(h_D)
    V, d = W_D.shape
    B = h_D.shape[0]
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    n_drafted = np.ascontiguousarray(n_drafted, dtype=np.int32)
    act = None if active is None else np.ascontiguousarray(active, dtype=np.uint8)
    token = np.full(B, -1, dtype=np.int32)
    conf = np.full(B, np.nan)
    halt = np.full(B, 255, dtype=np.uint8)
    feats = np.full((B, k + 2), np.nan)
    gap = np.full(B, np.nan)
    ids = np.full((B, k), -1, dtype=np.int32)
    probs = np.full((B, V), np.nan) if want_probs else None
    _check(lib().oracle_draft_step(
        _p(W_D, ctypes.c_uint16), _p(h_D, ctypes.c_uint16), V, d, B,
        _p(pos, ctypes.c_int32), _p(n_drafted, ctypes.c_int32), _p(act, ctypes.c_uint8),
        _p(clf.W1, ctypes.c_float), _p(clf.b1, ctypes.c_float), _p(clf.w2, ctypes.c_float),
        _p(clf.b2, ctypes.c_float), clf.H, k, ctypes.c_float(tau), int(sl_max),
        _p(token, ctypes.c_int32), _p(conf, ctypes.c_double), _p(halt, ctypes.c_uint8),
        _p(feats, ctypes.c_double), _p(probs, ctypes.c_double), _p(gap, ctypes.c_double),
        _p(ids, ctypes.c_int32), nthreads), "draft_step")
    return DraftStepResult(token, conf, halt, feats, gap, ids, probs)


def draft_step_ppl(W_D, h_D, n_drafted, nll_sum, ppl_max: float, sl_max: int, active=None, nthreads: int = 1):
    """Perplexity stopping rule (App. F).  Returns (token, ppl, halt, gap, new nll_sum)."""
    W_D, h_D = _u16(W_D), _u16(h_D)
    V, d = W_D.shape
    B = h_D.shape[0]
    n_drafted = np.ascontiguousarray(n_drafted, dtype=np.int32)
    nll = np.array(nll_sum, dtype=np.float64).copy()
    act = None if active is None else np.ascontiguousarray(active, dtype=np.uint8)
    token = np.full(B, -1, dtype=np.int32)
    ppl = np.full(B, np.nan)
    halt = np.full(B, 255, dtype=np.uint8)
    gap = np.full(B, np.nan)
    _check(lib().oracle_draft_step_ppl(
        _p(W_D, ctypes.c_uint16), _p(h_D, ctypes.c_uint16), V, d, B, _p(n_drafted, ctypes.c_int32),
        _p(act, ctypes.c_uint8), _p(nll, ctypes.c_double), ctypes.c_float(ppl_max), int(sl_max),
        _p(token, ctypes.c_int32), _p(ppl, ctypes.c_double), _p(halt, ctypes.c_uint8), _p(gap, ctypes.c_double),
        nthreads), "draft_step_ppl")
    return token, ppl, halt, gap, nll


@dataclass
class VerifyResult:
    n_accept: np.ndarray    # [B] int32
    bonus: np.ndarray       # [B] int32
    target_ids: np.ndarray  # [R] int32
    gap: np.ndarray         # [R] float64, top-2 logit gap per row


def verify_ragged(W_T, H_T, draft_ids, row_off, nthreads: int = 1) -> VerifyResult:
    W_T, H_T = _u16(W_T), _u16(H_T)
    V, d = W_T.shape
    row_off = np.ascontiguousarray(row_off, dtype=np.int32)
    B = row_off.shape[0] - 1
    R = int(row_off[-1]) if B >= 0 else 0
    assert H_T.shape[0] == R
    draft_ids = np.ascontiguousarray(draft_ids, dtype=np.int32)
    assert draft_ids.shape[0] == R - B
    n = np.full(B, -1, dtype=np.int32)
    bonus = np.full(B, -1, dtype=np.int32)
    tid = np.full(R, -1, dtype=np.int32)
    gap = np.full(R, np.nan)
    _check(lib().oracle_verify_ragged(
        _p(W_T, ctypes.c_uint16), _p(H_T, ctypes.c_uint16), V, d,
        _p(draft_ids, ctypes.c_int32) if draft_ids.size else None, _p(row_off, ctypes.c_int32), B,
        _p(n, ctypes.c_int32), _p(bonus, ctypes.c_int32), _p(tid, ctypes.c_int32),
        _p(gap, ctypes.c_double), nthreads), "verify_ragged")
    return VerifyResult(n, bonus, tid, gap)


def verify(W_T, H_T, draft_ids, B: int, SL: int, nthreads: int = 1) -> VerifyResult:
    W_T, H_T = _u16(W_T), _u16(H_T)
    V, d = W_T.shape
    R = B * (SL + 1)
    assert H_T.shape[0] == R
    draft_ids = np.ascontiguousarray(draft_ids, dtype=np.int32)
    assert draft_ids.shape[0] == B * SL
    n = np.full(B, -1, dtype=np.int32)
    bonus = np.full(B, -1, dtype=np.int32)
    tid = np.full(R, -1, dtype=np.int32)
    gap = np.full(R, np.nan)
    _check(lib().oracle_verify(
        _p(W_T, ctypes.c_uint16), _p(H_T, ctypes.c_uint16), V, d,
        _p(draft_ids, ctypes.c_int32) if draft_ids.size else None, B, SL,
        _p(n, ctypes.c_int32), _p(bonus, ctypes.c_int32), _p(tid, ctypes.c_int32),
        _p(gap, ctypes.c_double), nthreads), "verify")
    return VerifyResult(n, bonus, tid, gap)


# --------------------------------------------------------------------------- sampling at temperature 1
def sample_cdf(w, u: float):
    """Inverse-CDF draw from non-negative weights.  Returns (token, total weight)."""
    w = np.ascontiguousarray(w, dtype=np.float64)
    tok = ctypes.c_int32(-2)
    total = ctypes.c_double(0.0)
    _check(lib().oracle_sample_cdf(_p(w, ctypes.c_double), w.shape[0], ctypes.c_double(u), ctypes.byref(tok),
                                   ctypes.byref(total)), "sample_cdf")
    return int(tok.value), float(total.value)


@dataclass
class DraftSampleResult:
    token: np.ndarray      # [B] int32, drawn from y^D
    p_token: np.ndarray    # [B] float64, y^D(token)
    conf: np.ndarray       # [B] float64
    halt: np.ndarray       # [B] uint8
    feats: np.ndarray      # [B, k+2] float64
    probs: np.ndarray      # [B, V] float64


def draft_step_sample(W_D, h_D, pos, n_drafted, clf: Classifier, tau: float, sl_max: int, u,
                      active=None, k: int = K_TOP, nthreads: int = 1) -> DraftSampleResult:
    W_D, h_D = _u16(W_D), _u16(h_D)
    V, d = W_D.shape
    B = h_D.shape[0]
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    n_drafted = np.ascontiguousarray(n_drafted, dtype=np.int32)
    u = np.ascontiguousarray(u, dtype=np.float64)
    assert u.shape[0] == B
    act = None if active is None else np.ascontiguousarray(active, dtype=np.uint8)
    token = np.full(B, -1, dtype=np.int32)
    p_token = np.full(B, np.nan)
    conf = np.full(B, np.nan)
    halt = np.full(B, 255, dtype=np.uint8)
    feats = np.full((B, k + 2), np.nan)
    probs = np.full((B, V), np.nan)
    ctypes_f = ctypes.c_float
    fn = lib().oracle_draft_step_sample
    fn.restype = ctypes.c_int
    _check(fn(
        _p(W_D, ctypes.c_uint16), _p(h_D, ctypes.c_uint16), V, d, B,
        _p(pos, ctypes.c_int32), _p(n_drafted, ctypes.c_int32), _p(act, ctypes.c_uint8),
        _p(clf.W1, ctypes_f), _p(clf.b1, ctypes_f), _p(clf.w2, ctypes_f), _p(clf.b2, ctypes_f), clf.H, k,
        ctypes_f(tau), int(sl_max), _p(u, ctypes.c_double),
        _p(token, ctypes.c_int32), _p(p_token, ctypes.c_double), _p(conf, ctypes.c_double),
        _p(halt, ctypes.c_uint8), _p(feats, ctypes.c_double), _p(probs, ctypes.c_double), nthreads),
        "draft_step_sample")
    return DraftSampleResult(token, p_token, conf, halt, feats, probs)


def speculative_sample(yT, yD, tokens, ua, us: float):
    """One sequence of speculative sampling on given distributions.  yT [(SL+1), V], yD [SL, V].
    Returns (n_accept, next_token)."""
    yT = np.ascontiguousarray(yT, dtype=np.float64)
    SL = yT.shape[0] - 1
    V = yT.shape[1]
    yD = np.ascontiguousarray(yD, dtype=np.float64).reshape(SL, V)
    tokens = np.ascontiguousarray(tokens, dtype=np.int32)
    ua = np.ascontiguousarray(ua, dtype=np.float64)
    assert tokens.shape[0] == SL and ua.shape[0] == SL
    n = ctypes.c_int32(-1)
    nxt = ctypes.c_int32(-1)
    _check(lib().oracle_speculative_sample(
        _p(yT, ctypes.c_double), _p(yD, ctypes.c_double) if SL else None,
        _p(tokens, ctypes.c_int32) if SL else None, SL, V, _p(ua, ctypes.c_double) if SL else None,
        ctypes.c_double(us), ctypes.byref(n), ctypes.byref(nxt)), "speculative_sample")
    return int(n.value), int(nxt.value)


@dataclass
class VerifySampleResult:
    n_accept: np.ndarray    # [B] int32
    next_token: np.ndarray  # [B] int32
    y_T: np.ndarray         # [R, V] float64 target distributions


def verify_sample(W_T, H_T, draft_ids, draft_probs, row_off, ua, us, nthreads: int = 1) -> VerifySampleResult:
    """Stochastic verification.  draft_probs: float32 [steps, B, V] (step-major); ua packed like draft_ids; us [B]."""
    W_T, H_T = _u16(W_T), _u16(H_T)
    V, d = W_T.shape
    row_off = np.ascontiguousarray(row_off, dtype=np.int32)
    B = row_off.shape[0] - 1
    R = int(row_off[-1])
    assert H_T.shape[0] == R
    draft_ids = np.ascontiguousarray(draft_ids, dtype=np.int32)
    assert draft_ids.shape[0] == R - B
    ua = np.ascontiguousarray(ua, dtype=np.float64)
    us = np.ascontiguousarray(us, dtype=np.float64)
    assert ua.shape[0] == R - B and us.shape[0] == B
    dp = np.ascontiguousarray(draft_probs, dtype=np.float32)
    if R - B:
        max_sl = int(np.max(np.diff(row_off))) - 1
        assert dp.shape[0] >= max_sl and dp.shape[1] == B and dp.shape[2] == V
    n = np.full(B, -1, dtype=np.int32)
    nxt = np.full(B, -1, dtype=np.int32)
    yT = np.full((R, V), np.nan)
    _check(lib().oracle_verify_sample(
        _p(W_T, ctypes.c_uint16), _p(H_T, ctypes.c_uint16), V, d,
        _p(draft_ids, ctypes.c_int32) if draft_ids.size else None,
        _p(dp, ctypes.c_float) if draft_ids.size else None, _p(row_off, ctypes.c_int32), B,
        _p(ua, ctypes.c_double) if ua.size else None, _p(us, ctypes.c_double),
        _p(n, ctypes.c_int32), _p(nxt, ctypes.c_int32), _p(yT, ctypes.c_double), nthreads), "verify_sample")
    return VerifySampleResult(n, nxt, yT)


# --------------------------------------------------------------------------- bulk feature extraction (App. D)
def total_variation(p, q) -> float:
    p = np.ascontiguousarray(p, dtype=np.float64)
    q = np.ascontiguousarray(q, dtype=np.float64)
    assert p.shape == q.shape and p.ndim == 1
    tv = ctypes.c_double(-1.0)
    _check(lib().oracle_total_variation(_p(p, ctypes.c_double), _p(q, ctypes.c_double), p.shape[0], ctypes.byref(tv)),
           "total_variation")
    return float(tv.value)


@dataclass
class FeatureRows:
    feats_D: np.ndarray   # [N, k+2] float64
    feats_T: np.ndarray   # [N, k+2] float64
    tv: np.ndarray        # [N] float64
    label: np.ndarray     # [N] uint8, 1 = accepted
    token_D: np.ndarray   # [N] int32
    token_T: np.ndarray   # [N] int32
    gap_D: np.ndarray     # [N] float64, top-2 logit gaps
    gap_T: np.ndarray


def extract_features(W_D, H_D, W_T, H_T, pos, k: int = K_TOP, nthreads: int = 1) -> FeatureRows:
    W_D, H_D, W_T, H_T = _u16(W_D), _u16(H_D), _u16(W_T), _u16(H_T)
    V, d_D = W_D.shape
    V2, d_T = W_T.shape
    N = H_D.shape[0]
    assert V == V2 and H_T.shape[0] == N and H_D.shape[1] == d_D and H_T.shape[1] == d_T
    pos = np.ascontiguousarray(pos, dtype=np.int32)
    assert pos.shape[0] == N
    fD = np.full((N, k + 2), np.nan)
    fT = np.full((N, k + 2), np.nan)
    tv = np.full(N, np.nan)
    label = np.full(N, 255, dtype=np.uint8)
    tD = np.full(N, -1, dtype=np.int32)
    tT = np.full(N, -1, dtype=np.int32)
    gD = np.full(N, np.nan)
    gT = np.full(N, np.nan)
    _check(lib().oracle_extract_features(
        _p(W_D, ctypes.c_uint16), _p(H_D, ctypes.c_uint16), d_D, _p(W_T, ctypes.c_uint16), _p(H_T, ctypes.c_uint16),
        d_T, V, N, _p(pos, ctypes.c_int32), k, _p(fD, ctypes.c_double), _p(fT, ctypes.c_double),
        _p(tv, ctypes.c_double), _p(label, ctypes.c_uint8), _p(tD, ctypes.c_int32), _p(tT, ctypes.c_int32),
        _p(gD, ctypes.c_double), _p(gT, ctypes.c_double), nthreads), "extract_features")
    return FeatureRows(fD, fT, tv, label, tD, tT, gD, gT)


# --------------------------------------------------------------------------- whole iteration (Sec. 3)
@dataclass
class IterationResult:
    token: np.ndarray       # [sl_max, B] int32, -1 where the sequence had stopped
    conf: np.ndarray        # [sl_max, B] float64 (nan where not taken)
    halt: np.ndarray        # [sl_max, B] uint8 (255 where not taken)
    feats: np.ndarray       # [sl_max, B, k+2]
    gap_D: np.ndarray       # [sl_max, B] top-2 logit gap of each draft step
    sl: np.ndarray          # [B] int32 tokens drafted
    n_accept: np.ndarray | None   # [B]
    bonus: np.ndarray | None      # [B]
    target_ids: np.ndarray | None  # [B, sl_max+1], -1 beyond sl[b]
    gap_T: np.ndarray | None       # [B, sl_max+1]


def _clf_args(clf: Classifier):
    f = ctypes.c_float
    return _p(clf.W1, f), _p(clf.b1, f), _p(clf.w2, f), _p(clf.b2, f), clf.H


def draft_loop(W_D, h_D, pos0, clf: Classifier, tau: float, sl_max: int, sl_forced=None, k: int = K_TOP,
               nthreads: int = 1) -> IterationResult:
    """Draft phase of one iteration.  h_D: bf16 bits [sl_max, B, d]."""
    W_D, h_D = _u16(W_D), _u16(h_D)
    V, d = W_D.shape
    S, B = h_D.shape[0], h_D.shape[1]
    assert S == sl_max and h_D.shape[2] == d
    pos0 = np.ascontiguousarray(pos0, dtype=np.int32)
    forced = None if sl_forced is None else np.ascontiguousarray(sl_forced, dtype=np.int32)
    token = np.full((S, B), -1, dtype=np.int32)
    conf = np.full((S, B), np.nan)
    halt = np.full((S, B), 255, dtype=np.uint8)
    feats = np.full((S, B, k + 2), np.nan)
    gap = np.full((S, B), np.nan)
    sl = np.full(B, -1, dtype=np.int32)
    _check(lib().oracle_draft_loop(
        _p(W_D, ctypes.c_uint16), _p(h_D, ctypes.c_uint16), V, d, B, _p(pos0, ctypes.c_int32), *_clf_args(clf), k,
        ctypes.c_float(tau), int(sl_max), _p(forced, ctypes.c_int32), _p(token, ctypes.c_int32),
        _p(conf, ctypes.c_double), _p(halt, ctypes.c_uint8), _p(feats, ctypes.c_double), _p(gap, ctypes.c_double),
        _p(sl, ctypes.c_int32), nthreads), "draft_loop")
    return IterationResult(token, conf, halt, feats, gap, sl, None, None, None, None)


def verify_padded(W_T, H_T, sl, draft, stride_b: int, stride_j: int, nthreads: int = 1):
    """Verification in the fixed-shape layout.  H_T: bf16 bits [B, sl_max+1, d]; draft: int32, token j of
    sequence b at draft.flat[b * stride_b + j * stride_j].  Returns (n_accept, bonus, target_ids, gap)."""
    W_T, H_T = _u16(W_T), _u16(H_T)
    V, d = W_T.shape
    B, S1 = H_T.shape[0], H_T.shape[1]
    sl = np.ascontiguousarray(sl, dtype=np.int32)
    draft = None if draft is None else np.ascontiguousarray(draft, dtype=np.int32)
    n = np.full(B, -1, dtype=np.int32)
    bonus = np.full(B, -1, dtype=np.int32)
    tid = np.full((B, S1), -1, dtype=np.int32)
    gap = np.full((B, S1), np.nan)
    _check(lib().oracle_verify_padded(
        _p(W_T, ctypes.c_uint16), _p(H_T, ctypes.c_uint16), V, d, B, S1 - 1, _p(sl, ctypes.c_int32),
        _p(draft, ctypes.c_int32), ctypes.c_longlong(stride_b), ctypes.c_longlong(stride_j), _p(n, ctypes.c_int32),
        _p(bonus, ctypes.c_int32), _p(tid, ctypes.c_int32), _p(gap, ctypes.c_double), nthreads), "verify_padded")
    return n, bonus, tid, gap


def iteration(W_D, h_D, W_T, H_T, pos0, clf: Classifier, tau: float, sl_max: int, sl_forced=None, draft_ids=None,
              k: int = K_TOP, nthreads: int = 1) -> IterationResult:
    """One whole iteration: draft phase, then verification of what it drafted (draft_ids None) or of the
    ids given ([B, sl_max])."""
    W_D, h_D, W_T, H_T = _u16(W_D), _u16(h_D), _u16(W_T), _u16(H_T)
    V, d_D = W_D.shape
    d_T = W_T.shape[1]
    S, B = h_D.shape[0], h_D.shape[1]
    assert S == sl_max and H_T.shape == (B, S + 1, d_T) and W_T.shape[0] == V
    pos0 = np.ascontiguousarray(pos0, dtype=np.int32)
    forced = None if sl_forced is None else np.ascontiguousarray(sl_forced, dtype=np.int32)
    ids = None if draft_ids is None else np.ascontiguousarray(draft_ids, dtype=np.int32)
    assert ids is None or ids.shape == (B, S)
    token = np.full((S, B), -1, dtype=np.int32)
    conf = np.full((S, B), np.nan)
    halt = np.full((S, B), 255, dtype=np.uint8)
    feats = np.full((S, B, k + 2), np.nan)
    gapD = np.full((S, B), np.nan)
    sl = np.full(B, -1, dtype=np.int32)
    n = np.full(B, -1, dtype=np.int32)
    bonus = np.full(B, -1, dtype=np.int32)
    tid = np.full((B, S + 1), -1, dtype=np.int32)
    gapT = np.full((B, S + 1), np.nan)
    _check(lib().oracle_iteration(
        _p(W_D, ctypes.c_uint16), _p(h_D, ctypes.c_uint16), d_D, _p(W_T, ctypes.c_uint16), _p(H_T, ctypes.c_uint16),
        d_T, V, B, _p(pos0, ctypes.c_int32), *_clf_args(clf), k, ctypes.c_float(tau), int(sl_max),
        _p(forced, ctypes.c_int32), _p(ids, ctypes.c_int32), _p(token, ctypes.c_int32), _p(conf, ctypes.c_double),
        _p(halt, ctypes.c_uint8), _p(feats, ctypes.c_double), _p(gapD, ctypes.c_double), _p(sl, ctypes.c_int32),
        _p(n, ctypes.c_int32), _p(bonus, ctypes.c_int32), _p(tid, ctypes.c_int32), _p(gapT, ctypes.c_double),
        nthreads), "iteration")
    return IterationResult(token, conf, halt, feats, gapD, sl, n, bonus, tid, gapT)
