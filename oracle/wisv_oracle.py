"""Python face of the CPU oracle (test infrastructure only).

Loads the plain-C routines of ``wisv_oracle.c`` and composes them into one
verification round exactly in the order of Algorithm 1: LM-head logits, mismatch
localisation, decision head on the candidate positions, first-reject scan,
emission of the accepted length and the correction token.  Only tests, the smoke
check and the CPU-baseline leg of the benchmark may import this module; the
CUDA library never does.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Dict, Optional

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "wisv_oracle.c")
_LIB = os.path.join(_HERE, "libwisv_oracle.so")
_lib = None

ACT_RELU, ACT_GELU = 0, 1


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (portable flags; no -march)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".%d.tmp" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-fopenmp", "-shared", "-fPIC",
                               "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        lib = ctypes.CDLL(_LIB)
        c = ctypes
        P = c.c_void_p
        lib.wisv_oracle_threads.restype = c.c_int
        lib.wisv_oracle_lm_head.restype = c.c_int
        lib.wisv_oracle_lm_head.argtypes = [P, P, c.c_int64, c.c_int32, c.c_int32, P, P, P, P, P, P]
        lib.wisv_oracle_head.restype = c.c_int
        lib.wisv_oracle_head.argtypes = [P, P, P, c.c_double, c.c_int32, c.c_int32, c.c_int32,
                                         c.c_int32, c.c_int32, P, P, P, P, P, c.c_int64, P, P]
        lib.wisv_oracle_scan.restype = c.c_int
        lib.wisv_oracle_scan.argtypes = [c.c_int32, P, P, P, P, c.c_double, P, P, P]
        _lib = lib
    return _lib


def threads() -> int:
    return int(_load().wisv_oracle_threads())


def _p(a: Optional[np.ndarray]):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _c(a, dtype):
    return np.ascontiguousarray(a, dtype=dtype)


def lm_head(lm_head_bits: np.ndarray, target_hidden: np.ndarray,
            row_token: Optional[np.ndarray] = None, want_logits: bool = False) -> Dict[str, np.ndarray]:
    """Logits rows reduced to argmax / logsumexp / one requested logit / top-2 gap."""
    W = _c(lm_head_bits, np.uint16)
    Ht = _c(target_hidden, np.float32)
    V, H = W.shape
    R = Ht.shape[0]
    assert Ht.shape[1] == H
    tok = None if row_token is None else _c(row_token, np.int32)
    argmax = np.zeros(R, np.int32)
    lse = np.zeros(R, np.float64)
    tok_logit = np.full(R, np.nan, np.float64)
    gap = np.zeros(R, np.float64)
    logits = np.zeros((R, V), np.float64) if want_logits else None
    rc = _load().wisv_oracle_lm_head(_p(W), _p(Ht), R, H, V, _p(tok), _p(argmax), _p(lse),
                                     _p(tok_logit), _p(gap), _p(logits))
    if rc != 0:
        raise RuntimeError("wisv_oracle_lm_head failed: %d" % rc)
    out = dict(argmax=argmax, lse=lse, tok_logit=tok_logit, top2_gap=gap)
    if want_logits:
        out["logits"] = logits
    return out


def head(W1_bits, b1, w2, b2, H, H_d, d_c, act, draft_hidden, target_hidden, csi, tgt_row, req
         ) -> Dict[str, np.ndarray]:
    """Decision-head logit and rejection probability for P evaluated positions."""
    W1 = _c(W1_bits, np.uint16)
    d_J = W1.shape[0]
    assert W1.shape[1] == H_d + H + d_c
    hD = _c(draft_hidden, np.float32).reshape(-1, max(H_d, 1))
    Ht = _c(target_hidden, np.float32)
    cs = _c(csi, np.float32)
    tr = _c(tgt_row, np.int32)
    rq = _c(req, np.int32)
    P = tr.shape[0]
    s = np.zeros(P, np.float64)
    p = np.zeros(P, np.float64)
    rc = _load().wisv_oracle_head(_p(W1), _p(_c(b1, np.float32)), _p(_c(w2, np.float32)), float(b2),
                                  H, H_d, d_c, d_J, int(act), _p(hD), _p(Ht), _p(cs), _p(tr), _p(rq),
                                  P, _p(s), _p(p))
    if rc != 0:
        raise RuntimeError("wisv_oracle_head failed: %d" % rc)
    return dict(logit=s, prob=p)


def scan(k_off, cand, has_prob, prob, tau, argmax):
    """First-reject scan; returns (accept_len, correction_token)."""
    k_off = _c(k_off, np.int32)
    B = k_off.shape[0] - 1
    cand = _c(cand, np.uint8)
    has_prob = _c(has_prob, np.uint8)
    prob = _c(prob, np.float64)
    argmax = _c(argmax, np.int32)
    A = np.zeros(B, np.int32)
    corr = np.zeros(B, np.int32)
    rc = _load().wisv_oracle_scan(B, _p(k_off), _p(cand), _p(has_prob), _p(prob), float(tau),
                                  _p(argmax), _p(A), _p(corr))
    if rc != 0:
        raise RuntimeError("wisv_oracle_scan failed: %d" % rc)
    return A, corr


def hidden_as_f32(x) -> np.ndarray:
    """Hidden states as the fp32 array the definition starts from.

    The drafter uploads 16-bit hidden states (Section IV-A, b_h = 16): an fp16 array (numpy float16) is widened
    exactly; bf16 values arrive as uint16 bit patterns and are widened exactly as well.  The rounding to bf16 that
    precedes every matrix product is then applied by the C routines as for fp32 inputs: it leaves bf16 values as
    they are and rounds fp16 values to nearest even.
    """
    x = np.asarray(x)
    if x.dtype == np.uint16:
        return (x.astype(np.uint32) << np.uint32(16)).view(np.float32)
    return np.ascontiguousarray(x, dtype=np.float32)


def verify(*, lm_head_bits, W1_bits, b1, w2, b2, act, tau, k_len, target_hidden, draft_tokens,
           draft_hidden, csi, sel_off=None, sel_pos=None, draft_q=None, uniforms=None,
           head_row_shift: int = 0) -> Dict[str, np.ndarray]:
    """One verification round for a batch of windows.

    Row r = row_off[b] + i (i = 0..K_b) holds the target hidden state whose logits
    predict draft token i; row K_b gives the bonus token of a full accept.
    sel_off/sel_pos = None means full-hidden upload (draft_hidden is [T, H_d]);
    otherwise draft_hidden is the packed [M_sel, H_d] of selective-hidden upload.
    draft_q/uniforms given => candidates come from the speculative-sampling test
    u < min(1, p_T(y)/p_D(y)) (Eq. 1) instead of the greedy argmax comparison.
    """
    k_len = np.asarray(k_len, np.int32)
    B = k_len.shape[0]
    k_off = np.zeros(B + 1, np.int32)
    k_off[1:] = np.cumsum(k_len)
    row_off = k_off + np.arange(B + 1, dtype=np.int32)
    T, R = int(k_off[-1]), int(row_off[-1])
    W = _c(lm_head_bits, np.uint16)
    V, H = W.shape
    Ht = hidden_as_f32(target_hidden)
    assert Ht.shape == (R, H)
    draft_hidden = hidden_as_f32(draft_hidden)
    draft_tokens = _c(draft_tokens, np.int32)
    H_d = int(np.asarray(draft_hidden).shape[1]) if np.asarray(draft_hidden).ndim == 2 else 0
    csi = _c(csi, np.float32).reshape(B, -1)
    d_c = csi.shape[1]

    # window-row bookkeeping
    req_of_t = np.repeat(np.arange(B, dtype=np.int32), k_len)
    i_of_t = (np.arange(T, dtype=np.int32) - k_off[req_of_t]).astype(np.int32)
    row_of_t = (row_off[req_of_t] + i_of_t).astype(np.int32)
    row_token = np.full(R, -1, np.int32)
    row_token[row_of_t] = draft_tokens

    # Verify: logits -> argmax, logsumexp, target probability of the draft token
    lm = lm_head(W, Ht, row_token)
    p_draft = np.exp(lm["tok_logit"][row_of_t] - lm["lse"][row_of_t])

    # Localize: candidate set S
    if draft_q is None:
        cand = draft_tokens != lm["argmax"][row_of_t]
        alpha = None
    else:
        alpha = np.minimum(1.0, p_draft / np.asarray(draft_q, np.float64))
        cand = ~(np.asarray(uniforms, np.float64) < alpha)

    # positions whose drafter hidden state is available
    if sel_off is None:
        eval_t = np.arange(T, dtype=np.int32)
    else:
        sel_off = np.asarray(sel_off, np.int32)
        sel_pos = np.asarray(sel_pos, np.int32)
        req_of_sel = np.repeat(np.arange(B, dtype=np.int32), np.diff(sel_off))
        eval_t = (k_off[req_of_sel] + sel_pos).astype(np.int32)
    tgt_row = (row_of_t[eval_t] + head_row_shift).astype(np.int32)
    hd = head(W1_bits, b1, w2, b2, H, H_d, d_c, act, draft_hidden, Ht, csi, tgt_row, req_of_t[eval_t])

    has_prob = np.zeros(T, np.uint8)
    prob = np.zeros(T, np.float64)
    has_prob[eval_t] = 1
    prob[eval_t] = hd["prob"]

    A, corr = scan(k_off, cand.astype(np.uint8), has_prob, prob, tau, lm["argmax"])
    n_mismatch = np.bincount(req_of_t, weights=cand.astype(np.float64), minlength=B).astype(np.int32)   # |S| per request
    return dict(accept_len=A, correction_token=corr, argmax=lm["argmax"], lse=lm["lse"],
                top2_gap=lm["top2_gap"], p_draft=p_draft, cand=cand, n_mismatch=n_mismatch,
                head_prob=hd["prob"], head_logit=hd["logit"], eval_t=eval_t, has_prob=has_prob,
                prob_t=prob, alpha=alpha, k_off=k_off, row_off=row_off, row_of_t=row_of_t,
                req_of_t=req_of_t)
