"""ctypes binding of include/wisv.h (argument marshalling only)."""
from __future__ import annotations

import ctypes as C
import math
import os
import re
from dataclasses import dataclass
from typing import List, Optional

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "libwisv.so")
_HEADER = os.path.join(os.path.dirname(_HERE), "include", "wisv.h")
_lib = None

ACT_RELU, ACT_GELU = 0, 1
MODE_FH, MODE_SH = 0, 1
ACCEPT_GREEDY, ACCEPT_STOCHASTIC = 0, 2
DT_F32, DT_BF16, DT_F16 = 0, 1, 2


def _hidden_dtype(t) -> int:
    """WISV_DT_* of a hidden-state tensor (fp32, bf16 or fp16)."""
    if t is None:
        return DT_F32
    name = str(t.dtype)
    if name.endswith("float32"):
        return DT_F32
    if name.endswith("bfloat16"):
        return DT_BF16
    if name.endswith("float16"):
        return DT_F16
    raise ValueError("hidden states must be float32, bfloat16 or float16, not %s" % name)


class WisvError(RuntimeError):
    def __init__(self, code: int, what: str):
        super().__init__("%s failed: %s (%d)" % (what, _strerror(code), code))
        self.code = code


class _Config(C.Structure):
    _fields_ = [("H", C.c_int32), ("V", C.c_int32), ("H_d", C.c_int32), ("d_c", C.c_int32), ("d_J", C.c_int32),
                ("act", C.c_int32), ("head_row_shift", C.c_int32), ("tau", C.c_float),
                ("max_requests", C.c_int32), ("max_rows", C.c_int32), ("max_sel", C.c_int32),
                ("vocab_base", C.c_int32), ("vocab_total", C.c_int32)]


class _Weights(C.Structure):
    _fields_ = [("lm_head", C.c_void_p), ("W1", C.c_void_p), ("b1", C.c_void_p), ("w2", C.c_void_p),
                ("b2", C.c_float)]


class _Batch(C.Structure):
    _fields_ = [("B", C.c_int32), ("K", C.c_int32), ("k_off", C.c_void_p), ("T_total", C.c_int32),
                ("target_hidden", C.c_void_p), ("draft_tokens", C.c_void_p), ("draft_hidden", C.c_void_p),
                ("sel_off", C.c_void_p), ("sel_pos", C.c_void_p), ("M_sel", C.c_int32), ("csi", C.c_void_p),
                ("draft_q", C.c_void_p), ("uniforms", C.c_void_p), ("mode", C.c_uint32), ("tau", C.c_float),
                ("target_hidden_dtype", C.c_int32), ("draft_hidden_dtype", C.c_int32)]


class _Result(C.Structure):
    _fields_ = [("accept_len", C.c_void_p), ("correction_token", C.c_void_p), ("argmax", C.c_void_p),
                ("lse", C.c_void_p), ("p_draft", C.c_void_p), ("head_prob", C.c_void_p),
                ("mismatch_mask", C.c_void_p), ("n_mismatch", C.c_void_p), ("status", C.c_void_p)]


class _Tuning(C.Structure):
    _fields_ = [("lm_tile_n", C.c_int32), ("lm_stages", C.c_int32), ("head_tile_n", C.c_int32),
                ("head_stages", C.c_int32), ("lm_single_cta", C.c_int32), ("head_ctas", C.c_int32),
                ("lm_mma_m", C.c_int32), ("lm_kb_per_stage", C.c_int32), ("lm_teams", C.c_int32)]


class LinkParams(C.Structure):
    _fields_ = [("rate_up_bps", C.c_double), ("rate_down_bps", C.c_double), ("per_up", C.c_double),
                ("per_down", C.c_double), ("rtt_s", C.c_double), ("hdr_up_bits", C.c_double),
                ("hdr_down_bits", C.c_double), ("d_h", C.c_int32), ("b_h", C.c_int32), ("b_pos", C.c_int32)]


class LinkCost(C.Structure):
    _fields_ = [("b_id", C.c_int32), ("B_hid", C.c_double), ("B_fb", C.c_double), ("B_u_FH", C.c_double),
                ("B_u1_SH", C.c_double), ("B_req", C.c_double), ("B_u2_SH", C.c_double),
                ("T_comm_FH", C.c_double), ("T_comm_SH", C.c_double)]


def link_cost_round(link: "LinkParams", V: int, K_r: int, m_r: int) -> dict:
    """wisv_link_cost_round: payloads (bits) and communication latencies (s) of one round."""
    out = LinkCost()
    _check(load_library().wisv_link_cost_round(C.byref(link), V, K_r, m_r, C.byref(out)), "wisv_link_cost_round")
    return {n: getattr(out, n) for n, _ in LinkCost._fields_}


class PlanInfo(C.Structure):
    _fields_ = [(n, C.c_int32) for n in (
        "kernels", "head_in_lm_launch",
        "lm_pair", "lm_carry", "lm_tile_n", "lm_ctas", "lm_m_tiles", "lm_n_tiles", "lm_stages", "lm_smem_bytes",
        "lm_units_base", "lm_units_rem", "lm_tiles_per_cta", "lm_rounds", "lm_rounds_alone",
        "head_carry", "head_tile_n", "head_ctas", "head_m_tiles", "head_n_tiles", "head_k_splits",
        "head_kb_per_split", "head_stages", "head_smem_bytes", "head_units_base", "head_units_rem",
        "head_tiles_per_cta", "lm_n_cols", "lm_row_blocks", "lm_parts")]


def plan_host(*, H: int, V: int, H_d: int, d_c: int, d_J: int, R: int, P: int, sm_count: int = 148,
              max_smem_bytes: int = 232448):
    """wisv_plan_host: the launch plan for a batch shape on a device of the given size (host arithmetic only)."""
    cfg = _Config(H, V, H_d, d_c, d_J, ACT_GELU, 0, 0.5, 1, max(R, 1), 0, 0, 0)
    out = PlanInfo()
    lib = load_library()
    lib.wisv_plan_host.restype = C.c_int
    lib.wisv_plan_host.argtypes = [C.POINTER(_Config), C.c_int32, C.c_int32, C.c_int32, C.c_int32, C.POINTER(PlanInfo)]
    _check(lib.wisv_plan_host(C.byref(cfg), sm_count, max_smem_bytes, R, P, C.byref(out)), "wisv_plan_host")
    return {n: getattr(out, n) for n, _ in PlanInfo._fields_}


def choose_protocol(rtt_s: float) -> int:
    return int(load_library().wisv_choose_protocol(float(rtt_s)))


def exported_symbols() -> List[str]:
    """Function names declared in include/wisv.h."""
    text = open(_HEADER).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(wisv_[a-z_]+)\s*\(", text)))


def load_library(build_if_missing: bool = False):
    """Load libwisv.so (raises if it has not been built: there is no fallback)."""
    global _lib
    if _lib is not None:
        return _lib
    if build_if_missing:
        from . import build as _b
        _b.build()
    if not os.path.exists(_LIB_PATH):
        raise RuntimeError("libwisv.so is not built (run paper_2604_17701_b200/build.py); "
                           "the verifier has no fallback path")
    lib = C.CDLL(_LIB_PATH)
    P = C.c_void_p
    lib.wisv_version.restype = C.c_int
    lib.wisv_strerror.restype = C.c_char_p
    lib.wisv_strerror.argtypes = [C.c_int]
    lib.wisv_create.restype = C.c_int
    lib.wisv_create.argtypes = [C.POINTER(_Config), C.POINTER(_Weights), C.POINTER(P)]
    lib.wisv_destroy.restype = C.c_int
    lib.wisv_destroy.argtypes = [P]
    for name in ("wisv_verify", "wisv_verify_host", "wisv_localize", "wisv_decide"):
        f = getattr(lib, name)
        f.restype = C.c_int
        f.argtypes = [P, C.POINTER(_Batch), C.POINTER(_Result), P]
    lib.wisv_shard_rows.restype = C.c_int
    lib.wisv_shard_rows.argtypes = [P, C.POINTER(_Batch), P, P]
    lib.wisv_verify_gathered.restype = C.c_int
    lib.wisv_verify_gathered.argtypes = [P, C.POINTER(_Batch), P, C.c_int32, C.POINTER(_Result), P]
    lib.wisv_device_error.restype = C.c_int
    lib.wisv_device_error.argtypes = [P, P, C.POINTER(C.c_int32)]
    lib.wisv_profile_enable.restype = C.c_int
    lib.wisv_profile_enable.argtypes = [P, C.c_int32]
    lib.wisv_profile_read.restype = C.c_int
    lib.wisv_profile_read.argtypes = [P, C.c_int32, C.POINTER(C.c_float), C.c_int32, C.POINTER(C.c_int32)]
    lib.wisv_launch_count.restype = C.c_int64
    lib.wisv_launch_count.argtypes = [P]
    lib.wisv_plan.restype = C.c_int
    lib.wisv_plan.argtypes = [P, C.c_int32, C.c_int32] + [C.POINTER(C.c_int32)] * 6
    lib.wisv_debug_wait_probe.restype = C.c_int
    lib.wisv_debug_wait_probe.argtypes = [P, C.c_uint64, P]
    lib.wisv_debug_logits.restype = C.c_int
    lib.wisv_debug_logits.argtypes = [P, P, C.c_int32, P, P]
    lib.wisv_link_cost_round.restype = C.c_int
    lib.wisv_link_cost_round.argtypes = [C.POINTER(LinkParams), C.c_int32, C.c_int32, C.c_int32, C.POINTER(LinkCost)]
    lib.wisv_choose_protocol.restype = C.c_int
    lib.wisv_choose_protocol.argtypes = [C.c_double]
    lib.wisv_plan_kernels.restype = C.c_int
    lib.wisv_plan_kernels.argtypes = [P, C.c_int32, C.c_int32]
    lib.wisv_set_tuning.restype = C.c_int
    lib.wisv_set_tuning.argtypes = [P, C.POINTER(_Tuning)]
    lib.wisv_debug_poison.restype = C.c_int
    lib.wisv_debug_poison.argtypes = [P, P]
    lib.wisv_debug_poison_static.restype = C.c_int
    lib.wisv_debug_poison_static.argtypes = [P]
    lib.wisv_lm_head_reduce_static.restype = C.c_int
    lib.wisv_lm_head_reduce_static.argtypes = [P, C.c_int32, C.c_int32, P, C.c_int32, P, P, P]
    _lib = lib
    return lib


def _strerror(code: int) -> str:
    try:
        return load_library().wisv_strerror(code).decode()
    except Exception:
        return "error"


def _check(code: int, what: str):
    if code != 0:
        raise WisvError(code, what)


def _ptr(t) -> Optional[int]:
    return None if t is None else t.data_ptr()


@dataclass
class VerifyOutput:
    accept_len: "object"
    correction_token: "object"
    argmax: "object" = None
    lse: "object" = None
    p_draft: "object" = None
    head_prob: "object" = None
    mismatch_mask: "object" = None
    n_mismatch: "object" = None
    status: "object" = None


class BoundHostCall:
    """One wisv_verify_host call with its arguments already marshalled (see Verifier.bind_host)."""

    def __init__(self, verifier, batch, result, out, stream, keep):
        self._v, self._b, self._r, self.out, self._keep = verifier, batch, result, out, keep
        self._fn = verifier.lib.wisv_verify_host
        self._args = (verifier._h, C.byref(batch), C.byref(result), C.c_void_p(stream.cuda_stream))
        self._dev = verifier.device.index if verifier.device.index is not None else 0
        self._current_device = verifier._torch.cuda.current_device

    def __call__(self) -> "VerifyOutput":
        if self._current_device() != self._dev:
            with self._v._torch.cuda.device(self._dev):
                _check(self._fn(*self._args), "wisv_verify_host")
        else:
            _check(self._fn(*self._args), "wisv_verify_host")
        return self.out


class Verifier:
    """wisv_create / wisv_verify / wisv_destroy on torch CUDA tensors.

    lm_head: bf16 [V, H]; W1: bf16 [d_J, H_d + H + d_c]; b1, w2: fp32 [d_J].
    The tensors are borrowed: keep them alive as long as the Verifier.
    """

    def __init__(self, lm_head, W1, b1, w2, b2: float, *, H_d: int, d_c: int, act: int = ACT_GELU,
                 tau: float = 0.5, head_row_shift: int = 0, max_requests: int, max_rows: int, max_sel: int = 0,
                 vocab_base: int = 0, vocab_total: int = 0):
        import torch
        self._torch = torch
        self.lib = load_library()
        for t, dt in ((lm_head, torch.bfloat16), (W1, torch.bfloat16), (b1, torch.float32), (w2, torch.float32)):
            if not (t.is_cuda and t.is_contiguous() and t.dtype == dt):
                raise ValueError("weights must be contiguous CUDA tensors of the documented dtype")
        V, H = lm_head.shape
        d_J = W1.shape[0]
        if W1.shape[1] != H_d + H + d_c:
            raise ValueError("W1 must be [d_J, H_d + H + d_c]")
        self.H, self.V, self.H_d, self.d_c, self.d_J = H, V, H_d, d_c, d_J
        self._keep = (lm_head, W1, b1, w2)
        self.device = lm_head.device
        cfg = _Config(H, V, H_d, d_c, d_J, act, head_row_shift, tau, max_requests, max_rows, max_sel,
                      vocab_base, vocab_total)
        w = _Weights(lm_head.data_ptr(), W1.data_ptr(), b1.data_ptr(), w2.data_ptr(), float(b2))
        h = C.c_void_p()
        with torch.cuda.device(self.device):
            _check(self.lib.wisv_create(C.byref(cfg), C.byref(w), C.byref(h)), "wisv_create")
        self._h = h

    def close(self):
        if getattr(self, "_h", None):
            self._torch.cuda.synchronize(self.device)
            self.lib.wisv_destroy(self._h)
            self._h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    # ------------------------------------------------------------------ helpers
    def _batch(self, *, B, K, k_off, T, target_hidden, draft_tokens, draft_hidden, csi, sel_off, sel_pos,
               draft_q, uniforms, tau):
        mode = (MODE_SH if sel_off is not None else MODE_FH) | \
               (ACCEPT_STOCHASTIC if draft_q is not None else ACCEPT_GREEDY)
        M_sel = int(sel_pos.shape[0]) if sel_pos is not None else 0
        return _Batch(B, 0 if k_off is not None else K, _ptr(k_off), T, _ptr(target_hidden), _ptr(draft_tokens),
                      _ptr(draft_hidden), _ptr(sel_off), _ptr(sel_pos), M_sel, _ptr(csi), _ptr(draft_q),
                      _ptr(uniforms), mode, float("nan") if tau is None else float(tau),
                      _hidden_dtype(target_hidden), _hidden_dtype(draft_hidden))

    def _outputs(self, B, R, T, P, device, extras: bool, pin: bool = False):
        torch = self._torch
        kw = dict(device=device)
        if pin:
            kw = dict(device="cpu", pin_memory=True)
        out = VerifyOutput(torch.empty(B, dtype=torch.int32, **kw), torch.empty(B, dtype=torch.int32, **kw))
        if extras:
            out.argmax = torch.empty(R, dtype=torch.int32, **kw)
            out.lse = torch.empty(R, dtype=torch.float32, **kw)
            out.p_draft = torch.empty(T, dtype=torch.float32, **kw)
            out.head_prob = torch.empty(P, dtype=torch.float32, **kw)
            out.mismatch_mask = torch.empty(B, dtype=torch.int64, **kw)
            out.n_mismatch = torch.empty(B, dtype=torch.int32, **kw)
            out.status = torch.empty(B, dtype=torch.int32, **kw)
        return out

    @staticmethod
    def _result(o: VerifyOutput) -> _Result:
        return _Result(_ptr(o.accept_len), _ptr(o.correction_token), _ptr(o.argmax), _ptr(o.lse), _ptr(o.p_draft),
                       _ptr(o.head_prob), _ptr(o.mismatch_mask), _ptr(o.n_mismatch), _ptr(o.status))

    # ------------------------------------------------------------------ calls
    def verify(self, target_hidden, draft_tokens, draft_hidden, csi, *, B: int, K: int = 0, k_off=None,
               T: Optional[int] = None, sel_off=None, sel_pos=None, draft_q=None, uniforms=None,
               tau: Optional[float] = None, extras: bool = True, out: Optional[VerifyOutput] = None,
               stream=None) -> VerifyOutput:
        """wisv_verify on device tensors; asynchronous on the current (or given) torch stream."""
        torch = self._torch
        if T is None:
            T = B * K if k_off is None else int(draft_tokens.shape[0])
        R = T + B
        P = int(sel_pos.shape[0]) if sel_pos is not None else T
        if out is None:
            out = self._outputs(B, R, T, P, self.device, extras)
        b = self._batch(B=B, K=K, k_off=k_off, T=T, target_hidden=target_hidden, draft_tokens=draft_tokens,
                        draft_hidden=draft_hidden, csi=csi, sel_off=sel_off, sel_pos=sel_pos, draft_q=draft_q,
                        uniforms=uniforms, tau=tau)
        r = self._result(out)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        _check(self.lib.wisv_verify(self._h, C.byref(b), C.byref(r), C.c_void_p(st.cuda_stream)), "wisv_verify")
        return out

    def localize(self, target_hidden, draft_tokens, *, B: int, K: int = 0, k_off=None, T: Optional[int] = None,
                 draft_q=None, uniforms=None, out: Optional[VerifyOutput] = None, stream=None) -> VerifyOutput:
        """wisv_localize: LM head, argmax / log-sum-exp and the candidate sets S (first phase of SH)."""
        torch = self._torch
        if T is None:
            T = B * K if k_off is None else int(draft_tokens.shape[0])
        if out is None:
            out = self._outputs(B, T + B, T, 0, self.device, True)
            out.head_prob = None
        b = self._batch(B=B, K=K, k_off=k_off, T=T, target_hidden=target_hidden, draft_tokens=draft_tokens,
                        draft_hidden=None, csi=None, sel_off=None, sel_pos=None, draft_q=draft_q,
                        uniforms=uniforms, tau=None)
        r = self._result(out)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        _check(self.lib.wisv_localize(self._h, C.byref(b), C.byref(r), C.c_void_p(st.cuda_stream)), "wisv_localize")
        return out

    def decide(self, target_hidden, draft_hidden, csi, *, B: int, K: int = 0, k_off=None, T: int,
               sel_off=None, sel_pos=None, tau: Optional[float] = None, out: Optional[VerifyOutput] = None,
               stream=None) -> VerifyOutput:
        """wisv_decide: decision head on the uploaded hidden states and the first-reject scan (second phase)."""
        torch = self._torch
        P = int(sel_pos.shape[0]) if sel_pos is not None else T
        if out is None:
            out = VerifyOutput(torch.empty(B, dtype=torch.int32, device=self.device),
                               torch.empty(B, dtype=torch.int32, device=self.device))
            out.head_prob = torch.empty(P, dtype=torch.float32, device=self.device)
            out.mismatch_mask = torch.empty(B, dtype=torch.int64, device=self.device)
            out.n_mismatch = torch.empty(B, dtype=torch.int32, device=self.device)
            out.status = torch.empty(B, dtype=torch.int32, device=self.device)
        b = self._batch(B=B, K=K, k_off=k_off, T=T, target_hidden=target_hidden, draft_tokens=None,
                        draft_hidden=draft_hidden, csi=csi, sel_off=sel_off, sel_pos=sel_pos, draft_q=None,
                        uniforms=None, tau=tau)
        r = self._result(out)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        _check(self.lib.wisv_decide(self._h, C.byref(b), C.byref(r), C.c_void_p(st.cuda_stream)), "wisv_decide")
        return out

    def shard_rows(self, target_hidden, draft_tokens, *, B: int, K: int = 0, k_off=None, T: Optional[int] = None,
                   out=None, stream=None):
        """wisv_shard_rows: this vocabulary shard's per-row partials, a float32 tensor [R, 4] (16 bytes per row)."""
        torch = self._torch
        if T is None:
            T = B * K if k_off is None else int(draft_tokens.shape[0])
        if out is None:
            out = torch.empty((T + B, 4), dtype=torch.float32, device=self.device)
        b = self._batch(B=B, K=K, k_off=k_off, T=T, target_hidden=target_hidden, draft_tokens=draft_tokens,
                        draft_hidden=None, csi=None, sel_off=None, sel_pos=None, draft_q=None, uniforms=None,
                        tau=None)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        _check(self.lib.wisv_shard_rows(self._h, C.byref(b), out.data_ptr(), C.c_void_p(st.cuda_stream)),
               "wisv_shard_rows")
        return out

    def verify_gathered(self, gathered, target_hidden, draft_tokens, draft_hidden, csi, *, B: int, K: int = 0,
                        k_off=None, T: Optional[int] = None, sel_off=None, sel_pos=None, draft_q=None,
                        uniforms=None, tau: Optional[float] = None, out: Optional[VerifyOutput] = None,
                        stream=None) -> VerifyOutput:
        """wisv_verify_gathered: gathered is float32 [G, R, 4], the partials of all G vocabulary shards."""
        torch = self._torch
        if T is None:
            T = B * K if k_off is None else int(draft_tokens.shape[0])
        R = T + B
        P = int(sel_pos.shape[0]) if sel_pos is not None else T
        G = int(gathered.shape[0])
        if out is None:
            out = self._outputs(B, R, T, P, self.device, True)
        b = self._batch(B=B, K=K, k_off=k_off, T=T, target_hidden=target_hidden, draft_tokens=draft_tokens,
                        draft_hidden=draft_hidden, csi=csi, sel_off=sel_off, sel_pos=sel_pos, draft_q=draft_q,
                        uniforms=uniforms, tau=tau)
        r = self._result(out)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        _check(self.lib.wisv_verify_gathered(self._h, C.byref(b), gathered.data_ptr(), G, C.byref(r),
                                             C.c_void_p(st.cuda_stream)), "wisv_verify_gathered")
        return out

    def verify_host(self, target_hidden, draft_tokens, draft_hidden, csi, *, B: int, K: int = 0, k_off=None,
                    T: Optional[int] = None, sel_off=None, sel_pos=None, draft_q=None, uniforms=None,
                    tau: Optional[float] = None, extras: bool = False, out: Optional[VerifyOutput] = None,
                    stream=None) -> VerifyOutput:
        """wisv_verify_host on CPU tensors (pinned for asynchronous copies); returns after completion."""
        torch = self._torch
        if T is None:
            T = B * K if k_off is None else int(draft_tokens.shape[0])
        R = T + B
        P = int(sel_pos.shape[0]) if sel_pos is not None else T
        if out is None:
            out = self._outputs(B, R, T, P, "cpu", extras, pin=True)
        b = self._batch(B=B, K=K, k_off=k_off, T=T, target_hidden=target_hidden, draft_tokens=draft_tokens,
                        draft_hidden=draft_hidden, csi=csi, sel_off=sel_off, sel_pos=sel_pos, draft_q=draft_q,
                        uniforms=uniforms, tau=tau)
        r = self._result(out)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        with torch.cuda.device(self.device):
            _check(self.lib.wisv_verify_host(self._h, C.byref(b), C.byref(r), C.c_void_p(st.cuda_stream)),
                   "wisv_verify_host")
        return out

    def bind_host(self, target_hidden, draft_tokens, draft_hidden, csi, *, B: int, K: int = 0, k_off=None,
                  T: Optional[int] = None, sel_off=None, sel_pos=None, draft_q=None, uniforms=None,
                  tau: Optional[float] = None, extras: bool = False, out: Optional[VerifyOutput] = None,
                  stream=None) -> "BoundHostCall":
        """wisv_verify_host with the argument blocks built once, for a loop that reuses the same host buffers
        (a server refills its pinned input buffers in place and calls again): each call of the returned object
        is one wisv_verify_host on the buffers as they are then, and returns the same VerifyOutput."""
        torch = self._torch
        if T is None:
            T = B * K if k_off is None else int(draft_tokens.shape[0])
        R = T + B
        P = int(sel_pos.shape[0]) if sel_pos is not None else T
        if out is None:
            out = self._outputs(B, R, T, P, "cpu", extras, pin=True)
        b = self._batch(B=B, K=K, k_off=k_off, T=T, target_hidden=target_hidden, draft_tokens=draft_tokens,
                        draft_hidden=draft_hidden, csi=csi, sel_off=sel_off, sel_pos=sel_pos, draft_q=draft_q,
                        uniforms=uniforms, tau=tau)
        st = stream if stream is not None else torch.cuda.current_stream(self.device)
        keep = (target_hidden, draft_tokens, draft_hidden, csi, k_off, sel_off, sel_pos, draft_q, uniforms, st)
        return BoundHostCall(self, b, self._result(out), out, st, keep)

    def debug_logits(self, target_hidden):
        torch = self._torch
        R = target_hidden.shape[0]
        out = torch.empty((R, self.V), dtype=torch.float32, device=target_hidden.device)
        st = torch.cuda.current_stream(self.device)
        _check(self.lib.wisv_debug_logits(self._h, target_hidden.data_ptr(), R, out.data_ptr(),
                                          C.c_void_p(st.cuda_stream)), "wisv_debug_logits")
        return out

    def wait_probe(self, limit_cycles: int):
        st = self._torch.cuda.current_stream(self.device)
        _check(self.lib.wisv_debug_wait_probe(self._h, limit_cycles, C.c_void_p(st.cuda_stream)),
               "wisv_debug_wait_probe")

    def poison(self):
        st = self._torch.cuda.current_stream(self.device)
        _check(self.lib.wisv_debug_poison(self._h, C.c_void_p(st.cuda_stream)), "wisv_debug_poison")

    def device_error(self) -> int:
        st = self._torch.cuda.current_stream(self.device)
        v = C.c_int32(0)
        _check(self.lib.wisv_device_error(self._h, C.c_void_p(st.cuda_stream), C.byref(v)), "wisv_device_error")
        return v.value

    def plan(self, R: int, P: int):
        v = [C.c_int32(0) for _ in range(6)]
        _check(self.lib.wisv_plan(self._h, R, P, *[C.byref(x) for x in v]), "wisv_plan")
        keys = ("lm_tile_n", "lm_tiles", "lm_ctas", "head_tile_n", "head_tiles", "head_ctas")
        return dict(zip(keys, (x.value for x in v)))

    def plan_kernels(self, R: int, P: int) -> int:
        n = self.lib.wisv_plan_kernels(self._h, R, P)
        _check(min(n, 0), "wisv_plan_kernels")
        return n

    def set_tuning(self, lm_tile_n: int = 0, lm_stages: int = 0, head_tile_n: int = 0, head_stages: int = 0,
                   lm_single_cta: int = 0, head_ctas: int = 0, lm_mma_m: int = 0, lm_kb_per_stage: int = 0, lm_teams: int = 0):
        t = _Tuning(lm_tile_n, lm_stages, head_tile_n, head_stages, lm_single_cta, head_ctas, lm_mma_m, lm_kb_per_stage,
                    lm_teams)
        _check(self.lib.wisv_set_tuning(self._h, C.byref(t)), "wisv_set_tuning")

    def launch_count(self) -> int:
        return int(self.lib.wisv_launch_count(self._h))

    def profile_enable(self, n_calls: int):
        _check(self.lib.wisv_profile_enable(self._h, n_calls), "wisv_profile_enable")

    def profile_read(self, stage: int, cap: int = 4096):
        buf = (C.c_float * cap)()
        n = C.c_int32(0)
        _check(self.lib.wisv_profile_read(self._h, stage, buf, cap, C.byref(n)), "wisv_profile_read")
        return [buf[i] for i in range(n.value)]


def lm_head_reduce_static(lm_head, target_hidden, argmax, lse, stream=None):
    """wisv_lm_head_reduce_static on torch CUDA tensors the caller has already allocated.

    For callers that may not allocate device memory: nothing is allocated here
    either - inputs and outputs are the caller's, the scratch lives in the library
    image.  lm_head: bf16 [V, H]; target_hidden: fp32 [R, H]; argmax: int32 [R];
    lse: fp32 [R].  Asynchronous on the current (or given) torch stream.
    """
    import torch
    lib = load_library()
    V, H = lm_head.shape
    R = target_hidden.shape[0]
    st = stream if stream is not None else torch.cuda.current_stream(lm_head.device)
    with torch.cuda.device(lm_head.device):
        _check(lib.wisv_lm_head_reduce_static(lm_head.data_ptr(), V, H, target_hidden.data_ptr(), R,
                                              argmax.data_ptr(), lse.data_ptr(), C.c_void_p(st.cuda_stream)),
               "wisv_lm_head_reduce_static")
