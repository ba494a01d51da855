"""Workload assembly shared by the tests, the smoke check and the benchmark (harness, not product).

Builds one verification batch from the seeded generators, moves it to the device
and runs it through the binding of the CUDA library.  Nothing here is part of the
verification round: the reference argmax that the input recipe needs (draft
tokens are forced to match the target's prediction with a given probability) is
passed in by the caller.  ``gen/__init__`` does not import this module, so the
generators stay free of the CUDA package.
"""
from __future__ import annotations

from typing import Callable, Dict, Optional

import numpy as np

from . import synth as gen


def make_case(cfg: "gen.VerifyConfig", ref_argmax_fn: Callable[[np.ndarray, np.ndarray], np.ndarray],
              weights: Optional[Dict[str, np.ndarray]] = None) -> Dict[str, object]:
    """All inputs of one batch as numpy arrays.

    ref_argmax_fn(lm_head_bits [V,H], target_hidden [R,H]) -> int32 [R] supplies the
    target's greedy prediction per window row (an oracle or a library routine).
    """
    k_len = gen.window_lengths(cfg)
    k_off, row_off = gen.row_offsets(k_len)
    w = weights if weights is not None else gen.make_weights(cfg)
    h = gen.make_hidden(cfg, k_len)
    ref = np.asarray(ref_argmax_fn(w["lm_head"], h["target_hidden"]), np.int32)
    toks = gen.make_draft_tokens(cfg, k_len, ref)
    T = int(k_off[-1])
    case = dict(cfg=cfg, k_len=k_len, k_off=k_off, row_off=row_off, T=T, R=T + cfg.B, ref_argmax=ref,
                draft_tokens=toks, target_hidden=h["target_hidden"], csi=h["csi"],
                draft_hidden=h["draft_hidden"], sel_off=None, sel_pos=None, draft_q=None, uniforms=None, **w)
    if cfg.mode == "SH":
        rows = np.repeat(row_off[:-1], k_len) + (np.arange(T) - np.repeat(k_off[:-1], k_len))
        mismatch = toks != ref[rows]
        packed, sel_off, sel_pos = gen.pack_selective(h["draft_hidden"], k_len, mismatch)
        case.update(draft_hidden=packed, sel_off=sel_off, sel_pos=sel_pos)
    if cfg.stochastic:
        q, u = gen.make_stochastic_inputs(cfg, T)
        case.update(draft_q=q, uniforms=u)
    return case


def library_ref_argmax(lm_head_bits: np.ndarray, target_hidden: np.ndarray, device: str = "cpu",
                       chunk: int = 1024) -> np.ndarray:
    """Reference argmax for the input recipe at sizes a scalar oracle cannot reach.

    A plain torch library matmul (fp32, TF32 off) over bf16-rounded hidden states;
    used only to decide which draft tokens are forced to match.  It is input
    preparation: neither the verifier nor the oracle depends on it.
    """
    import torch
    prev = torch.backends.cuda.matmul.allow_tf32
    torch.backends.cuda.matmul.allow_tf32 = False
    try:
        W = torch.from_numpy(lm_head_bits.view(np.int16)).view(torch.bfloat16).to(device).float()
        out = np.empty(target_hidden.shape[0], np.int32)
        for lo in range(0, target_hidden.shape[0], chunk):
            x = torch.from_numpy(target_hidden[lo:lo + chunk]).to(device).to(torch.bfloat16).float()
            out[lo:lo + chunk] = torch.argmax(x @ W.T, dim=1).to(torch.int32).cpu().numpy()
        return out
    finally:
        torch.backends.cuda.matmul.allow_tf32 = prev


ACT = {"relu": 0, "gelu": 1}      # WISV_ACT_RELU, WISV_ACT_GELU


def to_device(case: Dict[str, object], device="cuda:0", weights_dev=None) -> Dict[str, object]:
    """The case with every array as a device tensor (weights_dev: model tensors already on the device, reused)."""
    import torch

    def dev(a, dtype=None):
        if a is None:
            return None
        t = torch.from_numpy(np.ascontiguousarray(a))
        return t.to(device)

    d = dict(case)
    if weights_dev is not None:
        d.update({k: weights_dev[k] for k in ("lm_head", "W1", "b1", "w2")})
    else:
        d["lm_head"] = torch.from_numpy(case["lm_head"].view(np.int16)).view(torch.bfloat16).to(device)
        d["W1"] = torch.from_numpy(case["W1"].view(np.int16)).view(torch.bfloat16).to(device)
    for k in (("b1", "w2") if weights_dev is None else ()) + ("target_hidden", "draft_tokens", "draft_hidden", "csi", "sel_off", "sel_pos",
              "draft_q", "uniforms"):
        d[k] = dev(case[k])
    cfg = case["cfg"]
    d["k_off_dev"] = dev(case["k_off"]) if cfg.K_hi > 0 else None
    return d


def make_verifier(dcase: Dict[str, object], *, act: Optional[str] = None, tau: Optional[float] = None,
                  head_row_shift: int = 0, max_requests: Optional[int] = None, max_rows: Optional[int] = None,
                  max_sel: int = 0, vocab_slice=None):
    from paper_2604_17701_b200 import binding
    cfg = dcase["cfg"]
    if vocab_slice is not None:
        # a context on rows [lo, hi) of the LM head (one vocabulary shard)
        lo, hi = vocab_slice
        return binding.Verifier(dcase["lm_head"][lo:hi], dcase["W1"], dcase["b1"], dcase["w2"], float(dcase["b2"]),
                                H_d=cfg.H_d, d_c=cfg.d_c, act=ACT[act or cfg.act],
                                tau=cfg.tau if tau is None else tau, head_row_shift=head_row_shift,
                                max_requests=max_requests or cfg.B, max_rows=max_rows or dcase["R"],
                                max_sel=max_sel, vocab_base=lo, vocab_total=cfg.V)
    return binding.Verifier(dcase["lm_head"], dcase["W1"], dcase["b1"], dcase["w2"], float(dcase["b2"]),
                            H_d=cfg.H_d, d_c=cfg.d_c, act=ACT[act or cfg.act],
                            tau=cfg.tau if tau is None else tau, head_row_shift=head_row_shift,
                            max_requests=max_requests or cfg.B, max_rows=max_rows or dcase["R"], max_sel=max_sel)


def run(verifier, dcase: Dict[str, object], *, tau: Optional[float] = None, extras: bool = True,
        out=None):
    """One wisv_verify call on a device-resident case."""
    cfg = dcase["cfg"]
    return verifier.verify(dcase["target_hidden"], dcase["draft_tokens"], dcase["draft_hidden"], dcase["csi"],
                           B=cfg.B, K=cfg.K if cfg.K_hi == 0 else 0, k_off=dcase["k_off_dev"], T=dcase["T"],
                           sel_off=dcase["sel_off"], sel_pos=dcase["sel_pos"], draft_q=dcase["draft_q"],
                           uniforms=dcase["uniforms"], tau=tau, extras=extras, out=out)
