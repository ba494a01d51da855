"""Parity harness: run the oracle on a case and compare a CUDA result with it.

Bars: argmax / accept_len / correction_token bit-exact outside near-ties (top-2
logit gap < 1e-2, |head prob - tau| < 2e-3, and for the stochastic test
|u - alpha| < 1e-2), which are excluded from the exact comparison and counted;
on a near-tie row several indices are correct, so the CUDA argmax is still
checked for validity: the oracle's logit at that index must lie within 1e-2 of
the oracle's maximum, and where the oracle's gap is exactly zero (duplicate
vocabulary rows) the lowest index is required bit-exactly.  Log-sum-exp within
1e-2 absolute; decision-head probabilities within 2e-3 absolute; the draft-token
probability within 2 % relative (it inherits the log-sum-exp tolerance).
"""
import numpy as np

import oracle

GAP_TIE = 1e-2
PROB_TIE = 2e-3
ALPHA_TIE = 1e-2
LSE_TOL = 1e-2
PROB_TOL = 2e-3

ACT = {"relu": oracle.ACT_RELU, "gelu": oracle.ACT_GELU}


def oracle_ref_argmax(lm_head_bits, target_hidden):
    return oracle.lm_head(lm_head_bits, target_hidden)["argmax"]


def run_oracle(case, *, act=None, tau=None, head_row_shift=0):
    cfg = case["cfg"]
    return oracle.verify(lm_head_bits=case["lm_head"], W1_bits=case["W1"], b1=case["b1"], w2=case["w2"],
                         b2=float(case["b2"]), act=ACT[act or cfg.act], tau=cfg.tau if tau is None else tau,
                         k_len=case["k_len"], target_hidden=case["target_hidden"],
                         draft_tokens=case["draft_tokens"], draft_hidden=case["draft_hidden"], csi=case["csi"],
                         sel_off=case["sel_off"], sel_pos=case["sel_pos"], draft_q=case["draft_q"],
                         uniforms=case["uniforms"], head_row_shift=head_row_shift)


def compare(case, ref, out, tau, requests=None):
    """Assert parity; returns counts of excluded near-ties.

    requests: optional subset of request indices the oracle was run on (ref is
    then indexed by the subset's own rows); None = whole batch.
    """
    g = {k: (getattr(out, k).cpu().numpy() if getattr(out, k) is not None else None)
         for k in ("accept_len", "correction_token", "argmax", "lse", "p_draft", "head_prob", "n_mismatch",
                   "mismatch_mask", "status")}
    k_len = np.asarray(case["k_len"])
    B = k_len.shape[0]
    k_off, row_off = ref["k_off"], ref["row_off"]
    gap = ref["top2_gap"]
    # a gap of exactly zero means bit-identical weight rows: both sides see equal logits and the lowest index is
    # the one correct answer, so such rows are compared exactly like any other
    row_tie = (gap < GAP_TIE) & (gap > 0.0)

    # per-row quantities
    assert np.max(np.abs(g["lse"] - ref["lse"])) <= LSE_TOL, "log-sum-exp outside tolerance"
    differs = g["argmax"] != ref["argmax"]
    bad = differs & ~row_tie
    assert not bad.any(), "argmax differs on rows %s (gaps %s)" % (np.nonzero(bad)[0][:8], gap[bad][:8])
    # near-tie rows: any index whose oracle logit is within the band of the oracle maximum is valid
    near = np.nonzero(differs & row_tie)[0]
    if near.size:
        V = np.asarray(case["lm_head"]).shape[0]
        assert np.all((g["argmax"][near] >= 0) & (g["argmax"][near] < V)), "argmax out of range on a near-tie row"
        rows2 = np.concatenate([near, near])
        toks2 = np.concatenate([g["argmax"][near], ref["argmax"][near]]).astype(np.int32)
        at = oracle.lm_head(case["lm_head"], np.asarray(case["target_hidden"])[rows2], row_token=toks2)["tok_logit"]
        short = at[near.size:] - at[:near.size]            # oracle maximum minus oracle logit at the GPU's index
        assert np.all(short >= 0.0) and np.all(short < GAP_TIE), \
            "near-tie rows %s: GPU argmax is not among the leading logits (short by %s)" % (near[:8], short[:8])
    rel = np.abs(g["p_draft"] - ref["p_draft"]) / np.maximum(ref["p_draft"], 1e-30)
    assert np.all(rel <= 2e-2), "draft-token probability outside tolerance"
    assert np.max(np.abs(g["head_prob"] - ref["head_prob"]), initial=0.0) <= PROB_TOL, "head probability outside tolerance"

    # per-request decisions
    prob_tie_t = np.zeros(ref["prob_t"].shape[0], bool)
    prob_tie_t[ref["eval_t"]] = np.abs(ref["head_prob"] - tau) < PROB_TIE
    if ref["alpha"] is not None:
        alpha_tie_t = np.abs(np.asarray(case["uniforms"], np.float64) - ref["alpha"]) < ALPHA_TIE
    else:
        alpha_tie_t = np.zeros_like(prob_tie_t)
    tainted = 0
    for b in range(B):
        Ao, Ag = int(ref["accept_len"][b]), int(g["accept_len"][b])
        hi = min(max(Ao, Ag), k_len[b])
        rows = slice(row_off[b], row_off[b] + hi + 1)
        toks = slice(k_off[b], k_off[b] + min(hi + 1, k_len[b]))
        if row_tie[rows].any() or prob_tie_t[toks].any() or alpha_tie_t[toks].any():
            tainted += 1
            continue
        assert Ag == Ao, "accept_len differs for request %d: gpu %d oracle %d" % (b, Ag, Ao)
        assert g["correction_token"][b] == ref["correction_token"][b], "correction token differs for request %d" % b
        assert 0 <= Ag <= k_len[b]
    # the candidate count agrees wherever no row of the window is a near-tie
    for b in range(B):
        rows = slice(row_off[b], row_off[b] + k_len[b] + 1)
        toks = slice(k_off[b], k_off[b] + k_len[b])
        if not row_tie[rows].any() and not alpha_tie_t[toks].any():
            assert g["n_mismatch"][b] == ref["n_mismatch"][b]
            mask = sum(1 << i for i in range(k_len[b]) if ref["cand"][k_off[b] + i])
            assert int(g["mismatch_mask"][b]) & ((1 << 64) - 1) == mask or int(g["mismatch_mask"][b]) == mask - (1 << 64)
    return dict(row_ties=int(row_tie.sum()), near_tie_rows_checked=int(near.size), rows=int(row_tie.shape[0]), tainted_requests=tainted, requests=B,
                prob_ties=int(prob_tie_t.sum()), alpha_ties=int(alpha_tie_t.sum()))
