"""The parity harness itself, on the CPU: what it must accept and what it must refuse on near-tie rows.

The "CUDA result" here is the oracle's own output with a mistake planted in it, so the checks of
tests/parity.py are shown to bite without a GPU.
"""
import numpy as np
import pytest
import torch

import gen
from gen import cases
from parity import compare, oracle_ref_argmax, run_oracle


class _Out:
    pass


def _as_output(ref):
    o = _Out()
    o.accept_len = torch.from_numpy(ref["accept_len"].astype(np.int32))
    o.correction_token = torch.from_numpy(ref["correction_token"].astype(np.int32))
    o.argmax = torch.from_numpy(ref["argmax"].astype(np.int32))
    o.lse = torch.from_numpy(ref["lse"].astype(np.float32))
    o.p_draft = torch.from_numpy(ref["p_draft"].astype(np.float32))
    o.head_prob = torch.from_numpy(ref["head_prob"].astype(np.float32))
    o.n_mismatch = torch.from_numpy(ref["n_mismatch"].astype(np.int32))
    mask = np.zeros(ref["accept_len"].shape[0], np.int64)
    for b in range(mask.shape[0]):
        for i in range(ref["k_off"][b + 1] - ref["k_off"][b]):
            if ref["cand"][ref["k_off"][b] + i]:
                mask[b] |= 1 << i
    o.mismatch_mask = torch.from_numpy(mask)
    o.status = torch.zeros(mask.shape[0], dtype=torch.int32)
    return o


def _case_with_near_and_exact_ties():
    cfg = gen.VerifyConfig("h", B=4, K=3, H=64, H_d=32, d_c=2, d_J=32, V=512, match_rate=0.5, seed=5)
    w = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in gen.make_weights(cfg).items()}
    base = cases.make_case(cfg, oracle_ref_argmax, weights=w)
    ref0 = run_oracle(base)
    r_near, r_exact = 1, 6
    a_near, a_exact = int(ref0["argmax"][r_near]), int(ref0["argmax"][r_exact])
    # twice the winning row (exact in bf16), so the planted maxima are far above the rest of their rows
    dbl = lambda row: np.where((row & 0x7F80) != 0, row + np.uint16(0x0080), row).astype(np.uint16)
    near_lo, near_hi, ex_lo, ex_hi = 100, 300, 40, 450
    W = w["lm_head"]
    W[near_lo] = dbl(W[a_near])
    W[near_hi] = W[near_lo]
    W[near_hi, 0] ^= 1                                  # one bf16 ulp in one weight: a near-tie, not a tie
    W[ex_lo] = dbl(W[a_exact])
    W[ex_hi] = W[ex_lo]
    case = cases.make_case(cfg, oracle_ref_argmax, weights=w)
    ref = run_oracle(case)
    assert 0.0 < ref["top2_gap"][r_near] < 1e-2 and ref["argmax"][r_near] in (near_lo, near_hi)
    assert ref["top2_gap"][r_exact] == 0.0 and ref["argmax"][r_exact] == ex_lo
    return cfg, case, ref, (r_near, near_lo, near_hi), (r_exact, ex_lo, ex_hi)


def test_harness_accepts_the_runner_up_of_a_near_tie_only():
    cfg, case, ref, (r_near, lo, hi), _ = _case_with_near_and_exact_ties()
    stats = compare(case, ref, _as_output(ref), cfg.tau)
    assert stats["row_ties"] >= 1 and stats["near_tie_rows_checked"] == 0
    other = hi if ref["argmax"][r_near] == lo else lo
    o = _as_output(ref)
    o.argmax[r_near] = other                            # the other leading index: valid
    assert compare(case, ref, o, cfg.tau)["near_tie_rows_checked"] == 1
    o.argmax[r_near] = (other + 1) % cfg.V              # any other index: must be refused
    with pytest.raises(AssertionError, match="near-tie"):
        compare(case, ref, o, cfg.tau)
    o.argmax[r_near] = cfg.V + 3
    with pytest.raises(AssertionError, match="out of range"):
        compare(case, ref, o, cfg.tau)


def test_harness_refuses_the_higher_index_of_an_exact_tie():
    cfg, case, ref, _, (r_exact, lo, hi) = _case_with_near_and_exact_ties()
    o = _as_output(ref)
    o.argmax[r_exact] = hi
    with pytest.raises(AssertionError, match="argmax differs"):
        compare(case, ref, o, cfg.tau)
