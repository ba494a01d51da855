"""The selective-hidden protocol in two calls (localize, then decide) against the one-call round and the oracle."""
import numpy as np
import pytest
import torch

import gen
from paper_2604_17701_b200 import WisvError
from gen import cases
from parity import compare, oracle_ref_argmax, run_oracle

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _cfg(**kw):
    base = dict(B=12, K=6, H=256, H_d=128, d_c=2, d_J=128, V=4096, match_rate=0.5, seed=31)
    base.update(kw)
    return gen.VerifyConfig("tp", **base)


@pytest.mark.parametrize("kw", [dict(), dict(K=0, K_lo=1, K_hi=10, B=40), dict(match_rate=1.0), dict(match_rate=0.0),
                                dict(B=1, K=8), dict(stochastic=True)],
                         ids=["uniform", "ragged", "emptyS", "fullS", "single", "stochastic"])
def test_localize_then_decide_equals_one_call(kw):
    cfg = _cfg(**kw)
    case = cases.make_case(cfg, oracle_ref_argmax)          # full-hidden traffic: dense draft hidden states
    if cfg.stochastic:
        base = run_oracle(case)
        case["draft_q"] = (base["p_draft"] * np.random.default_rng(2).uniform(0.5, 4.0, size=case["T"])).astype(np.float32)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    one = cases.run(v, d)
    torch.cuda.synchronize()

    kw_geo = dict(B=cfg.B, K=cfg.K if cfg.K_hi == 0 else 0, k_off=d["k_off_dev"], T=case["T"])
    loc = v.localize(d["target_hidden"], d["draft_tokens"], draft_q=d["draft_q"], uniforms=d["uniforms"], **kw_geo)
    torch.cuda.synchronize()
    assert torch.equal(loc.mismatch_mask, one.mismatch_mask) and torch.equal(loc.n_mismatch, one.n_mismatch)
    # the one-call round of a small batch divides the vocabulary over fewer CTAs (some evaluate the decision head in
    # the same launch): same logits, another fp32 summation order in the log-sum-exp
    assert torch.equal(loc.argmax, one.argmax)
    assert float((loc.lse - one.lse).abs().max()) < 1e-5
    assert torch.allclose(loc.p_draft, one.p_draft, rtol=1e-4, atol=0)
    # greedy result while no hidden state has arrived: first candidate position
    mask = loc.mismatch_mask.cpu().numpy().astype(np.uint64)
    first = np.array([next((i for i in range(case["k_len"][b]) if (int(mask[b]) >> i) & 1), case["k_len"][b])
                      for b in range(cfg.B)])
    assert np.array_equal(loc.accept_len.cpu().numpy(), first)

    # the device uploads exactly the hidden states the edge asked for (Algorithm 1: RequestHidden(S))
    sel = np.zeros(case["T"], bool)
    for b in range(cfg.B):
        for i in range(case["k_len"][b]):
            sel[case["k_off"][b] + i] = (int(mask[b]) >> i) & 1
    packed, sel_off, sel_pos = gen.pack_selective(case["draft_hidden"], case["k_len"], sel)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    dec = v.decide(d["target_hidden"], dev(packed), d["csi"], sel_off=dev(sel_off), sel_pos=dev(sel_pos), **kw_geo)
    torch.cuda.synchronize()
    assert v.device_error() == 0
    assert torch.equal(dec.accept_len, one.accept_len) and torch.equal(dec.correction_token, one.correction_token)
    assert torch.equal(dec.n_mismatch, one.n_mismatch)
    hp_one = one.head_prob.cpu().numpy()[sel]
    assert np.allclose(dec.head_prob.cpu().numpy(), hp_one, atol=1e-5)      # up to the fp32 summation order

    # and against the oracle on the selective-hidden traffic
    sh_case = dict(case, draft_hidden=packed, sel_off=sel_off, sel_pos=sel_pos)
    ref = run_oracle(sh_case)
    full = type("O", (), {})()
    for k in ("argmax", "lse", "p_draft"):
        setattr(full, k, getattr(loc, k))
    for k in ("accept_len", "correction_token", "head_prob", "n_mismatch", "mismatch_mask", "status"):
        setattr(full, k, getattr(dec, k))
    compare(sh_case, ref, full, cfg.tau)
    v.close()


def test_decide_needs_a_matching_localize():
    cfg = _cfg(B=4, K=4)
    case = cases.make_case(cfg, oracle_ref_argmax)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    with pytest.raises(WisvError) as e:                     # nothing pending
        v.decide(d["target_hidden"], d["draft_hidden"], d["csi"], B=4, K=4, T=16)
    assert e.value.code == -1
    v.localize(d["target_hidden"], d["draft_tokens"], B=4, K=4)
    with pytest.raises(WisvError) as e:                     # different geometry
        v.decide(d["target_hidden"], d["draft_hidden"], d["csi"], B=2, K=4, T=8)
    assert e.value.code == -2
    out = v.decide(d["target_hidden"], d["draft_hidden"], d["csi"], B=4, K=4, T=16)     # dense upload also works
    ref = cases.run(v, d)
    assert torch.equal(out.accept_len, ref.accept_len)
    with pytest.raises(WisvError):                          # consumed by the verify above
        v.decide(d["target_hidden"], d["draft_hidden"], d["csi"], B=4, K=4, T=16)
    v.close()


def test_decide_enqueued_right_behind_other_rounds_reads_its_own_inputs():
    """The decision-head launch of wisv_decide follows the pack kernel directly (no LM-head launch in between), so it
    must wait for the pack kernel before its first read.  A full-hidden round on other hidden states, then localize and
    decide with several hundred selected positions, all enqueued back to back with no host synchronisation: the
    result must equal one wisv_verify on the second batch."""
    cfg_a = _cfg(B=60, K=8, seed=91, match_rate=0.2, weight_seed=90)
    cfg_b = _cfg(B=60, K=8, seed=92, match_rate=0.2, weight_seed=90)
    w = gen.make_weights(cfg_a)
    case_a = cases.make_case(cfg_a, oracle_ref_argmax, weights=w)
    case_b = cases.make_case(cfg_b, oracle_ref_argmax, weights=w)
    da, db = cases.to_device(case_a, DEV), cases.to_device(case_b, DEV)
    v = cases.make_verifier(db, max_sel=case_b["T"])
    one = cases.run(v, db)
    torch.cuda.synchronize()
    mask = one.mismatch_mask.cpu().numpy().astype(np.uint64)
    sel = np.zeros(case_b["T"], bool)
    for b in range(cfg_b.B):
        for i in range(cfg_b.K):
            sel[b * cfg_b.K + i] = (int(mask[b]) >> i) & 1
    assert sel.sum() >= 300
    packed, sel_off, sel_pos = gen.pack_selective(case_b["draft_hidden"], case_b["k_len"], sel)
    dev = lambda a: torch.from_numpy(np.ascontiguousarray(a)).to(DEV)
    packed_d, sel_off_d, sel_pos_d = dev(packed), dev(sel_off), dev(sel_pos)
    geo = dict(B=cfg_b.B, K=cfg_b.K, T=case_b["T"])
    torch.cuda.synchronize()
    for _ in range(20):
        cases.run(v, da)                                    # leaves batch A's head inputs in the workspace
        v.localize(db["target_hidden"], db["draft_tokens"], **geo)
        dec = v.decide(db["target_hidden"], packed_d, db["csi"], sel_off=sel_off_d, sel_pos=sel_pos_d, **geo)
    torch.cuda.synchronize()
    assert v.device_error() == 0
    assert torch.equal(dec.accept_len, one.accept_len) and torch.equal(dec.correction_token, one.correction_token)
    assert np.allclose(dec.head_prob.cpu().numpy(), one.head_prob.cpu().numpy()[sel], atol=1e-5)
    v.close()
