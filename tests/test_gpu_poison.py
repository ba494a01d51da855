"""Stale or uninitialised scratch must never reach an output (the stand-in for a memory checker).

The kernels lean on "rows that are never read": MMA operands that run past the loaded activation rows, workspace
rows beyond the current batch, split-K scratch, partial buffers sized for the worst plan.  wisv_debug_poison fills
every scratch buffer the context owns with NaN / out-of-range patterns; a round that follows must give bit-identical
results to the same round on a clean workspace, equal the oracle, and leave the device error word at zero.
"""
import numpy as np
import pytest
import torch

import gen
from gen import cases
from parity import compare, oracle_ref_argmax, run_oracle

pytestmark = pytest.mark.gpu
DEV = "cuda:0"
FIELDS = ("accept_len", "correction_token", "argmax", "lse", "p_draft", "head_prob", "n_mismatch", "mismatch_mask",
          "status")


def _cfg(**kw):
    base = dict(B=8, K=4, H=256, H_d=128, d_c=2, d_J=128, V=4096, match_rate=0.5, seed=0, weight_seed=500)
    base.update(kw)
    return gen.VerifyConfig("poison", **base)


def _same(a, b, what):
    for k in FIELDS:
        assert torch.equal(getattr(a, k), getattr(b, k)), (what, k)


def test_large_batch_then_poison_then_small_batch():
    big_cfg, small_cfg = _cfg(B=100, K=4, seed=1), _cfg(B=2, K=3, seed=2)
    w = gen.make_weights(big_cfg)
    big = cases.make_case(big_cfg, oracle_ref_argmax, weights=w)
    small = cases.make_case(small_cfg, oracle_ref_argmax, weights=w)
    db, ds = cases.to_device(big, DEV), cases.to_device(small, DEV)
    v = cases.make_verifier(db)
    clean_small = cases.run(v, ds)
    clean_big = cases.run(v, db)
    torch.cuda.synchronize()
    v.poison()
    o_big = cases.run(v, db)                     # every workspace row of the batch is rewritten
    v.poison()
    o_small = cases.run(v, ds)                   # 8 live rows, 492 poisoned ones behind them
    o_small2 = cases.run(v, ds)                  # and once more on what the round itself left
    torch.cuda.synchronize()
    assert v.device_error() == 0
    _same(o_big, clean_big, "big")
    _same(o_small, clean_small, "small")
    _same(o_small2, clean_small, "small again")
    compare(big, run_oracle(big), o_big, big_cfg.tau)
    compare(small, run_oracle(small), o_small, small_cfg.tau)
    v.close()


def test_every_launch_plan_on_a_poisoned_workspace():
    """Seeded sweep over row counts around the plan boundaries, both upload modes, both acceptance rules and the
    launch plans the tuning switches select: poison, run, compare with the clean run and the oracle."""
    rng = np.random.default_rng(777)
    for it in range(24):
        K = int(rng.integers(1, 10))
        target_rows = int(rng.choice([5, 17, 63, 64, 65, 127, 128, 129, 200, 256, 257, 300, 384, 385, 520]))
        kw = dict(B=max(1, target_rows // (K + 1)), K=K, H=int(rng.choice([64, 72, 256])),
                  H_d=int(rng.choice([8, 40, 128])), d_c=int(rng.choice([0, 2, 3])),
                  d_J=int(rng.choice([16, 50, 128, 272])), V=int(rng.choice([17, 100, 1000, 4096, 5000, 40000])),
                  match_rate=float(rng.choice([0.0, 0.5, 1.0])), seed=5000 + it, weight_seed=-1,
                  mode=str(rng.choice(["FH", "SH"])), act=str(rng.choice(["gelu", "relu"])),
                  stochastic=bool(rng.random() < 0.25))
        cfg = _cfg(**kw)
        case = cases.make_case(cfg, oracle_ref_argmax)
        if cfg.stochastic:
            base = run_oracle(case)
            case["draft_q"] = (base["p_draft"] * rng.uniform(0.5, 4.0, size=case["T"])).astype(np.float32)
        ref = run_oracle(case)
        d = cases.to_device(case, DEV)
        # capacity far above the batch: most of the workspace is never written by these rounds
        v = cases.make_verifier(d, max_requests=cfg.B + 40, max_rows=case["R"] + 700, max_sel=case["T"] + 300)
        for tune in (dict(), dict(head_ctas=-1), dict(lm_single_cta=1), dict(head_ctas=3), dict(lm_mma_m=128), dict(lm_kb_per_stage=1)):
            v.set_tuning(**tune)
            clean = cases.run(v, d)
            torch.cuda.synchronize()
            v.poison()
            out = cases.run(v, d)
            torch.cuda.synchronize()
            assert v.device_error() == 0, (kw, tune)
            _same(out, clean, (kw, tune))
            compare(case, ref, out, cfg.tau)
        v.close()


def test_two_phase_and_sharded_flows_on_a_poisoned_workspace():
    cfg = _cfg(B=30, K=6, seed=9, match_rate=0.4)
    case = cases.make_case(cfg, oracle_ref_argmax)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d, max_requests=64, max_rows=700)
    geo = dict(B=cfg.B, K=cfg.K, T=case["T"])
    one = cases.run(v, d)
    torch.cuda.synchronize()
    v.poison()
    loc = v.localize(d["target_hidden"], d["draft_tokens"], **geo)
    dec = v.decide(d["target_hidden"], d["draft_hidden"], d["csi"], **geo)
    torch.cuda.synchronize()
    assert torch.equal(loc.argmax, one.argmax) and torch.equal(dec.accept_len, one.accept_len)
    assert torch.equal(dec.correction_token, one.correction_token)
    assert float((dec.head_prob - one.head_prob).abs().max()) < 1e-5
    v.poison()
    part = v.shard_rows(d["target_hidden"], d["draft_tokens"], **geo)
    out = v.verify_gathered(part.unsqueeze(0).contiguous(), d["target_hidden"], d["draft_tokens"], d["draft_hidden"],
                            d["csi"], **geo)
    torch.cuda.synchronize()
    assert v.device_error() == 0
    assert torch.equal(out.argmax, one.argmax) and torch.equal(out.accept_len, one.accept_len)
    compare(case, run_oracle(case), out, cfg.tau)
    v.close()
