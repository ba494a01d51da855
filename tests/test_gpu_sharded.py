"""LM head sharded by vocabulary: G contexts on slices of the LM head, their row partials gathered and merged.

One GPU stands in for the G GPUs: the shards run one after the other (no kernel waits for another), their
partials are stacked as an all-gather would, and the gathered round must equal the unsharded one.
"""
import numpy as np
import pytest
import torch

import gen
from gen import cases
from parity import compare, oracle_ref_argmax, run_oracle

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _cfg(**kw):
    base = dict(B=10, K=5, H=256, H_d=128, d_c=2, d_J=128, V=4096, match_rate=0.5, seed=41)
    base.update(kw)
    return gen.VerifyConfig("shard", **base)


@pytest.mark.parametrize("kw,cuts", [
    (dict(), [0, 2048, 4096]),                                   # two equal shards
    (dict(V=4099), [0, 1000, 3001, 4099]),                       # three uneven shards, odd vocabulary
    (dict(B=45, K=4, V=1500), [0, 700, 1500]),                   # 225 rows: CTA-pair kernel inside each shard
    (dict(K=0, K_lo=1, K_hi=9, B=16, mode="SH"), [0, 4096]),     # ragged, selective upload, one shard
    (dict(stochastic=True), [0, 1024, 2048, 3072, 4096]),        # four shards, sampling test
], ids=["G2", "G3odd", "G2pairs", "G1raggedSH", "G4stoch"])
def test_gathered_round_equals_unsharded_round(kw, cuts):
    cfg = _cfg(**kw)
    case = cases.make_case(cfg, oracle_ref_argmax)
    if cfg.stochastic:
        base = run_oracle(case)
        case["draft_q"] = (base["p_draft"] * np.random.default_rng(3).uniform(0.5, 4.0, size=case["T"])).astype(np.float32)
    d = cases.to_device(case, DEV)
    whole = cases.make_verifier(d)
    one = cases.run(whole, d)
    torch.cuda.synchronize()
    whole.close()

    geo = dict(B=cfg.B, K=cfg.K if cfg.K_hi == 0 else 0, k_off=d["k_off_dev"], T=case["T"])
    shards = [cases.make_verifier(d, vocab_slice=(lo, hi)) for lo, hi in zip(cuts[:-1], cuts[1:])]
    parts = torch.stack([v.shard_rows(d["target_hidden"], d["draft_tokens"], **geo) for v in shards])   # [G, R, 4]
    torch.cuda.synchronize()
    # the merge may run on any rank: take the last shard's context, and feed the shards in reverse order
    out = shards[-1].verify_gathered(parts.flip(0).contiguous(), d["target_hidden"], d["draft_tokens"],
                                     d["draft_hidden"], d["csi"], sel_off=d["sel_off"], sel_pos=d["sel_pos"],
                                     draft_q=d["draft_q"], uniforms=d["uniforms"], **geo)
    torch.cuda.synchronize()
    assert all(v.device_error() == 0 for v in shards)
    assert torch.equal(out.argmax, one.argmax)
    assert torch.equal(out.accept_len, one.accept_len) and torch.equal(out.correction_token, one.correction_token)
    assert torch.equal(out.n_mismatch, one.n_mismatch) and torch.equal(out.mismatch_mask, one.mismatch_mask)
    assert float((out.lse - one.lse).abs().max()) < 1e-5
    assert torch.allclose(out.p_draft, one.p_draft, rtol=1e-4, atol=0)
    # small batches evaluate the head inside the LM-head launch in a whole round but in a launch of its own here:
    # same products, another fp32 summation order
    assert float((out.head_prob - one.head_prob).abs().max()) < 1e-5
    compare(case, run_oracle(case), out, cfg.tau)
    for v in shards:
        v.close()


def test_shard_partials_are_per_shard_reductions():
    cfg = _cfg(B=3, K=3, V=600)
    case = cases.make_case(cfg, oracle_ref_argmax)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d, vocab_slice=(200, 600))
    part = v.shard_rows(d["target_hidden"], d["draft_tokens"], B=3, K=3).cpu().numpy()
    import oracle
    lm = oracle.lm_head(case["lm_head"][200:600], case["target_hidden"])
    assert np.array_equal(part[:, 1].view(np.int32), lm["argmax"] + 200)          # global token ids
    assert np.allclose(part[:, 0] + np.log(part[:, 2]), lm["lse"], atol=1e-4)
    toks = np.full(case["R"], -1)
    toks[np.repeat(case["row_off"][:-1], 3) + np.tile(np.arange(3), 3)] = case["draft_tokens"]
    owned = (toks >= 200) & (toks < 600)
    assert np.all(np.isneginf(part[~owned, 3])) and np.all(np.isfinite(part[owned, 3]))
    v.close()
