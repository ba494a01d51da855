"""CUDA path versus the CPU oracle, element by element, through the C ABI."""
import functools

import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2604_17701_b200 as wisv
from gen import cases
from parity import compare, oracle_ref_argmax, run_oracle

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


@functools.lru_cache(maxsize=4)
def _weights(cfg_key):
    return gen.make_weights(cfg_key)


def _shared_weights(cfg):
    # weights depend only on the model dimensions and the weight seed
    key = gen.VerifyConfig("w", B=1, K=1, H=cfg.H, H_d=cfg.H_d, d_c=cfg.d_c, d_J=cfg.d_J, V=cfg.V,
                           match_rate=0.0, seed=cfg.seed, weight_seed=cfg.weight_seed)
    return _weights(key)


def _small(name="s", **kw):
    base = dict(B=8, K=4, H=256, H_d=128, d_c=2, d_J=128, V=4096, match_rate=0.5, seed=0)
    base.update(kw)
    return gen.VerifyConfig(name, **base)


def _run(cfg, *, act=None, tau=None, shift=0, ref_fn=oracle_ref_argmax):
    case = cases.make_case(cfg, ref_fn, weights=_shared_weights(cfg))
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d, act=act, tau=tau, head_row_shift=shift)
    out = cases.run(v, d)
    torch.cuda.synchronize()
    assert v.device_error() == 0
    ref = run_oracle(case, act=act, tau=tau, head_row_shift=shift)
    stats = compare(case, ref, out, cfg.tau if tau is None else tau)
    v.close()
    return case, ref, out, stats


@pytest.mark.parametrize("B", [8, 52], ids=["R40", "R260"])     # one row tile; three row tiles, the last ragged
def test_raw_logits_match_oracle(B):
    cfg = _small(B=B, K=4)
    case = cases.make_case(cfg, oracle_ref_argmax)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    L = v.debug_logits(d["target_hidden"]).cpu().numpy()
    assert v.device_error() == 0
    ref = oracle.lm_head(case["lm_head"], case["target_hidden"], want_logits=True)["logits"]
    assert np.max(np.abs(L - ref)) < 2e-4
    v.close()


@pytest.mark.parametrize("act", ["gelu", "relu"])
@pytest.mark.parametrize("shift", [0, 1])
def test_tiny_config(act, shift):
    _run(gen.config("tiny"), act=act, shift=shift)


@pytest.mark.parametrize("kw", [
    dict(V=1000),                              # vocabulary tail inside a tile
    dict(V=4099, H=72, H_d=40),                # K tail (H not a multiple of 64), odd vocabulary
    dict(B=1, K=1),                            # smallest window
    dict(B=3, K=64, V=777),                    # longest window
    dict(B=40, K=4),                           # R = 200: two row tiles, ragged second tile
    dict(B=70, K=3, V=600, d_J=200),           # R = 280: three row tiles, head width not a tile multiple
    dict(B=100, K=4, V=700),                   # R = 500: two pair tiles of 256 rows, the last one ragged
    dict(B=16, K=0, K_lo=1, K_hi=9),           # ragged windows
    dict(match_rate=1.0),                      # full-match windows accept K
    dict(match_rate=0.0),                      # every position a candidate
    dict(d_c=0),                               # no CSI features
    dict(d_c=5, d_J=48),                       # odd CSI width
], ids=lambda kw: "-".join("%s%s" % (k, v) for k, v in kw.items()))
def test_shapes(kw):
    _run(_small(**kw))


@pytest.mark.parametrize("kw", [dict(B=2, K=8), dict(B=4, K=4, d_c=3), dict(B=3, K=1, H=72, H_d=40, d_J=50),
                                dict(B=5, K=3, act="relu"), dict(B=20, K=5, d_J=200)],
                         ids=["P16", "P16dc3", "P3odd", "P15relu", "P100"])
def test_split_k_head_matches_single_pass_head(kw):
    """One row tile of positions, the head in a launch of its own: the head GEMM splits K over CTAs;
    forcing a tile height turns that off."""
    cfg = _small(seed=17, **kw)
    case, ref, _, _ = _run(cfg)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    P = case["T"]
    v.set_tuning(head_ctas=-1)
    assert v.plan_kernels(case["R"], P) == 4
    for _ in range(2):                       # twice: the split-K tile counters must have reset themselves
        out = cases.run(v, d)
    torch.cuda.synchronize()
    assert v.device_error() == 0
    compare(case, ref, out, cfg.tau)
    v.set_tuning(head_ctas=-1, head_tile_n=16)
    o2 = cases.run(v, d)
    torch.cuda.synchronize()
    assert v.device_error() == 0
    compare(case, ref, o2, cfg.tau)
    assert float((o2.head_prob - out.head_prob).abs().max()) < 1e-5
    assert torch.equal(o2.accept_len, out.accept_len)
    v.set_tuning(head_ctas=-1)
    o3 = cases.run(v, d)
    assert torch.equal(o3.head_prob, out.head_prob)      # deterministic from call to call
    v.close()


@pytest.mark.parametrize("kw", [dict(B=2, K=8), dict(B=3, K=1, H=72, H_d=40, d_J=50), dict(B=20, K=5, d_J=200),
                                dict(B=14, K=8, d_c=3, act="relu"), dict(B=16, K=0, K_lo=1, K_hi=7)],
                         ids=["P16", "P3odd", "P100", "P112relu", "ragged"])
@pytest.mark.parametrize("head_ctas", [0, 1, 3, 40])
def test_one_launch_for_both_gemms_matches_separate_launches(kw, head_ctas):
    """At most 128 window rows and 128 head positions: LM-head CTAs and decision-head CTAs share a launch
    (three kernels per round); the result must not depend on how the CTAs are divided, and must equal the
    four-kernel round up to the fp32 summation order of the head partials."""
    cfg = _small(seed=29, **kw)
    case = cases.make_case(cfg, oracle_ref_argmax)
    ref = run_oracle(case)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    v.set_tuning(head_ctas=head_ctas)
    assert v.plan_kernels(case["R"], case["T"]) == 3
    plan = v.plan(case["R"], case["T"])
    assert plan["head_ctas"] >= 1 and plan["lm_ctas"] >= 1
    n0 = v.launch_count()
    for _ in range(2):
        out = cases.run(v, d)
    torch.cuda.synchronize()
    assert v.launch_count() - n0 == 6
    assert v.device_error() == 0
    compare(case, ref, out, cfg.tau)
    v.set_tuning(head_ctas=-1)
    sep = cases.run(v, d)
    torch.cuda.synchronize()
    assert torch.equal(sep.argmax, out.argmax) and torch.equal(sep.accept_len, out.accept_len)
    assert torch.equal(sep.correction_token, out.correction_token)
    assert float((sep.lse - out.lse).abs().max()) < 1e-5
    assert float((sep.head_prob - out.head_prob).abs().max()) < 1e-5
    v.close()


def test_cta_pair_kernel_matches_single_cta_kernel():
    """More than 128 window rows: the LM head runs on CTA pairs; the tuning switch forces the single-CTA kernel."""
    cfg = _small(B=50, K=4, V=1000, seed=23)               # 250 rows: one pair tile, second CTA ragged
    case, ref, out, _ = _run(cfg)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    plan = v.plan(case["R"], case["T"])
    assert plan["lm_ctas"] == 64 and plan["lm_tile_n"] == 32    # 32 units of 32 vocabulary rows, one per CTA pair
    assert v.plan_kernels(case["R"], case["T"]) == 3            # the decision head rides in the same launch
    v.set_tuning(lm_single_cta=1)
    assert v.plan(case["R"], case["T"])["lm_tiles"] == 8        # 2 row tiles x ceil(1000 / 256) tiles of 128 x 256
    assert v.plan_kernels(case["R"], case["T"]) == 4
    o2 = cases.run(v, d)
    torch.cuda.synchronize()
    assert v.device_error() == 0
    assert torch.equal(o2.argmax, out.argmax) and torch.equal(o2.accept_len, out.accept_len)
    assert float((o2.lse - out.lse).abs().max()) < 1e-5
    v.close()


@pytest.mark.parametrize("kw", [dict(B=26, K=4), dict(B=16, K=8, V=5000), dict(B=50, K=4, V=1000),
                                dict(B=28, K=8, d_J=200, V=4099), dict(B=40, K=0, K_lo=1, K_hi=9),
                                dict(B=30, K=6, mode="SH"), dict(B=25, K=9, stochastic=True)],
                         ids=["R130", "R144", "R250", "R252odd", "ragged", "SH", "stoch"])
@pytest.mark.parametrize("head_ctas", [0, 2, 5, -1], ids=["default", "h2", "h5", "separate"])
def test_two_row_tiles_pairs_with_head_clusters(kw, head_ctas):
    """129..256 window rows: the LM head runs on CTA pairs, each with one contiguous vocabulary range, and the
    decision head on extra clusters of the same launch (three kernels per round); -1 launches it separately."""
    cfg = _small(seed=37, **kw)
    case = cases.make_case(cfg, oracle_ref_argmax)
    if cfg.stochastic:
        base = run_oracle(case)
        case["draft_q"] = (base["p_draft"] * np.random.default_rng(5).uniform(0.5, 4.0, size=case["T"])).astype(np.float32)
    assert 128 < case["R"] <= 256
    ref = run_oracle(case)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    v.set_tuning(head_ctas=head_ctas)
    P = case["T"] if case["sel_pos"] is None else int(case["sel_pos"].shape[0])
    assert v.plan_kernels(case["R"], P) == (4 if head_ctas < 0 else 3)
    n0 = v.launch_count()
    for _ in range(2):
        out = cases.run(v, d)
    torch.cuda.synchronize()
    assert v.launch_count() - n0 == (8 if head_ctas < 0 else 6)
    assert v.device_error() == 0
    compare(case, ref, out, cfg.tau)
    v.set_tuning(lm_single_cta=1)
    one = cases.run(v, d)
    torch.cuda.synchronize()
    assert v.device_error() == 0
    assert torch.equal(one.argmax, out.argmax) and torch.equal(one.accept_len, out.accept_len)
    assert torch.equal(one.correction_token, out.correction_token)
    assert float((one.lse - out.lse).abs().max()) < 1e-5
    assert float((one.head_prob - out.head_prob).abs().max()) < 1e-5
    v.close()


@pytest.mark.parametrize("kw", [dict(B=60, K=4), dict(B=40, K=8, d_J=200), dict(B=100, K=4, V=2000),
                                dict(B=70, K=0, K_lo=2, K_hi=9, V=3000), dict(B=90, K=6, mode="SH")],
                         ids=["R300", "R360", "R500pairs", "ragged", "SH"])
def test_more_row_tiles_share_a_launch_when_it_costs_no_extra_round_of_tiles(kw):
    """More than 256 window rows: decision-head CTAs ride in the LM-head launch (single-CTA or pair kernel)
    whenever the LM head needs no additional round of tiles for it; the result must equal separate launches."""
    cfg = _small(seed=43, **kw)
    case = cases.make_case(cfg, oracle_ref_argmax)
    assert case["R"] > 256
    ref = run_oracle(case)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    P = case["T"] if case["sel_pos"] is None else int(case["sel_pos"].shape[0])
    # with so few vocabulary tiles the LM head is a single round of tiles and the automatic plan keeps the launches
    # apart (the head would outlast it); asking for head CTAs by hand skips that estimate, not the round check
    v.set_tuning(head_ctas=4)
    assert v.plan_kernels(case["R"], P) == 3
    out = cases.run(v, d)
    torch.cuda.synchronize()
    assert v.device_error() == 0
    compare(case, ref, out, cfg.tau)
    # a ragged last row tile with at most 64 rows runs on 64-row MMAs: forcing 128-row MMAs changes no bit
    v.set_tuning(head_ctas=4, lm_mma_m=128)
    big = cases.run(v, d)
    torch.cuda.synchronize()
    assert v.device_error() == 0
    for k in ("accept_len", "correction_token", "argmax", "lse", "p_draft", "head_prob", "n_mismatch", "status"):
        assert torch.equal(getattr(big, k), getattr(out, k)), k
    v.set_tuning(head_ctas=-1)
    assert v.plan_kernels(case["R"], P) == 4
    sep = cases.run(v, d)
    torch.cuda.synchronize()
    assert v.device_error() == 0
    assert torch.equal(sep.argmax, out.argmax) and torch.equal(sep.accept_len, out.accept_len)
    assert torch.equal(sep.correction_token, out.correction_token)
    # with fewer pairs for the LM head its teams cut the vocabulary into other ranges: the sums of exponentials are
    # added in another order
    assert float((sep.lse - out.lse).abs().max()) < 1e-5
    assert float((sep.head_prob - out.head_prob).abs().max()) < 1e-5
    v.close()


@pytest.mark.parametrize("B,K", [(1, 8), (4, 3), (2, 8), (8, 4), (7, 8), (8, 7), (13, 4)],
                         ids=["R9", "R16", "R18", "R40", "R63", "R64", "R65"])
@pytest.mark.parametrize("head_ctas", [0, -1], ids=["one_launch", "two_launches"])
def test_mma_of_64_rows_matches_mma_of_128_rows(B, K, head_ctas):
    """Up to 64 valid rows the GEMMs issue MMAs of 64 rows, whose accumulator rows sit in sixteen TMEM lanes of
    each quadrant; the products are the same, so forcing 128-row MMAs must not change a bit."""
    cfg = _small(B=B, K=K, seed=31, V=2000)
    case = cases.make_case(cfg, oracle_ref_argmax)
    ref = run_oracle(case)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    v.set_tuning(head_ctas=head_ctas)
    out = cases.run(v, d)
    torch.cuda.synchronize()
    assert v.device_error() == 0
    compare(case, ref, out, cfg.tau)
    L = v.debug_logits(d["target_hidden"])
    v.set_tuning(head_ctas=head_ctas, lm_mma_m=128)
    big = cases.run(v, d)
    L128 = v.debug_logits(d["target_hidden"])
    torch.cuda.synchronize()
    assert v.device_error() == 0
    assert torch.equal(L, L128)
    for k in ("accept_len", "correction_token", "argmax", "lse", "p_draft", "head_prob", "n_mismatch", "status"):
        assert torch.equal(getattr(big, k), getattr(out, k)), k
    v.close()


@pytest.mark.parametrize("tune", [dict(lm_tile_n=64), dict(lm_tile_n=256, lm_stages=2), dict(head_tile_n=64, head_stages=3)],
                         ids=lambda t: "-".join("%s%s" % kv for kv in t.items()))
def test_results_do_not_depend_on_the_launch_plan(tune):
    cfg = _small(B=20, K=5, seed=19)
    case = cases.make_case(cfg, oracle_ref_argmax)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    v.set_tuning(**tune)
    out = cases.run(v, d)
    torch.cuda.synchronize()
    assert v.device_error() == 0
    compare(case, run_oracle(case), out, cfg.tau)
    v.close()


@pytest.mark.parametrize("tau", [0.0, 0.35, 0.65, 1.5])
def test_thresholds(tau):
    case, ref, out, _ = _run(_small(B=24, K=6, seed=3), tau=tau)
    A = out.accept_len.cpu().numpy()
    if tau > 1:
        assert np.array_equal(A, case["k_len"])


@pytest.mark.parametrize("kw", [dict(), dict(K=0, K_lo=2, K_hi=12, B=32), dict(match_rate=1.0), dict(match_rate=0.0)],
                         ids=["uniform", "ragged", "emptyS", "fullS"])
def test_selective_hidden(kw):
    cfg = _small(mode="SH", seed=5, **{**dict(B=12, K=5), **kw})
    case, ref, out, _ = _run(cfg)
    # same decisions as full-hidden upload on the same traffic
    fh = cases.make_case(cfg.with_(mode="FH"), oracle_ref_argmax, weights=_shared_weights(cfg))
    d = cases.to_device(fh, DEV)
    v = cases.make_verifier(d)
    o2 = cases.run(v, d)
    assert torch.equal(o2.accept_len, out.accept_len) and torch.equal(o2.correction_token, out.correction_token)
    v.close()


def test_selective_hidden_missing_upload_is_rejected_and_flagged():
    cfg = _small(mode="SH", B=6, K=5, seed=7, match_rate=0.3)
    case = cases.make_case(cfg, oracle_ref_argmax)
    # drop the last uploaded hidden state of every request that has one
    keep, counts = [], []
    for b in range(cfg.B):
        lo, hi = int(case["sel_off"][b]), int(case["sel_off"][b + 1])
        kept = list(range(lo, max(lo, hi - 1)))
        keep += kept
        counts.append(len(kept))
    keep = np.asarray(keep, np.int64)
    case["sel_off"] = np.concatenate([[0], np.cumsum(counts)]).astype(np.int32)
    case["sel_pos"] = case["sel_pos"][keep]
    case["draft_hidden"] = case["draft_hidden"][keep]
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    out = cases.run(v, d)
    ref = run_oracle(case)
    compare(case, ref, out, cfg.tau)
    st = out.status.cpu().numpy()
    assert np.array_equal((st & 1) != 0, np.asarray(counts) < ref["n_mismatch"])
    v.close()


def test_selective_hidden_out_of_range_position_is_ignored_and_flagged():
    cfg = _small(mode="SH", B=6, K=5, seed=8, match_rate=0.3)
    case = cases.make_case(cfg, oracle_ref_argmax)
    b = next(i for i in range(cfg.B) if case["sel_off"][i + 1] - case["sel_off"][i] >= 2)
    j = int(case["sel_off"][b])                       # first uploaded entry of request b
    bad = dict(case)
    bad["sel_pos"] = case["sel_pos"].copy()
    bad["sel_pos"][j] = cfg.K + 3                     # not a window position
    d = cases.to_device(bad, DEV)
    v = cases.make_verifier(d)
    out = cases.run(v, d)
    torch.cuda.synchronize()
    st = out.status.cpu().numpy()
    assert st[b] & 8 and all(not (st[i] & 8) for i in range(cfg.B) if i != b)
    # same decisions as if that upload had never arrived
    keep = np.ones(case["sel_pos"].shape[0], bool)
    keep[j] = False
    less = dict(case)
    cnt = np.diff(case["sel_off"]).copy()
    cnt[b] -= 1
    less["sel_off"] = np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32)
    less["sel_pos"] = case["sel_pos"][keep]
    less["draft_hidden"] = case["draft_hidden"][keep]
    ref = run_oracle(less)
    A, Ao = out.accept_len.cpu().numpy(), ref["accept_len"]
    tie = np.zeros(cfg.B, bool)
    for i in range(cfg.B):
        rows = slice(ref["row_off"][i], ref["row_off"][i + 1])
        tie[i] = (ref["top2_gap"][rows] < 1e-2).any() or (np.abs(ref["prob_t"][ref["k_off"][i]:ref["k_off"][i + 1]] - cfg.tau) < 2e-3).any()
    assert np.array_equal(A[~tie], Ao[~tie])
    v.close()


def test_stochastic_acceptance():
    cfg = _small(B=32, K=6, seed=9, stochastic=True)
    case = cases.make_case(cfg, oracle_ref_argmax)
    # spread alpha = min(1, p/q) over (0, 1]: q = p_T(y) * U(0.5, 4)
    base = run_oracle(case)
    g = np.random.default_rng(1)
    case["draft_q"] = (base["p_draft"] * g.uniform(0.5, 4.0, size=case["T"])).astype(np.float32)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    for tau in (0.0, 0.5):
        out = cases.run(v, d, tau=tau)
        ref = run_oracle(case, tau=tau)
        st = compare(case, ref, out, tau)
        assert st["tainted_requests"] < cfg.B
    v.close()


def test_bad_token_ids_are_clamped_and_flagged():
    cfg = _small(B=4, K=4, seed=11)
    case = cases.make_case(cfg, oracle_ref_argmax)
    case["draft_tokens"] = case["draft_tokens"].copy()
    case["draft_tokens"][1] = cfg.V + 5
    case["draft_tokens"][9] = -3
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    out = cases.run(v, d)
    st = out.status.cpu().numpy()
    assert st[0] & 2 and st[2] & 2 and not (st[1] & 2) and not (st[3] & 2)
    A = out.accept_len.cpu().numpy()
    assert np.all(A >= 0) and np.all(A <= 4)
    v.close()


def test_host_buffer_entry_point_matches_device_entry_point():
    cfg = _small(B=9, K=5, seed=13)
    case = cases.make_case(cfg, oracle_ref_argmax)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    out = cases.run(v, d)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    ho = v.verify_host(pin(case["target_hidden"]), pin(case["draft_tokens"]), pin(case["draft_hidden"]),
                       pin(case["csi"]), B=cfg.B, K=cfg.K, extras=True)
    for k in ("accept_len", "correction_token", "argmax", "lse", "p_draft", "head_prob", "n_mismatch", "status"):
        assert torch.equal(getattr(ho, k), getattr(out, k).cpu()), k
    # pageable host memory works too (the copies are then synchronous staging copies)
    from paper_2604_17701_b200 import VerifyOutput
    page = lambda a: torch.from_numpy(np.ascontiguousarray(a).copy())
    po = VerifyOutput(torch.empty(cfg.B, dtype=torch.int32), torch.empty(cfg.B, dtype=torch.int32))
    po.argmax, po.lse = torch.empty(case["R"], dtype=torch.int32), torch.empty(case["R"], dtype=torch.float32)
    po.p_draft, po.head_prob = torch.empty(case["T"]), torch.empty(case["T"])
    po.mismatch_mask = torch.empty(cfg.B, dtype=torch.int64)
    po.n_mismatch, po.status = torch.empty(cfg.B, dtype=torch.int32), torch.empty(cfg.B, dtype=torch.int32)
    v.verify_host(page(case["target_hidden"]), page(case["draft_tokens"]), page(case["draft_hidden"]),
                  page(case["csi"]), B=cfg.B, K=cfg.K, extras=True, out=po)
    for k in ("accept_len", "correction_token", "argmax", "lse", "p_draft", "head_prob", "n_mismatch", "status"):
        assert torch.equal(getattr(po, k), getattr(out, k).cpu()), k
    v.close()


def test_bound_host_call_sees_buffers_refilled_in_place():
    """Serving loop: pinned buffers bound once, refilled in place, one wisv_verify_host per step; each step must
    equal a device-entry-point round on that step's data (also exercises the completion word, step after step)."""
    cfgs = [_small(B=6, K=5, seed=s, weight_seed=50) for s in (51, 52, 53)]       # one model, three batches
    built = [cases.make_case(c, oracle_ref_argmax, weights=_shared_weights(c)) for c in cfgs]
    d0 = cases.to_device(built[0], DEV)
    v = cases.make_verifier(d0)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    bufs = {k: pin(built[0][k]) for k in ("target_hidden", "draft_tokens", "draft_hidden", "csi")}
    call = v.bind_host(bufs["target_hidden"], bufs["draft_tokens"], bufs["draft_hidden"], bufs["csi"],
                       B=cfgs[0].B, K=cfgs[0].K, extras=True)
    for case in built * 2:
        for k, t in bufs.items():
            t.copy_(torch.from_numpy(np.ascontiguousarray(case[k])))
        ho = call()
        ref = cases.run(v, cases.to_device(case, DEV))
        torch.cuda.synchronize()
        for k in ("accept_len", "correction_token", "argmax", "lse", "p_draft", "head_prob", "n_mismatch", "status"):
            assert torch.equal(getattr(ho, k), getattr(ref, k).cpu()), k
        compare(case, run_oracle(case), ho, cfgs[0].tau)
    assert v.device_error() == 0
    v.close()


@pytest.mark.parametrize("pinned", [True, False])
def test_host_buffer_entry_point_ragged_selective_stochastic(pinned):
    """Every optional input (row offsets, selective positions, q and u of Eq. 1) through the packed host block; the
    target hidden states exceed the in-place limit (copy-engine path) while the draft ones stay below it."""
    cfg = _small(B=40, K=0, K_lo=1, K_hi=8, H=2048, H_d=128, mode="SH", stochastic=True, seed=71)
    case = cases.make_case(cfg, oracle_ref_argmax)
    assert case["R"] * cfg.H * 4 > (1 << 20) > case["sel_pos"].shape[0] * cfg.H_d * 4
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    out = cases.run(v, d)
    mk = (lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()) if pinned else \
        (lambda a: torch.from_numpy(np.ascontiguousarray(a).copy()))
    for _ in range(2):                           # the staging blocks are reused by the second call
        ho = v.verify_host(mk(case["target_hidden"]), mk(case["draft_tokens"]), mk(case["draft_hidden"]),
                           mk(case["csi"]), B=cfg.B, k_off=mk(case["k_off"]), T=case["T"], sel_off=mk(case["sel_off"]),
                           sel_pos=mk(case["sel_pos"]), draft_q=mk(case["draft_q"]), uniforms=mk(case["uniforms"]),
                           extras=True)
        for k in ("accept_len", "correction_token", "argmax", "lse", "p_draft", "head_prob", "mismatch_mask",
                  "n_mismatch", "status"):
            assert torch.equal(getattr(ho, k), getattr(out, k).cpu()), k
    assert v.device_error() == 0
    v.close()


def test_bounded_wait_gives_up_and_the_context_stays_usable():
    cfg = _small(B=4, K=4, seed=29)
    case = cases.make_case(cfg, oracle_ref_argmax)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    ref = cases.run(v, d)
    assert v.device_error() == 0
    v.wait_probe(2_000_000)                       # about 1 ms: a barrier nobody arrives on
    assert v.device_error() == 2                  # reported ...
    assert v.device_error() == 0                  # ... and cleared
    out = cases.run(v, d)                         # the context still works
    torch.cuda.synchronize()
    assert torch.equal(out.accept_len, ref.accept_len) and v.device_error() == 0
    v.close()


def test_empty_windows_and_empty_batch():
    """K_b = 0 for some or all requests: nothing to accept, the correction is the bonus-row argmax."""
    cfg = _small(B=6, K=0, K_lo=0, K_hi=2, seed=37)
    case = cases.make_case(cfg, oracle_ref_argmax)
    assert (case["k_len"] == 0).any()
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    out = cases.run(v, d)
    torch.cuda.synchronize()
    compare(case, run_oracle(case), out, cfg.tau)
    # every window empty: T = 0, only the B bonus rows go through the LM head
    k_off0 = torch.zeros(cfg.B + 1, dtype=torch.int32, device=DEV)
    rows = d["target_hidden"][:cfg.B].contiguous()
    o = v.verify(rows, d["draft_tokens"][:0], d["draft_hidden"][:0], d["csi"], B=cfg.B, k_off=k_off0, T=0)
    torch.cuda.synchronize()
    import oracle
    ref = oracle.lm_head(case["lm_head"], case["target_hidden"][:cfg.B])
    assert np.array_equal(o.accept_len.cpu().numpy(), np.zeros(cfg.B, np.int32))
    gap_ok = ref["top2_gap"] >= 1e-2
    assert np.array_equal(o.correction_token.cpu().numpy()[gap_ok], ref["argmax"][gap_ok])
    # no requests at all: accepted, nothing launched
    n = v.launch_count()
    v.verify(rows, d["draft_tokens"][:0], d["draft_hidden"][:0], d["csi"], B=0, K=4, T=0)
    assert v.launch_count() == n and v.device_error() == 0
    v.close()


def test_host_entry_point_with_selective_upload_and_sampling_test():
    cfg = _small(B=7, K=0, K_lo=2, K_hi=6, mode="SH", stochastic=True, seed=39)
    case = cases.make_case(cfg, oracle_ref_argmax)
    base = run_oracle(case)
    case["draft_q"] = (base["p_draft"] * np.random.default_rng(5).uniform(0.5, 4.0, size=case["T"])).astype(np.float32)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    out = cases.run(v, d)
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    ho = v.verify_host(pin(case["target_hidden"]), pin(case["draft_tokens"]), pin(case["draft_hidden"]),
                       pin(case["csi"]), B=cfg.B, k_off=pin(case["k_off"]), T=case["T"], sel_off=pin(case["sel_off"]),
                       sel_pos=pin(case["sel_pos"]), draft_q=pin(case["draft_q"]), uniforms=pin(case["uniforms"]),
                       extras=True)
    for k in ("accept_len", "correction_token", "argmax", "lse", "p_draft", "head_prob", "n_mismatch", "status"):
        assert torch.equal(getattr(ho, k), getattr(out, k).cpu()), k
    compare(case, run_oracle(case), out, cfg.tau)
    v.close()


def test_window_longer_than_the_limit_in_device_offsets_is_cut_and_flagged():
    """k_off lives on the device, so wisv_verify cannot see a window of more than 64 tokens: the device verifies its
    first 64 positions and says so in the request's status word; the other requests are untouched.  With host
    buffers the library sees the offsets and refuses the batch."""
    cfg = _small(B=4, K=0, K_lo=3, K_hi=9, seed=61, V=1000)
    k_len = np.array([5, 70, 3, 9], np.int32)                       # request 1 is too long; T = 87 <= 64 * B
    k_off, row_off = gen.row_offsets(k_len)
    w = _shared_weights(cfg)
    T, R = int(k_off[-1]), int(row_off[-1])
    g = np.random.default_rng(61)
    ht = g.standard_normal((R, cfg.H), dtype=np.float32)
    hd = g.standard_normal((T, cfg.H_d), dtype=np.float32)
    csi = g.uniform(1.0, 30.0, size=(cfg.B, cfg.d_c)).astype(np.float32)
    ref_am = oracle_ref_argmax(w["lm_head"], ht)
    rows = np.concatenate([row_off[b] + np.arange(k_len[b]) for b in range(cfg.B)])
    toks = np.where(g.random(T) < 0.8, ref_am[rows], g.integers(0, cfg.V, size=T)).astype(np.int32)
    case = dict(cfg=cfg, k_len=k_len, k_off=k_off, row_off=row_off, T=T, R=R, draft_tokens=toks, target_hidden=ht,
                csi=csi, draft_hidden=hd, sel_off=None, sel_pos=None, draft_q=None, uniforms=None, **w)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d, max_requests=cfg.B, max_rows=R)
    out = cases.run(v, d)
    torch.cuda.synchronize()
    assert v.device_error() == 0
    st = out.status.cpu().numpy()
    assert st[1] & 16 and not any(st[b] & 16 for b in (0, 2, 3))
    ref = run_oracle(case)                                          # the oracle has no window limit
    A, corr = out.accept_len.cpu().numpy(), out.correction_token.cpu().numpy()
    tie = ref["top2_gap"] < 1e-2
    ptie = np.abs(ref["head_prob"] - cfg.tau) < 2e-3
    for b in (0, 2, 3):
        if tie[row_off[b]:row_off[b + 1]].any() or ptie[k_off[b]:k_off[b + 1]].any():
            continue
        assert A[b] == ref["accept_len"][b] and corr[b] == ref["correction_token"][b]
    # the long window: verified over its first 64 positions only
    assert 0 <= A[1] <= 64
    if not tie[row_off[1]:row_off[1] + 65].any() and not ptie[k_off[1]:k_off[1] + 64].any():
        assert A[1] == min(int(ref["accept_len"][1]), 64)
    seen_rows = np.ones(R, bool)
    seen_rows[row_off[1] + 65:row_off[2]] = False                   # rows past the cut are not reported
    assert np.max(np.abs(out.lse.cpu().numpy() - ref["lse"])[seen_rows]) <= 1e-2
    pin = lambda a: torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    from paper_2604_17701_b200 import WisvError
    with pytest.raises(WisvError) as e:
        v.verify_host(pin(ht), pin(toks), pin(hd), pin(csi), B=cfg.B, k_off=pin(k_off), T=T)
    assert e.value.code == -2
    v.close()


def _as16(a, kind):
    """numpy view of a hidden-state array in a 16-bit upload format, and the same as a torch CPU tensor."""
    if kind == "f16":
        h = np.ascontiguousarray(a, np.float32).astype(np.float16)
        return h, torch.from_numpy(h.copy())
    bits = gen.f32_to_bf16_bits(a)
    return bits, torch.from_numpy(bits.view(np.int16).copy()).view(torch.bfloat16)


@pytest.mark.parametrize("th,dh", [("bf16", "f16"), ("f16", "bf16"), ("f32", "f16"), ("bf16", "f32")])
@pytest.mark.parametrize("kw", [dict(B=9, K=5), dict(B=30, K=6, mode="SH"), dict(B=70, K=0, K_lo=1, K_hi=7, V=3000)],
                         ids=["R54", "R210_SH", "R350_ragged"])
def test_sixteen_bit_hidden_states(kw, th, dh):
    """The drafter uploads hidden states with 16 bits per element (Section IV-A); the target's may be 16-bit too.
    bf16 is used as it is, fp16 is rounded to bf16 like fp32: against the oracle on the same 16-bit arrays, through
    the device entry point and the host-buffer one."""
    cfg = _small(seed=83, **kw)
    case = cases.make_case(cfg, oracle_ref_argmax)
    ocase, dev_t = dict(case), {}
    for key, kind in (("target_hidden", th), ("draft_hidden", dh)):
        if kind == "f32":
            dev_t[key] = torch.from_numpy(np.ascontiguousarray(case[key]))
        else:
            ocase[key], dev_t[key] = _as16(case[key], kind)
    ref = run_oracle(ocase)
    d = cases.to_device(case, DEV)
    d["target_hidden"], d["draft_hidden"] = dev_t["target_hidden"].to(DEV), dev_t["draft_hidden"].to(DEV)
    v = cases.make_verifier(d)
    out = cases.run(v, d)
    torch.cuda.synchronize()
    assert v.device_error() == 0
    compare(ocase, ref, out, cfg.tau)
    pin = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    ho = v.verify_host(dev_t["target_hidden"].pin_memory(), pin(case["draft_tokens"]), dev_t["draft_hidden"].pin_memory(),
                       pin(case["csi"]), B=cfg.B, K=cfg.K if cfg.K_hi == 0 else 0,
                       k_off=pin(case["k_off"]) if cfg.K_hi > 0 else None, T=case["T"], sel_off=pin(case["sel_off"]),
                       sel_pos=pin(case["sel_pos"]), extras=True)
    for k in ("accept_len", "correction_token", "argmax", "lse", "p_draft", "head_prob", "n_mismatch", "status"):
        assert torch.equal(getattr(ho, k), getattr(out, k).cpu()), k
    v.close()


@pytest.mark.parametrize("kw", [dict(B=320, K=9), dict(B=520, K=0, K_lo=2, K_hi=12, mode="SH", stochastic=True),
                                dict(B=380, K=9, h16=True)], ids=["uniform", "ragged_SH_stoch", "f16_uploads"])
def test_host_entry_point_pipelines_large_batches_group_by_group(kw):
    """More than 32 MB of hidden states: the host-buffer call cuts the batch into groups of whole requests and
    verifies one group while the next is in flight.  Windows are independent, so the result must equal the oracle and
    the one-piece device round (up to the fp32 summation order of the log-sum-exp, which follows the launch plan)."""
    kw = dict(kw)
    h16 = kw.pop("h16", False)
    cfg = _small(seed=91, H=2048, H_d=1024, V=1000, d_J=64, **kw)
    case = cases.make_case(cfg, oracle_ref_argmax)
    if cfg.stochastic:
        base = run_oracle(case)
        case["draft_q"] = (base["p_draft"] * np.random.default_rng(5).uniform(0.5, 4.0, size=case["T"])).astype(np.float32)
    ocase = dict(case)
    th_t = torch.from_numpy(np.ascontiguousarray(case["target_hidden"]))
    dh_t = torch.from_numpy(np.ascontiguousarray(case["draft_hidden"]))
    if h16:
        ocase["draft_hidden"], dh_t = _as16(case["draft_hidden"], "f16")
    n_bytes = th_t.numel() * th_t.element_size() + dh_t.numel() * dh_t.element_size()
    assert n_bytes > (32 << 20)
    ref = run_oracle(ocase)
    d = cases.to_device(case, DEV)
    d["draft_hidden"] = dh_t.to(DEV)
    v = cases.make_verifier(d)
    out = cases.run(v, d)
    torch.cuda.synchronize()
    compare(ocase, ref, out, cfg.tau)
    pin = lambda a: None if a is None else torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
    n0 = v.launch_count()
    for _ in range(2):                                   # twice: staging, events and offsets are reused
        ho = v.verify_host(th_t.pin_memory(), pin(case["draft_tokens"]), dh_t.pin_memory(), pin(case["csi"]), B=cfg.B,
                           K=cfg.K if cfg.K_hi == 0 else 0, k_off=pin(case["k_off"]) if cfg.K_hi > 0 else None,
                           T=case["T"], sel_off=pin(case["sel_off"]), sel_pos=pin(case["sel_pos"]),
                           draft_q=pin(case["draft_q"]), uniforms=pin(case["uniforms"]), extras=True)
    assert v.launch_count() - n0 >= 2 * 3 * 3            # at least three groups of at least three kernels per call
    assert v.device_error() == 0
    compare(ocase, ref, ho, cfg.tau)
    assert torch.equal(ho.argmax, out.argmax.cpu()) and torch.equal(ho.accept_len, out.accept_len.cpu())
    assert torch.equal(ho.correction_token, out.correction_token.cpu()) and torch.equal(ho.mismatch_mask, out.mismatch_mask.cpu())
    assert float((ho.lse - out.lse.cpu()).abs().max()) < 1e-4
    assert float((ho.head_prob - out.head_prob.cpu()).abs().max()) < 1e-5
    v.close()


def test_capacity_and_argument_errors():
    cfg = _small(B=4, K=4)
    case = cases.make_case(cfg, oracle_ref_argmax)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    from paper_2604_17701_b200 import WisvError
    with pytest.raises(WisvError) as e:
        v.verify(d["target_hidden"], d["draft_tokens"], d["draft_hidden"], d["csi"], B=5, K=4)
    assert e.value.code == -4
    with pytest.raises(WisvError) as e:
        v.verify(d["target_hidden"], d["draft_tokens"], d["draft_hidden"], d["csi"], B=1, K=65)
    assert e.value.code == -2
    with pytest.raises(WisvError) as e:
        v.verify(None, d["draft_tokens"], d["draft_hidden"], d["csi"], B=4, K=4)
    assert e.value.code == -1
    v.close()


# ------------------------------------------------------------------ 8B shapes

def _lib_ref(lm_head_bits, target_hidden):
    return cases.library_ref_argmax(lm_head_bits, target_hidden, device=DEV)


def _subset_case(case, reqs):
    """The same traffic restricted to a few whole requests (requests are independent)."""
    cfg = case["cfg"]
    k_len = case["k_len"][reqs]
    tok_idx = np.concatenate([np.arange(case["k_off"][b], case["k_off"][b + 1]) for b in reqs]).astype(np.int64)
    row_idx = np.concatenate([np.arange(case["row_off"][b], case["row_off"][b + 1]) for b in reqs]).astype(np.int64)
    k_off, row_off = gen.row_offsets(k_len)
    sub = dict(case)
    sub.update(cfg=cfg.with_(B=len(reqs)), k_len=k_len, k_off=k_off, row_off=row_off, T=int(k_off[-1]),
               R=int(row_off[-1]), target_hidden=case["target_hidden"][row_idx],
               draft_tokens=case["draft_tokens"][tok_idx], csi=case["csi"][reqs])
    if case["sel_off"] is not None:
        sel_idx = np.concatenate([np.arange(case["sel_off"][b], case["sel_off"][b + 1]) for b in reqs]).astype(np.int64)
        cnt = np.array([case["sel_off"][b + 1] - case["sel_off"][b] for b in reqs])
        sub.update(sel_off=np.concatenate([[0], np.cumsum(cnt)]).astype(np.int32), sel_pos=case["sel_pos"][sel_idx],
                   draft_hidden=case["draft_hidden"][sel_idx])
        ev_idx = sel_idx
    else:
        sub.update(draft_hidden=case["draft_hidden"][tok_idx])
        ev_idx = tok_idx
    for k in ("draft_q", "uniforms"):
        if case[k] is not None:
            sub[k] = case[k][tok_idx]
    return sub, row_idx, tok_idx, ev_idx


class _Sub:
    pass


def _subset_output(out, reqs, row_idx, tok_idx, ev_idx):
    s = _Sub()
    r, t, e, q = (torch.as_tensor(x, device=out.accept_len.device) for x in (row_idx, tok_idx, ev_idx, np.asarray(reqs)))
    s.accept_len, s.correction_token = out.accept_len[q], out.correction_token[q]
    s.n_mismatch, s.mismatch_mask, s.status = out.n_mismatch[q], out.mismatch_mask[q], out.status[q]
    s.argmax, s.lse, s.p_draft, s.head_prob = out.argmax[r], out.lse[r], out.p_draft[t], out.head_prob[e]
    return s


def _check_properties(case, out):
    """Properties that hold at any size, checked on the full batch."""
    k_len, k_off, row_off = case["k_len"], case["k_off"], case["row_off"]
    A = out.accept_len.cpu().numpy()
    corr = out.correction_token.cpu().numpy()
    am = out.argmax.cpu().numpy()
    assert np.all(A >= 0) and np.all(A <= k_len)
    assert np.array_equal(corr, am[row_off[:-1] + A])              # correction / bonus = argmax of row A
    assert np.all(np.isfinite(out.lse.cpu().numpy()))
    assert np.all(out.status.cpu().numpy() & ~1 == 0)
    if case["draft_q"] is None:
        rows = np.repeat(row_off[:-1], k_len) + (np.arange(case["T"]) - np.repeat(k_off[:-1], k_len))
        mism = case["draft_tokens"] != am[rows]
        first = np.array([next((i for i in range(k_len[b]) if mism[k_off[b] + i]), k_len[b]) for b in range(len(k_len))])
        assert np.all(A >= first)                                   # the head only extends the greedy span
        nm = out.n_mismatch.cpu().numpy()
        cnt = np.add.reduceat(mism.astype(np.int32), k_off[:-1])
        assert np.array_equal(nm, np.where(k_len > 0, cnt, 0))
    return A


def _sampled_parity(name, n_sample, seed_pick=0, cfg=None):
    cfg = cfg if cfg is not None else gen.config(name)
    case = cases.make_case(cfg, _lib_ref, weights=_shared_weights(cfg))
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    out = cases.run(v, d)
    torch.cuda.synchronize()
    assert v.device_error() == 0
    A = _check_properties(case, out)
    B = cfg.B
    if n_sample >= B:
        reqs = list(range(B))
    else:
        # first, last, requests straddling 128-row tile boundaries, then a seeded random fill
        picks = {0, B - 1}
        for edge in range(128, case["R"], 128):
            picks.add(int(np.searchsorted(case["row_off"], edge, side="right") - 1))
            if len(picks) >= n_sample // 2:
                break
        rest = [b for b in np.random.default_rng(seed_pick).permutation(B) if b not in picks]
        reqs = sorted(list(picks) + [int(b) for b in rest[:max(0, n_sample - len(picks))]])
    sub, row_idx, tok_idx, ev_idx = _subset_case(case, reqs)
    ref = run_oracle(sub)
    stats = compare(sub, ref, _subset_output(out, reqs, row_idx, tok_idx, ev_idx), cfg.tau)
    v.close()
    return case, out, A, stats


def test_8b_batch1_full_oracle():
    _sampled_parity("8b_b1", 1)


@pytest.mark.parametrize("name", ["8b_b16", "8b_b32"])
def test_8b_two_and_three_row_tiles_sampled(name):
    # 144 rows: CTA pairs with balanced vocabulary ranges + decision-head clusters; 288 rows: two teams of pairs, one
    # per row block of 144, with decision-head clusters in the same launch
    case, out, A, stats = _sampled_parity(name, 12)
    assert stats["tainted_requests"] < stats["requests"]


@pytest.mark.parametrize("name", ["8b_b64_m30", "8b_b64", "8b_b64_m95"])
def test_8b_batch64_sampled(name):
    case, out, A, stats = _sampled_parity(name, 16)
    assert stats["tainted_requests"] < stats["requests"]


def test_8b_selective_hidden_sampled():
    case, out, A, stats = _sampled_parity("8b_sh256", 24)
    assert stats["tainted_requests"] < stats["requests"]


def test_qwen_shapes_batch1_full_oracle():
    # H = 3584 (56 K blocks), V = 152064, H_d = 896: the second model pair of the paper's testbed
    _sampled_parity("qwen7b_b1", 1)


def test_qwen_shapes_longest_window_sampled():
    # K = 64, the largest draft length of Table I; 520 window rows over 5 row tiles
    case, out, A, stats = _sampled_parity("qwen7b_b8_k64", 2)
    assert stats["tainted_requests"] <= stats["requests"]


@pytest.mark.parametrize("name", ["8b_b512", "8b_b512_stoch"])
def test_8b_batch512_sampled(name):
    case, out, A, stats = _sampled_parity(name, 20)
    if name == "8b_b512":
        # i.i.d. per-position accept probability a = r' + (1 - r') P(p < tau): closed-form mean
        k = 16
        am = out.argmax.cpu().numpy()
        rows = np.repeat(case["row_off"][:-1], case["k_len"]) + (np.arange(case["T"]) - np.repeat(case["k_off"][:-1], case["k_len"]))
        mism = case["draft_tokens"] != am[rows]
        hp = out.head_prob.cpu().numpy()
        a = 1.0 - np.mean(mism & (hp >= 0.5))
        expect = a * (1 - a ** k) / (1 - a)
        var = np.var(A)
        assert abs(A.mean() - expect) < 4 * np.sqrt(var / len(A)) + 0.05


@pytest.mark.parametrize("B,K", [(100, 16), (1100, 16)], ids=["R1700_seven_row_blocks", "R18700_three_raster_groups"])
def test_8b_row_counts_beyond_the_bench_configurations_sampled(B, K):
    # 1700 rows: round-robin work items in one raster group, the decision head in its own launch with 128-column tiles;
    # 18700 rows: 74 row blocks in three raster groups, twice the rows of the largest bench configuration
    cfg = gen.config("8b_b512").with_(B=B, K=K, name="8b_b%d" % B, seed=4242 + B)
    case, out, A, stats = _sampled_parity(cfg.name, 12, cfg=cfg)
    v_plan = wisv.plan_host(H=cfg.H, V=cfg.V, H_d=cfg.H_d, d_c=cfg.d_c, d_J=cfg.d_J, R=case["R"], P=case["T"])
    assert v_plan["lm_pair"] == 1 and v_plan["lm_carry"] == 0 and v_plan["lm_row_blocks"] == -(-case["R"] // 256)
    assert stats["tainted_requests"] < stats["requests"]


def test_random_shapes_under_every_launch_plan():
    """Seeded sweep over row counts around the plan boundaries (64/65, 128/129, 256/257, 384/385 rows), odd
    vocabulary, hidden and head sizes, ragged windows, both upload modes and both acceptance rules: every case
    must match the oracle under the automatic plan, with the GEMMs launched separately, on the single-CTA LM
    head only, and with an odd number of decision-head CTAs - and all four must agree on argmax and accept_len."""
    rng = np.random.default_rng(2024)
    for it in range(40):
        ragged = rng.random() < 0.3
        K = int(rng.integers(1, 13))
        target_rows = int(rng.choice([5, 16, 17, 63, 64, 65, 127, 128, 129, 200, 255, 256, 257, 300, 384, 385, 520, 780,
                                      1040]))
        kw = dict(B=max(1, target_rows // (K + 1)), K=0 if ragged else K, H=int(rng.choice([64, 72, 128, 256])),
                  H_d=int(rng.choice([8, 40, 64, 128])), d_c=int(rng.choice([0, 2, 3])),
                  d_J=int(rng.choice([16, 48, 50, 128, 200, 272])),
                  V=int(rng.choice([17, 31, 100, 600, 1000, 2049, 4096, 5000, 40000])),
                  match_rate=float(rng.choice([0.0, 0.5, 0.9, 1.0])), seed=3000 + it,
                  mode=str(rng.choice(["FH", "SH"])), act=str(rng.choice(["gelu", "relu"])),
                  stochastic=bool(rng.random() < 0.2))
        if ragged:
            kw.update(K_lo=1, K_hi=K + 1)
        cfg = gen.VerifyConfig("rnd", **kw)
        case = cases.make_case(cfg, oracle_ref_argmax)
        if cfg.stochastic:
            base = run_oracle(case)
            case["draft_q"] = (base["p_draft"] * rng.uniform(0.5, 4.0, size=case["T"])).astype(np.float32)
        ref = run_oracle(case)
        d = cases.to_device(case, DEV)
        v = cases.make_verifier(d)
        outs = []
        for tune in (dict(), dict(head_ctas=-1), dict(lm_single_cta=1), dict(head_ctas=3), dict(lm_kb_per_stage=1),
                     dict(lm_kb_per_stage=4), dict(lm_teams=-1), dict(lm_teams=1, head_ctas=-1)):
            v.set_tuning(**tune)
            cases.run(v, d)
            out = cases.run(v, d)                       # twice: nothing may linger from the first call
            torch.cuda.synchronize()
            assert v.device_error() == 0, (kw, tune)
            compare(case, ref, out, cfg.tau)
            outs.append(out)
        for o in outs[1:]:
            assert torch.equal(o.argmax, outs[0].argmax) and torch.equal(o.accept_len, outs[0].accept_len), kw
        v.close()
