"""Exact ties between logits: the CUDA path must return the lowest token id at every place where it merges.

Greedy verification compares the draft token with the target's argmax and the emitted correction token is that
argmax (Section II-A; Algorithm 1, commit-and-correct), so a tie has to be broken the same way everywhere: the
lowest id (the oracle's strict '>' scan).  Duplicated rows of the LM head give bit-identical fp32 logits on the
GPU and bit-identical fp64 logits in the oracle, so the expected answer is exact.  The duplicates are planted so
that the equal maxima of a window row meet at each merge site of the kernels: inside one 16-column chunk of the
epilogue (one warp's 32 vocabulary rows in the CTA-pair kernel), in different chunks of one tile (different warps
there), in different tiles of one CTA's (or CTA pair's) carried vocabulary range, in different CTAs / pairs, in
the two halves of a pair tile (its two CTAs), in different vocabulary shards - under 64- and 128-row MMAs, carried
and per-tile partials, and through every entry point that reduces the LM head.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2604_17701_b200 as wisv
from gen import cases
from parity import compare, oracle_ref_argmax, run_oracle

DEV = "cuda:0"
V, H = 40000, 128
SM, SMEM = 148, 232448


def _cfg(B, K, **kw):
    base = dict(B=B, K=K, H=H, H_d=64, d_c=2, d_J=64, V=V, match_rate=0.6, seed=77, weight_seed=78)
    base.update(kw)
    return gen.VerifyConfig("ties", **base)


def _owner_fn(plan):
    """token id -> (CTA or pair, tile within its range, 16-column chunk, half of a pair tile) under `plan`."""
    pair, carry, tile_n = plan["lm_pair"], plan["lm_carry"], plan["lm_tile_n"]
    unit = 32 if pair else 16
    if not carry:
        tn = 256 if pair else tile_n
        return lambda v: (v // tn, 0, (v % tn) // 16, int(pair and (v % tn) >= tn // 2))
    groups = plan["lm_ctas"] // 2 if pair else plan["lm_ctas"]
    base, rem, tpc = plan["lm_units_base"], plan["lm_units_rem"], plan["lm_tiles_per_cta"]

    def owner(v):
        u = v // unit
        if u < rem * (base + 1):
            c, off, mine = u // (base + 1), u % (base + 1), base + 1
        else:
            c, off, mine = rem + (u - rem * (base + 1)) // base, (u - rem * (base + 1)) % base, base
        hq, hr = mine // tpc, mine % tpc
        t, start = 0, 0
        while True:
            h = hq + (1 if t < hr else 0)
            if off < start + h:
                break
            start += h
            t += 1
        in_tile = (off - start) * unit + v % unit
        return c, t, in_tile // 16, int(pair and in_tile >= h * unit // 2)
    return owner


def _find(rng, pred, used, tries=200000):
    for _ in range(tries):
        v = int(rng.integers(0, V))
        got = pred(v)
        if got and not (set(got) & used) and len(set(got)) == len(got) and all(0 <= x < V for x in got):
            return sorted(got)
    raise AssertionError("no placement found")


def _placements(plan, rng, n_groups):
    """Tie groups (sorted token ids) and the merge site each one exercises."""
    own = _owner_fn(plan)
    used, out = set(), []

    def add(name, pred):
        g = _find(rng, pred, used)
        used.update(g)
        out.append((name, g))

    def first(v, ds, cond):
        return next(((v, v + d) for d in ds if v + d < V and cond(own(v), own(v + d))), None)

    add("same_chunk", lambda v: v % 16 <= 8 and (v, v + 5))
    add("chunks_of_one_tile", lambda v: first(v, (16,), lambda a, b: a[:2] == b[:2] and a[2] != b[2]))
    add("three_in_one_tile", lambda v: v + 40 < V and own(v)[:2] == own(v + 40)[:2] and (v, v + 17, v + 40))
    add("different_ctas", lambda v: first(v, (3000,), lambda a, b: a[0] != b[0]))
    add("far_apart_three", lambda v: v < V // 4 and (v, v + V // 3 + 5, v + 2 * (V // 3) + 11))
    add("first_and_last_token", lambda v: (0, V - 1))
    if plan["lm_carry"] and plan["lm_tiles_per_cta"] > 1:
        add("tiles_of_one_cta", lambda v: first(v, (64, 96, 128, 160, 192, 224, 256),
                                                lambda a, b: a[0] == b[0] and a[1] != b[1]))
    if plan["lm_pair"]:
        add("halves_of_a_pair_tile", lambda v: first(v, (48, 96, 112, 128), lambda a, b: a[:2] == b[:2] and a[3] != b[3]))
    return out[:n_groups]


def _planted_case(cfg):
    """A case whose LM head has groups of identical rows, each group holding the top logit of one window row."""
    R, P = cfg.B * (cfg.K + 1), cfg.B * cfg.K
    plan = wisv.plan_host(H=cfg.H, V=cfg.V, H_d=cfg.H_d, d_c=cfg.d_c, d_J=cfg.d_J, R=R, P=P, sm_count=SM,
                          max_smem_bytes=SMEM)
    w = {k: (v.copy() if isinstance(v, np.ndarray) else v) for k, v in gen.make_weights(cfg).items()}
    k_len = gen.synth.window_lengths(cfg)
    ht = gen.make_hidden(cfg, k_len)["target_hidden"]
    base = oracle.lm_head(w["lm_head"], ht)
    rng = np.random.default_rng(cfg.seed)
    groups = _placements(plan, rng, R)
    # window rows with a clear winner, each with its own winning token, none of them a planted position
    planted_ids = {t for _, g in groups for t in g}
    rows, seen = [], set()
    for r in np.argsort(-base["top2_gap"]):
        a = int(base["argmax"][r])
        if a not in seen and a not in planted_ids:
            rows.append(int(r))
            seen.add(a)
        if len(rows) == len(groups):
            break
    assert len(rows) >= min(len(groups), 6)
    groups = groups[-len(rows):]                        # few window rows: the plan-specific sites come last, keep them
    W0 = w["lm_head"].copy()
    for r, (_, g) in zip(rows, groups):
        # twice the winning row of window row r (bf16 exponent + 1: exact) at every id of the group: the group's
        # logit on row r is twice the old maximum, far above every other logit of that row
        win = W0[int(base["argmax"][r])]
        doubled = np.where((win & 0x7F80) != 0, win + np.uint16(0x0080), win).astype(np.uint16)
        for t in g:
            w["lm_head"][t] = doubled
    case = cases.make_case(cfg, oracle_ref_argmax, weights=w)
    ref = run_oracle(case)
    expect = {}
    for r, (name, g) in zip(rows, groups):
        assert ref["top2_gap"][r] == 0.0 and ref["argmax"][r] == g[0], (name, g, ref["argmax"][r])
        others = np.delete(oracle.lm_head(w["lm_head"], case["target_hidden"][r:r + 1], want_logits=True)["logits"][0], g)
        assert ref["lse"][r] > others.max() + 0.2          # no third logit anywhere near the tied maximum
        expect[r] = (name, g)
    return case, ref, expect, plan


def _assert_planted(argmax, expect, what):
    am = argmax.cpu().numpy() if hasattr(argmax, "cpu") else np.asarray(argmax)
    for r, (name, g) in expect.items():
        assert am[r] == g[0], "%s: tie %s %s on row %d resolved to %d" % (what, name, g, r, am[r])


SHAPES = {"R9_mma64": (1, 8), "R100_mma128": (20, 4), "R200_pair_ranges": (40, 4), "R300_two_teams": (60, 4),
          "R512_two_teams": (64, 7), "R1040_pair_items": (130, 7)}


@pytest.mark.gpu
@pytest.mark.parametrize("shape", list(SHAPES), ids=list(SHAPES))
def test_lowest_token_id_wins_at_every_merge_site(shape):
    B, K = SHAPES[shape]
    cfg = _cfg(B, K)
    case, ref, expect, plan = _planted_case(cfg)
    R = case["R"]
    if shape == "R200_pair_ranges":
        assert plan["lm_pair"] and plan["lm_carry"] and plan["lm_tiles_per_cta"] > 1
    if shape == "R512_two_teams":
        assert plan["lm_pair"] and plan["lm_carry"] and (plan["lm_n_cols"], plan["lm_row_blocks"]) == (256, 2)
    if shape == "R300_two_teams":
        # two row blocks of 160, a team of pairs each, every pair with several tiles in its vocabulary range
        assert plan["lm_pair"] and plan["lm_carry"] and (plan["lm_n_cols"], plan["lm_row_blocks"]) == (160, 2)
        assert plan["lm_tiles_per_cta"] > 1 and plan["lm_parts"] == plan["lm_ctas"] // 2
    if shape == "R1040_pair_items":
        # five row blocks: work items (vocabulary tile of 256, row block) dealt out round-robin, partials per tile
        assert plan["lm_pair"] and not plan["lm_carry"] and plan["lm_row_blocks"] == 5
    if R <= 128:
        assert plan["lm_carry"] and plan["lm_tiles_per_cta"] > 1
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    geo = dict(B=cfg.B, K=cfg.K, T=case["T"])

    # one-call round: automatic plan, then other MMA heights, tile heights, kernels and launch splits
    tunings = [dict(), dict(lm_mma_m=128), dict(lm_single_cta=1), dict(head_ctas=-1), dict(lm_kb_per_stage=1),
               dict(head_ctas=-1, lm_single_cta=1, lm_mma_m=128)]
    if R <= 128:
        # other tile heights (with more rows the partial buffer is sized for the automatic tile and refuses finer ones)
        tunings += [dict(lm_tile_n=64), dict(lm_tile_n=176, lm_stages=3)]
    if R > 256:
        # the other way of dealing out the pair kernel's work: round-robin items instead of teams, and the reverse
        tunings += [dict(lm_teams=-1), dict(lm_teams=1), dict(lm_teams=-1, lm_kb_per_stage=4)]
    for tune in tunings:
        v.set_tuning(**tune)
        out = cases.run(v, d)
        torch.cuda.synchronize()
        assert v.device_error() == 0
        _assert_planted(out.argmax, expect, "wisv_verify %s" % tune)
        compare(case, ref, out, cfg.tau)
    v.set_tuning()

    # first phase of the two-call protocol
    loc = v.localize(d["target_hidden"], d["draft_tokens"], **geo)
    torch.cuda.synchronize()
    _assert_planted(loc.argmax, expect, "wisv_localize")
    assert np.array_equal(loc.argmax.cpu().numpy()[ref["top2_gap"] == 0.0], ref["argmax"][ref["top2_gap"] == 0.0])
    v.close()

    # vocabulary shards: the members of the far-apart groups live in different shards
    for cuts in ([0, 20000, V], [0, 13328, 26672, V], [0, 16, 39984, V]):
        shards = [cases.make_verifier(d, vocab_slice=(lo, hi)) for lo, hi in zip(cuts[:-1], cuts[1:])]
        parts = torch.stack([s.shard_rows(d["target_hidden"], d["draft_tokens"], **geo) for s in shards])
        for order in (parts, parts.flip(0).contiguous()):          # the merge must not depend on the gather order
            out = shards[0].verify_gathered(order, d["target_hidden"], d["draft_tokens"], d["draft_hidden"], d["csi"],
                                            **geo)
            torch.cuda.synchronize()
            _assert_planted(out.argmax, expect, "wisv_verify_gathered %s" % cuts)
            compare(case, ref, out, cfg.tau)
            if order is parts:
                for s in shards:                                       # a second gathered round needs a fresh shard pass
                    s.shard_rows(d["target_hidden"], d["draft_tokens"], **geo)
        assert all(s.device_error() == 0 for s in shards)
        for s in shards:
            s.close()

    # the allocation-free entry point (one row tile only)
    if R <= 128:
        lib = wisv.load_library()
        am = torch.full((R,), -7, dtype=torch.int32, device=DEV)
        lse = torch.zeros(R, dtype=torch.float32, device=DEV)
        st = torch.cuda.current_stream()
        rc = lib.wisv_lm_head_reduce_static(d["lm_head"].data_ptr(), V, H, d["target_hidden"].data_ptr(), R,
                                            am.data_ptr(), lse.data_ptr(), C.c_void_p(st.cuda_stream))
        assert rc == 0
        torch.cuda.synchronize()
        _assert_planted(am, expect, "wisv_lm_head_reduce_static")
        exact = (ref["top2_gap"] == 0.0) | (ref["top2_gap"] >= 1e-2)
        assert np.array_equal(am.cpu().numpy()[exact], ref["argmax"][exact])


def test_owner_map_matches_the_planner():
    """The helper that places the ties must describe the ranges the planner deals out (every token owned once,
    chunks and tiles inside the stated heights).  Host arithmetic only."""
    for R, P in ((9, 8), (100, 80), (200, 160), (300, 240), (512, 448)):
        plan = wisv.plan_host(H=H, V=V, H_d=64, d_c=2, d_J=64, R=R, P=P, sm_count=SM, max_smem_bytes=SMEM)
        own = _owner_fn(plan)
        groups = plan["lm_ctas"] // 2 if plan["lm_pair"] else plan["lm_ctas"]
        if R > 256:
            assert plan["lm_carry"] and plan["lm_row_blocks"] == 2
            groups //= plan["lm_row_blocks"]                  # teams of pairs: ownership inside a team
        seen = {}
        for v in range(0, V, 7):
            c, t, ch, half = own(v)
            assert 0 <= c < groups and 0 <= t < plan["lm_tiles_per_cta"] and 0 <= ch < plan["lm_tile_n"] // 16
            seen.setdefault(c, []).append(v)
        assert len(seen) == groups
        assert all(a == sorted(a) and a[-1] - a[0] < (plan["lm_units_base"] + 1) * (32 if plan["lm_pair"] else 16)
                   for a in seen.values())
