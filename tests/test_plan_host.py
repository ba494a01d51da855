"""The launch planner as host arithmetic (wisv_plan_host): invariants that must hold for every batch shape,
vocabulary size and device size, checked without a GPU."""
import itertools

import pytest

from paper_2604_17701_b200 import plan_host

DIMS_8B = dict(H=4096, V=128256, H_d=2048, d_c=2, d_J=1024)
SMEM = 232448


def _ranges(units_total, ctas, base, rem):
    """Units owned by each CTA (or pair) of a carried plan."""
    assert ctas * base + rem == units_total and 0 <= rem < max(ctas, 1)
    return [base + (1 if c < rem else 0) for c in range(ctas)]


def _check_carry(tile_n, tiles_per_cta, owned, unit):
    assert tile_n % unit == 0 and unit <= tile_n <= 256
    for u in owned:
        assert u >= 1                                        # no CTA is launched without work
        k = tiles_per_cta
        heights = [(u // k + (1 if i < u % k else 0)) * unit for i in range(k)]
        assert sum(heights) == u * unit                      # the tiles cover the range exactly once
        assert all(h in (0, tile_n - unit, tile_n) for h in heights)   # two tile heights (0: fewer units than tiles)
        assert max(heights) <= tile_n


@pytest.mark.parametrize("V", [17, 100, 1000, 4099, 32000, 128256, 152064, 262144])
@pytest.mark.parametrize("sm_count", [8, 132, 148, 160])
def test_carried_ranges_cover_the_vocabulary_exactly_once(V, sm_count):
    for R, P in ((1, 0), (9, 8), (64, 60), (65, 64), (128, 127), (129, 0), (129, 120), (200, 190), (256, 255)):
        p = plan_host(H=256, V=V, H_d=128, d_c=2, d_J=128, R=R, P=P, sm_count=sm_count, max_smem_bytes=SMEM)
        assert p["lm_carry"] == 1                            # up to 256 rows: always contiguous ranges
        unit = 32 if p["lm_pair"] else 16
        units_total = -(-V // unit)
        groups = p["lm_ctas"] // 2 if p["lm_pair"] else p["lm_ctas"]
        owned = _ranges(units_total, groups, p["lm_units_base"], p["lm_units_rem"])
        _check_carry(p["lm_tile_n"], p["lm_tiles_per_cta"], owned, unit)
        assert max(owned) - min(owned) <= 1                  # balanced to one unit
        assert p["lm_smem_bytes"] <= SMEM and p["lm_stages"] >= 2
        head_ctas = p["head_ctas"] if p["head_in_lm_launch"] else 0
        assert p["lm_ctas"] + head_ctas + (head_ctas % 2 if p["lm_pair"] else 0) <= sm_count
        assert p["kernels"] == (3 if (P == 0 or p["head_in_lm_launch"]) else 4)
        if P > 0:
            assert p["head_in_lm_launch"] == 1               # small batches never pay for a head launch
            assert p["head_smem_bytes"] <= SMEM
            if p["head_carry"]:
                owned_h = _ranges(-(-128 // 16), p["head_ctas"], p["head_units_base"], p["head_units_rem"])
                _check_carry(p["head_tile_n"], p["head_tiles_per_cta"], owned_h, 16)


def test_plans_at_the_task_shapes():
    p = plan_host(R=9, P=8, **DIMS_8B)                       # B=1, K=8
    assert (p["kernels"], p["lm_pair"], p["lm_carry"], p["lm_ctas"], p["head_ctas"]) == (3, 0, 1, 142, 6)
    assert p["lm_tile_n"] == 240 and p["lm_tiles_per_cta"] == 4 and p["lm_units_base"] == 56
    p = plan_host(R=144, P=128, **DIMS_8B)                   # B=16: pairs with head clusters
    assert (p["kernels"], p["lm_pair"], p["lm_carry"], p["lm_ctas"], p["head_ctas"]) == (3, 1, 1, 142, 6)
    assert (p["lm_n_cols"], p["lm_row_blocks"], p["lm_parts"]) == (144, 1, 142)     # the MMA's N is the row count up to 16
    p = plan_host(R=288, P=256, **DIMS_8B)                   # B=32: two row blocks of 144, nothing padded; two teams
    assert (p["kernels"], p["lm_pair"], p["lm_carry"], p["lm_n_cols"], p["lm_row_blocks"]) == (3, 1, 1, 144, 2)
    assert (p["lm_ctas"], p["lm_parts"], p["lm_rounds"], p["head_ctas"]) == (144, 72, 14, 2)   # of 36 pairs
    p = plan_host(R=576, P=512, **DIMS_8B)                   # B=64: three row blocks of 192; three teams of 24 pairs,
    assert (p["kernels"], p["lm_pair"], p["lm_carry"], p["lm_ctas"], p["lm_rounds"]) == (3, 1, 1, 144, 21)   # 21 tiles each
    assert (p["lm_n_cols"], p["lm_row_blocks"], p["lm_parts"], p["head_ctas"]) == (192, 3, 48, 4)
    assert (p["lm_units_base"], p["lm_units_rem"], p["lm_tiles_per_cta"]) == (167, 0, 21)     # 4008 units of 32 rows / 24
    p = plan_host(R=1100, P=1000, **DIMS_8B)                 # five row blocks: 14 pairs per team would need 36 tiles
    assert (p["lm_carry"], p["lm_row_blocks"], p["lm_parts"], p["lm_rounds"]) == (0, 5, 1002, 34)   # against 34 rounds
    p = plan_host(R=8704, P=8192, **DIMS_8B)                 # B=512, K=16: 74 pairs, 230.2 rounds of 256 x 256 items
    assert (p["kernels"], p["lm_pair"], p["lm_ctas"], p["lm_rounds"]) == (4, 1, 148, 231)
    assert (p["lm_n_cols"], p["lm_row_blocks"]) == (256, 34)


@pytest.mark.parametrize("R", [257, 288, 384, 385, 432, 504, 576, 640, 864, 1017, 1152, 1408, 2816, 8704])
def test_head_rides_along_only_when_the_lm_head_needs_no_extra_round(R):
    for P in (R - R // 9, max(1, R // 3)):
        p = plan_host(R=R, P=P, **DIMS_8B)
        groups = p["lm_ctas"] // 2 if p["lm_pair"] else p["lm_ctas"]
        if p["lm_carry"]:
            # teams of pairs, one per row block: a round is one tile of a pair's own vocabulary range, and the plan
            # is taken only when that is no more than round-robin items would need
            assert p["lm_row_blocks"] in (2, 3, 4) and groups % p["lm_row_blocks"] == 0
            assert p["lm_rounds"] == p["lm_tiles_per_cta"]
            assert p["lm_rounds"] <= -(-(p["lm_row_blocks"] * -(-128256 // 256)) // groups)
            team = groups // p["lm_row_blocks"]
            assert p["lm_parts"] == 2 * team
            assert team * p["lm_units_base"] + p["lm_units_rem"] == -(-128256 // 32)
        else:
            assert p["lm_rounds"] == -(-(p["lm_m_tiles"] * p["lm_n_tiles"]) // groups)
        if p["head_in_lm_launch"]:
            assert p["kernels"] == 3 and p["lm_rounds"] == p["lm_rounds_alone"]
            assert p["lm_ctas"] + p["head_ctas"] + (p["head_ctas"] % 2 if p["lm_pair"] else 0) <= 148
            head_rounds = -(-(p["head_m_tiles"] * p["head_n_tiles"]) // p["head_ctas"])
            assert head_rounds * 12 <= p["lm_rounds"] * 8     # the head finishes well inside the LM head's time
        else:
            assert p["kernels"] == 4 and p["lm_ctas"] == 148
        assert p["lm_smem_bytes"] <= SMEM and p["head_smem_bytes"] <= SMEM


def test_row_blocks_of_the_pair_kernel_pad_at_most_fifteen_rows_each():
    for R in (129, 144, 200, 256, 257, 288, 384, 385, 576, 600, 1017, 1280, 2816, 8704):
        p = plan_host(R=R, P=0, **DIMS_8B)
        assert p["lm_pair"] == 1
        nb, n = p["lm_row_blocks"], p["lm_n_cols"]
        assert nb == -(-R // 256) and n % 16 == 0 and 16 <= n <= 256
        assert nb * n >= R and nb * (n - 16) < R              # the narrowest width that covers the rows
        assert nb * n <= -(-R // 256) * 256                   # the blocks stay inside the rows the workspace holds
        assert p["lm_carry"] == (1 if nb <= 4 else 0)         # one team of pairs per row block up to four blocks
        assert p["lm_parts"] == (p["lm_ctas"] // nb if nb <= 4 else 2 * p["lm_n_tiles"])
    assert plan_host(R=128, P=0, **DIMS_8B)["lm_pair"] == 0


def test_decision_head_in_a_launch_of_its_own():
    # one row tile of positions: K split over about one work item per SM
    p = plan_host(R=8 * 9, P=64, **{**DIMS_8B, "V": 128256}, sm_count=148)
    assert p["head_in_lm_launch"] == 1                        # (small batches ride along; no split there)
    assert p["head_k_splits"] == 1
    # four row tiles of positions beside an LM head that cannot spare SMs: 64 column tiles of 64, K split in two,
    # 128 work items for 148 SMs
    p = plan_host(R=1100, P=512, **DIMS_8B)
    assert (p["head_in_lm_launch"], p["head_tile_n"], p["head_m_tiles"], p["head_n_tiles"]) == (0, 64, 4, 16)
    assert p["head_k_splits"] == 2 and p["head_kb_per_split"] == 48 and p["head_ctas"] == 128
    assert p["head_k_splits"] * p["head_kb_per_split"] >= 96  # the splits cover all 96 K blocks
    # six row tiles: no split; one round of 96 items 64 columns wide (a round of narrower tiles is shorter)
    p = plan_host(R=1100, P=768, **DIMS_8B)
    assert (p["head_in_lm_launch"], p["head_k_splits"], p["head_tile_n"]) == (0, 1, 64)
    assert p["head_m_tiles"] * p["head_n_tiles"] == 96
    # thirteen row tiles: 64-wide items would need two rounds, 128-wide ones fit in one
    p = plan_host(R=1800, P=1600, **DIMS_8B)
    assert (p["head_in_lm_launch"], p["head_k_splits"], p["head_tile_n"]) == (0, 1, 128)
    assert p["head_m_tiles"] * p["head_n_tiles"] == 104
    # twenty row tiles: one round of 256-wide items rather than two of 128-wide ones
    p = plan_host(R=2880, P=2560, **DIMS_8B)
    assert (p["head_k_splits"], p["head_tile_n"], p["head_m_tiles"] * p["head_n_tiles"]) == (1, 256, 80)
    # many row tiles: the widest tiles
    p = plan_host(R=8704, P=8192, **DIMS_8B)
    assert (p["head_k_splits"], p["head_tile_n"]) == (1, 256)


def test_bad_arguments_are_refused():
    from paper_2604_17701_b200 import WisvError
    for kw in (dict(R=0, P=0), dict(R=4, P=-1), dict(R=4, P=2, sm_count=1), dict(R=4, P=2, max_smem_bytes=1024)):
        with pytest.raises(WisvError):
            plan_host(**{**DIMS_8B, **kw})
