"""Host-side link model (Section IV-A) of the library against its oracle and a hand-worked fixture."""
import os

import numpy as np
import pytest

import paper_2604_17701_b200 as wisv
from oracle import link_model
from paper_2604_17701_b200 import build

GOLDEN = os.path.join(os.path.dirname(__file__), "golden", "link_hand_example.txt")
HAND = dict(V=128256, K_r=8, m_r=3, d_h=2048, b_h=16, b_pos=6, B_hdr_u=256.0, B_hdr_d=128.0,
            R_u=20e6, R_d=100e6, PER_u=0.1, PER_d=0.05, tau_RTT=0.05)


def _golden():
    vals = {}
    for line in open(GOLDEN):
        if line.startswith("#") or not line.strip():
            continue
        k, v = line.split()
        vals[k] = float(v)
    return vals


def _lib_cost(p):
    build.build()
    link = wisv.LinkParams(p["R_u"], p["R_d"], p["PER_u"], p["PER_d"], p["tau_RTT"], p["B_hdr_u"], p["B_hdr_d"],
                           p["d_h"], p["b_h"], p["b_pos"])
    return wisv.link_cost_round(link, p["V"], p["K_r"], p["m_r"])


def test_oracle_matches_hand_example():
    out = link_model.round_cost(**HAND)
    for k, v in _golden().items():
        assert abs(out[k] - v) <= 1e-15 * max(1.0, abs(v)), k


def test_library_matches_hand_example_and_oracle():
    out = _lib_cost(HAND)
    for k, v in _golden().items():
        assert abs(out[k] - v) <= 1e-15 * max(1.0, abs(v)), k
    g = np.random.default_rng(0)
    for _ in range(200):
        K = int(g.integers(0, 65))
        p = dict(V=int(g.integers(2, 300000)), K_r=K, m_r=int(g.integers(0, K + 1)), d_h=int(g.integers(0, 8192)),
                 b_h=int(g.choice([8, 16, 32])), b_pos=int(g.integers(0, 16)), B_hdr_u=float(g.integers(0, 1024)),
                 B_hdr_d=float(g.integers(0, 1024)), R_u=float(g.uniform(1e6, 1e9)), R_d=float(g.uniform(1e6, 1e9)),
                 PER_u=float(g.uniform(0, 0.5)), PER_d=float(g.uniform(0, 0.5)), tau_RTT=float(g.uniform(0, 0.2)))
        a, b = _lib_cost(p), link_model.round_cost(**p)
        for k in b:
            assert abs(a[k] - b[k]) <= 1e-12 * max(1.0, abs(b[k])), (k, p)


def test_selective_upload_saves_uplink_bits_and_costs_a_round_trip():
    fh = _lib_cost(dict(HAND, m_r=8))
    sh = _lib_cost(HAND)
    assert sh["B_u1_SH"] + sh["B_u2_SH"] < fh["B_u_FH"]                  # m_r < K_r: fewer hidden vectors uploaded
    assert fh["B_u_FH"] - (sh["B_u1_SH"] + sh["B_u2_SH"]) == (8 - 3) * 32768 - 256
    zero = _lib_cost(dict(HAND, R_u=1e15, R_d=1e15))
    assert abs(zero["T_comm_SH"] - zero["T_comm_FH"] - HAND["tau_RTT"]) < 1e-9   # SH pays one more RTT


def test_protocol_rule_and_argument_errors():
    assert wisv.choose_protocol(0.050) == wisv.MODE_FH and wisv.choose_protocol(0.002) == wisv.MODE_SH
    assert wisv.choose_protocol(0.010) == wisv.MODE_SH
    with pytest.raises(wisv.WisvError):
        _lib_cost(dict(HAND, m_r=9))                                     # m_r > K_r
    with pytest.raises(wisv.WisvError):
        _lib_cost(dict(HAND, PER_u=1.0))
