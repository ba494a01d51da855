"""Pins for the CPU oracle: what the paper and the mathematics fix, independent of the oracle.

Second opinions come from torch float64 library routines, closed forms, a
hand-worked fixture, exhaustive enumeration against the set definition of
Algorithm 1, and a pure-Python brute force on a tiny case.
"""
import itertools
import math
import os

import numpy as np
import pytest
import torch

import gen
import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bf16_bits(x):
    """bf16 bit patterns via torch's own conversion (independent of gen and the oracle)."""
    t = torch.as_tensor(np.asarray(x, np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def bf16_round64(x):
    return torch.as_tensor(np.asarray(x, np.float32)).to(torch.bfloat16).to(torch.float64)


def bits_to_f64(bits):
    return torch.as_tensor(np.asarray(bits).view(np.int16)).view(torch.bfloat16).to(torch.float64)


# ----------------------------------------------------------------------------- LM head

@pytest.mark.parametrize("R,H,V,seed", [(5, 72, 1000, 0), (40, 256, 4096, 1), (3, 8, 17, 2), (9, 33, 257, 3)])
def test_lm_head_matches_torch_float64(R, H, V, seed):
    g = np.random.default_rng(seed)
    W = bf16_bits(g.standard_normal((V, H)) * 0.05)
    Ht = g.standard_normal((R, H)).astype(np.float32)
    tok = g.integers(0, V, size=R).astype(np.int32)
    tok[0] = -1
    out = oracle.lm_head(W, Ht, tok, want_logits=True)
    L = bf16_round64(Ht) @ bits_to_f64(W).T
    assert np.allclose(out["logits"], L.numpy(), rtol=0, atol=1e-12)
    assert np.array_equal(out["argmax"], torch.argmax(L, dim=1).numpy())
    assert np.allclose(out["lse"], torch.logsumexp(L, dim=1).numpy(), rtol=0, atol=1e-12)
    top2 = torch.topk(L, 2, dim=1).values
    assert np.allclose(out["top2_gap"], (top2[:, 0] - top2[:, 1]).numpy(), atol=1e-12)
    assert math.isnan(out["tok_logit"][0])
    ref_tok = L[torch.arange(1, R), torch.as_tensor(tok[1:]).long()].numpy()
    assert np.allclose(out["tok_logit"][1:], ref_tok, atol=1e-12)


def test_lm_head_uniform_logits_closed_form():
    # all vocabulary rows identical => every logit equals x: lse = x + ln V, argmax = lowest id
    V, H = 300, 16
    W = np.tile(bf16_bits(np.full((1, H), 0.25)), (V, 1))
    Ht = np.ones((2, H), np.float32)
    Ht[1] *= 2
    out = oracle.lm_head(W, Ht)
    for r, x in enumerate((4.0, 8.0)):
        assert out["argmax"][r] == 0
        assert abs(out["lse"][r] - (x + math.log(V))) < 1e-12
        assert out["top2_gap"][r] == 0.0


def test_lm_head_shift_invariance_and_softmax_sums_to_one():
    g = np.random.default_rng(5)
    V, H = 64, 12
    Wf = g.standard_normal((V, H)) * 0.1
    Wf[:, 0] = 1.0                      # a direction every logit shares
    W = bf16_bits(Wf)
    x = g.standard_normal((1, H)).astype(np.float32)
    x[0, 0] = 0.5
    y = x.copy()
    y[0, 0] = 3.5                       # shifts every logit by exactly 3
    a = oracle.lm_head(W, x, want_logits=True)
    b = oracle.lm_head(W, y)
    assert a["argmax"][0] == b["argmax"][0]
    assert abs((b["lse"][0] - a["lse"][0]) - 3.0) < 1e-12
    assert abs(a["top2_gap"][0] - b["top2_gap"][0]) < 1e-12
    assert abs(np.exp(a["logits"][0] - a["lse"][0]).sum() - 1.0) < 1e-12
    # the draft-token probability exp(L[y] - lse) sums to one over all possible tokens
    tot = 0.0
    for v in range(V):
        o = oracle.lm_head(W, x, np.array([v], np.int32))
        tot += math.exp(o["tok_logit"][0] - o["lse"][0])
    assert abs(tot - 1.0) < 1e-12


def test_lm_head_planted_column_and_tie_break():
    V, H = 50, 8
    Wf = np.zeros((V, H))
    Wf[31, 2] = 4.0
    Wf[7, 2] = 4.0                      # same maximum at a lower index
    Wf[40, 2] = 2.0
    W = bf16_bits(Wf)
    x = np.zeros((1, H), np.float32)
    x[0, 2] = 1.0
    out = oracle.lm_head(W, x)
    assert out["argmax"][0] == 7 and out["top2_gap"][0] == 0.0
    Wf[7, 2] = 0.0
    out = oracle.lm_head(bf16_bits(Wf), x)
    assert out["argmax"][0] == 31 and abs(out["top2_gap"][0] - 2.0) < 1e-12
    # one dominant logit: lse -> max
    Wf[31, 2] = 60.0
    out = oracle.lm_head(bf16_bits(Wf), x)
    assert abs(out["lse"][0] - 60.0) < 1e-12


def test_hidden_states_round_to_nearest_even_bf16():
    # halfway cases: 1+2^-8 -> 1 (even), 1+3*2^-8 -> 1+2^-6 (even), just above half rounds up
    W = bf16_bits(np.array([[1.0]]))
    xs = np.array([[1 + 2.0 ** -8], [1 + 3 * 2.0 ** -8], [1 + 2.0 ** -8 + 2.0 ** -20], [-(1 + 2.0 ** -8)]],
                  np.float32)
    out = oracle.lm_head(W, xs, want_logits=True)
    assert out["logits"][:, 0].tolist() == [1.0, 1 + 2.0 ** -6, 1 + 2.0 ** -7, -1.0]


# ----------------------------------------------------------------------------- decision head

def _load_head_fixture():
    rows = []
    with open(os.path.join(GOLDEN, "head_hand_example.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            act, b2, s, p, rej = line.split()
            rows.append((act, float(b2), float(s), float(p), int(rej)))
    return rows


@pytest.mark.parametrize("row", _load_head_fixture())
def test_head_hand_example(row):
    act, b2, s_ref, p_ref, rej_ref = row
    W1 = bf16_bits(np.array([[1, 0, 2], [-1, 1, 0]], np.float32))
    out = oracle.head(W1, [0.0, 0.5], [0.5, 1.0], b2, H=1, H_d=1, d_c=1,
                      act=oracle.ACT_RELU if act == "relu" else oracle.ACT_GELU,
                      draft_hidden=np.array([[1.0]], np.float32), target_hidden=np.array([[-2.0]], np.float32),
                      csi=np.array([[0.5]], np.float32), tgt_row=[0], req=[0])
    assert abs(out["logit"][0] - s_ref) < 1e-12
    assert abs(out["prob"][0] - p_ref) < 1e-12
    # threshold rule: rejected iff p >= tau, through the scan on a one-token window
    A, _ = oracle.scan([0, 1], [1], [1], out["prob"], 0.5, [11, 22])
    assert (A[0] == 0) == bool(rej_ref)


def test_head_column_order_rounding_and_raw_csi():
    # pre = a*hD + b*hT + c*csi with distinct weights exposes a swapped block
    W1 = bf16_bits(np.array([[1.0, 0.5, 0.25]], np.float32))
    hD = np.array([[1 + 2.0 ** -8]], np.float32)       # rounds to 1.0
    hT = np.array([[3.0], [10.0]], np.float32)
    csi = np.array([[0.0], [0.3]], np.float32)          # 0.3 is not a bf16 value: must stay fp32
    out = oracle.head(W1, [0.0], [1.0], 0.0, H=1, H_d=1, d_c=1, act=oracle.ACT_RELU,
                      draft_hidden=hD, target_hidden=hT, csi=csi, tgt_row=[1], req=[1])
    expect = 1.0 + 0.5 * 10.0 + 0.25 * float(np.float32(0.3))
    assert abs(out["logit"][0] - expect) < 1e-15
    # all-zero first layer: p = sigmoid(b2)
    out = oracle.head(bf16_bits(np.zeros((4, 3))), np.zeros(4), np.ones(4), -0.75, H=1, H_d=1, d_c=1,
                      act=oracle.ACT_GELU, draft_hidden=hD, target_hidden=hT, csi=csi, tgt_row=[0], req=[0])
    assert abs(out["prob"][0] - 1 / (1 + math.exp(0.75))) < 1e-15


@pytest.mark.parametrize("act", ["relu", "gelu"])
def test_head_matches_torch_float64(act):
    g = np.random.default_rng(11)
    H, H_d, d_c, d_J, P, R, B = 40, 24, 2, 16, 9, 12, 3
    W1 = bf16_bits(g.standard_normal((d_J, H_d + H + d_c)) * 0.2)
    b1 = g.standard_normal(d_J).astype(np.float32)
    w2 = g.standard_normal(d_J).astype(np.float32)
    hD = g.standard_normal((P, H_d)).astype(np.float32)
    hT = g.standard_normal((R, H)).astype(np.float32)
    csi = (g.random((B, d_c)) * 30).astype(np.float32)
    tgt = g.integers(0, R, size=P).astype(np.int32)
    req = g.integers(0, B, size=P).astype(np.int32)
    out = oracle.head(W1, b1, w2, 0.3, H, H_d, d_c, oracle.ACT_RELU if act == "relu" else oracle.ACT_GELU,
                      hD, hT, csi, tgt, req)
    z = torch.cat([bf16_round64(hD), bf16_round64(hT)[torch.as_tensor(tgt).long()],
                   torch.as_tensor(csi).double()[torch.as_tensor(req).long()]], dim=1)
    pre = z @ bits_to_f64(W1).T + torch.as_tensor(b1).double()
    a = torch.relu(pre) if act == "relu" else torch.nn.functional.gelu(pre)
    s = a @ torch.as_tensor(w2).double() + 0.3
    assert np.allclose(out["logit"], s.numpy(), atol=1e-12)
    assert np.allclose(out["prob"], torch.sigmoid(s).numpy(), atol=1e-13)


# ----------------------------------------------------------------------------- scan / emission

def _set_definition(K, cand, has, rej_head):
    """Algorithm 1: j = min{i in S : rejected}, S = candidate positions; A = j or K."""
    S = [i for i in range(K) if cand[i] and (not has[i] or rej_head[i])]
    return min(S) if S else K


@pytest.mark.parametrize("K", [1, 2, 3, 4])
def test_scan_exhaustive_against_set_definition(K):
    tau = 0.5
    argmax = np.arange(100, 100 + K + 1, dtype=np.int32)
    for cand in itertools.product([0, 1], repeat=K):
        for has in itertools.product([0, 1], repeat=K):
            for rej in itertools.product([0, 1], repeat=K):
                prob = [0.9 if r else 0.1 for r in rej]
                A, corr = oracle.scan([0, K], cand, has, prob, tau, argmax)
                ref = _set_definition(K, cand, has, rej)
                assert A[0] == ref and 0 <= A[0] <= K
                assert corr[0] == argmax[ref]


def test_scan_threshold_is_inclusive_and_multi_request_offsets():
    # p == tau rejects (Eq. 27); requests index their own rows (K_b + 1 rows each)
    k_off = [0, 2, 2, 5]            # K = 2, 0, 3
    cand = [0, 1, 1, 0, 1]
    has = [1, 1, 1, 1, 1]
    prob = [0.99, 0.5, 0.49, 0.99, 0.5]
    argmax = np.arange(10, 10 + 5 + 3, dtype=np.int32)   # rows: b0 -> 10..12, b1 -> 13, b2 -> 14..17
    A, corr = oracle.scan(k_off, cand, has, prob, 0.5, argmax)
    assert A.tolist() == [1, 0, 2]
    assert corr.tolist() == [11, 13, 16]


def _tiny_case(seed=0, B=6, K=5, V=97, H=24, H_d=16, d_J=8, match=0.5):
    cfg = gen.VerifyConfig("t", B=B, K=K, H=H, H_d=H_d, d_c=2, d_J=d_J, V=V, match_rate=match, seed=seed)
    k = gen.synth.window_lengths(cfg)
    w = gen.make_weights(cfg)
    h = gen.make_hidden(cfg, k)
    ref = oracle.lm_head(w["lm_head"], h["target_hidden"])["argmax"]
    toks = gen.make_draft_tokens(cfg, k, ref)
    args = dict(lm_head_bits=w["lm_head"], W1_bits=w["W1"], b1=w["b1"], w2=w["w2"], b2=w["b2"],
                act=oracle.ACT_GELU, tau=0.5, k_len=k, target_hidden=h["target_hidden"],
                draft_tokens=toks, draft_hidden=h["draft_hidden"], csi=h["csi"])
    return cfg, k, ref, args


def test_verify_invariants_of_algorithm_1():
    cfg, k, ref, args = _tiny_case()
    out = oracle.verify(**args)
    A = out["accept_len"]
    row_off = out["row_off"]
    mism = args["draft_tokens"] != ref[out["row_of_t"]]
    assert np.array_equal(out["cand"], mism)
    first_mismatch = np.array([next((i for i in range(k[b]) if mism[out["k_off"][b] + i]), k[b])
                               for b in range(cfg.B)])
    assert np.all(A >= 0) and np.all(A <= k)
    assert np.all(A >= first_mismatch)                       # the head can only extend the span
    assert np.array_equal(out["correction_token"], ref[row_off[:-1] + A])
    # tau = 0: plain greedy speculative decoding; tau > 1: everything accepted (Section VI-B)
    g0 = oracle.verify(**{**args, "tau": 0.0})
    assert np.array_equal(g0["accept_len"], first_mismatch)
    g2 = oracle.verify(**{**args, "tau": 1.5})
    assert np.array_equal(g2["accept_len"], k)
    assert np.array_equal(g2["correction_token"], ref[row_off[1:] - 1])   # the bonus row
    # accepted length is monotone in tau
    prev = g0["accept_len"]
    for tau in (0.2, 0.4, 0.5, 0.6, 0.8, 1.01):
        cur = oracle.verify(**{**args, "tau": tau})["accept_len"]
        assert np.all(cur >= prev)
        prev = cur
    # a full-match window accepts K and emits the bonus token
    full = dict(args)
    full["draft_tokens"] = ref[out["row_of_t"]].astype(np.int32)
    fo = oracle.verify(**full)
    assert np.array_equal(fo["accept_len"], k) and fo["n_mismatch"].sum() == 0
    # a rejection at position i forces accept length i
    for b in range(cfg.B):
        if A[b] < k[b]:
            t = out["k_off"][b] + A[b]
            assert out["cand"][t] and out["prob_t"][t] >= 0.5
            assert not np.any(out["cand"][out["k_off"][b]:t] & (out["prob_t"][out["k_off"][b]:t] >= 0.5))


def test_full_hidden_equals_selective_hidden_and_matched_positions_are_ignored():
    cfg, k, ref, args = _tiny_case(seed=3)
    fh = oracle.verify(**args)
    packed, sel_off, sel_pos = gen.pack_selective(args["draft_hidden"], k, fh["cand"])
    sh = oracle.verify(**{**args, "draft_hidden": packed, "sel_off": sel_off, "sel_pos": sel_pos})
    assert np.array_equal(fh["accept_len"], sh["accept_len"])
    assert np.array_equal(fh["correction_token"], sh["correction_token"])
    assert np.allclose(sh["head_prob"], fh["head_prob"][fh["cand"]], atol=0)
    # the head is consulted only on S: hidden states at matched positions cannot matter
    scr = dict(args)
    hd = args["draft_hidden"].copy()
    hd[~fh["cand"]] = 123.0
    scr["draft_hidden"] = hd
    out = oracle.verify(**scr)
    assert np.array_equal(out["accept_len"], fh["accept_len"])
    # a mismatch whose hidden state was not uploaded is rejected (greedy fallback)
    none = oracle.verify(**{**args, "draft_hidden": packed[:0], "sel_off": np.zeros(cfg.B + 1, np.int32),
                            "sel_pos": np.zeros(0, np.int32)})
    g0 = oracle.verify(**{**args, "tau": 0.0})
    assert np.array_equal(none["accept_len"], g0["accept_len"])


def test_head_row_shift_uses_next_target_row():
    cfg, k, ref, args = _tiny_case(seed=4)
    a = oracle.verify(**args, head_row_shift=1)
    ht = args["target_hidden"]
    b = oracle.verify(**args)                                  # shift 0 on the same rows
    assert not np.allclose(a["head_prob"], b["head_prob"])
    # shift=1 on H equals shift=0 evaluated with the rows moved up by one (head only)
    tgt = a["row_of_t"] + 1
    direct = oracle.head(args["W1_bits"], args["b1"], args["w2"], args["b2"], cfg.H, cfg.H_d, cfg.d_c,
                         oracle.ACT_GELU, args["draft_hidden"], ht, args["csi"], tgt, a["req_of_t"])
    assert np.array_equal(a["head_prob"], direct["prob"])


def test_stochastic_acceptance_special_cases():
    cfg, k, ref, args = _tiny_case(seed=5)
    base = oracle.verify(**args)
    T = int(k.sum())
    u = np.random.default_rng(0).random(T).astype(np.float32)
    # q = p_T(y): alpha = 1, every token accepted whatever u in [0,1)
    o = oracle.verify(**{**args, "tau": 0.0, "draft_q": base["p_draft"], "uniforms": u})
    assert np.array_equal(o["accept_len"], k) and np.all(o["alpha"] == 1.0)
    # u = 0: accepted whenever p_T(y) > 0
    o = oracle.verify(**{**args, "tau": 0.0, "draft_q": np.ones(T), "uniforms": np.zeros(T)})
    assert np.array_equal(o["accept_len"], k)
    # q huge: alpha -> 0, rejected at the first position under tau = 0
    o = oracle.verify(**{**args, "tau": 0.0, "draft_q": np.full(T, 1e30), "uniforms": np.full(T, 0.5)})
    assert np.all(o["accept_len"] == 0)
    # alpha is min(1, p/q) and the test is strict u < alpha
    q = (base["p_draft"] * 2).astype(np.float64)
    o = oracle.verify(**{**args, "tau": 0.0, "draft_q": q, "uniforms": np.full(T, 0.5)})
    assert np.allclose(o["alpha"], 0.5) and np.all(o["cand"])


# ----------------------------------------------------------------------------- brute force

def _py_bf16(x):
    return float(torch.tensor(float(x), dtype=torch.float32).to(torch.bfloat16))


def test_whole_round_against_pure_python_brute_force():
    cfg, k, ref, args = _tiny_case(seed=9, B=3, K=3, V=13, H=6, H_d=4, d_J=3)
    out = oracle.verify(**{**args, "act": oracle.ACT_RELU})
    W = gen.bf16_bits_to_f32(args["lm_head_bits"]).astype(np.float64)
    W1 = gen.bf16_bits_to_f32(args["W1_bits"]).astype(np.float64)
    ht, hd, csi = args["target_hidden"], args["draft_hidden"], args["csi"]
    row = 0
    t = 0
    for b in range(cfg.B):
        amax = []
        for i in range(k[b] + 1):
            x = [_py_bf16(v) for v in ht[row + i]]
            L = [sum(x[h] * W[v, h] for h in range(cfg.H)) for v in range(cfg.V)]
            amax.append(max(range(cfg.V), key=lambda v: (L[v], -v)))
            lse = math.log(sum(math.exp(l) for l in L))
            assert abs(out["lse"][row + i] - lse) < 1e-12
            if i < k[b]:
                assert abs(out["p_draft"][t + i] - math.exp(L[args["draft_tokens"][t + i]] - lse)) < 1e-12
        A = k[b]
        for i in range(k[b]):
            if args["draft_tokens"][t + i] == amax[i]:
                continue
            z = [_py_bf16(v) for v in hd[t + i]] + [_py_bf16(v) for v in ht[row + i]] + [float(c) for c in csi[b]]
            s = float(args["b2"])
            for j in range(cfg.d_J):
                pre = sum(W1[j, kk] * z[kk] for kk in range(cfg.d_in)) + float(args["b1"][j])
                s += float(args["w2"][j]) * max(pre, 0.0)
            if 1 / (1 + math.exp(-s)) >= 0.5:
                A = i
                break
        assert out["accept_len"][b] == A
        assert out["correction_token"][b] == amax[A]
        row += k[b] + 1
        t += k[b]


def test_candidate_counts_with_empty_windows():
    cfg = gen.VerifyConfig("e", B=5, K=0, K_lo=0, K_hi=2, H=24, H_d=16, d_c=2, d_J=8, V=97, match_rate=0.0, seed=2)
    k = np.array([2, 0, 1, 0, 0], np.int32)
    w = gen.make_weights(cfg)
    h = gen.make_hidden(cfg, k)
    ref = oracle.lm_head(w["lm_head"], h["target_hidden"])["argmax"]
    toks = (ref[[0, 1, 4]] + 1) % cfg.V                         # every draft token mismatches
    out = oracle.verify(lm_head_bits=w["lm_head"], W1_bits=w["W1"], b1=w["b1"], w2=w["w2"], b2=w["b2"],
                        act=oracle.ACT_RELU, tau=0.0, k_len=k, target_hidden=h["target_hidden"],
                        draft_tokens=toks.astype(np.int32), draft_hidden=h["draft_hidden"], csi=h["csi"])
    assert out["n_mismatch"].tolist() == [2, 0, 1, 0, 0]
    assert out["accept_len"].tolist() == [0, 0, 0, 0, 0]
    assert np.array_equal(out["correction_token"], ref[[0, 3, 4, 6, 7]])     # first row of every window


# ----------------------------------------------------------------------------- 16-bit hidden states (Section IV-A, b_h = 16)

def test_sixteen_bit_hidden_states_follow_the_same_rounding_rule():
    """fp16 uploads are widened exactly and then rounded to bf16 (nearest even) like fp32 inputs; bf16 uploads are used
    as they are.  Second opinion: torch's own fp16 -> bf16 conversion and a float64 matmul."""
    import torch
    g = np.random.default_rng(12)
    V, H, R = 64, 48, 6
    W = gen.f32_to_bf16_bits(g.standard_normal((V, H), dtype=np.float32) * 0.1)
    x16 = g.standard_normal((R, H)).astype(np.float16)
    # halfway cases of the fp16 -> bf16 rounding: low three mantissa bits 100, kept bit even and odd
    bits = x16.view(np.uint16).copy()
    bits[0, :8] = (bits[0, :8] & np.uint16(0xFFF0)) | np.uint16(0x0004)       # kept bit 0: rounds down
    bits[0, 8:16] = (bits[0, 8:16] & np.uint16(0xFFF0)) | np.uint16(0x000C)   # kept bit 1: rounds up
    x16 = bits.view(np.float16)
    got = oracle.lm_head(W, oracle.hidden_as_f32(x16), want_logits=True)["logits"]
    xt = torch.from_numpy(x16.copy()).to(torch.bfloat16).to(torch.float64)       # library conversion, nearest even
    Wt = torch.from_numpy(gen.bf16_bits_to_f32(W)).to(torch.float64)
    assert np.allclose(got, (xt @ Wt.T).numpy(), rtol=0, atol=1e-12)
    # the two halfway groups really round in different directions
    r = xt[0].numpy()
    lo = x16[0].astype(np.float64)
    assert np.all(np.abs(r[:8]) < np.abs(lo[:8])) and np.all(np.abs(r[8:16]) > np.abs(lo[8:16]))
    # bf16 bit patterns are taken as they are
    xb = gen.f32_to_bf16_bits(g.standard_normal((R, H), dtype=np.float32))
    a = oracle.lm_head(W, oracle.hidden_as_f32(xb), want_logits=True)["logits"]
    b = oracle.lm_head(W, gen.bf16_bits_to_f32(xb), want_logits=True)["logits"]
    assert np.array_equal(a, b)
    assert np.allclose(a, (torch.from_numpy(gen.bf16_bits_to_f32(xb)).to(torch.float64) @ Wt.T).numpy(), rtol=0, atol=1e-12)


def test_round_with_sixteen_bit_uploads_equals_round_on_their_fp32_values():
    cfg = gen.VerifyConfig("h16", B=5, K=4, H=64, H_d=32, d_c=2, d_J=32, V=300, match_rate=0.5, seed=77)
    k_len = gen.synth.window_lengths(cfg)
    w = gen.make_weights(cfg)
    h = gen.make_hidden(cfg, k_len)
    ref_am = oracle.lm_head(w["lm_head"], h["target_hidden"])["argmax"]
    toks = gen.make_draft_tokens(cfg, k_len, ref_am)
    kw = dict(lm_head_bits=w["lm_head"], W1_bits=w["W1"], b1=w["b1"], w2=w["w2"], b2=float(w["b2"]), act=oracle.ACT_GELU,
              tau=0.5, k_len=k_len, draft_tokens=toks, csi=h["csi"])
    hd16 = h["draft_hidden"].astype(np.float16)
    ht_bits = gen.f32_to_bf16_bits(h["target_hidden"])
    a = oracle.verify(target_hidden=ht_bits, draft_hidden=hd16, **kw)
    b = oracle.verify(target_hidden=gen.bf16_bits_to_f32(ht_bits), draft_hidden=hd16.astype(np.float32), **kw)
    for k in ("accept_len", "correction_token", "argmax", "lse", "head_prob", "p_draft"):
        assert np.array_equal(a[k], b[k]), k
    # and the fp16 upload is a different input from the fp32 original: the head sees the rounded values
    c = oracle.verify(target_hidden=gen.bf16_bits_to_f32(ht_bits), draft_hidden=h["draft_hidden"], **kw)
    assert np.max(np.abs(c["head_logit"] - a["head_logit"])) > 0
