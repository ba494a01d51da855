"""The allocation-free LM-head entry point against the regular one and against the oracle.

Some callers of this library cannot allocate device memory (their host framework
has reserved the whole GPU, or they run in a loop that must not enter the CUDA
allocator), so they cannot create a verifier context.  wisv_lm_head_reduce_static
serves them from a fixed scratch array inside the library.  These tests call it
through the C ABI: twice in a row on different inputs against wisv_verify's
argmax and log-sum-exp on the same rows; at each of its stated limits (128 rows,
hidden size 8192, vocabulary 262144 - which fills the whole partial area) against
the CPU oracle, each followed by a small call that must not see what the large
one left behind; and with the scratch array filled with NaN beforehand.  The file
is collected last so that a run that stops at the first failure has already run
every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import gen
import oracle
import paper_2604_17701_b200 as wisv
from gen import cases
from parity import GAP_TIE, LSE_TOL, oracle_ref_argmax

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _reference_rows(cfg):
    case = cases.make_case(cfg, oracle_ref_argmax)
    d = cases.to_device(case, DEV)
    v = cases.make_verifier(d)
    out = cases.run(v, d)
    torch.cuda.synchronize()
    res = (d, out.argmax.clone(), out.lse.clone())
    v.close()
    return res


def _static_call(lm_head, hidden, am, lse):
    lib = wisv.load_library()
    V, H = lm_head.shape
    st = torch.cuda.current_stream()
    return lib.wisv_lm_head_reduce_static(lm_head.data_ptr(), V, H, hidden.data_ptr(), hidden.shape[0],
                                          am.data_ptr(), lse.data_ptr(), C.c_void_p(st.cuda_stream))


def test_static_entry_point_matches_verify_on_two_calls_in_a_row():
    # two different batches: the second has fewer rows, a vocabulary tail and other data,
    # so anything left in the shared scratch by the first call would show
    cfgs = [gen.VerifyConfig("a", B=20, K=5, H=256, H_d=128, d_c=2, d_J=128, V=4096, match_rate=0.5, seed=21),
            gen.VerifyConfig("b", B=3, K=4, H=320, H_d=128, d_c=2, d_J=128, V=1000, match_rate=0.5, seed=22)]
    refs = [_reference_rows(c) for c in cfgs]
    # outputs are allocated up front; the calls themselves allocate nothing
    outs = [(torch.full((r[1].shape[0],), -7, dtype=torch.int32, device=DEV),
             torch.zeros(r[1].shape[0], dtype=torch.float32, device=DEV)) for r in refs]
    for (d, _, _), (am, lse) in zip(refs, outs):
        assert _static_call(d["lm_head"], d["target_hidden"], am, lse) == 0
    torch.cuda.synchronize()
    for (d, ref_am, ref_lse), (am, lse) in zip(refs, outs):
        assert torch.equal(am, ref_am)
        assert float((lse - ref_lse).abs().max()) <= LSE_TOL


def _against_oracle(W_bits, hidden, am, lse):
    """argmax exact outside near-ties (and a valid leading index inside them), log-sum-exp within tolerance."""
    ref = oracle.lm_head(W_bits, hidden)
    am, lse = am.cpu().numpy(), lse.cpu().numpy()
    assert np.max(np.abs(lse - ref["lse"])) <= LSE_TOL
    differs = am != ref["argmax"]
    assert not (differs & (ref["top2_gap"] >= GAP_TIE)).any()
    near = np.nonzero(differs)[0]
    if near.size:
        assert np.all((am[near] >= 0) & (am[near] < W_bits.shape[0]))
        at = oracle.lm_head(W_bits, hidden[near], row_token=am[near].astype(np.int32))["tok_logit"]
        top = oracle.lm_head(W_bits, hidden[near], row_token=ref["argmax"][near])["tok_logit"]
        assert np.all(top - at < GAP_TIE)


def _weights_bits(V, H, seed):
    cfg = gen.VerifyConfig("w", B=1, K=1, H=H, H_d=8, d_c=0, d_J=16, V=V, match_rate=0.0, seed=seed)
    return gen.make_weights(cfg)["lm_head"]


@pytest.mark.parametrize("V,H,R", [(4096, 256, 128),        # the row limit: every lane of the row tile is a real row
                                   (1000, 8192, 24),        # the hidden-size limit: the whole bf16 row area
                                   (262144, 64, 16)],       # the vocabulary limit: 1024 tiles, the whole partial area
                         ids=["R128", "H8192", "V262144"])
def test_static_entry_point_at_its_limits_against_the_oracle(V, H, R):
    W_bits = _weights_bits(V, H, seed=300 + R)
    hid = np.random.default_rng(R).standard_normal((R, H), dtype=np.float32)
    W = torch.from_numpy(W_bits.view(np.int16)).view(torch.bfloat16).to(DEV)
    X = torch.from_numpy(hid).to(DEV)
    am = torch.full((R,), -7, dtype=torch.int32, device=DEV)
    lse = torch.zeros(R, dtype=torch.float32, device=DEV)
    # a small call on other data right behind the large one: nothing of the large call may linger
    Ws_bits = _weights_bits(700, 64, seed=400 + R)
    hs = np.random.default_rng(1000 + R).standard_normal((5, 64), dtype=np.float32)
    Ws = torch.from_numpy(Ws_bits.view(np.int16)).view(torch.bfloat16).to(DEV)
    Xs = torch.from_numpy(hs).to(DEV)
    am_s = torch.full((5,), -7, dtype=torch.int32, device=DEV)
    lse_s = torch.zeros(5, dtype=torch.float32, device=DEV)
    assert _static_call(W, X, am, lse) == 0
    assert _static_call(Ws, Xs, am_s, lse_s) == 0
    torch.cuda.synchronize()
    _against_oracle(W_bits, hid, am, lse)
    _against_oracle(Ws_bits, hs, am_s, lse_s)


def test_static_entry_point_does_not_read_what_it_has_not_written():
    """The scratch array filled with NaN bytes before each call: same bits as without."""
    lib = wisv.load_library()
    W_bits = _weights_bits(3000, 192, seed=55)
    W = torch.from_numpy(W_bits.view(np.int16)).view(torch.bfloat16).to(DEV)
    res = []
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    for R in (100, 7):                                       # the second call leaves 93 stale rows behind it
        hid = np.random.default_rng(R).standard_normal((R, 192), dtype=np.float32)
        X = torch.from_numpy(hid).to(DEV)
        outs = []
        for poison in (False, True, True):
            if poison:
                assert lib.wisv_debug_poison_static(st) == 0
            am = torch.full((R,), -7, dtype=torch.int32, device=DEV)
            lse = torch.zeros(R, dtype=torch.float32, device=DEV)
            assert _static_call(W, X, am, lse) == 0
            outs.append((am, lse))
        torch.cuda.synchronize()
        for am, lse in outs[1:]:
            assert torch.equal(am, outs[0][0]) and torch.equal(lse, outs[0][1])
        _against_oracle(W_bits, hid, *outs[0])
        res.append(outs)


def test_static_entry_point_rejects_sizes_beyond_its_scratch():
    lib = wisv.load_library()
    x = torch.zeros(16, dtype=torch.float32, device=DEV)
    p = x.data_ptr()
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert lib.wisv_lm_head_reduce_static(p, 4096, 256, p, 129, p, p, st) == -4      # too many rows
    assert lib.wisv_lm_head_reduce_static(p, 262145, 256, p, 8, p, p, st) == -4      # vocabulary too large
    assert lib.wisv_lm_head_reduce_static(p, 4096, 8200, p, 8, p, p, st) == -4       # hidden size too large
    assert lib.wisv_lm_head_reduce_static(None, 4096, 256, p, 8, p, p, st) == -1
