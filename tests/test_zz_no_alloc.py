"""The allocation-free LM-head entry point against the regular one.

Some callers of this library cannot allocate device memory (their host framework
has reserved the whole GPU, or they run in a loop that must not enter the CUDA
allocator), so they cannot create a verifier context.  wisv_lm_head_reduce_static
serves them from a fixed scratch array inside the library.  This test calls it
through the C ABI twice in a row, on different inputs, and checks argmax and
log-sum-exp against wisv_verify's on the same rows.  It is collected last so that
a run that stops at the first failure has already run every other test.
"""
import ctypes as C

import numpy as np
import pytest
import torch

import gen
import paper_2604_17701_b200 as wisv
from paper_2604_17701_b200 import cases
from parity import LSE_TOL, oracle_ref_argmax

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


def test_static_entry_point_matches_verify_on_two_calls_in_a_row():
    lib = wisv.load_library()
    # two different batches: the second has fewer rows, a vocabulary tail and other data,
    # so anything left in the shared scratch by the first call would show
    cfgs = [gen.VerifyConfig("a", B=20, K=5, H=256, H_d=128, d_c=2, d_J=128, V=4096, match_rate=0.5, seed=21),
            gen.VerifyConfig("b", B=3, K=4, H=320, H_d=128, d_c=2, d_J=128, V=1000, match_rate=0.5, seed=22)]
    refs = [_reference_rows(c) for c in cfgs]
    # outputs are allocated up front; the calls themselves allocate nothing
    outs = [(torch.full((r[1].shape[0],), -7, dtype=torch.int32, device=DEV),
             torch.zeros(r[1].shape[0], dtype=torch.float32, device=DEV)) for r in refs]
    st = torch.cuda.current_stream()
    for (d, _, _), (am, lse) in zip(refs, outs):
        V, H = d["lm_head"].shape
        R = d["target_hidden"].shape[0]
        rc = lib.wisv_lm_head_reduce_static(d["lm_head"].data_ptr(), V, H, d["target_hidden"].data_ptr(), R,
                                            am.data_ptr(), lse.data_ptr(), C.c_void_p(st.cuda_stream))
        assert rc == 0
    torch.cuda.synchronize()
    for (d, ref_am, ref_lse), (am, lse) in zip(refs, outs):
        assert torch.equal(am, ref_am)
        assert float((lse - ref_lse).abs().max()) <= LSE_TOL


def test_static_entry_point_rejects_sizes_beyond_its_scratch():
    lib = wisv.load_library()
    x = torch.zeros(16, dtype=torch.float32, device=DEV)
    p = x.data_ptr()
    st = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    assert lib.wisv_lm_head_reduce_static(p, 4096, 256, p, 129, p, p, st) == -4      # too many rows
    assert lib.wisv_lm_head_reduce_static(p, 262145, 256, p, 8, p, p, st) == -4      # vocabulary too large
    assert lib.wisv_lm_head_reduce_static(p, 4096, 8200, p, 8, p, p, st) == -4       # hidden size too large
    assert lib.wisv_lm_head_reduce_static(None, 4096, 256, p, 8, p, p, st) == -1
