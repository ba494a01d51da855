"""The seeded generators: determinism, layouts, storage conversion."""
import numpy as np
import torch

import gen


def test_bf16_storage_conversion_matches_torch():
    x = np.random.default_rng(0).standard_normal(10000).astype(np.float32)
    x[:4] = [1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, -0.0, 3.0e38]
    ours = gen.f32_to_bf16_bits(x)
    ref = torch.as_tensor(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, ref)
    assert np.array_equal(gen.bf16_bits_to_f32(ours), torch.as_tensor(x).to(torch.bfloat16).float().numpy())


def test_arrays_are_deterministic_and_order_independent():
    cfg = gen.config("tiny")
    k = gen.synth.window_lengths(cfg)
    a = gen.make_hidden(cfg, k)
    w = gen.make_weights(cfg)
    b = gen.make_hidden(cfg, k)
    assert all(np.array_equal(a[n], b[n]) for n in a)
    assert w["lm_head"].shape == (cfg.V, cfg.H) and w["lm_head"].dtype == np.uint16
    assert w["W1"].shape == (cfg.d_J, cfg.d_in)
    assert a["target_hidden"].shape == (cfg.B * (cfg.K + 1), cfg.H)
    assert a["draft_hidden"].shape == (cfg.B * cfg.K, cfg.H_d)
    assert 0 <= a["csi"][:, 0].min() and a["csi"][:, 0].max() <= 30
    assert 1 <= a["csi"][:, 1].min() and a["csi"][:, 1].max() <= 100
    other = gen.make_hidden(cfg.with_(seed=1), k)
    assert not np.array_equal(a["target_hidden"], other["target_hidden"])
    std = gen.bf16_bits_to_f32(w["lm_head"]).std()
    assert abs(std - 0.02) < 1e-3


def test_ragged_windows_and_offsets():
    cfg = gen.config("8b_sh256")
    k = gen.synth.window_lengths(cfg)
    assert k.shape == (256,) and k.min() >= 4 and k.max() <= 16
    k_off, row_off = gen.row_offsets(k)
    assert k_off[-1] == k.sum() and row_off[-1] == k.sum() + 256
    assert np.array_equal(np.diff(row_off), k + 1)


def test_draft_tokens_match_rate():
    cfg = gen.VerifyConfig("t", B=200, K=8, H=8, H_d=8, d_c=2, d_J=8, V=1000, match_rate=0.7, seed=3)
    k = gen.synth.window_lengths(cfg)
    _, row_off = gen.row_offsets(k)
    ref = np.arange(row_off[-1], dtype=np.int32) % 1000
    toks = gen.make_draft_tokens(cfg, k, ref)
    rows = np.concatenate([row_off[b] + np.arange(k[b]) for b in range(cfg.B)])
    rate = (toks == ref[rows]).mean()
    assert abs(rate - 0.7) < 0.04
    assert toks.min() >= 0 and toks.max() < 1000


def test_pack_selective_layout():
    k = np.array([3, 0, 2, 4], np.int32)
    hd = np.arange(9 * 2, dtype=np.float32).reshape(9, 2)
    sel = np.array([1, 0, 1, 0, 0, 0, 1, 1, 0], bool)
    packed, sel_off, sel_pos = gen.pack_selective(hd, k, sel)
    assert sel_off.tolist() == [0, 2, 2, 2, 4]
    assert sel_pos.tolist() == [0, 2, 1, 2]
    assert np.array_equal(packed, hd[[0, 2, 6, 7]])
    packed, sel_off, sel_pos = gen.pack_selective(hd, k, np.zeros(9, bool))
    assert packed.shape == (0, 2) and sel_off.tolist() == [0, 0, 0, 0, 0]


def test_pack_selective_with_empty_windows_at_the_end():
    k = np.array([2, 0, 3, 0, 0], np.int32)
    hd = np.arange(5 * 2, dtype=np.float32).reshape(5, 2)
    sel = np.array([0, 1, 1, 0, 1], bool)
    packed, sel_off, sel_pos = gen.pack_selective(hd, k, sel)
    assert sel_off.tolist() == [0, 1, 1, 3, 3, 3] and sel_pos.tolist() == [1, 0, 2]
    assert np.array_equal(packed, hd[[1, 2, 4]])
