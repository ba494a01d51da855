"""Counter-based seeded generators and input layouts.

Every array has its own Philox stream (key = [seed, stream id]) so its contents
do not depend on the order in which arrays are generated.  The shapes and value
distributions follow the 1B-drafter / 8B-target setting of the paper's
experiments (Section VI-A): bf16 LM head N(0, 0.02), fp32 hidden states N(0, 1),
CSI = [SNR dB ~ U(0,30), rate Mbps ~ U(1,100)], a two-layer decision head.
They stand in for recorded decoding traces, which need a dataset and trained
weights.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, replace
from typing import Dict, Optional, Tuple

import numpy as np

# stream ids (one per array)
_S_LM_HEAD, _S_W1, _S_B1, _S_W2, _S_HT, _S_HD, _S_CSI = 1, 2, 3, 4, 5, 6, 7
_S_KLEN, _S_MATCH, _S_RANDTOK, _S_Q, _S_U = 8, 9, 10, 11, 12

_CHUNK_ELEMS = 1 << 22  # fixed: chunk c of an array is its own Philox stream, so threads can fill it


@dataclass(frozen=True)
class VerifyConfig:
    name: str
    B: int            # requests
    K: int            # uniform window length (ignored when K_lo/K_hi set)
    H: int            # target hidden size
    H_d: int          # drafter hidden size
    d_c: int          # CSI feature count
    d_J: int          # decision-head hidden width
    V: int            # vocabulary size
    match_rate: float  # probability that a draft token is forced to the reference argmax
    mode: str = "FH"   # "FH" full-hidden upload | "SH" selective-hidden upload
    act: str = "gelu"  # "gelu" | "relu"
    tau: float = 0.5
    seed: int = 0
    stochastic: bool = False
    K_lo: int = 0      # ragged windows: K_b ~ U{K_lo..K_hi}
    K_hi: int = 0
    weight_seed: int = -1  # seed of the model weights; -1: same as seed

    @property
    def d_in(self) -> int:
        return self.H_d + self.H + self.d_c

    def with_(self, **kw) -> "VerifyConfig":
        return replace(self, **kw)


# one 8B-shaped model (LM head + decision head) serves every 8B workload
_8B = dict(H=4096, H_d=2048, d_c=2, d_J=1024, V=128256, weight_seed=1000)

# second model pair of the paper's testbed (Section VII): Qwen2.5-0.5B drafter -> Qwen2.5-7B target
_QWEN = dict(H=3584, H_d=896, d_c=2, d_J=1024, V=152064, weight_seed=2000)

CONFIGS: Dict[str, VerifyConfig] = {
    "tiny": VerifyConfig("tiny", B=8, K=4, H=256, H_d=128, d_c=2, d_J=128, V=4096,
                         match_rate=0.5, seed=0),
    "8b_b1": VerifyConfig("8b_b1", B=1, K=8, match_rate=0.7, seed=1, **_8B),
    # between the two: 144 and 288 window rows (two and three row tiles of 128)
    "8b_b16": VerifyConfig("8b_b16", B=16, K=8, match_rate=0.7, seed=8, **_8B),
    "8b_b32": VerifyConfig("8b_b32", B=32, K=8, match_rate=0.7, seed=9, **_8B),
    "8b_b64": VerifyConfig("8b_b64", B=64, K=8, match_rate=0.7, seed=3, **_8B),
    "8b_b64_m30": VerifyConfig("8b_b64_m30", B=64, K=8, match_rate=0.30, seed=2, **_8B),
    "8b_b64_m95": VerifyConfig("8b_b64_m95", B=64, K=8, match_rate=0.95, seed=4, **_8B),
    "8b_sh64": VerifyConfig("8b_sh64", B=64, K=8, match_rate=0.65, mode="SH", seed=13, **_8B),
    "8b_sh256": VerifyConfig("8b_sh256", B=256, K=0, K_lo=4, K_hi=16, match_rate=0.65,
                             mode="SH", seed=5, **_8B),
    "8b_b512": VerifyConfig("8b_b512", B=512, K=16, match_rate=0.7, seed=6, **_8B),
    "qwen7b_b1": VerifyConfig("qwen7b_b1", B=1, K=8, match_rate=0.7, seed=11, **_QWEN),
    "qwen7b_b8_k64": VerifyConfig("qwen7b_b8_k64", B=8, K=64, match_rate=0.9, seed=12, **_QWEN),
    "8b_b512_stoch": VerifyConfig("8b_b512_stoch", B=512, K=16, match_rate=0.7, seed=7,
                                  stochastic=True, **_8B),
}


def config(name: str) -> VerifyConfig:
    return CONFIGS[name]


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Storage conversion fp32 -> bf16 bit pattern (round to nearest even)."""
    b = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = ((b >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((b + r) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _normal_bf16(seed: int, stream: int, shape: Tuple[int, ...], std: float) -> np.ndarray:
    """bf16 bits of N(0, std); chunk c is drawn from stream (stream, c), independent of thread count."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.uint16)

    def fill(c: int) -> None:
        lo = c * _CHUNK_ELEMS
        hi = min(n, lo + _CHUNK_ELEMS)
        g = np.random.Generator(np.random.Philox(key=[int(seed), int(stream) + (c << 32)]))
        x = g.standard_normal(hi - lo, dtype=np.float32)
        x *= np.float32(std)
        out[lo:hi] = f32_to_bf16_bits(x)

    chunks = range((n + _CHUNK_ELEMS - 1) // _CHUNK_ELEMS)
    if len(chunks) > 1:
        with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as ex:
            list(ex.map(fill, chunks))
    else:
        for c in chunks:
            fill(c)
    return out.reshape(shape)


def window_lengths(cfg: VerifyConfig) -> np.ndarray:
    """K_b per request: uniform K, or U{K_lo..K_hi} for ragged windows."""
    if cfg.K_hi > 0:
        return _rng(cfg.seed, _S_KLEN).integers(cfg.K_lo, cfg.K_hi + 1, size=cfg.B).astype(np.int32)
    return np.full(cfg.B, cfg.K, dtype=np.int32)


def row_offsets(k_len: np.ndarray) -> Tuple[np.ndarray, np.ndarray]:
    """(k_off [B+1], row_off [B+1]): prefix sums of K_b and of K_b+1."""
    k_len = np.asarray(k_len, dtype=np.int64)
    k_off = np.zeros(k_len.size + 1, dtype=np.int32)
    k_off[1:] = np.cumsum(k_len)
    row_off = (k_off + np.arange(k_len.size + 1)).astype(np.int32)
    return k_off, row_off


def make_weights(cfg: VerifyConfig, lm_head: Optional[np.ndarray] = None) -> Dict[str, np.ndarray]:
    """LM head and decision-head parameters (lm_head given: reuse that array instead of drawing it again).

    lm_head: bf16 bits [V, H] ~ N(0, 0.02).  W1: bf16 bits [d_J, d_in] with columns
    ordered [h^D | h^T | c] (the order of Eq. 23), each column block drawn from its own
    sub-stream so a different concatenation order is a pure column permutation.
    """
    ws = cfg.weight_seed if cfg.weight_seed >= 0 else cfg.seed
    if lm_head is None:
        lm_head = _normal_bf16(ws, _S_LM_HEAD, (cfg.V, cfg.H), 0.02)
    # hidden-state columns ~ N(0, 1/sqrt(d_in)); CSI columns ~ N(0, 1/128) because the CSI
    # features are consumed unnormalised (tens of dB / Mbps) and would otherwise swamp z
    std1 = 1.0 / np.sqrt(cfg.d_in)
    blocks = []
    for j, (width, std) in enumerate(((cfg.H_d, std1), (cfg.H, std1), (cfg.d_c, 1.0 / 128.0))):
        blocks.append(_normal_bf16(ws, _S_W1 + 100 * (j + 1), (cfg.d_J, width), std))
    W1 = np.ascontiguousarray(np.concatenate(blocks, axis=1))
    b1 = (_rng(ws, _S_B1).standard_normal(cfg.d_J, dtype=np.float32) * np.float32(0.1))
    w2 = (_rng(ws, _S_W2).standard_normal(cfg.d_J, dtype=np.float32)
          * np.float32(1.0 / np.sqrt(cfg.d_J)))
    b2 = np.float32(0.0625)
    return dict(lm_head=lm_head, W1=W1, b1=b1, w2=w2, b2=b2)


def make_hidden(cfg: VerifyConfig, k_len: np.ndarray) -> Dict[str, np.ndarray]:
    """target_hidden fp32 [R, H], dense draft_hidden fp32 [T, H_d], csi fp32 [B, d_c]."""
    T = int(np.sum(k_len))
    R = T + cfg.B
    ht = _rng(cfg.seed, _S_HT).standard_normal((R, cfg.H), dtype=np.float32)
    hd = _rng(cfg.seed, _S_HD).standard_normal((T, cfg.H_d), dtype=np.float32)
    g = _rng(cfg.seed, _S_CSI)
    csi = np.empty((cfg.B, cfg.d_c), dtype=np.float32)
    for c in range(cfg.d_c):
        lo, hi = ((0.0, 30.0), (1.0, 100.0))[c % 2]  # SNR dB, rate Mbps, repeating
        csi[:, c] = g.uniform(lo, hi, size=cfg.B).astype(np.float32)
    return dict(target_hidden=ht, draft_hidden=hd, csi=csi)


def make_draft_tokens(cfg: VerifyConfig, k_len: np.ndarray, ref_argmax: np.ndarray) -> np.ndarray:
    """Draft tokens int32 [T].

    With probability match_rate a position takes ref_argmax of its window row (a
    model output the caller supplies, indexed by window row r = row_off[b] + i),
    otherwise a uniform token id.
    """
    k_off, row_off = row_offsets(k_len)
    T = int(k_off[-1])
    forced = _rng(cfg.seed, _S_MATCH).random(T) < cfg.match_rate
    rand_tok = _rng(cfg.seed, _S_RANDTOK).integers(0, cfg.V, size=T).astype(np.int32)
    rows = np.concatenate([row_off[b] + np.arange(k_len[b]) for b in range(len(k_len))]) \
        if T else np.zeros(0, dtype=np.int64)
    ref = np.asarray(ref_argmax, dtype=np.int32)[rows]
    return np.where(forced, ref, rand_tok).astype(np.int32)


def make_stochastic_inputs(cfg: VerifyConfig, T: int) -> Tuple[np.ndarray, np.ndarray]:
    """Draft-token probabilities q ~ U(0.05, 1) and uniforms u ~ U[0, 1), fp32 [T] each."""
    q = _rng(cfg.seed, _S_Q).uniform(0.05, 1.0, size=T).astype(np.float32)
    u = _rng(cfg.seed, _S_U).random(T, dtype=np.float32)
    return q, u


def pack_selective(draft_hidden: np.ndarray, k_len: np.ndarray, select: np.ndarray
                   ) -> Tuple[np.ndarray, np.ndarray, np.ndarray]:
    """Selective-hidden upload layout.

    select: bool [T], True where the drafter uploads its hidden state.  Returns
    (packed fp32 [M_sel, H_d], sel_off int32 [B+1], sel_pos int32 [M_sel]) with
    window-relative positions ascending inside each request.
    """
    k_off, _ = row_offsets(k_len)
    select = np.asarray(select, dtype=bool)
    idx = np.nonzero(select)[0]
    sel_off = np.zeros(len(k_len) + 1, dtype=np.int32)
    req_all = np.repeat(np.arange(len(k_len)), np.asarray(k_len, dtype=np.int64))
    counts = np.bincount(req_all, weights=select.astype(np.float64), minlength=len(k_len)).astype(np.int64)
    sel_off[1:] = np.cumsum(counts)
    req = np.searchsorted(k_off[1:], idx, side="right")
    sel_pos = (idx - k_off[req]).astype(np.int32)
    packed = np.ascontiguousarray(draft_hidden[idx], dtype=np.float32)
    return packed, sel_off, sel_pos
