"""Seeded synthetic inputs for the MRP drafting step.

This module only *generates data* (weights, backbone hidden states and logits, masks,
verification tokens) with the shapes and value distributions of the five benchmark
configurations; it holds none of the method's arithmetic and is the one module that both
the CUDA path's tests/benchmark and the CPU oracle's tests draw inputs from.  Everything is
numpy on the host, drawn from ``Generator(Philox(key=[seed, stream]))`` so that each tensor
has its own stream and does not depend on the order or the number of other draws.

Stand-in for the paper's workloads (SDAR-class shapes: V = 151936, d = 2048 / 4096, block
diffusion decoding): hidden states are N(0,1) plus a multiple of the LM-head row of a
"planted" token so that top-1 probabilities are peaked; base logits are the LM head applied
to those hidden states, computed once here and then treated as opaque input by both sides.
"""
from __future__ import annotations

import math
import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field

import numpy as np

# Stream ids (second word of the Philox key).
_S_WLM, _S_HEAD, _S_Z, _S_TOK, _S_STRENGTH, _S_MASK, _S_VERIFY = 1, 100, 2, 3, 4, 5, 6


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[int(seed), int(stream)]))


def bf16_round(x: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bfloat16 (ties to even); returns float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32)
    out = ((u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))))
           & np.uint32(0xFFFF0000))
    return out.view(np.float32)


def bf16_bits(x: np.ndarray) -> np.ndarray:
    """uint16 bit patterns of float32 values that are already bfloat16-representable."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16)


_CHUNK = 1 << 22


def _normal(seed, stream, shape, scale, dtype) -> np.ndarray:
    """N(0, scale^2) of ``shape``; chunk c is drawn from Philox(key=[seed, stream<<32 | c])
    so the values do not depend on how many threads fill the array."""
    n = int(np.prod(shape))
    out = np.empty(n, np.float32)

    def fill(c):
        i, j = c * _CHUNK, min(n, (c + 1) * _CHUNK)
        g = np.random.Generator(np.random.Philox(key=[int(seed), (int(stream) << 32) | c]))
        g.standard_normal(j - i, dtype=np.float32, out=out[i:j])
        out[i:j] *= np.float32(scale)
        if dtype == "bf16":
            out[i:j] = bf16_round(out[i:j])

    n_chunks = (n + _CHUNK - 1) // _CHUNK
    with ThreadPoolExecutor(max_workers=min(16, os.cpu_count() or 1)) as ex:
        list(ex.map(fill, range(n_chunks)))
    return out.reshape(shape)


@dataclass
class Weights:
    d: int
    F: int
    V: int
    dtype: str                      # "bf16" or "f32": storage type of weights and hidden states
    w_lm: np.ndarray                # [V, d] float32 (bf16-representable when dtype == "bf16")
    heads: list = field(default_factory=list)   # dicts gamma [d], w_gate [F,d], w_up [F,d], w_down [d,F]


def make_weights(d: int, F: int, V: int, n_heads: int, dtype: str, seed: int,
                 head_std: float = 0.02) -> Weights:
    """LM head ~ N(0, 1/d); each head: gamma = 1, SwiGLU matrices ~ N(0, head_std^2)."""
    w_lm = _normal(seed, _S_WLM, (V, d), 1.0 / math.sqrt(d), dtype)
    heads = []
    for k in range(n_heads):
        st = _S_HEAD + 4 * k
        heads.append({
            "gamma": np.ones(d, np.float32),
            "w_gate": _normal(seed, st, (F, d), head_std, dtype),
            "w_up": _normal(seed, st + 1, (F, d), head_std, dtype),
            "w_down": _normal(seed, st + 2, (d, F), head_std, dtype),
        })
    return Weights(d, F, V, dtype, w_lm, heads)


@dataclass
class ModuleWeights:
    """Weights of the token-conditioned MRP module (Sec. 3.2): frozen embedding table, fusion projection,
    D transformer layers.  float32 arrays (bf16-representable when dtype == "bf16")."""
    D: int
    n_attn_heads: int
    mask_token: int
    emb: np.ndarray                 # [V, d]
    w_proj: np.ndarray              # [d, 2d]
    layers: list = field(default_factory=list)   # dicts g_attn, w_q, w_k, w_v, w_o, g_mlp, w_gate, w_up, w_down


def make_module_weights(d: int, F: int, V: int, D: int, n_attn_heads: int, dtype: str, seed: int,
                        std: float = 0.02, proj_std: float | None = None) -> ModuleWeights:
    """Embeddings ~ N(0, 1); projection ~ N(0, proj_std^2) (default 1/sqrt(2d): an output of order one);
    layer matrices ~ N(0, std^2); norm weights 1 + 0.1 cos (non-trivial so that a dropped one shows)."""
    ps = proj_std if proj_std is not None else 1.0 / math.sqrt(2.0 * d)
    st = 500
    emb = _normal(seed, st, (V, d), 1.0, dtype)
    w_proj = _normal(seed, st + 1, (d, 2 * d), ps, dtype)
    layers = []
    for l in range(D):
        b = st + 10 * (l + 1)
        g1 = (1.0 + 0.1 * np.cos(np.arange(d) + l)).astype(np.float32)
        g2 = (1.0 + 0.1 * np.sin(np.arange(d) + l)).astype(np.float32)
        if dtype == "bf16":
            g1, g2 = bf16_round(g1), bf16_round(g2)
        layers.append({
            "g_attn": g1, "w_q": _normal(seed, b, (d, d), std, dtype), "w_k": _normal(seed, b + 1, (d, d), std, dtype),
            "w_v": _normal(seed, b + 2, (d, d), std, dtype), "w_o": _normal(seed, b + 3, (d, d), std, dtype),
            "g_mlp": g2, "w_gate": _normal(seed, b + 4, (F, d), std, dtype), "w_up": _normal(seed, b + 5, (F, d), std, dtype),
            "w_down": _normal(seed, b + 6, (d, F), std, dtype)})
    return ModuleWeights(D, n_attn_heads, V - 1, emb, w_proj, layers)


def planted_gain(s: np.ndarray, V: int, calibrated: bool = True) -> np.ndarray:
    """Logit advantage given to the planted token for a planted strength ``s``.

    Calibrated form: ln V + 1/2 + 2 (s - 1.7), so that the planted token's probability is
    about sigmoid(2 (s - 1.7) + N(0,1)): s = 1 -> 0.2, s = 3 -> 0.93, s = 4 -> 0.99.
    Literal form: ``s`` itself (the planted row is added with coefficient s).
    """
    s = np.asarray(s, np.float64)
    return (math.log(V) + 0.5 + 2.0 * (s - 1.7)) if calibrated else s


@dataclass
class Inputs:
    B: int
    L: int
    hidden: np.ndarray      # [B*L, d] float32 (storage-rounded)
    logits0: np.ndarray     # [B*L, V] float32; rows of unmasked positions are zero
    row_index: np.ndarray   # [M] int32, ascending dense positions b*L+i of masked rows
    planted: np.ndarray     # [B*L] int32 planted token per position
    strength: np.ndarray    # [B*L] float32 planted strength per position


def make_inputs(w: Weights, B: int, L: int, seed: int, s_lo: float, s_hi: float,
                mask_prob: float = 1.0, calibrated: bool = True, logits_fn=None,
                logits_rows: int | None = None, planted=None) -> Inputs:
    """Backbone outputs for one active block per sequence.

    ``mask_prob`` < 1 masks each position independently (at least one per block, by
    resampling the block); 1.0 masks every position.  ``logits_fn(hidden_rows)`` may replace
    the host matrix product that produces the base logits (e.g. an fp32 product on another
    device); whatever it returns is the input both sides then share.  ``logits_rows`` limits the
    base logits to the first that many masked rows (the others stay zero: for consumers that only
    touch a sample of the rows).  ``planted`` [B*L] overrides the uniformly drawn planted tokens
    (e.g. to put the top token of some rows at the two ends of the vocabulary).
    """
    n = B * L
    d, V = w.d, w.V
    z = _rng(seed, _S_Z).standard_normal((n, d), dtype=np.float32)
    drawn = _rng(seed, _S_TOK).integers(0, V, size=n, dtype=np.int64).astype(np.int32)
    planted = drawn if planted is None else np.asarray(planted, np.int32).reshape(n)
    u = _rng(seed, _S_STRENGTH).random(n)
    strength = (s_lo + (s_hi - s_lo) * u).astype(np.float32)
    rows = w.w_lm[planted]                                   # [n, d]
    if calibrated:
        g = planted_gain(strength, V, True)
        coef = g / np.maximum(np.sum(rows.astype(np.float64) ** 2, axis=1), 1e-30)
    else:
        coef = strength.astype(np.float64)
    hidden = (z.astype(np.float64) + coef[:, None] * rows).astype(np.float32)
    if w.dtype == "bf16":
        hidden = bf16_round(hidden)
    rm = _rng(seed, _S_MASK)
    if mask_prob >= 1.0:
        mask = np.ones((B, L), bool)
    else:
        mask = rm.random((B, L)) < mask_prob
        for b in range(B):
            while not mask[b].any():
                mask[b] = rm.random(L) < mask_prob
    row_index = np.flatnonzero(mask.reshape(-1)).astype(np.int32)
    logits0 = np.zeros((n, V), np.float32)
    step = 256
    n_logits = row_index.size if logits_rows is None else min(row_index.size, int(logits_rows))
    for i in range(0, n_logits, step):                       # base logits = LM head on h
        idx = row_index[i:min(i + step, n_logits)]
        logits0[idx] = logits_fn(hidden[idx]) if logits_fn else hidden[idx] @ w.w_lm.T
    return Inputs(B, L, hidden, logits0, row_index, planted, strength)


def make_verify_tokens(draft_tok: np.ndarray, V: int, seed: int, p_match: float = 0.7) -> np.ndarray:
    """Synthetic backbone verification tokens: equal to the draft with probability
    ``p_match`` per slot, otherwise uniform on [0, V)."""
    r = _rng(seed, _S_VERIFY)
    draft_tok = np.asarray(draft_tok, np.int32)
    keep = r.random(draft_tok.shape) < p_match
    rnd = r.integers(0, V, size=draft_tok.shape, dtype=np.int64).astype(np.int32)
    return np.where(keep, draft_tok, rnd).astype(np.int32)


# The five benchmark configurations (shapes, dtypes, value ranges, rule parameters).
CONFIGS = {
    0: dict(name="tiny_f32", dtype="f32", d=256, F=512, V=4096, n_heads=3, K=3, B=1, L=4,
            mask_prob=1.0, s_lo=3.0, s_hi=3.0, tau=0.9, mode="static", seed=0),
    1: dict(name="decode_1p7b", dtype="bf16", d=2048, F=4096, V=151936, n_heads=3, K=3, B=1,
            L=4, mask_prob=1.0, s_lo=1.0, s_hi=4.0, tau=0.9, mode="static", seed=1),
    2: dict(name="spec_8b", dtype="bf16", d=4096, F=8192, V=151936, n_heads=3, K=3, B=32, L=4,
            mask_prob=1.0, s_lo=1.0, s_hi=4.0, tau=0.9, mode="static", seed=2),
    3: dict(name="remask_8b", dtype="bf16", d=4096, F=8192, V=151936, n_heads=2, K=2, B=64,
            L=32, mask_prob=0.5, s_lo=0.5, s_hi=4.0, tau=0.5, mode="dynamic", seed=3),
}
SWEEP_ROWS = (1, 4, 16, 64, 256, 1024, 4096)
SWEEP_CHAIN = (1, 2, 4)


def sweep_config(M: int, K: int) -> dict:
    """One point of the roofline sweep (configuration 4): B = M sequences of one position."""
    p = SWEEP_ROWS.index(M) * len(SWEEP_CHAIN) + SWEEP_CHAIN.index(K)
    return dict(name="sweep_M%d_K%d" % (M, K), dtype="bf16", d=4096, F=8192, V=151936,
                n_heads=K, K=K, B=M, L=1, mask_prob=1.0, s_lo=1.0, s_hi=4.0, tau=0.9,
                mode="static", seed=4000 + p)


def make_config(cfg: dict, weights: Weights | None = None, logits_fn=None, planted=None):
    """Weights (unless given) and inputs of a configuration dict."""
    if weights is None:
        weights = make_weights(cfg["d"], cfg["F"], cfg["V"], cfg["n_heads"], cfg["dtype"],
                               cfg["seed"])
    inp = make_inputs(weights, cfg["B"], cfg["L"], cfg["seed"], cfg["s_lo"], cfg["s_hi"],
                      cfg["mask_prob"], logits_fn=logits_fn, planted=planted)
    return weights, inp
