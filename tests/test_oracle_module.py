"""Pins of the oracle's token-conditioned MRP module (Sec. 3.2; Algorithm 2, "Delta, delta <- g(x_t, h)").

The paper fixes the module's parts and leaves their details open, and prints no worked example; the
reading is the one in oracle/mrp_oracle.c.  The pins: the zero function, the reduction to the reduced
head the rest of the oracle implements, a second implementation on library routines, the single-position
closed form of attention, linearity of the LM head, locality of the block attention, equivariance."""
import numpy as np
import pytest
from scipy.special import expit, softmax

import oracle
from paper_2605_18817_b200 import synth


def problem(seed=3, d=16, F=24, V=40, D=2, heads=2, B=3, L=5, std=0.3):
    mw = synth.make_module_weights(d, F, V, D, heads, "f32", seed, std=std)
    rng = np.random.default_rng(seed)
    hidden = rng.standard_normal((B * L, d)).astype(np.float32)
    tokens = np.where(rng.random(B * L) < 0.5, -1, rng.integers(0, V - 1, B * L)).astype(np.int32)
    w_lm = (rng.standard_normal((V, d)) / np.sqrt(d)).astype(np.float32)
    return mw, hidden, tokens, w_lm


def run(mw, hidden, tokens, w_lm, B, L, rows=None, layers=None, w_proj=None):
    return oracle.module(hidden, tokens, B, L, mw.emb, mw.w_proj if w_proj is None else w_proj,
                         mw.layers if layers is None else layers, w_lm, mw.n_attn_heads, mw.mask_token, row_index=rows)


def library_module(mw, hidden, tokens, B, L, eps=1e-6):
    d = hidden.shape[1]
    H, dh = mw.n_attn_heads, d // mw.n_attn_heads
    tok = np.where(tokens >= 0, tokens, mw.mask_token)
    z = np.concatenate([hidden.astype(np.float64), mw.emb[tok].astype(np.float64)], axis=1) @ mw.w_proj.astype(np.float64).T

    def rms(x, g):
        return x / np.sqrt((x * x).mean(axis=1, keepdims=True) + eps) * g.astype(np.float64)

    for lay in mw.layers:
        n = rms(z, lay["g_attn"])
        q, k, v = (n @ lay[w].astype(np.float64).T for w in ("w_q", "w_k", "w_v"))
        q, k, v = (x.reshape(B, L, H, dh).transpose(0, 2, 1, 3) for x in (q, k, v))
        p = softmax(q @ k.transpose(0, 1, 3, 2) / np.sqrt(dh), axis=-1)
        o = (p @ v).transpose(0, 2, 1, 3).reshape(B * L, d)
        z = z + o @ lay["w_o"].astype(np.float64).T
        n = rms(z, lay["g_mlp"])
        g = n @ lay["w_gate"].astype(np.float64).T
        z = z + (g * expit(g) * (n @ lay["w_up"].astype(np.float64).T)) @ lay["w_down"].astype(np.float64).T
    return z


def test_zero_projection_is_the_zero_function():
    mw, hidden, tokens, w_lm = problem()
    dh, dl = run(mw, hidden, tokens, w_lm, 3, 5, rows=np.arange(15, dtype=np.int32), w_proj=np.zeros_like(mw.w_proj))
    assert not dh.any() and not dl.any()


def test_reduces_to_the_reduced_head_when_attention_is_off_and_the_projection_copies_h():
    # W_p = [I | 0], one layer, W_o = 0: Delta = h + W_down(silu(W_gate n) * W_up n), n = RMSNorm(h) g_mlp,
    # i.e. the hidden state after one step of the reduced head chain, which oracle.draft computes
    mw, hidden, tokens, w_lm = problem(D=1)
    d = hidden.shape[1]
    w_proj = np.concatenate([np.eye(d, dtype=np.float32), np.zeros((d, d), np.float32)], axis=1)
    lay = dict(mw.layers[0], w_o=np.zeros((d, d), np.float32))
    dh, _ = run(mw, hidden, tokens, w_lm, 3, 5, layers=[lay], w_proj=w_proj)
    head = {"gamma": lay["g_mlp"], "w_gate": lay["w_gate"], "w_up": lay["w_up"], "w_down": lay["w_down"]}
    ref = oracle.draft(hidden, np.zeros((15, w_lm.shape[0]), np.float32), [head], w_lm, want_hidden=True)
    assert np.allclose(dh, ref.hidden, rtol=0, atol=1e-12)


def test_matches_library_implementation_and_the_lm_head_is_linear():
    mw, hidden, tokens, w_lm = problem()
    rows = np.array([14, 0, 7, 3], np.int32)
    dh, dl = run(mw, hidden, tokens, w_lm, 3, 5, rows=rows)
    want = library_module(mw, hidden, tokens, 3, 5)
    assert np.abs(want).max() > 0.1
    assert np.allclose(dh, want, rtol=0, atol=1e-11)
    assert np.allclose(dl, dh[rows] @ w_lm.astype(np.float64).T, rtol=0, atol=1e-11)


def test_single_position_blocks_attention_returns_the_value_vector():
    # L = 1: the softmax over one position is 1, so o = v and the attention sub-layer is z + W_o W_v n
    mw, hidden, tokens, w_lm = problem(D=1, B=4, L=1)
    dh, _ = run(mw, hidden, tokens, w_lm, 4, 1)
    lay = mw.layers[0]
    tok = np.where(tokens >= 0, tokens, mw.mask_token)
    z = np.concatenate([hidden, mw.emb[tok]], axis=1).astype(np.float64) @ mw.w_proj.astype(np.float64).T
    n = z / np.sqrt((z * z).mean(axis=1, keepdims=True) + 1e-6) * lay["g_attn"]
    z = z + (n @ lay["w_v"].astype(np.float64).T) @ lay["w_o"].astype(np.float64).T
    n = z / np.sqrt((z * z).mean(axis=1, keepdims=True) + 1e-6) * lay["g_mlp"]
    g = n @ lay["w_gate"].astype(np.float64).T
    z = z + (g / (1 + np.exp(-g)) * (n @ lay["w_up"].astype(np.float64).T)) @ lay["w_down"].astype(np.float64).T
    assert np.allclose(dh, z, rtol=0, atol=1e-12)


def test_revealed_tokens_condition_the_other_positions_of_their_block_only():
    mw, hidden, tokens, w_lm = problem()
    B, L = 3, 5
    base, _ = run(mw, hidden, tokens, w_lm, B, L)
    t2 = tokens.copy()
    t2[6] = (max(tokens[6], 0) + 1) % (mw.emb.shape[0] - 1)          # position 1 of block 1 gets another token
    other, _ = run(mw, hidden, t2, w_lm, B, L)
    blk = np.arange(B * L) // L
    assert np.array_equal(other[blk != 1], base[blk != 1])            # other blocks: untouched
    assert np.all(np.abs(other[blk == 1] - base[blk == 1]).max(axis=1) > 1e-6)    # every position of the block moves
    # without the attention output projection there is no path between positions
    layers = [dict(l, w_o=np.zeros_like(l["w_o"])) for l in mw.layers]
    a, _ = run(mw, hidden, tokens, w_lm, B, L, layers=layers)
    b, _ = run(mw, hidden, t2, w_lm, B, L, layers=layers)
    keep = np.arange(B * L) != 6
    assert np.array_equal(a[keep], b[keep]) and np.abs(a[6] - b[6]).max() > 1e-6
    # a masked position is the [MASK] token's embedding
    t3 = np.where(tokens < 0, mw.mask_token, tokens).astype(np.int32)
    c, _ = run(mw, hidden, t3, w_lm, B, L)
    assert np.array_equal(c, base)


def test_positions_of_a_block_are_exchangeable():
    # no positional term: permuting the positions of a block permutes its outputs
    mw, hidden, tokens, w_lm = problem()
    B, L = 3, 5
    base, _ = run(mw, hidden, tokens, w_lm, B, L)
    perm = np.arange(B * L)
    perm[5:10] = 5 + np.array([3, 0, 4, 1, 2])
    out, _ = run(mw, hidden[perm], tokens[perm], w_lm, B, L)
    assert np.allclose(out, base[perm], rtol=0, atol=1e-12)


def test_numpy_statistics_agree_with_the_c_statistics():
    rng = np.random.default_rng(4)
    l = (rng.standard_normal((6, 50)) * 3).astype(np.float32)
    l[2, 7] = l[2, 3] = l[2].max() + 1.0                               # an exact tie: lowest index wins
    conf, lse, tok, margin = oracle.stats(l)
    w = synth.make_weights(8, 8, 50, 0, "f32", 1)
    r = oracle.draft(np.zeros((6, 8), np.float32), l, [], w.w_lm, K=0)
    assert np.allclose(conf, r.conf[0], atol=1e-15) and np.allclose(lse, r.lse[0], atol=1e-13)
    assert np.array_equal(tok, r.token[0]) and np.allclose(margin, r.margin[0], atol=1e-13)
    assert tok[2] == 3 and margin[2] == 0
