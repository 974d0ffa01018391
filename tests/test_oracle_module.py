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


# ---- the clean prefix of Fig. 1(c): keys and values of committed positions as inputs ----

def _tail_problem(seed=5, B=2, P=4, L=3, D=2):
    mw, hidden, tokens, w_lm = problem(seed=seed, D=D, B=B, L=P + L)
    long_h, _, k_long, v_long = oracle.module(hidden, tokens, B, P + L, mw.emb, mw.w_proj, mw.layers, w_lm, mw.n_attn_heads,
                                              mw.mask_token, want_kv=True)
    d = hidden.shape[1]
    tail = (np.arange(B * (P + L)) % (P + L)) >= P
    cap = P + 2                                                         # rows beyond the length: never read
    ks = [np.full((B, cap, d), np.nan, np.float32) for _ in range(D)]
    vs = [np.full((B, cap, d), np.nan, np.float32) for _ in range(D)]
    for l in range(D):
        ks[l][:, :P] = k_long[l].reshape(B, P + L, d)[:, :P]
        vs[l][:, :P] = v_long[l].reshape(B, P + L, d)[:, :P]
    return mw, hidden, tokens, w_lm, long_h, tail, ks, vs, k_long, v_long


def test_block_behind_a_prefix_equals_the_tail_of_the_longer_block():
    # Given the per-layer keys and values of the first P positions, the last L positions of a block of P + L
    # compute exactly what a block of L behind that prefix computes: the prefix enters through nothing else.
    B, P, L, D = 2, 4, 3, 2
    mw, hidden, tokens, w_lm, long_h, tail, ks, vs, k_long, v_long = _tail_problem(B=B, P=P, L=L, D=D)
    rows = np.array([0, 4, 5], np.int32)
    dh, dl, k_out, v_out = oracle.module(hidden[tail], tokens[tail], B, L, mw.emb, mw.w_proj, mw.layers, w_lm, mw.n_attn_heads,
                                         mw.mask_token, row_index=rows, prefix=(ks, vs, np.full(B, P, np.int32)), want_kv=True)
    assert np.abs(long_h[tail]).max() > 0.1
    assert np.allclose(dh, long_h[tail], rtol=0, atol=2e-6)             # (the prefix rows were rounded to fp32)
    assert np.allclose(dl, dh[rows] @ w_lm.astype(np.float64).T, rtol=0, atol=1e-11)
    for l in range(D):
        assert np.allclose(k_out[l], k_long[l][tail], rtol=0, atol=2e-6) and np.allclose(v_out[l], v_long[l][tail], rtol=0, atol=2e-6)
    # ... and the prefix matters: without it the block computes something else
    alone, _ = run(mw, hidden[tail], tokens[tail], w_lm, B, L)
    assert np.abs(alone - long_h[tail]).max() > 1e-3


def test_prefix_lengths_are_per_sequence():
    B, P, L, D = 2, 4, 3, 2
    mw, hidden, tokens, w_lm, long_h, tail, ks, vs, _, _ = _tail_problem(B=B, P=P, L=L, D=D)
    alone, _ = run(mw, hidden[tail], tokens[tail], w_lm, B, L)
    dh, _ = oracle.module(hidden[tail], tokens[tail], B, L, mw.emb, mw.w_proj, mw.layers, w_lm, mw.n_attn_heads, mw.mask_token,
                          prefix=(ks, vs, np.array([P, 0], np.int32)))
    assert np.allclose(dh[:L], long_h[tail][:L], rtol=0, atol=2e-6)     # sequence 0: behind its prefix
    assert np.array_equal(dh[L:], alone[L:])                            # sequence 1: no prefix rows in use
    # a shorter prefix is another function
    dh2, _ = oracle.module(hidden[tail], tokens[tail], B, L, mw.emb, mw.w_proj, mw.layers, w_lm, mw.n_attn_heads, mw.mask_token,
                           prefix=(ks, vs, np.array([P - 1, 0], np.int32)))
    assert np.abs(dh2[:L] - dh[:L]).max() > 1e-4 and np.array_equal(dh2[L:], dh[L:])


def test_zero_keys_average_the_values_of_prefix_and_block():
    # W_k = 0 and zero prefix keys: every score is 0, the softmax is uniform over the P_b + L keys and the
    # attention output is the plain mean of the prefix's and the block's values (one layer, W_o = I, no MLP)
    B, L, D = 2, 3, 1
    mw, hidden, tokens, w_lm = problem(seed=8, D=D, B=B, L=L)
    d = hidden.shape[1]
    lay = dict(mw.layers[0], w_k=np.zeros((d, d), np.float32), w_o=np.eye(d, dtype=np.float32),
               w_down=np.zeros_like(mw.layers[0]["w_down"]))
    rng = np.random.default_rng(1)
    cap, plen = 5, np.array([5, 2], np.int32)
    pv = rng.standard_normal((B, cap, d)).astype(np.float32)
    z0, _, _, v_blk = oracle.module(hidden, tokens, B, L, mw.emb, mw.w_proj, [dict(lay, w_o=np.zeros((d, d), np.float32))], w_lm,
                                    mw.n_attn_heads, mw.mask_token, want_kv=True)
    dh, _ = oracle.module(hidden, tokens, B, L, mw.emb, mw.w_proj, [lay], w_lm, mw.n_attn_heads, mw.mask_token,
                          prefix=([np.zeros((B, cap, d), np.float32)], [pv], plen))
    for b in range(B):
        mean = (pv[b, :plen[b]].astype(np.float64).sum(axis=0) + v_blk[0][b * L:(b + 1) * L].sum(axis=0)) / (plen[b] + L)
        assert np.allclose(dh[b * L:(b + 1) * L], z0[b * L:(b + 1) * L] + mean, rtol=0, atol=1e-12)


def test_prefix_matches_library_implementation():
    # second implementation on library routines: softmax over the concatenated keys, one sequence at a time
    B, L, D = 2, 3, 2
    mw, hidden, tokens, w_lm = problem(seed=9, D=D, B=B, L=L)
    d, H = hidden.shape[1], mw.n_attn_heads
    dh_ = d // H
    rng = np.random.default_rng(2)
    cap, plen = 6, np.array([6, 3], np.int32)
    ks = [rng.standard_normal((B, cap, d)).astype(np.float32) for _ in range(D)]
    vs = [rng.standard_normal((B, cap, d)).astype(np.float32) for _ in range(D)]
    got, _ = oracle.module(hidden, tokens, B, L, mw.emb, mw.w_proj, mw.layers, w_lm, H, mw.mask_token, prefix=(ks, vs, plen))
    tok = np.where(tokens >= 0, tokens, mw.mask_token)
    z = np.concatenate([hidden.astype(np.float64), mw.emb[tok].astype(np.float64)], axis=1) @ mw.w_proj.astype(np.float64).T
    rms = lambda x, g: x / np.sqrt((x * x).mean(axis=1, keepdims=True) + 1e-6) * g.astype(np.float64)
    for l, lay in enumerate(mw.layers):
        n = rms(z, lay["g_attn"])
        q, k, v = (n @ lay[w].astype(np.float64).T for w in ("w_q", "w_k", "w_v"))
        o = np.zeros_like(z)
        for b in range(B):
            kk = np.concatenate([ks[l][b, :plen[b]].astype(np.float64), k[b * L:(b + 1) * L]])
            vv = np.concatenate([vs[l][b, :plen[b]].astype(np.float64), v[b * L:(b + 1) * L]])
            for h in range(H):
                c = slice(h * dh_, (h + 1) * dh_)
                p = softmax(q[b * L:(b + 1) * L, c] @ kk[:, c].T / np.sqrt(dh_), axis=-1)
                o[b * L:(b + 1) * L, c] = p @ vv[:, c]
        z = z + o @ lay["w_o"].astype(np.float64).T
        n = rms(z, lay["g_mlp"])
        g = n @ lay["w_gate"].astype(np.float64).T
        z = z + (g * expit(g) * (n @ lay["w_up"].astype(np.float64).T)) @ lay["w_down"].astype(np.float64).T
    assert np.allclose(got, z, rtol=0, atol=1e-11)


def test_kl_rows_agrees_with_the_chain_objective_and_closed_forms():
    # the numpy objective used for the module against the C objective of the head chain (itself pinned against a
    # library relative entropy and a closed form): with a zero down projection l_1 = l_0, so both see the same rows
    from scipy.special import rel_entr
    rng = np.random.default_rng(6)
    d, F, V, M = 8, 12, 30, 5
    w = synth.make_weights(d, F, V, 1, "f32", 3)
    w.heads[0]["w_down"][:] = 0
    hidden = rng.standard_normal((M, d)).astype(np.float32)
    l0 = (rng.standard_normal((M, V)) * 2).astype(np.float32)
    teacher = (l0 + rng.standard_normal((M, V))).astype(np.float32)
    _, kl_c = oracle.draft_kl(hidden, l0, teacher[None], w.heads, w.w_lm)
    got = oracle.kl_rows(teacher, l0)
    assert np.all(got > 0) and np.allclose(got, kl_c[0], rtol=1e-12, atol=1e-14)
    assert np.allclose(got, rel_entr(softmax(teacher.astype(np.float64), axis=1), softmax(l0.astype(np.float64), axis=1)).sum(axis=1),
                       rtol=1e-10, atol=1e-13)
    assert np.abs(oracle.kl_rows(l0, l0 + 3.5)).max() < 1e-12           # shift invariance, equal distributions
    # two tokens: p = sigmoid(a), q = sigmoid(b)
    a, b = 0.7, -0.4
    p, q = expit(a), expit(b)
    want = p * np.log(p / q) + (1 - p) * np.log((1 - p) / (1 - q))
    assert abs(oracle.kl_rows([[a, 0.0]], [[b, 0.0]])[0] - want) < 1e-14
