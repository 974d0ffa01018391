"""Pins of the CPU oracle's drafting pass against what the paper and the mathematics fix.

None of these tests re-types the oracle's loops: they use special cases with known answers,
invariants, direct enumeration without the max-subtraction trick, and a second
implementation on numpy/scipy library routines.
"""
import math

import numpy as np
import pytest
from scipy.special import expit, logsumexp

import oracle
from paper_2605_18817_b200 import synth


def small_problem(seed=11, d=24, F=40, V=96, n_heads=3, rows=6, dtype="f32", head_std=0.3):
    w = synth.make_weights(d, F, V, n_heads, dtype, seed, head_std=head_std)
    for k, h in enumerate(w.heads):      # non-trivial gamma so a dropped gamma is caught
        h["gamma"] = (1.0 + 0.25 * np.cos(np.arange(d) + k)).astype(np.float32)
    inp = synth.make_inputs(w, rows, 1, seed, 1.0, 3.0)
    return w, inp


def library_draft(hidden, logits0, heads, w_lm, eps):
    """The same forward on library routines (fp64): rms norm, expit, matmul, logsumexp."""
    h = hidden.astype(np.float64)
    l = logits0.astype(np.float64)
    W = w_lm.astype(np.float64)
    stats = []

    def st(l):
        lse = logsumexp(l, axis=1)
        return np.exp(l.max(axis=1) - lse), lse, l.argmax(axis=1)

    stats.append(st(l))
    logits = []
    for hd in heads:
        rms = np.sqrt(np.mean(h * h, axis=1, keepdims=True) + eps)
        xh = h / rms * hd["gamma"].astype(np.float64)
        g = xh @ hd["w_gate"].astype(np.float64).T
        u = xh @ hd["w_up"].astype(np.float64).T
        a = g * expit(g) * u
        r = a @ hd["w_down"].astype(np.float64).T
        h = h + r
        l = l + r @ W.T
        stats.append(st(l))
        logits.append(l.copy())
    return stats, logits, h


def test_zero_residual_heads_leave_logits_unchanged():
    # "the zero function is already a reasonable approximation": W_down = 0 => delta = 0.
    w, inp = small_problem()
    for hd in w.heads:
        hd["w_down"] = np.zeros_like(hd["w_down"])
    r = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, want_logits=True, want_hidden=True)
    for k in range(1, 4):
        assert np.array_equal(r.token[k], r.token[0])
        assert np.array_equal(r.conf[k], r.conf[0])
        assert np.array_equal(r.lse[k], r.lse[0])
        assert np.array_equal(r.logits[k - 1], inp.logits0.astype(np.float64))
    assert np.array_equal(r.hidden, inp.hidden.astype(np.float64))


def test_softmax_normalisation_and_confidence_range():
    w, inp = small_problem()
    r = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, want_logits=True)
    V = w.V
    for k in range(1, 4):
        p = np.exp(r.logits[k - 1] - r.lse[k][:, None])
        assert np.allclose(p.sum(axis=1), 1.0, atol=1e-12)
        assert np.allclose(p.max(axis=1), r.conf[k], atol=1e-14)
    p0 = np.exp(inp.logits0.astype(np.float64) - r.lse[0][:, None])
    assert np.allclose(p0.sum(axis=1), 1.0, atol=1e-12)
    assert np.all(r.conf > 1.0 / V) and np.all(r.conf <= 1.0)


def test_chain_is_linear_in_the_residual():
    # l_K - l_0 = W_lm (h_K - h_0): every delta goes through the same LM head.
    w, inp = small_problem()
    r = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, want_logits=True, want_hidden=True)
    dh = r.hidden - inp.hidden.astype(np.float64)
    dl = r.logits[-1] - inp.logits0.astype(np.float64)
    assert np.allclose(dl, dh @ w.w_lm.astype(np.float64).T, rtol=0, atol=1e-10)
    assert np.abs(dl).max() > 1e-2          # the residual is not trivially zero
    # scaling the first head's output matrix by 1/2 halves delta_1 exactly (power of two)
    one = [dict(w.heads[0])]
    r1 = oracle.draft(inp.hidden, inp.logits0, one, w.w_lm, want_logits=True)
    one[0]["w_down"] = (0.5 * one[0]["w_down"]).astype(np.float32)
    r2 = oracle.draft(inp.hidden, inp.logits0, one, w.w_lm, want_logits=True)
    l0 = inp.logits0.astype(np.float64)
    assert np.allclose(r2.logits[0] - l0, 0.5 * (r1.logits[0] - l0), rtol=0, atol=1e-12)


def test_hand_example_closed_form():
    # d = F = 2, V = 3, identity gate/up/down, LM head rows e0, e1, e0+e1.
    h = np.array([[3.0, 4.0]], np.float32)
    l0 = np.array([[0.25, -0.5, 1.0]], np.float32)
    eye = np.eye(2, dtype=np.float32)
    heads = [dict(gamma=np.array([1.0, 2.0], np.float32), w_gate=eye, w_up=eye, w_down=eye)]
    w_lm = np.array([[1, 0], [0, 1], [1, 1]], np.float32)
    eps = 1e-6
    rstd = 1.0 / math.sqrt((9.0 + 16.0) / 2.0 + eps)
    x0, x1 = 3.0 * rstd * 1.0, 4.0 * rstd * 2.0
    a0 = x0 / (1.0 + math.exp(-x0)) * x0
    a1 = x1 / (1.0 + math.exp(-x1)) * x1
    l1 = [0.25 + a0, -0.5 + a1, 1.0 + a0 + a1]
    Z = sum(math.exp(v) for v in l1)
    r = oracle.draft(h, l0, heads, w_lm, eps=eps, want_logits=True, want_hidden=True)
    assert np.allclose(r.logits[0][0], l1, atol=1e-14)
    assert r.token[1, 0] == 2 and r.token[0, 0] == 2
    assert abs(r.conf[1, 0] - math.exp(l1[2]) / Z) < 1e-14
    assert abs(r.lse[1, 0] - math.log(Z)) < 1e-14
    assert abs(r.margin[1, 0] - (l1[2] - max(l1[0], l1[1]))) < 1e-14
    assert np.allclose(r.hidden[0], [3.0 + a0, 4.0 + a1], atol=1e-14)
    Z0 = sum(math.exp(float(v)) for v in l0[0])
    assert abs(r.conf[0, 0] - math.exp(1.0) / Z0) < 1e-14


def test_brute_force_tiny_vocabulary():
    # direct enumeration in pure Python, softmax without max subtraction
    w, inp = small_problem(seed=5, d=8, F=6, V=16, n_heads=2, rows=3)
    r = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm)
    d, F, V = 8, 6, 16
    for m in range(3):
        h = [float(x) for x in inp.hidden[m]]
        l = [float(x) for x in inp.logits0[m]]
        for k in range(0, 3):
            if k > 0:
                hd = w.heads[k - 1]
                ms = sum(x * x for x in h) / d
                xh = [h[j] / math.sqrt(ms + 1e-6) * float(hd["gamma"][j]) for j in range(d)]
                a = []
                for f in range(F):
                    g = sum(float(hd["w_gate"][f, j]) * xh[j] for j in range(d))
                    u = sum(float(hd["w_up"][f, j]) * xh[j] for j in range(d))
                    a.append(g / (1.0 + math.exp(-g)) * u)
                res = [sum(float(hd["w_down"][j, f]) * a[f] for f in range(F)) for j in range(d)]
                h = [h[j] + res[j] for j in range(d)]
                l = [l[v] + sum(float(w.w_lm[v, j]) * res[j] for j in range(d)) for v in range(V)]
            e = [math.exp(x) for x in l]
            Z = sum(e)
            p = [x / Z for x in e]
            best = max(range(V), key=lambda v: (p[v], -v))
            assert r.token[k, m] == best
            assert abs(r.conf[k, m] - p[best]) < 1e-12
            assert abs(r.lse[k, m] - math.log(Z)) < 1e-12


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
def test_matches_library_implementation(dtype):
    w, inp = small_problem(seed=21, d=64, F=96, V=640, n_heads=3, rows=7, dtype=dtype)
    r = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, want_logits=True, want_hidden=True)
    stats, logits, h = library_draft(inp.hidden, inp.logits0, w.heads, w.w_lm, 1e-6)
    for k in range(4):
        c, lse, tok = stats[k]
        assert np.allclose(r.conf[k], c, rtol=0, atol=1e-12)
        assert np.allclose(r.lse[k], lse, rtol=0, atol=1e-11)
        assert np.array_equal(r.token[k], tok)
    for k in range(3):
        assert np.allclose(r.logits[k], logits[k], rtol=0, atol=1e-10)
    assert np.allclose(r.hidden, h, rtol=0, atol=1e-11)


def test_matches_library_implementation_config0(tiny_cfg):
    cfg, w, inp = tiny_cfg
    r = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=cfg["K"], row_index=inp.row_index)
    stats, _, _ = library_draft(inp.hidden[inp.row_index], inp.logits0[inp.row_index], w.heads,
                                w.w_lm, 1e-6)
    for k in range(cfg["K"] + 1):
        assert np.allclose(r.conf[k], stats[k][0], rtol=0, atol=1e-12)
        assert np.array_equal(r.token[k], stats[k][2])


def test_row_index_gathers_rows_and_k_truncates_chain():
    w, inp = small_problem(rows=9)
    full = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm)
    idx = np.array([7, 2, 5], np.int32)
    sub = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=2, row_index=idx)
    assert sub.conf.shape == (3, 3)
    assert np.array_equal(sub.conf, full.conf[:3][:, idx])
    assert np.array_equal(sub.token, full.token[:3][:, idx])


def test_shift_and_permutation_invariance():
    w, inp = small_problem()
    r = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm)
    shifted = oracle.draft(inp.hidden, inp.logits0 + np.float32(2.0), w.heads, w.w_lm)
    assert np.array_equal(shifted.token, r.token)
    assert np.allclose(shifted.conf, r.conf, atol=1e-13)
    assert np.allclose(shifted.lse, r.lse + 2.0, atol=1e-12)
    perm = np.random.default_rng(0).permutation(w.V)
    rp = oracle.draft(inp.hidden, inp.logits0[:, perm], w.heads, w.w_lm[perm])
    assert np.array_equal(perm[rp.token], r.token)
    assert np.allclose(rp.conf, r.conf, atol=1e-13)
    assert np.allclose(rp.lse, r.lse, atol=1e-12)


def test_planted_token_wins_with_closed_form_confidence(tiny_cfg):
    cfg, w, inp = tiny_cfg
    r = oracle.draft(inp.hidden, inp.logits0, [], w.w_lm, K=0, row_index=inp.row_index)
    t = inp.planted[inp.row_index]
    assert np.array_equal(r.token[0], t)
    l = inp.logits0[inp.row_index].astype(np.float64)
    for m in range(len(t)):
        others = np.delete(l[m], t[m]) - l[m, t[m]]
        assert abs(r.conf[0, m] - 1.0 / (1.0 + np.exp(others).sum())) < 1e-13
    # calibrated strength 3 => confidences peaked (roughly sigmoid(2.6 + N(0,1)))
    assert np.all(r.conf[0] > 0.5)


def test_argmax_tie_goes_to_lowest_token_and_margin_is_zero():
    h = np.zeros((1, 4), np.float32)
    l0 = np.array([[0.0, 2.0, 2.0, -1.0, 2.0]], np.float32)
    r = oracle.draft(h, l0, [], np.zeros((5, 4), np.float32), K=0)
    assert r.token[0, 0] == 1 and r.margin[0, 0] == 0.0


def test_generator_confidence_calibration():
    # planted strength -> confidence mapping stated for the synthetic workloads
    w = synth.make_weights(64, 128, 4096, 0, "f32", 9)
    for s, lo, hi in ((1.0, 0.05, 0.5), (3.0, 0.8, 0.99), (4.0, 0.95, 1.0)):
        inp = synth.make_inputs(w, 64, 1, 9, s, s)
        r = oracle.draft(inp.hidden, inp.logits0, [], w.w_lm, K=0)
        assert lo < np.median(r.conf[0]) < hi, (s, np.median(r.conf[0]))


# ---- backbone logits from the hidden states (logits0=None): l_0 = W_lm n_0 ----

def test_from_hidden_equals_the_pass_on_precomputed_base_logits():
    """With base logits that are exactly representable the two entry points must agree: integer
    weights and hidden states make W_lm h an exact float32 matrix, so nothing is rounded."""
    rng = np.random.default_rng(3)
    w, inp = small_problem(seed=5)
    W = rng.integers(-3, 4, size=w.w_lm.shape).astype(np.float32)
    H = rng.integers(-2, 3, size=inp.hidden.shape).astype(np.float32)
    l0 = (H.astype(np.float64) @ W.astype(np.float64).T).astype(np.float32)
    a = oracle.draft(H, l0, w.heads, W, want_logits=True, want_hidden=True)
    b = oracle.draft(H, None, w.heads, W, want_logits=True, want_hidden=True)
    np.testing.assert_allclose(b.logits, a.logits, rtol=0, atol=1e-12)
    np.testing.assert_allclose(b.lse, a.lse, rtol=0, atol=1e-12)
    np.testing.assert_array_equal(b.token, a.token)
    np.testing.assert_allclose(b.hidden, a.hidden, rtol=0, atol=0)


def test_from_hidden_without_final_norm_every_step_is_the_lm_head_of_that_hidden_state():
    """l_k = l_0 + W_lm (h_k - h_0) = W_lm h_k: checked through two different outputs of the
    oracle (step-accumulated logits vs. a library matmul on its final hidden state)."""
    w, inp = small_problem(seed=8)
    for K in (1, 3):
        r = oracle.draft(inp.hidden, None, w.heads, w.w_lm, K=K, want_logits=True, want_hidden=True)
        direct = r.hidden @ w.w_lm.astype(np.float64).T
        np.testing.assert_allclose(r.logits[K - 1], direct, rtol=0, atol=1e-10)
        np.testing.assert_allclose(r.lse[K], logsumexp(direct, axis=1), rtol=0, atol=1e-10)


def test_from_hidden_final_norm_closed_form_on_one_hot_rows():
    """h_0 = c e_j: RMSNorm gives sqrt(d) sign(c) e_j (eps -> 0), so l_0 = sqrt(d) sign(c) g_j W_lm[:, j]."""
    d, V = 24, 96
    w, _ = small_problem(seed=9, d=d, V=V)
    g = (1.0 + 0.5 * np.sin(np.arange(d))).astype(np.float32)
    js = [0, 5, 23, 11]
    cs = [2.0, -3.0, 0.5, 7.0]
    H = np.zeros((4, d), np.float32)
    for i, (j, c) in enumerate(zip(js, cs)):
        H[i, j] = c
    r = oracle.draft(H, None, w.heads, w.w_lm, K=0, eps=0.0, final_gamma=g)
    for i, (j, c) in enumerate(zip(js, cs)):
        l = math.sqrt(d) * np.sign(c) * float(g[j]) * w.w_lm[:, j].astype(np.float64)
        assert r.token[0, i] == int(np.argmax(l))
        np.testing.assert_allclose(r.lse[0, i], logsumexp(l), rtol=0, atol=1e-12)
        np.testing.assert_allclose(r.conf[0, i], np.exp(l.max() - logsumexp(l)), rtol=0, atol=1e-12)


def test_from_hidden_final_norm_ignores_the_scale_of_the_hidden_state_at_step_zero():
    w, inp = small_problem(seed=10)
    g = (1.0 + 0.25 * np.cos(np.arange(w.d))).astype(np.float32)
    H = inp.hidden.astype(np.float32)
    a = oracle.draft(H, None, w.heads, w.w_lm, K=0, eps=0.0, final_gamma=g)
    b = oracle.draft(4.0 * H, None, w.heads, w.w_lm, K=0, eps=0.0, final_gamma=g)
    np.testing.assert_allclose(b.lse, a.lse, rtol=0, atol=1e-10)
    # and the library form of the same definition, with eps
    n0 = H.astype(np.float64) / np.sqrt(np.mean(H.astype(np.float64) ** 2, axis=1, keepdims=True) + 1e-6) * g
    c = oracle.draft(H, None, w.heads, w.w_lm, K=0, eps=1e-6, final_gamma=g)
    np.testing.assert_allclose(c.lse[0], logsumexp(n0 @ w.w_lm.astype(np.float64).T, axis=1), rtol=0, atol=1e-10)


def test_from_hidden_matches_library_implementation_with_final_norm():
    w, inp = small_problem(seed=12)
    g = (1.0 + 0.25 * np.cos(np.arange(w.d))).astype(np.float32)
    H = inp.hidden.astype(np.float64)
    n0 = H / np.sqrt(np.mean(H * H, axis=1, keepdims=True) + 1e-6) * g
    l0 = n0 @ w.w_lm.astype(np.float64).T
    stats, logits, _ = library_draft(inp.hidden, l0, w.heads, w.w_lm, 1e-6)
    r = oracle.draft(inp.hidden, None, w.heads, w.w_lm, eps=1e-6, final_gamma=g, want_logits=True)
    for k in range(len(w.heads) + 1):
        np.testing.assert_allclose(r.conf[k], stats[k][0], rtol=0, atol=1e-10)
        np.testing.assert_allclose(r.lse[k], stats[k][1], rtol=0, atol=1e-10)
        np.testing.assert_array_equal(r.token[k], stats[k][2])


# ---- probability of the step-0 argmax token under the updated logits (conf_first) ----

def test_conf_first_is_the_softmax_probability_of_the_step_zero_token():
    # library evaluation from the materialised logits: exp(l_k[tok_0] - logsumexp(l_k))
    w, inp = small_problem(seed=19, head_std=0.5)
    r = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, want_logits=True)
    assert np.array_equal(r.conf_first[0], r.conf[0])
    tok0 = r.token[0]
    rows = np.arange(tok0.size)
    moved = 0
    for k in range(1, 4):
        l = r.logits[k - 1]
        want = np.exp(l[rows, tok0] - logsumexp(l, axis=1))
        assert np.allclose(r.conf_first[k], want, rtol=0, atol=1e-14)
        same = r.token[k] == tok0
        assert np.array_equal(r.conf_first[k][same], r.conf[k][same])      # still on top: the confidence itself
        assert np.all(r.conf_first[k][~same] < r.conf[k][~same])           # displaced: strictly below the top
        moved += int((~same).sum())
    assert moved > 0                                                        # the case is exercised


def test_conf_first_with_zero_residual_heads_stays_at_the_backbone_confidence():
    w, inp = small_problem()
    for hd in w.heads:
        hd["w_down"] = np.zeros_like(hd["w_down"])
    r = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm)
    for k in range(4):
        assert np.array_equal(r.conf_first[k], r.conf[0])


# ---- the training objective: forward KL of the teacher against the corrected logits (Eq. (3)) ----

def _teacher(rng, logits, scale):
    """Teacher logits near the corrected logits (the residual is a small correction, Sec. 3.1)."""
    return (logits + scale * rng.standard_normal(logits.shape)).astype(np.float32)


def test_kl_matches_library_relative_entropy_and_is_zero_on_equal_distributions():
    from scipy.special import rel_entr, softmax
    w, inp = small_problem(seed=23, head_std=0.4)
    K, M, V = 3, inp.hidden.shape[0], w.V
    base = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, want_logits=True)
    rng = np.random.default_rng(5)
    teacher = _teacher(rng, base.logits, 0.7)
    r, kl = oracle.draft_kl(inp.hidden, inp.logits0, teacher, w.heads, w.w_lm)
    assert np.array_equal(r.conf, base.conf) and np.array_equal(r.token, base.token)
    want = rel_entr(softmax(teacher.astype(np.float64), axis=2), softmax(base.logits, axis=2)).sum(axis=2)
    assert kl.shape == (K, M) and np.all(kl > 0)
    assert np.allclose(kl, want, rtol=1e-10, atol=1e-13)
    # the direction matters: KL(q || p) differs
    other = rel_entr(softmax(base.logits, axis=2), softmax(teacher.astype(np.float64), axis=2)).sum(axis=2)
    assert np.abs(other - want).max() > 1e-3
    # a teacher that equals the corrected logits up to a constant per row is the same distribution: KL = 0
    # (the logits are unnormalised log-densities: the normalising constants cancel)
    # (fp32-exact inputs so that "equal" is exact: heads that produce nothing)
    for hd in w.heads:
        hd["w_down"] = np.zeros_like(hd["w_down"])
    t0 = np.repeat(inp.logits0[None, :, :], K, axis=0) + np.float32(2.5)
    _, kl0 = oracle.draft_kl(inp.hidden, inp.logits0, t0, w.heads, w.w_lm)
    assert np.abs(kl0).max() < 1e-12


def test_kl_two_token_closed_form():
    # V = 2, zero heads: KL((a, 1-a) || (b, 1-b)) = a ln(a/b) + (1-a) ln((1-a)/(1-b)), with a, b the
    # logistic function of the logit differences
    d, F, V = 8, 8, 2
    w = synth.make_weights(d, F, V, 1, "f32", 3)
    w.heads[0]["w_down"] = np.zeros_like(w.heads[0]["w_down"])
    hidden = np.ones((2, d), np.float32)
    logits0 = np.array([[0.5, -0.25], [2.0, 3.0]], np.float32)
    teacher = np.array([[[1.5, 0.0], [-1.0, 0.5]]], np.float32)
    _, kl = oracle.draft_kl(hidden, logits0, teacher, w.heads, w.w_lm)
    for m in range(2):
        a = 1.0 / (1.0 + math.exp(-(float(teacher[0, m, 0]) - float(teacher[0, m, 1]))))
        b = 1.0 / (1.0 + math.exp(-(float(logits0[m, 0]) - float(logits0[m, 1]))))
        want = a * math.log(a / b) + (1 - a) * math.log((1 - a) / (1 - b))
        assert abs(kl[0, m] - want) < 1e-14


def test_kl_row_index_and_chain_truncation():
    w, inp = small_problem(seed=29, rows=7)
    rng = np.random.default_rng(8)
    full = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, want_logits=True)
    teacher = _teacher(rng, full.logits, 0.5)
    _, kl = oracle.draft_kl(inp.hidden, inp.logits0, teacher, w.heads, w.w_lm)
    sub = np.array([5, 0, 3], np.int32)
    _, kl_sub = oracle.draft_kl(inp.hidden, inp.logits0, teacher[:2][:, sub], w.heads, w.w_lm, K=2, row_index=sub)
    assert np.array_equal(kl_sub, kl[:2][:, sub])
