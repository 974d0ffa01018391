"""Pins of the oracle's reveal / remask / verify rules: definitions restated with sorting
and set operations, closed forms, invariants, and the cap values printed from the paper's
formula (tests/golden/cap_values.txt)."""
import itertools
import os

import numpy as np
import pytest

import oracle

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def random_stats(rng, K, B, L, mask_prob=0.7, V=50):
    mask = rng.random((B, L)) < mask_prob
    row_index = np.flatnonzero(mask.reshape(-1)).astype(np.int32)
    M = row_index.size
    conf = rng.random((K + 1, M)).astype(np.float32)
    token = rng.integers(0, V, (K + 1, M)).astype(np.int32)
    return mask, row_index, conf, token


def test_cap_formula_matches_printed_values():
    rows = [l.split() for l in open(os.path.join(GOLDEN, "cap_values.txt")) if l[0] != "#"]
    assert len(rows) >= 8
    for n, L, m in rows:
        assert oracle.cap(int(n), int(L)) == int(m), (n, L, m)


def test_cap_floor_is_exact_on_multiples_of_ten():
    # 0.7 * 10 = 7 exactly in the formula; binary rounding must not turn it into 6
    assert oracle.cap(10, 32) == 7 and oracle.cap(20, 32) == 14 and oracle.cap(30, 32) == 21


@pytest.mark.parametrize("seed", range(6))
def test_static_picks_are_the_top_r_by_sorting(seed):
    rng = np.random.default_rng(seed)
    K, B, L = 3, 5, 8
    r_reveal, r_draft = 2, 1 + seed % 2
    mask, ri, conf, token = random_stats(rng, K, B, L)
    s = oracle.select(conf, token, ri, B, L, oracle.STATIC, r_reveal=r_reveal, r_draft=r_draft)
    Kd = K * r_draft
    for b in range(B):
        rows = [m for m in range(ri.size) if ri[m] // L == b]
        left = list(rows)
        drafts = []
        for k in range(K + 1):
            r = r_reveal if k == 0 else r_draft
            order = sorted(left, key=lambda m: (-conf[k, m], ri[m] % L))[:r]
            for m in order:
                dense = ri[m]
                assert s.step_of[dense] == k
                assert s.out_token[dense] == token[k, m]
                assert s.reveal_mask[dense] == (1 if k == 0 else 0)
                if k > 0:
                    drafts.append((ri[m] % L, token[k, m]))
                left.remove(m)
        for m in left:
            assert s.step_of[ri[m]] == -1 and s.out_token[ri[m]] == -1
        assert s.draft_len[b] == len(drafts)
        for q, (p, t) in enumerate(drafts):
            assert s.draft_pos[b, q] == p and s.draft_tok[b, q] == t
        assert np.all(s.draft_pos[b, len(drafts):] == -1)
        assert s.draft_tok.shape == (B, Kd)
    # unmasked positions are never touched; no remask in static mode
    assert np.all(s.step_of[~mask.reshape(-1)] == -1)
    assert not s.remask_mask.any()
    # picks are distinct positions and bounded in number
    assert (s.step_of >= 0).sum() <= B * (r_reveal + K * r_draft)


def test_static_brute_force_all_subsets_tiny():
    # the r most confident of n candidates = the size-r subset with the largest sorted key
    rng = np.random.default_rng(3)
    conf = rng.random((1, 5)).astype(np.float32)
    token = np.arange(5, dtype=np.int32)[None]
    s = oracle.select(conf, token, None, 1, 5, oracle.STATIC, r_reveal=2, r_draft=0)
    best = max(itertools.combinations(range(5), 2), key=lambda c: sorted(conf[0, list(c)], reverse=True))
    assert set(np.flatnonzero(s.reveal_mask)) == set(best)


@pytest.mark.parametrize("seed", range(6))
def test_dynamic_reveal_set_is_threshold_set(seed):
    rng = np.random.default_rng(100 + seed)
    K, B, L = 2, 6, 16
    tau = np.float32(0.5)
    mask, ri, conf, token = random_stats(rng, K, B, L)
    s = oracle.select(conf, token, ri, B, L, oracle.DYNAMIC_REMASK, tau=float(tau))
    dense_conf = np.full((K + 1, B * L), -1.0, np.float32)
    dense_conf[:, ri] = conf
    for b in range(B):
        sl = slice(b * L, (b + 1) * L)
        m = mask[b]
        R = m & (dense_conf[0, sl] >= tau)
        if m.any() and not R.any():
            R = np.zeros(L, bool)
            cand = np.flatnonzero(m)
            R[cand[np.argmax(dense_conf[0, sl][cand])]] = True
        assert np.array_equal(s.reveal_mask[sl].astype(bool), R)
        cmin = dense_conf[1:, sl].min(axis=0)
        rem = R & (cmin < tau)
        if R.any() and (R & ~rem).sum() == 0:
            cand = np.flatnonzero(R)
            rem[cand[np.argmax(dense_conf[0, sl][cand])]] = False
        assert np.array_equal(s.remask_mask[sl].astype(bool), rem)
        committed = R & ~rem
        tok0 = np.full(B * L, -1, np.int32)
        tok0[ri] = token[0]
        assert np.array_equal(s.out_token[sl], np.where(committed, tok0[sl], -1))
        assert np.array_equal(s.step_of[sl], np.where(committed, 0, -1))
    assert not s.draft_len.any()


def test_dynamic_threshold_extremes_and_boundary():
    rng = np.random.default_rng(7)
    K, B, L = 1, 4, 8
    mask, ri, conf, token = random_stats(rng, K, B, L, mask_prob=0.8)
    s0 = oracle.select(conf, token, ri, B, L, oracle.DYNAMIC_REMASK, tau=0.0)
    assert np.array_equal(s0.reveal_mask.astype(bool), mask.reshape(-1))
    assert not s0.remask_mask.any()
    s2 = oracle.select(conf, token, ri, B, L, oracle.DYNAMIC_REMASK, tau=1.5)
    for b in range(B):
        assert s2.reveal_mask[b * L:(b + 1) * L].sum() == (1 if mask[b].any() else 0)
        # forced reveal survives the remask step (progress guarantee)
        assert s2.remask_mask[b * L:(b + 1) * L].sum() == 0
    s3 = oracle.select(conf, token, ri, B, L, oracle.DYNAMIC_REMASK, tau=1.5, ensure_progress=False)
    assert not s3.reveal_mask.any() and np.all(s3.out_token == -1)
    # "at or above": a confidence equal to tau is revealed, and is not remasked at equality
    c = np.array([[0.5, 0.4], [0.5, 0.9]], np.float32)
    t = np.zeros((2, 2), np.int32)
    s = oracle.select(c, t, None, 1, 2, oracle.DYNAMIC_REMASK, tau=0.5)
    assert list(s.reveal_mask) == [1, 0] and list(s.remask_mask) == [0, 0]


def test_remask_policies_and_monotonicity():
    rng = np.random.default_rng(9)
    K, B, L = 3, 8, 16
    mask, ri, conf, token = random_stats(rng, K, B, L)
    prev = None
    for tau in (0.2, 0.4, 0.6, 0.8):
        a = oracle.select(conf, token, ri, B, L, oracle.DYNAMIC_REMASK, tau=tau,
                          ensure_progress=False)
        last = oracle.select(conf, token, ri, B, L, oracle.DYNAMIC_REMASK, tau=tau,
                             remask_policy=1, ensure_progress=False)
        assert np.array_equal(a.reveal_mask, last.reveal_mask)
        # policy ALL revokes a superset of policy LAST
        assert np.all(a.remask_mask >= last.remask_mask)
        # remask subset of reveal subset of masked
        assert np.all(a.remask_mask <= a.reveal_mask)
        assert np.all(a.reveal_mask.astype(bool) <= mask.reshape(-1))
        if prev is not None:      # raising tau never enlarges R
            assert np.all(a.reveal_mask <= prev)
        prev = a.reveal_mask
    # policy LAST looks only at step K
    dense = np.full(B * L, 2.0, np.float32)
    dense[ri] = conf[K]
    last = oracle.select(conf, token, ri, B, L, oracle.DYNAMIC_REMASK, tau=0.5, remask_policy=1,
                         ensure_progress=False)
    assert np.array_equal(last.remask_mask.astype(bool), last.reveal_mask.astype(bool) & (dense < 0.5))


def test_cap_keeps_the_most_confident():
    L = 16
    conf0 = np.linspace(0.99, 0.6, L).astype(np.float32)
    rng = np.random.default_rng(1)
    perm = rng.permutation(L)
    conf = np.stack([conf0[perm], np.ones(L, np.float32)])
    token = np.zeros((2, L), np.int32)
    s = oracle.select(conf, token, None, 1, L, oracle.DYNAMIC_REMASK, tau=0.5, use_cap=True)
    m = oracle.cap(L, L)
    assert m == 11 and s.reveal_mask.sum() == m
    assert set(np.flatnonzero(s.reveal_mask)) == set(np.argsort(-conf[0])[:m])
    s_off = oracle.select(conf, token, None, 1, L, oracle.DYNAMIC_REMASK, tau=0.5, use_cap=False)
    assert s_off.reveal_mask.sum() == L


def test_verify_prefix_and_positionwise():
    d = np.array([[5, 6, 7, 8], [1, 2, 3, 4], [9, 9, 9, 9], [1, 1, 1, 1]], np.int32)
    v = np.array([[5, 6, 0, 8], [1, 2, 3, 4], [0, 9, 9, 9], [1, 1, 1, 1]], np.int32)
    n = np.array([4, 4, 4, 2], np.int32)
    alen, amask = oracle.verify(d, v, n)
    assert list(alen) == [2, 4, 0, 2]
    assert amask.tolist() == [[1, 1, 0, 0], [1, 1, 1, 1], [0, 0, 0, 0], [1, 1, 0, 0]]
    alen, amask = oracle.verify(d, v, n, positionwise=True)
    assert list(alen) == [3, 4, 3, 2]
    assert amask.tolist() == [[1, 1, 0, 1], [1, 1, 1, 1], [0, 1, 1, 1], [1, 1, 0, 0]]


def test_verify_accept_length_is_first_mismatch_and_geometric_mean():
    from paper_2605_18817_b200 import synth
    B, Kd, V = 100000, 4, 151936
    rng = np.random.default_rng(0)
    d = rng.integers(0, V, (B, Kd)).astype(np.int32)
    v = synth.make_verify_tokens(d, V, seed=2, p_match=0.7)
    alen, amask = oracle.verify(d, v, np.full(B, Kd, np.int32))
    neq = d != v
    first = np.where(neq.any(axis=1), neq.argmax(axis=1), Kd)
    assert np.array_equal(alen, first)
    assert np.array_equal(amask.sum(axis=1), alen)
    # E[len] = sum_{j=1..4} 0.7^j = 1.7731 for a geometric accepted prefix
    expect = sum(0.7 ** j for j in range(1, 5))
    sd = alen.std() / np.sqrt(B)
    assert abs(alen.mean() - expect) < 4 * sd + 1e-3


# ---- the block-state transition x_t -> x_{t-1} (oracle.commit) ----

def _stats(rng, K, M, V=1000):
    return rng.random((K + 1, M)).astype(np.float32), rng.integers(0, V, (K + 1, M)).astype(np.int32)


def test_commit_hand_example_for_the_three_decoding_modes():
    # one block of 6 positions, position 2 already holds token 7
    tokens = np.array([-1, -1, 7, -1, -1, -1], np.int32)
    ri = np.array([0, 1, 3, 4, 5], np.int32)
    conf = np.array([[0.9, 0.2, 0.5, 0.1, 0.3],      # step 0: position 0 is the most confident
                     [0.0, 0.3, 0.8, 0.2, 0.1],      # step 1: position 3
                     [0.0, 0.6, 0.0, 0.7, 0.2]], np.float32)   # step 2: position 4
    tok = np.array([[10, 11, 13, 14, 15], [20, 21, 23, 24, 25], [30, 31, 33, 34, 35]], np.int32)
    sel = oracle.select(conf, tok, ri, 1, 6, oracle.STATIC)
    # Algorithm 2: reveals of every step are unmasked
    c = oracle.commit(tokens, sel, 1, 6)
    assert c.tokens.tolist() == [10, -1, 7, 23, 34, -1]
    assert c.row_index.tolist() == [1, 5] and c.block_masked.tolist() == [2]
    # Algorithm 3: the backbone accepts the first draft only
    c = oracle.commit(tokens, sel, 1, 6, accept_mask=np.array([[1, 0]], np.int8))
    assert c.tokens.tolist() == [10, -1, 7, 23, -1, -1]
    assert c.row_index.tolist() == [1, 4, 5]
    c = oracle.commit(tokens, sel, 1, 6, accept_mask=np.array([[0, 0]], np.int8))
    assert c.tokens.tolist() == [10, -1, 7, -1, -1, -1]
    # Algorithm 4: R = {0, 3} at tau = 0.45; the update drops position 0 below tau, so it is remasked
    sel = oracle.select(conf[:2], tok[:2], ri, 1, 6, oracle.DYNAMIC_REMASK, tau=0.45)
    assert sel.reveal_mask.tolist() == [1, 0, 0, 1, 0, 0] and sel.remask_mask.tolist() == [1, 0, 0, 0, 0, 0]
    c = oracle.commit(tokens, sel, 1, 6)
    assert c.tokens.tolist() == [-1, -1, 7, 13, -1, -1]


def test_commit_invariants_on_random_states():
    rng = np.random.default_rng(5)
    for case in range(30):
        B, L, K = 1 + case % 5, 1 + (case * 7) % 13, case % 4
        tokens = np.where(rng.random(B * L) < 0.6, -1, rng.integers(0, 99, B * L)).astype(np.int32)
        ri = np.flatnonzero(tokens < 0).astype(np.int32)
        if ri.size == 0:
            continue
        conf, tok = _stats(rng, K, ri.size)
        mode = oracle.STATIC if case % 2 == 0 else oracle.DYNAMIC_REMASK
        sel = oracle.select(conf, tok, ri, B, L, mode, tau=0.5, r_reveal=1 + case % 2, r_draft=1)
        acc = None
        if mode == oracle.STATIC and case % 4 == 0 and K > 0:
            vt = np.where(rng.random((B, K)) < 0.6, sel.draft_tok, -5).astype(np.int32)
            _, acc = oracle.verify(sel.draft_tok, vt, sel.draft_len)
        c = oracle.commit(tokens, sel, B, L, accept_mask=acc)
        was_masked = tokens < 0
        newly = was_masked & (c.tokens >= 0)
        assert np.array_equal(c.tokens[~was_masked], tokens[~was_masked])      # committed tokens never change
        assert np.array_equal(c.tokens[newly], sel.out_token[newly])            # new ones are the selected tokens
        assert np.array_equal(c.row_index, np.flatnonzero(c.tokens < 0))
        assert c.block_masked.sum() == c.row_index.size
        if acc is None:
            assert newly.sum() == (sel.out_token >= 0).sum()
        else:
            assert newly.sum() == (sel.step_of == 0).sum() + acc.sum()


def test_direct_decoding_loop_needs_ceil_L_over_K_plus_one_forwards():
    """Algorithm 2 with r = 1: every backbone forward unmasks min(K + 1, masked) positions of a
    block, so a block of L positions is done after ceil(L / (K + 1)) forwards, whatever the statistics."""
    rng = np.random.default_rng(9)
    for L, K in ((4, 1), (7, 2), (32, 3), (5, 0)):
        B = 3
        tokens = np.full(B * L, -1, np.int32)
        n = 0
        while (tokens < 0).any():
            ri = np.flatnonzero(tokens < 0).astype(np.int32)
            conf, tok = _stats(rng, K, ri.size)
            sel = oracle.select(conf, tok, ri, B, L, oracle.STATIC)
            tokens = oracle.commit(tokens, sel, B, L).tokens
            n += 1
            assert n <= L
        assert n == -(-L // (K + 1))


def test_commit_positionwise_acceptance_keeps_a_later_match():
    """Algorithm 3 read literally (per position): a later draft that the backbone confirms is kept
    even though an earlier one was rejected; with prefix acceptance it is not."""
    tokens = np.array([-1, -1, -1, -1], np.int32)
    ri = np.arange(4, dtype=np.int32)
    conf = np.array([[0.9, 0.1, 0.2, 0.3], [0.0, 0.8, 0.2, 0.3], [0.0, 0.0, 0.7, 0.3]], np.float32)
    tok = np.array([[1, 2, 3, 4], [11, 12, 13, 14], [21, 22, 23, 24]], np.int32)
    sel = oracle.select(conf, tok, ri, 1, 4, oracle.STATIC)
    assert sel.draft_pos.tolist() == [[1, 2]] and sel.draft_tok.tolist() == [[12, 23]]
    verify_tok = np.array([[99, 23]], np.int32)          # first draft rejected, second confirmed
    alen, amask = oracle.verify(sel.draft_tok, verify_tok, sel.draft_len, positionwise=False)
    assert alen.tolist() == [0] and amask.tolist() == [[0, 0]]
    assert oracle.commit(tokens, sel, 1, 4, accept_mask=amask).tokens.tolist() == [1, -1, -1, -1]
    alen, amask = oracle.verify(sel.draft_tok, verify_tok, sel.draft_len, positionwise=True)
    assert alen.tolist() == [1] and amask.tolist() == [[0, 1]]
    assert oracle.commit(tokens, sel, 1, 4, accept_mask=amask).tokens.tolist() == [1, -1, 23, -1]


def test_remask_by_the_revealed_token_hand_example():
    # one block of four masked positions, K = 2, tau = 0.5.  Position 0: stays confident and on the same
    # token.  Position 1: the top probability stays high but moves to another token at step 2, the
    # revealed token's own probability falls to 0.1.  Position 2: same token, confidence dips below tau
    # at step 1.  Position 3: never clears tau.
    conf = np.array([[0.9, 0.8, 0.7, 0.3],
                     [0.9, 0.8, 0.4, 0.3],
                     [0.9, 0.85, 0.7, 0.3]], np.float32)
    token = np.array([[5, 6, 7, 8],
                      [5, 6, 7, 8],
                      [5, 9, 7, 8]], np.int32)
    conf_first = np.array([[0.9, 0.8, 0.7, 0.3],
                           [0.9, 0.8, 0.4, 0.3],
                           [0.9, 0.1, 0.7, 0.3]], np.float32)
    want = {0: [0, 0, 1, 0],      # updated top-1 probability, all steps
            1: [0, 0, 0, 0],      # updated top-1 probability, last step
            2: [0, 1, 1, 0],      # probability of the revealed token, all steps
            3: [0, 1, 0, 0]}      # the argmax left the revealed token
    for policy, remask in want.items():
        s = oracle.select(conf, token, None, 1, 4, oracle.DYNAMIC_REMASK, tau=0.5, remask_policy=policy,
                          conf_first=conf_first)
        assert list(s.reveal_mask) == [1, 1, 1, 0], policy
        assert list(s.remask_mask) == remask, policy
        assert list(s.out_token) == [5 if not remask[0] else -1, 6 if not remask[1] else -1,
                                     7 if not remask[2] else -1, -1], policy


def test_remask_by_the_revealed_token_relations_between_the_policies():
    rng = np.random.default_rng(21)
    K, B, L = 3, 8, 16
    mask, ri, conf, token = random_stats(rng, K, B, L)
    M = ri.size
    # tokens move away from the step-0 token in some row-steps; where they stay, the revealed token's
    # probability is the top probability, where they move it is strictly smaller
    moved = rng.random((K + 1, M)) < 0.3
    moved[0] = False
    token = np.where(moved, token[0][None, :] + 1, token[0][None, :]).astype(np.int32)
    conf_first = np.where(moved, conf * rng.random((K + 1, M)).astype(np.float32) * 0.9, conf).astype(np.float32)
    for tau in (0.3, 0.5, 0.7):
        kw = dict(tau=tau, ensure_progress=False)
        p0 = oracle.select(conf, token, ri, B, L, oracle.DYNAMIC_REMASK, remask_policy=0, **kw)
        p2 = oracle.select(conf, token, ri, B, L, oracle.DYNAMIC_REMASK, remask_policy=2, conf_first=conf_first, **kw)
        p3 = oracle.select(conf, token, ri, B, L, oracle.DYNAMIC_REMASK, remask_policy=3, **kw)
        assert np.array_equal(p0.reveal_mask, p2.reveal_mask) and np.array_equal(p0.reveal_mask, p3.reveal_mask)
        # the revealed token's probability never exceeds the top probability: policy 2 revokes a superset
        assert np.all(p2.remask_mask >= p0.remask_mask)
        # policy 3 from its definition: revealed and moved at some step
        dense_moved = np.zeros(B * L, bool)
        dense_moved[ri] = moved[1:].any(axis=0)
        assert np.array_equal(p3.remask_mask.astype(bool), p3.reveal_mask.astype(bool) & dense_moved)
        # policy 2 from its definition
        dense_min = np.full(B * L, 2.0, np.float32)
        dense_min[ri] = conf_first[1:].min(axis=0)
        assert np.array_equal(p2.remask_mask.astype(bool), p2.reveal_mask.astype(bool) & (dense_min < np.float32(tau)))
    # with tokens that never move and conf_first = conf, policy 2 is policy 0 and policy 3 revokes nothing
    still = np.repeat(token[:1], K + 1, axis=0)
    a = oracle.select(conf, still, ri, B, L, oracle.DYNAMIC_REMASK, tau=0.5, remask_policy=0)
    b = oracle.select(conf, still, ri, B, L, oracle.DYNAMIC_REMASK, tau=0.5, remask_policy=2, conf_first=conf)
    c = oracle.select(conf, still, ri, B, L, oracle.DYNAMIC_REMASK, tau=0.5, remask_policy=3)
    assert np.array_equal(a.remask_mask, b.remask_mask) and not c.remask_mask.any()
