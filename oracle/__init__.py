"""CPU oracle for the MRP drafting step -- TEST INFRASTRUCTURE ONLY.

Thin ctypes access to ``mrp_oracle.c`` (plain C, fp64 arithmetic, OpenMP over independent
outputs).  Only tests, the smoke check and the benchmark's ``cpu_baseline`` / reference arm
may import this package; the product path never does.  Nothing here touches CUDA.

The functions mirror the paper's steps (Algorithms 2-4): ``draft`` runs the head chain and
the shared LM head and returns per-step softmax statistics, ``select`` applies the static /
dynamic reveal rules and the remask rule, ``verify`` computes accepted draft prefixes, ``commit``
applies the outcome to the block state (x_t -> x_{t-1}) and lists the positions still masked.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "mrp_oracle.c")
_LIB = os.path.join(_HERE, "libmrp_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile ``mrp_oracle.c`` into ``libmrp_oracle.so`` next to it (gcc, OpenMP)."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp.%d" % os.getpid()
    cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
    subprocess.run(cmd, check=True)
    os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.mrp_oracle_num_threads.restype = ctypes.c_int
        _lib.mrp_oracle_cap.restype = ctypes.c_int
        _lib.mrp_oracle_cap.argtypes = [ctypes.c_int, ctypes.c_int]
        _lib.mrp_oracle_draft.restype = ctypes.c_int
        _lib.mrp_oracle_draft_from_hidden.restype = ctypes.c_int
        _lib.mrp_oracle_draft_kl.restype = ctypes.c_int
        _lib.mrp_oracle_module.restype = ctypes.c_int
        _lib.mrp_oracle_module_prefix.restype = ctypes.c_int
        _lib.mrp_oracle_select.restype = ctypes.c_int
        _lib.mrp_oracle_verify.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().mrp_oracle_num_threads())


def cap(n_masked: int, L: int) -> int:
    """Max-accept cap m = min(max(floor(0.7 n), 5), L) (Sec. 4.4)."""
    return int(_load().mrp_oracle_cap(int(n_masked), int(L)))


def _f32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float32))


def _i32(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.int32))


def _p(a, ct):
    return a.ctypes.data_as(ctypes.POINTER(ct)) if a is not None else None


@dataclass
class DraftResult:
    conf: np.ndarray      # [(K+1), M] float64
    lse: np.ndarray       # [(K+1), M] float64
    token: np.ndarray     # [(K+1), M] int32
    margin: np.ndarray    # [(K+1), M] float64, top-1 minus top-2 logit
    logits: np.ndarray | None   # [K, M, V] float64
    hidden: np.ndarray | None   # [M, d] float64
    conf_first: np.ndarray | None = None   # [(K+1), M] float64: probability under step k of the step-0 argmax token


def draft(hidden, logits0, heads, w_lm, K=None, row_index=None, eps=1e-6,
          want_logits=False, want_hidden=False, final_gamma=None) -> DraftResult:
    """Head chain + shared LM head + softmax statistics (Algorithm 2, inner loop).

    ``heads`` is a sequence of dicts with float32-representable arrays ``gamma`` [d],
    ``w_gate`` [F,d], ``w_up`` [F,d], ``w_down`` [d,F]; ``hidden`` [rows,d]; ``logits0``
    [rows,V]; ``w_lm`` [V,d]; ``row_index`` selects the masked rows (None = all rows).
    ``logits0=None``: the backbone logits are computed from the hidden states with the shared
    LM head, ``l_0 = W_lm n_0``, ``n_0 = h_0`` or ``RMSNorm(h_0) * final_gamma``.
    """
    lib = _load()
    hidden = _f32(hidden)
    from_hidden = logits0 is None
    w_lm = _f32(w_lm)
    n_rows, d = hidden.shape
    V = w_lm.shape[0]
    assert w_lm.shape[1] == d
    if not from_hidden:
        assert final_gamma is None
        logits0 = _f32(logits0)
        assert logits0.shape == (n_rows, V)
    fg = None
    if final_gamma is not None:
        fg = _f32(final_gamma)
        assert fg.shape == (d,)
    K = len(heads) if K is None else int(K)
    assert 0 <= K <= len(heads)
    ri = None
    M = n_rows
    if row_index is not None:
        ri = _i32(row_index)
        M = ri.shape[0]
        assert M == 0 or (ri.min() >= 0 and ri.max() < n_rows)
    keep = []
    F = heads[0]["w_gate"].shape[0] if len(heads) else 1
    PtrArr = ctypes.POINTER(ctypes.c_float) * max(K, 1)
    arrs = {}
    for name, shape in (("gamma", (d,)), ("w_gate", (F, d)), ("w_up", (F, d)), ("w_down", (d, F))):
        lst = []
        for k in range(K):
            a = _f32(heads[k][name])
            assert a.shape == shape, (name, a.shape, shape)
            keep.append(a)
            lst.append(_p(a, ctypes.c_float))
        arrs[name] = PtrArr(*lst) if K else PtrArr()
    conf = np.zeros((K + 1, M), np.float64)
    lse = np.zeros((K + 1, M), np.float64)
    margin = np.zeros((K + 1, M), np.float64)
    token = np.zeros((K + 1, M), np.int32)
    logits = np.zeros((K, M, V), np.float64) if want_logits else None
    hid = np.zeros((M, d), np.float64) if want_hidden else None
    conf_first = np.zeros((K + 1, M), np.float64)
    fn = lib.mrp_oracle_draft_from_hidden if from_hidden else lib.mrp_oracle_draft
    rc = fn(
        ctypes.c_int(d), ctypes.c_int(F), ctypes.c_int(V), ctypes.c_int(K), ctypes.c_int(M),
        ctypes.c_double(eps), _p(hidden, ctypes.c_float),
        _p(fg, ctypes.c_float) if from_hidden else _p(logits0, ctypes.c_float),
        _p(ri, ctypes.c_int32), arrs["gamma"], arrs["w_gate"], arrs["w_up"], arrs["w_down"],
        _p(w_lm, ctypes.c_float), _p(conf, ctypes.c_double), _p(lse, ctypes.c_double),
        _p(token, ctypes.c_int32), _p(margin, ctypes.c_double), _p(logits, ctypes.c_double),
        _p(hid, ctypes.c_double), _p(conf_first, ctypes.c_double))
    if rc != 0:
        raise RuntimeError("mrp_oracle_draft failed (%d)" % rc)
    return DraftResult(conf, lse, token, margin, logits, hid, conf_first)


def draft_kl(hidden, logits0, teacher, heads, w_lm, K=None, row_index=None, eps=1e-6):
    """The drafting pass with the training objective (Algorithm 1, Eq. (3)): ``teacher`` [K, M, V]
    are the backbone's logits of every unrolled step's revealed sequence at the masked rows; returns
    (DraftResult, kl [K, M]) with kl = KL(softmax(teacher_k) || softmax(l_k))."""
    lib = _load()
    hidden, logits0, w_lm, teacher = _f32(hidden), _f32(logits0), _f32(w_lm), _f32(teacher)
    n_rows, d = hidden.shape
    V = w_lm.shape[0]
    K = len(heads) if K is None else int(K)
    ri, M = None, n_rows
    if row_index is not None:
        ri = _i32(row_index)
        M = ri.shape[0]
        assert M == 0 or (ri.min() >= 0 and ri.max() < n_rows)
    assert teacher.shape == (K, M, V) and logits0.shape == (n_rows, V) and K >= 1
    F = heads[0]["w_gate"].shape[0]
    PtrArr = ctypes.POINTER(ctypes.c_float) * K
    keep, arrs = [], {}
    for name, shape in (("gamma", (d,)), ("w_gate", (F, d)), ("w_up", (F, d)), ("w_down", (d, F))):
        lst = []
        for k in range(K):
            a = _f32(heads[k][name])
            assert a.shape == shape
            keep.append(a)
            lst.append(_p(a, ctypes.c_float))
        arrs[name] = PtrArr(*lst)
    conf, lse, margin = (np.zeros((K + 1, M), np.float64) for _ in range(3))
    token = np.zeros((K + 1, M), np.int32)
    kl = np.zeros((K, M), np.float64)
    rc = lib.mrp_oracle_draft_kl(
        ctypes.c_int(d), ctypes.c_int(F), ctypes.c_int(V), ctypes.c_int(K), ctypes.c_int(M),
        ctypes.c_double(eps), _p(hidden, ctypes.c_float), _p(logits0, ctypes.c_float), _p(ri, ctypes.c_int32),
        arrs["gamma"], arrs["w_gate"], arrs["w_up"], arrs["w_down"], _p(w_lm, ctypes.c_float),
        _p(teacher, ctypes.c_float), _p(conf, ctypes.c_double), _p(lse, ctypes.c_double),
        _p(token, ctypes.c_int32), _p(margin, ctypes.c_double), _p(kl, ctypes.c_double))
    if rc != 0:
        raise RuntimeError("mrp_oracle_draft_kl failed (%d)" % rc)
    return DraftResult(conf, lse, token, margin, None, None), kl


MODULE_LAYER_KEYS = ("g_attn", "w_q", "w_k", "w_v", "w_o", "g_mlp", "w_gate", "w_up", "w_down")


def module(hidden, tokens, B, L, emb, w_proj, layers, w_lm, n_attn_heads, mask_token, row_index=None, eps=1e-6,
           prefix=None, want_kv=False):
    """One application of the token-conditioned MRP module g(x_t, h) (Sec. 3.2; Algorithm 2) to the L
    positions of each of B blocks: returns (delta_h [B*L, d], delta_l [M, V]) in float64.  ``layers`` is a
    sequence of dicts with the arrays named in MODULE_LAYER_KEYS; ``tokens`` [B*L] with -1 = masked.
    ``prefix`` = (k, v, length) gives the clean prefix of Fig. 1(c): k, v are sequences of D arrays
    [B, cap, d] (the keys and values of the prefix positions per layer), length [B] the rows in use per
    sequence.  With ``want_kv`` the result gains (k, v): per layer the [B*L, d] float64 keys and values of
    the block's own positions."""
    lib = _load()
    hidden, emb, w_proj, w_lm = _f32(hidden), _f32(emb), _f32(w_proj), _f32(w_lm)
    tokens = _i32(tokens)
    n, d = hidden.shape
    assert n == B * L and tokens.shape == (n,) and w_proj.shape == (d, 2 * d) and emb.shape[1] == d
    V = w_lm.shape[0]
    D = len(layers)
    F = layers[0]["w_gate"].shape[0] if D else 1
    shapes = dict(g_attn=(d,), w_q=(d, d), w_k=(d, d), w_v=(d, d), w_o=(d, d), g_mlp=(d,), w_gate=(F, d), w_up=(F, d),
                  w_down=(d, F))
    PtrArr = ctypes.POINTER(ctypes.c_float) * max(D, 1)
    keep, arrs = [], {}
    for name in MODULE_LAYER_KEYS:
        lst = []
        for lay in layers:
            a = _f32(lay[name])
            assert a.shape == shapes[name], (name, a.shape)
            keep.append(a)
            lst.append(_p(a, ctypes.c_float))
        arrs[name] = PtrArr(*lst) if D else PtrArr()
    ri, M = None, 0
    if row_index is not None:
        ri = _i32(row_index)
        M = ri.shape[0]
    delta_h = np.zeros((n, d), np.float64)
    delta_l = np.zeros((M, V), np.float64)
    pk = pv = plen = None
    cap = 0
    if prefix is not None:
        ks, vs, length = prefix
        assert len(ks) == D and len(vs) == D
        plen = _i32(length)
        assert plen.shape == (B,)
        lk, lv = [], []
        for a, b in zip(ks, vs):
            a, b = _f32(a), _f32(b)
            assert a.ndim == 3 and a.shape == b.shape and a.shape[0] == B and a.shape[2] == d
            cap = a.shape[1]
            keep += [a, b]
            lk.append(_p(a, ctypes.c_float))
            lv.append(_p(b, ctypes.c_float))
        pk, pv = PtrArr(*lk), PtrArr(*lv)
    ko = vo = None
    k_out = v_out = None
    if want_kv:
        DArr = ctypes.POINTER(ctypes.c_double) * max(D, 1)
        k_out = [np.zeros((n, d), np.float64) for _ in range(D)]
        v_out = [np.zeros((n, d), np.float64) for _ in range(D)]
        ko = DArr(*[_p(a, ctypes.c_double) for a in k_out])
        vo = DArr(*[_p(a, ctypes.c_double) for a in v_out])
    rc = lib.mrp_oracle_module_prefix(
        ctypes.c_int(d), ctypes.c_int(F), ctypes.c_int(V), ctypes.c_int(D), ctypes.c_int(n_attn_heads), ctypes.c_int(B),
        ctypes.c_int(L), ctypes.c_int(mask_token), ctypes.c_double(eps), _p(hidden, ctypes.c_float),
        _p(tokens, ctypes.c_int32), _p(emb, ctypes.c_float), _p(w_proj, ctypes.c_float),
        *[arrs[k] for k in MODULE_LAYER_KEYS], _p(w_lm, ctypes.c_float), _p(ri, ctypes.c_int32), ctypes.c_int(M),
        _p(delta_h, ctypes.c_double), _p(delta_l, ctypes.c_double), pk, pv, _p(plen, ctypes.c_int32), ctypes.c_int(cap),
        ko, vo)
    if rc != 0:
        raise RuntimeError("mrp_oracle_module_prefix failed (%d)" % rc)
    if want_kv:
        return delta_h, delta_l, k_out, v_out
    return delta_h, delta_l


def kl_rows(teacher, logits):
    """KL(softmax(teacher[m]) || softmax(logits[m])) per row, by the definition of Eq. (3), in float64."""
    t, l = np.asarray(teacher, np.float64), np.asarray(logits, np.float64)
    lt = t - (t.max(axis=1, keepdims=True) + np.log(np.exp(t - t.max(axis=1, keepdims=True)).sum(axis=1, keepdims=True)))
    ll = l - (l.max(axis=1, keepdims=True) + np.log(np.exp(l - l.max(axis=1, keepdims=True)).sum(axis=1, keepdims=True)))
    return (np.exp(lt) * (lt - ll)).sum(axis=1)


def stats(logits):
    """(conf, lse, token, margin) of logit rows [M, V] by the definitions of Sec. 2, in float64."""
    l = np.asarray(logits, np.float64)
    mx = l.max(axis=1)
    tok = l.argmax(axis=1).astype(np.int32)
    lse = mx + np.log(np.exp(l - mx[:, None]).sum(axis=1))
    second = np.sort(l, axis=1)[:, -2] if l.shape[1] > 1 else np.full(l.shape[0], -np.inf)
    return np.exp(mx - lse), lse, tok, mx - second


@dataclass
class SelectResult:
    reveal_mask: np.ndarray   # [B*L] int8
    remask_mask: np.ndarray   # [B*L] int8
    out_token: np.ndarray     # [B*L] int32
    step_of: np.ndarray       # [B*L] int8
    draft_pos: np.ndarray     # [B, Kd] int32
    draft_tok: np.ndarray     # [B, Kd] int32
    draft_len: np.ndarray     # [B] int32


STATIC = 0
DYNAMIC_REMASK = 1


def select(conf, token, row_index, B, L, mode, tau=0.9, r_reveal=1, r_draft=1,
           use_cap=False, remask_policy=0, ensure_progress=True, conf_first=None) -> SelectResult:
    """Static top-r reveal/draft or dynamic threshold reveal + remask (Algorithms 2-4).
    ``remask_policy``: 0 = min over steps 1..K of the updated confidence, 1 = step K only,
    2 = min over steps of ``conf_first`` (probability of the token revealed at step 0),
    3 = revoke when the argmax left that token at any step."""
    lib = _load()
    conf = _f32(conf)
    token = _i32(token)
    cf = None
    if conf_first is not None:
        cf = _f32(conf_first)
        assert cf.shape == conf.shape
    Kp1, M = conf.shape
    assert token.shape == conf.shape
    K = Kp1 - 1
    ri = _i32(row_index) if row_index is not None else None
    Kd = K * max(int(r_draft), 0)
    out = SelectResult(
        np.zeros(B * L, np.int8), np.zeros(B * L, np.int8), np.zeros(B * L, np.int32),
        np.zeros(B * L, np.int8), np.zeros((B, Kd), np.int32), np.zeros((B, Kd), np.int32),
        np.zeros(B, np.int32))
    rc = lib.mrp_oracle_select(
        _p(conf, ctypes.c_float), _p(token, ctypes.c_int32), _p(ri, ctypes.c_int32),
        ctypes.c_int(M), ctypes.c_int(K), ctypes.c_int(B), ctypes.c_int(L), ctypes.c_int(mode),
        ctypes.c_float(tau), ctypes.c_int(r_reveal), ctypes.c_int(r_draft),
        ctypes.c_int(int(use_cap)), ctypes.c_int(int(remask_policy)),
        ctypes.c_int(int(ensure_progress)),
        _p(out.reveal_mask, ctypes.c_int8), _p(out.remask_mask, ctypes.c_int8),
        _p(out.out_token, ctypes.c_int32), _p(out.step_of, ctypes.c_int8),
        _p(out.draft_pos, ctypes.c_int32), _p(out.draft_tok, ctypes.c_int32),
        _p(out.draft_len, ctypes.c_int32), _p(cf, ctypes.c_float))
    if rc != 0:
        raise RuntimeError("mrp_oracle_select failed (%d)" % rc)
    return out


def verify(draft_tok, verify_tok, draft_len, positionwise=False):
    """Accepted-prefix length of drafted tokens against backbone tokens (Algorithm 3)."""
    lib = _load()
    draft_tok = _i32(draft_tok)
    verify_tok = _i32(verify_tok)
    draft_len = _i32(draft_len)
    B, Kd = draft_tok.shape
    assert verify_tok.shape == (B, Kd) and draft_len.shape == (B,)
    accept_len = np.zeros(B, np.int32)
    accept_mask = np.zeros((B, Kd), np.int8)
    rc = lib.mrp_oracle_verify(
        _p(draft_tok, ctypes.c_int32), _p(verify_tok, ctypes.c_int32),
        _p(draft_len, ctypes.c_int32), ctypes.c_int(B), ctypes.c_int(Kd),
        ctypes.c_int(int(positionwise)), _p(accept_len, ctypes.c_int32),
        _p(accept_mask, ctypes.c_int8))
    if rc != 0:
        raise RuntimeError("mrp_oracle_verify failed (%d)" % rc)
    return accept_len, accept_mask


@dataclass
class CommitResult:
    tokens: np.ndarray        # [B*L] int32, -1 = still masked
    row_index: np.ndarray     # [n_masked] int32, dense positions still masked, ascending
    block_masked: np.ndarray  # [B] int32


def commit(tokens, sel: SelectResult, B, L, accept_mask=None) -> CommitResult:
    """One transition x_t -> x_{t-1} of the block state (the last lines of Algorithms 2-4).

    ``tokens`` [B*L] holds the committed token of every position, -1 while it is masked.
    ``accept_mask=None``: every position the selection took is unmasked with its token --
    the reveals of all steps in direct decoding (Algorithm 2), the members of R that survived
    remasking in the dynamic regime (Algorithm 4).  With ``accept_mask`` [B, Kd] (speculative
    decoding, Algorithm 3): the step-0 reveals are unmasked, a drafted position only where the
    backbone accepted the draft; rejected drafts stay masked.  Plain loops, no arithmetic.
    """
    tokens = np.array(tokens, dtype=np.int32).reshape(B * L).copy()
    for p in range(B * L):
        if tokens[p] >= 0:
            continue
        if accept_mask is None:
            if sel.out_token[p] >= 0:
                tokens[p] = sel.out_token[p]
        elif sel.step_of[p] == 0:
            tokens[p] = sel.out_token[p]
    if accept_mask is not None:
        accept_mask = np.asarray(accept_mask).reshape(B, -1)
        for b in range(B):
            for s in range(accept_mask.shape[1]):
                if accept_mask[b, s] and sel.draft_pos[b, s] >= 0:
                    p = b * L + int(sel.draft_pos[b, s])
                    if tokens[p] < 0:
                        tokens[p] = sel.draft_tok[b, s]
    row_index = np.array([p for p in range(B * L) if tokens[p] < 0], dtype=np.int32)
    block_masked = np.array([int(np.sum(tokens[b * L:(b + 1) * L] < 0)) for b in range(B)], dtype=np.int32)
    return CommitResult(tokens, row_index, block_masked)
