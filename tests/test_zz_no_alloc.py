"""The allocation-free selection entry point, `mrp_reveal_remask_noalloc`.

It serves callers that cannot allocate device memory (an engine whose pool owns the GPU, a
plugin inside a foreign CUDA context, a path where cudaMalloc is forbidden) and so cannot
give `mrp_create` a workspace: its scratch is a fixed array inside the library.  The checks:
its outputs equal the CPU oracle's selection and those of the context-based
`mrp_reveal_remask` on several calls in a row (later ones on smaller problems, so anything an
earlier call left in the shared array would show), and sizes beyond the built-in capacity are
refused on the host.

This file sorts last on purpose: a run that stops at the first failure has by then run
every other test.
"""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from paper_2605_18817_b200 import binding, harness, synth

DEV = "cuda:0"
NAMES = ("reveal_mask", "remask_mask", "out_token", "step_of", "draft_pos", "draft_tok", "draft_len")


def _case(seed, K, B, L, mask_prob):
    rng = np.random.default_rng(seed)
    mask = rng.random((B, L)) < mask_prob
    mask[:, 0] |= ~mask.any(axis=1)
    ri = np.flatnonzero(mask.reshape(-1)).astype(np.int32)
    rng.shuffle(ri)
    conf = rng.random((K + 1, ri.size)).astype(np.float32)
    token = rng.integers(0, 50000, (K + 1, ri.size)).astype(np.int32)
    return ri, conf, token


def _both(ctx, ri, conf, token, B, L, mode, **kw):
    K, M = conf.shape[0] - 1, conf.shape[1]
    Kd = K * kw.get("r_draft", 1)
    c, t, r = (torch.from_numpy(a).to(DEV) for a in (conf, token, ri))
    ref = harness.alloc_select_out(B, L, Kd, DEV)
    harness.select(ctx, c, t, r, M, K, B, L, mode, ref, **kw)
    got = harness.alloc_select_out(B, L, Kd, DEV)
    for n in NAMES:                       # poison: every element must be written by the call
        getattr(got, n).fill_(77)
    binding.mrp_reveal_remask_noalloc(c, t, r, M, K, B, L, mode, **kw,
                                      **{n: getattr(got, n) for n in NAMES})
    torch.cuda.synchronize()
    omode = oracle.STATIC if mode == binding.MRP_SELECT_STATIC else oracle.DYNAMIC_REMASK
    want = oracle.select(conf, token, ri, B, L, omode, **kw)
    for n in NAMES:
        w = getattr(want, n)
        assert np.array_equal(getattr(got, n).cpu().numpy().reshape(w.shape), w), n
        assert torch.equal(getattr(got, n), getattr(ref, n)), n


@pytest.mark.gpu
def test_noalloc_selection_matches_context_entry_point_twice_in_a_row():
    w = synth.make_weights(16, 16, 32, 0, "f32", 1)
    heads, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(16, 16, 32, heads, w_lm, max_rows=4, max_seqs=2048, block_len=128)
    # first call: the full capacity (B * L = 65536 positions), densely masked; B * M > 2^22, the size
    # from which the context entry point goes through a dense position map as well
    ri, conf, token = _case(11, 2, 2048, 32, 0.9)
    assert 2048 * ri.size > (1 << 22)
    _both(ctx, ri, conf, token, 2048, 32, binding.MRP_SELECT_DYNAMIC_REMASK, tau=0.5)
    # second call: fewer, sparsely masked positions over the same part of the shared array
    ri, conf, token = _case(12, 3, 40, 16, 0.3)
    _both(ctx, ri, conf, token, 40, 16, binding.MRP_SELECT_STATIC, r_reveal=2, r_draft=1)
    ri, conf, token = _case(13, 1, 7, 100, 0.5)
    _both(ctx, ri, conf, token, 7, 100, binding.MRP_SELECT_DYNAMIC_REMASK, tau=0.7, use_cap=True,
          remask_policy=1)
    binding.mrp_destroy(ctx)


def test_noalloc_selection_refuses_sizes_beyond_its_capacity_on_the_host():
    lib = binding.lib
    p = binding.mrp_select_params(0, 0.5, 1, 1, 0, 0, 1)
    o = binding.mrp_select_out(8, 8, 8, 8, 8, 8, 8, None)    # never dereferenced: refused first
    B, L = binding.MRP_NOALLOC_MAX_POSITIONS // 32 + 1, 32
    rc = lib.mrp_reveal_remask_noalloc(None, None, None, 0, 1, B, L, ctypes.byref(p),
                                       ctypes.byref(o), None)
    assert rc == binding.MRP_ERR_CAPACITY
    assert b"capacity" in lib.mrp_status_string(rc)
    assert lib.mrp_reveal_remask_noalloc(None, None, None, 0, 1, 1, 2000, ctypes.byref(p),
                                         ctypes.byref(o), None) == 1
