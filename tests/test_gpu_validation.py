"""Caller-provided row indices are checked on the device before they are used as an address.

An entry of ``row_index`` outside its array raises MRP_DEV_BAD_INDEX (in the call's optional
status word and in the context's own) and the row is treated as absent: nothing is read or
written through it.  In selection a position named twice raises the bit as well and the row
listed last keeps the position.  The checks here: the bit, the results of the remaining rows
against the oracle, untouched guard bands around every output and around the workspace, and a
context that goes on working.

Every bad index used here stays within a few rows of its array, and the arrays that are indexed
sit inside larger allocations, so that even a missing guard would have read or written valid
memory: no case of this file can fault the GPU.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_18817_b200 import binding, harness, synth
from test_gpu_parity import DEV, TOL

pytestmark = pytest.mark.gpu

BAND = 4096          # guard elements on each side of a banded tensor


class Banded:
    """A tensor placed in the middle of a larger allocation whose margins hold a sentinel."""

    def __init__(self, shape, dtype, sentinel, fill=None):
        n = int(np.prod(shape))
        self.flat = torch.full((n + 2 * BAND,), sentinel, dtype=dtype, device=DEV)
        self.t = self.flat[BAND:BAND + n].view(shape)
        if fill is not None:
            self.t.fill_(fill)
        self.sentinel = sentinel
        self.n = n

    def intact(self) -> bool:
        lo, hi = self.flat[:BAND], self.flat[BAND + self.n:]
        return bool((lo == self.sentinel).all().item()) and bool((hi == self.sentinel).all().item())


def banded_draft_out(M, K):
    conf, lse = Banded((K + 1, M), torch.float32, -12345.0), Banded((K + 1, M), torch.float32, -12345.0)
    tok = Banded((K + 1, M), torch.int32, -77)
    out = harness.DraftOut(conf.t, lse.t, tok.t, None, None, None, torch.zeros(1, device=DEV, dtype=torch.int32))
    return out, (conf, lse, tok)


def padded_inputs(inp, dtype):
    """hidden / logits0 with spare rows before and after, so that an index a few rows out of range
    would still land in memory of this test."""
    pad = 8
    n, d = inp.hidden.shape
    V = inp.logits0.shape[1]
    hid = torch.zeros((n + 2 * pad, d), device=DEV, dtype=torch.bfloat16 if dtype == "bf16" else torch.float32)
    hid[pad:pad + n] = harness.to_device(inp.hidden, dtype, DEV)
    l0 = torch.full((n + 2 * pad, V), 1e30, device=DEV)          # would wreck the statistics if it were read
    l0[pad:pad + n] = torch.from_numpy(inp.logits0).to(DEV)
    return hid[pad:pad + n], l0[pad:pad + n]


@pytest.mark.parametrize("dtype,flags,d,F,V,B,L,K", [
    ("f32", 0, 72, 136, 1000, 5, 3, 2),                                 # CUDA-core kernels
    ("bf16", 0, 256, 512, 4096, 2, 4, 2),                               # few-row tensor-core kernels
    ("bf16", 0, 128, 256, 2048, 30, 4, 2),                              # row-major LM head (fp16 operand + top fix)
    ("bf16", binding.MRP_FLAG_EXACT_OPERANDS, 128, 256, 2048, 30, 4, 2),
])
@pytest.mark.parametrize("from_hidden", [False, True])
def test_draft_skips_row_indices_outside_the_input_arrays(dtype, flags, d, F, V, B, L, K, from_hidden):
    w = synth.make_weights(d, F, V, K, dtype, 21, head_std=0.05)
    inp = synth.make_inputs(w, B, L, 21, 1.0, 4.0)
    heads, w_lm = harness.upload_weights(w, DEV)
    n_rows = B * L
    ctx = binding.mrp_create(d, F, V, heads, w_lm, max_rows=n_rows, max_seqs=B, block_len=L, flags=flags,
                             guard_bytes=65536)
    hid, l0 = padded_inputs(inp, dtype)
    ri = np.arange(n_rows, dtype=np.int32)[::-1].copy()
    bad_at = {1: n_rows, 4: -1, n_rows - 2: n_rows + 3}
    for m, v in bad_at.items():
        ri[m] = v
    good = np.array([m for m in range(n_rows) if m not in bad_at])
    out, bands = banded_draft_out(n_rows, K)
    ri_t = torch.from_numpy(ri).to(DEV)
    if from_hidden:
        harness.draft_from_hidden(ctx, hid, None, ri_t, n_rows, K, out)
    else:
        harness.draft(ctx, hid, l0, ri_t, n_rows, K, out)
    torch.cuda.synchronize()
    assert int(out.status.item()) & binding.MRP_DEV_BAD_INDEX
    assert binding.mrp_fetch_status(ctx, clear=True) & binding.MRP_DEV_BAD_INDEX
    assert binding.mrp_fetch_status(ctx) == 0                         # the fetch above cleared the word
    assert all(b.intact() for b in bands) and binding.workspace_guards_intact(ctx)
    ref = oracle.draft(inp.hidden, None if from_hidden else inp.logits0, w.heads, w.w_lm, K=K, row_index=ri[good])
    tol = TOL[dtype]
    assert np.abs(out.conf.cpu().numpy()[:, good] - ref.conf).max() <= tol
    assert np.abs(out.lse.cpu().numpy()[:, good] - ref.lse).max() <= tol
    clear = ref.margin > 1e-2
    assert np.array_equal(out.token.cpu().numpy()[:, good][clear], ref.token[clear])
    # the skipped rows are those of an all-zero hidden state and logit row: finite and defined
    assert torch.isfinite(out.lse).all() and (out.token >= 0).all() and (out.token < V).all()
    # a smaller input array, declared through mrp_set_input_rows, moves the bound
    binding.mrp_set_input_rows(ctx, n_rows - 1)
    ok_ri = torch.arange(n_rows, device=DEV, dtype=torch.int32)
    out2, bands2 = banded_draft_out(n_rows, K)
    harness.draft(ctx, hid, l0, ok_ri, n_rows, K, out2)
    torch.cuda.synchronize()
    assert int(out2.status.item()) & binding.MRP_DEV_BAD_INDEX       # the last row is now out of range
    with pytest.raises(binding.MrpError):
        harness.draft(ctx, hid, l0, None, n_rows, K, out2)             # rows 0..M-1 do not all exist
    with pytest.raises(binding.MrpError):
        binding.mrp_set_input_rows(ctx, n_rows + 1)
    binding.mrp_set_input_rows(ctx, n_rows)
    # and the context goes on working
    binding.mrp_fetch_status(ctx, clear=True)
    out3, bands3 = banded_draft_out(n_rows, K)
    harness.draft(ctx, hid, l0, ok_ri, n_rows, K, out3)
    torch.cuda.synchronize()
    assert int(out3.status.item()) == 0 and binding.mrp_fetch_status(ctx) == 0
    ref3 = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=K)
    assert np.abs(out3.conf.cpu().numpy() - ref3.conf).max() <= tol
    assert all(b.intact() for b in bands2 + bands3) and binding.workspace_guards_intact(ctx)
    binding.mrp_destroy(ctx)


def banded_select_out(B, L, Kd):
    b = dict(
        reveal_mask=Banded((B * L,), torch.int8, 55), remask_mask=Banded((B * L,), torch.int8, 55),
        out_token=Banded((B * L,), torch.int32, -99), step_of=Banded((B * L,), torch.int8, 55),
        draft_pos=Banded((B, Kd), torch.int32, -99), draft_tok=Banded((B, Kd), torch.int32, -99),
        draft_len=Banded((B,), torch.int32, -99))
    return harness.SelectOut(**{k: v.t for k, v in b.items()}), list(b.values())


def surviving_rows(ri, n_pos):
    """Rows the selection keeps: position in range, and not named again by a later row."""
    last = {}
    for m, p in enumerate(ri):
        if 0 <= p < n_pos:
            last[int(p)] = m
    return np.array(sorted(last.values()), dtype=np.int64)


@pytest.mark.parametrize("B,L,mask_prob,path", [
    (9, 32, 0.6, "few rows: every block scans the row list"),
    (2048, 32, 0.2, "many rows: scatter into the dense map"),
    (2048, 32, 0.2, "allocation-free entry point"),
])
def test_selection_skips_bad_positions_and_resolves_duplicates(B, L, mask_prob, path):
    rng = np.random.default_rng(B + L)
    K = 2
    mask = rng.random((B, L)) < mask_prob
    ri = np.flatnonzero(mask.reshape(-1)).astype(np.int32)
    rng.shuffle(ri)
    M = ri.size
    if path.startswith("many"):
        assert B * M > (1 << 22)                     # what sends the context entry point to the dense map
    n_pos = B * L
    # out of range on both sides, and duplicates of positions listed elsewhere
    ri[3], ri[M // 2], ri[M - 1] = -2, n_pos, n_pos + 5
    ri[10], ri[11] = ri[40], ri[41]
    ri[M - 7] = ri[5]
    conf = rng.random((K + 1, M)).astype(np.float32)
    token = rng.integers(0, 1000, (K + 1, M)).astype(np.int32)
    keep = surviving_rows(ri, n_pos)
    assert keep.size == M - 6

    w = synth.make_weights(16, 16, 32, 0, "f32", 1)
    heads, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(16, 16, 32, heads, w_lm, max_rows=4, max_seqs=B, block_len=L, guard_bytes=65536)
    c, t, r = (torch.from_numpy(a).to(DEV) for a in (conf, token, ri))
    for mode, omode, kw in ((binding.MRP_SELECT_STATIC, oracle.STATIC, dict(r_reveal=2, r_draft=1)),
                            (binding.MRP_SELECT_DYNAMIC_REMASK, oracle.DYNAMIC_REMASK, dict(tau=0.5, use_cap=True))):
        sel, bands = banded_select_out(B, L, K)
        st = torch.zeros(1, device=DEV, dtype=torch.int32)
        args = dict(reveal_mask=sel.reveal_mask, remask_mask=sel.remask_mask, out_token=sel.out_token,
                    step_of=sel.step_of, draft_pos=sel.draft_pos, draft_tok=sel.draft_tok, draft_len=sel.draft_len,
                    status=st, **kw)
        if path.startswith("allocation-free"):
            binding.mrp_reveal_remask_noalloc(c, t, r, M, K, B, L, mode, **args)
        else:
            binding.mrp_reveal_remask(ctx, c, t, r, M, K, B, L, mode, **args)
        torch.cuda.synchronize()
        assert int(st.item()) == binding.MRP_DEV_BAD_INDEX
        if not path.startswith("allocation-free"):
            assert binding.mrp_fetch_status(ctx, clear=True) == binding.MRP_DEV_BAD_INDEX
        assert all(b.intact() for b in bands) and binding.workspace_guards_intact(ctx)
        o = oracle.select(conf[:, keep], token[:, keep], ri[keep], B, L, omode, **kw)
        for name in ("reveal_mask", "remask_mask", "out_token", "step_of", "draft_pos", "draft_tok", "draft_len"):
            got = getattr(sel, name).cpu().numpy()
            assert np.array_equal(got.reshape(getattr(o, name).shape), getattr(o, name)), (path, name)
    # clean input afterwards: no bit
    ri_ok = np.flatnonzero(mask.reshape(-1)).astype(np.int32)
    st = torch.zeros(1, device=DEV, dtype=torch.int32)
    sel, bands = banded_select_out(B, L, K)
    binding.mrp_reveal_remask(ctx, c[:, :ri_ok.size].contiguous(), t[:, :ri_ok.size].contiguous(),
                              torch.from_numpy(ri_ok).to(DEV), ri_ok.size, K, B, L, binding.MRP_SELECT_STATIC,
                              reveal_mask=sel.reveal_mask, remask_mask=sel.remask_mask, out_token=sel.out_token,
                              step_of=sel.step_of, draft_pos=sel.draft_pos, draft_tok=sel.draft_tok,
                              draft_len=sel.draft_len, status=st)
    torch.cuda.synchronize()
    assert int(st.item()) == 0 and binding.mrp_fetch_status(ctx) == 0
    binding.mrp_destroy(ctx)


def test_more_than_four_heads_stay_on_the_tensor_cores():
    """Chains longer than four heads run on the tcgen05 kernels too (one kernel per GEMM instead of
    the persistent chain kernel)."""
    K = 6
    w = synth.make_weights(256, 512, 4096, K, "bf16", 33, head_std=0.04)
    inp = synth.make_inputs(w, 3, 4, 33, 1.0, 4.0)
    heads, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(w.d, w.F, w.V, heads, w_lm, max_rows=12, max_seqs=3, block_len=4,
                             flags=binding.MRP_FLAG_REQUIRE_TENSOR_CORES)
    assert ctx.family == "tcgen05"
    hid = harness.to_device(inp.hidden, "bf16", DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    for k in (6, 5):
        out = harness.alloc_draft_out(12, k, w.V, w.d, DEV)
        harness.draft(ctx, hid, l0, None, 12, k, out)
        torch.cuda.synchronize()
        ref = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=k)
        assert np.abs(out.conf.cpu().numpy() - ref.conf).max() <= 2e-3
        assert np.abs(out.lse.cpu().numpy() - ref.lse).max() <= 2e-3
        assert int(out.status.item()) == 0
    binding.mrp_destroy(ctx)


def test_require_tensor_cores_refuses_shapes_only_the_cuda_cores_take():
    w = synth.make_weights(72, 136, 1000, 1, "bf16", 31)
    heads, w_lm = harness.upload_weights(w, DEV)
    with pytest.raises(binding.MrpError) as ei:
        binding.mrp_create(72, 136, 1000, heads, w_lm, max_rows=4, max_seqs=1, block_len=4,
                           flags=binding.MRP_FLAG_REQUIRE_TENSOR_CORES)
    assert ei.value.status == 2
    ctx = binding.mrp_create(72, 136, 1000, heads, w_lm, max_rows=4, max_seqs=1, block_len=4)
    assert ctx.family == "simt"
    binding.mrp_destroy(ctx)
