"""The 8-bit LM head (MRP_FLAG_FP8_LM): the library's e4m3 copy of W_lm against the reference encoder
bit for bit, and the drafting pass against the oracle run on the dequantised matrix."""
import numpy as np
import pytest
import torch

import oracle
from oracle import fp8
from paper_2605_18817_b200 import binding, harness, synth
from test_gpu_parity import DEV, check_stats

pytestmark = pytest.mark.gpu


def _ctx(w, max_rows, B, L, flags=0):
    heads, w_lm = harness.upload_weights(w, DEV)
    return binding.mrp_create(w.d, w.F, w.V, heads, w_lm, max_rows=max_rows, max_seqs=B, block_len=L,
                              flags=flags | binding.MRP_FLAG_FP8_LM)


@pytest.mark.parametrize("d,F,V,B,L,K", [
    (256, 512, 4096, 2, 4, 3),        # 32 row-steps: the widest operand
    (512, 1024, 2064, 1, 4, 2),       # vocabulary not a multiple of the tile
    (2048, 4096, 151936, 1, 4, 3),    # the decode configuration at full size
])
def test_drafting_pass_on_the_8_bit_lm_head(d, F, V, B, L, K):
    w = synth.make_weights(d, F, V, K, "bf16", 1 if d == 2048 else 93, head_std=0.05 if d <= 512 else 0.02)
    # rows of very different size, a zero row and a row whose largest entry is an exact power of two
    w.w_lm[5] = synth.bf16_round(w.w_lm[5] * 37.0)
    w.w_lm[6] = 0
    w.w_lm[7, 3] = 0.5
    inp = synth.make_inputs(w, B, L, 93, 1.0, 4.0)
    codes, scales, w8 = fp8.quantise_rows(w.w_lm)
    M = B * L
    ctx = _ctx(w, M, B, L)
    assert ctx.family == "tcgen05"
    got_codes, got_scales = binding.mrp_quantised_lm_head(ctx)
    assert np.array_equal(got_scales, scales)
    assert np.array_equal(got_codes, codes)
    hid = harness.to_device(inp.hidden, "bf16", DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    for from_hidden in (False, True):
        out = harness.alloc_draft_out(M, K, V, d, DEV, logits=True, hidden=True, conf_first=True)
        if from_hidden:
            harness.draft_from_hidden(ctx, hid, None, None, M, K, out)
        else:
            harness.draft(ctx, hid, l0, None, M, K, out)
        torch.cuda.synchronize()
        # the oracle, unchanged, on the matrix the context computes with
        ref = oracle.draft(inp.hidden, None if from_hidden else inp.logits0, w.heads, w8, K=K, want_logits=True,
                           want_hidden=True)
        check_stats(out, ref, "bf16")
        lg = out.logits.cpu().numpy().astype(np.float64)
        rms = np.sqrt((ref.logits ** 2).mean(axis=2, keepdims=True))
        assert np.all(np.abs(lg - ref.logits) <= 2e-2 * np.maximum(np.abs(ref.logits), rms))
        assert np.abs(out.hidden.cpu().numpy() - ref.hidden).max() <= 2e-2
        clear0 = ref.margin[0] > 1e-2
        assert np.abs(out.conf_first.cpu().numpy() - ref.conf_first)[:, clear0].max() <= 2e-3
    # a shorter chain and a row subset
    sub = np.array([2, 0], np.int32) if M >= 3 else np.array([0], np.int32)
    out = harness.alloc_draft_out(len(sub), 1, V, d, DEV)
    harness.draft(ctx, hid, l0, torch.from_numpy(sub).to(DEV), len(sub), 1, out)
    torch.cuda.synchronize()
    check_stats(out, oracle.draft(inp.hidden, inp.logits0, w.heads, w8, K=1, row_index=sub), "bf16")
    # the quantisation itself is visible against the unquantised head (that is what the flag trades)
    full = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=K)
    ref = oracle.draft(inp.hidden, inp.logits0, w.heads, w8, K=K)
    assert np.abs(full.lse - ref.lse)[1:].max() > 1e-4
    binding.mrp_destroy(ctx)


def test_8_bit_lm_head_is_refused_outside_the_decode_regime():
    w = synth.make_weights(256, 512, 2048, 2, "bf16", 5)
    heads, w_lm = harness.upload_weights(w, DEV)
    for kw in (dict(max_rows=16, max_seqs=4, block_len=4),                      # 48 row-steps
               dict(max_rows=4, max_seqs=1, block_len=4, flags=binding.MRP_FLAG_FORCE_SIMT)):
        flags = kw.pop("flags", 0) | binding.MRP_FLAG_FP8_LM
        with pytest.raises(binding.MrpError) as ei:
            binding.mrp_create(256, 512, 2048, heads, w_lm, flags=flags, **kw)
        assert ei.value.status == 2
    ctx = binding.mrp_create(256, 512, 2048, heads, w_lm, max_rows=4, max_seqs=1, block_len=4)
    with pytest.raises(binding.MrpError):
        binding.mrp_quantised_lm_head(ctx)                                       # no 8-bit copy in this context
    binding.mrp_destroy(ctx)


@pytest.mark.parametrize("d,F,V,D,heads,B,L", [
    (256, 512, 4096, 2, 2, 2, 4),        # 16 row-steps, the step as one cooperative kernel
    (512, 1024, 2064, 1, 4, 1, 5),       # ragged vocabulary, a block of five
    (2048, 4096, 151936, 3, 16, 1, 4),   # the decode configuration at full size, the paper's depth
])
def test_module_step_on_the_8_bit_lm_head(d, F, V, D, heads, B, L):
    """The token-conditioned module's step on an MRP_FLAG_FP8_LM context: its LM-head pass runs on the 8-bit copy,
    so its results are the oracle's module with the dequantised matrix as the LM head."""
    from test_gpu_module import upload_module
    big = d == 2048
    w = synth.make_weights(d, F, V, 1, "bf16", 1 if big else 95)
    mw = synth.make_module_weights(d, F, V, D, heads, "bf16", 11 if big else 95, std=0.02 if big else 0.06,
                                   proj_std=None if big else 0.3 / np.sqrt(2 * d))
    inp = synth.make_inputs(w, B, L, 95, 1.0, 4.0)
    _, _, w8 = fp8.quantise_rows(w.w_lm)
    n = B * L
    ctx = _ctx(w, n, B, L)
    emb, w_proj, layers = upload_module(mw, "bf16")
    binding.mrp_module_attach(ctx, emb, w_proj, layers, heads, mw.mask_token)
    tokens = np.full(n, -1, np.int32)
    tokens[::L] = 17
    hid0 = harness.to_device(inp.hidden, "bf16", DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    h_state = torch.empty((n, d), device=DEV, dtype=torch.float32)
    h_run = inp.hidden.astype(np.float64)
    l_run = inp.logits0.astype(np.float64)
    for s in range(2):
        ri = np.flatnonzero(tokens < 0).astype(np.int32)
        M = ri.size
        out = harness.alloc_draft_out(M, 1, V, d, DEV, hidden=True)
        binding.mrp_module_step(ctx, torch.from_numpy(tokens).to(DEV), hid0, h_state, l0, torch.from_numpy(ri).to(DEV), M, B, L,
                                s == 0, out.conf, out.lse, out.token, margin=out.margin, hidden_out=out.hidden, status=out.status)
        torch.cuda.synchronize()
        assert int(out.status.item()) == 0
        dh, dl = oracle.module(h_run.astype(np.float32), tokens, B, L, mw.emb, mw.w_proj, mw.layers, w8, heads, mw.mask_token,
                               row_index=ri)
        h_run = h_run.astype(np.float32).astype(np.float64) + dh
        l_run[ri] += dl
        conf, lse, tok, margin = oracle.stats(l_run[ri])
        assert np.abs(h_state.cpu().numpy() - h_run).max() <= 1e-3 * max(1.0, np.abs(h_run).max())
        assert np.abs(out.conf[1].cpu().numpy() - conf).max() <= 2e-3 and np.abs(out.lse[1].cpu().numpy() - lse).max() <= 2e-3
        clear = margin > 1e-2
        assert np.array_equal(out.token[1].cpu().numpy()[clear], tok[clear])
        # the quantisation is visible against the unquantised head
        if s == 0:
            _, dl_full = oracle.module(inp.hidden, tokens, B, L, mw.emb, mw.w_proj, mw.layers, w.w_lm, heads, mw.mask_token,
                                       row_index=ri)
            assert np.abs(dl_full - dl).max() > 1e-4
        # reveal the most confident masked position of every block for the next step
        for b in range(B):
            rows = [m for m in range(M) if ri[m] // L == b]
            if rows:
                best = max(rows, key=lambda m: conf[m])
                tokens[ri[best]] = tok[best]
    binding.mrp_destroy(ctx)
