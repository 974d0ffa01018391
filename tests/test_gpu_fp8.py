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
