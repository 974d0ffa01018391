"""Parity of the CUDA path (through the C ABI) against the CPU oracle on the same seeded
inputs.  Tolerances: integer outputs bit-exact wherever the oracle's top-2 logit margin
exceeds 1e-2; confidence and log-sum-exp within 2e-3 absolute on bf16 contexts (1e-5 on
fp32 contexts); materialised logits within 2e-2 relative to max(|logit|, row RMS)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_18817_b200 import binding, harness, synth

pytestmark = pytest.mark.gpu

DEV = "cuda:0"
TOL = {"f32": 1e-5, "bf16": 2e-3}


def run_gpu_draft(w, inp, K, flags=0, margin=True, logits=False, hidden=False, row_index="inp",
                  ctx=None):
    heads, w_lm = (None, None)
    own = ctx is None
    if own:
        heads, w_lm = harness.upload_weights(w, DEV)
        ctx = binding.mrp_create(w.d, w.F, w.V, heads, w_lm, max_rows=max(inp.B * inp.L, 1),
                                 max_seqs=inp.B, block_len=inp.L, flags=flags)
    ri = inp.row_index if isinstance(row_index, str) else row_index
    M = inp.hidden.shape[0] if ri is None else len(ri)
    hid = harness.to_device(inp.hidden, w.dtype, DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    ri_t = None if ri is None else torch.from_numpy(np.asarray(ri, np.int32)).to(DEV)
    out = harness.alloc_draft_out(M, K, w.V, w.d, DEV, margin=margin, logits=logits, hidden=hidden)
    harness.draft(ctx, hid, l0, ri_t, M, K, out)
    torch.cuda.synchronize()
    fam = ctx.family
    if own:
        binding.mrp_destroy(ctx)
    return out, fam


def run_gpu_draft_from_hidden(w, inp, K, final_gamma=None, flags=0, logits=False, hidden=False,
                              row_index="inp"):
    """mrp_draft_from_hidden on the same inputs: no base logits are handed over."""
    heads, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(w.d, w.F, w.V, heads, w_lm, max_rows=max(inp.B * inp.L, 1),
                             max_seqs=inp.B, block_len=inp.L, flags=flags)
    ri = inp.row_index if isinstance(row_index, str) else row_index
    M = inp.hidden.shape[0] if ri is None else len(ri)
    hid = harness.to_device(inp.hidden, w.dtype, DEV)
    g = None if final_gamma is None else harness.to_device(final_gamma, w.dtype, DEV)
    ri_t = None if ri is None else torch.from_numpy(np.asarray(ri, np.int32)).to(DEV)
    out = harness.alloc_draft_out(M, K, w.V, w.d, DEV, margin=True, logits=logits, hidden=hidden)
    harness.draft_from_hidden(ctx, hid, g, ri_t, M, K, out)
    torch.cuda.synchronize()
    fam = ctx.family
    binding.mrp_destroy(ctx)
    return out, fam


def check_stats(out, ref, dtype, cols=None):
    """Compare conf/lse/token of the GPU (all rows, or the columns `cols`) with the oracle."""
    tol = TOL[dtype]
    conf = out.conf.cpu().numpy().astype(np.float64)
    lse = out.lse.cpu().numpy().astype(np.float64)
    tok = out.token.cpu().numpy()
    if cols is not None:
        conf, lse, tok = conf[:, cols], lse[:, cols], tok[:, cols]
    assert conf.shape == ref.conf.shape
    assert np.abs(conf - ref.conf).max() <= tol, np.abs(conf - ref.conf).max()
    assert np.abs(lse - ref.lse).max() <= tol, np.abs(lse - ref.lse).max()
    clear = ref.margin > 1e-2
    assert clear.mean() > 0.5
    assert np.array_equal(tok[clear], ref.token[clear])
    if out.margin is not None:
        mg = out.margin.cpu().numpy().astype(np.float64)
        if cols is not None:
            mg = mg[:, cols]
        assert np.abs(mg - ref.margin).max() <= max(10 * tol, 2e-2)
    assert int(out.status.item()) == 0


def test_config0_fp32_all_outputs():
    cfg = synth.CONFIGS[0]
    w, inp = synth.make_config(cfg)
    out, fam = run_gpu_draft(w, inp, cfg["K"], logits=True, hidden=True)
    assert fam == "simt"
    ref = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=cfg["K"], row_index=inp.row_index,
                       want_logits=True, want_hidden=True)
    check_stats(out, ref, "f32")
    lg = out.logits.cpu().numpy().astype(np.float64)
    assert np.abs(lg - ref.logits).max() <= 1e-4
    assert np.abs(out.hidden.cpu().numpy() - ref.hidden).max() <= 1e-4


@pytest.mark.parametrize("dtype,flags", [("f32", 0), ("bf16", binding.MRP_FLAG_FORCE_SIMT)])
def test_ragged_shapes_on_cuda_cores(dtype, flags):
    # sizes that are not multiples of any tile: d, F, V ragged, odd row count, row subset
    w = synth.make_weights(72, 136, 1000, 3, dtype, 31, head_std=0.1)
    for k, h in enumerate(w.heads):
        h["gamma"] = (1.0 + 0.25 * np.cos(np.arange(72) + k)).astype(np.float32)
        if dtype == "bf16":
            h["gamma"] = synth.bf16_round(h["gamma"])
    inp = synth.make_inputs(w, 5, 3, 31, 1.0, 4.0, mask_prob=0.7)
    out, fam = run_gpu_draft(w, inp, 3, flags=flags, logits=True, hidden=True)
    assert fam == "simt"
    ref = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, row_index=inp.row_index,
                       want_logits=True, want_hidden=True)
    check_stats(out, ref, "f32")     # the CUDA-core family keeps fp32 intermediates
    assert np.abs(out.logits.cpu().numpy() - ref.logits).max() <= 1e-4
    assert np.abs(out.hidden.cpu().numpy() - ref.hidden).max() <= 1e-4
    # chain truncated to K = 1 and K = 0
    for K in (1, 0):
        o, _ = run_gpu_draft(w, inp, K, flags=flags)
        r = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=K, row_index=inp.row_index)
        check_stats(o, r, "f32")


@pytest.mark.parametrize("dtype,flags", [("f32", 0), ("bf16", binding.MRP_FLAG_FORCE_SIMT)])
@pytest.mark.parametrize("d,F,V,B,L", [(72, 136, 1000, 2, 3), (256, 512, 4096, 1, 4), (512, 264, 20000, 2, 4)])
def test_one_kernel_pass_for_a_few_short_rows(dtype, flags, d, F, V, B, L):
    """Up to 8 rows of up to 512 features run the whole drafting pass as one cooperative kernel on the CUDA
    cores: one launch, same results as one kernel per step (MRP_FLAG_NO_CHAIN) up to the merge order of the slices, oracle parity
    with every optional output, repeated calls (the grid barrier's counter carries over from call to call),
    the base logits computed in the pass, a row subset and an out-of-range row."""
    K = 3
    # (the fp32 tolerance is absolute, 1e-5: residuals that keep the logits near 10, where that is 10 ulp)
    w = synth.make_weights(d, F, V, K, dtype, 47, head_std=0.1 if d < 512 else 0.03)
    inp = synth.make_inputs(w, B, L, 47, 1.0, 4.0)
    M = len(inp.row_index)
    assert 1 <= M <= 8
    heads, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(d, F, V, heads, w_lm, max_rows=B * L, max_seqs=B, block_len=L, flags=flags)
    ctx1 = binding.mrp_create(d, F, V, heads, w_lm, max_rows=B * L, max_seqs=B, block_len=L,
                              flags=flags | binding.MRP_FLAG_NO_CHAIN)
    assert ctx.family == "simt"
    hid = harness.to_device(inp.hidden, w.dtype, DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    ri = torch.from_numpy(inp.row_index).to(DEV)
    ref = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=K, row_index=inp.row_index, want_logits=True,
                       want_hidden=True)
    status = torch.zeros(1, dtype=torch.int32, device=DEV)
    for rep in range(3):
        out = harness.alloc_draft_out(M, K, V, d, DEV, margin=True, logits=True, hidden=True, conf_first=True)
        out.status = status
        harness.draft(ctx, hid, l0, ri, M, K, out)
        torch.cuda.synchronize()
        assert ctx.last_launch_count == 1
        check_stats(out, ref, "f32")
        assert np.abs(out.logits.cpu().numpy() - ref.logits).max() <= 1e-4
        assert np.abs(out.hidden.cpu().numpy() - ref.hidden).max() <= 1e-4
        clear0 = ref.margin[0] > 1e-2
        assert np.abs(out.conf_first.cpu().numpy() - ref.conf_first)[:, clear0].max() <= 1e-5
    assert int(status.item()) == 0
    sep = harness.alloc_draft_out(M, K, V, d, DEV, margin=True)
    harness.draft(ctx1, hid, l0, ri, M, K, sep)
    torch.cuda.synchronize()
    assert ctx1.last_launch_count > 1
    assert torch.equal(sep.token, out.token)
    assert float((sep.conf - out.conf).abs().max()) <= 1e-5 and float((sep.lse - out.lse).abs().max()) <= 1e-5
    # shorter chain, row subset, base logits computed in the pass
    sub = inp.row_index[::2]
    o2 = harness.alloc_draft_out(len(sub), 2, V, d, DEV)
    harness.draft_from_hidden(ctx, hid, None, torch.from_numpy(sub).to(DEV), len(sub), 2, o2)
    torch.cuda.synchronize()
    assert ctx.last_launch_count == 1
    check_stats(o2, oracle.draft(inp.hidden, None, w.heads, w.w_lm, K=2, row_index=sub), "f32")
    # an out-of-range row reads as zeros and raises the status bit; the other rows are untouched by it
    bad = inp.row_index.copy()
    bad[-1] = B * L + 5
    o3 = harness.alloc_draft_out(M, K, V, d, DEV)
    o3.status = status
    harness.draft(ctx, hid, l0, torch.from_numpy(bad).to(DEV), M, K, o3)
    torch.cuda.synchronize()
    assert int(status.item()) & binding.MRP_DEV_BAD_INDEX
    if M > 1:
        assert torch.equal(o3.token[:, :M - 1], out.token[:, :M - 1])
        assert float((o3.conf[:, :M - 1] - out.conf[:, :M - 1]).abs().max()) <= 1e-5
    binding.mrp_destroy(ctx)
    binding.mrp_destroy(ctx1)


def test_empty_call_and_argument_errors():
    cfg = synth.CONFIGS[0]
    w, inp = synth.make_config(cfg)
    ctx = harness.create_for(cfg, w, DEV)
    out = harness.alloc_draft_out(4, 3, w.V, w.d, DEV)
    hid = harness.to_device(inp.hidden, w.dtype, DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    out.conf.fill_(-7.0)
    harness.draft(ctx, hid, l0, None, 0, 3, out)          # M = 0: nothing is written
    torch.cuda.synchronize()
    assert float(out.conf.min()) == -7.0 and ctx.last_launch_count == 0
    with pytest.raises(binding.MrpError):                  # M beyond max_rows
        harness.draft(ctx, hid, l0, None, 5, 3, out)
    with pytest.raises(binding.MrpError):                  # K beyond n_heads
        harness.draft(ctx, hid, l0, None, 4, 4, out)
    with pytest.raises(binding.MrpError):                  # missing required output
        binding.mrp_draft(ctx, hid, l0, None, 4, 3, None, out.lse, out.token)
    harness.draft(ctx, hid, l0, None, 4, 3, out)           # context still usable
    torch.cuda.synchronize()
    assert float(out.conf.min()) > 0
    binding.mrp_destroy(ctx)


def _rand_select_case(rng, K, B, L, mask_prob):
    mask = rng.random((B, L)) < mask_prob
    ri = np.flatnonzero(mask.reshape(-1)).astype(np.int32)
    rng.shuffle(ri)                                        # row order need not be ascending
    M = ri.size
    conf = rng.random((K + 1, M)).astype(np.float32)
    # plant exact ties and exact threshold hits
    if M > 3:
        conf[:, 1] = conf[:, 0]
        conf[0, 2] = np.float32(0.5)
    token = rng.integers(0, 1000, (K + 1, M)).astype(np.int32)
    # in about half of the row-steps the argmax is still the step-0 token
    token = np.where(rng.random((K + 1, M)) < 0.5, token[:1], token).astype(np.int32)
    return ri, conf, token


@pytest.fixture(scope="module")
def select_ctx():
    w = synth.make_weights(16, 16, 32, 0, "f32", 1)
    heads, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(16, 16, 32, heads, w_lm, max_rows=4, max_seqs=64, block_len=1024)
    yield ctx
    binding.mrp_destroy(ctx)


def _gpu_select(ctx, conf, token, ri, B, L, mode, **kw):
    K = conf.shape[0] - 1
    M = conf.shape[1]
    Kd = K * kw.get("r_draft", 1)
    out = harness.alloc_select_out(B, L, Kd, DEV)
    if kw.get("conf_first") is not None:
        kw = dict(kw, conf_first=torch.from_numpy(kw["conf_first"]).to(DEV))
    c = torch.from_numpy(conf).to(DEV)
    t = torch.from_numpy(token).to(DEV)
    r = torch.from_numpy(ri).to(DEV) if ri is not None else None
    harness.select(ctx, c, t, r, M, K, B, L, mode, out, **kw)
    torch.cuda.synchronize()
    return out


def _assert_select_equal(g, o):
    for name in ("reveal_mask", "remask_mask", "out_token", "step_of", "draft_pos", "draft_tok",
                 "draft_len"):
        a = getattr(g, name).cpu().numpy()
        b = getattr(o, name)
        assert np.array_equal(a.reshape(b.shape), b), name


@pytest.mark.parametrize("L", [1, 4, 16, 32, 33, 100, 1024])
def test_select_bit_exact_on_shared_statistics(select_ctx, L):
    rng = np.random.default_rng(L)
    for case in range(6):
        K = case % 4
        B = 1 + (case * 7) % 23
        ri, conf, token = _rand_select_case(rng, K, B, L, 0.3 + 0.1 * case)
        if ri.size == 0:
            continue
        kw = dict(r_reveal=1 + case % 3, r_draft=case % 3)
        g = _gpu_select(select_ctx, conf, token, ri, B, L, binding.MRP_SELECT_STATIC, **kw)
        o = oracle.select(conf, token, ri, B, L, oracle.STATIC, **kw)
        _assert_select_equal(g, o)
        # the revealed token's own probability: the top probability where the token stayed, less where it moved
        moved = token != token[:1]
        conf_first = np.where(moved, conf * np.float32(0.5), conf).astype(np.float32)
        for tau in (0.0, 0.3, 0.5, 0.8, 1.5):
            for cap in (False, True):
                for policy in (0, 1, 2, 3):
                    for prog in (True, False):
                        kw = dict(tau=tau, use_cap=cap, remask_policy=policy, ensure_progress=prog)
                        if policy == 2:
                            kw["conf_first"] = conf_first
                        g = _gpu_select(select_ctx, conf, token, ri, B, L,
                                        binding.MRP_SELECT_DYNAMIC_REMASK, **kw)
                        o = oracle.select(conf, token, ri, B, L, oracle.DYNAMIC_REMASK, **kw)
                        _assert_select_equal(g, o)


def test_select_with_no_masked_rows_writes_defaults(select_ctx):
    out = harness.alloc_select_out(3, 4, 2, DEV)
    empty_f = torch.empty((3, 0), device=DEV)
    empty_i = torch.empty((3, 0), device=DEV, dtype=torch.int32)
    harness.select(select_ctx, empty_f, empty_i, None, 0, 2, 3, 4, binding.MRP_SELECT_STATIC, out)
    torch.cuda.synchronize()
    assert not out.reveal_mask.any() and bool((out.out_token == -1).all())
    assert bool((out.draft_pos == -1).all()) and not out.draft_len.any()


def test_verify_bit_exact(select_ctx):
    rng = np.random.default_rng(5)
    for B, Kd in ((1, 1), (32, 3), (64, 4), (7, 12)):
        d = rng.integers(0, 50, (B, Kd)).astype(np.int32)
        v = synth.make_verify_tokens(d, 50, seed=B, p_match=0.7)
        n = rng.integers(0, Kd + 1, B).astype(np.int32)
        for pw in (False, True):
            al, am = harness.verify(select_ctx, torch.from_numpy(d).to(DEV), torch.from_numpy(v).to(DEV),
                                    torch.from_numpy(n).to(DEV), positionwise=pw)
            torch.cuda.synchronize()
            ol, om = oracle.verify(d, v, n, positionwise=pw)
            assert np.array_equal(al.cpu().numpy(), ol) and np.array_equal(am.cpu().numpy(), om)


def test_config0_static_selection_end_to_end():
    cfg = synth.CONFIGS[0]
    w, inp = synth.make_config(cfg)
    ctx = harness.create_for(cfg, w, DEV)
    K, B, L = cfg["K"], cfg["B"], cfg["L"]
    M = len(inp.row_index)
    hid = harness.to_device(inp.hidden, w.dtype, DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    ri = torch.from_numpy(inp.row_index).to(DEV)
    out = harness.alloc_draft_out(M, K, w.V, w.d, DEV)
    harness.draft(ctx, hid, l0, ri, M, K, out)
    sel = harness.alloc_select_out(B, L, K, DEV)
    harness.select(ctx, out.conf, out.token, ri, M, K, B, L, binding.MRP_SELECT_STATIC, sel)
    torch.cuda.synchronize()
    ref = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=K, row_index=inp.row_index)
    osel = oracle.select(ref.conf.astype(np.float32), ref.token, inp.row_index, B, L, oracle.STATIC)
    # the four confidences of this instance are separated by far more than the tolerance
    gaps = np.abs(ref.conf[:, :, None] - ref.conf[:, None, :])[:, ~np.eye(M, dtype=bool)]
    assert gaps.min() > 1e-4
    _assert_select_equal(sel, osel)
    binding.mrp_destroy(ctx)


@pytest.mark.parametrize("d,F,V,B,L,K", [
    (256, 512, 4096, 2, 4, 2),      # all row-steps stacked in one 128-row block
    (128, 256, 2048, 10, 4, 3),     # 160 row-steps: one accumulator per step, M < 128
    (192, 320, 4112, 150, 1, 2),    # two row blocks, vocabulary not a multiple of the tile
    (64, 64, 1024, 128, 1, 1),      # exactly one full row block
    (256, 512, 4096, 75, 4, 4),     # 300 rows, four accumulators
    (64, 128, 160, 3, 1, 1),        # fewer vocabulary units than CTAs
    (128, 256, 2048, 16, 1, 1),     # few-row kernels at their 32-row-step limit
    (128, 256, 2048, 32, 1, 2),     # few-row head kernels at 32 rows, row-major LM head
    (64, 12288, 2304, 5, 1, 2),     # gate/up: full 128-row weight tiles plus short tiles
    (19008, 64, 512, 3, 1, 1),      # down projection: full weight tiles plus short tiles
    (1024, 2048, 2048, 20, 1, 2),   # head chain with 32-row operands and two k-chunks per ring stage
    (512, 1024, 2048, 100, 1, 2),   # head chain with 128-row operands
    (128, 192, 2048, 90, 1, 2),     # the same with an odd number of gate/up weight tiles
    (64, 6144, 1024, 100, 1, 1),    # head chain, gate/up tiles not split: outputs finished straight from TMEM
    (64, 6144, 1024, 5, 1, 2),      # the same with few rows
    (64, 128, 160, 257, 1, 1),      # CTA pairs: three row blocks (the second pair half empty), fewer units than pairs
    (128, 256, 2064, 129, 1, 3),    # CTA pairs: one row past a block in the heads, four row blocks in the LM head
])
def test_tensor_core_family_small_shapes(d, F, V, B, L, K):
    # residuals inside the accuracy range the header states for the tensor-core kernels
    # (d * rms(h_k - h_0) <= MRP_RANGE_LIMIT; check_stats asserts that no status bit was raised)
    w = synth.make_weights(d, F, V, K, "bf16", 77, head_std=0.05 if d < 4096 else 0.02)
    for k, h in enumerate(w.heads):
        h["gamma"] = synth.bf16_round((1.0 + 0.25 * np.cos(np.arange(d) + k)).astype(np.float32))
    inp = synth.make_inputs(w, B, L, 77, 1.0, 4.0)
    out, fam = run_gpu_draft(w, inp, K, logits=True, hidden=True)
    assert fam == "tcgen05"
    ref = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=K, row_index=inp.row_index,
                       want_logits=True, want_hidden=True)
    check_stats(out, ref, "bf16")
    lg = out.logits.cpu().numpy().astype(np.float64)
    rms = np.sqrt((ref.logits ** 2).mean(axis=2, keepdims=True))
    assert np.all(np.abs(lg - ref.logits) <= 2e-2 * np.maximum(np.abs(ref.logits), rms))
    assert np.abs(out.hidden.cpu().numpy() - ref.hidden).max() <= 2e-2
    # without the optional outputs the statistics are identical
    out2, _ = run_gpu_draft(w, inp, K, margin=False)
    assert torch.equal(out2.conf, out.conf) and torch.equal(out2.token, out.token)
    # a row subset through row_index, shorter chain
    sub = inp.row_index[::3]
    out3, _ = run_gpu_draft(w, inp, max(K - 1, 1), row_index=sub)
    ref3 = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=max(K - 1, 1), row_index=sub)
    check_stats(out3, ref3, "bf16")
    # the row-major kernels alone, fully serialised launches: same results within tolerance
    out4, _ = run_gpu_draft(w, inp, K, flags=binding.MRP_FLAG_ROW_MAJOR_ONLY | binding.MRP_FLAG_NO_PDL)
    check_stats(out4, ref, "bf16")
    # the head chain as one kernel per GEMM instead of one persistent kernel
    out5, _ = run_gpu_draft(w, inp, K, flags=binding.MRP_FLAG_NO_CHAIN)
    check_stats(out5, ref, "bf16")
    # the row-major kernels one CTA per tile instead of CTA pairs
    if B * L > 128:
        out6, _ = run_gpu_draft(w, inp, K, flags=binding.MRP_FLAG_NO_CTA_PAIRS)
        check_stats(out6, ref, "bf16")


@pytest.mark.parametrize("d,F,V,M,K,std,beyond", [
    (19008, 64, 512, 3, 1, 0.02, False),        # d * rms about 14 000
    (19008, 64, 512, 3, 1, 0.05, True),         # about 220 000
    (4096, 8192, 4096, 40, 2, 0.02, False),     # the benchmark shapes' weights: about 11 000
    (4096, 8192, 4096, 40, 2, 0.04, True),      # about 98 000: beyond the range, and beyond the tolerance
])
def test_residuals_beyond_the_accuracy_range_raise_the_range_bit(d, F, V, M, K, std, beyond):
    """The tensor-core kernels keep confidence and log-sum-exp within 2e-3 while d * rms(h_k - h_0)
    stays below MRP_RANGE_LIMIT; a row-step beyond it is still computed but raises MRP_DEV_RANGE
    (the CUDA-core kernels, which accumulate by fp32 FMA, take the same input without the bit)."""
    w = synth.make_weights(d, F, V, K, "bf16", 77, head_std=std)
    inp = synth.make_inputs(w, M, 1, 77, 1.0, 4.0)
    ref = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=K, want_hidden=True)
    d_rms = d * np.sqrt(((ref.hidden - inp.hidden.astype(np.float64)) ** 2).mean(axis=1)).max()
    assert (d_rms > 2 * binding.MRP_RANGE_LIMIT) if beyond else (d_rms < 0.5 * binding.MRP_RANGE_LIMIT)
    out, fam = run_gpu_draft(w, inp, K)
    assert fam == "tcgen05"
    assert int(out.status.item()) == (binding.MRP_DEV_RANGE if beyond else 0)
    assert torch.isfinite(out.lse).all()
    if not beyond:
        check_stats(out, ref, "bf16")
    out_s, fam_s = run_gpu_draft(w, inp, K, flags=binding.MRP_FLAG_FORCE_SIMT)
    assert fam_s == "simt" and int(out_s.status.item()) == 0
    check_stats(out_s, ref, "bf16")


@pytest.mark.parametrize("flags", [0, binding.MRP_FLAG_FORCE_SIMT])
def test_non_finite_logits_raise_the_status_bit_and_leave_the_context_usable(flags):
    w = synth.make_weights(128, 256, 2048, 2, "bf16", 5, head_std=0.05)
    inp = synth.make_inputs(w, 2, 4, 5, 1.0, 4.0)
    heads, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(w.d, w.F, w.V, heads, w_lm, max_rows=8, max_seqs=2, block_len=4, flags=flags)
    hid = harness.to_device(inp.hidden, w.dtype, DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    bad = l0.clone()
    bad[3, 100] = float("inf")
    out = harness.alloc_draft_out(8, 2, w.V, w.d, DEV)
    harness.draft(ctx, hid, bad, None, 8, 2, out)
    torch.cuda.synchronize()
    assert int(out.status.item()) & binding.MRP_DEV_NONFINITE
    good = harness.alloc_draft_out(8, 2, w.V, w.d, DEV)
    harness.draft(ctx, hid, l0, None, 8, 2, good)
    torch.cuda.synchronize()
    assert int(good.status.item()) == 0
    ref = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=2)
    check_stats(good, ref, "bf16")
    binding.mrp_destroy(ctx)


def test_a_wait_that_nothing_completes_gives_up_and_reports():
    """Failure detection without a fault: the kernels' waits are bounded.  A barrier that nobody
    completes makes the wait run out (about 1.5 s); the kernel returns, the status word carries
    MRP_DEV_TIMEOUT and the context goes on working."""
    w = synth.make_weights(128, 256, 2048, 1, "bf16", 9, head_std=0.05)
    inp = synth.make_inputs(w, 1, 4, 9, 1.0, 4.0)
    heads, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(w.d, w.F, w.V, heads, w_lm, max_rows=4, max_seqs=1, block_len=4)
    st = torch.zeros(1, device=DEV, dtype=torch.int32)
    binding.mrp_selftest_wait_timeout(ctx, st)
    torch.cuda.synchronize()
    assert int(st.item()) & binding.MRP_DEV_TIMEOUT
    out, _ = run_gpu_draft(w, inp, 1, ctx=ctx)
    ref = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=1)
    check_stats(out, ref, "bf16")
    binding.mrp_destroy(ctx)


@pytest.mark.parametrize("dtype,flags,d,F,V,B,L,K", [
    ("f32", 0, 72, 136, 1000, 5, 3, 3),                                # CUDA-core kernels
    ("bf16", binding.MRP_FLAG_FORCE_SIMT, 72, 136, 1000, 5, 3, 2),
    ("bf16", 0, 256, 512, 4096, 2, 4, 3),                              # few-row tensor-core kernels
    ("bf16", 0, 128, 256, 2048, 30, 4, 3),                             # row-major LM head, fp16 operand
    ("bf16", binding.MRP_FLAG_EXACT_OPERANDS, 128, 256, 2048, 30, 4, 2),
])
def test_probability_of_the_step_zero_token_under_the_updated_logits(dtype, flags, d, F, V, B, L, K):
    """mrp_draft_out.conf_first against the oracle, with and without base logits handed over, and
    remask policy 2 / 3 driven by it end to end."""
    w = synth.make_weights(d, F, V, K, dtype, 61, head_std=0.12 if d < 128 else 0.08)   # residuals that move argmaxes
    inp = synth.make_inputs(w, B, L, 61, 0.5, 2.5)
    heads, w_lm = harness.upload_weights(w, DEV)
    M = B * L
    ctx = binding.mrp_create(d, F, V, heads, w_lm, max_rows=M, max_seqs=B, block_len=L, flags=flags)
    hid = harness.to_device(inp.hidden, w.dtype, DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    tol = TOL[dtype]
    moved_total = 0
    for from_hidden in (False, True):
        out = harness.alloc_draft_out(M, K, V, d, DEV, conf_first=True)
        out.conf_first.fill_(-1.0)
        if from_hidden:
            harness.draft_from_hidden(ctx, hid, None, None, M, K, out)
        else:
            harness.draft(ctx, hid, l0, None, M, K, out)
        torch.cuda.synchronize()
        ref = oracle.draft(inp.hidden, None if from_hidden else inp.logits0, w.heads, w.w_lm, K=K)
        check_stats(out, ref, dtype)
        # compare where the step-0 token is unambiguous (else the two sides may follow different tokens)
        clear0 = ref.margin[0] > 1e-2
        got = out.conf_first.cpu().numpy().astype(np.float64)
        assert np.abs(got - ref.conf_first)[:, clear0].max() <= tol
        assert np.array_equal(got[0], out.conf.cpu().numpy()[0].astype(np.float64))
        assert np.all(got <= out.conf.cpu().numpy() + 1e-7)
        moved_total += int((ref.token[1:] != ref.token[:1]).sum())
        # selection driven by the device's own statistics, policies 2 and 3, bit-exact against the oracle's rules
        for policy in (2, 3):
            sel = harness.alloc_select_out(B, L, K, DEV)
            harness.select(ctx, out.conf, out.token, None, M, K, B, L, binding.MRP_SELECT_DYNAMIC_REMASK, sel,
                           tau=0.3, remask_policy=policy, conf_first=out.conf_first)
            torch.cuda.synchronize()
            osel = oracle.select(out.conf.cpu().numpy(), out.token.cpu().numpy(), None, B, L, oracle.DYNAMIC_REMASK,
                                 tau=0.3, remask_policy=policy, conf_first=out.conf_first.cpu().numpy())
            _assert_select_equal(sel, osel)
    assert moved_total > 0
    with pytest.raises(binding.MrpError):          # policy 2 needs the array
        sel = harness.alloc_select_out(B, L, K, DEV)
        harness.select(ctx, out.conf, out.token, None, M, K, B, L, binding.MRP_SELECT_DYNAMIC_REMASK, sel,
                       tau=0.3, remask_policy=2)
    binding.mrp_destroy(ctx)


# ---- base logits stored as bf16 (mrp_draft_bf16_logits) ----

@pytest.mark.parametrize("dtype,flags,d,F,V,B,L,K", [
    ("f32", 0, 72, 136, 1000, 5, 3, 2),                                # CUDA-core kernels
    ("bf16", 0, 256, 512, 4096, 2, 4, 3),                              # few-row LM head
    ("bf16", 0, 128, 256, 2048, 30, 4, 3),                             # row-major LM head, fp16 operand + top fix
    ("bf16", binding.MRP_FLAG_EXACT_OPERANDS, 192, 320, 4112, 150, 1, 2),
])
def test_base_logits_stored_as_bf16(dtype, flags, d, F, V, B, L, K):
    """The bf16 values are the input: the oracle takes the same values promoted to fp32."""
    w = synth.make_weights(d, F, V, K, dtype, 81, head_std=0.05)
    inp = synth.make_inputs(w, B, L, 81, 1.0, 4.0, mask_prob=0.8)
    l0_r = synth.bf16_round(inp.logits0)
    heads, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(d, F, V, heads, w_lm, max_rows=B * L, max_seqs=B, block_len=L, flags=flags)
    M = inp.row_index.size
    hid = harness.to_device(inp.hidden, w.dtype, DEV)
    l0 = harness.to_device(l0_r, "bf16", DEV)
    ri = torch.from_numpy(inp.row_index).to(DEV)
    out = harness.alloc_draft_out(M, K, V, d, DEV, logits=True, conf_first=True)
    harness.draft(ctx, hid, l0, ri, M, K, out)
    torch.cuda.synchronize()
    ref = oracle.draft(inp.hidden, l0_r, w.heads, w.w_lm, K=K, row_index=inp.row_index, want_logits=True)
    check_stats(out, ref, dtype)
    lg = out.logits.cpu().numpy().astype(np.float64)
    rms = np.sqrt((ref.logits ** 2).mean(axis=2, keepdims=True))
    assert np.all(np.abs(lg - ref.logits) <= (1e-4 if dtype == "f32" else 2e-2) * np.maximum(np.abs(ref.logits), rms))
    clear0 = ref.margin[0] > 1e-2
    assert np.abs(out.conf_first.cpu().numpy() - ref.conf_first)[:, clear0].max() <= TOL[dtype]
    binding.mrp_destroy(ctx)


# ---- the training objective fused into the LM-head epilogue (mrp_draft_kl) ----

@pytest.mark.parametrize("dtype,flags,d,F,V,B,L,K", [
    ("f32", 0, 72, 136, 1000, 5, 3, 2),                                # CUDA-core kernels, ragged sizes
    ("bf16", binding.MRP_FLAG_FORCE_SIMT, 72, 136, 1000, 5, 3, 3),
    ("bf16", 0, 256, 512, 4096, 2, 4, 2),                              # 8 rows: one row block
    ("bf16", 0, 192, 320, 4112, 150, 1, 2),                            # 300 row-steps, ragged vocabulary tiles
    ("bf16", 0, 1024, 2048, 8192, 40, 4, 3),                           # several tiles per CTA, 480 row-steps
])
def test_kl_objective_fused_into_the_lm_head(dtype, flags, d, F, V, B, L, K):
    """kl[k, m] = KL(softmax(teacher_k) || softmax(l_k)) per masked row and unrolled step (Eq. (3)) against
    the oracle: absolute error within 2e-3 (bf16 contexts) / 1e-5 (fp32), and relative 2e-3 where the
    divergence is large; the ordinary statistics of the same call stay those of mrp_draft."""
    w = synth.make_weights(d, F, V, K, dtype, 71, head_std=0.05 if d <= 256 else 0.02)
    inp = synth.make_inputs(w, B, L, 71, 1.0, 4.0, mask_prob=0.8)
    ri = inp.row_index
    M = ri.size
    base = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=K, row_index=ri, want_logits=True)
    rng = np.random.default_rng(3)
    # teacher = corrected logits plus a perturbation of a few tenths: KL values from 1e-3 to order one
    scale = rng.uniform(0.02, 0.6, size=(K, M, 1))
    teacher = (base.logits + scale * rng.standard_normal(base.logits.shape)).astype(np.float32)
    ref, kl_ref = oracle.draft_kl(inp.hidden, inp.logits0, teacher, w.heads, w.w_lm, K=K, row_index=ri)
    heads, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(d, F, V, heads, w_lm, max_rows=B * L, max_seqs=B, block_len=L,
                             flags=flags | binding.MRP_FLAG_TRAINING_KL)
    hid = harness.to_device(inp.hidden, w.dtype, DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    out = harness.alloc_draft_out(M, K, V, d, DEV)
    kl = torch.full((K, M), -1.0, device=DEV)
    binding.mrp_draft_kl(ctx, hid, l0, torch.from_numpy(teacher).to(DEV), torch.from_numpy(ri).to(DEV), M, K,
                         out.conf, out.lse, out.token, kl, margin=out.margin, status=out.status)
    torch.cuda.synchronize()
    check_stats(out, ref, dtype)
    got = kl.cpu().numpy().astype(np.float64)
    tol = TOL[dtype]
    assert kl_ref.min() > 0 and kl_ref.max() > 1e-2
    assert np.all(np.abs(got - kl_ref) <= tol + 2e-3 * kl_ref), np.abs(got - kl_ref).max()
    # the ordinary entry point on the same context afterwards: nothing of the KL call lingers
    out2 = harness.alloc_draft_out(M, K, V, d, DEV)
    harness.draft(ctx, hid, l0, torch.from_numpy(ri).to(DEV), M, K, out2)
    torch.cuda.synchronize()
    check_stats(out2, ref, dtype)
    binding.mrp_destroy(ctx)
    # a context without the flag has no room for the partial sums
    ctx = binding.mrp_create(d, F, V, heads, w_lm, max_rows=B * L, max_seqs=B, block_len=L, flags=flags)
    with pytest.raises(binding.MrpError) as ei:
        binding.mrp_draft_kl(ctx, hid, l0, torch.from_numpy(teacher).to(DEV), torch.from_numpy(ri).to(DEV), M, K,
                             out.conf, out.lse, out.token, kl)
    assert ei.value.status == 2
    binding.mrp_destroy(ctx)


# ---- base logits computed from the hidden states in the LM-head pass (mrp_draft_from_hidden) ----

@pytest.mark.parametrize("dtype,flags,d,F,V,B,L,K", [
    ("f32", 0, 72, 136, 1000, 5, 3, 3),                                # CUDA-core kernels, ragged sizes
    ("bf16", binding.MRP_FLAG_FORCE_SIMT, 72, 136, 1000, 5, 3, 2),
    ("bf16", 0, 256, 512, 4096, 2, 4, 2),                              # few-row LM head + head chain
    ("bf16", 0, 2048, 4096, 4096, 1, 4, 3),                            # the same at the 1.7B-class width
    ("bf16", 0, 128, 256, 2048, 10, 4, 3),                             # row-major LM head, 160 row-steps
    ("bf16", 0, 192, 320, 4112, 150, 1, 2),                            # two row blocks + step-0 rows of their own
    ("bf16", binding.MRP_FLAG_ROW_MAJOR_ONLY, 256, 512, 4096, 2, 4, 2),
])
def test_base_logits_from_hidden_states(dtype, flags, d, F, V, B, L, K):
    w = synth.make_weights(d, F, V, K, dtype, 55, head_std=0.05 if d <= 256 else 0.02)
    inp = synth.make_inputs(w, B, L, 55, 1.0, 4.0)
    gam = (1.0 + 0.25 * np.cos(np.arange(d))).astype(np.float32)
    if dtype == "bf16":
        gam = synth.bf16_round(gam)
    for g in (None, gam):
        out, fam = run_gpu_draft_from_hidden(w, inp, K, final_gamma=g, flags=flags, logits=True, hidden=True)
        assert fam == ("simt" if (dtype == "f32" or flags & binding.MRP_FLAG_FORCE_SIMT) else "tcgen05")
        ref = oracle.draft(inp.hidden, None, w.heads, w.w_lm, K=K, row_index=inp.row_index,
                           final_gamma=g, want_logits=True, want_hidden=True)
        check_stats(out, ref, dtype)
        lg = out.logits.cpu().numpy().astype(np.float64)
        rms = np.sqrt((ref.logits ** 2).mean(axis=2, keepdims=True))
        rel = 1e-4 if dtype == "f32" else 2e-2
        assert np.all(np.abs(lg - ref.logits) <= rel * np.maximum(np.abs(ref.logits), rms))
        assert np.abs(out.hidden.cpu().numpy() - ref.hidden).max() <= (1e-4 if dtype == "f32" else 2e-2)
    # a row subset, a shorter chain, and no chain at all (step 0 only)
    sub = inp.row_index[::2]
    for k in (max(K - 1, 1), 0):
        out, _ = run_gpu_draft_from_hidden(w, inp, k, final_gamma=gam, flags=flags, row_index=sub, hidden=True)
        ref = oracle.draft(inp.hidden, None, w.heads, w.w_lm, K=k, row_index=sub, final_gamma=gam, want_hidden=True)
        check_stats(out, ref, dtype)
        assert np.abs(out.hidden.cpu().numpy() - ref.hidden).max() <= (1e-4 if dtype == "f32" else 2e-2)
    # the ordinary entry point afterwards on a fresh context: nothing of the mode lingers
    out, _ = run_gpu_draft(w, inp, K, flags=flags)
    ref = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=K, row_index=inp.row_index)
    check_stats(out, ref, dtype)


# ---- block-state transition (mrp_commit) ----

def _state_to_device(tokens, B, L):
    st = harness.alloc_block_state(B, L, DEV)
    st.tokens.copy_(torch.from_numpy(tokens))
    return st


def _assert_state_equal(st, ref):
    n = int(st.n_masked.item())
    assert n == ref.row_index.size
    assert np.array_equal(st.tokens.cpu().numpy(), ref.tokens)
    assert np.array_equal(st.row_index.cpu().numpy()[:n], ref.row_index)
    assert np.array_equal(st.block_masked.cpu().numpy(), ref.block_masked)


@pytest.mark.parametrize("L", [1, 4, 31, 32, 33, 100, 1024])
def test_commit_bit_exact_for_the_three_decoding_modes(select_ctx, L):
    rng = np.random.default_rng(100 + L)
    for case in range(8):
        K = case % 4
        B = 1 + (case * 7) % 23
        tokens = np.where(rng.random(B * L) < 0.3 + 0.08 * case, -1, rng.integers(0, 999, B * L)).astype(np.int32)
        ri = np.flatnonzero(tokens < 0).astype(np.int32)
        if ri.size == 0:
            continue
        conf = rng.random((K + 1, ri.size)).astype(np.float32)
        tok = rng.integers(0, 1000, (K + 1, ri.size)).astype(np.int32)
        mode = binding.MRP_SELECT_STATIC if case % 3 else binding.MRP_SELECT_DYNAMIC_REMASK
        kw = dict(tau=0.5) if mode == binding.MRP_SELECT_DYNAMIC_REMASK else dict(r_reveal=1 + case % 2, r_draft=1)
        sel = _gpu_select(select_ctx, conf, tok, ri, B, L, mode, **kw)
        osel = oracle.select(conf, tok, ri, B, L, oracle.STATIC if mode == binding.MRP_SELECT_STATIC else oracle.DYNAMIC_REMASK, **kw)
        _assert_select_equal(sel, osel)
        # direct decoding / remasking: everything selected is unmasked
        st = _state_to_device(tokens, B, L)
        harness.commit(select_ctx, sel, st, B, L, K)
        torch.cuda.synchronize()
        _assert_state_equal(st, oracle.commit(tokens, osel, B, L))
        # speculative decoding: drafts only where the backbone agreed
        if mode == binding.MRP_SELECT_STATIC and K > 0:
            vt = np.where(rng.random((B, K)) < 0.6, osel.draft_tok, -5).astype(np.int32)
            alen = torch.empty(B, device=DEV, dtype=torch.int32)
            amask = torch.empty((B, K), device=DEV, dtype=torch.int8)
            binding.mrp_verify(select_ctx, sel.draft_tok, torch.from_numpy(vt).to(DEV), sel.draft_len, B, K,
                               bool(case & 4), alen, amask)
            _, oacc = oracle.verify(osel.draft_tok, vt, osel.draft_len, positionwise=bool(case & 4))
            st = _state_to_device(tokens, B, L)
            harness.commit(select_ctx, sel, st, B, L, K, accept_mask=amask)
            torch.cuda.synchronize()
            _assert_state_equal(st, oracle.commit(tokens, osel, B, L, accept_mask=oacc))


@pytest.mark.parametrize("mode", ["direct", "speculative", "remask"])
def test_denoising_loop_with_the_block_state_on_the_device(select_ctx, mode):
    """Algorithms 2-4 as a loop: the statistics of every forward are synthetic (one random table
    per forward, gathered at the masked positions), selection, verification and the state
    transition run on the device; the oracle runs the same loop.  States must agree after
    every forward, and both must finish together."""
    rng = np.random.default_rng({"direct": 1, "speculative": 2, "remask": 3}[mode])
    B, L, K = 9, 32, 2 if mode != "remask" else 1
    tokens = np.full(B * L, -1, np.int32)
    st = _state_to_device(tokens, B, L)
    n_forwards = 0
    while (tokens < 0).any():
        conf_full = rng.random((K + 1, B * L)).astype(np.float32)
        tok_full = rng.integers(0, 1000, (K + 1, B * L)).astype(np.int32)
        n = int(st.n_masked.item())
        ri_dev = st.row_index[:n].clone()              # the device's own list of masked positions
        ri = np.flatnonzero(tokens < 0).astype(np.int32)
        assert np.array_equal(ri_dev.cpu().numpy(), ri)
        conf, tok = conf_full[:, ri], tok_full[:, ri]
        sel = harness.alloc_select_out(B, L, K, DEV)
        c, t = torch.from_numpy(np.ascontiguousarray(conf)).to(DEV), torch.from_numpy(np.ascontiguousarray(tok)).to(DEV)
        if mode == "remask":
            harness.select(select_ctx, c, t, ri_dev, n, K, B, L, binding.MRP_SELECT_DYNAMIC_REMASK, sel, tau=0.6)
            osel = oracle.select(conf, tok, ri, B, L, oracle.DYNAMIC_REMASK, tau=0.6)
            harness.commit(select_ctx, sel, st, B, L, K)
            ref = oracle.commit(tokens, osel, B, L)
        else:
            harness.select(select_ctx, c, t, ri_dev, n, K, B, L, binding.MRP_SELECT_STATIC, sel)
            osel = oracle.select(conf, tok, ri, B, L, oracle.STATIC)
            if mode == "direct":
                harness.commit(select_ctx, sel, st, B, L, K)
                ref = oracle.commit(tokens, osel, B, L)
            else:
                vt = np.where(rng.random((B, K)) < 0.7, osel.draft_tok, -5).astype(np.int32)
                alen = torch.empty(B, device=DEV, dtype=torch.int32)
                amask = torch.empty((B, K), device=DEV, dtype=torch.int8)
                binding.mrp_verify(select_ctx, sel.draft_tok, torch.from_numpy(vt).to(DEV), sel.draft_len, B, K,
                                   False, alen, amask)
                harness.commit(select_ctx, sel, st, B, L, K, accept_mask=amask)
                _, oacc = oracle.verify(osel.draft_tok, vt, osel.draft_len)
                ref = oracle.commit(tokens, osel, B, L, accept_mask=oacc)
        torch.cuda.synchronize()
        _assert_state_equal(st, ref)
        assert ref.row_index.size < ri.size                  # every forward makes progress
        tokens = ref.tokens
        n_forwards += 1
        assert n_forwards <= L
    if mode == "direct":
        assert n_forwards == -(-L // (K + 1))
    assert int(st.n_masked.item()) == 0 and int(st.block_masked.sum().item()) == 0


def test_commit_with_more_blocks_than_one_round_of_the_prefix_sum():
    w = synth.make_weights(16, 16, 32, 0, "f32", 1)
    heads, w_lm = harness.upload_weights(w, DEV)
    B, L, K = 2500, 3, 1
    ctx = binding.mrp_create(16, 16, 32, heads, w_lm, max_rows=4, max_seqs=B, block_len=L)
    rng = np.random.default_rng(77)
    tokens = np.where(rng.random(B * L) < 0.7, -1, rng.integers(0, 999, B * L)).astype(np.int32)
    ri = np.flatnonzero(tokens < 0).astype(np.int32)
    conf = rng.random((K + 1, ri.size)).astype(np.float32)
    tok = rng.integers(0, 1000, (K + 1, ri.size)).astype(np.int32)
    sel = _gpu_select(ctx, conf, tok, ri, B, L, binding.MRP_SELECT_STATIC)
    osel = oracle.select(conf, tok, ri, B, L, oracle.STATIC)
    st = _state_to_device(tokens, B, L)
    harness.commit(ctx, sel, st, B, L, K)
    torch.cuda.synchronize()
    _assert_state_equal(st, oracle.commit(tokens, osel, B, L))
    binding.mrp_destroy(ctx)


@pytest.mark.parametrize("d,F,V,B,L,K", [
    (2048, 4096, 4096, 1, 4, 3),      # head chain with grid barriers, few-row LM head
    (512, 1024, 2048, 100, 1, 2),     # 128-row chain: parked slices, tile barriers, row-major LM head
    (256, 512, 4096, 75, 4, 2),       # row-major kernels throughout
])
def test_repeated_calls_give_bit_identical_outputs(d, F, V, B, L, K):
    """Sums over CTAs are taken in a fixed order (slice order, fixed-point integer adds for the row
    sums of squares, fixed merge order of the softmax partials): 200 calls, no bit may move."""
    w = synth.make_weights(d, F, V, K, "bf16", 91, head_std=0.05 if d <= 512 else 0.02)
    inp = synth.make_inputs(w, B, L, 91, 1.0, 4.0)
    heads, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(w.d, w.F, w.V, heads, w_lm, max_rows=B * L, max_seqs=B, block_len=L)
    M = B * L
    hid = harness.to_device(inp.hidden, w.dtype, DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    out = harness.alloc_draft_out(M, K, w.V, w.d, DEV, margin=True, hidden=True)
    for from_hidden in (False, True):
        ref = None
        for i in range(200):
            if from_hidden:
                harness.draft_from_hidden(ctx, hid, None, None, M, K, out)
            else:
                harness.draft(ctx, hid, l0, None, M, K, out)
            if i % 40 == 0 or i == 199:
                torch.cuda.synchronize()
                cur = [t.clone() for t in (out.conf, out.lse, out.token, out.margin, out.hidden)]
                if ref is None:
                    ref = cur
                assert all(torch.equal(a, b) for a, b in zip(cur, ref)), i
        assert int(out.status.item()) == 0
    binding.mrp_destroy(ctx)


def test_draft_waits_for_the_base_logits_event_before_the_lm_head():
    """mrp_set_logits0_event: the base logits arrive late on another stream (after a sleep kernel);
    the call enqueued meanwhile must give the results of a call that had them from the start."""
    w = synth.make_weights(256, 512, 4096, 2, "bf16", 17, head_std=0.05)
    inp = synth.make_inputs(w, 2, 4, 17, 1.0, 4.0)
    heads, w_lm = harness.upload_weights(w, DEV)
    M, K = 8, 2
    hid = harness.to_device(inp.hidden, w.dtype, DEV)
    l0_host = torch.from_numpy(inp.logits0).pin_memory()
    for flags in (0, binding.MRP_FLAG_FORCE_SIMT, binding.MRP_FLAG_ROW_MAJOR_ONLY):
        ctx = binding.mrp_create(w.d, w.F, w.V, heads, w_lm, max_rows=M, max_seqs=2, block_len=4, flags=flags)
        ref = harness.alloc_draft_out(M, K, w.V, w.d, DEV)
        harness.draft(ctx, hid, l0_host.to(DEV), None, M, K, ref)
        torch.cuda.synchronize()
        l0 = torch.full((M, w.V), 1e30, device=DEV)          # poison until the late copy lands
        side, ready = torch.cuda.Stream(), torch.cuda.Event()
        with torch.cuda.stream(side):
            torch.cuda._sleep(40_000_000)                     # some 20 ms
            l0.copy_(l0_host, non_blocking=True)
            ready.record(side)
        binding.mrp_set_logits0_event(ctx, ready)
        out = harness.alloc_draft_out(M, K, w.V, w.d, DEV)
        harness.draft(ctx, hid, l0, None, M, K, out)
        torch.cuda.synchronize()
        assert torch.equal(out.conf, ref.conf) and torch.equal(out.token, ref.token) and torch.equal(out.lse, ref.lse)
        assert int(out.status.item()) == 0
        binding.mrp_set_logits0_event(ctx, None)
        binding.mrp_destroy(ctx)
