"""Full-size parity: the five benchmark configurations run through the C ABI at their real
shapes, in the launch configuration the benchmark times (default flags); the oracle recomputes
every row where there are at most 256, else 256 or more rows (whole blocks) spread so that every
128-row block of the stacked row-steps is hit, over all V columns.  Some of the compared rows have
their top token planted in the first and in the last 16 entries of the vocabulary, i.e. in the
first and the last CTA's range."""
import gc

import numpy as np
import pytest
import torch

import oracle
from paper_2605_18817_b200 import binding, harness, synth
from test_gpu_parity import DEV, _assert_select_equal, check_stats

pytestmark = pytest.mark.gpu


class Device:
    """Weights uploaded once, contexts created per (rows, seqs, block) shape."""

    def __init__(self, w):
        self.w = w
        self.heads, self.w_lm = harness.upload_weights(w, DEV)
        self.w_lm_f32 = None

    def logits_fn(self, rows):
        # base logits of the synthetic backbone: fp32 product on the device (input data)
        if self.w_lm_f32 is None:
            torch.backends.cuda.matmul.allow_tf32 = False
        x = torch.from_numpy(rows).to(DEV)
        out = torch.empty((x.shape[0], self.w.V), device=DEV)
        step = 16384
        for v0 in range(0, self.w.V, step):
            out[:, v0:v0 + step] = x @ self.w_lm[v0:v0 + step].float().T
        return out.cpu().numpy()

    def ctx(self, rows, seqs, block, n_heads=None, flags=0):
        heads = self.heads if n_heads is None else self.heads[:n_heads]
        return binding.mrp_create(self.w.d, self.w.F, self.w.V, heads, self.w_lm, max_rows=rows,
                                  max_seqs=seqs, block_len=block, flags=flags)


def spread_rows(M, n=256):
    """n row numbers spread evenly over 0..M-1 (all of them if M <= n), first and last included."""
    if M <= n:
        return np.arange(M)
    return np.unique(np.round(np.linspace(0, M - 1, n)).astype(np.int64))


def plant_vocabulary_ends(cfg, rows):
    """Planted tokens of a configuration with those of the dense positions `rows` moved to the two
    ends of the vocabulary, alternating."""
    n, V = cfg["B"] * cfg["L"], cfg["V"]
    planted = synth._rng(cfg["seed"], synth._S_TOK).integers(0, V, size=n, dtype=np.int64).astype(np.int32)
    for i, r in enumerate(rows):
        planted[r] = (i // 2) % 16 if i % 2 == 0 else V - 1 - (i // 2) % 16
    return planted


def gpu_draft(dev, ctx, inp, K, **kw):
    M = len(inp.row_index)
    hid = harness.to_device(inp.hidden, dev.w.dtype, DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    ri = torch.from_numpy(inp.row_index).to(DEV)
    out = harness.alloc_draft_out(M, K, dev.w.V, dev.w.d, DEV, **kw)
    harness.draft(ctx, hid, l0, ri, M, K, out)
    torch.cuda.synchronize()
    return out, ri


def test_config1_decode_shape_all_rows():
    cfg = synth.CONFIGS[1]
    w = synth.make_weights(cfg["d"], cfg["F"], cfg["V"], cfg["n_heads"], cfg["dtype"], cfg["seed"])
    dev = Device(w)
    _, inp = synth.make_config(cfg, w)
    ctx = dev.ctx(4, 1, 4)
    out, ri = gpu_draft(dev, ctx, inp, cfg["K"], logits=True, hidden=True)
    ref = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=cfg["K"], row_index=inp.row_index,
                       want_logits=True, want_hidden=True)
    check_stats(out, ref, "bf16")
    lg = out.logits.cpu().numpy().astype(np.float64)
    rms = np.sqrt((ref.logits ** 2).mean(axis=2, keepdims=True))
    assert np.all(np.abs(lg - ref.logits) <= 2e-2 * np.maximum(np.abs(ref.logits), rms))
    assert np.abs(out.hidden.cpu().numpy() - ref.hidden).max() <= 2e-2
    # static reveal + drafts, then verification against synthetic backbone tokens
    K, B, L, M = cfg["K"], 1, 4, 4
    sel = harness.alloc_select_out(B, L, K, DEV)
    harness.select(ctx, out.conf, out.token, ri, M, K, B, L, binding.MRP_SELECT_STATIC, sel)
    torch.cuda.synchronize()
    osel = oracle.select(out.conf.cpu().numpy(), out.token.cpu().numpy(), inp.row_index, B, L,
                         oracle.STATIC)
    _assert_select_equal(sel, osel)
    binding.mrp_destroy(ctx)


def test_config1_decode_shape_base_logits_from_hidden_states():
    """Config 1 through mrp_draft_from_hidden (no base logits handed over), with and without the
    backbone's final norm; all rows and all vocabulary entries against the oracle."""
    cfg = synth.CONFIGS[1]
    w = synth.make_weights(cfg["d"], cfg["F"], cfg["V"], cfg["n_heads"], cfg["dtype"], cfg["seed"])
    dev = Device(w)
    _, inp = synth.make_config(cfg, w)
    ctx = dev.ctx(4, 1, 4)
    K, M = cfg["K"], 4
    hid = harness.to_device(inp.hidden, w.dtype, DEV)
    ri = torch.from_numpy(inp.row_index).to(DEV)
    gam = synth.bf16_round((1.0 + 0.25 * np.cos(np.arange(w.d))).astype(np.float32))
    for g in (None, gam):
        out = harness.alloc_draft_out(M, K, w.V, w.d, DEV, logits=True, hidden=True)
        harness.draft_from_hidden(ctx, hid, None if g is None else harness.to_device(g, w.dtype, DEV),
                                  ri, M, K, out)
        torch.cuda.synchronize()
        ref = oracle.draft(inp.hidden, None, w.heads, w.w_lm, K=K, row_index=inp.row_index,
                           final_gamma=g, want_logits=True, want_hidden=True)
        check_stats(out, ref, "bf16")
        lg = out.logits.cpu().numpy().astype(np.float64)
        rms = np.sqrt((ref.logits ** 2).mean(axis=2, keepdims=True))
        assert np.all(np.abs(lg - ref.logits) <= 2e-2 * np.maximum(np.abs(ref.logits), rms))
    # without a final norm the synthetic base logits are W_lm h_0 rounded to fp32: the ordinary
    # entry point on those must give the same statistics up to that rounding
    out_b, _ = gpu_draft(dev, ctx, inp, K)
    out_a = harness.alloc_draft_out(M, K, w.V, w.d, DEV)
    harness.draft_from_hidden(ctx, hid, None, ri, M, K, out_a)
    torch.cuda.synchronize()
    assert torch.allclose(out_a.lse, out_b.lse, atol=1e-3) and torch.allclose(out_a.conf, out_b.conf, atol=1e-3)
    binding.mrp_destroy(ctx)


def test_config2_speculative_shape_sampled_rows_and_verify():
    cfg = synth.CONFIGS[2]
    w = synth.make_weights(cfg["d"], cfg["F"], cfg["V"], cfg["n_heads"], cfg["dtype"], cfg["seed"])
    dev = Device(w)
    _, inp = synth.make_config(cfg, w, logits_fn=dev.logits_fn, planted=plant_vocabulary_ends(cfg, range(0, 8)))
    K, B, L = cfg["K"], cfg["B"], cfg["L"]
    M = len(inp.row_index)
    assert M == 128
    ctx = dev.ctx(M, B, L)
    out, ri = gpu_draft(dev, ctx, inp, K)
    # every row of the configuration against the oracle
    ref = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=K, row_index=inp.row_index)
    check_stats(out, ref, "bf16")
    assert ref.token[0, 0] == 0 and ref.token[0, 1] == w.V - 1       # the planted ends of the vocabulary
    # selection on the device's own statistics is bit-exact against the oracle's rules
    sel = harness.alloc_select_out(B, L, K, DEV)
    harness.select(ctx, out.conf, out.token, ri, M, K, B, L, binding.MRP_SELECT_STATIC, sel)
    torch.cuda.synchronize()
    osel = oracle.select(out.conf.cpu().numpy(), out.token.cpu().numpy(), inp.row_index, B, L,
                         oracle.STATIC)
    _assert_select_equal(sel, osel)
    # verification: backbone tokens equal the draft with probability 0.7 per slot
    dt = sel.draft_tok.cpu().numpy()
    vt = synth.make_verify_tokens(dt, w.V, cfg["seed"], 0.7)
    al, am = harness.verify(ctx, sel.draft_tok, torch.from_numpy(vt).to(DEV), sel.draft_len)
    torch.cuda.synchronize()
    ol, om = oracle.verify(dt, vt, sel.draft_len.cpu().numpy())
    assert np.array_equal(al.cpu().numpy(), ol) and np.array_equal(am.cpu().numpy(), om)
    assert 0 < ol.mean() < K
    binding.mrp_destroy(ctx)
    del dev, w
    gc.collect()


def test_config3_remask_shape_sampled_blocks():
    cfg = synth.CONFIGS[3]
    w = synth.make_weights(cfg["d"], cfg["F"], cfg["V"], cfg["n_heads"], cfg["dtype"], cfg["seed"])
    dev = Device(w)
    _, inp = synth.make_config(cfg, w, logits_fn=dev.logits_fn, planted=plant_vocabulary_ends(cfg, range(0, 32)))
    K, B, L, tau = cfg["K"], cfg["B"], cfg["L"], cfg["tau"]
    M = len(inp.row_index)
    assert 850 < M < 1200
    ctx = dev.ctx(B * L, B, L)
    out, ri = gpu_draft(dev, ctx, inp, K)
    for policy in (0, 1):
        sel = harness.alloc_select_out(B, L, K, DEV)
        harness.select(ctx, out.conf, out.token, ri, M, K, B, L, binding.MRP_SELECT_DYNAMIC_REMASK,
                       sel, tau=tau, remask_policy=policy)
        torch.cuda.synchronize()
        # (i) the rules, bit-exact, on the device's own statistics
        osel = oracle.select(out.conf.cpu().numpy(), out.token.cpu().numpy(), inp.row_index, B, L,
                             oracle.DYNAMIC_REMASK, tau=tau, remask_policy=policy)
        _assert_select_equal(sel, osel)
        assert 0 < osel.remask_mask.sum() < osel.reveal_mask.sum()
    # (ii) end to end on every fourth block and the last (some 270 rows, two or more in every 128-row
    # block of the stacked row-steps), recomputed by the oracle
    blocks = sorted(set(range(0, B, 4)) | {B - 1})
    rows = np.flatnonzero(np.isin(inp.row_index // L, blocks))
    assert rows.size >= 256 and np.all(np.diff(rows) < 128)
    ref = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=K, row_index=inp.row_index[rows])
    check_stats(out, ref, "bf16", cols=rows)
    checked = 0
    sel_np = {n: getattr(sel, n).cpu().numpy() for n in ("reveal_mask", "remask_mask", "out_token")}
    for b in blocks:
        r = np.flatnonzero(inp.row_index[rows] // L == b)
        conf_b = ref.conf[:, r].astype(np.float32)
        if np.abs(conf_b - tau).min() < 2e-3 or (ref.margin[:, r] <= 1e-2).any():
            continue                      # a decision inside the tolerance band: not unique
        ri_b = (inp.row_index[rows][r] % L).astype(np.int32)
        o = oracle.select(conf_b, ref.token[:, r], ri_b, 1, L, oracle.DYNAMIC_REMASK, tau=tau,
                          remask_policy=1)
        sl = slice(b * L, (b + 1) * L)
        assert np.array_equal(sel_np["reveal_mask"][sl], o.reveal_mask)
        assert np.array_equal(sel_np["remask_mask"][sl], o.remask_mask)
        assert np.array_equal(sel_np["out_token"][sl], o.out_token)
        checked += 1
    assert checked >= 2
    binding.mrp_destroy(ctx)
    del dev, w
    gc.collect()


@pytest.fixture(scope="module")
def sweep_dev():
    w = synth.make_weights(4096, 8192, 151936, 4, "bf16", 4000)
    dev = Device(w)
    yield dev


@pytest.mark.parametrize("M,K", [(1, 1), (4, 2), (16, 4), (64, 2), (256, 4), (1024, 1), (4096, 4)])
def test_sweep_points_sampled_rows(sweep_dev, M, K):
    dev = sweep_dev
    cfg = synth.sweep_config(M, K)
    sample = spread_rows(M)
    _, inp = synth.make_config(cfg, dev.w, logits_fn=dev.logits_fn,
                               planted=plant_vocabulary_ends(cfg, [sample[0], sample[-1]]))
    ctx = dev.ctx(M, M, 1, n_heads=K)
    out, _ = gpu_draft(dev, ctx, inp, K, margin=False)
    ref = oracle.draft(inp.hidden, inp.logits0, dev.w.heads, dev.w.w_lm, K=K,
                       row_index=inp.row_index[sample])
    check_stats(out, ref, "bf16", cols=sample)
    # properties that hold at any size, checked on every row
    conf = out.conf.cpu().numpy()
    assert np.all(conf > 1.0 / dev.w.V) and np.all(conf <= 1.0 + 1e-6)
    tok = out.token.cpu().numpy()
    assert tok.min() >= 0 and tok.max() < dev.w.V
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    assert torch.equal(l0.argmax(dim=1).int().cpu(), out.token[0].cpu())
    assert torch.allclose(torch.logsumexp(l0, dim=1), out.lse[0], atol=2e-3)
    binding.mrp_destroy(ctx)


@pytest.mark.parametrize("M,K", [(4, 2), (64, 2), (256, 4), (1024, 1)])
def test_sweep_points_base_logits_from_hidden_states(sweep_dev, M, K):
    dev = sweep_dev
    cfg = synth.sweep_config(M, K)
    _, inp = synth.make_config(cfg, dev.w, logits_fn=dev.logits_fn)
    ctx = dev.ctx(M, M, 1, n_heads=K)
    hid = harness.to_device(inp.hidden, dev.w.dtype, DEV)
    ri = torch.from_numpy(inp.row_index).to(DEV)
    gam = synth.bf16_round((1.0 + 0.25 * np.cos(np.arange(dev.w.d))).astype(np.float32))
    out = harness.alloc_draft_out(M, K, dev.w.V, dev.w.d, DEV, margin=False)
    harness.draft_from_hidden(ctx, hid, harness.to_device(gam, dev.w.dtype, DEV), ri, M, K, out)
    torch.cuda.synchronize()
    sample = spread_rows(M)
    ref = oracle.draft(inp.hidden, None, dev.w.heads, dev.w.w_lm, K=K, row_index=inp.row_index[sample],
                       final_gamma=gam)
    check_stats(out, ref, "bf16", cols=sample)
    conf = out.conf.cpu().numpy()
    assert np.all(conf > 1.0 / dev.w.V) and np.all(conf <= 1.0 + 1e-6)
    binding.mrp_destroy(ctx)


@pytest.mark.parametrize("M,K", [(16, 2), (64, 4), (256, 1), (1024, 2), (4096, 4)])
def test_fp16_operand_mode_stays_close_to_exact_operands_on_every_row(sweep_dev, M, K):
    """Above 32 row-steps the LM head rounds its activation operand once to fp16 instead of
    carrying a bf16 hi + lo pair.  Every row-step of the call is compared with the same call
    under MRP_FLAG_EXACT_OPERANDS (itself checked against the oracle on sampled rows above):
    the two must agree well inside the 2e-3 tolerance, which leaves the exact path's own error
    as margin."""
    dev = sweep_dev
    cfg = synth.sweep_config(M, K)
    _, inp = synth.make_config(cfg, dev.w, logits_fn=dev.logits_fn)
    outs = []
    for flags in (0, binding.MRP_FLAG_EXACT_OPERANDS):
        ctx = dev.ctx(M, M, 1, n_heads=K, flags=flags)
        out, _ = gpu_draft(dev, ctx, inp, K, margin=True)
        outs.append(out)
        binding.mrp_destroy(ctx)
    a, b = outs
    dconf = (a.conf - b.conf).abs().max().item()
    dlse = (a.lse - b.lse).abs().max().item()
    print("M=%d K=%d max|dconf|=%.2e max|dlse|=%.2e" % (M, K, dconf, dlse))
    assert dconf <= 1.5e-3 and dlse <= 1.5e-3
    clear = b.margin > 1e-2
    assert torch.equal(a.token[clear], b.token[clear])
    assert torch.equal(a.conf[0], b.conf[0])          # step 0 never touches the operands


@pytest.mark.parametrize("M,K", [(16, 2), (64, 4), (256, 1), (1024, 2), (4096, 1)])
def test_fp16_operand_mode_of_the_base_logits_pass_stays_close_to_exact_operands(sweep_dev, M, K):
    """The same comparison for mrp_draft_from_hidden, where the base logits go through the
    operand as well: every row-step, step 0 included, against MRP_FLAG_EXACT_OPERANDS."""
    dev = sweep_dev
    cfg = synth.sweep_config(M, K)
    _, inp = synth.make_config(cfg, dev.w, logits_fn=dev.logits_fn)
    hid = harness.to_device(inp.hidden, dev.w.dtype, DEV)
    ri = torch.from_numpy(inp.row_index).to(DEV)
    gam = harness.to_device(synth.bf16_round((1.0 + 0.25 * np.cos(np.arange(dev.w.d))).astype(np.float32)),
                            dev.w.dtype, DEV)
    for g in (None, gam):
        outs = []
        for flags in (0, binding.MRP_FLAG_EXACT_OPERANDS):
            ctx = dev.ctx(M, M, 1, n_heads=K, flags=flags)
            out = harness.alloc_draft_out(M, K, dev.w.V, dev.w.d, DEV, margin=True)
            harness.draft_from_hidden(ctx, hid, g, ri, M, K, out)
            torch.cuda.synchronize()
            outs.append(out)
            binding.mrp_destroy(ctx)
        a, b = outs
        dconf = (a.conf - b.conf).abs().max().item()
        dlse = (a.lse - b.lse).abs().max().item()
        print("M=%d K=%d norm=%s max|dconf|=%.2e max|dlse|=%.2e" % (M, K, g is not None, dconf, dlse))
        assert dconf <= 1.5e-3 and dlse <= 1.5e-3
        clear = b.margin > 1e-2
        assert torch.equal(a.token[clear], b.token[clear])
