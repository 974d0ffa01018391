"""The token-conditioned MRP module (mrp_module_step) against the oracle's module, step by step through
the direct-decoding loop of Algorithm 2: after every MRP step the running hidden states, the statistics of
the running logits l <- l + delta and the reveal they drive are compared, and the tokens revealed so far
condition the next step on both sides."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_18817_b200 import binding, harness, synth
from test_gpu_parity import DEV, TOL

pytestmark = pytest.mark.gpu


def upload_module(mw, dtype):
    up = lambda a: harness.to_device(a, dtype, DEV)
    return up(mw.emb), up(mw.w_proj), [{k: up(v) for k, v in lay.items()} for lay in mw.layers]


@pytest.mark.parametrize("dtype,flags,d,F,V,D,heads,B,L,steps", [
    ("f32", 0, 64, 96, 512, 2, 4, 3, 4, 3),                                 # CUDA-core LM head
    ("bf16", binding.MRP_FLAG_FORCE_SIMT, 64, 96, 512, 1, 2, 2, 5, 2),
    ("bf16", 0, 256, 512, 4096, 3, 4, 1, 4, 3),                             # the paper's depth; few-row tcgen05 LM head
    ("bf16", 0, 128, 256, 2048, 2, 4, 10, 4, 2),                            # 80 row-steps: row-major LM head, fp16 operand
    ("bf16", 0, 256, 512, 4096, 0, 4, 2, 4, 1),                             # the fusion projection alone
    # more than four positions on a tensor-core context: the module's products run on the row-major tcgen05 kernel
    ("bf16", 0, 128, 256, 2048, 2, 4, 5, 32, 2),                            # 160 positions: two row blocks, blocks of 32
    ("bf16", 0, 192, 320, 2064, 3, 3, 3, 5, 2),                             # 15 positions, ragged tiles, three layers
    ("bf16", 0, 256, 512, 4096, 2, 4, 3, 4, 2),                             # 12 positions, three units per CTA
    ("bf16", 0, 512, 1024, 4096, 1, 4, 40, 4, 2),                           # 160 positions, two row blocks, wider model
    ("bf16", binding.MRP_FLAG_NO_CHAIN, 256, 512, 4096, 2, 4, 3, 4, 2),     # the few-row kernels, one launch per product
    ("bf16", 0, 256, 512, 4096, 3, 2, 2, 32, 2),                            # two blocks of 32: a layer as one kernel, 64 rows
    ("bf16", binding.MRP_FLAG_NO_CHAIN, 128, 256, 2048, 1, 4, 1, 48, 2),    # a block of 48 through the separate attention kernel
    # four positions or fewer: the module step is one cooperative kernel
    ("f32", 0, 64, 96, 512, 2, 4, 1, 4, 3),                                 # fp32 weights, ragged widths
    ("bf16", binding.MRP_FLAG_FORCE_SIMT, 256, 512, 1024, 2, 2, 1, 3, 2),   # 16-byte weight loads, block of three
    ("bf16", 0, 256, 512, 4096, 0, 4, 1, 4, 2),                             # no layers
    ("bf16", binding.MRP_FLAG_NO_CHAIN, 256, 512, 4096, 3, 4, 1, 4, 3),     # the same shape as one kernel per product
])
def test_module_steps_follow_the_oracle_through_direct_decoding(dtype, flags, d, F, V, D, heads, B, L, steps):
    w = synth.make_weights(d, F, V, 1, dtype, 41)
    mw = synth.make_module_weights(d, F, V, D, heads, dtype, 41, std=0.06, proj_std=0.3 / np.sqrt(2 * d))
    inp = synth.make_inputs(w, B, L, 41, 1.0, 3.0)
    n = B * L
    heads_dev, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(d, F, V, heads_dev, w_lm, max_rows=n, max_seqs=B, block_len=L, flags=flags)
    emb, w_proj, layers = upload_module(mw, dtype)
    binding.mrp_module_attach(ctx, emb, w_proj, layers, heads, mw.mask_token)
    hid0 = harness.to_device(inp.hidden, dtype, DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    h_state = torch.empty((n, d), device=DEV, dtype=torch.float32)
    tol = TOL[dtype] if dtype == "bf16" else 5e-5          # fp32: D layers of fp32 sums in front of the LM head

    tokens = np.full(n, -1, np.int32)                       # x_t: the active blocks, fully masked
    h_run = inp.hidden.astype(np.float64)                   # oracle's running h
    l_run = inp.logits0.astype(np.float64)                  # oracle's running l
    conf0, lse0, tok0, margin0 = oracle.stats(l_run)
    # the backbone's own reveal (Algorithm 2: r tokens of highest confidence before the MRP steps)
    sel = oracle.select(conf0[None, :].astype(np.float32), tok0[None, :], None, B, L, oracle.STATIC, r_reveal=1)
    tokens = np.where(sel.out_token >= 0, sel.out_token, tokens).astype(np.int32)
    for s in range(1, steps + 1):
        ri = np.flatnonzero(tokens < 0).astype(np.int32)
        M = ri.size
        if M == 0:
            break
        out = harness.alloc_draft_out(M, 1, V, d, DEV, hidden=True)
        binding.mrp_module_step(ctx, torch.from_numpy(tokens).to(DEV), hid0, h_state, l0, torch.from_numpy(ri).to(DEV),
                                M, B, L, s == 1, out.conf, out.lse, out.token, margin=out.margin,
                                hidden_out=out.hidden, status=out.status)
        torch.cuda.synchronize()
        assert int(out.status.item()) == 0
        dh, dl = oracle.module(h_run.astype(np.float32), tokens, B, L, mw.emb, mw.w_proj, mw.layers, w.w_lm, heads,
                               mw.mask_token, row_index=ri)
        assert D == 0 or np.abs(dh).max() > 1e-2
        h_run = h_run.astype(np.float32).astype(np.float64) + dh
        l_run[ri] += dl
        conf, lse, tok, margin = oracle.stats(l_run[ri])
        assert np.abs(h_state.cpu().numpy() - h_run).max() <= 1e-3 * max(1.0, np.abs(h_run).max())
        assert np.abs(out.hidden.cpu().numpy() - h_run[ri]).max() <= 1e-3 * max(1.0, np.abs(h_run).max())
        g_conf, g_lse, g_tok = (t.cpu().numpy() for t in (out.conf, out.lse, out.token))
        assert np.abs(g_conf[1] - conf).max() <= tol and np.abs(g_lse[1] - lse).max() <= tol
        assert np.abs(g_conf[0] - conf0[ri]).max() <= tol and np.abs(g_lse[0] - lse0[ri]).max() <= tol
        clear = margin > 1e-2
        assert np.array_equal(g_tok[1][clear], tok[clear])
        # reveal from the updated logits: the device's rule on its own statistics is the oracle's rule
        gsel = harness.alloc_select_out(B, L, 0, DEV)
        harness.select(ctx, out.conf[1:2].contiguous(), out.token[1:2].contiguous(), torch.from_numpy(ri).to(DEV), M, 0,
                       B, L, binding.MRP_SELECT_STATIC, gsel, r_reveal=1)
        torch.cuda.synchronize()
        osel_g = oracle.select(g_conf[1:2], g_tok[1:2], ri, B, L, oracle.STATIC, r_reveal=1)
        assert np.array_equal(gsel.out_token.cpu().numpy(), osel_g.out_token)
        # the oracle's own reveal conditions the next step on both sides
        osel = oracle.select(conf[None, :].astype(np.float32), tok[None, :], ri, B, L, oracle.STATIC, r_reveal=1)
        tokens = np.where(osel.out_token >= 0, osel.out_token, tokens).astype(np.int32)
    binding.mrp_destroy(ctx)


@pytest.mark.parametrize("B,L", [(2, 4), (1, 4)])          # one kernel per product / one kernel for the step
def test_module_step_checks_tokens_and_needs_an_attached_module(B, L):
    d, F, V = 64, 96, 512
    n = B * L
    w = synth.make_weights(d, F, V, 1, "f32", 43)
    mw = synth.make_module_weights(d, F, V, 1, 2, "f32", 43, std=0.05)
    inp = synth.make_inputs(w, B, L, 43, 1.0, 3.0)
    heads_dev, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(d, F, V, heads_dev, w_lm, max_rows=n, max_seqs=B, block_len=L)
    hid0 = harness.to_device(inp.hidden, "f32", DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    h_state = torch.empty((n, d), device=DEV)
    out = harness.alloc_draft_out(n, 1, V, d, DEV)
    tok = torch.full((n,), -1, device=DEV, dtype=torch.int32)
    with pytest.raises(binding.MrpError) as ei:
        binding.mrp_module_step(ctx, tok, hid0, h_state, l0, None, n, B, L, True, out.conf, out.lse, out.token)
    assert ei.value.status == 2
    emb, w_proj, layers = upload_module(mw, "f32")
    binding.mrp_module_attach(ctx, emb, w_proj, layers, 2, mw.mask_token)
    # a token id outside the embedding table is read as masked and raises the bit
    bad = tok.clone()
    bad[3] = V + 5
    binding.mrp_module_step(ctx, bad, hid0, h_state, l0, None, n, B, L, True, out.conf, out.lse, out.token, status=out.status)
    torch.cuda.synchronize()
    assert int(out.status.item()) == binding.MRP_DEV_BAD_INDEX
    ref = harness.alloc_draft_out(n, 1, V, d, DEV)
    binding.mrp_module_step(ctx, tok, hid0, h_state, l0, None, n, B, L, True, ref.conf, ref.lse, ref.token, status=ref.status)
    torch.cuda.synchronize()
    assert int(ref.status.item()) == 0 and torch.equal(ref.conf, out.conf) and torch.equal(ref.token, out.token)
    binding.mrp_destroy(ctx)


@pytest.mark.parametrize("which,L,blocks_checked", [
    (1, 4, 1),      # the decode shape, one block of 4: the step as one cooperative CUDA-core kernel
    (1, 16, 1),     # the same with the paper's block of 16: products on the few-row tensor-core kernels
    (2, 4, 2),      # 32 blocks of 4 at d = 4096: products on the row-major tensor-core kernel; oracle on two blocks
])
def test_module_step_at_the_benchmark_shapes(which, L, blocks_checked):
    """One module step at the shapes bench.py times (D = 3, 128 features per attention head), in the launch
    configuration it times, against the oracle on the first blocks (blocks do not see one another: Sec. 3.2,
    block-local attention): h <- h + Delta at every position of those blocks, statistics of their masked rows."""
    cfg = dict(synth.CONFIGS[which], L=L)
    d, F, V, B = cfg["d"], cfg["F"], cfg["V"], cfg["B"]
    n, n_attn, D = B * L, d // 128, 3
    w = synth.make_weights(d, F, V, 1, "bf16", cfg["seed"])
    heads_dev, w_lm = harness.upload_weights(w, DEV)
    _, inp = synth.make_config(cfg, w, logits_fn=harness.device_logits_fn(w_lm))
    mw = synth.make_module_weights(d, F, V, D, n_attn, "bf16", 11, std=0.02 if d < 4096 else 0.01)
    ctx = binding.mrp_create(d, F, V, heads_dev, w_lm, max_rows=n, max_seqs=B, block_len=L)
    up = lambda a: harness.to_device(a, "bf16", DEV)
    binding.mrp_module_attach(ctx, up(mw.emb), up(mw.w_proj), [{k: up(v) for k, v in lay.items()} for lay in mw.layers],
                              n_attn, mw.mask_token)
    tokens = np.full(n, -1, np.int32)
    tokens[::L] = 17                                   # one position of every block already revealed
    ri = np.flatnonzero(tokens < 0).astype(np.int32)
    M = ri.size
    hid0 = harness.to_device(inp.hidden, "bf16", DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    h_state = torch.empty((n, d), device=DEV, dtype=torch.float32)
    out = harness.alloc_draft_out(M, 1, V, d, DEV, hidden=True)
    binding.mrp_module_step(ctx, torch.from_numpy(tokens).to(DEV), hid0, h_state, l0, torch.from_numpy(ri).to(DEV), M, B, L,
                            True, out.conf, out.lse, out.token, margin=out.margin, hidden_out=out.hidden, status=out.status)
    torch.cuda.synchronize()
    assert int(out.status.item()) == 0
    ns = blocks_checked * L
    ri_s = np.flatnonzero(tokens[:ns] < 0).astype(np.int32)
    dh, dl = oracle.module(inp.hidden[:ns], tokens[:ns], blocks_checked, L, mw.emb, mw.w_proj, mw.layers, w.w_lm, n_attn,
                           mw.mask_token, row_index=ri_s)
    assert np.abs(dh).max() > 1e-2
    h_ref = inp.hidden[:ns].astype(np.float64) + dh
    assert np.abs(h_state[:ns].cpu().numpy() - h_ref).max() <= 1e-3 * max(1.0, np.abs(h_ref).max())
    conf, lse, tok, margin = oracle.stats(inp.logits0[ri_s].astype(np.float64) + dl)
    m_s = ri_s.size                                     # the checked blocks' masked rows come first in ri
    g_conf, g_lse, g_tok = (t.cpu().numpy() for t in (out.conf, out.lse, out.token))
    assert np.abs(g_conf[1, :m_s] - conf).max() <= TOL["bf16"] and np.abs(g_lse[1, :m_s] - lse).max() <= TOL["bf16"]
    clear = margin > 1e-2
    assert np.array_equal(g_tok[1, :m_s][clear], tok[clear])
    assert np.abs(out.hidden[:m_s].cpu().numpy() - h_ref[ri_s]).max() <= 1e-3 * max(1.0, np.abs(h_ref).max())
    binding.mrp_destroy(ctx)
    del ctx, w_lm, heads_dev, hid0, l0
    torch.cuda.empty_cache()


@pytest.mark.parametrize("dtype,flags,d,F,V,D,heads,B,L", [
    ("f32", 0, 64, 96, 512, 2, 4, 2, 4),                                 # CUDA-core kernels
    ("bf16", binding.MRP_FLAG_FORCE_SIMT, 64, 96, 512, 1, 2, 1, 4),     # ... the step as one cooperative kernel
    ("bf16", 0, 256, 512, 4096, 3, 4, 1, 4),                            # one tensor-core kernel per step, row-major KL LM head
    ("bf16", 0, 256, 512, 4096, 2, 4, 3, 16),                           # 48 positions
    ("bf16", 0, 128, 256, 2048, 2, 4, 5, 32),                           # 160 positions: row-major products
])
def test_module_step_with_the_training_objective(dtype, flags, d, F, V, D, heads, B, L):
    """mrp_module_step_kl: kl[m] = KL(softmax(teacher[m]) || softmax(l[m])) of the step (Eq. (3); Algorithm 1 trains the
    module with it) against the definition on the oracle's logits, over two unrolled steps; the ordinary outputs stay
    those of mrp_module_step."""
    w = synth.make_weights(d, F, V, 1, dtype, 61)
    mw = synth.make_module_weights(d, F, V, D, heads, dtype, 61, std=0.06, proj_std=0.3 / np.sqrt(2 * d))
    inp = synth.make_inputs(w, B, L, 61, 1.0, 3.0)
    n = B * L
    heads_dev, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(d, F, V, heads_dev, w_lm, max_rows=n, max_seqs=B, block_len=L,
                             flags=flags | binding.MRP_FLAG_TRAINING_KL)
    emb, w_proj, layers = upload_module(mw, dtype)
    binding.mrp_module_attach(ctx, emb, w_proj, layers, heads, mw.mask_token)
    hid0 = harness.to_device(inp.hidden, dtype, DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    h_state = torch.empty((n, d), device=DEV, dtype=torch.float32)
    rng = np.random.default_rng(5)
    tokens = np.full(n, -1, np.int32)
    tokens[::L] = rng.integers(0, V - 1, B)
    h_run = inp.hidden.astype(np.float64)
    l_run = inp.logits0.astype(np.float64)
    tol = TOL[dtype] if dtype == "bf16" else 5e-5
    for s in range(2):
        ri = np.flatnonzero(tokens < 0).astype(np.int32)
        M = ri.size
        dh, dl = oracle.module(h_run.astype(np.float32), tokens, B, L, mw.emb, mw.w_proj, mw.layers, w.w_lm, heads, mw.mask_token,
                               row_index=ri)
        h_run = h_run.astype(np.float32).astype(np.float64) + dh
        l_run[ri] += dl
        scale = rng.uniform(0.02, 0.6, size=(M, 1))
        teacher = (l_run[ri] + scale * rng.standard_normal((M, V))).astype(np.float32)
        kl_ref = oracle.kl_rows(teacher, l_run[ri])
        out = harness.alloc_draft_out(M, 1, V, d, DEV, hidden=True)
        kl = torch.full((M,), -1.0, device=DEV)
        binding.mrp_module_step_kl(ctx, torch.from_numpy(tokens).to(DEV), hid0, h_state, l0, torch.from_numpy(teacher).to(DEV),
                                   torch.from_numpy(ri).to(DEV), M, B, L, s == 0, out.conf, out.lse, out.token, kl,
                                   margin=out.margin, hidden_out=out.hidden, status=out.status)
        torch.cuda.synchronize()
        assert int(out.status.item()) == 0
        conf, lse, tok, margin = oracle.stats(l_run[ri])
        assert np.abs(h_state.cpu().numpy() - h_run).max() <= 1e-3 * max(1.0, np.abs(h_run).max())
        assert np.abs(out.conf[1].cpu().numpy() - conf).max() <= tol and np.abs(out.lse[1].cpu().numpy() - lse).max() <= tol
        clear = margin > 1e-2
        assert np.array_equal(out.token[1].cpu().numpy()[clear], tok[clear])
        got = kl.cpu().numpy().astype(np.float64)
        assert kl_ref.min() > 0 and kl_ref.max() > 1e-2
        assert np.all(np.abs(got - kl_ref) <= tol + 2e-3 * kl_ref), np.abs(got - kl_ref).max()
        for b in range(B):                                   # reveal a position per block for the next unrolled step
            rows = [m for m in range(M) if ri[m] // L == b]
            if rows:
                tokens[ri[rows[0]]] = int(rng.integers(0, V - 1))
    # nothing of the KL call lingers: the plain step runs on the same context afterwards
    h2 = torch.empty_like(h_state)
    ri_d = torch.from_numpy(np.flatnonzero(tokens < 0).astype(np.int32)).to(DEV)
    M2 = int(ri_d.numel())
    out3 = harness.alloc_draft_out(M2, 1, V, d, DEV)
    binding.mrp_module_step(ctx, torch.from_numpy(tokens).to(DEV), hid0, h2, l0, ri_d, M2, B, L, True, out3.conf, out3.lse,
                            out3.token, status=out3.status)
    torch.cuda.synchronize()
    assert int(out3.status.item()) == 0
    binding.mrp_destroy(ctx)
    # a context without the flag has no room for the partial sums
    ctx = binding.mrp_create(d, F, V, heads_dev, w_lm, max_rows=n, max_seqs=B, block_len=L, flags=flags)
    binding.mrp_module_attach(ctx, emb, w_proj, layers, heads, mw.mask_token)
    with pytest.raises(binding.MrpError) as ei:
        binding.mrp_module_step_kl(ctx, torch.from_numpy(tokens).to(DEV), hid0, h2, l0, torch.from_numpy(teacher).to(DEV), ri_d, M2,
                                   B, L, True, out3.conf, out3.lse, out3.token, kl)
    assert ei.value.status == 2
    binding.mrp_destroy(ctx)
