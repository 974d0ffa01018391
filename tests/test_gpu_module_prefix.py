"""mrp_module_step behind a clean prefix (Fig. 1(c)): the module's attention over the keys and values of the
committed prefix (mrp_module_set_prefix) and the block, against the oracle's module with the same prefix, on
every kernel path that serves the step; storing the block's own keys and values behind the prefix rows."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_18817_b200 import binding, harness, synth
from test_gpu_module import upload_module
from test_gpu_parity import DEV, TOL

pytestmark = pytest.mark.gpu


def tdt(dtype):
    return torch.float32 if dtype == "f32" else torch.bfloat16


def make_prefix(D, B, cap, d, plen, dtype, seed, poison=True):
    """Random caches in the context dtype; rows beyond a sequence's length hold NaN: a read of one shows."""
    g = torch.Generator().manual_seed(seed)
    caches = []
    for _ in range(D):
        k = torch.randn((B, cap, d), generator=g).to(tdt(dtype))
        v = torch.randn((B, cap, d), generator=g).to(tdt(dtype))
        if poison:
            for b in range(B):
                k[b, plen[b]:] = float("nan")
                v[b, plen[b]:] = float("nan")
        caches.append((k, v))
    return caches


def to_dev(host, heads):
    """The caches in the library's head-major layout, on the device."""
    return [(binding.prefix_to_head_major(k, heads).to(DEV), binding.prefix_to_head_major(v, heads).to(DEV)) for k, v in host]


def from_dev(t):
    """A device cache back in [sequences, positions, d] on the host."""
    return binding.prefix_from_head_major(t.cpu())


def as_oracle_prefix(caches, plen):
    ks = [np.nan_to_num(k.float().numpy(), nan=0.0) for k, _ in caches]
    vs = [np.nan_to_num(v.float().numpy(), nan=0.0) for _, v in caches]
    return ks, vs, np.asarray(plen, np.int32)


CASES = [
    # dtype, flags, d, F, V, D, heads, B, L, cap, prefix lengths
    ("f32", 0, 64, 96, 512, 2, 4, 2, 4, 40, [37, 5]),                                   # CUDA cores, one kernel per product
    ("f32", 0, 60, 96, 512, 1, 3, 1, 3, 70, [70]),                                      # heads of 20 features: scalar loads
    ("bf16", binding.MRP_FLAG_FORCE_SIMT, 64, 96, 512, 1, 2, 2, 5, 33, [0, 33]),
    ("bf16", 0, 256, 512, 4096, 3, 2, 1, 4, 200, [150]),                                # one cooperative tensor-core kernel
    ("bf16", 0, 256, 512, 4096, 2, 4, 3, 4, 72, [0, 70, 33]),                           # ... three blocks, ragged lengths
    ("bf16", 0, 256, 512, 4096, 2, 2, 2, 32, 40, [40, 7]),                              # ... 64 positions
    ("bf16", 0, 256, 512, 4096, 2, 1, 2, 32, 40, [40, 7]),                              # heads of 256 features: one kernel per product
    ("bf16", 0, 256, 512, 4096, 1, 4, 1, 4, 1500, [1500]),                              # a long prefix: keys split over CTAs
    ("bf16", binding.MRP_FLAG_NO_CHAIN, 256, 512, 4096, 1, 4, 2, 6, 700, [700, 130]),   # ... in the separate kernel, ragged
    ("bf16", binding.MRP_FLAG_NO_CHAIN, 256, 512, 4096, 2, 4, 3, 4, 72, [64, 1, 72]),   # few-row kernels, one per product
    ("bf16", 0, 128, 256, 2048, 2, 4, 5, 32, 48, [48, 0, 31, 32, 33]),                  # 160 positions: row-major kernels
    ("bf16", 0, 192, 320, 2064, 2, 3, 1, 4, 130, [129]),                                # d % 128 != 0: no one-kernel form
]


@pytest.mark.parametrize("dtype,flags,d,F,V,D,heads,B,L,cap,plen", CASES)
def test_module_step_behind_a_prefix_follows_the_oracle(dtype, flags, d, F, V, D, heads, B, L, cap, plen):
    w = synth.make_weights(d, F, V, 1, dtype, 47)
    mw = synth.make_module_weights(d, F, V, D, heads, dtype, 47, std=0.06, proj_std=0.3 / np.sqrt(2 * d))
    inp = synth.make_inputs(w, B, L, 47, 1.0, 3.0)
    n = B * L
    heads_dev, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(d, F, V, heads_dev, w_lm, max_rows=n, max_seqs=B, block_len=L, flags=flags)
    emb, w_proj, layers = upload_module(mw, dtype)
    binding.mrp_module_attach(ctx, emb, w_proj, layers, heads, mw.mask_token)
    host = make_prefix(D, B, cap, d, plen, dtype, 5)
    dev = to_dev(host, heads)
    plen_d = torch.tensor(plen, dtype=torch.int32, device=DEV)
    binding.mrp_module_set_prefix(ctx, dev, plen_d)
    hid0 = harness.to_device(inp.hidden, dtype, DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    h_state = torch.empty((n, d), device=DEV, dtype=torch.float32)
    tol = TOL[dtype] if dtype == "bf16" else 5e-5
    rng = np.random.default_rng(3)
    tokens = np.where(rng.random(n) < 0.4, rng.integers(0, V - 1, n), -1).astype(np.int32)
    tokens[0] = -1
    ri = np.flatnonzero(tokens < 0).astype(np.int32)
    M = ri.size
    out = harness.alloc_draft_out(M, 1, V, d, DEV, hidden=True)
    binding.mrp_module_step(ctx, torch.from_numpy(tokens).to(DEV), hid0, h_state, l0, torch.from_numpy(ri).to(DEV), M, B, L, True,
                            out.conf, out.lse, out.token, margin=out.margin, hidden_out=out.hidden, status=out.status)
    torch.cuda.synchronize()
    assert int(out.status.item()) == 0
    if dtype == "bf16" and flags == 0 and d % 128 == 0 and n <= 64 and d // heads <= 192:
        assert ctx.last_launch_count <= 4                    # the step was one kernel (+ the LM-head kernels)
    else:
        assert ctx.last_launch_count >= 4 + 5 * D
    pre = as_oracle_prefix(host, plen)
    dh, dl = oracle.module(inp.hidden, tokens, B, L, mw.emb, mw.w_proj, mw.layers, w.w_lm, heads, mw.mask_token, row_index=ri,
                           prefix=pre)
    alone, _ = oracle.module(inp.hidden, tokens, B, L, mw.emb, mw.w_proj, mw.layers, w.w_lm, heads, mw.mask_token)
    assert np.abs(dh - alone).max() > 1e-2                   # the prefix matters in this case
    h_run = inp.hidden.astype(np.float64) + dh
    conf, lse, tok, margin = oracle.stats(inp.logits0.astype(np.float64)[ri] + dl)
    scale = max(1.0, np.abs(h_run).max())
    assert np.abs(h_state.cpu().numpy() - h_run).max() <= 1e-3 * scale
    assert np.abs(out.hidden.cpu().numpy() - h_run[ri]).max() <= 1e-3 * scale
    g_conf, g_lse, g_tok = (t.cpu().numpy() for t in (out.conf, out.lse, out.token))
    assert np.abs(g_conf[1] - conf).max() <= tol and np.abs(g_lse[1] - lse).max() <= tol
    clear = margin > 1e-2
    assert np.array_equal(g_tok[1][clear], tok[clear])
    # the caches were only read
    for (k, v), (hk, hv) in zip(dev, host):
        assert torch.equal(from_dev(k).contiguous().view(torch.uint8), hk.view(torch.uint8))
        assert torch.equal(from_dev(v).contiguous().view(torch.uint8), hv.view(torch.uint8))
    # detached again, the step is the block-local one
    binding.mrp_module_set_prefix(ctx, None, None)
    binding.mrp_module_step(ctx, torch.from_numpy(tokens).to(DEV), hid0, h_state, l0, torch.from_numpy(ri).to(DEV), M, B, L, True,
                            out.conf, out.lse, out.token, status=out.status)
    torch.cuda.synchronize()
    assert int(out.status.item()) == 0
    assert np.abs(h_state.cpu().numpy() - (inp.hidden.astype(np.float64) + alone)).max() <= 1e-3 * scale
    binding.mrp_destroy(ctx)


@pytest.mark.parametrize("dtype,flags,d,F,V,D,heads,B,L,cap,plen", [
    ("f32", 0, 64, 96, 512, 2, 4, 2, 4, 40, [36, 5]),
    ("bf16", 0, 256, 512, 4096, 3, 2, 2, 4, 100, [96, 17]),                             # one cooperative tensor-core kernel
    ("bf16", binding.MRP_FLAG_NO_CHAIN, 256, 512, 4096, 2, 4, 2, 4, 72, [64, 1]),
    ("bf16", 0, 128, 256, 2048, 2, 4, 5, 32, 64, [32, 0, 31, 1, 30]),                   # row-major kernels
])
def test_committed_block_is_appended_and_serves_the_next_block(dtype, flags, d, F, V, D, heads, B, L, cap, plen):
    """A committed block (all tokens revealed) is run with append: its keys and values land behind the prefix rows
    as the oracle computes them, nothing else changes; the next block then attends to prefix + that block, as the
    oracle does with its own exported keys and values."""
    w = synth.make_weights(d, F, V, 1, dtype, 49)
    mw = synth.make_module_weights(d, F, V, D, heads, dtype, 49, std=0.06, proj_std=0.3 / np.sqrt(2 * d))
    inp = synth.make_inputs(w, B, L, 49, 1.0, 3.0)
    nxt = synth.make_inputs(w, B, L, 50, 1.0, 3.0)
    n = B * L
    heads_dev, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(d, F, V, heads_dev, w_lm, max_rows=n, max_seqs=B, block_len=L, flags=flags)
    emb, w_proj, layers = upload_module(mw, dtype)
    binding.mrp_module_attach(ctx, emb, w_proj, layers, heads, mw.mask_token)
    host = make_prefix(D, B, cap, d, plen, dtype, 6, poison=False)
    dev = to_dev(host, heads)
    plen_d = torch.tensor(plen, dtype=torch.int32, device=DEV)
    binding.mrp_module_set_prefix(ctx, dev, plen_d, append=True)
    rng = np.random.default_rng(4)
    tokens = rng.integers(0, V - 1, n).astype(np.int32)           # a clean block
    h_state = torch.empty((n, d), device=DEV, dtype=torch.float32)
    out = harness.alloc_draft_out(1, 1, V, d, DEV)
    binding.mrp_module_step(ctx, torch.from_numpy(tokens).to(DEV), harness.to_device(inp.hidden, dtype, DEV), h_state,
                            torch.from_numpy(inp.logits0).to(DEV), None, 0, B, L, True, out.conf, out.lse, out.token, status=out.status)
    torch.cuda.synchronize()
    assert int(out.status.item()) == 0
    pre = as_oracle_prefix(host, plen)
    _, _, k_o, v_o = oracle.module(inp.hidden, tokens, B, L, mw.emb, mw.w_proj, mw.layers, w.w_lm, heads, mw.mask_token, prefix=pre,
                                   want_kv=True)
    rel = 2.0 ** -8 if dtype == "bf16" else 1e-5
    grown = []
    for l, ((k, v), (hk, hv)) in enumerate(zip(dev, host)):
        gk, gv = from_dev(k).float().numpy(), from_dev(v).float().numpy()
        wk, wv = hk.float().numpy().copy(), hv.float().numpy().copy()
        mask = np.zeros((B, cap), bool)
        for b in range(B):
            mask[b, plen[b]:plen[b] + L] = True
            wk[b, plen[b]:plen[b] + L] = k_o[l][b * L:(b + 1) * L]
            wv[b, plen[b]:plen[b] + L] = v_o[l][b * L:(b + 1) * L]
        assert np.array_equal(gk[~mask], hk.float().numpy()[~mask]) and np.array_equal(gv[~mask], hv.float().numpy()[~mask])
        assert np.all(np.abs(gk - wk)[mask] <= rel * np.abs(wk[mask]) + 2e-3)
        assert np.all(np.abs(gv - wv)[mask] <= rel * np.abs(wv[mask]) + 2e-3)
        grown.append((gk, gv))
    # the next block of every sequence, behind prefix + the committed block (the device's own stored rows on both sides)
    plen2 = [p + L for p in plen]
    plen_d.copy_(torch.tensor(plen2, dtype=torch.int32))
    binding.mrp_module_set_prefix(ctx, dev, plen_d, append=False)
    tokens2 = np.full(n, -1, np.int32)
    ri = np.arange(n, dtype=np.int32)
    out2 = harness.alloc_draft_out(n, 1, V, d, DEV)
    binding.mrp_module_step(ctx, torch.from_numpy(tokens2).to(DEV), harness.to_device(nxt.hidden, dtype, DEV), h_state,
                            torch.from_numpy(nxt.logits0).to(DEV), torch.from_numpy(ri).to(DEV), n, B, L, True, out2.conf, out2.lse,
                            out2.token, status=out2.status)
    torch.cuda.synchronize()
    assert int(out2.status.item()) == 0
    dh, dl = oracle.module(nxt.hidden, tokens2, B, L, mw.emb, mw.w_proj, mw.layers, w.w_lm, heads, mw.mask_token, row_index=ri,
                           prefix=([g[0] for g in grown], [g[1] for g in grown], np.asarray(plen2, np.int32)))
    h_run = nxt.hidden.astype(np.float64) + dh
    assert np.abs(h_state.cpu().numpy() - h_run).max() <= 1e-3 * max(1.0, np.abs(h_run).max())
    conf, lse, tok, margin = oracle.stats(nxt.logits0.astype(np.float64) + dl)
    tol = TOL[dtype] if dtype == "bf16" else 5e-5
    assert np.abs(out2.conf[1].cpu().numpy() - conf).max() <= tol and np.abs(out2.lse[1].cpu().numpy() - lse).max() <= tol
    binding.mrp_destroy(ctx)


@pytest.mark.parametrize("dtype,B,L,d,heads", [("f32", 2, 4, 64, 4), ("bf16", 2, 4, 256, 2)])
def test_prefix_lengths_are_checked_on_the_device(dtype, B, L, d, heads):
    F, V, D, cap = 2 * d, 1024, 1, 24
    n = B * L
    w = synth.make_weights(d, F, V, 1, dtype, 51)
    mw = synth.make_module_weights(d, F, V, D, heads, dtype, 51, std=0.06)
    inp = synth.make_inputs(w, B, L, 51, 1.0, 3.0)
    heads_dev, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(d, F, V, heads_dev, w_lm, max_rows=n, max_seqs=B, block_len=L)
    with pytest.raises(binding.MrpError) as ei:               # no module attached
        binding.mrp_module_set_prefix(ctx, [], torch.zeros(B, dtype=torch.int32, device=DEV))
    assert ei.value.status == 2
    emb, w_proj, layers = upload_module(mw, dtype)
    binding.mrp_module_attach(ctx, emb, w_proj, layers, heads, mw.mask_token)
    host = make_prefix(D, B, cap, d, [cap, cap], dtype, 7, poison=False)
    dev = to_dev(host, heads)
    hid0 = harness.to_device(inp.hidden, dtype, DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    tok = torch.full((n,), -1, device=DEV, dtype=torch.int32)

    def step(plen, append):
        plen_d = torch.tensor(plen, dtype=torch.int32, device=DEV)
        binding.mrp_module_set_prefix(ctx, dev, plen_d, append=append)
        h = torch.empty((n, d), device=DEV, dtype=torch.float32)
        out = harness.alloc_draft_out(n, 1, V, d, DEV)
        binding.mrp_module_step(ctx, tok, hid0, h, l0, None, n, B, L, True, out.conf, out.lse, out.token, status=out.status)
        torch.cuda.synchronize()
        return h.cpu(), int(out.status.item())

    good, st = step([cap, 3], False)
    assert st == 0
    # a length beyond the cache or below zero: the bit, and the clamped length is used
    over, st = step([cap + 9, 3], False)
    assert st == binding.MRP_DEV_BAD_INDEX and torch.equal(over, good)
    under, st = step([cap, -2], False)
    zero, st0 = step([cap, 0], False)
    assert st == binding.MRP_DEV_BAD_INDEX and st0 == 0 and torch.equal(under, zero)
    # a block that does not fit behind its prefix is not stored, the other sequence's is
    before = [(k.clone(), v.clone()) for k, v in dev]
    _, st = step([cap - L + 1, 3], True)
    assert st == binding.MRP_DEV_BAD_INDEX
    for (k, v), (bk, bv) in zip(dev, before):
        assert torch.equal(k[0], bk[0]) and torch.equal(v[0], bv[0])
        k, bk = from_dev(k), from_dev(bk)
        assert not torch.equal(k[1, 3:3 + L], bk[1, 3:3 + L]) and torch.equal(k[1, 3 + L:], bk[1, 3 + L:]) and torch.equal(k[1, :3], bk[1, :3])
    binding.mrp_destroy(ctx)


@pytest.mark.parametrize("seed", [0, 1])
def test_random_shapes_behind_random_prefixes(seed):
    """Random small shapes, prefix lengths, kernel paths and token patterns: one step each against the oracle."""
    rng = np.random.default_rng(100 + seed)
    for case in range(14):
        dtype = "bf16" if rng.random() < 0.7 else "f32"
        heads = int(rng.choice([1, 2, 4]))
        d = int(rng.choice([64, 128, 256])) if dtype == "bf16" else int(rng.choice([48, 64, 96]))
        if d // heads > 256:
            heads = 2
        F, V, D = 2 * d, 1024, int(rng.integers(1, 4))
        L = int(rng.choice([1, 2, 4, 5, 8, 16, 33]))
        B = int(rng.integers(1, max(2, 70 // L)))
        cap = int(rng.choice([1, 31, 32, 33, 64, 100, 257, 700]))
        plen = [int(x) for x in rng.integers(0, cap + 1, B)]
        flags = int(rng.choice([0, 0, binding.MRP_FLAG_NO_CHAIN, binding.MRP_FLAG_FORCE_SIMT])) if dtype == "bf16" else 0
        n = B * L
        w = synth.make_weights(d, F, V, 1, dtype, 200 + case)
        mw = synth.make_module_weights(d, F, V, D, heads, dtype, 200 + case, std=0.06, proj_std=0.3 / np.sqrt(2 * d))
        inp = synth.make_inputs(w, B, L, 200 + case, 1.0, 3.0)
        heads_dev, w_lm = harness.upload_weights(w, DEV)
        ctx = binding.mrp_create(d, F, V, heads_dev, w_lm, max_rows=n, max_seqs=B, block_len=L, flags=flags)
        emb, w_proj, layers = upload_module(mw, dtype)
        binding.mrp_module_attach(ctx, emb, w_proj, layers, heads, mw.mask_token)
        host = make_prefix(D, B, cap, d, plen, dtype, 300 + case)
        dev = to_dev(host, heads)
        binding.mrp_module_set_prefix(ctx, dev, torch.tensor(plen, dtype=torch.int32, device=DEV))
        tokens = np.where(rng.random(n) < 0.5, rng.integers(0, V - 1, n), -1).astype(np.int32)
        tokens[int(rng.integers(0, n))] = -1
        ri = np.flatnonzero(tokens < 0).astype(np.int32)
        M = ri.size
        h_state = torch.empty((n, d), device=DEV, dtype=torch.float32)
        out = harness.alloc_draft_out(M, 1, V, d, DEV)
        binding.mrp_module_step(ctx, torch.from_numpy(tokens).to(DEV), harness.to_device(inp.hidden, dtype, DEV), h_state,
                                torch.from_numpy(inp.logits0).to(DEV), torch.from_numpy(ri).to(DEV), M, B, L, True, out.conf, out.lse,
                                out.token, status=out.status)
        torch.cuda.synchronize()
        what = (seed, case, dtype, flags, d, heads, D, B, L, cap, plen)
        assert int(out.status.item()) == 0, what
        dh, dl = oracle.module(inp.hidden, tokens, B, L, mw.emb, mw.w_proj, mw.layers, w.w_lm, heads, mw.mask_token, row_index=ri,
                               prefix=as_oracle_prefix(host, plen))
        h_run = inp.hidden.astype(np.float64) + dh
        assert np.abs(h_state.cpu().numpy() - h_run).max() <= 1e-3 * max(1.0, np.abs(h_run).max()), what
        conf, lse, tok, margin = oracle.stats(inp.logits0.astype(np.float64)[ri] + dl)
        tol = TOL[dtype] if dtype == "bf16" else 5e-5
        assert np.abs(out.conf[1].cpu().numpy() - conf).max() <= tol and np.abs(out.lse[1].cpu().numpy() - lse).max() <= tol, what
        clear = margin > 1e-2
        assert np.array_equal(out.token[1].cpu().numpy()[clear], tok[clear]), what
        binding.mrp_destroy(ctx)


@pytest.mark.parametrize("which,L,P,blocks_checked", [
    (1, 4, 1024, 1),     # decode shape, one block of 4 behind 1024 prefix positions: 9 key chunks per (block, head)
    (1, 16, 1024, 1),    # ... one block of 16: four query tiles per unit
    (2, 4, 300, 2),      # 32 blocks of 4 at d = 4096: the separate kernel, one unit per (block, head); oracle on two blocks
])
def test_prefix_at_the_benchmark_shapes(which, L, P, blocks_checked):
    """One module step behind a prefix at the shapes bench.py's module:P<n> workloads time (D = 3, 128 features per
    attention head, random caches), against the oracle on the first blocks."""
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
    plen = [P - (b % 3) for b in range(B)]
    host = make_prefix(D, B, P, d, plen, "bf16", 13)
    dev = to_dev(host, n_attn)
    binding.mrp_module_set_prefix(ctx, dev, torch.tensor(plen, dtype=torch.int32, device=DEV))
    tokens = np.full(n, -1, np.int32)
    tokens[::L] = 17
    ri = np.flatnonzero(tokens < 0).astype(np.int32)
    M = ri.size
    h_state = torch.empty((n, d), device=DEV, dtype=torch.float32)
    out = harness.alloc_draft_out(M, 1, V, d, DEV)
    binding.mrp_module_step(ctx, torch.from_numpy(tokens).to(DEV), harness.to_device(inp.hidden, "bf16", DEV), h_state,
                            torch.from_numpy(inp.logits0).to(DEV), torch.from_numpy(ri).to(DEV), M, B, L, True, out.conf, out.lse,
                            out.token, status=out.status)
    torch.cuda.synchronize()
    assert int(out.status.item()) == 0
    ns, Bs = blocks_checked * L, blocks_checked
    ri_s = np.flatnonzero(tokens[:ns] < 0).astype(np.int32)
    ks, vs, pl = as_oracle_prefix(host, plen)
    dh, dl = oracle.module(inp.hidden[:ns], tokens[:ns], Bs, L, mw.emb, mw.w_proj, mw.layers, w.w_lm, n_attn, mw.mask_token,
                           row_index=ri_s, prefix=([k[:Bs] for k in ks], [v[:Bs] for v in vs], pl[:Bs]))
    alone, _ = oracle.module(inp.hidden[:ns], tokens[:ns], Bs, L, mw.emb, mw.w_proj, mw.layers, w.w_lm, n_attn, mw.mask_token)
    assert np.abs(dh - alone).max() > 1e-3
    h_ref = inp.hidden[:ns].astype(np.float64) + dh
    assert np.abs(h_state[:ns].cpu().numpy() - h_ref).max() <= 1e-3 * max(1.0, np.abs(h_ref).max())
    conf, lse, tok, margin = oracle.stats(inp.logits0[ri_s].astype(np.float64) + dl)
    m_s = ri_s.size
    assert np.abs(out.conf[1, :m_s].cpu().numpy() - conf).max() <= TOL["bf16"]
    assert np.abs(out.lse[1, :m_s].cpu().numpy() - lse).max() <= TOL["bf16"]
    clear = margin > 1e-2
    assert np.array_equal(out.token[1, :m_s].cpu().numpy()[clear], tok[clear])
    binding.mrp_destroy(ctx)
    del ctx, w_lm, heads_dev, dev
    torch.cuda.empty_cache()
