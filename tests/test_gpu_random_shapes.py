"""Randomised parity sweep: the drafting pass and the module step against the oracle over random small shapes, row
counts, chain lengths and context flags, so that every kernel family and its switches (few-row / chain / row-major /
CTA pairs / one-kernel CUDA-core pass / the module's four paths) meets shapes nobody picked by hand.  Seeds are fixed:
a failing case prints the line that reproduces it."""
import numpy as np
import pytest
import torch

import oracle
from paper_2605_18817_b200 import binding, harness, synth
from test_gpu_parity import DEV, TOL, check_stats, run_gpu_draft, run_gpu_draft_from_hidden

pytestmark = pytest.mark.gpu


def _draft_case(rng, it, kind):
    dtype = "f32" if kind == "f32" else "bf16"
    flags = binding.MRP_FLAG_FORCE_SIMT if kind == "simt" else 0
    if kind == "tc":
        d = int(rng.choice([64, 128, 192, 256, 512, 1024]))
        F = int(rng.choice([64, 128, 320, 512, 1024, 2048]))
        V = int(rng.choice([160, 1024, 2048, 4112, 8192]))
        flags |= int(rng.choice([0, 0, 0, binding.MRP_FLAG_ROW_MAJOR_ONLY, binding.MRP_FLAG_NO_CTA_PAIRS,
                                 binding.MRP_FLAG_EXACT_OPERANDS, binding.MRP_FLAG_NO_CHAIN, binding.MRP_FLAG_NO_PDL]))
        B, L = [(1, 1), (2, 4), (10, 4), (33, 1), (64, 2), (129, 1), (75, 4), (257, 1), (40, 16), (512, 1),
                (130, 3)][int(rng.integers(0, 11))]
        std = 0.05
    else:
        d = int(rng.choice([24, 72, 128, 256, 512]))
        F = int(rng.choice([40, 136, 256, 512]))
        V = int(rng.choice([100, 1000, 4096]))
        flags |= int(rng.choice([0, 0, binding.MRP_FLAG_NO_CHAIN]))
        B, L = [(1, 1), (1, 4), (2, 4), (2, 3), (5, 3), (8, 1), (3, 2)][int(rng.integers(0, 7))]
        std = 0.1 if d < 512 else 0.03        # (the fp32 tolerance is absolute: logits of order 10)
    K = int(rng.integers(1, 5))
    mask_prob = float(rng.choice([1.0, 0.7, 0.4]))
    from_hidden = bool(rng.random() < 0.25)
    desc = f"{kind} d={d} F={F} V={V} B={B} L={L} K={K} mask={mask_prob} flags={flags} from_hidden={from_hidden}"
    w = synth.make_weights(d, F, V, K, dtype, 400 + it, head_std=std)
    inp = synth.make_inputs(w, B, L, 500 + it, 1.0, 4.0, mask_prob=mask_prob)
    if len(inp.row_index) == 0:
        return desc
    if from_hidden:
        out, _ = run_gpu_draft_from_hidden(w, inp, K, flags=flags)
        ref = oracle.draft(inp.hidden, None, w.heads, w.w_lm, K=K, row_index=inp.row_index)
    else:
        out, _ = run_gpu_draft(w, inp, K, flags=flags)
        ref = oracle.draft(inp.hidden, inp.logits0, w.heads, w.w_lm, K=K, row_index=inp.row_index)
    check_stats(out, ref, "bf16" if kind == "tc" else "f32")
    return desc


def _module_case(rng, it):
    d = int(rng.choice([64, 128, 192, 256, 512]))
    F = int(rng.choice([d, 2 * d, d + 64]))
    V = int(rng.choice([512, 2048, 2064, 4096]))
    D = int(rng.integers(0, 4))
    H = int(rng.choice([h for h in (1, 2, 4) if d % h == 0]))
    B, L = [(1, 4), (1, 3), (2, 4), (3, 5), (1, 16), (2, 16), (5, 32), (1, 64), (20, 4), (2, 2)][int(rng.integers(0, 10))]
    dtype = str(rng.choice(["bf16", "bf16", "f32"]))
    flags = int(rng.choice([0, 0, binding.MRP_FLAG_NO_CHAIN, binding.MRP_FLAG_ROW_MAJOR_ONLY]))
    desc = f"module {dtype} d={d} F={F} V={V} D={D} H={H} B={B} L={L} flags={flags}"
    w = synth.make_weights(d, F, V, 1, dtype, 100 + it)
    mw = synth.make_module_weights(d, F, V, D, H, dtype, 200 + it, std=0.05, proj_std=0.3 / np.sqrt(2 * d))
    inp = synth.make_inputs(w, B, L, 300 + it, 1.0, 3.0)
    n = B * L
    heads_dev, w_lm = harness.upload_weights(w, DEV)
    ctx = binding.mrp_create(d, F, V, heads_dev, w_lm, max_rows=n, max_seqs=B, block_len=L, flags=flags)
    up = lambda a: harness.to_device(a, dtype, DEV)
    binding.mrp_module_attach(ctx, up(mw.emb), up(mw.w_proj), [{k: up(v) for k, v in lay.items()} for lay in mw.layers], H,
                              mw.mask_token)
    tokens = np.where(rng.random(n) < 0.3, rng.integers(0, V, n), -1).astype(np.int32)
    if (tokens < 0).sum() == 0:
        tokens[0] = -1
    ri = np.flatnonzero(tokens < 0).astype(np.int32)
    M = ri.size
    hid0 = harness.to_device(inp.hidden, dtype, DEV)
    l0 = torch.from_numpy(inp.logits0).to(DEV)
    h_state = torch.empty((n, d), device=DEV)
    out = harness.alloc_draft_out(M, 1, V, d, DEV, hidden=True)
    tol = TOL["bf16"] if dtype == "bf16" else 5e-5
    h_run = inp.hidden.astype(np.float64)
    for s in (1, 2):                    # two applications on the same tokens: the second starts from the kept state
        binding.mrp_module_step(ctx, torch.from_numpy(tokens).to(DEV), hid0, h_state, l0, torch.from_numpy(ri).to(DEV), M, B, L,
                                s == 1, out.conf, out.lse, out.token, margin=out.margin, hidden_out=out.hidden, status=out.status)
        torch.cuda.synchronize()
        assert int(out.status.item()) == 0, desc
        dh, _ = oracle.module(h_run.astype(np.float32), tokens, B, L, mw.emb, mw.w_proj, mw.layers, w.w_lm, H, mw.mask_token,
                              row_index=ri)
        h_run = h_run.astype(np.float32).astype(np.float64) + dh
        # l = l_0 + W_lm (h - h_0) (Sec. 3.2): the oracle's own accumulation over both applications
        l_acc = inp.logits0[ri].astype(np.float64) + (h_run[ri] - inp.hidden[ri].astype(np.float64)) @ w.w_lm.astype(np.float64).T
        conf, lse, tok, margin = oracle.stats(l_acc)
        assert np.abs(h_state.cpu().numpy() - h_run).max() <= 1e-3 * max(1.0, np.abs(h_run).max()), desc
        g_conf, g_lse, g_tok = (t.cpu().numpy() for t in (out.conf, out.lse, out.token))
        assert np.abs(g_conf[1] - conf).max() <= tol and np.abs(g_lse[1] - lse).max() <= tol, desc
        clear = margin > 1e-2
        assert np.array_equal(g_tok[1][clear], tok[clear]), desc
    binding.mrp_destroy(ctx)
    return desc


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_random_shapes_against_the_oracle(seed):
    rng = np.random.default_rng(seed)
    for it in range(40):
        kind = str(rng.choice(["tc", "tc", "simt", "f32", "module", "module"]))
        try:
            _module_case(rng, it) if kind == "module" else _draft_case(rng, it, kind)
        except AssertionError as e:
            raise AssertionError("seed %d case %d (%s): %s" % (seed, it, kind, e)) from e
