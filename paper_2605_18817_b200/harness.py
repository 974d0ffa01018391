"""Device-memory plumbing around the binding: upload synthetic weights/inputs, allocate
output tensors, call the C ABI.  No arithmetic of the method happens here."""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np
import torch

from . import binding, synth


def to_device(a: np.ndarray, dtype: str, device) -> torch.Tensor:
    """float32 host array -> CUDA tensor in the storage dtype (bf16 values are exact)."""
    if dtype == "bf16":
        bits = synth.bf16_bits(a)
        return torch.from_numpy(bits.view(np.int16)).to(device).view(torch.bfloat16)
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).to(device)


def device_logits_fn(w_lm: torch.Tensor, chunk: int = 16384):
    """Input generation helper: base logits of the synthetic backbone as an fp32 product on
    the device (TF32 off), returned to the host; plugs into ``synth.make_inputs(logits_fn=)``."""
    def fn(rows: np.ndarray) -> np.ndarray:
        torch.backends.cuda.matmul.allow_tf32 = False
        x = torch.from_numpy(np.ascontiguousarray(rows, dtype=np.float32)).to(w_lm.device)
        out = torch.empty((x.shape[0], w_lm.shape[0]), device=w_lm.device)
        for v0 in range(0, w_lm.shape[0], chunk):
            out[:, v0:v0 + chunk] = x @ w_lm[v0:v0 + chunk].float().T
        return out.cpu().numpy()
    return fn


def upload_weights(w: synth.Weights, device):
    heads = [{k: to_device(v, w.dtype, device) for k, v in h.items()} for h in w.heads]
    return heads, to_device(w.w_lm, w.dtype, device)


@dataclass
class DraftOut:
    conf: torch.Tensor
    lse: torch.Tensor
    token: torch.Tensor
    margin: torch.Tensor | None
    logits: torch.Tensor | None
    hidden: torch.Tensor | None
    status: torch.Tensor
    conf_first: torch.Tensor | None = None


def alloc_draft_out(M, K, V, d, device, margin=True, logits=False, hidden=False, conf_first=False) -> DraftOut:
    f = dict(device=device, dtype=torch.float32)
    return DraftOut(
        torch.empty((K + 1, M), **f), torch.empty((K + 1, M), **f),
        torch.empty((K + 1, M), device=device, dtype=torch.int32),
        torch.empty((K + 1, M), **f) if margin else None,
        torch.empty((K, M, V), **f) if logits else None,
        torch.empty((M, d), **f) if hidden else None,
        torch.zeros(1, device=device, dtype=torch.int32),
        torch.empty((K + 1, M), **f) if conf_first else None)


def draft(ctx, hidden, logits0, row_index, M, K, out: DraftOut, stream=None):
    binding.mrp_draft(ctx, hidden, logits0, row_index, M, K, out.conf, out.lse, out.token,
                      out.margin, out.logits, out.hidden, out.status, stream=stream, conf_first=out.conf_first)
    return out


@dataclass
class BlockState:
    tokens: torch.Tensor        # [B*L] int32, -1 = masked
    row_index: torch.Tensor     # [B*L] int32
    n_masked: torch.Tensor      # [1] int32
    block_masked: torch.Tensor  # [B] int32


def alloc_block_state(B, L, device) -> BlockState:
    i32 = dict(device=device, dtype=torch.int32)
    return BlockState(torch.full((B * L,), -1, **i32), torch.arange(B * L, **i32),
                      torch.full((1,), B * L, **i32), torch.full((B,), L, **i32))


def commit(ctx, sel, state: BlockState, B, L, Kd, accept_mask=None, stream=None):
    binding.mrp_commit(ctx, B, L, Kd, out_token=sel.out_token, step_of=sel.step_of, draft_pos=sel.draft_pos,
                       draft_tok=sel.draft_tok, accept_mask=accept_mask, tokens=state.tokens,
                       row_index=state.row_index, n_masked=state.n_masked, block_masked=state.block_masked,
                       stream=stream)
    return state


def draft_from_hidden(ctx, hidden, final_gamma, row_index, M, K, out: DraftOut, stream=None):
    binding.mrp_draft_from_hidden(ctx, hidden, final_gamma, row_index, M, K, out.conf, out.lse, out.token,
                                  out.margin, out.logits, out.hidden, out.status, stream=stream,
                                  conf_first=out.conf_first)
    return out


@dataclass
class SelectOut:
    reveal_mask: torch.Tensor
    remask_mask: torch.Tensor
    out_token: torch.Tensor
    step_of: torch.Tensor
    draft_pos: torch.Tensor
    draft_tok: torch.Tensor
    draft_len: torch.Tensor


def alloc_select_out(B, L, Kd, device) -> SelectOut:
    i8 = dict(device=device, dtype=torch.int8)
    i32 = dict(device=device, dtype=torch.int32)
    return SelectOut(torch.empty(B * L, **i8), torch.empty(B * L, **i8), torch.empty(B * L, **i32),
                     torch.empty(B * L, **i8), torch.empty((B, Kd), **i32),
                     torch.empty((B, Kd), **i32), torch.empty(B, **i32))


def select(ctx, conf, token, row_index, M, K, B, L, mode, out: SelectOut, **kw):
    binding.mrp_reveal_remask(ctx, conf, token, row_index, M, K, B, L, mode,
                              reveal_mask=out.reveal_mask, remask_mask=out.remask_mask,
                              out_token=out.out_token, step_of=out.step_of,
                              draft_pos=out.draft_pos, draft_tok=out.draft_tok,
                              draft_len=out.draft_len, **kw)
    return out


def verify(ctx, draft_tok, verify_tok, draft_len, positionwise=False):
    B, Kd = draft_tok.shape
    accept_len = torch.empty(B, device=draft_tok.device, dtype=torch.int32)
    accept_mask = torch.empty((B, Kd), device=draft_tok.device, dtype=torch.int8)
    binding.mrp_verify(ctx, draft_tok, verify_tok, draft_len, B, Kd, positionwise, accept_len,
                       accept_mask)
    return accept_len, accept_mask


def create_for(cfg: dict, w: synth.Weights, device, max_rows=None, flags=0):
    """Context for a configuration dict plus the uploaded weights."""
    heads, w_lm = upload_weights(w, device)
    rows = cfg["B"] * cfg["L"] if max_rows is None else max_rows
    ctx = binding.mrp_create(w.d, w.F, w.V, heads, w_lm, max_rows=rows, max_seqs=cfg["B"],
                             block_len=cfg["L"], flags=flags)
    return ctx
