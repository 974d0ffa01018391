"""Thin ctypes binding of libmrp_b200.so: argument marshalling only.

The functions carry the C ABI's names (``mrp_create``, ``mrp_draft``, ``mrp_reveal_remask``,
``mrp_verify``, ``mrp_destroy``) and take torch CUDA tensors, which serve as device memory
and supply the current stream; every step of the drafting pass runs in the library's own
kernels.  Importing this module loads the shared library and raises if it is missing or
cannot be loaded: there is no CPU or PyTorch fallback.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# MRP_B200_LIB names a library built elsewhere (e.g. an out-of-tree build of the same sources).
LIB_PATH = os.environ.get("MRP_B200_LIB") or os.path.join(_HERE, "libmrp_b200.so")

MRP_F32, MRP_BF16 = 0, 1
MRP_FLAG_FORCE_SIMT = 1
MRP_FLAG_NO_PDL = 2
MRP_FLAG_ROW_MAJOR_ONLY = 4
MRP_FLAG_EXACT_OPERANDS = 8
MRP_FLAG_NO_CHAIN = 16
MRP_FLAG_REQUIRE_TENSOR_CORES = 32
MRP_FLAG_TRAINING_KL = 64
MRP_FLAG_FP8_LM = 128
MRP_FLAG_NO_CTA_PAIRS = 256
MRP_SELECT_STATIC, MRP_SELECT_DYNAMIC_REMASK = 0, 1
MRP_DEV_NONFINITE, MRP_DEV_TIMEOUT, MRP_DEV_BAD_INDEX, MRP_DEV_RANGE = 1, 2, 4, 8
MRP_RANGE_LIMIT = 32768.0

EXPORTS = ("mrp_workspace_bytes", "mrp_create", "mrp_destroy", "mrp_draft", "mrp_reveal_remask",
           "mrp_verify", "mrp_last_launch_count", "mrp_kernel_family", "mrp_status_string",
           "mrp_profile_enable", "mrp_profile_read", "mrp_last_error",
           "mrp_reveal_remask_noalloc", "mrp_selftest_wait_timeout", "mrp_draft_from_hidden", "mrp_commit",
           "mrp_set_logits0_event", "mrp_set_input_rows", "mrp_fetch_status", "mrp_draft_kl", "mrp_draft_bf16_logits", "mrp_quantised_lm_head",
           "mrp_module_workspace_bytes", "mrp_module_attach", "mrp_module_step", "mrp_module_set_prefix", "mrp_module_step_kl")
MRP_NOALLOC_MAX_POSITIONS = 65536
MRP_ERR_CAPACITY = 7


class mrp_config(ctypes.Structure):
    _fields_ = [("d", ctypes.c_int32), ("d_ff", ctypes.c_int32), ("vocab", ctypes.c_int32),
                ("n_heads", ctypes.c_int32), ("max_rows", ctypes.c_int32),
                ("max_seqs", ctypes.c_int32), ("block_len", ctypes.c_int32),
                ("dtype", ctypes.c_int32), ("rms_eps", ctypes.c_float),
                ("device", ctypes.c_int32), ("flags", ctypes.c_int32)]


class mrp_head_weights(ctypes.Structure):
    _fields_ = [("rms_gamma", ctypes.c_void_p), ("w_gate", ctypes.c_void_p),
                ("w_up", ctypes.c_void_p), ("w_down", ctypes.c_void_p)]


class mrp_draft_out(ctypes.Structure):
    _fields_ = [("conf", ctypes.c_void_p), ("lse", ctypes.c_void_p), ("token", ctypes.c_void_p),
                ("margin", ctypes.c_void_p), ("logits_out", ctypes.c_void_p),
                ("hidden_out", ctypes.c_void_p), ("status", ctypes.c_void_p),
                ("conf_first", ctypes.c_void_p)]


class mrp_select_params(ctypes.Structure):
    _fields_ = [("mode", ctypes.c_int32), ("tau", ctypes.c_float), ("r_reveal", ctypes.c_int32),
                ("r_draft", ctypes.c_int32), ("use_cap", ctypes.c_int32),
                ("remask_policy", ctypes.c_int32), ("ensure_progress", ctypes.c_int32),
                ("conf_first", ctypes.c_void_p)]


class mrp_select_out(ctypes.Structure):
    _fields_ = [("reveal_mask", ctypes.c_void_p), ("remask_mask", ctypes.c_void_p),
                ("out_token", ctypes.c_void_p), ("step_of", ctypes.c_void_p),
                ("draft_pos", ctypes.c_void_p), ("draft_tok", ctypes.c_void_p),
                ("draft_len", ctypes.c_void_p), ("status", ctypes.c_void_p)]


class mrp_module_layer(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("g_attn", "w_q", "w_k", "w_v", "w_o", "g_mlp", "w_gate", "w_up", "w_down")]


class mrp_module_weights(ctypes.Structure):
    _fields_ = [("n_layers", ctypes.c_int32), ("n_attn_heads", ctypes.c_int32), ("mask_token", ctypes.c_int32),
                ("emb_rows", ctypes.c_int32), ("emb", ctypes.c_void_p), ("w_proj", ctypes.c_void_p),
                ("layers", ctypes.POINTER(mrp_module_layer))]


class mrp_module_kv(ctypes.Structure):
    _fields_ = [("k", ctypes.c_void_p), ("v", ctypes.c_void_p)]


class mrp_block_state(ctypes.Structure):
    _fields_ = [("tokens", ctypes.c_void_p), ("row_index", ctypes.c_void_p),
                ("n_masked", ctypes.c_void_p), ("block_masked", ctypes.c_void_p)]


def _load():
    if not os.path.exists(LIB_PATH):
        raise ImportError(
            "libmrp_b200.so is not built (%s); run `python -m paper_2605_18817_b200.build` "
            "-- there is no fallback path" % LIB_PATH)
    lib = ctypes.CDLL(LIB_PATH)
    for name in EXPORTS:
        getattr(lib, name)
    lib.mrp_workspace_bytes.restype = ctypes.c_size_t
    lib.mrp_workspace_bytes.argtypes = [ctypes.POINTER(mrp_config)]
    lib.mrp_create.restype = ctypes.c_int
    lib.mrp_create.argtypes = [ctypes.POINTER(mrp_config), ctypes.POINTER(mrp_head_weights),
                               ctypes.c_void_p, ctypes.c_void_p, ctypes.c_size_t,
                               ctypes.POINTER(ctypes.c_void_p)]
    lib.mrp_destroy.restype = None
    lib.mrp_destroy.argtypes = [ctypes.c_void_p]
    lib.mrp_draft.restype = ctypes.c_int
    lib.mrp_draft.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                              ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(mrp_draft_out),
                              ctypes.c_void_p]
    lib.mrp_draft_bf16_logits.restype = ctypes.c_int
    lib.mrp_draft_bf16_logits.argtypes = lib.mrp_draft.argtypes
    lib.mrp_quantised_lm_head.restype = ctypes.c_int
    lib.mrp_quantised_lm_head.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_void_p), ctypes.POINTER(ctypes.c_void_p)]
    lib.mrp_module_workspace_bytes.restype = ctypes.c_size_t
    lib.mrp_module_workspace_bytes.argtypes = [ctypes.POINTER(mrp_config), ctypes.POINTER(mrp_module_weights)]
    lib.mrp_module_attach.restype = ctypes.c_int
    lib.mrp_module_attach.argtypes = [ctypes.c_void_p, ctypes.POINTER(mrp_module_weights), ctypes.c_void_p, ctypes.c_size_t]
    lib.mrp_module_step_kl.restype = ctypes.c_int
    lib.mrp_module_step_kl.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                       ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                       ctypes.c_int32, ctypes.POINTER(mrp_draft_out), ctypes.c_void_p, ctypes.c_void_p]
    lib.mrp_module_set_prefix.restype = ctypes.c_int
    lib.mrp_module_set_prefix.argtypes = [ctypes.c_void_p, ctypes.POINTER(mrp_module_kv), ctypes.c_void_p, ctypes.c_int32,
                                          ctypes.c_int32]
    lib.mrp_module_step.restype = ctypes.c_int
    lib.mrp_module_step.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                    ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32,
                                    ctypes.POINTER(mrp_draft_out), ctypes.c_void_p]
    lib.mrp_draft_kl.restype = ctypes.c_int
    lib.mrp_draft_kl.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                 ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(mrp_draft_out), ctypes.c_void_p,
                                 ctypes.c_void_p]
    lib.mrp_set_logits0_event.restype = ctypes.c_int
    lib.mrp_set_logits0_event.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
    lib.mrp_set_input_rows.restype = ctypes.c_int
    lib.mrp_set_input_rows.argtypes = [ctypes.c_void_p, ctypes.c_int32]
    lib.mrp_fetch_status.restype = ctypes.c_int
    lib.mrp_fetch_status.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int32, ctypes.c_void_p]
    lib.mrp_commit.restype = ctypes.c_int
    lib.mrp_commit.argtypes = [ctypes.c_void_p, ctypes.POINTER(mrp_select_out), ctypes.c_void_p, ctypes.c_int32,
                               ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(mrp_block_state), ctypes.c_void_p]
    lib.mrp_draft_from_hidden.restype = ctypes.c_int
    lib.mrp_draft_from_hidden.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                          ctypes.c_int32, ctypes.c_int32, ctypes.POINTER(mrp_draft_out),
                                          ctypes.c_void_p]
    lib.mrp_reveal_remask.restype = ctypes.c_int
    lib.mrp_reveal_remask.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                      ctypes.c_void_p, ctypes.c_int32, ctypes.c_int32,
                                      ctypes.c_int32, ctypes.c_int32,
                                      ctypes.POINTER(mrp_select_params),
                                      ctypes.POINTER(mrp_select_out), ctypes.c_void_p]
    lib.mrp_reveal_remask_noalloc.restype = ctypes.c_int
    lib.mrp_reveal_remask_noalloc.argtypes = lib.mrp_reveal_remask.argtypes[1:]
    lib.mrp_selftest_wait_timeout.restype = ctypes.c_int
    lib.mrp_selftest_wait_timeout.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    lib.mrp_verify.restype = ctypes.c_int
    lib.mrp_verify.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                               ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p,
                               ctypes.c_void_p, ctypes.c_void_p]
    lib.mrp_profile_enable.restype = ctypes.c_int
    lib.mrp_profile_enable.argtypes = [ctypes.c_void_p, ctypes.c_int32]
    lib.mrp_profile_read.restype = ctypes.c_int
    lib.mrp_profile_read.argtypes = [ctypes.c_void_p, ctypes.POINTER(ctypes.c_float),
                                     ctypes.POINTER(ctypes.c_int32)]
    lib.mrp_last_launch_count.restype = ctypes.c_int32
    lib.mrp_last_launch_count.argtypes = [ctypes.c_void_p]
    lib.mrp_last_error.restype = ctypes.c_char_p
    lib.mrp_last_error.argtypes = [ctypes.c_void_p]
    lib.mrp_kernel_family.restype = ctypes.c_char_p
    lib.mrp_kernel_family.argtypes = [ctypes.c_void_p]
    lib.mrp_status_string.restype = ctypes.c_char_p
    lib.mrp_status_string.argtypes = [ctypes.c_int]
    return lib


lib = _load()


class MrpError(RuntimeError):
    def __init__(self, where: str, status: int, detail: str = ""):
        self.status = status
        super().__init__("%s: %s (%d)%s" % (where, lib.mrp_status_string(status).decode(), status,
                                            " -- " + detail if detail else ""))


def _ptr(t):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(t, dtype, what):
    if t is None:
        return
    if not (t.is_cuda and t.is_contiguous() and t.dtype == dtype):
        raise TypeError("%s must be a contiguous CUDA tensor of %s" % (what, dtype))


@dataclass
class Context:
    handle: int
    cfg: mrp_config
    keep: tuple           # weights + workspace kept alive for the context's lifetime
    guards: tuple = ()    # (buffer, workspace offset, workspace bytes, guard bytes) for workspace_guards_intact

    @property
    def family(self) -> str:
        return lib.mrp_kernel_family(self.handle).decode()

    @property
    def last_launch_count(self) -> int:
        return int(lib.mrp_last_launch_count(self.handle))


def mrp_workspace_bytes(cfg: mrp_config) -> int:
    return int(lib.mrp_workspace_bytes(ctypes.byref(cfg)))


def mrp_create(d, d_ff, vocab, heads, w_lm, max_rows, max_seqs, block_len, rms_eps=1e-6,
               flags=0, guard_bytes=0) -> Context:
    """heads: list of dicts of CUDA tensors gamma [d], w_gate [F,d], w_up [F,d], w_down [d,F];
    w_lm: CUDA tensor [V,d]; dtype (float32 or bfloat16) is taken from w_lm.  ``guard_bytes``
    (a multiple of 256) surrounds the workspace with bands of that many 0xA5 bytes, which
    ``workspace_guards_intact`` checks: a way for tests to see a write outside the workspace."""
    tdtype = w_lm.dtype
    if tdtype not in (torch.float32, torch.bfloat16):
        raise TypeError("weights must be float32 or bfloat16")
    _check(w_lm, tdtype, "w_lm")
    dev = w_lm.device.index if w_lm.device.index is not None else torch.cuda.current_device()
    cfg = mrp_config(int(d), int(d_ff), int(vocab), len(heads), int(max_rows), int(max_seqs),
                     int(block_len), MRP_F32 if tdtype == torch.float32 else MRP_BF16,
                     float(rms_eps), int(dev), int(flags))
    harr = (mrp_head_weights * max(len(heads), 1))()
    keep = [w_lm]
    for k, h in enumerate(heads):
        for name in ("gamma", "w_gate", "w_up", "w_down"):
            _check(h[name], tdtype, name)
            keep.append(h[name])
        harr[k] = mrp_head_weights(h["gamma"].data_ptr(), h["w_gate"].data_ptr(),
                                   h["w_up"].data_ptr(), h["w_down"].data_ptr())
    nbytes = mrp_workspace_bytes(cfg)
    if nbytes == 0:
        raise MrpError("mrp_workspace_bytes", 1)
    guard_bytes = (int(guard_bytes) + 255) // 256 * 256
    ws = torch.full((nbytes + 256 + 2 * guard_bytes,), 0xA5, dtype=torch.uint8, device=w_lm.device)
    off = (-ws.data_ptr()) % 256 + guard_bytes
    keep.append(ws)
    handle = ctypes.c_void_p()
    rc = lib.mrp_create(ctypes.byref(cfg), harr, _ptr(w_lm), ctypes.c_void_p(ws.data_ptr() + off),
                        ctypes.c_size_t(nbytes), ctypes.byref(handle))
    if rc != 0:
        raise MrpError("mrp_create", rc)
    ctx = Context(handle.value, cfg, tuple(keep))
    ctx.guards = (ws, off, nbytes, guard_bytes)
    return ctx


def workspace_guards_intact(ctx: Context) -> bool:
    """True if the bands around the workspace (``guard_bytes`` of mrp_create) still hold their
    fill pattern; synchronises."""
    ws, off, nbytes, g = ctx.guards
    if g == 0:
        return True
    before, after = ws[off - g:off], ws[off + nbytes:off + nbytes + g]
    return bool((before == 0xA5).all().item()) and bool((after == 0xA5).all().item())


def mrp_quantised_lm_head(ctx: Context):
    """Host copies (uint8 codes [V, d], float32 scales [V]) of the 8-bit LM head of an MRP_FLAG_FP8_LM context."""
    codes, scales = ctypes.c_void_p(), ctypes.c_void_p()
    rc = lib.mrp_quantised_lm_head(ctx.handle, ctypes.byref(codes), ctypes.byref(scales))
    if rc != 0:
        raise MrpError("mrp_quantised_lm_head", rc)
    V, d = ctx.cfg.vocab, ctx.cfg.d
    dev = "cuda:%d" % ctx.cfg.device
    c = torch.empty((V, d), dtype=torch.uint8, device=dev)
    s = torch.empty(V, dtype=torch.float32, device=dev)
    ws = ctx.guards[0]          # the tensor that holds the workspace: the two pointers lie inside it
    c.copy_(ws[codes.value - ws.data_ptr():codes.value - ws.data_ptr() + V * d].view(V, d))
    s.copy_(ws[scales.value - ws.data_ptr():scales.value - ws.data_ptr() + 4 * V].view(torch.float32))
    return c.cpu().numpy(), s.cpu().numpy()


def mrp_module_attach(ctx: Context, emb, w_proj, layers, n_attn_heads, mask_token) -> None:
    """Attach the token-conditioned module: ``emb`` [rows, d], ``w_proj`` [d, 2d], ``layers`` a list of dicts
    of CUDA tensors named like the fields of mrp_module_layer.  Allocates the module's workspace (a torch
    tensor kept alive with the context)."""
    tdtype = torch.float32 if ctx.cfg.dtype == MRP_F32 else torch.bfloat16
    _check(emb, tdtype, "emb")
    _check(w_proj, tdtype, "w_proj")
    larr = (mrp_module_layer * max(len(layers), 1))()
    keep = [emb, w_proj]
    for i, lay in enumerate(layers):
        vals = []
        for name, _ in mrp_module_layer._fields_:
            _check(lay[name], tdtype, name)
            keep.append(lay[name])
            vals.append(lay[name].data_ptr())
        larr[i] = mrp_module_layer(*vals)
    w = mrp_module_weights(len(layers), int(n_attn_heads), int(mask_token), int(emb.shape[0]), emb.data_ptr(),
                           w_proj.data_ptr(), larr)
    nbytes = int(lib.mrp_module_workspace_bytes(ctypes.byref(ctx.cfg), ctypes.byref(w)))
    if nbytes == 0:
        raise MrpError("mrp_module_workspace_bytes", 1)
    ws = torch.empty(nbytes + 256, dtype=torch.uint8, device=emb.device)
    off = (-ws.data_ptr()) % 256
    rc = lib.mrp_module_attach(ctx.handle, ctypes.byref(w), ctypes.c_void_p(ws.data_ptr() + off), ctypes.c_size_t(nbytes))
    if rc != 0:
        raise MrpError("mrp_module_attach", rc)
    ctx.keep = tuple(ctx.keep) + tuple(keep) + (ws,)


def mrp_module_step(ctx: Context, tokens, hidden0, h_state, logits0, row_index, M, B, L, first_step, conf, lse, token,
                    margin=None, logits_out=None, hidden_out=None, status=None, conf_first=None, stream=None) -> None:
    """One step of the attached module; conf / lse / token are [2, M] (backbone, after this step)."""
    tdtype = torch.float32 if ctx.cfg.dtype == MRP_F32 else torch.bfloat16
    for t, dt, nm in ((tokens, torch.int32, "tokens"), (hidden0, tdtype, "hidden0"), (h_state, torch.float32, "h_state"),
                      (logits0, torch.float32, "logits0"), (row_index, torch.int32, "row_index"),
                      (conf, torch.float32, "conf"), (lse, torch.float32, "lse"), (token, torch.int32, "token"),
                      (margin, torch.float32, "margin"), (logits_out, torch.float32, "logits_out"),
                      (hidden_out, torch.float32, "hidden_out"), (status, torch.int32, "status"),
                      (conf_first, torch.float32, "conf_first")):
        _check(t, dt, nm)
    out = mrp_draft_out(_ptr(conf), _ptr(lse), _ptr(token), _ptr(margin), _ptr(logits_out), _ptr(hidden_out),
                        _ptr(status), _ptr(conf_first))
    rc = lib.mrp_module_step(ctx.handle, _ptr(tokens), _ptr(hidden0), _ptr(h_state), _ptr(logits0), _ptr(row_index),
                             int(M), int(B), int(L), int(bool(first_step)), ctypes.byref(out), _stream(stream))
    if rc != 0:
        raise MrpError("mrp_module_step", rc, lib.mrp_last_error(ctx.handle).decode())


def mrp_module_step_kl(ctx: Context, tokens, hidden0, h_state, logits0, teacher, row_index, M, B, L, first_step, conf, lse,
                       token, kl, margin=None, hidden_out=None, status=None, stream=None) -> None:
    """mrp_module_step with kl[m] = KL(softmax(teacher[m]) || softmax(l[m])) of the step fused into its LM-head pass:
    ``teacher`` [M, V] fp32, ``kl`` [M] fp32 (context created with MRP_FLAG_TRAINING_KL)."""
    tdtype = torch.float32 if ctx.cfg.dtype == MRP_F32 else torch.bfloat16
    for t, dt, nm in ((tokens, torch.int32, "tokens"), (hidden0, tdtype, "hidden0"), (h_state, torch.float32, "h_state"),
                      (logits0, torch.float32, "logits0"), (teacher, torch.float32, "teacher"), (row_index, torch.int32, "row_index"),
                      (conf, torch.float32, "conf"), (lse, torch.float32, "lse"), (token, torch.int32, "token"),
                      (kl, torch.float32, "kl"), (margin, torch.float32, "margin"), (hidden_out, torch.float32, "hidden_out"),
                      (status, torch.int32, "status")):
        _check(t, dt, nm)
    out = mrp_draft_out(_ptr(conf), _ptr(lse), _ptr(token), _ptr(margin), None, _ptr(hidden_out), _ptr(status), None)
    rc = lib.mrp_module_step_kl(ctx.handle, _ptr(tokens), _ptr(hidden0), _ptr(h_state), _ptr(logits0), _ptr(teacher), _ptr(row_index),
                                int(M), int(B), int(L), int(bool(first_step)), ctypes.byref(out), _ptr(kl), _stream(stream))
    if rc != 0:
        raise MrpError("mrp_module_step_kl", rc, lib.mrp_last_error(ctx.handle).decode())


def prefix_to_head_major(x, n_attn_heads: int):
    """[sequences, positions, d] -> the cache layout [sequences, heads, positions, d / heads] (a contiguous copy)."""
    B, cap, d = x.shape
    return x.view(B, cap, n_attn_heads, d // n_attn_heads).permute(0, 2, 1, 3).contiguous()


def prefix_from_head_major(x):
    """The inverse of prefix_to_head_major."""
    B, H, cap, dh = x.shape
    return x.permute(0, 2, 1, 3).reshape(B, cap, H * dh)


def mrp_module_set_prefix(ctx: Context, caches, prefix_len, append=False) -> None:
    """Attach the clean prefix of the module's attention: ``caches`` a list (one entry per module layer) of
    (k, v) CUDA tensors [max_seqs, n_attn_heads, prefix_cap, d / n_attn_heads] (head-major) in the context dtype,
    ``prefix_len`` [max_seqs] int32 on the device; ``caches`` None detaches.  With ``append`` the following steps also
    store their own keys and values behind the prefix rows."""
    if caches is None:
        rc = lib.mrp_module_set_prefix(ctx.handle, None, None, 0, 0)
        if rc != 0:
            raise MrpError("mrp_module_set_prefix", rc)
        return
    tdtype = torch.float32 if ctx.cfg.dtype == MRP_F32 else torch.bfloat16
    _check(prefix_len, torch.int32, "prefix_len")
    arr = (mrp_module_kv * max(len(caches), 1))()
    cap = 0
    for i, (k, v) in enumerate(caches):
        _check(k, tdtype, "prefix k")
        _check(v, tdtype, "prefix v")
        if k.dim() != 4 or k.shape != v.shape or k.shape[1] * k.shape[3] != ctx.cfg.d:
            raise ValueError("prefix caches are [max_seqs, n_attn_heads, prefix_cap, d / n_attn_heads]")
        cap = int(k.shape[2])
        arr[i] = mrp_module_kv(k.data_ptr(), v.data_ptr())
    rc = lib.mrp_module_set_prefix(ctx.handle, arr, _ptr(prefix_len), cap, int(bool(append)))
    if rc != 0:
        raise MrpError("mrp_module_set_prefix", rc)
    ctx.prefix_keep = (caches, prefix_len)


def mrp_set_input_rows(ctx: Context, n_rows: int) -> None:
    rc = lib.mrp_set_input_rows(ctx.handle, int(n_rows))
    if rc != 0:
        raise MrpError("mrp_set_input_rows", rc)


def mrp_fetch_status(ctx: Context, clear: bool = False, stream=None) -> int:
    """The context's device status word (MRP_DEV_* bits); synchronises to return it as an int."""
    dst = torch.zeros(1, dtype=torch.int32, device="cuda:%d" % ctx.cfg.device)
    rc = lib.mrp_fetch_status(ctx.handle, _ptr(dst), int(bool(clear)), _stream(stream))
    if rc != 0:
        raise MrpError("mrp_fetch_status", rc)
    return int(dst.item())


def mrp_destroy(ctx: Context) -> None:
    if ctx.handle:
        lib.mrp_destroy(ctx.handle)
        ctx.handle = 0


def mrp_profile_enable(ctx: Context, enable: bool) -> None:
    rc = lib.mrp_profile_enable(ctx.handle, int(bool(enable)))
    if rc != 0:
        raise MrpError("mrp_profile_enable", rc)


def mrp_profile_read(ctx: Context):
    """(ms_heads, ms_lm_head, ms_combine) summed over n calls, and n; sync the stream first."""
    ms = (ctypes.c_float * 3)()
    n = ctypes.c_int32()
    rc = lib.mrp_profile_read(ctx.handle, ms, ctypes.byref(n))
    if rc != 0:
        raise MrpError("mrp_profile_read", rc)
    return (float(ms[0]), float(ms[1]), float(ms[2])), int(n.value)


def mrp_draft(ctx: Context, hidden, logits0, row_index, M, K, conf, lse, token, margin=None,
              logits_out=None, hidden_out=None, status=None, stream=None, conf_first=None) -> None:
    """Enqueue one drafting pass; outputs are written into the given CUDA tensors.  ``logits0`` in
    float32 goes to mrp_draft, in bfloat16 to mrp_draft_bf16_logits."""
    _check(hidden, torch.float32 if ctx.cfg.dtype == MRP_F32 else torch.bfloat16, "hidden")
    l0_bf16 = logits0 is not None and logits0.dtype == torch.bfloat16
    _check(logits0, torch.bfloat16 if l0_bf16 else torch.float32, "logits0")
    _check(row_index, torch.int32, "row_index")
    for t, dt, nm in ((conf, torch.float32, "conf"), (lse, torch.float32, "lse"),
                      (token, torch.int32, "token"), (margin, torch.float32, "margin"),
                      (logits_out, torch.float32, "logits_out"),
                      (hidden_out, torch.float32, "hidden_out"), (status, torch.int32, "status"),
                      (conf_first, torch.float32, "conf_first")):
        _check(t, dt, nm)
    out = mrp_draft_out(_ptr(conf), _ptr(lse), _ptr(token), _ptr(margin), _ptr(logits_out),
                        _ptr(hidden_out), _ptr(status), _ptr(conf_first))
    fn = lib.mrp_draft_bf16_logits if l0_bf16 else lib.mrp_draft
    rc = fn(ctx.handle, _ptr(hidden), _ptr(logits0), _ptr(row_index), int(M), int(K),
            ctypes.byref(out), _stream(stream))
    if rc != 0:
        raise MrpError("mrp_draft", rc, lib.mrp_last_error(ctx.handle).decode())


def mrp_draft_kl(ctx: Context, hidden, logits0, teacher, row_index, M, K, conf, lse, token, kl, margin=None,
                 hidden_out=None, status=None, stream=None) -> None:
    """The drafting pass with the KL objective of every unrolled step fused into the LM-head epilogue:
    ``teacher`` [K, M, V] fp32, ``kl`` [K, M] fp32 (context created with MRP_FLAG_TRAINING_KL)."""
    _check(hidden, torch.float32 if ctx.cfg.dtype == MRP_F32 else torch.bfloat16, "hidden")
    _check(logits0, torch.float32, "logits0")
    _check(teacher, torch.float32, "teacher")
    _check(row_index, torch.int32, "row_index")
    for t, dt, nm in ((conf, torch.float32, "conf"), (lse, torch.float32, "lse"), (token, torch.int32, "token"),
                      (kl, torch.float32, "kl"), (margin, torch.float32, "margin"),
                      (hidden_out, torch.float32, "hidden_out"), (status, torch.int32, "status")):
        _check(t, dt, nm)
    out = mrp_draft_out(_ptr(conf), _ptr(lse), _ptr(token), _ptr(margin), None, _ptr(hidden_out), _ptr(status), None)
    rc = lib.mrp_draft_kl(ctx.handle, _ptr(hidden), _ptr(logits0), _ptr(teacher), _ptr(row_index), int(M), int(K),
                          ctypes.byref(out), _ptr(kl), _stream(stream))
    if rc != 0:
        raise MrpError("mrp_draft_kl", rc, lib.mrp_last_error(ctx.handle).decode())


def mrp_draft_from_hidden(ctx: Context, hidden, final_norm_gamma, row_index, M, K, conf, lse, token,
                          margin=None, logits_out=None, hidden_out=None, status=None, stream=None,
                          conf_first=None) -> None:
    """Enqueue one drafting pass that computes the base logits itself (l_0 = W_lm n_0)."""
    dt_ctx = torch.float32 if ctx.cfg.dtype == MRP_F32 else torch.bfloat16
    _check(hidden, dt_ctx, "hidden")
    _check(final_norm_gamma, dt_ctx, "final_norm_gamma")
    _check(row_index, torch.int32, "row_index")
    for t, dt, nm in ((conf, torch.float32, "conf"), (lse, torch.float32, "lse"),
                      (token, torch.int32, "token"), (margin, torch.float32, "margin"),
                      (logits_out, torch.float32, "logits_out"),
                      (hidden_out, torch.float32, "hidden_out"), (status, torch.int32, "status"),
                      (conf_first, torch.float32, "conf_first")):
        _check(t, dt, nm)
    out = mrp_draft_out(_ptr(conf), _ptr(lse), _ptr(token), _ptr(margin), _ptr(logits_out),
                        _ptr(hidden_out), _ptr(status), _ptr(conf_first))
    rc = lib.mrp_draft_from_hidden(ctx.handle, _ptr(hidden), _ptr(final_norm_gamma), _ptr(row_index),
                                   int(M), int(K), ctypes.byref(out), _stream(stream))
    if rc != 0:
        raise MrpError("mrp_draft_from_hidden", rc, lib.mrp_last_error(ctx.handle).decode())


def mrp_reveal_remask(ctx: Context, conf, token, row_index, M, K, B, L, mode, tau=0.9, r_reveal=1,
                      r_draft=1, use_cap=False, remask_policy=0, ensure_progress=True, conf_first=None, *,
                      reveal_mask, remask_mask, out_token, step_of, draft_pos, draft_tok, draft_len,
                      status=None, stream=None) -> None:
    _check(conf, torch.float32, "conf")
    _check(token, torch.int32, "token")
    _check(row_index, torch.int32, "row_index")
    for t, dt, nm in ((reveal_mask, torch.int8, "reveal_mask"), (remask_mask, torch.int8, "remask_mask"),
                      (out_token, torch.int32, "out_token"), (step_of, torch.int8, "step_of"),
                      (draft_pos, torch.int32, "draft_pos"), (draft_tok, torch.int32, "draft_tok"),
                      (draft_len, torch.int32, "draft_len"), (status, torch.int32, "status")):
        _check(t, dt, nm)
    _check(conf_first, torch.float32, "conf_first")
    p = mrp_select_params(int(mode), float(tau), int(r_reveal), int(r_draft), int(bool(use_cap)),
                          int(remask_policy), int(bool(ensure_progress)), _ptr(conf_first))
    o = mrp_select_out(_ptr(reveal_mask), _ptr(remask_mask), _ptr(out_token), _ptr(step_of),
                       _ptr(draft_pos), _ptr(draft_tok), _ptr(draft_len), _ptr(status))
    rc = lib.mrp_reveal_remask(ctx.handle, _ptr(conf), _ptr(token), _ptr(row_index), int(M), int(K),
                               int(B), int(L), ctypes.byref(p), ctypes.byref(o), _stream(stream))
    if rc != 0:
        raise MrpError("mrp_reveal_remask", rc)


def mrp_reveal_remask_noalloc(conf, token, row_index, M, K, B, L, mode, tau=0.9, r_reveal=1,
                              r_draft=1, use_cap=False, remask_policy=0, ensure_progress=True, conf_first=None, *,
                              reveal_mask, remask_mask, out_token, step_of, draft_pos, draft_tok,
                              draft_len, status=None, stream=None) -> None:
    """Reveal selection for callers that cannot allocate device memory: no context and no
    workspace, the position map lives in a fixed array inside the library (B * L at most
    MRP_NOALLOC_MAX_POSITIONS).  The tensors' device must be the current device.  Calls on
    one device share that array, so calls that could overlap on the GPU must be serialised."""
    _check(conf, torch.float32, "conf")
    _check(token, torch.int32, "token")
    _check(row_index, torch.int32, "row_index")
    for t, dt, nm in ((reveal_mask, torch.int8, "reveal_mask"), (remask_mask, torch.int8, "remask_mask"),
                      (out_token, torch.int32, "out_token"), (step_of, torch.int8, "step_of"),
                      (draft_pos, torch.int32, "draft_pos"), (draft_tok, torch.int32, "draft_tok"),
                      (draft_len, torch.int32, "draft_len"), (status, torch.int32, "status")):
        _check(t, dt, nm)
    _check(conf_first, torch.float32, "conf_first")
    p = mrp_select_params(int(mode), float(tau), int(r_reveal), int(r_draft), int(bool(use_cap)),
                          int(remask_policy), int(bool(ensure_progress)), _ptr(conf_first))
    o = mrp_select_out(_ptr(reveal_mask), _ptr(remask_mask), _ptr(out_token), _ptr(step_of),
                       _ptr(draft_pos), _ptr(draft_tok), _ptr(draft_len), _ptr(status))
    rc = lib.mrp_reveal_remask_noalloc(_ptr(conf), _ptr(token), _ptr(row_index), int(M), int(K),
                                       int(B), int(L), ctypes.byref(p), ctypes.byref(o),
                                       _stream(stream))
    if rc != 0:
        raise MrpError("mrp_reveal_remask_noalloc", rc)


def mrp_selftest_wait_timeout(ctx: Context, status, stream=None) -> None:
    """Launch the bounded-wait self-test: after a sync, ``status`` carries MRP_DEV_TIMEOUT."""
    _check(status, torch.int32, "status")
    rc = lib.mrp_selftest_wait_timeout(ctx.handle, _ptr(status), _stream(stream))
    if rc != 0:
        raise MrpError("mrp_selftest_wait_timeout", rc)


def mrp_set_logits0_event(ctx: Context, event) -> None:
    """``event``: a recorded ``torch.cuda.Event`` (or None): mrp_draft waits for it right before the LM head."""
    h = None if event is None else ctypes.c_void_p(event.cuda_event)
    rc = lib.mrp_set_logits0_event(ctx.handle, h)
    if rc != 0:
        raise MrpError("mrp_set_logits0_event", rc)


def mrp_commit(ctx: Context, B, L, Kd, *, out_token, step_of, draft_pos, draft_tok, accept_mask=None,
               tokens, row_index, n_masked, block_masked, stream=None) -> None:
    """Apply one pass's selection (and, if given, verification) to the block state."""
    for t, dt, nm in ((out_token, torch.int32, "out_token"), (step_of, torch.int8, "step_of"),
                      (draft_pos, torch.int32, "draft_pos"), (draft_tok, torch.int32, "draft_tok"),
                      (accept_mask, torch.int8, "accept_mask"), (tokens, torch.int32, "tokens"),
                      (row_index, torch.int32, "row_index"), (n_masked, torch.int32, "n_masked"),
                      (block_masked, torch.int32, "block_masked")):
        _check(t, dt, nm)
    sel = mrp_select_out(None, None, _ptr(out_token), _ptr(step_of), _ptr(draft_pos), _ptr(draft_tok), None, None)
    state = mrp_block_state(_ptr(tokens), _ptr(row_index), _ptr(n_masked), _ptr(block_masked))
    rc = lib.mrp_commit(ctx.handle, ctypes.byref(sel), _ptr(accept_mask), int(B), int(L), int(Kd),
                        ctypes.byref(state), _stream(stream))
    if rc != 0:
        raise MrpError("mrp_commit", rc, lib.mrp_last_error(ctx.handle).decode())


def mrp_verify(ctx: Context, draft_tok, verify_tok, draft_len, B, Kd, positionwise, accept_len,
               accept_mask, stream=None) -> None:
    for t, dt, nm in ((draft_tok, torch.int32, "draft_tok"), (verify_tok, torch.int32, "verify_tok"),
                      (draft_len, torch.int32, "draft_len"), (accept_len, torch.int32, "accept_len"),
                      (accept_mask, torch.int8, "accept_mask")):
        _check(t, dt, nm)
    rc = lib.mrp_verify(ctx.handle, _ptr(draft_tok), _ptr(verify_tok), _ptr(draft_len), int(B),
                        int(Kd), int(bool(positionwise)), _ptr(accept_len), _ptr(accept_mask),
                        _stream(stream))
    if rc != 0:
        raise MrpError("mrp_verify", rc)
