"""Thin ctypes binding of libbeagle.so (include/beagle.h).

Argument marshalling only: every step of the draft head runs in the CUDA
kernels behind the C ABI.  PyTorch supplies device memory (tensors) and the
current CUDA stream; nothing here computes.  Importing this module fails loudly
when the shared library has not been built -- there is no CPU fallback.
"""
from __future__ import annotations

import ctypes as C
import os
import weakref
from typing import Dict, Optional, Sequence, Tuple

import torch

from . import build as _build

BEAGLE_FP32, BEAGLE_BF16 = 0, 1
BEAGLE_MAX_CALL_BATCH = 64
STATUS_NAMES = {0: "OK", 1: "INVALID_ARG", 2: "SHAPE", 3: "CAPACITY", 4: "STATE", 5: "UNSUPPORTED", 6: "CUDA", 7: "DEVICE"}

WEIGHT_NAMES = ("embed", "g_q", "w_q", "w_k", "w_v", "w_o", "g_mlp", "w_gate", "w_up", "w_down", "w_lm")

EXPORTED_SYMBOLS = (
    "beagle_version", "beagle_query_sizes", "beagle_create", "beagle_destroy", "beagle_prefill_kv",
    "beagle_draft_step", "beagle_rollback", "beagle_reset_slot", "beagle_slot_lengths",
    "beagle_block_workspace_bytes", "beagle_block_forward", "beagle_verify_greedy", "beagle_last_error",
    "beagle_launch_count", "beagle_profile_enable", "beagle_profile_read", "beagle_profile_stage_count",
    "beagle_profile_stage_name", "beagle_verify_greedy_static", "beagle_check_device", "beagle_selftest_wait_timeout",
    "beagle_workspace_buffer", "beagle_block_workspace_buffer", "beagle_verify_sample", "beagle_block_loss", "beagle_draft_tree", "beagle_verify_tree_greedy",
    "beagle_block_grad_workspace_bytes", "beagle_block_grad", "beagle_quantize_rows_e4m3",
    "beagle_packed_weights_bytes", "beagle_pack_weights",
)

BUFFER_IDS = {"x": 0, "xn": 1, "q": 2, "o": 3, "y": 4, "yn": 5, "act": 6, "h": 7, "kt": 8, "vt": 9, "kp": 10, "vp": 11}


class BeagleConfig(C.Structure):
    _fields_ = [
        ("hidden", C.c_int32), ("n_q_heads", C.c_int32), ("n_kv_heads", C.c_int32), ("head_dim", C.c_int32),
        ("mlp_dim", C.c_int32), ("vocab", C.c_int32), ("dtype", C.c_int32), ("rms_eps", C.c_float),
        ("norm_q", C.c_int32), ("norm_mlp", C.c_int32), ("max_slots", C.c_int32), ("max_ctx", C.c_int32),
        ("max_draft", C.c_int32), ("rope_theta", C.c_float),
    ]


class BeagleWeights(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in WEIGHT_NAMES] + [("w_lm_fp8", C.c_void_p), ("w_lm_scale", C.c_void_p)]


class BeagleGrads(C.Structure):
    _fields_ = [(n, C.c_void_p) for n in WEIGHT_NAMES]


class BeagleError(RuntimeError):
    def __init__(self, status: int, message: str):
        super().__init__(f"beagle status {status} ({STATUS_NAMES.get(status, '?')}): {message}")
        self.status = status


_lib: Optional[C.CDLL] = None


def load_library(path: Optional[str] = None) -> C.CDLL:
    """Loads libbeagle.so (built in-tree by ``build.build()``); raises if it is missing."""
    global _lib
    if _lib is not None and path is None:
        return _lib
    # BEAGLE_LIBRARY: another build of the same library (the tests load the bounds-checking build this way)
    p = path or os.environ.get("BEAGLE_LIBRARY") or _build.LIB_PATH
    if not os.path.exists(p):
        raise ImportError(f"{p} not found: run `python -m paper_2505_24544_b200.build` (there is no fallback path)")
    lib = C.CDLL(p)
    vp, i32, i32p, szp = C.c_void_p, C.c_int32, C.POINTER(C.c_int32), C.POINTER(C.c_size_t)
    lib.beagle_version.restype = C.c_char_p
    lib.beagle_version.argtypes = []
    lib.beagle_query_sizes.argtypes = [C.POINTER(BeagleConfig), szp, szp]
    lib.beagle_create.argtypes = [C.POINTER(BeagleConfig), C.POINTER(BeagleWeights), vp, C.c_size_t, vp, C.c_size_t, C.POINTER(vp)]
    lib.beagle_destroy.argtypes = [vp]
    lib.beagle_prefill_kv.argtypes = [vp, i32, i32p, i32p, vp, vp]
    lib.beagle_draft_step.argtypes = [vp, i32, i32p, vp, i32, vp, i32, vp, vp, vp]
    lib.beagle_rollback.argtypes = [vp, i32, i32p]
    lib.beagle_reset_slot.argtypes = [vp, i32]
    lib.beagle_slot_lengths.argtypes = [vp, i32, i32p, i32p]
    lib.beagle_block_workspace_bytes.argtypes = [C.POINTER(BeagleConfig), i32, i32, szp]
    lib.beagle_block_forward.argtypes = [vp, i32, i32, vp, vp, i32, i32, i32, vp, vp, vp, vp, C.c_size_t, vp]
    lib.beagle_verify_greedy.argtypes = [vp, i32, i32, vp, vp, i32, vp, vp, vp, vp]
    lib.beagle_last_error.restype = C.c_char_p
    lib.beagle_last_error.argtypes = [vp]
    lib.beagle_profile_enable.argtypes = [vp, i32]
    lib.beagle_profile_enable.restype = C.c_int
    lib.beagle_profile_read.argtypes = [vp, C.POINTER(C.c_float), i32p]
    lib.beagle_profile_read.restype = C.c_int
    lib.beagle_profile_stage_count.argtypes = []
    lib.beagle_profile_stage_count.restype = C.c_int32
    lib.beagle_profile_stage_name.argtypes = [i32]
    lib.beagle_profile_stage_name.restype = C.c_char_p
    lib.beagle_verify_greedy_static.argtypes = [i32, i32, i32, vp, vp, i32, vp, vp, vp, C.c_char_p, C.c_size_t]
    lib.beagle_verify_greedy_static.restype = C.c_int
    lib.beagle_workspace_buffer.argtypes = [C.POINTER(BeagleConfig), i32, szp, i32p]
    lib.beagle_workspace_buffer.restype = C.c_int
    lib.beagle_block_workspace_buffer.argtypes = [C.POINTER(BeagleConfig), i32, i32, i32, szp, i32p]
    lib.beagle_block_workspace_buffer.restype = C.c_int
    lib.beagle_block_loss.argtypes = [vp, i32, i32, vp, vp, i32, i32, i32, i32, vp, i32, vp, vp, vp, vp, C.c_size_t, vp]
    lib.beagle_block_loss.restype = C.c_int
    lib.beagle_block_grad_workspace_bytes.argtypes = [C.POINTER(BeagleConfig), i32, i32, szp]
    lib.beagle_block_grad_workspace_bytes.restype = C.c_int
    lib.beagle_block_grad.argtypes = [vp, i32, i32, vp, vp, i32, i32, i32, i32, vp, i32, vp, C.c_float, C.POINTER(BeagleGrads), vp, vp,
                                      C.c_size_t, vp]
    lib.beagle_block_grad.restype = C.c_int
    lib.beagle_quantize_rows_e4m3.argtypes = [vp, i32, C.c_int64, i32, vp, vp, vp]
    lib.beagle_quantize_rows_e4m3.restype = C.c_int
    lib.beagle_draft_tree.argtypes = [vp, i32, vp, i32, i32, i32, vp, vp, vp, vp]
    lib.beagle_draft_tree.restype = C.c_int
    lib.beagle_verify_tree_greedy.argtypes = [vp, i32, vp, vp, vp, i32, vp, vp, vp, vp]
    lib.beagle_verify_tree_greedy.restype = C.c_int
    lib.beagle_verify_sample.argtypes = [vp, i32, i32, vp, vp, vp, i32, C.c_float, vp, vp, vp, vp, vp]
    lib.beagle_verify_sample.restype = C.c_int
    lib.beagle_packed_weights_bytes.argtypes = [C.POINTER(BeagleConfig), i32, szp]
    lib.beagle_packed_weights_bytes.restype = C.c_int
    lib.beagle_pack_weights.argtypes = [vp, vp, C.c_size_t, vp]
    lib.beagle_pack_weights.restype = C.c_int
    lib.beagle_check_device.argtypes = [vp, vp]
    lib.beagle_check_device.restype = C.c_int
    lib.beagle_selftest_wait_timeout.argtypes = [vp, vp]
    lib.beagle_selftest_wait_timeout.restype = C.c_int
    lib.beagle_launch_count.restype = C.c_int64
    lib.beagle_launch_count.argtypes = [vp]
    for name in ("beagle_query_sizes", "beagle_create", "beagle_destroy", "beagle_prefill_kv", "beagle_draft_step",
                 "beagle_rollback", "beagle_reset_slot", "beagle_slot_lengths", "beagle_block_workspace_bytes",
                 "beagle_block_forward", "beagle_verify_greedy"):
        getattr(lib, name).restype = C.c_int
    if path is None:
        _lib = lib
    return lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    if not t.is_contiguous():
        raise ValueError("tensor must be contiguous")
    return t.data_ptr()


def _i32_array(values: Sequence[int]):
    arr = (C.c_int32 * max(1, len(values)))(*[int(v) for v in values])
    return arr


def _stream() -> int:
    return torch.cuda.current_stream().cuda_stream


def torch_dtype(dtype_code: int) -> torch.dtype:
    return torch.bfloat16 if dtype_code == BEAGLE_BF16 else torch.float32


LIVE_CONTEXTS: "weakref.WeakSet[Context]" = weakref.WeakSet()      # open contexts (the tests check each one's device status)


class Context:
    """Owns the device buffers (as torch tensors) that the C context borrows, and the opaque handle."""

    def __init__(self, cfg: BeagleConfig, weights: Dict[str, torch.Tensor]):
        self.lib = load_library()
        self.cfg = cfg
        dt = torch_dtype(cfg.dtype)
        self.weights = {}
        w = BeagleWeights()
        for n in WEIGHT_NAMES:
            t = weights[n]
            if t.dtype != dt or not t.is_cuda or not t.is_contiguous():
                raise ValueError(f"weight {n}: expected contiguous {dt} CUDA tensor")
            self.weights[n] = t
            setattr(w, n, t.data_ptr())
        for n, want in (("w_lm_fp8", torch.uint8), ("w_lm_scale", torch.float32)):      # optional FP8 copy of the LM head
            t = weights.get(n)
            if t is not None:
                if t.dtype != want or not t.is_cuda or not t.is_contiguous():
                    raise ValueError(f"weight {n}: expected contiguous {want} CUDA tensor")
                self.weights[n] = t
                setattr(w, n, t.data_ptr())
        kv, ws = C.c_size_t(), C.c_size_t()
        st = self.lib.beagle_query_sizes(C.byref(cfg), C.byref(kv), C.byref(ws))
        if st != 0:
            raise BeagleError(st, "beagle_query_sizes rejected the configuration")
        dev = next(iter(self.weights.values())).device
        self.kv_buf = torch.empty(kv.value, dtype=torch.uint8, device=dev)
        self.ws_buf = torch.empty(ws.value, dtype=torch.uint8, device=dev)
        self.block_ws: Optional[torch.Tensor] = None
        self.packed_buf: Optional[torch.Tensor] = None
        handle = C.c_void_p()
        st = self.lib.beagle_create(C.byref(cfg), C.byref(w), self.kv_buf.data_ptr(), kv.value, self.ws_buf.data_ptr(),
                                    ws.value, C.byref(handle))
        if st != 0:
            raise BeagleError(st, "beagle_create failed")
        self.handle = handle
        LIVE_CONTEXTS.add(self)

    def check(self, st: int) -> None:
        if st != 0:
            raise BeagleError(st, self.lib.beagle_last_error(self.handle).decode())

    def close(self) -> None:
        if getattr(self, "handle", None):
            self.lib.beagle_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    @property
    def launch_count(self) -> int:
        return int(self.lib.beagle_launch_count(self.handle))


# ---- entry points, named as in include/beagle.h -----------------------------------------------

def beagle_prefill_kv(ctx: Context, seq_slot: Sequence[int], new_len: Sequence[int], hidden: Optional[torch.Tensor]) -> None:
    ctx.check(ctx.lib.beagle_prefill_kv(ctx.handle, len(seq_slot), _i32_array(seq_slot), _i32_array(new_len),
                                        _ptr(hidden), _stream()))


def beagle_draft_step(ctx: Context, seq_slot: Sequence[int], tokens_in: Optional[torch.Tensor], concat: bool,
                      tokens_out: Optional[torch.Tensor], logits_out: Optional[torch.Tensor] = None,
                      hidden_out: Optional[torch.Tensor] = None) -> None:
    """tokens_out may be a dense [batch] tensor or one column of a [batch, gamma] draft matrix."""
    stride, out_ptr = 1, None
    if tokens_out is not None:
        if tokens_out.dim() != 1 or tokens_out.dtype != torch.int32:
            raise ValueError("tokens_out must be a 1-D int32 tensor (a column view is fine)")
        stride, out_ptr = int(tokens_out.stride(0)), tokens_out.data_ptr()
    ctx.check(ctx.lib.beagle_draft_step(ctx.handle, len(seq_slot), _i32_array(seq_slot), _ptr(tokens_in), int(bool(concat)),
                                        out_ptr, stride, _ptr(logits_out), _ptr(hidden_out), _stream()))


def beagle_rollback(ctx: Context, seq_slot: Sequence[int]) -> None:
    ctx.check(ctx.lib.beagle_rollback(ctx.handle, len(seq_slot), _i32_array(seq_slot)))


def beagle_reset_slot(ctx: Context, slot: int) -> None:
    ctx.check(ctx.lib.beagle_reset_slot(ctx.handle, int(slot)))


def beagle_slot_lengths(ctx: Context, slot: int) -> Tuple[int, int]:
    a, b = C.c_int32(), C.c_int32()
    ctx.check(ctx.lib.beagle_slot_lengths(ctx.handle, int(slot), C.byref(a), C.byref(b)))
    return a.value, b.value


def beagle_block_workspace_bytes(ctx: Context, batch: int, S: int) -> int:
    n = C.c_size_t()
    st = ctx.lib.beagle_block_workspace_bytes(C.byref(ctx.cfg), batch, S, C.byref(n))
    if st != 0:
        raise BeagleError(st, "beagle_block_workspace_bytes")
    return n.value


def beagle_block_forward(ctx: Context, tokens: torch.Tensor, hidden: torch.Tensor, block: int, offset: int,
                         sim_steps: int, logits_out: Optional[torch.Tensor], argmax_out: Optional[torch.Tensor],
                         hidden_out: Optional[torch.Tensor]) -> None:
    batch, S = tokens.shape
    need = beagle_block_workspace_bytes(ctx, batch, S)
    if ctx.block_ws is None or ctx.block_ws.numel() < need:
        ctx.block_ws = None
        ctx.block_ws = torch.empty(need, dtype=torch.uint8, device=tokens.device)
    ctx.check(ctx.lib.beagle_block_forward(ctx.handle, batch, S, _ptr(tokens), _ptr(hidden), block, offset, sim_steps,
                                           _ptr(logits_out), _ptr(argmax_out), _ptr(hidden_out),
                                           ctx.block_ws.data_ptr(), ctx.block_ws.numel(), _stream()))


def beagle_block_loss(ctx: Context, tokens: torch.Tensor, hidden: torch.Tensor, block: int, offset: int, sim_steps: int, stage: str,
                      target_logits: Optional[torch.Tensor], target_ids: Optional[torch.Tensor], loss_out: torch.Tensor,
                      ce_out: Optional[torch.Tensor]) -> None:
    """stage: "early" (Eq. 4) or "late" (Eq. 7); loss_out fp32 [1]; ce_out fp32 [batch, S] or None."""
    batch, S = tokens.shape
    need = beagle_block_workspace_bytes(ctx, batch, S)
    if ctx.block_ws is None or ctx.block_ws.numel() < need:
        ctx.block_ws = None
        ctx.block_ws = torch.empty(need, dtype=torch.uint8, device=tokens.device)
    code = BEAGLE_FP32
    if target_logits is not None:
        if target_logits.dtype == torch.bfloat16:
            code = BEAGLE_BF16
        elif target_logits.dtype != torch.float32:
            raise ValueError("target_logits must be float32 or bfloat16")
    ctx.check(ctx.lib.beagle_block_loss(ctx.handle, batch, S, _ptr(tokens), _ptr(hidden), block, offset, sim_steps,
                                        {"early": 0, "late": 1}[stage], _ptr(target_logits), code, _ptr(target_ids), _ptr(loss_out),
                                        _ptr(ce_out), ctx.block_ws.data_ptr(), ctx.block_ws.numel(), _stream()))


def beagle_quantize_rows_e4m3(x: torch.Tensor) -> Tuple[torch.Tensor, torch.Tensor]:
    """Row-wise FP8 E4M3 quantisation of a [rows, cols] fp32 / bf16 CUDA tensor: (uint8 codes [rows, cols], fp32 scales [rows])."""
    if x.dim() != 2 or not x.is_cuda or not x.is_contiguous() or x.dtype not in (torch.float32, torch.bfloat16):
        raise ValueError("need a contiguous 2-D float32 / bfloat16 CUDA tensor")
    rows, cols = x.shape
    q = torch.empty(rows, cols, dtype=torch.uint8, device=x.device)
    scale = torch.empty(rows, dtype=torch.float32, device=x.device)
    st = load_library().beagle_quantize_rows_e4m3(x.data_ptr(), BEAGLE_BF16 if x.dtype == torch.bfloat16 else BEAGLE_FP32, rows, cols,
                                                  q.data_ptr(), scale.data_ptr(), _stream())
    if st != 0:
        raise BeagleError(st, "beagle_quantize_rows_e4m3")
    return q, scale


def beagle_block_grad_workspace_bytes(ctx: Context, batch: int, S: int) -> int:
    n = C.c_size_t()
    st = ctx.lib.beagle_block_grad_workspace_bytes(C.byref(ctx.cfg), batch, S, C.byref(n))
    if st != 0:
        raise BeagleError(st, "beagle_block_grad_workspace_bytes")
    return n.value


def beagle_block_grad(ctx: Context, tokens: torch.Tensor, hidden: torch.Tensor, block: int, offset: int, sim_steps: int, stage: str,
                      target_logits: Optional[torch.Tensor], target_ids: Optional[torch.Tensor], vloss_coef: float,
                      grads: Dict[str, Optional[torch.Tensor]], loss_out: torch.Tensor) -> None:
    """grads: parameter name -> fp32 tensor shaped like the parameter (missing / None: not computed); loss_out fp32 [3]."""
    batch, S = tokens.shape
    need = beagle_block_grad_workspace_bytes(ctx, batch, S)
    if ctx.block_ws is None or ctx.block_ws.numel() < need:
        ctx.block_ws = None
        ctx.block_ws = torch.empty(need, dtype=torch.uint8, device=tokens.device)
    code = BEAGLE_FP32
    if target_logits is not None:
        if target_logits.dtype == torch.bfloat16:
            code = BEAGLE_BF16
        elif target_logits.dtype != torch.float32:
            raise ValueError("target_logits must be float32 or bfloat16")
    g = BeagleGrads()
    for name in WEIGHT_NAMES:
        t = grads.get(name)
        if t is not None and t.dtype != torch.float32:
            raise ValueError("gradient buffers must be float32")
        setattr(g, name, _ptr(t))
    ctx.check(ctx.lib.beagle_block_grad(ctx.handle, batch, S, _ptr(tokens), _ptr(hidden), block, offset, sim_steps,
                                        {"early": 0, "late": 1}[stage], _ptr(target_logits), code, _ptr(target_ids), float(vloss_coef),
                                        C.byref(g), _ptr(loss_out), ctx.block_ws.data_ptr(), ctx.block_ws.numel(), _stream()))


def beagle_verify_greedy(ctx: Context, draft_tokens: torch.Tensor, target_logits: Optional[torch.Tensor],
                         target_ids: Optional[torch.Tensor], accept_len: torch.Tensor, out_tokens: torch.Tensor) -> None:
    batch, gamma = draft_tokens.shape
    code = BEAGLE_FP32
    if target_logits is not None:
        if target_logits.dtype == torch.bfloat16:
            code = BEAGLE_BF16
        elif target_logits.dtype != torch.float32:
            raise ValueError("target_logits must be float32 or bfloat16")
    ctx.check(ctx.lib.beagle_verify_greedy(ctx.handle, batch, gamma, _ptr(draft_tokens), _ptr(target_logits), code,
                                           _ptr(target_ids), _ptr(accept_len), _ptr(out_tokens), _stream()))


def beagle_verify_sample(ctx: Context, draft_tokens: torch.Tensor, draft_logits: torch.Tensor, target_logits: torch.Tensor,
                         u_accept: torch.Tensor, u_resample: torch.Tensor, accept_len: torch.Tensor, out_tokens: torch.Tensor,
                         temperature: float = 1.0) -> None:
    """draft_logits: fp32 [gamma, batch, V]; target_logits: [batch, gamma+1, V] fp32 or bf16; uniforms fp32."""
    batch, gamma = draft_tokens.shape
    if draft_logits.dtype != torch.float32 or u_accept.dtype != torch.float32 or u_resample.dtype != torch.float32:
        raise ValueError("draft_logits and the uniforms must be float32")
    if target_logits.dtype == torch.bfloat16:
        code = BEAGLE_BF16
    elif target_logits.dtype == torch.float32:
        code = BEAGLE_FP32
    else:
        raise ValueError("target_logits must be float32 or bfloat16")
    ctx.check(ctx.lib.beagle_verify_sample(ctx.handle, batch, gamma, _ptr(draft_tokens), _ptr(draft_logits), _ptr(target_logits), code,
                                           float(temperature), _ptr(u_accept), _ptr(u_resample), _ptr(accept_len), _ptr(out_tokens),
                                           _stream()))


def beagle_draft_tree(ctx: Context, slot: int, root_token: torch.Tensor, depth: int, topk: int, n_candidates: int,
                      tree_tokens: torch.Tensor, tree_parents: torch.Tensor, tree_scores: torch.Tensor) -> None:
    ctx.check(ctx.lib.beagle_draft_tree(ctx.handle, int(slot), _ptr(root_token), depth, topk, n_candidates, _ptr(tree_tokens),
                                        _ptr(tree_parents), _ptr(tree_scores), _stream()))


def beagle_verify_tree_greedy(ctx: Context, tree_tokens: torch.Tensor, tree_parents: torch.Tensor, target_ids: torch.Tensor,
                              accept_len: torch.Tensor, out_tokens: torch.Tensor, path: Optional[torch.Tensor] = None) -> None:
    ctx.check(ctx.lib.beagle_verify_tree_greedy(ctx.handle, tree_tokens.numel(), _ptr(tree_tokens), _ptr(tree_parents), _ptr(target_ids),
                                                out_tokens.numel(), _ptr(accept_len), _ptr(out_tokens), _ptr(path), _stream()))


def beagle_verify_greedy_static(draft_tokens: torch.Tensor, target_logits: torch.Tensor, accept_len: torch.Tensor,
                                out_tokens: torch.Tensor) -> None:
    """Greedy acceptance for callers that may not allocate: no context, no workspace -- the
    library's built-in device array serves as scratch (see include/beagle.h for the limits)."""
    batch, gamma = draft_tokens.shape
    if target_logits.dtype == torch.bfloat16:
        code = BEAGLE_BF16
    elif target_logits.dtype == torch.float32:
        code = BEAGLE_FP32
    else:
        raise ValueError("target_logits must be float32 or bfloat16")
    err = C.create_string_buffer(256)
    st = load_library().beagle_verify_greedy_static(batch, gamma, target_logits.shape[-1], _ptr(draft_tokens),
                                                    _ptr(target_logits), code, _ptr(accept_len), _ptr(out_tokens),
                                                    _stream(), err, len(err))
    if st != 0:
        raise BeagleError(st, err.value.decode())


def beagle_workspace_buffer(ctx: Context, name: str, rows: int) -> torch.Tensor:
    """View of an intermediate vector of the most recent draft step ([rows, width], storage type)."""
    off, width = C.c_size_t(), C.c_int32()
    st = ctx.lib.beagle_workspace_buffer(C.byref(ctx.cfg), BUFFER_IDS[name], C.byref(off), C.byref(width))
    if st != 0:
        raise BeagleError(st, f"beagle_workspace_buffer({name})")
    dt = torch_dtype(ctx.cfg.dtype)
    n = rows * width.value * dt.itemsize
    return ctx.ws_buf[off.value:off.value + n].view(dt).view(rows, width.value)


def beagle_block_workspace_buffer(ctx: Context, name: str, batch: int, S: int) -> torch.Tensor:
    """View of an intermediate matrix of the most recent block forward ([batch*S, width], storage type)."""
    off, width = C.c_size_t(), C.c_int32()
    st = ctx.lib.beagle_block_workspace_buffer(C.byref(ctx.cfg), batch, S, BUFFER_IDS[name], C.byref(off), C.byref(width))
    if st != 0:
        raise BeagleError(st, f"beagle_block_workspace_buffer({name})")
    dt = torch_dtype(ctx.cfg.dtype)
    rows = batch * S
    n = rows * width.value * dt.itemsize
    return ctx.block_ws[off.value:off.value + n].view(dt).view(rows, width.value)


def kv_cache_views(ctx: Context) -> Tuple[torch.Tensor, torch.Tensor]:
    """The caller-owned cache as ([slot, Hkv, max_ctx + max_draft, dh]) key and value tensors."""
    c = ctx.cfg
    dt = torch_dtype(c.dtype)
    cap = c.max_ctx + c.max_draft
    half = ctx.kv_buf.numel() // 2
    n = c.max_slots * c.n_kv_heads * cap * c.head_dim * dt.itemsize
    k = ctx.kv_buf[:n].view(dt).view(c.max_slots, c.n_kv_heads, cap, c.head_dim)
    v = ctx.kv_buf[half:half + n].view(dt).view(c.max_slots, c.n_kv_heads, cap, c.head_dim)
    return k, v


def beagle_packed_weights_bytes(cfg: BeagleConfig, with_fp8_lm_head: bool) -> int:
    n = C.c_size_t()
    st = load_library().beagle_packed_weights_bytes(C.byref(cfg), int(bool(with_fp8_lm_head)), C.byref(n))
    if st != 0:
        raise BeagleError(st, "beagle_packed_weights_bytes rejected the configuration")
    return int(n.value)


def beagle_pack_weights(ctx: Context, enable: bool = True) -> None:
    """Makes (or, enable=False, drops) the tile-major copies of the projection weights that draft steps of 9..64 rows stream.
    Call again after changing the weights in place."""
    if not enable:
        ctx.check(ctx.lib.beagle_pack_weights(ctx.handle, None, 0, _stream()))
        ctx.packed_buf = None
        return
    n = beagle_packed_weights_bytes(ctx.cfg, "w_lm_fp8" in ctx.weights)
    if n == 0:
        return
    if ctx.packed_buf is None or ctx.packed_buf.numel() < n:
        ctx.packed_buf = torch.empty(n, dtype=torch.uint8, device=ctx.kv_buf.device)
    ctx.check(ctx.lib.beagle_pack_weights(ctx.handle, ctx.packed_buf.data_ptr(), n, _stream()))


def beagle_selftest_wait_timeout(ctx: Context) -> None:
    """Launches the one-CTA kernel whose bounded wait runs out (test support for the device error path)."""
    ctx.check(ctx.lib.beagle_selftest_wait_timeout(ctx.handle, _stream()))


def beagle_check_device(ctx: Context) -> None:
    """Synchronises the current stream and raises if a kernel abandoned a bounded wait."""
    ctx.check(ctx.lib.beagle_check_device(ctx.handle, _stream()))


def beagle_profile_enable(ctx: Context, on: bool) -> None:
    ctx.check(ctx.lib.beagle_profile_enable(ctx.handle, int(bool(on))))


def beagle_profile_read(ctx: Context) -> Dict[str, Tuple[float, int]]:
    """{stage name: (accumulated ms, bracketed instances)} since the last read; synchronises."""
    n = ctx.lib.beagle_profile_stage_count()
    ms, cnt = (C.c_float * n)(), (C.c_int32 * n)()
    ctx.check(ctx.lib.beagle_profile_read(ctx.handle, ms, cnt))
    return {ctx.lib.beagle_profile_stage_name(i).decode(): (float(ms[i]), int(cnt[i])) for i in range(n) if cnt[i]}


# ---- convenience wrapper -----------------------------------------------------------------------

class BeagleHead:
    """A draft head on one GPU: allocates outputs and forwards to the entry points above."""

    def __init__(self, *, hidden: int, n_q_heads: int, n_kv_heads: int, head_dim: int, mlp_dim: int, vocab: int,
                 dtype: str, weights: Dict[str, torch.Tensor], max_slots: int, max_ctx: int, max_draft: int,
                 rms_eps: float = 1e-5, norm_q: bool = True, norm_mlp: bool = True, rope_theta: float = 0.0,
                 pack_weights: bool = True):
        """pack_weights: bf16 heads keep tile-major copies of the projection weights for draft steps of 9..64 rows
        (``beagle_pack_weights``; about the size of the weights without the embedding); after changing a weight tensor in
        place call ``beagle_pack_weights(head.ctx)`` again."""
        code = {"fp32": BEAGLE_FP32, "bf16": BEAGLE_BF16}[dtype]
        self.cfg = BeagleConfig(hidden, n_q_heads, n_kv_heads, head_dim, mlp_dim, vocab, code, rms_eps, int(norm_q),
                                int(norm_mlp), max_slots, max_ctx, max_draft, float(rope_theta))
        self.ctx = Context(self.cfg, weights)
        if pack_weights:
            beagle_pack_weights(self.ctx)
        self.weight_shapes = {n: tuple(weights[n].shape) for n in WEIGHT_NAMES}
        self.device = self.ctx.kv_buf.device
        self.dtype = torch_dtype(code)

    @classmethod
    def from_workload(cls, w, weights_np, device="cuda", max_slots=None, max_ctx=None, max_draft=None, rope_theta=0.0,
                      fp8_lm_head=False, pack_weights=True) -> "BeagleHead":
        """Uploads numpy float32 weights (already rounded to the storage type) and builds the head.
        fp8_lm_head: also make the FP8 copy of the LM head (used by draft steps of more than 8 rows)."""
        dt = torch.bfloat16 if w.dtype == "bf16" else torch.float32
        weights = {k: torch.from_numpy(v).to(device=device, dtype=dt).contiguous() for k, v in weights_np.items()}
        if fp8_lm_head:
            weights["w_lm_fp8"], weights["w_lm_scale"] = beagle_quantize_rows_e4m3(weights["w_lm"])
        return cls(hidden=w.hidden, n_q_heads=w.n_q_heads, n_kv_heads=w.n_kv_heads, head_dim=w.head_dim,
                   mlp_dim=w.mlp_dim, vocab=w.vocab, dtype=w.dtype, weights=weights,
                   max_slots=max_slots or w.batch, max_ctx=max_ctx or (w.ctx_max + 64),
                   max_draft=max_draft or max(w.gamma, 1), rms_eps=w.rms_eps, rope_theta=rope_theta, pack_weights=pack_weights)

    def prefill_kv(self, seq_slot, new_len, hidden):
        beagle_prefill_kv(self.ctx, seq_slot, new_len, hidden)

    def rollback(self, seq_slot):
        beagle_rollback(self.ctx, seq_slot)

    def draft_step(self, seq_slot, tokens_in=None, concat=True, want_logits=False, want_hidden=False):
        B = len(seq_slot)
        tokens_out = torch.empty(B, dtype=torch.int32, device=self.device)
        logits = torch.empty(B, self.cfg.vocab, dtype=torch.float32, device=self.device) if want_logits else None
        hidden = torch.empty(B, self.cfg.hidden, dtype=self.dtype, device=self.device) if want_hidden else None
        beagle_draft_step(self.ctx, seq_slot, tokens_in, concat, tokens_out, logits, hidden)
        return tokens_out, logits, hidden

    def block_forward(self, tokens, hidden, block, offset=0, sim_steps=1, want_logits=True, want_hidden=True):
        B, S = tokens.shape
        logits = torch.empty(B, S, self.cfg.vocab, dtype=torch.float32, device=self.device) if want_logits else None
        argmax = torch.empty(B, S, dtype=torch.int32, device=self.device)
        hid = torch.empty(B, S, self.cfg.hidden, dtype=self.dtype, device=self.device) if want_hidden else None
        beagle_block_forward(self.ctx, tokens, hidden, block, offset, sim_steps, logits, argmax, hid)
        return logits, argmax, hid

    def block_loss(self, tokens, hidden, block, offset, stage, sim_steps=1, target_logits=None, target_ids=None):
        B, S = tokens.shape
        loss = torch.empty(1, dtype=torch.float32, device=self.device)
        ce = torch.empty(B, S, dtype=torch.float32, device=self.device)
        beagle_block_loss(self.ctx, tokens, hidden, block, offset, sim_steps, stage, target_logits, target_ids, loss, ce)
        return loss, ce

    def block_grad(self, tokens, hidden, block, offset, stage, sim_steps=1, target_logits=None, target_ids=None, vloss_coef=0.0,
                   params=WEIGHT_NAMES):
        """One training step: returns (losses fp32 [3] = L, vloss, total; dict of fp32 gradients for `params`)."""
        grads = {n: torch.empty(tuple(getattr(self, "weight_shapes")[n]), dtype=torch.float32, device=self.device) for n in params}
        losses = torch.empty(3, dtype=torch.float32, device=self.device)
        beagle_block_grad(self.ctx, tokens, hidden, block, offset, sim_steps, stage, target_logits, target_ids, vloss_coef, grads, losses)
        return losses, grads

    def verify_greedy(self, draft_tokens, target_logits=None, target_ids=None):
        B, gamma = draft_tokens.shape
        accept = torch.empty(B, dtype=torch.int32, device=self.device)
        out = torch.empty(B, gamma + 1, dtype=torch.int32, device=self.device)
        beagle_verify_greedy(self.ctx, draft_tokens, target_logits, target_ids, accept, out)
        return accept, out

    def verify_sample(self, draft_tokens, draft_logits, target_logits, u_accept, u_resample, temperature=1.0):
        B, gamma = draft_tokens.shape
        accept = torch.empty(B, dtype=torch.int32, device=self.device)
        out = torch.empty(B, gamma + 1, dtype=torch.int32, device=self.device)
        beagle_verify_sample(self.ctx, draft_tokens, draft_logits, target_logits, u_accept, u_resample, accept, out, temperature)
        return accept, out

    def draft_tree(self, slot, root_token, depth, topk, n_candidates):
        tok = torch.empty(n_candidates, dtype=torch.int32, device=self.device)
        par = torch.empty(n_candidates, dtype=torch.int32, device=self.device)
        sc = torch.empty(n_candidates, dtype=torch.float32, device=self.device)
        beagle_draft_tree(self.ctx, slot, root_token, depth, topk, n_candidates, tok, par, sc)
        return tok, par, sc

    def verify_tree_greedy(self, tree_tokens, tree_parents, target_ids, out_cap):
        acc = torch.empty(1, dtype=torch.int32, device=self.device)
        out = torch.empty(out_cap, dtype=torch.int32, device=self.device)
        path = torch.empty(out_cap, dtype=torch.int32, device=self.device)
        beagle_verify_tree_greedy(self.ctx, tree_tokens, tree_parents, target_ids, acc, out, path)
        return acc, out, path

    def slot_lengths(self, slot):
        return beagle_slot_lengths(self.ctx, slot)

    @property
    def launch_count(self) -> int:
        return self.ctx.launch_count
