"""Thin Python binding of the Lynx C-ABI CUDA library (sm_100a).

Argument marshalling only: every step of the path runs in the library's kernels.  Torch is
used for device memory and streams.  There is no CPU fallback: if ``liblynx.so`` is missing
or a call returns an error status, an exception is raised.

Names mirror ``include/lynx.h``: split_quantize, recombine, anchor_attention,
merge_verify_attention, workspace_bytes.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
_LIB_PATH = os.path.join(_HERE, "liblynx.so")
_lib = None

D = 128


class LynxError(RuntimeError):
    pass


class _Plane(ctypes.Structure):
    _fields_ = [("anchor", ctypes.c_void_p), ("residual", ctypes.c_void_p), ("meta", ctypes.c_void_p)]


class _Shape(ctypes.Structure):
    _fields_ = [("num_q_heads", ctypes.c_int32), ("num_kv_heads", ctypes.c_int32),
                ("head_dim", ctypes.c_int32), ("block_tokens", ctypes.c_int32),
                ("num_blocks", ctypes.c_int32), ("max_blocks_per_seq", ctypes.c_int32)]


EXPORTS = ["lynx_split_quantize", "lynx_recombine", "lynx_workspace_bytes", "lynx_workspace_init",
           "lynx_anchor_attention", "lynx_merge_verify_attention", "lynx_anchor_attention_static",
           "lynx_bf16_workspace_bytes", "lynx_bf16_attention", "lynx_hier_quantize", "lynx_hier_dequantize",
           "lynx_token_verify", "lynx_workspace_lse", "lynx_bf16_workspace_lse", "lynx_lse_merge", "lynx_verify_decision", "lynx_split_quantize_bits", "lynx_recombine_bits",
           "lynx_check",
           "lynx_status_string", "lynx_version"]


def lib_path() -> str:
    return _LIB_PATH


def load():
    """Load liblynx.so (built in-tree by paper_2607_01831_b200/build.py). Fails loudly."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(_LIB_PATH):
        raise LynxError(f"{_LIB_PATH} is missing: build it with `python -m paper_2607_01831_b200.build` "
                        "(there is no CPU fallback)")
    lib = ctypes.CDLL(_LIB_PATH)
    vp, i32, i64, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float
    lib.lynx_split_quantize.argtypes = [vp, i64, vp, i32, i32, vp, vp, vp, vp]
    lib.lynx_split_quantize.restype = ctypes.c_int
    lib.lynx_recombine.argtypes = [vp, vp, vp, i64, vp, vp, vp]
    lib.lynx_recombine.restype = ctypes.c_int
    lib.lynx_workspace_bytes.argtypes = [ctypes.POINTER(_Shape), i32, i32]
    lib.lynx_workspace_bytes.restype = ctypes.c_size_t
    lib.lynx_workspace_init.argtypes = [vp, ctypes.c_size_t, vp]
    lib.lynx_workspace_init.restype = ctypes.c_int
    lib.lynx_anchor_attention.argtypes = [ctypes.POINTER(_Shape), vp, i32, i32, i32, _Plane, _Plane,
                                          vp, vp, f32, vp, vp, ctypes.c_size_t, vp]
    lib.lynx_anchor_attention.restype = ctypes.c_int
    lib.lynx_merge_verify_attention.argtypes = [ctypes.POINTER(_Shape), vp, i32, i32, i32, _Plane,
                                                _Plane, vp, vp, f32, vp, f32, f32, vp, vp, vp, vp,
                                                ctypes.c_size_t, vp]
    lib.lynx_merge_verify_attention.restype = ctypes.c_int
    lib.lynx_anchor_attention_static.argtypes = [ctypes.POINTER(_Shape), vp, i32, i32, i32, _Plane,
                                                 _Plane, vp, vp, f32, vp, vp]
    lib.lynx_anchor_attention_static.restype = ctypes.c_int
    lib.lynx_bf16_workspace_bytes.argtypes = [ctypes.POINTER(_Shape), i32, i32]
    lib.lynx_bf16_workspace_bytes.restype = ctypes.c_size_t
    lib.lynx_bf16_attention.argtypes = [ctypes.POINTER(_Shape), vp, i32, i32, i32, vp, vp, vp, vp, f32, vp, vp,
                                        ctypes.c_size_t, vp]
    lib.lynx_bf16_attention.restype = ctypes.c_int
    lib.lynx_hier_quantize.argtypes = [vp, i64, vp, vp, vp, vp, vp, vp, vp]
    lib.lynx_hier_quantize.restype = ctypes.c_int
    lib.lynx_hier_dequantize.argtypes = [vp, vp, i64, vp, vp, vp, vp, vp, vp]
    lib.lynx_hier_dequantize.restype = ctypes.c_int
    lib.lynx_token_verify.argtypes = [vp, vp, vp, vp, vp, ctypes.c_int32, ctypes.c_int32, ctypes.c_int32, vp, vp, vp]
    lib.lynx_token_verify.restype = ctypes.c_int
    lib.lynx_workspace_lse.argtypes = [ctypes.POINTER(_Shape), i32, i32, vp]
    lib.lynx_workspace_lse.restype = ctypes.c_void_p
    lib.lynx_bf16_workspace_lse.argtypes = [ctypes.POINTER(_Shape), i32, i32, vp]
    lib.lynx_bf16_workspace_lse.restype = ctypes.c_void_p
    lib.lynx_lse_merge.argtypes = [vp, vp, vp, vp, i64, vp, vp, vp]
    lib.lynx_lse_merge.restype = ctypes.c_int
    lib.lynx_verify_decision.argtypes = [vp, vp, i32, i32, i32, f32, f32, vp, vp, vp]
    lib.lynx_verify_decision.restype = ctypes.c_int
    lib.lynx_split_quantize_bits.argtypes = [vp, i64, i32, vp, vp, vp, vp]
    lib.lynx_split_quantize_bits.restype = ctypes.c_int
    lib.lynx_recombine_bits.argtypes = [vp, vp, vp, i64, i32, vp, vp, vp]
    lib.lynx_recombine_bits.restype = ctypes.c_int
    lib.lynx_check.argtypes = [vp, vp]
    lib.lynx_check.restype = ctypes.c_int
    lib.lynx_status_string.argtypes = [ctypes.c_int]
    lib.lynx_status_string.restype = ctypes.c_char_p
    lib.lynx_version.restype = ctypes.c_int
    _lib = lib
    return lib


def _ok(status: int, what: str):
    if status != 0:
        msg = load().lynx_status_string(status).decode()
        raise LynxError(f"{what}: status {status} ({msg})")


def _ptr(t: torch.Tensor | None):
    if t is None:
        return None
    if not t.is_cuda:
        raise LynxError("device tensors required")
    if not t.is_contiguous():
        raise LynxError("contiguous tensors required")
    return t.data_ptr()


def _stream():
    return torch.cuda.current_stream().cuda_stream


@dataclass
class Planes:
    """Quantised K or V: anchor / residual u8 [..., 64], meta f32 [..., 2] (device tensors)."""
    anchor: torch.Tensor
    residual: torch.Tensor | None
    meta: torch.Tensor

    def _c(self) -> _Plane:
        return _Plane(_ptr(self.anchor), _ptr(self.residual), _ptr(self.meta))


def alloc_planes(lead_shape, device) -> Planes:
    lead = tuple(lead_shape)
    return Planes(torch.empty(lead + (64,), dtype=torch.uint8, device=device),
                  torch.empty(lead + (64,), dtype=torch.uint8, device=device),
                  torch.empty(lead + (2,), dtype=torch.float32, device=device))


def split_quantize(src: torch.Tensor, out: Planes | None = None, block_ids: torch.Tensor | None = None,
                   rows_per_block: int = 0) -> Planes:
    """lynx_split_quantize: src BF16 [..., 128] -> Planes with the same leading shape."""
    if src.dtype != torch.bfloat16 or src.shape[-1] != D:
        raise LynxError("src must be BF16 [..., 128]")
    if out is None:
        out = alloc_planes(src.shape[:-1], src.device)
    n_rows = src.numel() // D
    nb = 0 if block_ids is None else block_ids.numel()
    _ok(load().lynx_split_quantize(_ptr(src), n_rows, _ptr(block_ids), nb, rows_per_block,
                                   _ptr(out.anchor), _ptr(out.residual), _ptr(out.meta), _stream()),
        "lynx_split_quantize")
    return out


def recombine(planes: Planes, want_codes: bool = True, want_bf16: bool = False):
    """lynx_recombine: returns (codes u8 [...,128] or None, dequantised BF16 [...,128] or None)."""
    lead = tuple(planes.anchor.shape[:-1])
    dev = planes.anchor.device
    codes = torch.empty(lead + (D,), dtype=torch.uint8, device=dev) if want_codes else None
    deq = torch.empty(lead + (D,), dtype=torch.bfloat16, device=dev) if want_bf16 else None
    n_rows = planes.anchor.numel() // 64
    _ok(load().lynx_recombine(_ptr(planes.anchor), _ptr(planes.residual), _ptr(planes.meta), n_rows,
                              _ptr(codes), _ptr(deq), _stream()), "lynx_recombine")
    return codes, deq


@dataclass
class Geometry:
    num_q_heads: int
    num_kv_heads: int
    block_tokens: int
    num_blocks: int
    max_blocks_per_seq: int
    head_dim: int = D

    def _c(self) -> _Shape:
        return _Shape(self.num_q_heads, self.num_kv_heads, self.head_dim, self.block_tokens,
                      self.num_blocks, self.max_blocks_per_seq)


def workspace_bytes(geo: Geometry, batch: int, n_q: int) -> int:
    return int(load().lynx_workspace_bytes(ctypes.byref(geo._c()), batch, n_q))


def make_workspace(geo: Geometry, batch: int, n_q: int, device) -> torch.Tensor:
    """Allocate and zero a workspace large enough for (batch, n_q) attention calls."""
    n = workspace_bytes(geo, batch, n_q)
    if n == 0:
        raise LynxError("unsupported attention shape")
    ws = torch.empty(n, dtype=torch.uint8, device=device)
    _ok(load().lynx_workspace_init(_ptr(ws), n, _stream()), "lynx_workspace_init")
    return ws


def check(workspace: torch.Tensor):
    """lynx_check: synchronises and raises if a kernel recorded a bad block id or a timeout."""
    _ok(load().lynx_check(_ptr(workspace), _stream()), "lynx_check")


def anchor_attention(geo: Geometry, q: torch.Tensor, K: Planes, V: Planes, block_table: torch.Tensor,
                     seq_lens: torch.Tensor, workspace: torch.Tensor, causal: bool = False,
                     softmax_scale: float = 0.0, out: torch.Tensor | None = None) -> torch.Tensor:
    """lynx_anchor_attention: q BF16 [B][n_q][Hq][128] -> float32 [B][n_q][Hq][128]."""
    B, n_q, Hq, d = q.shape
    if q.dtype != torch.bfloat16 or d != D or Hq != geo.num_q_heads:
        raise LynxError("q must be BF16 [B][n_q][Hq][128]")
    if out is None:
        out = torch.empty(B, n_q, Hq, D, dtype=torch.float32, device=q.device)
    _ok(load().lynx_anchor_attention(ctypes.byref(geo._c()), _ptr(q), B, n_q, int(causal), K._c(),
                                     V._c(), _ptr(block_table), _ptr(seq_lens), softmax_scale,
                                     _ptr(out), _ptr(workspace), workspace.numel(), _stream()),
        "lynx_anchor_attention")
    return out


def anchor_attention_static(geo: Geometry, q: torch.Tensor, K: Planes, V: Planes,
                            block_table: torch.Tensor, seq_lens: torch.Tensor, causal: bool = False,
                            softmax_scale: float = 0.0, out: torch.Tensor | None = None) -> torch.Tensor:
    """lynx_anchor_attention_static: anchor attention whose scratch memory is a fixed 8 MiB array
    inside the library, for callers that may not allocate a workspace.  Only `out` is allocated
    here when the caller does not pass it; the library call allocates nothing.  Calls share the
    array: keep them ordered on one stream.  Raises LynxError if the problem needs more scratch."""
    B, n_q, Hq, d = q.shape
    if q.dtype != torch.bfloat16 or d != D or Hq != geo.num_q_heads:
        raise LynxError("q must be BF16 [B][n_q][Hq][128]")
    if out is None:
        out = torch.empty(B, n_q, Hq, D, dtype=torch.float32, device=q.device)
    _ok(load().lynx_anchor_attention_static(ctypes.byref(geo._c()), _ptr(q), B, n_q, int(causal),
                                            K._c(), V._c(), _ptr(block_table), _ptr(seq_lens),
                                            softmax_scale, _ptr(out), _stream()),
        "lynx_anchor_attention_static")
    return out


def merge_verify_attention(geo: Geometry, q: torch.Tensor, K: Planes, V: Planes,
                           block_table: torch.Tensor, seq_lens: torch.Tensor, workspace: torch.Tensor,
                           draft_out: torch.Tensor | None = None, atol: float = 0.0, rtol: float = 0.0,
                           causal: bool = True, softmax_scale: float = 0.0,
                           out_full: torch.Tensor | None = None, first_reject: torch.Tensor | None = None,
                           dev: torch.Tensor | None = None):
    """lynx_merge_verify_attention -> (out_full f32 [B][k][Hq][128], first_reject i32 [B], dev f32 [B][k]).
    first_reject / dev are None when no draft is given."""
    B, k, Hq, d = q.shape
    if q.dtype != torch.bfloat16 or d != D or Hq != geo.num_q_heads:
        raise LynxError("q must be BF16 [B][k][Hq][128]")
    if out_full is None:
        out_full = torch.empty(B, k, Hq, D, dtype=torch.float32, device=q.device)
    if draft_out is not None:
        if draft_out.dtype != torch.float32 or tuple(draft_out.shape) != (B, k, Hq, D):
            raise LynxError("draft_out must be float32 [B][k][Hq][128]")
        if first_reject is None:
            first_reject = torch.empty(B, dtype=torch.int32, device=q.device)
        if dev is None:
            dev = torch.empty(B, k, dtype=torch.float32, device=q.device)
    _ok(load().lynx_merge_verify_attention(ctypes.byref(geo._c()), _ptr(q), B, k, int(causal), K._c(),
                                           V._c(), _ptr(block_table), _ptr(seq_lens), softmax_scale,
                                           _ptr(draft_out), atol, rtol, _ptr(out_full),
                                           _ptr(first_reject), _ptr(dev), _ptr(workspace),
                                           workspace.numel(), _stream()),
        "lynx_merge_verify_attention")
    return out_full, first_reject, dev


def bf16_attention(geo: Geometry, q: torch.Tensor, k_pages: torch.Tensor, v_pages: torch.Tensor,
                   block_table: torch.Tensor, seq_lens: torch.Tensor, workspace: torch.Tensor | None = None,
                   causal: bool = False, softmax_scale: float = 0.0, out: torch.Tensor | None = None) -> torch.Tensor:
    """lynx_bf16_attention: decode attention over dequantised BF16 pages [num_blocks][Hkv][bt][128]
    (what recombine(want_bf16=True) writes).  q BF16 [B][n_q][Hq][128] -> float32 [B][n_q][Hq][128]."""
    B, n_q, Hq, d = q.shape
    if q.dtype != torch.bfloat16 or d != D or Hq != geo.num_q_heads:
        raise LynxError("q must be BF16 [B][n_q][Hq][128]")
    if k_pages.dtype != torch.bfloat16 or v_pages.dtype != torch.bfloat16:
        raise LynxError("pages must be BF16")
    if out is None:
        out = torch.empty(B, n_q, Hq, D, dtype=torch.float32, device=q.device)
    if workspace is None:
        n = int(load().lynx_bf16_workspace_bytes(ctypes.byref(geo._c()), B, n_q))
        if n == 0:
            raise LynxError("unsupported attention shape")
        workspace = torch.empty(n, dtype=torch.uint8, device=q.device)
    _ok(load().lynx_bf16_attention(ctypes.byref(geo._c()), _ptr(q), B, n_q, int(causal), _ptr(k_pages),
                                   _ptr(v_pages), _ptr(block_table), _ptr(seq_lens), softmax_scale, _ptr(out),
                                   _ptr(workspace), workspace.numel(), _stream()), "lynx_bf16_attention")
    return out


def _lse_view(addr, workspace: torch.Tensor, B: int, n_q: int, Hq: int, what: str) -> torch.Tensor:
    if not addr:
        raise LynxError(f"{what}: unsupported shape")
    off = int(addr) - workspace.data_ptr()
    n = B * n_q * Hq * 4
    if workspace.dtype != torch.uint8 or off < 0 or off + n > workspace.numel():
        raise LynxError(f"{what}: the workspace is smaller than the call's")
    return workspace[off:off + n].view(torch.float32).view(B, n_q, Hq)


def workspace_lse(geo: Geometry, B: int, n_q: int, workspace: torch.Tensor) -> torch.Tensor:
    """lynx_workspace_lse: float32 [B][n_q][Hq] view, inside `workspace`, of the natural-log log-sum-exps the last
    anchor_attention / merge_verify_attention call with this (B, n_q) left there."""
    return _lse_view(load().lynx_workspace_lse(ctypes.byref(geo._c()), B, n_q, _ptr(workspace)), workspace, B, n_q,
                     geo.num_q_heads, "lynx_workspace_lse")


def bf16_workspace_lse(geo: Geometry, B: int, n_q: int, workspace: torch.Tensor) -> torch.Tensor:
    """lynx_bf16_workspace_lse: the same for the workspace of a bf16_attention call."""
    return _lse_view(load().lynx_bf16_workspace_lse(ctypes.byref(geo._c()), B, n_q, _ptr(workspace)), workspace, B,
                     n_q, geo.num_q_heads, "lynx_bf16_workspace_lse")


def lse_merge(out_a: torch.Tensor, lse_a: torch.Tensor, out_b: torch.Tensor, lse_b: torch.Tensor,
              out: torch.Tensor | None = None, want_lse: bool = False):
    """lynx_lse_merge: two attention results float32 [...][128] over disjoint key sets, with their log-sum-exps
    float32 [...], joined into the attention over the union.  Returns out, or (out, lse) with want_lse."""
    if out_a.dtype != torch.float32 or out_b.dtype != torch.float32 or out_a.shape != out_b.shape or out_a.shape[-1] != D:
        raise LynxError("out_a, out_b must be float32 [...][128] of one shape")
    rows = out_a.numel() // D
    if lse_a.dtype != torch.float32 or lse_b.dtype != torch.float32 or lse_a.numel() != rows or lse_b.numel() != rows:
        raise LynxError("lse_a, lse_b must be float32 with one value per row")
    if out is None:
        out = torch.empty_like(out_a)
    lse = torch.empty(out_a.shape[:-1], dtype=torch.float32, device=out_a.device) if want_lse else None
    _ok(load().lynx_lse_merge(_ptr(out_a), _ptr(lse_a), _ptr(out_b), _ptr(lse_b), rows, _ptr(out), _ptr(lse), _stream()),
        "lynx_lse_merge")
    return (out, lse) if want_lse else out


def split_quantize_bits(src: torch.Tensor, anchor_bits: int):
    """lynx_split_quantize_bits: src BF16 [...][128] -> (anchor u8 [...][16 A], residual u8 [...][16 (8 - A)],
    meta f32 [...][2]) for the split with A = anchor_bits top bits in the Anchor."""
    if src.dtype != torch.bfloat16 or src.shape[-1] != D:
        raise LynxError("src must be BF16 [...][128]")
    lead, rows = tuple(src.shape[:-1]), src.numel() // D
    anchor = torch.empty(lead + (16 * anchor_bits,), dtype=torch.uint8, device=src.device)
    residual = torch.empty(lead + (16 * (8 - anchor_bits),), dtype=torch.uint8, device=src.device)
    meta = torch.empty(lead + (2,), dtype=torch.float32, device=src.device)
    _ok(load().lynx_split_quantize_bits(_ptr(src), rows, anchor_bits, _ptr(anchor), _ptr(residual), _ptr(meta), _stream()),
        "lynx_split_quantize_bits")
    return anchor, residual, meta


def recombine_bits(anchor: torch.Tensor, residual: torch.Tensor | None, meta: torch.Tensor, anchor_bits: int,
                   want_codes: bool = True, want_bf16: bool = True):
    """lynx_recombine_bits -> (codes u8 [...][128] or None, dequantised BF16 [...][128] or None); residual None:
    the Anchor alone (bucket mid-points)."""
    lead, rows = tuple(anchor.shape[:-1]), anchor.numel() // (16 * anchor_bits)
    codes = torch.empty(lead + (D,), dtype=torch.uint8, device=anchor.device) if want_codes else None
    deq = torch.empty(lead + (D,), dtype=torch.bfloat16, device=anchor.device) if want_bf16 else None
    _ok(load().lynx_recombine_bits(_ptr(anchor), _ptr(residual), _ptr(meta), rows, anchor_bits, _ptr(codes), _ptr(deq),
                                   _stream()), "lynx_recombine_bits")
    return codes, deq


def verify_decision(out_full: torch.Tensor, draft_out: torch.Tensor, atol: float, rtol: float):
    """lynx_verify_decision: out_full, draft_out float32 [B][k][Hq][128] -> (first_reject i32 [B], dev f32 [B][k])."""
    if out_full.dtype != torch.float32 or draft_out.dtype != torch.float32 or out_full.shape != draft_out.shape \
            or out_full.dim() != 4 or out_full.shape[-1] != D:
        raise LynxError("out_full, draft_out must be float32 [B][k][Hq][128]")
    B, k, Hq, _ = out_full.shape
    first_reject = torch.empty(B, dtype=torch.int32, device=out_full.device)
    dev = torch.empty(B, k, dtype=torch.float32, device=out_full.device)
    _ok(load().lynx_verify_decision(_ptr(out_full), _ptr(draft_out), B, k, Hq, atol, rtol, _ptr(first_reject), _ptr(dev),
                                    _stream()), "lynx_verify_decision")
    return first_reject, dev


@dataclass
class HierPlanes:
    """Algorithm 1 output for pages of 256 tokens: packed nibbles and the per-channel metadata."""
    q_anc: torch.Tensor        # u8 [n_pages][256][64]
    q_res: torch.Tensor        # u8 [n_pages][256][64]
    gamma_min: torch.Tensor    # f32 [n_pages][128]
    gamma_scale: torch.Tensor  # f32 [n_pages][128]
    mu: torch.Tensor           # f32 [n_pages][8][128]
    sigma: torch.Tensor        # f32 [n_pages][8][128]


def hier_quantize(src: torch.Tensor) -> HierPlanes:
    """lynx_hier_quantize: src BF16 [n_pages][256][128] -> HierPlanes."""
    if src.dtype != torch.bfloat16 or src.dim() != 3 or tuple(src.shape[1:]) != (256, D):
        raise LynxError("src must be BF16 [n_pages][256][128]")
    n, dev = src.shape[0], src.device
    out = HierPlanes(torch.empty(n, 256, 64, dtype=torch.uint8, device=dev), torch.empty(n, 256, 64, dtype=torch.uint8, device=dev),
                     torch.empty(n, D, dtype=torch.float32, device=dev), torch.empty(n, D, dtype=torch.float32, device=dev),
                     torch.empty(n, 8, D, dtype=torch.float32, device=dev), torch.empty(n, 8, D, dtype=torch.float32, device=dev))
    _ok(load().lynx_hier_quantize(_ptr(src), n, _ptr(out.q_anc), _ptr(out.q_res), _ptr(out.gamma_min),
                                  _ptr(out.gamma_scale), _ptr(out.mu), _ptr(out.sigma), _stream()), "lynx_hier_quantize")
    return out


def hier_dequantize(h: HierPlanes, anchor_only: bool = False, out: torch.Tensor | None = None) -> torch.Tensor:
    """lynx_hier_dequantize -> BF16 [n_pages][256][128] (from the Anchor stream alone if asked)."""
    n = h.q_anc.shape[0]
    if out is None:
        out = torch.empty(n, 256, D, dtype=torch.bfloat16, device=h.q_anc.device)
    _ok(load().lynx_hier_dequantize(_ptr(h.q_anc), None if anchor_only else _ptr(h.q_res), n, _ptr(h.gamma_min),
                                    _ptr(h.gamma_scale), _ptr(h.mu), _ptr(h.sigma), _ptr(out), _stream()),
        "lynx_hier_dequantize")
    return out


def token_verify(p_probs: torch.Tensor, q_probs: torch.Tensor, draft_tokens: torch.Tensor, u: torch.Tensor,
                 r: torch.Tensor):
    """lynx_token_verify: p_probs f32 [B][k][V], q_probs f32 [B][k+1][V], draft_tokens i32 [B][k], u f32 [B][k],
    r f32 [B] -> (n_accepted i32 [B], next_token i32 [B])."""
    B, k, V = p_probs.shape
    if tuple(q_probs.shape) != (B, k + 1, V) or p_probs.dtype != torch.float32 or q_probs.dtype != torch.float32:
        raise LynxError("p_probs must be float32 [B][k][V], q_probs float32 [B][k+1][V]")
    if draft_tokens.dtype != torch.int32 or tuple(draft_tokens.shape) != (B, k):
        raise LynxError("draft_tokens must be int32 [B][k]")
    if u.dtype != torch.float32 or tuple(u.shape) != (B, k) or r.dtype != torch.float32 or tuple(r.shape) != (B,):
        raise LynxError("u must be float32 [B][k], r float32 [B]")
    for t in (p_probs, q_probs, draft_tokens, u, r):
        if not t.is_contiguous():
            raise LynxError("contiguous tensors required")
    n_acc = torch.empty(B, dtype=torch.int32, device=p_probs.device)
    nxt = torch.empty(B, dtype=torch.int32, device=p_probs.device)
    _ok(load().lynx_token_verify(_ptr(p_probs), _ptr(q_probs), _ptr(draft_tokens), _ptr(u), _ptr(r), B, k, V,
                                 _ptr(n_acc), _ptr(nxt), _stream()), "lynx_token_verify")
    return n_acc, nxt
