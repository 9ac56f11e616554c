"""CPU oracle for the Lynx split-stream quantisation hot path (TEST INFRASTRUCTURE).

A plain, slow C restatement (``lynx_oracle.c``) of what the CUDA library computes,
wrapped for numpy.  Only the tests, the smoke check and the benchmark's timed CPU
baseline may import this package; the product never does, and this package never
imports the product.  Quantisation is done in IEEE binary32 exactly as the paper's
linear grouped quantiser states it (Section 2.3), attention (Section 2) and the
accept/reject test (Section 4.3) in binary64.

Every function takes and returns numpy arrays on the host.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lynx_oracle.c")
_LIB = os.path.join(_HERE, "liblynx_oracle.so")
_lib = None

D = 128  # head_dim = group size


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (no fast-math, no contraction). Returns the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O2", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
               "-o", tmp, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
    return _lib


def _p(a: np.ndarray | None):
    if a is None:
        return ctypes.c_void_p(0)
    assert a.flags["C_CONTIGUOUS"], "oracle arrays must be C-contiguous"
    return ctypes.c_void_p(a.ctypes.data)


def threads() -> int:
    """Number of OpenMP threads the oracle runs with."""
    lib = _load()
    lib.lynx_oracle_threads.restype = ctypes.c_int
    return int(lib.lynx_oracle_threads())


def split_quantize(src_bf16_bits: np.ndarray, want_codes: bool = False):
    """src_bf16_bits: uint16 [..., 128] (BF16 bit patterns). Returns (anchor u8 [...,64],
    residual u8 [...,64], meta f32 [...,2]) and, if asked, codes u8 [...,128]."""
    src = np.ascontiguousarray(src_bf16_bits, dtype=np.uint16)
    assert src.shape[-1] == D
    lead = src.shape[:-1]
    n_rows = int(np.prod(lead, dtype=np.int64)) if lead else 1
    anchor = np.empty(lead + (64,), np.uint8)
    residual = np.empty(lead + (64,), np.uint8)
    meta = np.empty(lead + (2,), np.float32)
    codes = np.empty(lead + (D,), np.uint8) if want_codes else None
    _load().lynx_oracle_split_quantize(_p(src), ctypes.c_int64(n_rows), _p(anchor), _p(residual),
                                       _p(meta), _p(codes))
    return (anchor, residual, meta, codes) if want_codes else (anchor, residual, meta)


def recombine(anchor: np.ndarray, residual: np.ndarray, meta: np.ndarray,
              want_bf16: bool = True):
    """Returns (codes u8 [...,128], dequantised BF16 bits uint16 [...,128] or None)."""
    anchor = np.ascontiguousarray(anchor, np.uint8)
    residual = np.ascontiguousarray(residual, np.uint8)
    meta = np.ascontiguousarray(meta, np.float32)
    lead = anchor.shape[:-1]
    n_rows = int(np.prod(lead, dtype=np.int64)) if lead else 1
    codes = np.empty(lead + (D,), np.uint8)
    deq = np.empty(lead + (D,), np.uint16) if want_bf16 else None
    _load().lynx_oracle_recombine(_p(anchor), _p(residual), _p(meta), ctypes.c_int64(n_rows),
                                  _p(codes), _p(deq))
    return codes, deq


def attention(full: bool, q_bf16_bits: np.ndarray, k_planes, v_planes, block_table: np.ndarray,
              seq_lens: np.ndarray, num_kv_heads: int, block_tokens: int, causal: bool = False,
              softmax_scale: float | None = None) -> np.ndarray:
    """Attention over quantised paged K/V in binary64.

    q_bf16_bits: uint16 [B][n_q][Hq][128].  k_planes / v_planes: (anchor, residual-or-None,
    meta) with anchor/residual u8 [num_blocks][Hkv][block_tokens][64] and meta f32
    [num_blocks][Hkv][block_tokens][2].  block_table int32 [B][max_blocks]; seq_lens int32 [B].
    full=False uses the Anchor plane alone (bucket mid-point 16a+8); full=True uses 16a+r.
    Returns float64 [B][n_q][Hq][128].
    """
    q = np.ascontiguousarray(q_bf16_bits, np.uint16)
    B, n_q, Hq, d = q.shape
    assert d == D and Hq % num_kv_heads == 0
    ka, kr, km = k_planes
    va, vr, vm = v_planes
    ka = np.ascontiguousarray(ka, np.uint8); va = np.ascontiguousarray(va, np.uint8)
    km = np.ascontiguousarray(km, np.float32); vm = np.ascontiguousarray(vm, np.float32)
    if full:
        kr = np.ascontiguousarray(kr, np.uint8); vr = np.ascontiguousarray(vr, np.uint8)
    else:
        kr = vr = None
    bt = np.ascontiguousarray(block_table, np.int32)
    sl = np.ascontiguousarray(seq_lens, np.int32)
    assert bt.shape[0] == B and sl.shape == (B,)
    if softmax_scale is None:
        softmax_scale = 1.0 / np.sqrt(np.float64(D))
    out = np.empty((B, n_q, Hq, D), np.float64)
    _load().lynx_oracle_attention(
        ctypes.c_int(1 if full else 0), ctypes.c_int32(Hq), ctypes.c_int32(num_kv_heads),
        ctypes.c_int32(block_tokens), ctypes.c_int32(bt.shape[1]), _p(q), ctypes.c_int32(B),
        ctypes.c_int32(n_q), ctypes.c_int32(1 if causal else 0), _p(ka), _p(kr), _p(km), _p(va),
        _p(vr), _p(vm), _p(bt), _p(sl), ctypes.c_float(np.float32(softmax_scale)), _p(out))
    return out


def verify_decision(out_full: np.ndarray, draft_f32: np.ndarray, atol: float, rtol: float):
    """out_full float64 [B][k][Hq][128], draft float32 same shape.
    Returns (first_reject int32 [B], dev float64 [B][k])."""
    of = np.ascontiguousarray(out_full, np.float64)
    dr = np.ascontiguousarray(draft_f32, np.float32)
    B, k, Hq, d = of.shape
    assert dr.shape == of.shape and d == D
    fr = np.empty((B,), np.int32)
    dev = np.empty((B, k), np.float64)
    _load().lynx_oracle_verify_decision(_p(of), _p(dr), ctypes.c_int32(B), ctypes.c_int32(k),
                                        ctypes.c_int32(Hq), ctypes.c_double(atol),
                                        ctypes.c_double(rtol), _p(fr), _p(dev))
    return fr, dev


def attention_bf16_pages(q_bf16_bits: np.ndarray, k_pages_bits: np.ndarray, v_pages_bits: np.ndarray,
                         block_table: np.ndarray, seq_lens: np.ndarray, causal: bool = False,
                         softmax_scale: float | None = None) -> np.ndarray:
    """Attention over dequantised BF16 pages in binary64: the decode path the paper describes
    (Section 4.2: the dequantisation kernel scatters BF16 pages, the engine's attention reads them;
    Section 2: softmax(Q K^T / sqrt(d)) V).  Plain numpy, one (sequence, query, head) at a time.

    q_bf16_bits uint16 [B][n_q][Hq][128]; k/v_pages_bits uint16 [num_blocks][Hkv][block_tokens][128]
    (BF16 bit patterns); block_table int32 [B][max_blocks]; seq_lens int32 [B].  Query j of
    sequence b sees tokens [0, len) or, causal, [0, len - n_q + j + 1).  Returns float64
    [B][n_q][Hq][128]; a query that sees nothing gets zeros.
    """
    def f64(bits):
        return (np.ascontiguousarray(bits, np.uint16).astype(np.uint32) << 16).view(np.float32).astype(np.float64)
    q, kp, vp = f64(q_bf16_bits), f64(k_pages_bits), f64(v_pages_bits)
    B, n_q, Hq, d = q.shape
    _, Hkv, bt, _ = kp.shape
    assert d == D and Hq % Hkv == 0
    G = Hq // Hkv
    if softmax_scale is None:
        softmax_scale = 1.0 / np.sqrt(np.float64(D))
    scale = np.float64(np.float32(softmax_scale))
    out = np.zeros((B, n_q, Hq, D), np.float64)
    for b in range(B):
        length = min(max(int(seq_lens[b]), 0), block_table.shape[1] * bt)
        nblk = (length + bt - 1) // bt
        blocks = np.asarray(block_table[b, :nblk], np.int64)
        for h in range(Hq):
            k_rows = kp[blocks, h // G].reshape(-1, D)[:length]      # token t = row t % bt of block t / bt
            v_rows = vp[blocks, h // G].reshape(-1, D)[:length]
            for j in range(n_q):
                lim = length - n_q + j + 1 if causal else length
                if lim <= 0:
                    continue
                s = (k_rows[:lim] @ q[b, j, h]) * scale
                w = np.exp(s - s.max())
                out[b, j, h] = (w / w.sum()) @ v_rows[:lim]
    return out
