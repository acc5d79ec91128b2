"""ctypes wrapper around the fp64 CPU oracle (oda_oracle.c).

TEST INFRASTRUCTURE, NOT THE PRODUCT: only tests/, the smoke check and the
benchmark's CPU-baseline leg import this module.  It shares nothing with the
CUDA library; the arithmetic lives in oda_oracle.c, this file only marshals
numpy arrays.  bf16 tensors are passed as uint16 bit patterns.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from dataclasses import dataclass
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "oda_oracle.c")
_LIB = os.path.join(_HERE, "liboda_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile oda_oracle.c with gcc (OpenMP over independent units only)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + f".tmp{os.getpid()}"
        subprocess.check_call(
            ["gcc", "-O2", "-std=c99", "-fopenmp", "-fPIC", "-shared", "-o", tmp, _SRC, "-lm"]
        )
        os.replace(tmp, _LIB)
    return _LIB


class _Shape(ctypes.Structure):
    _fields_ = [
        ("num_layers", ctypes.c_int32),
        ("batch", ctypes.c_int32),
        ("num_q_heads", ctypes.c_int32),
        ("num_kv_heads", ctypes.c_int32),
        ("head_dim", ctypes.c_int32),
        ("block_size", ctypes.c_int32),
        ("max_blocks_per_seq", ctypes.c_int32),
        ("reserved", ctypes.c_int32),
        ("kv_layer_stride", ctypes.c_int64),
        ("kv_block_stride", ctypes.c_int64),
        ("kv_token_stride", ctypes.c_int64),
        ("kv_head_stride", ctypes.c_int64),
        ("sm_scale", ctypes.c_double),
    ]


def lib():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oda_oracle_attention.restype = ctypes.c_int
        _lib.oda_oracle_recall_head.restype = ctypes.c_int
        _lib.oda_oracle_flags.restype = ctypes.c_int
        _lib.oda_oracle_step.restype = ctypes.c_int
        _lib.oda_oracle_max_threads.restype = ctypes.c_int
        _lib.oda_oracle_write_current_kv.restype = ctypes.c_int
        _lib.oda_oracle_select_rows.restype = ctypes.c_int
        _lib.oda_oracle_full_head.restype = ctypes.c_int
        _lib.oda_oracle_full_head_param_count.restype = ctypes.c_int64
    return _lib


def host_threads() -> int:
    """Cores this process may run on (what the timed baseline reports)."""
    try:
        return len(os.sched_getaffinity(0))
    except AttributeError:  # pragma: no cover
        return os.cpu_count() or 1


@dataclass
class KVLayout:
    """Element strides of the paged cache; the D values of one token/head are contiguous."""

    layer_stride: int
    block_stride: int
    token_stride: int
    head_stride: int


def hnd_layout(num_blocks: int, num_kv_heads: int, block_size: int, head_dim: int) -> KVLayout:
    """[layers, blocks, kv_heads, block_size, D]"""
    return KVLayout(
        layer_stride=num_blocks * num_kv_heads * block_size * head_dim,
        block_stride=num_kv_heads * block_size * head_dim,
        token_stride=head_dim,
        head_stride=block_size * head_dim,
    )


def nhd_layout(num_blocks: int, num_kv_heads: int, block_size: int, head_dim: int) -> KVLayout:
    """[layers, blocks, block_size, kv_heads, D]"""
    return KVLayout(
        layer_stride=num_blocks * num_kv_heads * block_size * head_dim,
        block_stride=num_kv_heads * block_size * head_dim,
        token_stride=num_kv_heads * head_dim,
        head_stride=head_dim,
    )


class _Args:
    """Keeps every marshalled array alive until the C call has returned."""

    def __init__(self):
        self.keep = []

    def __call__(self, a, dtype) -> ctypes.c_void_p:
        if a is None:
            return ctypes.c_void_p(None)
        a = np.ascontiguousarray(a, dtype=dtype)
        self.keep.append(a)
        return ctypes.c_void_p(a.ctypes.data)


def _out(a: np.ndarray, dtype) -> ctypes.c_void_p:
    assert a.dtype == dtype and a.flags["C_CONTIGUOUS"]
    return ctypes.c_void_p(a.ctypes.data)


def _i32(x: Optional[Sequence[int]]) -> Optional[np.ndarray]:
    return None if x is None else np.ascontiguousarray(np.asarray(x, dtype=np.int32))


def _shape(q: np.ndarray, num_kv_heads: int, block_size: int, block_table: np.ndarray,
           layout: KVLayout, sm_scale: float) -> _Shape:
    L, B, Hq, D = q.shape
    scale = sm_scale if sm_scale else 1.0 / np.sqrt(float(D))
    return _Shape(L, B, Hq, num_kv_heads, D, block_size, block_table.shape[1] if B else 0, 0,
                  layout.layer_stride, layout.block_stride, layout.token_stride,
                  layout.head_stride, float(scale))


def attention(mode: str, q: np.ndarray, k_cache: np.ndarray, v_cache: np.ndarray,
              block_table: np.ndarray, seq_lens: np.ndarray, *, num_kv_heads: int,
              block_size: int, layout: KVLayout, layer_window: Sequence[int],
              layer_sinks: Sequence[int], layer_kv_index: Optional[Sequence[int]] = None,
              request_mask: Optional[np.ndarray] = None, layer_begin: int = 0,
              layer_end: Optional[int] = None, sm_scale: float = 0.0, nthreads: int = 1):
    """Softmax attention over the Local ('local') or Full ('full') set of Eq. 1.

    q [L,B,Hq,D] uint16 (bf16 bits); caches flat uint16; returns (out f64 [L,B,Hq,D],
    lse f64 [L,B,Hq]); layers outside [layer_begin, layer_end) and masked-out
    requests are left as NaN.
    """
    assert mode in ("local", "full")
    L, B, Hq, D = q.shape
    layer_end = L if layer_end is None else layer_end
    block_table = np.ascontiguousarray(block_table, dtype=np.int32).reshape(B, -1)
    sh = _shape(q, num_kv_heads, block_size, block_table, layout, sm_scale)
    out = np.full((L, B, Hq, D), np.nan, dtype=np.float64)
    lse = np.full((L, B, Hq), np.nan, dtype=np.float64)
    a = _Args()
    rc = lib().oda_oracle_attention(
        ctypes.byref(sh), ctypes.c_int(1 if mode == "full" else 0), a(layer_window, np.int32),
        a(layer_sinks, np.int32), a(layer_kv_index, np.int32), a(q, np.uint16),
        a(k_cache.reshape(-1), np.uint16), a(v_cache.reshape(-1), np.uint16),
        a(block_table, np.int32), a(seq_lens, np.int32), a(request_mask, np.uint8),
        ctypes.c_int(layer_begin), ctypes.c_int(layer_end), _out(out, np.float64),
        _out(lse, np.float64), ctypes.c_int(nthreads))
    if rc:
        raise ValueError(f"oda_oracle_attention rejected its arguments ({rc})")
    return out, lse


def recall_head(feat_ext: Optional[np.ndarray], attn_feat: Optional[np.ndarray], W1: np.ndarray,
                b1: np.ndarray, w2: np.ndarray, b2):
    """z = w2 . SiLU(W1 [feat_ext ; attn_feat] + b1) + b2 and sigmoid(z), fp64.  Returns (z, score)."""
    d_hidden, d_in = W1.shape
    B = feat_ext.shape[0] if feat_ext is not None else attn_feat.shape[0]
    d_ext = 0 if feat_ext is None else feat_ext.shape[1]
    d_attn = 0 if attn_feat is None else attn_feat.reshape(B, -1).shape[1]
    assert d_ext + d_attn == d_in
    z = np.empty(B, dtype=np.float64)
    s = np.empty(B, dtype=np.float64)
    a = _Args()
    rc = lib().oda_oracle_recall_head(
        ctypes.c_int(B), ctypes.c_int(d_ext), ctypes.c_int(d_attn), ctypes.c_int(d_hidden),
        a(feat_ext, np.float32), a(None if attn_feat is None else attn_feat.reshape(B, -1), np.float64),
        a(W1, np.float32), a(b1, np.float32), a(w2, np.float32),
        a(np.asarray(b2, dtype=np.float32).reshape(1), np.float32),
        _out(z, np.float64), _out(s, np.float64))
    if rc:
        raise ValueError(f"oda_oracle_recall_head rejected its arguments ({rc})")
    return z, s


def flags(z: Optional[np.ndarray], score: Optional[np.ndarray], tau: float,
          override_flags: Optional[np.ndarray] = None) -> np.ndarray:
    """Decision rule: override if given, else (z nonfinite) or (score > tau), strictly."""
    B = len(override_flags) if override_flags is not None else len(z)
    f = np.zeros(B, dtype=np.uint8)
    a = _Args()
    rc = lib().oda_oracle_flags(
        ctypes.c_int(B), a(z, np.float64), a(score, np.float64), ctypes.c_double(tau),
        a(override_flags, np.uint8), _out(f, np.uint8))
    if rc:
        raise ValueError(f"oda_oracle_flags rejected its arguments ({rc})")
    return f


@dataclass
class StepResult:
    out: np.ndarray        # [L,B,Hq,D] f64, selected
    lse: np.ndarray        # [L,B,Hq]
    out_local: np.ndarray  # [L,B,Hq,D]
    lse_local: np.ndarray
    z: np.ndarray          # [B] head logit
    score: np.ndarray      # [B] sigmoid(z)
    flags: np.ndarray      # [B] uint8


def step(q_local: np.ndarray, q_full: Optional[np.ndarray], k_cache: np.ndarray, v_cache: np.ndarray,
         block_table: np.ndarray, seq_lens: np.ndarray, *, num_kv_heads: int, block_size: int,
         layout: KVLayout, layer_window: Sequence[int], layer_sinks: Sequence[int],
         layer_gated: Sequence[int], layer_kv_index: Optional[Sequence[int]] = None,
         head: Optional[dict] = None, feat_ext: Optional[np.ndarray] = None, tau: float = 0.5,
         override_flags: Optional[np.ndarray] = None, sm_scale: float = 0.0,
         nthreads: int = 1) -> StepResult:
    """One ODA step on the attention stack (Algorithm 1, lines 1-7).

    head: dict(W1, b1, w2, b2, use_attn_out) or None (then override_flags is required).
    """
    L, B, Hq, D = q_local.shape
    block_table = np.ascontiguousarray(block_table, dtype=np.int32).reshape(B, -1)
    sh = _shape(q_local, num_kv_heads, block_size, block_table, layout, sm_scale)
    out = np.full((L, B, Hq, D), np.nan)
    lse = np.full((L, B, Hq), np.nan)
    out_l = np.full((L, B, Hq, D), np.nan)
    lse_l = np.full((L, B, Hq), np.nan)
    z = np.zeros(B)
    score = np.zeros(B)
    fl = np.zeros(B, dtype=np.uint8)
    a = _Args()
    if head is not None:
        W1 = np.ascontiguousarray(head["W1"], dtype=np.float32)
        d_hidden = W1.shape[0]
        use_attn = int(head.get("use_attn_out", 1))
        d_ext = 0 if feat_ext is None else feat_ext.shape[1]
        assert W1.shape[1] == d_ext + (Hq * D if use_attn and any(layer_gated) else 0)
        hw = (a(W1, np.float32), a(head["b1"], np.float32), a(head["w2"], np.float32),
              a(np.asarray(head["b2"], dtype=np.float32).reshape(1), np.float32))
    else:
        d_hidden = use_attn = d_ext = 0
        hw = (a(None, np.float32),) * 4
    rc = lib().oda_oracle_step(
        ctypes.byref(sh), a(layer_window, np.int32), a(layer_sinks, np.int32),
        a(layer_gated, np.uint8), a(layer_kv_index, np.int32), a(q_local, np.uint16),
        a(q_full, np.uint16), a(k_cache.reshape(-1), np.uint16), a(v_cache.reshape(-1), np.uint16),
        a(block_table, np.int32), a(seq_lens, np.int32), ctypes.c_int(d_ext),
        ctypes.c_int(use_attn), ctypes.c_int(d_hidden), a(feat_ext, np.float32), *hw,
        ctypes.c_double(tau), a(override_flags, np.uint8), _out(out, np.float64),
        _out(lse, np.float64), _out(out_l, np.float64), _out(lse_l, np.float64),
        _out(z, np.float64), _out(score, np.float64), _out(fl, np.uint8), ctypes.c_int(nthreads))
    if rc:
        raise ValueError(f"oda_oracle_step rejected its arguments ({rc})")
    return StepResult(out, lse, out_l, lse_l, z, score, fl)


def write_current_kv(k_cur: np.ndarray, v_cur: np.ndarray, k_cache: np.ndarray, v_cache: np.ndarray,
                     block_table: np.ndarray, seq_lens: np.ndarray, *, block_size: int, layout: KVLayout,
                     mask: Optional[np.ndarray] = None, layer_kv_index: Optional[Sequence[int]] = None) -> None:
    """Commit of the current token: k_cur/v_cur [L,B,Hkv,D] (bf16 bits) are written IN PLACE into
    the flat uint16 caches at position seq_len-1 of every request with mask != 0 (None = all)."""
    L, B, Hkv, D = k_cur.shape
    assert k_cache.dtype == np.uint16 and k_cache.flags["C_CONTIGUOUS"] and k_cache.flags["WRITEABLE"]
    assert v_cache.dtype == np.uint16 and v_cache.flags["C_CONTIGUOUS"] and v_cache.flags["WRITEABLE"]
    block_table = np.ascontiguousarray(block_table, dtype=np.int32).reshape(B, -1)
    sh = _Shape(L, B, Hkv, Hkv, D, block_size, block_table.shape[1], 0, layout.layer_stride,
                layout.block_stride, layout.token_stride, layout.head_stride, 1.0)
    a = _Args()
    rc = lib().oda_oracle_write_current_kv(
        ctypes.byref(sh), a(layer_kv_index, np.int32), a(k_cur, np.uint16), a(v_cur, np.uint16),
        a(mask, np.uint8), _out(k_cache.reshape(-1), np.uint16), _out(v_cache.reshape(-1), np.uint16),
        a(block_table, np.int32), a(seq_lens, np.int32))
    if rc:
        raise ValueError(f"oda_oracle_write_current_kv rejected its arguments ({rc})")


def select_rows(local: np.ndarray, full: np.ndarray, flags: np.ndarray) -> np.ndarray:
    """Selected-state rule per request: out[b] = flags[b] ? full[b] : local[b]."""
    assert local.shape == full.shape and local.dtype == full.dtype
    B = local.shape[0]
    lo = np.ascontiguousarray(local)
    fu = np.ascontiguousarray(full)
    out = np.empty_like(lo)
    a = _Args()
    rc = lib().oda_oracle_select_rows(
        ctypes.c_int(B), ctypes.c_int64(lo.nbytes // max(B, 1)), ctypes.c_void_p(lo.ctypes.data),
        ctypes.c_void_p(fu.ctypes.data), a(flags, np.uint8), ctypes.c_void_p(out.ctypes.data))
    if rc:
        raise ValueError(f"oda_oracle_select_rows rejected its arguments ({rc})")
    return out


@dataclass
class CommitStepResult:
    out: np.ndarray
    out_local: np.ndarray
    z: np.ndarray
    score: np.ndarray
    flags: np.ndarray
    hidden: Optional[np.ndarray]


def step_with_commit(q_local, q_full, k_cache, v_cache, block_table, seq_lens, *, k_cur_local, v_cur_local,
                     k_cur_full, v_cur_full, num_kv_heads, block_size, layout, layer_window, layer_sinks,
                     layer_gated, head=None, feat_ext=None, tau=0.5, override_flags=None,
                     hidden_local=None, hidden_full=None, layer_kv_index=None, nthreads=1) -> CommitStepResult:
    """Algorithm 1, lines 1-8, on the attention stack, with the current token's K/V supplied as
    candidates: the Local candidate is written at position seq_len-1 and Local runs; the head
    decides; for requests that recall, the Full candidate replaces it and Full runs on the gated
    layers; the selected branch supplies the output, the hidden row, and is what the caches
    (modified in place) keep."""
    L, B, Hq, D = q_local.shape
    kw = dict(num_kv_heads=num_kv_heads, block_size=block_size, layout=layout, layer_window=layer_window,
              layer_sinks=layer_sinks, layer_kv_index=layer_kv_index, nthreads=nthreads)
    write_current_kv(k_cur_local, v_cur_local, k_cache, v_cache, block_table, seq_lens,
                     block_size=block_size, layout=layout, layer_kv_index=layer_kv_index)
    out_local, _ = attention("local", q_local, k_cache, v_cache, block_table, seq_lens, **kw)
    gated = [l for l in range(L) if layer_gated[l]]
    if head is not None:
        attn = out_local[gated[-1]].reshape(B, -1) if (gated and head.get("use_attn_out", 1)) else None
        z, score = recall_head(feat_ext, attn, head["W1"], head["b1"], head["w2"], head["b2"])
    else:
        z, score = np.zeros(B), np.full(B, 0.5)
    fl = flags(z, score, tau, override_flags)
    write_current_kv(k_cur_full, v_cur_full, k_cache, v_cache, block_table, seq_lens, block_size=block_size,
                     layout=layout, mask=fl, layer_kv_index=layer_kv_index)
    out = out_local.copy()
    if fl.any() and gated:
        full, _ = attention("full", q_full if q_full is not None else q_local, k_cache, v_cache, block_table,
                            seq_lens, request_mask=fl, **kw)
        for l in gated:
            for b in range(B):
                if fl[b]:
                    out[l, b] = full[l, b]
    hidden = None if hidden_local is None else select_rows(hidden_local, hidden_full, fl)
    return CommitStepResult(out, out_local, z, score, fl, hidden)


def full_head_param_count(d_model: int, d_tower: int, d_ff: int, n_blocks: int) -> int:
    return int(lib().oda_oracle_full_head_param_count(ctypes.c_int(d_model), ctypes.c_int(d_tower),
                                                      ctypes.c_int(d_ff), ctypes.c_int(n_blocks)))


def full_head(params: np.ndarray, h_prev: np.ndarray, emb: np.ndarray, h_local: np.ndarray, *, d_tower: int,
              d_ff: int, n_blocks: int, eps: float = 1e-6):
    """The paper's recall head (three towers, interaction vector, fusion, SwiGLU blocks, scalar
    output) in fp64 on fp32 parameters.  Returns (q, sigmoid(q))."""
    B, d_model = h_prev.shape
    assert params.dtype == np.float32 and params.size == full_head_param_count(d_model, d_tower, d_ff, n_blocks)
    q = np.empty(B)
    sc = np.empty(B)
    a = _Args()
    rc = lib().oda_oracle_full_head(
        ctypes.c_int(B), ctypes.c_int(d_model), ctypes.c_int(d_tower), ctypes.c_int(d_ff), ctypes.c_int(n_blocks),
        ctypes.c_double(eps), a(params, np.float32), a(h_prev, np.float32), a(emb, np.float32),
        a(h_local, np.float32), _out(q, np.float64), _out(sc, np.float64))
    if rc:
        raise ValueError(f"oda_oracle_full_head rejected its arguments ({rc})")
    return q, sc
