"""Thin ctypes binding over the C-ABI library (include/oda.h): argument marshalling only.

torch is used for device memory and streams; every step of the path runs in the
library's kernels.  There is no fallback: if the library is missing, or a call
fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, field
from typing import Optional, Sequence

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liboda_b200.so")

VARIANT_AUTO, VARIANT_SIMT, VARIANT_TMA_MMA = 0, 1, 2

EXPORTS = [
    "oda_create", "oda_destroy", "oda_workspace_bytes", "oda_set_workspace", "oda_local_decode",
    "oda_recall_score", "oda_full_decode_gated", "oda_step", "oda_step_host",
    "oda_read_device_status", "oda_launch_count", "oda_resolved_variant", "oda_attention_grid",
    "oda_status_string", "oda_last_error", "oda_version", "oda_local_decode_static",
    "oda_local_decode_static_status",
    "oda_calibration_begin", "oda_calibration_end", "oda_calibration_spread",
    "oda_write_current_kv", "oda_select_rows", "oda_advance_seq_lens", "oda_full_head_param_count", "oda_full_head_scratch_bytes",
    "oda_recall_score_full", "oda_recall_score_full_pre", "oda_recall_preact", "oda_recall_finalize", "oda_merge_partials",
    "oda_recall_finalize_exchange", "oda_merge_partials_exchange", "oda_set_cache_resident_bytes",
]


class OdaError(RuntimeError):
    def __init__(self, status: int, what: str, detail: str = ""):
        super().__init__(f"{what}: status {status} ({detail})")
        self.status = status


class _Config(ctypes.Structure):
    _fields_ = [
        ("num_layers", ctypes.c_int32), ("num_q_heads", ctypes.c_int32),
        ("num_kv_heads", ctypes.c_int32), ("head_dim", ctypes.c_int32),
        ("block_size", ctypes.c_int32), ("max_batch", ctypes.c_int32),
        ("max_blocks_per_seq", ctypes.c_int32), ("out_dtype", ctypes.c_int32),
        ("sm_scale", ctypes.c_float), ("variant", ctypes.c_int32),
        ("layer_window", ctypes.c_void_p), ("layer_sinks", ctypes.c_void_p),
        ("layer_gated", ctypes.c_void_p), ("layer_kv_index", ctypes.c_void_p),
        ("kv_layer_stride", ctypes.c_int64), ("kv_block_stride", ctypes.c_int64),
        ("kv_token_stride", ctypes.c_int64), ("kv_head_stride", ctypes.c_int64),
        ("head_d_ext", ctypes.c_int32), ("head_use_attn_out", ctypes.c_int32),
        ("head_d_hidden", ctypes.c_int32), ("options", ctypes.c_int32),
    ]


class _FullHead(ctypes.Structure):
    _fields_ = [("d_model", ctypes.c_int32), ("d_tower", ctypes.c_int32), ("d_ff", ctypes.c_int32),
                ("n_blocks", ctypes.c_int32), ("eps", ctypes.c_float), ("variant", ctypes.c_int32),
                ("params", ctypes.c_void_p)]


class _ExchangeRank(ctypes.Structure):
    _fields_ = [("pre_local", ctypes.c_void_p), ("scores", ctypes.c_void_p), ("logits", ctypes.c_void_p),
                ("flags", ctypes.c_void_p), ("counters", ctypes.c_void_p)]


class _MergeExchangeRank(ctypes.Structure):
    _fields_ = [("part_out", ctypes.c_void_p), ("part_lse", ctypes.c_void_p), ("tokens_local", ctypes.c_void_p),
                ("flags", ctypes.c_void_p), ("out", ctypes.c_void_p), ("lse", ctypes.c_void_p)]


class _StepArgs(ctypes.Structure):
    _fields_ = [
        ("batch", ctypes.c_int32), ("advance_seq_lens", ctypes.c_int32),
        ("q_local", ctypes.c_void_p), ("q_full", ctypes.c_void_p),
        ("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p),
        ("block_table", ctypes.c_void_p), ("seq_lens", ctypes.c_void_p),
        ("feat_ext", ctypes.c_void_p),
        ("W1", ctypes.c_void_p), ("b1", ctypes.c_void_p), ("w2", ctypes.c_void_p), ("b2", ctypes.c_void_p),
        ("threshold", ctypes.c_float), ("pad", ctypes.c_int32),
        ("override_flags", ctypes.c_void_p),
        ("out", ctypes.c_void_p), ("lse", ctypes.c_void_p), ("scores", ctypes.c_void_p),
        ("logits", ctypes.c_void_p), ("flags", ctypes.c_void_p), ("counters", ctypes.c_void_p),
        ("k_cur_local", ctypes.c_void_p), ("v_cur_local", ctypes.c_void_p),
        ("k_cur_full", ctypes.c_void_p), ("v_cur_full", ctypes.c_void_p),
        ("hidden_local", ctypes.c_void_p), ("hidden_full", ctypes.c_void_p), ("hidden_out", ctypes.c_void_p),
        ("hidden_row_bytes", ctypes.c_int64),
        ("full_head", ctypes.c_void_p), ("head_h_prev", ctypes.c_void_p), ("head_emb", ctypes.c_void_p),
        ("head_h_local", ctypes.c_void_p), ("head_scratch", ctypes.c_void_p),
        ("head_scratch_bytes", ctypes.c_size_t),
    ]


_lib = None


def load_library():
    """dlopen the C-ABI library; raises if it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run __graft_entry__.build() (nvcc, sm_100a) first")
        lib = ctypes.CDLL(LIB_PATH)
        vp, i32, f32 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_float
        lib.oda_create.argtypes = [ctypes.POINTER(_Config), ctypes.POINTER(vp)]
        lib.oda_destroy.argtypes = [vp]
        lib.oda_destroy.restype = None
        lib.oda_workspace_bytes.argtypes = [vp, ctypes.POINTER(ctypes.c_size_t)]
        lib.oda_set_workspace.argtypes = [vp, vp, ctypes.c_size_t, vp]
        lib.oda_local_decode.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.oda_recall_score.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, f32, vp, vp, vp, vp, vp, vp]
        lib.oda_recall_preact.argtypes = [vp, i32, vp, vp, vp, ctypes.c_int64, vp, vp]
        lib.oda_recall_preact.restype = i32
        lib.oda_recall_finalize.argtypes = [vp, i32, vp, vp, vp, vp, f32, vp, vp, vp, vp, vp, vp]
        lib.oda_recall_finalize.restype = i32
        lib.oda_merge_partials.argtypes = [vp, i32, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp]
        lib.oda_merge_partials.restype = i32
        lib.oda_recall_finalize_exchange.argtypes = [vp, i32, i32, i32, i32, ctypes.POINTER(_ExchangeRank), vp, vp,
                                                     ctypes.c_uint32, ctypes.c_uint64, vp, vp, vp, f32, vp, vp]
        lib.oda_recall_finalize_exchange.restype = i32
        lib.oda_merge_partials_exchange.argtypes = [vp, i32, i32, i32, ctypes.POINTER(_MergeExchangeRank), vp, vp, vp,
                                                    ctypes.c_uint32, ctypes.c_uint64, i32, i32, i32, vp]
        lib.oda_merge_partials_exchange.restype = i32
        lib.oda_set_cache_resident_bytes.argtypes = [vp, ctypes.c_size_t]
        lib.oda_set_cache_resident_bytes.restype = i32
        lib.oda_full_decode_gated.argtypes = [vp, i32, i32, i32, vp, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.oda_step.argtypes = [vp, ctypes.POINTER(_StepArgs), vp]
        lib.oda_step_host.argtypes = [vp, ctypes.POINTER(_StepArgs), vp,
                                      ctypes.POINTER(ctypes.c_size_t), ctypes.POINTER(ctypes.c_size_t)]
        lib.oda_local_decode_static.argtypes = [i32, i32, i32, i32, i32, i32, f32, ctypes.c_int64,
                                                ctypes.c_int64, ctypes.c_int64, i32, vp, vp, vp, vp, vp,
                                                vp, vp, vp]
        lib.oda_local_decode_static_status.argtypes = [vp, ctypes.POINTER(i32)]
        lib.oda_write_current_kv.argtypes = [vp, i32, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.oda_select_rows.argtypes = [vp, i32, vp, vp, vp, vp, ctypes.c_int64, vp]
        lib.oda_advance_seq_lens.argtypes = [vp, i32, vp, vp]
        lib.oda_full_head_param_count.argtypes = [i32, i32, i32, i32]
        lib.oda_full_head_param_count.restype = ctypes.c_int64
        lib.oda_full_head_scratch_bytes.argtypes = [ctypes.POINTER(_FullHead), i32]
        lib.oda_full_head_scratch_bytes.restype = ctypes.c_size_t
        lib.oda_recall_score_full.argtypes = [vp, i32, ctypes.POINTER(_FullHead), vp, vp, vp, f32, vp, vp, vp, vp,
                                              vp, vp, ctypes.c_size_t, vp]
        lib.oda_recall_score_full_pre.argtypes = [vp, i32, ctypes.POINTER(_FullHead), vp, vp, vp, ctypes.c_size_t, vp]
        lib.oda_calibration_begin.argtypes = [vp, vp]
        lib.oda_calibration_end.argtypes = [vp, vp]
        lib.oda_calibration_spread.argtypes = [vp]
        lib.oda_calibration_spread.restype = ctypes.c_double
        lib.oda_read_device_status.argtypes = [vp, vp, ctypes.POINTER(i32)]
        lib.oda_launch_count.argtypes = [vp]
        lib.oda_launch_count.restype = ctypes.c_int64
        lib.oda_resolved_variant.argtypes = [vp]
        lib.oda_attention_grid.argtypes = [vp]
        lib.oda_status_string.argtypes = [ctypes.c_int]
        lib.oda_status_string.restype = ctypes.c_char_p
        lib.oda_last_error.argtypes = [vp]
        lib.oda_last_error.restype = ctypes.c_char_p
        lib.oda_version.restype = ctypes.c_char_p
        _lib = lib
    return _lib


@dataclass
class OdaConfig:
    num_layers: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    max_batch: int
    max_blocks_per_seq: int
    layer_window: Sequence[int]
    layer_sinks: Sequence[int]
    layer_gated: Sequence[int]
    kv_layer_stride: int
    kv_block_stride: int
    kv_token_stride: int
    kv_head_stride: int
    layer_kv_index: Optional[Sequence[int]] = None
    block_size: int = 16
    out_dtype: int = 0
    sm_scale: float = 0.0
    variant: int = VARIANT_AUTO
    head_d_ext: int = 0
    head_use_attn_out: int = 1
    head_d_hidden: int = 0
    serialize_launches: int = 0   # 1 = no programmatic dependent launch between the kernels of a step
    allow_empty: int = 0          # 1 = gated passes skip flagged requests of length 0 (sequence-sharded ranks)
    reuse_local: int = 0          # 1 = the gated pass reads only S^F \ S^L and merges with Local (q_full == q_local)
    _keep: list = field(default_factory=list, repr=False)

    def to_c(self) -> _Config:
        def arr(x, dt):
            if x is None:
                return None
            a = np.ascontiguousarray(np.asarray(x, dtype=dt))
            self._keep.append(a)
            return a.ctypes.data

        return _Config(
            self.num_layers, self.num_q_heads, self.num_kv_heads, self.head_dim, self.block_size,
            self.max_batch, self.max_blocks_per_seq, self.out_dtype, self.sm_scale, self.variant,
            arr(self.layer_window, np.int32), arr(self.layer_sinks, np.int32),
            arr(self.layer_gated, np.uint8), arr(self.layer_kv_index, np.int32),
            self.kv_layer_stride, self.kv_block_stride, self.kv_token_stride, self.kv_head_stride,
            self.head_d_ext, self.head_use_attn_out, self.head_d_hidden,
            (1 if self.serialize_launches else 0) | (2 if self.reuse_local else 0) | (4 if self.allow_empty else 0))


def _ptr(t) -> Optional[int]:
    """Device (or host) address of a torch tensor / numpy array / raw int; None stays NULL."""
    if t is None:
        return None
    if isinstance(t, int):
        return t
    if isinstance(t, np.ndarray):
        assert t.flags["C_CONTIGUOUS"]
        return t.ctypes.data
    assert t.is_contiguous(), "tensors handed to the library must be contiguous"
    return t.data_ptr()


def _stream() -> int:
    import torch

    return torch.cuda.current_stream().cuda_stream


class OdaContext:
    """Owns an oda_ctx_t and (optionally) its workspace tensor."""

    def __init__(self, cfg: OdaConfig, allocate_workspace: bool = True):
        self.lib = load_library()
        self.cfg = cfg
        self._h = ctypes.c_void_p()
        ccfg = cfg.to_c()
        st = self.lib.oda_create(ctypes.byref(ccfg), ctypes.byref(self._h))
        if st != 0:
            raise OdaError(st, "oda_create", self.lib.oda_status_string(st).decode())
        self.workspace = None
        if allocate_workspace:
            import torch

            self.workspace = torch.empty(self.workspace_bytes(), dtype=torch.uint8, device="cuda")
            self.set_workspace(self.workspace.data_ptr(), self.workspace.numel())

    def close(self):
        h = getattr(self, "_h", None)
        if h is not None and h.value:
            self.lib.oda_destroy(h)
            self._h = None

    __del__ = close

    def _check(self, st: int, what: str):
        if st != 0:
            raise OdaError(st, what, self.lib.oda_last_error(self._h).decode())

    def workspace_bytes(self) -> int:
        n = ctypes.c_size_t()
        self._check(self.lib.oda_workspace_bytes(self._h, ctypes.byref(n)), "oda_workspace_bytes")
        return n.value

    def set_workspace(self, ptr: int, nbytes: int, stream: Optional[int] = None):
        self._check(self.lib.oda_set_workspace(self._h, ptr, nbytes, _stream() if stream is None else stream),
                    "oda_set_workspace")

    def calibration_begin(self, stream=None):
        """Start recording per-SM streaming rates in the attention launches that follow."""
        self._check(self.lib.oda_calibration_begin(self._h, _stream() if stream is None else stream),
                    "oda_calibration_begin")

    def calibration_end(self, stream=None) -> float:
        """Fix the split of work across SMs from the recorded rates.  Returns slowest/fastest
        rate (0: not applied, e.g. no large launch was seen)."""
        self._check(self.lib.oda_calibration_end(self._h, _stream() if stream is None else stream),
                    "oda_calibration_end")
        return self.lib.oda_calibration_spread(self._h)

    # ---- the four calls of the path -------------------------------------------------
    def local_decode(self, layer_begin, layer_end, batch, q, k_cache, v_cache, block_table, seq_lens,
                     out, lse=None, stream=None):
        self._check(self.lib.oda_local_decode(
            self._h, layer_begin, layer_end, batch, _ptr(q), _ptr(k_cache), _ptr(v_cache),
            _ptr(block_table), _ptr(seq_lens), _ptr(out), _ptr(lse),
            _stream() if stream is None else stream), "oda_local_decode")

    def recall_score(self, batch, feat_ext, attn_out_last, W1, b1, w2, b2, threshold, override_flags,
                     scores, logits, flags, counters=None, stream=None):
        self._check(self.lib.oda_recall_score(
            self._h, batch, _ptr(feat_ext), _ptr(attn_out_last), _ptr(W1), _ptr(b1), _ptr(w2), _ptr(b2),
            float(threshold), _ptr(override_flags), _ptr(scores), _ptr(logits), _ptr(flags),
            _ptr(counters), _stream() if stream is None else stream), "oda_recall_score")

    def recall_preact(self, batch, feat_ext, attn_out_last, W1_cols, w1_row_stride, pre_out, stream=None):
        """This rank's share of W1 x; W1_cols is a device address (int) or a tensor."""
        w = W1_cols if isinstance(W1_cols, int) else _ptr(W1_cols)
        self._check(self.lib.oda_recall_preact(
            self._h, batch, _ptr(feat_ext), _ptr(attn_out_last), w, int(w1_row_stride), _ptr(pre_out),
            _stream() if stream is None else stream), "oda_recall_preact")

    def recall_finalize(self, batch, pre_sum, b1, w2, b2, threshold, override_flags, scores, logits, flags,
                        counters=None, stream=None):
        self._check(self.lib.oda_recall_finalize(
            self._h, batch, _ptr(pre_sum), _ptr(b1), _ptr(w2), _ptr(b2), float(threshold),
            _ptr(override_flags), _ptr(scores), _ptr(logits), _ptr(flags), _ptr(counters),
            _stream() if stream is None else stream), "oda_recall_finalize")

    def merge_partials(self, n_parts, layer_begin, layer_end, batch, parts_out, parts_lse, flags, out, lse=None,
                       part_tokens=None, stream=None):
        self._check(self.lib.oda_merge_partials(
            self._h, n_parts, layer_begin, layer_end, batch, _ptr(parts_out), _ptr(parts_lse), _ptr(part_tokens),
            _ptr(flags), _ptr(out), _ptr(lse), _stream() if stream is None else stream), "oda_merge_partials")

    def recall_finalize_exchange(self, batch, world, rank_base, ranks, recv, arrived, epoch, b1, w2, b2,
                                 threshold, override_flags=None, timeout_ns=0, stream=None):
        """ranks: list of dicts(pre_local, scores, flags[, logits, counters]) for the ranks this launch
        runs; recv / arrived: the receive buffers and flag arrays of ALL ranks of the group, in rank order."""
        n_local = len(ranks)
        arr = (_ExchangeRank * n_local)(*[
            _ExchangeRank(_ptr(r["pre_local"]), _ptr(r["scores"]), _ptr(r.get("logits")), _ptr(r["flags"]),
                          _ptr(r.get("counters"))) for r in ranks])
        recv_p = (ctypes.c_void_p * world)(*[_ptr(t) for t in recv])
        arr_p = (ctypes.c_void_p * world)(*[_ptr(t) for t in arrived])
        self._check(self.lib.oda_recall_finalize_exchange(
            self._h, batch, world, rank_base, n_local, arr, ctypes.cast(recv_p, ctypes.c_void_p),
            ctypes.cast(arr_p, ctypes.c_void_p), int(epoch), int(timeout_ns), _ptr(b1), _ptr(w2), _ptr(b2),
            float(threshold), _ptr(override_flags), _stream() if stream is None else stream),
            "oda_recall_finalize_exchange")

    def merge_partials_exchange(self, world, rank_base, ranks, recv_out, recv_lse, arrived, epoch, layer_begin,
                                layer_end, batch, timeout_ns=0, stream=None):
        """ranks: list of dicts(part_out, part_lse, out[, tokens_local, flags, lse]) for the ranks this launch runs."""
        n_local = len(ranks)
        arr = (_MergeExchangeRank * n_local)(*[
            _MergeExchangeRank(_ptr(r["part_out"]), _ptr(r["part_lse"]), _ptr(r.get("tokens_local")),
                               _ptr(r.get("flags")), _ptr(r["out"]), _ptr(r.get("lse"))) for r in ranks])
        tabs = [(ctypes.c_void_p * world)(*[_ptr(t) for t in tab]) for tab in (recv_out, recv_lse, arrived)]
        self._check(self.lib.oda_merge_partials_exchange(
            self._h, world, rank_base, n_local, arr, *[ctypes.cast(t, ctypes.c_void_p) for t in tabs], int(epoch),
            int(timeout_ns), layer_begin, layer_end, batch, _stream() if stream is None else stream),
            "oda_merge_partials_exchange")

    def full_decode_gated(self, layer_begin, layer_end, batch, q_full, k_cache, v_cache, block_table,
                          seq_lens, flags, out, lse=None, stream=None):
        self._check(self.lib.oda_full_decode_gated(
            self._h, layer_begin, layer_end, batch, _ptr(q_full), _ptr(k_cache), _ptr(v_cache),
            _ptr(block_table), _ptr(seq_lens), _ptr(flags), _ptr(out), _ptr(lse),
            _stream() if stream is None else stream), "oda_full_decode_gated")

    def recall_score_full(self, batch, params, d_tower, d_ff, n_blocks, h_prev, emb, h_local, threshold,
                          override_flags, scores, logits, flags, counters=None, eps=1e-6, scratch=None,
                          stream=None, variant=0):
        """The paper's full recall head; `params` is the flat fp32 parameter tensor (see oda.h)."""
        import torch

        head = _FullHead(h_prev.shape[1], d_tower, d_ff, n_blocks, eps, int(variant), _ptr(params))
        need = self.lib.oda_full_head_scratch_bytes(ctypes.byref(head), batch)
        if scratch is None:
            scratch = torch.empty(need, dtype=torch.uint8, device=h_prev.device)
        self._check(self.lib.oda_recall_score_full(
            self._h, batch, ctypes.byref(head), _ptr(h_prev), _ptr(emb), _ptr(h_local), float(threshold),
            _ptr(override_flags), _ptr(scores), _ptr(logits), _ptr(flags), _ptr(counters), _ptr(scratch),
            scratch.numel(), _stream() if stream is None else stream), "oda_recall_score_full")
        return scratch

    def recall_score_full_pre(self, batch, params, d_tower, d_ff, n_blocks, h_prev, emb, scratch, eps=1e-6,
                              stream=None):
        """First part of the paper's head (towers a, b and their share of the fusion product), left in
        `scratch` for a recall_score_full(..., variant=3) on the same scratch."""
        head = _FullHead(h_prev.shape[1], d_tower, d_ff, n_blocks, eps, 0, _ptr(params))
        self._check(self.lib.oda_recall_score_full_pre(
            self._h, batch, ctypes.byref(head), _ptr(h_prev), _ptr(emb), _ptr(scratch), scratch.numel(),
            _stream() if stream is None else stream), "oda_recall_score_full_pre")

    def full_head_scratch(self, batch, d_model, d_tower, d_ff, n_blocks, device="cuda"):
        """A scratch tensor large enough for the paper's head at this batch."""
        import torch

        head = _FullHead(d_model, d_tower, d_ff, n_blocks, 1e-6, 0, None)
        return torch.empty(self.lib.oda_full_head_scratch_bytes(ctypes.byref(head), batch), dtype=torch.uint8,
                           device=device)

    def write_current_kv(self, batch, k_cur, v_cur, mask, k_cache, v_cache, block_table, seq_lens, stream=None):
        self._check(self.lib.oda_write_current_kv(
            self._h, batch, _ptr(k_cur), _ptr(v_cur), _ptr(mask), _ptr(k_cache), _ptr(v_cache),
            _ptr(block_table), _ptr(seq_lens), _stream() if stream is None else stream), "oda_write_current_kv")

    def advance_seq_lens(self, batch, seq_lens, stream=None):
        """seq_lens[b] += 1 on the device (steps composed from the separate calls)."""
        self._check(self.lib.oda_advance_seq_lens(self._h, batch, _ptr(seq_lens),
                                                  _stream() if stream is None else stream), "oda_advance_seq_lens")

    def select_rows(self, batch, local, full, flags, out, stream=None):
        self._check(self.lib.oda_select_rows(
            self._h, batch, _ptr(local), _ptr(full), _ptr(flags), _ptr(out),
            out[0].numel() * out.element_size(), _stream() if stream is None else stream), "oda_select_rows")

    @staticmethod
    def step_args(batch, q_local, k_cache, v_cache, block_table, seq_lens, out, scores, flags,
                  q_full=None, feat_ext=None, head=None, threshold=0.5, override_flags=None, lse=None,
                  logits=None, counters=None, advance_seq_lens=False, k_cur_local=None, v_cur_local=None,
                  k_cur_full=None, v_cur_full=None, hidden_local=None, hidden_full=None,
                  hidden_out=None, full_head=None) -> _StepArgs:
        """full_head: dict(params, d_tower, d_ff, n_blocks, h_prev, emb, h_local, scratch[, eps, variant])
        to decide with the paper's own recall head."""
        h = head or {}
        row_bytes = 0 if hidden_out is None else hidden_out[0].numel() * hidden_out.element_size()
        fh = (None,) * 6
        keep = None
        if full_head is not None:
            keep = _FullHead(full_head["h_prev"].shape[1], full_head["d_tower"], full_head["d_ff"],
                             full_head["n_blocks"], full_head.get("eps", 1e-6), int(full_head.get("variant", 0)),
                             _ptr(full_head["params"]))
            fh = (ctypes.addressof(keep), _ptr(full_head["h_prev"]), _ptr(full_head["emb"]),
                  _ptr(full_head["h_local"]), _ptr(full_head["scratch"]), full_head["scratch"].numel())
        args = _StepArgs(
            batch, 1 if advance_seq_lens else 0, _ptr(q_local), _ptr(q_full), _ptr(k_cache),
            _ptr(v_cache), _ptr(block_table), _ptr(seq_lens), _ptr(feat_ext), _ptr(h.get("W1")),
            _ptr(h.get("b1")), _ptr(h.get("w2")), _ptr(h.get("b2")), float(threshold), 0,
            _ptr(override_flags), _ptr(out), _ptr(lse), _ptr(scores), _ptr(logits), _ptr(flags),
            _ptr(counters), _ptr(k_cur_local), _ptr(v_cur_local), _ptr(k_cur_full), _ptr(v_cur_full),
            _ptr(hidden_local), _ptr(hidden_full), _ptr(hidden_out), row_bytes, fh[0], fh[1], fh[2], fh[3],
            fh[4], fh[5] or 0)
        # the head descriptor and every buffer whose address is in the block must outlive the call
        args._keep = (keep, q_local, q_full, k_cache, v_cache, block_table, seq_lens, feat_ext, head, override_flags,
                      out, lse, scores, logits, flags, counters, k_cur_local, v_cur_local, k_cur_full, v_cur_full,
                      hidden_local, hidden_full, hidden_out, full_head)
        return args

    def step(self, args: _StepArgs, stream=None):
        self._check(self.lib.oda_step(self._h, ctypes.byref(args), _stream() if stream is None else stream),
                    "oda_step")

    def step_host(self, args: _StepArgs, stream=None):
        up, down = ctypes.c_size_t(), ctypes.c_size_t()
        self._check(self.lib.oda_step_host(self._h, ctypes.byref(args),
                                           _stream() if stream is None else stream,
                                           ctypes.byref(up), ctypes.byref(down)), "oda_step_host")
        return up.value, down.value

    def set_cache_resident_bytes(self, nbytes: int):
        """Local working set (leading layers) to keep in L2 between steps; 0 turns it off."""
        self._check(self.lib.oda_set_cache_resident_bytes(self._h, int(nbytes)), "oda_set_cache_resident_bytes")

    # ---- introspection ----------------------------------------------------------------
    def read_device_status(self, stream=None) -> int:
        code = ctypes.c_int32()
        st = self.lib.oda_read_device_status(self._h, _stream() if stream is None else stream,
                                             ctypes.byref(code))
        if st not in (0, 5):
            self._check(st, "oda_read_device_status")
        return code.value

    @property
    def launch_count(self) -> int:
        return self.lib.oda_launch_count(self._h)

    @property
    def variant(self) -> int:
        return self.lib.oda_resolved_variant(self._h)

    @property
    def attention_grid(self) -> int:
        return self.lib.oda_attention_grid(self._h)


def local_decode_static(batch, num_q_heads, num_kv_heads, head_dim, window, sinks, sm_scale,
                        kv_block_stride, kv_token_stride, kv_head_stride, max_blocks_per_seq, q,
                        k_cache, v_cache, block_table, seq_lens, out, lse=None, stream=None) -> None:
    """Local pass of one layer with no workspace: for callers that cannot allocate device memory
    (the scratch is a fixed array inside the library).  Limits: batch <= 16, batch*kv_heads <= 256.
    Calls on one device must not overlap; make the first call on a device outside stream capture."""
    st = load_library().oda_local_decode_static(
        batch, num_q_heads, num_kv_heads, head_dim, window, sinks, float(sm_scale), kv_block_stride,
        kv_token_stride, kv_head_stride, max_blocks_per_seq, _ptr(q), _ptr(k_cache), _ptr(v_cache),
        _ptr(block_table), _ptr(seq_lens), _ptr(out), _ptr(lse), _stream() if stream is None else stream)
    if st != 0:
        raise OdaError(st, "oda_local_decode_static", load_library().oda_status_string(st).decode())


def local_decode_static_status(stream=None) -> int:
    """Reads and clears the status word of the local_decode_static calls made on the current device
    (bit 0: a request had seq_len < 1 and was skipped; same bits as OdaContext.read_device_status).
    Synchronises the stream; allocates nothing."""
    code = ctypes.c_int32(0)
    st = load_library().oda_local_decode_static_status(_stream() if stream is None else stream, ctypes.byref(code))
    if st not in (0, 5):
        raise OdaError(st, "oda_local_decode_static_status", load_library().oda_status_string(st).decode())
    return int(code.value)


def version() -> str:
    return load_library().oda_version().decode()
