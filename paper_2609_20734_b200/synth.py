"""Seeded synthetic inputs, bit-identical on host (numpy) and device (one fill kernel).

This module holds no arithmetic of the attention method: it only produces
inputs.  Both the CPU oracle's tests and the CUDA path's tests draw from it, so
that the two sides see the same bits without either importing the other.

Recipe: a counter-based generator.  `key = mix64(mix64(seed) ^ stream * GOLD)`;
element `idx` of a stream gets the 16-bit code `mix64(key + idx * GOLD) >> 48`;
the code indexes a 65,536-entry table of standard-normal quantiles
`ndtri((code + 0.5) / 65536)`, built once on the host in fp64 and rounded to
bf16 (KV cache, queries) or scaled and rounded to fp32 (head weights, external
features).  Any slice of a tensor can therefore be regenerated on the host from
its linear element offsets without holding the whole tensor.
"""
from __future__ import annotations

import ctypes
import functools
import os
from typing import Optional

import numpy as np

GOLD = 0x9E3779B97F4A7C15
_M1 = 0xBF58476D1CE4E5B9
_M2 = 0x94D049BB133111EB
_MASK = (1 << 64) - 1

# stream ids (one per tensor kind)
STREAM_K, STREAM_V, STREAM_Q, STREAM_QFULL, STREAM_FEAT, STREAM_W1, STREAM_B1, STREAM_W2, \
    STREAM_B2, STREAM_FLAGS, STREAM_LENS, STREAM_TABLE = range(1, 13)


def _mix_int(x: int) -> int:
    x &= _MASK
    x = ((x ^ (x >> 30)) * _M1) & _MASK
    x = ((x ^ (x >> 27)) * _M2) & _MASK
    return x ^ (x >> 31)


def stream_key(seed: int, stream: int) -> int:
    return _mix_int(_mix_int(seed) ^ ((stream * GOLD) & _MASK))


def _mix_arr(x: np.ndarray) -> np.ndarray:
    with np.errstate(over="ignore"):
        x = (x ^ (x >> np.uint64(30))) * np.uint64(_M1)
        x = (x ^ (x >> np.uint64(27))) * np.uint64(_M2)
        return x ^ (x >> np.uint64(31))


def hash64(key: int, idx: np.ndarray) -> np.ndarray:
    idx = np.asarray(idx).astype(np.uint64)
    with np.errstate(over="ignore"):
        return _mix_arr(np.uint64(key) + idx * np.uint64(GOLD))


def code16(key: int, idx: np.ndarray) -> np.ndarray:
    return (hash64(key, idx) >> np.uint64(48)).astype(np.uint16)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round-to-nearest-even fp32 -> bf16 bit patterns (finite inputs)."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.asarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


@functools.lru_cache(maxsize=None)
def _quantiles_f64() -> np.ndarray:
    from scipy.special import ndtri

    return ndtri((np.arange(65536, dtype=np.float64) + 0.5) / 65536.0)


@functools.lru_cache(maxsize=None)
def gauss_table_bf16() -> np.ndarray:
    """65,536 bf16 bit patterns: the N(0,1) quantile of each 16-bit code."""
    t = f32_to_bf16_bits(_quantiles_f64().astype(np.float32))
    t.setflags(write=False)
    return t


def gauss_bf16(key: int, idx: np.ndarray) -> np.ndarray:
    """bf16 bit patterns ~ N(0,1) for the given linear element offsets."""
    return gauss_table_bf16()[code16(key, idx)]


def gauss_f32(key: int, idx: np.ndarray, std: float = 1.0) -> np.ndarray:
    return (_quantiles_f64()[code16(key, idx)] * std).astype(np.float32)


def gauss_bf16_tensor(seed: int, stream: int, shape, offset: int = 0) -> np.ndarray:
    n = int(np.prod(shape))
    return gauss_bf16(stream_key(seed, stream), np.arange(offset, offset + n, dtype=np.uint64)).reshape(shape)


def gauss_f32_tensor(seed: int, stream: int, shape, std: float = 1.0, offset: int = 0) -> np.ndarray:
    n = int(np.prod(shape))
    return gauss_f32(stream_key(seed, stream), np.arange(offset, offset + n, dtype=np.uint64), std).reshape(shape)


def bernoulli_flags(seed: int, step: int, batch: int, rate: float) -> np.ndarray:
    """Forced recall flags: request b at step k recalls iff a 24-bit hash < rate * 2^24."""
    idx = np.arange(batch, dtype=np.uint64) + np.uint64(step) * np.uint64(max(batch, 1))
    h = hash64(stream_key(seed, STREAM_FLAGS), idx) >> np.uint64(40)
    thr = np.uint64(min(max(int(round(rate * (1 << 24))), 0), 1 << 24))
    return (h < thr).astype(np.uint8)


def periodic_flags(step: int, batch: int, first_k: int, period: int = 16) -> np.ndarray:
    """Prescribed schedule: recall on the first `first_k` steps of every `period` steps."""
    return np.full(batch, 1 if (step % period) < first_k else 0, dtype=np.uint8)


def uniform_lengths(seed: int, batch: int, lo: int, hi: int) -> np.ndarray:
    """Per-request context lengths, uniform on [lo, hi]."""
    h = hash64(stream_key(seed, STREAM_LENS), np.arange(batch, dtype=np.uint64))
    return (lo + (h % np.uint64(hi - lo + 1)).astype(np.int64)).astype(np.int32)


def block_tables(seed: int, blocks_needed: np.ndarray, max_blocks_per_seq: int, shuffled: bool,
                 num_blocks: Optional[int] = None) -> tuple[np.ndarray, int]:
    """block_table [B, max_blocks_per_seq] (unused entries -1) and the pool size.

    Contiguous: request b owns consecutive physical blocks.  Shuffled: a seeded
    permutation of the pool (Fisher-Yates, numpy's), so logically adjacent pages
    are physically scattered and interleaved between requests.
    """
    blocks_needed = np.asarray(blocks_needed, dtype=np.int64)
    total = int(blocks_needed.sum())
    pool = total if num_blocks is None else num_blocks
    assert pool >= total and max_blocks_per_seq >= (blocks_needed.max() if len(blocks_needed) else 0)
    ids = np.arange(pool, dtype=np.int32)
    if shuffled:
        ids = np.random.RandomState(seed & 0x7FFFFFFF).permutation(pool).astype(np.int32)
    table = np.full((len(blocks_needed), max_blocks_per_seq), -1, dtype=np.int32)
    pos = 0
    for b, n in enumerate(blocks_needed):
        table[b, :n] = ids[pos:pos + n]
        pos += int(n)
    return table, pool


def kv_offsets(layer_stride: int, block_stride: int, token_stride: int, head_stride: int,
               kv_layer: int, blocks: np.ndarray, kv_head: int, block_size: int,
               head_dim: int) -> np.ndarray:
    """Linear element offsets [len(blocks), block_size, head_dim] of one (layer, kv head) slice."""
    blocks = np.asarray(blocks, dtype=np.int64)
    return (kv_layer * layer_stride + blocks[:, None, None] * block_stride + kv_head * head_stride
            + np.arange(block_size, dtype=np.int64)[None, :, None] * token_stride
            + np.arange(head_dim, dtype=np.int64)[None, None, :]).astype(np.uint64)


# ---------------------------------------------------------------- device side
_HERE = os.path.dirname(os.path.abspath(__file__))
_FILL_LIB = os.path.join(_HERE, "libsynth_fill.so")
_fill = None


def _fill_lib():
    global _fill
    if _fill is None:
        if not os.path.exists(_FILL_LIB):
            raise RuntimeError(f"{_FILL_LIB} is missing: run __graft_entry__.build() first")
        _fill = ctypes.CDLL(_FILL_LIB)
        _fill.synth_fill_bf16.restype = ctypes.c_int
        _fill.synth_fill_bf16.argtypes = [ctypes.c_void_p, ctypes.c_int64, ctypes.c_uint64,
                                          ctypes.c_int64, ctypes.c_void_p, ctypes.c_void_p]
    return _fill


_dev_tables = {}


def fill_bf16_device(tensor, seed: int, stream: int, offset: int = 0) -> None:
    """Fill a contiguous CUDA bf16 tensor with the same bits gauss_bf16() yields for
    linear offsets offset .. offset + numel - 1 of (seed, stream)."""
    import torch

    assert tensor.is_cuda and tensor.dtype == torch.bfloat16 and tensor.is_contiguous()
    dev = tensor.device.index
    if dev not in _dev_tables:
        tab = torch.from_numpy(gauss_table_bf16().view(np.int16).copy()).to(tensor.device)
        _dev_tables[dev] = tab
    with torch.cuda.device(dev):
        rc = _fill_lib().synth_fill_bf16(
            tensor.data_ptr(), tensor.numel(), stream_key(seed, stream), offset,
            _dev_tables[dev].data_ptr(), torch.cuda.current_stream().cuda_stream)
    if rc:
        raise RuntimeError(f"synth_fill_bf16 failed with CUDA error {rc}")


def bf16_bits_to_torch(bits: np.ndarray, device=None):
    import torch

    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16)).view(torch.bfloat16)
    return t if device is None else t.to(device)


def torch_to_bf16_bits(t) -> np.ndarray:
    import torch

    return t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
