"""Synthetic workloads shaped like the five benchmark configurations (shapes, lengths,
block-table structure, recall schedules).  Input description only: no arithmetic of the
attention method lives here.  Device tensors come from synth.fill_bf16_device, host slices
for a checker are regenerated from the same counters, so a 100-GB cache never has to exist
on the host.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Optional

import numpy as np

from . import synth

BASE_SEED = 20734
P = 16


@dataclass
class Workload:
    name: str
    L: int
    B: int
    Hq: int
    Hkv: int
    D: int
    windows: list
    sinks: list
    gated: list
    seq_lens0: np.ndarray            # context per request at step 0, current token included
    steps: int
    kv_index: Optional[list] = None  # layer -> physical cache layer (aliasing for huge stacks)
    shuffled: bool = False
    layout: str = "hnd"
    head: Optional[tuple] = None     # (d_ext, use_attn_out, d_hidden)
    recall_rate: float = 0.25
    schedule: str = "bernoulli"      # "bernoulli" | "periodic" | "head"
    seed: int = BASE_SEED
    threshold: float = 0.5
    reuse_local: bool = False        # gated pass reads only S^F \ S^L (valid here: q_full == q_local)

    @property
    def G(self):
        return self.Hq // self.Hkv

    @property
    def phys_layers(self):
        return self.L if self.kv_index is None else max(self.kv_index) + 1

    @property
    def blocks_needed(self):
        return (np.asarray(self.seq_lens0, dtype=np.int64) + self.steps + P - 1) // P

    @property
    def max_blocks_per_seq(self):
        return int(self.blocks_needed.max())

    @property
    def kv_token_bytes(self):
        """K and V bytes of one token of one layer (all KV heads)."""
        return 2 * self.Hkv * self.D * 2

    def strides(self, num_blocks):
        if self.layout == "hnd":   # [layers, blocks, kv_heads, P, D]
            return dict(layer=num_blocks * self.Hkv * P * self.D, block=self.Hkv * P * self.D,
                        token=self.D, head=P * self.D)
        return dict(layer=num_blocks * self.Hkv * P * self.D, block=self.Hkv * P * self.D,
                    token=self.Hkv * self.D, head=self.D)

    def tables(self):
        return synth.block_tables(self.seed, self.blocks_needed, self.max_blocks_per_seq, self.shuffled)

    def local_tokens(self, l, t):
        return min(t, self.sinks[l] + self.windows[l])

    def algorithmic_bytes(self, seq_lens, flags):
        """KV bytes the method must read in one step: window (+sinks) for every layer and request,
        plus the whole history for flagged requests on gated layers."""
        kb = self.kv_token_bytes
        local = sum(self.local_tokens(l, int(t)) for l in range(self.L) for t in seq_lens) * kb
        full = sum(int(t) - (self.local_tokens(l, int(t)) if self.reuse_local else 0)
                   for l in range(self.L) if self.gated[l] for t, f in zip(seq_lens, flags) if f) * kb
        return local, full

    def override_flags(self, step):
        if self.schedule == "bernoulli":
            return synth.bernoulli_flags(self.seed, step, self.B, self.recall_rate)
        if self.schedule == "periodic":
            return synth.periodic_flags(step, self.B, int(round(self.recall_rate * 16)))
        return None

    def q_host(self, step, which="local"):
        n = self.L * self.B * self.Hq * self.D
        stream = synth.STREAM_Q if which == "local" else synth.STREAM_QFULL
        return synth.gauss_bf16_tensor(self.seed, stream, (self.L, self.B, self.Hq, self.D), offset=step * n)

    def feat_host(self, step):
        d_ext = self.head[0] if self.head else 0
        if not d_ext:
            return None
        return synth.gauss_f32_tensor(self.seed, synth.STREAM_FEAT, (self.B, d_ext), offset=step * self.B * d_ext)

    def head_host(self):
        if not self.head:
            return None
        d_ext, use_attn, d_h = self.head
        d_in = d_ext + (self.Hq * self.D if use_attn and any(self.gated) else 0)
        return dict(W1=synth.gauss_f32_tensor(self.seed, synth.STREAM_W1, (d_h, d_in), std=0.02),
                    b1=synth.gauss_f32_tensor(self.seed, synth.STREAM_B1, (d_h,), std=0.02),
                    w2=synth.gauss_f32_tensor(self.seed, synth.STREAM_W2, (d_h,), std=0.02),
                    b2=synth.gauss_f32_tensor(self.seed, synth.STREAM_B2, (1,), std=0.02),
                    use_attn_out=use_attn)

    def host_unit(self, table, num_blocks, layer, b, g, t):
        """Compact host copy of what one (layer, request, kv head) unit reads: K/V bits of the
        request's first ceil(t/16) pages, as an HND cache with an identity block table."""
        st = self.strides(num_blocks)
        npg = (t + P - 1) // P
        kvl = layer if self.kv_index is None else self.kv_index[layer]
        offs = synth.kv_offsets(st["layer"], st["block"], st["token"], st["head"], kvl,
                                table[b, :npg], g, P, self.D)
        k = synth.gauss_bf16(synth.stream_key(self.seed, synth.STREAM_K), offs.reshape(-1))
        v = synth.gauss_bf16(synth.stream_key(self.seed, synth.STREAM_V), offs.reshape(-1))
        return k, v, np.arange(npg, dtype=np.int32)[None, :]


def _uniform(L, w, s, gated=1):
    return [w] * L, [s] * L, [gated] * L


def make(name: str, **ov) -> Workload:
    """The five benchmark configurations; keyword overrides shrink them for tests."""
    if name == "tiny":
        w, s, g = _uniform(1, 256, 4)
        wl = Workload("tiny", 1, 1, 4, 1, 64, w, s, g, np.array([2048], np.int32), 8,
                      head=(256, 1, 64), schedule="head")
    elif name == "llama8b":
        w, s, g = _uniform(32, 1024, 4)
        wl = Workload("llama8b", 32, 1, 32, 8, 128, w, s, g, np.array([32768], np.int32), 64)
    elif name == "batched":
        w, s, g = _uniform(32, 1024, 4)
        lens = synth.uniform_lengths(BASE_SEED, 16, 8192, 65536)
        wl = Workload("batched", 32, 16, 32, 8, 128, w, s, g, lens, 8, shuffled=True,
                      head=(0, 1, 256))
    elif name == "70b":
        w, s, g = _uniform(80, 2048, 4)
        wl = Workload("70b", 80, 4, 64, 8, 128, w, s, g, np.full(4, 131072, np.int32), 8,
                      kv_index=[l % 16 for l in range(80)], recall_rate=0.3)
    elif name == "hybrid":
        L = 48
        gated = [1 if l % 4 == 3 else 0 for l in range(L)]
        windows = [1024 if gated[l] else 512 for l in range(L)]
        sinks = [4 if gated[l] else 0 for l in range(L)]
        # fixed-window layers share 3 physical slices, gated layers get one each
        kv_index, ng = [], 0
        for l in range(L):
            if gated[l]:
                kv_index.append(3 + ng)
                ng += 1
            else:
                kv_index.append(l % 4)
        wl = Workload("hybrid", L, 4, 32, 8, 128, windows, sinks, gated,
                      np.full(4, 262144, np.int32), 8, kv_index=kv_index, head=(0, 1, 256),
                      recall_rate=0.15)
    elif name == "paper":
        # The paper's timing workload: batch 1, s=4 sinks + w=2048 window, one prompt per length
        # (4,139 ... 516,788 tokens) and a prescribed first-k-of-16 schedule.  The attention shape
        # is Qwen3-1.7B's public configuration (28 layers, 16 query / 8 KV heads, head_dim 128);
        # the paper itself only states the hidden size.
        w, s, g = _uniform(28, 2048, 4)
        wl = Workload("paper", 28, 1, 16, 8, 128, w, s, g, np.array([128852], np.int32), 16,
                      schedule="periodic", recall_rate=0.125)
    else:
        raise KeyError(name)
    return replace(wl, **ov) if ov else wl


def full_head_layout(d_model: int, d_tower: int, d_ff: int, n_blocks: int):
    """(name, shape) of the parameters of the paper's recall head in storage order: three towers
    (norm gain, weight, bias), the fusion projection, the SwiGLU blocks (norm gain, gate, up, down),
    the output norm gain, output vector and output bias."""
    out = []
    for i in range(3):
        out += [(f"g{i}", (d_model,)), (f"W{i}", (d_tower, d_model)), (f"b{i}", (d_tower,))]
    out += [("Wf", (d_tower, 9 * d_tower)), ("bf", (d_tower,))]
    for k in range(n_blocks):
        out += [(f"bg{k}", (d_tower,)), (f"Wg{k}", (d_ff, d_tower)), (f"Wu{k}", (d_ff, d_tower)),
                (f"Wd{k}", (d_tower, d_ff))]
    out += [("go", (d_tower,)), ("w", (d_tower,)), ("bias", (1,))]
    return out


def full_head_params(seed: int, d_model: int, d_tower: int, d_ff: int, n_blocks: int) -> np.ndarray:
    """Random-init parameters of the paper's head as one flat fp32 array: weights ~ N(0, 1/fan_in),
    biases ~ N(0, 0.1^2), norm gains 1 + N(0, 0.1^2)."""
    parts = []
    for i, (name, shape) in enumerate(full_head_layout(d_model, d_tower, d_ff, n_blocks)):
        std = 1.0 / np.sqrt(shape[-1]) if len(shape) == 2 else 0.1
        x = synth.gauss_f32_tensor(seed, 200 + i, shape, std=std)
        if name.startswith("g") or name.startswith("bg"):
            x = (1.0 + x).astype(np.float32)
        parts.append(x.reshape(-1))
    return np.concatenate(parts)


def full_head_input(seed: int, which: int, batch: int, d_model: int) -> np.ndarray:
    """Synthetic input of the paper's head: which = 0 preceding hidden state, 1 embedding, 2 Local
    hidden state; fp32 ~ N(0,1), [batch, d_model]."""
    return synth.gauss_f32_tensor(seed, 300 + which, (batch, d_model))


@dataclass
class DeviceState:
    wl: Workload
    table_host: np.ndarray
    num_blocks: int
    k_cache: object
    v_cache: object
    block_table: object
    seq_lens: object
    head: Optional[dict] = None
    extras: dict = field(default_factory=dict)


def materialize(wl: Workload, device="cuda") -> DeviceState:
    """Allocate and fill the device-resident state of a workload."""
    import torch

    table, nb = wl.tables()
    n = wl.phys_layers * nb * wl.Hkv * P * wl.D
    k = torch.empty(n, dtype=torch.bfloat16, device=device)
    v = torch.empty(n, dtype=torch.bfloat16, device=device)
    synth.fill_bf16_device(k, wl.seed, synth.STREAM_K)
    synth.fill_bf16_device(v, wl.seed, synth.STREAM_V)
    head = None
    hh = wl.head_host()
    if hh is not None:
        head = {kk: torch.from_numpy(np.ascontiguousarray(vv)).to(device) for kk, vv in hh.items()
                if kk != "use_attn_out"}
    return DeviceState(wl, table, nb, k, v, torch.from_numpy(table).to(device),
                       torch.from_numpy(np.asarray(wl.seq_lens0, dtype=np.int32)).to(device), head)


def q_device(wl: Workload, step: int, which="local", device="cuda"):
    import torch

    n = wl.L * wl.B * wl.Hq * wl.D
    q = torch.empty((wl.L, wl.B, wl.Hq, wl.D), dtype=torch.bfloat16, device=device)
    synth.fill_bf16_device(q, wl.seed, synth.STREAM_Q if which == "local" else synth.STREAM_QFULL,
                           offset=step * n)
    return q


def oda_config(wl: Workload, num_blocks: int, **kw):
    from .binding import OdaConfig

    st = wl.strides(num_blocks)
    d_ext, use_attn, d_h = wl.head if wl.head else (0, 0, 0)
    return OdaConfig(
        num_layers=wl.L, num_q_heads=wl.Hq, num_kv_heads=wl.Hkv, head_dim=wl.D, max_batch=wl.B,
        max_blocks_per_seq=wl.max_blocks_per_seq, layer_window=wl.windows, layer_sinks=wl.sinks,
        layer_gated=wl.gated, layer_kv_index=wl.kv_index, kv_layer_stride=st["layer"],
        kv_block_stride=st["block"], kv_token_stride=st["token"], kv_head_stride=st["head"],
        head_d_ext=d_ext, head_use_attn_out=use_attn, head_d_hidden=d_h,
        **{"reuse_local": int(wl.reuse_local), **kw})
