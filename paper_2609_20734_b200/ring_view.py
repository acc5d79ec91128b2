"""The Local workspace of the paper's runtime (appendix "Selected-state execution", paragraph on the
complete history and the Local workspace) as a variant: beside the complete paged history, every
request keeps a small second view that holds only what Local attention reads -- its sink positions
and a ring of the most recent positions -- and the commit of a step writes the selected K/V into both
views.

Here the second view is simply another paged cache with a periodic block table, so that the same
Local kernel reads it without a change:

  ring cache   [layers, B * (n_sink + R), kv_heads, 16, D]      (HND) -- R = window / 16 + 1 pages
  ring table   [B, max_blocks]: page p of request b ->  b * (n_sink + R) + (p if p < n_sink
                                                         else n_sink + (p - n_sink) mod R)

A window of w positions touches at most w / 16 + 1 consecutive pages, which the mod-R map sends to
distinct ring pages; position j + 16 R overwrites position j, which has left every window by then.
With s = 4 sinks and w = 2048 the view holds 16 + 129 * 16 slots per request and layer, of which at
most 4 + 2,047 committed positions plus the current one are live (the paper's 4 initial slots and
2,047-entry ring with the current candidate supplied separately).

Plumbing only: geometry, the table, and the initial copy of a prefix that already sits in the paged
history (index arithmetic and torch copies); attention and the per-step writes are the library's.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np

P = 16


@dataclass(frozen=True)
class RingGeometry:
    n_sink_pages: int      # pages that hold the sink positions (kept for ever)
    ring_pages: int        # R: pages of the ring of recent positions
    pages_per_request: int
    num_blocks: int        # blocks of the ring cache (all requests)


def geometry(batch: int, windows, sinks) -> RingGeometry:
    """Sized by the widest window / most sinks of the stack (the table is shared by all layers)."""
    n_sink = (max(sinks) + P - 1) // P
    ring = max(windows) // P + 1 + (1 if max(windows) % P else 0)
    per = n_sink + ring
    return RingGeometry(n_sink, ring, per, batch * per)


def ring_block(geo: RingGeometry, b: int, page: int) -> int:
    if page < geo.n_sink_pages:
        return b * geo.pages_per_request + page
    return b * geo.pages_per_request + geo.n_sink_pages + (page - geo.n_sink_pages) % geo.ring_pages


def table(geo: RingGeometry, batch: int, max_blocks: int) -> np.ndarray:
    """The periodic block table [batch, max_blocks] (does not depend on the lengths)."""
    pages = np.arange(max_blocks, dtype=np.int64)
    local = np.where(pages < geo.n_sink_pages, pages,
                     geo.n_sink_pages + (pages - geo.n_sink_pages) % geo.ring_pages)
    return (np.arange(batch, dtype=np.int64)[:, None] * geo.pages_per_request + local[None, :]).astype(np.int32)


def live_pages(geo: RingGeometry, t: int, window: int, sinks: int):
    """Logical pages whose ring copies a Local pass at length t reads (sinks, then the window)."""
    lo = max(0, t - window)
    pages = list(range(0, (min(sinks, t) + P - 1) // P)) + list(range(lo // P, (t + P - 1) // P))
    return sorted(set(pages))


def fill_from_paged(geo: RingGeometry, ring_k, ring_v, k_cache, v_cache, block_table_host, seq_lens_host,
                    windows, sinks, *, phys_layers: int, paged_blocks: int, kv_heads: int, head_dim: int):
    """Start-up copy: the pages a Local pass at the current lengths reads, from the paged history
    (HND, [phys_layers, paged_blocks, kv_heads, 16, D]) into the ring view.  torch indexing."""
    import torch

    pk = k_cache.view(phys_layers, paged_blocks, kv_heads * P * head_dim)
    pv = v_cache.view(phys_layers, paged_blocks, kv_heads * P * head_dim)
    rk = ring_k.view(phys_layers, geo.num_blocks, kv_heads * P * head_dim)
    rv = ring_v.view(phys_layers, geo.num_blocks, kv_heads * P * head_dim)
    src, dst = [], []
    for b, t in enumerate(np.asarray(seq_lens_host)):
        for page in live_pages(geo, int(t), max(windows), max(sinks)):
            src.append(int(block_table_host[b, page]))
            dst.append(ring_block(geo, b, page))
    src_t = torch.tensor(src, dtype=torch.long, device=k_cache.device)
    dst_t = torch.tensor(dst, dtype=torch.long, device=k_cache.device)
    rk[:, dst_t] = pk[:, src_t]
    rv[:, dst_t] = pv[:, src_t]
