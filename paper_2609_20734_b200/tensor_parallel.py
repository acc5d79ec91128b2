"""KV-head tensor parallelism for one decode step (Algorithm 1 sharded over attention heads).

Rank r of n owns KV heads [r*Hkv/n, (r+1)*Hkv/n), the query heads of their groups and the matching
columns of the recall head's first layer.  Attention needs no exchange: heads are independent.
The decision needs one: every rank multiplies its columns of W1 by its slice of the head input,
the [batch, d_hidden] products are summed over the ranks (the step's only collective), and every
rank applies bias, SiLU, the second layer and the decision rule to the same sums, so all ranks
gate the same requests.  Argument marshalling only: the arithmetic runs in the library's kernels
and the collective in torch.distributed.
"""
from __future__ import annotations

from dataclasses import dataclass


@dataclass(frozen=True)
class HeadShard:
    """What one rank owns."""
    rank: int
    world: int
    kv_heads: int          # KV heads on this rank
    q_heads: int           # query heads on this rank
    kv_head_begin: int     # first global KV head
    q_head_begin: int      # first global query head
    d_ext: int             # external head features this rank multiplies (rank 0 owns them all)
    col_begin: int         # first column of W1 this rank multiplies
    col_count: int         # number of columns
    d_in: int              # full row length of W1


def head_shard(rank: int, world: int, num_q_heads: int, num_kv_heads: int, head_dim: int,
               d_ext: int = 0, use_attn_out: bool = True) -> HeadShard:
    """Contiguous split of the KV heads; the head input is [feat_ext ; attention heads in order]."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("rank outside [0, world)")
    if num_kv_heads % world or num_q_heads % num_kv_heads:
        raise ValueError("KV heads must divide evenly over the ranks, and query heads over KV heads")
    kv = num_kv_heads // world
    g = num_q_heads // num_kv_heads
    q = kv * g
    d_attn = num_q_heads * head_dim if use_attn_out else 0
    own_ext = d_ext if rank == 0 else 0
    attn_cols = q * head_dim if use_attn_out else 0
    col_begin = 0 if rank == 0 else d_ext + rank * attn_cols
    return HeadShard(rank, world, kv, q, rank * kv, rank * q, own_ext, col_begin, own_ext + attn_cols,
                     d_ext + d_attn)


def sum_over_ranks(t, group=None):
    """The step's one collective: element-wise sum of a small fp32 tensor over the ranks."""
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized():
        dist.all_reduce(t, op=dist.ReduceOp.SUM, group=group)   # a one-rank group reduces to itself
    return t


def tp_local_and_preact(ctx, shard: HeadShard, batch, q_local, k_cache, v_cache, block_table, seq_lens, out,
                        *, W1, pre, feat_ext=None, lse=None):
    """Before the exchange: the Local pass over the rank's heads, then the rank's share of W1 x."""
    L = ctx.cfg.num_layers
    ctx.local_decode(0, L, batch, q_local, k_cache, v_cache, block_table, seq_lens, out, lse)
    gated = [l for l in range(L) if ctx.cfg.layer_gated[l]]
    # the head reads the Local output of the last gated layer, as the single-GPU step does
    attn_last = out[gated[-1]] if (ctx.cfg.head_use_attn_out and gated) else None
    ctx.recall_preact(batch, feat_ext if shard.d_ext else None, attn_last,
                      W1.data_ptr() + 4 * shard.col_begin, shard.d_in, pre)


def tp_decide_and_recompute(ctx, batch, q_full, k_cache, v_cache, block_table, seq_lens, out, *, pre_sum,
                            b1, w2, b2, threshold, scores, flags, logits=None, lse=None,
                            override_flags=None, counters=None):
    """After the exchange: the decision from the summed products, then the gated Full pass."""
    ctx.recall_finalize(batch, pre_sum, b1, w2, b2, threshold, override_flags, scores, logits, flags, counters)
    ctx.full_decode_gated(0, ctx.cfg.num_layers, batch, q_full, k_cache, v_cache, block_table, seq_lens,
                          flags, out, lse)


def tp_step(ctx, shard: HeadShard, batch, q_local, k_cache, v_cache, block_table, seq_lens, out, *,
            W1, b1, w2, b2, threshold, pre, scores, flags, feat_ext=None, q_full=None, logits=None,
            lse=None, override_flags=None, counters=None, all_reduce=sum_over_ranks):
    """One decode step on one rank.  `ctx` was created with the rank's head counts (and head_d_ext =
    shard.d_ext); caches, q and out hold the rank's heads only; W1 is the full [d_hidden, d_in]
    matrix (each rank reads only its columns).  `pre` is a [batch, d_hidden] fp32 device buffer.
    """
    tp_local_and_preact(ctx, shard, batch, q_local, k_cache, v_cache, block_table, seq_lens, out,
                        W1=W1, pre=pre, feat_ext=feat_ext, lse=lse)
    all_reduce(pre)
    tp_decide_and_recompute(ctx, batch, q_local if q_full is None else q_full, k_cache, v_cache, block_table,
                            seq_lens, out, pre_sum=pre, b1=b1, w2=w2, b2=b2, threshold=threshold,
                            scores=scores, flags=flags, logits=logits, lse=lse,
                            override_flags=override_flags, counters=counters)
    return flags


# ---- sequence sharding of the gated Full pass ------------------------------------------------
def sequence_shard(rank: int, world: int, seq_len: int, page: int = 16):
    """Contiguous split of a request's ceil(seq_len / page) pages over the ranks, as even as whole
    pages allow.  Returns (first page, end page, positions held); short requests leave the last
    ranks empty."""
    if world < 1 or not 0 <= rank < world:
        raise ValueError("rank outside [0, world)")
    pages = (int(seq_len) + page - 1) // page
    lo = (rank * pages + world - 1) // world
    hi = ((rank + 1) * pages + world - 1) // world
    held = max(0, min(int(seq_len), hi * page) - lo * page)
    return lo, hi, held


def gather_over_ranks(dst, src, group=None):
    """All-gather of equally shaped tensors into dst[rank] (dst has a leading world axis)."""
    import torch.distributed as dist

    if dist.is_available() and dist.is_initialized():
        dist.all_gather(list(dst.unbind(0)), src, group=group)   # dst[r] are contiguous views
    else:
        dst.copy_(src.reshape(dst.shape))
    return dst


def sp_full_step(ctx, world, batch, q_full, k_cache, v_cache, block_table_local, seq_lens_local, part_tokens,
                 flags, part_out, part_lse, parts_out, parts_lse, out, lse=None, gather=gather_over_ranks):
    """Gated Full pass of one rank of a sequence-sharded cache, then the exchange and the merge.
    The context is created with allow_empty = 1; block_table_local / seq_lens_local describe the
    positions this rank holds; part_tokens [world, batch] i32 holds every rank's counts; part_out /
    part_lse are this rank's [L, batch, Hq, D] / [L, batch, Hq] results and parts_* their gathered
    [world, ...] forms.  out / lse receive the whole-history rows of flagged requests."""
    L = ctx.cfg.num_layers
    ctx.full_decode_gated(0, L, batch, q_full, k_cache, v_cache, block_table_local, seq_lens_local, flags,
                          part_out, part_lse)
    gather(parts_out, part_out)
    gather(parts_lse, part_lse)
    ctx.merge_partials(world, 0, L, batch, parts_out, parts_lse, flags, out, lse, part_tokens=part_tokens)


# ---- the decision's exchange fused into the kernel (no collective call) ------------------------
class ExchangeBuffers:
    """Receive buffers and arrival flags of every rank of a group, as the library wants them: in
    rank order, each entry a tensor (ranks living in this process) or a raw device address (a
    peer's buffer mapped into this GPU's address space).  `epoch` counts the exchanges."""

    def __init__(self, recv, arrived, keep=None):
        self.recv, self.arrived, self.keep, self.epoch = recv, arrived, keep, 0

    @classmethod
    def local(cls, world, batch, d_hidden, device="cuda"):
        """All ranks in this process on one GPU: for checking the protocol with one cooperative launch."""
        import torch

        recv = [torch.zeros((2, world, batch, d_hidden), device=device) for _ in range(world)]
        arrived = [torch.zeros(world, dtype=torch.int32, device=device) for _ in range(world)]
        return cls(recv, arrived)

    @classmethod
    def symmetric(cls, group, batch, d_hidden, device="cuda"):
        """One rank per process and GPU: buffers in torch's symmetric memory, peers' addresses from
        its rendezvous.  Not tested on a GPU (this build had one): the addresses are used for plain
        peer stores only, never as the source of a copy-engine or tensor-map load."""
        import torch
        import torch.distributed as dist
        import torch.distributed._symmetric_memory as symm

        world = dist.get_world_size(group)
        recv = symm.empty((2, world, batch, d_hidden), dtype=torch.float32, device=device)
        arrived = symm.empty((world,), dtype=torch.int32, device=device)
        recv.zero_()
        arrived.zero_()
        h_recv = symm.rendezvous(recv, group)
        h_arr = symm.rendezvous(arrived, group)
        dist.barrier(group)    # every rank's flags are zero before the first exchange
        return cls([int(p) for p in h_recv.buffer_ptrs], [int(p) for p in h_arr.buffer_ptrs],
                   keep=(recv, arrived, h_recv, h_arr))

    def next_epoch(self):
        self.epoch += 1
        return self.epoch


def tp_step_fused(ctx, shard: HeadShard, batch, q_local, k_cache, v_cache, block_table, seq_lens, out, *,
                  W1, b1, w2, b2, threshold, pre, scores, flags, buffers: ExchangeBuffers, feat_ext=None,
                  q_full=None, logits=None, lse=None, override_flags=None, counters=None, timeout_ns=0):
    """tp_step with the all-reduce replaced by the library's own exchange kernel: Local pass, the rank's
    share of W1 x, then ONE kernel that pushes the share to every peer, waits for theirs and decides, then
    the gated Full pass.  Every rank of the group must make this call once per step."""
    tp_local_and_preact(ctx, shard, batch, q_local, k_cache, v_cache, block_table, seq_lens, out,
                        W1=W1, pre=pre, feat_ext=feat_ext, lse=lse)
    ctx.recall_finalize_exchange(batch, shard.world, shard.rank,
                                 [dict(pre_local=pre, scores=scores, logits=logits, flags=flags, counters=counters)],
                                 buffers.recv, buffers.arrived, buffers.next_epoch(), b1, w2, b2, threshold,
                                 override_flags=override_flags, timeout_ns=timeout_ns)
    ctx.full_decode_gated(0, ctx.cfg.num_layers, batch, q_local if q_full is None else q_full, k_cache, v_cache,
                          block_table, seq_lens, flags, out, lse)
    return flags


# ---- the sequence-sharded Full pass with the exchange inside the merge kernel ------------------
MERGE_BLOCKS = 64    # row blocks (and arrival flags per rank) of the fused exchange + merge


class MergeExchangeBuffers(ExchangeBuffers):
    """Receive buffers (partial rows and their log-sum-exps, two parities) and per-block arrival
    flags of every rank, in rank order; entries as in ExchangeBuffers."""

    def __init__(self, recv_out, recv_lse, arrived, keep=None):
        self.recv_out, self.recv_lse, self.arrived, self.keep, self.epoch = recv_out, recv_lse, arrived, keep, 0

    @classmethod
    def local(cls, world, num_layers, batch, q_heads, head_dim, device="cuda"):
        import torch

        rows = num_layers * batch * q_heads
        return cls([torch.zeros((2, world, rows, head_dim), device=device) for _ in range(world)],
                   [torch.zeros((2, world, rows), device=device) for _ in range(world)],
                   [torch.zeros((world, MERGE_BLOCKS), dtype=torch.int32, device=device) for _ in range(world)])

    @classmethod
    def symmetric(cls, group, num_layers, batch, q_heads, head_dim, device="cuda"):
        """One rank per process and GPU (torch's symmetric memory; plain peer stores only).  Not
        tested on a GPU: this build had one."""
        import torch
        import torch.distributed as dist
        import torch.distributed._symmetric_memory as symm

        world = dist.get_world_size(group)
        rows = num_layers * batch * q_heads
        bufs = [symm.empty((2, world, rows, head_dim), dtype=torch.float32, device=device),
                symm.empty((2, world, rows), dtype=torch.float32, device=device),
                symm.empty((world, MERGE_BLOCKS), dtype=torch.int32, device=device)]
        for t in bufs:
            t.zero_()
        hs = [symm.rendezvous(t, group) for t in bufs]
        dist.barrier(group)
        return cls(*[[int(p) for p in h.buffer_ptrs] for h in hs], keep=(bufs, hs))


def sp_full_step_fused(ctx, world, rank, batch, q_full, k_cache, v_cache, block_table_local, seq_lens_local, flags,
                       part_out, part_lse, out, lse=None, *, buffers: MergeExchangeBuffers, timeout_ns=0):
    """sp_full_step without a collective call: two launches, the gated Full pass over this rank's
    positions and the kernel that pushes its partial rows to the peers, waits for theirs block by
    block and merges.  seq_lens_local doubles as this rank's token counts."""
    L = ctx.cfg.num_layers
    ctx.full_decode_gated(0, L, batch, q_full, k_cache, v_cache, block_table_local, seq_lens_local, flags,
                          part_out, part_lse)
    ctx.merge_partials_exchange(world, rank, [dict(part_out=part_out, part_lse=part_lse, tokens_local=seq_lens_local,
                                                   flags=flags, out=out, lse=lse)],
                                buffers.recv_out, buffers.recv_lse, buffers.arrived, buffers.next_epoch(), 0, L, batch,
                                timeout_ns=timeout_ns)

