"""Sharded routing step over several GPUs: plumbing only (bounds, buffers, pointer tables, collectives).

One process per GPU.  Vocabulary sharding (decode batches): rank g keeps rows [v0, v1) of W on its GPU.
  * VocabShardedRouter: tlr_shard_summary, one all-gather of the 16-byte per-row summaries (n x 16 bytes per
    rank; NCCL on GPUs), tlr_shard_finish on the gathered block -- every rank ends with the full decision.
  * FusedVocabShardedRouter: the exchange fused into the kernels -- tlr_shard_push stores the summaries
    straight into every peer's exchange block and sets a flag there, tlr_shard_finish_fused waits for the
    flags on the device.  No collective call on the data path.
Row sharding (prefill batches): every rank routes its own rows; exchange_routed / merge_routed turn the
ranks' index lists into one list of global row numbers (an all-gather of counts and lists, one small kernel).
All arithmetic is in the library's kernels.
"""
from __future__ import annotations

import torch

from . import binding as B

GRANULE = 32          # shard boundaries fall on multiples of this many vocabulary rows


def shard_bounds(V: int, world: int, rank: int):
    """Contiguous, near-equal split of [0, V) at multiples of GRANULE rows: rows [v0, v1) of rank `rank`."""
    if not (0 <= rank < world) or V <= 0:
        raise ValueError("bad shard request")
    granules = (V + GRANULE - 1) // GRANULE
    if granules < world:
        raise ValueError("vocabulary too small for %d shards" % world)
    g0 = granules * rank // world
    g1 = granules * (rank + 1) // world
    return g0 * GRANULE, min(V, g1 * GRANULE)


def gather_summaries(local: torch.Tensor, group=None) -> torch.Tensor:
    """All-gather of the per-row summaries: local [n, 4] (16 bytes per row) -> [world, n, 4], rank-major."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    out = torch.empty((world,) + tuple(local.shape), dtype=local.dtype, device=local.device)
    dist.all_gather(list(out.unbind(0)), local.contiguous(), group=group)     # slot g = rank g's rows
    return out


class VocabShardedRouter:
    """Owner of one rank's context (on its rows of W), its summary buffers and the output tensors."""

    def __init__(self, W_shard: torch.Tensor, v_offset: int, max_n: int, world: int, group=None, wscale=None):
        """W_shard: this rank's rows of W, bf16 [V_local, d]; or, with wscale (float32 [V_local]), their e4m3 codes
        (decode batches of up to 128 rows, see tlr_create_fp8)."""
        fp8 = wscale is not None
        ok_dtype = W_shard.dtype in (torch.uint8, torch.float8_e4m3fn) if fp8 else W_shard.dtype == torch.bfloat16
        if not (W_shard.is_cuda and ok_dtype and W_shard.dim() == 2 and W_shard.is_contiguous()):
            raise ValueError("W_shard must be a contiguous CUDA [V_local, d] tensor, bf16 or (with wscale) e4m3 codes")
        self.W = W_shard
        self.wscale = wscale
        self.v_offset = int(v_offset)
        self.world = int(world)
        self.group = group
        self.max_n = max_n
        dev = W_shard.device
        with torch.cuda.device(dev):
            if fp8:
                self.ctx = B.tlr_create_fp8(W_shard.shape[1], W_shard.shape[0], W_shard, wscale, max_n)
            else:
                self.ctx = B.tlr_create(W_shard.shape[1], W_shard.shape[0], W_shard, max_n)
            self.summary = torch.empty((max_n, 4), dtype=torch.float32, device=dev)     # 16 bytes per row
            self.token = torch.empty(max_n, dtype=torch.int32, device=dev)
            self.conf = torch.empty(max_n, dtype=torch.float32, device=dev)
            self.entropy = torch.empty(max_n, dtype=torch.float32, device=dev)
            self.route_mask = torch.empty(max_n, dtype=torch.uint8, device=dev)
            self.routed_idx = torch.empty(max_n, dtype=torch.int32, device=dev)
            self.routed_count = torch.zeros(1, dtype=torch.int32, device=dev)

    def summarize(self, h: torch.Tensor, stream=None) -> torch.Tensor:
        n = h.shape[0]
        B.tlr_shard_summary(self.ctx, h, n, self.v_offset, self.summary, stream)
        return self.summary[:n]

    def finish(self, gathered: torch.Tensor, n: int, tau: float, stream=None):
        B.tlr_shard_finish(self.ctx, gathered, gathered.shape[0], n, tau, self.token, self.conf, self.entropy,
                           self.route_mask, self.routed_idx, self.routed_count, stream)
        return (self.token[:n], self.conf[:n], self.entropy[:n], self.route_mask[:n], self.routed_idx,
                self.routed_count)

    def route(self, h: torch.Tensor, tau: float):
        """Summary on this rank's shard, all-gather over the group, merge and decision on every rank."""
        n = h.shape[0]
        local = self.summarize(h)
        gathered = gather_summaries(local, self.group) if self.world > 1 else local.unsqueeze(0)
        return self.finish(gathered.contiguous(), n, tau)

    def close(self):
        if self.ctx is not None:
            B.tlr_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def symmetric_exchange_block(max_n: int, world: int, group=None):
    """One exchange block per rank in symmetric memory (every rank can store into every other rank's block).
    Returns (this rank's block as a uint8 tensor, zeroed; the device addresses of all ranks' blocks).
    Collective over the group.  Not exercised on more than one GPU by this repository's tests."""
    import torch.distributed as dist
    import torch.distributed._symmetric_memory as symm
    nbytes = B.tlr_shard_block_bytes(max_n, world)
    block = symm.empty(nbytes, dtype=torch.uint8, device=torch.device("cuda", torch.cuda.current_device()))
    block.zero_()
    handle = symm.rendezvous(block, group=group if group is not None else dist.group.WORLD)
    torch.cuda.synchronize()
    dist.barrier(group)                      # every block is zero before anyone's first push
    return block, [int(p) for p in handle.buffer_ptrs]


class FusedVocabShardedRouter:
    """One rank of the vocabulary-sharded step with the fused exchange: its context (on its rows of W), attached
    to the ranks' exchange blocks, and the output tensors."""

    def __init__(self, W_shard: torch.Tensor, v_offset: int, max_n: int, rank: int, world: int, peer_blocks,
                 wscale=None, keep=None):
        """peer_blocks: device addresses (or tensors) of all ranks' zeroed exchange blocks, entry `rank` this
        rank's own (see symmetric_exchange_block); `keep` is anything that must stay alive with them."""
        fp8 = wscale is not None
        self.W, self.wscale, self.keep = W_shard, wscale, keep
        self.v_offset, self.rank, self.world, self.max_n = int(v_offset), int(rank), int(world), max_n
        dev = W_shard.device
        with torch.cuda.device(dev):
            if fp8:
                self.ctx = B.tlr_create_fp8(W_shard.shape[1], W_shard.shape[0], W_shard, wscale, max_n)
            else:
                self.ctx = B.tlr_create(W_shard.shape[1], W_shard.shape[0], W_shard, max_n)
            B.tlr_shard_attach(self.ctx, self.rank, self.world, peer_blocks)
            self.token = torch.empty(max_n, dtype=torch.int32, device=dev)
            self.conf = torch.empty(max_n, dtype=torch.float32, device=dev)
            self.entropy = torch.empty(max_n, dtype=torch.float32, device=dev)
            self.route_mask = torch.empty(max_n, dtype=torch.uint8, device=dev)
            self.routed_idx = torch.empty(max_n, dtype=torch.int32, device=dev)
            self.routed_count = torch.zeros(1, dtype=torch.int32, device=dev)

    def push(self, h: torch.Tensor, stream=None):
        B.tlr_shard_push(self.ctx, h, h.shape[0], self.v_offset, stream)

    def finish(self, n: int, tau: float, stream=None):
        B.tlr_shard_finish_fused(self.ctx, n, tau, self.token, self.conf, self.entropy, self.route_mask,
                                 self.routed_idx, self.routed_count, stream)
        return (self.token[:n], self.conf[:n], self.entropy[:n], self.route_mask[:n], self.routed_idx,
                self.routed_count)

    def route(self, h: torch.Tensor, tau: float, stream=None):
        self.push(h, stream)
        return self.finish(h.shape[0], tau, stream)

    def close(self):
        if self.ctx is not None:
            B.tlr_destroy(self.ctx)
            self.ctx = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass


def row_offsets(rows_per_rank):
    """Global number of every rank's first row: the exclusive running sum of the ranks' row counts."""
    out, total = [], 0
    for r in rows_per_rank:
        out.append(total)
        total += int(r)
    return out


def exchange_routed(routed_idx: torch.Tensor, routed_count: torch.Tensor, n_local: int, group=None):
    """Row-sharded batches, the exchange: every rank contributes its routed_idx (capacity `cap` = its length, the
    same on every rank), its routed_count and its number of rows.  Returns (gathered_idx [world, cap],
    counts [world], offsets [world]), all int32 on routed_idx's device, the same on every rank."""
    import torch.distributed as dist
    world = dist.get_world_size(group)
    cap = routed_idx.shape[0]
    gathered = torch.empty((world, cap), dtype=torch.int32, device=routed_idx.device)
    dist.all_gather(list(gathered.unbind(0)), routed_idx.contiguous(), group=group)
    meta = torch.empty((world, 2), dtype=torch.int32, device=routed_idx.device)
    mine = torch.stack([routed_count.reshape(()).to(torch.int32),
                        torch.tensor(n_local, dtype=torch.int32, device=routed_idx.device)])
    dist.all_gather(list(meta.unbind(0)), mine, group=group)
    counts = meta[:, 0].contiguous()
    offsets = torch.tensor(row_offsets(meta[:, 1].tolist()), dtype=torch.int32, device=routed_idx.device)
    return gathered, counts, offsets


def merge_routed(gathered: torch.Tensor, counts: torch.Tensor, offsets: torch.Tensor, stream=None):
    """Row-sharded batches, the merge (one kernel): the global ascending list of routed rows and its length."""
    world, cap = gathered.shape
    out = torch.empty(world * cap, dtype=torch.int32, device=gathered.device)
    total = torch.zeros(1, dtype=torch.int32, device=gathered.device)
    B.tlr_rows_merge(gathered, counts, offsets, world, cap, out, total, stream)
    return out, total
