"""A per-layer bank split over several GPUs (one part per rank), or over several parts on one GPU.

The paper's outlook (Sec. VI-E) names sharing one cache between devices as future work.  Here every rank holds
a slice of the slots and sees the whole batch of query fingerprints; a lookup is

    scan of the local slice  ->  all-reduce(max) of one 64-bit word per query  ->  decision (same on every rank)

and every computed miss is stored by exactly one rank (miss number m goes to rank m mod world).  Only argument
marshalling and the exchange live here: the scan, the decision, the row copies and the inserts are the
library's kernels (llmcache_shard_scan, llmcache_shard_decide, llmcache_commit).  The exchange uses
torch.distributed (NCCL between GPUs, gloo in the CPU tests); nothing here waits on another rank inside a
kernel.
"""
from __future__ import annotations

from typing import List, Optional

import torch

from . import binding as L

_TOP = -(1 << 63)          # the top bit of a 64-bit word, as a signed integer


def slice_bounds(n_total: int, world: int, rank: int):
    """Slots [first, first + count) of part `rank` when n_total slots are cut into `world` nearly equal parts
    (the first n_total % world parts have one slot more)."""
    base, extra = divmod(n_total, world)
    first = rank * base + min(rank, extra)
    return first, base + (1 if rank < extra else 0)


def misses_of(rank: int, world: int, n_miss: int) -> torch.Tensor:
    """Positions (in the ascending miss list) of the misses that part `rank` stores: rank, rank + world, ..."""
    return torch.arange(rank, max(n_miss, rank), world, dtype=torch.int64)


def combine_words(words: torch.Tensor, group=None) -> torch.Tensor:
    """Element-wise UNSIGNED maximum over all ranks of a tensor of packed 64-bit best words (held as int64), in
    place.  Collectives compare int64 as signed numbers, so the top bit is flipped before and after: that maps
    the unsigned order onto the signed one."""
    import torch.distributed as dist
    words.bitwise_xor_(_TOP)
    dist.all_reduce(words, op=dist.ReduceOp.MAX, group=group)
    words.bitwise_xor_(_TOP)
    return words


def unsigned_max_(a: torch.Tensor, b: torch.Tensor) -> torch.Tensor:
    """a = element-wise unsigned maximum of the int64 tensors a and b (what combine_words computes across ranks)."""
    torch.maximum(a ^ _TOP, b ^ _TOP, out=a)
    a.bitwise_xor_(_TOP)
    return a


class ShardedBank:
    """`parts` banks that together form one bank of n_total slots.

    Multi-GPU: every rank builds ShardedBank(n_total, world=W, ranks=[rank], ...) (one local part) and passes its
    process group; probe_fp then all-reduces the words.  Single GPU (tests): ranks=range(W) puts all parts on one
    device; they are scanned one after the other into the same words, which is the same maximum.
    """

    def __init__(self, n_total: int, world: int, ranks: List[int], *, device=0, group=None, **bank_kw):
        self.n_total, self.world, self.ranks, self.group = n_total, world, list(ranks), group
        self.distributed = group is not None or (len(self.ranks) == 1 and world > 1)
        self.parts, self.base = [], []
        for r in self.ranks:
            first, count = slice_bounds(n_total, world, r)
            self.base.append(first)
            self.parts.append(L.Bank(device=device, capacity=count, **bank_kw))
        self.device = self.parts[0].device

    def close(self):
        for p in self.parts:
            p.close()

    def probe_fp(self, bufs: L.ProbeBuffers, B: int, h_out: Optional[torch.Tensor] = None, tau=None, stream=None):
        """Lookup of the B query fingerprints in bufs.fp over the whole bank.  bufs receives hit flags, slots of the
        whole bank, scores, index lists and counts; h_out[b] the stored output of every hit whose slot a local part
        owns (between GPUs the rows of the other parts' hits are fetched from their owners by the caller)."""
        words = torch.zeros(max(B, 1), dtype=torch.int64, device=self.device)
        for p, first in zip(self.parts, self.base):
            L.llmcache_shard_scan(p.handle, bufs.fp, B, first, words, stream)
        if self.distributed:
            combine_words(words, self.group)
        for i, (p, first) in enumerate(zip(self.parts, self.base)):
            w = words if i == len(self.parts) - 1 else words.clone()     # the decision consumes its words
            L.llmcache_shard_decide(p.handle, w, B, tau, first, self.n_total, h_out, bufs.io, stream)
        return words

    def commit(self, miss_out: Optional[torch.Tensor], bufs: L.ProbeBuffers, h_out: Optional[torch.Tensor] = None,
               stream=None):
        """Stores the computed outputs of the misses: miss number m (ascending miss order) goes to part m mod world.
        miss_out: [M, n*d] in miss order (None for keys-only banks).  Returns {rank: (positions in the miss list,
        slots of the whole bank or -1)}.  Reads the miss count on the host."""
        M = int(bufs.counts[1])
        out = {}
        for p, first, r in zip(self.parts, self.base, self.ranks):
            mine = misses_of(r, self.world, M).to(self.device)
            share = L.ProbeBuffers(max(len(mine), 1), bufs.fp.shape[1], self.device, pinned_counts=False)
            share.miss_idx[: len(mine)] = bufs.miss_idx[:M][mine]
            share.counts[0] = bufs.counts[0]
            share.counts[1] = len(mine)
            io = share.io
            io.fp, io.rq = bufs.fp.data_ptr(), bufs.rq.data_ptr()       # fingerprints of the whole batch
            io.hit, io.slot, io.score, io.hit_idx = (bufs.hit.data_ptr(), bufs.slot.data_ptr(), bufs.score.data_ptr(),
                                                     bufs.hit_idx.data_ptr())
            io.generation = bufs.io.generation
            rows = miss_out[mine].contiguous() if miss_out is not None else None
            if len(mine) == 0 and p.desc.store_act:      # nothing to store: the library still wants a valid pointer
                rows = torch.zeros((1, p.n * p.d), dtype=torch.bfloat16, device=self.device)
            L.llmcache_commit(p.handle, rows, io, h_out, share.new_slot, stream)
            torch.cuda.synchronize(self.device)
            local = share.new_slot[: len(mine)]
            out[r] = (mine, torch.where(local >= 0, local + first, local))
        return out
