"""One THC round across GPUs, one worker per rank (the paper's Section 2 remark that a PS
colocated with every worker makes the scheme an all-reduce, and Algorithm 3's two exchanges).

Rank i holds worker i's gradient.  The round:

  1. preliminary stage (Section 5.3; Algorithm 3 "send ||x_i||, receive ell"): every rank
     computes its own M_i per RHT block (thc_prepare on one worker); all_reduce(max) gives
     M = max_i M_i, the value thc_prepare returns for all workers together (the map from the
     norm to the fp32 M is monotone);
  2. thc_compress of the rank's own gradient (worker id = rank);
  3. "send Z_i": the RHT blocks are split into world-size contiguous ranges and rank q acts as
     the PS of range q, so an all-to-all moves every rank's packed indices of range q to q;
  4. thc_aggregate over the n received slices (Algorithm 2's PS line);
  5. "receive Y": all-gather of the w-bit sums;
  6. thc_decompress with divisor n.

Every slice lands in the rank's own memory (a plain collective) before a kernel reads it.  Per
rank and round the exchanges move about d (b + w)/8 bytes each way instead of the 8 d of an
fp32 ring all-reduce.

The exchange logic takes the per-rank steps as an `ops` object, so that it can be exercised on
CPU process groups; the only implementation in this package, CudaOps, calls the library.
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def block_ranges(nblocks: int, world: int):
    """Contiguous ranges of RHT blocks, one per rank: the first nblocks % world ranks get one
    block more.  Returns a list of (first, count)."""
    base, extra = divmod(nblocks, world)
    out, first = [], 0
    for q in range(world):
        cnt = base + (1 if q < extra else 0)
        out.append((first, cnt))
        first += cnt
    return out


class CudaOps:
    """The per-rank steps on the rank's GPU through the C ABI (thc.Context)."""

    def __init__(self, ctx, d: int, device):
        self.ctx, self.d, self.device = ctx, d, device
        self.sz = ctx.sizes(d, 1)
        self.workspace = torch.empty(self.sz.workspace_bytes, dtype=torch.uint8, device=device)

    def local_scales(self, grad):
        scales = torch.empty(self.sz.nblocks, dtype=torch.float32, device=self.device)
        self.ctx.prepare([grad], self.d, scales, self.workspace)
        return scales

    def compress(self, grad, rnd: int, scales, worker: int):
        packed = torch.empty(self.sz.packed_bytes, dtype=torch.uint8, device=self.device)
        self.ctx.compress([grad], self.d, rnd, scales, [packed], self.workspace, worker_base=worker)
        return packed

    def aggregate(self, slices, coords: int):
        """slices: n tensors of packed indices covering `coords` coordinates (whole blocks)."""
        sz = self.ctx.sizes(coords, len(slices))
        total = torch.empty(sz.sum_bytes, dtype=torch.uint8, device=self.device)
        self.ctx.aggregate(slices, coords, total)
        return total

    def decompress(self, total, divisor: int, rnd: int, scales):
        out = torch.empty(self.d, dtype=torch.float32, device=self.device)
        self.ctx.decompress(total, divisor, self.d, rnd, scales, out, self.workspace)
        return out


class DataParallelRound:
    """The exchange steps of one round; `ops` supplies the four per-rank steps.

    bits / acc_bits / log2_block / d fix the byte counts of the slices: a range of c blocks is
    c * B * bits / 8 bytes of indices and c * B * acc_bits / 8 bytes of sums.
    """

    def __init__(self, ops, d: int, log2_block: int, bits: int, acc_bits: int, group=None):
        self.ops, self.d, self.bits, self.acc_bits = ops, d, bits, acc_bits
        self.group = group
        self.world = dist.get_world_size(group)
        self.rank = dist.get_rank(group)
        self.block = 1 << log2_block
        self.nblocks = (d + self.block - 1) // self.block
        self.ranges = block_ranges(self.nblocks, self.world)
        if (self.block * bits) % 128 != 0 and self.world > 1:
            raise ValueError("slices of packed indices must start on 16-byte boundaries")

    def _idx_bytes(self, blocks: int) -> int:
        return blocks * self.block * self.bits // 8

    def _sum_bytes(self, blocks: int) -> int:
        return blocks * self.block * self.acc_bits // 8

    def step(self, grad, rnd: int):
        """Returns (out, scales, packed, total): the decompressed average and the intermediates
        (for checks).  Collectives are issued on the current stream of the tensors' device."""
        ops, world, rank = self.ops, self.world, self.rank
        # 1. scales: max over workers of the per-worker M
        scales = ops.local_scales(grad)
        dist.all_reduce(scales, op=dist.ReduceOp.MAX, group=self.group)
        # 2. own indices
        packed = ops.compress(grad, rnd, scales, rank)
        # 3. all-to-all: range q of every worker goes to rank q
        in_splits = [self._idx_bytes(c) for (_, c) in self.ranges]
        mine = self.ranges[rank][1]
        recv = torch.empty(world * self._idx_bytes(mine), dtype=torch.uint8, device=packed.device)
        out_splits = [self._idx_bytes(mine)] * world
        dist.all_to_all_single(recv, packed, output_split_sizes=out_splits, input_split_sizes=in_splits,
                               group=self.group)
        # 4. the PS line on the own range
        if mine > 0:
            slices = list(recv.split(self._idx_bytes(mine)))
            part = ops.aggregate(slices, mine * self.block)
        else:
            part = torch.empty(0, dtype=torch.uint8, device=packed.device)
        # 5. all-gather of the sums (ranges may differ by one block: padded to the longest)
        longest = self._sum_bytes(self.ranges[0][1])
        padded = torch.zeros(longest, dtype=torch.uint8, device=packed.device)
        padded[: part.numel()] = part
        gathered = torch.empty(world * longest, dtype=torch.uint8, device=packed.device)
        dist.all_gather_into_tensor(gathered, padded, group=self.group)
        total = torch.cat([gathered[q * longest: q * longest + self._sum_bytes(c)]
                           for q, (_, c) in enumerate(self.ranges)])
        # 6. estimate + inverse RHT with divisor n
        out = ops.decompress(total, world, rnd, scales)
        return out, scales, packed, total
