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

PeerMemoryRound is the same round without the two data collectives, for the GPUs of one node:
every rank's packed indices and sums live in buffers all ranks can address (CudaIpcPeers: CUDA
IPC mappings, NVLink peer memory between GPUs), the thc_aggregate kernel of rank q loads range q
of every worker's indices straight from the owners' memory (compute and transfer in one kernel,
plain loads only), and q stores its sums into every rank's buffer.  Two stream-ordered fences
per round (a one-element all-reduce each) replace the all-to-all and the all-gather; no kernel
ever waits on another rank.

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
    """The per-rank steps on the rank's GPU through the C ABI (thc.Context).  Buffers are
    allocated once: what a step returns is overwritten by the same step of the next round."""

    def __init__(self, ctx, d: int, device):
        self.ctx, self.d, self.device = ctx, d, device
        self.sz = ctx.sizes(d, 1)
        u8 = dict(dtype=torch.uint8, device=device)
        self.workspace = torch.empty(self.sz.workspace_bytes, **u8)
        self.scales = torch.empty(self.sz.nblocks, dtype=torch.float32, device=device)
        self.packed = torch.empty(self.sz.packed_bytes, **u8)
        self.out = torch.empty(d, dtype=torch.float32, device=device)
        self._part = {}

    def local_scales(self, grad):
        self.ctx.prepare([grad], self.d, self.scales, self.workspace)
        return self.scales

    def compress(self, grad, rnd: int, scales, worker: int, out=None):
        packed = out if out is not None else self.packed
        self.ctx.compress([grad], self.d, rnd, scales, [packed], self.workspace, worker_base=worker)
        return packed

    def aggregate(self, slices, coords: int, out=None):
        """slices: n tensors of packed indices covering `coords` coordinates (whole blocks);
        they may live in another rank's memory."""
        total = out
        if total is None:
            key = (coords, len(slices))
            if key not in self._part:
                self._part[key] = torch.empty(self.ctx.sizes(coords, len(slices)).sum_bytes,
                                              dtype=torch.uint8, device=self.device)
            total = self._part[key]
        self.ctx.aggregate(slices, coords, total)
        return total

    def decompress(self, total, divisor: int, rnd: int, scales):
        self.ctx.decompress(total, divisor, self.d, rnd, scales, self.out, self.workspace)
        return self.out


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
        self._recv = self._padded = self._gathered = self._total = None

    def _idx_bytes(self, blocks: int) -> int:
        return blocks * self.block * self.bits // 8

    def _sum_bytes(self, blocks: int) -> int:
        return blocks * self.block * self.acc_bits // 8

    def _buffers(self, like):
        if self._recv is None:
            u8 = dict(dtype=torch.uint8, device=like.device)
            mine = self.ranges[self.rank][1]
            longest = self._sum_bytes(self.ranges[0][1])
            self._recv = torch.empty(self.world * self._idx_bytes(mine), **u8)
            self._gathered = torch.empty(self.world * longest, **u8)
            self._even = all(c == self.ranges[0][1] for _, c in self.ranges)
            # ranges of equal length: the gathered sums are the sum buffer; else ranges are
            # padded to the longest for the all-gather and copied out
            self._padded = None if self._even else torch.zeros(longest, **u8)
            self._total = self._gathered if self._even else torch.empty(self._sum_bytes(self.nblocks), **u8)
        return self._recv, self._padded, self._gathered, self._total

    def step(self, grad, rnd: int):
        """Returns (out, scales, packed, total): the decompressed average and the intermediates
        (for checks; buffers of this object and of `ops`, overwritten by the next step).
        Collectives are issued on the current stream of the tensors' device."""
        ops, world, rank = self.ops, self.world, self.rank
        # 1. scales: max over workers of the per-worker M
        scales = ops.local_scales(grad)
        dist.all_reduce(scales, op=dist.ReduceOp.MAX, group=self.group)
        # 2. own indices
        packed = ops.compress(grad, rnd, scales, rank)
        recv, padded, gathered, total = self._buffers(packed)
        # 3. all-to-all: range q of every worker goes to rank q
        in_splits = [self._idx_bytes(c) for (_, c) in self.ranges]
        mine = self.ranges[rank][1]
        out_splits = [self._idx_bytes(mine)] * world
        dist.all_to_all_single(recv, packed, output_split_sizes=out_splits, input_split_sizes=in_splits,
                               group=self.group)
        # 4. the PS line on the own range, 5. all-gather of the sums
        longest = self._sum_bytes(self.ranges[0][1])
        slices = list(recv.split(self._idx_bytes(mine))) if mine > 0 else []
        if self._even:
            part = gathered[rank * longest: (rank + 1) * longest]
            ops.aggregate(slices, mine * self.block, out=part)
            dist.all_gather_into_tensor(gathered, part, group=self.group)
        else:
            if mine > 0:
                ops.aggregate(slices, mine * self.block, out=padded[: self._sum_bytes(mine)])
            dist.all_gather_into_tensor(gathered, padded, group=self.group)
            at = 0
            for q, (_, c) in enumerate(self.ranges):
                n = self._sum_bytes(c)
                total[at: at + n].copy_(gathered[q * longest: q * longest + n])
                at += n
        # 6. estimate + inverse RHT with divisor n
        out = ops.decompress(total, world, rnd, scales)
        return out, scales, packed, total


class CudaIpcPeers:
    """Device buffers of this rank that every rank of the node can address.

    share(nbytes) allocates nbytes on this rank's GPU, hands its CUDA IPC handle to the other
    ranks of the group and returns one uint8 tensor per rank: the own buffer and the others'
    mappings (peer memory over NVLink when the owners are other GPUs).  All GPUs of the node must
    be visible to every process.  close() drops the mappings on all ranks before any owner
    frees its buffer."""

    def __init__(self, device, group=None):
        self.device, self.group = device, group
        self.world, self.rank = dist.get_world_size(group), dist.get_rank(group)
        self._own, self._mapped = [], []

    def share(self, nbytes: int):
        local = torch.empty(max(nbytes, 1), dtype=torch.uint8, device=self.device)[:nbytes]
        self._own.append(local)
        if self.world == 1:
            return [local]
        from torch.multiprocessing.reductions import reduce_tensor
        # one handle per reader: torch counts the readers of a shared CUDA block per handle
        mine = [None if q == self.rank else reduce_tensor(local) for q in range(self.world)]
        handles = [None] * self.world
        dist.all_gather_object(handles, mine, group=self.group)
        bufs = []
        for q in range(self.world):
            if q == self.rank:
                bufs.append(local)
            else:
                fn, args = handles[q][self.rank]
                bufs.append(fn(*args))
        self._mapped.append([b for q, b in enumerate(bufs) if q != self.rank])
        return bufs

    def close(self):
        if torch.cuda.is_available():
            torch.cuda.synchronize()
        self._mapped.clear()
        if self.world > 1:
            dist.barrier(group=self.group)
        self._own.clear()


class PeerMemoryRound(DataParallelRound):
    """The round over buffers all ranks can address: `peers.share(nbytes)` returns one uint8
    tensor per rank (index = owner).  The caller keeps `peers` and this object alive together
    and drops this object (its views of the peers' buffers) before peers.close()."""

    def __init__(self, ops, peers, d: int, log2_block: int, bits: int, acc_bits: int, group=None):
        super().__init__(ops, d, log2_block, bits, acc_bits, group)
        self.packed = peers.share(self._idx_bytes(self.nblocks))
        self.total = peers.share(self._sum_bytes(self.nblocks))
        self._token = torch.zeros(1, dtype=torch.int32, device=self.packed[self.rank].device)

    def _fence(self):
        """Everything every rank enqueued before its fence is complete before anything a rank
        enqueues after it starts: a collective on the compute stream cannot finish anywhere
        before every rank has reached it."""
        dist.all_reduce(self._token, group=self.group)

    def step(self, grad, rnd: int):
        ops, world, rank = self.ops, self.world, self.rank
        scales = ops.local_scales(grad)
        dist.all_reduce(scales, op=dist.ReduceOp.MAX, group=self.group)
        # own indices, into the buffer the other ranks read.  No rank still reads the previous
        # round's: all aggregates were complete at that round's second fence.
        ops.compress(grad, rnd, scales, rank, out=self.packed[rank])
        self._fence()
        first, mine = self.ranges[rank]
        if mine > 0:
            lo, hi = self._idx_bytes(first), self._idx_bytes(first + mine)
            slo, shi = self._sum_bytes(first), self._sum_bytes(first + mine)
            part = self.total[rank][slo:shi]
            # the PS line on the own range: the kernel loads the n slices from their owners
            ops.aggregate([self.packed[q][lo:hi] for q in range(world)], mine * self.block, out=part)
            for q in range(world):                  # "receive Y", pushed
                if q != rank:
                    self.total[q][slo:shi].copy_(part, non_blocking=True)
        self._fence()
        out = ops.decompress(self.total[rank], world, rnd, scales)
        return out, scales, self.packed[rank], self.total[rank]
