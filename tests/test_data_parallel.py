"""The multi-GPU round (one worker per rank; all_reduce(max) of the scales, all-to-all of the
packed indices, local PS aggregation of a block range, all-gather of the sums, local decompress;
and its peer-memory form, where the aggregate step reads the other ranks' buffers and pushes its
sums into them between two fences) on CPU process groups.  The exchange logic of paper_2302_08545_b200.data_parallel is run by
2, 3 and 4 gloo ranks whose per-rank steps are bound to the CPU oracle (the product binds them to
the CUDA library only); every rank's result must equal the oracle's single-process round over
all workers bit for bit: scales, the rank's own indices, the sums and the output."""
import os
import socket
import subprocess
import sys

import pytest

from paper_2302_08545_b200.data_parallel import block_ranges

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

WORKER = r"""
import os, sys
sys.path.insert(0, os.environ["THC_ROOT"])
import numpy as np, torch
import torch.distributed as dist
from oracle import oracle as O
from paper_2302_08545_b200.data_parallel import DataParallelRound, PeerMemoryRound

dist.init_process_group("gloo")
rank, world = dist.get_rank(), dist.get_world_size()
nblk = int(os.environ["THC_BLOCKS"])               # 7 blocks: uneven ranges for 2, 3 and 4 ranks; 8: even for 2 and 4
k, d, rnd = 8, 256 * (nblk - 1) + 77, 5
T = (0, 3, 5, 7, 9, 11, 13, 14, 15, 17, 19, 21, 23, 25, 27, 30)
cfg = O.Config(bits=4, granularity=30, table=T, t_p=2.1538746940614564, log2_block=k,
               seed=0x0123456789ABCDEF)
w = O.acc_bits(world, 30)
dt = {8: np.uint8, 16: np.uint16, 32: np.uint32}[w]
x = (np.random.default_rng(99).standard_normal((world, d)) * np.linspace(0.5, 2.0, world)[:, None]).astype(np.float32)

class OracleOps:                                   # the four per-rank steps, on host tensors
    def local_scales(self, grad):
        return torch.from_numpy(O.scales(grad.numpy()[None, :], cfg))
    def compress(self, grad, rnd, scales, worker, out=None):
        r = O.rht_forward(grad.numpy(), cfg, rnd)
        res = torch.from_numpy(O.pack(O.quantize(r, scales.numpy(), cfg, rnd, worker), 4))
        return res if out is None else out.copy_(res)
    def aggregate(self, slices, coords, out=None):
        packed = np.stack([np.array(s.numpy()) for s in slices])
        res = torch.from_numpy(O.aggregate(packed, coords, cfg, w).view(np.uint8).copy())
        return res if out is None else out.copy_(res)
    def decompress(self, total, divisor, rnd, scales):
        return torch.from_numpy(O.decompress(np.array(total.numpy()).view(dt), divisor, d, scales.numpy(), cfg, rnd))

class FilePeers:                                   # buffers all ranks address: files mapped by every rank
    count = 0
    def share(self, nbytes):
        name = os.path.join(os.environ["THC_OUT"], "buf%d_rank%%d.bin" % self.count)
        self.count += 1
        np.memmap(name % rank, dtype=np.uint8, mode="w+", shape=(nbytes,)).flush()
        dist.barrier()
        return [torch.from_numpy(np.memmap(name % q, dtype=np.uint8, mode="r+", shape=(nbytes,))) for q in range(world)]

if os.environ["THC_MODE"] == "peer":
    dp = PeerMemoryRound(OracleOps(), FilePeers(), d, k, 4, w)
else:
    dp = DataParallelRound(OracleOps(), d, k, 4, w)
for rnd in (5, 6):                                 # the second round reuses the peer buffers
    xr = (x * (1.0 + 0.25 * (rnd - 5))).astype(np.float32)
    out, scales, packed, total = dp.step(torch.from_numpy(xr[rank].copy()), rnd)
    ref = O.thc_round(xr, cfg, rnd)
    assert np.array_equal(scales.numpy().view(np.uint32), ref["scales"].view(np.uint32))
    assert np.array_equal(np.array(packed.numpy()), ref["packed"][rank])
    assert np.array_equal(np.array(total.numpy()).view(dt), ref["sum"])
    assert np.array_equal(out.numpy().view(np.uint32), ref["out"].view(np.uint32))
dist.barrier()
dist.destroy_process_group()
open(os.path.join(os.environ["THC_OUT"], f"rank{rank}.ok"), "w").write("ok")
"""


def _free_port() -> int:
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def test_block_ranges_cover_every_block_once():
    for nblocks in (1, 7, 8, 25, 132):
        for world in (1, 2, 3, 4, 8):
            r = block_ranges(nblocks, world)
            assert len(r) == world and r[0][0] == 0 and sum(c for _, c in r) == nblocks
            assert all(r[q][0] + r[q][1] == r[q + 1][0] for q in range(world - 1))
            assert max(c for _, c in r) - min(c for _, c in r) <= 1 and r[0][1] == max(c for _, c in r)


@pytest.mark.parametrize("world,blocks,mode", [(2, 7, "collective"), (3, 7, "collective"), (4, 7, "collective"),
                                               (2, 8, "collective"), (4, 8, "collective"),
                                               (2, 7, "peer"), (3, 7, "peer"), (4, 7, "peer")])
def test_round_across_gloo_ranks_equals_the_single_process_round(tmp_path, world, blocks, mode):
    script = tmp_path / "worker.py"
    script.write_text(WORKER)
    env = dict(os.environ, THC_ROOT=ROOT, THC_OUT=str(tmp_path), THC_MODE=mode, THC_BLOCKS=str(blocks),
               MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={world}",
           "--master-addr", "127.0.0.1", "--master-port", str(_free_port()), str(script)]
    res = subprocess.run(cmd, capture_output=True, text=True, env=env, timeout=300)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-3000:]
    assert all((tmp_path / f"rank{r}.ok").exists() for r in range(world))
