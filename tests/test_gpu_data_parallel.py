"""The multi-GPU round with its product binding (CUDA library + NCCL) at world size 1, the only
size NCCL allows on a single GPU: every collective of the round runs (on one rank they copy),
and the result must equal the plain single-process round on the same gradient bit for bit.  The
peer-memory form also runs as 2 and 3 processes on the one GPU (CUDA IPC mappings between them,
gloo for the fences) against the oracle.  The exchange logic at world sizes 2 to 4 is covered
on CPU in test_data_parallel.py."""
import os
import socket

import numpy as np
import pytest

from paper_2302_08545_b200 import workloads as W

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("k,d", [(20, 3 * (1 << 20) + 4321), (10, 33_001)])
def test_one_rank_nccl_round_equals_the_single_process_round(k, d):
    import torch
    import torch.distributed as dist
    from paper_2302_08545_b200 import runner
    from paper_2302_08545_b200.data_parallel import CudaOps, DataParallelRound
    w = W.Workload("dp_x", n=1, d=d, log2_block=k, bits=4, granularity=30, table=W.TABLES[(4, 30)],
                   data_seed=55)
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=dev)
    try:
        ctx = runner.context_for(w)
        r = runner.Round(ctx, 1, d, "f32")
        W.fill_torch(w, r.grads)
        r.run(2)
        torch.cuda.synchronize()
        dp = DataParallelRound(CudaOps(ctx, d, dev), d, k, 4, r.sz.acc_bits)
        out, scales, packed, total = dp.step(r.grads[0], 2)
        torch.cuda.synchronize()
        assert torch.equal(scales, r.scales)
        assert torch.equal(packed, r.packed[0])
        assert torch.equal(total, r.total.view(torch.uint8))
        assert np.array_equal(out.cpu().numpy().view(np.uint32), r.out.cpu().numpy().view(np.uint32))
        assert ctx.status() == 0
    finally:
        dist.destroy_process_group()


def test_one_rank_peer_memory_round_equals_the_single_process_round():
    import torch
    import torch.distributed as dist
    from paper_2302_08545_b200 import runner
    from paper_2302_08545_b200.data_parallel import CudaIpcPeers, CudaOps, PeerMemoryRound
    k, d = 20, 2 * (1 << 20) + 99
    w = W.Workload("dp_peer1", n=1, d=d, log2_block=k, bits=4, granularity=30, table=W.TABLES[(4, 30)],
                   data_seed=56)
    dev = torch.device("cuda", 0)
    torch.cuda.set_device(dev)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    os.environ["MASTER_ADDR"], os.environ["MASTER_PORT"] = "127.0.0.1", str(port)
    dist.init_process_group("nccl", rank=0, world_size=1, device_id=dev)
    try:
        ctx = runner.context_for(w)
        r = runner.Round(ctx, 1, d, "f32")
        W.fill_torch(w, r.grads)
        peers = CudaIpcPeers(dev)
        dp = PeerMemoryRound(CudaOps(ctx, d, dev), peers, d, k, 4, r.sz.acc_bits)
        for rnd in (2, 3):
            r.run(rnd)
            out, scales, packed, total = dp.step(r.grads[0], rnd)
            torch.cuda.synchronize()
            assert torch.equal(scales, r.scales)
            assert torch.equal(packed, r.packed[0])
            assert torch.equal(total, r.total.view(torch.uint8))
            assert np.array_equal(out.cpu().numpy().view(np.uint32), r.out.cpu().numpy().view(np.uint32))
        assert ctx.status() == 0
        del dp
        peers.close()
    finally:
        dist.destroy_process_group()


PEER_WORKER = r"""
import os, sys, datetime, traceback, faulthandler
faulthandler.enable()
sys.path.insert(0, os.environ["THC_ROOT"])
import numpy as np, torch
import torch.distributed as dist
from oracle import oracle as O
from paper_2302_08545_b200 import runner, workloads as W
from paper_2302_08545_b200.data_parallel import CudaIpcPeers, CudaOps, PeerMemoryRound

dist.init_process_group("gloo", timeout=datetime.timedelta(seconds=90))
rank, world = dist.get_rank(), dist.get_world_size()
outdir = os.environ["THC_OUT"]
dev = torch.device("cuda", 0)                      # every rank on the one GPU: kernels never wait on a rank
torch.cuda.set_device(dev)
k, d = 15, 5 * (1 << 15) + 1234                    # 6 blocks: ranges of 3 + 3 or 2 + 2 + 2
w = W.Workload("dp_peer", n=world, d=d, log2_block=k, bits=4, granularity=30, table=W.TABLES[(4, 30)],
               data_seed=57)
cfg = O.Config(bits=4, granularity=30, table=tuple(w.table), t_p=w.t_p, log2_block=k, seed=w.seed)
x = (np.random.default_rng(57).standard_normal((world, d)) * np.linspace(0.5, 2.0, world)[:, None]).astype(np.float32)
ctx = runner.context_for(w)
peers = CudaIpcPeers(dev)
try:
    probe = peers.share(4096)
except Exception as e:                             # no CUDA IPC between processes on this machine
    open(os.path.join(outdir, f"rank{rank}.noipc"), "w").write(repr(e))
    sys.exit(0)
del probe
dp = PeerMemoryRound(CudaOps(ctx, d, dev), peers, d, k, 4, w.acc_bits)
dt = {8: np.uint8, 16: np.uint16, 32: np.uint32}[w.acc_bits]
ok = True
try:
    for rnd in (4, 5, 6):                          # later rounds reuse the shared buffers
        xr = (x * (1.0 + 0.5 * (rnd - 4))).astype(np.float32)
        grad = torch.from_numpy(xr[rank].copy()).to(dev)
        out, scales, packed, total = dp.step(grad, rnd)
        torch.cuda.synchronize()
        got = [t.cpu().numpy() for t in (scales, packed, total, out)]
        ref = O.thc_round(xr, cfg, rnd)
        assert np.array_equal(got[0].view(np.uint32), ref["scales"].view(np.uint32))
        assert np.array_equal(got[1], ref["packed"][rank])
        assert np.array_equal(got[2].view(dt), ref["sum"])
        assert np.array_equal(got[3].view(np.uint32), ref["out"].view(np.uint32))
    assert ctx.status() == 0
except Exception:
    ok = False
    traceback.print_exc()
torch.cuda.synchronize()
del dp
peers.close()                                      # mappings dropped on every rank before an owner frees
dist.destroy_process_group()
if ok:
    open(os.path.join(outdir, f"rank{rank}.ok"), "w").write("ok")
sys.exit(0 if ok else 1)
"""


@pytest.mark.parametrize("world", [2, 3])
def test_peer_memory_round_between_processes_equals_the_oracle(tmp_path, world):
    """Two and three ranks as processes that share the one GPU: each rank's thc_aggregate reads
    the other processes' packed indices through CUDA IPC mappings and its sums are pushed into
    their buffers.  The ranks meet only on the host (gloo); no kernel waits on another rank."""
    import subprocess
    import sys
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    script = tmp_path / "peer_worker.py"
    script.write_text(PEER_WORKER)
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    env = dict(os.environ, THC_ROOT=root, THC_OUT=str(tmp_path), MASTER_ADDR="127.0.0.1", OMP_NUM_THREADS="1")
    cmd = [sys.executable, "-m", "torch.distributed.run", "--nnodes=1", f"--nproc-per-node={world}",
           "--master-addr", "127.0.0.1", "--master-port", str(port), str(script)]
    res = subprocess.run(cmd, capture_output=True, text=True, env=env, timeout=600)
    assert res.returncode == 0, res.stdout[-3000:] + res.stderr[-3000:]
    refused = [tmp_path / f"rank{r}.noipc" for r in range(world) if (tmp_path / f"rank{r}.noipc").exists()]
    if refused:
        pytest.skip("CUDA IPC between processes is unavailable here: " + refused[0].read_text()[:200])
    assert all((tmp_path / f"rank{r}.ok").exists() for r in range(world))
