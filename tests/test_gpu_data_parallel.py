"""The multi-GPU round with its product binding (CUDA library + NCCL) at world size 1, the only
size a single GPU allows: every collective of the round runs (on one rank they copy), and the
result must equal the plain single-process round on the same gradient bit for bit.  The
exchange logic at world sizes 2 to 4 is covered on CPU in test_data_parallel.py."""
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
