"""The tensor-sharded step with the real CUDA stepper, on a process group of one rank.

One GPU is all a test run gets here, so the multi-rank exchange is covered on the CPU (two
gloo ranks, tests/test_dist_cpu.py); this test runs the same code path end to end on the GPU --
bucketed reduce-scatter of the gradients (NCCL), the CUDA step on fp32 views of the summed
segment, bucketed all-gather of the parameters -- and checks the result against the oracle."""
import os

import numpy as np
import pytest

from paper_2307_02047_b200 import synth
from tests.parity_util import TOL_STEP1, TOL_STEP10, err_signed, to_torch_grad

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("bucket_elems", [4096, 1 << 26])
def test_sharded_step_world_size_one_matches_oracle(oracle, bucket_elems):
    import torch
    import torch.distributed as dist
    from paper_2307_02047_b200 import binding
    from paper_2307_02047_b200.sharded import ShardedCame
    assert torch.cuda.is_available()
    torch.cuda.set_device(0)
    os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
    os.environ.setdefault("MASTER_PORT", str(29700 + os.getpid() % 200))
    created = not dist.is_initialized()
    if created:
        dist.init_process_group("nccl", rank=0, world_size=1, device_id=torch.device("cuda", 0))
    try:
        ts = (synth.mat("a", 257, 1032), synth.mat("b", 96, 520), synth.vec("v", 1001),
              synth.mat("c", 33, 65), synth.mat("d", 300, 1))
        hp = dict(synth.PAPER_HPARAMS, weight_decay=0.01, grad_scale=0.5)
        w = synth.Workload("sharded", ts, synth.BF16, "normal_fixed", 1e-3, 0.0, (), 3, hp)
        p_host = synth.make_params(w, 51)
        params = [torch.from_numpy(p).cuda() for p in p_host]
        grads = [torch.empty(t.shape, dtype=torch.bfloat16, device="cuda") for t in ts]
        sh = ShardedCame(params, grads, bucket_elems=bucket_elems)
        assert sh.owner == [0] * len(ts) and sh.collectives_per_step == 2 * sh.n_buckets
        if bucket_elems == 4096:
            assert sh.n_buckets > 10
        orc = oracle.OracleOptimizer(p_host)
        for step in (1, 2, 3):
            g_host = synth.make_grads(w, 51, step)
            for dg, g in zip(grads, g_host):
                dg.copy_(to_torch_grad(torch, g, "cuda"))
            sh.step(**hp)
            orc.step([synth.widen(g) * 0.5 for g in g_host], **dict(hp, grad_scale=1.0))
            torch.cuda.synchronize()
            tol = TOL_STEP1 if step == 1 else TOL_STEP10
            for p, ref in zip(params, orc.p):
                assert err_signed(p.cpu().numpy(), ref) <= tol
        sh.close()
    finally:
        if created:
            dist.destroy_process_group()
