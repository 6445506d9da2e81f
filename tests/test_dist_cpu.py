"""The N > 1 plumbing of the benchmark, exercised with two gloo ranks on the CPU: the job's
step time is the slowest rank's, throughput counts every rank's replica, and only rank 0 of
the oracle arm does any work."""
import json
import os
import subprocess
import sys

import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import bench
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port), RANK=str(rank),
                      WORLD_SIZE=str(world), LOCAL_RANK=str(rank))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    assert bench.dist_env() == (rank, rank, world)
    ms = bench.max_over_ranks(10.0 + 5.0 * rank, world, torch.device("cpu"))
    dist.barrier()
    q.put((rank, ms, bench.job_value(world, 1000, ms)))
    dist.destroy_process_group()


def test_two_ranks_take_the_slowest_time():
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 29500 + os.getpid() % 2000
    procs = [ctx.Process(target=_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    out = sorted(q.get(timeout=120) for _ in procs)
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert [o[1] for o in out] == [15.0, 15.0]              # max over ranks on both
    assert out[0][2] == 2 * 1000 / 15e-3                    # both replicas counted


def test_single_rank_is_identity():
    sys.path.insert(0, ROOT)
    import bench
    assert bench.max_over_ranks(3.5, 1, None) == 3.5
    assert bench.job_value(1, 10, 2.0) == 5000.0


def test_reference_arm_other_ranks_do_nothing():
    env = dict(os.environ, RANK="1", LOCAL_RANK="1", WORLD_SIZE="2")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True,
                         text=True, timeout=120)
    assert res.returncode == 0 and res.stdout.strip() == ""


# ---------------------------------------------------------------------------
# tensor-sharded step: two gloo ranks, the oracle as the injected local stepper
# ---------------------------------------------------------------------------
def test_partition_by_bytes_balances_and_is_deterministic():
    sys.path.insert(0, ROOT)
    from paper_2307_02047_b200.sharded import partition_by_bytes
    sizes = [100, 90, 50, 40, 30, 10, 10, 5]
    own = partition_by_bytes(sizes, 2)
    loads = [sum(s for s, o in zip(sizes, own) if o == r) for r in range(2)]
    assert abs(loads[0] - loads[1]) <= max(sizes) and sum(loads) == sum(sizes)
    assert own == partition_by_bytes(sizes, 2)
    assert partition_by_bytes(sizes, 1) == [0] * len(sizes)
    assert sorted(set(partition_by_bytes([7] * 8, 8))) == list(range(8))


def test_segment_layout_covers_every_element_once():
    sys.path.insert(0, ROOT)
    from paper_2307_02047_b200.sharded import (ALIGN_ELEMS, bucket_pieces, partition_by_bytes,
                                               segment_layout)
    numels = [960, 128, 33, 320, 7, 4096, 1]
    for world in (1, 2, 3):
        for bucket in (8, 64, 1000, 1 << 20):
            owner = partition_by_bytes([4 * n for n in numels], world)
            offset, seg_len, chunk, nb = segment_layout(numels, owner, world, bucket)
            assert seg_len == nb * chunk and chunk % ALIGN_ELEMS == 0
            assert all(o % ALIGN_ELEMS == 0 for o in offset)          # 32-byte aligned fp32 views
            pieces = bucket_pieces(numels, owner, offset, chunk, nb)
            seen = [0] * len(numels)
            cells = set()
            for b, plist in enumerate(pieces):
                for (i, lo, hi, r, dst) in plist:
                    assert r == owner[i] and 0 <= lo < hi <= numels[i] and dst + hi - lo <= chunk
                    assert b * chunk + dst == offset[i] + lo                   # where it sits in the segment
                    seen[i] += hi - lo
                    for c in range(dst, dst + hi - lo):
                        assert (b, r, c) not in cells                          # no two pieces overlap
                        cells.add((b, r, c))
            assert seen == numels


def _sharded_worker(rank, world, port, q):
    sys.path.insert(0, ROOT)
    import numpy as np
    from oracle import came_oracle
    from paper_2307_02047_b200 import synth
    from paper_2307_02047_b200.sharded import ShardedCame
    os.environ.update(MASTER_ADDR="127.0.0.1", MASTER_PORT=str(port))
    dist.init_process_group("gloo", rank=rank, world_size=world)
    ts = (synth.mat("a", 24, 40), synth.mat("b", 16, 8), synth.vec("v", 33), synth.mat("c", 5, 64))
    hp = dict(synth.PAPER_HPARAMS, weight_decay=0.01)
    w = synth.Workload("sh", ts, synth.F32, "normal_fixed", 1e-3, 0.0, (), 3, hp)
    params = [torch.from_numpy(x.astype(np.float64)) for x in synth.make_params(w, 1)]
    grads = [torch.zeros_like(p) for p in params]

    class OracleLocal:                      # stands in for the CUDA context on this CPU test
        def __init__(self, p, g):
            self.p, self.g = p, g
            self.o = came_oracle.OracleOptimizer([x.numpy() for x in p])
        def step(self, **h):
            gs = h.pop("grad_scale")
            self.o.step([x.numpy() * gs for x in self.g], **h)
            for dst, src in zip(self.p, self.o.p):
                dst.copy_(torch.from_numpy(src))

    # small buckets: several collectives per step, tensors straddling bucket boundaries
    sh = ShardedCame(params, grads, make_local=OracleLocal, bucket_elems=256)
    assert sh.n_buckets >= 3 and sh.collectives_per_step == 2 * sh.n_buckets
    for step in (1, 2, 3):
        for i, g in enumerate(grads):       # each rank has its own micro-batch gradient
            g.copy_(torch.from_numpy(synth.widen(synth.make_grad(w, 100 + rank, i, step))))
        sh.step(**hp)
    q.put((rank, sh.owner, [p.numpy().copy() for p in params]))
    dist.barrier()
    dist.destroy_process_group()


def test_sharded_step_equals_single_process_mean_gradient():
    import numpy as np
    sys.path.insert(0, ROOT)
    from oracle import came_oracle
    from paper_2307_02047_b200 import synth
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    port = 31500 + os.getpid() % 2000
    procs = [ctx.Process(target=_sharded_worker, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    out = sorted((q.get(timeout=180) for _ in procs), key=lambda o: o[0])
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert out[0][1] == out[1][1] and set(out[0][1]) == {0, 1}       # same partition, both ranks used
    # reference: one process stepping on the mean of the two ranks' gradients
    ts = (synth.mat("a", 24, 40), synth.mat("b", 16, 8), synth.vec("v", 33), synth.mat("c", 5, 64))
    hp = dict(synth.PAPER_HPARAMS, weight_decay=0.01)
    w = synth.Workload("sh", ts, synth.F32, "normal_fixed", 1e-3, 0.0, (), 3, hp)
    ref = came_oracle.OracleOptimizer(synth.make_params(w, 1))
    for step in (1, 2, 3):
        gs = [(synth.widen(synth.make_grad(w, 100, i, step)) + synth.widen(synth.make_grad(w, 101, i, step))) * 0.5
              for i in range(len(ts))]
        ref.step(gs, **hp)
    for r in range(2):
        for got, want in zip(out[r][2], ref.p):
            np.testing.assert_allclose(got, want, rtol=1e-12, atol=0)


def test_reference_arm_prints_the_contract_line():
    """bench.py --impl reference (the CPU oracle on a bounded sample) prints one JSON line with
    the keys the benchmark contract names; no GPU is touched."""
    env = dict(os.environ, RANK="0", LOCAL_RANK="0", WORLD_SIZE="1", CUDA_VISIBLE_DEVICES="")
    res = subprocess.run([sys.executable, os.path.join(ROOT, "bench.py"), "--impl", "reference",
                          "--steps", "1", "--warmup", "0"], env=env, capture_output=True,
                         text=True, timeout=600)
    assert res.returncode == 0, res.stderr[-2000:]
    lines = [l for l in res.stdout.splitlines() if l.strip()]
    assert len(lines) == 1
    d = json.loads(lines[0])
    assert d["impl"] == "reference" and d["metric"] == "came_params_updated_per_sec"
    assert d["unit"] == "params/s" and d["value"] > 0 and d["higher_is_better"] is True
    assert d["steps"] == 1 and d["warmup"] == 0 and d["gpu_launches"] == 0
    assert d["cpu_baseline"]["kind"] == "oracle" and d["cpu_baseline"]["cores"] >= 1
    assert d["cpu_baseline"]["value"] == d["value"] and d["cpu_baseline"]["sample"]
    assert d["e2e"] == {"value": d["value"], "unit": "params/s", "h2d_bytes_per_step": 0,
                        "d2h_bytes_per_step": 0}
    assert d["config"]["workload"] == "llama7b"
