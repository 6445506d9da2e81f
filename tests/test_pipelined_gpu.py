"""The pipelined schedule (one persistent grid per step, CAME_TUNE_SCHEDULE = 2) against the
one-grid-per-phase schedule and against the CPU oracle.

The two schedules run the same tile routines, and every reduction adds its partial sums in a
fixed order, so with the same tile size they must agree bit for bit whatever the order in
which the persistent grid's blocks happen to run.  The bounded wait that the pipelined grid
uses for its "phase done" flags is exercised on its own, on a flag that nothing sets: it must
give up after its limit, report it, and leave the device usable."""
import numpy as np
import pytest

from paper_2307_02047_b200 import synth
from tests.parity_util import gate, run_paired
from tests.test_api_gpu import Buffers, HP, W_ODD, _run_steps, _same

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env(oracle):
    import torch
    from paper_2307_02047_b200 import binding
    assert torch.cuda.is_available()
    binding.load()
    return torch, binding, oracle


class tuned:
    """came_tune settings for the duration of a with-block (restored to their defaults)."""

    def __init__(self, binding, **kv):
        self.b, self.kv = binding, kv

    def __enter__(self):
        for k, v in self.kv.items():
            self.b.came_tune(getattr(self.b, "CAME_TUNE_" + k), v)

    def __exit__(self, *exc):
        for k in self.kv:
            self.b.came_tune(getattr(self.b, "CAME_TUNE_" + k), 0)


W_MANY = synth.Workload(
    "many", tuple([synth.mat(f"a{i}", 96 + 8 * i, 520) for i in range(6)] +
                  [synth.vec(f"v{i}", 700 + i) for i in range(3)] +
                  [synth.mat("wide", 40, 4104), synth.mat("tall", 3000, 72), synth.mat("col", 900, 1),
                   synth.mat("row", 1, 2050), synth.vec("one", 1)]),
    synth.BF16, "normal_fixed", 1e-3, 0.0, (), 4, HP)


@pytest.mark.parametrize("order", [0, 1])
@pytest.mark.parametrize("w", [W_ODD, W_MANY], ids=["odd", "many"])
def test_pipelined_is_bit_identical_to_phase_grids(env, w, order):
    torch, binding, _ = env
    snaps = []
    for sched in (binding.CAME_SCHEDULE_PHASE_GRIDS, binding.CAME_SCHEDULE_PIPELINED):
        # same tile size in both, small groups so that the pipeline has many stages
        with tuned(binding, SCHEDULE=sched, TILE_ELEMS=4096, PIPE_GROUP_BYTES=300_000, PIPE_ORDER=order):
            buf = Buffers(torch, binding, w, 31)
            ctx = binding.came_create(buf.descs)
        assert binding.came_query(ctx, binding.CAME_Q_SCHEDULE) == (sched == binding.CAME_SCHEDULE_PIPELINED)
        if sched == binding.CAME_SCHEDULE_PIPELINED:
            assert binding.came_query(ctx, binding.CAME_Q_LAUNCHES_PER_STEP) == 1
            assert binding.came_query(ctx, binding.CAME_Q_PIPE_GROUPS) >= 3
        _run_steps(torch, binding, buf, ctx, 31, 1, 4)
        assert binding.came_query(ctx, binding.CAME_Q_DEVICE_ERROR) == 0
        buf.check_guards()
        snaps.append(buf.snapshot())
        binding.came_destroy(ctx)
    assert _same(*snaps), "the pipelined grid and the phase grids disagree"


@pytest.mark.parametrize("name,steps", [("toy", 10), ("mat:1500x1288:bf16", 10), ("mat:1x65536", 3),
                                        ("mat:65536x1", 3), ("mat:2048x2048", 5)])
def test_pipelined_parity_single_sets(env, name, steps):
    torch, binding, oracle = env
    with tuned(binding, SCHEDULE=2):
        gate(run_paired(torch, binding, oracle, synth.workload(name), seed=33, steps=steps,
                        check_at=(1, steps)), "pipelined/" + name)


@pytest.mark.parametrize("algorithm", ["came", "adafactor"])
def test_pipelined_parity_many_tensors_flags_and_modes(env, algorithm):
    torch, binding, oracle = env
    hp = dict(HP, lr=1e-3, weight_decay=0.1, grad_scale=0.25)
    w = synth.Workload("many_wd", W_MANY.tensors, synth.F32, "student_t3", 1e-3, 0.0, (), 10, hp)
    flags = [0] * len(w.tensors)
    flags[1] = binding.CAME_T_NO_WEIGHT_DECAY
    flags[6] = binding.CAME_T_VEC_NO_CONFIDENCE
    with tuned(binding, SCHEDULE=2, PIPE_GROUP_BYTES=400_000):
        gate(run_paired(torch, binding, oracle, w, seed=35, steps=10, check_at=(1, 10), flags=flags,
                        algorithm=algorithm, bf16_copy=True), "pipelined/many/" + algorithm)


def test_pipelined_bert_base_ten_steps(env):
    """The BERT-base-shaped set at full size with the schedule's default tile and group sizes:
    a dozen or so pipeline stages, the embedding a stage of its own."""
    torch, binding, oracle = env
    w = synth.workload("bert_base")
    with tuned(binding, SCHEDULE=2):
        gate(run_paired(torch, binding, oracle, w, seed=2, steps=10, check_at=(1, 10), workers=16),
             "pipelined/bert_base")


def test_pipelined_graph_replay_and_clear(env):
    torch, binding, _ = env
    with tuned(binding, SCHEDULE=2, PIPE_GROUP_BYTES=300_000):
        a = Buffers(torch, binding, W_ODD, 13)
        ctx = binding.came_create(a.descs)
        a.set_grads(13, 1)
        for step in (1, 2, 3, 4):
            binding.came_step(ctx, binding.make_hparams(step, **HP), None, torch.cuda.current_stream().cuda_stream)
        torch.cuda.synchronize()
        binding.came_destroy(ctx)

        b = Buffers(torch, binding, W_ODD, 13)
        ctx = binding.came_create(b.descs)
    b.set_grads(13, 1)
    stream = torch.cuda.current_stream().cuda_stream
    binding.came_step(ctx, binding.make_hparams(1, **HP), None, stream)
    torch.cuda.synchronize()
    # clearing a healthy context is harmless: counters, flags and the step epoch restart at zero
    binding.came_clear_device_error(ctx, stream)
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        binding.came_step(ctx, binding.make_hparams(2, **HP), None, side.cuda_stream)
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        binding.came_step(ctx, binding.make_hparams(3, **HP), None, torch.cuda.current_stream().cuda_stream)
    for _ in range(2):          # steps 3 and 4: the step number lives on the device, not in the launch
        graph.replay()
    torch.cuda.synchronize()
    assert binding.came_query(ctx, binding.CAME_Q_DEVICE_ERROR) == 0
    binding.came_destroy(ctx)
    assert _same(a.snapshot(), b.snapshot())


def test_bounded_wait_gives_up_and_reports(env):
    """A wait for a flag that nothing sets must end at its limit with the error word set, and
    the device must be usable afterwards."""
    torch, binding, oracle = env
    for limit_ns in (200_000, 5_000_000):
        r = binding.came_selftest_wait_timeout(0, limit_ns)
        assert r["timed_out"] == 1 and r["error_word"] == 1
        assert limit_ns * 1e-6 * 0.5 <= r["elapsed_ms"] <= limit_ns * 1e-6 + 50.0, r
    with pytest.raises(binding.CameError) as e:
        binding.came_selftest_wait_timeout(0, 5_000_000_000)      # limits above 1 s are refused
    assert e.value.status == 11
    with tuned(binding, SCHEDULE=2):
        gate(run_paired(torch, binding, oracle, synth.workload("toy"), seed=1, steps=2, check_at=(1, 2)))
