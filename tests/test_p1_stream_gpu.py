"""The streaming form of the first phase (persistent grid, per-thread rings of asynchronous
copies; CAME_TUNE_P1_STREAM) against the one-block-per-tile form.

Both add the same numbers in the same order, so every state tensor must agree bit for bit,
for every load width, ring depth and tile size, with ragged tiles, when gradients are re-bound
every step, and through the host-buffer step."""
import numpy as np
import pytest

from paper_2307_02047_b200 import synth
from tests.parity_util import gate, run_paired, to_torch_grad
from tests.test_api_gpu import Buffers, HP, W_ODD, _run_steps, _same
from tests.test_pipelined_gpu import W_MANY, tuned

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env(oracle):
    import torch
    from paper_2307_02047_b200 import binding
    assert torch.cuda.is_available()
    binding.load()
    return torch, binding, oracle


W_F32 = synth.Workload(
    "f32kinds", (synth.mat("x8", 300, 1032), synth.mat("x4", 77, 1028), synth.mat("x1", 50, 1030),
                 synth.mat("tall", 5000, 72), synth.mat("wide", 9, 8200), synth.mat("col", 700, 1),
                 synth.vec("v", 3000), synth.mat("one", 1, 1)),
    synth.F32, "normal_fixed", 1e-3, 0.0, (), 4, HP)


def _final_state(torch, binding, w, seed, steps=4, **tune):
    with tuned(binding, **tune):
        buf = Buffers(torch, binding, w, seed)
        ctx = binding.came_create(buf.descs)
    grid = binding.came_query(ctx, binding.CAME_Q_P1_STREAM_GRID)
    _run_steps(torch, binding, buf, ctx, seed, 1, steps)
    buf.check_guards()
    snap = buf.snapshot()
    binding.came_destroy(ctx)
    return snap, grid


@pytest.mark.parametrize("w", [W_ODD, W_MANY, W_F32], ids=["odd", "many", "f32kinds"])
@pytest.mark.parametrize("tile", [0, 4096, 65536])
def test_streaming_p1_is_bit_identical(env, w, tile):
    torch, binding, _ = env
    ref, grid_off = _final_state(torch, binding, w, 41, P1_STREAM=1, TILE_ELEMS=tile)
    assert grid_off == 0
    for ring in (1, 2, 3, 4):
        got, grid_on = _final_state(torch, binding, w, 41, P1_STREAM=2, P1_STREAM_RING=ring, TILE_ELEMS=tile)
        assert grid_on > 0
        assert _same(ref, got), f"streaming P1 (ring {ring}) differs from the per-tile form"


def test_streaming_p1_follows_rebound_gradients(env):
    """The streaming kernel reads gradient addresses from its own tile records; they must
    follow the pointers passed to came_step."""
    torch, binding, _ = env
    stream = torch.cuda.current_stream().cuda_stream
    ref, _ = _final_state(torch, binding, W_MANY, 43, steps=3, P1_STREAM=1)
    with tuned(binding, P1_STREAM=2):
        b = Buffers(torch, binding, W_MANY, 43)
        ctx = binding.came_create(b.descs)
    assert binding.came_query(ctx, binding.CAME_Q_P1_STREAM_GRID) > 0
    keep = []
    for step in (1, 2, 3):
        gs = [to_torch_grad(torch, synth.make_grad(W_MANY, 43, i, step), "cuda:0").reshape(-1).clone()
              for i in range(len(W_MANY.tensors))]
        keep.append(gs)
        binding.came_step(ctx, binding.make_hparams(step, **HP), [g.data_ptr() for g in gs], stream)
    torch.cuda.synchronize()
    binding.came_destroy(ctx)
    assert _same(ref, b.snapshot())


@pytest.mark.parametrize("name", ["mat:1500x1288:bf16", "mat:2048x2048", "mat:4100x1028"])
def test_streaming_p1_parity_with_oracle(env, name):
    torch, binding, oracle = env
    with tuned(binding, P1_STREAM=2, P1_STREAM_RING=3):
        gate(run_paired(torch, binding, oracle, synth.workload(name), seed=45, steps=5, check_at=(1, 5)),
             "p1_stream/" + name)
