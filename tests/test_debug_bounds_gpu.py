"""The bounds-checking build (-DCAME_DEBUG_BOUNDS) on awkward shapes.

Every tile's index arithmetic is checked on the device against the tensor's shape and the
launch plan; a violation would be masked out and recorded, never trapped.  On the shapes that
stress the planner (1 x n, n x 1, columns not a multiple of the vector width, rows not a
multiple of the tile, single elements, many tensors, all three schedules) the record must
stay empty, and the checked build must produce the ordinary build's results bit for bit."""
import pytest

from paper_2307_02047_b200 import synth
from tests.test_api_gpu import Buffers, HP, W_ODD, _run_steps, _same
from tests.test_p1_stream_gpu import W_F32
from tests.test_pipelined_gpu import W_MANY, tuned

pytestmark = pytest.mark.gpu


def _run(torch, binding, w, seed, **tune):
    with tuned(binding, **tune):
        buf = Buffers(torch, binding, w, seed)
        ctx = binding.came_create(buf.descs)
    _run_steps(torch, binding, buf, ctx, seed, 1, 3)
    buf.check_guards()
    snap = buf.snapshot()
    binding.came_destroy(ctx)
    return snap


@pytest.mark.parametrize("w", [W_ODD, W_MANY, W_F32], ids=["odd", "many", "f32kinds"])
@pytest.mark.parametrize("tune", [dict(), dict(TILE_ELEMS=4096), dict(SCHEDULE=2, PIPE_GROUP_BYTES=300_000),
                                  dict(P1_STREAM=2)], ids=["default", "small_tiles", "pipelined", "p1_stream"])
def test_checked_build_records_nothing_and_matches(w, tune):
    import torch
    from paper_2307_02047_b200 import binding
    assert torch.cuda.is_available()
    want = _run(torch, binding, w, 61, **tune)
    with binding.using_debug_build():
        got = _run(torch, binding, w, 61, **tune)
        rec = binding.came_debug_bounds(0)
    assert rec["code"] == 0 and rec["threads"] == 0, rec
    assert _same(want, got)
