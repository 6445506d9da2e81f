"""GPU tests of the C ABI beyond numerics: error paths that must not launch, resume,
run-to-run determinism, gradient re-binding, the host-buffer step, queries, profiling and
guard bands around every buffer (no out-of-bounds write for awkward shapes)."""
import ctypes

import numpy as np
import pytest

from paper_2307_02047_b200 import synth
from tests.parity_util import to_torch_grad

pytestmark = pytest.mark.gpu
HP = dict(synth.PAPER_HPARAMS)
GUARD = 64          # floats of sentinel on each side of every buffer
SENT = 1232.0      # exactly representable in bf16 and fp32


@pytest.fixture(scope="module")
def env():
    import torch
    from paper_2307_02047_b200 import binding
    assert torch.cuda.is_available()
    binding.load()
    return torch, binding


class Buffers:
    """All tensors of a workload carved out of guarded arenas, as raw descriptors."""

    def __init__(self, torch, binding, w, seed):
        self.torch, self.w = torch, w
        self.guards = []
        self.p, self.g, self.m, self.r, self.c, self.R, self.C = ([] for _ in range(7))
        params = synth.make_params(w, seed)
        self.descs = []
        for i, t in enumerate(w.tensors):
            p = self._guarded(t.numel, torch.float32); p.copy_(torch.from_numpy(params[i]).reshape(-1))
            gdt = torch.bfloat16 if w.grad_dtype == synth.BF16 else torch.float32
            g = self._guarded(t.numel, gdt)
            m = self._guarded(t.numel, torch.float32)
            r = self._guarded(t.rows, torch.float32); R = self._guarded(t.rows, torch.float32)
            c = self._guarded(t.cols, torch.float32) if t.ndim == 2 else None
            C = self._guarded(t.cols, torch.float32) if t.ndim == 2 else None
            for lst, x in zip((self.p, self.g, self.m, self.r, self.c, self.R, self.C),
                              (p, g, m, r, c, R, C)):
                lst.append(x)
            ptr = lambda x: x.data_ptr() if x is not None else None
            self.descs.append(binding.came_tensor(
                ptr(p), ptr(g), ptr(m), ptr(r), ptr(c), ptr(R), ptr(C), t.rows, t.cols, t.ndim,
                binding.CAME_BF16 if w.grad_dtype == synth.BF16 else binding.CAME_F32, 0, 0))

    def _guarded(self, n, dtype):
        torch = self.torch
        per = 4 // torch.empty(0, dtype=dtype).element_size()      # elements per float slot
        pad = GUARD * per
        body = (n + 63) // 64 * 64                                  # keeps the next guard 16-B aligned
        arena = torch.full((pad + body + pad,), SENT, dtype=dtype, device="cuda:0")
        self.guards.append((arena, pad, n))
        return arena[pad:pad + n]

    def set_grads(self, seed, step):
        for i, g in enumerate(self.g):
            g.copy_(to_torch_grad(self.torch, synth.make_grad(self.w, seed, i, step), "cuda:0").reshape(-1))

    def check_guards(self):
        for arena, pad, n in self.guards:
            a = arena.float().cpu().numpy()
            assert np.all(a[:pad] == SENT) and np.all(a[pad + n:] == SENT), "guard band overwritten"

    def snapshot(self):
        self.torch.cuda.synchronize()
        return [x.clone() for lst in (self.p, self.m, self.r, self.R, self.c, self.C)
                for x in lst if x is not None]


W_ODD = synth.Workload("odd", (synth.mat("a", 257, 1030), synth.mat("b", 33, 65), synth.mat("c", 1, 200),
                               synth.mat("d", 300, 1), synth.mat("e", 640, 1024), synth.vec("v", 1001),
                               synth.vec("s", 1)), synth.BF16, "normal_fixed", 1e-3, 0.0, (), 3, HP)


def _run_steps(torch, binding, buf, ctx, seed, first, last):
    stream = torch.cuda.current_stream().cuda_stream
    for step in range(first, last + 1):
        buf.set_grads(seed, step)
        binding.came_step(ctx, binding.make_hparams(step, **HP), None, stream)
    torch.cuda.synchronize()


def _same(a, b):
    return all(bool((x == y).all()) for x, y in zip(a, b))


def test_guard_bands_and_determinism(env):
    torch, binding = env
    snaps = []
    for _ in range(2):
        buf = Buffers(torch, binding, W_ODD, 3)
        ctx = binding.came_create(buf.descs)
        _run_steps(torch, binding, buf, ctx, 3, 1, 3)
        buf.check_guards()
        snaps.append(buf.snapshot())
        binding.came_destroy(ctx)
    assert _same(*snaps), "two identical runs differ: the reductions are not deterministic"


def test_resume_is_bit_exact(env):
    torch, binding = env
    a = Buffers(torch, binding, W_ODD, 5)
    ctx = binding.came_create(a.descs)
    _run_steps(torch, binding, a, ctx, 5, 1, 6)
    binding.came_destroy(ctx)
    b = Buffers(torch, binding, W_ODD, 5)
    ctx = binding.came_create(b.descs)
    _run_steps(torch, binding, b, ctx, 5, 1, 3)
    binding.came_destroy(ctx)
    ctx = binding.came_create(b.descs, flags=binding.CAME_CREATE_KEEP_STATE)
    assert binding.came_query(ctx, binding.CAME_Q_LAST_STEP) == 0
    _run_steps(torch, binding, b, ctx, 5, 4, 6)       # a resumed context accepts any first step
    binding.came_destroy(ctx)
    assert _same(a.snapshot(), b.snapshot())


def test_errors_do_not_launch(env):
    torch, binding = env
    buf = Buffers(torch, binding, W_ODD, 7)
    ctx = binding.came_create(buf.descs)
    _run_steps(torch, binding, buf, ctx, 7, 1, 1)
    before = buf.snapshot()
    stream = torch.cuda.current_stream().cuda_stream
    bad = [(dict(HP), 3, 6), (dict(HP), 1, 6), (dict(HP, beta1=1.0), 2, 5), (dict(HP, beta3=-0.1), 2, 5),
           (dict(HP, clip_d=0.0), 2, 5), (dict(HP, lr=float("nan")), 2, 5), (dict(HP, eps2=-1.0), 2, 5),
           (dict(HP, weight_decay=-1.0), 2, 5), (dict(HP), 0, 6)]
    for hp, step, status in bad:
        with pytest.raises(binding.CameError) as e:
            binding.came_step(ctx, binding.make_hparams(step, **hp), None, stream)
        assert e.value.status == status
    assert _same(before, buf.snapshot())
    assert binding.came_query(ctx, binding.CAME_Q_LAST_STEP) == 1
    assert binding.came_last_error(ctx) != ""
    with pytest.raises(binding.CameError) as e:
        binding.came_step(ctx, binding.make_hparams(2, **HP), [0] * len(buf.descs), stream)
    assert e.value.status == 1
    with pytest.raises(binding.CameError) as e:
        binding.came_query(ctx, 99)
    assert e.value.status == 11
    binding.came_destroy(ctx)
    with pytest.raises(binding.CameError) as e:
        binding.came_create(buf.descs, device=4096)
    assert e.value.status == 7


def test_gradient_rebinding_and_host_step(env):
    torch, binding = env
    stream = torch.cuda.current_stream().cuda_stream
    # reference: gradients copied into the buffers given at create
    a = Buffers(torch, binding, W_ODD, 9)
    ctx = binding.came_create(a.descs)
    _run_steps(torch, binding, a, ctx, 9, 1, 3)
    binding.came_destroy(ctx)
    # (1) fresh gradient buffers passed to every step
    b = Buffers(torch, binding, W_ODD, 9)
    ctx = binding.came_create(b.descs)
    keep = []
    for step in (1, 2, 3):
        gs = [to_torch_grad(torch, synth.make_grad(W_ODD, 9, i, step), "cuda:0").reshape(-1).clone()
              for i in range(len(W_ODD.tensors))]
        keep.append(gs)
        binding.came_step(ctx, binding.make_hparams(step, **HP), [g.data_ptr() for g in gs], stream)
    torch.cuda.synchronize()
    binding.came_destroy(ctx)
    assert _same(a.snapshot(), b.snapshot())
    # (2) the host-buffer entry point: pinned gradients in, parameters out
    c = Buffers(torch, binding, W_ODD, 9)
    ctx = binding.came_create(c.descs)
    outs = [torch.empty(t.numel, dtype=torch.float32).pin_memory() for t in W_ODD.tensors]
    for step in (1, 2, 3):
        hg = [to_torch_grad(torch, synth.make_grad(W_ODD, 9, i, step), "cpu").reshape(-1).pin_memory()
              for i in range(len(W_ODD.tensors))]
        binding.came_step_host(ctx, binding.make_hparams(step, **HP), [g.data_ptr() for g in hg],
                               [o.data_ptr() for o in outs], stream)
        torch.cuda.synchronize()
    binding.came_destroy(ctx)
    assert _same(a.snapshot(), c.snapshot())
    for o, p in zip(outs, c.p):
        assert bool((o == p.cpu()).all())


def test_queries_and_profiling(env):
    torch, binding = env
    w = synth.workload("toy")
    buf = Buffers(torch, binding, w, 11)
    ctx = binding.came_create(buf.descs)
    q = lambda k: binding.came_query(ctx, k)
    nm, nv = 512 * 256, 256
    assert q(binding.CAME_Q_NUMEL) == nm + nv
    assert q(binding.CAME_Q_MATRIX_NUMEL) == nm
    assert q(binding.CAME_Q_STATE_BYTES) == 4 * (nm + 2 * (512 + 256)) + 12 * nv
    assert q(binding.CAME_Q_STREAM_BYTES) == nm * 32 + 16 * (512 + 256) + nv * 36
    assert q(binding.CAME_Q_COMPULSORY_BYTES) == nm * 20 + 16 * (512 + 256) + nv * 36
    assert q(binding.CAME_Q_LAUNCHES_PER_STEP) == 4 and q(binding.CAME_Q_NUM_PHASES) == 4
    assert q(binding.CAME_Q_NUM_TILES) >= 1 and q(binding.CAME_Q_WORKSPACE_BYTES) > 0
    with pytest.raises(binding.CameError):
        binding.came_get_phase_ms(ctx)                 # nothing profiled yet
    binding.came_set_profiling(ctx, True)
    _run_steps(torch, binding, buf, ctx, 11, 1, 4)
    ms = binding.came_get_phase_ms(ctx)
    names = [binding.came_phase_name(ctx, i) for i in range(len(ms))]
    assert names == ["p1_reduce_g2", "p2_sum_u2", "p3_momentum_instability", "p4_apply"]
    assert all(0.0 < x < 50.0 for x in ms)
    binding.came_destroy(ctx)


def test_rank3_tensor_is_the_matrix_of_merged_leading_dims(env, oracle):
    torch, binding = env
    from tests.parity_util import err_signed
    w = synth.workload("mat:96x520")
    p0 = synth.make_params(w, 31)[0]
    g0 = synth.make_grad(w, 31, 0, 1)
    p = torch.from_numpy(p0.reshape(8, 12, 520).copy()).cuda()
    g = torch.from_numpy(g0.reshape(8, 12, 520).copy()).cuda()
    opt = binding.CameOptimizer([p], [g])
    opt.step(**HP)
    torch.cuda.synchronize()
    orc = oracle.OracleOptimizer([p0])
    orc.step([synth.widen(g0)], **HP)
    assert p.shape == (8, 12, 520)
    assert err_signed(p.cpu().numpy().reshape(96, 520), orc.p[0]) <= 1e-5
    opt.close()


def test_cuda_graph_replay_matches_eager_launches(env):
    """came_step neither synchronises nor allocates, so a caller may capture it in a CUDA graph
    and replay it; the replayed steps must equal eagerly launched ones bit for bit."""
    torch, binding = env
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
    side = torch.cuda.Stream()
    side.wait_stream(torch.cuda.current_stream())
    with torch.cuda.stream(side):
        binding.came_step(ctx, binding.make_hparams(1, **HP), None, side.cuda_stream)   # warm-up, eager
    torch.cuda.current_stream().wait_stream(side)
    torch.cuda.synchronize()
    graph = torch.cuda.CUDAGraph()
    with torch.cuda.graph(graph):
        binding.came_step(ctx, binding.make_hparams(2, **HP), None,
                          torch.cuda.current_stream().cuda_stream)
    for _ in range(3):          # steps 2, 3, 4 (capture itself runs nothing)
        graph.replay()
    torch.cuda.synchronize()
    binding.came_destroy(ctx)
    assert _same(a.snapshot(), b.snapshot())


def test_grouped_schedule_and_pipelined_host_step_are_bit_identical(env):
    """Scheduling knobs change launch order only: running group by group, or pipelining the
    host-buffer step over several groups, must reproduce the one-grid-per-phase result exactly."""
    torch, binding = env
    ref = Buffers(torch, binding, W_ODD, 15)
    ctx = binding.came_create(ref.descs)
    _run_steps(torch, binding, ref, ctx, 15, 1, 3)
    binding.came_destroy(ctx)
    want = ref.snapshot()

    binding.came_tune(binding.CAME_TUNE_SCHED_GROUP_BYTES, 100_000)     # ~ one or two tensors per group
    try:
        a = Buffers(torch, binding, W_ODD, 15)
        ctx = binding.came_create(a.descs)
        _run_steps(torch, binding, a, ctx, 15, 1, 3)
        binding.came_destroy(ctx)
    finally:
        binding.came_tune(binding.CAME_TUNE_SCHED_GROUP_BYTES, 0)
    assert _same(want, a.snapshot())

    binding.came_tune(binding.CAME_TUNE_HOST_GROUP_BYTES, 50_000)
    try:
        b = Buffers(torch, binding, W_ODD, 15)
        ctx = binding.came_create(b.descs)
        stream = torch.cuda.current_stream().cuda_stream
        outs = [torch.empty(t.numel, dtype=torch.float32).pin_memory() for t in W_ODD.tensors]
        for step in (1, 2, 3):
            hg = [to_torch_grad(torch, synth.make_grad(W_ODD, 15, i, step), "cpu").reshape(-1).pin_memory()
                  for i in range(len(W_ODD.tensors))]
            binding.came_step_host(ctx, binding.make_hparams(step, **HP), [g.data_ptr() for g in hg],
                                   [o.data_ptr() for o in outs], stream)
            torch.cuda.current_stream().synchronize()      # the caller's stream alone is enough
        binding.came_destroy(ctx)
    finally:
        binding.came_tune(binding.CAME_TUNE_HOST_GROUP_BYTES, 0)
    assert _same(want, b.snapshot())
    for o, p in zip(outs, b.p):
        assert bool((o == p.cpu()).all())


def test_two_contexts_on_two_streams_do_not_interfere(env):
    """Contexts share nothing on the device: stepping two of them concurrently on different
    streams gives each the result it gets alone."""
    torch, binding = env
    alone = []
    for seed in (21, 22):
        b = Buffers(torch, binding, W_ODD, seed)
        ctx = binding.came_create(b.descs)
        _run_steps(torch, binding, b, ctx, seed, 1, 3)
        binding.came_destroy(ctx)
        alone.append(b.snapshot())
    bufs = [Buffers(torch, binding, W_ODD, seed) for seed in (21, 22)]
    ctxs = [binding.came_create(b.descs) for b in bufs]
    streams = [torch.cuda.Stream(), torch.cuda.Stream()]
    for step in (1, 2, 3):
        for b, seed in zip(bufs, (21, 22)):
            b.set_grads(seed, step)
        torch.cuda.synchronize()
        for ctx, st in zip(ctxs, streams):
            binding.came_step(ctx, binding.make_hparams(step, **HP), None, st.cuda_stream)
        torch.cuda.synchronize()
    for ctx in ctxs:
        binding.came_destroy(ctx)
    assert _same(alone[0], bufs[0].snapshot()) and _same(alone[1], bufs[1].snapshot())


def test_replacement_gradient_must_match_the_planned_load_width(env):
    """The launch plan is fixed at create.  A tensor planned for 256-bit fp32 gradient loads
    rejects a replacement pointer at 16 mod 32 before anything is launched; a tensor planned
    for 128-bit loads accepts it and gives the result of the aligned buffer."""
    torch, binding = env
    w = synth.Workload("align", (synth.mat("a", 64, 1024), synth.mat("b", 64, 1028)), synth.F32,
                       "normal_fixed", 1e-3, 0.0, (), 2, HP)
    assert binding.came_plan_tensor(64, 1024, 2, 0, True)["vec"] == 8
    assert binding.came_plan_tensor(64, 1028, 2, 0, True)["vec"] == 4
    stream = torch.cuda.current_stream().cuda_stream
    ref = Buffers(torch, binding, w, 17)
    ctx = binding.came_create(ref.descs)
    _run_steps(torch, binding, ref, ctx, 17, 1, 2)
    binding.came_destroy(ctx)

    buf = Buffers(torch, binding, w, 17)
    for x in buf.g:
        assert x.data_ptr() % 32 == 0
    ctx = binding.came_create(buf.descs)
    _run_steps(torch, binding, buf, ctx, 17, 1, 1)
    before = buf.snapshot()
    buf.set_grads(17, 2)
    shifted = []
    for g in buf.g:                       # the same values, 16 bytes into a larger buffer
        big = torch.zeros(g.numel() + 16, dtype=torch.float32, device="cuda:0")
        off = ((16 - big.data_ptr() % 32) % 32) // 4
        view = big[off:off + g.numel()]
        view.copy_(g)
        assert view.data_ptr() % 32 == 16
        shifted.append((big, view))
    with pytest.raises(binding.CameError) as e:
        binding.came_step(ctx, binding.make_hparams(2, **HP),
                          [shifted[0][1].data_ptr(), buf.g[1].data_ptr()], stream)
    assert e.value.status == 4 and "32-byte" in str(e.value)
    assert _same(before, buf.snapshot())
    assert binding.came_query(ctx, binding.CAME_Q_LAST_STEP) == 1
    binding.came_step(ctx, binding.make_hparams(2, **HP),
                      [buf.g[0].data_ptr(), shifted[1][1].data_ptr()], stream)
    torch.cuda.synchronize()
    binding.came_destroy(ctx)
    buf.check_guards()
    assert _same(ref.snapshot(), buf.snapshot())


def test_step_with_another_device_current_is_refused(env):
    torch, binding = env
    if torch.cuda.device_count() < 2:
        pytest.skip("needs two GPUs; the comparison itself is covered by the CPU test of came_device_status")
    buf = Buffers(torch, binding, synth.workload("toy"), 19)
    ctx = binding.came_create(buf.descs, device=0)
    buf.set_grads(19, 1)
    before = buf.snapshot()
    with torch.cuda.device(1):
        with pytest.raises(binding.CameError) as e:
            binding.came_step(ctx, binding.make_hparams(1, **HP), None, 0)
    assert e.value.status == 7
    assert _same(before, buf.snapshot())
    binding.came_destroy(ctx)
