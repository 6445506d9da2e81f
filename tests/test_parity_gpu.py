"""GPU parity: the CUDA library, called through its C ABI, against the CPU float64 oracle
on identical seeded inputs.  Gates: 1e-5 after one step, 1e-4 after ten steps."""
import numpy as np
import pytest

from paper_2307_02047_b200 import synth
from tests.parity_util import TOL_STEP1, TOL_STEP10, gate, run_paired

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def env(oracle):
    import torch
    from paper_2307_02047_b200 import binding
    assert torch.cuda.is_available(), "GPU tests need a CUDA device"
    binding.load()
    return torch, binding, oracle


def _gate(res):
    gate(res)


def test_toy_config_ten_steps(env):
    torch, binding, oracle = env
    _gate(run_paired(torch, binding, oracle, synth.workload("toy"), seed=1, steps=10, check_at=(1, 10)))


SHAPES = [(1, 1), (1, 37), (37, 1), (5, 3), (33, 65), (64, 256), (257, 1030), (1000, 72),
          (300, 2052), (2, 4096), (1, 65536), (65536, 1), (777, 768), (513, 3072)]


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("shape", SHAPES)
def test_single_matrix_shapes(env, shape, dtype):
    torch, binding, oracle = env
    w = synth.workload(f"mat:{shape[0]}x{shape[1]}" + (":bf16" if dtype == "bf16" else ""))
    _gate(run_paired(torch, binding, oracle, w, seed=3, steps=3, check_at=(1, 3)))


@pytest.mark.parametrize("tile", [4096, 8192, 65536])
def test_tile_sizes_span_many_tiles(env, tile):
    torch, binding, oracle = env
    binding.came_tune(binding.CAME_TUNE_TILE_ELEMS, tile)
    try:
        w = synth.workload("mat:1500x1288:bf16")
        _gate(run_paired(torch, binding, oracle, w, seed=5, steps=10, check_at=(1, 10)))
    finally:
        binding.came_tune(binding.CAME_TUNE_TILE_ELEMS, 0)


@pytest.mark.parametrize("n", [1, 7, 256, 4097, 100003])
def test_vectors(env, n):
    torch, binding, oracle = env
    w = synth.Workload("v", (synth.vec("b", n),), synth.F32, "normal_fixed", 1e-3, 0.0, (), 3,
                       dict(synth.PAPER_HPARAMS))
    _gate(run_paired(torch, binding, oracle, w, seed=7, steps=3, check_at=(1, 3)))


def test_flags_weight_decay_and_no_confidence(env):
    torch, binding, oracle = env
    ts = (synth.mat("w0", 130, 264), synth.mat("w1", 64, 128), synth.vec("b0", 300), synth.vec("b1", 300))
    # lr * lambda * |theta| is 2e-4 of the first update here: a dropped decay term, or a
    # dropped opt-out flag, moves the cumulative update by 20 times the step-1 gate
    hp = dict(synth.PAPER_HPARAMS, lr=1e-3, weight_decay=0.1)
    w = synth.Workload("flags", ts, synth.BF16, "student_t3", 1e-3, 0.0, (), 10, hp)
    flags = [0, binding.CAME_T_NO_WEIGHT_DECAY, binding.CAME_T_VEC_NO_CONFIDENCE,
             binding.CAME_T_NO_WEIGHT_DECAY]
    _gate(run_paired(torch, binding, oracle, w, seed=9, steps=10, check_at=(1, 10), flags=flags))


def test_zero_rows_everywhere(env):
    torch, binding, oracle = env
    ts = (synth.mat("e", 3000, 256), synth.mat("w", 256, 1024), synth.vec("b", 256))
    w = synth.Workload("z", ts, synth.BF16, "normal_loguniform", 0.0, 0.0, (), 10,
                       dict(synth.PAPER_HPARAMS))
    w = synth.with_zero_rows_everywhere(w, 0.2)
    res = run_paired(torch, binding, oracle, w, seed=11, steps=10, check_at=(1, 10))
    _gate(res)


def test_other_hyperparameters(env):
    torch, binding, oracle = env
    hp = dict(lr=1e-3, beta1=0.8, beta2=0.99, beta3=0.999, eps1=1e-12, eps2=1e-6, clip_d=0.5,
              weight_decay=0.1)
    _gate(run_paired(torch, binding, oracle, synth.workload("toy"), seed=13, steps=10,
                     check_at=(1, 10), hparams=hp))
    hp0 = dict(synth.PAPER_HPARAMS, beta1=0.0, clip_d=100.0)
    _gate(run_paired(torch, binding, oracle, synth.workload("toy"), seed=13, steps=3,
                     check_at=(1, 3), hparams=hp0))


# ---------------------------------------------------------------------------
# Algorithm 1 (Adafactor with momentum) on the same kernels
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("name", ["toy", "mat:257x1030:bf16", "mat:1x4096", "mat:777x768"])
def test_adafactor_mode(env, name):
    torch, binding, oracle = env
    w = synth.workload(name)
    hp = dict(w.hparams, weight_decay=0.01)
    _gate(run_paired(torch, binding, oracle, w, seed=17, steps=10, check_at=(1, 10), hparams=hp,
                     algorithm="adafactor"))


def test_adafactor_mode_needs_no_instability_state(env):
    torch, binding, oracle = env
    w = synth.workload("toy")
    params = synth.make_params(w, 19)
    p = [torch.from_numpy(x).cuda() for x in params]
    g = [torch.from_numpy(x).cuda() for x in synth.make_grads(w, 19, 1)]
    m = [torch.empty_like(x) for x in p]
    r = [torch.empty(512, device="cuda"), torch.empty(256, device="cuda")]
    c = torch.empty(256, device="cuda")
    descs = [binding.came_tensor(p[0].data_ptr(), g[0].data_ptr(), m[0].data_ptr(), r[0].data_ptr(),
                                 c.data_ptr(), None, None, 512, 256, 2, 0, 0, 0),
             binding.came_tensor(p[1].data_ptr(), g[1].data_ptr(), m[1].data_ptr(), r[1].data_ptr(),
                                 None, None, None, 256, 1, 1, 0, 0, 0)]
    with pytest.raises(binding.CameError) as e:
        binding.came_create(descs)                      # Algorithm 2 needs R and C
    assert e.value.status == 1
    ctx = binding.came_create(descs, flags=binding.CAME_CREATE_ADAFACTOR)
    assert binding.came_query(ctx, binding.CAME_Q_LAUNCHES_PER_STEP) == 3
    binding.came_step(ctx, binding.make_hparams(1, **w.hparams), None,
                      torch.cuda.current_stream().cuda_stream)
    torch.cuda.synchronize()
    orc = oracle.OracleOptimizer(params, algorithm="adafactor")
    orc.step([synth.widen(x) for x in synth.make_grads(w, 19, 1)], **w.hparams)
    from tests.parity_util import err_signed
    assert err_signed(p[0].cpu().numpy(), orc.p[0]) <= TOL_STEP1
    assert err_signed(p[1].cpu().numpy(), orc.p[1]) <= TOL_STEP1
    binding.came_destroy(ctx)


# ---------------------------------------------------------------------------
# steps either side of the path, fused into its passes: gradient pre-scale, bf16 copy of theta
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("algorithm", ["came", "adafactor"])
def test_grad_scale_and_bf16_copy(env, algorithm):
    torch, binding, oracle = env
    ts = (synth.mat("a", 257, 1032), synth.mat("b", 300, 516), synth.mat("c", 33, 65),
          synth.vec("v", 1001))
    for dt in (synth.BF16, synth.F32):
        hp = dict(synth.PAPER_HPARAMS, grad_scale=1.0 / 48.0, eps1=1e-12)
        w = synth.Workload("fused", ts, dt, "normal_fixed", 1e-3, 0.0, (), 10, hp)
        _gate(run_paired(torch, binding, oracle, w, seed=23, steps=10, check_at=(1, 10),
                         algorithm=algorithm, bf16_copy=True))


def test_grad_scale_is_validated(env):
    torch, binding, oracle = env
    w = synth.workload("toy")
    p = [torch.from_numpy(x).cuda() for x in synth.make_params(w, 1)]
    g = [torch.from_numpy(x).cuda() for x in synth.make_grads(w, 1, 1)]
    opt = binding.CameOptimizer(p, g)
    with pytest.raises(binding.CameError) as e:
        opt.step(**dict(w.hparams, grad_scale=-2.0))
    assert e.value.status == 5
    opt.close()


# ---------------------------------------------------------------------------
# degenerate inputs
# ---------------------------------------------------------------------------
def test_all_zero_gradients_stay_finite_and_match(env):
    torch, binding, oracle = env
    ts = (synth.mat("a", 130, 264), synth.mat("b", 1, 40), synth.vec("v", 300))
    hp = dict(synth.PAPER_HPARAMS, weight_decay=0.01)
    w = synth.Workload("zeros", ts, synth.BF16, "normal_fixed", 0.0, 0.0, (), 3, hp)   # scale 0: g == 0
    res = run_paired(torch, binding, oracle, w, seed=27, steps=3, check_at=(1, 3))
    _gate(res)


def test_nan_in_one_tensor_does_not_touch_the_others(env):
    """Tensors are independent in Algorithm 2; a non-finite gradient propagates inside its own
    tensor only (the paper has no skip logic, and none is added)."""
    torch, binding, oracle = env
    ts = (synth.mat("a", 64, 264), synth.mat("b", 130, 520), synth.vec("v", 300), synth.vec("u", 77))
    w = synth.Workload("nan", ts, synth.F32, "normal_fixed", 1e-3, 0.0, (), 2, dict(synth.PAPER_HPARAMS))
    outs = []
    for poison in (False, True):
        p = [torch.from_numpy(x).cuda() for x in synth.make_params(w, 29)]
        g = [torch.from_numpy(x).cuda() for x in synth.make_grads(w, 29, 1)]
        if poison:
            g[0][3, 5] = float("nan")
            g[2][10] = float("inf")
        opt = binding.CameOptimizer(p, g)
        opt.step(**w.hparams)
        opt.step(**w.hparams)
        torch.cuda.synchronize()
        outs.append([x.clone() for x in p] + [x.clone() for x in opt.m] + [opt.r[1].clone(), opt.C[1].clone()])
        if poison:
            assert not bool(p[0].isfinite().all()) and not bool(p[2].isfinite().all())
        opt.close()
    clean, dirty = outs
    for i in (1, 3, 5, 7, 8, 9):                      # everything belonging to tensors 1 and 3
        assert bool((clean[i] == dirty[i]).all())


# ---------------------------------------------------------------------------
# seeded random sweep: shapes, gradient types, tile sizes, hyper-parameters, flags
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("case", range(24))
def test_random_configurations(env, case):
    torch, binding, oracle = env
    rng = np.random.default_rng(1000 + case)
    def dim():
        k = rng.integers(0, 4)
        return int([rng.integers(1, 9), rng.integers(9, 200), rng.integers(200, 1500),
                    8 * rng.integers(16, 300)][k])
    ts = []
    for i in range(int(rng.integers(1, 5))):
        if rng.random() < 0.25:
            ts.append(synth.vec(f"v{i}", int(rng.integers(1, 6000))))
        else:
            ts.append(synth.mat(f"m{i}", dim(), dim()))
    dt = synth.BF16 if rng.random() < 0.5 else synth.F32
    hp = dict(lr=float(10 ** rng.uniform(-5, -2)), beta1=float(rng.choice([0.0, 0.5, 0.9, 0.99])),
              beta2=float(rng.choice([0.9, 0.999])), beta3=float(rng.choice([0.99, 0.9999])),
              eps1=float(rng.choice([1e-30, 1e-16, 1e-9])), eps2=float(rng.choice([1e-16, 1e-8])),
              clip_d=float(rng.choice([0.1, 1.0, 100.0])), weight_decay=float(rng.choice([0.0, 0.01])),
              grad_scale=float(rng.choice([1.0, 0.125, 3.0])))
    kind = str(rng.choice(["normal_fixed", "student_t3"]))
    w = synth.Workload(f"rand{case}", tuple(ts), dt, kind, float(10 ** rng.uniform(-5, -1)), 0.0, (), 4, hp)
    flags = []
    for t in ts:
        f = binding.CAME_T_NO_WEIGHT_DECAY if rng.random() < 0.3 else 0
        if t.ndim == 1 and rng.random() < 0.3:
            f |= binding.CAME_T_VEC_NO_CONFIDENCE
        flags.append(f)
    binding.came_tune(binding.CAME_TUNE_TILE_ELEMS, int(rng.choice([0, 4096, 16384])))
    try:
        res = run_paired(torch, binding, oracle, w, seed=case, steps=4, check_at=(1, 4), flags=flags,
                         algorithm="adafactor" if rng.random() < 0.2 else "came",
                         bf16_copy=bool(rng.random() < 0.3))
    finally:
        binding.came_tune(binding.CAME_TUNE_TILE_ELEMS, 0)
    _gate(res)
