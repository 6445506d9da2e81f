"""CPU-only checks of the C-ABI library: it loads, exports every symbol the header declares,
rejects bad arguments before touching CUDA, and its host-side tile planner covers every
matrix exactly once.  No GPU compute is called here."""
import ctypes
import os
import re

import pytest

from paper_2307_02047_b200 import binding, synth

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _declared_functions():
    text = open(os.path.join(ROOT, "include", "came_b200.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    return sorted(set(re.findall(r"\b(came_[a-z_]+)\s*\(", text)))


def test_every_declared_symbol_is_exported():
    L = binding.load()
    names = _declared_functions()
    assert len(names) >= 10
    for n in names:
        assert hasattr(L, n), f"{n} declared in the header but not exported"
    assert sorted(binding.EXPORTED) == names


def _desc(rows=8, cols=8, ndim=2, dt=0, base=0x10000, flags=0, **over):
    d = dict(param=base, grad=base + 0x1000, m=base + 0x2000, r=base + 0x3000,
             c=(base + 0x4000) if ndim == 2 else None, R=base + 0x5000,
             C=(base + 0x6000) if ndim == 2 else None)
    d.update(over)
    return binding.came_tensor(d["param"], d["grad"], d["m"], d["r"], d["c"], d["R"], d["C"],
                               rows, cols, ndim, dt, flags, 0)


@pytest.mark.parametrize("desc,status", [
    (dict(ndim=3), 2), (dict(rows=0), 2), (dict(cols=0), 2), (dict(ndim=1, cols=4), 2),
    (dict(dt=7), 3), (dict(param=None), 1), (dict(c=None), 1), (dict(C=None), 1),
    (dict(m=0x10008), 4), (dict(grad=0x10002), 4), (dict(flags=2), 2),
])
def test_create_rejects_bad_descriptors_without_cuda(desc, status):
    with pytest.raises(binding.CameError) as e:
        binding.came_create([_desc(**desc)])
    assert e.value.status == status
    assert binding.came_last_error(None) != ""


def test_create_null_and_count():
    L = binding.load()
    ctx = ctypes.c_void_p()
    assert L.came_create(None, None, 1, 0, 0) == 1
    assert L.came_create(ctypes.byref(ctx), None, 1, 0, 0) == 1
    arr = (binding.came_tensor * 1)(_desc())
    assert L.came_create(ctypes.byref(ctx), arr, 0, 0, 0) == 2
    assert L.came_create(ctypes.byref(ctx), arr, 1, 0, 0xF0) == 11
    assert ctx.value is None
    assert L.came_step(None, None, None, None) == 1
    assert L.came_destroy(None) == 1
    assert binding.came_status_string(5) == "CAME_ERR_HPARAM"


def test_create_without_gpu_reports_device_error():
    import torch
    if torch.cuda.is_available():
        pytest.skip("a GPU is present")
    with pytest.raises(binding.CameError) as e:
        binding.came_create([_desc()])
    assert e.value.status == 7      # CAME_ERR_DEVICE: no silent CPU fallback


SHAPES = [(1, 1), (1, 65536), (65536, 1), (30522, 768), (768, 3072), (3072, 768), (4096, 11008),
          (11008, 4096), (128256, 4096), (16384, 16384), (513, 1030), (50257, 1024), (7, 13)]


@pytest.mark.parametrize("dt", [0, 1])
@pytest.mark.parametrize("target", [0, 4096, 65536])
@pytest.mark.parametrize("shape", SHAPES)
def test_plan_covers_matrix_exactly(shape, dt, target):
    rows, cols = shape
    p = binding.came_plan_tensor(rows, cols, 2, dt, True, target)
    vec, tx, tr = p["vec"], p["threads_x"], p["tile_rows"]
    assert vec in (1, 4, 8) and tx in (32, 64, 128, 256)
    assert cols % vec == 0
    sw = tx * vec
    ty = 256 // tx
    assert tr >= 1 and tr % ty == 0
    # row blocks and column strips tile the matrix with no gap and no overlap
    assert (p["n_rb"] - 1) * tr < rows <= p["n_rb"] * tr
    assert (p["n_cb"] - 1) * sw < cols <= p["n_cb"] * sw
    assert p["n_rb"] <= 256 or tr >= rows // 256
    if dt == 1:
        assert vec in (1, 8)
    if cols % 8 == 0:
        assert vec == 8          # 256-bit accesses whenever rows start 32-byte aligned


def test_plan_unaligned_bf16_falls_back_to_scalar():
    assert binding.came_plan_tensor(64, 1024, 2, 1, False, 0)["vec"] == 1
    assert binding.came_plan_tensor(64, 1024, 2, 0, False, 0)["vec"] == 4
    assert binding.came_plan_tensor(64, 1022, 2, 0, True, 0)["vec"] == 1
    assert binding.came_plan_tensor(64, 1024, 2, 0, True, 0)["vec"] == 8
    assert binding.came_plan_tensor(64, 1028, 2, 0, True, 0)["vec"] == 4


def test_plan_rejects_bad_arguments():
    L = binding.load()
    o = [ctypes.c_int32() for _ in range(5)]
    refs = [ctypes.byref(x) for x in o]
    assert L.came_plan_tensor(0, 4, 2, 0, 1, 0, *refs) == 2
    assert L.came_plan_tensor(4, 4, 2, 9, 1, 0, *refs) == 3
    assert L.came_plan_tensor(4, 4, 2, 0, 1, 0, None, *refs[1:]) == 1
    assert L.came_tune(99, 1) == 11


def test_workload_shapes_match_the_named_models():
    counts = {"toy": (1, 1, 512 * 256 + 256), "bert_base": (74, 120, 108_888_576),
              "bert_large": (146, 240, 334_088_192), "gpt2_medium": (98, 192, 354_821_120),
              "llama7b": (226, 65, 6_738_415_616)}
    for name, (nm, nv, numel) in counts.items():
        w = synth.workload(name)
        assert sum(t.ndim == 2 for t in w.tensors) == nm
        assert sum(t.ndim == 1 for t in w.tensors) == nv
        assert w.numel == numel


def test_header_is_plain_c():
    """The boundary is a C ABI: the header must compile as C99 on its own."""
    import subprocess, tempfile
    with tempfile.TemporaryDirectory() as d:
        src = os.path.join(d, "t.c")
        with open(src, "w") as f:
            f.write('#include "came_b200.h"\nint main(void) { came_hparams h; (void)h; return 0; }\n')
        res = subprocess.run(["gcc", "-std=c99", "-Wall", "-Wextra", "-pedantic", "-Werror",
                              "-fsyntax-only", "-I", os.path.join(ROOT, "include"), src],
                             capture_output=True, text=True)
        assert res.returncode == 0, res.stderr


# ---------------------------------------------------------------------------
# alignment and device checks that must hold before anything is launched
# ---------------------------------------------------------------------------
def test_static_plan_follows_the_gradient_pointer_alignment():
    """The allocation-free entry point plans 256-bit loads of fp32 gradients only for a
    32-byte aligned pointer; a pointer at 16 mod 32 (a view into a flat buffer) gets 128-bit
    loads, never a wider access than its alignment allows."""
    base, r, c = 0x7f0000000000, 0x7f0000100000, 0x7f0000200000
    F32, BF16 = binding.CAME_F32, binding.CAME_BF16
    plan = binding.came_factor_update_static_plan
    assert plan(base, F32, 512, 1024, r, c)["vec"] == 8
    assert plan(base + 16, F32, 512, 1024, r, c)["vec"] == 4
    assert plan(base + 16, F32, 512, 1028, r, c)["vec"] == 4        # cols % 8 != 0
    assert plan(base, F32, 512, 1028, r, c)["vec"] == 4
    assert plan(base + 16, F32, 512, 1030, r, c)["vec"] == 1
    assert plan(base + 16, BF16, 512, 1024, r, c)["vec"] == 8       # one 128-bit load of 8 bf16
    for off in (4, 8, 2):
        with pytest.raises(binding.CameError) as e:
            plan(base + off, F32, 512, 1024, r, c)
        assert e.value.status == 4
    with pytest.raises(binding.CameError) as e:
        plan(base, F32, 3_000_000, 4, r, c)
    assert e.value.status == 11
    assert plan(base, F32, 4096, 4096, r, c)["scratch_bytes"] <= binding.CAME_STATIC_SCRATCH_BYTES
    for a in range(0, 64, 16):
        v = plan(base + a, F32, 64, 4096, r, c)["vec"]
        assert (base + a) % binding.came_required_grad_alignment(F32, v) == 0


def test_required_gradient_alignment():
    assert binding.came_required_grad_alignment(binding.CAME_F32, 8) == 32
    assert binding.came_required_grad_alignment(binding.CAME_F32, 4) == 16
    assert binding.came_required_grad_alignment(binding.CAME_F32, 1) == 16
    assert binding.came_required_grad_alignment(binding.CAME_BF16, 8) == 16
    assert binding.came_required_grad_alignment(binding.CAME_BF16, 1) == 16


def test_device_status_comparison():
    assert binding.came_device_status(0, 0) == 0
    assert binding.came_device_status(3, 3) == 0
    assert binding.came_device_status(0, 1) == 7
    assert binding.came_device_status(1, 0) == 7
    assert binding.came_device_status(-1, -1) == 7


def test_lr_warmup_is_a_linear_ramp_to_the_peak():
    f = binding.came_lr_warmup
    assert f(2e-4, 0.0, 1, 10) == pytest.approx(2e-5, rel=1e-15)
    assert f(2e-4, 0.0, 5, 10) == pytest.approx(1e-4, rel=1e-15)
    assert f(2e-4, 0.0, 10, 10) == 2e-4
    assert f(2e-4, 0.0, 11, 10) == 2e-4
    assert f(2e-4, 1e-5, 0, 10) == 1e-5
    assert f(2e-4, 1e-5, 4, 8) == pytest.approx(1e-5 + 0.5 * (2e-4 - 1e-5), rel=1e-15)
    assert f(6e-4, 0.0, 3, 0) == 6e-4
    vals = [f(3e-4, 0.0, t, 100) for t in range(0, 120)]
    assert all(b >= a for a, b in zip(vals, vals[1:])) and max(vals) == 3e-4


def test_create_rejects_overlapping_buffers_without_cuda():
    """Two buffers that share memory are refused before any CUDA call (status 12)."""
    def wide(base=0x100000, **over):          # a 64 x 64 matrix, buffers 64 KiB apart (param is 16 KiB)
        f = dict(param=base, grad=base + 0x10000, m=base + 0x20000, r=base + 0x30000,
                 c=base + 0x40000, R=base + 0x50000, C=base + 0x60000)
        f.update(over)
        return binding.came_tensor(f["param"], f["grad"], f["m"], f["r"], f["c"], f["R"], f["C"],
                                   64, 64, 2, 0, 0, 0)
    numel_bytes = 4 * 64 * 64
    for over in (dict(grad=0x100000 + 64),                          # grad starts inside param
                 dict(m=0x110000 + numel_bytes - 16),               # m starts on grad's last 16 bytes
                 dict(r=0x120000 + numel_bytes - 16),               # r overlaps the end of m
                 dict(C=0x130000)):                                 # C on top of r
        with pytest.raises(binding.CameError) as e:
            binding.came_create([wide(**over)])
        assert e.value.status == 12, (over, e.value.status)
        assert "overlap" in str(e.value)
    # two tensors sharing one gradient buffer
    a = wide()
    b = wide(base=0x800000, grad=0x110000)
    with pytest.raises(binding.CameError) as e:
        binding.came_create([a, b])
    assert e.value.status == 12 and "tensor 0" in str(e.value) and "tensor 1" in str(e.value)
    # buffers that touch but do not overlap pass this check: the next one to fail is the device's
    import torch
    if not torch.cuda.is_available():
        with pytest.raises(binding.CameError) as e:
            binding.came_create([wide(grad=0x100000 + numel_bytes)])
        assert e.value.status == 7
    assert binding.came_status_string(12) == "CAME_ERR_OVERLAP"


def test_debug_build_exports_the_same_symbols_and_ordinary_build_has_no_record():
    L = binding.load_debug()
    for n in _declared_functions():
        assert hasattr(L, n), f"{n} missing from the bounds-checking build"
    with pytest.raises(binding.CameError) as e:
        binding.came_debug_bounds(0)                 # ordinary build: no record to read
    assert e.value.status == 11
