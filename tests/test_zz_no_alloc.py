"""The allocation-free entry point, came_factor_update_static, against came_step and against
the CPU oracle.

Some users of this library cannot allocate device memory when they step the optimizer: the
device heap belongs to their framework's memory pool, or an allocation's hidden
synchronisation would stall their loop, or their memory budget is fixed and audited at
start-up.  came_create allocates a workspace, so those users get one entry point that
keeps its partial sums in a fixed array inside the library.  These tests call it through the
C ABI twice in a row (the second call meets whatever the first left in that array) and
check r, c and sqrt(sum r) against what the ordinary came_step path produces from the same
gradients, and against the float64 oracle's row/column EMA of the first two lines of
Algorithm 2.  Every load width of the entry point is covered: 8 bf16 per thread, 8 fp32
(256-bit, 32-byte aligned gradient), 4 fp32 (128-bit: columns not a multiple of 8, or a
gradient pointer that is only 16-byte aligned) and one element at a time.

Collected last on purpose: a failure here cannot hide the result of any other test.
"""
import numpy as np
import pytest

from paper_2307_02047_b200 import synth
from tests.parity_util import TOL_STEP1, TOL_STEP10, err_positive, to_torch_grad

pytestmark = pytest.mark.gpu

CASES = [("mat:1500x1288:bf16", 0, 8), ("mat:513x1030", 0, 1), ("mat:4096x1024:bf16", 0, 8),
         ("mat:700x2048", 0, 8),        # fp32, cols % 8 == 0, 32-byte aligned: 256-bit loads
         ("mat:700x2044", 0, 4),        # fp32, cols % 4 == 0 only: 128-bit loads
         ("mat:700x2048", 16, 4)]       # fp32 view 16 bytes into a buffer: must fall back to 128-bit


@pytest.mark.parametrize("name,byte_offset,want_vec", CASES)
def test_static_scratch_matches_came_step_and_oracle_twice(name, byte_offset, want_vec, oracle):
    import torch
    from paper_2307_02047_b200 import binding
    assert torch.cuda.is_available()
    w = synth.workload(name)
    t = w.tensors[0]
    hp = dict(w.hparams)
    dev = "cuda:0"
    params = [torch.from_numpy(synth.make_params(w, 21)[0]).to(dev)]
    g_dev = [to_torch_grad(torch, synth.make_grad(w, 21, 0, 1), dev)]
    opt = binding.CameOptimizer(params, g_dev)              # the existing entry points
    r = torch.zeros(t.rows, dtype=torch.float32, device=dev)
    c = torch.zeros(t.cols, dtype=torch.float32, device=dev)
    ssr = torch.zeros(4, dtype=torch.float32, device=dev)
    gdt = binding.CAME_BF16 if w.grad_dtype == synth.BF16 else binding.CAME_F32
    # the gradient as the static entry point sees it: the same values, optionally at an offset
    esz = g_dev[0].element_size()
    big = torch.zeros(t.numel + 64, dtype=g_dev[0].dtype, device=dev)
    start = ((byte_offset - big.data_ptr() % 32) % 32) // esz
    g_static = big[start:start + t.numel]
    assert g_static.data_ptr() % 32 == byte_offset
    # the plan is checked on the host before anything runs on that pointer
    plan = binding.came_factor_update_static_plan(g_static.data_ptr(), gdt, t.rows, t.cols,
                                                  r.data_ptr(), c.data_ptr(), hp["beta2"], hp["eps1"])
    assert plan["vec"] == want_vec
    assert g_static.data_ptr() % binding.came_required_grad_alignment(gdt, plan["vec"]) == 0
    r64, c64 = np.zeros(t.rows), np.zeros(t.cols)           # the oracle's r_t, c_t
    stream = torch.cuda.current_stream().cuda_stream
    for step in (1, 2):
        g_host = synth.make_grad(w, 21, 0, step)
        g_dev[0].copy_(to_torch_grad(torch, g_host, dev))
        g_static.copy_(g_dev[0].reshape(-1))
        opt.step(**hp)
        binding.came_factor_update_static(g_static.data_ptr(), gdt, t.rows, t.cols, r.data_ptr(),
                                          c.data_ptr(), hp["beta2"], hp["eps1"], ssr.data_ptr(),
                                          0, stream)
        torch.cuda.synchronize()
        g64 = synth.widen(g_host)
        oracle.factor_ema(np.ascontiguousarray(g64 * g64), hp["eps1"], hp["beta2"], r64, c64)
        tol = TOL_STEP1 if step == 1 else TOL_STEP10
        assert err_positive(r.cpu().numpy(), opt.r[0].cpu().numpy()) <= tol
        assert err_positive(c.cpu().numpy(), opt.c[0].cpu().numpy()) <= tol
        assert err_positive(r.cpu().numpy(), r64) <= tol
        assert err_positive(c.cpu().numpy(), c64) <= tol
        want = float(np.sqrt(opt.r[0].double().sum().item()))
        assert abs(float(ssr[0].item()) - want) <= tol * want
        assert abs(float(ssr[0].item()) - np.sqrt(r64.sum())) <= tol * np.sqrt(r64.sum())
    opt.close()


def test_static_scratch_rejects_what_does_not_fit():
    import torch
    from paper_2307_02047_b200 import binding
    g = torch.zeros(16, dtype=torch.float32, device="cuda:0")
    # 3M rows: the per-row partial sums and scales alone exceed the 8 MiB array
    with pytest.raises(binding.CameError) as e:
        binding.came_factor_update_static(g.data_ptr(), binding.CAME_F32, 3_000_000, 4,
                                          g.data_ptr(), g.data_ptr(), 0.999, 1e-30)
    assert e.value.status == 11 and "scratch" in str(e.value)
    with pytest.raises(binding.CameError) as e:
        binding.came_factor_update_static(g.data_ptr(), binding.CAME_F32, 4, 4, g.data_ptr(),
                                          g.data_ptr(), 1.5, 1e-30)
    assert e.value.status == 5
    with pytest.raises(binding.CameError) as e:         # misaligned pointers never reach a kernel
        binding.came_factor_update_static(g.data_ptr() + 4, binding.CAME_F32, 2, 4, g.data_ptr(),
                                          g.data_ptr(), 0.999, 1e-30)
    assert e.value.status == 4
