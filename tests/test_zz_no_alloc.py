"""The allocation-free entry point, came_factor_update_static, against came_step.

Some users of this library cannot allocate device memory when they step the optimizer: the
device heap belongs to their framework's memory pool, or an allocation's hidden
synchronisation would stall their loop, or their memory budget is fixed and audited at
start-up.  came_create allocates a workspace, so those users get one entry point that
keeps its partial sums in a fixed array inside the library.  This test calls it through the
C ABI twice in a row (the second call meets whatever the first left in that array) and
checks r and c against what the ordinary came_step path produces from the same gradients.

Collected last on purpose: a failure here cannot hide the result of any other test.
"""
import numpy as np
import pytest

from paper_2307_02047_b200 import synth
from tests.parity_util import TOL_STEP1, TOL_STEP10, err_positive, to_torch_grad

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("name", ["mat:1500x1288:bf16", "mat:513x1030", "mat:4096x1024:bf16"])
def test_static_scratch_matches_came_step_twice(name):
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
    stream = torch.cuda.current_stream().cuda_stream
    for step in (1, 2):
        if step > 1:
            g_dev[0].copy_(to_torch_grad(torch, synth.make_grad(w, 21, 0, step), dev))
        opt.step(**hp)
        binding.came_factor_update_static(g_dev[0].data_ptr(), gdt, t.rows, t.cols, r.data_ptr(),
                                          c.data_ptr(), hp["beta2"], hp["eps1"], ssr.data_ptr(),
                                          0, stream)
        torch.cuda.synchronize()
        tol = TOL_STEP1 if step == 1 else TOL_STEP10
        assert err_positive(r.cpu().numpy(), opt.r[0].cpu().numpy()) <= tol
        assert err_positive(c.cpu().numpy(), opt.c[0].cpu().numpy()) <= tol
        want = float(np.sqrt(opt.r[0].double().sum().item()))
        assert abs(float(ssr[0].item()) - want) <= tol * want
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
