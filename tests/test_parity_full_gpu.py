"""Full-size GPU parity: the five workload configurations at their real sizes, in the launch
configuration the benchmark times (default tile planning, all tensors in one context).

BERT-base/-large- and GPT-2-medium-shaped sets are checked in full against the oracle at
steps 1 and 10.  The LLaMA-7B-shaped set (6.74 B parameters) runs in full on the GPU while the
oracle, which is exact per tensor because tensors are independent, follows one tensor of every
distinct shape element by element.  The large single matrices of the shape sweep are checked
in full.  Gates: 1e-5 after step 1, 1e-4 afterwards.
"""
import os

import pytest

from paper_2307_02047_b200 import synth
from tests.parity_util import TOL_STEP1, TOL_STEP10, run_paired

pytestmark = pytest.mark.gpu
WORKERS = max(1, min(16, os.cpu_count() or 1))


@pytest.fixture(scope="module")
def env(oracle):
    import torch
    from paper_2307_02047_b200 import binding
    assert torch.cuda.is_available()
    binding.load()
    return torch, binding, oracle


def _gate(res, label=""):
    assert res
    print("PARITY", label, {k: {n: float("%.3g" % e) for n, e in v.items()} for k, v in res.items()})
    for step, worst in res.items():
        tol = TOL_STEP1 if step == 1 else TOL_STEP10
        for name, e in worst.items():
            assert e <= tol, f"step {step}: {name} error {e:.3e} > {tol:.0e}  ({worst})"


@pytest.mark.parametrize("name", ["bert_base", "bert_large", "gpt2_medium"])
def test_model_shaped_sets_steps_1_and_10(env, name):
    torch, binding, oracle = env
    w = synth.workload(name)
    _gate(run_paired(torch, binding, oracle, w, seed=2, steps=10, check_at=(1, 10), workers=WORKERS), name)


def test_bert_large_zero_rows_in_every_matrix(env):
    torch, binding, oracle = env
    w = synth.with_zero_rows_everywhere(synth.workload("bert_large"))
    # the oracle follows the embeddings, one layer's matrices and a few vectors
    idx = [0, 1] + list(range(2, 18)) + [1000 % len(w.tensors)]
    _gate(run_paired(torch, binding, oracle, w, seed=4, steps=3, check_at=(1, 3), oracle_idx=idx,
                     workers=WORKERS), "bert_large+zero_rows")


def test_llama7b_full_set_sampled_tensors(env):
    torch, binding, oracle = env
    w = synth.workload("llama7b")
    names = {t.name: i for i, t in enumerate(w.tensors)}
    idx = [names[n] for n in ("tok_emb", "l0.wq", "l0.w_gate", "l0.w_down", "l0.norm1",
                              "l17.wo", "l31.w_up", "l31.norm2", "norm_f")]
    _gate(run_paired(torch, binding, oracle, w, seed=6, steps=2, check_at=(1, 2), oracle_idx=idx,
                     workers=WORKERS), "llama7b")


@pytest.mark.parametrize("shape", [(1024, 1024), (4096, 4096), (8192, 8192), (16384, 16384),
                                   (128256, 4096)])
def test_shape_sweep_large_matrices(env, shape):
    torch, binding, oracle = env
    w = synth.workload(f"mat:{shape[0]}x{shape[1]}")
    steps = 5 if shape[0] * shape[1] <= 1 << 26 else 2
    _gate(run_paired(torch, binding, oracle, w, seed=8, steps=steps, check_at=(1, steps),
                     workers=WORKERS), w.name)


def test_bert_base_adafactor_mode(env):
    torch, binding, oracle = env
    w = synth.workload("bert_base")
    _gate(run_paired(torch, binding, oracle, w, seed=2, steps=10, check_at=(1, 10), workers=WORKERS,
                     algorithm="adafactor"), "bert_base/adafactor")


def test_matrix_with_more_than_2_pow_31_elements(env):
    """Index arithmetic beyond 32 bits.  A matrix that is a K x K tiling of a small base block B
    has, by Algorithm 2's own algebra, r and R equal to K times the base's (tiled), c and C
    likewise, and v, u, m, S, theta equal to the base's in every copy (the factor K*K cancels
    in r c / sum r).  So the oracle steps the base block and every copy of the 2.2 G-element
    result is checked against it."""
    torch, binding, oracle = env
    import numpy as np
    from tests.parity_util import err_signed, err_positive
    nb, mb, K = 1024, 2056, 32                      # 32768 x 65792 = 2,155,872,256 elements
    w = synth.workload(f"mat:{nb}x{mb}:bf16")
    hp = dict(w.hparams)
    p0 = synth.make_params(w, 41)[0]
    dev = "cuda:0"
    p = torch.from_numpy(p0).to(dev).repeat(K, K).contiguous()
    g = torch.empty((nb * K, mb * K), dtype=torch.bfloat16, device=dev)
    assert p.numel() > 2 ** 31
    opt = binding.CameOptimizer([p], [g])
    orc = oracle.OracleOptimizer([p0])
    for step in (1, 2):
        gb = synth.make_grad(w, 41, 0, step)
        g.copy_(torch.from_numpy(gb.view(np.int16)).view(torch.bfloat16).to(dev).repeat(K, K))
        opt.step(**hp)
        orc.step([synth.widen(gb)], **hp)
    torch.cuda.synchronize()
    tol = TOL_STEP10
    ref_p = torch.from_numpy(orc.p[0]).to(dev)
    ref_m = torch.from_numpy(orc.m[0]).to(dev)
    rms_p, rms_m = float(ref_p.square().mean().sqrt()), float(ref_m.square().mean().sqrt())
    worst_p = worst_m = 0.0
    for bi in range(K):                              # one block row at a time keeps temporaries small
        blk_p = p[bi * nb:(bi + 1) * nb].view(nb, K, mb).double()
        blk_m = opt.m[0][bi * nb:(bi + 1) * nb].view(nb, K, mb).double()
        ep = ((blk_p - ref_p[:, None, :]).abs() / (ref_p.abs()[:, None, :] + rms_p)).max()
        em = ((blk_m - ref_m[:, None, :]).abs() / (ref_m.abs()[:, None, :] + rms_m)).max()
        worst_p, worst_m = max(worst_p, float(ep)), max(worst_m, float(em))
    assert worst_p <= tol and worst_m <= tol, (worst_p, worst_m)
    for got, want in ((opt.r[0], np.tile(orc.r[0], K) * K), (opt.c[0], np.tile(orc.c[0], K) * K),
                      (opt.R[0], np.tile(orc.R[0], K) * K), (opt.C[0], np.tile(orc.C[0], K) * K)):
        assert err_positive(got.cpu().numpy(), want) <= tol
    print("PARITY >2^31", dict(p=worst_p, m=worst_m))
    opt.close()
