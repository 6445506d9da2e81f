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
