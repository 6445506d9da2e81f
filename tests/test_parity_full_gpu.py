"""Full-size GPU parity: the five workload configurations at their real sizes and at their
stated step counts, in the launch configuration the benchmark times (default tile planning,
all tensors in one context).

BERT-base/-large- and GPT-2-medium-shaped sets run their 100 / 50 / 20 steps and are checked
in full against the oracle at steps 1, 10 and the last.  The LLaMA-7B-shaped set (6.74 B
parameters) runs its 5 steps in full on the GPU while the oracle, which is exact per tensor
because tensors are independent, follows one tensor of every distinct shape element by
element.  The single matrices of the shape sweep run their 5 steps and are checked in full.
Gates: 1e-5 after step 1, 1e-4 at every later checked step, on p, m, r, c, R, C and on the
cumulative update theta_t - theta_0; the strict element-wise figures for p and m are printed.
"""
import json
import os

import pytest

from paper_2307_02047_b200 import synth
from tests.parity_util import TOL_STEP1, TOL_STEP10, gate, run_paired

pytestmark = pytest.mark.gpu
WORKERS = max(1, min(16, os.cpu_count() or 1))
# CAME_PARITY_FULL=1 runs every configuration to its stated step count (about 15 minutes for
# the whole GPU suite).  Without it the three longest runs stop earlier, so that the suite
# stays well inside a 20-minute budget on a slower host: the BERT-large-shaped set at step 20
# of 50, the GPT-2-medium-shaped set at 10 of 20 and the 128256 x 4096 matrix at 2 of 5;
# everything else (the BERT-base-shaped set's 100 steps included) always runs in full.
FULL = os.environ.get("CAME_PARITY_FULL", "0") == "1"


def _steps(configured: int, short: int) -> int:
    return configured if FULL else min(configured, short)


@pytest.fixture(scope="module")
def env(oracle):
    import torch
    from paper_2307_02047_b200 import binding
    assert torch.cuda.is_available()
    binding.load()
    return torch, binding, oracle


def _gate(res, label=""):
    gate(res, label)
    log = os.environ.get("CAME_PARITY_LOG")        # optional: one JSON line per run, for the record
    if log:
        with open(log, "a") as f:
            f.write(json.dumps({"label": label, "errors": {str(k): v for k, v in res.items()}}) + "\n")


@pytest.mark.parametrize("name", ["bert_base", "bert_large", "gpt2_medium"])
def test_model_shaped_sets_at_their_configured_step_counts(env, name):
    torch, binding, oracle = env
    w = synth.workload(name)
    assert w.steps == {"bert_base": 100, "bert_large": 50, "gpt2_medium": 20}[name]
    steps = _steps(w.steps, {"bert_base": 100, "bert_large": 20, "gpt2_medium": 10}[name])
    _gate(run_paired(torch, binding, oracle, w, seed=2, steps=steps, check_at=(1, 10, steps),
                     workers=WORKERS), name)


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
    assert w.steps == 5
    names = {t.name: i for i, t in enumerate(w.tensors)}
    idx = [names[n] for n in ("tok_emb", "l0.wq", "l0.w_gate", "l0.w_down", "l0.norm1",
                              "l17.wo", "l31.w_up", "l31.norm2", "norm_f")]
    _gate(run_paired(torch, binding, oracle, w, seed=6, steps=w.steps, check_at=(1, w.steps),
                     oracle_idx=idx, workers=WORKERS, device_fill_others=True), "llama7b")


@pytest.mark.parametrize("shape", synth.SWEEP_SHAPES)
def test_shape_sweep_five_steps(env, shape):
    torch, binding, oracle = env
    w = synth.workload(f"mat:{shape[0]}x{shape[1]}")
    assert w.steps == 5
    steps = _steps(w.steps, 2 if shape[0] * shape[1] > 1 << 28 else 5)
    _gate(run_paired(torch, binding, oracle, w, seed=8, steps=steps, check_at=(1, steps),
                     workers=WORKERS), w.name)


def test_bert_base_adafactor_mode(env):
    torch, binding, oracle = env
    w = synth.workload("bert_base")
    steps = _steps(w.steps, 10)             # all 100 steps with CAME_PARITY_FULL=1
    _gate(run_paired(torch, binding, oracle, w, seed=2, steps=steps, check_at=(1, 10, steps), workers=WORKERS,
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
