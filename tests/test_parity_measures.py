"""CPU checks of the error measures the GPU parity tests gate on (tests/parity_util.py).

A gate is only worth what it can see.  Mistakes are planted in the ORACLE's output, on the
CPU, and each measure must flag them; the rounding that storing theta in fp32 forces on any
implementation must pass."""
import numpy as np

from paper_2307_02047_b200 import synth
from tests.parity_util import (TOL_STEP1, TOL_STEP10, err_positive, err_signed, err_strict,
                               err_update, gate)


def _run(oracle, hp, steps, seed=3, shape=(96, 200)):
    w = synth.Workload("m", (synth.mat("w", *shape),), synth.F32, "normal_fixed", 1e-3, 0.0, (),
                       steps, hp)
    p0 = synth.make_params(w, seed)
    orc = oracle.OracleOptimizer(p0)
    for t in range(1, steps + 1):
        orc.step([synth.widen(g) for g in synth.make_grads(w, seed, t)], **hp)
    return p0[0], orc


def test_update_gate_sees_an_error_in_the_last_line_that_the_gate_on_theta_misses(oracle):
    hp = dict(synth.PAPER_HPARAMS)
    p0, orc = _run(oracle, hp, 1)
    ref = orc.p[0]
    wrong = p0.astype(np.float64) + (ref - p0) * (1.0 + 2.5e-5)    # update off by 2.5e-5 relative
    assert err_signed(wrong, ref) <= TOL_STEP1                      # theta alone does not notice
    assert err_update(wrong, ref, p0, 1) > 1.5 * TOL_STEP1          # the update gate does
    assert err_update(ref, ref, p0, 1) == 0.0


def test_update_gate_catches_a_dropped_weight_decay_term(oracle):
    hp = dict(synth.PAPER_HPARAMS, lr=1e-3, weight_decay=0.1)
    p0, with_wd = _run(oracle, hp, 1)
    _, without = _run(oracle, dict(hp, weight_decay=0.0), 1)
    assert err_update(without.p[0], with_wd.p[0], p0, 1) > 5 * TOL_STEP1
    p0, with_wd = _run(oracle, hp, 10)
    _, without = _run(oracle, dict(hp, weight_decay=0.0), 10)
    assert err_update(without.p[0], with_wd.p[0], p0, 10) > 2 * TOL_STEP10


def test_update_gate_passes_the_rounding_of_fp32_storage(oracle):
    """theta kept in fp32 and rounded once per step (everything else exact) must pass, also
    when the learning rate is so small that the update is a few ulps of theta."""
    for lr in (2e-4, 1e-5, 1e-7):
        hp = dict(synth.PAPER_HPARAMS, lr=lr)
        w = synth.Workload("m", (synth.mat("w", 64, 96),), synth.F32, "normal_fixed", 1e-3, 0.0,
                           (), 10, hp)
        p0 = synth.make_params(w, 5)
        exact, rounded = oracle.OracleOptimizer(p0), oracle.OracleOptimizer(p0)
        for t in range(1, 11):
            g = [synth.widen(x) for x in synth.make_grads(w, 5, t)]
            exact.step(g, **hp)
            rounded.step(g, **hp)
            rounded.p[0][...] = rounded.p[0].astype(np.float32).astype(np.float64)
            tol = TOL_STEP1 if t == 1 else TOL_STEP10
            assert err_update(rounded.p[0], exact.p[0], p0[0], t) <= tol / 10


def test_positive_and_strict_measures():
    ref = np.array([1.0, 2.0, 4.0])
    assert err_positive(ref * (1 + 1e-6), ref) == np.float64(1e-6).item() or \
        abs(err_positive(ref * (1 + 1e-6), ref) - 1e-6) < 1e-12
    assert err_positive(np.array([1.0, 2.0, 0.5]), np.array([1.0, 2.0, 0.0])) == float("inf")
    assert abs(err_strict(np.array([1.0, -2.002]), np.array([1.0, -2.0])) - 1e-3) < 1e-12
    assert err_strict(np.zeros(3), np.zeros(3)) == 0.0


def test_gate_ignores_the_informational_strict_figures():
    gate({1: dict(p=1e-7, strict_p=0.5), 10: dict(m=5e-5, strict_m=3.0)})
    for bad in ({1: dict(p=2e-5)}, {10: dict(dp=2e-4)}):
        try:
            gate(bad)
        except AssertionError:
            continue
        raise AssertionError("gate let an error above tolerance through")
