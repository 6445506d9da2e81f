"""Pins for the CPU float64 oracle: each test checks it against something other than
itself -- a closed form, an invariant of the mathematics, a limit case, or a dense
(unfactored) brute force written here in numpy from the paper's equations.

Citations are to the paper's Algorithm 1 (Adafactor with momentum), Algorithm 2
(CAME), Eq. 1 (update clipping) and Eq. 2 (rank-1 factorisation).
"""
import os

import numpy as np
import pytest

from paper_2307_02047_b200 import synth

HP = dict(lr=2e-4, beta1=0.9, beta2=0.999, beta3=0.9999, eps1=1e-30, eps2=1e-16,
          clip_d=1.0, weight_decay=0.0)
GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand_g(rng, n, m, scale=1e-3):
    return rng.standard_normal((n, m)) * scale


def _zeros_state(n, m):
    return (np.zeros((n, m)), np.zeros(n), np.zeros(m), np.zeros(n), np.zeros(m))


def _run(oracle, theta0, grads, hp, want_uhat=False):
    n, m = theta0.shape
    theta = theta0.copy()
    mom, r, c, R, C = _zeros_state(n, m)
    out = None
    for g in grads:
        out = oracle.matrix_step(theta, np.ascontiguousarray(g), mom, r, c, R, C,
                                 oracle.hparams(**hp), want_uhat=want_uhat)
    return theta, mom, r, c, R, C, out


# ---------------------------------------------------------------------------
# dense brute force: Algorithm 2 with the two second moments kept as FULL n x m
# EMAs (V for g^2 + eps1, W for U + eps2) and Eq. 2 applied to them afresh each
# step: row factor = V 1_m, column factor = 1_n^T V, normaliser 1_n^T V 1_m.
# Because the EMA is linear this must equal the factored recursion.
# ---------------------------------------------------------------------------
def dense_bruteforce(theta0, grads, hp):
    n, m = theta0.shape
    theta = theta0.copy()
    mom = np.zeros((n, m)); V = np.zeros((n, m)); W = np.zeros((n, m))
    ones_n, ones_m = np.ones(n), np.ones(m)
    for g in grads:
        V = hp["beta2"] * V + (1 - hp["beta2"]) * (g * g + hp["eps1"])
        vhat = np.outer(V @ ones_m, ones_n @ V) / (ones_n @ V @ ones_m)
        u = g / np.sqrt(vhat)
        rms = np.sqrt(np.mean(u * u))
        uhat = u / max(1.0, rms / hp["clip_d"])
        mom = hp["beta1"] * mom + (1 - hp["beta1"]) * uhat
        U = (uhat - mom) ** 2
        W = hp["beta3"] * W + (1 - hp["beta3"]) * (U + hp["eps2"])
        shat = np.outer(W @ ones_m, ones_n @ W) / (ones_n @ W @ ones_m)
        theta = theta - hp["lr"] * (mom / np.sqrt(shat) + hp["weight_decay"] * theta)
    return theta, mom, V @ ones_m, ones_n @ V, W @ ones_m, ones_n @ W


@pytest.mark.parametrize("n,m", [(3, 5), (7, 4), (1, 6), (6, 1), (16, 16)])
def test_dense_bruteforce_multi_step(oracle, n, m):
    rng = np.random.default_rng(100 + n * 31 + m)
    theta0 = rng.standard_normal((n, m)) * 0.02
    grads = [_rand_g(rng, n, m) for _ in range(6)]
    # second setting: eps1 and eps2 large enough to be visible in every quantity
    for hp in (dict(HP, beta3=0.99), dict(HP, beta3=0.99, eps1=3e-7, eps2=2e-3, clip_d=0.7)):
        got = _run(oracle, theta0, grads, hp)[:6]
        want = dense_bruteforce(theta0, grads, hp)
        for a, b, name in zip(got, want, "theta m r c R C".split()):
            np.testing.assert_allclose(a, b, rtol=1e-10, atol=0, err_msg=name)


def test_dense_bruteforce_weight_decay_definition(oracle):
    # weight decay is not in the paper; this only pins the oracle to the stated definition
    rng = np.random.default_rng(5)
    theta0 = rng.standard_normal((4, 6)) * 0.02
    grads = [_rand_g(rng, 4, 6) for _ in range(3)]
    hp = dict(HP, weight_decay=0.01)
    got = _run(oracle, theta0, grads, hp)[0]
    want = dense_bruteforce(theta0, grads, hp)[0]
    np.testing.assert_allclose(got, want, rtol=1e-12)
    # and lambda = 0 is a different result (the term is really there)
    assert np.max(np.abs(got - _run(oracle, theta0, grads, HP)[0])) > 1e-9


# ---------------------------------------------------------------------------
# Eq. 2: marginals and optimality of the rank-1 factorisation
# ---------------------------------------------------------------------------
def test_rank1_marginals(oracle):
    rng = np.random.default_rng(1)
    Vfull = rng.random((9, 13)) + 0.01
    W = Vfull.sum(axis=1)          # V 1_m
    H = Vfull.sum(axis=0)          # 1_n^T V  (un-normalised column factor)
    approx = oracle.rank1(W, H)    # W H / (1_n^T W)
    np.testing.assert_allclose(approx.sum(axis=1), W, rtol=1e-13)
    np.testing.assert_allclose(approx.sum(axis=0), H, rtol=1e-13)
    np.testing.assert_allclose(approx.sum(), Vfull.sum(), rtol=1e-13)
    # transposed operands would break this asymmetric check:
    assert approx.shape == (9, 13)
    np.testing.assert_allclose(approx[2, 5], W[2] * H[5] / W.sum(), rtol=1e-14)


def _gen_kl(P, Q):
    return float(np.sum(P * np.log(P / Q) - P + Q))


def test_rank1_minimises_generalised_kl(oracle):
    rng = np.random.default_rng(2)
    Vfull = rng.random((6, 8)) + 0.05
    W, H = Vfull.sum(axis=1), Vfull.sum(axis=0)
    best = _gen_kl(Vfull, oracle.rank1(W, H))
    for _ in range(200):
        a = W * np.exp(rng.standard_normal(6) * 0.05)
        b = H * np.exp(rng.standard_normal(8) * 0.05) / W.sum()
        assert _gen_kl(Vfull, np.outer(a, b)) >= best - 1e-12


def test_factor_ema_sums_and_eps_inside_sum(oracle):
    rng = np.random.default_rng(3)
    X = rng.random((5, 7))
    row = rng.random(5); col = rng.random(7)
    row0, col0 = row.copy(), col.copy()
    eps, beta = 0.25, 0.75
    oracle.factor_ema(X, eps, beta, row, col)
    # eps is added per ELEMENT before summing: 7 eps per row, 5 eps per column
    np.testing.assert_allclose(row, beta * row0 + (1 - beta) * (X.sum(axis=1) + 7 * eps), rtol=1e-14)
    np.testing.assert_allclose(col, beta * col0 + (1 - beta) * (X.sum(axis=0) + 5 * eps), rtol=1e-14)


def test_beta2_zero_gives_plain_sums(oracle):
    rng = np.random.default_rng(4)
    theta0 = rng.standard_normal((5, 3))
    grads = [_rand_g(rng, 5, 3) for _ in range(3)]
    hp = dict(HP, beta2=0.0, eps1=0.0)
    _, _, r, c, _, _, _ = _run(oracle, theta0, grads, hp)
    g = grads[-1]
    np.testing.assert_allclose(r, (g * g).sum(axis=1), rtol=1e-14)
    np.testing.assert_allclose(c, (g * g).sum(axis=0), rtol=1e-14)


# ---------------------------------------------------------------------------
# rank-1 squared gradients: the factored second moment is exact
# ---------------------------------------------------------------------------
def test_rank1_gradients_exact_second_moment(oracle):
    n, m = 6, 9
    hp = dict(HP, eps1=0.0)
    theta = np.zeros((n, m)); mom, r, c, R, C = _zeros_state(n, m)
    Vexact = np.zeros((n, m))
    for step in range(1, 5):
        g, a, b = synth.rank1_sign_matrix(n, m, seed=11, step=step)
        oracle.matrix_step(theta, g, mom, r, c, R, C, oracle.hparams(**hp))
        Vexact = hp["beta2"] * Vexact + (1 - hp["beta2"]) * g * g
        np.testing.assert_allclose(oracle.rank1(r, c), Vexact, rtol=1e-12)
    # after step 1 specifically: v = (1 - beta2) G^2
    theta = np.zeros((n, m)); mom, r, c, R, C = _zeros_state(n, m)
    g, a, b = synth.rank1_sign_matrix(n, m, seed=11, step=1)
    oracle.matrix_step(theta, g, mom, r, c, R, C, oracle.hparams(**hp))
    np.testing.assert_allclose(oracle.rank1(r, c), (1 - hp["beta2"]) * np.outer(a, b), rtol=1e-12)


def _read_golden(name):
    out = {}
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            k, v = line.split()
            out[k] = float(v)
    return out


def test_closed_form_first_step_golden(oracle):
    gold = _read_golden("closed_form_first_step.txt")
    n, m = 8, 12
    hp = dict(HP, eps1=0.0)
    g, a, b = synth.rank1_sign_matrix(n, m, seed=3, step=1)
    sgn = np.sign(g)
    rng = np.random.default_rng(0)
    theta0 = rng.standard_normal((n, m)) * 0.02
    theta, mom, r, c, R, C, (diag, uhat) = _run(oracle, theta0, [g], hp, want_uhat=True)
    np.testing.assert_allclose(diag["rms_u"], gold["abs_u"], rtol=1e-12)
    np.testing.assert_allclose(uhat, gold["abs_uhat"] * sgn, rtol=1e-12)
    np.testing.assert_allclose(mom, gold["abs_m"] * sgn, rtol=1e-12)
    np.testing.assert_allclose(R, (1 - hp["beta3"]) * m * (gold["U"] + hp["eps2"]), rtol=1e-10)
    np.testing.assert_allclose(C, (1 - hp["beta3"]) * n * (gold["U"] + hp["eps2"]), rtol=1e-10)
    np.testing.assert_allclose(oracle.rank1(R, C), gold["S"], rtol=1e-9)
    np.testing.assert_allclose(theta - theta0, -gold["abs_delta_theta"] * sgn, rtol=1e-9, atol=1e-16)
    np.testing.assert_allclose(diag["sum_r"], (1 - hp["beta2"]) * a.sum() * b.sum(), rtol=1e-12)


def test_closed_form_general_hparams(oracle):
    # same closed form with other hyper-parameters, clip threshold and eps2 visible
    n, m = 5, 7
    hp = dict(lr=3e-3, beta1=0.8, beta2=0.99, beta3=0.9, eps1=0.0, eps2=1e-2, clip_d=2.5,
              weight_decay=0.0)
    g, a, b = synth.rank1_sign_matrix(n, m, seed=4, step=1)
    sgn = np.sign(g)
    theta0 = np.zeros((n, m))
    theta, mom, r, c, R, C, (diag, uhat) = _run(oracle, theta0, [g], hp, want_uhat=True)
    d, b1, b3, e2 = hp["clip_d"], hp["beta1"], hp["beta3"], hp["eps2"]
    np.testing.assert_allclose(uhat, d * sgn, rtol=1e-12)
    np.testing.assert_allclose(mom, (1 - b1) * d * sgn, rtol=1e-12)
    S = (1 - b3) * ((b1 * d) ** 2 + e2)
    np.testing.assert_allclose(theta, -hp["lr"] * (1 - b1) * d * sgn / np.sqrt(S), rtol=1e-12)


def test_no_clip_when_rms_below_d(oracle):
    # with d above RMS(u) the update is not scaled (Eq. 1: max(1, .) = 1)
    n, m = 5, 7
    hp = dict(HP, eps1=0.0, clip_d=100.0)
    g, a, b = synth.rank1_sign_matrix(n, m, seed=4, step=1)
    _, _, _, _, _, _, (diag, uhat) = _run(oracle, np.zeros((n, m)), [g], hp, want_uhat=True)
    np.testing.assert_allclose(np.abs(uhat), 1 / np.sqrt(1 - hp["beta2"]), rtol=1e-12)


def test_clip_property_generic(oracle):
    rng = np.random.default_rng(6)
    for d in (0.3, 1.0, 50.0):
        hp = dict(HP, clip_d=d)
        g = _rand_g(rng, 9, 11)
        _, _, _, _, _, _, (diag, uhat) = _run(oracle, np.zeros((9, 11)), [g], hp, want_uhat=True)
        rms_hat = np.sqrt(np.mean(uhat ** 2))
        np.testing.assert_allclose(rms_hat, min(diag["rms_u"], d), rtol=1e-12)
        # RMS is over ALL components (root of the MEAN), not a norm
        assert diag["rms_u"] == pytest.approx(31.6, rel=0.2)


def test_beta1_zero(oracle):
    rng = np.random.default_rng(7)
    n, m = 6, 5
    hp = dict(HP, beta1=0.0)
    g = _rand_g(rng, n, m)
    theta0 = rng.standard_normal((n, m))
    theta, mom, r, c, R, C, (diag, uhat) = _run(oracle, theta0, [g], hp, want_uhat=True)
    np.testing.assert_allclose(mom, uhat, rtol=0, atol=0)
    np.testing.assert_allclose(R, (1 - hp["beta3"]) * m * hp["eps2"], rtol=1e-12)
    np.testing.assert_allclose(C, (1 - hp["beta3"]) * n * hp["eps2"], rtol=1e-12)
    np.testing.assert_allclose(theta - theta0,
                               -hp["lr"] * uhat / np.sqrt((1 - hp["beta3"]) * hp["eps2"]), rtol=1e-9)


# ---------------------------------------------------------------------------
# whole-step invariants
# ---------------------------------------------------------------------------
def test_reduces_to_algorithm1_for_r_c_m(oracle):
    rng = np.random.default_rng(8)
    n, m = 7, 6
    theta0 = rng.standard_normal((n, m)) * 0.02
    grads = [_rand_g(rng, n, m) for _ in range(5)]
    _, mom, r, c, _, _, _ = _run(oracle, theta0, grads, HP)
    th = theta0.copy(); mo = np.zeros((n, m)); rr = np.zeros(n); cc = np.zeros(m)
    for g in grads:
        oracle.adafactor_matrix_step(th, np.ascontiguousarray(g), mo, rr, cc, oracle.hparams(**HP))
    np.testing.assert_array_equal(mom, mo)
    np.testing.assert_array_equal(r, rr)
    np.testing.assert_array_equal(c, cc)
    # Algorithm 1's parameter line: theta_t = theta_{t-1} - eta m_t (checked on one more step)
    th2 = th.copy(); mo2 = mo.copy()
    oracle.adafactor_matrix_step(th2, grads[0], mo2, rr, cc, oracle.hparams(**HP))
    np.testing.assert_allclose(th2, th - HP["lr"] * mo2, rtol=1e-14)


def test_power_of_two_scale_invariance(oracle):
    rng = np.random.default_rng(9)
    n, m = 6, 10
    theta0 = rng.standard_normal((n, m)) * 0.02
    grads = [_rand_g(rng, n, m) for _ in range(4)]
    hp = dict(HP, eps1=0.0)
    base = _run(oracle, theta0, grads, hp)
    scaled = _run(oracle, theta0, [g * 2.0 ** 7 for g in grads], hp)
    for k in (0, 1, 4, 5):                       # theta, m, R, C unchanged
        np.testing.assert_allclose(scaled[k], base[k], rtol=1e-13)
    np.testing.assert_allclose(scaled[2], base[2] * 4.0 ** 7, rtol=1e-13)   # r
    np.testing.assert_allclose(scaled[3], base[3] * 4.0 ** 7, rtol=1e-13)   # c


def test_transpose_equivariance(oracle):
    rng = np.random.default_rng(10)
    n, m = 5, 8
    theta0 = rng.standard_normal((n, m)) * 0.02
    grads = [_rand_g(rng, n, m) for _ in range(4)]
    a = _run(oracle, theta0, grads, HP)
    b = _run(oracle, np.ascontiguousarray(theta0.T), [np.ascontiguousarray(g.T) for g in grads], HP)
    np.testing.assert_allclose(b[0].T, a[0], rtol=1e-11)
    np.testing.assert_allclose(b[1].T, a[1], rtol=1e-11)
    np.testing.assert_allclose(b[2], a[3], rtol=1e-12)   # r of the transpose = c
    np.testing.assert_allclose(b[3], a[2], rtol=1e-12)
    np.testing.assert_allclose(b[4], a[5], rtol=1e-11)
    np.testing.assert_allclose(b[5], a[4], rtol=1e-11)


def test_permutation_equivariance(oracle):
    rng = np.random.default_rng(11)
    n, m = 6, 7
    theta0 = rng.standard_normal((n, m)) * 0.02
    grads = [_rand_g(rng, n, m) for _ in range(3)]
    pr, pc = rng.permutation(n), rng.permutation(m)
    a = _run(oracle, theta0, grads, HP)
    b = _run(oracle, np.ascontiguousarray(theta0[pr][:, pc]),
             [np.ascontiguousarray(g[pr][:, pc]) for g in grads], HP)
    np.testing.assert_allclose(b[0], a[0][pr][:, pc], rtol=1e-11)
    np.testing.assert_allclose(b[2], a[2][pr], rtol=1e-12)
    np.testing.assert_allclose(b[3], a[3][pc], rtol=1e-12)
    np.testing.assert_allclose(b[4], a[4][pr], rtol=1e-11)
    np.testing.assert_allclose(b[5], a[5][pc], rtol=1e-11)


def test_state_does_not_depend_on_parameters(oracle):
    rng = np.random.default_rng(12)
    n, m = 4, 9
    grads = [_rand_g(rng, n, m) for _ in range(3)]
    a = _run(oracle, np.zeros((n, m)), grads, HP)
    b = _run(oracle, rng.standard_normal((n, m)), grads, HP)
    for k in range(1, 6):
        np.testing.assert_array_equal(a[k], b[k])


def test_zero_gradient_rows_stay_finite(oracle):
    # rows with all-zero gradients live on eps1 alone; nothing may become NaN/inf
    rng = np.random.default_rng(13)
    n, m = 8, 6
    g = _rand_g(rng, n, m); g[2] = 0.0; g[5] = 0.0
    theta0 = rng.standard_normal((n, m)) * 0.02
    theta, mom, r, c, R, C, _ = _run(oracle, theta0, [g, g], HP)
    for x in (theta, mom, r, c, R, C):
        assert np.all(np.isfinite(x))
    np.testing.assert_allclose(r[2], (1 - 0.999 ** 2) * m * HP["eps1"], rtol=1e-9)
    assert np.all(mom[2] == 0.0)


# ---------------------------------------------------------------------------
# vector path
# ---------------------------------------------------------------------------
@pytest.mark.parametrize("as_row", [False, True])
def test_vector_equals_degenerate_matrix(oracle, as_row):
    rng = np.random.default_rng(14)
    N = 37
    theta0 = rng.standard_normal(N) * 0.02
    grads = [rng.standard_normal(N) * 1e-3 for _ in range(5)]
    hp = dict(HP, beta3=0.99, weight_decay=0.003, eps1=3e-7, eps2=2e-3)
    th = theta0.copy(); mo = np.zeros(N); v = np.zeros(N); S = np.zeros(N)
    for g in grads:
        oracle.vector_step(th, g, mo, v, S, oracle.hparams(**hp))
    shape = (1, N) if as_row else (N, 1)
    out = _run(oracle, theta0.reshape(shape), [g.reshape(shape) for g in grads], hp)
    np.testing.assert_allclose(out[0].ravel(), th, rtol=1e-11)
    np.testing.assert_allclose(out[1].ravel(), mo, rtol=1e-11)
    # N x 1: r = v and R = S;  1 x N: c = v and C = S
    np.testing.assert_allclose(out[3] if as_row else out[2], v, rtol=1e-12)
    np.testing.assert_allclose(out[5] if as_row else out[4], S, rtol=1e-11)


def test_vector_no_confidence_is_algorithm1_last_line(oracle):
    rng = np.random.default_rng(15)
    N = 11
    theta0 = rng.standard_normal(N)
    g = rng.standard_normal(N) * 1e-3
    th = theta0.copy(); mo = np.zeros(N); v = np.zeros(N); S = np.full(N, 7.0)
    oracle.vector_step(th, g, mo, v, S, oracle.hparams(**HP), no_confidence=True)
    np.testing.assert_allclose(th, theta0 - HP["lr"] * mo, rtol=1e-14)
    assert np.all(S == 7.0)


def test_optimizer_driver_lists(oracle):
    w = synth.workload("toy")
    params = synth.make_params(w, seed=1)
    opt = oracle.OracleOptimizer(params)
    for step in (1, 2):
        grads = [synth.widen(g) for g in synth.make_grads(w, 1, step)]
        opt.step(grads, **w.hparams)
    assert opt.p[0].shape == (512, 256) and opt.p[1].shape == (256,)
    # first-step magnitude predicted by the closed form (~2.2e-3 per step at the defaults)
    d = np.abs(opt.p[0] - params[0].astype(np.float64))
    assert 1e-3 < d.mean() < 1e-2


def test_vector_no_confidence_equals_algorithm1_on_a_column_matrix(oracle):
    # the alternate vector reading is Algorithm 1 applied to the vector as an N x 1 matrix
    rng = np.random.default_rng(16)
    N = 23
    theta0 = rng.standard_normal(N) * 0.02
    grads = [rng.standard_normal(N) * 1e-3 for _ in range(4)]
    hp = dict(HP, weight_decay=0.002, eps1=3e-7)
    th = theta0.copy(); mo = np.zeros(N); v = np.zeros(N); S = np.zeros(N)
    TH = theta0.reshape(N, 1).copy(); MO = np.zeros((N, 1)); r = np.zeros(N); c = np.zeros(1)
    for g in grads:
        oracle.vector_step(th, g, mo, v, S, oracle.hparams(**hp), no_confidence=True)
        oracle.adafactor_matrix_step(TH, np.ascontiguousarray(g.reshape(N, 1)), MO, r, c,
                                     oracle.hparams(**hp))
    np.testing.assert_allclose(th, TH.ravel(), rtol=1e-11)
    np.testing.assert_allclose(mo, MO.ravel(), rtol=1e-11)
    np.testing.assert_allclose(v, r, rtol=1e-12)


try:
    from hypothesis import given, settings, strategies as st
    _HAVE_HYPOTHESIS = True
except Exception:                                     # pragma: no cover
    _HAVE_HYPOTHESIS = False


if _HAVE_HYPOTHESIS:
    @settings(max_examples=25, deadline=None)
    @given(n=st.integers(1, 12), m=st.integers(1, 12), k=st.integers(-12, 12),
           seed=st.integers(0, 10_000), steps=st.integers(1, 4))
    def test_property_invariances_on_random_shapes(n, m, k, seed, steps):
        """On arbitrary small shapes: power-of-two gradient scaling (eps1 = 0) leaves theta, m,
        R, C unchanged and scales r, c by 4^k; transposing the problem transposes the result;
        and the dense-EMA brute force agrees."""
        from oracle import came_oracle as oracle
        rng = np.random.default_rng(seed)
        theta0 = rng.standard_normal((n, m)) * 0.02
        grads = [_rand_g(rng, n, m) for _ in range(steps)]
        hp = dict(HP, eps1=0.0, beta3=0.99)
        base = _run(oracle, theta0, grads, hp)
        scaled = _run(oracle, theta0, [g * 2.0 ** k for g in grads], hp)
        for i in (0, 1, 4, 5):
            np.testing.assert_allclose(scaled[i], base[i], rtol=1e-12)
        np.testing.assert_allclose(scaled[2], base[2] * 4.0 ** k, rtol=1e-12)
        np.testing.assert_allclose(scaled[3], base[3] * 4.0 ** k, rtol=1e-12)
        tr = _run(oracle, np.ascontiguousarray(theta0.T), [np.ascontiguousarray(g.T) for g in grads], hp)
        np.testing.assert_allclose(tr[0].T, base[0], rtol=1e-9)
        np.testing.assert_allclose(tr[2], base[3], rtol=1e-10)
        np.testing.assert_allclose(tr[4], base[5], rtol=1e-9)
        want = dense_bruteforce(theta0, grads, hp)
        for a, b in zip(base[:6], want):
            np.testing.assert_allclose(a, b, rtol=1e-9)
