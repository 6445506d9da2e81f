"""The seeded input generators: determinism, independence of draw order, exact bf16 rounding."""
import numpy as np

from paper_2307_02047_b200 import synth


def test_draws_are_keyed_not_sequential():
    w = synth.workload("toy")
    a = synth.make_grad(w, 5, 0, 3)
    _ = synth.make_grad(w, 5, 1, 2)
    b = synth.make_grad(w, 5, 0, 3)
    np.testing.assert_array_equal(a, b)
    assert not np.array_equal(a, synth.make_grad(w, 5, 0, 4))
    assert not np.array_equal(a, synth.make_grad(w, 6, 0, 3))
    assert a.dtype == np.float32 and a.shape == (512, 256)
    assert 0.8e-3 < a.std() < 1.2e-3
    p = synth.make_params(w, 5)
    assert 0.018 < p[0].std() < 0.022


def test_bf16_rounding_is_nearest_even_and_exact_to_widen():
    x = np.array([1.0, 1.00390625, 1.005859375, 1.001953125, -2.5, 3.14159, 1e-30, 0.0], np.float32)
    bits = synth.f32_to_bf16_bits(x)
    back = synth.bf16_bits_to_f32(bits)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7: goes to even (1.0); 1 + 1.5*2^-8 rounds up
    assert back[0] == 1.0 and back[1] == 1.0 and back[2] == 1.0078125 and back[3] == 1.0
    assert np.all(np.abs(back - x) <= np.abs(x) * 2.0 ** -8)
    assert synth.widen(bits).dtype == np.float64
    np.testing.assert_array_equal(synth.widen(bits), back.astype(np.float64))


def test_workload_recipes():
    w = synth.workload("bert_large")
    g = synth.make_grad(w, 1, 1, 1)         # position embedding, bf16 with zeroed rows
    assert g.dtype == np.uint16
    zero_rows = np.all(g == 0, axis=1).mean()
    assert 0.1 < zero_rows < 0.3
    s = [synth.tensor_sigma(w, 1, i) for i in range(20)]
    assert min(s) >= 1e-5 and max(s) <= 1e-2 and len(set(s)) == 20
    w4 = synth.workload("gpt2_medium")
    g4 = synth.widen(synth.make_grad(w4, 1, 1, 1))
    k = np.mean(g4 ** 4) / np.mean(g4 ** 2) ** 2      # heavy tails: kurtosis far above 3
    assert k > 6
    assert w4.hparams["weight_decay"] == 0.01
    wz = synth.with_zero_rows_everywhere(synth.workload("toy"))
    assert wz.zero_row_tensors == (0,)


def test_rank1_sign_matrix():
    g, a, b = synth.rank1_sign_matrix(4, 6, seed=2, step=1)
    np.testing.assert_allclose(g * g, np.outer(a, b), rtol=1e-14)
    g2, a2, b2 = synth.rank1_sign_matrix(4, 6, seed=2, step=2)
    np.testing.assert_array_equal(a, a2)
    assert not np.array_equal(np.sign(g), np.sign(g2))
