"""Host-side checks of the synthetic input recipe (no GPU, no method arithmetic)."""
import numpy as np

from paper_2509_24899_b200 import workloads as W


def test_splitmix64_reference_value_and_schedule():
    # first output of SplitMix64 seeded with 0 (published test vector of the generator)
    assert next(W.splitmix64_stream(0)) == 0xE220A8397B1DCDAF
    sched = W.stack_schedule(0)
    assert len(sched) == 30 and set(sched) <= set(W.STACK_RATES)
    assert sched[:6] == [1, 1, 0, 0, 8, 1]
    assert {r: sched.count(r) for r in W.STACK_RATES} == {1: 8, 4: 5, 8: 6, 16: 5, 0: 6}


def test_bf16_rounding_is_nearest_even():
    x = np.array([1.0, 1.0 + 2 ** -8, 1.0 + 3 * 2 ** -8, 1.0 + 2 ** -7, -2.5, 0.0], dtype=np.float32)
    back = W.bf16_bits_to_f32(W.f32_to_bf16_bits(x))
    # ties go to the even mantissa: 1+2^-8 -> 1, 1+3*2^-8 -> 1+2^-6
    assert back.tolist() == [1.0, 1.0, 1.0 + 2 ** -6, 1.0 + 2 ** -7, -2.5, 0.0]


def test_generate_shapes_seed_and_distribution():
    wl = W.CONFIGS["tiny"]
    a, b = W.generate(wl), W.generate(wl)
    assert all(np.array_equal(a[k], b[k]) for k in a)
    assert a["q"].shape == (1, 2, 1024, 64) and a["wq"].shape == (2, 64, 64)
    assert a["q"].dtype == np.uint16
    wl2 = W.Workload("t", B=1, H=2, d=128, F=128, grid=(1, 6, 8), block=(1, 6, 8), rate=8, seed=5)
    g = W.generate(wl2)
    q = W.bf16_bits_to_f64(g["q"])
    np.testing.assert_allclose(np.sqrt((q ** 2).mean(-1)), 1.0, atol=5e-3)   # unit RMS per token
    w = W.bf16_bits_to_f64(g["wk"])
    lim = np.sqrt(6.0 / 256)
    assert np.abs(w).max() <= lim * 1.01 and abs(w.std() - lim / np.sqrt(3)) < 0.01
    h1 = W.generate(wl2, heads=1)
    assert np.array_equal(h1["q"][:, 0], g["q"][:, 0]) and h1["wq"].shape[0] == 1
    assert W.CONFIGS["wan81"].N == 32760 and W.CONFIGS["wan161cfg"].N == 63960
    assert W.stack_layer(4).rate == 8 and W.stack_layer(4).seed == 4004
