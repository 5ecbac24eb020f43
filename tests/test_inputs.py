"""Host-side checks of the seeded input generators."""
import numpy as np

import pm_inputs as I


def test_rng_is_a_pure_function_of_its_coordinates():
    a = I.normal(7, 3, 1000)
    b = I.normal(7, 3, 1000)
    np.testing.assert_array_equal(a, b)
    np.testing.assert_array_equal(I.normal(7, 3, 10, offset=5), a[5:15])
    assert np.abs(I.normal(7, 4, 1000) - a).max() > 0.1


def test_normal_moments():
    x = I.normal(11, 1, 200000)
    assert abs(x.mean()) < 0.01 and abs(x.std() - 1.0) < 0.01
    assert abs((x ** 3).mean()) < 0.05 and abs((x ** 4).mean() - 3.0) < 0.1


def test_pipemare_delays():
    assert I.pipemare_delays(4) == ([7, 5, 3, 1], [0, 0, 0, 0])
    assert I.pipemare_delays(4, n_micro=2)[0] == [4, 3, 2, 1]


def test_cfg_shapes():
    c1, c3 = I.cfg1(), I.cfg3()
    assert c1.n_stages == 4 and c1.tau_fwd == [7, 5, 3, 1] and c1.microbatch == 32
    assert c3.n_stages == 32 and c3.tau_fwd[0] == 63 and len(c3.stages[0]) == 2
    x, y = I.batch(c1, 0)
    assert x.shape == (32, 256) and y.shape == (32, 256) and x.dtype == np.float32
    assert (y >= 0).all()                    # the teacher ends in ReLU
    x2, _ = I.batch(c1, 1)
    assert np.abs(x - x2).max() > 0.1


def test_bf16_inputs_are_representable():
    wl = I.cfg3_small()
    x, _ = I.batch(wl, 0)
    np.testing.assert_array_equal(I.round_to_bf16(x), x)
    assert (x.view(np.uint32) & 0xFFFF == 0).all()


def test_update_sweep_layout():
    case = I.update_sweep_case(1000, 8)
    assert sum(case["counts"]) == 1000
    assert all(o % 64 == 0 for o in case["offsets"])
    assert case["tau_fwd"][0] == 15 and case["tau_fwd"][-1] == 1
    assert case["w"].shape == (case["total"],)
    o, c = case["offsets"][1], case["counts"][1]
    assert (case["w"][o:o + c] != 0).all() and (case["w"][o + c:case["offsets"][2]] == 0).all()


def test_zipf_ranks_are_skewed():
    r = I.zipf_ranks(3, 9, 20000, 1000, 1.1)
    assert r.min() >= 0 and r.max() < 1000
    assert (r == 0).mean() > 5 * (r == 9).mean() * 0.5
