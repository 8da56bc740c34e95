"""MINIROCKET, host side of the library (no GPU): parameters against the reference generator, biases of the
host-side fit against the oracle's."""
import numpy as np
import pytest

import oracle
import paper_2301_08527_b200 as rk
from rocket_inputs import ar1_spike_series, generate_minirocket


@pytest.mark.parametrize("C,L,F", [(1, 64, 500), (20, 5000, 10000), (5, 50000, 10000), (9, 300, 84), (5, 49, 168), (3, 57, 840),
                                   (2, 4097, 2688), (4, 1001, 1680), (2, 9, 84), (1, 25, 252)])
def test_library_parameters_equal_the_reference_generator(C, L, F):
    ref = generate_minirocket(8527, C, L, F)
    m = rk.MiniRocket.create(8527, C, L, F)
    a = m.host_arrays()
    assert (m.F, m.n_combos) == (ref.F, ref.n_combos)
    for name in ("taps", "dilation", "kernel_index", "padded", "num_channels", "channel_idx", "feature_offset"):
        assert np.array_equal(a[name], getattr(ref, name)), name
    assert np.array_equal(a["example_draw"], ref.example_draw)
    np.testing.assert_allclose(a["quantile"], ref.quantile, rtol=0, atol=1e-12)
    m.close()


def test_host_fit_gives_the_oracles_biases():
    C, L, N = 6, 2000, 5
    ref = generate_minirocket(21, C, L, 84 * 30)
    X = ar1_spike_series(22, N, C, L)
    m = rk.MiniRocket.create(21, C, L, 84 * 30)
    m.fit(X)
    got = m.host_arrays()["bias"].astype(np.float64)
    # the library carries the reference generator's quantiles to within an ulp: fit the oracle with the library's
    p = generate_minirocket(21, C, L, 84 * 30)
    p.quantile = m.host_arrays()["quantile"]
    want = oracle.minirocket_fit(p, X)
    np.testing.assert_allclose(got, want, rtol=1e-6, atol=1e-6)
    m.close()


@pytest.mark.parametrize("L", [9, 10, 17, 63, 64, 100, 999, 4099, 50001, 200000, 1000003])
def test_a_handle_exists_for_any_series_length(L):
    # creation chooses, per dilation, how the kernel tiles the dilated view; every dilation of every length
    # from the shortest (9 samples: dilation 1 only) upwards must find a tiling
    m = rk.MiniRocket.create(3, 3, L, 84 * 12)
    a = m.host_arrays()
    assert a["dilation"].min() == 1 and a["dilation"].max() <= max(1, (L - 1) // 8)
    m.close()


def test_argument_checks():
    lib = rk.load_library()
    import ctypes
    h = ctypes.c_void_p()
    assert lib.rocket_mini_create(1, 0, 100, 840, ctypes.byref(h)) == -1
    assert lib.rocket_mini_create(1, 2, 8, 840, ctypes.byref(h)) == -1
    assert lib.rocket_mini_create(1, 2, 100, 83, ctypes.byref(h)) == -1
    m = rk.MiniRocket.create(1, 2, 100, 840)
    assert lib.rocket_mini_transform(m.handle, ctypes.c_void_p(16), 1, 2, 100, ctypes.c_void_p(16), None) == -1   # not fitted
    assert lib.rocket_mini_fit(m.handle, None, 3) == -1
    m.set_biases(np.zeros(m.F, np.float32))
    assert lib.rocket_mini_transform(m.handle, ctypes.c_void_p(16), 1, 3, 100, ctypes.c_void_p(16), None) == -2   # shape
    with pytest.raises(rk.RocketError):
        m.set_biases(np.full(m.F, np.nan, np.float32))
    m.close()
