"""MINIROCKET transform on the device against the oracle (oracle/minirocket_oracle.c), through the C ABI.

Tolerance: the feature is a count over n outputs; as for the hard PPV of ROCKET, outputs within 1e-5 of the
bias are undecidable in fp32, so a count c is accepted iff P+ - 1e-4 n <= c <= P+ + AMB + 1e-4 n with
P+ = #{z > bias + 1e-5} and AMB = #{|z - bias| <= 1e-5} from the oracle.  The fp32 biases of the library's fit
feed both sides.
"""
from types import SimpleNamespace

import numpy as np
import pytest

import oracle
import paper_2301_08527_b200 as rk
from rocket_inputs import ar1_spike_series, generate_minirocket, random_walk_series

import parity as P

pytestmark = pytest.mark.gpu


def _check(C, L, N, F, seed, series=ar1_spike_series, examples=None):
    import torch
    p = generate_minirocket(seed, C, L, F)
    X = series(seed + 1, N, C, L)
    m = rk.MiniRocket.create(seed, C, L, F)
    m.fit(X)
    arrays = m.host_arrays()
    p.quantile = arrays["quantile"]
    bias = arrays["bias"].astype(np.float64)
    np.testing.assert_allclose(bias, oracle.minirocket_fit(p, X), rtol=1e-6, atol=1e-6)
    feat = m.transform(torch.from_numpy(X).cuda()).cpu().numpy()
    m.close()
    sel = np.arange(N) if examples is None else np.asarray(examples)
    ref = oracle.minirocket_transform(p, X[sel], bias)
    band = SimpleNamespace(ppv=ref.ppv, pos_eps=ref.pos_eps, amb=ref.amb, out_len=np.broadcast_to(ref.n_out[None, :], ref.ppv.shape))
    assert np.all(np.isfinite(feat)) and np.all((feat >= 0) & (feat <= 1))
    return P.check_hard_ppv(feat[sel], band)


@pytest.mark.parametrize("C,L,N,F", [(3, 700, 3, 84 * 12), (1, 64, 4, 84 * 40), (20, 5000, 4, 10000), (2, 9, 3, 84), (7, 4099, 2, 84 * 20),
                                     (5, 49, 1, 168)])
def test_minirocket_small_full(C, L, N, F):
    _check(C, L, N, F, seed=31 + L)


@pytest.mark.parametrize("C,L,N,F", [(2, 777, 2, 84 * 32), (5, 12001, 2, 84 * 32), (3, 30003, 1, 84 * 32), (1, 2050, 3, 84 * 64)])
def test_minirocket_every_tile_shape(C, L, N, F):
    # 32 dilations per kernel: tiles of whole rows and of 256-column blocks, ragged last column tiles, runs of 9
    # to 63 rows, series lengths that are no multiple of anything
    _check(C, L, N, F, seed=77 + L)


def test_minirocket_univariate_random_walks():
    _check(1, 512, 16, 10000, seed=8527, series=random_walk_series)


def test_minirocket_paper_scale_two_examples_of_a_batch():
    # 20 channels x 50,000 steps, 9,996 features: the shape of the paper's examples; the oracle checks two
    # examples of a batch of six in full
    _check(20, 50000, 6, 10000, seed=8527, examples=[1, 4])


def test_minirocket_two_runs_are_identical_and_biases_can_be_installed():
    import torch
    C, L, N = 4, 3000, 3
    X = ar1_spike_series(5, N, C, L)
    m = rk.MiniRocket.create(6, C, L, 84 * 25)
    m.fit(X)
    Xd = torch.from_numpy(X).cuda()
    a, b = m.transform(Xd).cpu().numpy(), m.transform(Xd).cpu().numpy()
    assert a.tobytes() == b.tobytes()
    m2 = rk.MiniRocket.create(6, C, L, 84 * 25)
    m2.set_biases(m.host_arrays()["bias"])
    assert m2.transform(Xd).cpu().numpy().tobytes() == a.tobytes()
    out = torch.empty((0, m.F), device="cuda")
    assert m.transform(torch.empty((0, C, L), device="cuda")).shape == (0, m.F)
    m.close(); m2.close()
