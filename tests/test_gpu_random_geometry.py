"""Randomised geometry against the oracle: kernels with any mix of lengths (fast-path and generic),
dilations up to the largest that fits (few rows of the dilated view: the wide tiles), symmetric, zero
and arbitrary paddings, channel subsets, on series lengths from 64 to 30,000; hard, soft and backward
passes of every case within the tolerances of parity.py."""
import numpy as np
import pytest

import oracle
import paper_2301_08527_b200 as rk
from rocket_inputs import ar1_spike_series, kernels_from_lists, normal_array

import parity as P

pytestmark = pytest.mark.gpu


def _random_kernels(rng, C, L):
    ks = []
    for _ in range(int(rng.integers(20, 120))):
        ln = int(rng.choice([7, 9, 11])) if rng.random() < 0.9 else int(rng.choice([3, 5]))
        dmax = max(1, (L - 1) // (ln - 1))
        mode = rng.random()
        if mode < 0.5:
            d = int(np.floor(2 ** rng.uniform(0, np.log2(dmax))))
        elif mode < 0.8:
            d = int(rng.integers(max(1, dmax // 3), dmax + 1))
        else:
            d = int(rng.integers(40, 140)) if dmax >= 140 else int(rng.integers(1, dmax + 1))
        d = max(1, min(d, dmax))
        pm = rng.random()
        p = 0 if pm < 0.4 else ((ln - 1) * d // 2 if pm < 0.8 else int(rng.integers(0, (ln - 1) * d + 3)))
        if L + 2 * p - (ln - 1) * d < 1:
            p = (ln - 1) * d // 2
        m = int(rng.integers(1, min(C, ln) + 1))
        ks.append(dict(dilation=d, padding=p, channels=sorted(rng.choice(C, m, replace=False).tolist()),
                       weights=rng.normal(size=(m, ln)), bias=float(rng.uniform(-1, 1))))
    return kernels_from_lists(C, L, ks)


@pytest.mark.parametrize("seed", [11, 12, 13])
def test_random_geometry_all_passes(seed):
    import torch
    rng = np.random.default_rng(seed)
    for _ in range(10):
        C = int(rng.choice([1, 2, 5, 20]))
        L = int(rng.choice([64, 256, 1000, 2048, 5000, 12000, 30000]))
        N = int(rng.choice([1, 2, 3, 13]))
        kp = _random_kernels(rng, C, L)
        X = ar1_spike_series(int(rng.integers(1 << 30)), N, C, L)
        lam, shift = float(rng.choice([1.0, 10.0, 100.0])), float(rng.choice([3.0, -3.0]))
        p = rk.RocketParams.from_kernel_params(kp)
        Xd = torch.from_numpy(X).cuda()
        ref = oracle.forward(kp, X, lam=lam, shift=shift)
        ppv, mx = P.split_features(rk.rocket_transform(p, Xd).cpu().numpy())
        P.check_hard_ppv(ppv, ref)
        P.check_max(mx, ref)
        feat, arg = rk.rocket_transform_soft(p, Xd, lam, shift)
        soft, mx2 = P.split_features(feat.cpu().numpy())
        P.check_soft_ppv(soft, ref)
        P.check_max(mx2, ref)
        P.check_argmax(arg.cpu().numpy(), ref)
        g = normal_array(int(rng.integers(1 << 30)), (N, 2 * kp.K))
        dW, db = rk.rocket_transform_soft_backward(p, Xd, lam, shift, torch.from_numpy(g).cuda(), arg)
        rW, rb = oracle.backward(kp, X, g, arg.cpu().numpy(), lam=lam, shift=shift)
        P.check_grads(dW.cpu().numpy(), db.cpu().numpy(), rW, rb)
        assert p.device_status() == 0
        p.close()
