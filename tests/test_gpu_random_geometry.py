"""Randomised geometry against the oracle: kernels with any mix of lengths (fast-path and generic),
dilations up to the largest that fits (few rows of the dilated view: the wide tiles), symmetric, zero
and arbitrary paddings, channel subsets, on series lengths from 64 to 50,001 (multiples of four floats and
not); hard, soft and backward
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
        L = int(rng.choice([64, 256, 1000, 2048, 4099, 5000, 12000, 30000, 50001]))
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


def test_backward_with_padding_beyond_eight_dilations_on_the_fused_kernels():
    # paddings of 8 d to 10 d (legal for caller-supplied kernels) put outputs more than 8 rows of the dilated
    # view before the first sample; the argmax term of the gradient must survive there.  Every kernel has a
    # fast-path length, so the fused backward kernels serve the whole set.
    import torch
    rng = np.random.default_rng(77)
    C, L, N = 2, 64, 6
    ks = []
    for i in range(80):
        ln = int(rng.choice([9, 11]))
        d = int(rng.integers(2, 7)) if ln == 9 else int(rng.integers(2, 7))
        p = int(rng.integers(8 * d + 1, (ln - 1) * d + 1)) if (ln - 1) * d > 8 * d else 8 * d
        m = int(rng.integers(1, 3))
        ks.append(dict(dilation=d, padding=p, channels=sorted(rng.choice(C, m, replace=False).tolist()),
                       weights=rng.normal(size=(m, ln)), bias=float(rng.uniform(0.5, 1.0))))
    kp = kernels_from_lists(C, L, ks)
    X = -np.abs(ar1_spike_series(78, N, C, L))          # negative samples: the bias alone wins in the padding
    lam, shift = 10.0, 3.0
    g = normal_array(79, (N, 2 * kp.K))
    ref = oracle.forward(kp, X, lam=lam, shift=shift)
    far_left = (ref.argmax - kp.padding[None, :]) < -8 * kp.dilation[None, :]
    assert far_left.sum() >= 10                           # the case is exercised
    p = rk.RocketParams.from_kernel_params(kp)
    Xd = torch.from_numpy(X).cuda()
    feat, arg = rk.rocket_transform_soft(p, Xd, lam, shift)
    P.check_argmax(arg.cpu().numpy(), ref)
    dW, db = rk.rocket_transform_soft_backward(p, Xd, lam, shift, torch.from_numpy(g).cuda(),
                                               torch.from_numpy(ref.argmax.astype(np.int32)).cuda())
    rdW, rdb = oracle.backward(kp, X, g, ref.argmax, lam=lam, shift=shift)
    P.check_grads(dW.cpu().numpy(), db.cpu().numpy(), rdW, rdb)
    P.check_grads(np.zeros(0), db.cpu().numpy(), np.zeros(0), rdb)
    p.close()
