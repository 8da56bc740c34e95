"""Half-precision hard transform on the device (rocket_transform_f16) against the half-precision oracle
(oracle/rocket_f16_oracle.c: binary16 samples, weights and biases, one rounding per fused multiply-add, bias
first, channels in the kernel's order, taps 0 .. len - 1) - bit for bit, counts and maxima - and against the
double-precision oracle within the looser bounds of a binary16 accumulation (PPV: counts within 5e-3 n + 2 of one
another - a kernel whose dilation leaves a hundred outputs moves PPV by 1e-2 with a single output near zero; max:
1e-2 of max(|max|, 1))."""
import numpy as np
import pytest

import oracle
import paper_2301_08527_b200 as rk
from rocket_inputs import ar1_spike_series, generate_kernels, kernels_from_lists, random_walk_series

import parity as P

pytestmark = pytest.mark.gpu

F16_PPV_ATOL = 5e-3
F16_MAX_RTOL = 1e-2


def _fast_only(kp):
    """The kernels the fused kernels take (lengths 7, 9, 11), as a parameter set of their own."""
    keep = [k for k in range(kp.K) if int(kp.length[k]) in (7, 9, 11)]
    ks = []
    for k in keep:
        m, ln = int(kp.num_channels[k]), int(kp.length[k])
        ks.append(dict(dilation=int(kp.dilation[k]), padding=int(kp.padding[k]),
                       channels=kp.channel_idx[kp.channel_offset[k]:kp.channel_offset[k + 1]].tolist(),
                       weights=kp.weights[kp.weight_offset[k]:kp.weight_offset[k + 1]].reshape(m, ln), bias=float(kp.bias[k])))
    return kernels_from_lists(kp.C, kp.L, ks)


def _check_bitwise(kp, X, feat, pn=None, pk=None):
    ppv, mx = P.split_features(feat)
    if pn is None:
        ref = oracle.forward_f16(kp, X)
    else:
        ref = oracle.forward_f16_pairs(kp, X, pn, pk)
        ppv, mx = ppv[pn, pk], mx[pn, pk]
    n = ref.out_len.astype(np.float64)
    cnt = np.round(ppv.astype(np.float64) * n).astype(np.int64)
    assert np.all(np.abs(ppv.astype(np.float64) * n - cnt) <= 1e-6 * n + 1e-3)
    bad = np.argwhere(cnt != ref.count)
    assert bad.size == 0, "counts differ from the half-precision oracle at %s: %s vs %s" % (bad[:5], cnt[tuple(bad[0])], ref.count[tuple(bad[0])])
    assert np.array_equal(mx.astype(np.float64), ref.max), "maxima differ from the half-precision oracle"
    return ref


def _check_loose(kp, X, feat, pn=None, pk=None):
    ppv, mx = P.split_features(feat)
    ref = oracle.forward(kp, X) if pn is None else oracle.forward_pairs(kp, X, pn, pk)
    if pn is not None:
        ppv, mx = ppv[pn, pk], mx[pn, pk]
    n = ref.out_len.astype(np.float64)
    e_ppv = np.abs(ppv - ref.ppv).max()
    e_max = (np.abs(mx - ref.max) / np.maximum(np.abs(ref.max), 1.0)).max()
    assert np.all(np.abs(ppv - ref.ppv) * n <= F16_PPV_ATOL * n + 2.0), "PPV count further than 5e-3 n + 2 from double precision"
    assert e_max <= F16_MAX_RTOL, e_max
    return e_ppv, e_max


@pytest.mark.parametrize("C,L,K,N,series", [(1, 512, 400, 5, random_walk_series), (20, 5000, 600, 3, ar1_spike_series),
                                            (5, 4099, 300, 2, ar1_spike_series), (3, 50001, 60, 1, ar1_spike_series),
                                            (20, 1000, 1500, 13, ar1_spike_series)])
def test_f16_small_full_bit_for_bit(C, L, K, N, series):
    import torch
    kp = generate_kernels(61 + L, K, C, L)
    X = series(62 + L, N, C, L)
    p = rk.RocketParams.from_kernel_params(kp)
    feat = rk.rocket_transform_f16(p, torch.from_numpy(X).cuda()).cpu().numpy()
    assert p.device_status() == 0
    p.close()
    _check_bitwise(kp, X, feat)
    print("half precision against double precision: PPV %.2e, max %.2e" % _check_loose(kp, X, feat))


@pytest.mark.parametrize("seed", [21, 22])
def test_f16_random_geometry_bit_for_bit(seed):
    import torch
    import test_gpu_random_geometry as G
    rng = np.random.default_rng(seed)
    for _ in range(8):
        C = int(rng.choice([1, 2, 5, 20])); L = int(rng.choice([64, 256, 1000, 2048, 4099, 12000, 30000]))
        N = int(rng.choice([1, 2, 13]))
        kp = _fast_only(G._random_kernels(rng, C, L))
        X = ar1_spike_series(int(rng.integers(1 << 30)), N, C, L)
        p = rk.RocketParams.from_kernel_params(kp)
        feat = rk.rocket_transform_f16(p, torch.from_numpy(X).cuda()).cpu().numpy()
        assert p.device_status() == 0
        p.close()
        _check_bitwise(kp, X, feat)


def test_f16_paper_scale_sampled_pairs_bit_for_bit():
    import torch
    C, L, K, N = 20, 50000, 10000, 14
    kp = generate_kernels(8527, K, C, L)
    X = ar1_spike_series(2301, N, C, L)
    p = rk.RocketParams.from_kernel_params(kp)
    feat = rk.rocket_transform_f16(p, torch.from_numpy(X).cuda()).cpu().numpy()
    assert p.device_status() == 0
    p.close()
    rng = np.random.default_rng(3)
    pk = rng.choice(K, 600, replace=False).astype(np.int32)
    pn = rng.integers(0, N, size=600).astype(np.int32)
    _check_bitwise(kp, X, feat, pn, pk)
    print("half precision against double precision at 20 x 50,000: PPV %.2e, max %.2e" % _check_loose(kp, X, feat, pn, pk))
    # every pair: PPV in [0, 1], finite maxima
    ppv, mx = P.split_features(feat)
    assert np.all((ppv >= 0) & (ppv <= 1)) and np.all(np.isfinite(mx))


def test_f16_is_refused_for_kernels_outside_the_fused_kernels():
    import torch
    kp = kernels_from_lists(1, 64, [dict(weights=[[1.0, 0.0, -1.0]], bias=0.0)])      # length 3
    p = rk.RocketParams.from_kernel_params(kp)
    with pytest.raises(Exception):
        rk.rocket_transform_f16(p, torch.zeros((1, 1, 64), device="cuda"))
    p.close()
