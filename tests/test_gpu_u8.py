"""GPU-vs-oracle parity of the 8-bit entry points (raw intensities scaled per channel, Sections 4.1
and 4.3) through the C ABI: fused route, fp32-copy route, host-buffer form; hard and soft."""
import numpy as np
import pytest

import oracle
import paper_2301_08527_b200 as rk
from paper_2301_08527_b200 import binding
from rocket_inputs import channel_statistics, generate_kernels, intensity_series_u8, kernels_from_lists

import parity as P

pytestmark = pytest.mark.gpu


def _dev(a):
    import torch
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def _check_hard(kp, X8, mean, inv_std, feat, pn=None, pk=None):
    x = oracle.scale_u8(X8, mean, inv_std)
    ppv, mx = P.split_features(feat)
    if pn is None:
        ref = oracle.forward(kp, x)
        P.check_hard_ppv(ppv, ref)
        P.check_max(mx, ref)
    else:
        ref = oracle.forward_pairs(kp, x, pn, pk)
        P.check_hard_ppv(ppv[pn, pk], ref)
        P.check_max(mx[pn, pk], ref)


@pytest.mark.parametrize("path", [0, 1])
@pytest.mark.parametrize("C,L,K,N", [(20, 1000, 400, 3), (3, 516, 300, 2), (5, 4099, 200, 2), (1, 512, 300, 13)])
def test_hard_u8_small_full(path, C, L, K, N):
    # path 0 takes the fused route when L % 4 == 0, the fp32-copy route otherwise; path 1 always the copy
    kp = generate_kernels(31, K, C, L)
    X8 = intensity_series_u8(41, N, C, L)
    mean, inv_std = channel_statistics(X8)
    p = rk.RocketParams.from_kernel_params(kp)
    p.set_path(path)
    feat = rk.rocket_transform_u8(p, _dev(X8), mean, inv_std).cpu().numpy()
    assert p.device_status() == 0
    p.close()
    _check_hard(kp, X8, mean, inv_std, feat)


def test_hard_u8_equals_fp32_entry_point_on_the_scaled_input_bitwise():
    # the same fp32 samples reach the same kernels: the two entry points must agree bit for bit
    import torch
    kp = generate_kernels(32, 500, 20, 5000)
    X8 = intensity_series_u8(42, 14, 20, 5000)      # 14 examples: two chunks through the fused kernels
    mean, inv_std = channel_statistics(X8)
    p = rk.RocketParams.from_kernel_params(kp)
    x32 = (_dev(X8).to(torch.float32) - _dev(mean).view(1, -1, 1)) * _dev(inv_std).view(1, -1, 1)
    a = rk.rocket_transform_u8(p, _dev(X8), mean, inv_std)
    b = rk.rocket_transform(p, x32.contiguous())
    assert torch.equal(a, b)
    p.close()


@pytest.mark.parametrize("lam,shift", [(10.0, 3.0), (1.0, -3.0)])
def test_soft_u8_small_full(lam, shift):
    kp = generate_kernels(33, 300, 20, 1000)
    X8 = intensity_series_u8(43, 3, 20, 1000)
    mean, inv_std = channel_statistics(X8)
    p = rk.RocketParams.from_kernel_params(kp)
    feat, arg = rk.rocket_transform_soft_u8(p, _dev(X8), mean, inv_std, lam, shift)
    feat, arg = feat.cpu().numpy(), arg.cpu().numpy()
    p.close()
    ref = oracle.forward(kp, oracle.scale_u8(X8, mean, inv_std), lam=lam, shift=shift)
    soft, mx = P.split_features(feat)
    P.check_soft_ppv(soft, ref)
    P.check_max(mx, ref)
    P.check_argmax(arg, ref)


def test_hard_u8_paper_scale_sampled_and_host_form():
    # the shape bench.py times for this entry point: N=60, C=20, L=50,000, K=10,000
    import torch
    kp = generate_kernels(8527, 10000, 20, 50000)
    X8 = intensity_series_u8(2302, 60, 20, 50000)
    mean, inv_std = channel_statistics(X8)
    p = rk.RocketParams.from_kernel_params(kp)
    feat_t = rk.rocket_transform_u8(p, _dev(X8), mean, inv_std)
    feat = feat_t.cpu().numpy()
    assert p.device_status() == 0
    ppv, mx = P.split_features(feat)
    assert np.all(np.isfinite(feat)) and np.all((ppv >= 0) & (ppv <= 1)) and np.array_equal(ppv > 0, mx > 0)
    rng = np.random.default_rng(3)
    ks = rng.choice(10000, 1000, replace=False)
    pn = np.concatenate([np.full(1000, 23), np.tile(np.arange(60), 10)]).astype(np.int32)
    pk = np.concatenate([ks, np.repeat(rng.choice(10000, 10, replace=False), 60)]).astype(np.int32)
    _check_hard(kp, X8, mean, inv_std, feat, pn, pk)
    host = torch.empty((60, 20000), dtype=torch.float32).pin_memory()
    binding.rocket_transform_u8_host(p, torch.from_numpy(X8).pin_memory(), mean, inv_std, host)
    assert torch.equal(host, feat_t.cpu())
    p.close()


def test_u8_argument_errors_and_edge_cases():
    import torch
    kp = generate_kernels(34, 64, 2, 64)
    p = rk.RocketParams.from_kernel_params(kp)
    X8 = _dev(intensity_series_u8(44, 2, 2, 64))
    with pytest.raises(ValueError):
        rk.rocket_transform_u8(p, X8, np.zeros(3), np.ones(3))
    with pytest.raises(rk.RocketError):
        rk.rocket_transform_u8(p, X8, np.array([0.0, np.nan]), np.ones(2))
    with pytest.raises(rk.RocketError):
        rk.rocket_transform_u8(p, _dev(np.zeros((2, 3, 64), np.uint8)), np.zeros(2), np.ones(2))
    empty = rk.rocket_transform_u8(p, torch.empty((0, 2, 64), dtype=torch.uint8, device="cuda"), np.zeros(2), np.ones(2))
    assert empty.shape == (0, 128)
    # a constant channel scaled to zero: every output is the bias
    kc = kernels_from_lists(1, 64, [dict(dilation=1, padding=0, channels=[0], weights=[[1, -2, 3, -4, 5, -6, 3]], bias=0.25)])
    pc = rk.RocketParams.from_kernel_params(kc)
    f = rk.rocket_transform_u8(pc, _dev(np.full((1, 1, 64), 77, np.uint8)), np.array([77.0]), np.array([2.0])).cpu().numpy()
    assert f[0, 0] == 1.0 and f[0, 1] == 0.25
    pc.close()
    p.close()
