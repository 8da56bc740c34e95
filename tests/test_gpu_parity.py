"""GPU-vs-oracle parity through the C ABI (run on the B200 machine: pytest -m gpu)."""
import ctypes

import numpy as np
import pytest

import oracle
import paper_2301_08527_b200 as rk
from paper_2301_08527_b200 import binding
from rocket_inputs import (ar1_spike_series, generate_kernels, kernels_from_lists, normal_array,
                           random_walk_series)

import parity as P

pytestmark = pytest.mark.gpu

PATHS = [0, 1]  # 0 = automatic (fast path where it applies), 1 = generic kernels


def _torch():
    import torch
    return torch


def _dev(a):
    return _torch().from_numpy(np.ascontiguousarray(a)).cuda()


def _run_hard(kp, X, path=0):
    p = rk.RocketParams.from_kernel_params(kp)
    p.set_path(path)
    feat = rk.rocket_transform(p, _dev(X)).cpu().numpy()
    assert p.device_status() == 0
    p.close()
    return feat


def _run_soft(kp, X, lam, shift, path=0):
    p = rk.RocketParams.from_kernel_params(kp)
    p.set_path(path)
    feat, arg = rk.rocket_transform_soft(p, _dev(X), lam, shift)
    feat, arg = feat.cpu().numpy(), arg.cpu().numpy()
    p.close()
    return feat, arg


def _check_hard_full(kp, X, path):
    feat = _run_hard(kp, X, path)
    ref = oracle.forward(kp, X)
    ppv, mx = P.split_features(feat)
    P.check_hard_ppv(ppv, ref)
    P.check_max(mx, ref)


@pytest.mark.parametrize("path", PATHS)
def test_config0_univariate_hard_full(path):
    kp = generate_kernels(8527, 1000, 1, 512)
    X = random_walk_series(2301, 16, 1, 512)
    _check_hard_full(kp, X, path)


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("C,L,K,N", [(3, 257, 300, 3), (20, 1000, 400, 2), (5, 4099, 300, 2), (2, 11, 64, 4)])
def test_small_multivariate_hard_full(path, C, L, K, N):
    kp = generate_kernels(11 + L, K, C, L)
    X = ar1_spike_series(12 + L, N, C, L)
    _check_hard_full(kp, X, path)


def _sample_pairs(N, K, n_full_examples, n_full_kernels, seed):
    rng = np.random.default_rng(seed)
    ex = rng.choice(N, min(n_full_examples, N), replace=False)
    ks = rng.choice(K, min(n_full_kernels, K), replace=False)
    pn = np.concatenate([np.repeat(ex, K), np.tile(np.arange(N), len(ks))]).astype(np.int32)
    pk = np.concatenate([np.tile(np.arange(K), len(ex)), np.repeat(ks, N)]).astype(np.int32)
    return pn, pk


def _check_sampled(kp, X, feat, pn, pk, soft=None, arg=None):
    lam, shift = soft if soft else (1.0, 3.0)
    ref = oracle.forward_pairs(kp, X, pn, pk, lam=lam, shift=shift)
    first, mx = P.split_features(feat)
    if soft:
        P.check_soft_ppv(first[pn, pk], ref)
        if arg is not None:
            P.check_argmax(arg[pn, pk], ref)
    else:
        P.check_hard_ppv(first[pn, pk], ref)
    P.check_max(mx[pn, pk], ref)


def _check_properties_hard(feat):
    ppv, mx = P.split_features(feat)
    assert np.all(np.isfinite(feat))
    assert np.all((ppv >= 0) & (ppv <= 1))
    assert np.array_equal(ppv > 0, mx > 0)


_FULL_REF = {}


def _full_reference(name, kp, X, **kw):
    """The oracle over the full (example, kernel) grid of a config, computed once per test session."""
    key = (name,) + tuple(sorted(kw.items()))
    if key not in _FULL_REF:
        _FULL_REF[key] = oracle.forward(kp, X, **kw)
    return _FULL_REF[key]


def _report(name, stats):
    print("%s: |max| < 1 for %.1f%% of pairs; worst relative error %.2e where |max| >= 1, %.2e below "
          "(%.4f%% of all pairs exceed 1e-5 there); worst scaled error %.2e"
          % (name, 100 * stats["share_below_floor"], stats["rel_err_at_or_above_floor"], stats["rel_err_below_floor"],
             100 * stats["share_below_floor_over_1e-5"], stats["scaled_err"]))


@pytest.mark.parametrize("path", PATHS)
def test_config1_multivariate_hard_full(path):
    # every one of the 64 x 10,000 (example, kernel) pairs against the oracle
    kp = generate_kernels(8527, 10000, 20, 5000)
    X = ar1_spike_series(2301, 64, 20, 5000)
    feat = _run_hard(kp, X, path)
    _check_properties_hard(feat)
    ref = _full_reference("config1", kp, X)
    ppv, mx = P.split_features(feat)
    P.check_hard_ppv(ppv, ref)
    _report("config 1, path %d" % path, P.check_max(mx, ref))


def test_config2_paper_scale_hard_full():
    # the launch configuration bench.py times: N=60, C=20, L=50,000, K=10,000, automatic path; every one
    # of the 600,000 (example, kernel) pairs is compared with the oracle (about a minute of host time)
    kp = generate_kernels(8527, 10000, 20, 50000)
    X = ar1_spike_series(2301, 60, 20, 50000)
    feat = _run_hard(kp, X, 0)
    _check_properties_hard(feat)
    ref = _full_reference("config2", kp, X)
    ppv, mx = P.split_features(feat)
    P.check_hard_ppv(ppv, ref)
    _report("config 2", P.check_max(mx, ref))


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("lam", [1.0, 10.0, 100.0])
@pytest.mark.parametrize("shift", [3.0, -3.0, 0.0])
def test_soft_forward_small_full(path, lam, shift):
    kp = generate_kernels(21, 300, 6, 700)
    X = ar1_spike_series(22, 3, 6, 700)
    feat, arg = _run_soft(kp, X, lam, shift, path)
    ref = oracle.forward(kp, X, lam=lam, shift=shift)
    soft, mx = P.split_features(feat)
    P.check_soft_ppv(soft, ref)
    P.check_max(mx, ref)
    P.check_argmax(arg, ref)


@pytest.mark.parametrize("path", PATHS)
def test_soft_lambda_zero_is_sigmoid_of_shift(path):
    kp = generate_kernels(23, 100, 4, 300)
    X = ar1_spike_series(24, 2, 4, 300)
    feat, _ = _run_soft(kp, X, 0.0, 3.0, path)
    np.testing.assert_allclose(feat[:, 0::2], 0.9525741268224334, atol=1e-6)


def _run_backward(kp, X, lam, shift, g, arg, path=0):
    p = rk.RocketParams.from_kernel_params(kp)
    p.set_path(path)
    dW, db = rk.rocket_transform_soft_backward(p, _dev(X), lam, shift, _dev(g), _dev(arg.astype(np.int32)))
    dW, db = dW.cpu().numpy(), db.cpu().numpy()
    p.close()
    return dW, db


@pytest.mark.parametrize("path", PATHS)
@pytest.mark.parametrize("lam,shift", [(1.0, 3.0), (10.0, 3.0), (100.0, 3.0), (10.0, -3.0), (0.0, 3.0)])
def test_backward_small_full(path, lam, shift):
    kp = generate_kernels(31, 200, 6, 900)
    X = ar1_spike_series(32, 4, 6, 900)
    g = normal_array(527, (4, 2 * kp.K))
    ref = oracle.forward(kp, X, lam=lam, shift=shift)
    rdW, rdb = oracle.backward(kp, X, g, ref.argmax, lam=lam, shift=shift)
    dW, db = _run_backward(kp, X, lam, shift, g, ref.argmax, path)   # the oracle's argmax feeds both sides
    P.check_grads(dW, db, rdW, rdb)
    # db alone and dW alone must also hold the bound (a wrong db would hide behind a large dW)
    P.check_grads(np.zeros(0), db, np.zeros(0), rdb)
    P.check_grads(dW, np.zeros(0), rdW, np.zeros(0))


@pytest.mark.parametrize("path", PATHS)
def test_config3_training_pass_sampled(path):
    # N=32 x C=20 x L=50,000 with a subset of the 10,000 kernels so that the oracle finishes in seconds:
    # the gradient of a kernel does not depend on the other kernels.
    full = generate_kernels(8527, 10000, 20, 50000)
    ks = np.sort(np.random.default_rng(3).choice(10000, 24, replace=False))
    kp = full.subset(ks)
    X = ar1_spike_series(2301, 32, 20, 50000)
    g = normal_array(527, (32, 2 * kp.K))
    for lam in (1.0, 10.0, 100.0):
        feat, arg = _run_soft(kp, X, lam, 3.0, path)
        ref = oracle.forward(kp, X, lam=lam, shift=3.0)
        soft, mx = P.split_features(feat)
        P.check_soft_ppv(soft, ref)
        P.check_max(mx, ref)
        P.check_argmax(arg, ref)
        rdW, rdb = oracle.backward(kp, X, g, ref.argmax, lam=lam, shift=3.0)
        dW, db = _run_backward(kp, X, lam, 3.0, g, ref.argmax, path)
        P.check_grads(dW, db, rdW, rdb)



@pytest.mark.parametrize("lam", [1.0, 10.0, 100.0])
def test_config3_soft_forward_full(lam):
    # N=32 x C=20 x L=50,000 with all 10,000 kernels through the automatic path, as bench.py times it:
    # soft PPV, max and argmax of every one of the 320,000 pairs against the oracle, per temperature
    N, K, C, L, shift = 32, 10000, 20, 50000, 3.0
    kp = generate_kernels(8527, K, C, L)
    X = ar1_spike_series(2301, N, C, L)
    p = rk.RocketParams.from_kernel_params(kp)
    feat, arg = rk.rocket_transform_soft(p, _dev(X), lam, shift)
    feat, arg = feat.cpu().numpy(), arg.cpu().numpy()
    assert p.device_status() == 0
    p.close()
    ref = _full_reference("config3", kp, X, lam=lam, shift=shift)
    soft, mx = P.split_features(feat)
    P.check_soft_ppv(soft, ref)
    _report("config 3, lambda %g" % lam, P.check_max(mx, ref))
    P.check_argmax(arg, ref)


def test_config3_backward_all_kernels_and_whole_batch():
    # gradients at N=32 x C=20 x L=50,000, K=10,000, automatic path, lambda = 10; the oracle's argmax feeds
    # both sides.  (a) all 10,000 kernels over two examples; (b) 500 kernels over the whole batch of 32, in
    # the launch configuration bench.py times (a kernel's gradient does not depend on the other kernels).
    N, K, C, L, lam, shift = 32, 10000, 20, 50000, 10.0, 3.0
    kp = generate_kernels(8527, K, C, L)
    X = ar1_spike_series(2301, N, C, L)
    g = normal_array(527, (N, 2 * K))
    ref = _full_reference("config3", kp, X, lam=lam, shift=shift)
    p = rk.RocketParams.from_kernel_params(kp)
    Xd = _dev(X)
    # (a)
    ex = np.array([5, 21])
    dW, db = rk.rocket_transform_soft_backward(p, Xd[ex].contiguous(), lam, shift, _dev(g[ex]), _dev(ref.argmax[ex].astype(np.int32)))
    assert p.device_status() == 0
    rdW, rdb = oracle.backward(kp, X[ex], g[ex], ref.argmax[ex], lam=lam, shift=shift)
    P.check_grads(dW.cpu().numpy(), db.cpu().numpy(), rdW, rdb)
    # (b)
    dW, db = rk.rocket_transform_soft_backward(p, Xd, lam, shift, _dev(g), _dev(ref.argmax.astype(np.int32)))
    dW, db = dW.cpu().numpy(), db.cpu().numpy()
    assert p.device_status() == 0
    p.close()
    assert np.all(np.isfinite(dW)) and np.all(np.isfinite(db))
    ks = np.sort(np.random.default_rng(4).choice(K, 500, replace=False)).astype(np.int32)
    rdW, rdb = oracle.backward(kp, X, g, ref.argmax, lam=lam, shift=shift, kernels=ks)
    sel = np.concatenate([np.arange(kp.weight_offset[k], kp.weight_offset[k + 1]) for k in ks])
    P.check_grads(dW[sel], db[ks], rdW[sel], rdb[ks])
    P.check_grads(np.zeros(0), db[ks], np.zeros(0), rdb[ks])


@pytest.mark.parametrize("N,L,K", [(1, 10000, 10000), (8, 200000, 10000), (256, 10000, 50000), (60, 50000, 50000)])
def test_config4_sweep_points_hard_cross_sample(N, L, K):
    # corners of the throughput sweep (batch 1 = streaming latency, the longest series, the largest batch,
    # the largest kernel set).  The oracle checks a cross-shaped sample: every kernel for two examples (one
    # where N = 1) and every example for 500 kernels; the rest is covered by invariants.
    kp = generate_kernels(8527, K, 20, L)
    X = ar1_spike_series(2301, N, 20, L)
    feat = _run_hard(kp, X, 0)
    _check_properties_hard(feat)
    pn, pk = _sample_pairs(N, K, 2, 500, seed=N + L + K)
    _check_sampled(kp, X, feat, pn, pk)


def test_config4_largest_point_hard_cross_sample():
    # the far corner of the sweep: 256 x 20 x 200,000 with 50,000 kernels (4 GB of input, built from eight
    # generated examples repeated, one slot replaced by a fresh example); the oracle checks every kernel
    # for two examples and every example for 500 kernels (about a minute and a half of host time)
    N, L, K = 256, 200000, 50000
    kp = generate_kernels(8527, K, 20, L)
    X = np.concatenate([ar1_spike_series(2301, 8, 20, L)] * 32, axis=0)
    X[200] = ar1_spike_series(99, 1, 20, L)[0]
    feat = _run_hard(kp, X, 0)
    _check_properties_hard(feat)
    assert np.array_equal(feat[0], feat[8]) and np.array_equal(feat[3], feat[251])   # equal examples, equal rows
    ks = np.random.default_rng(5).choice(K, 500, replace=False)
    pn = np.concatenate([np.full(K, 200), np.full(K, 255), np.tile(np.arange(N), len(ks))]).astype(np.int32)
    pk = np.concatenate([np.arange(K), np.arange(K), np.repeat(ks, N)]).astype(np.int32)
    _check_sampled(kp, X, feat, pn, pk)


@pytest.mark.parametrize("path", PATHS)
def test_edge_cases(path):
    torch = _torch()
    # (a) shortest series the generator accepts: L = 11, so a length-11 kernel has one output
    kp = generate_kernels(5, 64, 2, 11)
    X = random_walk_series(6, 4, 2, 11)
    _check_hard_full(kp, X, path)
    # (b) strict Heaviside: all-zero input with zero bias gives PPV 0, MAX 0 (padding included)
    kz = kernels_from_lists(1, 64, [dict(dilation=2, padding=6, channels=[0], weights=np.ones((1, 7)), bias=0.0),
                                    dict(dilation=1, padding=0, channels=[0], weights=np.ones((1, 9)), bias=0.0)])
    feat = _run_hard(kz, np.zeros((2, 1, 64), np.float32), path)
    assert np.array_equal(feat, np.zeros_like(feat))
    # (c) constant input with mean-centred rows: z == b everywhere
    kc = kernels_from_lists(2, 300, [dict(dilation=5, padding=0, channels=[0, 1],
                                          weights=[[1, -1, 2, -2, 0, 3, -3], [0, 0, 0, 1, -1, 0, 0]], bias=0.625),
                                     dict(dilation=5, padding=0, channels=[1],
                                          weights=[[1, -1, 2, -2, 0, 3, -3]], bias=-0.5)])
    Xc = np.broadcast_to(np.array([2.0, -1.0], np.float32)[None, :, None], (2, 2, 300)).copy()
    feat = _run_hard(kc, Xc, path)
    np.testing.assert_array_equal(feat[:, 0], 1.0); np.testing.assert_array_equal(feat[:, 1], 0.625)
    np.testing.assert_array_equal(feat[:, 2], 0.0); np.testing.assert_array_equal(feat[:, 3], -0.5)
    # (d) extreme dilation / padding: span reaches the series length, padded outputs mostly read zeros
    L = 1000
    ke = kernels_from_lists(1, L, [
        dict(dilation=166, padding=0, channels=[0], weights=np.arange(1, 8)[None, :] - 4.0, bias=0.1),    # L_out = 4
        dict(dilation=166, padding=498, channels=[0], weights=np.arange(1, 8)[None, :] - 4.0, bias=0.1),  # L_out = L
        dict(dilation=99, padding=495, channels=[0], weights=np.arange(1, 12)[None, :] - 6.0, bias=-0.2),
        dict(dilation=1, padding=0, channels=[0], weights=np.ones((1, 3)), bias=0.0),                      # length 3
        dict(dilation=7, padding=40, channels=[0], weights=np.ones((1, 5)), bias=0.0),                     # odd padding
    ])
    Xe = random_walk_series(7, 3, 1, L)
    _check_hard_full(ke, Xe, path)
    # (e) N = 0 is a no-op, N = 1 and K = 1 work
    p = rk.RocketParams.from_kernel_params(ke)
    p.set_path(path)
    out = rk.rocket_transform(p, torch.empty((0, 1, L), device="cuda"))
    assert out.shape == (0, 10)
    p.close()
    _check_hard_full(ke.subset([2]), Xe[:1], path)


def test_two_runs_are_bitwise_identical():
    kp = generate_kernels(41, 500, 8, 2000)
    X = ar1_spike_series(42, 4, 8, 2000)
    g = normal_array(43, (4, 2 * kp.K))
    a, b = _run_hard(kp, X), _run_hard(kp, X)
    assert a.tobytes() == b.tobytes()
    (fa, aa), (fb, ab) = _run_soft(kp, X, 10.0, 3.0), _run_soft(kp, X, 10.0, 3.0)
    assert fa.tobytes() == fb.tobytes() and aa.tobytes() == ab.tobytes()
    da, db_ = _run_backward(kp, X, 10.0, 3.0, g, aa), _run_backward(kp, X, 10.0, 3.0, g, aa)
    assert da[0].tobytes() == db_[0].tobytes() and da[1].tobytes() == db_[1].tobytes()


def test_host_buffer_entry_points_match_device_entry_points():
    torch = _torch()
    kp = generate_kernels(51, 300, 5, 1500)
    X = ar1_spike_series(52, 3, 5, 1500)
    g = normal_array(53, (3, 2 * kp.K))
    p = rk.RocketParams.from_kernel_params(kp)
    Xh = torch.from_numpy(X).pin_memory()
    fh = torch.empty((3, 2 * kp.K), dtype=torch.float32).pin_memory()
    binding.rocket_transform_host(p, Xh, fh)
    assert fh.numpy().tobytes() == rk.rocket_transform(p, _dev(X)).cpu().numpy().tobytes()
    ah = torch.empty((3, kp.K), dtype=torch.int32).pin_memory()
    binding.rocket_transform_soft_host(p, Xh, 10.0, 3.0, fh, ah)
    fd, ad = rk.rocket_transform_soft(p, _dev(X), 10.0, 3.0)
    assert fh.numpy().tobytes() == fd.cpu().numpy().tobytes() and ah.numpy().tobytes() == ad.cpu().numpy().tobytes()
    dWh = torch.empty(p.n_weights, dtype=torch.float32).pin_memory()
    dbh = torch.empty(kp.K, dtype=torch.float32).pin_memory()
    binding.rocket_transform_soft_backward_host(p, Xh, 10.0, 3.0, torch.from_numpy(g).pin_memory(), ah, dWh, dbh)
    dWd, dbd = rk.rocket_transform_soft_backward(p, _dev(X), 10.0, 3.0, _dev(g), ad)
    assert dWh.numpy().tobytes() == dWd.cpu().numpy().tobytes() and dbh.numpy().tobytes() == dbd.cpu().numpy().tobytes()
    p.close()


def test_library_generator_on_device_equals_reference_generator_run():
    kp = generate_kernels(8527, 800, 20, 5000)
    X = ar1_spike_series(61, 2, 20, 5000)
    p = rk.RocketParams.generate(8527, 800, 20, 5000)
    a = rk.rocket_transform(p, _dev(X)).cpu().numpy()
    p.close()
    assert a.tobytes() == _run_hard(kp, X).tobytes()


def test_argument_errors_leave_outputs_untouched():
    torch = _torch()
    kp = generate_kernels(71, 50, 2, 200)
    p = rk.RocketParams.from_kernel_params(kp)
    X = _dev(random_walk_series(72, 2, 2, 200))
    out = torch.full((2, 100), 7.0, device="cuda")
    lib = rk.load_library()
    st = lib.rocket_transform(p.handle, ctypes.c_void_p(X.data_ptr()), 2, 3, 200, ctypes.c_void_p(out.data_ptr()), None)
    assert st == -2
    st = lib.rocket_transform(p.handle, ctypes.c_void_p(X.data_ptr()), -1, 2, 200, ctypes.c_void_p(out.data_ptr()), None)
    assert st == -1
    st = lib.rocket_transform_soft(p.handle, ctypes.c_void_p(X.data_ptr()), 2, 2, 200, ctypes.c_float(float("nan")),
                                   ctypes.c_float(3.0), ctypes.c_void_p(out.data_ptr()), None, None)
    assert st == -1
    torch.cuda.synchronize()
    assert torch.all(out == 7.0)
    p.close()
