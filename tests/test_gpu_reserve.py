"""rocket_params_reserve: after it, device calls within the reserved size allocate nothing."""
import numpy as np
import pytest

import oracle
import paper_2301_08527_b200 as rk
from rocket_inputs import ar1_spike_series, generate_kernels, kernels_from_lists, normal_array

import parity as P

pytestmark = pytest.mark.gpu


def _kernels_with_generic_lengths(C, L):
    rng = np.random.default_rng(5)
    ks = []
    for i in range(60):
        ln = [3, 5, 7, 9, 11][i % 5]
        d = int(rng.integers(1, max(2, (L - 1) // (ln - 1) // 2)))
        ks.append(dict(dilation=d, padding=(ln - 1) * d // 2 if i % 2 else 0, channels=sorted(rng.choice(C, 2, replace=False).tolist()),
                       weights=rng.normal(size=(2, ln)), bias=float(rng.uniform(-1, 1))))
    return kernels_from_lists(C, L, ks)


@pytest.mark.parametrize("case", ["fused kernels only", "fused and generic kernels", "generic path"])
def test_calls_after_reserve_do_not_allocate(case):
    import torch
    C, L, N = 6, 4000, 30                      # three chunks of the fused kernels' batch size
    kp = generate_kernels(91, 400, C, L) if case != "fused and generic kernels" else _kernels_with_generic_lengths(C, L)
    X = ar1_spike_series(92, N, C, L)
    g = normal_array(93, (N, 2 * kp.K))
    Xd = torch.from_numpy(X).cuda()
    gd = torch.from_numpy(g).cuda()
    X8 = torch.from_numpy(np.clip(np.round(X * 40 + 128), 0, 255).astype(np.uint8)).cuda()
    mean, istd = np.full(C, 128.0, np.float32), np.full(C, 1 / 40.0, np.float32)
    p = rk.RocketParams.from_kernel_params(kp)
    if case == "generic path":
        p.set_path(1)
    feat = torch.empty((N, 2 * kp.K), device="cuda")
    arg = torch.empty((N, kp.K), dtype=torch.int32, device="cuda")
    dW = torch.empty((p.n_weights,), device="cuda")
    db = torch.empty((kp.K,), device="cuda")
    p.reserve(N, rk.PASS_HARD | rk.PASS_SOFT | rk.PASS_BACKWARD | rk.PASS_U8_INPUT)
    torch.cuda.synchronize()
    before = rk.device_alloc_count()
    for n in (N, 7, N):                                     # smaller calls fit as well
        rk.rocket_transform(p, Xd[:n], out=feat[:n])
        rk.rocket_transform_soft(p, Xd[:n], 10.0, 3.0, out=feat[:n], argmax_out=arg[:n])
        rk.rocket_transform_soft_backward(p, Xd[:n], 10.0, 3.0, gd[:n], arg[:n], dW, db)
        rk.rocket_transform_u8(p, X8[:n], mean, istd, out=feat[:n])
    torch.cuda.synchronize()
    assert rk.device_alloc_count() == before, "a device call allocated after rocket_params_reserve"
    assert p.device_status() == 0
    # and the reserved workspace gives the right answers
    ref = oracle.forward(kp, X, lam=10.0, shift=3.0)
    sfeat, sarg = rk.rocket_transform_soft(p, Xd, 10.0, 3.0)
    soft, mx = P.split_features(sfeat.cpu().numpy())
    P.check_soft_ppv(soft, ref)
    P.check_max(mx, ref)
    dW2, db2 = rk.rocket_transform_soft_backward(p, Xd, 10.0, 3.0, gd, torch.from_numpy(ref.argmax.astype(np.int32)).cuda())
    rdW, rdb = oracle.backward(kp, X, g, ref.argmax, lam=10.0, shift=3.0)
    P.check_grads(dW2.cpu().numpy(), db2.cpu().numpy(), rdW, rdb)
    # a larger call than reserved still works (and may allocate)
    p.reserve(N + 5, rk.PASS_HARD)
    p.close()


def test_reserve_rejects_bad_arguments():
    kp = generate_kernels(94, 20, 2, 200)
    p = rk.RocketParams.from_kernel_params(kp)
    lib = rk.load_library()
    assert lib.rocket_params_reserve(p.handle, 0, 1) == -1
    assert lib.rocket_params_reserve(p.handle, 4, 0) == -1
    assert lib.rocket_params_reserve(p.handle, 4, 16) == -1
    assert lib.rocket_params_reserve(None, 4, 1) == -1
    p.close()
