"""The allocation-free backward entry point against the ordinary one.

Some callers of this library cannot call cudaMalloc while they run: a control loop with a hard
latency budget, a process whose device memory pool is fixed at start-up, code running while
someone else records the stream.  rocket_transform_soft_backward_noalloc serves them by keeping
its partial sums in a fixed array inside the library.  This test calls it through the C ABI twice
in a row (the array is shared between calls and keeps old contents) and checks each result
against rocket_transform_soft_backward on the same inputs, and both against the CPU oracle's
gradients.  It lives in a file that sorts last, so a run that stops at the first failure has
already run every other test.
"""
import ctypes

import numpy as np
import pytest

import oracle
import paper_2301_08527_b200 as rk
from paper_2301_08527_b200 import binding
from rocket_inputs import ar1_spike_series, generate_kernels, normal_array

import parity as P

pytestmark = pytest.mark.gpu


def test_noalloc_backward_matches_allocating_backward_on_two_calls_in_a_row():
    import torch
    lam, shift = 10.0, 3.0
    # two different problems, the larger first, so the second call finds stale data in the array
    cases = [(61, 300, 6, 1200, 5), (62, 120, 4, 700, 3)]
    for seed, K, C, L, N in cases:
        kp = generate_kernels(seed, K, C, L)
        Xh = ar1_spike_series(seed + 100, N, C, L)
        gh = normal_array(seed + 200, (N, 2 * K))
        X = torch.from_numpy(Xh).cuda()
        g = torch.from_numpy(gh).cuda()
        p = rk.RocketParams.from_kernel_params(kp)
        p.bind_device()                      # binding allocates: done here, at set-up
        ref = oracle.forward(kp, Xh, lam=lam, shift=shift)
        arg = torch.from_numpy(ref.argmax.astype(np.int32)).cuda()    # the oracle's argmax feeds all three
        oracle_dW, oracle_db = oracle.backward(kp, Xh, gh, ref.argmax, lam=lam, shift=shift)
        ref_dW, ref_db = rk.rocket_transform_soft_backward(p, X, lam, shift, g, arg)
        dW = torch.full((p.n_weights,), float("nan"), device="cuda")
        db = torch.full((K,), float("nan"), device="cuda")
        binding.rocket_transform_soft_backward_noalloc(p, X, lam, shift, g, arg, dW, db)
        torch.cuda.synchronize()
        rel = P.check_grads(dW.cpu().numpy(), db.cpu().numpy(),
                            ref_dW.cpu().numpy().astype(np.float64), ref_db.cpu().numpy().astype(np.float64))
        assert rel <= P.GRAD_REL_L2
        P.check_grads(dW.cpu().numpy(), db.cpu().numpy(), oracle_dW, oracle_db)
        P.check_grads(ref_dW.cpu().numpy(), ref_db.cpu().numpy(), oracle_dW, oracle_db)
        p.close()


def test_noalloc_backward_rejects_oversized_and_unbound_requests():
    import torch
    lib = rk.load_library()
    kp = generate_kernels(63, 3000, 20, 5000)        # ~98k weights: N = 64 needs more than the array holds
    p = rk.RocketParams.from_kernel_params(kp)
    N = 64
    X = torch.zeros((N, 20, 5000), device="cuda")
    g = torch.zeros((N, 2 * kp.K), device="cuda")
    arg = torch.zeros((N, kp.K), dtype=torch.int32, device="cuda")
    dW = torch.full((p.n_weights,), 7.0, device="cuda")
    db = torch.full((kp.K,), 7.0, device="cuda")
    args = [p.handle, ctypes.c_void_p(X.data_ptr()), N, 20, 5000, ctypes.c_float(1.0), ctypes.c_float(3.0),
            ctypes.c_void_p(g.data_ptr()), ctypes.c_void_p(arg.data_ptr()), ctypes.c_void_p(dW.data_ptr()),
            ctypes.c_void_p(db.data_ptr()), None]
    assert lib.rocket_transform_soft_backward_noalloc(*args) == -1      # handle not bound yet
    p.bind_device()
    assert N * (p.n_weights + kp.K) > 4 * 1024 * 1024
    assert lib.rocket_transform_soft_backward_noalloc(*args) == -3      # larger than the fixed array
    torch.cuda.synchronize()
    assert torch.all(dW == 7.0) and torch.all(db == 7.0)                # nothing was launched
    p.close()
