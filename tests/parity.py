"""Shared comparison rules for the GPU-vs-oracle parity tests (tolerances written out here).

  max          |gpu - oracle| <= 1e-5 * max(|oracle|, 1): the stated bound, relative error <= 1e-5,
               wherever |oracle| >= 1, and the same bound with |oracle| replaced by 1 below that
               (inputs are z-normalised and biases lie in [-1, 1), so 1 is the scale of the summed
               terms; a purely relative test would reject correctly rounded fp32 sums whose value
               happens to fall near zero: a sum of 30-120 products of size ~1 carries an fp32
               rounding error of a few 1e-7 whatever its own size).  check_max returns the share of
               pairs under the floor and the worst purely relative error on both sides of it.
  hard PPV     count accepted iff  P+ - 1e-4 n <= count <= P+ + AMB + 1e-4 n,  where P+ counts
               oracle outputs above 1e-5 and AMB those within 1e-5 of zero (their sign is not
               decidable in fp32)
  soft PPV     |gpu - oracle| <= 1e-5
  argmax       equal wherever the oracle's gap to the runner-up exceeds 1e-5 * max(1, |max|);
               elsewhere the GPU's index must still be a valid output index
  gradients    relative L2 error over concat(dW, db) <= 1e-4
"""
import numpy as np

MAX_RTOL = 1e-5
PPV_ATOL = 1e-4
AMB_EPS = 1e-5
SOFT_ATOL = 1e-5
GRAD_REL_L2 = 1e-4


def check_max(gpu_max, ref):
    """Asserts the max rule; returns a dict with the worst scaled error, the share of pairs whose
    |oracle max| lies under the floor of 1, and the worst purely relative error at or above / below
    the floor (the latter is reported, not asserted)."""
    gpu_max = np.asarray(gpu_max, np.float64)
    ref_max = np.asarray(ref.max, np.float64)
    assert np.all(np.isfinite(gpu_max))
    diff = np.abs(gpu_max - ref_max)
    err = diff / np.maximum(np.abs(ref_max), 1.0)
    assert err.max(initial=0.0) <= MAX_RTOL, "max err %.3g (scaled) at %s" % (err.max(), np.argmax(err))
    big = np.abs(ref_max) >= 1.0
    with np.errstate(divide="ignore", invalid="ignore"):
        rel = np.where(ref_max != 0.0, diff / np.abs(ref_max), np.where(diff == 0.0, 0.0, np.inf))
    rel_big = float(rel[big].max(initial=0.0))
    assert rel_big <= MAX_RTOL, "max relative err %.3g where |max| >= 1" % rel_big
    return {"scaled_err": float(err.max(initial=0.0)), "share_below_floor": float(1.0 - big.mean()) if big.size else 0.0,
            "rel_err_at_or_above_floor": rel_big, "rel_err_below_floor": float(rel[~big].max(initial=0.0)),
            "share_below_floor_over_1e-5": float((rel[~big] > MAX_RTOL).sum() / big.size) if big.size else 0.0}


def check_hard_ppv(gpu_ppv, ref):
    n = ref.out_len.astype(np.float64)
    cnt = np.asarray(gpu_ppv, np.float64) * n
    # the device stores count / n in fp32: recover the integer
    cnt_i = np.round(cnt)
    assert np.all(np.abs(cnt - cnt_i) <= 1e-6 * n + 1e-3), "PPV * n is not an integer"
    lo = ref.pos_eps - PPV_ATOL * n
    hi = ref.pos_eps + ref.amb + PPV_ATOL * n
    bad = (cnt_i < lo - 1e-9) | (cnt_i > hi + 1e-9)
    assert not bad.any(), "hard PPV outside the accepted band at %s" % (np.argwhere(bad)[:5],)
    return float(np.max(np.abs(np.asarray(gpu_ppv, np.float64) - ref.ppv), initial=0.0))


def check_soft_ppv(gpu_soft, ref):
    err = np.abs(np.asarray(gpu_soft, np.float64) - ref.soft)
    assert err.max(initial=0.0) <= SOFT_ATOL, "soft PPV abs err %.3g" % err.max()
    return float(err.max(initial=0.0))


def check_argmax(gpu_arg, ref):
    gpu_arg = np.asarray(gpu_arg)
    assert np.all((gpu_arg >= 0) & (gpu_arg < ref.out_len))
    decided = ref.gap > 1e-5 * np.maximum(1.0, np.abs(ref.max))
    assert np.array_equal(gpu_arg[decided], ref.argmax[decided])
    return float(decided.mean()) if decided.size else 1.0


def check_grads(gpu_dW, gpu_db, ref_dW, ref_db):
    a = np.concatenate([np.asarray(gpu_dW, np.float64).ravel(), np.asarray(gpu_db, np.float64).ravel()])
    b = np.concatenate([ref_dW.ravel(), ref_db.ravel()])
    assert np.all(np.isfinite(a))
    denom = np.linalg.norm(b)
    rel = np.linalg.norm(a - b) / denom if denom > 0 else np.linalg.norm(a - b)
    assert rel <= GRAD_REL_L2, "gradient rel L2 err %.3g" % rel
    return float(rel)


def split_features(feat):
    """[N, 2K] interleaved -> (first feature [N, K], max [N, K])."""
    feat = np.asarray(feat)
    return feat[:, 0::2], feat[:, 1::2]
