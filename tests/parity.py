"""Helpers shared by the GPU parity tests (comparison rules only; no arithmetic
of the method lives here)."""
import math

import numpy as np

TOL_F32 = 1e-4      # reductions over fp32 inputs, relative
TOL_BF16 = 1e-3     # bf16 Gram path, relative


def rel_close(a, b, tol):
    return abs(a - b) <= tol * max(abs(a), abs(b), 1e-300)


def assert_test_result(gpu, ora, params, tol, *, stat_tol=None, what=""):
    """gpu: binding.TestResult; ora: oracle NormTestResult; params: binding.TestParams.

    Scalars within `tol` relative.  Decisions are compared exactly whenever the
    oracle's statistic is farther than the tolerance from the threshold that
    decides them: integers for b_req, b_cur for GROW, switch_n*b_max for
    ACCUMULATE, multiples of b_max for accum_steps."""
    stat_tol = tol if stat_tol is None else stat_tol
    assert gpu.device_status == 0, what
    assert gpu.batch_count == ora.batch_count, what
    if ora.flags & 16:        # a non-finite sum: no statistic, only the plan is defined
        assert gpu.flags == ora.flags and gpu.b_req == ora.b_req, (what, gpu.flags, ora.flags)
        assert (gpu.accum_steps, gpu.b_micro) == (ora.accum_steps, ora.b_micro), what
        assert gpu.stat == 0.0 and gpu.variance == 0.0, what
        return {"decisive": True}
    assert rel_close(gpu.sum_sqnorm, ora.sum_sqnorm, tol), (what, gpu.sum_sqnorm, ora.sum_sqnorm)
    assert rel_close(gpu.mean_sqnorm, ora.mean_sqnorm, tol), (what, gpu.mean_sqnorm, ora.mean_sqnorm)
    special = ora.flags & (4 | 8)
    assert (gpu.flags & (4 | 8)) == special, (what, gpu.flags, ora.flags)
    if special:
        assert gpu.b_req == ora.b_req and gpu.flags == ora.flags, what
        assert (gpu.accum_steps, gpu.b_micro) == (ora.accum_steps, ora.b_micro), what
        return {"decisive": True}
    # variance: absolute error scaled by the size of the terms it is formed from
    v_scale = max(abs(ora.variance), 1e-300)
    assert abs(gpu.variance - ora.variance) <= stat_tol * v_scale + 1e-30, (what, gpu.variance, ora.variance)
    assert rel_close(gpu.stat, ora.stat, 2 * stat_tol) or abs(gpu.stat - ora.stat) < 1e-30, (what, gpu.stat, ora.stat)
    s = ora.stat
    band = 2 * stat_tol * abs(s)
    uncapped = params.b_cap == 0 or math.ceil(s) < params.b_cap
    dec_breq = (not uncapped) or abs(s - round(s)) > band or s < 1.0 - band
    out = {"decisive": dec_breq, "frac": s - math.floor(s)}
    if dec_breq:
        assert gpu.b_req == ora.b_req, (what, gpu.b_req, ora.b_req, s)
        assert gpu.flags == ora.flags, (what, gpu.flags, ora.flags)
        assert (gpu.accum_steps, gpu.b_micro) == (ora.accum_steps, ora.b_micro), what
        return out
    assert abs(gpu.b_req - ora.b_req) <= 1, (what, gpu.b_req, ora.b_req)
    if abs(s - params.b_cur) > band + 1:
        assert (gpu.flags & 1) == (ora.flags & 1), what
    thr = params.switch_n * params.b_max
    if abs(s - thr) > band + 1:
        assert (gpu.flags & 2) == (ora.flags & 2), what
        if abs(s / params.b_max - round(s / params.b_max)) * params.b_max > band + 1:
            assert (gpu.accum_steps, gpu.b_micro) == (ora.accum_steps, ora.b_micro), what
    return out


def ulp32(mag):
    """Spacing of float32 at magnitude mag (array)."""
    m = np.maximum(np.abs(mag), np.float64(np.finfo(np.float32).tiny)).astype(np.float32)
    return np.spacing(m).astype(np.float64)


def assert_outer_step(theta_gpu, mom_gpu, theta_ref, mom_ref, theta_old, mom_old, d_ref, lr, mu, what=""):
    """Elementwise within 2 fp32 ulp, the ulp taken at the largest magnitude that
    enters the final subtraction (theta, theta', lr*u) resp. (v', mu*v, d)."""
    th = theta_gpu.astype(np.float64)
    v = mom_gpu.astype(np.float64)
    lr_u = theta_old - theta_ref
    mag_t = np.maximum(np.maximum(np.abs(theta_old), np.abs(theta_ref)), np.abs(lr_u))
    mag_v = np.maximum(np.maximum(np.abs(mom_ref), np.abs(mu * mom_old)), np.abs(d_ref))
    et = np.abs(th - theta_ref) / ulp32(mag_t)
    ev = np.abs(v - mom_ref) / ulp32(mag_v)
    assert et.max() <= 2.0, (what, "theta", float(et.max()), int(et.argmax()))
    assert ev.max() <= 2.0, (what, "momentum", float(ev.max()), int(ev.argmax()))
    return float(et.max()), float(ev.max())
