"""ctypes binding of libadloco.so: the same entry points as include/adloco.h,
taking torch tensors.  Argument marshalling only -- every step of the path runs
in the CUDA kernels behind the C ABI.  There is no fallback: if the library is
not built or no CUDA device is present, loading or the first call fails.
"""
from __future__ import annotations

import ctypes as C
import os
from dataclasses import dataclass

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libadloco.so")

OK = 0
ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_ALIGNMENT, ERR_CUDA, ERR_WORKSPACE, ERR_TIMEOUT = -1, -2, -3, -4, -5, -6
F32, BF16 = 0, 1
FLAG_GROW, FLAG_ACCUMULATE, FLAG_UNDEFINED, FLAG_ZERO_MEAN, FLAG_NONFINITE = 1, 2, 4, 8, 16

# every symbol that include/adloco.h declares
EXPORTS = (
    "adloco_create", "adloco_destroy", "adloco_status_string", "adloco_last_cuda_error", "adloco_launch_count",
    "adloco_set_wait_limit", "adloco_device_status",
    "adloco_norm_test", "adloco_test_decide", "adloco_norm_test_host", "adloco_norm_test_noalloc", "adloco_inner_product_test", "adloco_gram_sqnorm", "adloco_linear_sqnorm", "adloco_linear_sqnorm_group", "adloco_vector_param_sqnorm", "adloco_embedding_sqnorm",
    "adloco_accum_create", "adloco_accum_reset", "adloco_accum_destroy", "adloco_accumulate",
    "adloco_accum_finalize", "adloco_outer_step", "adloco_outer_step_host", "adloco_check_merge", "adloco_merge",
    "adloco_pseudo_gradient", "adloco_outer_apply", "adloco_refresh_instance",
)


class TestParams(C.Structure):
    __test__ = False
    _fields_ = [("eta", C.c_double), ("ddof", C.c_int32), ("switch_n", C.c_int32),
                ("b_cur", C.c_int64), ("b_max", C.c_int64), ("b_cap", C.c_int64)]


class TestSums(C.Structure):
    __test__ = False
    _fields_ = [("sum_sqnorm", C.c_double), ("sum_sq_gsum", C.c_double), ("centred_ss", C.c_double),
                ("batch_count", C.c_int64), ("has_centred", C.c_int32), ("device_status", C.c_int32)]


class TestResult(C.Structure):
    __test__ = False
    _fields_ = [("sum_sqnorm", C.c_double), ("mean_sqnorm", C.c_double), ("variance", C.c_double),
                ("stat", C.c_double), ("batch_count", C.c_int64), ("b_req", C.c_int64),
                ("accum_steps", C.c_int64), ("b_micro", C.c_int64), ("flags", C.c_uint32),
                ("device_status", C.c_int32)]

    def as_dict(self):
        return {n: getattr(self, n) for n, _ in self._fields_}


class IpParams(C.Structure):
    _fields_ = [("theta", C.c_double), ("nu", C.c_double), ("ddof", C.c_int32), ("reserved", C.c_int32),
                ("b_cur", C.c_int64), ("b_cap", C.c_int64)]


class IpResult(C.Structure):
    _fields_ = [("var_ip", C.c_double), ("stat_ip", C.c_double), ("var_orth", C.c_double),
                ("stat_orth", C.c_double), ("mean_sqnorm", C.c_double), ("batch_count", C.c_int64),
                ("b_ip", C.c_int64), ("b_aug", C.c_int64), ("flags", C.c_uint32), ("device_status", C.c_int32)]


class LinearLayer(C.Structure):
    _fields_ = [("X", C.c_void_p), ("D", C.c_void_p), ("d_in", C.c_int64), ("d_out", C.c_int64),
                ("grad_sum", C.c_void_p)]


LINEAR_METHODS = {"auto": 0, "gram": 1, "direct": 2, "pair": 3, "gram_one_cta": 4, "gram_pair": 5}


class AdlocoError(RuntimeError):
    def __init__(self, status: int, msg: str):
        super().__init__(msg)
        self.status = status


_lib = None


def load_library() -> C.CDLL:
    """Loads libadloco.so (built in-tree by paper_2508_18182_b200.build); raises if absent."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise OSError(f"{LIB_PATH} is not built: run `python -m paper_2508_18182_b200.build`")
    lib = C.CDLL(LIB_PATH)
    vp, i32, i64, f32 = C.c_void_p, C.c_int32, C.c_int64, C.c_float
    sig = {
        "adloco_create": (C.c_int, [C.POINTER(vp), C.c_int]),
        "adloco_destroy": (C.c_int, [vp]),
        "adloco_status_string": (C.c_char_p, [C.c_int]),
        "adloco_last_cuda_error": (C.c_char_p, [vp]),
        "adloco_launch_count": (i64, [vp]),
        "adloco_set_wait_limit": (C.c_int, [vp, C.c_uint64]),
        "adloco_device_status": (C.c_int, [vp, C.POINTER(C.c_int32), C.c_int, vp]),
        "adloco_norm_test": (C.c_int, [vp, vp, C.c_int, i64, i64, i64, C.POINTER(TestParams), vp, vp, vp, vp, vp, vp]),
        "adloco_test_decide": (C.c_int, [vp, vp, C.POINTER(TestParams), vp, vp, vp]),
        "adloco_norm_test_host": (C.c_int, [vp, vp, i64, i64, i64, C.POINTER(TestParams), vp, vp, vp]),
        "adloco_norm_test_noalloc": (C.c_int, [vp, i64, i64, i64, C.POINTER(TestParams), vp, vp, vp, vp]),
        "adloco_inner_product_test": (C.c_int, [vp, vp, C.c_int, i64, i64, i64, C.POINTER(IpParams), vp, vp, vp, vp, vp, vp]),
        "adloco_gram_sqnorm": (C.c_int, [vp, vp, vp, i64, i64, i64, i64, vp, C.c_int, vp, C.c_int, vp]),
        "adloco_linear_sqnorm": (C.c_int, [vp, vp, vp, i64, i64, i64, i64, vp, C.c_int, vp, C.c_int, C.c_int, vp]),
        "adloco_linear_sqnorm_group": (C.c_int, [vp, C.POINTER(LinearLayer), i32, i64, i64, vp, C.c_int, C.c_int, C.c_int, vp]),
        "adloco_vector_param_sqnorm": (C.c_int, [vp, vp, vp, i64, i64, i64, vp, C.c_int, vp, C.c_int, vp]),
        "adloco_embedding_sqnorm": (C.c_int, [vp, vp, vp, i64, i64, i64, i64, vp, C.c_int, vp, C.c_int, vp]),
        "adloco_accum_create": (C.c_int, [vp, C.POINTER(vp), C.POINTER(vp), C.POINTER(i64), i32]),
        "adloco_accum_reset": (C.c_int, [vp, vp, vp]),
        "adloco_accum_destroy": (C.c_int, [vp]),
        "adloco_accumulate": (C.c_int, [vp, vp, vp, C.c_int, i64, i64, i64, vp, vp]),
        "adloco_accum_finalize": (C.c_int, [vp, vp, C.POINTER(TestParams), vp, vp, vp, vp]),
        "adloco_outer_step": (C.c_int, [vp, C.POINTER(vp), C.c_int, i32, i64, vp, vp, vp, vp, f32, f32, C.c_int,
                                        C.POINTER(vp), vp]),
        "adloco_outer_step_host": (C.c_int, [vp, C.POINTER(vp), C.c_int, i32, i64, vp, vp, f32, f32, C.c_int, vp]),
        "adloco_pseudo_gradient": (C.c_int, [vp, vp, vp, C.c_int, i64, vp, vp]),
        "adloco_outer_apply": (C.c_int, [vp, vp, i32, i64, vp, vp, vp, vp, f32, f32, C.c_int, vp]),
        "adloco_refresh_instance": (C.c_int, [vp, vp, vp, C.c_int, i64, vp]),
        "adloco_check_merge": (C.c_int, [C.POINTER(i64), i32, i32, C.POINTER(i32)]),
        "adloco_merge": (C.c_int, [vp, C.POINTER(vp), C.POINTER(i64), C.c_int, i32, i64, vp, C.POINTER(i32), vp]),
    }
    for name, (res, args) in sig.items():
        fn = getattr(lib, name)
        fn.restype, fn.argtypes = res, args
    _lib = lib
    return lib


def _ptr(t):
    return None if t is None else C.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return C.c_void_p(stream.cuda_stream)


def _dtype_code(dt):
    if dt == torch.float32:
        return F32
    if dt == torch.bfloat16:
        return BF16
    raise AdlocoError(ERR_UNSUPPORTED, f"unsupported dtype {dt}")


def make_params(eta, ddof=1, b_cur=1, b_max=1, b_cap=0, switch_n=2) -> TestParams:
    return TestParams(float(eta), int(ddof), int(switch_n), int(b_cur), int(b_max), int(b_cap))


class Context:
    """One adloco_ctx on a CUDA device."""

    def __init__(self, device: int = 0):
        self.lib = load_library()
        h = C.c_void_p()
        rc = self.lib.adloco_create(C.byref(h), int(device))
        if rc != OK:
            raise AdlocoError(rc, f"adloco_create: {self.lib.adloco_status_string(rc).decode()}")
        self.h = h
        self.device = torch.device("cuda", int(device))
        # small device/pinned scratch for results (torch owns the memory)
        self._res_dev = torch.zeros(TestResult_size(), dtype=torch.uint8, device=self.device)
        self._res_host = torch.zeros(TestResult_size(), dtype=torch.uint8).pin_memory()
        self._sums_dev = torch.zeros(C.sizeof(TestSums), dtype=torch.uint8, device=self.device)

    def close(self):
        if getattr(self, "h", None):
            torch.cuda.synchronize(self.device)
            self.lib.adloco_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def check(self, rc: int, what: str):
        if rc != OK:
            msg = self.lib.adloco_status_string(rc).decode()
            if rc == ERR_CUDA:
                msg += ": " + self.lib.adloco_last_cuda_error(self.h).decode()
            raise AdlocoError(rc, f"{what}: {msg}")

    def set_wait_limit(self, limit_ns: int):
        self.check(self.lib.adloco_set_wait_limit(self.h, int(limit_ns)), "adloco_set_wait_limit")

    def device_status(self, clear: bool = True, stream=None) -> int:
        v = C.c_int32(0)
        self.check(self.lib.adloco_device_status(self.h, C.byref(v), int(clear), _stream(stream)), "adloco_device_status")
        return v.value

    @property
    def launch_count(self) -> int:
        return int(self.lib.adloco_launch_count(self.h))

    def _read_result(self, stream=None) -> TestResult:
        (stream or torch.cuda.current_stream()).synchronize()
        return TestResult.from_buffer_copy(self._res_host.numpy().tobytes())

    def read_sums(self, sums_dev=None) -> TestSums:
        t = self._sums_dev if sums_dev is None else sums_dev
        return TestSums.from_buffer_copy(t.cpu().numpy().tobytes())

    # ------------------------------------------------------------------ norm test
    def norm_test(self, G, params: TestParams, *, per_sample_sqnorm=None, grad_sum=None, stream=None,
                  sync=True):
        """adloco_norm_test on a [B, P] float32 CUDA tensor (rows may be strided).
        Returns the TestResult (after synchronising) or None when sync=False."""
        B, P = G.shape
        stride = G.stride(0) if B > 1 else max(G.stride(0), P)
        if G.stride(1) != 1:
            raise AdlocoError(ERR_INVALID_ARG, "columns must be contiguous")
        rc = self.lib.adloco_norm_test(self.h, _ptr(G), _dtype_code(G.dtype), B, P, stride, C.byref(params),
                                       _ptr(per_sample_sqnorm), _ptr(grad_sum), _ptr(self._sums_dev),
                                       _ptr(self._res_dev), _ptr(self._res_host), _stream(stream))
        self.check(rc, "adloco_norm_test")
        return self._read_result(stream) if sync else None

    def test_decide(self, params: TestParams, *, sums_dev=None, stream=None, sync=True):
        """adloco_test_decide on the sums of the last norm_test (or the given device sums)."""
        s = self._sums_dev if sums_dev is None else sums_dev
        rc = self.lib.adloco_test_decide(self.h, _ptr(s), C.byref(params), _ptr(self._res_dev),
                                         _ptr(self._res_host), _stream(stream))
        self.check(rc, "adloco_test_decide")
        return self._read_result(stream) if sync else None

    def norm_test_host(self, G_host, params: TestParams, *, per_sample_sqnorm_host=None, stream=None):
        """adloco_norm_test_host on a [B, P] float32 HOST tensor (ideally pinned)."""
        B, P = G_host.shape
        res = TestResult()
        rc = self.lib.adloco_norm_test_host(self.h, _ptr(G_host), B, P, G_host.stride(0) if B > 1 else P,
                                            C.byref(params), _ptr(per_sample_sqnorm_host),
                                            C.cast(C.byref(res), C.c_void_p), _stream(stream))
        self.check(rc, "adloco_norm_test_host")
        return res

    def inner_product_test(self, G, grad_sum, *, theta, nu, ddof=1, b_cur=1, b_cap=0, inner_products=None,
                           sums_dev=None, stream=None) -> IpResult:
        """adloco_inner_product_test on the G whose norm test (with grad_sum) has just run on this context."""
        B, P = G.shape
        stride = G.stride(0) if B > 1 else max(G.stride(0), P)
        p = IpParams(float(theta), float(nu), int(ddof), 0, int(b_cur), int(b_cap))
        if not hasattr(self, "_ip_dev"):
            self._ip_dev = torch.zeros(C.sizeof(IpResult), dtype=torch.uint8, device=self.device)
            self._ip_host = torch.zeros(C.sizeof(IpResult), dtype=torch.uint8).pin_memory()
        s = self._sums_dev if sums_dev is None else sums_dev
        rc = self.lib.adloco_inner_product_test(self.h, _ptr(G), _dtype_code(G.dtype), B, P, stride, C.byref(p),
                                                _ptr(grad_sum), _ptr(s), _ptr(inner_products), _ptr(self._ip_dev),
                                                _ptr(self._ip_host), _stream(stream))
        self.check(rc, "adloco_inner_product_test")
        (stream or torch.cuda.current_stream()).synchronize()
        return IpResult.from_buffer_copy(self._ip_host.numpy().tobytes())

    # ------------------------------------------------------------------ Gram path
    def gram_sqnorm(self, X, D, per_sample_sqnorm, *, accumulate_norms=False, grad_sum=None,
                    accumulate_sum=False, stream=None):
        B, T, d_in = X.shape
        d_out = D.shape[2]
        if X.dtype != torch.bfloat16 or D.dtype != torch.bfloat16 or not X.is_contiguous() or not D.is_contiguous():
            raise AdlocoError(ERR_INVALID_ARG, "X and D must be contiguous bfloat16")
        rc = self.lib.adloco_gram_sqnorm(self.h, _ptr(X), _ptr(D), B, T, d_in, d_out, _ptr(per_sample_sqnorm),
                                         int(accumulate_norms), _ptr(grad_sum), int(accumulate_sum),
                                         _stream(stream))
        self.check(rc, "adloco_gram_sqnorm")

    def linear_sqnorm(self, X, D, per_sample_sqnorm, *, method="auto", accumulate_norms=False, grad_sum=None,
                      accumulate_sum=False, stream=None):
        """adloco_linear_sqnorm: method is "auto", "gram", "direct" or "pair"."""
        B, T, d_in = X.shape
        d_out = D.shape[2]
        if X.dtype != torch.bfloat16 or D.dtype != torch.bfloat16 or not X.is_contiguous() or not D.is_contiguous():
            raise AdlocoError(ERR_INVALID_ARG, "X and D must be contiguous bfloat16")
        code = LINEAR_METHODS[method]
        rc = self.lib.adloco_linear_sqnorm(self.h, _ptr(X), _ptr(D), B, T, d_in, d_out, _ptr(per_sample_sqnorm),
                                           int(accumulate_norms), _ptr(grad_sum), int(accumulate_sum), code,
                                           _stream(stream))
        self.check(rc, "adloco_linear_sqnorm")

    def make_layer_group(self, layers):
        """Marshals [(X, D, grad_sum or None), ...] (bf16 [B, T, d] tensors of one B and T) into the
        array adloco_linear_sqnorm_group takes; the result can be reused while the tensors live."""
        arr = (LinearLayer * len(layers))()
        B, T = layers[0][0].shape[0], layers[0][0].shape[1]
        for k, (X, D, S) in enumerate(layers):
            if (X.dtype != torch.bfloat16 or D.dtype != torch.bfloat16 or not X.is_contiguous() or not D.is_contiguous()
                    or X.shape[:2] != (B, T) or D.shape[:2] != (B, T)):
                raise AdlocoError(ERR_INVALID_ARG, "X and D must be contiguous bfloat16 [B, T, d] with one B and T")
            if S is not None and (S.dtype != torch.float32 or tuple(S.shape) != (D.shape[2], X.shape[2]) or not S.is_contiguous()):
                raise AdlocoError(ERR_INVALID_ARG, "grad_sum must be contiguous float32 [d_out, d_in]")
            arr[k] = LinearLayer(X.data_ptr(), D.data_ptr(), X.shape[2], D.shape[2], None if S is None else S.data_ptr())
        return arr, len(layers), B, T

    def linear_sqnorm_group(self, group, per_sample_sqnorm, *, method="auto", accumulate_norms=False,
                            accumulate_sum=False, stream=None):
        """adloco_linear_sqnorm_group on a group from make_layer_group (or a list of (X, D, S) triples);
        method is "auto", "direct" or "pair"."""
        if isinstance(group, (list, tuple)) and not isinstance(group[0], C.Array):
            group = self.make_layer_group(group)
        arr, n, B, T = group
        rc = self.lib.adloco_linear_sqnorm_group(self.h, arr, n, B, T, _ptr(per_sample_sqnorm), int(accumulate_norms),
                                                 int(accumulate_sum), LINEAR_METHODS[method], _stream(stream))
        self.check(rc, "adloco_linear_sqnorm_group")

    def vector_param_sqnorm(self, D, per_sample_sqnorm, *, X=None, accumulate_norms=False, grad_sum=None,
                            accumulate_sum=False, stream=None):
        """adloco_vector_param_sqnorm: bias (X=None) or elementwise gain (X given)."""
        B, T, d = D.shape
        if D.dtype != torch.bfloat16 or not D.is_contiguous() or (X is not None and (X.shape != D.shape or not X.is_contiguous())):
            raise AdlocoError(ERR_INVALID_ARG, "D (and X) must be contiguous bfloat16 of one shape")
        rc = self.lib.adloco_vector_param_sqnorm(self.h, _ptr(D), _ptr(X), B, T, d, _ptr(per_sample_sqnorm),
                                                 int(accumulate_norms), _ptr(grad_sum), int(accumulate_sum),
                                                 _stream(stream))
        self.check(rc, "adloco_vector_param_sqnorm")

    def embedding_sqnorm(self, token_ids, D, V, per_sample_sqnorm, *, accumulate_norms=False, grad_sum=None,
                         accumulate_sum=False, stream=None):
        """adloco_embedding_sqnorm: token_ids int32 [B, T], D bf16 [B, T, d], table of V rows."""
        B, T, d = D.shape
        if token_ids.dtype != torch.int32 or tuple(token_ids.shape) != (B, T) or not token_ids.is_contiguous():
            raise AdlocoError(ERR_INVALID_ARG, "token_ids must be contiguous int32 [B, T]")
        if D.dtype != torch.bfloat16 or not D.is_contiguous():
            raise AdlocoError(ERR_INVALID_ARG, "D must be contiguous bfloat16")
        rc = self.lib.adloco_embedding_sqnorm(self.h, _ptr(token_ids), _ptr(D), B, T, d, int(V), _ptr(per_sample_sqnorm),
                                              int(accumulate_norms), _ptr(grad_sum), int(accumulate_sum), _stream(stream))
        self.check(rc, "adloco_embedding_sqnorm")

    # ------------------------------------------------------------------ outer step
    def outer_step(self, instances, theta_in, mom_in, *, lr, momentum, nesterov=True, theta_out=None,
                   mom_out=None, writeback=None, stream=None):
        """adloco_outer_step; theta_out / mom_out default to in-place."""
        K = len(instances)
        P = theta_in.numel()
        arr = (C.c_void_p * K)(*[t.data_ptr() for t in instances])
        wb = None
        if writeback is not None:
            wb = (C.c_void_p * K)(*[(t.data_ptr() if t is not None else None) for t in writeback])
        theta_out = theta_in if theta_out is None else theta_out
        mom_out = mom_in if mom_out is None else mom_out
        rc = self.lib.adloco_outer_step(self.h, arr, _dtype_code(instances[0].dtype), K, P, _ptr(theta_in),
                                        _ptr(theta_out), _ptr(mom_in), _ptr(mom_out), float(lr), float(momentum),
                                        int(bool(nesterov)), wb, _stream(stream))
        self.check(rc, "adloco_outer_step")
        return theta_out, mom_out

    def outer_step_host(self, instances_host, theta_host, mom_host, *, lr, momentum, nesterov=True, stream=None):
        K = len(instances_host)
        arr = (C.c_void_p * K)(*[t.data_ptr() for t in instances_host])
        rc = self.lib.adloco_outer_step_host(self.h, arr, _dtype_code(instances_host[0].dtype), K,
                                             theta_host.numel(), _ptr(theta_host), _ptr(mom_host), float(lr),
                                             float(momentum), int(bool(nesterov)), _stream(stream))
        self.check(rc, "adloco_outer_step_host")

    # ------------------------------------------------------------------ outer step around an exchange
    def pseudo_gradient(self, theta, instance, out, *, stream=None):
        """adloco_pseudo_gradient: out = theta - instance (fp32 [P])."""
        rc = self.lib.adloco_pseudo_gradient(self.h, _ptr(theta), _ptr(instance), _dtype_code(instance.dtype),
                                             theta.numel(), _ptr(out), _stream(stream))
        self.check(rc, "adloco_pseudo_gradient")

    def outer_apply(self, pseudo_grad_sum, K, theta, mom, *, lr, momentum, nesterov=True, stream=None):
        """adloco_outer_apply, in place on the slices theta and mom."""
        rc = self.lib.adloco_outer_apply(self.h, _ptr(pseudo_grad_sum), int(K), theta.numel(), _ptr(theta), _ptr(theta),
                                         _ptr(mom), _ptr(mom), float(lr), float(momentum), int(bool(nesterov)),
                                         _stream(stream))
        self.check(rc, "adloco_outer_apply")

    def refresh_instance(self, theta, instance, *, stream=None):
        """adloco_refresh_instance: instance = theta rounded to the instance's type."""
        rc = self.lib.adloco_refresh_instance(self.h, _ptr(theta), _ptr(instance), _dtype_code(instance.dtype),
                                              theta.numel(), _stream(stream))
        self.check(rc, "adloco_refresh_instance")

    # ------------------------------------------------------------------ merge
    def merge(self, members, weights, out, *, stream=None) -> int:
        K = len(members)
        arr = (C.c_void_p * K)(*[t.data_ptr() for t in members])
        w = (C.c_int64 * K)(*[int(x) for x in weights])
        rep = C.c_int32(-1)
        rc = self.lib.adloco_merge(self.h, arr, w, _dtype_code(members[0].dtype), K, members[0].numel(),
                                   _ptr(out), C.byref(rep), _stream(stream))
        self.check(rc, "adloco_merge")
        return rep.value


def norm_test_noalloc(G, params: TestParams, result_dev, result_host, *, per_sample_sqnorm=None, stream=None):
    """adloco_norm_test_noalloc on the current device: no context, and nothing
    is allocated by the library.  `result_dev` (device) and `result_host`
    (pinned host) are uint8 tensors of at least sizeof(TestResult) bytes that the
    caller owns.  Returns the TestResult after synchronising the stream."""
    lib = load_library()
    if G.dtype != torch.float32 or G.stride(1) != 1:
        raise AdlocoError(ERR_UNSUPPORTED, "adloco_norm_test_noalloc takes float32 rows with contiguous columns")
    B, P = G.shape
    stride = G.stride(0) if B > 1 else max(G.stride(0), P)
    rc = lib.adloco_norm_test_noalloc(_ptr(G), B, P, stride, C.byref(params), _ptr(per_sample_sqnorm),
                                      _ptr(result_dev), _ptr(result_host), _stream(stream))
    if rc != OK:
        raise AdlocoError(rc, "adloco_norm_test_noalloc: " + lib.adloco_status_string(rc).decode())
    (stream or torch.cuda.current_stream()).synchronize()
    return TestResult.from_buffer_copy(result_host.numpy().tobytes()[:C.sizeof(TestResult)])


def shard_bounds(P: int, rank: int, world: int, align: int = 8):
    """[begin, end) of rank `rank`'s slice when a flat parameter vector of P elements is
    cut into `world` contiguous slices whose starts are multiples of `align` elements
    (8 keeps fp32 and bf16 slices 16-byte aligned).  The slices are disjoint and cover
    [0, P); trailing ranks may get an empty slice when P is small."""
    if not (0 <= rank < world) or P < 0 or align < 1:
        raise ValueError("bad shard request")
    units = -(-P // align)
    lo = min(P, (units * rank // world) * align)
    hi = min(P, (units * (rank + 1) // world) * align)
    return lo, hi


def outer_step_shard(ctx, instances, theta, mom, rank: int, world: int, *, lr, momentum, nesterov=True,
                     writeback=None, stream=None):
    """The outer step on this rank's slice of the parameter vector.  The update is
    elementwise, so when every GPU holds its slice of theta, of the momentum and of all K
    instances, the sharded outer step needs no exchange at all: each rank calls this on its
    own buffers (here: views into full-length tensors).  Returns the slice bounds."""
    lo, hi = shard_bounds(theta.numel(), rank, world)
    if hi > lo:
        wb = None if writeback is None else [None if t is None else t[lo:hi] for t in writeback]
        ctx.outer_step([t[lo:hi] for t in instances], theta[lo:hi], mom[lo:hi], lr=lr, momentum=momentum,
                       nesterov=nesterov, writeback=wb, stream=stream)
    return lo, hi


def TestResult_size() -> int:
    return C.sizeof(TestResult)


def check_merge(b_req, w: int):
    """adloco_check_merge (host only)."""
    lib = load_library()
    k = len(b_req)
    arr = (C.c_int64 * max(k, 1))(*[int(x) for x in b_req])
    out = (C.c_int32 * max(w, 1))()
    n = lib.adloco_check_merge(arr, k, int(w), out)
    if n < 0:
        raise AdlocoError(n, "adloco_check_merge: " + lib.adloco_status_string(n).decode())
    return [out[i] for i in range(n)]


class Accumulator:
    """adloco_accum over caller-owned float32 sum buffers (switch mode)."""

    def __init__(self, ctx: Context, sum_bufs):
        self.ctx = ctx
        self.bufs = list(sum_bufs)
        n = len(self.bufs)
        ptrs = (C.c_void_p * n)(*[t.data_ptr() for t in self.bufs])
        sizes = (C.c_int64 * n)(*[t.numel() for t in self.bufs])
        h = C.c_void_p()
        rc = ctx.lib.adloco_accum_create(ctx.h, C.byref(h), ptrs, sizes, n)
        ctx.check(rc, "adloco_accum_create")
        self.h = h

    def reset(self, stream=None):
        self.ctx.check(self.ctx.lib.adloco_accum_reset(self.ctx.h, self.h, _stream(stream)), "adloco_accum_reset")

    def accumulate(self, G=None, *, per_sample_sqnorm=None, b_micro=None, stream=None):
        if G is not None:
            b, P = G.shape
            stride = G.stride(0) if b > 1 else max(G.stride(0), P)
            rc = self.ctx.lib.adloco_accumulate(self.ctx.h, self.h, _ptr(G), _dtype_code(G.dtype), b, P, stride,
                                                _ptr(per_sample_sqnorm), _stream(stream))
        else:
            b = per_sample_sqnorm.numel() if b_micro is None else int(b_micro)
            rc = self.ctx.lib.adloco_accumulate(self.ctx.h, self.h, None, F32, b, 0, 0,
                                                _ptr(per_sample_sqnorm), _stream(stream))
        self.ctx.check(rc, "adloco_accumulate")

    def finalize(self, params: TestParams, *, stream=None, sync=True):
        c = self.ctx
        rc = c.lib.adloco_accum_finalize(c.h, self.h, C.byref(params), _ptr(c._sums_dev), _ptr(c._res_dev),
                                         _ptr(c._res_host), _stream(stream))
        c.check(rc, "adloco_accum_finalize")
        return c._read_result(stream) if sync else None

    def close(self):
        if getattr(self, "h", None):
            torch.cuda.synchronize(self.ctx.device)
            self.ctx.lib.adloco_accum_destroy(self.h)
            self.h = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
