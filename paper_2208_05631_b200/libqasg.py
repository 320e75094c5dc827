"""ctypes binding of libqasg.so: argument marshalling only.

Every function has the name and the argument order of its C entry point (see
include/qasg.h, which documents meaning, layout and ownership).  Tensors are torch CUDA
tensors; the binding passes their data pointers, sizes and the current CUDA stream.
Nothing here computes: if the shared library is missing or a call fails, an exception
is raised - there is no CPU path.
"""
import ctypes
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "lib", "libqasg.so")

OK = 0
(ERR_INVALID_ARG, ERR_ALIGNMENT, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_NONFINITE, ERR_BAD_CODE,
 ERR_BAD_INDEX) = range(1, 9)
Q_THRESHOLD, Q_TERNARY_STOCH, Q_NONE = 0, 1, 2
RULE_CMD, RULE_RDA = 0, 1
CREATE_NO_CODE_SCRATCH = 1
CREATE_SERIAL_LAUNCHES = 2
OPT_STREAM_ROW_BYTES, OPT_STREAM_LAG, OPT_WAIT_POLLS, OPT_ONE_LAUNCH_STEP_BYTES = 0, 1, 2, 3
LAG_AUTO = 0xFFFFFFFF

# Names every build of the library must export (checked by the CPU tests).
EXPORTS = [
    "qasg_create", "qasg_destroy", "qasg_code_words", "qasg_quantize_pack", "qasg_decode_average",
    "qasg_cmd_step", "qasg_rda_step", "qasg_step", "qasg_step_host", "qasg_logreg_grad_dense",
    "qasg_logreg_grad_csr", "qasg_last_async_status", "qasg_launch_count", "qasg_status_string",
    "qasg_profile_begin", "qasg_profile_end", "qasg_kernel_name", "qasg_quantize_pack_static", "qasg_requantize", "qasg_step_double",
    "qasg_select_quantize_pack", "qasg_indicator_or", "qasg_step_select",
    "qasg_logreg_grad_csr_touched", "qasg_quantize_pack_touched", "qasg_step_touched",
    "qasg_optimal_scratch_bytes", "qasg_quantize_pack_optimal", "qasg_set_option", "qasg_wait_selftest",
]
STATIC_MAX_WORKERS = 16
KERNEL_COUNT = 26


class QasgError(RuntimeError):
    def __init__(self, status, where):
        self.status = int(status)
        super().__init__("%s: %s (status %d)" % (where, status_string(status), status))


class Params(ctypes.Structure):
    _fields_ = [("struct_size", ctypes.c_uint32), ("quantizer", ctypes.c_uint32),
                ("thr_coef", ctypes.c_float), ("lambda_", ctypes.c_float), ("eta", ctypes.c_float),
                ("delta", ctypes.c_float), ("seed", ctypes.c_uint64)]


def make_params(lam=1e-3, eta=0.1, delta=1e-8, quantizer=Q_THRESHOLD, thr_coef=0.75, seed=0):
    return Params(ctypes.sizeof(Params), int(quantizer), float(thr_coef), float(lam), float(eta),
                  float(delta), int(seed))


_lib = None


def load():
    """Loads libqasg.so (once).  Raises if it has not been built."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError("libqasg.so is missing: build it with `python -m paper_2208_05631_b200.build`")
    lib = ctypes.CDLL(LIB_PATH)
    vp, u64, u32, i32 = ctypes.c_void_p, ctypes.c_uint64, ctypes.c_uint32, ctypes.c_int
    pp = ctypes.POINTER(Params)
    lib.qasg_create.argtypes = [ctypes.POINTER(vp), i32, u64, u32, u32]
    lib.qasg_destroy.argtypes = [vp]
    lib.qasg_code_words.argtypes = [u64]
    lib.qasg_code_words.restype = u64
    lib.qasg_quantize_pack.argtypes = [vp, vp, u64, u64, u32, u64, pp, vp, vp, vp, vp, vp]
    lib.qasg_decode_average.argtypes = [vp, vp, vp, u64, u32, vp, vp]
    lib.qasg_cmd_step.argtypes = [vp, vp, vp, vp, u64, u64, pp, vp]
    lib.qasg_rda_step.argtypes = [vp, vp, vp, vp, vp, u64, u64, pp, vp]
    lib.qasg_step.argtypes = [vp, i32, vp, u64, u64, u32, u64, pp, vp, vp, vp, vp, vp, vp]
    lib.qasg_requantize.argtypes = [vp, vp, vp, u64, u32, u64, pp, vp, vp, vp, vp, vp]
    lib.qasg_step_double.argtypes = [vp, i32, vp, u64, u64, u32, u64, pp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.qasg_select_quantize_pack.argtypes = [vp, i32, vp, u64, u64, u32, u64, pp, vp, vp, vp, vp, vp, vp, vp, vp,
                                              vp, vp]
    lib.qasg_indicator_or.argtypes = [vp, vp, u64, u32, vp, vp, vp]
    lib.qasg_step_select.argtypes = [vp, i32, i32, vp, u64, u64, u32, u64, pp, vp, vp, vp, vp, vp, vp, vp, vp, vp,
                                     vp]
    lib.qasg_step_host.argtypes = [vp, i32, vp, u64, u64, u32, u64, pp, vp, vp, vp, vp, vp, vp, vp, vp]
    lib.qasg_logreg_grad_dense.argtypes = [vp, vp, vp, u64, u64, u32, ctypes.POINTER(u64), vp, u32, u64,
                                           vp, vp, u64, vp]
    lib.qasg_logreg_grad_csr.argtypes = [vp, vp, vp, vp, vp, u64, u64, u32, ctypes.POINTER(u64), vp, u32,
                                         u64, vp, vp, u64, vp]
    lib.qasg_logreg_grad_csr_touched.argtypes = [vp, vp, vp, vp, vp, u64, u64, u32, ctypes.POINTER(u64), vp, u32,
                                                 u64, vp, vp, u64, vp, vp]
    lib.qasg_quantize_pack_touched.argtypes = [vp, vp, u64, u64, u32, u64, pp, vp, vp, vp, vp, vp, vp]
    lib.qasg_step_touched.argtypes = [vp, i32, vp, u64, u64, u32, u64, pp, vp, vp, vp, vp, vp, vp, vp]
    lib.qasg_optimal_scratch_bytes.argtypes = [u64]
    lib.qasg_optimal_scratch_bytes.restype = u64
    lib.qasg_quantize_pack_optimal.argtypes = [vp, vp, u64, u64, u32, pp, vp, vp, vp, vp, vp, u64, vp]
    lib.qasg_set_option.argtypes = [vp, i32, u64]
    lib.qasg_wait_selftest.argtypes = [vp, u32, vp]
    lib.qasg_last_async_status.argtypes = [vp, vp]
    lib.qasg_launch_count.argtypes = [vp]
    lib.qasg_launch_count.restype = u64
    lib.qasg_profile_begin.argtypes = [vp]
    lib.qasg_profile_end.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(u64)]
    lib.qasg_kernel_name.argtypes = [i32]
    lib.qasg_kernel_name.restype = ctypes.c_char_p
    lib.qasg_quantize_pack_static.argtypes = [i32, vp, u64, u64, u32, ctypes.c_float, vp, vp, vp, vp, vp]
    lib.qasg_status_string.argtypes = [i32]
    lib.qasg_status_string.restype = ctypes.c_char_p
    _lib = lib
    return lib


def status_string(status):
    return load().qasg_status_string(int(status)).decode()


def _check(status, where):
    if status != OK:
        raise QasgError(status, where)


def _ptr(t):
    if t is None:
        return None
    if isinstance(t, int):
        return t
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        return torch.cuda.current_stream().cuda_stream
    return stream if isinstance(stream, int) else stream.cuda_stream


def _shards(shard_row0):
    arr = (ctypes.c_uint64 * len(shard_row0))(*[int(v) for v in shard_row0])
    return arr


class Context:
    """Owns one qasg_ctx.  Methods mirror the C entry points."""

    def __init__(self, d_max, M_max, device=0, flags=0):
        self._h = ctypes.c_void_p()
        self.device = int(device)
        _check(load().qasg_create(ctypes.byref(self._h), self.device, int(d_max), int(M_max), int(flags)),
               "qasg_create")

    def close(self):
        if self._h:
            load().qasg_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def quantize_pack(self, g, d, ld_g, M, t, params, codes, scales, thresholds=None, counts=None,
                      stream=None):
        _check(load().qasg_quantize_pack(self._h, _ptr(g), d, ld_g, M, t, ctypes.byref(params), _ptr(codes),
                                         _ptr(scales), _ptr(thresholds), _ptr(counts), _stream(stream)),
               "qasg_quantize_pack")

    def decode_average(self, codes, scales, d, M, gbar, stream=None):
        _check(load().qasg_decode_average(self._h, _ptr(codes), _ptr(scales), d, M, _ptr(gbar),
                                          _stream(stream)), "qasg_decode_average")

    def cmd_step(self, q, x, h, d, t, params, stream=None):
        _check(load().qasg_cmd_step(self._h, _ptr(q), _ptr(x), _ptr(h), d, t, ctypes.byref(params),
                                    _stream(stream)), "qasg_cmd_step")

    def rda_step(self, q, x, h, z, d, t, params, stream=None):
        _check(load().qasg_rda_step(self._h, _ptr(q), _ptr(x), _ptr(h), _ptr(z), d, t, ctypes.byref(params),
                                    _stream(stream)), "qasg_rda_step")

    def step(self, rule, g, d, ld_g, M, t, params, x, h, z=None, codes_out=None, scales_out=None,
             stream=None):
        _check(load().qasg_step(self._h, rule, _ptr(g), d, ld_g, M, t, ctypes.byref(params), _ptr(x), _ptr(h),
                                _ptr(z), _ptr(codes_out), _ptr(scales_out), _stream(stream)), "qasg_step")

    def requantize(self, codes, scales, d, M, t, params, qcodes, qscale, qthreshold=None, qcount=None,
                   stream=None):
        _check(load().qasg_requantize(self._h, _ptr(codes), _ptr(scales), d, M, t, ctypes.byref(params),
                                      _ptr(qcodes), _ptr(qscale), _ptr(qthreshold), _ptr(qcount),
                                      _stream(stream)), "qasg_requantize")

    def step_double(self, rule, g, d, ld_g, M, t, params, x, h, z=None, codes_out=None, scales_out=None,
                    qcodes_out=None, qscale_out=None, stream=None):
        _check(load().qasg_step_double(self._h, rule, _ptr(g), d, ld_g, M, t, ctypes.byref(params), _ptr(x),
                                       _ptr(h), _ptr(z), _ptr(codes_out), _ptr(scales_out), _ptr(qcodes_out),
                                       _ptr(qscale_out), _stream(stream)), "qasg_step_double")

    def select_quantize_pack(self, rule, g, d, ld_g, M, t, params, x, h, z, codes, scales, thresholds=None,
                             counts=None, indicators=None, selected=None, stream=None):
        _check(load().qasg_select_quantize_pack(self._h, rule, _ptr(g), d, ld_g, M, t, ctypes.byref(params),
                                                _ptr(x), _ptr(h), _ptr(z), _ptr(codes), _ptr(scales),
                                                _ptr(thresholds), _ptr(counts), _ptr(indicators), _ptr(selected),
                                                _stream(stream)), "qasg_select_quantize_pack")

    def indicator_or(self, indicators, d, M, isyn, ksyn, stream=None):
        _check(load().qasg_indicator_or(self._h, _ptr(indicators), d, M, _ptr(isyn), _ptr(ksyn), _stream(stream)),
               "qasg_indicator_or")

    def step_select(self, rule, double_quant, g, d, ld_g, M, t, params, x, h, z=None, codes_out=None,
                    scales_out=None, indicators_out=None, selected_out=None, isyn_out=None, ksyn_out=None,
                    stream=None):
        _check(load().qasg_step_select(self._h, rule, int(bool(double_quant)), _ptr(g), d, ld_g, M, t,
                                       ctypes.byref(params), _ptr(x), _ptr(h), _ptr(z), _ptr(codes_out),
                                       _ptr(scales_out), _ptr(indicators_out), _ptr(selected_out), _ptr(isyn_out),
                                       _ptr(ksyn_out), _stream(stream)), "qasg_step_select")

    def step_host(self, rule, g_host, d, ld_g, M, t, params, x_host, h_host, z_host, g_dev, x_dev, h_dev,
                  z_dev, stream=None):
        _check(load().qasg_step_host(self._h, rule, _ptr(g_host), d, ld_g, M, t, ctypes.byref(params),
                                     _ptr(x_host), _ptr(h_host), _ptr(z_host), _ptr(g_dev), _ptr(x_dev),
                                     _ptr(h_dev), _ptr(z_dev), _stream(stream)), "qasg_step_host")

    def logreg_grad_dense(self, X, y, n_rows, d, M, shard_row0, batch_rows, B, t, x, g, ld_g, stream=None):
        _check(load().qasg_logreg_grad_dense(self._h, _ptr(X), _ptr(y), n_rows, d, M, _shards(shard_row0),
                                             _ptr(batch_rows), B, t, _ptr(x), _ptr(g), ld_g,
                                             _stream(stream)), "qasg_logreg_grad_dense")

    def logreg_grad_csr(self, rowptr, colidx, vals, y, n_rows, d, M, shard_row0, batch_rows, B, t, x, g,
                        ld_g, stream=None):
        _check(load().qasg_logreg_grad_csr(self._h, _ptr(rowptr), _ptr(colidx), _ptr(vals), _ptr(y), n_rows,
                                           d, M, _shards(shard_row0), _ptr(batch_rows), B, t, _ptr(x),
                                           _ptr(g), ld_g, _stream(stream)), "qasg_logreg_grad_csr")

    def logreg_grad_csr_touched(self, rowptr, colidx, vals, y, n_rows, d, M, shard_row0, batch_rows, B, t, x, g,
                                ld_g, touched, stream=None):
        _check(load().qasg_logreg_grad_csr_touched(self._h, _ptr(rowptr), _ptr(colidx), _ptr(vals), _ptr(y),
                                                   n_rows, d, M, _shards(shard_row0), _ptr(batch_rows), B, t,
                                                   _ptr(x), _ptr(g), ld_g, _ptr(touched), _stream(stream)),
               "qasg_logreg_grad_csr_touched")

    def quantize_pack_touched(self, g, d, ld_g, M, t, params, touched, codes, scales, thresholds=None,
                              counts=None, stream=None):
        _check(load().qasg_quantize_pack_touched(self._h, _ptr(g), d, ld_g, M, t, ctypes.byref(params),
                                                 _ptr(touched), _ptr(codes), _ptr(scales), _ptr(thresholds),
                                                 _ptr(counts), _stream(stream)), "qasg_quantize_pack_touched")

    def step_touched(self, rule, g, d, ld_g, M, t, params, touched, x, h, z=None, codes_out=None,
                     scales_out=None, stream=None):
        _check(load().qasg_step_touched(self._h, rule, _ptr(g), d, ld_g, M, t, ctypes.byref(params),
                                        _ptr(touched), _ptr(x), _ptr(h), _ptr(z), _ptr(codes_out),
                                        _ptr(scales_out), _stream(stream)), "qasg_step_touched")

    def quantize_pack_optimal(self, g, d, ld_g, M, params, codes, scales, scratch, thresholds=None, counts=None,
                              stream=None):
        """scratch: a device tensor of at least optimal_scratch_bytes(d) bytes."""
        _check(load().qasg_quantize_pack_optimal(self._h, _ptr(g), d, ld_g, M, ctypes.byref(params), _ptr(codes),
                                                 _ptr(scales), _ptr(thresholds), _ptr(counts), _ptr(scratch),
                                                 scratch.numel() * scratch.element_size(), _stream(stream)),
               "qasg_quantize_pack_optimal")

    def set_option(self, option, value):
        _check(load().qasg_set_option(self._h, int(option), int(value)), "qasg_set_option")

    def wait_selftest(self, max_polls, stream=None):
        _check(load().qasg_wait_selftest(self._h, int(max_polls), _stream(stream)), "qasg_wait_selftest")

    def last_async_status(self, stream=None):
        return int(load().qasg_last_async_status(self._h, _stream(stream)))

    def profile_begin(self):
        _check(load().qasg_profile_begin(self._h), "qasg_profile_begin")

    def profile_end(self):
        """Returns {kernel name: (total ms, launches)} for the kernels launched since profile_begin."""
        ms = (ctypes.c_double * KERNEL_COUNT)()
        n = (ctypes.c_uint64 * KERNEL_COUNT)()
        _check(load().qasg_profile_end(self._h, ms, n), "qasg_profile_end")
        return {load().qasg_kernel_name(k).decode(): (float(ms[k]), int(n[k]))
                for k in range(KERNEL_COUNT) if n[k]}

    def launch_count(self):
        return int(load().qasg_launch_count(self._h))


def optimal_scratch_bytes(d):
    return int(load().qasg_optimal_scratch_bytes(d))


def quantize_pack_static(device, g, d, ld_g, M, thr_coef, codes, scales, thresholds=None, counts=None,
                          stream=None):
    """qasg_quantize_pack_static: the threshold quantizer without a context and without any
    allocation (the scratch is a fixed array inside the library; at most STATIC_MAX_WORKERS
    workers; calls that overlap on the GPU race on it)."""
    _check(load().qasg_quantize_pack_static(int(device), _ptr(g), d, ld_g, M, float(thr_coef), _ptr(codes),
                                            _ptr(scales), _ptr(thresholds), _ptr(counts), _stream(stream)),
           "qasg_quantize_pack_static")


def code_words(d):
    return int(load().qasg_code_words(int(d)))
