"""Thin ctypes binding of the C ABI in ``include/wfq.h`` (argument marshalling only).

Every step of the computation runs in the CUDA kernels of ``libwfq.so``.  PyTorch is
used by callers for device memory and streams; this module only passes raw pointers.
If the library has not been built the import-time loader raises: there is no
fallback path.
"""
import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libwfq.so")

WFQ_OK, WFQ_ERR_INVALID_ARG, WFQ_ERR_UNSUPPORTED, WFQ_ERR_ALLOC = 0, 1, 2, 3
WFQ_ERR_NOT_PREPARED, WFQ_ERR_CUDA, WFQ_ERR_TIMEOUT, WFQ_ERR_SCRATCH_TOO_SMALL = 4, 5, 6, 7
WFQ_STATIC_SCRATCH_FLOATS = 4 * 1024 * 1024
WFQ_F32, WFQ_F16, WFQ_BF16 = 0, 1, 2
WFQ_ACT_NONE, WFQ_ACT_RELU, WFQ_ACT_SILU = 0, 1, 2
WFQ_Y_FP32, WFQ_Y_TILE, WFQ_Y_ROW = 0, 1, 2
WFQ_NCHW, WFQ_NHWC = 0, 1
WFQ_BUF_XQ, WFQ_BUF_SX, WFQ_BUF_WQ, WFQ_BUF_SW, WFQ_BUF_Y, WFQ_BUF_STATUS = range(6)
WFQ_DEBUG_WAIT_CYCLES, WFQ_DEBUG_SKIP_INPUT_ITEM, WFQ_DEBUG_INPUT_TRANSFORM_KERNEL = range(3)
WFQ_DEBUG_SKIP_GEMM_STAGE = 3
WFQ_DEBUG_GEMM_SHAPE = 4

# every symbol include/wfq.h declares
EXPORTS = [
    "wfq_plan_create", "wfq_plan_set_input_dtype", "wfq_plan_workspace_bytes",
    "wfq_plan_set_workspace", "wfq_prepare_filters", "wfq_conv_forward",
    "wfq_conv_forward_host", "wfq_input_transform_quantize", "wfq_gemm_dequantize",
    "wfq_output_transform", "wfq_debug_gemm_acc32", "wfq_debug_get",
    "wfq_check_device_status", "wfq_plan_destroy", "wfq_status_string", "wfq_version",
    "wfq_quantize_filters_static", "wfq_plan_set_debug_option", "wfq_debug_int8_mma_rate",
    "wfq_plan_set_epilogue", "wfq_plan_set_full_quant", "wfq_plan_set_output_dtype", "wfq_plan_set_weight_bits",
    "wfq_conv_forward_host_async", "wfq_filters_bytes", "wfq_filters_export", "wfq_filters_import",
    "wfq_plan_set_input_layout",
]

_lib = None


class WfqError(RuntimeError):
    def __init__(self, status, what):
        self.status = status
        super().__init__(f"{what}: {status_string(status)} ({status})")


def load():
    """Load libwfq.so and declare the prototypes.  Raises if the library is missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} is missing: build it with "
                           "`python -m paper_2412_19867_b200.build` (no CPU fallback exists)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    lib.wfq_plan_create.argtypes = [ctypes.POINTER(vp)] + [ci] * 9
    lib.wfq_plan_set_input_dtype.argtypes = [vp, ci]
    lib.wfq_plan_workspace_bytes.argtypes = [vp]
    lib.wfq_plan_workspace_bytes.restype = sz
    lib.wfq_plan_set_workspace.argtypes = [vp, vp, sz]
    lib.wfq_prepare_filters.argtypes = [vp, vp, vp, vp, vp, vp]
    lib.wfq_conv_forward.argtypes = [vp, vp, vp, vp]
    lib.wfq_conv_forward_host.argtypes = [vp, vp, vp, vp]
    lib.wfq_conv_forward_host_async.argtypes = [vp, vp, vp, vp]
    lib.wfq_filters_bytes.argtypes = [vp]
    lib.wfq_filters_bytes.restype = ctypes.c_size_t
    lib.wfq_filters_export.argtypes = [vp, vp, ctypes.c_size_t, vp]
    lib.wfq_filters_import.argtypes = [vp, vp, ctypes.c_size_t, vp]
    lib.wfq_input_transform_quantize.argtypes = [vp, vp, vp]
    lib.wfq_gemm_dequantize.argtypes = [vp, vp]
    lib.wfq_output_transform.argtypes = [vp, vp, vp]
    lib.wfq_debug_gemm_acc32.argtypes = [vp, vp, vp]
    lib.wfq_debug_get.argtypes = [vp, ci, ctypes.POINTER(vp), ctypes.POINTER(sz)]
    lib.wfq_check_device_status.argtypes = [vp, vp, ctypes.POINTER(ci)]
    lib.wfq_plan_destroy.argtypes = [vp]
    lib.wfq_quantize_filters_static.argtypes = [vp, ci, ci, ci, ci, vp, vp, vp, vp]
    lib.wfq_plan_set_epilogue.argtypes = [vp, vp, ci]
    lib.wfq_plan_set_full_quant.argtypes = [vp, ci, ci]
    lib.wfq_plan_set_output_dtype.argtypes = [vp, ci]
    lib.wfq_plan_set_weight_bits.argtypes = [vp, ci]
    lib.wfq_plan_set_input_layout.argtypes = [vp, ci]
    lib.wfq_plan_set_debug_option.argtypes = [vp, ci, ctypes.c_longlong]
    lib.wfq_debug_int8_mma_rate.argtypes = [vp, ci, ci, ctypes.POINTER(ctypes.c_longlong), vp]
    lib.wfq_status_string.argtypes = [ci]
    lib.wfq_status_string.restype = ctypes.c_char_p
    lib.wfq_version.restype = ci
    for name in EXPORTS:
        fn = getattr(lib, name)
        if fn.restype is ctypes.c_int and name not in ("wfq_version",):
            fn.restype = ci
    _lib = lib
    return lib


def status_string(status):
    return load().wfq_status_string(int(status)).decode()


def _check(status, what):
    if status != WFQ_OK:
        raise WfqError(status, what)


def _host_floats(values):
    if values is None:
        return None, None
    arr = (ctypes.c_float * len(values))(*[float(v) for v in values])
    return arr, ctypes.cast(arr, ctypes.c_void_p)


# ---- the C calls, same names, raw pointers (ints) in and out ------------------------

def wfq_plan_create(N, C, K, H, W, m, r=3, group_size=64, bits=8):
    plan = ctypes.c_void_p()
    _check(load().wfq_plan_create(ctypes.byref(plan), N, C, K, H, W, m, r, group_size, bits),
           "wfq_plan_create")
    return plan


def wfq_plan_set_input_dtype(plan, dtype):
    _check(load().wfq_plan_set_input_dtype(plan, dtype), "wfq_plan_set_input_dtype")


def wfq_plan_set_epilogue(plan, bias_dev, act=WFQ_ACT_NONE):
    _check(load().wfq_plan_set_epilogue(plan, bias_dev, act), "wfq_plan_set_epilogue")


def wfq_plan_set_input_layout(plan, layout):
    _check(load().wfq_plan_set_input_layout(plan, layout), "wfq_plan_set_input_layout")


def wfq_plan_set_weight_bits(plan, bits):
    _check(load().wfq_plan_set_weight_bits(plan, bits), "wfq_plan_set_weight_bits")


def wfq_plan_set_output_dtype(plan, dtype):
    _check(load().wfq_plan_set_output_dtype(plan, dtype), "wfq_plan_set_output_dtype")


def wfq_plan_set_full_quant(plan, quant_input, y_mode):
    _check(load().wfq_plan_set_full_quant(plan, int(quant_input), y_mode), "wfq_plan_set_full_quant")


def wfq_plan_workspace_bytes(plan):
    return int(load().wfq_plan_workspace_bytes(plan))


def wfq_plan_set_workspace(plan, dev_ptr, nbytes):
    _check(load().wfq_plan_set_workspace(plan, dev_ptr, nbytes), "wfq_plan_set_workspace")


def wfq_prepare_filters(plan, w_dev, sB=None, sG=None, sA=None, stream=0):
    kb, pb = _host_floats(sB)
    kg, pg = _host_floats(sG)
    ka, pa = _host_floats(sA)
    _check(load().wfq_prepare_filters(plan, w_dev, pb, pg, pa, stream), "wfq_prepare_filters")


def wfq_conv_forward(plan, x_dev, y_dev, stream=0):
    _check(load().wfq_conv_forward(plan, x_dev, y_dev, stream), "wfq_conv_forward")


def wfq_conv_forward_host(plan, x_host, y_host, stream=0):
    _check(load().wfq_conv_forward_host(plan, x_host, y_host, stream), "wfq_conv_forward_host")


def wfq_filters_bytes(plan):
    return int(load().wfq_filters_bytes(plan))


def wfq_filters_export(plan, stream=0):
    """The prepared filters of the plan as a bytes-like host buffer (ctypes array)."""
    n = wfq_filters_bytes(plan)
    buf = (ctypes.c_char * n)()
    _check(load().wfq_filters_export(plan, ctypes.cast(buf, ctypes.c_void_p), n, stream), "wfq_filters_export")
    return buf


def wfq_filters_import(plan, blob, stream=0):
    raw = bytes(blob)
    _check(load().wfq_filters_import(plan, ctypes.cast(ctypes.c_char_p(raw), ctypes.c_void_p), len(raw), stream),
           "wfq_filters_import")


def wfq_conv_forward_host_async(plan, x_host, y_host, stream=0):
    _check(load().wfq_conv_forward_host_async(plan, x_host, y_host, stream), "wfq_conv_forward_host_async")


def wfq_input_transform_quantize(plan, x_dev, stream=0):
    _check(load().wfq_input_transform_quantize(plan, x_dev, stream), "wfq_input_transform_quantize")


def wfq_gemm_dequantize(plan, stream=0):
    _check(load().wfq_gemm_dequantize(plan, stream), "wfq_gemm_dequantize")


def wfq_output_transform(plan, y_dev, stream=0):
    _check(load().wfq_output_transform(plan, y_dev, stream), "wfq_output_transform")


def wfq_debug_gemm_acc32(plan, acc_dev, stream=0):
    _check(load().wfq_debug_gemm_acc32(plan, acc_dev, stream), "wfq_debug_gemm_acc32")


def wfq_debug_get(plan, which):
    ptr, nbytes = ctypes.c_void_p(), ctypes.c_size_t()
    _check(load().wfq_debug_get(plan, which, ctypes.byref(ptr), ctypes.byref(nbytes)), "wfq_debug_get")
    return ptr.value, nbytes.value


def wfq_check_device_status(plan, stream=0):
    where = ctypes.c_int(0)
    st = load().wfq_check_device_status(plan, stream, ctypes.byref(where))
    return st, where.value


def wfq_quantize_filters_static(w_dev, K, C, m, group_size, sG, wq_dev, sw_dev, stream=0):
    """Allocation-free filter quantization into caller-owned device buffers."""
    keep, pg = _host_floats(sG)
    _check(load().wfq_quantize_filters_static(w_dev, K, C, m, group_size, pg, wq_dev, sw_dev, stream),
           "wfq_quantize_filters_static")


def wfq_plan_set_debug_option(plan, option, value):
    _check(load().wfq_plan_set_debug_option(plan, option, value), "wfq_plan_set_debug_option")


def wfq_debug_int8_mma_rate(plan, n_cols, mmas_per_sm, stream=0):
    """Enqueues the tensor-pipe rate kernel; returns the integer operations it performs."""
    ops = ctypes.c_longlong(0)
    _check(load().wfq_debug_int8_mma_rate(plan, n_cols, mmas_per_sm, ctypes.byref(ops), stream),
           "wfq_debug_int8_mma_rate")
    return ops.value


def wfq_plan_destroy(plan):
    _check(load().wfq_plan_destroy(plan), "wfq_plan_destroy")


# ---- convenience wrapper holding torch tensors for the device buffers ----------------

class _DevicePointer:
    """Exposes a raw device pointer through __cuda_array_interface__ (no copy)."""

    def __init__(self, ptr, shape, typestr):
        self.__cuda_array_interface__ = {"shape": tuple(shape), "typestr": typestr,
                                         "data": (int(ptr), False), "version": 2}


class Conv:
    """One layer: plan + workspace + prepared filters, driven with torch CUDA tensors."""

    def __init__(self, N, C, K, H, W, m, group_size, in_dtype="f16", device="cuda:0"):
        import torch
        self.torch = torch
        self.shape = (N, C, K, H, W)
        self.m, self.gs = m, group_size
        self.device = torch.device(device)
        self.in_dtype = in_dtype
        self.plan = wfq_plan_create(N, C, K, H, W, m, 3, group_size, 8)
        wfq_plan_set_input_dtype(self.plan, WFQ_F16 if in_dtype == "f16" else WFQ_F32)
        nbytes = wfq_plan_workspace_bytes(self.plan)
        # torch's caching allocator returns 512-byte aligned blocks; over-allocate and
        # round the base up to the 1024-byte alignment the TMA tiles want
        self._ws = torch.empty(nbytes + 1024, dtype=torch.uint8, device=self.device)
        base = (self._ws.data_ptr() + 1023) // 1024 * 1024
        with torch.cuda.device(self.device):
            wfq_plan_set_workspace(self.plan, base, nbytes)
        n = m + 2
        self.P, self.G = n * n, C // group_size
        self.T = N * (-(-H // m)) * (-(-W // m))
        self.Tp = (self.T + 31) // 32 * 32
        self.Ts = (self.T + 127) // 128 * 128
        self.Kp = (K + 127) // 128 * 128

    def _stream(self):
        return self.torch.cuda.current_stream(self.device).cuda_stream

    def prepare(self, w, sB=None, sG=None, sA=None):
        torch = self.torch
        assert w.is_cuda and w.dtype == torch.float32 and w.is_contiguous()
        with torch.cuda.device(self.device):
            wfq_prepare_filters(self.plan, w.data_ptr(), sB, sG, sA, self._stream())

    def set_input_layout(self, layout):
        """"nchw" (default) or "nhwc": forward() then takes x of shape (N, H, W, C)."""
        self.in_layout = layout
        wfq_plan_set_input_layout(self.plan, WFQ_NHWC if layout == "nhwc" else WFQ_NCHW)

    def set_weight_bits(self, bits):
        """8 (default) or 4; call before prepare()."""
        wfq_plan_set_weight_bits(self.plan, bits)

    def set_output_dtype(self, dtype):
        """"f32" (default), "f16" or "bf16": element type of the tensors forward() returns or fills."""
        self.out_dtype = dtype
        wfq_plan_set_output_dtype(self.plan, {"f32": WFQ_F32, "f16": WFQ_F16, "bf16": WFQ_BF16}[dtype])

    def set_epilogue(self, bias=None, act=WFQ_ACT_NONE):
        """bias: fp32 CUDA tensor [K] or None; kept alive by this object."""
        if bias is not None:
            assert bias.is_cuda and bias.dtype == self.torch.float32 and bias.is_contiguous()
            assert bias.numel() == self.shape[2]
        self._bias = bias
        wfq_plan_set_epilogue(self.plan, None if bias is None else bias.data_ptr(), act)

    def forward(self, x, y=None):
        torch = self.torch
        N, C, K, H, W = self.shape
        xs = (N, H, W, C) if getattr(self, "in_layout", "nchw") == "nhwc" else (N, C, H, W)
        assert x.is_cuda and x.is_contiguous() and tuple(x.shape) == xs
        assert x.dtype == (torch.float16 if self.in_dtype == "f16" else torch.float32)
        ydt = {"f32": torch.float32, "f16": torch.float16, "bf16": torch.bfloat16}[getattr(self, "out_dtype", "f32")]
        if y is None:
            y = torch.empty((N, K, H, W), dtype=ydt, device=self.device)
        assert y.dtype == ydt and y.is_contiguous() and tuple(y.shape) == (N, K, H, W)
        with torch.cuda.device(self.device):
            wfq_conv_forward(self.plan, x.data_ptr(), y.data_ptr(), self._stream())
        return y

    def forward_host(self, x_host, y_host):
        """x_host / y_host: CPU tensors (pinned for speed); synchronous."""
        with self.torch.cuda.device(self.device):
            wfq_conv_forward_host(self.plan, x_host.data_ptr(), y_host.data_ptr(), self._stream())
        return y_host

    def forward_host_async(self, x_host, y_host, stream=None):
        """The same without the final wait; `stream`: a torch.cuda.Stream (default: the current
        one).  y_host is valid after that stream has been synchronised."""
        sptr = self._stream() if stream is None else stream.cuda_stream
        with self.torch.cuda.device(self.device):
            wfq_conv_forward_host_async(self.plan, x_host.data_ptr(), y_host.data_ptr(), sptr)
        return y_host

    def buffer(self, which):
        """A torch tensor aliasing an internal buffer, shaped per include/wfq.h."""
        torch = self.torch
        ptr, nbytes = wfq_debug_get(self.plan, which)
        N, C, K, H, W = self.shape
        shapes = {WFQ_BUF_XQ: ((self.P, self.T, C), "|i1", 1),
                  WFQ_BUF_SX: ((self.P, self.G, self.Ts), "<f4", 4),
                  WFQ_BUF_WQ: ((self.P, K, C), "|i1", 1),
                  WFQ_BUF_SW: ((self.P, self.G, self.Kp), "<f4", 4),
                  WFQ_BUF_Y: ((self.P, K, self.Tp), "<f4", 4),
                  WFQ_BUF_STATUS: ((4,), "<i4", 4)}
        shape, typestr, esz = shapes[which]
        count = 1
        for d in shape:
            count *= d
        assert count * esz == nbytes, (which, shape, nbytes)
        holder = _DevicePointer(ptr, shape, typestr)
        with torch.cuda.device(self.device):
            return torch.as_tensor(holder, device=self.device)

    def write_buffer(self, which, tensor):
        """Overwrite an internal buffer (feeding a later stage with chosen operands)."""
        dst = self.buffer(which)
        dst.copy_(tensor.to(self.device).reshape(dst.shape))
        self.torch.cuda.synchronize(self.device)

    def check_status(self):
        st, where = wfq_check_device_status(self.plan, self._stream())
        if st != WFQ_OK:
            raise WfqError(st, f"device status (wait id {where})")

    def close(self):
        if self.plan is not None:
            wfq_plan_destroy(self.plan)
            self.plan = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass
