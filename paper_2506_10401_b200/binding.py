"""ctypes binding of libhct.so: argument marshalling only, same names as include/hct.h."""
from __future__ import annotations

import ctypes
import os

PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(PKG, "libhct.so")

HCT_OK = 0
HCT_ERR_INVALID_ARG, HCT_ERR_PARSE, HCT_ERR_GRAPH, HCT_ERR_UNSUPPORTED, HCT_ERR_COMPILE = 1, 2, 3, 4, 5
HCT_ERR_CUDA, HCT_ERR_TIMEOUT, HCT_ERR_ARCH, HCT_ERR_OOM = 6, 7, 8, 9
HCT_F32, HCT_BF16 = 0, 1
HCT_DEVICE_NONE = -1

EXPORTS = [
    "hct_graph_create", "hct_graph_run", "hct_graph_status", "hct_graph_destroy", "hct_graph_num_inputs",
    "hct_graph_num_outputs", "hct_graph_tensor_info", "hct_graph_workspace_bytes", "hct_graph_num_kernels",
    "hct_graph_cost", "hct_graph_plan_text", "hct_graph_kernel_source", "hct_graph_kernel_name", "hct_last_error",
    "hct_version", "hct_gemm_bias_relu_f32_static", "hct_graph_create_scheduled", "hct_graph_autotune", "hct_graph_schedule",
    "hct_graph_input_layout",
    "hct_graph_output_layout",
]

HCT_STATIC_SCRATCH_BYTES = 8 << 20


class HctError(RuntimeError):
    def __init__(self, code: int, message: str):
        super().__init__(f"hct error {code}: {message}")
        self.code = code
        self.message = message


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library.  Fails loudly when it has not been built: there is no other execution path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing; run `python -m paper_2506_10401_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        vp, cp, ci, sz = ctypes.c_void_p, ctypes.c_char_p, ctypes.c_int, ctypes.c_size_t
        L.hct_graph_create.argtypes = [cp, sz, ci, ctypes.POINTER(vp)]
        L.hct_graph_create.restype = ci
        L.hct_graph_run.argtypes = [vp, ctypes.POINTER(vp), ci, ctypes.POINTER(vp), ci, vp, sz, vp]
        L.hct_graph_run.restype = ci
        L.hct_graph_status.argtypes = [vp]
        L.hct_graph_status.restype = ci
        L.hct_graph_destroy.argtypes = [vp]
        L.hct_graph_destroy.restype = ci
        L.hct_graph_num_inputs.argtypes = [vp]
        L.hct_graph_num_inputs.restype = ci
        L.hct_graph_num_outputs.argtypes = [vp]
        L.hct_graph_num_outputs.restype = ci
        L.hct_graph_tensor_info.argtypes = [vp, ci, ci, ctypes.POINTER(cp), ctypes.POINTER(ci), ctypes.POINTER(ci),
                                            ctypes.POINTER(ctypes.c_int64)]
        L.hct_graph_tensor_info.restype = ci
        L.hct_graph_workspace_bytes.argtypes = [vp]
        L.hct_graph_workspace_bytes.restype = sz
        L.hct_graph_input_layout.argtypes = [vp, ci]
        L.hct_graph_input_layout.restype = ci
        L.hct_graph_output_layout.argtypes = [vp, ci]
        L.hct_graph_output_layout.restype = ci
        L.hct_graph_num_kernels.argtypes = [vp]
        L.hct_graph_num_kernels.restype = ci
        L.hct_graph_cost.argtypes = [vp, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_double)]
        L.hct_graph_cost.restype = ci
        L.hct_graph_plan_text.argtypes = [vp]
        L.hct_graph_plan_text.restype = cp
        L.hct_graph_kernel_source.argtypes = [vp, ci]
        L.hct_graph_kernel_source.restype = cp
        L.hct_graph_kernel_name.argtypes = [vp, ci]
        L.hct_graph_kernel_name.restype = cp
        L.hct_last_error.argtypes = []
        L.hct_last_error.restype = cp
        L.hct_gemm_bias_relu_f32_static.argtypes = [vp, vp, vp, vp, ctypes.c_int64, ctypes.c_int64, ctypes.c_int64, ci, ci, vp]
        L.hct_gemm_bias_relu_f32_static.restype = ci
        L.hct_version.argtypes = []
        L.hct_version.restype = cp
        L.hct_graph_create_scheduled.argtypes = [cp, sz, ci, cp, ctypes.POINTER(vp)]
        L.hct_graph_create_scheduled.restype = ci
        L.hct_graph_autotune.argtypes = [cp, sz, ci, ctypes.POINTER(vp), ci, ctypes.POINTER(vp), ci, vp, sz, vp, ci, ctypes.POINTER(vp)]
        L.hct_graph_autotune.restype = ci
        L.hct_graph_schedule.argtypes = [vp]
        L.hct_graph_schedule.restype = cp
        _lib = L
    return _lib


def _check(rc: int):
    if rc != HCT_OK:
        raise HctError(rc, lib().hct_last_error().decode())


def hct_version() -> str:
    return lib().hct_version().decode()


def hct_graph_create(spec: str, device: int = 0) -> ctypes.c_void_p:
    raw = spec.encode()
    out = ctypes.c_void_p()
    _check(lib().hct_graph_create(raw, len(raw), device, ctypes.byref(out)))
    return out


def hct_graph_create_scheduled(spec: str, device: int = 0, schedule: str | None = None) -> ctypes.c_void_p:
    raw = spec.encode()
    out = ctypes.c_void_p()
    _check(lib().hct_graph_create_scheduled(raw, len(raw), device, None if schedule is None else schedule.encode(), ctypes.byref(out)))
    return out


def hct_graph_autotune(spec: str, device: int, inputs, outputs, workspace: int = 0, workspace_bytes: int = 0, cuda_stream: int = 0,
                       max_trials: int = 16) -> ctypes.c_void_p:
    """inputs / outputs: device addresses as for hct_graph_run.  Returns the fastest handle."""
    raw = spec.encode()
    n_in, n_out = len(inputs), len(outputs)
    a_in = (ctypes.c_void_p * max(n_in, 1))(*inputs)
    a_out = (ctypes.c_void_p * max(n_out, 1))(*outputs)
    out = ctypes.c_void_p()
    _check(lib().hct_graph_autotune(raw, len(raw), device, a_in, n_in, a_out, n_out, workspace, workspace_bytes, cuda_stream,
                                    max_trials, ctypes.byref(out)))
    return out


def hct_graph_schedule(g) -> str:
    return lib().hct_graph_schedule(g).decode()


def hct_graph_run(g, inputs, outputs, workspace: int = 0, workspace_bytes: int = 0, cuda_stream: int = 0):
    """inputs / outputs: sequences of device addresses (ints), in spec order."""
    n_in, n_out = len(inputs), len(outputs)
    a_in = (ctypes.c_void_p * max(n_in, 1))(*inputs)
    a_out = (ctypes.c_void_p * max(n_out, 1))(*outputs)
    _check(lib().hct_graph_run(g, a_in, n_in, a_out, n_out, workspace, workspace_bytes, cuda_stream))


def hct_graph_status(g):
    _check(lib().hct_graph_status(g))


def hct_graph_destroy(g):
    _check(lib().hct_graph_destroy(g))


def hct_graph_num_inputs(g) -> int:
    return lib().hct_graph_num_inputs(g)


def hct_graph_num_outputs(g) -> int:
    return lib().hct_graph_num_outputs(g)


def hct_graph_tensor_info(g, is_output: bool, idx: int):
    name, dtype, rank = ctypes.c_char_p(), ctypes.c_int(), ctypes.c_int()
    shape = (ctypes.c_int64 * 4)()
    _check(lib().hct_graph_tensor_info(g, int(is_output), idx, ctypes.byref(name), ctypes.byref(dtype), ctypes.byref(rank), shape))
    return name.value.decode(), dtype.value, tuple(shape[i] for i in range(rank.value))


def hct_graph_workspace_bytes(g) -> int:
    return lib().hct_graph_workspace_bytes(g)


def hct_graph_input_layout(g, idx: int) -> int:
    return lib().hct_graph_input_layout(g, idx)


def hct_graph_output_layout(g, idx: int) -> int:
    return lib().hct_graph_output_layout(g, idx)


def hct_graph_num_kernels(g) -> int:
    return lib().hct_graph_num_kernels(g)


def hct_graph_cost(g):
    b, f = ctypes.c_double(), ctypes.c_double()
    _check(lib().hct_graph_cost(g, ctypes.byref(b), ctypes.byref(f)))
    return b.value, f.value


def hct_graph_plan_text(g) -> str:
    return lib().hct_graph_plan_text(g).decode()


def hct_graph_kernel_source(g, idx: int) -> str:
    s = lib().hct_graph_kernel_source(g, idx)
    return s.decode() if s is not None else ""


def hct_graph_kernel_name(g, idx: int) -> str:
    s = lib().hct_graph_kernel_name(g, idx)
    return s.decode() if s is not None else ""


def hct_gemm_bias_relu_f32_static(a: int, b: int, bias: int, out: int, m: int, k: int, n: int, apply_relu: bool = True,
                                  device: int = 0, cuda_stream: int = 0):
    """relu(A*B + bias) on device addresses, using the library's built-in scratch instead of a workspace."""
    _check(lib().hct_gemm_bias_relu_f32_static(a, b, bias, out, m, k, n, int(apply_relu), device, cuda_stream))
