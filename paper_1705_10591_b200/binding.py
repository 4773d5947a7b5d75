"""ctypes binding of libconv2d_b200.so: same names and argument order as the C header.

Pointers are passed as integers (``tensor.data_ptr()`` / ``ndarray.ctypes.data``),
streams as the integer ``torch.cuda.current_stream().cuda_stream``.  Nothing here
computes anything and nothing falls back to another implementation: if the
library is missing or a call fails, an exception is raised.
"""
from __future__ import annotations

import ctypes
from pathlib import Path

ALGO_AUTO, ALGO_FFMA, ALGO_TF32, ALGO_16BIT = 0, 1, 2, 3
OPERAND_BF16, OPERAND_FP16 = 0, 1
FLAG_WEIGHTS_PACKED = 1

_LIB_PATH = Path(__file__).resolve().parent / "libconv2d_b200.so"
_lib = None


class Conv2dError(RuntimeError):
    """A library call returned a status other than CONV2D_OK."""

    def __init__(self, status: int, where: str):
        self.status = int(status)
        super().__init__(f"{where}: status {self.status} ({conv2d_status_string(self.status)})")


def library_path() -> Path:
    return _LIB_PATH


def load_library() -> ctypes.CDLL:
    """Loads the shared library (built in-tree by ``python -m paper_1705_10591_b200.build``)."""
    global _lib
    if _lib is not None:
        return _lib
    if not _LIB_PATH.exists():
        raise FileNotFoundError(
            f"{_LIB_PATH} is missing: build it with `python -m paper_1705_10591_b200.build` "
            "(there is no fallback implementation)")
    lib = ctypes.CDLL(str(_LIB_PATH))
    vp, i, sz, u = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t, ctypes.c_uint
    lib.conv2d_fwd_workspace_size.argtypes = [i] * 7 + [i, ctypes.POINTER(sz)]
    lib.conv2d_fwd_workspace_size.restype = i
    lib.conv2d_fwd_plan_describe.argtypes = [i] * 7 + [i, ctypes.c_char_p, sz]
    lib.conv2d_fwd_plan_describe.restype = i
    lib.conv2d_fwd_single_channel.argtypes = [vp, vp, vp] + [i] * 6 + [vp, sz, u, vp]
    lib.conv2d_fwd_single_channel.restype = i
    lib.conv2d_fwd_general.argtypes = [vp, vp, vp] + [i] * 7 + [i, vp, sz, u, vp]
    lib.conv2d_fwd_general.restype = i
    lib.conv2d_fwd_general_16bit.argtypes = [vp, vp, vp] + [i] * 7 + [i, vp, sz, u, vp]
    lib.conv2d_fwd_general_16bit.restype = i
    lib.conv2d_fwd_padded_workspace_size.argtypes = [i] * 9 + [i, ctypes.POINTER(sz)]
    lib.conv2d_fwd_padded_workspace_size.restype = i
    lib.conv2d_fwd_general_padded.argtypes = [vp, vp, vp] + [i] * 9 + [i, vp, sz, u, vp]
    lib.conv2d_fwd_general_padded.restype = i
    lib.conv2d_fwd_strided_workspace_size.argtypes = [i] * 10 + [i, ctypes.POINTER(sz)]
    lib.conv2d_fwd_strided_workspace_size.restype = i
    lib.conv2d_fwd_general_strided.argtypes = [vp, vp, vp] + [i] * 10 + [i, vp, sz, u, vp]
    lib.conv2d_fwd_general_strided.restype = i
    lib.conv2d_fwd_general_noalloc.argtypes = [vp, vp, vp] + [i] * 7 + [i, vp]
    lib.conv2d_fwd_general_noalloc.restype = i
    lib.conv2d_fwd_host.argtypes = [vp] * 6 + [i] * 7 + [i, vp, sz, vp]
    lib.conv2d_fwd_host.restype = i
    lib.conv2d_get_status.argtypes = [vp, vp]
    lib.conv2d_get_status.restype = i
    lib.conv2d_status_string.argtypes = [i]
    lib.conv2d_status_string.restype = ctypes.c_char_p
    lib.conv2d_launch_count.argtypes = []
    lib.conv2d_launch_count.restype = ctypes.c_ulonglong
    _lib = lib
    return lib


def _check(status: int, where: str) -> None:
    if status != 0:
        raise Conv2dError(status, where)


def conv2d_status_string(status: int) -> str:
    return load_library().conv2d_status_string(int(status)).decode()


def conv2d_launch_count() -> int:
    return int(load_library().conv2d_launch_count())


def conv2d_fwd_workspace_size(N, C, H, W, K, R, S, algo=ALGO_AUTO) -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().conv2d_fwd_workspace_size(N, C, H, W, K, R, S, algo, ctypes.byref(out)),
           "conv2d_fwd_workspace_size")
    return int(out.value)


def conv2d_fwd_plan_describe(N, C, H, W, K, R, S, algo=ALGO_AUTO) -> dict:
    """The library's description of its tensor-core plan for a shape, as a dict of its key=value pairs."""
    buf = ctypes.create_string_buffer(1024)
    _check(load_library().conv2d_fwd_plan_describe(N, C, H, W, K, R, S, algo, buf, len(buf)), "conv2d_fwd_plan_describe")
    out = {}
    for pair in buf.value.decode().split():
        key, _, val = pair.partition("=")
        try:
            out[key] = int(val)
        except ValueError:
            try:
                out[key] = float(val)
            except ValueError:
                out[key] = val
    return out


def conv2d_fwd_single_channel(x_ptr, w_ptr, y_ptr, N, H, W, K, R, S,
                              workspace_ptr=0, workspace_bytes=0, flags=0, stream=0) -> None:
    _check(load_library().conv2d_fwd_single_channel(x_ptr, w_ptr, y_ptr, N, H, W, K, R, S,
                                                    workspace_ptr or None, workspace_bytes, flags, stream or None),
           "conv2d_fwd_single_channel")


def conv2d_fwd_general(x_ptr, w_ptr, y_ptr, N, C, H, W, K, R, S, algo=ALGO_AUTO,
                       workspace_ptr=0, workspace_bytes=0, flags=0, stream=0) -> None:
    _check(load_library().conv2d_fwd_general(x_ptr, w_ptr, y_ptr, N, C, H, W, K, R, S, algo,
                                             workspace_ptr or None, workspace_bytes, flags, stream or None),
           "conv2d_fwd_general")


def conv2d_fwd_general_16bit(x_ptr, w_ptr, y_ptr, N, C, H, W, K, R, S, operand=OPERAND_BF16,
                             workspace_ptr=0, workspace_bytes=0, flags=0, stream=0) -> None:
    """x, w: device tensors of bf16 or fp16 elements (as `operand` says); y: device fp32 tensor."""
    _check(load_library().conv2d_fwd_general_16bit(x_ptr, w_ptr, y_ptr, N, C, H, W, K, R, S, operand,
                                                   workspace_ptr or None, workspace_bytes, flags, stream or None),
           "conv2d_fwd_general_16bit")


def conv2d_fwd_padded_workspace_size(N, C, H, W, K, R, S, pad_h, pad_w, algo=ALGO_AUTO) -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().conv2d_fwd_padded_workspace_size(N, C, H, W, K, R, S, pad_h, pad_w, algo, ctypes.byref(out)),
           "conv2d_fwd_padded_workspace_size")
    return int(out.value)


def conv2d_fwd_general_padded(x_ptr, w_ptr, y_ptr, N, C, H, W, K, R, S, pad_h, pad_w, algo=ALGO_AUTO,
                              workspace_ptr=0, workspace_bytes=0, flags=0, stream=0) -> None:
    """Zero padding of pad_h rows / pad_w columns on every side; y is [N, K, H+2*pad_h-R+1, W+2*pad_w-S+1]."""
    _check(load_library().conv2d_fwd_general_padded(x_ptr, w_ptr, y_ptr, N, C, H, W, K, R, S, pad_h, pad_w, algo,
                                                    workspace_ptr or None, workspace_bytes, flags, stream or None),
           "conv2d_fwd_general_padded")


def conv2d_fwd_strided_workspace_size(N, C, H, W, K, R, S, pad_h, pad_w, stride, algo=ALGO_AUTO) -> int:
    out = ctypes.c_size_t(0)
    _check(load_library().conv2d_fwd_strided_workspace_size(N, C, H, W, K, R, S, pad_h, pad_w, stride, algo,
                                                            ctypes.byref(out)), "conv2d_fwd_strided_workspace_size")
    return int(out.value)


def conv2d_fwd_general_strided(x_ptr, w_ptr, y_ptr, N, C, H, W, K, R, S, pad_h, pad_w, stride, algo=ALGO_AUTO,
                               workspace_ptr=0, workspace_bytes=0, flags=0, stream=0) -> None:
    """Zero padding and stride; y is [N, K, (H+2*pad_h-R)//stride+1, (W+2*pad_w-S)//stride+1]."""
    _check(load_library().conv2d_fwd_general_strided(x_ptr, w_ptr, y_ptr, N, C, H, W, K, R, S, pad_h, pad_w, stride, algo,
                                                     workspace_ptr or None, workspace_bytes, flags, stream or None),
           "conv2d_fwd_general_strided")


def conv2d_fwd_general_noalloc(x_ptr, w_ptr, y_ptr, N, C, H, W, K, R, S, wait=0, stream=0) -> None:
    """Tensor-core convolution whose scratch is the library's own fixed device array (see the header)."""
    _check(load_library().conv2d_fwd_general_noalloc(x_ptr, w_ptr, y_ptr, N, C, H, W, K, R, S,
                                                     int(wait), stream or None),
           "conv2d_fwd_general_noalloc")


def conv2d_fwd_host(x_host_ptr, w_host_ptr, y_host_ptr, x_ptr, w_ptr, y_ptr, N, C, H, W, K, R, S,
                    algo=ALGO_AUTO, workspace_ptr=0, workspace_bytes=0, stream=0) -> None:
    _check(load_library().conv2d_fwd_host(x_host_ptr, w_host_ptr, y_host_ptr, x_ptr, w_ptr, y_ptr,
                                          N, C, H, W, K, R, S, algo,
                                          workspace_ptr or None, workspace_bytes, stream or None),
           "conv2d_fwd_host")


def conv2d_get_status(workspace_ptr=0, stream=0) -> None:
    """Waits for the stream; raises if a kernel reported a device-side timeout."""
    _check(load_library().conv2d_get_status(workspace_ptr or None, stream or None), "conv2d_get_status")
