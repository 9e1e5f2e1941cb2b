"""ctypes binding of libdivision.so: the same entry points as include/division.h, argument marshalling only.

Every step of compress / decompress runs inside the CUDA library.  PyTorch appears here only as the
owner of device memory and streams.  If the library has not been built the import of the symbols
fails loudly; nothing falls back to the CPU.
"""
from __future__ import annotations

import ctypes
import os
from ctypes import c_char_p, c_int32, c_int64, c_size_t, c_uint32, c_uint64, c_void_p

LIB_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "libdivision.so")

DIV_OK = 0
DIV_ERR_NULL, DIV_ERR_SHAPE, DIV_ERR_PARAM, DIV_ERR_ALIGN, DIV_ERR_CAPACITY, DIV_ERR_CUDA, DIV_ERR_TIMEOUT = range(1, 8)
DIV_F32, DIV_BF16 = 0, 1
DIV_FLAG_FORCE_TWO_PASS = 1
DIV_FLAG_NO_STRIP_KERNEL = 2
DIV_FLAG_NO_LAGGED_KERNEL = 4
DIV_FLAG_NO_PLANE_KERNELS = 8
DIV_FLAG_NO_LINE_KERNELS = 16
DIV_FLAG_NO_STAGED_KERNEL = 32
DIV_FLAG_TWO_LAUNCH_PLANES = 64
DTYPE_CODES = {"f32": DIV_F32, "bf16": DIV_BF16}

EXPORTED_SYMBOLS = (
    "div_compressed_bytes", "div_compress", "div_compress_ex", "div_compress_static", "div_read_static_status",
    "div_debug_compress_starved",
    "div_decompress", "div_plan_query",
    "div_compressed_bytes_3d", "div_compress_3d", "div_decompress_3d",
    "div_mask_bytes", "div_relu_forward", "div_dropout_forward", "div_mask_backward",
    "div_planegroup_bytes", "div_planegroup_compress", "div_planegroup_decompress", "div_planegroup_plan_query",
    "div_read_device_status", "div_status_string",
)


class DivDesc(ctypes.Structure):
    _fields_ = [("n", c_int64), ("c", c_int64), ("h", c_int64), ("w", c_int64),
                ("block", c_int32), ("qbits", c_int32), ("x_dtype", c_int32), ("lfc_dtype", c_int32)]


class DivDesc3D(ctypes.Structure):
    _fields_ = [("n", c_int64), ("c", c_int64), ("d", c_int64), ("h", c_int64), ("w", c_int64),
                ("block", c_int32), ("qbits", c_int32), ("x_dtype", c_int32), ("lfc_dtype", c_int32)]


class DivLayout(ctypes.Structure):
    _fields_ = [(name, c_uint64) for name in (
        "lfc_off", "lfc_bytes", "packed_off", "packed_bytes", "stats_off", "stats_bytes",
        "total_bytes", "closed_form_bytes", "raw_bytes", "workspace_bytes")]


class DivPlan(ctypes.Structure):
    _fields_ = [("fused", c_int32), ("grid", c_int32), ("threads", c_int32), ("stages", c_int32),
                ("lag", c_int32), ("smem_bytes", c_int32), ("chunk_elems", c_int64),
                ("chunks_per_sample", c_int64), ("decompress_fast", c_int32), ("reserved", c_int32)]


class DivisionError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} (status {status})")


_lib = None


def lib() -> ctypes.CDLL:
    """The loaded library; raises if it was never built (there is no other implementation to run)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(
                f"{LIB_PATH} is missing: build it with `python -m paper_2208_04187_b200.build` "
                "(or __graft_entry__.build()); this package has no CPU fallback")
        L = ctypes.CDLL(LIB_PATH)
        L.div_compressed_bytes.argtypes = [ctypes.POINTER(DivDesc), ctypes.POINTER(DivLayout)]
        L.div_compressed_bytes.restype = c_int32
        L.div_compress.argtypes = [ctypes.POINTER(DivDesc), c_void_p, c_void_p, c_size_t, c_void_p, c_size_t,
                                   c_uint64, c_void_p]
        L.div_compress.restype = c_int32
        L.div_compress_ex.argtypes = L.div_compress.argtypes + [c_uint32]
        L.div_compress_ex.restype = c_int32
        L.div_compress_static.argtypes = [ctypes.POINTER(DivDesc), c_void_p, c_void_p, c_size_t, c_uint64, c_void_p]
        L.div_compress_static.restype = c_int32
        L.div_read_static_status.argtypes = [c_void_p, ctypes.POINTER(c_int32)]
        L.div_read_static_status.restype = c_int32
        L.div_debug_compress_starved.argtypes = L.div_compress_ex.argtypes + [c_uint64]
        L.div_debug_compress_starved.restype = c_int32
        L.div_decompress.argtypes = [ctypes.POINTER(DivDesc), c_void_p, c_size_t, c_void_p, c_void_p]
        L.div_decompress.restype = c_int32
        L.div_plan_query.argtypes = [ctypes.POINTER(DivDesc), c_uint32, ctypes.POINTER(DivPlan)]
        L.div_plan_query.restype = c_int32
        L.div_planegroup_bytes.argtypes = [ctypes.POINTER(DivDesc), ctypes.POINTER(DivLayout)]
        L.div_planegroup_bytes.restype = c_int32
        L.div_planegroup_compress.argtypes = [ctypes.POINTER(DivDesc), c_void_p, c_void_p, c_size_t, c_uint64, c_void_p,
                                              c_uint32]
        L.div_planegroup_compress.restype = c_int32
        L.div_planegroup_decompress.argtypes = L.div_decompress.argtypes
        L.div_planegroup_decompress.restype = c_int32
        L.div_planegroup_plan_query.argtypes = L.div_plan_query.argtypes
        L.div_planegroup_plan_query.restype = c_int32
        L.div_compressed_bytes_3d.argtypes = [ctypes.POINTER(DivDesc3D), ctypes.POINTER(DivLayout)]
        L.div_compressed_bytes_3d.restype = c_int32
        L.div_compress_3d.argtypes = [ctypes.POINTER(DivDesc3D), c_void_p, c_void_p, c_size_t, c_void_p, c_size_t, c_uint64,
                                      c_void_p]
        L.div_compress_3d.restype = c_int32
        L.div_decompress_3d.argtypes = [ctypes.POINTER(DivDesc3D), c_void_p, c_size_t, c_void_p, c_void_p]
        L.div_decompress_3d.restype = c_int32
        L.div_mask_bytes.argtypes = [c_uint64, ctypes.POINTER(c_uint64)]
        L.div_mask_bytes.restype = c_int32
        L.div_relu_forward.argtypes = [c_void_p, c_void_p, c_void_p, c_size_t, c_uint64, c_int32, c_void_p]
        L.div_relu_forward.restype = c_int32
        L.div_dropout_forward.argtypes = [c_void_p, c_void_p, c_void_p, c_size_t, c_uint64, c_int32, c_uint64, c_uint32,
                                          c_void_p]
        L.div_dropout_forward.restype = c_int32
        L.div_mask_backward.argtypes = [c_void_p, c_size_t, c_void_p, c_void_p, c_uint64, c_int32, c_void_p]
        L.div_mask_backward.restype = c_int32
        L.div_read_device_status.argtypes = [c_void_p, c_void_p, ctypes.POINTER(c_int32)]
        L.div_read_device_status.restype = c_int32
        L.div_status_string.argtypes = [c_int32]
        L.div_status_string.restype = c_char_p
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().div_status_string(int(status)).decode()


def make_desc(n, c, h, w, block, qbits, x_dtype="f32", lfc_dtype="f32") -> DivDesc:
    return DivDesc(int(n), int(c), int(h), int(w), int(block), int(qbits),
                   DTYPE_CODES[x_dtype], DTYPE_CODES[lfc_dtype])


def _check(status: int, where: str):
    if status != DIV_OK:
        raise DivisionError(status, where)


def div_compressed_bytes(desc: DivDesc) -> DivLayout:
    out = DivLayout()
    _check(lib().div_compressed_bytes(ctypes.byref(desc), ctypes.byref(out)), "div_compressed_bytes")
    return out


def div_plan_query(desc: DivDesc, flags: int = 0) -> DivPlan:
    out = DivPlan()
    _check(lib().div_plan_query(ctypes.byref(desc), int(flags), ctypes.byref(out)), "div_plan_query")
    return out


def div_compress(desc: DivDesc, x_ptr: int, comp_ptr: int, comp_capacity: int, ws_ptr: int, ws_bytes: int,
                 seed: int, stream: int = 0, flags: int = 0) -> None:
    """Raw-pointer call (device pointers as integers, stream as a cudaStream_t handle)."""
    st = lib().div_compress_ex(ctypes.byref(desc), c_void_p(x_ptr), c_void_p(comp_ptr), comp_capacity,
                               c_void_p(ws_ptr), ws_bytes, c_uint64(seed & (2 ** 64 - 1)), c_void_p(stream),
                               int(flags))
    _check(st, "div_compress")


DIV_STATIC_MAX_SAMPLES = 1024


def div_compress_static(desc: DivDesc, x_ptr: int, comp_ptr: int, comp_capacity: int, seed: int, stream: int = 0) -> None:
    """div_compress with the scratch taken from a fixed array inside the library (nothing is allocated).

    For callers that cannot allocate device memory where they compress; at most DIV_STATIC_MAX_SAMPLES
    samples; calls on one device must not overlap on the GPU (they share the array).
    """
    st = lib().div_compress_static(ctypes.byref(desc), c_void_p(x_ptr), c_void_p(comp_ptr), comp_capacity,
                                   c_uint64(seed & (2 ** 64 - 1)), c_void_p(stream))
    _check(st, "div_compress_static")


def div_read_static_status(stream: int = 0) -> int:
    """Device-side status of the last div_compress_static on the current device (DIV_OK or DIV_ERR_TIMEOUT)."""
    out = c_int32(0)
    _check(lib().div_read_static_status(c_void_p(stream), ctypes.byref(out)), "div_read_static_status")
    return out.value


def div_decompress(desc: DivDesc, comp_ptr: int, comp_bytes: int, xhat_ptr: int, stream: int = 0) -> None:
    st = lib().div_decompress(ctypes.byref(desc), c_void_p(comp_ptr), comp_bytes, c_void_p(xhat_ptr),
                              c_void_p(stream))
    _check(st, "div_decompress")


def div_planegroup_bytes(desc: DivDesc) -> DivLayout:
    """Layout of the per-plane form: one bfloat16 (delta, Delta) pair per (sample, channel) plane."""
    out = DivLayout()
    _check(lib().div_planegroup_bytes(ctypes.byref(desc), ctypes.byref(out)), "div_planegroup_bytes")
    return out


def div_planegroup_plan_query(desc: DivDesc, flags: int = 0) -> DivPlan:
    out = DivPlan()
    _check(lib().div_planegroup_plan_query(ctypes.byref(desc), int(flags), ctypes.byref(out)),
           "div_planegroup_plan_query")
    return out


def div_planegroup_compress(desc: DivDesc, x_ptr: int, comp_ptr: int, comp_capacity: int, seed: int,
                            stream: int = 0, flags: int = 0) -> None:
    st = lib().div_planegroup_compress(ctypes.byref(desc), c_void_p(x_ptr), c_void_p(comp_ptr), comp_capacity,
                                       c_uint64(seed & (2 ** 64 - 1)), c_void_p(stream), int(flags))
    _check(st, "div_planegroup_compress")


def div_planegroup_decompress(desc: DivDesc, comp_ptr: int, comp_bytes: int, xhat_ptr: int, stream: int = 0) -> None:
    st = lib().div_planegroup_decompress(ctypes.byref(desc), c_void_p(comp_ptr), comp_bytes, c_void_p(xhat_ptr),
                                         c_void_p(stream))
    _check(st, "div_planegroup_decompress")


def make_desc_3d(n, c, d, h, w, block, qbits, x_dtype="f32", lfc_dtype="f32") -> DivDesc3D:
    return DivDesc3D(int(n), int(c), int(d), int(h), int(w), int(block), int(qbits), DTYPE_CODES[x_dtype], DTYPE_CODES[lfc_dtype])


def div_compressed_bytes_3d(desc: DivDesc3D) -> DivLayout:
    out = DivLayout()
    _check(lib().div_compressed_bytes_3d(ctypes.byref(desc), ctypes.byref(out)), "div_compressed_bytes_3d")
    return out


def div_compress_3d(desc: DivDesc3D, x_ptr: int, comp_ptr: int, comp_capacity: int, ws_ptr: int, ws_bytes: int,
                    seed: int, stream: int = 0) -> None:
    _check(lib().div_compress_3d(ctypes.byref(desc), c_void_p(x_ptr), c_void_p(comp_ptr), comp_capacity, c_void_p(ws_ptr),
                                 ws_bytes, c_uint64(seed & (2 ** 64 - 1)), c_void_p(stream)), "div_compress_3d")


def div_decompress_3d(desc: DivDesc3D, comp_ptr: int, comp_bytes: int, xhat_ptr: int, stream: int = 0) -> None:
    _check(lib().div_decompress_3d(ctypes.byref(desc), c_void_p(comp_ptr), comp_bytes, c_void_p(xhat_ptr), c_void_p(stream)),
           "div_decompress_3d")


def div_mask_bytes(total: int) -> int:
    out = c_uint64(0)
    _check(lib().div_mask_bytes(c_uint64(total), ctypes.byref(out)), "div_mask_bytes")
    return out.value


def div_relu_forward(x_ptr: int, y_ptr: int, mask_ptr: int, mask_capacity: int, total: int, dtype: str = "f32",
                     stream: int = 0) -> None:
    _check(lib().div_relu_forward(c_void_p(x_ptr), c_void_p(y_ptr), c_void_p(mask_ptr), mask_capacity, c_uint64(total),
                                  DTYPE_CODES[dtype], c_void_p(stream)), "div_relu_forward")


def div_dropout_forward(x_ptr: int, y_ptr: int, mask_ptr: int, mask_capacity: int, total: int, seed: int,
                        drop_threshold: int, dtype: str = "f32", stream: int = 0) -> None:
    _check(lib().div_dropout_forward(c_void_p(x_ptr), c_void_p(y_ptr), c_void_p(mask_ptr), mask_capacity, c_uint64(total),
                                     DTYPE_CODES[dtype], c_uint64(seed & (2 ** 64 - 1)), c_uint32(drop_threshold),
                                     c_void_p(stream)), "div_dropout_forward")


def div_mask_backward(mask_ptr: int, mask_bytes: int, grad_out_ptr: int, grad_in_ptr: int, total: int,
                      dtype: str = "f32", stream: int = 0) -> None:
    _check(lib().div_mask_backward(c_void_p(mask_ptr), mask_bytes, c_void_p(grad_out_ptr), c_void_p(grad_in_ptr),
                                   c_uint64(total), DTYPE_CODES[dtype], c_void_p(stream)), "div_mask_backward")


def div_read_device_status(ws_ptr: int, stream: int = 0) -> int:
    out = c_int32(0)
    _check(lib().div_read_device_status(c_void_p(ws_ptr), c_void_p(stream), ctypes.byref(out)),
           "div_read_device_status")
    return out.value


# ----------------------------------------------------------------------------------------
# torch conveniences: buffers and pointers only
# ----------------------------------------------------------------------------------------
def _torch():
    import torch
    return torch


def torch_dtype(name: str):
    torch = _torch()
    return {"f32": torch.float32, "bf16": torch.bfloat16}[name]


def current_stream_handle() -> int:
    """cudaStream_t of torch's current stream on the current device, as an integer."""
    torch = _torch()
    raw = getattr(torch._C, "_cuda_getCurrentRawStream", None)      # one C call instead of building a Stream object
    if raw is not None:
        return int(raw(torch.cuda.current_device()))
    return int(torch.cuda.current_stream().cuda_stream)


class Codec:
    """Device buffers for one descriptor (blob, workspace) and the two calls on torch tensors."""

    def __init__(self, n, c, h, w, block, qbits, x_dtype="f32", lfc_dtype="f32", device="cuda"):
        torch = _torch()
        self.x_dtype, self.lfc_dtype = x_dtype, lfc_dtype
        self.desc = make_desc(n, c, h, w, block, qbits, x_dtype, lfc_dtype)
        self.layout = div_compressed_bytes(self.desc)
        self.shape = (n, c, h, w)
        self.device = torch.device(device)
        self.blob = torch.zeros(int(self.layout.total_bytes), dtype=torch.uint8, device=self.device)
        self.workspace = torch.zeros(int(self.layout.workspace_bytes), dtype=torch.uint8, device=self.device)

    def plan(self, flags: int = 0) -> DivPlan:
        return div_plan_query(self.desc, flags)

    def compress(self, x, seed: int = 0, flags: int = 0, blob=None):
        """x: contiguous CUDA tensor of shape N x C x H x W in the descriptor's dtype."""
        torch = _torch()
        blob = self.blob if blob is None else blob
        if not (x.is_cuda and x.is_contiguous() and tuple(x.shape) == self.shape
                and x.dtype == torch_dtype(self.x_dtype)):
            raise ValueError("x must be a contiguous CUDA tensor matching the descriptor")
        div_compress(self.desc, x.data_ptr(), blob.data_ptr(), blob.numel(), self.workspace.data_ptr(),
                     self.workspace.numel(), seed, current_stream_handle(), flags)
        return blob

    def decompress(self, blob=None, out=None):
        torch = _torch()
        blob = self.blob if blob is None else blob
        if out is None:
            out = torch.empty(self.shape, dtype=torch_dtype(self.x_dtype), device=self.device)
        div_decompress(self.desc, blob.data_ptr(), blob.numel(), out.data_ptr(), current_stream_handle())
        return out

    def device_status(self) -> int:
        return div_read_device_status(self.workspace.data_ptr(), current_stream_handle())


class PlaneGroupCodec:
    """Codec with one bfloat16 (delta, Delta) pair per (sample, channel) plane; no workspace."""

    def __init__(self, n, c, h, w, block, qbits, x_dtype="f32", lfc_dtype="f32", device="cuda"):
        torch = _torch()
        self.x_dtype, self.lfc_dtype = x_dtype, lfc_dtype
        self.desc = make_desc(n, c, h, w, block, qbits, x_dtype, lfc_dtype)
        self.layout = div_planegroup_bytes(self.desc)
        self.shape = (n, c, h, w)
        self.device = torch.device(device)
        self.blob = torch.zeros(int(self.layout.total_bytes), dtype=torch.uint8, device=self.device)

    def plan(self, flags: int = 0) -> DivPlan:
        return div_planegroup_plan_query(self.desc, flags)

    def compress(self, x, seed: int = 0, flags: int = 0, blob=None):
        torch = _torch()
        blob = self.blob if blob is None else blob
        if not (x.is_cuda and x.is_contiguous() and tuple(x.shape) == self.shape
                and x.dtype == torch_dtype(self.x_dtype)):
            raise ValueError("x must be a contiguous CUDA tensor matching the descriptor")
        div_planegroup_compress(self.desc, x.data_ptr(), blob.data_ptr(), blob.numel(), seed,
                                current_stream_handle(), flags)
        return blob

    def decompress(self, blob=None, out=None):
        torch = _torch()
        blob = self.blob if blob is None else blob
        if out is None:
            out = torch.empty(self.shape, dtype=torch_dtype(self.x_dtype), device=self.device)
        div_planegroup_decompress(self.desc, blob.data_ptr(), blob.numel(), out.data_ptr(), current_stream_handle())
        return out
