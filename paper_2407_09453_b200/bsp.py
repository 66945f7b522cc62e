"""Thin ctypes binding of libbsp.so: same names as the C ABI (include/bsp.h), argument marshalling only.

Every function takes torch CUDA tensors (device memory and streams are PyTorch's), passes raw device
pointers to the library and raises ``BspError`` on a non-zero status.  All arithmetic runs in the CUDA
kernels; there is no CPU path.  Importing this module does not load the library; the first call does, and
fails loudly if the library is missing.
"""
from __future__ import annotations

import ctypes as C
import os

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libbsp.so")

OK, ERR_NULL, ERR_SHAPE, ERR_BLOCK, ERR_DTYPE, ERR_CAPACITY, ERR_INDEX, ERR_CUDA, ERR_TIMEOUT = range(9)
F32, BF16, I8, I32 = 0, 1, 2, 3
NORM_L2, NORM_L1, NORM_VAR = 0, 1, 2
SCOPE_LAYER, SCOPE_ROW = 0, 1

EXPORTS = ["bsp_mask_workspace_bytes", "bsp_mask", "bsp_mask_static", "bsp_packed_bytes",
           "bsp_compact_workspace_bytes", "bsp_compact_nnz", "bsp_compact", "bsp_conv_workspace_bytes", "bsp_gemm",
           "bsp_conv2d", "bsp_gemm_q8", "bsp_conv2d_q8", "bsp_conv2d_chain", "bsp_conv2d_chain_q8", "bsp_conv_kernel_name", "bsp_spgemm",
           "bsp_index_to_relative", "bsp_index_from_relative", "bsp_check", "bsp_status_string"]


class BspError(RuntimeError):
    def __init__(self, status: int, what: str):
        self.status = status
        super().__init__(f"{what}: bsp_status {status} ({status_string(status)})")


class WDesc(C.Structure):
    _fields_ = [("O", C.c_int), ("I", C.c_int), ("H", C.c_int), ("K", C.c_int), ("bo", C.c_int),
                ("bi", C.c_int), ("wtype", C.c_int)]


class XDesc(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("N", "L", "J", "stride_h", "stride_w", "pad_h", "pad_w")]


class Bcsr(C.Structure):
    _fields_ = [("row_ptr", C.c_void_p), ("col_idx", C.c_void_p), ("payload", C.c_void_p),
                ("packed", C.c_void_p), ("nnz", C.c_int64)]


_lib = None


def lib():
    """The loaded shared library (built by paper_2407_09453_b200.build); no fallback if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2407_09453_b200.build` "
                               "(or __graft_entry__.build()); there is no CPU fallback")
        L = C.CDLL(LIB_PATH)
        for n in ("bsp_mask_workspace_bytes", "bsp_packed_bytes", "bsp_compact_workspace_bytes",
                  "bsp_conv_workspace_bytes"):
            getattr(L, n).restype = C.c_size_t
        L.bsp_status_string.restype = C.c_char_p
        L.bsp_conv_kernel_name.restype = C.c_char_p
        for n in ("bsp_mask", "bsp_mask_static", "bsp_compact_nnz", "bsp_compact", "bsp_gemm", "bsp_conv2d",
                  "bsp_gemm_q8", "bsp_conv2d_q8", "bsp_conv2d_chain", "bsp_conv2d_chain_q8", "bsp_spgemm", "bsp_index_to_relative", "bsp_index_from_relative", "bsp_check"):
            getattr(L, n).restype = C.c_int
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().bsp_status_string(C.c_int(status)).decode()


_TORCH_DT = {torch.float32: F32, torch.bfloat16: BF16, torch.int8: I8, torch.int32: I32}


def dtype_code(t: torch.dtype) -> int:
    return _TORCH_DT[t]


def _ptr(t):
    return C.c_void_p(0 if t is None else t.data_ptr())


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return C.c_void_p(s.cuda_stream)


def _raise(rc, what):
    if rc != OK:
        raise BspError(rc, what)


def wdesc(O, I, H, K, bo, bi, wtype) -> WDesc:
    return WDesc(O, I, H, K, bo, bi, wtype if isinstance(wtype, int) else dtype_code(wtype))


def new_workspace(nbytes: int, device="cuda") -> torch.Tensor:
    """A zero-filled device workspace (the first 256 bytes hold the latched status word)."""
    return torch.zeros(max(int(nbytes), 256), dtype=torch.uint8, device=device)


def bsp_mask_workspace_bytes(wd: WDesc) -> int:
    return int(lib().bsp_mask_workspace_bytes(C.byref(wd)))


def bsp_mask(wd: WDesc, W, norm, scope, n_zero, gamma, scores_opt, ws, stream=None):
    _raise(lib().bsp_mask(C.byref(wd), _ptr(W), C.c_int(norm), C.c_int(scope), C.c_int64(n_zero), _ptr(gamma),
                          _ptr(scores_opt), _ptr(ws), _stream(stream)), "bsp_mask")


def bsp_packed_bytes(wd: WDesc, nnz: int) -> int:
    return int(lib().bsp_packed_bytes(C.byref(wd), C.c_int64(nnz)))


def bsp_compact_workspace_bytes(wd: WDesc) -> int:
    return int(lib().bsp_compact_workspace_bytes(C.byref(wd)))


def bsp_compact_nnz(wd: WDesc, gamma, ws, stream=None) -> int:
    out = C.c_int64(0)
    _raise(lib().bsp_compact_nnz(C.byref(wd), _ptr(gamma), C.byref(out), _ptr(ws), _stream(stream)),
           "bsp_compact_nnz")
    return int(out.value)


def bsp_compact(wd: WDesc, W, gamma, row_ptr, col_idx, payload, packed, capacity_blocks, ws, stream=None):
    _raise(lib().bsp_compact(C.byref(wd), _ptr(W), _ptr(gamma), _ptr(row_ptr), _ptr(col_idx), _ptr(payload),
                             _ptr(packed), C.c_int64(capacity_blocks), _ptr(ws), _stream(stream)), "bsp_compact")


def bcsr(row_ptr, col_idx, payload, packed, nnz) -> Bcsr:
    return Bcsr(_ptr(row_ptr).value, _ptr(col_idx).value, _ptr(payload).value, _ptr(packed).value, int(nnz))


def bsp_conv_workspace_bytes(wd: WDesc, xd: XDesc) -> int:
    return int(lib().bsp_conv_workspace_bytes(C.byref(wd), C.byref(xd)))


def bsp_gemm(wd: WDesc, w: Bcsr, X, P, bias, Y, ytype, ws, stream=None):
    _raise(lib().bsp_gemm(C.byref(wd), C.byref(w), _ptr(X), C.c_int64(P), _ptr(bias), _ptr(Y), C.c_int(ytype),
                          _ptr(ws), _stream(stream)), "bsp_gemm")


def bsp_conv2d(wd: WDesc, w: Bcsr, xd: XDesc, X, bias, Y, ytype, ws, stream=None):
    _raise(lib().bsp_conv2d(C.byref(wd), C.byref(w), C.byref(xd), _ptr(X), _ptr(bias), _ptr(Y), C.c_int(ytype),
                            _ptr(ws), _stream(stream)), "bsp_conv2d")


def bsp_conv2d_q8(wd: WDesc, w: Bcsr, xd: XDesc, X, bias, shift, Y, ws, stream=None):
    _raise(lib().bsp_conv2d_q8(C.byref(wd), C.byref(w), C.byref(xd), _ptr(X), _ptr(bias), _ptr(shift), _ptr(Y), _ptr(ws),
                               _stream(stream)), "bsp_conv2d_q8")


def bsp_gemm_q8(wd: WDesc, w: Bcsr, X, P, bias, shift, Y, ws, stream=None):
    _raise(lib().bsp_gemm_q8(C.byref(wd), C.byref(w), _ptr(X), C.c_int64(P), _ptr(bias), _ptr(shift), _ptr(Y), _ptr(ws),
                             _stream(stream)), "bsp_gemm_q8")


def bsp_conv2d_chain(wd1: WDesc, w1: Bcsr, wd2: WDesc, w2: Bcsr, xd: XDesc, X, bias1, relu, bias2, Y, ytype, ws, stream=None):
    _raise(lib().bsp_conv2d_chain(C.byref(wd1), C.byref(w1), C.byref(wd2), C.byref(w2), C.byref(xd), _ptr(X), _ptr(bias1),
                                  C.c_int(1 if relu else 0), _ptr(bias2), _ptr(Y), C.c_int(ytype), _ptr(ws), _stream(stream)),
           "bsp_conv2d_chain")


def bsp_conv2d_chain_q8(wd1: WDesc, w1: Bcsr, wd2: WDesc, w2: Bcsr, xd: XDesc, X, bias1, shift1, relu, bias2, shift2, Y, ws, stream=None):
    _raise(lib().bsp_conv2d_chain_q8(C.byref(wd1), C.byref(w1), C.byref(wd2), C.byref(w2), C.byref(xd), _ptr(X), _ptr(bias1),
                                     _ptr(shift1), C.c_int(1 if relu else 0), _ptr(bias2), _ptr(shift2), _ptr(Y), _ptr(ws),
                                     _stream(stream)), "bsp_conv2d_chain_q8")


def bsp_spgemm(wa: WDesc, a: Bcsr, wb: WDesc, b: Bcsr, Cm, ws, stream=None):
    _raise(lib().bsp_spgemm(C.byref(wa), C.byref(a), C.byref(wb), C.byref(b), _ptr(Cm), _ptr(ws), _stream(stream)), "bsp_spgemm")


def bsp_index_to_relative(NBo, row_ptr, col_idx, rel, stream=None):
    _raise(lib().bsp_index_to_relative(C.c_int(NBo), _ptr(row_ptr), _ptr(col_idx), _ptr(rel), _stream(stream)), "bsp_index_to_relative")


def bsp_index_from_relative(NBo, row_ptr, rel, col_idx, stream=None):
    _raise(lib().bsp_index_from_relative(C.c_int(NBo), _ptr(row_ptr), _ptr(rel), _ptr(col_idx), _stream(stream)),
           "bsp_index_from_relative")


def bsp_mask_static(wd: WDesc, W, norm, scope, n_zero, gamma, stream=None):
    _raise(lib().bsp_mask_static(C.byref(wd), _ptr(W), C.c_int(norm), C.c_int(scope), C.c_int64(n_zero), _ptr(gamma),
                                 _stream(stream)), "bsp_mask_static")


def bsp_check(ws, stream=None):
    _raise(lib().bsp_check(_ptr(ws), _stream(stream)), "bsp_check")


def conv_kernel_name(wd: WDesc, xd: XDesc) -> str:
    """Name of the product kernel that bsp_conv2d / bsp_gemm launch for these descriptors."""
    r = lib().bsp_conv_kernel_name(C.byref(wd), C.byref(xd))
    if r is None:
        raise BspError(ERR_SHAPE, "bsp_conv_kernel_name")
    return r.decode()


def launches_per_step(wd: WDesc) -> int:
    """Kernel launches of one bsp_mask + bsp_compact + bsp_conv2d/bsp_gemm pass.  General path: score, select; the
    compaction; the product kernel.  Small layers take one launch for the mask (up to 4096 blocks)."""
    nb = (wd.O // wd.bo) * (wd.I // wd.bi)
    return (1 if nb <= 4096 else 2) + 1 + 1


class SparseLayer:
    """Device buffers of one compacted layer plus the calls that fill and use them (marshalling only)."""

    def __init__(self, O, I, H, K, bo, bi, wtype: torch.dtype, capacity_blocks=None, device="cuda",
                 canonical=True):
        self.wd = wdesc(O, I, H, K, bo, bi, wtype)
        self.wtype = wtype
        self.NBo, self.NBi = O // bo, I // bi
        NB = self.NBo * self.NBi
        self.capacity = NB if capacity_blocks is None else int(capacity_blocks)
        self.gamma = torch.empty(NB, dtype=torch.uint8, device=device)
        self.row_ptr = torch.empty(self.NBo + 1, dtype=torch.int32, device=device)
        self.col_idx = torch.empty(max(self.capacity, 1), dtype=torch.int32, device=device)
        self.payload = (torch.empty(max(self.capacity, 1) * bo * H * K * bi, dtype=wtype, device=device)
                        if canonical else None)
        self.packed = torch.empty(bsp_packed_bytes(self.wd, self.capacity), dtype=torch.uint8, device=device)
        self.ws = new_workspace(max(bsp_mask_workspace_bytes(self.wd), bsp_compact_workspace_bytes(self.wd)),
                                device)
        self.nnz = self.capacity

    def mask(self, W, n_zero, norm=NORM_L2, scope=SCOPE_LAYER, scores=None, stream=None):
        bsp_mask(self.wd, W, norm, scope, n_zero, self.gamma, scores, self.ws, stream)
        self.nnz = (self.NBo * self.NBi - n_zero) if scope == SCOPE_LAYER else self.NBo * (self.NBi - n_zero)

    def compact(self, W, gamma=None, stream=None):
        if gamma is not None:
            self.gamma.copy_(gamma.reshape(-1))
        bsp_compact(self.wd, W, self.gamma, self.row_ptr, self.col_idx, self.payload, self.packed, self.capacity,
                    self.ws, stream)

    def handle(self) -> Bcsr:
        return bcsr(self.row_ptr, self.col_idx, self.payload, self.packed, min(self.nnz, self.capacity))

    def conv2d(self, X, bias, Y, stride=(1, 1), pad=(0, 0), stream=None):
        N, L, J, _ = X.shape
        xd = XDesc(N, L, J, stride[0], stride[1], pad[0], pad[1])
        bsp_conv2d(self.wd, self.handle(), xd, X, bias, Y, dtype_code(Y.dtype), self.ws, stream)

    def gemm(self, X, bias, Y, stream=None):
        bsp_gemm(self.wd, self.handle(), X, X.shape[0], bias, Y, dtype_code(Y.dtype), self.ws, stream)

    def conv2d_q8(self, X, bias, shift, Y, stride=(1, 1), pad=(0, 0), stream=None):
        N, L, J, _ = X.shape
        xd = XDesc(N, L, J, stride[0], stride[1], pad[0], pad[1])
        bsp_conv2d_q8(self.wd, self.handle(), xd, X, bias, shift, Y, self.ws, stream)

    def gemm_q8(self, X, bias, shift, Y, stream=None):
        bsp_gemm_q8(self.wd, self.handle(), X, X.shape[0], bias, shift, Y, self.ws, stream)

    def check(self, stream=None):
        bsp_check(self.ws, stream)
