"""ctypes front end of the plain-C CPU oracle ``bsp_oracle.c``.

TEST INFRASTRUCTURE ONLY: imported by the tests, the smoke check and the benchmark's CPU-baseline
leg.  Nothing here touches the CUDA library.  ``build()`` compiles the C file with gcc next to
this module; every wrapper takes and returns numpy arrays.

Conventions (paper's Introduction): W [O][H][K][I], X [N][L][J][I], Y [pixels][O], Gamma
[NB_o][NB_i] of 0/1 bytes, compact form = (row_ptr [NB_o+1], col_idx [nnz], payload
[nnz][b_o][H][K][b_i]).  Float tensors are float32 arrays (bf16 data are passed as the float32
values they represent); 8-bit integer tensors are int8 arrays.
"""
from __future__ import annotations

import ctypes as C
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bsp_oracle.c")
_LIB = os.path.join(_HERE, "libbsp_oracle.so")
_lib = None

NORM_L2, NORM_L1, NORM_VAR = 0, 1, 2
SCOPE_LAYER, SCOPE_ROW = 0, 1


class WDesc(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("O", "I", "H", "K", "bo", "bi")]


class XDesc(C.Structure):
    _fields_ = [(n, C.c_int) for n in ("N", "L", "J", "stride_h", "stride_w", "pad_h", "pad_w")]


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (-O2, OpenMP) if the shared object is missing or stale."""
    if (not force and os.path.exists(_LIB)
            and os.path.getmtime(_LIB) >= os.path.getmtime(_SRC)):
        return _LIB
    tmp = _LIB + ".tmp%d" % os.getpid()
    subprocess.check_call(["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-Wall",
                           "-o", tmp, _SRC])
    os.replace(tmp, _LIB)
    return _LIB


def lib():
    global _lib
    if _lib is None:
        _lib = C.CDLL(build())
        _lib.ref_set_threads.restype = C.c_int
    return _lib


def set_threads(n: int = 0) -> int:
    """Set the OpenMP thread count (0 keeps it) and return the count in effect."""
    return int(lib().ref_set_threads(C.c_int(n)))


def _p(a):
    return None if a is None else a.ctypes.data_as(C.c_void_p)


def _check(rc, what):
    if rc != 0:
        raise RuntimeError(f"oracle {what} failed with code {rc}")


def out_hw(L, J, H, K, stride_h=1, stride_w=1, pad_h=0, pad_w=0):
    return (L + 2 * pad_h - H) // stride_h + 1, (J + 2 * pad_w - K) // stride_w + 1


def scores(W: np.ndarray, bo: int, bi: int, norm: int = NORM_L2) -> np.ndarray:
    """Block importance [NB_o][NB_i]: float64 for float32 weights, int64 for int8 weights."""
    O, H, K, I = W.shape
    wd = WDesc(O, I, H, K, bo, bi)
    W = np.ascontiguousarray(W)
    if W.dtype == np.int8:
        s = np.empty((O // bo, I // bi), dtype=np.int64)
        _check(lib().ref_scores_i8(C.byref(wd), _p(W), C.c_int(norm), _p(s)), "scores_i8")
    else:
        assert W.dtype == np.float32
        s = np.empty((O // bo, I // bi), dtype=np.float64)
        _check(lib().ref_scores_f32(C.byref(wd), _p(W), C.c_int(norm), _p(s)), "scores_f32")
    return s


def mask(score: np.ndarray, n_zero: int, scope: int = SCOPE_LAYER) -> np.ndarray:
    """Gamma [NB_o][NB_i] uint8 with the n_zero lowest (score, index) blocks zeroed."""
    NBo, NBi = score.shape
    score = np.ascontiguousarray(score)
    g = np.empty((NBo, NBi), dtype=np.uint8)
    if score.dtype == np.int64:
        rc = lib().ref_mask(C.c_int(NBo), C.c_int(NBi), None, _p(score), C.c_int(scope),
                            C.c_int64(n_zero), _p(g))
    else:
        assert score.dtype == np.float64
        rc = lib().ref_mask(C.c_int(NBo), C.c_int(NBi), _p(score), None, C.c_int(scope),
                            C.c_int64(n_zero), _p(g))
    _check(rc, "mask")
    return g


def compact(W: np.ndarray, gamma: np.ndarray, bo: int, bi: int):
    """(row_ptr int32 [NB_o+1], col_idx int32 [nnz], payload [nnz][b_o][H][K][b_i])."""
    O, H, K, I = W.shape
    wd = WDesc(O, I, H, K, bo, bi)
    W = np.ascontiguousarray(W)
    gamma = np.ascontiguousarray(gamma, dtype=np.uint8)
    NBo, NBi = O // bo, I // bi
    cap = NBo * NBi
    row_ptr = np.zeros(NBo + 1, dtype=np.int32)
    col_idx = np.zeros(cap, dtype=np.int32)
    payload = np.zeros((cap, bo, H, K, bi), dtype=W.dtype)
    nnz = C.c_int64(0)
    _check(lib().ref_compact(C.byref(wd), _p(W), C.c_int(W.dtype.itemsize), _p(gamma), _p(row_ptr),
                             _p(col_idx), _p(payload), C.c_int64(cap), C.byref(nnz)), "compact")
    n = int(nnz.value)
    return row_ptr, col_idx[:n].copy(), payload[:n].copy()


def _pix(pix):
    if pix is None:
        return None, 0
    pix = np.ascontiguousarray(pix, dtype=np.int64)
    return pix, pix.size


def conv2d(wshape, bo, bi, row_ptr, col_idx, payload, X, bias=None, stride=(1, 1), pad=(0, 0),
           pix=None) -> np.ndarray:
    """Block-sparse convolution from the compact structure; rows = pixels (all, or ``pix``)."""
    O, H, K, I = wshape
    N, L, J, I2 = X.shape
    assert I2 == I
    wd = WDesc(O, I, H, K, bo, bi)
    xd = XDesc(N, L, J, stride[0], stride[1], pad[0], pad[1])
    M, Nw = out_hw(L, J, H, K, stride[0], stride[1], pad[0], pad[1])
    pixa, npix = _pix(pix)
    rows = npix if pix is not None else N * M * Nw
    X = np.ascontiguousarray(X)
    payload = np.ascontiguousarray(payload)
    row_ptr = np.ascontiguousarray(row_ptr, dtype=np.int32)
    col_idx = np.ascontiguousarray(col_idx, dtype=np.int32)
    if X.dtype == np.int8:
        assert payload.dtype == np.int8
        b = None if bias is None else np.ascontiguousarray(bias, dtype=np.int32)
        Y = np.empty((rows, O), dtype=np.int32)
        _check(lib().ref_conv2d_i8(C.byref(wd), C.byref(xd), _p(row_ptr), _p(col_idx), _p(payload), _p(X),
                                   _p(b), _p(pixa), C.c_int64(npix), _p(Y)), "conv2d_i8")
    else:
        assert X.dtype == np.float32 and payload.dtype == np.float32
        b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
        Y = np.empty((rows, O), dtype=np.float64)
        _check(lib().ref_conv2d_f32(C.byref(wd), C.byref(xd), _p(row_ptr), _p(col_idx), _p(payload), _p(X),
                                    _p(b), _p(pixa), C.c_int64(npix), _p(Y)), "conv2d_f32")
    return Y


def gemm(O, I, bo, bi, row_ptr, col_idx, payload, X, bias=None, pix=None) -> np.ndarray:
    """Block-sparse FC product; X [P][I] -> Y [P][O] (all rows, or the rows listed in ``pix``)."""
    P = X.shape[0]
    assert X.shape[1] == I
    pixa, npix = _pix(pix)
    rows = npix if pix is not None else P
    X = np.ascontiguousarray(X)
    payload = np.ascontiguousarray(payload)
    row_ptr = np.ascontiguousarray(row_ptr, dtype=np.int32)
    col_idx = np.ascontiguousarray(col_idx, dtype=np.int32)
    if X.dtype == np.int8:
        b = None if bias is None else np.ascontiguousarray(bias, dtype=np.int32)
        Y = np.empty((rows, O), dtype=np.int32)
        _check(lib().ref_gemm_i8(C.c_int(O), C.c_int(I), C.c_int(bo), C.c_int(bi), _p(row_ptr), _p(col_idx),
                                 _p(payload), _p(X), C.c_int64(P), _p(b), _p(pixa), C.c_int64(npix), _p(Y)),
               "gemm_i8")
    else:
        assert X.dtype == np.float32 and payload.dtype == np.float32
        b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
        Y = np.empty((rows, O), dtype=np.float64)
        _check(lib().ref_gemm_f32(C.c_int(O), C.c_int(I), C.c_int(bo), C.c_int(bi), _p(row_ptr), _p(col_idx),
                                  _p(payload), _p(X), C.c_int64(P), _p(b), _p(pixa), C.c_int64(npix), _p(Y)),
               "gemm_f32")
    return Y


def requant_i8(y32: np.ndarray, shift: np.ndarray) -> np.ndarray:
    """int32 [rows][O] (accumulator + bias) -> int8: value / 2^shift[o], nearest with halves away from zero, saturated."""
    y32 = np.ascontiguousarray(y32, dtype=np.int32)
    shift = np.ascontiguousarray(shift, dtype=np.int32)
    rows, O = y32.shape
    assert shift.shape == (O,)
    y8 = np.empty((rows, O), dtype=np.int8)
    _check(lib().ref_requant_i8(C.c_int64(rows), C.c_int(O), _p(y32), _p(shift), _p(y8)), "requant_i8")
    return y8


def round_bf16(v: np.ndarray) -> np.ndarray:
    """float64 -> nearest bfloat16 (ties to even), returned as float32."""
    v = np.ascontiguousarray(v, dtype=np.float64)
    out = np.empty(v.shape, dtype=np.float32)
    _check(lib().ref_round_bf16(C.c_int64(v.size), _p(v), _p(out)), "round_bf16")
    return out


def chain2(w1shape, bo1, bi1, c1, X, b1, relu, O2, bo2, bi2, c2, b2, stride=(1, 1), pad=(0, 0)) -> np.ndarray:
    """Two consecutive layers with the tensor between them stored as bfloat16 (Section "Depth-wise Tiling"):
    T = bf16(act(W1 * X + b1)), Y = W2 * T + b2 with a 1x1 second layer.  c1, c2 are (row_ptr, col_idx, payload) of
    the two layers; rows of the result = output positions."""
    T = conv2d(w1shape, bo1, bi1, c1[0], c1[1], c1[2], X, b1, stride, pad)
    if relu:
        _check(lib().ref_relu_f64(C.c_int64(T.size), _p(T)), "relu")
    Tb = round_bf16(T)
    O1 = w1shape[0]
    return gemm(O2, O1, bo2, bi2, c2[0], c2[1], np.asarray(c2[2]).reshape(-1, bo2, bi2), Tb, b2)


def chain2_q8(w1shape, bo1, bi1, c1, X, b1, shift1, relu, O2, bo2, bi2, c2, b2, shift2=None, stride=(1, 1), pad=(0, 0)) -> np.ndarray:
    """The 8-bit chain (Section "Depth-wise Tiling" with the tensors of Section "Compiler and its Code generation"): the
    tensor between the layers is the requantised int8 output of layer one, T = act(requant(W1 * X + b1, shift1)); Y is
    the int32 result W2 * T + b2 of the 1x1 second layer, or its requantised int8 form when shift2 is given."""
    T32 = conv2d(w1shape, bo1, bi1, c1[0], c1[1], c1[2], X, b1, stride, pad)
    T8 = requant_i8(T32, shift1)
    if relu:
        T8 = np.maximum(T8, 0).astype(np.int8)
    O1 = w1shape[0]
    Y32 = gemm(O2, O1, bo2, bi2, c2[0], c2[1], np.asarray(c2[2]).reshape(-1, bo2, bi2), T8, b2)
    return Y32 if shift2 is None else requant_i8(Y32, shift2)


def spgemm(kb, a, b) -> np.ndarray:
    """C = (Gamma . A)(Omega . B)^t from two compact forms (row_ptr, col_idx, payload [nnz][kb][kb]) with kb x kb blocks;
    dense float64 [NBa*kb][NBb*kb]."""
    (arp, aci, apl), (brp, bci, bpl) = a, b
    NBa, NBb = len(arp) - 1, len(brp) - 1
    apl = np.ascontiguousarray(apl, dtype=np.float32).reshape(-1, kb, kb)
    bpl = np.ascontiguousarray(bpl, dtype=np.float32).reshape(-1, kb, kb)
    Cm = np.empty((NBa * kb, NBb * kb), dtype=np.float64)
    _check(lib().ref_spgemm_f32(C.c_int(NBa), C.c_int(NBb), C.c_int(kb),
                                _p(np.ascontiguousarray(arp, dtype=np.int32)), _p(np.ascontiguousarray(aci, dtype=np.int32)), _p(apl),
                                _p(np.ascontiguousarray(brp, dtype=np.int32)), _p(np.ascontiguousarray(bci, dtype=np.int32)), _p(bpl),
                                _p(Cm)), "spgemm_f32")
    return Cm


def index_to_relative(row_ptr, col_idx) -> np.ndarray:
    """Relative column index of a compact form: first kept block of a row absolute, the others as distances."""
    row_ptr = np.ascontiguousarray(row_ptr, dtype=np.int32)
    col_idx = np.ascontiguousarray(col_idx, dtype=np.int32)
    rel = np.empty_like(col_idx)
    _check(lib().ref_index_to_relative(C.c_int(len(row_ptr) - 1), _p(row_ptr), _p(col_idx), _p(rel)), "index_to_relative")
    return rel


def index_from_relative(row_ptr, rel) -> np.ndarray:
    row_ptr = np.ascontiguousarray(row_ptr, dtype=np.int32)
    rel = np.ascontiguousarray(rel, dtype=np.int32)
    col = np.empty_like(rel)
    _check(lib().ref_index_from_relative(C.c_int(len(row_ptr) - 1), _p(row_ptr), _p(rel), _p(col)), "index_from_relative")
    return col


def dense_conv2d(W, X, bias=None, stride=(1, 1), pad=(0, 0)) -> np.ndarray:
    """Textbook dense convolution (cross-correlation) with bias; float64 or int64 [pixels][O]."""
    O, H, K, I = W.shape
    N, L, J, _ = X.shape
    wd = WDesc(O, I, H, K, 1, 1)
    xd = XDesc(N, L, J, stride[0], stride[1], pad[0], pad[1])
    M, Nw = out_hw(L, J, H, K, stride[0], stride[1], pad[0], pad[1])
    W = np.ascontiguousarray(W)
    X = np.ascontiguousarray(X)
    if X.dtype == np.int8:
        b = None if bias is None else np.ascontiguousarray(bias, dtype=np.int32)
        Y = np.empty((N * M * Nw, O), dtype=np.int64)
        _check(lib().ref_dense_conv2d_i8(C.byref(wd), C.byref(xd), _p(W), _p(X), _p(b), _p(Y)), "dense_i8")
    else:
        b = None if bias is None else np.ascontiguousarray(bias, dtype=np.float32)
        Y = np.empty((N * M * Nw, O), dtype=np.float64)
        _check(lib().ref_dense_conv2d_f32(C.byref(wd), C.byref(xd), _p(W), _p(X), _p(b), _p(Y)), "dense_f32")
    return Y


def apply_mask(W: np.ndarray, gamma: np.ndarray, bo: int, bi: int) -> np.ndarray:
    """Gamma (.) W of Eq. (1): every weight of a block with Gamma = 0 set to zero."""
    full = np.repeat(np.repeat(gamma.astype(bool), bo, axis=0), bi, axis=1)    # [O][I]
    return np.where(full[:, None, None, :], W, np.zeros((), dtype=W.dtype)).astype(W.dtype)
