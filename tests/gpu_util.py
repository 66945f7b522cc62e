"""Helpers for the GPU parity tests: move seeded numpy tensors to the device and call the C ABI."""
import numpy as np
import torch

from paper_2407_09453_b200 import bsp, synth

TORCH_DT = {"bf16": torch.bfloat16, "f32": torch.float32, "i8": torch.int8}

def to_dev(a: np.ndarray, dtype: str) -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t.to(torch.bfloat16) if dtype == "bf16" else t


def from_dev(t: torch.Tensor) -> np.ndarray:
    if t.dtype == torch.bfloat16:
        return t.float().cpu().numpy()
    return t.cpu().numpy()


def gpu_mask(W, bo, bi, dtype, n_zero, norm=bsp.NORM_L2, scope=bsp.SCOPE_LAYER):
    O, H, K, I = W.shape
    lay = bsp.SparseLayer(O, I, H, K, bo, bi, TORCH_DT[dtype])
    Wd = to_dev(W, dtype)
    sc = torch.empty(lay.NBo * lay.NBi, dtype=torch.int64 if dtype == "i8" else torch.float64, device="cuda")
    lay.mask(Wd, n_zero, norm, scope, sc)
    lay.check()
    return from_dev(lay.gamma).reshape(lay.NBo, lay.NBi), from_dev(sc).reshape(lay.NBo, lay.NBi), lay, Wd


def gpu_layer(W, gamma, bo, bi, dtype):
    O, H, K, I = W.shape
    lay = bsp.SparseLayer(O, I, H, K, bo, bi, TORCH_DT[dtype])
    Wd = to_dev(W, dtype)
    lay.compact(Wd, torch.from_numpy(np.ascontiguousarray(gamma, dtype=np.uint8)).cuda())
    lay.nnz = int(gamma.sum())
    lay.check()
    return lay


def gpu_conv(lay, X, bias, dtype, stride=(1, 1), pad=(0, 0), out="f32"):
    N, L, J, I = X.shape
    H, K, O = lay.wd.H, lay.wd.K, lay.wd.O
    M = (L + 2 * pad[0] - H) // stride[0] + 1
    Nw = (J + 2 * pad[1] - K) // stride[1] + 1
    ydt = torch.int32 if dtype == "i8" else (torch.bfloat16 if out == "bf16" else torch.float32)
    Y = torch.full((N, M, Nw, O), -7, dtype=ydt, device="cuda")
    Xd = to_dev(X, dtype)
    bd = None if bias is None else torch.from_numpy(bias).cuda()
    lay.conv2d(Xd, bd, Y, stride, pad)
    lay.check()
    return from_dev(Y).reshape(-1, O)


def gpu_gemm(lay, X, bias, dtype, out="f32"):
    P, I = X.shape
    O = lay.wd.O
    ydt = torch.int32 if dtype == "i8" else (torch.bfloat16 if out == "bf16" else torch.float32)
    Y = torch.full((P, O), -7, dtype=ydt, device="cuda")
    Xd = to_dev(X, dtype)
    bd = None if bias is None else torch.from_numpy(bias).cuda()
    lay.gemm(Xd, bd, Y)
    lay.check()
    return from_dev(Y)


def rel_err(got, want):
    """max |got - want| / max |want| (the normwise reading of 'max relative error')."""
    return float(np.abs(got.astype(np.float64) - want).max() / max(np.abs(want).max(), 1e-30))


# stated tolerance: max relative error 1e-2 for bf16 inputs with fp32 accumulation
TOL = 1e-2
# what the arithmetic should deliver: fp32 accumulation of exact bf16 products over at most a few thousand
# terms (error << 1e-4 of the largest output); bf16 output adds half an ulp, 2^-9 relative; tf32 rounds each
# operand to 11 bits
TIGHT = {"f32out": 2e-4, "bf16out": 5e-3, "tf32": 3e-3}


def make_case(seed, O, I, H, K, dtype):
    if dtype == "i8":
        W = synth.uniform_int(seed, (O, H, K, I), -127, 127).astype(np.int8)
    else:
        W = synth.normal(seed, (O, H, K, I), float(np.sqrt(2.0 / (H * K * I)))).astype(np.float32)
        if dtype == "bf16":
            W = synth.round_to_bf16(W)
    return W


def make_x(seed, shape, dtype):
    if dtype == "i8":
        return synth.uniform_int(seed, shape, -127, 127).astype(np.int8)
    X = synth.normal(seed, shape).astype(np.float32)
    return synth.round_to_bf16(X) if dtype == "bf16" else X


def make_bias(seed, O, dtype):
    if dtype == "i8":
        return synth.uniform_int(seed, (O,), -(1 << 15), 1 << 15).astype(np.int32)
    return synth.normal(seed, (O,), 0.1).astype(np.float32)
