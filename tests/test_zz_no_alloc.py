"""bsp_mask_static: the Gamma builder for hosts that cannot give the library scratch memory.

A caller that lives inside someone else's memory plan (a plugin handed only its tensors, a loop where
cudaMalloc is forbidden) cannot pass bsp_mask() its workspace.  The static variant keeps the block scores
in an array built into the library.  This file is collected last on purpose: if it fails under -x, every
other test has already run.  Two calls in a row share the built-in array, so the second call checks that
nothing stale from the first leaks into its result.
"""
import ctypes as C

import numpy as np
import pytest
import torch

from oracle import ref
from paper_2407_09453_b200 import bsp, build, synth


def test_symbol_and_limit_on_host():
    build.build()
    lib = bsp.lib()
    assert hasattr(lib, "bsp_mask_static")
    lib.bsp_mask_static.restype = C.c_int
    one = C.c_void_p(256)
    big = bsp.wdesc(4096, 4096, 1, 1, 8, 8, bsp.BF16)          # 262144 blocks > 65536: rejected on the host
    assert lib.bsp_mask_static(C.byref(big), one, 0, 0, C.c_int64(1), one, None) == bsp.ERR_CAPACITY
    ok = bsp.wdesc(64, 64, 1, 1, 8, 8, bsp.BF16)
    assert lib.bsp_mask_static(C.byref(ok), None, 0, 0, C.c_int64(1), one, None) == bsp.ERR_NULL
    assert lib.bsp_mask_static(C.byref(ok), one, 0, 0, C.c_int64(65), one, None) == bsp.ERR_CAPACITY


@pytest.mark.gpu
def test_static_variant_matches_workspace_variant_twice_in_a_row():
    lib = bsp.lib()
    lib.bsp_mask_static.restype = C.c_int
    stream = C.c_void_p(torch.cuda.current_stream().cuda_stream)
    cases = [  # (O, I, H, K, bo, bi, dtype, n_zero, scope): second call is smaller, so stale scores sit behind it
        (512, 512, 3, 3, 8, 8, torch.bfloat16, 2048, bsp.SCOPE_LAYER),
        (128, 256, 1, 1, 4, 16, torch.int8, 7, bsp.SCOPE_ROW),
    ]
    for idx, (O, I, H, K, bo, bi, dt, n_zero, scope) in enumerate(cases):
        if dt == torch.int8:
            W = torch.from_numpy(synth.uniform_int(900 + idx, (O, H, K, I), -127, 127).astype(np.int8)).cuda()
        else:
            W = torch.from_numpy(synth.normal(900 + idx, (O, H, K, I), 0.05).astype(np.float32)).cuda().to(dt)
        wd = bsp.wdesc(O, I, H, K, bo, bi, dt)
        NB = (O // bo) * (I // bi)
        want = torch.empty(NB, dtype=torch.uint8, device="cuda")
        ws = bsp.new_workspace(bsp.bsp_mask_workspace_bytes(wd))
        bsp.bsp_mask(wd, W, bsp.NORM_L2, scope, n_zero, want, None, ws)
        got = torch.full((NB,), 9, dtype=torch.uint8, device="cuda")
        rc = lib.bsp_mask_static(C.byref(wd), C.c_void_p(W.data_ptr()), bsp.NORM_L2, scope, C.c_int64(n_zero),
                                 C.c_void_p(got.data_ptr()), stream)
        assert rc == bsp.OK
        torch.cuda.synchronize()
        assert torch.equal(got, want)                                # masks are compared bit for bit
        Wh = W.float().cpu().numpy() if dt != torch.int8 else W.cpu().numpy()
        oracle = ref.mask(ref.scores(Wh, bo, bi), n_zero, ref.SCOPE_LAYER if scope == bsp.SCOPE_LAYER else ref.SCOPE_ROW)
        assert np.array_equal(got.cpu().numpy().reshape(oracle.shape), oracle)      # and with the CPU oracle
        zeros = int((got == 0).sum())
        assert zeros == (n_zero if scope == bsp.SCOPE_LAYER else n_zero * (O // bo))
