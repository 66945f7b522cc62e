"""GPU parity of the block-sparse x block-sparse product and of the relative column index against the oracle, through the
C ABI: the product within the fp32-accumulation tolerance (bf16 or fp32 blocks), the index bit for bit."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2407_09453_b200 import bsp, synth
from gpu_util import gpu_layer, make_case, rel_err

pytestmark = pytest.mark.gpu


def run_spgemm(seed, Oa, Ob, I, dtype, fa, fb):
    A = make_case(seed, Oa, I, 1, 1, dtype)
    B = make_case(seed + 10, Ob, I, 1, 1, dtype)
    ga = synth.random_gamma(seed + 1, Oa // 8, I // 8, int(round(fa * (Oa // 8) * (I // 8))))
    gb = synth.random_gamma(seed + 11, Ob // 8, I // 8, int(round(fb * (Ob // 8) * (I // 8))))
    la, lb = gpu_layer(A, ga, 8, 8, dtype), gpu_layer(B, gb, 8, 8, dtype)
    la.nnz, lb.nnz = int(ga.sum()), int(gb.sum())
    Cm = torch.full((Oa, Ob), -7.0, dtype=torch.float32, device="cuda")
    bsp.bsp_spgemm(la.wd, la.handle(), lb.wd, lb.handle(), Cm, la.ws)
    la.check()
    want = ref.spgemm(8, ref.compact(A, ga, 8, 8), ref.compact(B, gb, 8, 8))
    got = Cm.cpu().numpy()
    assert rel_err(got, want) <= 2e-5 if want.any() else np.array_equal(got, want)
    # blocks of C whose rows share no kept column are exactly zero
    share = (ga.astype(np.int32) @ gb.astype(np.int32).T) > 0
    full = np.repeat(np.repeat(share, 8, axis=0), 8, axis=1)
    assert np.all(got[~full] == 0.0)
    return got


@pytest.mark.parametrize("dtype", ["f32", "bf16"])
@pytest.mark.parametrize("fa,fb", [(0.5, 0.5), (0.0, 0.75), (0.9, 0.9), (1.0, 0.3)])
def test_spgemm_against_the_oracle(dtype, fa, fb):
    run_spgemm(901, 136, 200, 320, dtype, fa, fb)


def test_spgemm_many_rows_and_long_lists():
    """More rows of B than one sweep of the warps covers, and column lists longer than one 32-entry look-up."""
    run_spgemm(911, 64, 2048, 1024, "bf16", 0.5, 0.5)


def test_spgemm_argument_errors():
    la = bsp.SparseLayer(64, 64, 1, 1, 8, 8, torch.bfloat16)
    lb = bsp.SparseLayer(64, 128, 1, 1, 8, 8, torch.bfloat16)
    Cm = torch.zeros((64, 64), dtype=torch.float32, device="cuda")
    with pytest.raises(bsp.BspError) as e:
        bsp.bsp_spgemm(la.wd, la.handle(), lb.wd, lb.handle(), Cm, la.ws)
    assert e.value.status == bsp.ERR_SHAPE                   # the reduction dimensions differ
    l4 = bsp.SparseLayer(64, 64, 1, 1, 4, 16, torch.bfloat16)
    with pytest.raises(bsp.BspError) as e:
        bsp.bsp_spgemm(la.wd, la.handle(), l4.wd, l4.handle(), Cm, la.ws)
    assert e.value.status == bsp.ERR_BLOCK


def test_relative_index_round_trip_bit_exact():
    W = make_case(921, 256, 1024, 1, 1, "bf16")
    gamma = synth.random_gamma(922, 32, 128, 2500)
    gamma[5, :] = 0                                          # an empty row
    lay = gpu_layer(W, gamma, 8, 8, "bf16")
    nnz = int(gamma.sum())
    rel = torch.full((nnz,), -1, dtype=torch.int32, device="cuda")
    back = torch.full((nnz,), -1, dtype=torch.int32, device="cuda")
    bsp.bsp_index_to_relative(32, lay.row_ptr, lay.col_idx, rel)
    bsp.bsp_index_from_relative(32, lay.row_ptr, rel, back)
    torch.cuda.synchronize()
    rp, ci, _ = ref.compact(W, gamma, 8, 8)
    assert np.array_equal(rel.cpu().numpy(), ref.index_to_relative(rp, ci))
    assert np.array_equal(back.cpu().numpy(), ci)
