"""GPU parity: Gamma builder and compaction against the CPU oracle, bit for bit, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import ref
from paper_2407_09453_b200 import bsp, synth
from gpu_util import gpu_layer, gpu_mask, from_dev, make_case, to_dev, TORCH_DT

pytestmark = pytest.mark.gpu

SHAPES = [(8, 8), (4, 16), (16, 4)]


@pytest.mark.parametrize("dtype", ["bf16", "f32", "i8"])
@pytest.mark.parametrize("bo,bi", SHAPES)
@pytest.mark.parametrize("norm", [bsp.NORM_L2, bsp.NORM_L1])
def test_scores_and_gamma_bit_exact(dtype, bo, bi, norm):
    O, I, H, K = 96, 160, 3, 3
    W = make_case(101, O, I, H, K, dtype)
    NB = (O // bo) * (I // bi)
    want_s = ref.scores(W, bo, bi, norm)
    for n_zero in (NB // 2, 1, NB - 1):
        g, s, _, _ = gpu_mask(W, bo, bi, dtype, n_zero, norm)
        assert np.array_equal(s.view(np.uint64), want_s.view(np.uint64))      # identical bit patterns
        assert np.array_equal(g, ref.mask(want_s, n_zero))
        assert int((g == 0).sum()) == n_zero                                   # Eq. (2)


@pytest.mark.parametrize("dtype", ["bf16", "i8"])
def test_gamma_row_scope_and_extremes(dtype):
    bo = bi = 8
    O, I, H, K = 64, 256, 1, 1
    W = make_case(103, O, I, H, K, dtype)
    want_s = ref.scores(W, bo, bi)
    g, s, _, _ = gpu_mask(W, bo, bi, dtype, 9, scope=bsp.SCOPE_ROW)
    assert np.array_equal(g, ref.mask(want_s, 9, ref.SCOPE_ROW)) and np.all((g == 0).sum(axis=1) == 9)
    for n_zero in (0, 32):
        g, _, _, _ = gpu_mask(W, bo, bi, dtype, n_zero, scope=bsp.SCOPE_ROW)
        assert np.all(g == (1 if n_zero == 0 else 0))
    NB = g.size
    assert gpu_mask(W, bo, bi, dtype, 0)[0].all() and not gpu_mask(W, bo, bi, dtype, NB)[0].any()


def test_gamma_ties_broken_by_index():
    """int8 scores collide all the time; equal weights make every score equal."""
    bo = bi = 8
    W = np.full((64, 1, 1, 64), 5, dtype=np.int8)
    g, s, _, _ = gpu_mask(W, bo, bi, "i8", 23)
    assert np.array_equal(g.ravel(), np.r_[np.zeros(23, np.uint8), np.ones(41, np.uint8)])
    W = synth.uniform_int(107, (128, 1, 1, 256), -3, 3).astype(np.int8)        # few distinct scores
    want_s = ref.scores(W, bo, bi)
    assert len(np.unique(want_s)) < want_s.size // 2
    for n_zero in (100, 256, 301):
        g, s, _, _ = gpu_mask(W, bo, bi, "i8", n_zero)
        assert np.array_equal(g, ref.mask(want_s, n_zero))


def test_gamma_ties_in_a_layer_of_many_blocks():
    """8192 blocks with few distinct int8 scores: the multi-CTA select must zero equal keys lowest index first,
    across the slices of different CTAs."""
    bo = bi = 8
    W = synth.uniform_int(131, (512, 1, 1, 1024), -3, 3).astype(np.int8)
    want_s = ref.scores(W, bo, bi)
    assert len(np.unique(want_s)) < want_s.size // 8
    for n_zero in (1, 4097, want_s.size - 1):
        g, s, _, _ = gpu_mask(W, bo, bi, "i8", n_zero)
        assert np.array_equal(g, ref.mask(want_s, n_zero))
    g, _, _, _ = gpu_mask(W, bo, bi, "i8", 40, scope=bsp.SCOPE_ROW)
    assert np.array_equal(g, ref.mask(want_s, 40, ref.SCOPE_ROW))


def test_gamma_large_layer_many_select_passes():
    """More blocks than one pass of the selecting CTA covers (4096x2048 / 8x8 = 131072 blocks)."""
    bo = bi = 8
    W = synth.round_to_bf16(synth.normal(109, (2048, 1, 1, 1024), 1 / 32.0).astype(np.float32))
    want_s = ref.scores(W, bo, bi)
    g, s, _, _ = gpu_mask(W, bo, bi, "bf16", want_s.size // 2)
    assert np.array_equal(s.view(np.uint64), want_s.view(np.uint64))
    assert np.array_equal(g, ref.mask(want_s, want_s.size // 2))


@pytest.mark.parametrize("dtype", ["bf16", "f32", "i8"])
@pytest.mark.parametrize("bo,bi", SHAPES)
def test_compact_bit_exact(dtype, bo, bi):
    O, I, H, K = 128, 96, 3, 2
    W = make_case(113, O, I, H, K, dtype)
    NBo, NBi = O // bo, I // bi
    for nz in ((NBo * NBi) // 2, 0, NBo * NBi, 5):
        gamma = synth.random_gamma(115 + nz, NBo, NBi, nz)
        lay = gpu_layer(W, gamma, bo, bi, dtype)
        rp, ci, pl = ref.compact(W, gamma, bo, bi)
        nnz = len(ci)
        assert np.array_equal(from_dev(lay.row_ptr), rp)
        assert np.array_equal(from_dev(lay.col_idx)[:nnz], ci)
        got = from_dev(lay.payload)[:pl.size].reshape(pl.shape)
        assert np.array_equal(got, pl if dtype != "bf16" else pl.astype(np.float32))
        assert bsp.bsp_compact_nnz(lay.wd, lay.gamma, lay.ws) == nnz


@pytest.mark.parametrize("dtype", ["bf16", "i8"])
@pytest.mark.parametrize("bo,bi", SHAPES)
def test_compact_more_blocks_than_the_single_launch_path_takes(dtype, bo, bi):
    """8192 blocks: the count / scan / fill launches instead of the one-launch kernel of small layers."""
    O, I, H, K = 512, 1024, 1, 1
    W = make_case(123, O, I, H, K, dtype)
    NBo, NBi = O // bo, I // bi
    assert NBo * NBi > 4096
    gamma = synth.random_gamma(125, NBo, NBi, (NBo * NBi) // 3)
    lay = gpu_layer(W, gamma, bo, bi, dtype)
    rp, ci, pl = ref.compact(W, gamma, bo, bi)
    assert np.array_equal(from_dev(lay.row_ptr), rp)
    assert np.array_equal(from_dev(lay.col_idx)[:len(ci)], ci)
    got = from_dev(lay.payload)[:pl.size].reshape(pl.shape)
    assert np.array_equal(got, pl if dtype != "bf16" else pl.astype(np.float32))


@pytest.mark.parametrize("dtype", ["bf16", "i8", "f32"])
def test_mask_and_compact_of_weights_at_an_odd_address(dtype):
    """W starting four bytes into an allocation: the 16-byte loads of the score and copy loops must give way to
    narrower ones, with the same bits out; an address that is not a multiple of four is refused."""
    bo = bi = 8
    O, I, H, K = 64, 72, 3, 3
    W = make_case(127, O, I, H, K, dtype)
    skip = {"bf16": 2, "i8": 4, "f32": 1}[dtype]
    big = torch.empty(W.size + 16, dtype=TORCH_DT[dtype], device="cuda")
    Wd = big[skip:skip + W.size].view(O, H, K, I)
    Wd.copy_(to_dev(W, dtype))
    assert Wd.data_ptr() % 16 == 4
    lay = bsp.SparseLayer(O, I, H, K, bo, bi, TORCH_DT[dtype])
    if dtype != "f32":
        odd = big[1:1 + W.size].view(O, H, K, I)
        with pytest.raises(bsp.BspError) as e:
            lay.mask(odd, 1)
        assert e.value.status == bsp.ERR_SHAPE
    sc = torch.empty(lay.NBo * lay.NBi, dtype=torch.int64 if dtype == "i8" else torch.float64, device="cuda")
    n_zero = lay.NBo * lay.NBi // 2
    lay.mask(Wd, n_zero, scores=sc)
    lay.compact(Wd)
    lay.check()
    want_s = ref.scores(W, bo, bi)
    assert np.array_equal(from_dev(sc).view(np.uint64), want_s.reshape(-1).view(np.uint64))
    g = ref.mask(want_s, n_zero)
    assert np.array_equal(from_dev(lay.gamma).reshape(g.shape), g)
    rp, ci, pl = ref.compact(W, g, bo, bi)
    assert np.array_equal(from_dev(lay.row_ptr), rp) and np.array_equal(from_dev(lay.col_idx)[:len(ci)], ci)
    got = from_dev(lay.payload)[:pl.size].reshape(pl.shape)
    assert np.array_equal(got, pl if dtype != "bf16" else pl.astype(np.float32))


def test_compact_capacity_overflow_is_latched():
    bo = bi = 8
    W = make_case(117, 64, 64, 1, 1, "bf16")
    lay = bsp.SparseLayer(64, 64, 1, 1, bo, bi, torch.bfloat16, capacity_blocks=10)
    gamma = synth.random_gamma(119, 8, 8, 32)
    lay.compact(to_dev(W, "bf16"), torch.from_numpy(gamma).cuda())
    with pytest.raises(bsp.BspError) as e:
        lay.check()
    assert e.value.status == bsp.ERR_CAPACITY
    lay.check()                                                                # cleared after being read


def test_mask_then_compact_round_trip_to_masked_dense():
    bo = bi = 8
    O, I, H, K = 256, 256, 3, 3
    W = make_case(121, O, I, H, K, "bf16")
    g, s, lay, Wd = gpu_mask(W, bo, bi, "bf16", 512)
    lay.compact(Wd)
    lay.check()
    rp, ci = from_dev(lay.row_ptr), from_dev(lay.col_idx)
    pl = from_dev(lay.payload).reshape(-1, bo, H, K, bi)
    back = np.zeros_like(W)
    for l in range(O // bo):
        for n in range(rp[l], rp[l + 1]):
            back[l * bo:(l + 1) * bo, :, :, ci[n] * bi:(ci[n] + 1) * bi] = pl[n]
    assert rp[-1] == 512 and np.array_equal(back, ref.apply_mask(W, g, bo, bi))


@pytest.mark.parametrize("dtype", ["bf16", "f32"])
@pytest.mark.parametrize("bo,bi", SHAPES)
@pytest.mark.parametrize("H,K,O,I", [(3, 3, 96, 160), (1, 1, 256, 512), (1, 7, 32, 64)])
def test_variance_scores_and_gamma_bit_exact(dtype, bo, bi, H, K, O, I):
    """Variance importance (float weights): blocks get their own offsets so that the mean matters and the ranking
    differs from the L2 one; scores are compared as bit patterns (the kernel keeps the oracle's order of the sums and
    rounds the subtraction, the square and the addition one by one), Gamma bit for bit."""
    W = make_case(131, O, I, H, K, dtype)
    NBo, NBi = O // bo, I // bi
    shift = synth.normal(132, (NBo, NBi), 0.05).astype(np.float32)
    W = W + np.repeat(np.repeat(shift, bo, axis=0), bi, axis=1)[:, None, None, :]
    W = synth.round_to_bf16(W.astype(np.float32)) if dtype == "bf16" else W.astype(np.float32)
    want_s = ref.scores(W, bo, bi, ref.NORM_VAR)
    NB = NBo * NBi
    g, s, _, _ = gpu_mask(W, bo, bi, dtype, NB // 2, bsp.NORM_VAR)
    assert np.array_equal(s.view(np.uint64), want_s.view(np.uint64))
    want_g = ref.mask(want_s, NB // 2)
    assert np.array_equal(g, want_g)
    assert not np.array_equal(want_g, ref.mask(ref.scores(W, bo, bi, ref.NORM_L2), NB // 2))
    g_row, _, _, _ = gpu_mask(W, bo, bi, dtype, 3, bsp.NORM_VAR, bsp.SCOPE_ROW)
    assert np.array_equal(g_row, ref.mask(want_s, 3, ref.SCOPE_ROW))


def test_variance_of_int8_weights_is_refused():
    W = make_case(133, 64, 64, 1, 1, "i8")
    with pytest.raises(bsp.BspError) as e:
        gpu_mask(W, 8, 8, "i8", 4, bsp.NORM_VAR)
    assert e.value.status == bsp.ERR_DTYPE


def test_bounded_wait_runs_out_and_the_workspace_recovers():
    """A wait that nothing can satisfy ends by itself: the arrival word of the grid barrier in the workspace header is
    preset (by the host: the contract says it starts at zero) so that no CTA of the one-launch Gamma builder ever counts
    as the last arriver.  Every CTA's bounded wait expires, the kernel returns, bsp_check reports BSP_ERR_TIMEOUT once and
    clears the barrier words, and the next call on the same workspace is bit-exact."""
    W = make_case(141, 128, 128, 3, 3, "bf16")
    lay = bsp.SparseLayer(128, 128, 3, 3, 8, 8, torch.bfloat16)
    Wd = to_dev(W, "bf16")
    lay.ws.view(torch.int32)[2] = 0x40000000          # arrivals so far: far more than any grid
    lay.mask(Wd, 128)
    with pytest.raises(bsp.BspError) as e:
        lay.check()
    assert e.value.status == bsp.ERR_TIMEOUT
    assert lay.ws.view(torch.int32)[:4].abs().sum().item() == 0      # status and barrier words cleared by bsp_check
    lay.check()
    lay.mask(Wd, 128)
    lay.check()
    want = ref.mask(ref.scores(W, 8, 8), 128)
    assert np.array_equal(from_dev(lay.gamma).reshape(16, 16), want)
