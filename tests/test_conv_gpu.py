"""GPU parity: the CUDA library (through its C ABI) against the CPU oracle on the same seeded inputs.

Tolerances (global max norm over the whole output, both sides):
  fp32:  max|err| <= 1e-3 * max|ref|
  bf16 inputs, fp32 accumulation, bf16 outputs:  max|err| <= 2e-2 * max|ref|
A comparison is void unless at least 10 % of the reference outputs are non-zero.
"""
import numpy as np
import pytest
import torch

import oracle
import rt3d_synth as synth
import paper_2007_09835_b200 as rt3d
from paper_2007_09835_b200 import nets

pytestmark = pytest.mark.gpu

TOL = {torch.float32: 1e-3, torch.bfloat16: 2e-2}


def check(y, ref, dtype, what=""):
    assert y.shape == ref.shape, (y.shape, ref.shape)
    assert np.isfinite(y).all(), f"{what}: non-finite output"
    scale = np.abs(ref).max()
    assert (ref != 0).mean() >= 0.10, f"{what}: reference is mostly zero, comparison void"
    err = np.abs(y - ref).max()
    assert err <= TOL[dtype] * scale, f"{what}: max|err| {err:.4g} > {TOL[dtype]} * {scale:.4g}"
    return err / scale


def run_case(spec, n, t, h, w, g_m, g_n, mask_kind, mask_arg, dtype, algo, cfg=7, layer=0, dense=False,
             x_pitch=None, bias=True):
    L = synth.make_layer(spec, cfg, layer, g_m, g_n, mask_kind, mask_arg)
    x = synth.make_input(cfg * 100 + layer, (n, t, h, w, spec.cin))
    b = L["bias"] if bias else None
    ref = oracle.conv3d(x, L["w"], None if dense else L["mask"], b, spec.stride, spec.pad, spec.relu,
                        round_bf16=(dtype == torch.bfloat16))
    lay = nets.ConvLayer(spec, L["w"], b, L["mask"], g_m, g_n, dtype, dense=dense)
    xd = nets.to_device(x, dtype, x_pitch)
    y = lay(xd, algo=algo)
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    return nets.to_numpy(y, spec.cout), ref, lay, xd, y


# ----------------------------------------------------------------------- cfg0 (fp32)
@pytest.mark.parametrize("relu", [True, False])
def test_cfg0_fp32_kgs_14_of_27(relu):
    spec = synth.ConvSpec("cfg0", 16, 32, (3, 3, 3), (1, 1, 1), (1, 1, 1), relu)
    y, ref, *_ = run_case(spec, 1, 8, 28, 28, 4, 4, "exact_per_group", 14, torch.float32, rt3d.ALGO_AUTO, cfg=0)
    check(y, ref, torch.float32, "cfg0")


def test_cfg0_dense_path_fp32():
    spec = synth.ConvSpec("cfg0", 16, 32, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    y, ref, *_ = run_case(spec, 1, 8, 28, 28, 4, 4, "none", None, torch.float32, rt3d.ALGO_AUTO, cfg=0, dense=True)
    check(y, ref, torch.float32, "cfg0 dense")


# ------------------------------------------------------------- CUDA-core kernel, odd shapes
SIMT_CASES = [
    # cin, cout, k, stride, pad, (n,t,h,w), g_m, g_n, density
    (5, 6, (3, 3, 3), (1, 1, 1), (1, 1, 1), (2, 4, 5, 6), 4, 4, 0.5),
    (3, 45, (1, 7, 7), (1, 2, 2), (0, 3, 3), (1, 3, 20, 22), 4, 4, 0.4),
    (45, 64, (3, 1, 1), (1, 1, 1), (1, 0, 0), (1, 5, 6, 7), 4, 4, 0.4),
    (24, 40, (3, 3, 3), (2, 2, 2), (1, 1, 1), (1, 6, 9, 9), 8, 4, 0.3),
    (16, 16, (1, 1, 1), (2, 2, 2), (0, 0, 0), (2, 4, 6, 6), 8, 8, 0.6),
    (7, 9, (2, 2, 1), (1, 1, 1), (0, 1, 0), (1, 4, 4, 4), 3, 2, 0.5),
]


@pytest.mark.parametrize("case", SIMT_CASES)
@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_simt_kernel_against_oracle(case, dtype):
    cin, cout, k, stride, pad, (n, t, h, w), g_m, g_n, d = case
    spec = synth.ConvSpec("s", cin, cout, k, stride, pad, True)
    y, ref, *_ = run_case(spec, n, t, h, w, g_m, g_n, "bernoulli", d, dtype, rt3d.ALGO_SIMT)
    check(y, ref, dtype, f"simt {case}")


# ------------------------------------------------------------- tensor-core kernel, small shapes
UMMA_CASES = [
    # cin, cout, k, stride, pad, (n,t,h,w), g_m, g_n, density
    (64, 64, (3, 3, 3), (1, 1, 1), (1, 1, 1), (2, 4, 8, 8), 4, 4, 0.4),      # 4 full tiles
    (64, 64, (3, 3, 3), (1, 1, 1), (1, 1, 1), (1, 3, 7, 9), 4, 4, 0.4),      # ragged boxes
    (128, 256, (3, 3, 3), (1, 1, 1), (1, 1, 1), (1, 4, 12, 12), 4, 4, 0.4),  # 2 chunks, n_tile 256
    (96, 80, (3, 3, 3), (1, 1, 1), (1, 1, 1), (1, 2, 8, 8), 8, 4, 0.5),      # partial chunk, n_tile 80
    (144, 45, (3, 1, 1), (1, 1, 1), (1, 0, 0), (1, 6, 6, 6), 4, 4, 0.4),     # ragged M, 3x1x1
    (64, 512, (1, 1, 1), (1, 1, 1), (0, 0, 0), (2, 2, 9, 9), 8, 8, 0.5),     # two bundles, Ks = 1
    (3, 64, (3, 3, 3), (1, 1, 1), (1, 1, 1), (1, 4, 10, 10), 4, 4, 0.3),     # C_in = 3 (pitch 8)
    (64, 64, (1, 3, 3), (1, 1, 1), (0, 1, 1), (3, 5, 6, 6), 4, 4, 0.4),
]


@pytest.mark.parametrize("case", UMMA_CASES)
def test_umma_kernel_against_oracle(case):
    cin, cout, k, stride, pad, (n, t, h, w), g_m, g_n, d = case
    spec = synth.ConvSpec("u", cin, cout, k, stride, pad, True)
    y, ref, *_ = run_case(spec, n, t, h, w, g_m, g_n, "bernoulli", d, torch.bfloat16, rt3d.ALGO_UMMA)
    check(y, ref, torch.bfloat16, f"umma {case}")


SMALLC_CASES = [
    # C_in <= 8 at pitch 8, stride 1: the staged-halo kernel with location-pair MMAs
    (3, 64, (3, 3, 3), (1, 1, 1), (1, 1, 1), (2, 5, 33, 19), 4, 4, 0.3),     # ragged 16x8 tiles, several frames
    (3, 64, (3, 3, 3), (1, 1, 1), (1, 1, 1), (1, 3, 32, 16), 4, 4, 1.0),     # all 27 locations (odd count)
    (8, 45, (1, 7, 7), (1, 1, 1), (0, 3, 3), (1, 2, 20, 20), 4, 4, 0.5),     # 49 locations, ragged C_out
    (1, 16, (3, 1, 1), (1, 1, 1), (1, 0, 0), (1, 6, 9, 9), 4, 4, 0.7),
    (5, 256, (2, 2, 2), (1, 1, 1), (0, 0, 0), (1, 4, 18, 10), 8, 4, 0.5),    # no padding, even kernel
    (3, 32, (3, 3, 3), (1, 1, 1), (0, 1, 2), (1, 5, 17, 9), 4, 4, 0.05),     # very sparse: few pairs
    (3, 45, (1, 7, 7), (1, 2, 2), (0, 3, 3), (2, 3, 56, 40), 4, 4, 0.4),     # R(2+1)D stem: 4 stride phases
    (3, 64, (3, 3, 3), (2, 2, 2), (1, 1, 1), (1, 7, 35, 21), 4, 4, 0.6),     # strided in t, h and w, ragged
    (8, 32, (3, 5, 3), (1, 3, 1), (1, 2, 1), (1, 3, 50, 12), 8, 8, 0.5),     # stride 3 along h only
    (4, 16, (1, 2, 2), (1, 2, 2), (0, 0, 0), (1, 2, 32, 32), 4, 4, 1.0),     # kernel = stride: each phase one tap
]


@pytest.mark.parametrize("case", SMALLC_CASES)
def test_small_cin_kernel_against_oracle(case):
    cin, cout, k, stride, pad, (n, t, h, w), g_m, g_n, d = case
    spec = synth.ConvSpec("c", cin, cout, k, stride, pad, True)
    y, ref, lay, xd, yt = run_case(spec, n, t, h, w, g_m, g_n, "bernoulli", d, torch.bfloat16, rt3d.ALGO_UMMA)
    check(y, ref, torch.bfloat16, f"small-cin {case}")
    ys = nets.to_numpy(lay(xd, algo=rt3d.ALGO_SIMT), cout)
    check(ys, ref, torch.bfloat16, f"small-cin simt {case}")


def test_small_cin_padding_channels():
    """Channels 3..7 of a 3-channel input at pitch 8 are padding.  By default nothing the caller left there
    may reach the result; with x_pad_zero the caller vouches for zeros and the kernel fetches whole rows."""
    spec = synth.ConvSpec("c1", 3, 64, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    L = synth.make_layer(spec, 7, 21, 4, 4, "bernoulli", 0.4)
    x = synth.make_input(721, (2, 5, 21, 19, 3))
    ref = oracle.conv3d(x, L["w"], L["mask"], L["bias"], spec.stride, spec.pad, True, round_bf16=True)
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    xd = nets.to_device(x)
    y0 = lay(xd).clone()
    assert rt3d.rt3d_last_plan()["kernel"] == 3
    check(nets.to_numpy(y0, 64), ref, torch.bfloat16, "small-C default")
    y1 = lay(xd, x_pad_zero=True)
    assert rt3d.rt3d_last_plan()["kernel"] == 3
    assert torch.equal(y0, y1)                               # same arithmetic, only the loads differ
    dirty = xd.clone()
    dirty[..., 3:] = float("nan")                            # garbage in the padding channels
    y2 = lay(dirty)
    assert torch.equal(y0, y2)


def test_small_cin_bias_enters_through_the_accumulator():
    """The first-layer kernel adds the bias by one extra MMA (bias split into two bf16 terms) instead of in the
    epilogue.  The usual synthetic bias is too small for the layer tolerance to notice a wrong one, so: a bias
    of order 3 with full fp32 mantissas over a weak convolution; the result must be within half a bf16 step
    of the oracle's."""
    for cout, stride in ((64, (1, 1, 1)), (45, (1, 2, 2)), (24, (1, 1, 1))):
        spec = synth.ConvSpec("c1", 3, cout, (3, 3, 3), stride, (1, 1, 1), False)
        L = synth.make_layer(spec, 2, 31, 4, 4, "bernoulli", 0.5)
        bias = (np.random.default_rng(31).standard_normal(cout) * 3.0).astype(np.float32)
        w = (L["w"] * 0.01).astype(np.float32)
        x = synth.make_input(731, (2, 4, 32, 24, 3))
        ref = oracle.conv3d(x, w, L["mask"], bias, stride, (1, 1, 1), False, round_bf16=True)
        lay = nets.ConvLayer(spec, w, bias, L["mask"], 4, 4, torch.bfloat16)
        y = nets.to_numpy(lay(nets.to_device(x), x_pad_zero=True), cout)
        assert rt3d.rt3d_last_plan()["kernel"] == 3
        assert rt3d.rt3d_last_device_status() == rt3d.OK
        assert np.abs(y - ref).max() <= np.abs(ref).max() * 2.0 ** -8, (cout, stride)


def test_small_cin_all_pruned_outputs_bias():
    spec = synth.ConvSpec("c", 3, 32, (3, 3, 3), (1, 1, 1), (1, 1, 1), False)
    L = synth.make_layer(spec, 7, 4, 4, 4, "bernoulli", 0.5)
    L["mask"][:] = 0
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    y = nets.to_numpy(lay(nets.to_device(synth.make_input(704, (1, 2, 16, 8, 3))), algo=rt3d.ALGO_UMMA), 32)
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    np.testing.assert_array_equal(y, np.broadcast_to(oracle.bf16_round(L["bias"]), y.shape))


UMMA_STRIDED = [
    (64, 64, (3, 3, 3), (2, 2, 2), (1, 1, 1), (1, 6, 11, 12), 4, 4, 0.4),
    (64, 230, (1, 3, 3), (1, 2, 2), (0, 1, 1), (1, 4, 14, 14), 4, 4, 0.4),
    (230, 128, (3, 1, 1), (2, 1, 1), (1, 0, 0), (1, 8, 7, 7), 4, 4, 0.4),
    (64, 128, (1, 1, 1), (2, 2, 2), (0, 0, 0), (2, 4, 10, 10), 4, 4, 1.0),
    (3, 45, (1, 7, 7), (1, 2, 2), (0, 3, 3), (1, 2, 28, 28), 4, 4, 0.4),
]


@pytest.mark.parametrize("case", UMMA_STRIDED)
def test_umma_kernel_strided(case):
    cin, cout, k, stride, pad, (n, t, h, w), g_m, g_n, d = case
    spec = synth.ConvSpec("u", cin, cout, k, stride, pad, False)
    y, ref, *_ = run_case(spec, n, t, h, w, g_m, g_n, "bernoulli", d, torch.bfloat16, rt3d.ALGO_UMMA)
    check(y, ref, torch.bfloat16, f"umma strided {case}")


PAIR_CASES = [
    # CTA-pair kernel (two tiles per MMA, weight tile shared by the pair)
    (64, 64, (1, 1, 1), (1, 1, 1), (0, 0, 0), (1, 4, 8, 8), 4, 4, 0.5),        # one pair, one step
    (128, 256, (3, 3, 3), (1, 1, 1), (1, 1, 1), (1, 4, 12, 12), 4, 4, 0.4),    # odd tile count: dummy second tile
    (64, 512, (3, 3, 3), (2, 2, 2), (1, 1, 1), (1, 8, 20, 20), 8, 4, 0.4),     # two bundles, strided
    (96, 224, (1, 3, 3), (1, 1, 1), (0, 1, 1), (2, 3, 17, 15), 8, 8, 0.4),     # ragged boxes, partial chunk, n_tile 224
    (64, 45, (3, 1, 1), (1, 1, 1), (1, 0, 0), (1, 6, 10, 10), 4, 4, 0.4),      # n_tile 48: one 32-column piece + 16-column tail
]


@pytest.mark.parametrize("case", PAIR_CASES)
@pytest.mark.parametrize("dense", [False, True])
def test_umma_pair_kernel_against_oracle(case, dense):
    cin, cout, k, stride, pad, (n, t, h, w), g_m, g_n, d = case
    spec = synth.ConvSpec("p", cin, cout, k, stride, pad, True)
    y, ref, lay, xd, yt = run_case(spec, n, t, h, w, g_m, g_n, "none" if dense else "bernoulli", d, torch.bfloat16,
                                   rt3d.ALGO_UMMA_PAIR, dense=dense)
    check(y, ref, torch.bfloat16, f"pair {case}")
    y1 = nets.to_numpy(lay(xd, algo=rt3d.ALGO_UMMA), cout)      # single-CTA kernel (may split K: other sum order)
    check(y1, ref, torch.bfloat16, f"single {case}")
    assert np.abs(y1 - y).max() <= 1e-2 * np.abs(ref).max()


TAIL_CASES = [
    # more tile pairs than CTA pairs, a last round that is not full, and long K: the left-over tiles are cut
    # along K and shared by the pairs (fp32 partials through scratch, fixed summation order)
    (256, 256, (3, 3, 3), (4, 8, 28, 28), False),      # 98 tile pairs on 74 CTA pairs, one step per hand-shake
    (256, 512, (3, 3, 3), (2, 8, 28, 28), False),      # two bundles, left-over items all in the second
    (256, 128, (3, 3, 3), (4, 8, 28, 28), False),      # narrow bundle: two steps per hand-shake
    (256, 256, (3, 3, 3), (4, 8, 28, 28), True),       # dense path (computed steps)
    (256, 256, (3, 3, 3), (4, 8, 27, 29), False),      # ragged boxes
]


@pytest.mark.parametrize("case", TAIL_CASES)
def test_pair_kernel_tail_split_against_oracle(case):
    cin, cout, k, (n, t, h, w), dense = case
    spec = synth.ConvSpec("t", cin, cout, k, (1, 1, 1), tuple(kk // 2 for kk in k), True)
    y, ref, lay, xd, yt = run_case(spec, n, t, h, w, 4, 4, "none" if dense else "bernoulli", 0.4, torch.bfloat16,
                                   rt3d.ALGO_AUTO, dense=dense)
    plan = rt3d.rt3d_last_plan()
    assert plan["kernel"] in (2, 7) and plan["tail_workers"] > 0, plan     # 7: narrow bundle, one deeper input tile per kt group
    check(y, ref, torch.bfloat16, f"tail split {case}")
    first = yt.clone()
    for _ in range(3):                       # flags reset themselves; the sum order is fixed
        lay(xd, yt)
        torch.cuda.synchronize()
        assert torch.equal(first, yt)
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    y1 = nets.to_numpy(lay(xd, algo=rt3d.ALGO_UMMA), cout)      # single-CTA kernel: whole tiles, other sum order
    assert rt3d.rt3d_last_plan()["kernel"] == 1
    assert np.abs(y1 - y).max() <= 1e-2 * np.abs(ref).max()


HALO_CASES = [
    # resident-weight kernel for thin stride-1 layers: cin, cout, k, pad, (n,t,h,w), dense
    (64, 144, (1, 3, 3), (0, 1, 1), (2, 4, 24, 20), False),     # R(2+1)D stage-2 spatial conv; ragged tiles
    (144, 64, (3, 1, 1), (1, 0, 0), (2, 6, 12, 16), False),     # its temporal conv: partial last chunk, tile 16 frames deep
    (45, 64, (3, 1, 1), (1, 0, 0), (1, 5, 9, 11), False),       # stem temporal conv: 45 channels at pitch 48
    (32, 32, (3, 3, 3), (1, 1, 1), (1, 4, 20, 12), False),      # 3x3x3: block of 3 x 18 x 10 voxels
    (64, 128, (1, 1, 1), (0, 0, 0), (3, 3, 17, 9), False),      # one location: no halo; odd tile count
    (64, 144, (1, 3, 3), (0, 1, 1), (1, 3, 16, 16), True),      # dense path (computed steps)
    (64, 96, (1, 3, 3), (0, 0, 0), (1, 2, 19, 21), False),      # no padding: output smaller than input
    (128, 64, (3, 1, 1), (0, 0, 0), (1, 9, 8, 8), False),       # two full chunks, no temporal padding
]


@pytest.mark.parametrize("case", HALO_CASES)
def test_umma_halo_kernel_against_oracle(case):
    cin, cout, k, pad, (n, t, h, w), dense = case
    spec = synth.ConvSpec("h", cin, cout, k, (1, 1, 1), pad, True)
    y, ref, lay, xd, yt = run_case(spec, n, t, h, w, 4, 4, "none" if dense else "bernoulli", 0.4, torch.bfloat16,
                                   rt3d.ALGO_UMMA_HALO, dense=dense)
    assert rt3d.rt3d_last_plan()["kernel"] == 4
    check(y, ref, torch.bfloat16, f"halo {case}")
    y1 = nets.to_numpy(lay(xd, algo=rt3d.ALGO_UMMA), cout)      # step-per-location kernel, same weights
    assert rt3d.rt3d_last_plan()["kernel"] in (1, 2)
    assert np.abs(y1 - y).max() <= 1e-2 * np.abs(ref).max()


def test_umma_halo_kernel_refusals_and_auto_choice():
    big = synth.ConvSpec("h", 128, 256, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)          # weights far beyond shared memory
    L = synth.make_layer(big, 7, 1, 4, 4, "bernoulli", 0.4)
    lay = nets.ConvLayer(big, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    xd = nets.to_device(synth.make_input(1, (1, 2, 8, 8, 128)))
    with pytest.raises(rt3d.Rt3dError) as e:
        lay(xd, algo=rt3d.ALGO_UMMA_HALO)
    assert e.value.status == rt3d.ERR_UNSUPPORTED
    strided = synth.ConvSpec("h", 64, 64, (1, 3, 3), (1, 2, 2), (0, 1, 1), True)
    L = synth.make_layer(strided, 7, 2, 4, 4, "bernoulli", 0.4)
    lay = nets.ConvLayer(strided, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    with pytest.raises(rt3d.Rt3dError) as e:
        lay(nets.to_device(synth.make_input(1, (1, 2, 16, 16, 64))), algo=rt3d.ALGO_UMMA_HALO)
    assert e.value.status == rt3d.ERR_UNSUPPORTED
    # a thin layer with at least one tile per SM: the library picks the resident-weight kernel by itself
    thin = synth.ConvSpec("h", 64, 144, (1, 3, 3), (1, 1, 1), (0, 1, 1), True)
    L = synth.make_layer(thin, 7, 3, 4, 4, "bernoulli", 0.4)
    lay = nets.ConvLayer(thin, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    x = synth.make_input(2, (2, 4, 48, 56, 64))
    y = nets.to_numpy(lay(nets.to_device(x)), 144)
    assert rt3d.rt3d_last_plan()["kernel"] == 4
    ref = oracle.conv3d(x, L["w"], L["mask"], L["bias"], thin.stride, thin.pad, True, round_bf16=True)
    check(y, ref, torch.bfloat16, "halo auto")


WIDE_GROUP_CASES = [
    # kernel groups matched to the tensor-core footprint (beyond the paper's 4..8): exact step skipping
    (256, 256, (3, 3, 3), (2, 8, 14, 14), 256, 64, 0.25),
    (256, 256, (3, 3, 3), (2, 8, 14, 14), 128, 64, 0.25),
    (128, 256, (3, 3, 3), (4, 8, 14, 14), 64, 64, 0.5),
    (192, 160, (1, 3, 3), (2, 4, 14, 14), 32, 16, 0.3),
    (256, 256, (3, 3, 3), (1, 2, 7, 7), 256, 64, 0.125),       # few tiles: K split over short lists
]


@pytest.mark.parametrize("case", WIDE_GROUP_CASES)
def test_wide_kernel_groups_against_oracle(case):
    cin, cout, k, (n, t, h, w), g_m, g_n, d = case
    spec = synth.ConvSpec("g", cin, cout, k, (1, 1, 1), tuple(kk // 2 for kk in k), True)
    y, ref, lay, xd, yt = run_case(spec, n, t, h, w, g_m, g_n, "bernoulli", d, torch.bfloat16, rt3d.ALGO_AUTO)
    check(y, ref, torch.bfloat16, f"wide groups {case}")
    with pytest.raises(rt3d.Rt3dError) as e:               # the CUDA-core kernel stops at 8 x 8 groups
        lay(xd, algo=rt3d.ALGO_SIMT)
    assert e.value.status == rt3d.ERR_UNSUPPORTED


SPLITK_CASES = [
    # few output tiles, long K: the tensor-core kernel splits K across CTAs and reduces fp32 partials
    (256, 256, (3, 3, 3), (1, 1, 1), (1, 1, 1), (1, 2, 7, 7), 4, 4, 0.4),
    (512, 512, (3, 3, 3), (1, 1, 1), (1, 1, 1), (2, 2, 7, 7), 4, 4, 0.3),
    (192, 230, (3, 3, 3), (1, 1, 1), (1, 1, 1), (1, 4, 9, 9), 8, 4, 0.4),      # ragged C_out, 3 m-tiles
    (576, 96, (3, 1, 1), (1, 1, 1), (1, 0, 0), (1, 4, 7, 7), 4, 4, 0.4),
]


@pytest.mark.parametrize("case", SPLITK_CASES)
@pytest.mark.parametrize("dense", [False, True])
def test_umma_split_k_against_oracle(case, dense):
    cin, cout, k, stride, pad, (n, t, h, w), g_m, g_n, d = case
    spec = synth.ConvSpec("k", cin, cout, k, stride, pad, True)
    y, ref, lay, xd, yt = run_case(spec, n, t, h, w, g_m, g_n, "none" if dense else "bernoulli", d, torch.bfloat16,
                                   rt3d.ALGO_UMMA, dense=dense)
    check(y, ref, torch.bfloat16, f"split-k {case}")
    first = yt.clone()
    for _ in range(3):                       # arrival counters reset themselves; the sum order is fixed
        lay(xd, yt, algo=rt3d.ALGO_UMMA)
        torch.cuda.synchronize()
        assert torch.equal(first, yt)
    assert rt3d.rt3d_last_device_status() == rt3d.OK


def test_umma_dense_entry_point():
    spec = synth.ConvSpec("u", 128, 128, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    y, ref, *_ = run_case(spec, 2, 4, 8, 8, 4, 4, "none", None, torch.bfloat16, rt3d.ALGO_UMMA, dense=True)
    check(y, ref, torch.bfloat16, "umma dense")


def test_umma_bundle_with_every_group_pruned_outputs_bias():
    spec = synth.ConvSpec("u", 64, 512, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    L = synth.make_layer(spec, 7, 3, 4, 4, "bernoulli", 0.4)
    L["mask"][256:] = 0                                   # second bundle of 256 channels: nothing kept
    x = synth.make_input(703, (1, 2, 8, 8, 64))
    ref = oracle.conv3d(x, L["w"], L["mask"], L["bias"], spec.stride, spec.pad, True, round_bf16=True)
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    y = nets.to_numpy(lay(nets.to_device(x), algo=rt3d.ALGO_UMMA), 512)
    check(y, ref, torch.bfloat16, "empty bundle")
    np.testing.assert_allclose(y[..., 256:], np.broadcast_to(np.maximum(L["bias"][256:], 0), y[..., 256:].shape),
                               rtol=1e-2, atol=1e-4)


def test_umma_and_simt_agree_and_are_deterministic():
    spec = synth.ConvSpec("u", 128, 64, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    y1, ref, lay, xd, yt = run_case(spec, 1, 4, 10, 10, 4, 4, "bernoulli", 0.4, torch.bfloat16, rt3d.ALGO_UMMA)
    first = yt.clone()
    lay(xd, yt, algo=rt3d.ALGO_UMMA)
    torch.cuda.synchronize()
    assert torch.equal(first, yt)                          # no atomics, no split-K: bitwise repeatable
    ys = nets.to_numpy(lay(xd, algo=rt3d.ALGO_SIMT), 64)
    check(ys, ref, torch.bfloat16, "simt")
    assert np.abs(ys - y1).max() <= 2e-2 * np.abs(ref).max()


def test_output_pitch_guard_band_untouched():
    spec = synth.ConvSpec("u", 64, 40, (3, 3, 3), (1, 1, 1), (1, 1, 1), False)
    L = synth.make_layer(spec, 7, 5, 4, 4, "bernoulli", 0.5)
    x = synth.make_input(705, (1, 2, 6, 6, 64))
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    for algo in (rt3d.ALGO_UMMA, rt3d.ALGO_SIMT):
        y = torch.full((1, 2, 6, 6, 48), 777.0, dtype=torch.bfloat16, device="cuda")   # pitch 48 > 40 channels
        lay(nets.to_device(x), y, algo=algo)
        torch.cuda.synchronize()
        assert (y[..., 40:] == 777.0).all()
        ref = oracle.conv3d(x, L["w"], L["mask"], L["bias"], spec.stride, spec.pad, False, round_bf16=True)
        check(nets.to_numpy(y, 40), ref, torch.bfloat16, "pitch")


# ------------------------------------------------------------------------- cfg1, full size
@pytest.mark.parametrize("mode", ["kgs", "dense", "vanilla"])
def test_cfg1_c3d_conv3a_full_size(mode):
    spec = synth.ConvSpec("conv3a", 128, 256, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    if mode == "kgs":
        args = ("bernoulli", 0.4)
    elif mode == "vanilla":
        args = ("vanilla_total", round(64 * 32 * 0.4))
    else:
        args = ("none", None)
    y, ref, *_ = run_case(spec, 8, 8, 28, 28, 4, 4, *args, torch.bfloat16, rt3d.ALGO_AUTO, cfg=1,
                          dense=(mode == "dense"))
    rel = check(y, ref, torch.bfloat16, f"cfg1 {mode}")
    assert rel < 1e-2
    assert rt3d.rt3d_last_plan()["kernel"] in (2, 7)           # CTA pairs: 196 tile pairs on 74 pairs of SMs


# ------------------------------------------------------------------ host entry point, glue
def test_conv3d_host_entry_point_matches_device_call():
    spec = synth.ConvSpec("h", 64, 64, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    L = synth.make_layer(spec, 7, 9, 4, 4, "bernoulli", 0.4)
    x = synth.make_input(709, (2, 4, 8, 8, 64))
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    yd = lay(nets.to_device(x))
    xh = torch.from_numpy(x).to(torch.bfloat16).pin_memory()
    yh = torch.zeros((2, 4, 8, 8, 64), dtype=torch.bfloat16).pin_memory()
    bh = torch.from_numpy(L["bias"]).pin_memory()
    rt3d.rt3d_conv3d_host(rt3d.tensor_desc(xh), lay.packed, bh, rt3d.tensor_desc(yh), spec.stride, spec.pad, True)
    assert torch.equal(yh, yd.cpu())


def test_conv3d_host_entry_point_pipelines_large_batches_in_chunks():
    """Above 8 MiB the host entry point copies, convolves and copies back chunks of whole clips on three
    streams.  Every output element must arrive, in the right place (11 clips = chunks of one or two clips)."""
    spec = synth.ConvSpec("h", 64, 128, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    L = synth.make_layer(spec, 7, 10, 4, 4, "bernoulli", 0.4)
    x = synth.make_input(710, (11, 4, 28, 28, 64))
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, torch.bfloat16)
    yd = lay(nets.to_device(x)).cpu().float()
    xh = torch.from_numpy(x).to(torch.bfloat16).pin_memory()
    yh = torch.full((11, 4, 28, 28, 128), 55.0, dtype=torch.bfloat16).pin_memory()
    bh = torch.from_numpy(L["bias"]).pin_memory()
    launches = rt3d.rt3d_launch_count()
    for _ in range(2):                                   # the second call reuses streams, events and staging
        rt3d.rt3d_conv3d_host(rt3d.tensor_desc(xh), lay.packed, bh, rt3d.tensor_desc(yh), spec.stride, spec.pad, True)
    assert rt3d.rt3d_launch_count() - launches == 16     # eight chunks per call
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    assert (yd != 0).float().mean() > 0.1
    assert (yh.float() - yd).abs().max() <= 1e-2 * yd.abs().max()
    ref0 = oracle.conv3d(x[10:], L["w"], L["mask"], L["bias"], spec.stride, spec.pad, True, round_bf16=True)
    check(yh[10:].float().numpy(), ref0, torch.bfloat16, "host path, last clip")


def test_maxpool_and_add_relu_against_oracle():
    for dtype in (torch.bfloat16, torch.float32):
        for c, shape, pool in ((64, (2, 4, 8, 8), synth.PoolSpec("p", (2, 2, 2), (2, 2, 2), (0, 0, 0))),
                               (64, (1, 3, 14, 14), synth.PoolSpec("p", (1, 2, 2), (1, 2, 2), (0, 0, 0))),
                               (16, (1, 2, 7, 7), synth.PoolSpec("p", (2, 2, 2), (2, 2, 2), (0, 1, 1))),
                               (5, (1, 2, 6, 6), synth.PoolSpec("p", (2, 2, 2), (2, 2, 2), (0, 0, 0))),
                               # unit stride along w: four outputs per thread share their column maxima
                               (32, (2, 5, 9, 13), synth.PoolSpec("p", (3, 3, 3), (1, 1, 1), (1, 1, 1))),
                               (16, (1, 4, 7, 4), synth.PoolSpec("p", (3, 3, 3), (1, 1, 1), (1, 1, 1))),
                               (16, (1, 4, 7, 3), synth.PoolSpec("p", (3, 3, 3), (1, 1, 1), (1, 1, 1))),
                               (24, (2, 6, 11, 10), synth.PoolSpec("p", (3, 3, 3), (2, 2, 1), (1, 1, 1))),
                               (8, (1, 3, 12, 17), synth.PoolSpec("p", (1, 3, 3), (1, 1, 1), (0, 1, 1))),
                               (8, (1, 3, 12, 17), synth.PoolSpec("p", (1, 3, 3), (1, 2, 1), (0, 0, 0)))):
            x = synth.make_input(800 + c, shape + (c,))
            xr = oracle.bf16_round(x) if dtype == torch.bfloat16 else x
            y = nets.to_numpy(nets.maxpool(nets.to_device(x, dtype), c, pool), c)
            np.testing.assert_array_equal(y, oracle.maxpool3d(xr, pool.k, pool.stride, pool.pad))
        a = synth.make_input(901, (2, 3, 5, 5, 24))
        b = synth.make_input(902, (2, 3, 5, 5, 24))
        ar, br = (oracle.bf16_round(a), oracle.bf16_round(b)) if dtype == torch.bfloat16 else (a, b)
        for relu in (True, False):
            y = nets.to_numpy(nets.add_relu(nets.to_device(a, dtype), nets.to_device(b, dtype), 24, relu), 24)
            ref = oracle.add_relu(ar, br, relu)
            if dtype == torch.bfloat16:
                ref = oracle.bf16_round(ref)
            np.testing.assert_array_equal(y, ref)


def test_cost_model_counts_kept_macs():
    spec = synth.ConvSpec("c", 16, 32, (3, 3, 3), (1, 1, 1), (1, 1, 1), True)
    L = synth.make_layer(spec, 0, 0, 4, 4, "exact_per_group", 14)
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 4, 4, torch.float32)
    x = nets.to_device(synth.make_input(0, (1, 8, 28, 28, 16)), torch.float32)
    kept, dense, nbytes = lay.cost(x)
    assert dense == spec.dense_macs(1, 8, 28, 28)
    assert kept * 27 == dense * 14
    assert nbytes == (6272 * 16 + 6272 * 32) * 4 + 448 * 16 * 4 + 448 * 2 + 33 * 4 + 32 * 4


@pytest.mark.parametrize("algo", ["auto", "pair", "simt"])
def test_padding_channels_of_the_output(algo):
    """300 output channels at a pitch of 320: the padding channels 304..319 must be left alone by every kernel; the four
    padding channels that share the last 16-byte unit of a row with channels 296..299 are either left alone (CUDA-core
    kernel, per-element stores) or written as zeros (bulk stores of the tensor-core kernels move whole units)."""
    spec = synth.ConvSpec("pad", 16, 300, (1, 3, 2), (1, 2, 1), (0, 1, 1), True)
    L = synth.make_layer(spec, 51, 58, 8, 8, "bernoulli", 0.2)
    x = synth.make_input(6158, (8, 4, 32, 9, 16))
    ref = oracle.conv3d(x, L["w"], L["mask"], L["bias"], spec.stride, spec.pad, True, round_bf16=True)
    lay = nets.ConvLayer(spec, L["w"], L["bias"], L["mask"], 8, 8, torch.bfloat16)
    xd = nets.to_device(x)
    y = torch.full(tuple(lay.out_shape(xd)[:4]) + (320,), 9.0, dtype=torch.bfloat16, device="cuda")
    lay(xd, y, algo={"auto": rt3d.ALGO_AUTO, "pair": rt3d.ALGO_UMMA_PAIR, "simt": rt3d.ALGO_SIMT}[algo])
    assert rt3d.rt3d_last_device_status() == rt3d.OK
    check(nets.to_numpy(y, 300), ref, torch.bfloat16, f"padding {algo}")
    assert (y[..., 304:] == 9.0).all()
    unit = y[..., 300:304]
    assert ((unit == 9.0) | (unit == 0.0)).all()
    if algo == "simt":
        assert (unit == 9.0).all()
