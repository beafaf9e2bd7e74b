"""Host logic of the library (no GPU): rt3d_pack_kgs against the oracle's pack, bit for bit;
the derived tensor-core weight layout against the canonical arrays; argument errors."""
import numpy as np
import pytest

import oracle
import rt3d_synth as synth
import paper_2007_09835_b200 as rt3d


def _layer(M, N, k, g_m, g_n, density, seed):
    spec = synth.ConvSpec("t", N, M, k, (1, 1, 1), (0, 0, 0))
    return synth.make_layer(spec, 9, seed, g_m, g_n, "bernoulli", density)


@pytest.mark.parametrize("M,N,k,g_m,g_n", [(32, 16, (3, 3, 3), 4, 4), (6, 5, (3, 3, 3), 4, 4), (64, 64, (3, 3, 3), 8, 4),
                                           (45, 3, (1, 7, 7), 4, 4), (40, 24, (3, 1, 1), 8, 8), (7, 9, (2, 2, 1), 3, 2),
                                           (128, 128, (3, 3, 3), 64, 64), (200, 70, (1, 3, 3), 128, 16)])
@pytest.mark.parametrize("dtype", [rt3d.RT3D_F32, rt3d.RT3D_BF16])
def test_pack_bit_exact_against_oracle(M, N, k, g_m, g_n, dtype):
    L = _layer(M, N, k, g_m, g_n, 0.4, M + N)
    ref = oracle.pack_kgs(L["w"], L["mask"], g_m, g_n, to_bf16=(dtype == rt3d.RT3D_BF16))
    got = rt3d.rt3d_pack_kgs(L["w"], L["mask"], g_m, g_n, dtype).view()
    assert got["nnz"] == ref["nnz"] and got["P"] == ref["P"] and got["Q"] == ref["Q"] and got["Ks"] == ref["Ks"]
    assert bool(got["is_vanilla"]) == ref["is_vanilla"]
    assert got["group_ptr"].tobytes() == ref["group_ptr"].tobytes()
    assert got["pos_idx"].tobytes() == ref["pos_idx"].tobytes()
    assert got["tiles"].tobytes() == ref["tiles"].tobytes()


def test_pack_all_kept_all_pruned_and_vanilla():
    L = _layer(16, 16, (3, 3, 3), 4, 4, 0.5, 1)
    v = rt3d.rt3d_pack_kgs(L["w"], None, 4, 4, rt3d.RT3D_F32).view()
    assert v["nnz"] == 16 * 27 and v["is_vanilla"] == 1
    v = rt3d.rt3d_pack_kgs(L["w"], np.zeros_like(L["mask"]), 4, 4, rt3d.RT3D_F32).view()
    assert v["nnz"] == 0 and (v["group_ptr"] == 0).all()
    gm = synth.vanilla_mask_exact_total(4, 4, 27, 5, 3)
    mask = synth.expand_group_mask(gm, 16, 16, 4, 4, 3, 3, 3)
    v = rt3d.rt3d_pack_kgs(L["w"], mask, 4, 4, rt3d.RT3D_BF16).view()
    ref = oracle.pack_kgs(L["w"], mask, 4, 4, True)
    assert v["is_vanilla"] == 1 and v["nnz"] == 5 * 27 and v["tiles"].tobytes() == ref["tiles"].tobytes()
    d = rt3d.rt3d_pack_dense(L["w"], rt3d.RT3D_BF16).view()
    assert d["is_dense"] == 1 and d["nnz"] == 16 * 27


def test_pack_errors():
    L = _layer(8, 8, (3, 3, 3), 4, 4, 0.5, 2)
    bad = np.ones_like(L["mask"])
    bad[1, 1, 0, 0, 0] = 0
    with pytest.raises(rt3d.Rt3dError) as e:
        rt3d.rt3d_pack_kgs(L["w"], bad, 4, 4, rt3d.RT3D_F32)
    assert e.value.status == rt3d.ERR_MASK_NOT_GROUP_UNIFORM
    for g_m, g_n, dt in ((0, 4, 0), (4, 257, 0), (4, 4, 7)):
        with pytest.raises(rt3d.Rt3dError) as e:
            rt3d.rt3d_pack_kgs(L["w"], None, g_m, g_n, dt)
        assert e.value.status == rt3d.ERR_INVALID_ARG


@pytest.mark.parametrize("dtype", [rt3d.RT3D_F32, rt3d.RT3D_BF16])
def test_unpack_roundtrip(dtype):
    L = _layer(10, 7, (3, 3, 3), 4, 4, 0.45, 5)
    back = rt3d.rt3d_pack_kgs(L["w"], L["mask"], 4, 4, dtype).unpack_to_dense()
    expect = L["w"] * L["mask"]
    if dtype == rt3d.RT3D_BF16:
        expect = oracle.bf16_round(expect)
    np.testing.assert_array_equal(back, expect)


@pytest.mark.parametrize("M,N,k,g_m,g_n,n_tile", [(256, 128, (3, 3, 3), 4, 4, 0), (256, 128, (3, 3, 3), 4, 4, 64),
                                                  (45, 3, (1, 7, 7), 4, 4, 0), (144, 64, (1, 3, 3), 8, 4, 0),
                                                  (64, 230, (3, 1, 1), 8, 8, 32), (512, 70, (1, 1, 1), 4, 4, 0),
                                                  (256, 128, (3, 3, 3), 64, 64, 64), (256, 256, (3, 3, 3), 256, 64, 0)])
def test_tensor_core_layout_holds_exactly_the_masked_weights(M, N, k, g_m, g_n, n_tile):
    L = _layer(M, N, k, g_m, g_n, 0.3, 11)
    pk = rt3d.rt3d_pack_kgs(L["w"], L["mask"], g_m, g_n, rt3d.RT3D_BF16)
    np.testing.assert_array_equal(pk.unpack_device_layout(n_tile), oracle.bf16_round(L["w"] * L["mask"]))
    # the t-grouped order of the same layout (its group tables are checked inside the call)
    np.testing.assert_array_equal(pk.unpack_device_layout(n_tile, t_groups=True), oracle.bf16_round(L["w"] * L["mask"]))
    with pytest.raises(rt3d.Rt3dError):
        rt3d.rt3d_pack_kgs(L["w"], L["mask"], g_m, g_n, rt3d.RT3D_F32).unpack_device_layout(n_tile)


def test_wide_groups_drop_whole_steps_from_the_layout():
    # groups as wide as a bundle and as deep as a chunk: a pruned (location, chunk) is not a step at all
    spec = synth.ConvSpec("t", 256, 256, (3, 3, 3), (1, 1, 1), (1, 1, 1))
    L = synth.make_layer(spec, 9, 2, 256, 64, "exact_total", (1 * 4 * 27) // 4)
    pk = rt3d.rt3d_pack_kgs(L["w"], L["mask"], 256, 64, rt3d.RT3D_BF16)
    assert pk.view()["nnz"] == 27
    np.testing.assert_array_equal(pk.unpack_device_layout(256), oracle.bf16_round(L["w"] * L["mask"]))


def test_vanilla_high_rate_skips_steps_in_layout():
    # whole groups removed at 8x with narrow bundles: some (location, chunk) steps vanish entirely
    spec = synth.ConvSpec("t", 256, 64, (3, 3, 3), (1, 1, 1), (1, 1, 1))
    L = synth.make_layer(spec, 9, 1, 4, 4, "vanilla_total", (16 * 64) // 8)
    pk = rt3d.rt3d_pack_kgs(L["w"], L["mask"], 4, 4, rt3d.RT3D_BF16)
    np.testing.assert_array_equal(pk.unpack_device_layout(16), oracle.bf16_round(L["w"] * L["mask"]))
    np.testing.assert_array_equal(pk.unpack_device_layout(16, t_groups=True), oracle.bf16_round(L["w"] * L["mask"]))


@pytest.mark.parametrize("M,N,k,g_m,g_n,density", [(256, 256, (3, 3, 3), 8, 8, 0.125), (256, 128, (3, 3, 3), 4, 4, 0.4),
                                                   (230, 72, (1, 3, 3), 8, 4, 0.2), (64, 40, (3, 1, 1), 8, 8, 0.3),
                                                   (512, 64, (3, 3, 3), 64, 64, 0.5), (40, 16, (3, 3, 3), 8, 8, 0.05),
                                                   (300, 256, (3, 3, 3), 16, 16, 0.25)])
def test_sub_tile_layout_holds_exactly_the_masked_weights(M, N, k, g_m, g_n, density):
    # blocks of 16 x 16 channels + per-step command headers: rebuilt weights equal W * mask after bf16 rounding, and the
    # library's own consistency checks (first step starts every range, block indices in range, zeros outside) pass
    L = _layer(M, N, k, g_m, g_n, density, 3)
    pk = rt3d.rt3d_pack_kgs(L["w"], L["mask"], g_m, g_n, rt3d.RT3D_BF16)
    np.testing.assert_array_equal(pk.unpack_sub_layout(0), oracle.bf16_round(L["w"] * L["mask"]))
