"""GPU parity of the device-side pruning step (group norms, reweighted penalties, KGS mask) against the oracle.

Norms and penalties are fp32 on the device and double on the oracle: relative tolerance 1e-5 / 1e-4
(sums of at most a few thousand non-negative terms).  The keep / prune decision is a comparison of the
fp32 norm with a threshold; thresholds are put half way between two neighbouring norms whose gap is far
above one ulp, so both sides decide on the same side; the expanded mask is then compared bit for bit
and must pack to exactly the same canonical arrays as the oracle's mask.
"""
import numpy as np
import pytest
import torch

import oracle
import rt3d_synth as synth
import paper_2007_09835_b200 as rt3d

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("M,N,k,g_m,g_n", [(256, 128, (3, 3, 3), 4, 4), (45, 3, (1, 7, 7), 4, 4),
                                           (230, 64, (1, 3, 3), 8, 4), (512, 512, (3, 3, 3), 8, 8),
                                           (64, 230, (3, 1, 1), 4, 4), (256, 256, (3, 3, 3), 256, 64)])
@pytest.mark.parametrize("norm", [1, 2])
def test_group_norms_penalty_mask_and_pack(M, N, k, g_m, g_n, norm):
    spec = synth.ConvSpec("r", N, M, k, (1, 1, 1), (0, 0, 0))
    w = synth.make_layer(spec, 6, M + N + norm, g_m, g_n, "none", None)["w"]
    Ks = k[0] * k[1] * k[2]
    P, Q = synth.n_groups(M, N, g_m, g_n)
    ref = oracle.group_norms(w, g_m, g_n, norm)
    wd = torch.from_numpy(w).cuda()
    nd = torch.empty((P, Q, Ks), dtype=torch.float32, device="cuda")
    rt3d.rt3d_kgs_group_norms(wd, g_m, g_n, norm, nd)
    got = nd.cpu().numpy()
    np.testing.assert_allclose(got, ref, rtol=1e-5, atol=0)
    # threshold in the widest gap near the median norm
    srt = np.sort(ref.ravel())
    lo = max(1, int(0.45 * srt.size)); hi = max(lo + 1, int(0.55 * srt.size))
    j = lo + int(np.argmax(np.diff(srt[lo:hi + 1])))
    thr = float(0.5 * (float(srt[j]) + float(srt[j + 1])))
    assert srt[j + 1] - srt[j] > 1e-5 * srt[j + 1]
    pen_ref, keep_ref = oracle.reweight(ref, 1e-3, thr)
    pen = torch.empty_like(nd)
    keep = torch.empty((P, Q, Ks), dtype=torch.uint8, device="cuda")
    rt3d.rt3d_kgs_reweight(nd, 1e-3, thr, pen, keep)
    np.testing.assert_allclose(pen.cpu().numpy(), pen_ref, rtol=1e-4, atol=0)
    np.testing.assert_array_equal(keep.cpu().numpy(), keep_ref)
    mask = torch.empty((M, N) + k, dtype=torch.uint8, device="cuda")
    rt3d.rt3d_kgs_expand_mask(keep, M, N, *k, g_m, g_n, mask)
    mask_h = mask.cpu().numpy()
    np.testing.assert_array_equal(mask_h, synth.expand_group_mask(keep_ref, M, N, g_m, g_n, *k))
    pk = rt3d.rt3d_pack_kgs(w, mask_h, g_m, g_n, rt3d.RT3D_BF16).view()       # the mask is a KGS mask
    assert pk["nnz"] == int(keep_ref.sum())


def test_reweight_argument_errors():
    n = torch.ones(8, device="cuda")
    for eps in (0.0, -1.0):
        with pytest.raises(rt3d.Rt3dError) as e:
            rt3d.rt3d_kgs_reweight(n, eps, 0.5, torch.empty_like(n), None)
        assert e.value.status == rt3d.ERR_INVALID_ARG
    with pytest.raises(rt3d.Rt3dError):
        rt3d.rt3d_kgs_reweight(n, 1e-3, 0.5, None, None)
    w = torch.ones((4, 4, 1, 1, 1), device="cuda")
    with pytest.raises(rt3d.Rt3dError):
        rt3d.rt3d_kgs_group_norms(w, 4, 4, 3, torch.empty((1, 1, 1), device="cuda"))
