"""Pins for the CPU oracle: everything here runs without a GPU and never touches the CUDA path.

Each test checks the oracle against something other than itself: a structurally different
brute force, hand-worked values, closed forms, a library convolution, the identities the
paper states (mask of ones = dense conv; vanilla sparsity is a special case of KGS;
2-D conv is 3-D conv with temporal size 1) and the model totals the paper prints.
"""
import itertools
import os

import numpy as np
import pytest
import torch

import oracle
import rt3d_synth as synth

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def _rand(shape, seed, lo=-1.0, hi=1.0):
    return np.random.default_rng(seed).uniform(lo, hi, size=shape).astype(np.float32)


# ------------------------------------------------------------------ hand-worked fixtures
def _parse_hand_cases():
    cases, cur = [], {}
    for line in open(os.path.join(GOLDEN, "hand_worked_conv.txt")):
        line = line.strip()
        if line.startswith("#"):
            continue
        if not line:
            if cur:
                cases.append(cur)
                cur = {}
            continue
        key, rest = line.split(None, 1)
        if key in ("x", "w"):
            dims, vals = rest.split("|")
            cur[key] = np.array(vals.split(), dtype=np.float32).reshape([int(d) for d in dims.split()])
        elif key in ("stride", "pad"):
            cur[key] = tuple(int(v) for v in rest.split())
        elif key == "y":
            cur["y"] = np.array(rest.split(), dtype=np.float32)
    if cur:
        cases.append(cur)
    return cases


def test_hand_worked_examples():
    cases = _parse_hand_cases()
    assert len(cases) == 4
    for c in cases:
        for fn in (oracle.conv3d, oracle.conv3d_scatter):
            y = fn(c["x"], c["w"], stride=c["stride"], pad=c["pad"])
            np.testing.assert_array_equal(y.ravel(), c["y"])


# ------------------------------------------------------- gather form vs scatter brute force
@pytest.mark.parametrize("k", [(1, 1, 1), (2, 1, 3), (3, 3, 3), (1, 3, 3), (3, 1, 1), (2, 2, 2)])
@pytest.mark.parametrize("stride,pad", [((1, 1, 1), (0, 0, 0)), ((1, 1, 1), (1, 1, 1)),
                                        ((2, 2, 2), (1, 1, 1)), ((1, 2, 2), (0, 1, 1)),
                                        ((2, 1, 1), (1, 0, 0))])
def test_gather_equals_scatter_bruteforce(k, stride, pad):
    seed = hash((k, stride, pad)) & 0xFFFF
    for (n, t, h, w, c, M) in [(1, 3, 4, 5, 2, 3), (2, 5, 3, 4, 5, 2), (1, 4, 5, 3, 1, 1)]:
        if any(d + 2 * p < kk for d, p, kk in zip((t, h, w), pad, k)):
            continue
        x = _rand((n, t, h, w, c), seed)
        wt = _rand((M, c) + k, seed + 1)
        b = _rand((M,), seed + 2)
        mask = (np.random.default_rng(seed + 3).uniform(size=wt.shape) < 0.6).astype(np.uint8)
        for relu in (False, True):
            ya = oracle.conv3d(x, wt, mask, b, stride, pad, relu)
            yb = oracle.conv3d_scatter(x, wt, mask, b, stride, pad, relu)
            assert ya.shape == yb.shape
            np.testing.assert_allclose(ya, yb, rtol=0, atol=2e-6)


def test_impulse_response_pins_axis_order_and_orientation():
    # x = delta at voxel v0, channel c0  =>  y[v0 - loc + pad, m] = W[m, c0, loc]
    M, N, k, pad = 3, 2, (3, 3, 3), (1, 1, 1)
    t, h, w = 5, 6, 7
    wt = _rand((M, N) + k, 11)
    v0, c0 = (2, 3, 4), 1
    x = np.zeros((1, t, h, w, N), np.float32)
    x[0, v0[0], v0[1], v0[2], c0] = 1.0
    y = oracle.conv3d(x, wt, pad=pad)
    expect = np.zeros_like(y)
    for kt, kh, kw in itertools.product(range(3), repeat=3):
        expect[0, v0[0] - kt + 1, v0[1] - kh + 1, v0[2] - kw + 1, :] = wt[:, c0, kt, kh, kw]
    np.testing.assert_array_equal(y, expect)


def test_closed_form_ones_counts_kept_inbounds_taps():
    # x = 1, W = 1, b = 0: every output equals the number of kept, in-bounds (tap, channel) pairs.
    M, N, g_m, g_n = 6, 5, 4, 4                       # ragged groups on both axes
    k, pad, stride = (3, 3, 3), (1, 1, 1), (1, 2, 1)
    t, h, w = 4, 5, 3
    P, Q = synth.n_groups(M, N, g_m, g_n)
    gm = synth.kgs_mask_bernoulli(P, Q, 27, 0.5, 77)
    mask = synth.expand_group_mask(gm, M, N, g_m, g_n, *k)
    y = oracle.conv3d(np.ones((1, t, h, w, N), np.float32), np.ones((M, N) + k, np.float32), mask,
                      stride=stride, pad=pad)
    To, Ho, Wo = y.shape[1:4]
    for to, ho, wo, m in itertools.product(range(To), range(Ho), range(Wo), range(M)):
        cnt = 0
        for kt, kh, kw in itertools.product(range(3), repeat=3):
            ti, hi, wi = to * stride[0] + kt - 1, ho * stride[1] + kh - 1, wo * stride[2] + kw - 1
            if 0 <= ti < t and 0 <= hi < h and 0 <= wi < w:
                kpos = (kt * 3 + kh) * 3 + kw
                for c in range(N):
                    cnt += int(gm[m // g_m, c // g_n, kpos])
        assert y[0, to, ho, wo, m] == cnt


def test_t_equals_one_reduces_to_conv2d():
    # Section 1 footnote: 2-D convolution is the 3-D one with temporal size 1.
    x = _rand((2, 1, 9, 8, 5), 5)
    wt = _rand((4, 5, 1, 3, 3), 6)
    b = _rand((4,), 7)
    for stride, pad in (((1, 1), (1, 1)), ((2, 2), (1, 1)), ((1, 2), (0, 1))):
        y3 = oracle.conv3d(x, wt, None, b, (1,) + stride, (0,) + pad, relu=True)
        y2 = oracle.conv2d(x[:, 0], wt[:, :, 0], b, stride, pad, relu=True)
        np.testing.assert_allclose(y3[:, 0], y2, rtol=0, atol=2e-6)


@pytest.mark.parametrize("k,stride,pad", [((3, 3, 3), (1, 1, 1), (1, 1, 1)),
                                          ((1, 7, 7), (1, 2, 2), (0, 3, 3)),
                                          ((3, 1, 1), (2, 1, 1), (1, 0, 0)),
                                          ((1, 1, 1), (2, 2, 2), (0, 0, 0))])
def test_library_convolution_float64(k, stride, pad):
    # The plain definition coincides with the library's conv3d (cross-correlation, zero pad).
    x = _rand((2, 6, 9, 10, 7), 21)
    wt = _rand((5, 7) + k, 22)
    b = _rand((5,), 23)
    y = oracle.conv3d(x, wt, None, b, stride, pad)
    xt = torch.from_numpy(x).double().permute(0, 4, 1, 2, 3)
    ref = torch.nn.functional.conv3d(xt, torch.from_numpy(wt).double(), torch.from_numpy(b).double(),
                                     stride=stride, padding=pad).permute(0, 2, 3, 4, 1).numpy()
    np.testing.assert_allclose(y, ref.astype(np.float32), rtol=0, atol=2e-6)


# --------------------------------------------------------------------------- masking
def _kgs_case(seed=3, M=10, N=7, g_m=4, g_n=4, density=0.45):
    k = (3, 3, 3)
    x = _rand((1, 4, 6, 5, N), seed)
    wt = _rand((M, N) + k, seed + 1)
    b = _rand((M,), seed + 2)
    P, Q = synth.n_groups(M, N, g_m, g_n)
    gm = synth.kgs_mask_bernoulli(P, Q, 27, density, seed + 3)
    return x, wt, b, gm, synth.expand_group_mask(gm, M, N, g_m, g_n, *k)


def test_mask_of_ones_equals_dense():
    x, wt, b, _, mask = _kgs_case()
    y0 = oracle.conv3d(x, wt, None, b, pad=(1, 1, 1))
    y1 = oracle.conv3d(x, wt, np.ones_like(mask), b, pad=(1, 1, 1))
    np.testing.assert_array_equal(y0, y1)


def test_pruned_group_contributes_exactly_zero():
    x, wt, b, gm, mask = _kgs_case()
    y0 = oracle.conv3d(x, wt, mask, b, pad=(1, 1, 1))
    garbage = wt.copy()
    garbage[mask == 0] = 1e30          # pruned weights must never be read into the sum
    y1 = oracle.conv3d(x, garbage, mask, b, pad=(1, 1, 1))
    np.testing.assert_array_equal(y0, y1)
    # an output channel whose groups are all pruned yields act(bias)
    mask2 = mask.copy()
    mask2[0:4] = 0
    y2 = oracle.conv3d(x, wt, mask2, b, pad=(1, 1, 1), relu=True)
    np.testing.assert_array_equal(y2[..., 0:4], np.broadcast_to(np.maximum(b[0:4], 0), y2[..., 0:4].shape))


def test_disjoint_masks_are_additive():
    x, wt, b, gm, mask = _kgs_case()
    other = synth.expand_group_mask(1 - gm, wt.shape[0], wt.shape[1], 4, 4, 3, 3, 3)
    ya = oracle.conv3d(x, wt, mask, None, pad=(1, 1, 1)).astype(np.float64)
    yb = oracle.conv3d(x, wt, other, None, pad=(1, 1, 1)).astype(np.float64)
    yd = oracle.conv3d(x, wt, None, None, pad=(1, 1, 1)).astype(np.float64)
    np.testing.assert_allclose(ya + yb, yd, rtol=0, atol=3e-6)


def test_vanilla_is_special_case_of_kgs():
    # Section 3: a vanilla mask (whole groups) is a KGS mask; packing marks it as such.
    M, N, k = 8, 8, (3, 3, 3)
    wt = _rand((M, N) + k, 9)
    gm = synth.vanilla_mask_exact_total(2, 2, 27, 2, 5)
    mask = synth.expand_group_mask(gm, M, N, 4, 4, *k)
    pk = oracle.pack_kgs(wt, mask, 4, 4)
    assert pk["is_vanilla"] and pk["nnz"] == 2 * 27
    gm2 = synth.kgs_mask_exact_per_group(2, 2, 27, 14, 5)
    pk2 = oracle.pack_kgs(wt, synth.expand_group_mask(gm2, M, N, 4, 4, *k), 4, 4)
    assert not pk2["is_vanilla"] and pk2["nnz"] == 4 * 14


# ------------------------------------------------------------------------------ pack
@pytest.mark.parametrize("M,N,g_m,g_n", [(8, 8, 4, 4), (6, 5, 4, 4), (16, 12, 8, 4), (9, 17, 8, 8), (3, 3, 4, 4)])
@pytest.mark.parametrize("to_bf16", [False, True])
def test_pack_roundtrip_and_counts(M, N, g_m, g_n, to_bf16):
    k = (3, 3, 3)
    wt = _rand((M, N) + k, M * 31 + N)
    P, Q = synth.n_groups(M, N, g_m, g_n)
    gm = synth.kgs_mask_bernoulli(P, Q, 27, 0.4, M + N)
    mask = synth.expand_group_mask(gm, M, N, g_m, g_n, *k)
    pk = oracle.pack_kgs(wt, mask, g_m, g_n, to_bf16)
    assert pk["nnz"] == int(gm.sum())
    np.testing.assert_array_equal(np.diff(pk["group_ptr"]), gm.reshape(P * Q, 27).sum(1))
    for g in range(P * Q):                                    # ascending locations inside a group
        seg = pk["pos_idx"][pk["group_ptr"][g]:pk["group_ptr"][g + 1]]
        np.testing.assert_array_equal(seg, np.nonzero(gm.reshape(P * Q, 27)[g])[0])
    back = oracle.unpack_kgs(pk, M, N, *k, g_m, g_n)
    expect = wt * mask
    if to_bf16:
        expect = torch.from_numpy(expect).to(torch.bfloat16).float().numpy()
    np.testing.assert_array_equal(back, expect)
    # ragged tiles are zero filled: total tile mass equals the masked weight mass
    tiles = pk["tiles"] if not to_bf16 else oracle.bf16_widen(pk["tiles"])
    assert np.isclose(np.abs(tiles).sum(dtype=np.float64), np.abs(back).sum(dtype=np.float64))


def test_pack_tile_element_order_by_direct_indexing():
    """Pins the order INSIDE a tile without going through the oracle's own unpack: element [i][j] of the
    tile stored for group (p, q) at kernel location kpos is W[p*g_m + i][q*g_n + j][kpos], zero where the
    kernel does not exist (ragged last groups).  A non-square group size and weights that encode their own
    (m, n, kpos) make a transposed or differently flattened layout fail."""
    M, N, k, g_m, g_n = 19, 14, (2, 3, 2), 8, 4
    Ks = k[0] * k[1] * k[2]
    m_i, n_i, k_i = np.meshgrid(np.arange(M), np.arange(N), np.arange(Ks), indexing="ij")
    # m + n/16 + kpos/256 + 1: distinct per (m, n, kpos); 5 + 4 + 4 significant bits, but bf16 keeps 8, so
    # the bf16 case uses a code with 8 bits that is still distinct inside every tile and across locations
    codes = {False: (1.0 + m_i + n_i / 16.0 + k_i / 256.0), True: (1.0 + (m_i % 8) * 16 + (n_i % 4) * 4 + (k_i % 4))}
    P, Q = synth.n_groups(M, N, g_m, g_n)
    gm = synth.kgs_mask_bernoulli(P, Q, Ks, 0.5, 77)
    mask = synth.expand_group_mask(gm, M, N, g_m, g_n, *k)
    for to_bf16 in (False, True):
        wv = codes[to_bf16].astype(np.float32).reshape((M, N) + k)
        pk = oracle.pack_kgs(wv, mask, g_m, g_n, to_bf16)
        tiles = pk["tiles"] if not to_bf16 else oracle.bf16_widen(pk["tiles"])
        assert tiles.shape == (pk["nnz"], g_m, g_n) and pk["nnz"] > 0
        w3 = wv.reshape(M, N, Ks)
        seen_ragged = False
        for p in range(P):
            for q in range(Q):
                g = p * Q + q
                for e in range(pk["group_ptr"][g], pk["group_ptr"][g + 1]):
                    kpos = int(pk["pos_idx"][e])
                    for i in range(g_m):
                        for j in range(g_n):
                            m, n = p * g_m + i, q * g_n + j
                            inside = m < M and n < N
                            seen_ragged |= not inside
                            assert tiles[e, i, j] == (w3[m, n, kpos] if inside else 0.0), (to_bf16, p, q, kpos, i, j)
        assert seen_ragged


def test_pack_rejects_non_uniform_mask():
    wt = _rand((8, 8, 3, 3, 3), 1)
    mask = np.ones_like(wt, dtype=np.uint8)
    mask[1, 2, 0, 1, 2] = 0
    with pytest.raises(oracle.MaskNotGroupUniform):
        oracle.pack_kgs(wt, mask, 4, 4)
    mask[0:4, 0:4, 0, 1, 2] = 0
    assert oracle.pack_kgs(wt, mask, 4, 4)["nnz"] == 4 * 27 - 1


def test_pack_kept_location_with_zero_weights_is_stored():
    wt = np.zeros((4, 4, 1, 1, 2), np.float32)
    mask = np.ones_like(wt, dtype=np.uint8)
    mask[..., 1] = 0
    pk = oracle.pack_kgs(wt, mask, 4, 4)
    assert pk["nnz"] == 1 and pk["pos_idx"][0] == 0


# -------------------------------------------------------------------- bf16 rounding
def test_bf16_rne_matches_library_rounding():
    rng = np.random.default_rng(0)
    bits = rng.integers(0, 2 ** 32, size=1 << 20, dtype=np.uint64).astype(np.uint32)
    hand = np.array([0x3F808000, 0x3F818000, 0x3F808001, 0x3F80FFFF, 0x00000001, 0x80000000, 0x00000000,
                     0x7F7FFFFF, 0x7F800000, 0xFF800000, 0x00008000, 0x00018000, 0x3F7FFFFF], dtype=np.uint32)
    bits = np.concatenate([bits, hand])
    f = bits.view(np.float32)
    keep = ~np.isnan(f)
    f = f[keep]
    got = oracle.bf16_bits(f)
    ref = torch.from_numpy(f).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    np.testing.assert_array_equal(got, ref)
    # ties go to even: 1 + 2^-8 (exactly half way between 1 and 1+2^-7) rounds down to 1
    assert oracle.bf16_bits(np.array([1.0 + 2.0 ** -8], np.float32))[0] == 0x3F80
    assert oracle.bf16_bits(np.array([1.0 + 3 * 2.0 ** -8], np.float32))[0] == 0x3F82


def test_bf16_mode_rounds_inputs_not_sums():
    x, wt, b, gm, mask = _kgs_case(seed=13)
    y = oracle.conv3d(x, wt, mask, b, pad=(1, 1, 1), round_bf16=True)
    y2 = oracle.conv3d(oracle.bf16_round(x), oracle.bf16_round(wt * mask), None, b, pad=(1, 1, 1))
    np.testing.assert_array_equal(y, y2)
    assert np.abs(y - oracle.conv3d(x, wt, mask, b, pad=(1, 1, 1))).max() > 0


# ---------------------------------------------------------------- pooling and add
def test_maxpool_ramp_closed_form_and_library():
    n, t, h, w, c = 1, 4, 6, 6, 3
    x = np.arange(n * t * h * w * c, dtype=np.float32).reshape(n, t, h, w, c)   # strictly increasing
    y = oracle.maxpool3d(x, (2, 2, 2), (2, 2, 2))
    np.testing.assert_array_equal(y, x[:, 1::2, 1::2, 1::2, :])                # max = last corner of each window
    xr = _rand((2, 2, 7, 7, 4), 3)
    y = oracle.maxpool3d(xr, (2, 2, 2), (2, 2, 2), (0, 1, 1))
    ref = torch.nn.functional.max_pool3d(torch.from_numpy(xr).permute(0, 4, 1, 2, 3), (2, 2, 2), (2, 2, 2),
                                         (0, 1, 1)).permute(0, 2, 3, 4, 1).numpy()
    assert y.shape == (2, 1, 4, 4, 4)
    np.testing.assert_array_equal(y, ref)


def test_add_relu():
    # hand values: sums that are exact in binary, one negative, one exactly zero, one positive
    a = np.array([[1.5, -2.0, 0.25], [-0.5, 3.0, -4.0]], np.float32)
    b = np.array([[0.5, 1.0, -0.25], [-0.5, -1.0, 4.5]], np.float32)
    np.testing.assert_array_equal(oracle.add_relu(a, b, False), np.array([[2.0, -1.0, 0.0], [-1.0, 2.0, 0.5]], np.float32))
    np.testing.assert_array_equal(oracle.add_relu(a, b, True), np.array([[2.0, 0.0, 0.0], [0.0, 2.0, 0.5]], np.float32))
    # and commutativity / idempotence of the activation on random data
    x, y = _rand((3, 5), 1), _rand((3, 5), 2)
    r = oracle.add_relu(x, y, True)
    np.testing.assert_array_equal(r, oracle.add_relu(y, x, True))
    np.testing.assert_array_equal(oracle.add_relu(r, np.zeros_like(r), True), r)
    assert (r >= 0).all() and (r[oracle.add_relu(x, y, False) > 0] > 0).all()


# -------------------------------------------------------------------- workload shapes
def _paper_totals():
    rows = {}
    for line in open(os.path.join(GOLDEN, "paper_model_totals.txt")):
        if line.startswith("#") or not line.strip():
            continue
        model, size, after, rate = line.split()
        rows.setdefault(model, []).append((float(size), float(after), float(rate)))
    return rows


def test_layer_plans_reproduce_paper_totals():
    totals = _paper_totals()
    # C3D-shaped stack
    t, h, w = 16, 112, 112
    macs, params = 0, 0
    for op in synth.c3d_plan():
        if isinstance(op, synth.ConvSpec):
            macs += op.dense_macs(1, t, h, w)
            params += op.n_weights() + op.cout
            t, h, w = op.out_extent(t, h, w)
        else:
            t, h, w = [(d + 2 * p - k) // s + 1 for d, p, k, s in zip((t, h, w), op.pad, op.k, op.stride)]
    assert (t, h, w) == (1, 4, 4)
    fc = 8192 * 4096 + 4096 + 4096 * 4096 + 4096 + 4096 * 101 + 101
    lo = min((a - 0.05) * (r - 0.05) for _, a, r in totals["c3d"])
    hi = max((a + 0.05) * (r + 0.05) for _, a, r in totals["c3d"])
    assert lo <= macs / 1e9 <= hi, (macs, lo, hi)
    assert abs((params + fc) * 4 / 2 ** 20 - totals["c3d"][0][0]) < 1.0
    # R(2+1)D-18-shaped
    stem, blocks = synth.r2plus1d18_plan()
    t, h, w = 16, 112, 112
    macs, params = 0, 0
    for cv in stem:
        macs += cv.dense_macs(1, t, h, w); params += cv.n_weights() + cv.cout
        t, h, w = cv.out_extent(t, h, w)
    for blk in blocks:
        t0, h0, w0 = t, h, w
        for cv in blk.convs:
            macs += cv.dense_macs(1, t, h, w); params += cv.n_weights() + cv.cout
            t, h, w = cv.out_extent(t, h, w)
        if blk.shortcut is not None:
            macs += blk.shortcut.dense_macs(1, t0, h0, w0); params += blk.shortcut.n_weights() + blk.shortcut.cout
            assert blk.shortcut.out_extent(t0, h0, w0) == (t, h, w)
    assert (t, h, w) == (2, 7, 7)
    lo = min((a - 0.05) * (r - 0.05) for _, a, r in totals["r2plus1d"])
    hi = max((a + 0.05) * (r + 0.05) for _, a, r in totals["r2plus1d"])
    assert lo <= macs / 1e9 <= hi, (macs, lo, hi)
    fc = 512 * 400 + 400
    assert abs((params + fc) * 4 / 2 ** 20 - totals["r2plus1d"][0][0]) < 1.5


# -------------------------------------------------------------------- generator sanity
def test_s3d_plan_is_consistent():
    """The paper gives no S3D totals (only its 2.1x FLOPs pruning rate), so this pins the plan's internal
    consistency: every op consumes what the previous one produces, Inception branches concatenate to the
    next block's input width, extents follow the pooling schedule, slices stay 16-byte aligned."""
    plan = synth.s3d_plan()
    t, h, w, c = 16, 224, 224, 3
    n_convs = 0
    for op in plan:
        if isinstance(op, synth.ConvSpec):
            assert op.cin == c, op.name
            t, h, w = op.out_extent(t, h, w)
            c = op.cout
            n_convs += 1
        elif isinstance(op, synth.PoolSpec):
            t, h, w = [(d + 2 * p - k) // s + 1 for d, p, k, s in zip((t, h, w), op.pad, op.k, op.stride)]
        else:
            assert op.cin == c, op.name
            for br in (op.b1, op.b2):
                assert br[0].cin == c and br[1].cin == br[0].cout and br[2].cin == br[1].cout == br[2].cout
            assert op.b3.cin == c and op.b0.cin == c
            assert [(d + 2 * p - k) // s + 1 for d, p, k, s in zip((t, h, w), op.pool.pad, op.pool.k, op.pool.stride)] == [t, h, w]
            for sp in op.convs():
                assert sp.out_extent(t, h, w) == (t, h, w)            # branches keep the extents
                assert sp.cout % 8 == 0                               # channel slices start on 16-byte boundaries
            c = op.cout
            n_convs += 8
    assert (t, h, w, c) == (2, 7, 7, 1024)
    assert n_convs == 5 + 9 * 8 == len(synth.s3d_convs(plan))
    assert [op.cout for op in plan if isinstance(op, synth.InceptionSpec)] == [256, 480, 512, 512, 512, 528, 832, 832, 1024]


def test_generator_is_counter_based_and_calibrated():
    a = synth.splitmix64(123, 0, 1000)
    b = synth.splitmix64(123, 500, 500)
    np.testing.assert_array_equal(a[500:], b)
    u = synth.uniform_pm1(1, (200000,))
    g = synth.normal(2, (200000,), 0.05)
    assert abs(u.mean()) < 0.01 and abs(u.std() - 1 / np.sqrt(3)) < 0.01 and u.min() >= -1 and u.max() < 1
    assert abs(g.mean()) < 1e-3 and abs(g.std() - 0.05) < 1e-3
    gm = synth.kgs_mask_exact_per_group(8, 4, 27, 14, 9)
    assert (gm.sum(-1) == 14).all()
    assert synth.kgs_mask_exact_total(64, 64, 27, 12345, 3).sum() == 12345
    v = synth.vanilla_mask_exact_total(64, 64, 27, 100, 3)
    assert v.sum() == 2700 and set(np.unique(v.sum(-1))) == {0, 27}


# ----------------------------------------------------- group norms and reweighting (Section 4)
def test_group_norms_closed_forms_and_library():
    M, N, k, g_m, g_n = 10, 7, (3, 3, 3), 4, 4
    ones = np.ones((M, N) + k, np.float32)
    n1 = oracle.group_norms(ones, g_m, g_n, 1)
    n2 = oracle.group_norms(ones, g_m, g_n, 2)
    rows = np.minimum(g_m, M - np.arange(0, M, g_m))          # kernels that exist in ragged groups
    cols = np.minimum(g_n, N - np.arange(0, N, g_n))
    cnt = np.outer(rows, cols).astype(np.float64)
    np.testing.assert_array_equal(n1, np.broadcast_to(cnt[..., None], n1.shape).astype(np.float32))
    np.testing.assert_allclose(n2, np.broadcast_to(np.sqrt(cnt)[..., None], n2.shape), rtol=1e-7)
    w = _rand((M, N) + k, 4)
    for g in (1, 2):                                           # library norm on each reshaped group
        got = oracle.group_norms(w, g_m, g_n, g)
        for p in range(3):
            for q in range(2):
                blk = w[p * g_m:(p + 1) * g_m, q * g_n:(q + 1) * g_n].reshape(-1, 27).astype(np.float64)
                np.testing.assert_allclose(got[p, q], np.linalg.norm(blk, ord=g, axis=0), rtol=1e-6)
        np.testing.assert_allclose(oracle.group_norms(-2.5 * w, g_m, g_n, g), 2.5 * got, rtol=1e-6)   # homogeneity


def test_reweight_penalty_and_mask():
    norms = np.array([0.0, 0.1, 0.5, 2.0], np.float32)
    pen, keep = oracle.reweight(norms, 1e-3, 0.3)
    np.testing.assert_allclose(pen, [1000.0, 1 / 0.011, 1 / 0.251, 1 / 4.001], rtol=1e-6)   # 1 / (n^2 + eps)
    assert (np.diff(pen) < 0).all()                     # larger groups are penalised less
    np.testing.assert_array_equal(keep, [0, 0, 1, 1])
    # a mask made this way is a KGS mask: the packer accepts it and keeps exactly those locations
    w = _rand((8, 8, 3, 3, 3), 5)
    n = oracle.group_norms(w, 4, 4, 2)
    thr = float(np.median(n))
    _, gk = oracle.reweight(n, 1e-3, thr)
    mask = synth.expand_group_mask(gk, 8, 8, 4, 4, 3, 3, 3)
    assert oracle.pack_kgs(w, mask, 4, 4)["nnz"] == int(gk.sum()) == int((n > thr).sum())
