"""Seeded synthetic inputs and workload shapes for the RT3D conv3d hot path.

This module is the only code shared by the CPU oracle's tests and the CUDA library's
tests / benchmark.  It holds no arithmetic of the method (no convolution, no packing,
no rounding of weights): only a counter-based random generator, the mask recipes and
the layer shape tables of the two video networks the paper measures (C3D and
R(2+1)D, Section 5 "Experimental Setup").  Every value is a pure function of
(seed, stream key, element index), so generation is order independent.

Value distributions: weights N(0, 0.05^2), activations U(-1, 1), bias N(0, 0.01^2).
Masks are drawn at kernel-group level (one bit per (group, kernel location), the KGS
scheme of Section 3) and expanded to one byte per weight.
"""
from __future__ import annotations

import dataclasses
import numpy as np

BASE_SEED = 200709835
_PHI = np.uint64(0x9E3779B97F4A7C15)
_M1 = np.uint64(0xBF58476D1CE4E5B9)
_M2 = np.uint64(0x94D049BB133111EB)

ROLE_WEIGHT, ROLE_INPUT, ROLE_BIAS, ROLE_MASK = 1, 2, 3, 4


def stream_key(seed: int, cfg: int, layer: int, role: int) -> int:
    """64-bit key of one random stream: seed xor (cfg*2^32 + layer*2^16 + role)."""
    return (int(seed) ^ ((int(cfg) << 32) + (int(layer) << 16) + int(role))) & 0xFFFFFFFFFFFFFFFF


def splitmix64(key: int, start: int, count: int) -> np.ndarray:
    """Counter-based splitmix64: element i is mix(key + (start+i+1)*phi), uint64."""
    with np.errstate(over="ignore"):
        idx = np.arange(start + 1, start + count + 1, dtype=np.uint64)
        z = np.uint64(key) + idx * _PHI
        z = (z ^ (z >> np.uint64(30))) * _M1
        z = (z ^ (z >> np.uint64(27))) * _M2
        z = z ^ (z >> np.uint64(31))
    return z


def uniform01(key: int, count: int, start: int = 0) -> np.ndarray:
    """Doubles in [0, 1): top 53 bits of each 64-bit draw."""
    return (splitmix64(key, start, count) >> np.uint64(11)).astype(np.float64) * (1.0 / 9007199254740992.0)


def uniform_pm1(key: int, shape) -> np.ndarray:
    """float32 tensor of U(-1, 1) draws."""
    n = int(np.prod(shape))
    return (2.0 * uniform01(key, n) - 1.0).astype(np.float32).reshape(shape)


def normal(key: int, shape, sigma: float) -> np.ndarray:
    """float32 tensor of N(0, sigma^2) draws (Box-Muller, one output per uniform pair)."""
    n = int(np.prod(shape))
    u = uniform01(key, 2 * n)
    u1 = np.maximum(u[0::2], 2.0 ** -53)
    u2 = u[1::2]
    g = np.sqrt(-2.0 * np.log(u1)) * np.cos(2.0 * np.pi * u2)
    return (sigma * g).astype(np.float32).reshape(shape)


# ----------------------------------------------------------------------------- masks
def n_groups(M: int, N: int, g_m: int, g_n: int):
    """P = ceil(M/g_m), Q = ceil(N/g_n) kernel groups (Section 4)."""
    return -(-M // g_m), -(-N // g_n)


def kgs_mask_exact_per_group(P: int, Q: int, Ks: int, k: int, key: int) -> np.ndarray:
    """Each group keeps exactly k of its Ks kernel locations: the k smallest of Ks random keys."""
    r = splitmix64(key, 0, P * Q * Ks).reshape(P * Q, Ks)
    order = np.argsort(r, axis=1, kind="stable")
    gm = np.zeros((P * Q, Ks), dtype=np.uint8)
    np.put_along_axis(gm, order[:, :k], 1, axis=1)
    return gm.reshape(P, Q, Ks)


def kgs_mask_bernoulli(P: int, Q: int, Ks: int, density: float, key: int) -> np.ndarray:
    """Each (group, location) kept independently with probability `density`
    (per-group kept count is Binomial(Ks, density))."""
    u = uniform01(key, P * Q * Ks)
    return (u < density).astype(np.uint8).reshape(P, Q, Ks)


def kgs_mask_exact_total(P: int, Q: int, Ks: int, kept: int, key: int) -> np.ndarray:
    """Exactly `kept` (group, location) pairs kept, uniformly over all P*Q*Ks pairs."""
    r = splitmix64(key, 0, P * Q * Ks)
    order = np.argsort(r, kind="stable")
    gm = np.zeros(P * Q * Ks, dtype=np.uint8)
    gm[order[:kept]] = 1
    return gm.reshape(P, Q, Ks)


def vanilla_mask_exact_total(P: int, Q: int, Ks: int, kept_groups: int, key: int) -> np.ndarray:
    """Vanilla structured sparsity: exactly `kept_groups` whole groups kept."""
    r = splitmix64(key, 0, P * Q)
    order = np.argsort(r, kind="stable")
    g = np.zeros(P * Q, dtype=np.uint8)
    g[order[:kept_groups]] = 1
    return np.repeat(g[:, None], Ks, axis=1).reshape(P, Q, Ks)


def expand_group_mask(gmask: np.ndarray, M: int, N: int, g_m: int, g_n: int,
                      Kt: int, Kh: int, Kw: int) -> np.ndarray:
    """Group-level mask [P,Q,Ks] -> per-weight uint8 mask [M,N,Kt,Kh,Kw]."""
    P, Q, Ks = gmask.shape
    assert Ks == Kt * Kh * Kw
    full = np.repeat(np.repeat(gmask, g_m, axis=0), g_n, axis=1)[:M, :N]
    return np.ascontiguousarray(full.reshape(M, N, Kt, Kh, Kw))


# ------------------------------------------------------------------------- layer specs
@dataclasses.dataclass(frozen=True)
class ConvSpec:
    """One 3-D convolution layer.  Activations are NDHWC, weights [M][N][Kt][Kh][Kw]."""
    name: str
    cin: int
    cout: int
    k: tuple          # (Kt, Kh, Kw)
    stride: tuple     # (st, sh, sw)
    pad: tuple        # (pt, ph, pw)
    relu: bool = True

    def out_extent(self, t: int, h: int, w: int):
        return tuple((d + 2 * p - kk) // s + 1
                     for d, p, kk, s in zip((t, h, w), self.pad, self.k, self.stride))

    def dense_macs(self, n: int, t: int, h: int, w: int) -> int:
        to, ho, wo = self.out_extent(t, h, w)
        return n * to * ho * wo * self.cout * self.cin * self.k[0] * self.k[1] * self.k[2]

    def n_weights(self) -> int:
        return self.cout * self.cin * self.k[0] * self.k[1] * self.k[2]


@dataclasses.dataclass(frozen=True)
class PoolSpec:
    name: str
    k: tuple
    stride: tuple
    pad: tuple


def c3d_plan():
    """C3D-shaped stack: eight 3x3x3 stride-1 pad-1 convs with ReLU, five max-pools.
    Returns a list of ConvSpec / PoolSpec in execution order; input is 16x112x112x3."""
    chans = [3, 64, 128, 256, 256, 512, 512, 512, 512]
    names = ["conv1", "conv2", "conv3a", "conv3b", "conv4a", "conv4b", "conv5a", "conv5b"]
    pool_after = {"conv1": PoolSpec("pool1", (1, 2, 2), (1, 2, 2), (0, 0, 0)),
                  "conv2": PoolSpec("pool2", (2, 2, 2), (2, 2, 2), (0, 0, 0)),
                  "conv3b": PoolSpec("pool3", (2, 2, 2), (2, 2, 2), (0, 0, 0)),
                  "conv4b": PoolSpec("pool4", (2, 2, 2), (2, 2, 2), (0, 0, 0)),
                  "conv5b": PoolSpec("pool5", (2, 2, 2), (2, 2, 2), (0, 1, 1))}
    plan = []
    for i, nm in enumerate(names):
        plan.append(ConvSpec(nm, chans[i], chans[i + 1], (3, 3, 3), (1, 1, 1), (1, 1, 1), True))
        if nm in pool_after:
            plan.append(pool_after[nm])
    return plan


def c3d_fc_tail(n_classes: int = 101):
    """The three fully connected layers that follow pool5 of the C3D-shaped stack, as 1x1x1 convolutions over
    the flattened 1 x 4 x 4 x 512 feature block (flattened in memory order h, w, c): 8192 -> 4096 -> 4096 ->
    classes, ReLU after the first two.  Not pruned (the paper's FLOPs rates are over the conv layers)."""
    one = lambda nm, ci, co, relu: ConvSpec(nm, ci, co, (1, 1, 1), (1, 1, 1), (0, 0, 0), relu)  # noqa: E731
    return [one("fc6", 8192, 4096, True), one("fc7", 4096, 4096, True), one("fc8", 4096, n_classes, False)]


def r2plus1d_mid(cin: int, cout: int) -> int:
    """Width of the intermediate tensor of a factorised (2+1)D block, chosen so the
    factorised pair has about as many parameters as the 3x3x3 conv it replaces."""
    return (27 * cin * cout) // (9 * cin + 3 * cout)


@dataclasses.dataclass(frozen=True)
class ResBlockSpec:
    """One residual block of the R(2+1)D-18-shaped network: two factorised convs
    (spatial 1x3x3 then temporal 3x1x1 each), optional 1x1x1 strided projection."""
    name: str
    convs: tuple          # (spatial1, temporal1, spatial2, temporal2)
    shortcut: object      # ConvSpec or None


def r2plus1d18_plan():
    """R(2+1)D-18-shaped network.  Returns (stem convs, list of ResBlockSpec)."""
    stem = (ConvSpec("stem.s", 3, 45, (1, 7, 7), (1, 2, 2), (0, 3, 3), True),
            ConvSpec("stem.t", 45, 64, (3, 1, 1), (1, 1, 1), (1, 0, 0), True))
    blocks = []
    cin = 64
    for stage, width in zip((2, 3, 4, 5), (64, 128, 256, 512)):
        for b in (1, 2):
            down = (stage > 2 and b == 1)
            mid = r2plus1d_mid(cin, width)
            ss = (1, 2, 2) if down else (1, 1, 1)
            ts = (2, 1, 1) if down else (1, 1, 1)
            pre = f"s{stage}b{b}"
            convs = (ConvSpec(pre + ".c1.s", cin, mid, (1, 3, 3), ss, (0, 1, 1), True),
                     ConvSpec(pre + ".c1.t", mid, width, (3, 1, 1), ts, (1, 0, 0), True),
                     ConvSpec(pre + ".c2.s", width, mid, (1, 3, 3), (1, 1, 1), (0, 1, 1), True),
                     ConvSpec(pre + ".c2.t", mid, width, (3, 1, 1), (1, 1, 1), (1, 0, 0), False))
            sc = ConvSpec(pre + ".sc", cin, width, (1, 1, 1), (2, 2, 2), (0, 0, 0), False) if down else None
            blocks.append(ResBlockSpec(pre, convs, sc))
            cin = width
    return stem, blocks


# --------------------------------------------------------------------- layer instances
@dataclasses.dataclass(frozen=True)
class InceptionSpec:
    """One Inception block of the S3D-shaped network: four branches whose outputs are concatenated along
    the channels in this order: 1x1x1; 1x1x1 then separable 3x3x3 (1x3x3 + 3x1x1); the same again with other
    widths; 3x3x3 stride-1 max-pool then 1x1x1.  Every conv is followed by ReLU."""
    name: str
    b0: ConvSpec
    b1: tuple            # (1x1x1 reduce, 1x3x3, 3x1x1)
    b2: tuple            # (1x1x1 reduce, 1x3x3, 3x1x1)
    pool: PoolSpec
    b3: ConvSpec

    @property
    def cin(self):
        return self.b0.cin

    @property
    def cout(self):
        return self.b0.cout + self.b1[2].cout + self.b2[2].cout + self.b3.cout

    def convs(self):
        return (self.b0,) + tuple(self.b1) + tuple(self.b2) + (self.b3,)


def _sep3(name, cin, cout):
    return (ConvSpec(name + ".s", cin, cout, (1, 3, 3), (1, 1, 1), (0, 1, 1), True),
            ConvSpec(name + ".t", cout, cout, (3, 1, 1), (1, 1, 1), (1, 0, 0), True))


def s3d_plan():
    """S3D-shaped network (separable 3-D Inception): list of ConvSpec / PoolSpec / InceptionSpec in execution
    order; input is 16 x 224 x 224 x 3.  Widths are those of the Inception-v1 table the architecture uses."""
    plan = [ConvSpec("conv1.s", 3, 64, (1, 7, 7), (1, 2, 2), (0, 3, 3), True),
            ConvSpec("conv1.t", 64, 64, (7, 1, 1), (2, 1, 1), (3, 0, 0), True),
            PoolSpec("pool1", (1, 3, 3), (1, 2, 2), (0, 1, 1)),
            ConvSpec("conv2b", 64, 64, (1, 1, 1), (1, 1, 1), (0, 0, 0), True)]
    plan += list(_sep3("conv2c", 64, 192))
    plan.append(PoolSpec("pool2", (1, 3, 3), (1, 2, 2), (0, 1, 1)))
    table = [("mixed3b", 192, 64, 96, 128, 16, 32, 32), ("mixed3c", 256, 128, 128, 192, 32, 96, 64), "pool3",
             ("mixed4b", 480, 192, 96, 208, 16, 48, 64), ("mixed4c", 512, 160, 112, 224, 24, 64, 64),
             ("mixed4d", 512, 128, 128, 256, 24, 64, 64), ("mixed4e", 512, 112, 144, 288, 32, 64, 64),
             ("mixed4f", 528, 256, 160, 320, 32, 128, 128), "pool4",
             ("mixed5b", 832, 256, 160, 320, 32, 128, 128), ("mixed5c", 832, 384, 192, 384, 48, 128, 128)]
    for row in table:
        if row == "pool3":
            plan.append(PoolSpec("pool3", (3, 3, 3), (2, 2, 2), (1, 1, 1)))
        elif row == "pool4":
            plan.append(PoolSpec("pool4", (2, 2, 2), (2, 2, 2), (0, 0, 0)))
        else:
            nm, cin, b0, b1a, b1b, b2a, b2b, b3 = row
            one = lambda tag, ci, co: ConvSpec(f"{nm}.{tag}", ci, co, (1, 1, 1), (1, 1, 1), (0, 0, 0), True)  # noqa: E731
            plan.append(InceptionSpec(nm, one("b0", cin, b0),
                                      (one("b1a", cin, b1a),) + _sep3(nm + ".b1", b1a, b1b),
                                      (one("b2a", cin, b2a),) + _sep3(nm + ".b2", b2a, b2b),
                                      PoolSpec(nm + ".pool", (3, 3, 3), (1, 1, 1), (1, 1, 1)), one("b3", cin, b3)))
    return plan


def s3d_convs(plan):
    """All ConvSpec of an S3D-shaped plan in execution order."""
    out = []
    for op in plan:
        if isinstance(op, ConvSpec):
            out.append(op)
        elif isinstance(op, InceptionSpec):
            out += list(op.convs())
    return out


def make_layer(spec: ConvSpec, cfg: int, layer: int, g_m: int, g_n: int, mask_kind: str,
               mask_arg, seed: int = BASE_SEED):
    """Draw weights, bias and a KGS / vanilla mask for one layer.

    mask_kind: "none" | "exact_per_group" (mask_arg = k) | "bernoulli" (mask_arg = density)
               | "exact_total" (mask_arg = kept pairs) | "vanilla_total" (mask_arg = kept groups)
    Returns dict(w [M,N,Kt,Kh,Kw] f32, bias [M] f32, mask uint8 like w or None, gmask [P,Q,Ks] or None).
    """
    M, N = spec.cout, spec.cin
    Kt, Kh, Kw = spec.k
    Ks = Kt * Kh * Kw
    w = normal(stream_key(seed, cfg, layer, ROLE_WEIGHT), (M, N, Kt, Kh, Kw), 0.05)
    b = normal(stream_key(seed, cfg, layer, ROLE_BIAS), (M,), 0.01)
    P, Q = n_groups(M, N, g_m, g_n)
    mk = stream_key(seed, cfg, layer, ROLE_MASK)
    if mask_kind == "none":
        gmask = None
    elif mask_kind == "exact_per_group":
        gmask = kgs_mask_exact_per_group(P, Q, Ks, int(mask_arg), mk)
    elif mask_kind == "bernoulli":
        gmask = kgs_mask_bernoulli(P, Q, Ks, float(mask_arg), mk)
    elif mask_kind == "exact_total":
        gmask = kgs_mask_exact_total(P, Q, Ks, int(mask_arg), mk)
    elif mask_kind == "vanilla_total":
        gmask = vanilla_mask_exact_total(P, Q, Ks, int(mask_arg), mk)
    else:
        raise ValueError(mask_kind)
    mask = None if gmask is None else expand_group_mask(gmask, M, N, g_m, g_n, Kt, Kh, Kw)
    return {"w": w, "bias": b, "mask": mask, "gmask": gmask}


def make_input(cfg: int, shape, seed: int = BASE_SEED) -> np.ndarray:
    """Activation tensor [n,t,h,w,c] of U(-1,1) float32 draws."""
    return uniform_pm1(stream_key(seed, cfg, 0, ROLE_INPUT), shape)


def kept_fraction(gmask, spec: ConvSpec, g_m: int, g_n: int) -> float:
    """Kept MACs / dense MACs of a layer, counting only weights that exist (ragged groups)."""
    if gmask is None:
        return 1.0
    m = expand_group_mask(gmask, spec.cout, spec.cin, g_m, g_n, *spec.k)
    return float(m.sum()) / m.size
