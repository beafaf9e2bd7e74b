"""Oracle-side forward passes of the two network-shaped workloads (test infrastructure).

Built only from the oracle and the shared shape tables; shares nothing with the CUDA path.
Each layer's output is rounded to bfloat16 before it feeds the next layer, mirroring the
storage precision of the bf16 data flow.  For every op the function records the exact input
it consumed (already bf16-representable) and the un-rounded float output, so a test can hand
the same input to the CUDA library (teacher forcing) and compare against the output.
"""
import numpy as np

import oracle
import rt3d_synth as synth


def make_c3d_layers(cfg, density, g_m=4, g_n=4, dense=False):
    plan = synth.c3d_plan()
    layers = {}
    for i, op in enumerate(plan):
        if isinstance(op, synth.ConvSpec):
            layers[op.name] = synth.make_layer(op, cfg, i, g_m, g_n, "none" if dense else "bernoulli", density)
    return plan, layers


def c3d_reference(plan, layers, x):
    """x: float32 [n,16,112,112,3] (bf16-representable).  Returns (records, final) where
    records[name] = (input, output_unrounded)."""
    rec = {}
    cur = x
    for op in plan:
        if isinstance(op, synth.ConvSpec):
            L = layers[op.name]
            out = oracle.conv3d(cur, L["w"], L["mask"], L["bias"], op.stride, op.pad, op.relu, round_bf16=True)
            rec[op.name] = (cur, out)
            cur = oracle.bf16_round(out)
        else:
            out = oracle.maxpool3d(cur, op.k, op.stride, op.pad)
            rec[op.name] = (cur, out)
            cur = out
    return rec, cur


def make_r2plus1d_layers(cfg, density, g_m=4, g_n=4):
    stem, blocks = synth.r2plus1d18_plan()
    specs = list(stem)
    for blk in blocks:
        specs += list(blk.convs)
        if blk.shortcut is not None:
            specs.append(blk.shortcut)
    layers = {sp.name: synth.make_layer(sp, cfg, i, g_m, g_n, "bernoulli", density) for i, sp in enumerate(specs)}
    return stem, blocks, layers


def r2plus1d_reference(stem, blocks, layers, x):
    rec = {}

    def conv(sp, inp):
        L = layers[sp.name]
        out = oracle.conv3d(inp, L["w"], L["mask"], L["bias"], sp.stride, sp.pad, sp.relu, round_bf16=True)
        rec[sp.name] = (inp, out)
        return oracle.bf16_round(out)

    cur = x
    for sp in stem:
        cur = conv(sp, cur)
    for blk in blocks:
        inp = cur
        for sp in blk.convs:
            cur = conv(sp, cur)
        sc = inp if blk.shortcut is None else conv(blk.shortcut, inp)
        out = oracle.add_relu(cur, sc, True)
        rec[blk.name + ".out"] = ((cur, sc), out)
        cur = oracle.bf16_round(out)
    return rec, cur


def make_s3d_layers(cfg, density, g_m=4, g_n=4):
    plan = synth.s3d_plan()
    layers = {sp.name: synth.make_layer(sp, cfg, i, g_m, g_n, "bernoulli", density)
              for i, sp in enumerate(synth.s3d_convs(plan))}
    return plan, layers


def s3d_reference(plan, layers, x):
    """Oracle forward of the S3D-shaped network; records[name] = (input, unrounded output) per conv / pool,
    records[block] = (input, concatenated bf16 output) per Inception block."""
    rec = {}

    def conv(sp, inp):
        L = layers[sp.name]
        out = oracle.conv3d(inp, L["w"], L["mask"], L["bias"], sp.stride, sp.pad, sp.relu, round_bf16=True)
        rec[sp.name] = (inp, out)
        return oracle.bf16_round(out)

    def pool(sp, inp):
        out = oracle.maxpool3d(inp, sp.k, sp.stride, sp.pad)
        rec[sp.name] = (inp, out)
        return out

    cur = x
    for op in plan:
        if isinstance(op, synth.ConvSpec):
            cur = conv(op, cur)
        elif isinstance(op, synth.PoolSpec):
            cur = pool(op, cur)
        else:
            inp = cur
            parts = [conv(op.b0, inp)]
            for br in (op.b1, op.b2):
                t = inp
                for sp in br:
                    t = conv(sp, t)
                parts.append(t)
            parts.append(conv(op.b3, pool(op.pool, inp)))
            cur = np.concatenate(parts, axis=-1)
            rec[op.name] = (inp, cur)
    return rec, cur


def make_c3d_fc_layers(cfg):
    return {sp.name: synth.make_layer(sp, cfg, 100 + i, 4, 4, "none", None) for i, sp in enumerate(synth.c3d_fc_tail())}


def c3d_fc_reference(fc_layers, feat):
    """feat: bf16-representable pool5 output [n,1,4,4,512]; returns records and the logits [n,1,1,1,101]."""
    rec = {}
    cur = feat.reshape(feat.shape[0], 1, 1, 1, -1)
    for sp in synth.c3d_fc_tail():
        L = fc_layers[sp.name]
        out = oracle.conv3d(cur, L["w"], None, L["bias"], sp.stride, sp.pad, sp.relu, round_bf16=True)
        rec[sp.name] = (cur, out)
        cur = oracle.bf16_round(out)
    return rec, cur
