"""Seeded random network weights, packed as the library's weight blob.

Only random draws and byte packing happen here; nothing of the network's arithmetic.  Draws:
convolution and fully-connected weights He-normal (std = sqrt(2 / fan_in)); folded batch-norm
scale ~ N(1, 0.1) and bias ~ N(0, 0.1); fully-connected biases ~ N(0, 0.1).  The last linear
layer of each head is then multiplied by a stored scalar (head_scales.json, written by the
oracle's calibration script) so that policy and value outputs are not saturated.

Blob layout (little-endian): a 64-byte header
    8 bytes magic "AZNETv1\\0", then uint32 version(=1), in_planes, blocks, channels,
    policy_head, value_head, tensor_count, and zero padding to 64 bytes,
followed by raw float32 tensors, in this order, with no per-tensor headers:
    input conv   W[C][P][3][3], scale[C], bias[C]
    per block    W1[C][C][3][3], scale1[C], bias1[C], W2[C][C][3][3], scale2[C], bias2[C]
    policy head  (0) Wp[73][C], bp[73]
                 (1) Wpc[32][C], scale_pc[32], bias_pc[32], Wpf[1858][2048], bpf[1858]
    value head   Wvc[32][C], scale_vc[32], bias_vc[32], Wv1[128][2048], bv1[128],
                 Wv2[V][128], bv2[V]   (V = 1 scalar head, 3 win/draw/loss head)
"""
import json
import os
import struct
from collections import OrderedDict

import numpy as np

from .configs import HEAD_CHANNELS, POLICY_SIZE, VALUE_HIDDEN, VALUE_SIZE, Config

MAGIC = b"AZNETv1\0"
HEADER_BYTES = 64
_SCALES_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "head_scales.json")


def tensor_shapes(cfg: Config) -> "OrderedDict[str, tuple]":
    C, P = cfg.channels, cfg.in_planes
    t = OrderedDict()
    t["in.w"], t["in.scale"], t["in.bias"] = (C, P, 3, 3), (C,), (C,)
    for b in range(cfg.blocks):
        t[f"b{b}.w1"], t[f"b{b}.scale1"], t[f"b{b}.bias1"] = (C, C, 3, 3), (C,), (C,)
        t[f"b{b}.w2"], t[f"b{b}.scale2"], t[f"b{b}.bias2"] = (C, C, 3, 3), (C,), (C,)
    if cfg.policy_head == 0:
        t["p.w"], t["p.bias"] = (73, C), (73,)
    else:
        t["p.cw"], t["p.cscale"], t["p.cbias"] = (HEAD_CHANNELS, C), (HEAD_CHANNELS,), (HEAD_CHANNELS,)
        t["p.fw"], t["p.fbias"] = (POLICY_SIZE[1], HEAD_CHANNELS * 64), (POLICY_SIZE[1],)
    t["v.cw"], t["v.cscale"], t["v.cbias"] = (HEAD_CHANNELS, C), (HEAD_CHANNELS,), (HEAD_CHANNELS,)
    t["v.w1"], t["v.b1"] = (VALUE_HIDDEN, HEAD_CHANNELS * 64), (VALUE_HIDDEN,)
    V = VALUE_SIZE[cfg.value_head]
    t["v.w2"], t["v.b2"] = (V, VALUE_HIDDEN), (V,)
    return t


def head_scales(name: str):
    """(policy, value) multipliers stored for the named weight set; (1, 1) if none stored."""
    try:
        with open(_SCALES_PATH) as f:
            table = json.load(f)
    except OSError:
        return 1.0, 1.0
    entry = table.get(name)
    if entry is None:
        return 1.0, 1.0
    return float(entry["policy"]), float(entry["value"])


def draw_tensors(cfg: Config, policy_scale: float = None, value_scale: float = None):
    """Named float32 tensors in blob order."""
    if policy_scale is None or value_scale is None:
        ps, vs = head_scales(cfg.weights_name)
        policy_scale = ps if policy_scale is None else policy_scale
        value_scale = vs if value_scale is None else value_scale
    rng = np.random.Generator(np.random.PCG64(cfg.weight_seed))
    out = OrderedDict()
    for name, shape in tensor_shapes(cfg).items():
        leaf = name.split(".")[1]
        if "scale" in leaf:
            a = rng.normal(1.0, 0.1, size=shape)
        elif "bias" in leaf or leaf in ("b1", "b2"):
            a = rng.normal(0.0, 0.1, size=shape)
        else:
            fan_in = int(np.prod(shape[1:]))
            a = rng.normal(0.0, np.sqrt(2.0 / fan_in), size=shape)
        out[name] = a.astype(np.float32)
    if cfg.branch_scale != 1.0:
        for b in range(cfg.blocks):
            for k in (f"b{b}.scale2", f"b{b}.bias2"):
                out[k] = (out[k] * np.float32(cfg.branch_scale)).astype(np.float32)
    last_policy = ("p.w", "p.bias") if cfg.policy_head == 0 else ("p.fw", "p.fbias")
    for k in last_policy:
        out[k] = (out[k] * np.float32(policy_scale)).astype(np.float32)
    for k in ("v.w2", "v.b2"):
        out[k] = (out[k] * np.float32(value_scale)).astype(np.float32)
    return out


def pack_blob(cfg: Config, tensors) -> np.ndarray:
    header = MAGIC + struct.pack("<7I", 1, cfg.in_planes, cfg.blocks, cfg.channels,
                                 cfg.policy_head, cfg.value_head, len(tensors))
    header = header + b"\0" * (HEADER_BYTES - len(header))
    parts = [np.frombuffer(header, dtype=np.uint8)]
    for name, shape in tensor_shapes(cfg).items():
        a = np.ascontiguousarray(tensors[name], dtype="<f4")
        assert a.shape == tuple(shape), (name, a.shape, shape)
        parts.append(a.reshape(-1).view(np.uint8))
    return np.concatenate(parts)


def make_blob(cfg: Config, policy_scale: float = None, value_scale: float = None) -> np.ndarray:
    return pack_blob(cfg, draw_tensors(cfg, policy_scale, value_scale))
