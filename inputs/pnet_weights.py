"""Seeded random weights of the paper's own network, packed as its weight blob.

Only random draws and byte packing happen here.  Convolutions and linear maps He-normal
(std = sqrt(2 / fan_in)); folded batch-norm scale ~ N(1, 0.1) and bias ~ N(0, 0.1); linear biases
~ N(0, 0.1).  The residual branch scale 1/sqrt(blocks) is folded into every block's second scale
and bias, as the paper does at export (Sec. 4.3.6).  The query map and the promotion offsets are
multiplied by one stored scalar and the last value layer by another (pnet_head_scales.json,
written by the oracle's calibration script) so that the outputs are not saturated.

Blob layout (little-endian): 64-byte header = 8 bytes "AZPNET1\\0", uint32 version (= 1), blocks,
channels, key size, value channels, value hidden units, tensor count, zero padding; then raw
float32 tensors in the order of `tensor_shapes`.
"""
import json
import os
import struct
from collections import OrderedDict
from dataclasses import dataclass

import numpy as np

MAGIC = b"AZPNET1\0"
PLANES = 52
ACTIONS = 1880
MASK_WORDS = 30
_SCALES_PATH = os.path.join(os.path.dirname(os.path.abspath(__file__)), "pnet_head_scales.json")


@dataclass(frozen=True)
class PNetConfig:
    name: str
    blocks: int
    channels: int
    batch: int
    position_seed: int
    weight_seed: int
    key: int = 128
    value_channels: int = 2
    value_hidden: int = 48
    plies: tuple = (0, 160)
    precision: int = 1           # 1 = bf16, 3 = int8 tower (heads and pooled context in floating point)
    weights_like: str = ""       # name of the configuration whose head scales this one reuses

    # the same vocabulary as the other workloads' Config, so that callers can treat both alike
    in_planes = PLANES
    policy_head = 2
    value_head = 1
    policy_size = ACTIONS
    value_size = 3
    mask_words = MASK_WORDS


# the paper's network ladder (App. D.3): 12 x 128 and 14 x 160 (the reported checkpoint's size)
PNET_CONFIGS = {
    "p12": PNetConfig("p12", 12, 128, 1024, 20260961, 9371201),
    "p14": PNetConfig("p14", 14, 160, 320, 20260962, 9371401),
    # the largest stage of the paper's ladder (App. D.3)
    "p19": PNetConfig("p19", 19, 176, 296, 20260964, 9371901),
    # p12 with the backbone's convolutions in int8, the precision the paper deploys (Sec. 4.3.6)
    "p12i": PNetConfig("p12i", 12, 128, 1024, 20260961, 9371201, precision=3, weights_like="p12"),
    # the reported checkpoint's size in the precision the paper deploys it in (Sec. 4.3.6, App. B.1)
    "p14i": PNetConfig("p14i", 14, 160, 320, 20260962, 9371401, precision=3, weights_like="p14"),
}


def tiny(name="ptiny", blocks=3, channels=16, batch=8, weight_seed=5252, key=8) -> PNetConfig:
    return PNetConfig(name, blocks, channels, batch, 20260963, weight_seed, key=key)


def pooled(block: int) -> bool:
    """Every second block carries the global context: blocks 1, 3, 5, ..."""
    return block % 2 == 1


def tensor_shapes(cfg: PNetConfig) -> "OrderedDict[str, tuple]":
    C, K = cfg.channels, cfg.key
    P, R = C // 4, C - C // 4
    t = OrderedDict()
    t["in.w"], t["in.scale"], t["in.bias"] = (C, PLANES, 3, 3), (C,), (C,)
    for b in range(cfg.blocks):
        t[f"b{b}.w1"], t[f"b{b}.scale1"], t[f"b{b}.bias1"] = (C, C, 3, 3), (C,), (C,)
        if pooled(b):
            t[f"b{b}.gw"] = (R, 2 * P)
        t[f"b{b}.w2"] = (C, R if pooled(b) else C, 3, 3)
        t[f"b{b}.scale2"], t[f"b{b}.bias2"] = (C,), (C,)
    t["t.w"], t["t.b"] = (K, C), (K,)
    t["q.w"], t["q.b"] = (K, K), (K,)
    t["k.w"], t["k.b"] = (K, K), (K,)
    t["o.w"], t["o.b"] = (4, K), (4,)
    t["v.cw"], t["v.cscale"], t["v.cbias"] = (cfg.value_channels, C), (cfg.value_channels,), (cfg.value_channels,)
    t["v.w1"], t["v.b1"] = (cfg.value_hidden, cfg.value_channels * 64), (cfg.value_hidden,)
    t["v.w2"], t["v.b2"] = (3, cfg.value_hidden), (3,)
    return t


def head_scales(name: str):
    try:
        with open(_SCALES_PATH) as f:
            entry = json.load(f).get(name)
    except OSError:
        entry = None
    if entry is None:
        return 1.0, 1.0
    return float(entry["policy"]), float(entry["value"])


def draw_tensors(cfg: PNetConfig, policy_scale: float = None, value_scale: float = None):
    if policy_scale is None or value_scale is None:
        ps, vs = head_scales(cfg.weights_like or cfg.name)
        policy_scale = ps if policy_scale is None else policy_scale
        value_scale = vs if value_scale is None else value_scale
    rng = np.random.Generator(np.random.PCG64(cfg.weight_seed))
    out = OrderedDict()
    for name, shape in tensor_shapes(cfg).items():
        leaf = name.split(".")[1]
        if "scale" in leaf:
            a = rng.normal(1.0, 0.1, size=shape)
        elif "bias" in leaf or leaf in ("b", "b1", "b2"):
            a = rng.normal(0.0, 0.1, size=shape)
        else:
            fan_in = int(np.prod(shape[1:]))
            a = rng.normal(0.0, np.sqrt(2.0 / fan_in), size=shape)
        out[name] = a.astype(np.float32)
    branch = np.float32(cfg.blocks ** -0.5) if cfg.blocks else np.float32(1.0)
    for b in range(cfg.blocks):
        for k in (f"b{b}.scale2", f"b{b}.bias2"):
            out[k] = (out[k] * branch).astype(np.float32)
    for k in ("q.w", "q.b", "o.w", "o.b"):
        out[k] = (out[k] * np.float32(policy_scale)).astype(np.float32)
    for k in ("v.w2", "v.b2"):
        out[k] = (out[k] * np.float32(value_scale)).astype(np.float32)
    return out


def pack_blob(cfg: PNetConfig, tensors) -> np.ndarray:
    header = MAGIC + struct.pack("<7I", 1, cfg.blocks, cfg.channels, cfg.key, cfg.value_channels,
                                 cfg.value_hidden, len(tensors))
    header = header + b"\0" * (64 - len(header))
    parts = [np.frombuffer(header, dtype=np.uint8)]
    for name, shape in tensor_shapes(cfg).items():
        a = np.ascontiguousarray(tensors[name], dtype="<f4")
        assert a.shape == tuple(shape), (name, a.shape, shape)
        parts.append(a.reshape(-1).view(np.uint8))
    return np.concatenate(parts)


def make_blob(cfg: PNetConfig, policy_scale: float = None, value_scale: float = None) -> np.ndarray:
    return pack_blob(cfg, draw_tensors(cfg, policy_scale, value_scale))


def parameter_count(cfg: PNetConfig) -> int:
    return int(sum(np.prod(s) for s in tensor_shapes(cfg).values()))
