"""Pins of oracle/quant_emul.py, and the floors it gives for the reduced-precision towers.

The emulation rounds the operands of every tensor-core product to the format in question and keeps
everything else exact.  Its rounding functions are pinned here against what defines the formats (the
code points themselves, ties, saturation) and against a library's converters; its exact mode against
the C oracle.  The floors asserted at the end are the figures the design notes quote: no kernel can be
closer to the fp64 oracle than these, whatever its quality.
"""
import json
import os

import numpy as np
import pytest
import torch

import oracle
from inputs import configs, positions, weights
from oracle import quant_emul as qe


def all_e4m3_values():
    """The 254 finite code points of e4m3, from their definition: sign, 4 exponent bits (bias 7), 3 mantissa bits;
    exponent field 0 is subnormal (m/8 * 2^-6); exponent 15 with mantissa 7 is NaN."""
    vals = []
    for e in range(16):
        for m in range(8):
            if e == 15 and m == 7:
                continue
            v = (m / 8.0) * 2.0 ** -6 if e == 0 else (1.0 + m / 8.0) * 2.0 ** (e - 7)
            vals += [v, -v]
    return np.array(sorted(set(vals)))


def test_e4m3_code_points_ties_and_saturation():
    vals = all_e4m3_values()
    assert vals.max() == 448.0 and len(vals) == 253              # +0 and -0 coincide
    t = torch.from_numpy(vals)
    assert torch.equal(qe.round_e4m3(t), t)                       # every code point is a fixed point
    pos = vals[vals >= 0]
    mid = (pos[:-1] + pos[1:]) / 2
    got = qe.round_e4m3(torch.from_numpy(mid)).numpy()
    # a midpoint goes to the neighbour with the even mantissa: the neighbours alternate even / odd, index 0 is zero
    want = np.where(np.arange(len(mid)) % 2 == 0, pos[:-1], pos[1:])
    assert (got == want).all()
    # just off the midpoint: the nearer neighbour
    assert (qe.round_e4m3(torch.from_numpy(mid * (1 + 1e-9))).numpy() == pos[1:]).all()
    assert (qe.round_e4m3(torch.from_numpy(mid * (1 - 1e-9))).numpy() == pos[:-1]).all()
    big = torch.tensor([448.0, 449.0, 464.0, 480.0, 1e6, -1e6], dtype=torch.float64)
    assert qe.round_e4m3(big).tolist() == [448.0, 448.0, 448.0, 448.0, 448.0, -448.0]
    # relative error of a normal number is at most half a unit in the last place, 2^-4
    x = torch.from_numpy(np.random.default_rng(1).uniform(2.0 ** -6, 448.0, 20000))
    assert float(((qe.round_e4m3(x) - x).abs() / x).max()) <= 2.0 ** -4


def test_rounding_agrees_with_the_library_converters():
    rng = np.random.default_rng(2)
    x = torch.from_numpy(np.concatenate([rng.normal(0, s, 20000) for s in (1e-3, 0.1, 3.0, 100.0)]))
    x32 = x.to(torch.float32).to(torch.float64)                   # the library converts from float32
    lib = x32.to(torch.float32).clamp(-448, 448).to(torch.float8_e4m3fn).to(torch.float64)
    assert torch.equal(qe.round_e4m3(x32), lib)
    assert torch.equal(qe.round_bf16(x32), x32.to(torch.float32).to(torch.bfloat16).to(torch.float64))
    # bf16 ties: 1 + 2^-8 lies half-way between 1 and 1 + 2^-7 -> even mantissa (1); 1 + 3 * 2^-8 -> 1 + 2^-6
    t = torch.tensor([1 + 2.0 ** -8, 1 + 3 * 2.0 ** -8, -(1 + 2.0 ** -8), 2.0 ** -130], dtype=torch.float64)
    assert qe.round_bf16(t).tolist() == [1.0, 1 + 2.0 ** -6, -1.0, 2.0 ** -130]
    assert qe.round_u8(torch.tensor([-3.0, 0.5, 1.5, 2.5, 254.6, 300.0], dtype=torch.float64)).tolist() == [0, 0, 2, 2, 255, 255]
    assert qe.round_s8(torch.tensor([-200.0, -127.5, -0.5, 0.5, 126.5, 127.5], dtype=torch.float64)).tolist() == [-127, -127, 0, 0, 126, 127]


def test_split_operands_carry_about_twice_the_bits():
    x = torch.from_numpy(np.random.default_rng(3).uniform(1.0, 448.0, 20000))
    hi, lo = qe._split(x, qe.round_e4m3)
    assert torch.equal(hi, qe.round_e4m3(x)) and torch.equal(lo, qe.round_e4m3(lo))
    assert float(((hi + lo - x).abs() / x).max()) <= 2.0 ** -7     # remainder <= 2^-4 |x|, itself rounded to 2^-4


@pytest.mark.parametrize("policy_head,value_head", [(0, 0), (1, 1)])
def test_exact_mode_is_the_oracle(policy_head, value_head):
    cfg = configs.tiny_config(blocks=2, channels=16, policy_head=policy_head, value_head=value_head, batch=6)
    tensors = weights.draw_tensors(cfg, 0.05, 0.1)
    blob = weights.pack_blob(cfg, tensors)
    recs = positions.cur_records(positions.generate(77, 6, (0, 90))[0])
    masks, planes, pol0, val0, raw = oracle.evaluate(blob, recs, 19, policy_head, want_raw=True, want_tower=True)
    net = qe.ResidualTower(cfg, tensors)
    h = net.run(torch.from_numpy(planes), qe.Spec("exact"))
    pol, val, lg, z = net.heads(h, masks, lambda t: t)
    assert np.abs(h.numpy() - raw["tower"]).max() <= 1e-12 * np.abs(raw["tower"]).max()
    assert np.abs(pol.numpy() - pol0).max() <= 1e-12 and np.abs(val.numpy() - val0).max() <= 1e-12
    assert np.abs(z.numpy() - raw["value_pre"]).max() <= 1e-12
    # an 8-bit spec whose rounding is switched off must also reproduce it: the scales cancel exactly enough
    ident = lambda t: t
    old = qe._limits
    try:
        qe._limits = lambda kind: (448.0, 448.0, ident, ident)
        sa, _ = net.calibrate(torch.from_numpy(planes), qe.Spec("e4m3"))
        h8 = net.run(torch.from_numpy(planes), qe.Spec("e4m3"), sa=sa)
    finally:
        qe._limits = old
    hb = net.run(torch.from_numpy(planes), qe.Spec("bf16"))
    # (layer 0 keeps bf16 operands in an 8-bit spec; the rest is exact here, so the result lies nearer to exact than bf16 does)
    assert (h8 - torch.from_numpy(raw["tower"])).abs().max() <= (hb - torch.from_numpy(raw["tower"])).abs().max() * 1.5


def test_paper_network_exact_mode_is_the_oracle():
    from inputs import pnet_weights
    cfg = pnet_weights.tiny(blocks=4, channels=16, key=8)
    tensors = pnet_weights.draw_tensors(cfg, 1.0, 1.0)
    blob = pnet_weights.pack_blob(cfg, tensors)
    rec, _ = positions.generate_moves(99, 5, (0, 120))
    masks, planes, pol0, val0, raw = oracle.pnet_evaluate(blob, rec, want_raw=True, want_tower=True)
    net = qe.PaperTower(cfg, tensors)
    h = net.run(torch.from_numpy(planes), qe.Spec("exact"))
    pol, val, lg, z = net.heads(h, masks, lambda t: t)
    assert np.abs(h.numpy() - raw["tower"]).max() <= 1e-11
    assert np.abs(pol.numpy() - pol0).max() <= 1e-11 and np.abs(val.numpy() - val0).max() <= 1e-11


# ---- the floors --------------------------------------------------------------------------------------

def test_bf16_floor_of_the_20x128_towers():
    # bf16 operands, exact accumulation: the towers end 0.4-0.7 % rms off; what the value heads make of that
    # differs by weight set: a tenth of the spread for c2's scalar head, under a hundredth for c3's
    c2 = qe.residual_report("c2", 64, (qe.Spec("bf16"),))["bf16"]
    c3 = qe.residual_report("c3", 64, (qe.Spec("bf16"),))["bf16"]
    print("c2", c2)
    print("c3", c3)
    assert 0.004 < c2["tower_rms"] < 0.008 and 0.003 < c3["tower_rms"] < 0.008
    assert 0.06 < c2["value_pre_rms_over_spread"] < 0.15
    assert c3["value_pre_rms_over_spread"] < 0.02
    assert c2["policy_max_abs"] < 2e-2 and c3["policy_max_abs"] < 2e-2
    # at a spread of 0.5 the floor of c2's tanh output alone is beyond the 2e-2 bar; c3's is far inside
    c2w = qe.residual_report("c2", 64, (qe.Spec("bf16"),), value_spread=0.5)["bf16"]
    assert c2w["value_max_abs"] > 2e-2
    assert c3["value_max_abs"] < 1e-2 and 0.4 < c3["value_pre_spread"] < 0.65


def test_e4m3_floor_of_the_plain_residual_tower():
    # c4 as specified: e4m3 weights and activations with per-channel scales, exact accumulation, bf16 heads; with
    # and without the bias correction.  The tower ends 7-10 % rms off and the policy beyond the 5e-2 bar, before any
    # kernel is involved.  (64 positions, ranges from 128 calibration positions to keep the test short; the stored
    # figures in tests/golden/quant_floors.json come from 128 / 512.)
    rep = qe.residual_report("c4", 64, (qe.Spec("e4m3"), qe.Spec("e4m3", bias_correction=True),
                                        qe.Spec("e4m3", split_w=True, split_a=True)), n_cal=128)
    for k, v in rep.items():
        print(k, v)
    plain, bc, split = rep["e4m3"], rep["e4m3, bias correction"], rep["e4m3, split weights, split activations"]
    assert 0.07 < plain["tower_rms"] < 0.11 and 0.055 < bc["tower_rms"] < 0.09
    assert plain["policy_max_abs"] > 5e-2 and bc["policy_max_abs"] > 5e-2
    # two e4m3 numbers per operand (three products per layer) bring it inside with room to spare
    assert split["tower_rms"] < 0.01 and split["policy_max_abs"] < 2e-2 and split["value_max_abs"] < 2e-2


def test_stored_floors_are_what_the_emulation_gives():
    with open(qe.GOLDEN) as f:
        table = json.load(f)
    for name in ("c2", "c2@0.5", "c3", "c5", "c5@0.5", "c4", "c4b", "p12"):
        assert name in table, name
    # one entry recomputed in full: the file is the emulation's output, not typed in
    n, spread, specs = qe.FLOOR_RUNS["c2"]
    rep = qe.residual_report("c2", n, specs, value_spread=spread)
    for k, v in rep["bf16"].items():
        assert abs(v - table["c2"]["bf16"][k]) <= 1e-9 * max(1.0, abs(v)), k
    assert os.path.getsize(qe.GOLDEN) < 64 * 1024
