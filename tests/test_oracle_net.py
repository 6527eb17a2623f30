"""Pins for the oracle's network arithmetic and masked softmax (CPU only)."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from inputs import configs, positions, weights


def im2col_conv(w: np.ndarray, x: np.ndarray) -> np.ndarray:
    """Brute force: build the [64][cin*9] patch matrix and multiply by the [cin*9][cout] weights."""
    cout, cin = w.shape[:2]
    cols = np.zeros((64, cin * 9))
    for y in range(8):
        for xx in range(8):
            for ci in range(cin):
                for ky in range(3):
                    for kx in range(3):
                        yy, xc = y + ky - 1, xx + kx - 1
                        if 0 <= yy < 8 and 0 <= xc < 8:
                            cols[y * 8 + xx, ci * 9 + ky * 3 + kx] = x[ci, yy, xc]
    out = cols @ w.reshape(cout, cin * 9).astype(np.float64).T
    return out.T.reshape(cout, 8, 8)


@pytest.mark.parametrize("cin,cout", [(1, 1), (3, 5), (19, 8), (16, 16)])
def test_direct_summation_equals_im2col_product(cin, cout):
    rng = np.random.default_rng(cin * 100 + cout)
    w = rng.normal(size=(cout, cin, 3, 3)).astype(np.float32)
    x = rng.normal(size=(cin, 8, 8))
    assert np.abs(oracle.conv3x3(w, x) - im2col_conv(w, x)).max() < 1e-12


def test_conv_closed_forms():
    rng = np.random.default_rng(0)
    x = rng.normal(size=(4, 8, 8))
    ident = np.zeros((4, 4, 3, 3), dtype=np.float32)
    for c in range(4):
        ident[c, c, 1, 1] = 1.0
    assert (oracle.conv3x3(ident, x) == x).all()
    # all-ones kernel on all-ones planes counts the on-board neighbours: 9 inside, 6 on an edge,
    # 4 in a corner, times the number of input channels
    ones = oracle.conv3x3(np.ones((2, 5, 3, 3), dtype=np.float32), np.ones((5, 8, 8)))
    assert ones[0, 3, 3] == 45 and ones[1, 0, 4] == 30 and ones[0, 7, 0] == 20 and ones[1, 4, 7] == 30
    # a kernel with a single off-centre tap shifts the plane: W[.,.,0,2] reads in[y-1][x+1]
    shift = np.zeros((1, 1, 3, 3), dtype=np.float32)
    shift[0, 0, 0, 2] = 1.0
    plane = np.arange(64, dtype=np.float64).reshape(1, 8, 8)
    got = oracle.conv3x3(shift, plane)[0]
    assert got[3, 2] == plane[0, 2, 3] and got[0, 0] == 0 and got[5, 7] == 0


def test_conv_matches_library_float64():
    rng = np.random.default_rng(5)
    w = rng.normal(size=(24, 40, 3, 3)).astype(np.float32)
    x = rng.normal(size=(40, 8, 8))
    ref = F.conv2d(torch.from_numpy(x)[None], torch.from_numpy(w.astype(np.float64)), padding=1)[0].numpy()
    assert np.abs(oracle.conv3x3(w, x) - ref).max() < 1e-10


def torch_forward(cfg, T, planes):
    """The same network as a float64 composition of library ops."""
    tt = {k: torch.from_numpy(v.astype(np.float64)) for k, v in T.items()}
    sb = lambda x, s, b: x * tt[s].view(1, -1, 1, 1) + tt[b].view(1, -1, 1, 1)
    h = F.relu(sb(F.conv2d(torch.from_numpy(planes), tt["in.w"], padding=1), "in.scale", "in.bias"))
    for b in range(cfg.blocks):
        t = F.relu(sb(F.conv2d(h, tt[f"b{b}.w1"], padding=1), f"b{b}.scale1", f"b{b}.bias1"))
        h = F.relu(h + sb(F.conv2d(t, tt[f"b{b}.w2"], padding=1), f"b{b}.scale2", f"b{b}.bias2"))
    if cfg.policy_head == 0:
        logits = (F.conv2d(h, tt["p.w"][:, :, None, None]) + tt["p.bias"].view(1, -1, 1, 1)).flatten(1)
    else:
        pc = F.relu(sb(F.conv2d(h, tt["p.cw"][:, :, None, None]), "p.cscale", "p.cbias"))
        logits = F.linear(pc.flatten(1), tt["p.fw"], tt["p.fbias"])
    vc = F.relu(sb(F.conv2d(h, tt["v.cw"][:, :, None, None]), "v.cscale", "v.cbias"))
    z = F.linear(F.relu(F.linear(vc.flatten(1), tt["v.w1"], tt["v.b1"])), tt["v.w2"], tt["v.b2"])
    value = torch.tanh(z) if cfg.value_head == 0 else torch.softmax(z, dim=1)
    return h.numpy(), logits.numpy(), z.numpy(), value.numpy()


@pytest.mark.parametrize("policy_head,value_head,in_planes", [(0, 0, 19), (1, 1, 19), (1, 1, 112), (0, 1, 112)])
def test_whole_network_matches_library_composition(policy_head, value_head, in_planes):
    cfg = configs.tiny_config(in_planes=in_planes, blocks=3, channels=24, policy_head=policy_head,
                              value_head=value_head, weight_seed=100 + policy_head + 2 * value_head)
    T = weights.draw_tensors(cfg, 0.05, 0.2)
    blob = weights.pack_blob(cfg, T)
    rec, _ = positions.generate(77, 12, (0, 60))
    recs = positions.records_for_planes(in_planes, rec)
    masks, planes, policy, value, raw = oracle.evaluate(blob, recs, in_planes, policy_head,
                                                        want_raw=True, want_tower=True)
    h, logits, z, val = torch_forward(cfg, T, planes)
    scale = np.abs(h).max()
    assert np.abs(raw["tower"] - h).max() < 1e-9 * scale
    assert np.abs(raw["logits"] - logits).max() < 1e-9 * max(1.0, np.abs(logits).max())
    assert np.abs(raw["value_pre"] - z).max() < 1e-9 * max(1.0, np.abs(z).max())
    assert np.abs(value - val).max() < 1e-9
    # masked softmax against the library's softmax with -inf on illegal entries
    for i in range(recs.shape[0]):
        bits = np.unpackbits(masks[i].view(np.uint8), bitorder="little")[: cfg.policy_size].astype(bool)
        lg = torch.from_numpy(np.where(bits, logits[i], -np.inf))
        assert np.abs(torch.softmax(lg, 0).numpy() - policy[i]).max() < 1e-12
        assert (policy[i][~bits] == 0.0).all()
        assert abs(policy[i].sum() - 1.0) < 1e-12
    if value_head == 0:
        assert (np.abs(value) <= 1.0).all()
    else:
        assert np.abs(value.sum(axis=1) - 1.0).max() < 1e-12 and (value >= 0).all()


def test_residual_block_with_zero_branch_is_the_identity_on_nonnegative_input():
    cfg = configs.tiny_config(blocks=2, channels=8)
    T = weights.draw_tensors(cfg, 1.0, 1.0)
    for b in range(cfg.blocks):
        T[f"b{b}.w2"][:] = 0
        T[f"b{b}.bias2"][:] = 0
    rec, _ = positions.generate(1, 4, (0, 40))
    recs = positions.cur_records(rec)
    _, planes, _, _, raw = oracle.evaluate(weights.pack_blob(cfg, T), recs, 19, 0, want_tower=True)
    T0 = {k: v for k, v in T.items()}
    cfg0 = configs.tiny_config(blocks=0, channels=8)
    T0 = {k: v for k, v in T.items() if not k.startswith("b")}
    _, _, _, _, raw0 = oracle.evaluate(weights.pack_blob(cfg0, T0), recs, 19, 0, want_tower=True)
    assert (raw["tower"] == raw0["tower"]).all() and raw["tower"].min() >= 0


def test_residual_add_comes_before_the_second_activation():
    # one block, conv2 = -identity with unit scale: h + (-t) where t = relu(conv1(h)).  With conv1 =
    # identity, t = h (h >= 0) and the block must output relu(h - h) = 0.
    cfg = configs.tiny_config(blocks=1, channels=8)
    T = weights.draw_tensors(cfg, 1.0, 1.0)
    for k, sign in (("b0.w1", 1.0), ("b0.w2", -1.0)):
        T[k][:] = 0
        for c in range(8):
            T[k][c, c, 1, 1] = sign
    for k in ("b0.scale1", "b0.scale2"):
        T[k][:] = 1
    for k in ("b0.bias1", "b0.bias2"):
        T[k][:] = 0
    rec, _ = positions.generate(2, 3, (0, 40))
    _, _, _, _, raw = oracle.evaluate(weights.pack_blob(cfg, T), positions.cur_records(rec), 19, 0, want_tower=True)
    assert np.abs(raw["tower"]).max() < 1e-12
    T["b0.bias2"][:] = 0.25          # bias lands inside the final ReLU: output = relu(0 + 0.25)
    _, _, _, _, raw = oracle.evaluate(weights.pack_blob(cfg, T), positions.cur_records(rec), 19, 0, want_tower=True)
    assert np.abs(raw["tower"] - 0.25).max() < 1e-12


def test_masked_softmax_invariants():
    rng = np.random.default_rng(9)
    logits = rng.normal(size=1858) * 3
    mask = np.zeros(30, dtype=np.uint64)
    legal = rng.choice(1858, size=31, replace=False)
    for i in legal:
        mask[i >> 6] |= np.uint64(1) << np.uint64(i & 63)
    p = oracle.masked_softmax(logits, mask)
    assert abs(p.sum() - 1) < 1e-12 and (p[np.setdiff1d(np.arange(1858), legal)] == 0).all()
    assert np.abs(oracle.masked_softmax(logits + 123.456, mask) - p).max() < 1e-12      # shift invariance
    assert np.abs(oracle.masked_softmax(np.full(1858, 2.5), mask)[legal] - 1 / 31).max() < 1e-15
    # a huge illegal logit must not disturb the legal ones
    big = logits.copy()
    big[np.setdiff1d(np.arange(1858), legal)[0]] = 1e6
    assert np.abs(oracle.masked_softmax(big, mask) - p).max() == 0
    # ratio of two legal probabilities is exp of the logit difference
    a, b = legal[0], legal[1]
    assert abs(np.log(p[a] / p[b]) - (logits[a] - logits[b])) < 1e-9
    # no legal move: all-zero row
    assert (oracle.masked_softmax(logits, np.zeros(30, dtype=np.uint64)) == 0).all()


def test_stored_head_scales_give_unsaturated_outputs():
    cfg = configs.CONFIGS["c1"]
    blob = weights.make_blob(cfg)
    rec = positions.for_config(cfg, 32, calibration=True)
    masks, _, policy, value, raw = oracle.evaluate(blob, positions.cur_records(rec), 19, 0, want_raw=True)
    top = policy.max(axis=1)
    assert 0.05 < top.mean() < 0.6 and np.abs(value).max() < 0.999
