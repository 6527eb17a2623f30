"""Pins of the oracle's implementation of the paper's network (Sec. 3.2, 4.3, App. D.1): the whole
network against a float64 composition of library operators, and closed forms that single out the
capped activation, the pooled context, the query-key score and the promotion offsets."""
import numpy as np
import pytest
import torch
import torch.nn.functional as F

import oracle
from inputs import pnet_weights as pw
from inputs import positions


def library_forward(cfg, tensors, planes, masks):
    """float64 composition of library operators, written from the description of the network."""
    t = {k: torch.from_numpy(np.asarray(v, dtype=np.float64)) for k, v in tensors.items()}
    x = torch.from_numpy(planes)
    C, P = cfg.channels, cfg.channels // 4
    R = C - P

    def bn(y, s, b):
        return y * t[s].view(1, -1, 1, 1) + t[b].view(1, -1, 1, 1)

    def cap(y):
        return torch.clamp(y, 0.0, 6.0)

    h = cap(bn(F.conv2d(x, t["in.w"], padding=1), "in.scale", "in.bias"))
    for b in range(cfg.blocks):
        y = bn(F.conv2d(h, t[f"b{b}.w1"], padding=1), f"b{b}.scale1", f"b{b}.bias1")
        if pw.pooled(b):
            pool = cap(y[:, R:])
            g_in = torch.cat([pool.mean(dim=(2, 3)), pool.amax(dim=(2, 3))], dim=1)
            y = cap(y[:, :R] + (g_in @ t[f"b{b}.gw"].T).view(-1, R, 1, 1))
        else:
            y = cap(y)
        y = bn(F.conv2d(y, t[f"b{b}.w2"], padding=1), f"b{b}.scale2", f"b{b}.bias2")
        h = cap(h + y)
    n = h.shape[0]
    feat = h.reshape(n, C, 64)
    u = torch.einsum("kc,ncs->nks", t["t.w"], feat) + t["t.b"].view(1, -1, 1)
    q = torch.einsum("jk,nks->njs", t["q.w"], u) + t["q.b"].view(1, -1, 1)
    k = torch.einsum("jk,nks->njs", t["k.w"], u) + t["k.b"].view(1, -1, 1)
    o = torch.einsum("pk,nks->nps", t["o.w"], u) + t["o.b"].view(1, -1, 1)
    score = torch.einsum("ndf,ndt->nft", q, k) / np.sqrt(cfg.key)
    logits = torch.zeros((n, pw.ACTIONS), dtype=torch.float64)
    for f in range(64):
        for to in range(64):
            i = oracle.policy_index(2, 0, f, to, 0, 0)
            if i >= 0:
                logits[:, i] = score[:, f, to]
            for promo in (1, 2, 3, 4):
                j = oracle.policy_index(2, 0, f, to, promo, 0)
                if j >= 0:
                    logits[:, j] = score[:, f, to] + o[:, 4 - promo, f]
    bits = torch.from_numpy(np.unpackbits(masks.view(np.uint8), axis=1, bitorder="little")[:, :pw.ACTIONS].astype(bool))
    policy = torch.softmax(logits.masked_fill(~bits, -np.inf), dim=1)
    v = torch.relu(bn(F.conv2d(h, t["v.cw"].view(cfg.value_channels, C, 1, 1)), "v.cscale", "v.cbias"))
    hid = torch.relu(v.reshape(n, -1) @ t["v.w1"].T + t["v.b1"])
    value = torch.softmax(hid @ t["v.w2"].T + t["v.b2"], dim=1)
    return policy.numpy(), value.numpy(), logits.numpy(), h.numpy()


def inputs_for(cfg, n, seed=77):
    rec, _ = positions.generate_moves(seed, n, (0, 160))
    return rec, oracle.encode52(rec), oracle.legal_masks(np.ascontiguousarray(rec["cur"]), 2)


@pytest.mark.parametrize("blocks,channels,key", [(3, 16, 8), (4, 32, 16), (1, 8, 4), (0, 8, 4)])
def test_whole_network_against_a_float64_library_composition(blocks, channels, key):
    cfg = pw.tiny(blocks=blocks, channels=channels, key=key)
    tensors = pw.draw_tensors(cfg, 1.0, 1.0)
    rec, planes, masks = inputs_for(cfg, 12)
    pol, val, extra = oracle.pnet_forward(pw.pack_blob(cfg, tensors), planes, masks, want_raw=True, want_tower=True)
    lp, lv, ll, lh = library_forward(cfg, tensors, planes, masks)
    assert np.abs(extra["tower"] - lh).max() < 1e-10
    assert np.abs(extra["logits"] - ll).max() < 1e-9
    assert np.abs(pol - lp).max() < 1e-10 and np.abs(val - lv).max() < 1e-10
    bits = np.unpackbits(masks.view(np.uint8), axis=1, bitorder="little")[:, :pw.ACTIONS].astype(bool)
    assert (pol[~bits] == 0).all() and np.abs(pol.sum(axis=1) - 1).max() < 1e-12 and np.abs(val.sum(axis=1) - 1).max() < 1e-12


def test_activations_are_capped_at_six():
    cfg = pw.tiny(blocks=3, channels=16, key=8)
    tensors = pw.draw_tensors(cfg, 1.0, 1.0)
    for k in ("in.scale", "b0.scale1", "b1.scale1", "b2.scale2"):
        tensors[k] = tensors[k] * np.float32(500.0)
    rec, planes, masks = inputs_for(cfg, 6)
    _, _, extra = oracle.pnet_forward(pw.pack_blob(cfg, tensors), planes, masks, want_tower=True)
    tw = extra["tower"]
    assert tw.min() >= 0.0 and tw.max() == 6.0 and (tw == 6.0).mean() > 0.05


def test_identity_query_and_key_give_a_symmetric_score_and_offsets_add_exactly():
    cfg = pw.tiny(blocks=2, channels=16, key=8)
    tensors = pw.draw_tensors(cfg, 1.0, 1.0)
    eye = np.eye(cfg.key, dtype=np.float32)
    tensors["q.w"], tensors["k.w"] = eye, eye.copy()
    tensors["q.b"][:] = 0
    tensors["k.b"][:] = 0
    tensors["o.w"][:] = 0
    tensors["o.b"][:] = np.array([1.0, 2.0, 3.0, 4.0], dtype=np.float32)       # queen, rook, bishop, knight
    rec, planes, masks = inputs_for(cfg, 5)
    _, _, extra = oracle.pnet_forward(pw.pack_blob(cfg, tensors), planes, masks, want_raw=True)
    lg = extra["logits"]
    # q = k = token: the score of (f, t) is the Gram matrix entry, the same for (t, f)
    checked = 0
    for f in range(64):
        for to in range(f + 1, 64):
            i, j = oracle.policy_index(2, 0, f, to, 0, 0), oracle.policy_index(2, 0, to, f, 0, 0)
            if i >= 0 and j >= 0:
                assert np.abs(lg[:, i] - lg[:, j]).max() < 1e-12
                checked += 1
    assert checked == 1792 // 2
    # a promotion action = its pair's score plus the piece's offset
    for f in range(48, 56):
        for to in (f + 7, f + 8, f + 9):
            if to < 64 and abs((to & 7) - (f & 7)) <= 1:
                pair = oracle.policy_index(2, 0, f, to, 0, 0)
                for promo, off in ((4, 1.0), (3, 2.0), (2, 3.0), (1, 4.0)):
                    assert np.abs(lg[:, oracle.policy_index(2, 0, f, to, promo, 0)] - lg[:, pair] - off).max() < 1e-12


def test_pooled_context_by_hand_on_a_constant_board():
    # one pooled block whose first convolution is zero: its normalised output is the bias, the same on
    # every square, so mean = max = cap(bias) on the pooled channels and the context is a plain product
    cfg = pw.tiny(blocks=2, channels=8, key=4)
    tensors = pw.draw_tensors(cfg, 1.0, 1.0)
    tensors["b1.w1"][:] = 0
    tensors["b1.w2"][:] = 0
    rec, planes, masks = inputs_for(cfg, 3)
    # a second convolution that copies its input channel r (centre tap) to output channel r
    R = 6
    for r in range(R):
        tensors["b1.w2"][r, r, 1, 1] = 1.0
    tensors["b1.scale2"][:] = 1.0
    tensors["b1.bias2"][:] = 0.0
    _, _, e1 = oracle.pnet_forward(pw.pack_blob(cfg, tensors), planes, masks, want_tower=True)
    b1 = tensors["b1.bias1"].astype(np.float64)
    pooled = np.clip(b1[R:], 0, 6)
    g = tensors["b1.gw"].astype(np.float64) @ np.concatenate([pooled, pooled])
    t_reg = np.clip(b1[:R] + g, 0, 6)                        # what the second convolution copies
    # the block's input h0 = the output of the same network cut after block 0 (tensors copied as they
    # are, so block 0 keeps the branch scale it was folded with)
    cfg1 = pw.tiny(blocks=1, channels=8, key=4)
    t1 = {k: v for k, v in tensors.items() if not k.startswith("b1.")}
    _, _, eh = oracle.pnet_forward(pw.pack_blob(cfg1, t1), planes, masks, want_tower=True)
    h0 = eh["tower"]
    want = np.clip(h0 + np.concatenate([t_reg, np.zeros(2)]).reshape(1, 8, 1, 1), 0, 6)
    assert np.abs(e1["tower"] - want).max() < 1e-12
