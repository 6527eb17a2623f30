"""ORACLE side — test infrastructure, not the product: what reduced-precision OPERANDS cost.

The CUDA towers multiply bf16, e4m3 or 8-bit integer operands on the tensor cores and accumulate in
fp32 / int32.  No kernel of that kind can be closer to the fp64 oracle than the arithmetic it is
told to use.  This module computes that floor on the CPU: the network of `net_oracle.c` /
`pnet_oracle.c` written once more with library primitives (float64 `conv2d`, `linear`), in which
every operand of a tensor-core product is first rounded to the format in question and everything
else — accumulation, the residual stream, biases, activations — stays exact (float64).  What is
rounded, and with which scales, follows the readings the library documents for its 8-bit towers
(Sec. 4.3.6: trunk convolutions quantised after training, ranges from a few hundred calibration
positions, start block and heads at higher precision):

  bf16   every convolution and head operand rounded to bfloat16 (nearest even)
  e4m3   layers after the input layer: activations a / sa[ci] with sa = calibration maximum / 448,
         weights (bn_scale * W * sa[ci]) / ws[co] with ws = max|.| / 448, both rounded to e4m3
         (saturating, nearest even); input layer and heads as bf16
  int8   the same with unsigned 8-bit activations (maximum / 255, round to nearest, clamp) and
         signed 8-bit weights (max / 127)
  options: operands split into a rounded value plus the rounded remainder (two e4m3 numbers per
         operand), the last blocks kept in bf16, and the per-channel bias correction of the
         calibration step (mean pre-activation of every layer matched to the bf16 tower's on the
         calibration positions, shifts limited to a quarter of the channel's range).

Nothing here is shared with the CUDA library, and the library never imports it.  The rounding
functions are pinned in tests/test_quant_emul.py against closed forms and a library's converters;
the exact mode is pinned against the C oracle.  `python -m oracle.quant_emul --write` stores the
floors the GPU parity tests compare against in tests/golden/quant_floors.json (oracle calls only).
"""
import json
import os
import sys
from dataclasses import dataclass

import numpy as np
import torch
import torch.nn.functional as F

import oracle
from inputs import configs, pnet_weights, positions, weights

GOLDEN = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "tests", "golden", "quant_floors.json")


# ---- rounding to the operand formats (float64 in, float64 out) ------------------------------------

def round_bf16(x: torch.Tensor) -> torch.Tensor:
    """Nearest bfloat16, ties to even: float32 bit pattern, rounded at bit 16."""
    u = x.to(torch.float32).contiguous().view(torch.int32).to(torch.int64) & 0xFFFFFFFF
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    u = torch.where(u >= 2 ** 31, u - 2 ** 32, u).to(torch.int32)
    return u.view(torch.float32).to(torch.float64)


def round_e4m3(x: torch.Tensor) -> torch.Tensor:
    """Nearest e4m3 (4 exponent bits, bias 7, 3 mantissa bits, no infinities), ties to even,
    saturating at +-448.  Normal numbers 2^e * (1 + m/8), e in -6..8; below 2^-6 the spacing stays
    2^-9 (subnormals)."""
    a = x.abs().clamp(max=448.0)
    e = torch.floor(torch.log2(a.clamp(min=2.0 ** -20))).clamp(min=-6.0, max=8.0)
    step = torch.exp2(e - 3.0)
    q = torch.round(a / step) * step            # torch.round: half to even
    return torch.sign(x) * q.clamp(max=448.0)


def round_u8(x: torch.Tensor) -> torch.Tensor:
    return torch.round(x).clamp(0.0, 255.0)


def round_s8(x: torch.Tensor) -> torch.Tensor:
    return torch.round(x).clamp(-127.0, 127.0)


@dataclass(frozen=True)
class Spec:
    kind: str = "exact"             # exact | bf16 | e4m3 | int8
    split_w: bool = False           # 8-bit weights as a rounded value plus the rounded remainder
    split_a: bool = False           # 8-bit activations likewise
    bias_correction: bool = False
    bf16_last_blocks: int = 0       # this many blocks at the end keep bf16 operands
    dequantised_weights_only: bool = False   # weights rounded as `kind` says, activations exact

    @property
    def label(self) -> str:
        parts = [self.kind]
        if self.dequantised_weights_only:
            parts.append("weights only")
        if self.split_w:
            parts.append("split weights")
        if self.split_a:
            parts.append("split activations")
        if self.bf16_last_blocks:
            parts.append(f"last {self.bf16_last_blocks} blocks bf16")
        if self.bias_correction:
            parts.append("bias correction")
        return ", ".join(parts)


def _limits(kind):
    """(largest activation code, largest weight code, activation rounding, weight rounding)."""
    if kind == "e4m3":
        return 448.0, 448.0, round_e4m3, round_e4m3
    if kind == "int8":
        return 255.0, 127.0, round_u8, round_s8
    raise ValueError(kind)


def _split(x, rnd):
    hi = rnd(x)
    return hi, rnd(x - hi)


class ResidualTower:
    """The plain residual tower of the five workloads (input convolution, then blocks of convolution,
    folded normalisation, ReLU, convolution, folded normalisation, residual addition, ReLU)."""

    def __init__(self, cfg, tensors):
        self.cfg = cfg
        self.t = {k: torch.from_numpy(np.asarray(v, dtype=np.float64)) for k, v in tensors.items()}
        self.layers = [("in.w", "in.scale", "in.bias")]
        for b in range(cfg.blocks):
            self.layers += [(f"b{b}.w1", f"b{b}.scale1", f"b{b}.bias1"), (f"b{b}.w2", f"b{b}.scale2", f"b{b}.bias2")]

    def folded(self, l):
        w, s, b = self.layers[l]
        return self.t[w] * self.t[s].view(-1, 1, 1, 1), self.t[b]

    def _is_8bit(self, l, spec):
        L = len(self.layers)
        return spec.kind in ("e4m3", "int8") and l > 0 and l < L - 2 * spec.bf16_last_blocks

    def conv(self, l, a, spec, sa):
        W, bias = self.folded(l)
        if spec.kind == "exact":
            y = F.conv2d(a, W, padding=1)
        elif not self._is_8bit(l, spec):
            y = F.conv2d(round_bf16(a), round_bf16(W), padding=1)
        else:
            amax, wmax, ra, rw = _limits(spec.kind)
            Wp = W * sa[l].view(1, -1, 1, 1)
            ws = Wp.abs().amax(dim=(1, 2, 3)).clamp_min(1e-30) / wmax
            wq, aq = Wp / ws.view(-1, 1, 1, 1), a / sa[l].view(1, -1, 1, 1)
            if spec.dequantised_weights_only:
                y = F.conv2d(aq, rw(wq), padding=1)
            elif spec.split_w or spec.split_a:
                w_hi, w_lo = _split(wq, rw)
                a_hi, a_lo = _split(aq, ra)
                y = F.conv2d(a_hi, w_hi, padding=1)
                if spec.split_a:
                    y = y + F.conv2d(a_lo, w_hi, padding=1)
                if spec.split_w:
                    y = y + F.conv2d(a_hi, w_lo, padding=1)
            else:
                y = F.conv2d(ra(aq), rw(wq), padding=1)
            y = y * ws.view(1, -1, 1, 1)
        return y + bias.view(1, -1, 1, 1)

    def run(self, x, spec, sa=None, corr=None, stats=None, fit=None):
        """x [n][P][8][8].  `stats`: dict filled with per-layer output maxima and mean pre-activations.
        `fit`: mean pre-activations to match; corrections are then derived layer by layer on THIS input
        (the calibration positions) and stored in `corr`."""
        L = len(self.layers)
        outs, pres = [], []

        def layer(l, a, residual=None):
            z = self.conv(l, a, spec, sa)
            if residual is not None:
                z = z + residual
            if corr is not None and fit is not None and self._is_8bit(l, spec):
                top = fit["absmax"][l]
                c = fit["mean"][l] - z.mean(dim=(0, 2, 3))
                c = torch.where(top > 1e-20, torch.minimum(torch.maximum(c, -0.25 * top), 0.25 * top), torch.zeros_like(c))
                corr[l] = c
            if corr is not None and corr.get(l) is not None:
                z = z + corr[l].view(1, -1, 1, 1)
            pres.append(z)
            out = torch.relu(z)
            outs.append(out)
            return out

        h = layer(0, x)
        for b in range(self.cfg.blocks):
            t = layer(1 + 2 * b, h)
            h = layer(2 + 2 * b, t, residual=h)
        if stats is not None:
            stats["absmax"] = [o.amax(dim=(0, 2, 3)) for o in outs]
            stats["mean"] = [z.mean(dim=(0, 2, 3)) for z in pres]
        assert len(outs) == L
        return h

    def calibrate(self, x_cal, spec):
        """Ranges from the bf16 tower on the calibration positions, then (optionally) the bias correction."""
        stats = {}
        self.run(x_cal, Spec("bf16"), stats=stats)
        amax = _limits(spec.kind)[0]
        sa = [None] + [m.clamp_min(1e-30) / amax for m in stats["absmax"][:-1]]
        corr = None
        if spec.bias_correction:
            corr = {}
            self.run(x_cal, spec, sa=sa, corr=corr, fit=stats)
        return sa, corr

    def dequantised_tensors(self, tensors, sa, kind):
        """The network's float32 tensors with every 8-bit layer's weights replaced by what their 8-bit codes stand
        for (scale folded in, the layer's own scale set to one).  Fed to the fp64 oracle, this is the network an 8-bit
        tower would compute if its ACTIVATIONS were exact: comparing a kernel against it isolates the activations'
        share of the error."""
        _, wmax, _, rw = _limits(kind)
        out = dict(tensors)
        for l in range(1, len(self.layers)):
            w, s, b = self.layers[l]
            W, _ = self.folded(l)
            Wp = W * sa[l].view(1, -1, 1, 1)
            ws = Wp.abs().amax(dim=(1, 2, 3)).clamp_min(1e-30) / wmax
            deq = rw(Wp / ws.view(-1, 1, 1, 1)) * ws.view(-1, 1, 1, 1) / sa[l].view(1, -1, 1, 1)
            out[w] = deq.numpy().astype(np.float32)
            out[s] = np.ones_like(np.asarray(tensors[s]))
        return out

    def heads(self, h, masks, q):
        """Heads with operands rounded by q (identity for the exact network): policy, value, raw logits, value
        pre-activation."""
        cfg, t = self.cfg, self.t
        sb = lambda x, s, b: x * t[s].view(1, -1, 1, 1) + t[b].view(1, -1, 1, 1)
        hh = q(h)
        if cfg.policy_head == 0:
            lg = (F.conv2d(hh, q(t["p.w"])[:, :, None, None]) + t["p.bias"].view(1, -1, 1, 1)).flatten(1)
        else:
            pc = q(torch.relu(F.conv2d(hh, q(t["p.cw"] * t["p.cscale"].view(-1, 1))[:, :, None, None]) + t["p.cbias"].view(1, -1, 1, 1)))
            lg = F.linear(pc.flatten(1), q(t["p.fw"]), t["p.fbias"])
        vc = q(torch.relu(F.conv2d(hh, q(t["v.cw"] * t["v.cscale"].view(-1, 1))[:, :, None, None]) + t["v.cbias"].view(1, -1, 1, 1)))
        z = F.linear(torch.relu(F.linear(vc.flatten(1), q(t["v.w1"]), t["v.b1"])), t["v.w2"], t["v.b2"])
        val = torch.tanh(z) if cfg.value_head == 0 else torch.softmax(z, 1)
        bits = torch.from_numpy(np.unpackbits(masks.view(np.uint8), axis=1, bitorder="little")[:, : cfg.policy_size].astype(bool))
        pol = torch.softmax(torch.where(bits, lg, torch.full_like(lg, -float("inf"))), 1)
        return pol, val, lg, z


class PaperTower:
    """The paper's own network (Sec. 3.2, 4.3.3, 4.3.6, App. D.1): activations capped at six, residual branch
    scaled (folded into the second convolution), pooled context in blocks 1, 3, 5, ..., query-key policy head."""

    def __init__(self, cfg, tensors):
        self.cfg = cfg
        self.t = {k: torch.from_numpy(np.asarray(v, dtype=np.float64)) for k, v in tensors.items()}

    def run(self, x, spec):
        cfg, t = self.cfg, self.t
        C = cfg.channels
        R = C - C // 4
        cap = lambda y: torch.clamp(y, 0.0, 6.0)
        q = (lambda z: z) if spec.kind == "exact" else round_bf16

        def conv(a, w, s, b):
            return F.conv2d(q(a), q(t[w] * t[s].view(-1, 1, 1, 1)), padding=1) + t[b].view(1, -1, 1, 1)

        h = cap(conv(x, "in.w", "in.scale", "in.bias"))
        for b in range(cfg.blocks):
            y = conv(h, f"b{b}.w1", f"b{b}.scale1", f"b{b}.bias1")
            if pnet_weights.pooled(b):
                pool = cap(y[:, R:])
                g = torch.cat([pool.mean(dim=(2, 3)), pool.amax(dim=(2, 3))], 1)
                y = cap(y[:, :R] + (g @ t[f"b{b}.gw"].T).view(-1, R, 1, 1))
            else:
                y = cap(y)
            h = cap(h + conv(y, f"b{b}.w2", f"b{b}.scale2", f"b{b}.bias2"))
        return h

    def heads(self, h, masks, q):
        """Token projection composed into the query and key maps, as a deployment would (it has no activation)."""
        cfg, t = self.cfg, self.t
        C, n = cfg.channels, h.shape[0]
        feat = q(h).reshape(n, C, 64)
        wq = q((t["q.w"] @ t["t.w"]) / np.sqrt(cfg.key))
        bq = (t["q.w"] @ t["t.b"] + t["q.b"]) / np.sqrt(cfg.key)
        wk, bk = q(t["k.w"] @ t["t.w"]), t["k.w"] @ t["t.b"] + t["k.b"]
        qq = torch.einsum("jc,ncs->njs", wq, feat) + bq.view(1, -1, 1)
        kk = torch.einsum("jc,ncs->njs", wk, feat) + bk.view(1, -1, 1)
        u = torch.einsum("kc,ncs->nks", t["t.w"], feat) + t["t.b"].view(1, -1, 1)
        o = torch.einsum("pk,nks->nps", t["o.w"], u) + t["o.b"].view(1, -1, 1)
        score = torch.einsum("ndf,ndt->nft", qq, kk)
        lg = torch.zeros((n, 1880), dtype=torch.float64)
        for f in range(64):
            for to in range(64):
                i = oracle.policy_index(2, 0, f, to, 0, 0)
                if i >= 0:
                    lg[:, i] = score[:, f, to]
                for pr in (1, 2, 3, 4):
                    j = oracle.policy_index(2, 0, f, to, pr, 0)
                    if j >= 0:
                        lg[:, j] = score[:, f, to] + o[:, 4 - pr, f]
        bits = torch.from_numpy(np.unpackbits(masks.view(np.uint8), axis=1, bitorder="little")[:, :1880].astype(bool))
        pol = torch.softmax(lg.masked_fill(~bits, -np.inf), 1)
        v = torch.relu(F.conv2d(h, t["v.cw"].view(-1, C, 1, 1)) * t["v.cscale"].view(1, -1, 1, 1) + t["v.cbias"].view(1, -1, 1, 1))
        hid = torch.relu(v.reshape(n, -1) @ t["v.w1"].T + t["v.b1"])
        z = hid @ t["v.w2"].T + t["v.b2"]
        return pol, torch.softmax(z, 1), lg, z


# ---- figures of merit -----------------------------------------------------------------------------

def figures(h, pol, val, z, h0, pol0, val0, z0):
    """Errors of an emulated network against the exact one (all float64 tensors / arrays)."""
    as_t = lambda a: a if isinstance(a, torch.Tensor) else torch.from_numpy(np.asarray(a, dtype=np.float64))
    h0, pol0, val0, z0 = as_t(h0), as_t(pol0), as_t(val0), as_t(z0)
    gap = torch.sort(pol0, dim=1, descending=True).values
    clear = (gap[:, 0] - gap[:, 1]) > 2e-2
    same = pol.argmax(1) == pol0.argmax(1)
    # spread of the value head over positions: of the pre-activation for the scalar head, of the centred logits
    # (what the softmax sees) for the win/draw/loss head
    zc0 = z0 - z0.mean(dim=1, keepdim=True) if z0.shape[1] > 1 else z0
    zc = z - z.mean(dim=1, keepdim=True) if z.shape[1] > 1 else z
    comp_corr = [float(np.corrcoef(val[:, k].numpy(), val0[:, k].numpy())[0, 1]) for k in range(val0.shape[1])]
    return {
        "value_min_component_corr": min(comp_corr),
        "tower_rms": float(((h - h0).pow(2).mean() / h0.pow(2).mean()).sqrt()),
        "policy_max_abs": float((pol - pol0).abs().max()),
        "value_max_abs": float((val - val0).abs().max()),
        "argmax_agreement": float(same.double().mean()),
        "argmax_agreement_clear_gap": float(same[clear].double().mean()) if bool(clear.any()) else 1.0,
        "value_pre_rms_over_spread": float((zc - zc0).pow(2).mean().sqrt() / zc0.std()),
        "value_pre_spread": float(zc0.std()),
    }


def residual_report(name, n, specs, n_cal=configs.CALIBRATION_COUNT, value_spread=None):
    """Emulates workload `name` on its first n positions under every Spec in `specs`.
    value_spread: rescale the value head's last layer so that its pre-activation has this spread over positions
    instead of the one its stored head scale was chosen for (inputs/head_scales.json, "value_spread")."""
    cfg = configs.CONFIGS[name]
    tensors = weights.draw_tensors(cfg)
    if value_spread is not None:
        with open(weights._SCALES_PATH) as f:
            stored = float(json.load(f)[cfg.weights_name]["value_spread"])
        for k in ("v.w2", "v.b2"):
            tensors[k] = (tensors[k] * np.float32(value_spread / stored)).astype(np.float32)
    blob = weights.pack_blob(cfg, tensors)
    recs = positions.records_for_planes(cfg.in_planes, positions.for_config(cfg, n))
    masks, planes, pol0, val0, raw = oracle.evaluate(blob, recs, cfg.in_planes, cfg.policy_head, want_raw=True, want_tower=True)
    net = ResidualTower(cfg, tensors)
    x = torch.from_numpy(planes)
    x_cal = None
    out = {}
    for spec in specs:
        sa = corr = None
        if spec.kind in ("e4m3", "int8"):
            if x_cal is None:
                cal = positions.records_for_planes(cfg.in_planes, positions.for_config(cfg, n_cal, calibration=True))
                x_cal = torch.from_numpy(oracle.encode(cal, cfg.in_planes))
            sa, corr = net.calibrate(x_cal, spec)
        h = net.run(x, spec, sa=sa, corr=corr)
        q = (lambda z: z) if spec.kind == "exact" else round_bf16
        pol, val, _, z = net.heads(h, masks, q)
        out[spec.label] = figures(h, pol, val, z, raw["tower"], pol0, val0, raw["value_pre"])
    return out


def paper_report(name, n):
    cfg = pnet_weights.PNET_CONFIGS[name]
    tensors = pnet_weights.draw_tensors(cfg)
    blob = pnet_weights.pack_blob(cfg, tensors)
    rec, _ = positions.generate_moves(cfg.position_seed, n, cfg.plies)
    masks, planes, pol0, val0, raw = oracle.pnet_evaluate(blob, rec, want_raw=True, want_tower=True)
    net = PaperTower(cfg, tensors)
    x = torch.from_numpy(planes)
    out = {}
    for spec in (Spec("exact"), Spec("bf16")):
        h = net.run(x, spec)
        q = (lambda z: z) if spec.kind == "exact" else round_bf16
        pol, val, _, z = net.heads(h, masks, q)
        z0 = torch.log(torch.from_numpy(val0))            # the oracle returns probabilities; logits up to a common shift
        out[spec.label] = figures(h, pol, val, z, raw["tower"], pol0, val0, z0)
    return out


FLOOR_RUNS = {
    # name: (positions, value spread or None for the stored head scale, specs)
    "c2": (128, None, (Spec("bf16"),)),
    "c2@0.5": (128, 0.5, (Spec("bf16"),)),
    "c3": (128, None, (Spec("bf16"),)),
    "c5": (48, None, (Spec("bf16"),)),
    "c5@0.5": (48, 0.5, (Spec("bf16"),)),
    "c4": (128, None, (Spec("e4m3"), Spec("e4m3", bias_correction=True), Spec("e4m3", dequantised_weights_only=True),
                       Spec("e4m3", split_w=True, bias_correction=True), Spec("e4m3", split_a=True, bias_correction=True),
                       Spec("e4m3", split_w=True, split_a=True), Spec("e4m3", bf16_last_blocks=4, bias_correction=True),
                       Spec("int8", bias_correction=True))),
    "c4b": (128, None, (Spec("e4m3"), Spec("e4m3", bias_correction=True))),
}


def main(argv):
    write = "--write" in argv
    names = [a for a in argv if not a.startswith("--")] or list(FLOOR_RUNS) + ["p12"]
    table = {}
    if write and os.path.exists(GOLDEN):
        with open(GOLDEN) as f:
            table = json.load(f)
    for name in names:
        if name in pnet_weights.PNET_CONFIGS:
            rep = paper_report(name, 256)
        else:
            n, spread, specs = FLOOR_RUNS[name]
            rep = residual_report(name.split("@")[0], n, specs, value_spread=spread)
        table[name] = rep
        for label, fig in rep.items():
            print(f"{name:8s} {label:50s} " + " ".join(f"{k}={v:.4g}" for k, v in fig.items()), flush=True)
    if write:
        with open(GOLDEN, "w") as f:
            json.dump(table, f, indent=1, sort_keys=True)
            f.write("\n")


if __name__ == "__main__":
    main(sys.argv[1:])
