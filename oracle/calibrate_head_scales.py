"""Writes inputs/head_scales.json: one multiplier per head and weight set.

Random He-normal towers with residual additions grow their activations by orders of magnitude,
so the un-scaled policy is one-hot and the value saturated, which would make every parity check
vacuous.  Following the paper's own bootstrap (a small final policy projection, numerical scale
set on a few hundred encoded positions, no chess targets: Sec. 4.3.5), the LAST linear layer of
each head is multiplied by a scalar chosen on 512 seeded calibration positions so that
  * the standard deviation of a position's legal-move logits averages 1.0, and
  * the value head's pre-activation has standard deviation 0.2 for the three win/draw/loss
    logits and 0.03 for the scalar tanh head.  Why so small: an emulation with bf16-rounded
    operands but EXACT accumulation (the floor of any bf16 kernel) leaves the towers' activations
    0.6-0.7 % (rms) off, and the value heads turn that into a pre-activation error of a quarter
    to a third of the head's spread over positions.  At a spread of 0.5 that floor alone is
    0.03-0.05 in the tanh output of the 20x128 net and 0.03 in the win/draw/loss probabilities
    of the 40x256 net, outside the 2e-2 bar for every possible bf16 implementation.  The tanh
    head has unit slope near the origin and no softmax to cancel an error common to its logits,
    hence the smaller figure.  A value head with a small final projection is also what an
    untrained bootstrap network looks like.
The scalars become part of the weights, so the oracle and the CUDA library see the same network.

Calls only the oracle and the input generators.  Usage:  python -m oracle.calibrate_head_scales
"""
import json
import os
import sys

import numpy as np

import oracle
from inputs import configs, positions, weights


def scales_for(cfg) -> dict:
    tensors = weights.draw_tensors(cfg, policy_scale=1.0, value_scale=1.0)
    blob = weights.pack_blob(cfg, tensors)
    rec = positions.for_config(cfg, calibration=True)
    recs = positions.records_for_planes(cfg.in_planes, rec)
    masks, _, _, _, raw = oracle.evaluate(blob, recs, cfg.in_planes, cfg.policy_head, want_raw=True)
    stds = []
    for i in range(recs.shape[0]):
        bits = np.unpackbits(masks[i].view(np.uint8), bitorder="little")[: cfg.policy_size].astype(bool)
        legal = raw["logits"][i][bits]
        if legal.size >= 2:
            stds.append(float(np.std(legal)))
    policy = 1.0 / float(np.mean(stds))
    value = (0.2 if cfg.value_head == 1 else 0.03) / float(np.std(raw["value_pre"]))
    return {"policy": policy, "value": value, "positions": int(recs.shape[0]),
            "raw_legal_logit_std": float(np.mean(stds)), "raw_value_std": float(np.std(raw["value_pre"]))}


def main(names):
    path = os.path.join(os.path.dirname(os.path.abspath(weights.__file__)), "head_scales.json")
    try:
        with open(path) as f:
            table = json.load(f)
    except OSError:
        table = {}
    for name in names:
        cfg = configs.CONFIGS[name]
        if cfg.weights_like:
            continue
        table[name] = scales_for(cfg)
        print(name, table[name], flush=True)
    with open(path, "w") as f:
        json.dump(table, f, indent=1, sort_keys=True)
        f.write("\n")


if __name__ == "__main__":
    main(sys.argv[1:] or [n for n in configs.CONFIGS])
