"""Writes inputs/pnet_head_scales.json: the two multipliers of the paper-network weight sets.

Same purpose and recipe as calibrate_head_scales.py (Sec. 4.3.5: a small final policy projection,
numerical scale set on a few hundred encoded positions, no chess targets).  On 512 seeded
calibration positions of each configuration:
  * the query map and the promotion offsets are scaled together so that the standard deviation of a
    position's legal-action logits averages 1.0 (the logits are linear in that scalar);
  * the last value layer is scaled so that the three win/draw/loss logits, centred per position,
    have standard deviation 0.2.
Calls only the oracle and the input generators.  Usage:  python -m oracle.calibrate_pnet_head_scales
"""
import json
import os
import sys

import numpy as np

import oracle
from inputs import pnet_weights as pw
from inputs import positions

CALIBRATION_SEED_OFFSET = 777_000_000
CALIBRATION_COUNT = 512


def calibration_records(cfg):
    rec, _ = positions.generate_moves(cfg.position_seed + CALIBRATION_SEED_OFFSET, CALIBRATION_COUNT, cfg.plies)
    return rec


def scales_for(cfg) -> dict:
    blob = pw.make_blob(cfg, 1.0, 1.0)
    rec = calibration_records(cfg)
    masks, _, _, value, extra = oracle.pnet_evaluate(blob, rec, want_raw=True)
    stds = []
    for i in range(rec.shape[0]):
        bits = np.unpackbits(masks[i].view(np.uint8), bitorder="little")[: pw.ACTIONS].astype(bool)
        legal = extra["logits"][i][bits]
        if legal.size >= 2:
            stds.append(float(np.std(legal)))
    logp = np.log(value)
    centred = logp - logp.mean(axis=1, keepdims=True)
    return {"policy": 1.0 / float(np.mean(stds)), "value": 0.2 / float(np.std(centred)),
            "positions": int(rec.shape[0]), "raw_legal_logit_std": float(np.mean(stds)),
            "raw_value_logit_std": float(np.std(centred))}


def main(names):
    path = os.path.join(os.path.dirname(os.path.abspath(pw.__file__)), "pnet_head_scales.json")
    try:
        with open(path) as f:
            table = json.load(f)
    except OSError:
        table = {}
    for name in names:
        table[name] = scales_for(pw.PNET_CONFIGS[name])
        print(name, table[name], flush=True)
    with open(path, "w") as f:
        json.dump(table, f, indent=1, sort_keys=True)
        f.write("\n")


if __name__ == "__main__":
    main(sys.argv[1:] or [n for n, c in pw.PNET_CONFIGS.items() if not c.weights_like])
