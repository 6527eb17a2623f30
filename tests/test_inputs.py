"""The seeded input generators: determinism, recipe, and the stored batch hashes (CPU only)."""
import hashlib
import json
import os

import numpy as np

from inputs import configs, positions, weights


def test_positions_are_deterministic_and_follow_the_ply_recipe():
    a, pa = positions.generate(1234, 300, (0, 40), (40, 160))
    b, pb = positions.generate(1234, 300, (0, 40), (40, 160))
    assert a.tobytes() == b.tobytes() and (pa == pb).all()
    assert (pa[0::2] <= 40).all() and (pa[1::2] >= 40).all() and pa.max() <= 160
    # index-addressed: a slice of the stream equals the same indices of the whole
    c, _ = positions.generate(1234, 50, (0, 40), (40, 160), first_index=100)
    assert c.tobytes() == a[100:150].tobytes()
    assert (a["n_hist"] == np.minimum(pa, 7)).all()
    assert (a["cur"]["halfmove"] <= pa).all()
    assert (a["cur"]["stm"] == pa % 2).all()
    for i in range(300):
        assert len(positions.legal_moves(a[i])) >= 1            # never a terminal position
        assert bin(int(a["cur"]["pieces"][i, 5])).count("1") == 1 and bin(int(a["cur"]["pieces"][i, 11])).count("1") == 1


def test_zero_plies_is_the_start_position():
    a, p = positions.generate(5, 4, (0, 0))
    start = positions.record_from_fen("rnbqkbnr/pppppppp/8/8/8/8/PPPPPPPP/RNBQKBNR w KQkq - 0 1")
    for i in range(4):
        assert a["cur"][i].tobytes() == start[0].tobytes() and a["n_hist"][i] == 0


def test_stored_hashes_of_the_config_batches(golden_dir):
    with open(os.path.join(golden_dir, "input_hashes.json")) as f:
        stored = json.load(f)
    for name in ("c1", "c2", "c3"):
        cfg = configs.CONFIGS[name]
        rec = positions.for_config(cfg)
        assert hashlib.sha256(rec.tobytes()).hexdigest() == stored[name]["positions"], name
    cfg = configs.CONFIGS["c1"]
    assert hashlib.sha256(weights.make_blob(cfg).tobytes()).hexdigest() == stored["c1"]["weights"]


def test_weight_blob_layout_and_statistics():
    cfg = configs.CONFIGS["c2"]
    T = weights.draw_tensors(cfg, 1.0, 1.0)
    blob = weights.pack_blob(cfg, T)
    n_params = sum(int(np.prod(s)) for s in weights.tensor_shapes(cfg).values())
    assert blob.nbytes == 64 + 4 * n_params
    assert bytes(blob[:8]) == b"AZNETv1\0"
    hdr = np.frombuffer(blob[8:36].tobytes(), dtype="<u4")
    assert list(hdr[:6]) == [1, 19, 20, 128, 0, 0] and hdr[6] == len(T)
    w = T["b3.w1"]
    assert abs(w.std() - np.sqrt(2.0 / (128 * 9))) < 0.02 * np.sqrt(2.0 / (128 * 9))
    assert abs(T["b3.scale1"].mean() - 1) < 0.05 and abs(T["b3.bias2"].mean()) < 0.05
    # first tensor sits right behind the header
    assert (np.frombuffer(blob[64:64 + 16].tobytes(), dtype="<f4") == T["in.w"].reshape(-1)[:4]).all()
    # c4 reuses c2's weights
    assert weights.make_blob(configs.CONFIGS["c4"]).tobytes() == weights.make_blob(cfg).tobytes()
