"""Seeded synthetic chess positions (random legal playouts) as library position records.

Thin ctypes wrapper over chessgen.c.  Records are numpy structured arrays whose memory layout
is exactly the library's 784-byte record with history; `cur_records` gives the 104-byte
history-free record used by the 19-plane networks.
"""
import ctypes
import os

import numpy as np

from . import _cbuild
from .configs import CALIBRATION_COUNT, CALIBRATION_SEED_OFFSET, Config

CUR_DTYPE = np.dtype([
    ("pieces", "<u8", (12,)),
    ("stm", "u1"), ("castling", "u1"), ("ep_square", "u1"), ("halfmove", "u1"),
    ("repetitions", "u1"), ("pad", "u1", (3,)),
])
H8_DTYPE = np.dtype([
    ("cur", CUR_DTYPE),
    ("hist_pieces", "<u8", (7, 12)),
    ("hist_rep", "u1", (7,)),
    ("n_hist", "u1"),
])
M8_DTYPE = np.dtype([
    ("cur", CUR_DTYPE),
    ("move_from", "u1", (8,)), ("move_to", "u1", (8,)),
    ("n_moves", "u1"), ("pad", "u1", (7,)),
])
assert CUR_DTYPE.itemsize == 104 and H8_DTYPE.itemsize == 784 and M8_DTYPE.itemsize == 128

_lib = None


def _load():
    global _lib
    if _lib is None:
        here = os.path.dirname(os.path.abspath(__file__))
        path = _cbuild.build_shared(os.path.join(here, "chessgen.c"), "chessgen")
        lib = ctypes.CDLL(path)
        lib.azgen_positions.restype = ctypes.c_int
        lib.azgen_positions.argtypes = [ctypes.c_uint64, ctypes.c_int64, ctypes.c_int,
                                        ctypes.c_int, ctypes.c_int, ctypes.c_int, ctypes.c_int,
                                        ctypes.c_void_p, ctypes.c_void_p]
        lib.azgen_positions_moves.restype = ctypes.c_int
        lib.azgen_positions_moves.argtypes = lib.azgen_positions.argtypes
        assert lib.azgen_move_record_bytes() == M8_DTYPE.itemsize
        lib.azgen_legal_moves.restype = ctypes.c_int
        lib.azgen_legal_moves.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
        assert lib.azgen_record_bytes() == H8_DTYPE.itemsize
        _lib = lib
    return _lib


def build() -> str:
    """Compile the generator (used by the repo-level build step)."""
    _load()
    return "chessgen"


def generate(seed: int, count: int, plies_even=(0, 80), plies_odd=None, first_index: int = 0):
    """`count` records with history, plus each record's ply count."""
    plies_odd = plies_odd or plies_even
    rec = np.zeros(count, dtype=H8_DTYPE)
    plies = np.zeros(count, dtype=np.int32)
    rc = _load().azgen_positions(seed, first_index, count, plies_even[0], plies_even[1],
                                 plies_odd[0], plies_odd[1], rec.ctypes.data, plies.ctypes.data)
    if rc != 0:
        raise ValueError("azgen_positions rejected its arguments")
    return rec, plies


def generate_moves(seed: int, count: int, plies_even=(0, 80), plies_odd=None, first_index: int = 0):
    """The same positions as `generate`, as 128-byte records with the last eight moves (most recent
    first, castling as the king's own move) instead of the last seven boards."""
    plies_odd = plies_odd or plies_even
    rec = np.zeros(count, dtype=M8_DTYPE)
    plies = np.zeros(count, dtype=np.int32)
    rc = _load().azgen_positions_moves(seed, first_index, count, plies_even[0], plies_even[1],
                                       plies_odd[0], plies_odd[1], rec.ctypes.data, plies.ctypes.data)
    if rc != 0:
        raise ValueError("azgen_positions_moves rejected its arguments")
    return rec, plies


def for_config(cfg: Config, count: int = None, first_index: int = 0, calibration: bool = False):
    """The config's batch (or `count` positions of the same stream); records with history."""
    if count is None:
        count = CALIBRATION_COUNT if calibration else cfg.batch
    seed = cfg.position_seed + (CALIBRATION_SEED_OFFSET if calibration else 0)
    rec, _ = generate(seed, count, cfg.plies_even, cfg.plies_odd, first_index)
    return rec


def cur_records(rec_h8: np.ndarray) -> np.ndarray:
    """Contiguous 104-byte records (no history) of the same positions."""
    return np.ascontiguousarray(rec_h8["cur"])


def records_for_planes(cfg_in_planes: int, rec_h8: np.ndarray) -> np.ndarray:
    """The record array a network with that many input planes consumes."""
    return rec_h8 if cfg_in_planes == 112 else cur_records(rec_h8)


def legal_moves(record) -> list:
    """Legal moves of one record as sorted (from, to, promo) triples; promo 0 none,1 N,2 B,3 R,4 Q."""
    cur = np.ascontiguousarray(record["cur"] if "cur" in (record.dtype.names or ()) else record)
    buf = np.zeros(256 * 3, dtype=np.uint8)
    n = _load().azgen_legal_moves(cur.ctypes.data, buf.ctypes.data)
    return [tuple(int(v) for v in buf[3 * i:3 * i + 3]) for i in range(n)]


def record_from_fen(fen: str) -> np.ndarray:
    """One 104-byte record from a FEN string (text parsing only; repetitions = 0)."""
    parts = fen.split()
    rec = np.zeros(1, dtype=CUR_DTYPE)
    order = "PNBRQKpnbrqk"
    rank, file = 7, 0
    for ch in parts[0]:
        if ch == "/":
            rank -= 1
            file = 0
        elif ch.isdigit():
            file += int(ch)
        else:
            rec["pieces"][0, order.index(ch)] |= np.uint64(1) << np.uint64(rank * 8 + file)
            file += 1
    rec["stm"] = 0 if parts[1] == "w" else 1
    c = parts[2] if len(parts) > 2 else "-"
    rec["castling"] = sum(b for k, b in (("K", 1), ("Q", 2), ("k", 4), ("q", 8)) if k in c)
    ep = parts[3] if len(parts) > 3 else "-"
    rec["ep_square"] = 64 if ep == "-" else (ord(ep[0]) - 97) + 8 * (int(ep[1]) - 1)
    rec["halfmove"] = min(int(parts[4]), 255) if len(parts) > 4 else 0
    return rec
