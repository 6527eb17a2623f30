"""ORACLE — test infrastructure, not the product.

A plain, slow CPU implementation (C, double precision) of what leaf evaluation computes:
legal-move masks, input planes, the residual policy/value network and the masked softmax.
Only tests, the smoke check and the benchmark's CPU-baseline leg may import this package; the
CUDA library never does, and this package imports nothing of the CUDA library.

The C sources are compiled on first use with the host's gcc (OpenMP for the per-position loop).
"""
import ctypes
import hashlib
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SOURCES = ("chess_oracle.c", "net_oracle.c", "pnet_oracle.c", "mcts_oracle.c")
_lib = None


def _cpu_tag() -> str:
    try:
        with open("/proc/cpuinfo") as f:
            for line in f:
                if line.startswith("flags"):
                    return hashlib.sha1(line.encode()).hexdigest()[:8]
    except OSError:
        pass
    return "generic"


def build() -> str:
    """Compile the oracle's C files into one shared library beside them; returns its path."""
    h = hashlib.sha1()
    for s in _SOURCES:
        with open(os.path.join(_HERE, s), "rb") as f:
            h.update(f.read())
    out = os.path.join(_HERE, f"liboracle_{h.hexdigest()[:10]}_{_cpu_tag()}.so")
    if not os.path.exists(out):
        tmp = out + f".tmp{os.getpid()}"
        cmd = ["gcc", "-O3", "-march=native", "-std=c11", "-ffp-contract=off", "-fopenmp", "-shared", "-fPIC",
               *[os.path.join(_HERE, s) for s in _SOURCES], "-lm", "-o", tmp]
        subprocess.run(cmd, check=True)
        os.replace(tmp, out)
    return out


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build())
        vp, ci = ctypes.c_void_p, ctypes.c_int
        lib.orc_perft.restype = ctypes.c_uint64
        lib.orc_perft.argtypes = [vp, ci]
        lib.orc_legal_moves.restype = ci
        lib.orc_legal_moves.argtypes = [vp, vp]
        lib.orc_flat_count.restype = ci
        lib.orc_policy_index.restype = ci
        lib.orc_policy_index.argtypes = [ci] * 6
        lib.orc_legal_masks.restype = ci
        lib.orc_legal_masks.argtypes = [vp, ci, ci, ci, vp]
        lib.orc_encode.restype = ci
        lib.orc_encode.argtypes = [vp, ci, ci, ci, vp]
        lib.orc_encode52.restype = ci
        lib.orc_encode52.argtypes = [vp, ci, ci, vp]
        lib.orc_apply_moves.restype = ci
        lib.orc_apply_moves.argtypes = [vp, ci, ci, ci, vp, vp]
        lib.orc_in_check.restype = ci
        lib.orc_in_check.argtypes = [vp]
        lib.orc_synth_eval.restype = ci
        lib.orc_synth_eval.argtypes = [vp, ci, ctypes.c_uint64, vp, vp, vp]
        lib.orc_mcts_search.restype = ci
        lib.orc_mcts_search.argtypes = [vp, ci, ci, ci, ci, ctypes.c_float, ctypes.c_float, ctypes.c_float, ctypes.c_uint64,
                                        ci, ci, vp, vp, vp, vp, vp, vp, vp]
        lib.orc_mcts_new.restype = vp
        lib.orc_mcts_new.argtypes = [vp, ci, ci, ctypes.c_float, ctypes.c_float, ctypes.c_float, ctypes.c_uint64, ci, ci]
        lib.orc_mcts_run.restype = ci
        lib.orc_mcts_run.argtypes = [vp, ci, ci]
        lib.orc_mcts_advance.restype = ci
        lib.orc_mcts_advance.argtypes = [vp, ci]
        lib.orc_mcts_read.restype = ci
        lib.orc_mcts_read.argtypes = [vp] * 9
        lib.orc_mcts_root_noise.restype = ci
        lib.orc_mcts_root_noise.argtypes = [vp, vp, ctypes.c_float]
        lib.orc_mcts_node.restype = ci
        lib.orc_mcts_node.argtypes = [vp, ci, vp, vp]
        lib.orc_mcts_free.restype = None
        lib.orc_mcts_free.argtypes = [vp]
        lib.orc_pnet_forward.restype = ci
        lib.orc_pnet_forward.argtypes = [vp, ctypes.c_size_t, vp, vp, ci, vp, vp, vp, vp]
        lib.orc_conv3x3.restype = None
        lib.orc_conv3x3.argtypes = [vp, vp, ci, ci, vp]
        lib.orc_masked_softmax.restype = None
        lib.orc_masked_softmax.argtypes = [vp, vp, ci, vp]
        lib.orc_forward.restype = ci
        lib.orc_forward.argtypes = [vp, ctypes.c_size_t, vp, vp, ci, vp, vp, vp, vp, vp]
        lib.orc_threads.restype = ci
        _lib = lib
    return _lib


POLICY_SIZE = {0: 73 * 64, 1: 1858}
MASK_WORDS = {0: 73, 1: 30, 2: 30}


def _records(records):
    rec = np.ascontiguousarray(records)
    return rec, rec.dtype.itemsize, rec.shape[0] if rec.ndim else 1


def perft(record, depth: int) -> int:
    rec = np.ascontiguousarray(record)
    return int(_load().orc_perft(rec.ctypes.data, depth))


def legal_moves(record):
    """Sorted (from, to, promo) triples; promo 0 none, 1 N, 2 B, 3 R, 4 Q; castling as the king's move."""
    rec = np.ascontiguousarray(record)
    buf = np.zeros(256 * 3, dtype=np.uint8)
    n = _load().orc_legal_moves(rec.ctypes.data, buf.ctypes.data)
    return sorted(tuple(int(v) for v in buf[3 * i:3 * i + 3]) for i in range(n))


def flat_count() -> int:
    return int(_load().orc_flat_count())


def policy_index(head: int, stm: int, frm: int, to: int, promo: int = 0, castle: int = 0) -> int:
    return int(_load().orc_policy_index(head, stm, frm, to, promo, castle))


def legal_masks(records, head: int) -> np.ndarray:
    """uint64 [n][73 or 30]: bit (i & 63) of word (i >> 6) set iff policy index i is legal.
    head 0: 73 move planes, 1: flat 1,858 list, 2: the paper's 1,880 actions (30 words)."""
    rec, stride, n = _records(records)
    masks = np.zeros((n, MASK_WORDS[head]), dtype=np.uint64)
    rc = _load().orc_legal_masks(rec.ctypes.data, stride, n, head, masks.ctypes.data)
    if rc != 0:
        raise RuntimeError("a legal move had no policy index")
    return masks


def encode(records, in_planes: int) -> np.ndarray:
    """float64 [n][in_planes][8][8] input planes, mover-oriented."""
    rec, stride, n = _records(records)
    if in_planes == 112 and stride != 784:
        raise ValueError("the 112-plane encoding needs records with history")
    planes = np.zeros((n, in_planes, 8, 8), dtype=np.float64)
    if _load().orc_encode(rec.ctypes.data, stride, n, in_planes, planes.ctypes.data) != 0:
        raise ValueError("unsupported plane count")
    return planes


def apply_moves(records, head: int, actions) -> np.ndarray:
    """Successor records (same layout) of `records` after the legal actions `actions` (policy indices of `head`)."""
    rec, stride, n = _records(records)
    act = np.ascontiguousarray(actions, dtype=np.int32)
    out = np.zeros_like(rec)
    if _load().orc_apply_moves(rec.ctypes.data, stride, n, head, act.ctypes.data, out.ctypes.data) != 0:
        raise ValueError("an action is not a legal move of its position")
    return out


def synth_eval(record, head: int, seed: int):
    """The stand-in evaluator of the search tests: (actions, priors float32, value float32) of one position."""
    rec = np.ascontiguousarray(record)
    actions = np.zeros(256, dtype=np.int32)
    priors = np.zeros(256, dtype=np.float32)
    value = np.zeros(1, dtype=np.float32)
    k = _load().orc_synth_eval(rec.ctypes.data, head, seed, actions.ctypes.data, priors.ctypes.data, value.ctypes.data)
    if k < 0:
        raise RuntimeError("a legal move had no policy index")
    return actions[:k].copy(), priors[:k].copy(), float(value[0])


def mcts_search(record, head: int, simulations: int, leaves: int = 1, c_puct: float = 1.5, fpu_reduction: float = 0.2,
                discount: float = 0.99, seed: int = 0, node_cap: int | None = None, edge_cap: int | None = None) -> dict:
    """Sequential tree search of one game with the stand-in evaluator (Eq. 1; constants of App. D.2)."""
    rec, stride, n = _records(record)
    assert n == 1
    node_cap = node_cap or simulations * leaves + 2
    edge_cap = edge_cap or node_cap * 64
    actions = np.zeros(256, dtype=np.int32)
    visits = np.zeros(256, dtype=np.int32)
    w = np.zeros(256, dtype=np.float32)
    prior = np.zeros(256, dtype=np.float32)
    counts = np.zeros(4, dtype=np.int32)
    nvis = np.zeros(node_cap, dtype=np.int32)
    wsum = np.zeros(node_cap, dtype=np.float32)
    k = _load().orc_mcts_search(rec.ctypes.data, stride, head, simulations, leaves, c_puct, fpu_reduction, discount, seed,
                                node_cap, edge_cap, actions.ctypes.data, visits.ctypes.data, w.ctypes.data,
                                prior.ctypes.data, counts.ctypes.data, nvis.ctypes.data, wsum.ctypes.data)
    if k < 0:
        raise ValueError("bad search arguments")
    return {"actions": actions[:k].copy(), "visits": visits[:k].copy(), "w": w[:k].copy(), "prior": prior[:k].copy(),
            "n_nodes": int(counts[0]), "n_edges": int(counts[1]), "flags": int(counts[2]), "idle": int(counts[3]),
            "node_nvis": nvis[:counts[0]].copy(), "node_wsum": wsum[:counts[0]].copy()}


class MctsTree:
    """A search of one game that lives across played moves (the subtree under the played move is kept)."""

    def __init__(self, record, head: int, leaves: int = 1, c_puct: float = 1.5, fpu_reduction: float = 0.2,
                 discount: float = 0.99, seed: int = 0, node_cap: int = 1024, edge_cap: int | None = None):
        rec, stride, n = _records(record)
        assert n == 1
        self.dtype, self.leaves, self.node_cap = rec.dtype, leaves, node_cap
        self.handle = _load().orc_mcts_new(rec.ctypes.data, stride, head, c_puct, fpu_reduction, discount, seed,
                                           node_cap, edge_cap or node_cap * 64)
        if not self.handle:
            raise ValueError("bad search arguments")

    def run(self, simulations: int):
        if _load().orc_mcts_run(self.handle, simulations, self.leaves) != 0:
            raise ValueError("bad search arguments")

    def advance(self, action: int):
        """Plays `action` at the root; ValueError if the root has no such move."""
        if _load().orc_mcts_advance(self.handle, int(action)) != 0:
            raise ValueError("the root has no such move")

    def read(self) -> dict:
        actions = np.zeros(256, dtype=np.int32)
        visits = np.zeros(256, dtype=np.int32)
        w = np.zeros(256, dtype=np.float32)
        prior = np.zeros(256, dtype=np.float32)
        counts = np.zeros(4, dtype=np.int32)
        nvis = np.zeros(self.node_cap, dtype=np.int32)
        wsum = np.zeros(self.node_cap, dtype=np.float32)
        root = np.zeros(1, dtype=self.dtype)
        k = _load().orc_mcts_read(self.handle, actions.ctypes.data, visits.ctypes.data, w.ctypes.data, prior.ctypes.data,
                                  counts.ctypes.data, nvis.ctypes.data, wsum.ctypes.data, root.ctypes.data)
        return {"actions": actions[:k].copy(), "visits": visits[:k].copy(), "w": w[:k].copy(), "prior": prior[:k].copy(),
                "n_nodes": int(counts[0]), "n_edges": int(counts[1]), "flags": int(counts[2]), "idle": int(counts[3]),
                "node_nvis": nvis[:counts[0]].copy(), "node_wsum": wsum[:counts[0]].copy(), "root": root}

    def root_noise(self, noise, epsilon: float) -> int:
        """Mixes caller-drawn noise into the priors of the current root's edges; returns how many edges changed."""
        eta = np.ascontiguousarray(noise, dtype=np.float32)
        assert eta.size >= 256
        return int(_load().orc_mcts_root_noise(self.handle, eta.ctypes.data, epsilon))

    def node(self, index: int):
        """(record, parent index) of one node, for inspection."""
        rec = np.zeros(1, dtype=self.dtype)
        parent = np.zeros(1, dtype=np.int32)
        if _load().orc_mcts_node(self.handle, index, rec.ctypes.data, parent.ctypes.data) != 0:
            raise IndexError(index)
        return rec, int(parent[0])

    def close(self):
        if self.handle:
            _load().orc_mcts_free(self.handle)
            self.handle = None

    def __del__(self):
        self.close()


def encode52(records) -> np.ndarray:
    """float64 [n][52][8][8]: the input planes of the paper's network (App. D.1, Table D.1) from
    128-byte records that carry the last eight moves."""
    rec, stride, n = _records(records)
    if stride != 128:
        raise ValueError("the 52-plane encoding needs 128-byte records with the last eight moves")
    planes = np.zeros((n, 52, 8, 8), dtype=np.float64)
    _load().orc_encode52(rec.ctypes.data, stride, n, planes.ctypes.data)
    return planes


def pnet_forward(blob: np.ndarray, planes: np.ndarray, masks: np.ndarray, want_raw=False, want_tower=False):
    """The paper's network on encoded planes [n][52][8][8] and 1,880-action masks [n][30]:
    (policy [n][1880], value [n][3] win/draw/loss) and, on request, a dict with the raw policy
    logits and the backbone's output [n][C][8][8]."""
    b = np.ascontiguousarray(blob, dtype=np.uint8)
    pl = np.ascontiguousarray(planes, dtype=np.float64)
    mk = np.ascontiguousarray(masks, dtype=np.uint64)
    n = pl.shape[0]
    channels = int(np.frombuffer(b[16:20].tobytes(), dtype="<u4")[0])
    policy = np.zeros((n, 1880), dtype=np.float64)
    value = np.zeros((n, 3), dtype=np.float64)
    raw = np.zeros((n, 1880), dtype=np.float64) if want_raw else None
    tower = np.zeros((n, channels, 8, 8), dtype=np.float64) if want_tower else None
    rc = _load().orc_pnet_forward(b.ctypes.data, b.size, pl.ctypes.data, mk.ctypes.data, n, policy.ctypes.data,
                                  value.ctypes.data, raw.ctypes.data if want_raw else None,
                                  tower.ctypes.data if want_tower else None)
    if rc != 0:
        raise ValueError("malformed network blob")
    if want_raw or want_tower:
        return policy, value, {"logits": raw, "tower": tower}
    return policy, value


def pnet_evaluate(blob: np.ndarray, records, **kw):
    """Records with the last eight moves -> (masks, planes, policy, value[, extras]) of the paper's network."""
    masks = legal_masks(np.ascontiguousarray(records["cur"]), 2)
    planes = encode52(records)
    out = pnet_forward(blob, planes, masks, **kw)
    return (masks, planes) + tuple(out)


def conv3x3(weight: np.ndarray, x: np.ndarray) -> np.ndarray:
    """weight float32 [cout][cin][3][3], x float64 [cin][8][8] -> float64 [cout][8][8]."""
    w = np.ascontiguousarray(weight, dtype=np.float32)
    xin = np.ascontiguousarray(x, dtype=np.float64)
    cout, cin = w.shape[0], w.shape[1]
    out = np.zeros((cout, 8, 8), dtype=np.float64)
    _load().orc_conv3x3(w.ctypes.data, xin.ctypes.data, cin, cout, out.ctypes.data)
    return out


def masked_softmax(logits: np.ndarray, mask_words: np.ndarray) -> np.ndarray:
    lg = np.ascontiguousarray(logits, dtype=np.float64)
    mk = np.ascontiguousarray(mask_words, dtype=np.uint64)
    out = np.zeros_like(lg)
    _load().orc_masked_softmax(lg.ctypes.data, mk.ctypes.data, lg.shape[0], out.ctypes.data)
    return out


def forward(blob: np.ndarray, planes: np.ndarray, masks: np.ndarray, want_raw: bool = False,
            want_tower: bool = False):
    """Network + masked softmax on already-encoded planes.

    Returns (policy [n][4672|1858], value [n][1|3]) and, on request, a dict with the raw logits,
    the value head's pre-activation and the tower's final activations.
    """
    blob = np.ascontiguousarray(blob, dtype=np.uint8)
    hdr = np.frombuffer(blob[8:36].tobytes(), dtype="<u4")
    channels, policy_head, value_head = int(hdr[3]), int(hdr[4]), int(hdr[5])
    pl = np.ascontiguousarray(planes, dtype=np.float64)
    mk = np.ascontiguousarray(masks, dtype=np.uint64)
    n = pl.shape[0]
    npol, V = POLICY_SIZE[policy_head], 3 if value_head else 1
    policy = np.zeros((n, npol), dtype=np.float64)
    value = np.zeros((n, V), dtype=np.float64)
    raw_l = np.zeros((n, npol), dtype=np.float64) if want_raw else None
    raw_v = np.zeros((n, V), dtype=np.float64) if want_raw else None
    tower = np.zeros((n, channels, 8, 8), dtype=np.float64) if want_tower else None
    ptr = lambda a: a.ctypes.data if a is not None else None
    rc = _load().orc_forward(blob.ctypes.data, blob.nbytes, pl.ctypes.data, mk.ctypes.data, n,
                             policy.ctypes.data, value.ctypes.data, ptr(raw_l), ptr(raw_v), ptr(tower))
    if rc != 0:
        raise ValueError("malformed weight blob")
    if want_raw or want_tower:
        return policy, value, {"logits": raw_l, "value_pre": raw_v, "tower": tower}
    return policy, value


def evaluate(blob: np.ndarray, records, in_planes: int, policy_head: int, **kw):
    """The whole path: masks from the rules, planes from the records, network, masked softmax."""
    masks = legal_masks(records, policy_head)
    planes = encode(records, in_planes)
    return (masks, planes) + tuple(forward(blob, planes, masks, **kw))


def threads() -> int:
    return int(_load().orc_threads())
