"""Pins for the oracle's chess rules, policy index maps, legal masks and plane encoder (CPU only)."""
import os

import numpy as np
import pytest

import oracle
from inputs import positions

START = "rnbqkbnr/pppppppp/8/8/8/8/PPPPPPPP/RNBQKBNR w KQkq - 0 1"


def sq(name: str) -> int:
    return (ord(name[0]) - 97) + 8 * (int(name[1]) - 1)


def popcounts(masks: np.ndarray) -> np.ndarray:
    return np.unpackbits(masks.view(np.uint8), axis=1).sum(axis=1)


def mask_bits(row: np.ndarray, n: int) -> np.ndarray:
    return np.unpackbits(row.view(np.uint8), bitorder="little")[:n].astype(bool)


def mirror(rec: np.ndarray) -> np.ndarray:
    """Colour-flipped, rank-mirrored twin of 104-byte records."""
    out = rec.copy()
    for i in range(rec.shape[0]):
        for p in range(12):
            bb = int(rec["pieces"][i, p])
            flipped = int.from_bytes(bb.to_bytes(8, "little")[::-1], "little")   # reverse ranks
            out["pieces"][i, (p + 6) % 12] = flipped
        c = int(rec["castling"][i])
        out["castling"][i] = ((c & 3) << 2) | ((c >> 2) & 3)
        out["stm"][i] = 1 - int(rec["stm"][i])
        e = int(rec["ep_square"][i])
        out["ep_square"][i] = e ^ 56 if e < 64 else 64
    return out


def perft_cases(golden_dir):
    cases = []
    with open(os.path.join(golden_dir, "perft.txt")) as f:
        for line in f:
            if line.startswith("#") or "|" not in line:
                continue
            fen, counts = line.split("|")
            cases.append((fen.strip(), [int(c) for c in counts.split()]))
    return cases


def test_perft_start_position_counts_fixed_by_the_task(golden_dir):
    rec = positions.record_from_fen(START)
    assert [oracle.perft(rec, d) for d in (1, 2, 3, 4)] == [20, 400, 8902, 197281]


def test_perft_published_positions(golden_dir):
    for fen, counts in perft_cases(golden_dir):
        rec = positions.record_from_fen(fen)
        got = [oracle.perft(rec, d + 1) for d in range(len(counts))]
        assert got == counts, fen


def test_perft_is_colour_symmetric(golden_dir):
    # the mirrored twin of a position has the same move tree
    for fen, counts in perft_cases(golden_dir)[1:]:
        rec = mirror(positions.record_from_fen(fen))
        assert [oracle.perft(rec, d + 1) for d in range(3)] == counts[:3], fen


def test_move_sets_agree_with_the_generators_separate_rules_code():
    rec, _ = positions.generate(99, 6000, (0, 120))
    cur = positions.cur_records(rec)
    for i in range(cur.shape[0]):
        assert oracle.legal_moves(cur[i]) == positions.legal_moves(cur[i]), i


def test_en_passant_that_uncovers_a_rank_attack_is_illegal():
    rec = positions.record_from_fen("8/8/8/8/k2Pp2Q/8/8/3K4 b - d3 0 1")
    moves = oracle.legal_moves(rec)
    assert (sq("e4"), sq("d3"), 0) not in moves
    assert (sq("e4"), sq("e3"), 0) in moves
    rec2 = positions.record_from_fen("8/8/8/8/3Pp3/8/k7/3K4 b - d3 0 1")
    assert (sq("e4"), sq("d3"), 0) in oracle.legal_moves(rec2)


def test_castling_rules():
    free = oracle.legal_moves(positions.record_from_fen("4k3/8/8/8/8/8/8/R3K2R w KQ - 0 1"))
    assert len(free) == 26 and (sq("e1"), sq("g1"), 0) in free and (sq("e1"), sq("c1"), 0) in free
    # f1 attacked: no short castling, long castling still fine
    thru = oracle.legal_moves(positions.record_from_fen("4kr2/8/8/8/8/8/8/R3K2R w KQ - 0 1"))
    assert (sq("e1"), sq("g1"), 0) not in thru and (sq("e1"), sq("c1"), 0) in thru
    # b1 attacked only: long castling is still legal (the king does not cross b1)
    b1 = oracle.legal_moves(positions.record_from_fen("1r2k3/8/8/8/8/8/8/R3K2R w KQ - 0 1"))
    assert (sq("e1"), sq("c1"), 0) in b1
    # in check: no castling at all
    chk = oracle.legal_moves(positions.record_from_fen("4r1k1/8/8/8/8/8/8/R3K2R w KQ - 0 1"))
    assert (sq("e1"), sq("g1"), 0) not in chk and (sq("e1"), sq("c1"), 0) not in chk
    # no rights: no castling
    none = oracle.legal_moves(positions.record_from_fen("4k3/8/8/8/8/8/8/R3K2R w - - 0 1"))
    assert len(none) == 24


def test_promotions_come_in_four_pieces():
    moves = oracle.legal_moves(positions.record_from_fen("1n5k/P7/8/8/8/8/8/K7 w - - 0 1"))
    promos = sorted(m for m in moves if m[0] == sq("a7"))
    assert promos == sorted([(sq("a7"), sq("a8"), p) for p in (1, 2, 3, 4)] +
                            [(sq("a7"), sq("b8"), p) for p in (1, 2, 3, 4)])


# ---- policy index maps --------------------------------------------------------------------

def geometric_moves():
    """Every (from, to, promo) a piece could make in mover-oriented coordinates."""
    out = []
    for f in range(64):
        for t in range(64):
            if f == t:
                continue
            df, dr = (t & 7) - (f & 7), (t >> 3) - (f >> 3)
            ray = df == 0 or dr == 0 or abs(df) == abs(dr)
            jump = sorted((abs(df), abs(dr))) == [1, 2]
            if ray or jump:
                out.append((f, t, 0))
            if (f >> 3) == 6 and dr == 1 and abs(df) <= 1:
                out.extend((f, t, p) for p in (1, 2, 3))
    return out


def test_action_space_counts_match_the_papers_structure():
    moves = geometric_moves()
    pairs = [m for m in moves if m[2] == 0]
    promo_pairs = {(m[0], m[1]) for m in moves if m[2]}
    # 1,792 ray-or-knight pairs; 22 promotion (from, to) pairs -> 88 actions with four pieces in
    # the paper's list, 66 with three pieces here (queen promotion rides on the plain pair)
    assert len(pairs) == 1792 and len(promo_pairs) == 22
    assert 1792 + 4 * len(promo_pairs) == 1880
    assert len(moves) == 1858 == oracle.flat_count()


@pytest.mark.parametrize("head,size", [(0, 4672), (1, 1858)])
def test_index_maps_are_injective(head, size):
    moves = geometric_moves()
    idx = [oracle.policy_index(head, 0, f, t, p, 0) for f, t, p in moves]
    assert min(idx) >= 0 and max(idx) < size
    assert len(set(idx)) == len(moves) == 1858      # exactly 1,858 of the 4,672 cells are reachable
    if head == 1:
        assert sorted(idx) == list(range(1858))
        plain = [i for (f, t, p), i in zip(moves, idx) if p == 0]
        assert plain == sorted(plain) and plain == list(range(1792))   # (from, to) ascending order


def test_the_papers_1880_action_list():
    # Sec. 3.2 / App. D.1: 1,792 ray-or-knight pairs plus 88 promotions with four pieces each
    moves = [m for m in geometric_moves() if m[2] == 0]
    promos = [(f, t, p) for f in range(48, 56) for t in (f + 7, f + 8, f + 9)
              if abs((t & 7) - (f & 7)) <= 1 and t < 64 for p in (4, 3, 2, 1)]      # queen, rook, bishop, knight
    assert len(moves) == 1792 and len(promos) == 88
    idx = [oracle.policy_index(2, 0, f, t, p, 0) for f, t, p in moves + promos]
    assert idx == list(range(1880))                   # this very order, no gaps, nothing twice
    # plain pairs are numbered as in the 1,858 list
    assert [oracle.policy_index(1, 0, f, t, 0, 0) for f, t, _ in moves] == idx[:1792]
    # by hand: a7-a8=Q is the first promotion action, h7-h8=N the last; b7xa8=R: a-file has 2 combinations
    assert oracle.policy_index(2, 0, sq("a7"), sq("a8"), 4, 0) == 1792
    assert oracle.policy_index(2, 0, sq("h7"), sq("h8"), 1, 0) == 1879
    assert oracle.policy_index(2, 0, sq("b7"), sq("a8"), 3, 0) == 1792 + 4 * 2 + 1
    # Black's promotion is the mover's promotion; a promotion from anywhere else has no action
    assert oracle.policy_index(2, 1, sq("a2"), sq("a1"), 4, 0) == 1792
    assert oracle.policy_index(2, 0, sq("a6"), sq("a7"), 4, 0) == -1
    # masks: one bit per legal move, promotions on their own actions and not on the plain pair
    rec, _ = positions.generate(23, 1200, (0, 200))
    cur = positions.cur_records(rec)
    m2 = oracle.legal_masks(cur, 2)
    n = np.array([len(oracle.legal_moves(cur[i])) for i in range(cur.shape[0])])
    assert (popcounts(m2) == n).all()
    promo_rec = positions.record_from_fen("1r2k3/P7/8/8/8/8/8/4K3 w - - 0 1")
    bits = mask_bits(oracle.legal_masks(promo_rec, 2)[0], 1920)
    assert not bits[1880:].any()
    for to in ("a8", "b8"):
        for piece in (1, 2, 3, 4):
            assert bits[oracle.policy_index(2, 0, sq("a7"), sq(to), piece, 0)]
        assert not bits[oracle.policy_index(2, 0, sq("a7"), sq(to), 0, 0)]
    assert bits.sum() == len(oracle.legal_moves(promo_rec)) == 8 + 5


def test_index_73_plane_examples_by_hand():
    # plane = 7*direction + distance-1 with directions N, NE, E, SE, S, SW, W, NW; index = plane*64 + from
    assert oracle.policy_index(0, 0, sq("e2"), sq("e4"), 0, 0) == (7 * 0 + 1) * 64 + sq("e2")
    assert oracle.policy_index(0, 0, sq("a1"), sq("h8"), 0, 0) == (7 * 1 + 6) * 64 + sq("a1")
    assert oracle.policy_index(0, 0, sq("g1"), sq("f3"), 0, 0) == (56 + 7) * 64 + sq("g1")   # (-1,+2)
    assert oracle.policy_index(0, 0, sq("b1"), sq("c3"), 0, 0) == (56 + 0) * 64 + sq("b1")   # (+1,+2)
    # under-promotion to a rook, capturing towards the a-file, from b7
    assert oracle.policy_index(0, 0, sq("b7"), sq("a8"), 3, 0) == (64 + 3 * 2 + 0) * 64 + sq("b7")
    # queen promotion uses the one-step north plane
    assert oracle.policy_index(0, 0, sq("b7"), sq("b8"), 4, 0) == 0 * 64 + sq("b7")
    # Black's e7-e5 is the mover's e2-e4
    assert oracle.policy_index(0, 1, sq("e7"), sq("e5"), 0, 0) == oracle.policy_index(0, 0, sq("e2"), sq("e4"), 0, 0)
    # castling is king -> own rook square: short = east by 3, long = west by 4 (both colours)
    for stm, e, g, c in ((0, "e1", "g1", "c1"), (1, "e8", "g8", "c8")):
        assert oracle.policy_index(0, stm, sq(e), sq(g), 0, 1) == (7 * 2 + 2) * 64 + sq("e1")
        assert oracle.policy_index(0, stm, sq(e), sq(c), 0, 2) == (7 * 6 + 3) * 64 + sq("e1")
        assert oracle.policy_index(1, stm, sq(e), sq(g), 0, 1) == oracle.policy_index(1, 0, sq("e1"), sq("h1"), 0, 0)


def test_masks_count_legal_moves_and_agree_between_heads():
    rec, _ = positions.generate(7, 1500, (0, 160))
    cur = positions.cur_records(rec)
    m0, m1 = oracle.legal_masks(cur, 0), oracle.legal_masks(cur, 1)
    n = np.array([len(oracle.legal_moves(cur[i])) for i in range(cur.shape[0])])
    assert (popcounts(m0) == n).all() and (popcounts(m1) == n).all() and n.min() >= 1
    start = positions.record_from_fen(START)
    assert popcounts(oracle.legal_masks(start, 0))[0] == 20
    # no bit beyond the last index
    assert not mask_bits(m1[0], 1920)[1858:].any()


def test_masks_are_identical_for_the_colour_mirrored_twin():
    rec, _ = positions.generate(11, 800, (0, 120))
    cur = positions.cur_records(rec)
    twin = mirror(cur)
    for head in (0, 1):
        assert (oracle.legal_masks(cur, head) == oracle.legal_masks(twin, head)).all()


def test_castling_and_en_passant_bits_in_a_real_mask():
    rec = positions.record_from_fen("r3k2r/8/8/3pP3/8/8/8/R3K2R w KQkq d6 0 1")
    for head in (0, 1):
        bits = mask_bits(oracle.legal_masks(rec, head)[0], 4672 if head == 0 else 1858)
        assert bits[oracle.policy_index(head, 0, sq("e1"), sq("h1"), 0, 0)]     # short castling
        assert bits[oracle.policy_index(head, 0, sq("e1"), sq("a1"), 0, 0)]     # long castling
        assert bits[oracle.policy_index(head, 0, sq("e5"), sq("d6"), 0, 0)]     # en passant pair
        assert not bits[oracle.policy_index(head, 0, sq("e1"), sq("g1"), 0, 0)]  # king cannot step two


# ---- plane encoder -------------------------------------------------------------------------

def test_start_position_planes_by_hand():
    pl = oracle.encode(positions.record_from_fen(START), 19)[0]
    assert pl.shape == (19, 8, 8)
    assert (pl[0, 1] == 1).all() and pl[0].sum() == 8            # own pawns on row 1
    assert (pl[6, 6] == 1).all() and pl[6].sum() == 8            # opponent pawns on row 6
    assert pl[5, 0, 4] == 1 and pl[5].sum() == 1                 # own king on e1 (row 0, column 4)
    assert pl[11, 7, 4] == 1 and pl[4, 0, 3] == 1                # opponent king e8, own queen d1
    assert pl[3, 0, 0] == 1 and pl[3, 0, 7] == 1 and pl[3].sum() == 2
    assert (pl[12] == 0).all() and (pl[13:17] == 1).all()
    assert (pl[17] == 0).all() and (pl[18] == 0).all()


def test_black_to_move_is_reflected_and_colour_swapped():
    rec = positions.record_from_fen("rnbqkbnr/pppppppp/8/8/4P3/8/PPPP1PPP/RNBQKBNR b KQkq e3 0 1")
    pl = oracle.encode(rec, 19)[0]
    assert (pl[0, 1] == 1).all()                                 # Black's pawns are "own", on row 1
    assert pl[6, 4, 4] == 1 and pl[6, 6, 4] == 0                 # White's e4 pawn seen from Black: row 4
    assert pl[5, 0, 4] == 1 and (pl[12] == 1).all()


def test_piece_planes_hold_exactly_the_boards_pieces():
    rec, _ = positions.generate(3, 2000, (0, 160))
    cur = positions.cur_records(rec)
    pl = oracle.encode(cur, 19)
    n_pieces = np.array([sum(bin(int(b)).count("1") for b in cur["pieces"][i]) for i in range(cur.shape[0])])
    assert (pl[:, :12].sum(axis=(1, 2, 3)) == n_pieces).all()
    assert set(np.unique(pl[:, :12])) <= {0.0, 1.0}
    assert (pl[:, :12].sum(axis=1) <= 1).all()                   # at most one piece per square
    hm = np.minimum(cur["halfmove"].astype(np.int64), 100)
    expect = (hm.astype(np.float32) / np.float32(100.0)).astype(np.float64)
    assert (pl[:, 17, 0, 0] == expect).all() and (pl[:, 17] == pl[:, 17, :1, :1]).all()
    assert (pl[:, 18, 0, 0] == (cur["repetitions"] >= 1)).all()
    assert (pl[:, 12, 0, 0] == cur["stm"]).all()


def test_mirrored_twin_gives_the_same_planes_except_the_side_plane():
    rec, _ = positions.generate(5, 500, (0, 120))
    cur = positions.cur_records(rec)
    a, b = oracle.encode(cur, 19), oracle.encode(mirror(cur), 19)
    keep = [p for p in range(19) if p != 12]
    assert (a[:, keep] == b[:, keep]).all()
    assert (a[:, 12] == 1 - b[:, 12]).all()


def test_halfmove_plane_is_capped_at_100():
    rec = positions.record_from_fen("4k3/8/8/8/8/8/8/4K2R w K - 137 90")
    pl = oracle.encode(rec, 19)[0]
    assert (pl[17] == 1.0).all()
    assert (pl[13] == 1).all() and (pl[14] == 0).all() and (pl[15] == 0).all()


def test_history_planes():
    rec, plies = positions.generate(21, 400, (0, 30))
    pl = oracle.encode(rec, 112)
    cur19 = oracle.encode(positions.cur_records(rec), 19)
    assert (pl[:, 0:12] == cur19[:, 0:12]).all()                 # step 0 is the current board
    assert (pl[:, 12] == cur19[:, 18]).all()
    assert (pl[:, 104:108] == cur19[:, 13:17]).all()
    assert (pl[:, 108] == cur19[:, 12]).all() and (pl[:, 109] == cur19[:, 17]).all()
    assert (pl[:, 110] == 0).all() and (pl[:, 111] == 1).all()
    for i in range(rec.shape[0]):
        n = min(int(plies[i]), 7)
        assert int(rec["n_hist"][i]) == n
        assert (pl[i, 13 * (n + 1):104] == 0).all()              # missing history is zero-filled
        for t in range(1, n + 1):
            # board t plies ago, oriented by the CURRENT mover: encode it as a position of its own
            # with the current side to move and compare the piece planes
            old = np.zeros(1, dtype=positions.CUR_DTYPE)
            old["pieces"][0] = rec["hist_pieces"][i, t - 1]
            old["stm"] = rec["cur"]["stm"][i]
            old["ep_square"] = 64
            assert (pl[i, 13 * t:13 * t + 12] == oracle.encode(old, 19)[0, :12]).all()
            assert (pl[i, 13 * t + 12, 0, 0] == (rec["hist_rep"][i, t - 1] >= 1))
            # consecutive boards differ by one move: between 2 and 4 squares change
            prev = rec["hist_pieces"][i, t - 2] if t >= 2 else rec["cur"]["pieces"][i]
            changed = 0
            for p in range(12):
                changed |= int(prev[p]) ^ int(rec["hist_pieces"][i, t - 1, p])
            assert 2 <= bin(changed).count("1") <= 4
