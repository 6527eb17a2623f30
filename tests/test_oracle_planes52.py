"""Pins of the oracle's 52-plane encoder (App. D.1, Table D.1) against what the table and the rules
of chess fix: hand-built positions, counting identities, colour-mirror symmetry, and agreement of
the checker plane with "is the mover in check" as the move generators see it."""
import numpy as np

import oracle
from inputs import positions


def m8_from_fen(fen, moves=()):
    rec = np.zeros(1, dtype=positions.M8_DTYPE)
    rec["cur"] = positions.record_from_fen(fen)
    rec["n_moves"] = len(moves)
    for t, (f, to) in enumerate(moves):
        rec["move_from"][0, t], rec["move_to"][0, t] = f, to
    return rec


def sq(name):
    return (ord(name[0]) - 97) + 8 * (int(name[1]) - 1)


def test_start_position_by_hand():
    p = oracle.encode52(m8_from_fen("rnbqkbnr/pppppppp/8/8/8/8/PPPPPPPP/RNBQKBNR w KQkq - 0 1"))[0]
    assert p[0, 1].sum() == 8 and p[0].sum() == 8                    # own pawns on row 1
    assert p[6, 6].sum() == 8 and p[6].sum() == 8                    # opponent pawns on row 6
    assert p[5, 0, 4] == 1 and p[11, 7, 4] == 1                      # kings on the e-file
    assert (p[12:16] == 1).all()                                     # all four castling rights
    assert p[16].sum() == 16 and p[17].sum() == 16 and (p[16, :2] == 1).all() and (p[17, 6:] == 1).all()
    assert p[18:38].sum() == 0                                       # no check, no en passant, no repetition, no history
    assert p[38, 0, 0] == 1 and p[38, 0, 1] == 0 and p[38, 1, 0] == 0 and p[38].sum() == 32
    assert (p[39] == 0).all() and (p[40:46] == 0).all() and (p[46] == 0).all()
    assert [p[47 + k, 0, 0] for k in range(5)] == [8, 2, 2, 2, 1]


def test_black_to_move_is_reflected_and_recoloured():
    # after 1. e4: Black to move, en-passant square e3, last move e2-e4
    p = oracle.encode52(m8_from_fen("rnbqkbnr/pppppppp/8/8/4P3/8/PPPP1PPP/RNBQKBNR b KQkq e3 0 1",
                                    [(sq("e2"), sq("e4"))]))[0]
    assert p[0, 1].sum() == 8                                        # Black's pawns are "own", on row 1 of the tensor
    assert p[6, 4, 4] == 1 and p[6, 6].sum() == 7                    # the white e-pawn: rank 4 -> row 7-3 = 4
    assert p[19].sum() == 1 and p[19, 5, 4] == 1                     # e3 -> row 7-2 = 5
    assert p[22].sum() == 1 and p[22, 6, 4] == 1 and p[23].sum() == 1 and p[23, 4, 4] == 1
    assert p[24:38].sum() == 0
    assert p[38, 0, 0] == 1                                          # the checkerboard does not move with the board


def test_checkers_castling_move_bishops_material_and_clock():
    # White to move: Kg1 Rf1 (castled two plies ago), Bc4; Black: Ke8, Bc8, Qh4 (no check), Nf3 (check)
    fen = "2b1k3/8/8/8/2B4q/5n2/8/5RK1 w - - 37 30"
    p = oracle.encode52(m8_from_fen(fen, [(sq("g5"), sq("f3")), (sq("e1"), sq("g1"))]))[0]
    assert p[18].sum() == 1 and p[18, 2, 5] == 1                     # only the knight on f3 checks
    assert p[24, 0, 4] == 1 and p[25, 0, 6] == 1                     # castling two plies back: king e1 -> g1
    assert (p[12:16] == 0).all()
    assert (p[39] == 0).all()                                        # c4 and c8 are both light squares
    assert (p[46] == 37).all()
    # balances own - opponent: P 0, N -1, B 0, R +1, Q -1, K 0; own counts P N B R Q
    assert [p[40 + k, 3, 3] for k in range(6)] == [0, -1, 0, 1, -1, 0]
    assert [p[47 + k, 7, 7] for k in range(5)] == [0, 0, 1, 1, 0]
    # the same with Black's bishop on d8 (dark) and a clock beyond the cap
    p2 = oracle.encode52(m8_from_fen("3bk3/8/8/8/2B4q/5n2/8/5RK1 w - - 137 30"))[0]
    assert (p2[39] == 1).all() and (p2[46] == 100).all()


def test_opposite_bishops_flag_exact():
    light = "4k3/8/8/8/2B5/8/8/4K3 w - - 0 1"                        # c4 is a light square
    for their, expect in (("2b1k3", 0), ("3bk3", 1)):               # c8 light, d8 dark
        fen = light.replace("4k3", their, 1)
        assert oracle.encode52(m8_from_fen(fen))[0][39, 0, 0] == expect
    two = "2bbk3/8/8/8/2B5/8/8/4K3 w - - 0 1"
    assert oracle.encode52(m8_from_fen(two))[0][39].sum() == 0


def test_counting_identities_and_mirror_symmetry_on_generated_positions():
    rec, plies = positions.generate_moves(20260952, 400, (0, 120))
    p = oracle.encode52(rec)
    cur = rec["cur"]
    for i in range(len(rec)):
        n_pieces = sum(bin(int(b)).count("1") for b in cur["pieces"][i])
        assert p[i, :12].sum() == n_pieces and p[i, 16].sum() + p[i, 17].sum() == n_pieces
        assert (p[i, 16] == p[i, 0:6].sum(axis=0)).all() and (p[i, 17] == p[i, 6:12].sum(axis=0)).all()
        k = min(int(plies[i]), 8)
        assert p[i, 22:38].sum() == 2 * k and all(p[i, 22 + j].sum() == 1 for j in range(2 * k))
        # the most recent move ended on a square now held by the opponent of the mover (the side that made it)
        if k:
            assert (p[i, 23] * p[i, 17]).sum() == 1
        # checkers are opponent pieces, two at most
        assert (p[i, 18] <= p[i, 17]).all() and p[i, 18].sum() <= 2
        assert p[i, 20, 0, 0] >= p[i, 21, 0, 0]
        assert set(np.unique(p[i, :40])) <= {0.0, 1.0}
        assert p[i, 45, 0, 0] == 0 and 0 <= p[i, 46, 0, 0] <= 100
    # colour mirror: exchanging colours and reflecting ranks (and the move squares) must not change the planes
    m = rec.copy()
    def flip_bb(b):
        b = int(b)
        return sum(((b >> (8 * r)) & 0xFF) << (8 * (7 - r)) for r in range(8))
    for i in range(len(rec)):
        for k in range(6):
            m["cur"]["pieces"][i, k] = flip_bb(cur["pieces"][i, 6 + k])
            m["cur"]["pieces"][i, 6 + k] = flip_bb(cur["pieces"][i, k])
        m["cur"]["stm"][i] = 1 - cur["stm"][i]
        c = int(cur["castling"][i])
        m["cur"]["castling"][i] = ((c & 3) << 2) | ((c >> 2) & 3)
        if cur["ep_square"][i] < 64:
            m["cur"]["ep_square"][i] = int(cur["ep_square"][i]) ^ 56
        m["move_from"][i] = rec["move_from"][i] ^ 56
        m["move_to"][i] = rec["move_to"][i] ^ 56
    assert (oracle.encode52(m) == p).all()


def _attackers_of_king(record):
    """Squares of the pieces that attack the mover's king: plain 8x8 array walk, written out here."""
    board = [[None] * 8 for _ in range(8)]
    for k in range(12):
        b = int(record["pieces"][k])
        for s in range(64):
            if (b >> s) & 1:
                board[s >> 3][s & 7] = (k // 6, "PNBRQK"[k % 6])      # (colour 0 white / 1 black, kind)
    me = int(record["stm"])
    (kr, kf), = [(r, f) for r in range(8) for f in range(8) if board[r][f] == (me, "K")]
    out = set()

    def at(r, f):
        return board[r][f] if 0 <= r < 8 and 0 <= f < 8 else None

    pawn_dr = 1 if me == 0 else -1                                    # enemy pawns sit one rank further up the board
    for df in (-1, 1):
        if at(kr + pawn_dr, kf + df) == (1 - me, "P"):
            out.add((kr + pawn_dr) * 8 + kf + df)
    for dr, df in ((1, 2), (2, 1), (2, -1), (1, -2), (-1, -2), (-2, -1), (-2, 1), (-1, 2)):
        if at(kr + dr, kf + df) == (1 - me, "N"):
            out.add((kr + dr) * 8 + kf + df)
    for dr, df, kinds in [(1, 0, "RQ"), (-1, 0, "RQ"), (0, 1, "RQ"), (0, -1, "RQ"),
                          (1, 1, "BQ"), (1, -1, "BQ"), (-1, 1, "BQ"), (-1, -1, "BQ")]:
        r, f = kr + dr, kf + df
        while 0 <= r < 8 and 0 <= f < 8 and board[r][f] is None:
            r, f = r + dr, f + df
        hit = at(r, f)
        if hit is not None and hit[0] == 1 - me and hit[1] in kinds:
            out.add(r * 8 + f)
    return out


def test_checker_plane_against_a_brute_force_walk():
    rec, _ = positions.generate_moves(20260953, 3000, (0, 160))
    p = oracle.encode52(rec)
    n_check = 0
    for i in range(len(rec)):
        flip = 56 if rec["cur"]["stm"][i] else 0
        got = {int(s) ^ flip for s in np.flatnonzero(p[i, 18].reshape(64))}
        want = _attackers_of_king(rec["cur"][i])
        assert got == want, (i, got, want)
        n_check += bool(want)
    assert n_check > 50                                              # the sample does contain checks
