"""Pins of the oracle's "apply an action" step: the tree of successors reached through the legal masks
and the action lists reproduces the published perft counts, and hand-built moves change the record the
way the rules say."""
import numpy as np
import pytest

import oracle
from inputs import positions

START = "rnbqkbnr/pppppppp/8/8/8/8/PPPPPPPP/RNBQKBNR w KQkq - 0 1"
KIWI = "r3k2r/p1ppqpb1/bn2pnp1/3PN3/1p2P3/2N2Q1p/PPPBBPPP/R3K2R w KQkq - 0 1"      # castling, en passant, promotions near


def sq(name):
    return (ord(name[0]) - 97) + 8 * (int(name[1]) - 1)


def children(rec, head, size):
    masks = oracle.legal_masks(rec, head)
    bits = np.unpackbits(masks.view(np.uint8), axis=1, bitorder="little")[:, :size].astype(bool)
    parent, action = np.nonzero(bits)
    return oracle.apply_moves(rec[parent], head, action.astype(np.int32))


@pytest.mark.parametrize("head,size", [(0, 4672), (1, 1858), (2, 1880)])
def test_successor_tree_reproduces_perft(head, size):
    # under-promotions are separate actions in every list; queen promotion is separate only in the 1,880 list,
    # so the action tree of the start position has the perft counts 20 / 400 / 8,902 in all three
    level = positions.record_from_fen(START)
    for want in (20, 400, 8902):
        level = children(level, head, size)
        assert level.shape[0] == want
    # a position with castling, en passant and captures: 48 / 2,039 (published perft of this position)
    level = positions.record_from_fen(KIWI)
    for want in (48, 2039):
        level = children(level, head, size)
        assert level.shape[0] == want


def test_hand_built_moves():
    def play(fen, head, frm, to, promo=0, castle=0):
        rec = positions.record_from_fen(fen)
        a = oracle.policy_index(head, int(rec["stm"][0]), sq(frm), sq(to), promo, castle)
        return oracle.apply_moves(rec, head, [a])[0]
    r = play(START, 1, "e2", "e4")
    assert r["stm"] == 1 and r["ep_square"] == sq("e3") and r["halfmove"] == 0 and r["castling"] == 15
    assert (int(r["pieces"][0]) >> sq("e4")) & 1 and not (int(r["pieces"][0]) >> sq("e2")) & 1
    r = play("r3k2r/8/8/8/8/8/8/R3K2R w KQkq - 7 20", 0, "e1", "g1", castle=1)        # short castling: king to g1, rook to f1
    assert (int(r["pieces"][5]) >> sq("g1")) & 1 and (int(r["pieces"][3]) >> sq("f1")) & 1 and not (int(r["pieces"][3]) >> sq("h1")) & 1
    assert r["castling"] == 12 and r["halfmove"] == 8 and r["ep_square"] == 64
    r = play("r3k2r/8/8/8/8/8/8/R3K2R b KQkq - 0 20", 2, "e8", "c8", castle=2)        # Black castles long
    assert (int(r["pieces"][11]) >> sq("c8")) & 1 and (int(r["pieces"][9]) >> sq("d8")) & 1 and r["castling"] == 3
    r = play("4k3/8/8/3pP3/8/8/8/4K3 w - d6 0 1", 1, "e5", "d6")                      # en passant removes the d5 pawn
    assert int(r["pieces"][6]) == 0 and (int(r["pieces"][0]) >> sq("d6")) & 1 and r["halfmove"] == 0
    r = play("1r2k3/P7/8/8/8/8/8/4K3 w - - 5 1", 2, "a7", "b8", promo=2)              # capture-promotion to a bishop
    assert (int(r["pieces"][2]) >> sq("b8")) & 1 and int(r["pieces"][0]) == 0 and int(r["pieces"][9]) == 0
    r = play("1r2k3/P7/8/8/8/8/8/4K3 w - - 5 1", 1, "a7", "a8")                       # plain action in the 1,858 list = queen
    assert (int(r["pieces"][4]) >> sq("a8")) & 1
    r = play("4k3/8/8/8/8/8/8/R3K2R w KQ - 0 1", 1, "h1", "h8")                       # the rook leaves home: that right is gone
    assert r["castling"] == 2
    with pytest.raises(ValueError):
        oracle.apply_moves(positions.record_from_fen(START), 1, [oracle.policy_index(1, 0, sq("e2"), sq("e5"))])


def test_history_and_move_records_are_pushed():
    rec, _ = positions.generate(31, 40, (3, 60))
    m8, _ = positions.generate_moves(31, 40, (3, 60))
    for r, head, size in ((rec, 1, 1858), (m8, 2, 1880)):
        masks = oracle.legal_masks(np.ascontiguousarray(r["cur"]), head)
        first = [int(np.flatnonzero(np.unpackbits(masks[i].view(np.uint8), bitorder="little")[:size])[0]) for i in range(40)]
        out = oracle.apply_moves(r, head, first)
        cur_only = oracle.apply_moves(np.ascontiguousarray(r["cur"]), head, first)
        assert (out["cur"] == cur_only).all()
        if head == 1:
            assert (out["hist_pieces"][:, 0] == r["cur"]["pieces"]).all() and (out["hist_pieces"][:, 1:] == r["hist_pieces"][:, :6]).all()
            assert (out["n_hist"] == np.minimum(r["n_hist"] + 1, 7)).all() and (out["hist_rep"][:, 0] == r["cur"]["repetitions"]).all()
        else:
            assert (out["move_from"][:, 1:] == r["move_from"][:, :7]).all() and (out["move_to"][:, 1:] == r["move_to"][:, :7]).all()
            assert (out["n_moves"] == np.minimum(r["n_moves"] + 1, 8)).all()
            # the pushed move's origin is empty afterwards and its destination holds a piece of the side that moved
            for i in range(40):
                occ = 0
                for b in out["cur"]["pieces"][i]:
                    occ |= int(b)
                assert not (occ >> int(out["move_from"][i, 0])) & 1 and (occ >> int(out["move_to"][i, 0])) & 1
