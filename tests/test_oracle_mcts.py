"""Pins of the oracle's tree search (Eq. 1, Sec. 3.4; constants of App. D.2) and of the stand-in evaluator
it searches with: bookkeeping invariants, the first two selections recomputed by hand from Eq. 1, forced
mates whose backed-up value the discount fixes, and the accounting of parallel leaves."""
import numpy as np
import pytest

import oracle
from inputs import positions

START = "rnbqkbnr/pppppppp/8/8/8/8/PPPPPPPP/RNBQKBNR w KQkq - 0 1"
MATE_IN_1 = "6k1/5ppp/8/8/8/8/8/R3K3 w Q - 0 1"          # Ra8 mates
MATE_IN_2 = "7k/8/5K2/8/8/8/8/6R1 w - - 0 1"             # king and rook against a cornered king: mate in two, none in one


def sq(name):
    return (ord(name[0]) - 97) + 8 * (int(name[1]) - 1)


def test_stand_in_evaluator_is_a_distribution_over_the_legal_actions():
    rec, _ = positions.generate(5, 30, (2, 80))
    cur = np.ascontiguousarray(rec["cur"])
    values = []
    for i in range(30):
        for head, size in ((1, 1858), (2, 1880)):
            a, p, v = oracle.synth_eval(cur[i], head, 7)
            mask = oracle.legal_masks(cur[i:i + 1], head)[0]
            bits = np.flatnonzero(np.unpackbits(mask.view(np.uint8), bitorder="little")[:size])
            assert (a == bits).all() and (p > 0).all() and abs(float(p.astype(np.float64).sum()) - 1) < 1e-5
            assert -0.75 <= v < 0.75
        a2, p2, v2 = oracle.synth_eval(cur[i], 2, 8)
        assert v2 != v or not np.array_equal(p2, p)          # the seed matters
        values.append(v)
    assert len(set(values)) > 25 and min(values) < -0.3 and max(values) > 0.3
    a, p, v = oracle.synth_eval(cur[0], 2, 7)
    b, q, w = oracle.synth_eval(cur[0], 2, 7)
    assert np.array_equal(p, q) and v == w


@pytest.mark.parametrize("head", [1, 2])
def test_bookkeeping_invariants(head):
    rec = positions.record_from_fen(START)
    r = oracle.mcts_search(rec, head, 300)
    assert r["flags"] == 0 and r["idle"] == 0
    assert r["visits"].sum() == 300 and r["n_nodes"] == 301          # every traversal ends in a new node here
    assert r["node_nvis"][0] == 301 and (r["node_nvis"][1:] >= 1).all()
    assert len(r["actions"]) == 20 and abs(float(r["prior"].sum()) - 1) < 1e-5
    # a node's visits = its own evaluation + the traversals that went on through it: the sum over all nodes
    # counts each traversal once per node of its path
    assert r["node_nvis"].sum() > 2 * 300
    q = r["w"][r["visits"] > 0] / r["visits"][r["visits"] > 0]
    assert (np.abs(q) <= 0.99 * 0.75 + 1e-6).all()                    # |value| <= 0.75, one ply of discount at least


def test_first_two_selections_follow_eq_1():
    rec, _ = positions.generate(11, 24, (2, 60))
    cur = np.ascontiguousarray(rec["cur"])
    checked = 0
    for i in range(24):
        a, p, v0 = oracle.synth_eval(cur[i], 1, 3)
        if len(a) < 2:
            continue
        one = oracle.mcts_search(cur[i:i + 1], 1, 1, seed=3)
        first = int(np.argmax(p))                                      # all Q equal: the largest prior wins, first of equals
        assert one["visits"][first] == 1 and one["visits"].sum() == 1
        child = oracle.apply_moves(cur[i:i + 1], 1, [int(a[first])])
        ca, cp, v1 = oracle.synth_eval(child[0], 1, 3)
        if len(ca) == 0 or child[0]["halfmove"] >= 100:
            continue
        w1 = -0.99 * v1
        assert abs(float(one["w"][first]) - w1) < 1e-6
        fpu = (v0 + w1) / 2 - 0.2
        score = fpu + 1.5 * p.astype(np.float64) * 1.0 / 1.0           # sqrt(max(1, N(s))) with N(s) = 1
        score[first] = w1 + 1.5 * float(p[first]) * 1.0 / 2.0
        order = np.sort(score)
        if order[-1] - order[-2] < 1e-5:
            continue                                                    # too close to call in float64
        second = int(np.argmax(score))
        two = oracle.mcts_search(cur[i:i + 1], 1, 2, seed=3)
        want = np.zeros(len(a), dtype=np.int32)
        want[first] += 1
        want[second] += 1
        assert (two["visits"] == want).all()
        checked += 1
    assert checked >= 15


def test_forced_mates_back_up_the_discounted_result():
    rec = positions.record_from_fen(MATE_IN_1)
    r = oracle.mcts_search(rec, 2, 400)
    mate = oracle.policy_index(2, 0, sq("a1"), sq("a8"))
    i = int(np.flatnonzero(r["actions"] == mate)[0])
    assert r["visits"][i] > 200 and abs(float(r["w"][i]) / int(r["visits"][i]) - 0.99) < 1e-5
    assert r["n_nodes"] < 400                                           # visits of the mated node open no new node
    rec = positions.record_from_fen(MATE_IN_2)
    r = oracle.mcts_search(rec, 2, 4000)
    # White mates by force but not in one move: the search settles on a winning line, and no root move can be
    # worth more than a mate three plies below it
    i = int(np.argmax(r["visits"]))
    assert r["visits"][i] > 2000
    q = r["w"].astype(np.float64) / np.maximum(r["visits"], 1)
    assert 0.85 < q[i] and (q <= 0.99 ** 3 + 1e-6).all()


def test_stalemate_and_fifty_move_leaves_are_draws():
    # Black to move is stalemated: the root itself is terminal, every traversal ends there with value 0
    r = oracle.mcts_search(positions.record_from_fen("7k/5Q2/6K1/8/8/8/8/8 b - - 0 1"), 2, 10)
    assert len(r["actions"]) == 0 and r["n_nodes"] == 1 and r["node_nvis"][0] == 11 and r["node_wsum"][0] == 0
    # halfmove clock 99: every quiet successor is a fifty-move draw, captures and pawn moves are not
    r = oracle.mcts_search(positions.record_from_fen("4k3/8/8/8/8/8/4P3/4K3 w - - 99 80"), 2, 50)
    pawn = {oracle.policy_index(2, 0, sq("e2"), sq("e3")), oracle.policy_index(2, 0, sq("e2"), sq("e4"))}
    for a, n, w in zip(r["actions"], r["visits"], r["w"]):
        if int(a) not in pawn and n > 0:
            assert w == 0


@pytest.mark.parametrize("leaves", [2, 8])
def test_parallel_leaves_accounting(leaves):
    rec = positions.record_from_fen(START)
    r = oracle.mcts_search(rec, 2, 100, leaves=leaves)
    # the root's step idles its other slots; afterwards every traversal is either counted or given up
    assert r["visits"].sum() + r["idle"] == 100 * leaves + (leaves - 1)
    assert r["n_nodes"] == 1 + r["visits"].sum()
    # the traversals of the first counted step take different root moves: a reservation counts as a lost visit
    one = oracle.mcts_search(rec, 2, 1, leaves=leaves)
    assert one["visits"].max() == 1 and one["visits"].sum() == leaves


def test_pools_that_fill_up_are_reported():
    rec = positions.record_from_fen(START)
    r = oracle.mcts_search(rec, 2, 100, node_cap=40, edge_cap=40 * 64)
    assert r["flags"] & 1 and r["n_nodes"] == 40 and r["visits"].sum() + r["idle"] == 100
    r = oracle.mcts_search(rec, 2, 100, node_cap=128, edge_cap=300)
    assert r["flags"] & 2 and r["n_edges"] <= 300 and r["visits"].sum() == 100


def test_played_moves_keep_their_subtree():
    rec = positions.record_from_fen(START)
    t = oracle.MctsTree(rec, 2, seed=4, node_cap=700)
    t.run(300)
    before = t.read()
    best = int(np.argmax(before["visits"]))
    action, n_child = int(before["actions"][best]), int(before["visits"][best])
    t.advance(action)
    after = t.read()
    # the new root is the old child: its position is the successor, its visits are the old edge's, and every visit
    # through it had opened exactly one node of its subtree (no terminal nodes this early in the game)
    assert (after["root"].view(np.uint8) == oracle.apply_moves(rec, 2, [action]).view(np.uint8)).all()
    assert after["node_nvis"][0] == n_child and after["n_nodes"] == n_child and after["visits"].sum() == n_child - 1
    # the kept statistics are the old ones: every (visits, value sum) pair of the new tree occurs in the old one
    old = {(int(n), np.float32(w).tobytes()) for n, w in zip(before["node_nvis"], before["node_wsum"])}
    assert all((int(n), np.float32(w).tobytes()) in old for n, w in zip(after["node_nvis"], after["node_wsum"]))
    # breadth-first renumbering: a node's visits never exceed its parent's, so the root comes first and the
    # first level (the root's visited edges, in edge order) follows
    level1 = after["visits"][after["visits"] > 0]
    assert (after["node_nvis"][1:1 + len(level1)] == level1).all()
    # the search goes on from the kept statistics
    t.run(100)
    more = t.read()
    assert more["node_nvis"][0] == n_child + 100 and more["visits"].sum() == n_child - 1 + 100
    with pytest.raises(ValueError):
        t.advance(1879)                                                  # a promotion cannot be legal here
    t.close()


def test_a_move_without_a_subtree_starts_a_fresh_tree():
    rec = positions.record_from_fen(START)
    t = oracle.MctsTree(rec, 2, seed=6, node_cap=300)
    t.run(5)
    r = t.read()
    unvisited = int(r["actions"][np.flatnonzero(r["visits"] == 0)[0]])
    t.advance(unvisited)
    assert t.read()["n_nodes"] == 1 and len(t.read()["actions"]) == 0      # waiting for its root evaluation
    t.run(120)
    got = t.read()
    want = oracle.mcts_search(oracle.apply_moves(rec, 2, [unvisited]), 2, 120, seed=6, node_cap=300)
    assert (got["visits"] == want["visits"]).all() and (got["w"].view(np.uint32) == want["w"].view(np.uint32)).all()
    assert (got["node_nvis"] == want["node_nvis"]).all()
    t.close()


def test_a_game_played_by_the_search_follows_the_rules():
    rec = positions.record_from_fen(START)
    t = oracle.MctsTree(rec, 2, leaves=2, seed=8, node_cap=400)
    cur = rec
    for ply in range(30):
        t.run(60)
        r = t.read()
        if len(r["actions"]) == 0:
            break
        a = int(r["actions"][int(np.argmax(r["visits"]))])
        cur = oracle.apply_moves(cur, 2, [a])
        t.advance(a)
        assert (t.read()["root"].view(np.uint8) == cur.view(np.uint8)).all()
    assert ply >= 10
    t.close()


def same_position(a, b):
    return (a["pieces"] == b["pieces"]).all() and a["stm"] == b["stm"] and a["castling"] == b["castling"] and a["ep_square"] == b["ep_square"]


def test_repetitions_across_played_moves():
    # the knights go out and come back, twice: the start position has then occurred twice before
    rec = positions.record_from_fen(START)
    shuffle = [("g1", "f3", 0), ("g8", "f6", 1), ("f3", "g1", 0), ("f6", "g8", 1)]
    # counts along the way: first round 0 0 0 1 (the start position again), second round 1 1 1 2
    t2 = oracle.MctsTree(rec, 2, seed=1, node_cap=200)
    seen = []
    for rnd in range(2):
        for frm, to, stm in shuffle:
            t2.run(0)                                                  # the root's own evaluation: it learns its moves
            t2.advance(oracle.policy_index(2, stm, sq(frm), sq(to)))
            seen.append(int(t2.read()["root"]["repetitions"][0]))
    assert seen == [0, 0, 0, 1, 1, 1, 1, 2]
    # a position that has occurred twice before is a draw: its evaluation finds no moves to search
    t2.run(5)
    r = t2.read()
    assert len(r["actions"]) == 0 and r["n_nodes"] == 1 and r["node_wsum"][0] == 0
    # a pawn move in between cuts the history off
    t3 = oracle.MctsTree(rec, 2, seed=1, node_cap=200)
    for frm, to, stm in shuffle[:2] + [("e2", "e4", 0), ("f6", "g8", 1), ("f3", "g1", 0)]:
        t3.run(0)
        t3.advance(oracle.policy_index(2, stm, sq(frm), sq(to)))
    assert int(t3.read()["root"]["repetitions"][0]) == 0
    for tr in (t2, t3):
        tr.close()


def test_repetition_counts_inside_a_tree_against_a_brute_force_walk():
    # few pieces: paths that return to an earlier position are common within a few plies
    repeated = 0
    for fen, seed in (("8/8/8/4k3/8/8/3QK3/8 w - - 10 40", 3), ("8/8/8/8/8/5k2/8/4K2R b - - 20 60", 5), ("8/8/8/4k3/8/8/3QK3/8 w - - 10 40", 9)):
        rec = positions.record_from_fen(fen)
        t = oracle.MctsTree(rec, 2, seed=seed, node_cap=3001)
        t.run(3000)
        n = t.read()["n_nodes"]
        nodes = [t.node(i) for i in range(n)]
        parents_with_children = {p for _, p in nodes}
        for i, (r, parent) in enumerate(nodes):
            cur = r[0]
            want, k, p = 0, 1, parent
            while p >= 0 and k <= int(cur["halfmove"]):
                pr = nodes[p][0][0]
                if same_position(pr, cur):
                    want = int(pr["repetitions"]) + 1
                    break
                p, k = nodes[p][1], k + 1
            assert int(cur["repetitions"]) == want, i
            repeated += want >= 1
            if want >= 2:
                assert i not in parents_with_children                     # a drawn node is never expanded
        t.close()
    assert repeated >= 10


def test_root_noise_mixes_into_the_root_priors_only():
    rec = positions.record_from_fen(START)
    t = oracle.MctsTree(rec, 2, seed=2, node_cap=400)
    assert t.root_noise(np.zeros(256, dtype=np.float32), 0.25) == 0             # the root has not been evaluated yet
    t.run(0)
    before = t.read()["prior"]
    eta = np.random.default_rng(5).dirichlet([0.3] * 20).astype(np.float32)     # App. D.2: alpha 0.3
    noise = np.zeros(256, dtype=np.float32)
    noise[:20] = eta
    assert t.root_noise(noise, 0.25) == 20
    after = t.read()["prior"]
    want = (np.float32(0.75) * before).astype(np.float32) + (np.float32(0.25) * eta).astype(np.float32)
    assert (after.view(np.uint32) == want.view(np.uint32)).all() and abs(float(after.sum()) - 1) < 1e-5
    # the search follows the noisy priors: its first traversal takes the largest of them
    t.run(1)
    r = t.read()
    assert r["visits"][int(np.argmax(after))] == 1
    # epsilon 0 changes nothing; the noise stays at the root's edges and nowhere else
    t2 = oracle.MctsTree(rec, 2, seed=2, node_cap=400)
    t2.run(0)
    t2.root_noise(noise, 0.0)
    assert (t2.read()["prior"].view(np.uint32) == before.view(np.uint32)).all()
    t.close()
    t2.close()
