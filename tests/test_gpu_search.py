"""The GPU search driver (Eq. 1, Sec. 3.4, 4.1, 5.1; App. D.2) against the oracle's sequential search:
successor positions bit-exact, the stand-in evaluator bit-exact, and with that evaluator whole trees equal
node by node (visit counts as integers, value sums as float32 bit patterns).  With a network as evaluator the
trees cannot be compared across precisions; the bookkeeping invariants and the root priors are checked."""
import numpy as np
import pytest
import torch

import oracle
from inputs import pnet_weights as pw
from inputs import positions

pytestmark = pytest.mark.gpu

START = "rnbqkbnr/pppppppp/8/8/8/8/PPPPPPPP/RNBQKBNR w KQkq - 0 1"
SPECIAL = [START,
           "r3k2r/p1ppqpb1/bn2pnp1/3PN3/1p2P3/2N2Q1p/PPPBBPPP/R3K2R w KQkq - 0 1",
           "6k1/5ppp/8/8/8/8/8/R3K3 w Q - 0 1",
           "7k/8/5K2/8/8/8/8/6R1 w - - 0 1",
           "7k/5Q2/6K1/8/8/8/8/8 b - - 0 1",
           "4k3/8/8/8/8/8/4P3/4K3 w - - 99 80",
           "1r2k3/P7/8/8/8/8/8/4K3 w - - 5 1",
           "4k3/8/8/3pP3/8/8/8/4K3 w - d6 0 1"]
SIZE = {0: 4672, 1: 1858, 2: 1880}


def records(head, stride, n, seed):
    """n generated records of the given layout, the special positions in front."""
    if stride == 128:
        rec, _ = positions.generate_moves(seed, n, (0, 160))
    else:
        rec, _ = positions.generate(seed, n, (0, 160))
        if stride == 104:
            rec = positions.cur_records(rec)
    rec = rec.copy()
    for i, fen in enumerate(SPECIAL):
        cur = positions.record_from_fen(fen)[0]
        if stride == 104:
            rec[i] = cur
        else:
            rec[i] = np.zeros((), dtype=rec.dtype)
            rec[i]["cur"] = cur
    return rec


def cur_of(rec):
    return np.ascontiguousarray(rec["cur"]) if rec.dtype.names and "cur" in rec.dtype.names else rec


@pytest.mark.parametrize("head,stride", [(0, 784), (1, 104), (2, 128), (0, 104), (1, 784)])
def test_successor_positions_are_bit_exact(head, stride):
    import paper_2609_37447_b200 as az
    rec = records(head, stride, 400, 20260980 + head)
    masks = oracle.legal_masks(cur_of(rec), head)
    bits = np.unpackbits(masks.view(np.uint8), axis=1, bitorder="little")[:, :SIZE[head]].astype(bool)
    parent, action = np.nonzero(bits)
    assert len(parent) > 8000
    src = np.ascontiguousarray(rec[parent])
    want = oracle.apply_moves(src, head, action.astype(np.int32))
    pos = az.records_to_device(src)
    out = torch.zeros_like(pos)
    act = torch.from_numpy(action.astype(np.int32)).cuda()
    status = torch.zeros(1, dtype=torch.int32, device="cuda")
    az.az_apply_moves(pos, stride, len(parent), head, act, out, status)
    torch.cuda.synchronize()
    got = out.cpu().numpy().view(np.uint8).reshape(len(parent), stride)
    ref = want.view(np.uint8).reshape(len(parent), stride)
    bad = np.flatnonzero((got != ref).any(axis=1))
    assert len(bad) == 0, (len(bad), parent[bad[:5]], action[bad[:5]])
    assert int(status.item()) == 0
    # an action whose origin is empty leaves a copy and raises the flag
    empty = torch.full((1,), int(oracle.policy_index(head, 0, 27, 35)), dtype=torch.int32, device="cuda")
    az.az_apply_moves(pos[:1], stride, 1, head, empty, out[:1], status)
    torch.cuda.synchronize()
    assert int(status.item()) == az.AZ_SEARCH_FLAG_BAD_ACTION and (out[:1].cpu() == pos[:1].cpu()).all()


@pytest.mark.parametrize("head,stride", [(1, 104), (2, 128)])
def test_stand_in_evaluator_is_bit_exact(head, stride):
    import paper_2609_37447_b200 as az
    rec = records(head, stride, 300, 20260985)
    n = rec.shape[0]
    pos = az.records_to_device(rec)
    masks = torch.zeros((n, 30), dtype=torch.int64, device="cuda")
    az.az_legal_masks(pos, stride, n, head, masks)
    legal = torch.full((n, az.AZ_MAX_LEGAL), -1.0, device="cuda")
    counts = torch.zeros(n, dtype=torch.int32, device="cuda")
    value = torch.zeros(n, device="cuda")
    az.az_standin_evaluate(pos, stride, masks, n, head, 77, legal, counts, value)
    torch.cuda.synchronize()
    legal, counts, value = legal.cpu().numpy(), counts.cpu().numpy(), value.cpu().numpy()
    cur = cur_of(rec)
    for i in range(n):
        a, p, v = oracle.synth_eval(cur[i], head, 77)
        assert counts[i] == len(a)
        assert (legal[i, :len(a)].view(np.uint32) == p.view(np.uint32)).all() and (legal[i, len(a):] == -1.0).all()
        assert np.float32(v).view(np.uint32) == value[i].view(np.uint32)


def run_gpu_search(az, rec, head, stride, sims, leaves, groups, max_nodes, max_edges, seed, c_puct=1.5, runs=1):
    cfg = az.make_search_config(rec.shape[0], head, stride, leaves=leaves, groups=groups, max_nodes=max_nodes,
                                max_edges=max_edges, evaluator=az.AZ_SEARCH_EVAL_STANDIN, c_puct=c_puct, seed=seed)
    s = az.az_search_create(None, cfg)
    az.az_search_set_roots(s, rec)
    for _ in range(runs):
        az.az_search_run(s, sims // runs)
    out = []
    for g in range(rec.shape[0]):
        a, n, w, p = az.az_search_root(s, g)
        counts, nvis, wsum = az.az_search_tree(s, g)
        out.append((a, n, w, p, counts, nvis, wsum))
    az.az_search_destroy(s)
    return out


def compare_with_oracle(got, rec, head, sims, leaves, max_nodes, max_edges, seed, c_puct=1.5):
    for g, (a, n, w, p, counts, nvis, wsum) in enumerate(got):
        want = oracle.mcts_search(rec[g:g + 1], head, sims, leaves=leaves, c_puct=c_puct, seed=seed,
                                  node_cap=max_nodes, edge_cap=max_edges)
        where = f"game {g}"
        assert (a == want["actions"]).all(), where
        assert (p.view(np.uint32) == want["prior"].view(np.uint32)).all(), where
        assert (n == want["visits"]).all(), (where, n, want["visits"])
        assert (w.view(np.uint32) == want["w"].view(np.uint32)).all(), where
        assert tuple(counts) == (want["n_nodes"], want["n_edges"], want["flags"], want["idle"]), where
        assert (nvis == want["node_nvis"]).all(), where
        assert (wsum.view(np.uint32) == want["node_wsum"].view(np.uint32)).all(), where


@pytest.mark.parametrize("head,stride,leaves,groups", [(2, 128, 1, 1), (2, 128, 4, 2), (1, 104, 1, 2), (1, 104, 8, 1), (0, 784, 2, 2)])
def test_trees_equal_the_oracles_node_by_node(head, stride, leaves, groups):
    import paper_2609_37447_b200 as az
    rec = records(head, stride, 29, 20260990 + leaves)               # 29 games: an odd split over two groups, a ragged last block
    sims, nodes = 240, 240 * leaves + 2
    got = run_gpu_search(az, rec, head, stride, sims, leaves, groups, nodes, 48 * nodes, seed=5)
    compare_with_oracle(got, rec, head, sims, leaves, nodes, 48 * nodes, seed=5)


def test_runs_add_up_and_other_constants():
    import paper_2609_37447_b200 as az
    rec = records(2, 128, 12, 20260995)
    # three runs of 100 steps are one search of 300; the evaluation constants of App. B.1 (c = 1.0)
    got = run_gpu_search(az, rec, 2, 128, 300, 2, 2, 700, 700 * 48, seed=9, c_puct=1.0, runs=3)
    compare_with_oracle(got, rec, 2, 300, 2, 700, 700 * 48, seed=9, c_puct=1.0)


def test_full_pools_are_reported_like_the_oracles():
    import paper_2609_37447_b200 as az
    rec = records(2, 128, 10, 20260996)
    got = run_gpu_search(az, rec, 2, 128, 150, 2, 1, 60, 60 * 48, seed=3)
    compare_with_oracle(got, rec, 2, 150, 2, 60, 60 * 48, seed=3)
    assert any(c[4][2] & az.AZ_SEARCH_FLAG_NODES_FULL for c in got)
    got = run_gpu_search(az, rec, 2, 128, 150, 1, 1, 200, 400, seed=3)
    compare_with_oracle(got, rec, 2, 150, 1, 200, 400, seed=3)
    assert any(c[4][2] & az.AZ_SEARCH_FLAG_EDGES_FULL for c in got)


@pytest.mark.parametrize("games", [592, 640])
def test_many_games_in_the_benchmarks_launch_configuration(games):
    """Two groups of 296 games (the benchmark's default: one two-board group per SM) and of 320 (the paper's batch,
    Sec. 5.1), 64 steps; sampled games against the oracle."""
    import paper_2609_37447_b200 as az
    rec = records(2, 128, games, 20260997)
    got = run_gpu_search(az, rec, 2, 128, 64, 1, 2, 80, 80 * 64, seed=11)
    half = games // 2
    pick = [0, 1, 2, 3, 4, 5, 6, 7, 100, half - 1, half, half + 1, 400, games - 1]
    compare_with_oracle([got[g] for g in pick], rec[pick], 2, 64, 1, 80, 80 * 64, seed=11)
    for a, n, w, p, counts, nvis, wsum in got:
        assert n.sum() + counts[3] == 64 or len(a) == 0


def test_root_visits_of_all_games_in_one_copy():
    import paper_2609_37447_b200 as az
    rec = records(2, 128, 33, 20260994)
    s = az.az_search_create(None, az.make_search_config(33, 2, 128, leaves=2, max_nodes=300, evaluator=az.AZ_SEARCH_EVAL_STANDIN, seed=2))
    az.az_search_set_roots(s, rec)
    az.az_search_run(s, 120)
    actions = np.full((33, az.AZ_MAX_LEGAL), -1, dtype=np.int32)
    visits = np.full((33, az.AZ_MAX_LEGAL), -1, dtype=np.int32)
    counts = np.zeros(33, dtype=np.int32)
    az.az_search_root_visits(s, actions, visits, counts)
    for g in range(33):
        a, n, w, p = az.az_search_root(s, g)
        assert counts[g] == len(a) and (actions[g, :len(a)] == a).all() and (visits[g, :len(a)] == n).all()
    az.az_search_destroy(s)


def read_gpu_tree(az, s, g):
    a, n, w, p = az.az_search_root(s, g)
    counts, nvis, wsum = az.az_search_tree(s, g)
    return a, n, w, p, counts, nvis, wsum


def same_tree(got, want, where):
    a, n, w, p, counts, nvis, wsum = got
    assert (a == want["actions"]).all() and (n == want["visits"]).all(), where
    assert (w.view(np.uint32) == want["w"].view(np.uint32)).all() and (p.view(np.uint32) == want["prior"].view(np.uint32)).all(), where
    assert tuple(counts) == (want["n_nodes"], want["n_edges"], want["flags"], want["idle"]), (where, counts, want["n_nodes"], want["n_edges"])
    assert (nvis == want["node_nvis"]).all() and (wsum.view(np.uint32) == want["node_wsum"].view(np.uint32)).all(), where


@pytest.mark.parametrize("head,stride,leaves", [(2, 128, 1), (1, 784, 3)])
def test_games_played_by_the_search_keep_their_subtrees_like_the_oracles(head, stride, leaves):
    """Every game plays its most visited move after each search; trees, positions and moves equal the oracle's
    at every ply (stand-in evaluator on both sides)."""
    import paper_2609_37447_b200 as az
    rec = records(head, stride, 21, 20261001)
    n, sims, cap = rec.shape[0], 50, 50 * leaves * 14 + 2
    s = az.az_search_create(None, az.make_search_config(n, head, stride, leaves=leaves, groups=2, max_nodes=cap, max_edges=cap * 48,
                                                        evaluator=az.AZ_SEARCH_EVAL_STANDIN, seed=13))
    az.az_search_set_roots(s, rec)
    trees = [oracle.MctsTree(rec[g:g + 1], head, leaves=leaves, seed=13, node_cap=cap, edge_cap=cap * 48) for g in range(n)]
    moved = 0
    for ply in range(12):
        az.az_search_run(s, sims)
        want_play = []
        for g in range(n):
            trees[g].run(sims)
            want = trees[g].read()
            same_tree(read_gpu_tree(az, s, g), want, f"ply {ply} game {g}")
            want_play.append(int(want["actions"][int(np.argmax(want["visits"]))]) if len(want["actions"]) else -1)
        played = az.az_search_advance(s)
        assert (played == np.array(want_play)).all()
        roots = az.az_search_root_positions(s, rec.dtype)
        for g in range(n):
            if want_play[g] >= 0:
                trees[g].advance(want_play[g])
                moved += 1
            want = trees[g].read()
            assert (roots[g:g + 1].view(np.uint8) == want["root"].view(np.uint8)).all(), f"ply {ply} game {g}"
            same_tree(read_gpu_tree(az, s, g), want, f"after the move of ply {ply}, game {g}")
    assert moved > 10 * (n - 3)
    az.az_search_destroy(s)
    for t in trees:
        t.close()


def test_repetitions_inside_trees_and_across_played_moves():
    """Endgames with few pieces, where paths return to earlier positions: repetition counts in the records, drawn
    leaves and the history across played moves equal the oracle's (which a brute-force walk pins)."""
    import paper_2609_37447_b200 as az
    fens = ["8/8/8/4k3/8/8/3QK3/8 w - - 10 40", "8/8/8/8/8/5k2/8/4K2R b - - 20 60", "8/8/4k3/8/8/3K4/8/R7 w - - 30 70",
            "8/5k2/8/8/8/8/2Q5/K7 b - - 4 50", "7k/8/8/8/8/8/R7/K7 w - - 0 1"]
    rec, _ = positions.generate_moves(1, len(fens), (0, 2))
    rec = rec.copy()
    for i, fen in enumerate(fens):
        rec[i] = np.zeros((), dtype=rec.dtype)
        rec[i]["cur"] = positions.record_from_fen(fen)[0]
    n, sims, cap = len(fens), 400, 2600
    s = az.az_search_create(None, az.make_search_config(n, 2, 128, leaves=1, groups=2, max_nodes=cap, max_edges=cap * 32,
                                                        evaluator=az.AZ_SEARCH_EVAL_STANDIN, seed=17))
    az.az_search_set_roots(s, rec)
    trees = [oracle.MctsTree(rec[g:g + 1], 2, seed=17, node_cap=cap, edge_cap=cap * 32) for g in range(n)]
    repeated_nodes, repeated_roots = 0, 0
    for ply in range(10):
        az.az_search_run(s, sims)
        for g in range(n):
            trees[g].run(sims)
            want = trees[g].read()
            same_tree(read_gpu_tree(az, s, g), want, f"ply {ply} game {g}")
            if ply == 0:
                repeated_nodes += sum(int(trees[g].node(i)[0]["cur"]["repetitions"][0]) >= 1 for i in range(want["n_nodes"]))
        # the least visited tried move: shuffles rather than progress
        actions = np.full(n, -1, dtype=np.int32)
        for g in range(n):
            r = trees[g].read()
            tried = np.flatnonzero(r["visits"] > 0)
            if len(tried):
                actions[g] = int(r["actions"][tried[np.argmin(r["visits"][tried])]])
        played = az.az_search_advance(s, actions)
        assert (played == actions).all()
        roots = az.az_search_root_positions(s, rec.dtype)
        for g in range(n):
            if actions[g] >= 0:
                trees[g].advance(int(actions[g]))
            want = trees[g].read()
            assert (roots[g:g + 1].view(np.uint8) == want["root"].view(np.uint8)).all(), f"ply {ply} game {g}"
            repeated_roots += int(want["root"]["cur"]["repetitions"][0]) >= 1
    assert repeated_nodes >= 5
    az.az_search_destroy(s)
    for t in trees:
        t.close()


def test_given_moves_none_unvisited_and_impossible_ones():
    import paper_2609_37447_b200 as az
    rec = records(2, 128, 12, 20261002)
    n = rec.shape[0]
    s = az.az_search_create(None, az.make_search_config(n, 2, 128, leaves=1, groups=1, max_nodes=400, evaluator=az.AZ_SEARCH_EVAL_STANDIN, seed=21))
    az.az_search_set_roots(s, rec)
    trees = [oracle.MctsTree(rec[g:g + 1], 2, seed=21, node_cap=400, edge_cap=400 * 64) for g in range(n)]
    az.az_search_run(s, 12)
    actions = np.full(n, -1, dtype=np.int32)
    for g in range(n):
        trees[g].run(12)
        r = trees[g].read()
        if len(r["actions"]) == 0:
            continue
        if g % 3 == 0:                                           # a move the search never tried: a fresh tree
            actions[g] = int(r["actions"][np.flatnonzero(r["visits"] == 0)[0]])
        elif g % 3 == 1:                                         # the least visited of the tried moves
            tried = np.flatnonzero(r["visits"] > 0)
            actions[g] = int(r["actions"][tried[np.argmin(r["visits"][tried])]])
    bad = 9
    actions[bad] = 1879 if not (trees[bad].read()["actions"] == 1879).any() else 1878      # not a move of that root
    played = az.az_search_advance(s, actions)
    for g in range(n):
        if g == bad:
            assert played[g] == -1 and az.az_search_tree(s, g, nodes=False)[0][2] & az.AZ_SEARCH_FLAG_BAD_ACTION
            continue
        assert played[g] == actions[g]
        if actions[g] >= 0:
            trees[g].advance(int(actions[g]))
    # the next run: fresh trees evaluate their roots in a step of their own while the others sit it out
    az.az_search_run(s, 40)
    for g in range(n):
        trees[g].run(40)
        got = read_gpu_tree(az, s, g)
        want = trees[g].read()
        if g == bad:
            want["flags"] |= az.AZ_SEARCH_FLAG_BAD_ACTION
        same_tree(got, want, f"game {g}")
    az.az_search_destroy(s)
    for t in trees:
        t.close()


def test_random_configurations_against_the_oracle():
    """Thirty seeded configurations (games, leaves, groups, action list, record layout, pool sizes, constants),
    each searched, moved and searched again on both sides."""
    import paper_2609_37447_b200 as az
    rng = np.random.default_rng(20261010)
    for case in range(30):
        head, stride = [(0, 104), (0, 784), (1, 104), (1, 784), (2, 128)][int(rng.integers(5))]
        games, leaves, groups = int(rng.integers(1, 10)), int(rng.choice([1, 1, 2, 3, 5, 8, 16])), int(rng.integers(1, 3))
        sims = int(rng.integers(5, 70))
        cap = int(rng.choice([sims * leaves * 3 + 2, max(8, sims * leaves // 2)]))          # roomy, or a pool that fills up
        ecap = int(rng.choice([cap * 48, cap * 12]))
        c_puct, fpu, disc = float(rng.choice([1.5, 1.0, 3.0, 0.0])), float(rng.choice([0.2, 0.0, 0.5])), float(rng.choice([0.99, 1.0, 0.9]))
        seed = int(rng.integers(1 << 30))
        rec = records(head, stride, max(games, 9), 20261011 + case)[rng.permutation(max(games, 9))[:games]]
        rec = np.ascontiguousarray(rec)
        cfg = az.make_search_config(games, head, stride, leaves=leaves, groups=groups, max_nodes=cap, max_edges=ecap,
                                    evaluator=az.AZ_SEARCH_EVAL_STANDIN, c_puct=c_puct, fpu_reduction=fpu, discount=disc, seed=seed)
        s = az.az_search_create(None, cfg)
        az.az_search_set_roots(s, rec)
        trees = [oracle.MctsTree(rec[g:g + 1], head, leaves=leaves, c_puct=c_puct, fpu_reduction=fpu, discount=disc, seed=seed,
                                 node_cap=cap, edge_cap=ecap) for g in range(games)]
        for phase in range(3):
            az.az_search_run(s, sims)
            for g in range(games):
                trees[g].run(sims)
                same_tree(read_gpu_tree(az, s, g), trees[g].read(), f"case {case} phase {phase} game {g}")
            played = az.az_search_advance(s)
            for g in range(games):
                r = trees[g].read()
                want = int(r["actions"][int(np.argmax(r["visits"]))]) if len(r["actions"]) else -1
                assert played[g] == want, f"case {case} phase {phase} game {g}"
                if want >= 0:
                    trees[g].advance(want)
        az.az_search_destroy(s)
        for t in trees:
            t.close()


def test_search_with_the_network_as_evaluator():
    import paper_2609_37447_b200 as az
    cfg = pw.PNetConfig("ts", 2, 128, 64, 20260998, 4500)
    blob = pw.make_blob(cfg, 0.1, 0.6)
    arch = az.make_arch(52, cfg.blocks, cfg.channels, 2, 1, cfg.precision, 128)
    net = az.az_load_net(arch, blob)
    rec = records(2, 128, 40, 20260999)
    n = rec.shape[0]
    sc = az.make_search_config(n, 2, 128, leaves=2, groups=2, max_nodes=256, evaluator=az.AZ_SEARCH_EVAL_NET)
    s = az.az_search_create(net, sc)
    az.az_search_set_roots(s, rec)
    ms = az.az_search_run(s, 100)
    assert ms > 0 and az.az_search_launches_per_step(s) == 3 + az.az_launches_per_evaluate(net, 40)
    # the root priors are the evaluator's own output for the root positions
    pos = az.records_to_device(rec)
    masks = torch.zeros((n, 30), dtype=torch.int64, device="cuda")
    az.az_legal_masks(pos, 128, n, 2, masks)
    legal = torch.zeros((n, az.AZ_MAX_LEGAL), device="cuda")
    counts = torch.zeros(n, dtype=torch.int32, device="cuda")
    value = torch.zeros((n, 3), device="cuda")
    az.az_evaluate_legal(net, pos, masks, n, legal, counts, value)
    torch.cuda.synchronize()
    legal, counts, value = legal.cpu().numpy(), counts.cpu().numpy(), value.cpu().numpy()
    want_masks = oracle.legal_masks(cur_of(rec), 2)
    for g in range(n):
        a, nv, w, p = az.az_search_root(s, g)
        c, nvis, wsum = az.az_search_tree(s, g)
        bits = np.flatnonzero(np.unpackbits(want_masks[g].view(np.uint8), bitorder="little")[:1880])
        if len(bits) == 0 or rec[g]["cur"]["halfmove"] >= 100:
            assert len(a) == 0 and c[0] == 1
            continue
        assert (a == bits).all() and c[2] == 0
        assert (p.view(np.uint32) == legal[g, :counts[g]].view(np.uint32)).all()
        assert nv.sum() + c[3] == 200 + 1 and c[0] <= 1 + nv.sum()       # the root's step idles its second row
        assert nvis[0] == 1 + nv.sum() and (np.abs(w) <= nv + 1e-4).all()
        # the root's value sum starts with its own evaluation: win minus loss
        assert abs(float(wsum[0]) - float(w.sum()) - float(value[g, 0] - value[g, 2])) < 1e-3
    az.az_search_destroy(s)
    # a second search object on the same net, one group, gives the same trees as two groups (the order of the
    # steps of different games does not matter)
    s1 = az.az_search_create(net, az.make_search_config(n, 2, 128, leaves=2, groups=1, max_nodes=256))
    s2 = az.az_search_create(net, az.make_search_config(n, 2, 128, leaves=2, groups=2, max_nodes=256))
    for s in (s1, s2):
        az.az_search_set_roots(s, rec)
        az.az_search_run(s, 60)
    for g in range(n):
        r1, r2 = az.az_search_root(s1, g), az.az_search_root(s2, g)
        assert all((x.view(np.uint32) == y.view(np.uint32)).all() for x, y in zip(r1, r2))
    az.az_search_destroy(s1)
    az.az_search_destroy(s2)
    assert az.az_device_status(net) & ~1 == 0                            # only "a position had no legal move" may be set
    az.az_free_net(net)


@pytest.mark.parametrize("in_planes,head,value_head,precision,channels", [(19, 1, 1, 1, 128), (112, 0, 0, 1, 128), (19, 0, 0, 0, 32)])
def test_search_over_the_residual_tower_configs(in_planes, head, value_head, precision, channels):
    """The classic networks as evaluators: tensor-core path with its second workspace (two groups side by side),
    the 112-plane records with history, and the FP32-ALU path (one workspace: the groups take turns)."""
    import paper_2609_37447_b200 as az
    from inputs import configs, weights
    cfg = configs.tiny_config(in_planes=in_planes, blocks=2, channels=channels, policy_head=head, value_head=value_head,
                              precision=precision, batch=64)
    blob = weights.make_blob(cfg, 0.02, 0.05)
    net = az.az_load_net(az.make_arch(in_planes, 2, channels, head, value_head, precision, 64), blob)
    stride = 784 if in_planes == 112 else 104
    rec = records(head, stride, 31, 20261003)
    n, size = rec.shape[0], SIZE[head]
    results = []
    for groups in (2, 1):
        s = az.az_search_create(net, az.make_search_config(n, head, stride, leaves=2, groups=groups, max_nodes=200))
        az.az_search_set_roots(s, rec)
        az.az_search_run(s, 40)
        played = az.az_search_advance(s)
        az.az_search_run(s, 40)
        out = []
        for g in range(n):
            a, nv, w, p = az.az_search_root(s, g)
            c, nvis, wsum = az.az_search_tree(s, g)
            out.append((a, nv, w, p, c, nvis, wsum, played[g]))
            assert c[2] == 0 and (nvis[0] == 1 + nv.sum() or len(a) == 0)
            assert (np.abs(w) <= nv + 1e-4).all() and (len(a) == 0 or abs(float(p.sum()) - 1) < 1e-3)
        results.append(out)
        az.az_search_destroy(s)
    # one group and two groups: the same trees, bit for bit
    for x, y in zip(*results):
        assert all(np.atleast_1d(u).tobytes() == np.atleast_1d(v).tobytes() for u, v in zip(x, y))
    # the moves played are legal moves of the roots
    masks = oracle.legal_masks(cur_of(rec), head)
    for g in range(n):
        pl = int(results[0][g][7])
        if pl >= 0:
            assert (int(masks[g, pl >> 6]) >> (pl & 63)) & 1
    assert az.az_device_status(net) & ~1 == 0
    az.az_free_net(net)


def test_degenerate_runs():
    """No steps at all (only the roots are evaluated), a single game with the maximum number of leaves, roots set anew."""
    import paper_2609_37447_b200 as az
    rec = records(2, 128, 9, 20261030)
    s = az.az_search_create(None, az.make_search_config(9, 2, 128, leaves=az.AZ_SEARCH_MAX_LEAVES, groups=2, max_nodes=600,
                                                        evaluator=az.AZ_SEARCH_EVAL_STANDIN, seed=4))
    az.az_search_set_roots(s, rec)
    az.az_search_run(s, 0)
    for g in range(9):
        want = oracle.mcts_search(rec[g:g + 1], 2, 0, leaves=16, seed=4, node_cap=600)
        same_tree(read_gpu_tree(az, s, g), want, f"game {g}")
        assert want["n_nodes"] == 1 and want["visits"].sum() == 0
    az.az_search_run(s, 30)
    az.az_search_set_roots(s, rec[::-1].copy())              # new roots: the old trees are gone
    az.az_search_run(s, 20)
    for g in range(9):
        want = oracle.mcts_search(rec[8 - g:9 - g], 2, 20, leaves=16, seed=4, node_cap=600)
        same_tree(read_gpu_tree(az, s, g), want, f"game {g} after the reset")
    az.az_search_destroy(s)
    one = az.az_search_create(None, az.make_search_config(1, 2, 128, leaves=16, groups=2, max_nodes=900,
                                                          evaluator=az.AZ_SEARCH_EVAL_STANDIN, seed=4))
    az.az_search_set_roots(one, rec[:1])
    az.az_search_run(one, 50)
    same_tree(read_gpu_tree(az, one, 0), oracle.mcts_search(rec[:1], 2, 50, leaves=16, seed=4, node_cap=900), "one game")
    az.az_search_destroy(one)


def test_some_games_start_anew_while_the_others_go_on():
    import paper_2609_37447_b200 as az
    rec = records(2, 128, 14, 20261040)
    fresh = records(2, 128, 12, 20261041)[9:12]
    s = az.az_search_create(None, az.make_search_config(14, 2, 128, leaves=2, groups=2, max_nodes=500, evaluator=az.AZ_SEARCH_EVAL_STANDIN, seed=6))
    az.az_search_set_roots(s, rec)
    trees = [oracle.MctsTree(rec[g:g + 1], 2, leaves=2, seed=6, node_cap=500, edge_cap=500 * 64) for g in range(14)]
    az.az_search_run(s, 60)
    az.az_search_advance(s)
    for g in range(14):
        trees[g].run(60)
        r = trees[g].read()
        if len(r["actions"]):
            trees[g].advance(int(r["actions"][int(np.argmax(r["visits"]))]))
    picked = [11, 0, 6]
    az.az_search_replace_roots(s, picked, fresh)
    for i, g in enumerate(picked):
        trees[g].close()
        trees[g] = oracle.MctsTree(fresh[i:i + 1], 2, leaves=2, seed=6, node_cap=500, edge_cap=500 * 64)
    az.az_search_run(s, 45)
    roots = az.az_search_root_positions(s, rec.dtype)
    for g in range(14):
        trees[g].run(45)
        want = trees[g].read()
        same_tree(read_gpu_tree(az, s, g), want, f"game {g}")
        assert (roots[g:g + 1].view(np.uint8) == want["root"].view(np.uint8)).all()
    with pytest.raises(az.AzError) as e:
        az.az_search_replace_roots(s, [14], fresh[:1])
    assert e.value.code == az.AZ_ERR_BAD_ARG
    with pytest.raises(az.AzError) as e:
        az.az_search_replace_roots(s, [3, 3], fresh[:2])
    assert e.value.code == az.AZ_ERR_BAD_ARG
    az.az_search_replace_roots(s, [], fresh[:0])
    az.az_search_destroy(s)
    for t in trees:
        t.close()


def test_root_noise_like_the_oracles():
    """A self-play style loop: evaluate the roots, mix Dirichlet noise (drawn here) into their priors, search, play,
    and again on the kept subtrees' roots; trees equal the oracle's throughout."""
    import paper_2609_37447_b200 as az
    rec = records(2, 128, 11, 20261060)
    n = rec.shape[0]
    s = az.az_search_create(None, az.make_search_config(n, 2, 128, leaves=2, groups=2, max_nodes=700, evaluator=az.AZ_SEARCH_EVAL_STANDIN, seed=8))
    az.az_search_set_roots(s, rec)
    trees = [oracle.MctsTree(rec[g:g + 1], 2, leaves=2, seed=8, node_cap=700, edge_cap=700 * 64) for g in range(n)]
    rng = np.random.default_rng(77)
    early = az.az_search_root_noise(s, np.zeros((n, az.AZ_MAX_LEGAL), dtype=np.float32), 0.25)
    assert (early == 0).all()                                            # no root has been evaluated yet
    for move in range(4):
        az.az_search_run(s, 0)                                           # roots that are new evaluate themselves
        noise = np.zeros((n, az.AZ_MAX_LEGAL), dtype=np.float32)
        for g in range(n):
            trees[g].run(0)
            k = len(trees[g].read()["actions"])
            if k:
                noise[g, :k] = rng.dirichlet([0.3] * k).astype(np.float32)
        changed = az.az_search_root_noise(s, noise, 0.25)
        for g in range(n):
            assert changed[g] == trees[g].root_noise(noise[g], 0.25)
        az.az_search_run(s, 50)
        for g in range(n):
            trees[g].run(50)
            same_tree(read_gpu_tree(az, s, g), trees[g].read(), f"move {move} game {g}")
        played = az.az_search_advance(s)
        for g in range(n):
            if played[g] >= 0:
                trees[g].advance(int(played[g]))
    with pytest.raises(az.AzError) as e:
        az.az_search_root_noise(s, np.zeros((n, az.AZ_MAX_LEGAL), dtype=np.float32), 1.5)
    assert e.value.code == az.AZ_ERR_BAD_ARG
    az.az_search_destroy(s)
    for t in trees:
        t.close()


def test_run_in_two_halves():
    import paper_2609_37447_b200 as az
    rec = records(2, 128, 16, 20261020)
    cfg = az.make_search_config(16, 2, 128, leaves=2, groups=2, max_nodes=500, evaluator=az.AZ_SEARCH_EVAL_STANDIN, seed=5)
    a, b = az.az_search_create(None, cfg), az.az_search_create(None, cfg)
    for s in (a, b):
        az.az_search_set_roots(s, rec)
    az.az_search_run(a, 200)
    az.az_search_run_async(b, 200)
    for call in (lambda: az.az_search_root(b, 0), lambda: az.az_search_advance(b), lambda: az.az_search_run_async(b, 1),
                 lambda: az.az_search_set_roots(b, rec), lambda: az.az_search_tree(b, 0)):
        with pytest.raises(az.AzError) as e:
            call()
        assert e.value.code == az.AZ_ERR_BUSY
    assert az.az_search_wait(b) > 0
    with pytest.raises(az.AzError) as e:
        az.az_search_wait(b)
    assert e.value.code == az.AZ_ERR_BAD_ARG
    for g in range(16):
        x, y = read_gpu_tree(az, a, g), read_gpu_tree(az, b, g)
        assert all(np.atleast_1d(u).tobytes() == np.atleast_1d(v).tobytes() for u, v in zip(x, y))
    az.az_search_run_async(b, 50)                     # destroying a search with a run pending waits for it
    az.az_search_destroy(b)
    az.az_search_destroy(a)


def test_bad_arguments():
    import paper_2609_37447_b200 as az
    # az_apply_moves: empty batches are no-ops, in == out and unknown strides or lists are refused
    rec = records(2, 128, 9, 20261050)
    pos = az.records_to_device(rec)
    out = torch.zeros_like(pos)
    act = torch.zeros(9, dtype=torch.int32, device="cuda")
    az.az_apply_moves(pos, 128, 0, 2, act, out)
    for args in ((pos, 128, 9, 2, act, pos), (pos, 120, 9, 2, act, out), (pos, 128, 9, 3, act, out), (pos, 128, -1, 2, act, out)):
        with pytest.raises(az.AzError) as e:
            az.az_apply_moves(*args)
        assert e.value.code == az.AZ_ERR_BAD_ARG
    masks = torch.zeros((9, 30), dtype=torch.int64, device="cuda")
    legal = torch.zeros((9, az.AZ_MAX_LEGAL), device="cuda")
    counts = torch.zeros(9, dtype=torch.int32, device="cuda")
    value = torch.zeros(9, device="cuda")
    az.az_standin_evaluate(pos, 128, masks, 0, 2, 1, legal, counts, value)
    with pytest.raises(az.AzError) as e:
        az.az_standin_evaluate(pos, 100, masks, 9, 2, 1, legal, counts, value)
    assert e.value.code == az.AZ_ERR_BAD_ARG
    # an all-zero mask row is a position without moves: count 0, the value still comes
    az.az_standin_evaluate(pos, 128, masks, 9, 2, 1, legal, counts, value)
    torch.cuda.synchronize()
    assert (counts.cpu().numpy() == 0).all() and (value.cpu().numpy() != 0).any()
    for kw in ({"leaves": 17}, {"groups": 3}, {"max_nodes": 1}):
        with pytest.raises(az.AzError) as e:
            az.az_search_create(None, az.make_search_config(4, 2, 128, evaluator=az.AZ_SEARCH_EVAL_STANDIN, **kw))
        assert e.value.code == az.AZ_ERR_BAD_ARG
    with pytest.raises(az.AzError) as e:
        az.az_search_create(None, az.make_search_config(4, 2, 128))       # a network evaluator needs a network
    assert e.value.code == az.AZ_ERR_BAD_ARG
    with pytest.raises(az.AzError) as e:
        az.az_search_create(None, az.make_search_config(4, 2, 100, evaluator=az.AZ_SEARCH_EVAL_STANDIN))
    assert e.value.code == az.AZ_ERR_BAD_ARG
    cfg = pw.PNetConfig("tb", 0, 128, 8, 20260998, 4501)
    net = az.az_load_net(az.make_arch(52, 0, 128, 2, 1, cfg.precision, 8), pw.make_blob(cfg, 0.1, 0.6))
    with pytest.raises(az.AzError) as e:
        az.az_search_create(net, az.make_search_config(20, 2, 128, groups=2))    # 10 rows per step, the net takes 8
    assert e.value.code == az.AZ_ERR_BATCH_TOO_LARGE
    with pytest.raises(az.AzError) as e:
        az.az_search_create(net, az.make_search_config(4, 1, 104))               # the net's action list is the 1,880 one
    assert e.value.code == az.AZ_ERR_BAD_ARCH
    az.az_free_net(net)
