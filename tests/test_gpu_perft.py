"""Perft on the GPU: the tree of legal moves is walked with az_legal_masks (children of a position = the set
bits of its mask) and az_apply_moves (the successor under each action), and the leaf counts are compared with
the published counts of tests/golden/perft.txt -- facts of chess, independent of the oracle.  Exercises
castling (also through attacked squares), en passant (also the discovered-check case), promotions and
under-promotions, pins and double checks in both kernels, through both from-to action lists and the 73 planes."""
import os

import numpy as np
import pytest
import torch

from inputs import positions

pytestmark = pytest.mark.gpu
SIZE = {0: 4672, 1: 1858, 2: 1880}
WORDS = {0: 73, 1: 30, 2: 30}
CHUNK = 1 << 17


def perft_cases(golden_dir):
    with open(os.path.join(golden_dir, "perft.txt")) as f:
        for line in f:
            if line.strip() and not line.startswith("#"):
                fen, counts = line.split("|")
                yield fen.strip(), [int(c) for c in counts.split()]


def children(az, pos, head):
    """All successors of the positions in `pos` ([n][104] uint8 on the GPU), in chunks."""
    out = []
    shifts = torch.arange(64, device="cuda", dtype=torch.int64)
    for lo in range(0, pos.shape[0], CHUNK):
        part = pos[lo:lo + CHUNK].contiguous()
        n = part.shape[0]
        masks = torch.zeros((n, WORDS[head]), dtype=torch.int64, device="cuda")
        az.az_legal_masks(part, 104, n, head, masks)
        bits = ((masks.unsqueeze(2) >> shifts) & 1).bool().reshape(n, -1)[:, :SIZE[head]]
        parent, action = torch.nonzero(bits, as_tuple=True)
        if parent.numel() == 0:
            continue
        src = part[parent].contiguous()
        dst = torch.empty_like(src)
        status = torch.zeros(1, dtype=torch.int32, device="cuda")
        az.az_apply_moves(src, 104, src.shape[0], head, action.to(torch.int32).contiguous(), dst, status)
        assert int(status.item()) == 0
        out.append(dst)
    return torch.cat(out) if out else pos[:0]


def leaf_count(az, pos, head):
    total = 0
    for lo in range(0, pos.shape[0], CHUNK):
        part = pos[lo:lo + CHUNK].contiguous()
        masks = torch.zeros((part.shape[0], WORDS[head]), dtype=torch.int64, device="cuda")
        az.az_legal_masks(part, 104, part.shape[0], head, masks)
        m = masks.view(torch.uint8)                           # population count; bits above a list's size are never set
        total += sum(int(((m >> k) & 1).sum()) for k in range(8))
    return total


@pytest.mark.parametrize("head", [1, 2, 0])
def test_gpu_perft_reproduces_the_published_counts(golden_dir, head):
    import paper_2609_37447_b200 as az
    for fen, counts in perft_cases(golden_dir):
        level = az.records_to_device(positions.record_from_fen(fen))
        budget = 5_000_000 if head != 0 else 500_000          # the 73-plane masks are 2.4 times as wide
        for depth, want in enumerate(counts, start=1):
            if want > budget:
                break
            assert leaf_count(az, level, head) == want, (fen, depth)
            if depth < len(counts) and counts[depth] <= budget:
                level = children(az, level, head)
                assert level.shape[0] == want, (fen, depth)
