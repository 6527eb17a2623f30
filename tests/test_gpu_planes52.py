"""The CUDA 52-plane encoder (App. D.1, Table D.1) against the oracle's: bit-exact, both output types,
on generated positions, hand-built ones, an empty batch and a ragged size."""
import numpy as np
import pytest
import torch

import oracle
from inputs import pnet_weights, positions

pytestmark = pytest.mark.gpu


def gpu_planes(az, rec, dtype):
    n = rec.shape[0]
    pos = az.records_to_device(rec)
    out = torch.full((n, 64, 64), -3.0, dtype=dtype, device="cuda")
    az.az_encode52(pos, n, out)
    torch.cuda.synchronize()
    return out.float().cpu().numpy()


@pytest.mark.parametrize("dtype", [torch.float32, torch.bfloat16])
def test_encoding52_is_bit_exact(dtype):
    import paper_2609_37447_b200 as az
    rec, _ = positions.generate_moves(20260960, 4099, (0, 200))      # several blocks and a ragged tail
    got = gpu_planes(az, rec, dtype)
    want = oracle.encode52(rec).reshape(-1, 52, 64).transpose(0, 2, 1)   # [n][square][channel]
    assert (got[:, :, :52] == want).all()
    assert (got[:, :, 52:] == 0).all()
    # the sample exercises every plane that can be non-zero (the king balance never is; repetitions are
    # rare in random play and covered by the hand-built records below)
    seen = np.abs(want.reshape(-1, 52)).max(axis=0) > 0
    assert seen[[c for c in range(52) if c not in (20, 21, 45)]].all()


def test_encoding52_hand_built_and_degenerate_sizes():
    import paper_2609_37447_b200 as az
    rec = np.zeros(3, dtype=positions.M8_DTYPE)
    rec["cur"][0] = positions.record_from_fen("rnbqkbnr/pppppppp/8/8/4P3/8/PPPP1PPP/RNBQKBNR b KQkq e3 0 1")[0]
    rec["n_moves"][0] = 1
    rec["move_from"][0, 0], rec["move_to"][0, 0] = 12, 28
    rec["cur"][1] = positions.record_from_fen("3bk3/8/8/8/2B4q/5n2/8/5RK1 w - - 137 30")[0]
    rec["cur"][1]["repetitions"] = 2
    rec["cur"][2] = positions.record_from_fen("4k3/8/8/8/8/8/4q3/4K3 w - - 0 1")[0]      # queen gives check from e2
    got = gpu_planes(az, rec, torch.float32)
    want = oracle.encode52(rec).reshape(-1, 52, 64).transpose(0, 2, 1)
    assert (got[:, :, :52] == want).all()
    assert got[2, 12, 18] == 1 and got[1, 0, 20] == 1 and got[1, 0, 21] == 1
    # an empty batch is a no-op; null pointers with a non-empty batch are refused
    az.az_encode52(az.records_to_device(rec), 0, torch.zeros((1, 64, 64), device="cuda"))
    with pytest.raises(az.AzError) as e:
        az._check(az._lib.az_encode52(None, 1, 0, None, None), "az_encode52")
    assert e.value.code == az.AZ_ERR_BAD_ARG


def test_encoder52_fused_into_the_tower_kernel_is_bit_exact():
    # Inside az_evaluate the 52 planes are written by the tower kernel's epilogue warps straight into the
    # shared-memory frame, not by the stand-alone encoder.  A network of the paper's kind without blocks
    # whose input convolution passes plane c to channel c as +x/32 and to channel 64 + c as -x/32
    # (centre tap, scale one, bias zero) shows them: the activation keeps max(., 0) of each (and 100/32
    # stays under its cap of six), x = 32 * (channel c - channel 64 + c), every value exact in bf16.
    import paper_2609_37447_b200 as az
    n = 1301                                                               # more than two rounds, a lone last board
    cfg = pnet_weights.PNetConfig("pid", 0, 128, n, 20260965, 77)
    t = pnet_weights.draw_tensors(cfg, 1.0, 1.0)
    w = np.zeros((128, 52, 3, 3), dtype=np.float32)
    w[np.arange(52), np.arange(52), 1, 1] = 1.0 / 32
    w[64 + np.arange(52), np.arange(52), 1, 1] = -1.0 / 32
    t["in.w"], t["in.scale"], t["in.bias"] = w, np.ones(128, np.float32), np.zeros(128, np.float32)
    net = az.az_load_net(az.make_arch(52, 0, 128, 2, 1, 1, n), pnet_weights.pack_blob(cfg, t))
    rec, _ = positions.generate_moves(20260966, n, (0, 200))
    tower = torch.full((n, 64, 128), 9.0, dtype=torch.bfloat16, device="cuda")
    az.az_tower(net, az.records_to_device(rec), n, tower)
    torch.cuda.synchronize()
    got = tower.float().cpu().numpy()
    want = oracle.encode52(rec).reshape(-1, 52, 64).transpose(0, 2, 1)   # [n][square][channel]
    assert (32.0 * (got[:, :, :52] - got[:, :, 64:116]) == want).all()
    assert (got[:, :, 52:64] == 0).all() and (got[:, :, 116:] == 0).all()
    assert az.az_device_status(net) == 0
    az.az_free_net(net)
