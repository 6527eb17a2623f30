"""az_tower_static, the entry point for callers that cannot allocate device memory (a plugin in a
host application that owns the device's memory pool, a real-time serving thread that must not
enter the allocator): it keeps its plane scratch in a fixed array inside the library.  It has to
give exactly what az_tower gives, call after call, although every call reuses the same scratch.

Collected last on purpose (file name), and written to pass both on its own in a fresh process and
after the rest of the GPU suite.
"""
import numpy as np
import pytest
import torch

import oracle
from inputs import configs, positions, weights

pytestmark = pytest.mark.gpu


def test_static_scratch_tower_matches_az_tower_on_two_calls_in_a_row():
    import paper_2609_37447_b200 as az
    cfg = configs.tiny_config(blocks=2, channels=128, precision=1, batch=256, weight_seed=321)
    blob = weights.make_blob(cfg, 1.0, 1.0)
    arch = az.make_arch(cfg.in_planes, cfg.blocks, cfg.channels, cfg.policy_head, cfg.value_head, cfg.precision, 300)
    net = az.az_load_net(arch, blob)
    rec, _ = positions.generate(8086, 300, (0, 120))
    cur = positions.cur_records(rec)
    calls = [(cur[:200], 200), (cur[200:237], 37)]          # a larger batch first, then a ragged smaller one
    for recs, n in calls:
        pos = az.records_to_device(recs)
        want = torch.full((n, 64, 128), 7.0, dtype=torch.bfloat16, device="cuda")
        got = torch.full((n, 64, 128), -7.0, dtype=torch.bfloat16, device="cuda")
        az.az_tower(net, pos, n, want)
        az.az_tower_static(net, pos, n, got)
        torch.cuda.synchronize()
        a, b = want.float().cpu().numpy(), got.float().cpu().numpy()
        assert np.isfinite(b).all()
        # same kernels, same inputs: identical bits expected; the bound is the suite's bf16 bar
        assert np.abs(a - b).max() <= 2e-2 * max(1.0, np.abs(a).max())
        assert (a == b).all()
        # and not merely equal to each other: rows spread over the call against the CPU oracle's tower
        rows = np.unique(np.array([0, 1, n // 2, n - 2, n - 1]))
        ref = oracle.evaluate(blob, recs[rows], 19, cfg.policy_head, want_tower=True)[4]["tower"]    # [rows][C][8][8]
        mine = b[rows].transpose(0, 2, 1).reshape(len(rows), 128, 8, 8)
        assert np.abs(mine - ref).max() <= 2e-2 * 3 ** 0.5 * np.abs(ref).max()
    assert az.az_device_status(net) == 0
    # beyond the fixed scratch the call refuses instead of overrunning it
    pos = az.records_to_device(cur[:257])
    out = torch.zeros((257, 64, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(az.AzError) as e:
        az.az_tower_static(net, pos, 257, out)
    assert e.value.code == az.AZ_ERR_BATCH_TOO_LARGE
    # a caller that has switched to another GPU since az_load_net is refused: that GPU's copy of the array is not
    # the one this network's kernels can use (needs a second GPU; a one-GPU machine has no other device to switch to)
    if torch.cuda.device_count() > 1:
        with torch.cuda.device(1):
            with pytest.raises(az.AzError) as e:
                az.az_tower_static(net, az.records_to_device(cur[:4]), 4, out)
        assert e.value.code == az.AZ_ERR_BAD_ARG
    az.az_free_net(net)
    # the 8-bit towers are refused whether calibrated or not: this entry point is the bf16 tower's
    cfg8 = configs.tiny_config(blocks=1, channels=128, precision=2, batch=16, weight_seed=322)
    net8 = az.az_load_net(az.make_arch(19, 1, 128, 0, 0, 2, 16), weights.make_blob(cfg8, 1.0, 1.0))
    pos8 = az.records_to_device(cur[:16])
    out8 = torch.zeros((16, 64, 128), dtype=torch.bfloat16, device="cuda")
    for calibrated in (False, True):
        if calibrated:
            az.az_calibrate(net8, pos8, 16)
        with pytest.raises(az.AzError) as e:
            az.az_tower_static(net8, pos8, 16, out8)
        assert e.value.code == az.AZ_ERR_UNSUPPORTED
    az.az_free_net(net8)
    # networks without the tensor-core tower are refused, not silently routed elsewhere
    cfg32 = configs.tiny_config(blocks=1, channels=32, precision=0, batch=4)
    net32 = az.az_load_net(az.make_arch(19, 1, 32, 0, 0, 0, 4), weights.make_blob(cfg32))
    with pytest.raises(az.AzError) as e:
        az.az_tower_static(net32, az.records_to_device(cur[:4]), 4, torch.zeros((4, 64, 32), device="cuda"))
    assert e.value.code == az.AZ_ERR_UNSUPPORTED
    az.az_free_net(net32)
