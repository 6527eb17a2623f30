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
    assert az.az_device_status(net) == 0
    # beyond the fixed scratch the call refuses instead of overrunning it
    pos = az.records_to_device(cur[:257])
    out = torch.zeros((257, 64, 128), dtype=torch.bfloat16, device="cuda")
    with pytest.raises(az.AzError) as e:
        az.az_tower_static(net, pos, 257, out)
    assert e.value.code == az.AZ_ERR_BATCH_TOO_LARGE
    az.az_free_net(net)
    # networks without the tensor-core tower are refused, not silently routed elsewhere
    cfg32 = configs.tiny_config(blocks=1, channels=32, precision=0, batch=4)
    net32 = az.az_load_net(az.make_arch(19, 1, 32, 0, 0, 0, 4), weights.make_blob(cfg32))
    with pytest.raises(az.AzError) as e:
        az.az_tower_static(net32, az.records_to_device(cur[:4]), 4, torch.zeros((4, 64, 32), device="cuda"))
    assert e.value.code == az.AZ_ERR_UNSUPPORTED
    az.az_free_net(net32)
