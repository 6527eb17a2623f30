"""Runtime behaviour of the library on the GPU: host-buffer entry point, CUDA-graph replay, event
timing of the tower, and the failure path of the bounded device-side waits (made to run out on a
barrier nothing arrives on; nothing hangs, the context stays usable)."""
import numpy as np
import pytest
import torch

from inputs import configs, positions, weights

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def setup():
    import paper_2609_37447_b200 as az
    cfg = configs.tiny_config(blocks=3, channels=128, policy_head=1, value_head=1, precision=1, batch=96, weight_seed=77)
    blob = weights.make_blob(cfg, 0.02, 0.05)
    net = az.az_load_net(az.make_arch(19, 3, 128, 1, 1, 1, 128), blob)
    recs = positions.cur_records(positions.generate(4711, 96, (0, 100))[0])
    pos = az.records_to_device(recs)
    masks = torch.zeros((96, 30), dtype=torch.int64, device="cuda")
    az.az_legal_masks(pos, 104, 96, 1, masks)
    policy = torch.zeros((96, 1858), device="cuda")
    value = torch.zeros((96, 3), device="cuda")
    az.az_evaluate(net, pos, masks, 96, policy, value)
    torch.cuda.synchronize()
    yield az, net, recs, pos, masks, policy.clone(), value.clone()
    az.az_free_net(net)


def test_host_buffer_entry_point_gives_the_same_results(setup):
    az, net, recs, pos, masks, policy, value = setup
    pos_h = torch.from_numpy(np.ascontiguousarray(recs).view(np.uint8).reshape(96, -1).copy()).pin_memory()
    masks_h = masks.cpu().pin_memory()
    pol_h = torch.full((96, 1858), -1.0).pin_memory()
    val_h = torch.full((96, 3), -1.0).pin_memory()
    az.az_evaluate_host(net, pos_h, masks_h, 96, pol_h, val_h)          # returns after the results landed
    assert torch.equal(pol_h, policy.cpu()) and torch.equal(val_h, value.cpu())
    # pageable numpy buffers work too
    pol_n, val_n = np.zeros((96, 1858), np.float32), np.zeros((96, 3), np.float32)
    az.az_evaluate_host(net, pos_h.numpy(), masks_h.numpy(), 96, pol_n, val_n)
    assert (pol_n == policy.cpu().numpy()).all() and (val_n == value.cpu().numpy()).all()


def test_pipelined_host_entry_matches_and_bounds_its_queue(setup):
    az, net, recs, pos, masks, policy, value = setup
    pos_h = torch.from_numpy(np.ascontiguousarray(recs).view(np.uint8).reshape(96, -1).copy()).pin_memory()
    masks_h = masks.cpu().pin_memory()
    # six batches of different sizes through two slots; every result must equal the synchronous one
    sizes = [96, 17, 64, 96, 1, 50]
    outs = [(torch.full((96, 1858), -1.0).pin_memory(), torch.full((96, 3), -1.0).pin_memory()) for _ in sizes]
    tickets = []
    for i, n in enumerate(sizes):
        if len(tickets) == az.AZ_HOST_SLOTS:
            az.az_wait_host(net, tickets.pop(0))
        tickets.append(az.az_submit_host(net, pos_h, masks_h, n, outs[i][0], None, None, outs[i][1]))
    for t in tickets:
        az.az_wait_host(net, t)
    for (pol_h, val_h), n in zip(outs, sizes):
        assert torch.equal(pol_h[:n], policy.cpu()[:n]) and torch.equal(val_h[:n], value.cpu()[:n])
        assert (pol_h[n:] == -1.0).all()
    # legal-moves-only output through the same queue
    legal_ref = torch.zeros((96, az.AZ_MAX_LEGAL), device="cuda")
    counts_ref = torch.zeros((96,), dtype=torch.int32, device="cuda")
    az.az_evaluate_legal(net, pos, masks, 96, legal_ref, counts_ref, torch.zeros_like(value))
    torch.cuda.synchronize()
    legal_h = torch.zeros((96, az.AZ_MAX_LEGAL)).pin_memory()
    counts_h = torch.zeros((96,), dtype=torch.int32).pin_memory()
    val_h = torch.zeros((96, 3)).pin_memory()
    az.az_wait_host(net, az.az_submit_host(net, pos_h, masks_h, 96, None, legal_h, counts_h, val_h))
    assert torch.equal(counts_h, counts_ref.cpu()) and torch.equal(val_h, value.cpu())
    for b in range(96):
        assert torch.equal(legal_h[b, :counts_h[b]], legal_ref.cpu()[b, :counts_h[b]])
    # a third submission while two are in flight is refused and queues nothing; a stale ticket is an error
    t0 = az.az_submit_host(net, pos_h, masks_h, 96, outs[0][0], None, None, outs[0][1])
    t1 = az.az_submit_host(net, pos_h, masks_h, 96, outs[1][0], None, None, outs[1][1])
    with pytest.raises(az.AzError) as err:
        az.az_submit_host(net, pos_h, masks_h, 96, outs[2][0], None, None, outs[2][1])
    assert err.value.code == az.AZ_ERR_BUSY
    az.az_wait_host(net, t0)
    az.az_wait_host(net, t1)
    with pytest.raises(az.AzError) as err:
        az.az_wait_host(net, t0)
    assert err.value.code == az.AZ_ERR_BAD_ARG
    assert az.az_device_status(net) == 0


def test_legal_moves_only_output_matches_the_dense_policy(setup):
    az, net, recs, pos, masks, policy, value = setup
    legal = torch.full((96, az.AZ_MAX_LEGAL), -1.0, device="cuda")
    counts = torch.full((96,), -1, dtype=torch.int32, device="cuda")
    val = torch.zeros_like(value)
    az.az_evaluate_legal(net, pos, masks, 96, legal, counts, val)
    torch.cuda.synchronize()
    dense = policy.cpu().numpy()
    bits = np.unpackbits(az.masks_to_numpy(masks).view(np.uint8), axis=1, bitorder="little")[:, :1858].astype(bool)
    lg, cn = legal.cpu().numpy(), counts.cpu().numpy()
    assert torch.equal(val, value)
    for b in range(96):
        idx = np.flatnonzero(bits[b])                      # ascending policy index = order of the mask's set bits
        assert cn[b] == idx.size
        assert np.abs(lg[b, :idx.size] - dense[b, idx]).max() < 1e-6
        assert (lg[b, idx.size:] == -1.0).all()              # entries beyond the count are left alone
    # host-buffer form
    pos_h = torch.from_numpy(np.ascontiguousarray(recs).view(np.uint8).reshape(96, -1).copy()).pin_memory()
    lg_h = torch.zeros((96, az.AZ_MAX_LEGAL)).pin_memory()
    cn_h = torch.zeros((96,), dtype=torch.int32).pin_memory()
    val_h = torch.zeros((96, 3)).pin_memory()
    az.az_evaluate_legal_host(net, pos_h, masks.cpu().pin_memory(), 96, lg_h, cn_h, val_h)
    assert torch.equal(cn_h, counts.cpu()) and torch.equal(val_h, value.cpu())
    for b in range(96):
        assert torch.equal(lg_h[b, :cn[b]], legal[b, :cn[b]].cpu())


def test_evaluation_replays_from_a_cuda_graph(setup):
    az, net, recs, pos, masks, policy, value = setup
    pol_g = torch.zeros_like(policy)
    val_g = torch.zeros_like(value)
    stream = torch.cuda.Stream()
    with torch.cuda.stream(stream):
        az.az_evaluate(net, pos, masks, 96, pol_g, val_g, stream)       # first call outside the capture
        stream.synchronize()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph, stream=stream):
            az.az_evaluate(net, pos, masks, 96, pol_g, val_g, torch.cuda.current_stream())
        pol_g.zero_()
        val_g.zero_()
        for _ in range(3):
            graph.replay()
        stream.synchronize()
    assert torch.equal(pol_g, policy) and torch.equal(val_g, value)


def test_tower_event_timing_counts_passes(setup):
    az, net, recs, pos, masks, policy, value = setup
    pol = torch.zeros_like(policy)
    val = torch.zeros_like(value)
    az.az_profile_tower(net, True)
    az.az_tower_time(net)
    for _ in range(5):
        az.az_evaluate(net, pos, masks, 96, pol, val)
    ms, passes = az.az_tower_time(net)
    az.az_profile_tower(net, False)
    assert passes == 5 and 0.0 < ms < 50.0
    az.az_evaluate(net, pos, masks, 96, pol, val)
    assert az.az_tower_time(net) == (0.0, 0)
    assert az.az_launches_per_evaluate(net, 96) == 3
    # every third evaluation only (the third, sixth, ... after the call): 7 evaluations, 2 timed; results unchanged
    az.az_profile_tower(net, True, every=3)
    for _ in range(7):
        az.az_evaluate(net, pos, masks, 96, pol, val)
    ms, passes = az.az_tower_time(net)
    az.az_profile_tower(net, False)
    assert passes == 2 and 0.0 < ms < 50.0
    torch.cuda.synchronize()
    assert torch.equal(pol, policy) and torch.equal(val, value)
    with pytest.raises(az.AzError):
        az.az_profile_tower(net, True, every=-2)


def test_a_wait_that_runs_out_is_reported_and_leaves_the_context_usable(setup):
    az, net, recs, pos, masks, policy, value = setup
    assert az.az_selftest_wait_timeout() == az.AZ_ERR_DEVICE_TIMEOUT
    assert az.az_selftest_wait_timeout() == az.AZ_ERR_DEVICE_TIMEOUT   # repeatable
    pol = torch.zeros_like(policy)
    val = torch.zeros_like(value)
    az.az_evaluate(net, pos, masks, 96, pol, val)                      # the device still works
    torch.cuda.synchronize()
    assert torch.equal(pol, policy) and torch.equal(val, value)
    assert az.az_device_status(net) == 0
