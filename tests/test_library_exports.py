"""The C-ABI library loads without a GPU and exports every function the headers under include/ declare."""
import ctypes
import glob
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def declared_functions():
    names = set()
    for header in sorted(glob.glob(os.path.join(ROOT, "include", "*.h"))):
        with open(header) as f:
            text = re.sub(r"/\*.*?\*/", "", f.read(), flags=re.S)
        names |= set(re.findall(r"\b(az_[a-z0-9_]+)\s*\(", text))
    return sorted(names)


@pytest.fixture(scope="module")
def lib():
    import __graft_entry__
    return ctypes.CDLL(__graft_entry__.load_build_module().build())


def test_every_declared_entry_point_is_exported(lib):
    names = declared_functions()
    assert {"az_load_net", "az_evaluate", "az_encode", "az_legal_masks", "az_free_net", "az_search_run", "az_apply_moves"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name


def test_binding_lists_the_same_names():
    import paper_2609_37447_b200 as az
    assert sorted(az.EXPORTS) == declared_functions()
    for name in az.EXPORTS:
        assert callable(getattr(az, name))


def test_host_only_helpers(lib):
    import paper_2609_37447_b200 as az
    arch = az.make_arch(19, 20, 128, 1, 1, 1, 1024)
    assert (az.az_position_bytes(arch), az.az_policy_size(arch), az.az_mask_words(arch),
            az.az_value_size(arch), az.az_plane_channels(arch)) == (104, 1858, 30, 3, 32)
    arch = az.make_arch(112, 40, 256, 0, 0, 1, 16)
    assert (az.az_position_bytes(arch), az.az_policy_size(arch), az.az_mask_words(arch),
            az.az_value_size(arch), az.az_plane_channels(arch)) == (784, 4672, 73, 1, 128)
    assert az.az_strerror(0) == "ok" and "batch" in az.az_strerror(az.AZ_ERR_BATCH_TOO_LARGE)
    # argument errors are reported before any CUDA call
    with pytest.raises(az.AzError) as e:
        az.az_load_net(az.make_arch(19, 1, 30, 0, 0, 0, 4), b"\0" * 128)
    assert e.value.code == az.AZ_ERR_BAD_ARCH
    with pytest.raises(az.AzError) as e:
        az.az_load_net(az.make_arch(19, 1, 32, 0, 0, 0, 4), b"\0" * 128)
    assert e.value.code == az.AZ_ERR_BAD_WEIGHTS


def test_search_arguments_are_checked_before_any_cuda_call(lib):
    import paper_2609_37447_b200 as az
    for kw in ({"leaves": 0}, {"leaves": 17}, {"groups": 0}, {"groups": 3}, {"max_nodes": 1}, {"c_puct": -1.0}, {"discount": 0.0}):
        with pytest.raises(az.AzError) as e:
            az.az_search_create(None, az.make_search_config(4, 2, 128, evaluator=az.AZ_SEARCH_EVAL_STANDIN, **kw))
        assert e.value.code == az.AZ_ERR_BAD_ARG, kw
    with pytest.raises(az.AzError) as e:
        az.az_search_create(None, az.make_search_config(4, 2, 128))           # the network evaluator needs a network
    assert e.value.code == az.AZ_ERR_BAD_ARG
    with pytest.raises(az.AzError) as e:
        az.az_search_create(None, az.make_search_config(4, 3, 128, evaluator=az.AZ_SEARCH_EVAL_STANDIN))   # no such action list
    assert e.value.code == az.AZ_ERR_BAD_ARG
    cfg = az.make_search_config(4, 2, 128)
    assert (cfg.c_puct, cfg.fpu_reduction, cfg.discount) == (1.5, pytest.approx(0.2), pytest.approx(0.99))   # App. D.2
