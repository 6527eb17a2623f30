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
