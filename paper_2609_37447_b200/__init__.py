"""Python binding of the az_eval C library (argument marshalling only).

Every function has the name and meaning of the C entry point declared in include/az_eval.h; all
computation happens in the library's CUDA kernels.  PyTorch supplies device memory and streams.
There is no fallback: if libazeval.so is missing or fails to load, importing raises.
"""
import ctypes
import os
from dataclasses import dataclass

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.environ.get("AZ_EVAL_LIB") or os.path.join(_HERE, "libazeval.so")

AZ_ABI_VERSION = 1
AZ_OK = 0
AZ_ERR_BAD_ARG, AZ_ERR_BAD_ARCH, AZ_ERR_BAD_WEIGHTS, AZ_ERR_BATCH_TOO_LARGE = -1, -2, -3, -4
AZ_ERR_CUDA, AZ_ERR_DEVICE_TIMEOUT, AZ_ERR_NOT_CALIBRATED, AZ_ERR_UNSUPPORTED, AZ_ERR_BUSY = -5, -6, -7, -8, -9
AZ_HOST_SLOTS = 2
AZ_POLICY_PLANES73, AZ_POLICY_FLAT1858, AZ_POLICY_FROMTO1880 = 0, 1, 2
AZ_VALUE_TANH, AZ_VALUE_WDL = 0, 1
AZ_PREC_FP32, AZ_PREC_BF16, AZ_PREC_FP8_E4M3, AZ_PREC_INT8, AZ_PREC_FP8_E4M3_X2, AZ_PREC_FP8_E4M3_X2A = 0, 1, 2, 3, 4, 5

EXPORTS = ("az_position_bytes", "az_policy_size", "az_mask_words", "az_value_size", "az_plane_channels",
           "az_load_net", "az_load_net_ex", "az_free_net", "az_evaluate", "az_evaluate_legal", "az_evaluate_legal_host", "az_evaluate_host", "az_submit_host", "az_wait_host", "az_encode", "az_encode52", "az_tower", "az_tower_static", "az_legal_masks",
           "az_calibrate", "az_calibrate_ex", "az_device_status", "az_profile_tower", "az_tower_time", "az_selftest_wait_timeout", "az_launches_per_evaluate", "az_strerror",
           "az_last_cuda_error",
           "az_apply_moves", "az_standin_evaluate", "az_search_create", "az_search_destroy", "az_search_set_roots", "az_search_replace_roots",
           "az_search_run", "az_search_run_async", "az_search_wait", "az_search_root", "az_search_root_visits", "az_search_advance", "az_search_root_noise", "az_search_root_positions", "az_search_tree", "az_search_launches_per_step")


class az_arch(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint32) for n in ("abi_version", "in_planes", "blocks", "channels",
                                               "policy_head", "value_head", "precision", "max_batch")]


class az_search_config(ctypes.Structure):
    _fields_ = [(n, ctypes.c_uint32) for n in ("games", "leaves", "groups", "max_nodes", "max_edges", "evaluator",
                                               "policy_head", "position_bytes")] + \
               [("c_puct", ctypes.c_float), ("fpu_reduction", ctypes.c_float), ("discount", ctypes.c_float),
                ("reserved", ctypes.c_uint32), ("seed", ctypes.c_uint64)]


AZ_SEARCH_EVAL_NET, AZ_SEARCH_EVAL_STANDIN = 0, 1
AZ_SEARCH_MAX_LEAVES, AZ_SEARCH_MAX_DEPTH = 16, 128
AZ_SEARCH_FLAG_NODES_FULL, AZ_SEARCH_FLAG_EDGES_FULL, AZ_SEARCH_FLAG_DEPTH, AZ_SEARCH_FLAG_BAD_ACTION = 1, 2, 4, 8


class AzError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        detail = _lib.az_last_cuda_error().decode() if code == AZ_ERR_CUDA else ""
        super().__init__(f"{where}: {_lib.az_strerror(code).decode()} ({code}) {detail}".strip())


def _load_library():
    if not os.path.exists(LIB_PATH):
        raise ImportError(f"{LIB_PATH} is missing: build it with `python -m paper_2609_37447_b200.build` "
                          "(there is no CPU fallback)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    ap = ctypes.POINTER(az_arch)
    for name in ("az_position_bytes", "az_policy_size", "az_mask_words", "az_value_size", "az_plane_channels"):
        getattr(lib, name).restype = sz
        getattr(lib, name).argtypes = [ap]
    lib.az_load_net.restype = ci
    lib.az_load_net.argtypes = [ap, vp, sz, ctypes.POINTER(vp)]
    lib.az_load_net_ex.restype = ci
    lib.az_load_net_ex.argtypes = [ap, vp, sz, ctypes.c_uint32, ctypes.POINTER(vp)]
    lib.az_free_net.restype = None
    lib.az_free_net.argtypes = [vp]
    lib.az_evaluate.restype = ci
    lib.az_evaluate.argtypes = [vp, vp, vp, ci, vp, vp, vp]
    lib.az_evaluate_legal.restype = ci
    lib.az_evaluate_legal.argtypes = [vp, vp, vp, ci, vp, vp, vp, vp]
    lib.az_evaluate_legal_host.restype = ci
    lib.az_evaluate_legal_host.argtypes = [vp, vp, vp, ci, vp, vp, vp, vp]
    lib.az_evaluate_host.restype = ci
    lib.az_evaluate_host.argtypes = [vp, vp, vp, ci, vp, vp, vp]
    lib.az_submit_host.restype = ci
    lib.az_submit_host.argtypes = [vp, vp, vp, ci, vp, vp, vp, vp, ctypes.POINTER(ci)]
    lib.az_wait_host.restype = ci
    lib.az_wait_host.argtypes = [vp, ci]
    lib.az_profile_tower.restype = ci
    lib.az_profile_tower.argtypes = [vp, ci]
    lib.az_tower_time.restype = ci
    lib.az_tower_time.argtypes = [vp, ctypes.POINTER(ctypes.c_float), ctypes.POINTER(ci)]
    lib.az_encode.restype = ci
    lib.az_encode.argtypes = [vp, vp, ci, vp, vp]
    lib.az_encode52.restype = ci
    lib.az_encode52.argtypes = [vp, ci, ci, vp, vp]
    lib.az_tower.restype = ci
    lib.az_tower.argtypes = [vp, vp, ci, vp, vp]
    lib.az_tower_static.restype = ci
    lib.az_tower_static.argtypes = [vp, vp, ci, vp, vp]
    lib.az_legal_masks.restype = ci
    lib.az_legal_masks.argtypes = [vp, sz, ci, ci, vp, vp]
    lib.az_calibrate.restype = ci
    lib.az_calibrate.argtypes = [vp, vp, ci, vp]
    lib.az_calibrate_ex.restype = ci
    lib.az_calibrate_ex.argtypes = [vp, vp, ci, ctypes.c_uint32, vp]
    lib.az_device_status.restype = ci
    lib.az_device_status.argtypes = [vp, vp, ctypes.POINTER(ctypes.c_uint32)]
    lib.az_selftest_wait_timeout.restype = ci
    lib.az_selftest_wait_timeout.argtypes = [vp]
    lib.az_launches_per_evaluate.restype = ci
    lib.az_launches_per_evaluate.argtypes = [vp, ci]
    lib.az_strerror.restype = ctypes.c_char_p
    lib.az_strerror.argtypes = [ci]
    lib.az_last_cuda_error.restype = ctypes.c_char_p
    lib.az_last_cuda_error.argtypes = []
    lib.az_apply_moves.restype = ci
    lib.az_apply_moves.argtypes = [vp, sz, ci, ci, vp, vp, vp, vp]
    lib.az_standin_evaluate.restype = ci
    lib.az_standin_evaluate.argtypes = [vp, sz, vp, ci, ci, ctypes.c_uint64, vp, vp, vp, vp]
    lib.az_search_create.restype = ci
    lib.az_search_create.argtypes = [vp, ctypes.POINTER(az_search_config), ctypes.POINTER(vp)]
    lib.az_search_destroy.restype = None
    lib.az_search_destroy.argtypes = [vp]
    lib.az_search_set_roots.restype = ci
    lib.az_search_set_roots.argtypes = [vp, vp]
    lib.az_search_replace_roots.restype = ci
    lib.az_search_replace_roots.argtypes = [vp, vp, ci, vp]
    lib.az_search_run.restype = ci
    lib.az_search_run.argtypes = [vp, ci, ctypes.POINTER(ctypes.c_float)]
    lib.az_search_run_async.restype = ci
    lib.az_search_run_async.argtypes = [vp, ci]
    lib.az_search_wait.restype = ci
    lib.az_search_wait.argtypes = [vp, ctypes.POINTER(ctypes.c_float)]
    lib.az_search_root.restype = ci
    lib.az_search_root.argtypes = [vp, ci, vp, vp, vp, vp, ctypes.POINTER(ctypes.c_int32)]
    lib.az_search_root_visits.restype = ci
    lib.az_search_root_visits.argtypes = [vp, vp, vp, vp]
    lib.az_search_advance.restype = ci
    lib.az_search_advance.argtypes = [vp, vp, vp]
    lib.az_search_root_noise.restype = ci
    lib.az_search_root_noise.argtypes = [vp, vp, ctypes.c_float, vp]
    lib.az_search_root_positions.restype = ci
    lib.az_search_root_positions.argtypes = [vp, vp]
    lib.az_search_tree.restype = ci
    lib.az_search_tree.argtypes = [vp, ci, vp, vp, vp]
    lib.az_search_launches_per_step.restype = ci
    lib.az_search_launches_per_step.argtypes = [vp]
    return lib


_lib = _load_library()


def _check(code: int, where: str):
    if code != AZ_OK:
        raise AzError(code, where)


def _stream_ptr(stream) -> int:
    if stream is None:
        stream = torch.cuda.current_stream()
    return int(stream.cuda_stream)


def _dev_ptr(t: torch.Tensor, name: str) -> int:
    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.is_contiguous()):
        raise TypeError(f"{name} must be a contiguous CUDA tensor")
    return t.data_ptr()


def make_arch(in_planes, blocks, channels, policy_head, value_head, precision, max_batch) -> az_arch:
    return az_arch(AZ_ABI_VERSION, in_planes, blocks, channels, policy_head, value_head, precision, max_batch)


def az_position_bytes(arch: az_arch) -> int:
    return int(_lib.az_position_bytes(ctypes.byref(arch)))


def az_policy_size(arch: az_arch) -> int:
    return int(_lib.az_policy_size(ctypes.byref(arch)))


def az_mask_words(arch: az_arch) -> int:
    return int(_lib.az_mask_words(ctypes.byref(arch)))


def az_value_size(arch: az_arch) -> int:
    return int(_lib.az_value_size(ctypes.byref(arch)))


def az_plane_channels(arch: az_arch) -> int:
    return int(_lib.az_plane_channels(ctypes.byref(arch)))


@dataclass
class Net:
    """Handle of a loaded network (owns device weights and workspace; call az_free_net when done)."""
    handle: int
    arch: az_arch

    @property
    def act_dtype(self):
        return torch.float32 if self.arch.precision == AZ_PREC_FP32 else torch.bfloat16


def az_load_net(arch: az_arch, weights_host) -> Net:
    """weights_host: the weight blob as bytes / numpy uint8 array (host memory)."""
    blob = np.ascontiguousarray(np.frombuffer(weights_host, dtype=np.uint8) if isinstance(weights_host, (bytes, bytearray))
                                else weights_host, dtype=np.uint8)
    out = ctypes.c_void_p()
    _check(_lib.az_load_net(ctypes.byref(arch), blob.ctypes.data, blob.nbytes, ctypes.byref(out)), "az_load_net")
    return Net(out.value, arch)


AZ_LOAD_TOWER_CTA_PAIRS = 1
AZ_LOAD_TOWER_SINGLE_CTAS = 2


def az_load_net_ex(arch: az_arch, weights_host, flags=0) -> Net:
    """az_load_net with options (AZ_LOAD_TOWER_CTA_PAIRS: insist on the tower kernel as clusters of two CTAs, the
    default where the shape has that form; AZ_LOAD_TOWER_SINGLE_CTAS: never)."""
    blob = np.ascontiguousarray(np.frombuffer(weights_host, dtype=np.uint8) if isinstance(weights_host, (bytes, bytearray))
                                else weights_host, dtype=np.uint8)
    out = ctypes.c_void_p()
    _check(_lib.az_load_net_ex(ctypes.byref(arch), blob.ctypes.data, blob.nbytes, flags, ctypes.byref(out)), "az_load_net_ex")
    return Net(out.value, arch)


def az_free_net(net: Net):
    if net is not None and net.handle:
        _lib.az_free_net(net.handle)
        net.handle = 0


def az_evaluate(net: Net, positions_dev, legal_masks_dev, batch, policy_dev, value_dev, stream=None):
    """(positions, legal_masks) -> (policy, value), written into the caller's device tensors."""
    _check(_lib.az_evaluate(net.handle, _dev_ptr(positions_dev, "positions"), _dev_ptr(legal_masks_dev, "legal_masks"),
                            batch, _dev_ptr(policy_dev, "policy"), _dev_ptr(value_dev, "value"), _stream_ptr(stream)),
           "az_evaluate")


def _host_ptr(t, name: str) -> int:
    if isinstance(t, torch.Tensor):
        if t.is_cuda or not t.is_contiguous():
            raise TypeError(f"{name} must be a contiguous host tensor")
        return t.data_ptr()
    if isinstance(t, np.ndarray) and t.flags["C_CONTIGUOUS"]:
        return t.ctypes.data
    raise TypeError(f"{name} must be a contiguous host tensor or numpy array")


def az_evaluate_host(net: Net, positions_host, legal_masks_host, batch, policy_host, value_host, stream=None):
    """az_evaluate with host buffers (pinned or pageable); returns after the results have landed."""
    _check(_lib.az_evaluate_host(net.handle, _host_ptr(positions_host, "positions"), _host_ptr(legal_masks_host, "legal_masks"),
                                 batch, _host_ptr(policy_host, "policy"), _host_ptr(value_host, "value"),
                                 _stream_ptr(stream)), "az_evaluate_host")


AZ_MAX_LEGAL = 256


def az_evaluate_legal(net: Net, positions_dev, legal_masks_dev, batch, legal_policy_dev, legal_counts_dev, value_dev, stream=None):
    """az_evaluate with the policy over the legal moves only: [batch][AZ_MAX_LEGAL] float32 + [batch] int32 counts."""
    _check(_lib.az_evaluate_legal(net.handle, _dev_ptr(positions_dev, "positions"), _dev_ptr(legal_masks_dev, "legal_masks"),
                                  batch, _dev_ptr(legal_policy_dev, "legal_policy"), _dev_ptr(legal_counts_dev, "legal_counts"),
                                  _dev_ptr(value_dev, "value"), _stream_ptr(stream)), "az_evaluate_legal")


def az_evaluate_legal_host(net: Net, positions_host, legal_masks_host, batch, legal_policy_host, legal_counts_host, value_host, stream=None):
    _check(_lib.az_evaluate_legal_host(net.handle, _host_ptr(positions_host, "positions"), _host_ptr(legal_masks_host, "legal_masks"),
                                       batch, _host_ptr(legal_policy_host, "legal_policy"), _host_ptr(legal_counts_host, "legal_counts"),
                                       _host_ptr(value_host, "value"), _stream_ptr(stream)), "az_evaluate_legal_host")


def az_submit_host(net: Net, positions_host, legal_masks_host, batch, policy_host, legal_policy_host, legal_counts_host, value_host) -> int:
    """Queues one evaluation on host buffers and returns its ticket (dense output if policy_host is given)."""
    ticket = ctypes.c_int(-1)
    opt = lambda t, name: None if t is None else _host_ptr(t, name)
    _check(_lib.az_submit_host(net.handle, _host_ptr(positions_host, "positions"), _host_ptr(legal_masks_host, "legal_masks"), batch,
                               opt(policy_host, "policy"), opt(legal_policy_host, "legal_policy"), opt(legal_counts_host, "legal_counts"),
                               _host_ptr(value_host, "value"), ctypes.byref(ticket)), "az_submit_host")
    return int(ticket.value)


def az_wait_host(net: Net, ticket: int):
    _check(_lib.az_wait_host(net.handle, ticket), "az_wait_host")


def az_profile_tower(net: Net, enable, every: int = 1):
    """enable False / 0: off; True: every `every`-th evaluation's tower pass is bracketed with events."""
    _check(_lib.az_profile_tower(net.handle, int(every) if enable else 0), "az_profile_tower")


def az_tower_time(net: Net):
    """(summed milliseconds, passes) of the tower since the last read."""
    ms, n = ctypes.c_float(0), ctypes.c_int(0)
    _check(_lib.az_tower_time(net.handle, ctypes.byref(ms), ctypes.byref(n)), "az_tower_time")
    return float(ms.value), int(n.value)


def az_encode(net: Net, positions_dev, batch, planes_dev, stream=None):
    _check(_lib.az_encode(net.handle, _dev_ptr(positions_dev, "positions"), batch, _dev_ptr(planes_dev, "planes"),
                          _stream_ptr(stream)), "az_encode")


def az_encode52(positions_dev, batch, planes_dev, stream=None):
    """128-byte move-history records -> [batch][64][64] planes (float32 or bfloat16 by the tensor's dtype)."""
    bf16 = 1 if planes_dev.dtype == torch.bfloat16 else 0
    if not bf16 and planes_dev.dtype != torch.float32:
        raise TypeError("planes must be float32 or bfloat16")
    _check(_lib.az_encode52(_dev_ptr(positions_dev, "positions"), batch, bf16, _dev_ptr(planes_dev, "planes"),
                            _stream_ptr(stream)), "az_encode52")


def az_tower(net: Net, positions_dev, batch, tower_dev, stream=None):
    _check(_lib.az_tower(net.handle, _dev_ptr(positions_dev, "positions"), batch, _dev_ptr(tower_dev, "tower"),
                         _stream_ptr(stream)), "az_tower")


def az_tower_static(net: Net, positions_dev, batch, tower_dev, stream=None):
    """az_tower without any device allocation: the plane scratch is a fixed array inside the library.

    For callers that may not allocate on the device (a host application that owns all device memory,
    a real-time thread that must stay clear of the allocator).  At most 256 positions per call, bf16
    128-channel networks only; all calls share the one scratch array, so do not overlap them on the GPU.
    """
    _check(_lib.az_tower_static(net.handle, _dev_ptr(positions_dev, "positions"), batch, _dev_ptr(tower_dev, "tower"),
                                _stream_ptr(stream)), "az_tower_static")


def az_legal_masks(positions_dev, position_stride, batch, policy_head, masks_dev, stream=None):
    _check(_lib.az_legal_masks(_dev_ptr(positions_dev, "positions"), position_stride, batch, policy_head,
                               _dev_ptr(masks_dev, "masks"), _stream_ptr(stream)), "az_legal_masks")


def az_calibrate(net: Net, positions_dev, n, stream=None):
    _check(_lib.az_calibrate(net.handle, _dev_ptr(positions_dev, "positions"), n, _stream_ptr(stream)), "az_calibrate")


AZ_CALIBRATE_NO_BIAS_CORRECTION = 1


def az_calibrate_ex(net: Net, positions_dev, n, flags=0, stream=None):
    _check(_lib.az_calibrate_ex(net.handle, _dev_ptr(positions_dev, "positions"), n, flags, _stream_ptr(stream)), "az_calibrate_ex")


def az_device_status(net: Net, stream=None) -> int:
    status = ctypes.c_uint32(0)
    code = _lib.az_device_status(net.handle, _stream_ptr(stream), ctypes.byref(status))
    if code not in (AZ_OK, AZ_ERR_DEVICE_TIMEOUT):
        raise AzError(code, "az_device_status")
    return int(status.value)


def az_selftest_wait_timeout(stream=None) -> int:
    """Returns the library's code: AZ_ERR_DEVICE_TIMEOUT means the bounded wait ran out as it should."""
    return int(_lib.az_selftest_wait_timeout(_stream_ptr(stream)))


def az_launches_per_evaluate(net: Net, batch: int) -> int:
    return int(_lib.az_launches_per_evaluate(net.handle, batch))


def az_strerror(code: int) -> str:
    return _lib.az_strerror(code).decode()


def az_last_cuda_error() -> str:
    return _lib.az_last_cuda_error().decode()


# ---- small marshalling helpers used by tests and the benchmark ----------------------------------

def az_apply_moves(positions_dev, position_stride, batch, policy_head, actions_dev, out_positions_dev, status_dev=None, stream=None):
    _check(_lib.az_apply_moves(_dev_ptr(positions_dev, "positions"), position_stride, batch, policy_head,
                               _dev_ptr(actions_dev, "actions"), _dev_ptr(out_positions_dev, "out_positions"),
                               _dev_ptr(status_dev, "status") if status_dev is not None else None, _stream_ptr(stream)),
           "az_apply_moves")


def az_standin_evaluate(positions_dev, position_stride, legal_masks_dev, batch, policy_head, seed, legal_policy_dev,
                        legal_counts_dev, value_dev, stream=None):
    _check(_lib.az_standin_evaluate(_dev_ptr(positions_dev, "positions"), position_stride, _dev_ptr(legal_masks_dev, "legal_masks"),
                                    batch, policy_head, seed, _dev_ptr(legal_policy_dev, "legal_policy"),
                                    _dev_ptr(legal_counts_dev, "legal_counts"), _dev_ptr(value_dev, "value"), _stream_ptr(stream)),
           "az_standin_evaluate")


@dataclass
class Search:
    """Handle of a batched tree search (owns the trees in device memory; call az_search_destroy when done)."""
    handle: int
    config: az_search_config


def make_search_config(games, policy_head, position_bytes, leaves=1, groups=2, max_nodes=1024, max_edges=None,
                       evaluator=AZ_SEARCH_EVAL_NET, c_puct=1.5, fpu_reduction=0.2, discount=0.99, seed=0) -> az_search_config:
    return az_search_config(games, leaves, groups, max_nodes, max_edges or 64 * max_nodes, evaluator, policy_head,
                            position_bytes, c_puct, fpu_reduction, discount, 0, seed)


def az_search_create(net, config: az_search_config) -> Search:
    out = ctypes.c_void_p()
    _check(_lib.az_search_create(net.handle if net is not None else None, ctypes.byref(config), ctypes.byref(out)), "az_search_create")
    return Search(out.value, config)


def az_search_destroy(search: Search):
    if search is not None and search.handle:
        _lib.az_search_destroy(search.handle)
        search.handle = 0


def az_search_set_roots(search: Search, positions_host: np.ndarray):
    rec = np.ascontiguousarray(positions_host)
    if rec.nbytes != search.config.games * search.config.position_bytes:
        raise ValueError("positions_host must hold one record per game")
    _check(_lib.az_search_set_roots(search.handle, rec.ctypes.data), "az_search_set_roots")


def az_search_replace_roots(search: Search, games, positions_host: np.ndarray):
    """New root records for the listed games only (their trees are emptied); the other games go on."""
    idx = np.ascontiguousarray(games, dtype=np.int32)
    rec = np.ascontiguousarray(positions_host)
    if rec.nbytes != idx.size * search.config.position_bytes:
        raise ValueError("one record per listed game expected")
    _check(_lib.az_search_replace_roots(search.handle, idx.ctypes.data, int(idx.size), rec.ctypes.data), "az_search_replace_roots")


def az_search_run(search: Search, simulations: int) -> float:
    """Runs `simulations` steps on every tree; returns the device time in milliseconds."""
    ms = ctypes.c_float(0)
    _check(_lib.az_search_run(search.handle, simulations, ctypes.byref(ms)), "az_search_run")
    return float(ms.value)


def az_search_run_async(search: Search, simulations: int):
    """Queues `simulations` steps on every tree and returns; az_search_wait collects them."""
    _check(_lib.az_search_run_async(search.handle, simulations), "az_search_run_async")


def az_search_wait(search: Search) -> float:
    ms = ctypes.c_float(0)
    _check(_lib.az_search_wait(search.handle, ctypes.byref(ms)), "az_search_wait")
    return float(ms.value)


def az_search_root(search: Search, game: int):
    """(actions, visits, value sums, priors) of the root's edges of one game."""
    a = np.zeros(AZ_MAX_LEGAL, dtype=np.int32)
    n = np.zeros(AZ_MAX_LEGAL, dtype=np.int32)
    w = np.zeros(AZ_MAX_LEGAL, dtype=np.float32)
    p = np.zeros(AZ_MAX_LEGAL, dtype=np.float32)
    k = ctypes.c_int32(0)
    _check(_lib.az_search_root(search.handle, game, a.ctypes.data, n.ctypes.data, w.ctypes.data, p.ctypes.data, ctypes.byref(k)),
           "az_search_root")
    return a[:k.value].copy(), n[:k.value].copy(), w[:k.value].copy(), p[:k.value].copy()


def az_search_root_visits(search: Search, actions_host: np.ndarray, visits_host: np.ndarray, counts_host: np.ndarray):
    """Root actions and visit counts of all games into int32 host arrays [games][AZ_MAX_LEGAL] (x2) and [games]."""
    g = search.config.games
    for arr, shape in ((actions_host, (g, AZ_MAX_LEGAL)), (visits_host, (g, AZ_MAX_LEGAL)), (counts_host, (g,))):
        if arr.dtype != np.int32 or arr.shape != shape or not arr.flags.c_contiguous:
            raise TypeError("int32 C-contiguous arrays of [games][AZ_MAX_LEGAL], [games][AZ_MAX_LEGAL], [games] expected")
    _check(_lib.az_search_root_visits(search.handle, actions_host.ctypes.data, visits_host.ctypes.data, counts_host.ctypes.data),
           "az_search_root_visits")


def az_search_advance(search: Search, actions_host=None) -> np.ndarray:
    """Plays one move per game (actions_host: int32 policy indices, -1 = none; None: the most visited root move).
    Returns the actions played, -1 where a game's tree stayed as it was."""
    played = np.zeros(search.config.games, dtype=np.int32)
    act = None
    if actions_host is not None:
        act = np.ascontiguousarray(actions_host, dtype=np.int32)
        if act.shape != (search.config.games,):
            raise ValueError("one action per game expected")
    _check(_lib.az_search_advance(search.handle, act.ctypes.data if act is not None else None, played.ctypes.data), "az_search_advance")
    return played


def az_search_root_noise(search: Search, noise_host: np.ndarray, epsilon: float) -> np.ndarray:
    """Mixes caller-drawn noise ([games][AZ_MAX_LEGAL] float32) into the priors of every game's current root;
    returns the number of edges changed per game."""
    eta = np.ascontiguousarray(noise_host, dtype=np.float32)
    if eta.shape != (search.config.games, AZ_MAX_LEGAL):
        raise ValueError("noise must be [games][AZ_MAX_LEGAL]")
    changed = np.zeros(search.config.games, dtype=np.int32)
    _check(_lib.az_search_root_noise(search.handle, eta.ctypes.data, epsilon, changed.ctypes.data), "az_search_root_noise")
    return changed


def az_search_root_positions(search: Search, dtype) -> np.ndarray:
    """The current root records of all games as a numpy array of the given record dtype."""
    out = np.zeros(search.config.games, dtype=dtype)
    if out.dtype.itemsize != search.config.position_bytes:
        raise ValueError("dtype does not match the search's position records")
    _check(_lib.az_search_root_positions(search.handle, out.ctypes.data), "az_search_root_positions")
    return out


def az_search_tree(search: Search, game: int, nodes: bool = True):
    """counts (nodes, edges, flags, traversals given up) and, with nodes=True, per-node visit counts and value sums."""
    counts = np.zeros(4, dtype=np.int32)
    if not nodes:
        _check(_lib.az_search_tree(search.handle, game, counts.ctypes.data, None, None), "az_search_tree")
        return counts, None, None
    nvis = np.zeros(search.config.max_nodes, dtype=np.int32)
    wsum = np.zeros(search.config.max_nodes, dtype=np.float32)
    _check(_lib.az_search_tree(search.handle, game, counts.ctypes.data, nvis.ctypes.data, wsum.ctypes.data), "az_search_tree")
    return counts, nvis[:counts[0]].copy(), wsum[:counts[0]].copy()


def az_search_launches_per_step(search: Search) -> int:
    return int(_lib.az_search_launches_per_step(search.handle))


def records_to_device(records: np.ndarray, device="cuda") -> torch.Tensor:
    """A numpy record array (104- or 784-byte records) as a uint8 device tensor [n][record_bytes]."""
    raw = np.ascontiguousarray(records).view(np.uint8).reshape(records.shape[0], -1)
    return torch.from_numpy(raw.copy()).to(device)


def masks_to_numpy(masks_dev: torch.Tensor) -> np.ndarray:
    return masks_dev.cpu().numpy().view(np.uint64)
