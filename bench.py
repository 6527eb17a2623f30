"""Benchmark of batched leaf evaluation: leaf evals/sec on the 20x128 bf16 batch-1024 workload.

A step is one az_evaluate call (encode -> tower -> heads -> masked softmax) on one batch of
synthetic positions that already sits in device memory.  One process per GPU; with N > 1
(torchrun) every rank evaluates its own batch (weak scaling, no collective on the data path).

  python bench.py [--gpus N] [--steps K] [--warmup W] [--config c3] [--impl ours|reference]

Prints ONE JSON line (rank 0).  `--impl reference` times the CPU oracle instead.
"""
import argparse
import json
import os
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from inputs import configs, pnet_weights, positions, weights  # noqa: E402

METRIC = "leaf evals/sec, 20x128 bf16 batch 1024"      # the headline workload (c3); other workloads name themselves
UNIT = "evals/s"


def metric_of(cfg) -> str:
    if cfg.name == "c3" and cfg.batch == 1024:
        return METRIC
    net = f"{cfg.blocks}x{cfg.channels}"
    return f"leaf evals/sec, {net} {DTYPE[cfg.precision]} batch {cfg.batch} (workload {cfg.name})"
WORKLOADS = {
    "c1": "c1: 6x64 fp32 batch 64, 73-plane policy + tanh value",
    "c2": "c2: 20x128 bf16 batch 256, 73-plane policy + tanh value",
    "c3": "c3: 20x128 bf16 batch 1024, flat-1858 policy + WDL value",
    "c5": "c5: 40x256 bf16, 112 history planes, flat-1858 policy + WDL value (batch sweep via --batch)",
    "c4": "c4: 20x128 FP8-e4m3 tower (bf16 heads) batch 4096, 73-plane policy + tanh value",
    "c4b": "c4b: c4 with residual branches scaled by 1/sqrt(20)",
    "c4x": "c4x: c4 as specified (plain weights, e4m3 weights and activations) with every operand as a pair of e4m3 numbers "
           "(three products per layer), batch 4096",
    "c4a": "c4a: c4 with pairs of e4m3 numbers for the activations only (two products per layer), batch 4096",
    "c4p": "c4p: c4 as specified (plain weights) with the tower in int8, batch 4096",
    "c4i": "c4i: c4b with the tower in int8 (u8 activations x s8 weights, int32 accumulation), batch 4096",
    "p12": "p12: the paper's own network, 12x128 bf16 batch 1024 (52 planes, capped scaled blocks, pooled context, "
           "query-key policy over 1,880 actions, WDL value)",
    "p12i": "p12i: p12 with the backbone's convolutions in int8 (pooled context and heads in floating point), batch 1024",
    "p14": "p14: the paper's own network at its reported size, 14x160 bf16, batch 320 as the paper serves it "
           "(App. D.3); --batch for other sizes",
    "p19": "p19: the paper's own network at the largest size of its ladder, 19x176 bf16, batch 296 (one round); --batch for other sizes",
    "p14i": "p14i: p14 with the backbone's convolutions in int8, the precision the paper deploys; batch 320, --batch for other sizes",
    "s14i": "s14i: the search of s14 over the int8 14x160 network",
    "s14": "s14: batched tree search (Eq. 1, c 1.5, first-play reduction 0.2, discount 0.99) over the paper's 14x160 "
           "network: two groups of games, each step one batch of leaf positions per group (296 rows = one two-board "
           "group per SM; the paper serves 320, App. D.3: --batch 320), one traversal per game and step",
    "s12": "s12: the same search over the 12x128 network (--batch 592: one round of two-group CTAs)",
    "s12i": "s12i: the same search over the int8 12x128 network",
}
SEARCH_NETS = {"s14": "p14", "s12": "p12", "s14i": "p14i", "s12i": "p12i"}
SEARCH_METRIC = "searches/sec (tree traversals with their leaf evaluation)"
SEARCH_UNIT = "searches/s"


def is_pnet(cfg) -> bool:
    return cfg.in_planes == 52


def get_config(name: str):
    name = SEARCH_NETS.get(name, name)
    return pnet_weights.PNET_CONFIGS[name] if name in pnet_weights.PNET_CONFIGS else configs.CONFIGS[name]


def make_records(cfg, count, first_index=0):
    """Position records of the workload, in the layout its network consumes."""
    if is_pnet(cfg):
        return positions.generate_moves(cfg.position_seed, count, cfg.plies, first_index=first_index)[0]
    return positions.records_for_planes(cfg.in_planes, positions.for_config(cfg, count, first_index=first_index))


def make_blob(cfg):
    return pnet_weights.make_blob(cfg) if is_pnet(cfg) else weights.make_blob(cfg)
DTYPE = {0: "f32", 1: "bf16", 2: "fp8_e4m3", 3: "int8", 4: "fp8_e4m3 (operand pairs)", 5: "fp8_e4m3 (activation pairs)"}

# DRAM bytes (read + write) of one launch of the dominant kernel come from the ncu capture of that workload,
# summarised under profiles/: each summary ends with a line
#     traffic_model: fixed_bytes=<weights and constants, read once per launch> per_position_bytes=<grows with the batch>
# taken from its dram__bytes_read.sum + dram__bytes_write.sum (captured at a batch of a few hundred; the per-position
# part scales in proportion, the weights do not).  No capture of a workload: no traffic figure.
TRAFFIC_PROFILES = {
    "c1": "tower_f32_kernel_c1_batch64.md",
    "c3": "tower_tc_kernel_c3_batch592.md",
    "c4": "tower_tc_kernel_fp8_c4_batch592.md", "c4b": "tower_tc_kernel_fp8_c4_batch592.md",
    "c4i": "tower_tc_kernel_int8_c4i_batch592.md", "c4p": "tower_tc_kernel_int8_c4i_batch592.md",
    "c5": "tower_tc_kernel_c5_batch296.md",
    "p14": "tower_tc_kernel_p14_batch296.md",
    "p14i": "tower_tc_kernel_int8_p14i_batch296.md",
}


def tower_traffic_bytes(cfg, batch):
    name = TRAFFIC_PROFILES.get(cfg.name)
    if name is None:
        return None, None
    try:
        with open(os.path.join(ROOT, "profiles", name)) as f:
            for line in f:
                if line.startswith("traffic_model:"):
                    kv = dict(item.split("=") for item in line.split()[1:])
                    return float(kv["fixed_bytes"]) + batch * float(kv["per_position_bytes"]), f"profiles/{name}"
    except (OSError, KeyError, ValueError):
        pass
    return None, None


def tower_flops_per_position(cfg) -> float:
    """Dense convolution count 2*64*9*Cin*Cout per layer; channel padding is not counted."""
    c = cfg.channels
    if is_pnet(cfg):
        # second convolutions of the pooled blocks (1, 3, 5, ...) read 3C/4 channels; the fused query/key
        # layer (a 1x1 convolution C -> 256) is part of the kernel's work
        pooled = cfg.blocks // 2
        return 2.0 * 64 * (9 * (cfg.in_planes * c + (2 * cfg.blocks - pooled) * c * c + pooled * c * (3 * c // 4)) + c * 256)
    return 2.0 * 64 * 9 * (cfg.in_planes * c + 2 * cfg.blocks * c * c)


def load_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as f:
            p = json.load(f)
        return {"bf16_tflops": float(p["bf16_tflops"]), "bf16_tflops_sustained": float(p.get("bf16_tflops_sustained", p["bf16_tflops"])),
                "hbm_gbs": float(p["hbm_gbs"]), "source": "measured"}
    except (OSError, KeyError, ValueError):
        return {"bf16_tflops": 1590.0, "bf16_tflops_sustained": 1400.0, "hbm_gbs": 6650.0, "source": "fallback"}


NOMINAL_DENSE_TFLOPS = {0: None, 1: 2250.0, 2: 4500.0, 3: 4500.0, 4: 4500.0, 5: 4500.0}    # datasheet, dense, per GPU


def measure_8bit_peak(int8: bool, seconds: float = 4.0):
    """The library GEMM of the 8-bit type at 8192^3, measured here the way the bf16 peaks were measured for
    MEASURED_PEAKS.json: best of ten launches (burst) and back to back for `seconds` (sustained), CUDA events.
    Returns {"burst": TFLOP/s, "sustained": TFLOP/s, "how": ...} or None when the library call is not available."""
    import torch
    n = 8192
    try:
        if int8:
            a = torch.randint(-127, 128, (n, n), dtype=torch.int8, device="cuda")
            b = torch.randint(-127, 128, (n, n), dtype=torch.int8, device="cuda")
            run = lambda: torch._int_mm(a, b)
            how = "torch._int_mm int8 8192^3"
        else:
            a = torch.randn(n, n, device="cuda").to(torch.float8_e4m3fn)
            b = torch.randn(n, n, device="cuda").to(torch.float8_e4m3fn).t()          # column-major second operand
            one = torch.ones((), dtype=torch.float32, device="cuda")
            run = lambda: torch._scaled_mm(a, b, scale_a=one, scale_b=one, out_dtype=torch.bfloat16)
            how = "torch._scaled_mm e4m3 8192^3"
        for _ in range(3):
            run()
        torch.cuda.synchronize()
        flops = 2.0 * n ** 3
        best = float("inf")
        for _ in range(10):
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(); run(); e1.record(); torch.cuda.synchronize()
            best = min(best, e0.elapsed_time(e1))
        reps = max(10, int(seconds * 1e3 / best))
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record()
        for _ in range(reps):
            run()
        e1.record(); torch.cuda.synchronize()
        return {"burst": flops / (best * 1e-3) / 1e12, "sustained": flops * reps / (e0.elapsed_time(e1) * 1e-3) / 1e12,
                "how": f"{how}: best of 10 (burst), {reps} launches back to back (sustained), measured in this run"}
    except Exception as exc:            # the library has no such GEMM here: say so, fall back to the nominal ratio
        return {"error": f"{type(exc).__name__}: {exc}"[:200]}


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons through NVML while the timed region runs."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.samples, self.reasons, self.max_mhz = index, [], set(), None
        self._stop_event = threading.Event()
        self.ok = False
        try:
            import pynvml
            self.nv = pynvml
            pynvml.nvmlInit()
            self.h = pynvml.nvmlDeviceGetHandleByIndex(index)
            self.max_mhz = int(pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM))
            self.ok = True
        except Exception:
            pass

    def run(self):
        if not self.ok:
            return
        nv = self.nv
        names = {
            getattr(nv, "nvmlClocksEventReasonGpuIdle", 0x1): None,
            getattr(nv, "nvmlClocksEventReasonSwPowerCap", 0x4): "sw_power_cap",
            getattr(nv, "nvmlClocksThrottleReasonHwSlowdown", 0x8): "hw_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonSwThermalSlowdown", 0x20): "sw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwThermalSlowdown", 0x40): "hw_thermal_slowdown",
            getattr(nv, "nvmlClocksThrottleReasonHwPowerBrakeSlowdown", 0x80): "hw_power_brake",
        }
        while not self._stop_event.is_set():
            try:
                self.samples.append(int(nv.nvmlDeviceGetClockInfo(self.h, nv.NVML_CLOCK_SM)))
                try:
                    r = int(nv.nvmlDeviceGetCurrentClocksEventReasons(self.h))
                except Exception:
                    r = int(nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.h))
                for bit, name in names.items():
                    if name and (r & bit):
                        self.reasons.add(name)
            except Exception:
                pass
            time.sleep(0.002)

    def stop(self):
        self._stop_event.set()
        if self.is_alive():
            self.join(timeout=2)
        return {"sm_mhz": float(np.median(self.samples)) if self.samples else None,
                "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": len(self.samples)}


def oracle_rate(cfg, blob, recs, sample: int):
    """The CPU oracle, as it stands, on the first `sample` positions: (evals/s, seconds, threads)."""
    import oracle
    sub = recs[:sample]
    t0 = time.perf_counter()
    if is_pnet(cfg):
        oracle.pnet_evaluate(blob, sub)
    else:
        oracle.evaluate(blob, sub, cfg.in_planes, cfg.policy_head)
    dt = time.perf_counter() - t0
    return sub.shape[0] / dt, dt, oracle.threads()


def run_reference(args, cfg):
    """--impl reference: the oracle on the host cores; each step a bounded sample of the workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    blob = make_blob(cfg)
    recs = make_records(cfg, cfg.batch)
    sample = min(cfg.batch, 128)
    for _ in range(args.warmup):
        oracle_rate(cfg, blob, recs, min(sample, 16))
    total_t, total_n, threads = 0.0, 0, 1
    for _ in range(args.steps):
        rate, dt, threads = oracle_rate(cfg, blob, recs, sample)
        total_t += dt
        total_n += sample
    value = total_n / total_t
    sample_txt = f"first {sample} positions of the {cfg.batch}-position batch per step"
    print(json.dumps({
        "impl": "reference", "metric": metric_of(cfg), "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": WORKLOADS[cfg.name], "sample": sample_txt},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample_txt},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def oracle_search_rate(recs, sims: int, games: int):
    """The oracle's sequential search with its stand-in evaluator (no network) on `games` roots: (searches/s, seconds)."""
    import oracle
    t0 = time.perf_counter()
    for g in range(games):
        oracle.mcts_search(recs[g:g + 1], 2, sims, seed=1)
    dt = time.perf_counter() - t0
    return games * sims / dt, dt


def run_search_reference(args, name):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    cfg = get_config(name)
    recs = make_records(cfg, 64)
    for _ in range(args.warmup):
        oracle_search_rate(recs, 50, 2)
    total_t, total_n = 0.0, 0
    for _ in range(args.steps):
        rate, dt = oracle_search_rate(recs, 400, 8)
        total_t += dt
        total_n += 8 * 400
    value = total_n / total_t
    sample_txt = ("8 games x 400 traversals per step, sequential, the oracle's stand-in evaluator in place of the network "
                  "(the oracle has no network-backed search: an upper bound of its search rate)")
    print(json.dumps({
        "impl": "reference", "metric": SEARCH_METRIC, "value": value, "unit": SEARCH_UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * total_t / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "config": {"workload": WORKLOADS[name], "sample": sample_txt},
        "cpu_baseline": {"value": value, "unit": SEARCH_UNIT, "cores": 1, "kind": "oracle", "sample": sample_txt},
        "e2e": {"value": value, "unit": SEARCH_UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
        "gpu_launches": 0,
    }))


def run_search(args, name):
    """Search workloads: a step is one search step of every game (one leaf batch per group)."""
    import torch
    import torch.distributed as dist

    import paper_2609_37447_b200 as az
    from paper_2609_37447_b200 import sharding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))
    cfg = get_config(name)
    rows = args.batch if args.batch > 0 else 296     # one two-board group per SM and group of games (148 SMs)
    leaves = max(1, args.leaves)
    games = 2 * rows // leaves
    recs = make_records(cfg, games, first_index=sharding.rank_first_index(rank, games))
    blob = make_blob(cfg)
    net = az.az_load_net(az.make_arch(cfg.in_planes, cfg.blocks, cfg.channels, cfg.policy_head, cfg.value_head, cfg.precision, rows), blob)
    if cfg.precision >= 2:      # 8-bit backbone: fix the activation ranges on the seeded calibration positions first
        cal = positions.generate_moves(cfg.position_seed + configs.CALIBRATION_SEED_OFFSET, configs.CALIBRATION_COUNT, cfg.plies)[0]
        az.az_calibrate(net, az.records_to_device(cal), cal.shape[0])
    nodes = (args.steps + args.warmup) * leaves + 2

    def new_search():
        sc = az.make_search_config(games, 2, 128, leaves=leaves, groups=2, max_nodes=nodes, max_edges=48 * nodes)
        s = az.az_search_create(net, sc)
        az.az_search_set_roots(s, recs)
        return s

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    actions = np.zeros((games, az.AZ_MAX_LEGAL), dtype=np.int32)
    visits = np.zeros((games, az.AZ_MAX_LEGAL), dtype=np.int32)
    counts = np.zeros(games, dtype=np.int32)

    def done(s):
        az.az_search_root_visits(s, actions, visits, counts)
        return int(visits[np.arange(az.AZ_MAX_LEGAL)[None, :] < counts[:, None]].sum())

    # ---- device-timed: warm-up steps, then K steps queued in one call, timed by events on the search's stream
    s = new_search()
    az.az_search_run(s, args.warmup)
    before = done(s)
    az.az_profile_tower(net, True)
    az.az_tower_time(net)
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    ms = az.az_search_run(s, args.steps)
    barrier()
    clocks = sampler.stop()
    tower_ms, tower_passes = az.az_tower_time(net)
    az.az_profile_tower(net, False)
    searched = done(s) - before
    flags = 0
    for g in range(games):
        flags |= int(az.az_search_tree(s, g, nodes=False)[0][2])
    launches = az.az_search_launches_per_step(s) * 2 * args.steps
    az.az_search_destroy(s)

    # ---- end to end: roots from host memory, K steps (plus the roots' own), the root visit counts back to the host
    # (the search object is allocated beforehand, like the network; the timed region starts with the roots on the host)
    s = new_search()
    az.az_search_run(s, 3)
    barrier()
    t0 = time.perf_counter()
    az.az_search_set_roots(s, recs)
    az.az_search_run(s, args.steps)
    searched_e2e = done(s)
    e2e_s = time.perf_counter() - t0
    barrier()
    az.az_search_destroy(s)
    status = az.az_device_status(net)

    # ---- optional: games in progress.  Every game plays its most visited move after each K-step search and keeps
    # the subtree under it (Sec. 3.3); wall clock over all moves, moves read back to the host
    play = None
    if args.moves > 0:
        nodes_play = 6 * args.steps * leaves + 2
        sc = az.make_search_config(games, 2, 128, leaves=leaves, groups=2, max_nodes=nodes_play, max_edges=48 * nodes_play)
        s = az.az_search_create(net, sc)
        az.az_search_set_roots(s, recs)
        az.az_search_run(s, args.steps)
        az.az_search_advance(s)
        barrier()
        t0 = time.perf_counter()
        run_ms, moved, restarted, spare_at = 0.0, 0, 0, 0
        spare = make_records(cfg, games, first_index=sharding.rank_first_index(rank, games) + world * games)
        for _ in range(args.moves):
            run_ms += az.az_search_run(s, args.steps)
            played = az.az_search_advance(s)
            moved += int((played >= 0).sum())
            over = np.flatnonzero(played < 0)                   # the game has ended: the next one starts in its place
            if over.size:
                pick = (spare_at + np.arange(over.size)) % games
                az.az_search_replace_roots(s, over, np.ascontiguousarray(spare[pick]))
                spare_at = int((spare_at + over.size) % games)
                restarted += int(over.size)
        play_s = time.perf_counter() - t0
        barrier()
        flags_play, kept = 0, []
        for g in range(0, games, max(1, games // 32)):
            c = az.az_search_tree(s, g, nodes=False)[0]
            flags_play |= int(c[2])
            kept.append(int(c[0]))
        az.az_search_destroy(s)
        play = {"moves_per_game": args.moves, "moves_played": moved, "games_restarted": restarted, "searches_per_s": games * leaves * args.steps * args.moves / play_s,
                "moves_per_s": moved / play_s, "ms_per_move_all_games": 1e3 * play_s / args.moves,
                "ms_in_search_per_move": run_ms / args.moves, "tree_flags": flags_play,
                "kept_nodes_median": float(np.median(kept)),
                "note": "wall clock over az_search_run + az_search_advance (+ az_search_replace_roots for games that ended) per move; "
                        "every traversal of a step counted"}

    ms_max, e2e_ms = sharding.max_over_ranks([ms, e2e_s * 1e3], device="cuda")
    if rank == 0:
        peaks = load_peaks()
        flops = tower_flops_per_position(cfg) * rows
        total_s = ms_max * 1e-3
        achieved = flops * 2 * args.steps / total_s / 1e12
        sustained = total_s >= 1.0
        peak_tf = peaks["bf16_tflops_sustained" if sustained else "bf16_tflops"] * (2.0 if cfg.precision >= 2 else 1.0)
        out = {
            "metric": SEARCH_METRIC, "value": world * searched / total_s, "unit": SEARCH_UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms_max / args.steps,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": DTYPE[cfg.precision], "data": "synthetic",
            "config": {"workload": WORKLOADS[name], "games_per_gpu": games, "rows_per_batch": rows, "leaves": leaves,
                       "l2": "not flushed: the steps run back to back on the device without returning to the host; the trees "
                             f"({games * nodes * (160 + 48 * 24) / 1e6:.0f} MB) exceed L2",
                       "timing": "CUDA events around the queued steps on the search's stream; max over ranks",
                       "device_status": status, "tree_flags": flags, "evaluations": rows * 2 * args.steps},
            "e2e": {"value": world * searched_e2e / (e2e_ms * 1e-3), "unit": SEARCH_UNIT,
                    "h2d_bytes_per_step": int(recs.nbytes / args.steps), "d2h_bytes_per_step": int((actions.nbytes + visits.nbytes + counts.nbytes) / args.steps),
                    "ms_per_step": e2e_ms / args.steps,
                    "api": "az_search_set_roots (roots from host memory) + az_search_run + az_search_root_visits "
                           "(root visit counts to host memory); bytes are per step of the K-step search"},
            "gpu_launches": launches,
            "clocks": clocks,
            "roofline": {"kernel": "tower_tc_kernel", "bound": "tensor", "achieved": achieved, "peak": peak_tf, "unit": "TFLOP/s",
                         "frac": achieved / peak_tf, "traffic": None,
                         "peak_source": f"of {peaks['source']} ({'sustained' if sustained else 'burst'} bf16 GEMM"
                                        + (" x 2, nominal 8-bit/bf16 ratio)" if cfg.precision >= 2 else ")"),
                         "note": "whole-loop figure: the tower's flops of all leaf batches over the search's elapsed time (the two "
                                 "groups' launches overlap, so a per-launch duration would count the shared time twice)",
                         "avg_launch_ms_overlapped": tower_ms / max(tower_passes, 1), "launches_timed": tower_passes,
                         "flops_per_launch": flops},
        }
        if play is not None:
            out["games_in_progress"] = play
        if not args.no_cpu_baseline:
            rate, dt = oracle_search_rate(recs, 8000, 128)
            out["cpu_baseline"] = {"value": rate, "unit": SEARCH_UNIT, "cores": 1, "kind": "oracle",
                                   "sample": f"128 games x 8,000 traversals, sequential, stand-in evaluator in place of the network "
                                             f"(the oracle has no network-backed search), {dt:.1f} s"}
        print(json.dumps(out))
    az.az_free_net(net)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=50)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--config", default="c3", choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--batch", type=int, default=0, help="override the workload's batch (profiling captures on a smaller case)")
    ap.add_argument("--leaves", type=int, default=1, help="search workloads: traversals per tree and step")
    ap.add_argument("--tower-timing-every", type=int, default=4,
                    help="the library's events around the tower kernel (roofline) on every n-th timed step (they cost the step its "
                         "dependent launch's overlap); 1 with fewer than 8 steps")
    ap.add_argument("--single-ctas", action="store_true",
                    help="load the network with AZ_LOAD_TOWER_SINGLE_CTAS: the one-CTA tower kernel instead of clusters of two CTAs "
                         "(the default for bf16 128-channel residual networks), for comparisons")
    ap.add_argument("--legs", default="all", choices=["all", "device"],
                    help="device: only the device-resident timed leg (short runs for profiler captures)")
    ap.add_argument("--moves", type=int, default=0, help="search workloads: also time this many played moves per game, each after "
                                                         "a search of --steps steps (subtrees kept)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.config in SEARCH_NETS:
        if args.impl == "reference":
            run_search_reference(args, args.config)
        else:
            run_search(args, args.config)
        return
    cfg = get_config(args.config)
    if args.batch > 0:
        import dataclasses
        cfg = dataclasses.replace(cfg, batch=args.batch)
    if args.impl == "reference":
        run_reference(args, cfg)
        return

    import torch
    import torch.distributed as dist

    import paper_2609_37447_b200 as az
    from paper_2609_37447_b200 import sharding

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local_rank)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local_rank))

    # ---- inputs: every rank evaluates its own batch of the same stream (weak scaling)
    B = cfg.batch
    recs = make_records(cfg, B, first_index=sharding.rank_first_index(rank, B))
    blob = make_blob(cfg)
    arch = az.make_arch(cfg.in_planes, cfg.blocks, cfg.channels, cfg.policy_head, cfg.value_head, cfg.precision, B)
    net = az.az_load_net_ex(arch, blob, az.AZ_LOAD_TOWER_SINGLE_CTAS) if args.single_ctas else az.az_load_net(arch, blob)
    if cfg.precision >= 2:      # 8-bit tower: fix the activation ranges on the seeded calibration positions first
        if is_pnet(cfg):
            cal = positions.generate_moves(cfg.position_seed + configs.CALIBRATION_SEED_OFFSET, configs.CALIBRATION_COUNT, cfg.plies)[0]
        else:
            cal = positions.records_for_planes(cfg.in_planes, positions.for_config(cfg, calibration=True))
        az.az_calibrate(net, az.records_to_device(cal), cal.shape[0])
    pos_dev = az.records_to_device(recs)
    masks_dev = torch.zeros((B, cfg.mask_words), dtype=torch.int64, device="cuda")
    az.az_legal_masks(pos_dev, recs.dtype.itemsize, B, cfg.policy_head, masks_dev)
    policy_dev = torch.zeros((B, cfg.policy_size), dtype=torch.float32, device="cuda")
    value_dev = torch.zeros((B, cfg.value_size), dtype=torch.float32, device="cuda")
    flush = torch.empty(256 * 1024 * 1024, dtype=torch.uint8, device="cuda")   # > 126 MB L2
    torch.cuda.synchronize()

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- device-resident timing: K steps, L2 flushed before each, each step bracketed by events
    for _ in range(args.warmup):
        az.az_evaluate(net, pos_dev, masks_dev, B, policy_dev, value_dev)
    torch.cuda.synchronize()
    # the tower's own duration (roofline) is taken on every fourth step: the library's events between the tower's
    # launch and the head kernel's cost an evaluation the overlap of its dependent launch (about 9 us at batch 1024)
    timed_every = max(1, args.tower_timing_every) if args.steps >= 8 else 1
    az.az_profile_tower(net, True, every=timed_every)
    az.az_tower_time(net)
    starts = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    ends = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps)]
    sampler = ClockSampler(local_rank)
    barrier()
    sampler.start()
    for i in range(args.steps):
        flush.fill_(i & 0xFF)
        starts[i].record()
        az.az_evaluate(net, pos_dev, masks_dev, B, policy_dev, value_dev)
        ends[i].record()
    barrier()
    clocks = sampler.stop()
    step_ms = [s.elapsed_time(e) for s, e in zip(starts, ends)]
    total_ms = float(sum(step_ms))
    tower_ms, tower_passes = az.az_tower_time(net)
    az.az_profile_tower(net, False)
    status = az.az_device_status(net)

    # ---- the same back to back without flushing (steady-state serving: weights stay in L2)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    barrier()
    ev0.record()
    for _ in range(args.steps):
        az.az_evaluate(net, pos_dev, masks_dev, B, policy_dev, value_dev)
    ev1.record()
    barrier()
    b2b_ms = ev0.elapsed_time(ev1)

    # ---- sustained: at least two seconds of evaluations back to back, clocks sampled throughout.  The timed region
    # above is a few milliseconds at boost clocks; this leg shows what holds once the power cap has settled.
    sustained = None
    if args.legs == "all" and cfg.precision != 0:
        n_sus = max(args.steps, int(2500.0 / max(b2b_ms / args.steps, 1e-3)))     # (the library times the first 4096 tower passes)
        az.az_profile_tower(net, True, every=8)
        az.az_tower_time(net)
        sus_sampler = ClockSampler(local_rank)
        barrier()
        sus_sampler.start()
        ev0.record()
        for _ in range(n_sus):
            az.az_evaluate(net, pos_dev, masks_dev, B, policy_dev, value_dev)
        ev1.record()
        barrier()
        sus_clocks = sus_sampler.stop()
        sus_ms = ev0.elapsed_time(ev1)
        sus_tower_ms, sus_passes = az.az_tower_time(net)
        az.az_profile_tower(net, False)
        sustained = {"steps": n_sus, "ms": sus_ms, "tower_ms": sus_tower_ms, "passes": sus_passes, "clocks": sus_clocks}

    host = None
    if args.legs == "all":
        host = host_legs(az, torch, args, cfg, net, recs, masks_dev, B, barrier)

    # ---- the library GEMM of the 8-bit operand type, measured here (MEASURED_PEAKS.json has bf16 only)
    peak8 = None
    if cfg.precision >= 2 and rank == 0 and args.legs == "all":
        peak8 = measure_8bit_peak(cfg.precision == 3)

    # ---- max over ranks
    times = [total_ms, b2b_ms, tower_ms] + ([sustained["ms"]] if sustained else [0.0]) + (host["times_ms"] if host else [0.0] * 4)
    total_ms, b2b_ms, tower_ms_max, sus_ms_max, e2e_ms, e2e_legal_ms, e2e_pipe_ms, e2e_pipe_legal_ms = sharding.max_over_ranks(times, device="cuda")

    if rank == 0:
        peaks = load_peaks()
        evals = world * B * args.steps
        flops = tower_flops_per_position(cfg) * B
        tower_avg_ms = tower_ms / max(tower_passes, 1)
        achieved = flops / (tower_avg_ms * 1e-3) / 1e12 if tower_passes else None
        traffic, traffic_source = tower_traffic_bytes(cfg, B)
        # a tower launch of a few hundred microseconds between L2 flushes is a burst; launches of milliseconds back to
        # back for the whole timed region run under the power cap like the sustained GEMM
        long_launch = tower_avg_ms >= 2.0
        which = "sustained" if long_launch else "burst"
        if cfg.precision >= 2 and peak8 is not None and "error" not in peak8:
            peak_tf, peak_sus = peak8[which], peak8["sustained"]
            peak_note = f"of measured ({which}; {peak8['how']})"
        elif cfg.precision >= 2:
            peak_tf = peaks["bf16_tflops_sustained" if long_launch else "bf16_tflops"] * 2.0
            peak_sus = peaks["bf16_tflops_sustained"] * 2.0
            peak_note = (f"of {peaks['source']} ({which} bf16 GEMM x 2, the nominal 8-bit/bf16 ratio; no 8-bit library GEMM was measured"
                         + (": " + peak8["error"] if peak8 else " in this run") + ")")
        else:
            peak_tf = peaks["bf16_tflops_sustained" if long_launch else "bf16_tflops"]
            peak_sus = peaks["bf16_tflops_sustained"]
            peak_note = f"of {peaks['source']} ({which} bf16 GEMM; sustained is used when a tower launch takes 2 ms or more)"
        roof_kernel, roof_bound = "tower_tc_kernel", "tensor"
        nominal = NOMINAL_DENSE_TFLOPS[cfg.precision]
        if cfg.precision == 0:
            # the fp32 network runs on the FP32 FMA pipes: 148 SMs x 128 FMA per clock x 2 x the maximum SM clock
            roof_kernel, roof_bound = "tower_f32_kernel", "alu"
            peak_tf = 148 * 128 * 2 * (clocks.get("sm_max_mhz") or 1965) * 1e6 / 1e12
            peak_sus, nominal = peak_tf, peak_tf
            peak_note = "derived: 148 SMs x 128 FP32 FMA per clock x 2 x the maximum SM clock"
        out = {
            "metric": metric_of(cfg), "value": evals / (total_ms * 1e-3), "unit": UNIT, "n_gpus": world,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": total_ms / args.steps,
            "ms_per_step_median": float(np.median(step_ms)), "ms_per_step_best": float(min(step_ms)),
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": DTYPE[cfg.precision], "data": "synthetic",
            "config": {"workload": WORKLOADS[cfg.name], "batch_per_gpu": B, "l2": "flushed before every step (256 MB write)",
                       "timing": "CUDA events around each step on the launch stream, summed; max over ranks",
                       "device_status": status, "tower_cta_pairs": bool(not args.single_ctas and cfg.precision != 0 and (cfg.channels == 128 or (cfg.channels == 256 and cfg.precision == 1 and B > 148)))},
            "back_to_back": {"value": evals / (b2b_ms * 1e-3), "unit": UNIT, "ms_per_step": b2b_ms / args.steps,
                             "note": "no L2 flush between steps"},
            "gpu_launches": args.steps * az.az_launches_per_evaluate(net, B),
            "clocks": clocks,
            "roofline": {"kernel": roof_kernel, "bound": roof_bound, "achieved": achieved, "peak": peak_tf,
                         "unit": "TFLOP/s", "frac": (achieved / peak_tf) if achieved else None,
                         "frac_of_nominal_dense_peak": (achieved / nominal) if achieved and nominal else None,
                         "nominal_dense_peak": nominal,
                         "traffic": traffic, "traffic_source": traffic_source, "peak_source": peak_note,
                         "avg_launch_ms": tower_avg_ms, "launches_timed": tower_passes, "timed_every_nth_step": timed_every,
                         "flops_per_launch": flops},
        }
        if sustained:
            sus_tower_avg = sustained["tower_ms"] / max(sustained["passes"], 1)
            sus_ach = flops / (sus_tower_avg * 1e-3) / 1e12 if sustained["passes"] else None
            mhz = sustained["clocks"].get("sm_mhz")
            out["sustained"] = {
                "value": world * B * sustained["steps"] / (sus_ms_max * 1e-3), "unit": UNIT, "steps": sustained["steps"],
                "seconds": sus_ms_max * 1e-3, "ms_per_step": sus_ms_max / sustained["steps"], "clocks": sustained["clocks"],
                "ms_per_step_x_sm_mhz": (sus_ms_max / sustained["steps"]) * mhz if mhz else None,
                "tower_avg_launch_ms": sus_tower_avg, "tower_achieved": sus_ach, "tower_peak_sustained": peak_sus,
                "tower_frac_of_sustained_peak": (sus_ach / peak_sus) if sus_ach else None,
                "tower_frac_of_nominal_dense_peak": (sus_ach / nominal) if sus_ach and nominal else None,
                "note": "evaluations back to back on one stream for two seconds and more, no L2 flush, clocks sampled throughout; "
                        "the tower's launches timed by events inside the library",
            }
        if host:
            h2d, d2h, d2h_legal = host["h2d"], host["d2h"], host["d2h_legal"]
            out["config"]["policy_checksum"] = host["checksum"]
            out["e2e"] = {"value": evals / (e2e_pipe_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                          "ms_per_step": e2e_pipe_ms / args.steps,
                          "api": "az_submit_host / az_wait_host, pinned host buffers, two batches in flight (dense policy out)"}
            out["e2e_sync"] = {"value": evals / (e2e_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                               "ms_per_step": e2e_ms / args.steps, "api": "az_evaluate_host, pinned host buffers, one batch at a time"}
            out["e2e_legal_moves_only"] = {"value": evals / (e2e_pipe_legal_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                                           "d2h_bytes_per_step": int(d2h_legal), "ms_per_step": e2e_pipe_legal_ms / args.steps,
                                           "api": "az_submit_host / az_wait_host, legal-moves-only policy out, two batches in flight"}
            out["e2e_legal_moves_only_sync"] = {"value": evals / (e2e_legal_ms * 1e-3), "unit": UNIT, "h2d_bytes_per_step": int(h2d),
                                                "d2h_bytes_per_step": int(d2h_legal), "ms_per_step": e2e_legal_ms / args.steps,
                                                "api": "az_evaluate_legal_host, pinned host buffers, one batch at a time"}
        if not args.no_cpu_baseline and args.legs == "all":
            # about twenty core-seconds of the oracle: 500 positions at 20 x 128 (it runs some 25 positions per
            # second and core there), fewer in proportion to the tower's work for the larger networks
            sample = max(16, int(500 * 757e6 / tower_flops_per_position(cfg))) if cfg.channels >= 128 else cfg.batch
            sample = min(sample, B)
            rate, dt, threads = oracle_rate(cfg, blob, recs, sample)
            out["cpu_baseline"] = {"value": rate, "unit": UNIT, "cores": threads, "kind": "oracle",
                                   "sample": f"first {sample} positions of the batch, {dt:.1f} s"}
        print(json.dumps(out))
    az.az_free_net(net)
    if world > 1:
        dist.destroy_process_group()


def host_legs(az, torch, args, cfg, net, recs, masks_dev, B, barrier):
    """The end-to-end legs: the same evaluation through the entry points that take HOST buffers, every step copying its
    inputs in from pinned host memory and its results out.  Returns wall-clock times in ms and the bytes moved per step."""
    pos_host = torch.from_numpy(np.ascontiguousarray(recs).view(np.uint8).reshape(B, -1).copy()).pin_memory()
    masks_host = masks_dev.cpu().pin_memory()
    policy_host = torch.zeros((B, cfg.policy_size), dtype=torch.float32).pin_memory()
    value_host = torch.zeros((B, cfg.value_size), dtype=torch.float32).pin_memory()
    for _ in range(3):
        az.az_evaluate_host(net, pos_host, masks_host, B, policy_host, value_host)
    barrier()
    t0 = time.perf_counter()
    for i in range(args.steps):
        az.az_evaluate_host(net, pos_host, masks_host, B, policy_host, value_host)
    torch.cuda.synchronize()
    e2e_s = time.perf_counter() - t0
    barrier()
    h2d = pos_host.numel() + masks_host.numel() * 8
    d2h = (policy_host.numel() + value_host.numel()) * 4
    # the same with the policy returned over the legal moves only (1 KB per position instead of 7.4 KB)
    legal_host = torch.zeros((B, az.AZ_MAX_LEGAL), dtype=torch.float32).pin_memory()
    counts_host = torch.zeros((B,), dtype=torch.int32).pin_memory()
    for _ in range(3):
        az.az_evaluate_legal_host(net, pos_host, masks_host, B, legal_host, counts_host, value_host)
    barrier()
    t0 = time.perf_counter()
    for i in range(args.steps):
        az.az_evaluate_legal_host(net, pos_host, masks_host, B, legal_host, counts_host, value_host)
    torch.cuda.synchronize()
    e2e_legal_s = time.perf_counter() - t0
    barrier()
    d2h_legal = (legal_host.numel() + counts_host.numel() + value_host.numel()) * 4
    checksum = float(policy_host.sum())            # every row sums to one

    # pipelined: az_submit_host / az_wait_host with two batches in flight, each with its own pinned input and output
    # buffers; every step still copies its inputs in and its results out
    def pipelined(dense: bool) -> float:
        bufs = []
        for _ in range(az.AZ_HOST_SLOTS):
            bufs.append((pos_host.clone().pin_memory(), masks_host.clone().pin_memory(),
                         torch.zeros_like(policy_host).pin_memory() if dense else None,
                         None if dense else torch.zeros_like(legal_host).pin_memory(),
                         None if dense else torch.zeros_like(counts_host).pin_memory(),
                         torch.zeros_like(value_host).pin_memory()))

        def run(steps: int):
            tickets = []
            for i in range(steps):
                if len(tickets) == az.AZ_HOST_SLOTS:
                    az.az_wait_host(net, tickets.pop(0))
                p, m, pol, leg, cnt, val = bufs[i % az.AZ_HOST_SLOTS]
                tickets.append(az.az_submit_host(net, p, m, B, pol, leg, cnt, val))
            for t in tickets:
                az.az_wait_host(net, t)

        run(4)
        barrier()
        t0 = time.perf_counter()
        run(args.steps)
        dt = time.perf_counter() - t0
        barrier()
        return dt

    e2e_pipe_s = pipelined(True)
    e2e_pipe_legal_s = pipelined(False)
    return {"times_ms": [e2e_s * 1e3, e2e_legal_s * 1e3, e2e_pipe_s * 1e3, e2e_pipe_legal_s * 1e3],
            "h2d": h2d, "d2h": d2h, "d2h_legal": d2h_legal, "checksum": checksum}


if __name__ == "__main__":
    main()
