#!/usr/bin/env python
"""Benchmark of the VScan reduction path (Stage 1 + Stage 2) on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--impl vscan|reference]

One step = one pass of the whole path (score x2 -> select -> merge -> prune) over one batch of the
LLaVA-NeXT workload (32 images x 5 crops x 576 patches = 2880 visual tokens per image, bf16).
Prints one JSON line.  `value` is images/s with inputs resident in HBM (CUDA-graph replays, CUDA
events, max over ranks); `e2e` is the same pass with pinned-host inputs copied in and results copied
out inside the timed region; `roofline` is the dominant kernel's algorithmic bytes over its CUDA-event
duration against the measured HBM copy bandwidth; `cpu_baseline` is the numpy oracle on the host.
With N > 1 every rank runs an independent replica of the batch (the path has no exchange step).
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np  # noqa: E402

from synth import CONFIGS, schedule_points, stage1_inputs, stage2_inputs, sweep_config  # noqa: E402

METRIC = "VScan reduction images/s (Stage1+Stage2) at 2880 visual tokens"
UNIT = "images/s"
FALLBACK_HBM_GBS = 6650.0
MERGE_KERNELS = ("merge_cluster", "order_members", "kept_inv_norm", "assign_simt", "assign_tensor", "group_mean", "merge_persistent", "pack_kept")


# ------------------------------------------------------------------ algorithmic work per step
def algorithmic_bytes(cfg) -> dict:
    """Bytes each call has to move per step (whole batch): every input byte read once, every output
    byte written once.  The K rows of the Stage-2 survivors are read by the scoring (the whole visual
    span of K) and are not charged a second time to the compaction."""
    e, I, B = cfg.elem_bytes, cfg.instances, cfg.B
    k_survivors = B * cfg.Hkv * cfg.k2 * cfg.d * e          # part of the span the scoring already read
    row = {
        "row_mean": I * (cfg.H * cfg.L * e + cfg.N * 4),                       # un-fused ROW-mode score
        "select": I * (2 * cfg.N * 4 + cfg.K1 * 4),                            # un-fused selection
        "score_select": 2 * I * cfg.H * cfg.L * e + I * (2 * cfg.N * 4 + cfg.K1 * 4),   # Eq. 2 + Eq. 3 fused
        "merge": I * (cfg.N * cfg.D * e + cfg.K1 * 4 + cfg.K1 * cfg.D * e),     # X once + merged out
        "qk_softmax": B * (cfg.Hkv * cfg.n_vis * cfg.d * e + cfg.Hq * cfg.d * e),
        "prune_topk": B * cfg.k2 * 4,
        "compact": B * 2 * cfg.S_out * (cfg.Dh * e + 2 * cfg.Hkv * cfg.d * e + cfg.pos_planes * 4) - k_survivors,
    }
    row["prune_fused"] = row["qk_softmax"] + row["prune_topk"] + row["compact"]   # Stage 2 in one launch
    # the step as it is launched: fused score + select, the merge call, Stage 2
    row["step"] = row["score_select"] + row["merge"] + row["prune_fused"]
    row["stage2_only"] = row["prune_fused"]
    return row


def merge_flops(cfg) -> float:
    return 2.0 * cfg.instances * (cfg.N - cfg.K1) * cfg.K1 * cfg.D


def measured_peaks() -> tuple[float, str]:
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        return float(json.load(open(path))["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


FALLBACK_BF16_TFLOPS_SUSTAINED = 1400.0   # an earlier measurement on this machine, used when the measured file is absent


def measured_tensor_peak() -> tuple[float, str]:
    """Dense bf16 TFLOP/s of a library matrix product timed inside a long loop (the figure for a kernel that is
    timed inside a step)."""
    try:
        return float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["bf16_tflops_sustained"]), "measured"
    except Exception:
        return FALLBACK_BF16_TFLOPS_SUSTAINED, "fallback"


# ------------------------------------------------------------------ clocks during the timed region
class ClockSampler(threading.Thread):
    REASONS = {0x4: "sw_power_cap", 0x8: "hw_slowdown", 0x20: "sw_thermal_slowdown",
               0x40: "hw_thermal_slowdown", 0x80: "hw_power_brake_slowdown", 0x2: "applications_clocks_setting"}

    def __init__(self, device_index: int, period_s: float = 0.004):
        super().__init__(daemon=True)
        self.period, self.samples, self.reason_bits, self.max_mhz = period_s, [], 0, None
        self._stop_evt = threading.Event()
        self.ok = False
        try:
            import pynvml
            import torch
            pynvml.nvmlInit()
            self.nv = pynvml
            try:
                uuid = "GPU-" + str(torch.cuda.get_device_properties(device_index).uuid)
                self.h = pynvml.nvmlDeviceGetHandleByUUID(uuid.encode())
            except Exception:
                self.h = pynvml.nvmlDeviceGetHandleByIndex(device_index)
            self.max_mhz = pynvml.nvmlDeviceGetMaxClockInfo(self.h, pynvml.NVML_CLOCK_SM)
            self.ok = True
        except Exception:
            self.ok = False

    def _reasons(self):
        for fn in ("nvmlDeviceGetCurrentClocksEventReasons", "nvmlDeviceGetCurrentClocksThrottleReasons"):
            f = getattr(self.nv, fn, None)
            if f is not None:
                try:
                    return int(f(self.h))
                except Exception:
                    pass
        return 0

    def sample_once(self):
        try:
            self.samples.append(self.nv.nvmlDeviceGetClockInfo(self.h, self.nv.NVML_CLOCK_SM))
            self.reason_bits |= self._reasons()
        except Exception:
            pass

    def run(self):
        if not self.ok:
            return
        while not self._stop_evt.is_set():
            self.sample_once()
            time.sleep(self.period)

    def finish(self) -> dict:
        self._stop_evt.set()
        if self.is_alive():
            self.join(timeout=2)
        if not self.ok or not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": [], "samples": 0}
        reasons = [name for bit, name in self.REASONS.items() if self.reason_bits & bit]
        return {"sm_mhz": float(np.median(self.samples)), "sm_max_mhz": self.max_mhz, "reasons": reasons,
                "samples": len(self.samples)}


# ------------------------------------------------------------------ oracle timing (CPU baseline)
def oracle_threads() -> int:
    try:
        from threadpoolctl import threadpool_info
        return max([p.get("num_threads", 1) for p in threadpool_info()] + [1])
    except Exception:
        return os.cpu_count() or 1


def oracle_image(cfg, s1, s2, img: int):
    """The whole path for one image on the CPU oracle: its C crops through Stage 1, its sequence
    through Stage 2."""
    from oracle import vscan_oracle as vo
    for c in range(cfg.C):
        i = img * cfg.C + c
        sg = vo.score_row(s1["attn_g"][i], cfg.cls)
        sl = vo.score_row(s1["attn_l"][i], cfg.cls)
        kept = vo.select_global_local(sg, sl, cfg.frames, cfg.grid_h, cfg.grid_w, cfg.win_h, cfg.win_w,
                                      cfg.k_w, cfg.k_g)[0]
        vo.merge(s1["x"][i], cfg.cls, kept)
    vo.llm_prune(s2["q_last"][img], s2["k"][img], s2["v"][img], s2["hidden"][img], s2["pos_ids"][:, img],
                 cfg.n_sys, cfg.n_vis, cfg.n_txt, cfg.k2, s2["scale"])


def time_oracle(cfg, budget_s: float = 12.0, max_images: int = 16):
    n = min(cfg.B, max_images)
    s1 = stage1_inputs(cfg, 0, n * cfg.C)
    s2 = stage2_inputs(cfg, 0, n)
    oracle_image(cfg, s1, s2, 0)            # warm numpy / BLAS
    done, t0 = 0, time.perf_counter()
    while True:
        oracle_image(cfg, s1, s2, done % n)
        done += 1
        el = time.perf_counter() - t0
        if el >= budget_s:
            break
    return {"value": done / el, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle",
            "threads": f"1 Python thread; numpy's BLAS pool of {oracle_threads()} threads inside the matrix products",
            "sample": f"{done} images of the {cfg.name} workload ({cfg.C} crops + 1 sequence each), "
                      f"{el:.1f} s of numpy fp64"}


def run_reference(args, cfg):
    """The oracle as the reference arm: one image of the workload per step."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    n = 4
    s1 = stage1_inputs(cfg, 0, n * cfg.C)
    s2 = stage2_inputs(cfg, 0, n)
    for w in range(max(args.warmup, 1)):
        oracle_image(cfg, s1, s2, w % n)
    t0 = time.perf_counter()
    for i in range(args.steps):
        oracle_image(cfg, s1, s2, i % n)
    el = time.perf_counter() - t0
    value = args.steps / el
    sample = f"1 image ({cfg.C} crops + 1 sequence) of the workload per step, numpy fp64 oracle on the host"
    print(json.dumps({
        "impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": 1e3 * el / args.steps,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
        "config": {"workload": cfg.name, "images_per_step": 1},
        "cpu_baseline": {"value": value, "unit": UNIT, "cores": oracle_threads(), "kind": "oracle", "sample": sample},
        "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }))


# ------------------------------------------------------------------ multi-rank plumbing
def dist_setup(n_gpus: int):
    """-> (rank, world, local_rank, dist or None).  One process per GPU under torchrun."""
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if world <= 1:
        return 0, 1, 0, None
    import torch.distributed as dist
    dist.init_process_group(os.environ.get("VSCAN_BENCH_BACKEND", "nccl"))
    return dist.get_rank(), world, int(os.environ.get("LOCAL_RANK", "0")), dist


def max_over_ranks(value_ms: float, dist, device) -> float:
    if dist is None:
        return value_ms
    import torch
    t = torch.tensor([value_ms], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


# ------------------------------------------------------------------ the GPU arm
def build_sets(cfg, n_sets: int, device):
    """Generate one batch on the host (at most 32 distinct images, tiled beyond that); the other sets
    are the same batch with the images rotated, so that consecutive steps touch different memory."""
    import torch
    dt = torch.float32 if cfg.dtype == "f32" else torch.bfloat16
    gen_b = min(cfg.B, 32)
    s1, s2 = stage1_inputs(cfg, 0, gen_b * cfg.C), stage2_inputs(cfg, 0, gen_b)

    def tile(t, total, axis=0):
        reps = -(-total // t.shape[axis])
        if reps > 1:
            t = torch.cat([t] * reps, dim=axis)
        return t.narrow(axis, 0, total)

    base = {name: torch.from_numpy(a).to(device=device, dtype=dt)
            for name, a in (("attn_g", s1["attn_g"]), ("attn_l", s1["attn_l"]), ("x", s1["x"]),
                            ("q_last", s2["q_last"]), ("k", s2["k"]), ("v", s2["v"]), ("hidden", s2["hidden"]))}
    pos = torch.from_numpy(s2["pos_ids"]).to(device)
    sets = []
    for r in range(n_sets):
        d = {}
        for name, t in base.items():
            per_image = cfg.C if name in ("attn_g", "attn_l", "x") else 1
            d[name] = tile(torch.roll(t, r * per_image, dims=0), cfg.B * per_image).contiguous()
        d["pos_ids"] = tile(pos, cfg.B, axis=1).contiguous()
        sets.append(d)
    return sets


def measure(args, cfg, rank, world, local_rank, dist, with_e2e=True, with_cpu=True, run_stage1=True):
    """Times one workload on this rank's GPU; rank 0 gets the JSON-able result dict, others None."""
    import torch

    import paper_2505_22654_b200 as vs
    from paper_2505_22654_b200 import binding as vb

    device = torch.device("cuda", local_rank)

    n_sets = args.sets
    warmup = max(args.warmup, 3)
    sets = build_sets(cfg, n_sets, device)
    reducers = [vs.VScanReducer.from_config(cfg, device=device, merge_path=args.merge_path,
                                            overlap_stages=args.overlap_stages, run_stage1=run_stage1)
                for _ in range(n_sets)]
    stream = torch.cuda.Stream(device)
    launches_per_step = 0
    with torch.cuda.stream(stream):
        for w in range(warmup):
            before = vs.kernel_launches()
            reducers[w % n_sets].run(**sets[w % n_sets])
            launches_per_step = vs.kernel_launches() - before
        stream.synchronize()
        graphs = []
        if not args.no_graph:
            for r in range(n_sets):
                g = torch.cuda.CUDAGraph()
                with torch.cuda.graph(g, stream=stream):
                    reducers[r].run(**sets[r])
                graphs.append(g)
            for i in range(warmup):
                graphs[i % n_sets].replay()
            stream.synchronize()

        def step(i):
            if graphs:
                graphs[i % n_sets].replay()
            else:
                reducers[i % n_sets].run(**sets[i % n_sets])

        # ---- timed region: exactly K steps between barriers and synchronisations
        sampler = ClockSampler(local_rank)
        ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        if dist is not None:
            dist.barrier()
        torch.cuda.synchronize()
        sampler.start()
        ev0.record(stream)
        for i in range(args.steps):
            step(i)
        ev1.record(stream)
        if sampler.ok:
            sampler.sample_once()       # at least one sample while the queue is still draining
        ev1.synchronize()
        torch.cuda.synchronize()
        clocks = sampler.finish()
        if dist is not None:
            dist.barrier()
        ms_total = max_over_ranks(ev0.elapsed_time(ev1), dist, device)
        # a bounded device-side wait that ran out leaves unwritten rows behind: such a run is not a measurement
        status = max(r.check() for r in reducers)

        # ---- per-kernel durations: the same steps launched directly, each kernel between two events
        prof_steps = max(1, min(args.steps, 30))
        cap = prof_steps * launches_per_step + 8
        vb.profile_begin(cap)
        for i in range(prof_steps):
            reducers[i % n_sets].run(**sets[i % n_sets])
        records = vb.profile_end(cap)
        per_kernel = {}
        for name, ms in records:
            per_kernel.setdefault(name, []).append(ms)

        # ---- end to end: pinned host buffers in and out, copies inside the timed region
        e2e = None
        red, dev_in = reducers[0], sets[0]
        if with_e2e:
            host_in = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True).copy_(v) for k, v in dev_in.items()}
            outs = {"merged": red.merged, **{k: red.out2[k] for k in ("kept_vis", "hidden", "k", "v", "pos")}}
            host_out = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True) for k, v in outs.items()}
            e_steps = max(1, min(args.steps, 8))
            dev_slots = [dev_in, sets[1 % n_sets]]
            red.run_host_many([host_in] * 2, [host_out] * 2, dev_slots)
            stream.synchronize()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            # every step uploads its inputs and downloads its results; uploads, passes and downloads
            # of neighbouring steps overlap on three streams
            red.run_host_many([host_in] * e_steps, [host_out] * e_steps, dev_slots)
            e1.record(stream)
            e1.synchronize()
            e_ms = max_over_ranks(e0.elapsed_time(e1), dist, device)
            e2e = {"value": world * cfg.B * e_steps / (e_ms * 1e-3), "unit": UNIT,
                   "h2d_bytes_per_step": int(sum(t.numel() * t.element_size() for t in host_in.values())),
                   "d2h_bytes_per_step": int(sum(t.numel() * t.element_size() for t in host_out.values())),
                   "steps": e_steps, "ms_per_step": e_ms / e_steps}

    line = None
    if rank == 0:
        peak, peak_kind = measured_peaks()
        alg = algorithmic_bytes(cfg)
        if not run_stage1:
            alg["step"] = alg["stage2_only"]
        ms_step = ms_total / args.steps
        kernels = {}
        total_k = sum(sum(v) for v in per_kernel.values())
        for name, v in per_kernel.items():
            kernels[name] = {"launches_per_step": len(v) / prof_steps, "avg_us": 1e3 * float(np.mean(v)),
                             "share": sum(v) / total_k}
        merge_names = [n for n in kernels if n in MERGE_KERNELS]
        dominant = max(kernels, key=lambda n: kernels[n]["share"])
        # the merge call is several kernels that share one pass over the features: its algorithmic
        # bytes are charged to whichever of them is being reported
        dom_bytes = alg["merge"] if dominant in merge_names else alg[dominant]
        achieved = dom_bytes / (kernels[dominant]["avg_us"] * 1e-6) / 1e9
        traffic = None
        try:
            traffic = json.load(open(os.path.join(ROOT, "profiles", "dram_traffic.json"))).get(cfg.name, {}).get(dominant)
        except Exception:
            pass
        cpu = time_oracle(cfg) if (world == 1 and with_cpu and not args.no_cpu_baseline) else None
        step_gbs = alg["step"] / (ms_step * 1e-3) / 1e9
        roof = {"kernel": dominant, "bound": "hbm", "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "traffic": traffic, "peak_kind": f"of {peak_kind}",
                "algorithmic_bytes_per_launch": dom_bytes}
        peak_tf, tf_kind = measured_tensor_peak()
        if dominant in ("assign_tensor", "merge_persistent") and \
                merge_flops(cfg) / (peak_tf * 1e12) > dom_bytes / (peak * 1e9):
            # the similarity contraction takes longer at the tensor peak than its bytes at the HBM peak: a contraction
            tf = merge_flops(cfg) / (kernels[dominant]["avg_us"] * 1e-6) / 1e12
            roof = {"kernel": dominant, "bound": "tensor", "achieved": tf, "peak": peak_tf, "unit": "TFLOP/s",
                    "frac": tf / peak_tf, "traffic": traffic, "peak_kind": f"of {tf_kind} (bf16, sustained)",
                    "algorithmic_flops_per_launch": merge_flops(cfg)}
        line = {
            "metric": METRIC, "value": world * cfg.B * args.steps / (ms_total * 1e-3), "unit": UNIT,
            "n_gpus": world, "steps": args.steps, "warmup": warmup, "ms_per_step": ms_step,
            "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": cfg.dtype,
            "data": "synthetic",
            "config": {"workload": cfg.name, "images_per_step": cfg.B, "crops_per_image": cfg.C,
                       "visual_tokens_per_image": cfg.C * cfg.N, "kept_per_crop": cfg.K1, "stage2_keep": cfg.k2,
                       "launch": "cuda graph replay" if graphs else "stream launches",
                       "l2": f"inputs+outputs {alg['step'] / 1e6:.0f} MB per step > 126 MB L2; "
                             f"{n_sets} rotating buffer sets",
                       "parallelism": "replicas only" if world > 1 else "single GPU"},
            "step_hbm": {"algorithmic_bytes": alg["step"], "achieved_gbs": step_gbs, "frac": step_gbs / peak,
                         "peak_gbs": peak, "peak_kind": peak_kind},
            "roofline": roof,
            "kernels": kernels,
            "merge": {"flops_per_step": merge_flops(cfg),
                      "us": sum(kernels[n]["avg_us"] * kernels[n]["launches_per_step"] for n in merge_names),
                      "assign_kernel": next((n for n in ("merge_cluster", "merge_persistent", "assign_tensor", "assign_simt") if n in kernels), None)},
            "gpu_launches": launches_per_step * args.steps,
            "status": status,
            "clocks": clocks,
            "e2e": e2e,
            "cpu_baseline": cpu,
        }
    del sets, reducers, graphs
    torch.cuda.empty_cache()
    return line


def run_vscan(args, cfg):
    import torch

    from paper_2505_22654_b200 import binding as vb

    rank, world, local_rank, dist = dist_setup(args.gpus)
    if not torch.cuda.is_available():
        raise RuntimeError("bench.py needs a CUDA device: the VScan path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    vb.lib()
    if args.sweep:
        run_sweep(args, rank, world, local_rank, dist)
    else:
        line = measure(args, cfg, rank, world, local_rank, dist)
        if world == 1 and not args.no_other_workloads and args.workload == "2":
            line["other_workloads"] = other_workloads(args, rank, world, local_rank, dist)
        if rank == 0:
            print(json.dumps(line))
    if dist is not None:
        dist.destroy_process_group()


def other_workloads(args, rank, world, local_rank, dist) -> dict:
    """Short runs of the 576-token batch workload and the 16384-token workload beside the headline line: images/s,
    step time, step HBM fraction and, for the tensor-bound one, the assignment kernel against the sustained bf16 peak."""
    peak_tf = 1395.5
    try:
        peak_tf = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["bf16_tflops_sustained"])
    except Exception:
        pass
    out = {}
    steps, sets = args.steps, args.sets
    for idx in (1, 3):
        cfg = CONFIGS[idx]
        args.steps, args.sets = 20, 2
        line = measure(args, cfg, rank, world, local_rank, dist, with_e2e=False, with_cpu=False)
        k = line["kernels"]
        assign = line["merge"]["assign_kernel"]
        out[cfg.name] = {
            "images_per_s": round(line["value"], 1), "ms_per_step": round(line["ms_per_step"], 4),
            "step_hbm_frac": round(line["step_hbm"]["frac"], 3), "status": line["status"],
            "kernels_us": {n: round(v["avg_us"] * v["launches_per_step"], 1) for n, v in k.items()},
            "assign_kernel": assign,
            "assign_frac_of_sustained_bf16": round(merge_flops(cfg) / (k[assign]["avg_us"] * 1e-6) / 1e12 / peak_tf, 3) if assign else None,
        }
    args.steps, args.sets = steps, sets
    return out


def run_sweep(args, rank, world, local_rank, dist):
    """Every named workload plus the batch x retention sweep at the 2880-token shape; one JSON line per
    point.  For each retention level the merge is also timed on the CUDA-core path at batch 32, which
    places the crossover between the two similarity paths."""
    from synth import SWEEP_BATCHES, SWEEP_BUDGETS
    peak_tf = 1395.5
    try:
        peak_tf = float(json.load(open(os.path.join(ROOT, "MEASURED_PEAKS.json")))["bf16_tflops_sustained"])
    except Exception:
        pass
    points = [("config%d" % i, CONFIGS[i], 0) for i in (0, 1, 2, 3)]
    points += [("sweep b=%d %s" % (b, r), sweep_config(b, r), 0) for r in SWEEP_BUDGETS for b in SWEEP_BATCHES]
    points += [("simt b=32 %s" % r, sweep_config(32, r), 1) for r in SWEEP_BUDGETS]
    points += [("tensor b=32 %s" % r, sweep_config(32, r), 2) for r in SWEEP_BUDGETS]
    points = [(label, cfg, path, True) for label, cfg, path in points]
    # the paper's pruning schedules as throughput points (Table 1, Table 6(a)/(b), App. B.1)
    points += [(label, cfg, 0, s1) for label, cfg, s1 in schedule_points()]
    if args.sweep_filter:
        points = [p for p in points if args.sweep_filter in p[0]]
    if rank == 0 and (not args.sweep_filter or args.sweep_filter in "fma"):
        from paper_2505_22654_b200 import binding as vb
        print(json.dumps({"point": "fp32 fma rate (ceiling of the CUDA-core similarity path)",
                          "tflops": round(vb.fma_rate_tflops(), 2)}), flush=True)
    if rank == 0 and (not args.sweep_filter or args.sweep_filter in "ragged"):
        import torch
        print(json.dumps(measure_ragged(args, torch.device("cuda", local_rank))), flush=True)
    if rank == 0 and (not args.sweep_filter or args.sweep_filter in "received"):
        import torch
        print(json.dumps(measure_received(args, torch.device("cuda", local_rank), peak_tf)), flush=True)
    for label, cfg, path, s1 in points:
        args.merge_path = path
        steps = args.steps
        args.steps = max(10, min(steps, int(2e5 / max(cfg.B, 1)) // 10 * 10)) if cfg.B > 64 else steps
        line = measure(args, cfg, rank, world, local_rank, dist, with_e2e=False, with_cpu=False, run_stage1=s1)
        args.steps = steps
        if rank != 0:
            continue
        k = line["kernels"]
        assign = line["merge"]["assign_kernel"]
        out = {"point": label, "workload": cfg.name, "B": cfg.B, "K1": cfg.K1, "n_vis": cfg.n_vis, "k2": cfg.k2,
               "dtype": cfg.dtype, "status": line["status"],
               "images_per_s": round(line["value"], 1), "ms_per_step": round(line["ms_per_step"], 4),
               "hbm_frac": round(line["step_hbm"]["frac"], 3), "merge_us": round(line["merge"]["us"], 1),
               "assign_kernel": assign, "assign_us": round(k[assign]["avg_us"], 1) if assign else None,
               "assign_tensor_frac": round(merge_flops(cfg) / (k[assign]["avg_us"] * 1e-6) / 1e12 / peak_tf, 4) if assign else None,
               "kernels_us": {n: round(v["avg_us"] * v["launches_per_step"], 1) for n, v in k.items()},
               "clocks_mhz": line["clocks"]["sm_mhz"], "reasons": line["clocks"]["reasons"]}
        print(json.dumps(out), flush=True)


def measure_received(args, device, peak_tf):
    """The no-[CLS] score source at the 16384-token shape (4 instances x 16 heads, head dim 128): received
    attention from q and k in two tensor-core passes over the score matrix, which is never stored."""
    import torch

    from paper_2505_22654_b200 import binding as vb
    B, H, N, d = 4, 16, 16384, 128
    g = torch.Generator(device="cpu").manual_seed(0)
    q = torch.randn((B, H, N, d), generator=g).to(torch.bfloat16).to(device)
    k = torch.randn((B, H, N, d), generator=g).to(torch.bfloat16).to(device)
    out = torch.empty((B, N), dtype=torch.float32, device=device)
    ws = vb.Workspace(0, device)
    stream = torch.cuda.Stream(device)
    with torch.cuda.stream(stream):
        L = vb.lib()
        import ctypes as C
        desc = vb.ScoreDesc(mode=vb.SCORE_RECEIVED, dtype=vb.BF16, q=q.data_ptr(), k=k.data_ptr(), batch=B, q_heads=H,
                            kv_heads=H, seq_len=N, head_dim=d, scale=d ** -0.5, scores=out.data_ptr())
        ws.reserve(L.vscan_score_workspace_bytes(C.byref(desc)))
        vb.vscan_score_received(q, k, d ** -0.5, out=out, workspace=ws)
        stream.synchronize()
        n = 3
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n):
            vb.vscan_score_received(q, k, d ** -0.5, out=out, workspace=ws)
        e1.record(stream)
        e1.synchronize()
        status = vb.vscan_check(ws)
    ms = e0.elapsed_time(e1) / n
    flops = 2 * 2.0 * B * H * N * N * d
    return {"point": "received attention from q, k: 4 x 16 heads x 16384 tokens x 128", "ms": round(ms, 3),
            "tflops": round(flops / (ms * 1e-3) / 1e12, 1), "tensor_frac": round(flops / (ms * 1e-3) / 1e12 / peak_tf, 3),
            "exp_per_s": round(2.0 * B * H * N * N / (ms * 1e-3) / 1e12, 2), "status": status,
            "score_sum_per_instance": [round(float(v), 4) for v in out.sum(dim=1).tolist()]}


def measure_ragged(args, device):
    """One mixed-resolution batch through the ragged entry points (dynamic-resolution shapes, Sec. 5.1 "Models"):
    instances of 576 to 16384 tokens sorted by size, 11.1 % of each kept, then sequences of matching lengths pruned
    to half.  CUDA events over repeated calls; inputs (63 MB + 1.1 GB) rotate through three packed copies."""
    import torch

    from paper_2505_22654_b200 import binding as vb
    dt, D, H, Hq, Hkv, d, Dh = torch.bfloat16, 1280, 16, 28, 4, 128, 3584
    mix = [(1, 24, 24)] * 8 + [(1, 32, 32)] * 8 + [(1, 48, 48)] * 4 + [(4, 32, 32)] * 2 + [(9, 32, 32)] + [(16, 32, 32)]
    g = torch.Generator(device="cpu").manual_seed(0)
    toks = [f * a * b for f, a, b in mix]
    kw = [1] * len(mix)                                                   # one local token per 4 x 4 window
    kg = [max(1, round(0.111 * n) - n // 16) for n in toks]               # the rest of the 11.1 % globally
    k1 = [n // 16 + k for n, k in zip(toks, kg)]
    attn = [torch.softmax(3 * torch.randn((H, n), generator=g), dim=-1).to(dt).to(device) for n in toks]
    xs = [torch.randn((n, D), generator=g).to(dt).to(device) for n in toks]
    n_sys, n_txt = [0] * len(mix), [128] * len(mix)
    k2 = [k // 2 for k in k1]
    q = torch.randn((len(mix), Hq, d), generator=g).to(dt).to(device)
    ks = [(torch.randn((Hkv, k + 128, d), generator=g) * d ** -0.5).to(dt).to(device) for k in k1]
    hs = [torch.randn((k + 128, Dh), generator=g).to(dt).to(device) for k in k1]
    ps = [torch.arange(k + 128, dtype=torch.int32, device=device) for k in k1]
    stream = torch.cuda.Stream(device)
    with torch.cuda.stream(stream):
        def step():
            _, _, w1 = vb.vscan_stage1_ragged(attn, attn, xs, 0, mix, 4, 4, kw, kg)
            _, w2 = vb.vscan_llm_prune_ragged(q, ks, ks, hs, ps, n_sys, k1, n_txt, k2, d ** -0.5)
            return w1, w2
        before = vb.kernel_launches()
        w1, w2 = step()
        launches = vb.kernel_launches() - before
        stream.synchronize()
        n = 10
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        e0.record(stream)
        for _ in range(n):
            w1, w2 = step()
        e1.record(stream)
        e1.synchronize()
        status = max(vb.vscan_check(w1), vb.vscan_check(w2))
    ms = e0.elapsed_time(e1) / n
    return {"point": "ragged: 24 images of 576..16384 tokens in one call per stage (packing by the binding included)",
            "images": len(mix), "tokens": sum(toks), "kept": sum(k1), "ms_per_call_pair": round(ms, 3),
            "images_per_s": round(len(mix) / (ms * 1e-3), 1), "kernel_launches": launches, "status": status}


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="vscan", choices=["vscan", "reference"])
    ap.add_argument("--workload", default="2", help="0-3, or sweep:<batch>:<retention>")
    ap.add_argument("--sets", type=int, default=3, help="rotating buffer sets")
    ap.add_argument("--merge-path", type=int, default=0, help="0 auto, 1 CUDA cores, 2 tensor cores")
    ap.add_argument("--no-graph", action="store_true")
    ap.add_argument("--overlap-stages", action="store_true", help="Stage 1 and Stage 2 as two parallel branches")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-other-workloads", action="store_true", help="skip the short runs of the other named workloads")
    ap.add_argument("--sweep", action="store_true",
                    help="all named workloads, the batch x retention sweep and the paper's pruning schedules")
    ap.add_argument("--sweep-filter", default="", help="with --sweep: only the points whose label contains this")
    args = ap.parse_args()
    if args.workload.startswith("sweep:"):
        _, b, r = args.workload.split(":")
        cfg = sweep_config(int(b), r)
    else:
        cfg = CONFIGS[int(args.workload)]
    if args.impl == "reference":
        run_reference(args, cfg)
    else:
        run_vscan(args, cfg)


if __name__ == "__main__":
    main()
