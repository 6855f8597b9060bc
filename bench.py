#!/usr/bin/env python
"""Benchmark of the SSD-SGD update path on B200.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

One "step" is one whole iteration of the method (server aggregate + momentum-SGD and all K
workers' GLU updates, with the pre_weight refreshes and pulls the schedule asks for) over one
batch of synthetic gradients, through the fused ssd_step entry point.  The timed steps are all
in the steps-delay stage (the SSD-SGD warm-up stage and the first GLU call run before timing).
Prints ONE JSON line.  With --gpus N > 1 (under torchrun) every rank runs an independent
replica: the method's state lives on one GPU and there is no exchange between GPUs.
"""
from __future__ import annotations

import argparse
import hashlib
import json
import os
import statistics
import subprocess
import sys
import tempfile
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

import numpy as np
import torch

METRIC = "ssd_sgd_update_bandwidth"
UNIT = "GB/s"
NOMINAL_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0

# name -> layout, workers, server lr, momentum, SSD warm-up iterations, delay steps, gradient sigma
WORKLOADS = {
    "resnet20_K4": dict(layout="resnet20", K=4, lr=0.1, m=0.9, W=2, k=4, sigma=1e-2),
    "resnet56_K8": dict(layout="resnet56", K=8, lr=0.1, m=0.9, W=5, k=4, sigma=1e-2),
    "resnet50_K8": dict(layout="resnet50", K=8, lr=0.1, m=0.9, W=8, k=4, sigma=1e-3),
    "vgg16_K16": dict(layout="vgg16", K=16, lr=0.01, m=0.9, W=4, k=4, sigma=1e-3),
}
DEFAULT_WORKLOAD = "vgg16_K16"

# DRAM bytes per PARAMETER of one step_kernel launch (dram__bytes_read.sum + dram__bytes_write.sum
# from an ncu capture of a small flat arena: 2^24 parameters, K = 16 float32 workers, 4.4 GB
# resident), by iteration flags (0 plain, 2 refresh, 4 pull).  The kernel streams every byte once,
# so its traffic grows in proportion to the parameter count and a full-size launch is this figure
# times its parameters.  Valid only for K = 16 float32 and the kernel sources with this digest;
# otherwise the bench line carries traffic = null.
NCU_TRAFFIC = {"digest": "76c747b132b71595", "K": 16, "grad_dtype": "f32", "captured_params": 1 << 24,
               "bytes_per_param": {0: 269.880, 2: 332.624, 4: 332.893}}
TARGET_TIMED_MS = 2000.0      # repeats of the timed region are added until about this much GPU time


def kernel_digest() -> str:
    h = hashlib.sha256()
    for name in ("ssd_kernels.cuh", "ssd_ring.cuh", "ssd_sgd.cu"):
        with open(os.path.join(ROOT, "paper_2012_05396_b200", "csrc", name), "rb") as fh:
            h.update(fh.read())
    return h.hexdigest()[:16]


def step_bytes_per_param(K: int, sg: int, flags: int, shared_pre: bool = False, local_sgd: bool = False,
                         merged_dev: bool = False) -> int:
    """Algorithmic bytes one fused delay-stage step moves per parameter: K gradients, K local
    weights read and written, K pre_weights read, w and mom read and written; a refresh adds K
    pre_weight stores, a pull adds K device-weight stores (and trades nothing else).  With one
    shared pre_weight buffer it is read once and refreshed once instead of K times.  Without
    separate device weights (merged_dev) a pull iteration is the server update plus K stores of the
    new global weight (plus, where it also writes pre_weight, the old local weights going there)."""
    pre_copies = 1 if shared_pre else K
    if merged_dev and flags & 4:
        writes_pre = bool(flags & 3) and not local_sgd
        return K * sg + 16 + 4 * K + (8 * pre_copies if writes_pre else 0)
    if local_sgd:       # plain-SGD local updater: no pre_weight traffic at all
        return K * (sg + 8) + 16 + (4 * K if flags & 4 else 0)
    b = K * (sg + 8) + 4 * pre_copies + 16
    if flags & 2:       # refresh
        b += 4 * pre_copies
    if flags & 4:       # pull
        b += 4 * K
    return b


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


class ClockSampler:
    """nvidia-smi clock samples of one GPU while the timed region runs."""

    QUERY = ("clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.hw_slowdown,"
             "clocks_event_reasons.hw_thermal_slowdown,clocks_event_reasons.sw_thermal_slowdown,"
             "clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index = index
        self.proc = None
        self.file = None

    def start(self):
        try:
            self.file = tempfile.NamedTemporaryFile("w+", suffix=".csv", delete=False)
            self.proc = subprocess.Popen(
                ["nvidia-smi", "-i", str(self.index), f"--query-gpu={self.QUERY}",
                 "--format=csv,noheader,nounits", "-lms", "20"],
                stdout=self.file, stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self):
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        self.file.flush()
        self.file.seek(0)
        sm, smax, reasons = [], [], set()
        names = ("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap")
        for line in self.file.read().splitlines():
            f = [x.strip() for x in line.split(",")]
            if len(f) < 7:
                continue
            try:
                sm.append(float(f[0]))
                smax.append(float(f[1]))
            except ValueError:
                continue
            for name, val in zip(names, f[3:7]):
                if val.lower().startswith("active"):
                    reasons.add(name)
        self.file.close()
        os.unlink(self.file.name)
        if sm:
            out.update(sm_mhz=statistics.median(sm), sm_max_mhz=max(smax), reasons=sorted(reasons),
                       samples=len(sm))
        return out


def dist_setup(n_gpus: int):
    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    if n_gpus > 1 and world != n_gpus:
        raise SystemExit(f"--gpus {n_gpus} needs torchrun with {n_gpus} ranks (WORLD_SIZE={world})")
    return world, rank, local


def max_over_ranks(value: float, device, world: int) -> float:
    """The slowest rank's time: every rank gets the maximum (identity for a single rank)."""
    if world <= 1:
        return float(value)
    import torch.distributed as dist
    t = torch.tensor([value], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, ms_max: float) -> float:
    """Units all replicas processed per second, over the slowest rank's time."""
    return units_per_rank * world / (ms_max * 1e-3)


def oracle_sample_run(wl, n_sample: int, steps: int, grads_host, w0_host):
    """Times the CPU oracle, as it stands, on the first n_sample arena elements for `steps`
    delay-stage iterations.  Returns (seconds, bytes moved, params updated, threads used)."""
    import oracle
    hp = oracle.Hyper(K=wl["K"], lr=wl["lr"], m=wl["m"], W=wl["W"], k=wl["k"])
    st = oracle.State(hp, w0_host[:n_sample], fill=0.0)
    for n in range(wl["W"] + 1):                      # SSD warm-up stage and the first GLU call: untimed
        st.step(grads_host[n % len(grads_host)])
    moved = 0
    t0 = time.perf_counter()
    for n in range(steps):
        _, flags = st.step(grads_host[n % len(grads_host)])
        moved += step_bytes_per_param(wl["K"], 4, flags) * n_sample
    dt = time.perf_counter() - t0
    return dt, moved, n_sample * steps, 1


def oracle_all_cores_run(wl, n_sample: int, steps: int, grads_host, w0_host, threads: int):
    """The same oracle, untouched, run by `threads` host threads on disjoint element ranges of the
    sample (the update is elementwise; the C calls release the interpreter lock).  Returns seconds."""
    import oracle
    from concurrent.futures import ThreadPoolExecutor
    hp = oracle.Hyper(K=wl["K"], lr=wl["lr"], m=wl["m"], W=wl["W"], k=wl["k"])
    bounds = [n_sample * t // threads for t in range(threads + 1)]
    parts = []
    for t in range(threads):
        lo, hi = bounds[t], bounds[t + 1]
        st = oracle.State(hp, w0_host[lo:hi], fill=0.0)
        gs = [[np.ascontiguousarray(g[lo:hi]) for g in gset] for gset in grads_host]
        parts.append((st, gs))

    def advance(part, first, count):
        st, gs = part
        for n in range(first, first + count):
            st.step(gs[n % len(gs)])

    with ThreadPoolExecutor(threads) as pool:
        list(pool.map(lambda part: advance(part, 0, wl["W"] + 1), parts))       # untimed, as above
        t0 = time.perf_counter()
        list(pool.map(lambda part: advance(part, wl["W"] + 1, steps), parts))
        return time.perf_counter() - t0


def run_reference(args, wl_name, wl):
    """--impl reference: the CPU oracle on the host cores, a bounded sample per step."""
    from paper_2012_05396_b200 import synth
    lay = synth.get_layout(wl["layout"])
    n_sample = min(lay.padded_numel, 1 << 22)
    K = wl["K"]
    w0 = synth.init_weights(lay)[:n_sample].numpy() if lay.padded_numel <= (1 << 22) else \
        synth.normal(synth.stream_key(synth.SEED, synth.STREAM_WEIGHT), n_sample, 0.02).numpy()
    sets = []
    for s in range(2):
        sets.append([synth.normal(synth.stream_key(synth.SEED, synth.STREAM_GRAD, s, i), n_sample,
                                  wl["sigma"]).numpy() for i in range(K)])
    import oracle
    hp = oracle.Hyper(K=K, lr=wl["lr"], m=wl["m"], W=wl["W"], k=wl["k"])
    st = oracle.State(hp, w0, fill=0.0)
    for n in range(wl["W"] + 1 + args.warmup):
        st.step(sets[n % 2])
    moved = 0
    t0 = time.perf_counter()
    for n in range(args.steps):
        _, flags = st.step(sets[n % 2])
        moved += step_bytes_per_param(K, 4, flags) * n_sample
    dt = time.perf_counter() - t0
    gbs = moved / dt / 1e9
    sample = f"first {n_sample} of {lay.padded_numel} arena elements per step, all {K} workers"
    line = {
        "impl": "reference", "metric": METRIC, "value": gbs, "unit": UNIT, "n_gpus": args.gpus,
        "steps": args.steps, "warmup": args.warmup, "ms_per_step": dt / args.steps * 1e3,
        "higher_is_better": True, "scaling": "weak", "vs_baseline": None, "dtype": "f32",
        "data": "synthetic", "params_per_s": n_sample * args.steps / dt,
        "config": {"workload": wl_name, "layout": wl["layout"], "workers": K, "delay_k": wl["k"],
                   "grad_dtype": "f32", "sample": sample},
        "cpu_baseline": {"value": gbs, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
        "e2e": {"value": gbs, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
    }
    print(json.dumps(line))


def host_step_bytes(K: int, sg: int, flags: int, stage_delay: bool, host_grads: bool, host_pre: bool,
                    read_back: bool):
    """(host-to-device, device-to-host) bytes per parameter of one ssd_step_host call."""
    h2d = K * sg if host_grads else 0
    d2h = 4 if read_back else 0
    if host_pre and stage_delay:
        if not flags & 1:            # every GLU call but the first reads pre_weight
            h2d += 4
        if flags & 3:                # the first call and the refreshes write it back
            d2h += 4
    return h2d, d2h


def time_regions(run_region, repeats: int, world: int, dev_name: str):
    """Times `repeats` regions on the current stream, each bracketed by a barrier and a device
    synchronisation on both sides; returns per region (ms over ranks' maximum, per-step ms list)."""
    import torch.distributed as dist
    out = []
    for _ in range(repeats):
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        events = run_region()
        torch.cuda.synchronize()
        if world > 1:
            dist.barrier()
        total = events[0].elapsed_time(events[-1])
        steps = [events[i].elapsed_time(events[i + 1]) for i in range(len(events) - 1)]
        out.append((max_over_ranks(total, dev_name, world), steps))
    return out


def kernel_table(peak: float):
    """Every update kernel on two more workloads of 25M parameters and more, measured in this process
    with the sweep's method (CUDA events between back-to-back launches, buffer sets rotated so that
    nothing is served from L2): the ResNet-50 layout with K = 8 float32 workers and a flat 2^26
    tensor with K = 16 bfloat16 workers."""
    from paper_2012_05396_b200 import sweep, synth
    rows = []
    cases = [("resnet50_K8_f32", synth.get_layout("resnet50").numels, 25, 8, "f32"),
             ("flat2p26_K16_bf16", None, 26, 16, "bf16")]
    for name, numels, log2n, K, dtype in cases:
        for rec in sweep.point(log2n, K, dtype, ["sync", "glu", "step", "step_merged"], 20, peak, numels=numels):
            if "gbs" not in rec:
                rows.append({"workload": name, "kernel": rec["kernel"], "skipped": rec.get("skipped")})
                continue
            rows.append({"workload": name, "kernel": rec["kernel"], "params": rec["params"], "workers": K,
                         "grad_dtype": dtype, "algorithmic_bytes": rec["bytes_per_launch"],
                         "ms": rec["ms_median"], "gbs": rec["gbs"], "frac_of_measured": rec["gbs"] / peak,
                         "frac_of_nominal_8TBs": rec["gbs"] / NOMINAL_HBM_GBS})
    return rows


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=20)
    ap.add_argument("--warmup", type=int, default=4)
    ap.add_argument("--workload", default=DEFAULT_WORKLOAD, choices=sorted(WORKLOADS))
    ap.add_argument("--impl", default="b200", choices=["b200", "reference"])
    ap.add_argument("--repeats", type=int, default=0,
                    help="timed regions of --steps steps each (0 = at least 5, more until about 2 s of GPU time)")
    ap.add_argument("--e2e-steps", type=int, default=4)
    ap.add_argument("--no-host-pre", action="store_true", help="skip the host-resident pre_weight legs")
    ap.add_argument("--no-kernel-table", action="store_true", help="skip the per-kernel table")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-graph", action="store_true",
                    help="skip the CUDA-graph replay leg (it runs for L2-resident workloads only)")
    ap.add_argument("--per-tensor", action="store_true",
                    help="per-tensor hyper-parameters: weight decay 5e-4 on conv/FC weights only")
    ap.add_argument("--shared-pre", action="store_true",
                    help="one pre_weight buffer shared by all workers (fewer algorithmic bytes, counted as such)")
    ap.add_argument("--merged-dev", action="store_true",
                    help="no separate device weights (w_dev[i] is w_loc[i]): pull iterations skip the local update")
    ap.add_argument("--local-sgd", action="store_true",
                    help="workers update with plain SGD (Eq. 5) instead of GLU (fewer algorithmic bytes, counted as such)")
    ap.add_argument("--threads", type=int, default=0, help="threads per block (0 = library default)")
    ap.add_argument("--blocks-per-sm", type=int, default=0, help="resident blocks per SM (0 = default)")
    args = ap.parse_args()
    wl_name, wl = args.workload, WORKLOADS[args.workload]

    world, rank, local = dist_setup(args.gpus)
    if args.impl == "reference":
        if rank == 0:
            run_reference(args, wl_name, wl)
        return

    from paper_2012_05396_b200 import binding as B
    from paper_2012_05396_b200 import build as libbuild
    from paper_2012_05396_b200 import synth
    from paper_2012_05396_b200.state import DeviceState, alloc_arenas

    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device; there is no CPU path")
    if rank == 0:
        libbuild.build_library()
    torch.cuda.set_device(local)
    dev_name = f"cuda:{local}"
    if world > 1:
        import torch.distributed as dist
        dist.init_process_group("nccl", device_id=torch.device(dev_name))
        dist.barrier()

    K, sg = wl["K"], 4
    lay = synth.get_layout(wl["layout"])
    N = lay.padded_numel
    n_sets = 2
    need = ((2 + 3 * K) * N * 4 + n_sets * K * N * sg) * 1.05
    free, _total = torch.cuda.mem_get_info()
    if need > free:
        raise SystemExit(f"workload needs {need / 2**30:.1f} GiB, only {free / 2**30:.1f} GiB free")

    nan = float("nan")
    hp = B.make_hparams(K, wl["lr"], wl["m"], wl["W"], wl["k"], wd=5e-4 if args.per_tensor else 0.0,
                        lr_local=nan, alpha=nan, beta=nan, rescale=nan, grad_dtype=B.SSD_F32,
                        local_updater=B.SSD_LOCAL_SGD if args.local_sgd else B.SSD_LOCAL_GLU)
    w0 = synth.init_weights(lay, device=dev_name)
    st = DeviceState(lay.numels, hp, w0, device=dev_name, fill=0.0, shared_pre=args.shared_pre,
                     merged_dev=args.merged_dev)
    if args.per_tensor:
        table = torch.empty(st.ctx.ssd_tensor_table_bytes(), dtype=torch.uint8, device=dev_name)
        st.ctx.ssd_set_tensor_scales(None, [1.0 if kind == "he" else 0.0 for kind in lay.kinds], table)
    if args.threads or args.blocks_per_sm:
        st.ctx.ssd_set_launch(args.threads, args.blocks_per_sm)
    mask = synth.valid_mask(lay, dev_name) if N != lay.numel else None
    grad_sets = []
    for s in range(n_sets):                       # each set of K gradient arenas is one allocation
        arenas = alloc_arenas(K, N, torch.float32, dev_name)
        for i in range(K):
            arenas[i].copy_(synth.gradient(lay, s, i, wl["sigma"], device=dev_name, mask=mask))
        grad_sets.append(arenas)
    stream = torch.cuda.current_stream()
    state_bytes = st.bytes()
    l2_note = "inputs larger than L2 (no flush needed)" if state_bytes > 4 * 126e6 \
        else "L2-resident: not an HBM measurement"

    # SSD warm-up stage + first GLU call, then the bench's own warm-up steps (all untimed); the
    # last of them are timed roughly to choose the number of repeats.
    warm = max(args.warmup, 3)
    for n in range(wl["W"] + 1):
        st.ctx.ssd_step(grad_sets[n % n_sets])
    torch.cuda.synchronize()
    t0 = time.perf_counter()
    for n in range(warm):
        st.ctx.ssd_step(grad_sets[n % n_sets])
    torch.cuda.synchronize()
    est_region_ms = (time.perf_counter() - t0) / warm * args.steps * 1e3
    est_region_ms = max_over_ranks(est_region_ms, dev_name, world)
    repeats = args.repeats or int(min(50, max(5, -(-TARGET_TIMED_MS // max(est_region_ms, 1e-3)))))

    flags_per_region = []
    launches0 = st.ctx.ssd_kernel_launches()

    def region():
        it0 = st.ctx.ssd_get_counters()[0]
        flags_per_region.append([st.ctx.ssd_schedule(it0 + n)[1] for n in range(args.steps)])
        ev = [torch.cuda.Event(enable_timing=True) for _ in range(args.steps + 1)]
        ev[0].record(stream)
        for n in range(args.steps):
            st.ctx.ssd_step(grad_sets[n % n_sets])
            ev[n + 1].record(stream)
        return ev

    sampler = ClockSampler(local)
    sampler.start()
    time.sleep(0.3)
    t_wall = time.perf_counter()
    regions = time_regions(region, repeats, world, dev_name)
    t_wall = time.perf_counter() - t_wall
    clocks = sampler.stop()
    launches = st.ctx.ssd_kernel_launches() - launches0

    def region_bytes(flags):
        return [step_bytes_per_param(K, sg, f, args.shared_pre, args.local_sgd, args.merged_dev) * N for f in flags]

    rates = [whole_job_rate(float(sum(region_bytes(f))), world, ms) / 1e9
             for f, (ms, _) in zip(flags_per_region, regions)]
    order = sorted(range(repeats), key=lambda r: rates[r])
    mid = order[repeats // 2]                                     # the median region is the one reported
    value, total_ms, per_launch_ms = rates[mid], regions[mid][0], regions[mid][1]
    bytes_per_launch = region_bytes(flags_per_region[mid])
    peak, peak_kind = measured_peak()
    # the dominant (only) kernel of the timed region: mean over every launch of every region
    all_ms = [ms for _, steps in regions for ms in steps]
    all_bytes = [b for f in flags_per_region for b in region_bytes(f)]
    achieved = (sum(all_bytes) / len(all_bytes)) / (statistics.mean(all_ms) * 1e-3) / 1e9
    by_flags = {}
    for f, (_, steps) in zip(flags_per_region, regions):
        for fl, ms in zip(f, steps):
            by_flags.setdefault(fl & 6, []).append(ms)
    names = {0: "plain", 2: "refresh", 4: "pull", 6: "refresh+pull"}
    per_kind = {names[fl]: {"launches": len(ms), "ms_median": statistics.median(ms),
                            "gbs": step_bytes_per_param(K, sg, fl, args.shared_pre, args.local_sgd, args.merged_dev) * N
                            / (statistics.median(ms) * 1e-3) / 1e9}
                for fl, ms in sorted(by_flags.items())}
    traffic = None
    plain_config = not (args.shared_pre or args.local_sgd or args.per_tensor or args.threads or args.blocks_per_sm
                        or args.merged_dev)
    if NCU_TRAFFIC["digest"] == kernel_digest() and NCU_TRAFFIC["K"] == K and plain_config:
        per = NCU_TRAFFIC["bytes_per_param"]
        kinds = [f & 6 for fl in flags_per_region for f in fl]
        if all(kd in per for kd in kinds):
            traffic = statistics.mean(per[kd] for kd in kinds) * N

    line = {
        "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
        "warmup": warm, "ms_per_step": total_ms / args.steps, "higher_is_better": True,
        "scaling": "weak", "vs_baseline": None, "dtype": "f32", "data": "synthetic",
        "repeats": {"count": repeats, "reported": "median", "value_min": min(rates), "value_max": max(rates),
                    "timed_ms_total": sum(ms for ms, _ in regions)},
        "params_per_s": whole_job_rate(float(N) * args.steps, world, total_ms),
        "frac_of_nominal_8TBs": value / world / NOMINAL_HBM_GBS,
        "wall_ms_per_step": t_wall / (args.steps * repeats) * 1e3,
        "config": {"workload": wl_name, "layout": wl["layout"], "params": lay.numel, "tensors": lay.num_tensors,
                   "workers": K, "delay_k": wl["k"], "ssd_warmup_iters": wl["W"], "grad_dtype": "f32",
                   "stage": "steps-delay", "kernel": "fused ssd_step", "replicas": world,
                   "hyper_parameters": "per tensor" if args.per_tensor else "uniform",
                   "pre_weight": "one shared buffer" if args.shared_pre else "one buffer per worker",
                   "local_updater": "sgd" if args.local_sgd else "glu",
                   "device_weights": "the local weights (no separate buffers)" if args.merged_dev
                   else "one buffer per worker",
                   "device_bytes": state_bytes + n_sets * K * N * sg, "l2": l2_note},
        "clocks": clocks,
        "gpu_launches": args.steps, "gpu_launches_all_repeats": launches,
        "roofline": {"bound": "hbm", "kernel": "step_kernel (pull iterations: sync_kernel)" if args.merged_dev
                     else "step_kernel", "achieved": achieved, "peak": peak,
                     "unit": "GB/s", "frac": achieved / peak, "peak_kind": peak_kind, "traffic": traffic,
                     "traffic_source": None if traffic is None else
                     f"ncu DRAM counters on {NCU_TRAFFIC['captured_params']} parameters, scaled by parameter count",
                     "algorithmic_bytes_per_launch": sum(all_bytes) / len(all_bytes),
                     "launch_ms": {"mean": statistics.mean(all_ms), "min": min(all_ms), "max": max(all_ms)},
                     "by_iteration_kind": per_kind},
    }

    # ---- launch-bound workloads: one schedule period replayed from a CUDA graph ----
    if state_bytes <= 4 * 126e6 and not args.no_graph:
        k = wl["k"]
        it, lu, _, _ = st.ctx.ssd_get_counters()
        graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
        with torch.cuda.graph(graph, stream=side):
            for j in range(k):
                st.ctx.ssd_step(grad_sets[j % n_sets])
        g_flags = [st.ctx.ssd_schedule(it + j)[1] for j in range(k)]
        periods = max(1, args.steps // k) * 10

        def replay():
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(periods):
                graph.replay()
            e1.record(stream)
            return [e0, e1]
        replay()
        g_ms = time_regions(replay, 1, world, dev_name)[0][0]
        # the counters moved at capture time only: account for the replayed periods
        st.ctx.ssd_set_counters(it + k * (2 * periods + 1), lu + k * (2 * periods + 1))
        g_bytes = float(sum(step_bytes_per_param(K, sg, f, args.shared_pre, args.local_sgd) * N for f in g_flags)) * periods
        line["graph_replay"] = {"ms_per_step": g_ms / (periods * k), "value": whole_job_rate(g_bytes, world, g_ms) / 1e9,
                                "unit": UNIT, "steps_per_graph": k, "replays": periods,
                                "note": "one schedule period of fused steps captured once and replayed"}

    # ---- end to end: gradients arrive in pinned host memory, the new global weight is read back ----
    def e2e_run(state, host_grads, staging, host_w, host_pre):
        """Times --e2e-steps calls of ssd_step_host (one untimed call first); host_grads None =
        the gradients stay on the device."""
        state.ctx.ssd_step_host(host_grads, staging, host_w)
        torch.cuda.synchronize()
        it0 = state.ctx.ssd_get_counters()[0]
        e_flags = [state.ctx.ssd_schedule(it0 + n)[1] for n in range(args.e2e_steps)]

        def run():
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            for _ in range(args.e2e_steps):
                state.ctx.ssd_step_host(host_grads, staging, host_w)
            e1.record(stream)
            return [e0, e1]
        e_ms = time_regions(run, 1, world, dev_name)[0][0]
        shared = args.shared_pre or host_pre
        e_bytes = float(sum(step_bytes_per_param(K, sg, f, shared, args.local_sgd) * N for f in e_flags))
        moved = [host_step_bytes(K, sg, f, True, host_grads is not None, host_pre, host_w is not None)
                 for f in e_flags]
        return {"value": whole_job_rate(e_bytes, world, e_ms) / 1e9, "unit": UNIT,
                "h2d_bytes_per_step": statistics.mean(m[0] for m in moved) * N,
                "d2h_bytes_per_step": statistics.mean(m[1] for m in moved) * N,
                "steps": args.e2e_steps, "ms_per_step": e_ms / args.e2e_steps, "call": "ssd_step_host"}

    cpu_sample = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        n_sample = min(N, 1 << 23)                # the oracle's inputs: host copies of the same gradients
        cpu_sample = ([[g[:n_sample].cpu().numpy() for g in gs] for gs in grad_sets], w0[:n_sample].cpu().numpy())

    e2e = host_pre_legs = None
    if args.e2e_steps > 0:
        host_grads = [torch.empty(N, dtype=torch.float32).pin_memory() for _ in range(K)]
        for i in range(K):
            host_grads[i].copy_(grad_sets[0][i])
        host_w = torch.empty(N, dtype=torch.float32).pin_memory()
        staging = grad_sets[1]
        e2e = e2e_run(st, host_grads, staging, host_w, False)
        e2e["pre_weight"] = line["config"]["pre_weight"] + ", in device memory"
        if not args.no_host_pre and not args.local_sgd:
            # the same workload with pre_weight in ONE pinned host arena (Section 3.5 of the paper)
            device_pre_bytes = (1 if args.shared_pre else K) * N * 4
            del st
            torch.cuda.empty_cache()
            st = DeviceState(lay.numels, hp, w0, device=dev_name, fill=0.0, host_pre=True, pre_slots=3)
            if args.per_tensor:
                st.ctx.ssd_set_tensor_scales(None, [1.0 if kind == "he" else 0.0 for kind in lay.kinds], table)
            for n in range(wl["W"] + 1):              # SSD warm-up stage and the first GLU call
                st.ctx.ssd_step_host(None, grad_sets[n % n_sets], None)
            host_pre_legs = {
                "pre_weight": "one pinned host arena, streamed through 3 device slices of 2^24 elements",
                "device_bytes_saved": device_pre_bytes - st.pre_slices.numel() * 4,
                "host_gradients": e2e_run(st, host_grads, staging, host_w, True),
                # gradients already on the device: only pre_weight crosses the bus; compare with ms_per_step
                "device_gradients": e2e_run(st, None, grad_sets[0], None, True)}
        del host_grads, host_w
    line["e2e"] = e2e
    if host_pre_legs:
        line["e2e_host_pre_weight"] = host_pre_legs

    # ---- every kernel on two more workloads (single-GPU runs only) ----
    if world == 1 and not args.no_kernel_table:
        del st, grad_sets
        torch.cuda.empty_cache()
        line["kernels"] = kernel_table(peak)

    # ---- the CPU oracle on the host cores, bounded sample (rank 0, single GPU runs only) ----
    if cpu_sample is not None:
        g_host, w_host = cpu_sample
        o_steps = 2 * wl["k"]
        dt, moved, params, cores = oracle_sample_run(wl, n_sample, o_steps, g_host, w_host)
        line["cpu_baseline"] = {
            "value": moved / dt / 1e9, "unit": UNIT, "cores": cores, "kind": "oracle",
            "host_cores": os.cpu_count(), "params_per_s": params / dt, "ms_per_step_sample": dt / o_steps * 1e3,
            "sample": f"first {n_sample} of {N} arena elements, all {K} workers, {o_steps} delay-stage steps"}
        threads = os.cpu_count() or 1
        if threads > 1:
            dt_all = oracle_all_cores_run(wl, n_sample, o_steps, g_host, w_host, threads)
            line["cpu_baseline"]["all_cores"] = {"value": moved / dt_all / 1e9, "unit": UNIT, "cores": threads,
                                                 "params_per_s": params / dt_all}

    if rank == 0:
        print(json.dumps(line))
    if world > 1:
        import torch.distributed as dist
        dist.barrier()
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
