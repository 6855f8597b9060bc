"""Bandwidth sweep of the three update kernels on a flat parameter buffer.

    python -m paper_2012_05396_b200.sweep --log2n 16 20 24 26 28 --K 1 4 16 32 --dtype f32 bf16

For every point it times, with CUDA events on the launching stream (3 warm-up + `--reps` timed
launches, median and minimum reported):
    sync    ssd_server_sync_update               K*sg + 16 bytes per parameter
    glu     ssd_worker_glu_update, plain flags   sg + 12 bytes per parameter and worker
    step    ssd_step in the steps-delay stage    K*(sg+12) + 16 (+4K on refresh, +4K on pull)
    step_merged  the same for a context without separate device weights: only its pull iterations
            differ (server update + K stores of the new global weight, K*(sg+4) + 16) and only they
            are reported
and prints one JSON object per point.  State and gradients are uniform(-1,1) from the seeded
generators.  Points whose footprint is below 1 GB rotate over several independent buffer sets (at
least 1 GB together), so that a launch never finds its data in the 126 MB L2 left by the previous
one; points below four times the L2 size are still marked "l2" (they last microseconds and show
launch latency).  Points that do not fit in free device memory are reported as skipped.
"""
from __future__ import annotations

import argparse
import json
import statistics
import sys

import torch

from . import binding as B
from . import build as libbuild
from . import synth
from .state import DeviceState, alloc_arenas

L2_BYTES = 126e6


def measured_peak() -> float:
    """The HBM copy rate measured on this machine (MEASURED_PEAKS.json at the repository root), else the
    earlier measurement of 6650 GB/s."""
    import os
    path = os.path.join(os.path.dirname(os.path.dirname(os.path.abspath(__file__))), "MEASURED_PEAKS.json")
    try:
        with open(path) as fh:
            return float(json.load(fh)["hbm_gbs"])
    except Exception:
        return 6650.0


def time_launches(fn, reps: int, warmup: int = 3):
    stream = torch.cuda.current_stream()
    for _ in range(warmup):
        fn()
    ev = [torch.cuda.Event(enable_timing=True) for _ in range(reps + 1)]
    torch.cuda.synchronize()
    ev[0].record(stream)
    for r in range(reps):
        fn()
        ev[r + 1].record(stream)
    torch.cuda.synchronize()
    ms = [ev[r].elapsed_time(ev[r + 1]) for r in range(reps)]
    return statistics.median(ms), min(ms)


def _grads(n, K, dtype):
    out = alloc_arenas(K, n, torch.bfloat16 if dtype == "bf16" else torch.float32)
    for i in range(K):
        g = synth.uniform_buffer(synth.STREAM_GRAD, n, worker=i, device="cuda")
        g.mul_(1e-3)                     # keeps the state bounded over many repetitions
        out[i].copy_(g)                  # rounds to nearest even for bfloat16
    return out


def _hp(K, k, dtype):
    nan = float("nan")
    return B.make_hparams(K, 0.1, 0.9, 0, k, lr_local=nan, alpha=nan, beta=nan, rescale=nan,
                          grad_dtype=B.SSD_BF16 if dtype == "bf16" else B.SSD_F32)


def _fits(nbytes):
    torch.cuda.empty_cache()             # blocks cached from the previous point count as free
    free, _ = torch.cuda.mem_get_info()
    return nbytes * 1.03 + (1 << 30) <= free


def point(log2n: int, K: int, dtype: str, kernels, reps: int, peak: float, threads: int = 0, bps: int = 0,
          vw: int = 0, batch: int = 0, staging: int = 0, numels=None):
    """One sweep point: a flat tensor of 2^log2n elements, or the tensor list `numels` of a model
    layout (log2n is then only a label)."""
    numels = [1 << log2n] if numels is None else [int(x) for x in numels]
    n = B.ssd_arena_numel(numels)
    sg = 2 if dtype == "bf16" else 4
    out = []

    def emit(kernel, footprint, bytes_per_launch, med, mn):
        gbs = bytes_per_launch / (med * 1e-3) / 1e9
        out.append({"log2n": log2n, "params": n, "K": K, "grad_dtype": dtype, "kernel": kernel,
                    "footprint_bytes": footprint, "l2": footprint < 4 * L2_BYTES,
                    "bytes_per_launch": bytes_per_launch, "ms_median": med, "ms_min": mn, "gbs": gbs,
                    "gbs_best": bytes_per_launch / (mn * 1e-3) / 1e9, "frac_of_8TBs": gbs / 8000.0,
                    "frac_of_measured": gbs / peak, "params_per_s": n / (med * 1e-3)})

    def skip(kernel, footprint):
        out.append({"log2n": log2n, "K": K, "grad_dtype": dtype, "kernel": kernel,
                    "footprint_bytes": footprint, "skipped": "does not fit in free device memory"})

    def tune(st):
        if threads or bps:
            st.ctx.ssd_set_launch(threads, bps)
        if vw or batch:
            st.ctx.ssd_set_kernel_shape(vw, batch)
        if staging:
            st.ctx.ssd_set_staging(staging)       # fused step through the shared-memory ring

    def copies(footprint):
        """Independent buffer sets to rotate over, so that no launch finds its data in the 126 MB L2:
        at least 1 GB in total (at most 8 sets)."""
        return max(1, min(8, -(-int(1e9) // footprint)))

    w0 = synth.uniform_buffer(synth.STREAM_WEIGHT, n, device="cuda")
    if "sync" in kernels:
        # the server alone: a context without a delay stage needs no worker state
        fp = 2 * n * 4 + K * n * sg
        R = copies(fp)
        if _fits(fp * R):
            sets = []
            for _ in range(R):
                st = DeviceState(numels, _hp(K, 0, dtype), w0, worker_state=False)
                tune(st)
                sets.append((st, _grads(n, K, dtype)))
            turn = {"i": 0}

            def sync():
                st, grads = sets[turn["i"]]
                st.ctx.ssd_server_sync_update(grads)
                turn["i"] = (turn["i"] + 1) % R
            med, mn = time_launches(sync, reps)
            emit("sync", fp, (K * sg + 16) * n, med, mn)
            del sets
        else:
            skip("sync", fp)
    if "glu" in kernels:
        # one launch updates one worker, so the worker count does not enter; rotate over the buffers
        # of enough workers that consecutive launches never touch the same memory
        fp1 = 3 * n * 4 + n * sg                     # one worker's buffers
        Kg = max(min(K, 4), min(8, -(-int(1e9) // fp1)))
        fp = (2 + 3 * Kg) * n * 4 + Kg * n * sg
        if _fits(fp):
            st = DeviceState(numels, _hp(Kg, 4, dtype), w0, fill=0.0)
            tune(st)
            grads = _grads(n, Kg, dtype)
            for i in range(Kg):
                st.pre[i].copy_(st.w_loc[i])
            state = {"i": 0}

            def glu():
                i = state["i"]
                st.ctx.ssd_worker_glu_update(i, grads[i], 0)
                state["i"] = (i + 1) % Kg
            med, mn = time_launches(glu, reps)
            emit("glu", fp, (sg + 12) * n, med, mn)
            del st, grads
        else:
            skip("glu", fp)
    for merged in (False, True):
        if ("step_merged" if merged else "step") not in kernels:
            continue
        fp = (2 + (2 if merged else 3) * K) * n * 4 + K * n * sg
        R = copies(fp)
        if _fits(fp * R):
            sets = []
            for _ in range(R):
                st = DeviceState(numels, _hp(K, 4, dtype), w0, fill=0.0, merged_dev=merged)
                tune(st)
                grads = _grads(n, K, dtype)
                st.ctx.ssd_step(grads)                               # first GLU call
                sets.append((st, grads))
            stream = torch.cuda.current_stream()
            per_flag = {}
            total = R * (4 + max(reps, 8))                           # every set goes through the same schedule
            ev = [torch.cuda.Event(enable_timing=True) for _ in range(total + 1)]
            flags_of = []
            ev[0].record(stream)
            for r in range(total):                                   # enqueued back to back, as a training loop does
                st, grads = sets[r % R]
                flags_of.append(st.ctx.ssd_get_counters()[3])
                st.ctx.ssd_step(grads)
                ev[r + 1].record(stream)
            torch.cuda.synchronize()
            for r in range(4 * R, total):
                per_flag.setdefault(flags_of[r], []).append(ev[r].elapsed_time(ev[r + 1]))
            for flags, ms in sorted(per_flag.items()):
                b = K * (sg + 12) + 16 + (4 * K if flags & 2 else 0) + (4 * K if flags & 4 else 0)
                name = "step" + ("+refresh" if flags & 2 else "") + ("+pull" if flags & 4 else "")
                if merged:
                    if not flags & 4:
                        continue                                     # the other iterations are the plain form's
                    b, name = K * (sg + 4) + 16, "step+pull (merged device weights)"
                emit(name, fp, b * n, statistics.median(ms), min(ms))
            del sets
            st = grads = None                                        # the loop variables still held the last set
        else:
            skip("step_merged" if merged else "step", fp)
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--log2n", type=int, nargs="+", default=[16, 18, 20, 22, 24, 26, 28])
    ap.add_argument("--K", type=int, nargs="+", default=[1, 4, 16, 32])
    ap.add_argument("--dtype", nargs="+", default=["f32", "bf16"], choices=["f32", "bf16"])
    ap.add_argument("--kernels", nargs="+", default=["sync", "glu", "step"], choices=["sync", "glu", "step", "step_merged"])
    ap.add_argument("--reps", type=int, default=20)
    ap.add_argument("--peak", type=float, default=0.0,
                    help="HBM copy rate in GB/s for the 'of measured' column (0 = read MEASURED_PEAKS.json, "
                         "else the pool's earlier figure of 6650)")
    ap.add_argument("--threads", type=int, default=0)
    ap.add_argument("--blocks-per-sm", type=int, default=0)
    ap.add_argument("--vector-elems", type=int, default=0, choices=[0, 4, 8, 16])
    ap.add_argument("--batch", type=int, default=0, choices=[0, 1, 2, 4, 8])
    ap.add_argument("--staging", type=int, default=0,
                    help="stages of the shared-memory ring for the fused step (0 = register path)")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("the sweep needs a CUDA device")
    libbuild.build_library()
    if args.peak <= 0:
        args.peak = measured_peak()
    for log2n in args.log2n:
        for K in args.K:
            for dtype in args.dtype:
                for rec in point(log2n, K, dtype, args.kernels, args.reps, args.peak, args.threads,
                                 args.blocks_per_sm, args.vector_elems, args.batch, args.staging):
                    print(json.dumps(rec), flush=True)


if __name__ == "__main__":
    main()
