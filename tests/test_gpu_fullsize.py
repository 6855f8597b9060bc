"""The full-size configurations on the GPU, in the launch shape the benchmark times.

Where the oracle cannot sweep every element in seconds, it follows a sample of arena elements
through the whole schedule: the update is elementwise in the parameter index, so the oracle run on
the gathered elements (same hyper-parameters, same gradients at those indices) is the exact
expected value for those positions of the full-size GPU result.  Samples hold every tensor's first
and last element, the elements around every padding gap, both ends of the arena and a seeded
random draw.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2012_05396_b200 import binding as B
from paper_2012_05396_b200 import synth
from paper_2012_05396_b200.state import DeviceState
from tests.gpu_common import assert_same, compare_states, make_hp, oracle_grad

pytestmark = pytest.mark.gpu


def sample_indices(lay, n_random=4096, seed=5):
    N = lay.padded_numel
    picks = [np.arange(0, min(N, 64)), np.arange(max(0, N - 64), N)]
    for off, cnt in zip(lay.offsets, lay.numels):
        edge = np.array([off, off + 1, off + cnt - 2, off + cnt - 1, off + cnt, off + cnt + 1, off - 1])
        picks.append(edge[(edge >= 0) & (edge < N)])
    picks.append(np.random.default_rng(seed).integers(0, N, n_random))
    return np.unique(np.concatenate(picks)).astype(np.int64)


def run_sampled(layout_name, K, W, k, iters, sigma, lr, m, per_tensor=False):
    lay = synth.get_layout(layout_name)
    ohp, chp = make_hp(K, lr, m, W, k, wd=5e-4 if per_tensor else 0.0)
    idx = sample_indices(lay)
    tidx = torch.from_numpy(idx)
    w0 = synth.init_weights(lay, device="cuda")
    dev = DeviceState(lay.numels, chp, w0)
    if per_tensor:
        # no weight decay on BN and bias tensors, a tenth of the learning rate on the classifier
        wd_mult = [1.0 if kind == "he" else 0.0 for kind in lay.kinds]
        lr_mult = [0.1 if name.startswith("fc") else 1.0 for name in lay.names]
        ends = [lay.offsets[t + 1] if t + 1 < lay.num_tensors else lay.padded_numel
                for t in range(lay.num_tensors)]
        ohp.set_tensor_scales(ends, lr_mult, wd_mult, arena_index=idx)
        table = torch.empty(dev.ctx.ssd_tensor_table_bytes(), dtype=torch.uint8, device="cuda")
        dev.ctx.ssd_set_tensor_scales(lr_mult, wd_mult, table)
    ref = oracle.State(ohp, w0[tidx.cuda()].cpu().numpy())
    mask = synth.valid_mask(lay, "cuda") if lay.padded_numel != lay.numel else None
    for n in range(iters):
        grads = [synth.gradient(lay, n, i, sigma, device="cuda", mask=mask) for i in range(K)]
        dev.ctx.ssd_step(grads)
        ref.step([synth.gradient_at(lay, n, i, sigma, tidx).numpy() for i in range(K)])
        del grads
    torch.cuda.synchronize()
    compare_states(dev, ref, f"{layout_name} K={K} k={k}", idx=idx)
    assert dev.ctx.ssd_kernel_launches() == iters
    # the sample really is the full-size run's data: weights of the sampled positions came from
    # the device arena, gradients from the same counter-based stream
    g = synth.gradient(lay, 0, 0, sigma, device="cuda", mask=mask)
    assert torch.equal(g[tidx.cuda()].cpu(), synth.gradient_at(lay, 0, 0, sigma, tidx))


def test_config_resnet50_K8_every_element():
    # ResNet-50 layout (25.6M parameters, 161 tensors), K=8, sigma 1e-3, W=8, k=4, 50 iterations
    lay = synth.get_layout("resnet50")
    K, W, k, iters = 8, 8, 4, 50
    ohp, chp = make_hp(K, 0.1, 0.9, W, k)
    w0 = synth.init_weights(lay, device="cuda")
    dev = DeviceState(lay.numels, chp, w0)
    ref = oracle.State(ohp, w0.cpu().numpy())
    for n in range(iters):
        grads = [synth.gradient(lay, n, i, 1e-3, device="cuda") for i in range(K)]
        dev.ctx.ssd_step(grads)
        ref.step([g.cpu().numpy() for g in grads])
        if n in (W - 1, W, W + k - 1, W + k):
            torch.cuda.synchronize()
            compare_states(dev, ref, f"resnet50 iter {n}")
    torch.cuda.synchronize()
    compare_states(dev, ref, "resnet50 final")


@pytest.mark.parametrize("k", [2, 8])
def test_config_resnet50_K8_other_delays_sampled(k):
    run_sampled("resnet50", 8, 8, k, 50, 1e-3, 0.1, 0.9)


def test_config_resnet50_K8_per_tensor_hyper_parameters_sampled():
    run_sampled("resnet50", 8, 8, 4, 24, 1e-3, 0.1, 0.9, per_tensor=True)


class ThreadedOracle:
    """The CPU oracle, as it stands, run by several host threads on disjoint element ranges of one
    slice (the update is elementwise in the parameter index; the C calls release the interpreter lock)."""

    def __init__(self, ohp, w0_slice, threads):
        from concurrent.futures import ThreadPoolExecutor
        n = w0_slice.shape[0]
        self.bounds = [n * t // threads for t in range(threads + 1)]
        self.parts = [oracle.State(ohp, w0_slice[lo:hi]) for lo, hi in zip(self.bounds, self.bounds[1:])]
        self.pool = ThreadPoolExecutor(threads)

    def step(self, grads):
        def one(t):
            lo, hi = self.bounds[t], self.bounds[t + 1]
            return self.parts[t].step([g[lo:hi] for g in grads])
        return list(self.pool.map(one, range(len(self.parts))))[0]

    def buffer(self, name, worker=None):
        pick = (lambda st: getattr(st, name)) if worker is None else (lambda st: getattr(st, name)[worker])
        return np.concatenate([pick(st) for st in self.parts])

    def close(self):
        self.pool.shutdown()


def test_config_vgg16_K16_every_element():
    # VGG-16 layout (138M parameters), K=16, sigma 1e-3, lr 0.01, m 0.9, W=4, k=4, 20 iterations: the
    # workload and launch shape bench.py times.  The GPU runs the whole schedule at full size; then the
    # oracle follows EVERY element through the same schedule, one slice of 2^24 elements at a time
    # (gradients regenerated for the slice from the counter-based stream, host memory bounded), and all
    # 2 + 3K buffers of the slice are compared bit for bit.
    import os
    K, W, k, iters, sigma = 16, 4, 4, 20, 1e-3
    lay = synth.get_layout("vgg16")
    N = lay.padded_numel
    need = ((2 + 4 * K) * N * 4 + (8 << 30))
    if torch.cuda.mem_get_info()[0] < need:
        pytest.skip("not enough free device memory for the VGG-16 K=16 state")
    ohp, chp = make_hp(K, 0.01, 0.9, W, k)
    w0 = synth.init_weights(lay, device="cuda")
    dev = DeviceState(lay.numels, chp, w0)
    mask = synth.valid_mask(lay, "cuda") if N != lay.numel else None
    for n in range(iters):
        grads = [synth.gradient(lay, n, i, sigma, device="cuda", mask=mask) for i in range(K)]
        dev.ctx.ssd_step(grads)
        del grads
    torch.cuda.synchronize()
    assert dev.ctx.ssd_kernel_launches() == iters and dev.guards_intact()

    threads = max(1, len(os.sched_getaffinity(0)))
    slice_elems = 1 << 24
    keys = [[synth.stream_key(synth.SEED, synth.STREAM_GRAD, n, i) for i in range(K)] for n in range(iters)]
    stage_buf = torch.empty((K, slice_elems), dtype=torch.float32).pin_memory()
    compared = 0
    for lo in range(0, N, slice_elems):
        hi = min(N, lo + slice_elems)
        idx = torch.arange(lo, hi, dtype=torch.int64, device="cuda")
        ref = ThreadedOracle(ohp, w0[lo:hi].cpu().numpy(), threads)
        host = stage_buf[:, :hi - lo]
        for n in range(iters):
            for i in range(K):
                g = synth.normal_at(keys[n][i], idx, sigma)
                if mask is not None:
                    g = g * mask[lo:hi]
                host[i].copy_(g, non_blocking=True)
            torch.cuda.synchronize()
            ref.step([host[i].numpy() for i in range(K)])
        tag = f"vgg16 K=16 elements [{lo}, {hi})"
        assert_same(dev.w[lo:hi], ref.buffer("w"), tag + " w")
        assert_same(dev.mom[lo:hi], ref.buffer("mom"), tag + " mom")
        for i in range(K):
            for name in ("w_loc", "pre", "w_dev"):
                assert_same(getattr(dev, name)[i][lo:hi], ref.buffer(name, i), f"{tag} {name}[{i}]")
        assert (ref.parts[0].iter, ref.parts[0].loc_update) == dev.ctx.ssd_get_counters()[:2]
        ref.close()
        compared += hi - lo
    assert compared == N
    # the regenerated slices really are the full-size run's gradients
    g = synth.gradient(lay, 3, 5, sigma, device="cuda", mask=mask)
    idx = torch.arange(N - 4096, N, dtype=torch.int64, device="cuda")
    assert torch.equal(g[N - 4096:], synth.normal_at(keys[3][5], idx, sigma) * (1 if mask is None else mask[N - 4096:]))


def sweep_buffer(stream, n, worker, device, idx=None):
    """One uniform(-1,1) buffer of the bandwidth sweep; only its elements at `idx` when given."""
    if idx is None:
        return synth.uniform_buffer(stream, n, worker=worker, device=device)
    return synth.uniform_at(synth.stream_key(synth.SEED, stream, 0, worker), idx)


def sweep_point(n, K, bf16, glu_flags, sampled):
    """One server update, then one GLU update per worker, from primed uniform(-1,1) state."""
    ohp, chp = make_hp(K, 0.1, 0.9, 0, 4, bf16=bf16)
    idx = tidx = None
    if sampled:
        idx = np.unique(np.concatenate([np.arange(64), np.arange(n - 64, n),
                                        np.random.default_rng(n + K).integers(0, n, 4096)])).astype(np.int64)
        tidx = torch.from_numpy(idx)

    def host(stream, worker=0):
        """The oracle's copy of a buffer: the sampled elements, or all of them."""
        return sweep_buffer(stream, n, worker, "cpu", tidx).numpy().copy()

    # the device state is filled in place, one buffer at a time (the largest points nearly fill the GPU)
    dev = DeviceState([n], chp, sweep_buffer(synth.STREAM_WEIGHT, n, 0, "cuda"))
    dev.mom.copy_(sweep_buffer(synth.STREAM_MOM, n, 0, "cuda"))
    grads = []
    for i in range(K):
        dev.w_loc[i].copy_(sweep_buffer(synth.STREAM_WLOC, n, i, "cuda"))
        dev.pre[i].copy_(sweep_buffer(synth.STREAM_PRE, n, i, "cuda"))
        g = sweep_buffer(synth.STREAM_GRAD, n, i, "cuda")
        grads.append(synth.to_bf16(g) if bf16 else g)
    ref = oracle.State(ohp, host(synth.STREAM_WEIGHT))
    ref.mom[:] = host(synth.STREAM_MOM)
    ref_grads = []
    for i in range(K):
        ref.w_loc[i][:] = host(synth.STREAM_WLOC, i)
        ref.pre[i][:] = host(synth.STREAM_PRE, i)
        g = sweep_buffer(synth.STREAM_GRAD, n, i, "cpu", tidx)
        ref_grads.append(oracle_grad(synth.to_bf16(g) if bf16 else g, bf16))
    dev.ctx.ssd_server_sync_update(grads)
    oracle.server_update(ohp, ref_grads, ref.w, ref.mom)
    for i in range(K):
        dev.ctx.ssd_worker_glu_update(i, grads[i], glu_flags)
        oracle.glu_update(ohp, ref_grads[i], ref.w_loc[i], ref.pre[i], ref.w_dev[i], ref.w, glu_flags)
    torch.cuda.synchronize()
    tag = f"sweep n={n} K={K} bf16={bf16} flags={glu_flags}"
    assert_same(dev.w, ref.w, tag + " w", idx)
    assert_same(dev.mom, ref.mom, tag + " mom", idx)
    for i in range(K):
        for name in ("w_loc", "pre", "w_dev"):
            assert_same(getattr(dev, name)[i], getattr(ref, name)[i], f"{tag} {name}[{i}]", idx)


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("K", [1, 4, 16, 32])
def test_sweep_points_every_element(K, bf16):
    for n in (1 << 16, 1 << 20):
        sweep_point(n, K, bf16, 0, sampled=False)


@pytest.mark.parametrize("bf16", [False, True])
def test_sweep_refresh_and_pull_variants(bf16):
    sweep_point(1 << 22, 4, bf16, B.SSD_FLAG_REFRESH, sampled=False)
    sweep_point(1 << 22, 4, bf16, B.SSD_FLAG_PULL, sampled=False)
    sweep_point(1 << 26, 4, bf16, B.SSD_FLAG_REFRESH | B.SSD_FLAG_PULL, sampled=True)


@pytest.mark.parametrize("K,bf16", [(4, False), (32, True), (32, False)])
def test_sweep_largest_size_sampled(K, bf16):
    n = 1 << 28
    torch.cuda.empty_cache()
    need = ((2 + 4 * K) * 4 + K * (2 if bf16 else 4)) * n + (8 << 30)      # state, gradients, generator scratch
    if torch.cuda.mem_get_info()[0] < need:
        pytest.skip(f"needs {need / 2**30:.0f} GiB of free device memory")
    sweep_point(n, K, bf16, 0, sampled=True)


def test_step_host_in_chunks_equals_one_step():
    # An arena longer than one 2^24-element chunk: ssd_step_host pipelines two chunks over its side
    # streams and must leave exactly the state of ssd_step on device-resident gradients (which the
    # tests above tie to the oracle), also with per-tensor scalars, whose lookup depends on position.
    lay = synth.get_layout("resnet50")
    K, W, k = 2, 1, 2
    _, chp = make_hp(K, 0.1, 0.9, W, k, wd=5e-4)
    w0 = synth.init_weights(lay, device="cuda")
    a, b = DeviceState(lay.numels, chp, w0), DeviceState(lay.numels, chp, w0)
    wd_mult = [1.0 if kind == "he" else 0.0 for kind in lay.kinds]
    lr_mult = [0.5 if name.startswith("s3") else 1.0 for name in lay.names]
    tables = [torch.empty(s.ctx.ssd_tensor_table_bytes(), dtype=torch.uint8, device="cuda") for s in (a, b)]
    a.ctx.ssd_set_tensor_scales(lr_mult, wd_mult, tables[0])
    b.ctx.ssd_set_tensor_scales(lr_mult, wd_mult, tables[1])
    staging = [torch.empty(b.n, dtype=torch.float32, device="cuda") for _ in range(K)]
    w_out = torch.empty(b.n, dtype=torch.float32).pin_memory()
    chunks = -(-b.n // (1 << 24))
    assert chunks == 2
    for n in range(5):
        grads = [synth.gradient(lay, n, i, 1e-3, device="cuda") for i in range(K)]
        host = [g.cpu().pin_memory() for g in grads]
        a.ctx.ssd_step(grads)
        b.ctx.ssd_step_host(host, staging, w_out)
        torch.cuda.synchronize()
        assert torch.equal(w_out.view(torch.int32), a.w.cpu().view(torch.int32)), f"w_out iter {n}"
    for name in ("w", "mom"):
        assert torch.equal(getattr(a, name).view(torch.int32), getattr(b, name).view(torch.int32)), name
    for i in range(K):
        for name in ("w_loc", "pre", "w_dev"):
            assert torch.equal(getattr(a, name)[i].view(torch.int32), getattr(b, name)[i].view(torch.int32)), name
    assert b.ctx.ssd_kernel_launches() == 5 * chunks and a.ctx.ssd_get_counters()[:2] == b.ctx.ssd_get_counters()[:2]
