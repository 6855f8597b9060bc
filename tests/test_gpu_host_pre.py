"""pre_weight kept in host memory (Section 3.5 of the paper) and the host-gradient pipeline.

ssd_step_host streams the arena through the GPU in chunks.  With ssd_set_host_pre_weight the one
pre_weight of all workers lives in a pinned host arena and travels with the gradients.  Every
result here is compared with the CPU oracle bit for bit: the oracle keeps K pre_weights, which
must all equal the one host arena.
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


def pinned(t: torch.Tensor) -> torch.Tensor:
    return t.cpu().pin_memory()


def run_host_pipeline(lay, K, W, k, iters, bf16, host_pre, chunk=0, slots=2, host_grads=True, wd=1e-3,
                      per_tensor=False, check_every=1):
    ohp, chp = make_hp(K, 0.1, 0.9, W, k, wd=wd, bf16=bf16)
    w0 = synth.init_weights(lay)
    dev = DeviceState(lay.numels, chp, w0, host_pre=host_pre, pre_slots=slots, host_chunk=chunk)
    if chunk and not host_pre:
        dev.ctx.ssd_set_host_chunk(chunk)
    if per_tensor:
        ends = [lay.offsets[t + 1] if t + 1 < lay.num_tensors else lay.padded_numel for t in range(lay.num_tensors)]
        lr_mult = [0.5 if t % 3 == 0 else 1.0 for t in range(lay.num_tensors)]
        wd_mult = [1.0 if kind == "he" else 0.0 for kind in lay.kinds]
        ohp.set_tensor_scales(ends, lr_mult, wd_mult)
        table = torch.empty(dev.ctx.ssd_tensor_table_bytes(), dtype=torch.uint8, device="cuda")
        dev.ctx.ssd_set_tensor_scales(lr_mult, wd_mult, table)
    ref = oracle.State(ohp, w0.numpy())
    gdtype = torch.bfloat16 if bf16 else torch.float32
    staging = [torch.empty(dev.n, dtype=gdtype, device="cuda") for _ in range(K)]
    w_out = torch.empty(dev.n, dtype=torch.float32).pin_memory()
    seen = set()
    for n in range(iters):
        grads = [synth.gradient(lay, n, i, 1e-2, device="cuda") for i in range(K)]
        if bf16:
            grads = [synth.to_bf16(g) for g in grads]
        if host_grads:
            host = [pinned(g) for g in grads]
            dev.ctx.ssd_step_host(host, staging, w_out)
        else:                                   # gradients already on the device: only pre_weight and w travel
            for s, g in zip(staging, grads):
                s.copy_(g)
            dev.ctx.ssd_step_host(None, staging, w_out)
        stage, flags = ref.step([oracle_grad(g, bf16) for g in grads])
        seen.add((stage, flags))
        if (n + 1) % check_every == 0 or n == iters - 1:
            torch.cuda.synchronize()
            tag = f"iter {n} stage {stage} flags {flags}"
            assert_same(w_out, ref.w, tag + " w read back")
            compare_states(dev, ref, tag)
    chunks = -(-dev.n // (chunk or (1 << 24)))
    assert dev.ctx.ssd_kernel_launches() == iters * chunks
    # the schedule went through first, pull and refresh iterations
    bits_seen = 0
    for s, f in seen:
        if s == B.SSD_STAGE_DELAY:
            bits_seen |= f
    assert bits_seen & 7 == 7
    return dev, ref, chunks


@pytest.mark.parametrize("bf16", [False, True])
def test_host_pre_weight_two_full_size_chunks(bf16):
    # ResNet-50 layout: 25.6M elements = two chunks of 2^24; K=2, W=1, k=3: copy, first, plain, pull, refresh
    lay = synth.get_layout("resnet50")
    dev, ref, chunks = run_host_pipeline(lay, 2, 1, 3, 9, bf16, host_pre=True, check_every=4)
    assert chunks == 2
    assert not any(t.is_cuda for t in dev.pre)              # pre_weight never had a device arena


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("slots", [1, 2, 3])
def test_host_pre_weight_more_chunks_than_slices(bf16, slots):
    # ResNet-56 layout (0.85M elements) in chunks of 65 536: 14 chunks through 1..3 device slices, the last
    # chunk ragged; per-tensor scalars make the result depend on the arena position of every chunk
    lay = synth.get_layout("resnet56")
    dev, ref, chunks = run_host_pipeline(lay, 3, 2, 2, 10, bf16, host_pre=True, chunk=1 << 16, slots=slots,
                                         per_tensor=True)
    assert chunks == 14 and dev.n % (1 << 16) != 0


def test_host_pre_weight_with_device_resident_gradients():
    lay = synth.get_layout("resnet56")
    run_host_pipeline(lay, 4, 0, 4, 11, False, host_pre=True, chunk=1 << 17, slots=2, host_grads=False)


@pytest.mark.parametrize("bf16", [False, True])
def test_step_host_with_device_pre_weight_in_chunks(bf16):
    # the same pipeline with pre_weight in device arenas (one per worker), 2 chunks of 2^24 and many small ones
    run_host_pipeline(synth.get_layout("resnet50"), 2, 1, 2, 6, bf16, host_pre=False, check_every=3)
    run_host_pipeline(synth.get_layout("resnet56"), 3, 1, 2, 7, bf16, host_pre=False, chunk=1 << 15, per_tensor=True)


def test_host_pre_weight_k1_and_single_worker():
    # k = 1: every delay iteration pulls and (from the second on) refreshes; K = 1: one worker
    lay = synth.get_layout("resnet20")
    for K, W, k in ((1, 1, 2), (2, 0, 1), (5, 2, 1)):
        ohp, chp = make_hp(K, 0.1, 0.9, W, k, wd=1e-3)
        w0 = synth.init_weights(lay)
        dev = DeviceState(lay.numels, chp, w0, host_pre=True, pre_slots=2, host_chunk=1 << 16)
        ref = oracle.State(ohp, w0.numpy())
        staging = [torch.empty(dev.n, dtype=torch.float32, device="cuda") for _ in range(K)]
        for n in range(W + 6):
            host = [pinned(synth.gradient(lay, n, i, 1e-2)) for i in range(K)]
            dev.ctx.ssd_step_host(host, staging, None)          # no read-back of w
            ref.step([h.numpy() for h in host])
            torch.cuda.synchronize()
            compare_states(dev, ref, f"K={K} W={W} k={k} iter {n}")


def test_host_pre_weight_survives_a_checkpoint():
    # the host arena is part of the state: a new context over restored buffers continues bit for bit
    lay = synth.get_layout("resnet20")
    K, W, k = 3, 1, 3
    ohp, chp = make_hp(K, 0.1, 0.9, W, k)
    w0 = synth.init_weights(lay)
    ref = oracle.State(ohp, w0.numpy())
    a = DeviceState(lay.numels, chp, w0, host_pre=True, host_chunk=1 << 16)
    staging = [torch.empty(a.n, dtype=torch.float32, device="cuda") for _ in range(K)]

    def step(dev, n):
        host = [pinned(synth.gradient(lay, n, i, 1e-2)) for i in range(K)]
        dev.ctx.ssd_step_host(host, staging, None)
        torch.cuda.synchronize()
        return host

    for n in range(6):
        ref.step([h.numpy() for h in step(a, n)])
    it, lu, _, _ = a.ctx.ssd_get_counters()
    b = DeviceState(lay.numels, chp, a.w, host_pre=True, host_chunk=1 << 16, pre_slots=3)
    b.mom.copy_(a.mom)
    b.host_pre.copy_(a.host_pre)
    for i in range(K):
        b.w_loc[i].copy_(a.w_loc[i])
        b.w_dev[i].copy_(a.w_dev[i])
    b.ctx.ssd_set_counters(it, lu)
    for n in range(6, 13):
        ref.step([h.numpy() for h in step(b, n)])
    compare_states(b, ref, "resumed")


def test_plain_sgd_updater_needs_no_pre_weight_at_all():
    # Eq. 5 as local updater never touches pre_weight: a context created without pre_weight buffers (and
    # without a host arena) runs every delay-stage call, fused, split and through the host pipeline
    lay = synth.get_layout("resnet20")
    K, W, k = 3, 1, 2
    ohp, chp = make_hp(K, 0.1, 0.9, W, k, wd=1e-3, lr_loc=0.25, local_sgd=True)
    w0 = synth.init_weights(lay)
    full = DeviceState(lay.numels, chp, w0)                    # only for its arenas
    ctx = B.Context(lay.numels, chp, full.w, full.mom, full.w_loc, None, full.w_dev)
    ref = oracle.State(ohp, w0.numpy())
    staging = [torch.empty(full.n, dtype=torch.float32, device="cuda") for _ in range(K)]
    for n in range(9):
        grads = [synth.gradient(lay, n, i, 1e-2, device="cuda") for i in range(K)]
        if n % 3 == 0:
            ctx.ssd_step(grads)
        elif n % 3 == 1:
            ctx.ssd_server_sync_update(grads)
            for i in range(K):
                ctx.ssd_worker_local_step(i, grads[i])
            ctx.ssd_advance()
        else:
            host = [pinned(g) for g in grads]
            ctx.ssd_step_host(host, staging, None)
        torch.cuda.synchronize()
        ref.step([g.cpu().numpy() for g in grads])
    assert_same(full.w, ref.w, "w")
    assert_same(full.mom, ref.mom, "mom")
    for i in range(K):
        assert_same(full.w_loc[i], ref.w_loc[i], f"w_loc[{i}]")
        assert_same(full.w_dev[i], ref.w_dev[i], f"w_dev[{i}]")
    assert full.guards_intact()


def test_random_host_pipelines():
    # seeded draw over arena sizes, chunk sizes, slice counts, schedules, gradient types and where the
    # gradients and pre_weight live; every iteration compared with the oracle
    rng = np.random.default_rng(35)
    for case in range(16):
        T = int(rng.integers(1, 6))
        numels = [int(rng.choice([3, 100, 1000, 4099, 30000, 70001])) for _ in range(T)]
        K = int(rng.choice([1, 2, 3, 5, 8]))
        W, k = int(rng.integers(0, 3)), int(rng.integers(1, 5))
        bf16, host_pre, host_grads = bool(rng.integers(2)), bool(rng.integers(3) > 0), bool(rng.integers(2))
        chunk = int(rng.choice([1024, 4096, 1 << 15, 1 << 17]))
        slots = int(rng.integers(1, 5))
        lay = synth.Layout("t")
        for i, cnt in enumerate(numels):
            lay.add(f"x{i}", cnt, "he", 8)
        tag = f"case {case}: numels={numels} K={K} W={W} k={k} bf16={bf16} host_pre={host_pre} " \
              f"host_grads={host_grads} chunk={chunk} slots={slots}"
        ohp, chp = make_hp(K, 0.1, 0.9, W, k, wd=0.01, bf16=bf16)
        w0 = synth.init_weights(lay, seed=case)
        dev = DeviceState(lay.numels, chp, w0, host_pre=host_pre, pre_slots=slots, host_chunk=chunk)
        if not host_pre:
            dev.ctx.ssd_set_host_chunk(chunk)
        ref = oracle.State(ohp, w0.numpy())
        gdtype = torch.bfloat16 if bf16 else torch.float32
        staging = [torch.empty(dev.n, dtype=gdtype, device="cuda") for _ in range(K)]
        w_out = torch.empty(dev.n, dtype=torch.float32).pin_memory()
        for n in range(W + 2 * k + 2):
            grads = [synth.gradient(lay, n, i, 0.05, seed=case, device="cuda") for i in range(K)]
            if bf16:
                grads = [synth.to_bf16(g) for g in grads]
            if host_grads:
                host = [pinned(g) for g in grads]
                dev.ctx.ssd_step_host(host, staging, w_out)
            else:
                for s, g in zip(staging, grads):
                    s.copy_(g)
                dev.ctx.ssd_step_host(None, staging, w_out)
            ref.step([oracle_grad(g, bf16) for g in grads])
            torch.cuda.synchronize()
            assert_same(w_out, ref.w, f"{tag} iter {n} w read back")
            compare_states(dev, ref, f"{tag} iter {n}")


def test_two_contexts_on_two_host_threads_and_streams():
    # a context is used by one host thread at a time; two threads with a context and a stream each run
    # their schedules concurrently and neither disturbs the other
    import threading
    lay = synth.get_layout("resnet56")
    K, W, k, iters = 3, 1, 2, 12
    results, errors = {}, []

    def work(tid):
        try:
            torch.cuda.set_device(0)
            ohp, chp = make_hp(K, 0.1, 0.9, W, k, wd=1e-3 * (tid + 1))
            w0 = synth.init_weights(lay, seed=100 + tid)
            stream = torch.cuda.Stream()
            with torch.cuda.stream(stream):
                dev = DeviceState(lay.numels, chp, w0)
                ref = oracle.State(ohp, w0.numpy())
                for n in range(iters):
                    grads = [synth.gradient(lay, n, i, 1e-2, seed=100 + tid, device="cuda") for i in range(K)]
                    dev.ctx.ssd_step(grads, stream=stream)
                    ref.step([g.cpu().numpy() for g in grads])
                stream.synchronize()
            results[tid] = (dev, ref)
        except Exception as exc:                      # surfaced in the main thread below
            errors.append(exc)

    threads = [threading.Thread(target=work, args=(t,)) for t in range(2)]
    for t in threads:
        t.start()
    for t in threads:
        t.join()
    assert not errors, errors
    torch.cuda.synchronize()
    for tid, (dev, ref) in results.items():
        compare_states(dev, ref, f"thread {tid}")
