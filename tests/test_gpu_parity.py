"""CUDA path against the CPU oracle, element by element, through the C ABI (needs a B200)."""
import itertools

import numpy as np
import pytest
import torch

import oracle
from paper_2012_05396_b200 import binding as B
from paper_2012_05396_b200 import synth
from paper_2012_05396_b200.state import DeviceState
from tests import golden_trace
from tests.gpu_common import (assert_same, compare_states, gpu_iteration, make_hp, oracle_grad)

pytestmark = pytest.mark.gpu
f32 = np.float32


@pytest.mark.parametrize("mode", ["fused", "split"])
@pytest.mark.parametrize("name", golden_trace.ALL)
def test_hand_traces_on_the_gpu(name, mode):
    tr = golden_trace.load(name)
    h = tr.hp
    K = int(h["K"])
    _, hp = make_hp(K, h["lr"], h["m"], int(h["W"]), int(h["k"]), wd=h["wd"], lr_loc=h["lr_loc"],
                    alpha=h["alpha"], beta=h["beta"], rescale=h["rescale"])
    dev = DeviceState([len(tr.w0)], hp, torch.from_numpy(tr.w0))
    for it in tr.iters:
        stage, flags = dev.ctx.ssd_schedule(it.n)
        assert (stage, flags) == (it.stage, it.flags)
        grads = [torch.from_numpy(it.grads[i]).cuda() for i in range(K)]
        gpu_iteration(dev, grads, mode)
        torch.cuda.synchronize()
        assert dev.ctx.ssd_worker_weights(0)[1] == it.view
        for key, exp in it.server.items():
            assert_same(getattr(dev, key), exp, f"{name} iter {it.n} {key}")
        for (key, i), exp in it.worker.items():
            assert_same(getattr(dev, key)[i], exp, f"{name} iter {it.n} {key}[{i}]")


def run_both(numels, K, W, k, iters, sigma, mode, wd=0.0, bf16=False, seed=synth.SEED, lr=0.1, m=0.9,
             check_every=1, w0=None):
    ohp, chp = make_hp(K, lr, m, W, k, wd=wd, bf16=bf16)
    lay = synth.Layout("t")
    for n in numels:
        lay.add("x", n, "he", 16)
    if w0 is None:
        w0 = synth.init_weights(lay, seed)
    dev = DeviceState(lay.numels, chp, w0)
    ref = oracle.State(ohp, w0.numpy())
    mask = synth.valid_mask(lay, "cuda")
    for n in range(iters):
        grads = [synth.gradient(lay, n, i, sigma, seed, "cuda", mask) for i in range(K)]
        if bf16:
            grads = [synth.to_bf16(g) for g in grads]
        gpu_iteration(dev, grads, mode)
        stage, flags = ref.step([oracle_grad(g, bf16) for g in grads])
        if (n + 1) % check_every == 0 or n == iters - 1:
            torch.cuda.synchronize()
            compare_states(dev, ref, f"iter {n} stage {stage} flags {flags}")
    return dev, ref


@pytest.mark.parametrize("mode", ["fused", "split"])
@pytest.mark.parametrize("bf16", [False, True])
def test_tiny_and_ragged_sizes(mode, bf16):
    # vector tails (n % 4 != 0), single elements, several tensors with padding between them
    for numels, K, W, k in [([1], 1, 1, 1), ([3], 2, 0, 2), ([5], 3, 2, 3), ([7, 1, 2], 5, 1, 2),
                            ([17], 4, 2, 4), ([4, 4], 8, 3, 1), ([1023], 17, 2, 2), ([4097, 33], 32, 1, 3)]:
        run_both(numels, K, W, k, W + 3 * max(k, 1) + 2, 0.05, mode, wd=0.01, bf16=bf16)


@pytest.mark.parametrize("mode", ["fused", "split"])
def test_every_small_schedule(mode):
    for W, k in itertools.product(range(4), range(4)):
        run_both([37, 6], 3, W, k, 11, 0.1, mode, wd=0.001)


def test_multi_wave_grid_with_partial_last_trip():
    # more vectors than one wave of blocks covers, the last trip only partly filled, smallest launch shape
    ohp, chp = make_hp(6, 0.1, 0.9, 1, 2)
    n = 148 * 64 * 4 * 5 + 36
    lay = synth.flat(n)
    w0 = synth.init_weights(lay)
    dev = DeviceState(lay.numels, chp, w0)
    dev.ctx.ssd_set_launch(64, 1)
    ref = oracle.State(ohp, w0.numpy())
    for it in range(5):
        grads = [synth.gradient(lay, it, i, 0.02, device="cuda") for i in range(6)]
        gpu_iteration(dev, grads, "fused")
        ref.step([oracle_grad(g, False) for g in grads])
    torch.cuda.synchronize()
    compare_states(dev, ref, "multi-wave")


def test_config_resnet20_K4():
    # ResNet-20 layout, K=4, He-init, N(0, 1e-2) gradients, lr 0.1, m 0.9, W=2, k=4, 20 iterations
    lay = synth.get_layout("resnet20")
    for mode in ("fused", "split"):
        run_both(lay.numels, 4, 2, 4, 20, 1e-2, mode)


def test_config_resnet56_K8():
    # ResNet-56 layout, K=8, W=5, k=4, 100 iterations
    lay = synth.get_layout("resnet56")
    run_both(lay.numels, 8, 5, 4, 100, 1e-2, "fused", check_every=7)


def test_server_alone_is_synchronous_sgd():
    # zero delay: ssd_step never leaves the warm-up stage and equals ssd_server_sync_update alone
    lay = synth.get_layout("resnet20")
    ohp, chp = make_hp(4, 0.1, 0.9, 3, 0, wd=1e-4)
    w0 = synth.init_weights(lay)
    a = DeviceState(lay.numels, chp, w0)
    b = DeviceState(lay.numels, chp, w0, worker_state=False)      # server state only
    ref = oracle.State(ohp, w0.numpy())
    for n in range(6):
        grads = [synth.gradient(lay, n, i, 1e-2, device="cuda") for i in range(4)]
        a.ctx.ssd_step(grads)
        b.ctx.ssd_server_sync_update(grads)
        ref.step([oracle_grad(g, False) for g in grads])
    torch.cuda.synchronize()
    compare_states(a, ref, "k=0")
    assert_same(b.w, ref.w, "server-only w")
    assert_same(b.mom, ref.mom, "server-only mom")
    assert b.ctx.ssd_get_counters()[0] == 0
    with pytest.raises(B.SsdError) as e:
        b.ctx.ssd_broadcast_weights()
    assert e.value.status == B.SSD_ERR_STATE


def test_glu_update_flags_one_by_one():
    # ssd_worker_glu_update with explicit flags from primed uniform(-1,1) state (sweep workload)
    n = (1 << 16) + 8
    for bf16 in (False, True):
        ohp, chp = make_hp(2, 0.1, 0.9, 0, 4, wd=0.01, bf16=bf16)
        for flags in range(8):
            w0 = synth.uniform_buffer(synth.STREAM_WEIGHT, n)
            dev = DeviceState([n], chp, w0)
            ref = oracle.State(ohp, w0.numpy())
            for i in range(2):
                wl = synth.uniform_buffer(synth.STREAM_WLOC, n, worker=i)
                pr = synth.uniform_buffer(synth.STREAM_PRE, n, worker=i)
                dev.w_loc[i].copy_(wl); dev.pre[i].copy_(pr)
                ref.w_loc[i][:] = wl.numpy(); ref.pre[i][:] = pr.numpy()
                g = synth.uniform_buffer(synth.STREAM_GRAD, n, worker=i, device="cuda")
                if bf16:
                    g = synth.to_bf16(g)
                dev.ctx.ssd_worker_glu_update(i, g, flags)
                oracle.glu_update(ohp, oracle_grad(g, bf16), ref.w_loc[i], ref.pre[i], ref.w_dev[i],
                                  ref.w, flags)
            torch.cuda.synchronize()
            for i in range(2):
                for name in ("w_loc", "pre", "w_dev"):
                    assert_same(getattr(dev, name)[i], getattr(ref, name)[i], f"flags {flags} {name}[{i}]")
            assert_same(dev.w, ref.w, "w untouched")


def test_broadcast_weights_and_zero_warmup():
    lay = synth.get_layout("resnet20")
    ohp, chp = make_hp(3, 0.1, 0.9, 0, 2)
    w0 = synth.init_weights(lay)
    dev = DeviceState(lay.numels, chp, w0)
    for t in dev.w_loc:
        t.fill_(float("nan"))
    dev.ctx.ssd_broadcast_weights()
    torch.cuda.synchronize()
    for t in dev.w_loc:
        assert torch.equal(t, dev.w)
    ref = oracle.State(ohp, w0.numpy())
    for n in range(5):
        grads = [synth.gradient(lay, n, i, 1e-2, device="cuda") for i in range(3)]
        dev.ctx.ssd_step(grads)
        ref.step([oracle_grad(g, False) for g in grads])
    torch.cuda.synchronize()
    compare_states(dev, ref, "W=0")


def test_checkpoint_resume_is_bit_exact():
    lay = synth.get_layout("resnet20")
    _, chp = make_hp(4, 0.1, 0.9, 2, 4)
    w0 = synth.init_weights(lay)
    full = DeviceState(lay.numels, chp, w0)
    half = DeviceState(lay.numels, chp, w0)
    def grads(n):
        return [synth.gradient(lay, n, i, 1e-2, device="cuda") for i in range(4)]
    for n in range(14):
        full.ctx.ssd_step(grads(n))
    for n in range(7):
        half.ctx.ssd_step(grads(n))
    it, lu, _, _ = half.ctx.ssd_get_counters()
    resumed = DeviceState(lay.numels, chp, half.w)          # a new context over restored buffers
    resumed.mom.copy_(half.mom)
    for i in range(4):
        resumed.w_loc[i].copy_(half.w_loc[i]); resumed.pre[i].copy_(half.pre[i])
        resumed.w_dev[i].copy_(half.w_dev[i])
    resumed.ctx.ssd_set_counters(it, lu)
    for n in range(7, 14):
        resumed.ctx.ssd_step(grads(n))
    torch.cuda.synchronize()
    for name in ("w", "mom"):
        assert_same(getattr(resumed, name), getattr(full, name).cpu().numpy(), name)
    for i in range(4):
        for name in ("w_loc", "pre", "w_dev"):
            assert_same(getattr(resumed, name)[i], getattr(full, name)[i].cpu().numpy(), f"{name}[{i}]")


def test_step_host_moves_gradients_and_returns_weights():
    lay = synth.get_layout("resnet20")
    ohp, chp = make_hp(4, 0.1, 0.9, 1, 2)
    w0 = synth.init_weights(lay)
    dev = DeviceState(lay.numels, chp, w0)
    ref = oracle.State(ohp, w0.numpy())
    staging = [torch.empty(dev.n, dtype=torch.float32, device="cuda") for _ in range(4)]
    w_out = torch.empty(dev.n, dtype=torch.float32).pin_memory()
    for n in range(4):
        host = [synth.gradient(lay, n, i, 1e-2).pin_memory() for i in range(4)]
        dev.ctx.ssd_step_host(host, staging, w_out)
        torch.cuda.synchronize()
        ref.step([h.numpy() for h in host])
        assert_same(w_out, ref.w, f"host w iter {n}")
    compare_states(dev, ref, "step_host")
    assert dev.ctx.ssd_kernel_launches() == 4


@pytest.mark.parametrize("bf16", [False, True])
def test_every_kernel_shape_and_alignment_gives_the_same_bits(bf16):
    # 256-bit and 128-bit access paths, every load batch, a length with n % 8 == 4, and buffers that
    # are only 16-byte aligned (which must fall back to 128-bit accesses on their own)
    K, W, k, iters = 5, 1, 2, 6
    n = 8 * 1031 + 4
    ohp, chp = make_hp(K, 0.1, 0.9, W, k, wd=0.01, bf16=bf16)
    lay = synth.flat(n)
    w0 = synth.init_weights(lay)
    grads = [[synth.gradient(lay, it, i, 0.05, device="cuda") for i in range(K)] for it in range(iters)]
    if bf16:
        grads = [[synth.to_bf16(g) for g in gs] for gs in grads]
    ref = oracle.State(ohp, w0.numpy())
    for gs in grads:
        ref.step([oracle_grad(g, bf16) for g in gs])

    def offset_copy(t, elems):
        """A copy of t that starts `elems` elements into a fresh allocation (16-byte aligned only)."""
        buf = torch.empty(t.numel() + 16, dtype=t.dtype, device="cuda")
        view = buf[elems:elems + t.numel()]
        view.copy_(t)
        assert view.data_ptr() % 32 == 16 and view.data_ptr() % 16 == 0
        return view

    for vw, batch in [(0, 0), (16, 1), (16, 2), (16, 4), (16, 8), (8, 1), (8, 2), (8, 4), (8, 8), (4, 1), (4, 2),
                      (4, 4), (4, 8)]:
        for mode in ("fused", "split"):
            dev = DeviceState(lay.numels, chp, w0)
            dev.ctx.ssd_set_kernel_shape(vw, batch)
            for gs in grads:
                gpu_iteration(dev, gs, mode)
            torch.cuda.synchronize()
            compare_states(dev, ref, f"shape vw={vw} batch={batch} {mode}")
    # a thread count above what the 16-element kernels are compiled for is brought down, not refused
    dev = DeviceState(lay.numels, chp, w0)
    dev.ctx.ssd_set_kernel_shape(16, 2)
    dev.ctx.ssd_set_launch(512, 1)
    for gs in grads:
        gpu_iteration(dev, gs, "fused")
    torch.cuda.synchronize()
    compare_states(dev, ref, "vw=16 with 512 threads asked")
    # misaligned gradient buffers (float32 only matters) and misaligned state
    shift = 8 if bf16 else 4
    dev = DeviceState(lay.numels, chp, w0)
    for gs in grads:
        gpu_iteration(dev, [offset_copy(g, shift) for g in gs], "fused")
    torch.cuda.synchronize()
    compare_states(dev, ref, "misaligned gradients")
    dev = DeviceState(lay.numels, chp, w0)
    state = DeviceState.__new__(DeviceState)
    state.numels, state.n, state.K, state.device = dev.numels, dev.n, K, dev.device
    state.slabs = []
    state.w, state.mom = offset_copy(dev.w, 4), offset_copy(dev.mom, 4)
    state.w_loc = [offset_copy(t, 4) for t in dev.w_loc]
    state.pre = [offset_copy(t, 4) for t in dev.pre]
    state.w_dev = [offset_copy(t, 4) for t in dev.w_dev]
    state.ctx = B.Context(lay.numels, chp, state.w, state.mom, state.w_loc, state.pre, state.w_dev)
    for gs in grads:
        gpu_iteration(state, gs, "fused")
    torch.cuda.synchronize()
    compare_states(state, ref, "misaligned state")


def tensor_ends(lay):
    offs = lay.offsets
    return [offs[t + 1] if t + 1 < lay.num_tensors else lay.padded_numel for t in range(lay.num_tensors)]


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("mode", ["fused", "split"])
def test_per_tensor_scales_and_lr_schedule(mode, bf16):
    # tensors of odd sizes so that 8-element vectors straddle tensor boundaries; decay only on some
    # tensors, a larger lr on others; the lr drops in the middle of the delay stage
    K, W, k, iters = 3, 2, 3, 12
    lay = synth.Layout("t")
    for n in (5, 1, 10, 3, 64, 7, 1024, 2, 36, 4100):
        lay.add("x", n, "he", 16)
    T = lay.num_tensors
    lr_mult = [1.0, 0.5, 2.0, 1.0, 0.25, 1.0, 1.0, 4.0, 1.0, 0.5]
    wd_mult = [1.0, 0.0, 3.0, 0.0, 1.0, 0.0, 1.0, 0.0, 2.0, 1.0]
    ohp, chp = make_hp(K, 0.1, 0.9, W, k, wd=0.01, bf16=bf16)
    ohp.set_tensor_scales(tensor_ends(lay), lr_mult, wd_mult)
    w0 = synth.init_weights(lay)
    ref = oracle.State(ohp, w0.numpy())
    for vw in (0, 4, 16):
        dev = DeviceState(lay.numels, chp, w0)
        dev.ctx.ssd_set_kernel_shape(vw, 0)
        table = torch.empty(dev.ctx.ssd_tensor_table_bytes(), dtype=torch.uint8, device="cuda")
        dev.ctx.ssd_set_tensor_scales(lr_mult, wd_mult, table)
        ohp.lr, ohp.lr_loc = np.float32(0.1), np.float32(4.0) * np.float32(0.1)
        ref = oracle.State(ohp, w0.numpy())
        for n in range(iters):
            if n == 7:
                dev.ctx.ssd_set_lr(0.05, 0.125)
                ohp.lr, ohp.lr_loc = np.float32(0.05), np.float32(0.125)
            grads = [synth.gradient(lay, n, i, 0.05, device="cuda") for i in range(K)]
            if bf16:
                grads = [synth.to_bf16(g) for g in grads]
            gpu_iteration(dev, grads, mode)
            ref.step([oracle_grad(g, bf16) for g in grads])
            torch.cuda.synchronize()
            compare_states(dev, ref, f"per-tensor vw={vw} iter {n}")


def test_per_tensor_scales_can_be_switched_off_again():
    lay = synth.get_layout("resnet20")
    K = 2
    ohp, chp = make_hp(K, 0.1, 0.9, 1, 2, wd=1e-3)
    w0 = synth.init_weights(lay)
    dev = DeviceState(lay.numels, chp, w0)
    ref = oracle.State(ohp, w0.numpy())
    wd_mult = [1.0 if kind == "he" else 0.0 for kind in lay.kinds]       # no decay on BN and bias
    table = torch.empty(dev.ctx.ssd_tensor_table_bytes(), dtype=torch.uint8, device="cuda")
    for n in range(8):
        if n == 2:
            dev.ctx.ssd_set_tensor_scales(None, wd_mult, table)
            ohp.set_tensor_scales(tensor_ends(lay), [1.0] * lay.num_tensors, wd_mult)
        if n == 6:
            dev.ctx.ssd_set_tensor_scales(None, None, None)
            ohp.tensor_end = None
        grads = [synth.gradient(lay, n, i, 1e-2, device="cuda") for i in range(K)]
        dev.ctx.ssd_step(grads)
        ref.step([oracle_grad(g, False) for g in grads])
    torch.cuda.synchronize()
    compare_states(dev, ref, "per-tensor on/off")


@pytest.mark.parametrize("bf16", [False, True])
def test_shared_pre_weight_gives_the_same_results(bf16):
    # one pre_weight buffer for all K workers: ssd_step reads it once per element; every worker's
    # pre_weight in the oracle must equal it
    K, W, k, iters = 5, 2, 3, 13
    lay = synth.get_layout("resnet20")
    ohp, chp = make_hp(K, 0.1, 0.9, W, k, wd=1e-3, bf16=bf16)
    w0 = synth.init_weights(lay)
    for vw, batch in ((0, 0), (4, 4), (8, 2), (16, 1)):
        dev = DeviceState(lay.numels, chp, w0, shared_pre=True)
        assert len({t.data_ptr() for t in dev.pre}) == 1
        dev.ctx.ssd_set_kernel_shape(vw, batch)
        ref = oracle.State(ohp, w0.numpy())
        for n in range(iters):
            grads = [synth.gradient(lay, n, i, 1e-2, device="cuda") for i in range(K)]
            if bf16:
                grads = [synth.to_bf16(g) for g in grads]
            dev.ctx.ssd_step(grads)
            ref.step([oracle_grad(g, bf16) for g in grads])
            torch.cuda.synchronize()
            compare_states(dev, ref, f"shared pre vw={vw} iter {n}")
    # the per-worker calls cannot be used with a shared pre_weight
    with pytest.raises(B.SsdError) as e:
        dev.ctx.ssd_worker_glu_update(0, grads[0], 0)
    assert e.value.status == B.SSD_ERR_STATE
    with pytest.raises(B.SsdError) as e:
        dev.ctx.ssd_worker_local_step(0, grads[0])
    assert e.value.status == B.SSD_ERR_STATE


def test_layout_with_empty_tensors_and_per_tensor_scales():
    # zero-length tensors occupy no arena space; per-tensor lookups must skip them on both sides
    K = 2
    lay = synth.Layout("t")
    for n in (0, 5, 0, 0, 9, 16, 0):
        lay.add("x", n, "he", 4)
    assert lay.padded_numel == 8 + 12 + 16
    lr_mult = [9.0, 1.0, 9.0, 9.0, 0.5, 2.0, 9.0]
    wd_mult = [9.0, 0.0, 9.0, 9.0, 1.0, 2.0, 9.0]
    ohp, chp = make_hp(K, 0.1, 0.9, 1, 2, wd=0.01)
    ohp.set_tensor_scales(tensor_ends(lay), lr_mult, wd_mult)
    w0 = synth.init_weights(lay)
    dev = DeviceState(lay.numels, chp, w0)
    assert [dev.ctx.ssd_tensor_offset(t) for t in range(7)] == lay.offsets == [0, 0, 8, 8, 8, 20, 36]
    table = torch.empty(dev.ctx.ssd_tensor_table_bytes(), dtype=torch.uint8, device="cuda")
    dev.ctx.ssd_set_tensor_scales(lr_mult, wd_mult, table)
    ref = oracle.State(ohp, w0.numpy())
    for n in range(7):
        grads = [synth.gradient(lay, n, i, 0.05, device="cuda") for i in range(K)]
        dev.ctx.ssd_step(grads)
        ref.step([oracle_grad(g, False) for g in grads])
    torch.cuda.synchronize()
    compare_states(dev, ref, "empty tensors")


def test_plain_c_program_reproduces_the_hand_trace(tmp_path):
    # the boundary is usable from plain C: compile a C program against include/ssd_sgd.h, link it
    # with the library and the CUDA runtime, run it
    import os
    import subprocess
    from paper_2012_05396_b200 import build as libbuild
    root = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
    lib = libbuild.build_library()
    cuda = os.environ.get("CUDA_HOME", "/usr/local/cuda")
    exe = str(tmp_path / "trace_demo")
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-I", os.path.join(root, "include"),
                           "-I", os.path.join(cuda, "include"), os.path.join(root, "tests", "c_abi", "trace_demo.c"),
                           lib, "-L", os.path.join(cuda, "lib64"), "-lcudart", "-o", exe,
                           "-Wl,-rpath," + os.path.dirname(lib), "-Wl,-rpath," + os.path.join(cuda, "lib64")])
    r = subprocess.run([exe], capture_output=True, text=True, timeout=120)
    assert r.returncode == 0, r.stdout + r.stderr
    assert "trace reproduced from C" in r.stdout


@pytest.mark.parametrize("mode", ["fused", "split"])
@pytest.mark.parametrize("bf16", [False, True])
def test_plain_sgd_local_updater(mode, bf16):
    # Eq. 5 as the workers' updater: no grad_sync, pre_weight never read or written
    K, W, k, iters = 3, 2, 3, 11
    lay = synth.get_layout("resnet20")
    ohp, chp = make_hp(K, 0.1, 0.9, W, k, wd=1e-3, lr_loc=0.25, bf16=bf16, local_sgd=True)
    w0 = synth.init_weights(lay)
    dev = DeviceState(lay.numels, chp, w0)
    ref = oracle.State(ohp, w0.numpy())
    for n in range(iters):
        grads = [synth.gradient(lay, n, i, 1e-2, device="cuda") for i in range(K)]
        if bf16:
            grads = [synth.to_bf16(g) for g in grads]
        gpu_iteration(dev, grads, mode)
        ref.step([oracle_grad(g, bf16) for g in grads])
    torch.cuda.synchronize()
    compare_states(dev, ref, "local SGD")                   # pre stays at its NaN fill on both sides


def test_work_is_ordered_on_the_callers_stream():
    # everything is enqueued on the stream it is given: a side stream, with the gradients produced on
    # that stream right before each call and no host synchronisation in between
    K, W, k, iters = 4, 1, 2, 9
    lay = synth.get_layout("resnet56")
    ohp, chp = make_hp(K, 0.1, 0.9, W, k)
    w0 = synth.init_weights(lay)
    dev = DeviceState(lay.numels, chp, w0)
    ref = oracle.State(ohp, w0.numpy())
    side = torch.cuda.Stream()
    staging = [torch.empty(dev.n, dtype=torch.float32, device="cuda") for _ in range(K)]
    w_out = torch.empty(dev.n, dtype=torch.float32).pin_memory()
    torch.cuda.synchronize()
    kept = []
    with torch.cuda.stream(side):
        for n in range(iters):
            grads = [synth.gradient(lay, n, i, 1e-2, device="cuda") for i in range(K)]
            kept.append(grads)
            if n % 3 == 2:                                  # mix in the host-gradient entry point
                host = [g.cpu().pin_memory() for g in grads]
                dev.ctx.ssd_step_host(host, staging, w_out, stream=side)
                kept.append(host)
            else:
                dev.ctx.ssd_step(grads, stream=side)
    side.synchronize()
    for n in range(iters):
        ref.step([synth.gradient(lay, n, i, 1e-2).numpy() for i in range(K)])
    compare_states(dev, ref, "side stream")
    assert_same(w_out, ref.w, "w read back by the last step, which was a host step")


@pytest.mark.parametrize("bf16", [False, True])
def test_layer_by_layer_stepping_equals_one_step(bf16):
    # groups of tensors updated in reverse network order (the order in which a backward pass delivers
    # gradients), with group boundaries that are only 16-byte aligned, per-tensor scales and a shared
    # pre_weight; every iteration must equal one ssd_step over the whole arena
    K, W, k, iters = 3, 2, 2, 8
    lay = synth.Layout("t")
    for i, cnt in enumerate((5, 1, 10, 3, 64, 7, 1024, 2, 36, 4100, 12, 9, 20000, 4, 4, 33)):
        lay.add(f"x{i}", cnt, "he" if i % 3 else "zero", 16)
    T = lay.num_tensors
    ohp, chp = make_hp(K, 0.1, 0.9, W, k, wd=1e-3, bf16=bf16)
    w0 = synth.init_weights(lay)
    whole = DeviceState(lay.numels, chp, w0, shared_pre=True)
    layered = DeviceState(lay.numels, chp, w0, shared_pre=True)
    wd_mult = [1.0 if kind == "he" else 0.0 for kind in lay.kinds]
    ends = [lay.offsets[t + 1] if t + 1 < T else lay.padded_numel for t in range(T)]
    ohp.set_tensor_scales(ends, [1.0] * T, wd_mult)
    ref = oracle.State(ohp, w0.numpy())                    # and both must equal the CPU oracle
    tables = [torch.empty(s.ctx.ssd_tensor_table_bytes(), dtype=torch.uint8, device="cuda") for s in (whole, layered)]
    whole.ctx.ssd_set_tensor_scales(None, wd_mult, tables[0])
    layered.ctx.ssd_set_tensor_scales(None, wd_mult, tables[1])
    assert any(o % 8 == 4 for o in lay.offsets)            # some groups start off the 256-bit grid
    groups, t = [], 0
    for size in itertools.cycle((1, 3, 2, 7)):
        if t >= T:
            break
        groups.append((t, min(size, T - t)))
        t += size
    for n in range(iters):
        grads = [synth.gradient(lay, n, i, 1e-2, device="cuda") for i in range(K)]
        if bf16:
            grads = [synth.to_bf16(g) for g in grads]
        whole.ctx.ssd_step(grads)
        for first, count in reversed(groups):
            layered.ctx.ssd_step_tensors(grads, first, count)
        layered.ctx.ssd_advance()
        ref.step([oracle_grad(g, bf16) for g in grads])
        torch.cuda.synchronize()
        compare_states(layered, ref, f"layer groups, iter {n}")
        for name in ("w", "mom"):
            assert torch.equal(getattr(whole, name).view(torch.int32), getattr(layered, name).view(torch.int32)), (name, n)
        for i in range(K):
            for name in ("w_loc", "pre", "w_dev"):
                assert torch.equal(getattr(whole, name)[i].view(torch.int32),
                                   getattr(layered, name)[i].view(torch.int32)), (name, i, n)
    assert whole.ctx.ssd_get_counters() == layered.ctx.ssd_get_counters()
    assert layered.ctx.ssd_kernel_launches() == iters * len(groups)
    with pytest.raises(B.SsdError) as e:
        layered.ctx.ssd_step_tensors(grads, T - 1, 2)
    assert e.value.status == B.SSD_ERR_ARG


def test_random_combinations_of_every_option():
    # seeded draw over layouts, K, schedule, gradient type, per-tensor scales, shared pre_weight, local
    # updater, kernel shape and the way an iteration is issued (whole step, layer groups, split calls)
    rng = np.random.default_rng(20201205)
    for case in range(40):
        T = int(rng.integers(1, 9))
        numels = [int(rng.choice([0, 1, 3, 4, 5, 8, 17, 64, 100, 1000, 4099])) for _ in range(T)]
        if sum(numels) == 0:
            numels[0] = 6
        K = int(rng.choice([1, 2, 3, 4, 7, 8, 16, 32]))
        W, k = int(rng.integers(0, 4)), int(rng.integers(0, 5))
        bf16, per_tensor = bool(rng.integers(2)), bool(rng.integers(2))
        local_sgd = bool(rng.integers(4) == 0)
        shared = bool(rng.integers(2)) and K > 1 and k > 0
        issue = str(rng.choice(["step", "layers"] if shared else ["step", "layers", "split"]))
        vw, batch = int(rng.choice([0, 4, 8, 16])), int(rng.choice([0, 1, 2, 4, 8]))
        iters = W + 2 * max(k, 1) + 2
        tag = f"case {case}: numels={numels} K={K} W={W} k={k} bf16={bf16} pt={per_tensor} sgd={local_sgd} " \
              f"shared={shared} issue={issue} shape=({vw},{batch})"
        lay = synth.Layout("t")
        for i, cnt in enumerate(numels):
            lay.add(f"x{i}", cnt, "he", 8)
        ohp, chp = make_hp(K, 0.1, 0.9, W, k, wd=0.01, bf16=bf16, local_sgd=local_sgd)
        w0 = synth.init_weights(lay, seed=case)
        dev = DeviceState(lay.numels, chp, w0, shared_pre=shared)
        dev.ctx.ssd_set_kernel_shape(vw, batch)
        if per_tensor:
            lr_mult = [float(x) for x in rng.choice([0.25, 0.5, 1.0, 2.0], T)]
            wd_mult = [float(x) for x in rng.choice([0.0, 1.0, 3.0], T)]
            ohp.set_tensor_scales(tensor_ends(lay), lr_mult, wd_mult)
            table = torch.empty(dev.ctx.ssd_tensor_table_bytes(), dtype=torch.uint8, device="cuda")
            dev.ctx.ssd_set_tensor_scales(lr_mult, wd_mult, table)
        ref = oracle.State(ohp, w0.numpy())
        for n in range(iters):
            grads = [synth.gradient(lay, n, i, 0.05, seed=case, device="cuda") for i in range(K)]
            if bf16:
                grads = [synth.to_bf16(g) for g in grads]
            if issue == "step":
                dev.ctx.ssd_step(grads)
            elif issue == "layers":
                for t in reversed(range(T)):
                    dev.ctx.ssd_step_tensors(grads, t, 1)
                dev.ctx.ssd_advance()
            else:
                gpu_iteration(dev, grads, "split")
            ref.step([oracle_grad(g, bf16) for g in grads])
        torch.cuda.synchronize()
        compare_states(dev, ref, tag)


def test_fused_steps_replayed_from_a_cuda_graph():
    # one period of k delay-stage iterations captured into a CUDA graph and replayed for later periods,
    # the gradients written into the same buffers before each replay; the counters are set by hand
    K, W, k, periods = 4, 2, 4, 3
    lay = synth.get_layout("resnet20")
    ohp, chp = make_hp(K, 0.1, 0.9, W, k, wd=1e-3)
    w0 = synth.init_weights(lay)
    dev = DeviceState(lay.numels, chp, w0)
    ref = oracle.State(ohp, w0.numpy())
    slots = [[torch.empty(dev.n, dtype=torch.float32, device="cuda") for _ in range(K)] for _ in range(k)]

    def fill(n, j):
        grads = [synth.gradient(lay, n, i, 1e-2, device="cuda") for i in range(K)]
        for s, g in zip(slots[j], grads):
            s.copy_(g)
        ref.step([g.cpu().numpy() for g in grads])

    n = 0
    for _ in range(W + 1 + k):                     # warm-up, first GLU call, one whole period outside capture
        fill(n, n % k)
        dev.ctx.ssd_step(slots[n % k])
        n += 1
    torch.cuda.synchronize()
    compare_states(dev, ref, "before capture")
    base = n
    # capture the next period (its launches do not run now: the state is untouched, the counters move)
    graph, side = torch.cuda.CUDAGraph(), torch.cuda.Stream()
    it0, lu0, _, _ = dev.ctx.ssd_get_counters()
    with torch.cuda.graph(graph, stream=side):
        for j in range(k):
            dev.ctx.ssd_step(slots[(base + j) % k])
    assert dev.ctx.ssd_get_counters()[:2] == (it0 + k, lu0 + k)
    dev.ctx.ssd_set_counters(it0, lu0)
    for p in range(periods):
        for j in range(k):
            fill(n, n % k)
            n += 1
        graph.replay()
        it, lu, _, _ = dev.ctx.ssd_get_counters()
        dev.ctx.ssd_set_counters(it + k, lu + k)
        torch.cuda.synchronize()
        compare_states(dev, ref, f"after replay {p}")


@pytest.mark.parametrize("bf16", [False, True])
def test_staged_step_kernel_gives_the_same_bits(bf16):
    # the bulk-copy / shared-memory ring variant of the fused step: every flag of the schedule, several
    # ring depths, per-tensor scalars, tiles with a ragged end, layer-group ranges
    K, W, k, iters = 4, 1, 3, 9
    lay = synth.Layout("t")
    for i, cnt in enumerate((5000, 3, 2048, 64, 4100, 12, 8)):
        lay.add(f"x{i}", cnt, "he", 16)
    ohp, chp = make_hp(K, 0.1, 0.9, W, k, wd=0.01, bf16=bf16)
    lr_mult = [1.0, 0.5, 2.0, 1.0, 0.25, 1.0, 4.0]
    wd_mult = [1.0, 0.0, 3.0, 0.0, 1.0, 0.0, 2.0]
    w0 = synth.init_weights(lay)
    for stages, per_tensor, layers in ((2, False, False), (3, True, False), (8, False, True), (4, True, True)):
        if per_tensor:
            ohp.set_tensor_scales(tensor_ends(lay), lr_mult, wd_mult)
        else:
            ohp.tensor_end = None
        dev = DeviceState(lay.numels, chp, w0)
        dev.ctx.ssd_set_staging(stages)
        if per_tensor:
            table = torch.empty(dev.ctx.ssd_tensor_table_bytes(), dtype=torch.uint8, device="cuda")
            dev.ctx.ssd_set_tensor_scales(lr_mult, wd_mult, table)
        ref = oracle.State(ohp, w0.numpy())
        for n in range(iters):
            grads = [synth.gradient(lay, n, i, 0.05, device="cuda") for i in range(K)]
            if bf16:
                grads = [synth.to_bf16(g) for g in grads]
            if layers:
                for first, count in ((4, 3), (1, 3), (0, 1)):
                    dev.ctx.ssd_step_tensors(grads, first, count)
                dev.ctx.ssd_advance()
            else:
                dev.ctx.ssd_step(grads)
            ref.step([oracle_grad(g, bf16) for g in grads])
            torch.cuda.synchronize()
            compare_states(dev, ref, f"ring stages={stages} pt={per_tensor} layers={layers} iter {n}")
        assert dev.ctx.ssd_staging_error() == 0
    with pytest.raises(B.SsdError):
        dev.ctx.ssd_set_staging(9)
    with pytest.raises(B.SsdError):
        dev.ctx.ssd_set_staging(1)
