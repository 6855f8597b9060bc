"""Contexts without separate device weights (w_dev[i] is w_loc[i]) against the CPU oracle.

Algorithm 1 hands the local update's result to the worker's devices on a pull iteration and then
overwrites the local weight with the pulled global weight.  A caller that keeps one buffer for both
never sees that result, so the library skips the local update on pull iterations.  The oracle
is the plain algorithm with its K device-weight buffers; w, mom, every w_loc and every pre_weight
must equal it bit for bit on every iteration (compare_states leaves out only w_dev).
"""
import itertools

import pytest
import torch

import oracle
from paper_2012_05396_b200 import binding as B
from paper_2012_05396_b200 import synth
from paper_2012_05396_b200.state import DeviceState
from tests.gpu_common import compare_states, gpu_iteration, make_hp, oracle_grad

pytestmark = pytest.mark.gpu


def flat_layout(numels):
    lay = synth.Layout("t")
    for n in numels:
        lay.add("x", n, "he", 16)
    return lay


def run_merged(lay, K, W, k, iters, mode, bf16=False, wd=1e-3, shared_pre=False, local_sgd=False,
               per_tensor=False, shape=None, check_every=1, staging=0):
    ohp, chp = make_hp(K, 0.1, 0.9, W, k, wd=wd, bf16=bf16, local_sgd=local_sgd)
    w0 = synth.init_weights(lay)
    dev = DeviceState(lay.numels, chp, w0, merged_dev=True, shared_pre=shared_pre)
    assert all(a.data_ptr() == b.data_ptr() for a, b in zip(dev.w_dev, dev.w_loc))
    if per_tensor:
        ends = [lay.offsets[t + 1] if t + 1 < lay.num_tensors else lay.padded_numel for t in range(lay.num_tensors)]
        lr_mult = [0.5 if t % 3 == 0 else 1.0 for t in range(lay.num_tensors)]
        wd_mult = [1.0 if kind == "he" else 0.0 for kind in lay.kinds]
        ohp.set_tensor_scales(ends, lr_mult, wd_mult)
        table = torch.empty(dev.ctx.ssd_tensor_table_bytes(), dtype=torch.uint8, device="cuda")
        dev.ctx.ssd_set_tensor_scales(lr_mult, wd_mult, table)
    if shape:
        dev.ctx.ssd_set_kernel_shape(*shape)
    if staging:
        dev.ctx.ssd_set_staging(staging)
    ref = oracle.State(ohp, w0.numpy())
    mask = synth.valid_mask(lay, "cuda")
    seen = 0
    for n in range(iters):
        grads = [synth.gradient(lay, n, i, 1e-2, device="cuda", mask=mask) for i in range(K)]
        if bf16:
            grads = [synth.to_bf16(g) for g in grads]
        gpu_iteration(dev, grads, mode)
        stage, flags = ref.step([oracle_grad(g, bf16) for g in grads])
        if stage == B.SSD_STAGE_DELAY:
            seen |= flags
        if (n + 1) % check_every == 0 or n == iters - 1:
            torch.cuda.synchronize()
            compare_states(dev, ref, f"K={K} W={W} k={k} iter {n} stage {stage} flags {flags}")
    return dev, ref, seen


@pytest.mark.parametrize("mode", ["fused", "split"])
@pytest.mark.parametrize("bf16", [False, True])
def test_merged_device_weights_small_schedules(mode, bf16):
    # ragged sizes, every (W, k) up to 3: k = 1 pulls and writes pre_weight in the same iteration
    for W, k in itertools.product(range(3), range(1, 4)):
        _, _, seen = run_merged(flat_layout([37, 6, 1023]), 3, W, k, W + 3 * k + 2, mode, bf16=bf16)
        assert seen & 7 == 7                 # first, refresh and pull iterations all occurred


@pytest.mark.parametrize("bf16", [False, True])
def test_merged_device_weights_resnet56_layout(bf16):
    # several waves of blocks, per-tensor scalars, K not a multiple of the load batch
    lay = synth.get_layout("resnet56")
    run_merged(lay, 5, 2, 4, 12, "fused", bf16=bf16, per_tensor=True, check_every=3)
    run_merged(lay, 9, 1, 1, 6, "fused", bf16=bf16, per_tensor=True, check_every=2)


def test_merged_device_weights_shared_pre_weight_and_plain_sgd():
    lay = synth.get_layout("resnet20")
    run_merged(lay, 4, 1, 1, 6, "fused", shared_pre=True)
    run_merged(lay, 4, 2, 3, 10, "fused", shared_pre=True)
    run_merged(lay, 4, 1, 2, 8, "fused", local_sgd=True)
    run_merged(lay, 3, 0, 1, 5, "split", local_sgd=True)


@pytest.mark.parametrize("bf16", [False, True])
def test_merged_device_weights_with_the_staged_fused_step(bf16):
    # the shared-memory ring runs the iterations without a pull; the pulls stay on the register path
    lay = flat_layout([70001, 12, 4099])
    dev, _, seen = run_merged(lay, 3, 1, 3, 9, "fused", bf16=bf16, staging=3)
    assert seen & 7 == 7 and dev.ctx.ssd_staging_error() == 0


@pytest.mark.parametrize("bf16", [False, True])
def test_merged_pull_kernel_in_every_shape(bf16):
    # k = 1 runs the pull-and-write-pre_weight kernel at every delay iteration: all vectors and batches
    lay = flat_layout([4097, 33, 100003])
    for vw, batch in itertools.product((4, 8, 16), (1, 2, 4, 8)):
        run_merged(lay, 7, 1, 1, 5, "fused", bf16=bf16, shape=(vw, batch), check_every=5)


def test_merged_device_weights_layer_groups_and_host_pipeline():
    # the range forms: ssd_step_tensors over groups of layers, ssd_step_host over chunks, and a
    # host-resident pre_weight (one pinned arena) whose slice is not fetched on pull iterations
    lay = synth.get_layout("resnet56")
    K = 3
    for k in (1, 3):
        ohp, chp = make_hp(K, 0.1, 0.9, 1, k, wd=1e-3)
        w0 = synth.init_weights(lay)
        groups = DeviceState(lay.numels, chp, w0, merged_dev=True)
        piped = DeviceState(lay.numels, chp, w0, merged_dev=True)
        piped.ctx.ssd_set_host_chunk(1 << 16)
        hosted = DeviceState(lay.numels, chp, w0, merged_dev=True, host_pre=True, pre_slots=2, host_chunk=1 << 16)
        ref = oracle.State(ohp, w0.numpy())
        staging = [torch.empty(groups.n, dtype=torch.float32, device="cuda") for _ in range(K)]
        T = lay.num_tensors
        cuts = [0, 1, 7, 60, 61, T]
        for n in range(2 + 3 * k):
            host = [synth.gradient(lay, n, i, 1e-2).pin_memory() for i in range(K)]
            grads = [h.cuda() for h in host]
            for a, b in reversed(list(zip(cuts[:-1], cuts[1:]))):          # last layers first, as backward does
                groups.ctx.ssd_step_tensors(grads, a, b - a)
            groups.ctx.ssd_advance()
            piped.ctx.ssd_step_host(host, staging, None)
            torch.cuda.synchronize()
            hosted.ctx.ssd_step_host(host, staging, None)
            ref.step([h.numpy() for h in host])
            torch.cuda.synchronize()
            for name, dev in (("layer groups", groups), ("host pipeline", piped), ("host pre_weight", hosted)):
                compare_states(dev, ref, f"{name} k={k} iter {n}")


def test_merged_device_weights_checkpoint_and_views():
    # resume in the middle of a period; the view a worker computes its next gradient on
    lay = flat_layout([5000])
    K, W, k = 2, 1, 3
    ohp, chp = make_hp(K, 0.1, 0.9, W, k)
    w0 = synth.init_weights(lay)
    dev = DeviceState(lay.numels, chp, w0, merged_dev=True)
    ref = oracle.State(ohp, w0.numpy())
    views = []
    for n in range(6):
        grads = [synth.gradient(lay, n, i, 1e-2, device="cuda") for i in range(K)]
        dev.ctx.ssd_step(grads)
        ref.step([g.cpu().numpy() for g in grads])
        weights, view = dev.ctx.ssd_worker_weights(1)
        views.append(view)
        assert weights == (dev.w.data_ptr() if view == B.SSD_VIEW_GLOBAL else dev.w_loc[1].data_ptr())
    assert views == [B.SSD_VIEW_LOCAL] * 6          # W = 1: the hand-over copy comes with iteration 0
    torch.cuda.synchronize()
    saved = [t.clone() for t in [dev.w, dev.mom, *dev.w_loc, *dev.pre]]
    counters = dev.ctx.ssd_get_counters()[:2]
    resumed = DeviceState(lay.numels, chp, w0, merged_dev=True)
    for dst, src in zip([resumed.w, resumed.mom, *resumed.w_loc, *resumed.pre], saved):
        dst.copy_(src)
    resumed.ctx.ssd_set_counters(*counters)
    for n in range(6, 11):
        grads = [synth.gradient(lay, n, i, 1e-2, device="cuda") for i in range(K)]
        resumed.ctx.ssd_step(grads)
        ref.step([g.cpu().numpy() for g in grads])
    torch.cuda.synchronize()
    compare_states(resumed, ref, "resumed")
