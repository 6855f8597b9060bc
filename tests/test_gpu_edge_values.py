"""The ends of the binary32 range on the GPU: subnormals, signed zeros, overflow.

The arithmetic contract is IEEE 754 binary32 with gradual underflow: subnormal inputs are used
as they are and subnormal results are kept (no flush to zero).  The CPU oracle is pinned to that
by exact rational arithmetic (tests/test_oracle_pins.py); here the CUDA kernels must match the
oracle bit for bit on inputs that live at both ends of the range.  A kernel built to flush
subnormals, or with approximate arithmetic, fails these tests.  Where the arithmetic itself
produces a NaN (inf - inf, 0 * inf) only its being a NaN is compared.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2012_05396_b200 import binding as B
from paper_2012_05396_b200.state import DeviceState
from tests.gpu_common import assert_same, compare_states, make_hp

pytestmark = pytest.mark.gpu
f32 = np.float32
U = 2.0 ** -149
TINY_NORMAL = 2.0 ** -126
BIG = float(np.finfo(f32).max)


def edge_buffer(rng, n, regime):
    """n float32 values: 'small' around and below the smallest normal, 'large' near the largest finite
    value, 'mixed' both plus ordinary magnitudes, zeros of both signs and infinities."""
    small = np.array([0.0, U, 2 * U, 3 * U, 5 * U, 1000 * U, 2.0 ** -127, TINY_NORMAL, 1.5 * TINY_NORMAL,
                      TINY_NORMAL - U, 1e-38, 1e-39, 1e-40, 1e-42, 1e-44, 3e-37, 1e-36])
    large = np.array([BIG, BIG / 2, BIG / 3, 2.0 ** 127, 1e38, 3e38, 1e37, 2.0 ** 126, 1e30])
    if regime == "small":
        pool = small
    elif regime == "large":
        pool = large
    else:
        pool = np.concatenate([small, large, [1.0, 0.1, 1e-3, 1e-20, 1e20, np.inf]])
    picks = rng.choice(pool, n) * rng.choice([-1.0, 1.0], n)
    wobble = 1.0 + 0.25 * rng.random(n)                    # spread the mantissas, stay in the regime
    if regime == "large":
        wobble = 1.0 - 0.25 * rng.random(n)
    out = (picks * wobble).astype(f32)
    out[rng.random(n) < 0.05] = f32(-0.0)
    return out


def count_subnormal(a):
    a = np.abs(a[np.isfinite(a)])
    return int(np.count_nonzero((a > 0) & (a < TINY_NORMAL)))


@pytest.mark.parametrize("bf16", [False, True])
@pytest.mark.parametrize("regime", ["small", "large", "mixed"])
def test_single_calls_on_edge_values(regime, bf16):
    # one server update and one GLU call per worker and flag combination, from primed state
    rng = np.random.default_rng(99)
    n, K = 8 * 4099 + 4, 3
    ohp, chp = make_hp(K, 0.1, 0.9, 0, 4, wd=0.01, bf16=bf16)
    w0 = edge_buffer(rng, n, regime)
    subnormal_results = 0
    for flags in (0, B.SSD_FLAG_REFRESH, B.SSD_FLAG_PULL, B.SSD_FLAG_FIRST, B.SSD_FLAG_REFRESH | B.SSD_FLAG_PULL):
        dev = DeviceState([n], chp, torch.from_numpy(w0))
        ref = oracle.State(ohp, w0)
        mom = edge_buffer(rng, n, regime)
        dev.mom.copy_(torch.from_numpy(mom)); ref.mom[:] = mom
        grads, ref_grads = [], []
        for i in range(K):
            wl, pr = edge_buffer(rng, n, regime), edge_buffer(rng, n, regime)
            pr[::7] = wl[::7]                                # grad_sync exactly zero on some elements
            dev.w_loc[i].copy_(torch.from_numpy(wl)); dev.pre[i].copy_(torch.from_numpy(pr))
            ref.w_loc[i][:] = wl; ref.pre[i][:] = pr
            g = torch.from_numpy(edge_buffer(rng, n, regime)).cuda()
            if bf16:
                g = g.to(torch.bfloat16)                     # subnormal bfloat16 values stay subnormal
                ref_grads.append(g.cpu().view(torch.int16).numpy().view(np.uint16))
            else:
                ref_grads.append(g.cpu().numpy())
            grads.append(g)
        dev.ctx.ssd_server_sync_update(grads)
        with np.errstate(all="ignore"):
            oracle.server_update(ohp, ref_grads, ref.w, ref.mom)
        for i in range(K):
            dev.ctx.ssd_worker_glu_update(i, grads[i], flags)
            oracle.glu_update(ohp, ref_grads[i], ref.w_loc[i], ref.pre[i], ref.w_dev[i], ref.w, flags)
        torch.cuda.synchronize()
        tag = f"{regime} bf16={bf16} flags={flags}"
        assert_same(dev.w, ref.w, tag + " w", generated_nans=True)
        assert_same(dev.mom, ref.mom, tag + " mom", generated_nans=True)
        for i in range(K):
            for name in ("w_loc", "pre", "w_dev"):
                if name == "w_dev" and not flags & B.SSD_FLAG_PULL:
                    continue
                assert_same(getattr(dev, name)[i], getattr(ref, name)[i], f"{tag} {name}[{i}]", generated_nans=True)
        assert dev.guards_intact()
        subnormal_results += count_subnormal(ref.mom) + sum(count_subnormal(x) for x in ref.w_loc)
    if regime == "small":
        assert subnormal_results > 10000                   # the expected values really are subnormal
    if regime == "large":
        assert np.isinf(ref.w).sum() + np.isinf(ref.mom).sum() > 100


@pytest.mark.parametrize("bf16", [False, True])
def test_whole_schedule_in_the_subnormal_range(bf16):
    # weights, momenta and gradients stay around the smallest normal for a whole schedule, fused step,
    # every vector width: products such as lr*(g + wd*w), m*mom and (pre - w')*c are subnormal throughout
    rng = np.random.default_rng(7)
    K, W, k, iters = 4, 1, 3, 9
    n = 16 * 1031 + 12
    ohp, chp = make_hp(K, 0.1, 0.9, W, k, wd=0.01, bf16=bf16)
    w0 = edge_buffer(rng, n, "small")
    gs = [[edge_buffer(rng, n, "small") for _ in range(K)] for _ in range(iters)]
    ref = oracle.State(ohp, w0)
    dev_grads, seen_subnormal = [], 0
    for it in range(iters):
        tg = [torch.from_numpy(g).cuda() for g in gs[it]]
        if bf16:
            tg = [g.to(torch.bfloat16) for g in tg]
        dev_grads.append(tg)
        ref.step([g.cpu().view(torch.int16).numpy().view(np.uint16) if bf16 else g.cpu().numpy() for g in tg])
        seen_subnormal += count_subnormal(ref.mom) + count_subnormal(ref.w_loc[0])
    assert seen_subnormal > 5000
    for vw in (0, 4, 8, 16):
        dev = DeviceState([n], chp, torch.from_numpy(w0))
        dev.ctx.ssd_set_kernel_shape(vw, 0)
        for it in range(iters):
            dev.ctx.ssd_step(dev_grads[it])
        torch.cuda.synchronize()
        compare_states(dev, ref, f"subnormal schedule vw={vw} bf16={bf16}", generated_nans=True)
