"""Helpers shared by the GPU parity tests: run a schedule on both sides and compare bit patterns."""
import numpy as np
import torch

import oracle
from paper_2012_05396_b200 import binding as B
from paper_2012_05396_b200 import synth
from paper_2012_05396_b200.state import DeviceState

# The arithmetic is defined operation by operation (binary32, no fused multiply-add, fixed
# summation order), so the CUDA result is unique and must equal the oracle's bit for bit.  That
# is stricter than the stated floating-point bar, which is also asserted:
REL_TOL, ABS_TOL = 1e-6, 1e-7


def bits(a):
    if isinstance(a, torch.Tensor):
        a = a.detach().cpu().numpy()
    return np.ascontiguousarray(a).view(np.uint32)


def assert_same(got, want, what, idx=None, generated_nans=False):
    """Bit equality of every element.  generated_nans: where the oracle's value is a NaN that the
    arithmetic produced (inf - inf, 0 * inf), only "is a NaN" is compared: IEEE 754 leaves the sign
    and payload of such a NaN open, and x86 and the GPU choose differently."""
    if isinstance(got, torch.Tensor):
        if idx is not None:                       # gather on the device: the arena may be GiB-sized
            got = got[torch.from_numpy(np.asarray(idx)).to(got.device)]
            idx = None
        g = got.detach().cpu().numpy()
    else:
        g = got
    if idx is not None:
        g = g[idx]
    gb, wb = bits(g), bits(want)
    if generated_nans:
        nan = np.isnan(want)
        assert np.array_equal(np.isnan(g), nan), f"{what}: NaNs in different places"
        gb, wb = np.where(nan, 0, gb), np.where(nan, 0, wb)
    if not np.array_equal(gb, wb):
        bad = np.nonzero(gb != wb)[0]
        j = int(bad[0])
        raise AssertionError(f"{what}: {bad.size} of {wb.size} elements differ; first at {j}: "
                             f"cuda {g[j]!r} oracle {want[j]!r}")
    finite = np.isfinite(want)
    err = np.abs(g[finite].astype(np.float64) - want[finite].astype(np.float64))
    assert np.all(err <= ABS_TOL + REL_TOL * np.abs(want[finite].astype(np.float64))), what


def make_hp(K, lr, m, W, k, wd=0.0, lr_loc=None, alpha=2.0, beta=0.5, rescale=None, bf16=False,
            local_sgd=False):
    """The same hyper-parameters for both sides (defaults resolved by each side on its own)."""
    nan = float("nan")
    o = oracle.Hyper(K=K, lr=lr, m=m, W=W, k=k, wd=wd, lr_loc=lr_loc, alpha=alpha, beta=beta,
                     rescale=rescale, grad_bf16=bf16, local_sgd=local_sgd)
    c = B.make_hparams(K, lr, m, W, k, wd=wd, lr_local=nan if lr_loc is None else lr_loc,
                       alpha=alpha, beta=beta, rescale=nan if rescale is None else rescale,
                       grad_dtype=B.SSD_BF16 if bf16 else B.SSD_F32,
                       local_updater=B.SSD_LOCAL_SGD if local_sgd else B.SSD_LOCAL_GLU)
    return o, c


def oracle_grad(g: torch.Tensor, bf16: bool):
    """Device gradient tensor -> the numpy array the oracle consumes."""
    if bf16:
        return synth.bf16_bits(g)
    return g.detach().cpu().numpy()


def compare_states(dev: DeviceState, ref: oracle.State, tag, idx=None, generated_nans=False):
    kw = dict(idx=idx, generated_nans=generated_nans)
    # merged device weights: the device-weight output of pull iterations is not produced (the next
    # gradient is computed on the pulled weight); everything else is the oracle's, bit for bit
    merged = getattr(dev, "merged_dev", False)
    assert_same(dev.w, ref.w, f"{tag} w", **kw)
    assert_same(dev.mom, ref.mom, f"{tag} mom", **kw)
    for i in range(dev.K):
        assert_same(dev.w_loc[i], ref.w_loc[i], f"{tag} w_loc[{i}]", **kw)
        assert_same(dev.pre[i], ref.pre[i], f"{tag} pre[{i}]", **kw)
        if not merged:
            assert_same(dev.w_dev[i], ref.w_dev[i], f"{tag} w_dev[{i}]", **kw)
    # nothing was stored outside the arenas (guard words before, between and after them)
    for slab in getattr(dev, "slabs", []):
        assert slab.guards_intact(), f"{tag}: guard words overwritten next to arenas {slab.damaged_gaps()}"
    it, lu, _, _ = dev.ctx.ssd_get_counters()
    assert (it, lu) == (ref.iter, ref.loc_update), tag
    for i in range(dev.K):
        view = dev.ctx.ssd_worker_weights(i)[1]
        assert view == (B.SSD_VIEW_LOCAL if merged and ref.view == B.SSD_VIEW_DEVICE else ref.view), tag


def gpu_iteration(dev: DeviceState, grads, mode):
    """One iteration on the GPU: 'fused' = ssd_step, 'split' = server + K local steps + advance."""
    if mode == "fused":
        dev.ctx.ssd_step(grads)
    else:
        dev.ctx.ssd_server_sync_update(grads)
        for i in range(dev.K):
            dev.ctx.ssd_worker_local_step(i, grads[i])
        dev.ctx.ssd_advance()
