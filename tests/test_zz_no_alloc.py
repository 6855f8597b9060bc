"""The allocation-free entry point, ssd_server_sync_update_static.

Some users of this library cannot allocate device memory at the point where they call it (their
host program's memory pool owns the whole GPU, or allocation is forbidden where they run), so
they cannot provide the device table that per-tensor hyper-parameters normally need.  For them
the library keeps that table in a fixed array of its own device image.  These tests check that
the call gives exactly what the ordinary route gives (caller-allocated table, then
ssd_server_sync_update), on two calls in a row, and that layouts beyond the array's capacity
are refused.  The file name sorts last so that a run stopping at the first failure has
already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2012_05396_b200 import binding as B
from paper_2012_05396_b200 import build as libbuild
from paper_2012_05396_b200 import synth
from paper_2012_05396_b200.state import DeviceState


def test_layouts_beyond_the_static_table_are_refused():
    libbuild.build_library()
    T = B.SSD_STATIC_TABLE_MAX_TENSORS + 1
    hp = B.make_hparams(2, 0.1, 0.9, 0, 0)
    ctx = B.Context([4] * T, hp, 0x10000000, 0x20000000)
    with pytest.raises(B.SsdError) as e:
        ctx.ssd_server_sync_update_static([0x30000000, 0x40000000])
    assert e.value.status == B.SSD_ERR_TOO_LARGE and "SSD_STATIC_TABLE_MAX_TENSORS" in str(e.value)
    assert ctx.ssd_kernel_launches() == 0


@pytest.mark.gpu
@pytest.mark.parametrize("bf16", [False, True])
def test_static_table_update_equals_the_caller_allocated_route(bf16):
    K = 4
    lay = synth.get_layout("resnet20")
    lr_mult = [0.1 if name.startswith("fc") else 1.0 for name in lay.names]
    wd_mult = [1.0 if kind == "he" else 0.0 for kind in lay.kinds]          # no decay on BN and bias
    hp = B.make_hparams(K, 0.1, 0.9, 0, 0, wd=5e-4, grad_dtype=B.SSD_BF16 if bf16 else B.SSD_F32)
    w0 = synth.init_weights(lay)
    ordinary = DeviceState(lay.numels, hp, w0, worker_state=False)
    static = DeviceState(lay.numels, hp, w0, worker_state=False)
    table = torch.empty(ordinary.ctx.ssd_tensor_table_bytes(), dtype=torch.uint8, device="cuda")
    ordinary.ctx.ssd_set_tensor_scales(lr_mult, wd_mult, table)
    for call in range(2):                                                   # two calls in a row
        grads = [synth.gradient(lay, call, i, 1e-2, device="cuda") for i in range(K)]
        if bf16:
            grads = [synth.to_bf16(g) for g in grads]
        if call == 1:                                                       # the second call changes the scales
            lr_mult = [2.0 * v for v in lr_mult]
            ordinary.ctx.ssd_set_tensor_scales(lr_mult, wd_mult, table)
        ordinary.ctx.ssd_server_sync_update(grads)
        static.ctx.ssd_server_sync_update_static(grads, lr_mult, wd_mult)
        torch.cuda.synchronize()
        # same arithmetic, same order: the two routes must agree bit for bit
        assert torch.equal(static.w.view(torch.int32), ordinary.w.view(torch.int32)), f"w differs after call {call}"
        assert torch.equal(static.mom.view(torch.int32), ordinary.mom.view(torch.int32)), f"mom differs after call {call}"
    assert not torch.equal(static.w, w0.cuda())
    assert static.ctx.ssd_kernel_launches() == 2


@pytest.mark.gpu
@pytest.mark.parametrize("bf16", [False, True])
def test_static_table_update_against_the_cpu_oracle(bf16):
    # The same call checked directly against the CPU oracle's per-tensor server update, bit for bit, on
    # two calls in a row.  Also: a warm call changes the amount of free device memory by nothing, and a
    # table the context got through ssd_set_tensor_scales is neither used nor disturbed by it.
    from tests.gpu_common import assert_same, oracle_grad
    K = 3
    lay = synth.get_layout("resnet56")
    ends = [lay.offsets[t + 1] if t + 1 < lay.num_tensors else lay.padded_numel for t in range(lay.num_tensors)]
    own_lr = [0.5] * lay.num_tensors                        # the context's own table: something else entirely
    own_wd = [2.0] * lay.num_tensors
    hp = B.make_hparams(K, 0.1, 0.9, 0, 0, wd=5e-4, grad_dtype=B.SSD_BF16 if bf16 else B.SSD_F32)
    w0 = synth.init_weights(lay)
    dev = DeviceState(lay.numels, hp, w0, worker_state=False)
    own = torch.empty(dev.ctx.ssd_tensor_table_bytes(), dtype=torch.uint8, device="cuda")
    dev.ctx.ssd_set_tensor_scales(own_lr, own_wd, own)
    ohp = oracle.Hyper(K=K, lr=0.1, m=0.9, W=0, k=0, wd=5e-4, grad_bf16=bf16)
    ref_w, ref_mom = w0.numpy().copy(), np.zeros(dev.n, np.float32)
    for call in range(3):
        grads = [synth.gradient(lay, call, i, 1e-2, device="cuda") for i in range(K)]
        if bf16:
            grads = [synth.to_bf16(g) for g in grads]
        lr_mult = [(0.1 if name.startswith("fc") else 1.0) * (call + 1) for name in lay.names]
        wd_mult = [1.0 if kind == "he" else 0.0 for kind in lay.kinds]
        torch.cuda.synchronize()
        free_before = torch.cuda.mem_get_info()[0]
        if call < 2:
            dev.ctx.ssd_server_sync_update_static(grads, lr_mult, wd_mult)
            ohp.set_tensor_scales(ends, lr_mult, wd_mult)
            if call == 1:                                    # (the first call did the one-time address look-up)
                torch.cuda.synchronize()
                assert torch.cuda.mem_get_info()[0] >= free_before, "the warm call took device memory"
        else:                                                # the ordinary call still uses the context's own table
            dev.ctx.ssd_server_sync_update(grads)
            ohp.set_tensor_scales(ends, own_lr, own_wd)
        torch.cuda.synchronize()
        oracle.server_update(ohp, [oracle_grad(g, bf16) for g in grads], ref_w, ref_mom)
        assert_same(dev.w, ref_w, f"w after call {call}")
        assert_same(dev.mom, ref_mom, f"mom after call {call}")
    assert dev.guards_intact()
