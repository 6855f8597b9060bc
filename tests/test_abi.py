"""Host-side checks of the C ABI that need no GPU: exports, validation, schedule, counters."""
import ctypes as C
import math
import os
import re

import pytest

import oracle
from paper_2012_05396_b200 import binding as B
from paper_2012_05396_b200 import build as libbuild

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module", autouse=True)
def built():
    libbuild.build_library()


def fake_ptrs(K, base=0x10000000, step=0x1000000):
    """Aligned, distinct, never dereferenced addresses (no launch happens in this file)."""
    a = [base + i * step for i in range(2 + 3 * K)]
    return a[0], a[1], a[2:2 + K], a[2 + K:2 + 2 * K], a[2 + 2 * K:]


def make_ctx(K=4, W=2, k=4, numels=(10, 7, 64), **kw):
    w, mom, wl, pre, wdv = fake_ptrs(K)
    hp = B.make_hparams(K, kw.pop("lr", 0.1), kw.pop("momentum", 0.9), W, k, **kw)
    return B.Context(numels, hp, w, mom, wl, pre, wdv)


def test_library_exports_every_declared_symbol():
    header = open(os.path.join(ROOT, "include", "ssd_sgd.h")).read()
    header = re.sub(r"/\*.*?\*/", "", header, flags=re.S)
    declared = set(re.findall(r"\b(ssd_[a-z_0-9]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    raw = C.CDLL(B.LIB_PATH)
    for name in declared:
        assert getattr(raw, name) is not None


def test_status_strings():
    L = B.lib()
    texts = [L.ssd_status_str(s).decode() for s in range(7)]
    assert texts[0] == "ok" and len(set(texts)) == 7
    assert L.ssd_status_str(99).decode() == "unknown status"


def test_arena_numel_and_offsets():
    assert B.ssd_arena_numel([10, 7, 64]) == 12 + 8 + 64
    assert B.ssd_arena_numel([1]) == 4
    ctx = make_ctx()
    assert [ctx.ssd_tensor_offset(t) for t in range(3)] == [0, 12, 20]
    with pytest.raises(B.SsdError) as e:
        ctx.ssd_tensor_offset(3)
    assert e.value.status == B.SSD_ERR_ARG
    for bad in ([], [0], [-1, 4], [1 << 40]):
        with pytest.raises(B.SsdError) as e:
            B.ssd_arena_numel(bad)
        assert e.value.status == B.SSD_ERR_LAYOUT


def test_layout_offsets_match_the_generator_module():
    from paper_2012_05396_b200 import synth
    lay = synth.get_layout("resnet56")
    assert B.ssd_arena_numel(lay.numels) == lay.padded_numel
    ctx = make_ctx(numels=lay.numels)
    assert [ctx.ssd_tensor_offset(t) for t in range(lay.num_tensors)] == lay.offsets


@pytest.mark.parametrize("field,value,status", [
    ("K", 0, B.SSD_ERR_ARG), ("K", 33, B.SSD_ERR_ARG), ("lr", 0.0, B.SSD_ERR_ARG),
    ("lr", -1.0, B.SSD_ERR_ARG), ("lr", math.inf, B.SSD_ERR_ARG), ("lr", math.nan, B.SSD_ERR_ARG),
    ("momentum", 1.0, B.SSD_ERR_ARG), ("momentum", -0.1, B.SSD_ERR_ARG),
    ("wd", math.nan, B.SSD_ERR_ARG), ("warmup_iters", -1, B.SSD_ERR_ARG), ("delay_k", -1, B.SSD_ERR_ARG),
    ("grad_dtype", 2, B.SSD_ERR_ARG), ("alpha", math.inf, B.SSD_ERR_ARG), ("local_updater", 2, B.SSD_ERR_ARG),
])
def test_init_rejects_bad_hyper_parameters(field, value, status):
    K = 4
    w, mom, wl, pre, wdv = fake_ptrs(K)
    hp = B.make_hparams(K, 0.1, 0.9, 2, 4)
    setattr(hp, field, value)
    if field == "K" and value > K:
        w, mom, wl, pre, wdv = fake_ptrs(value)
    with pytest.raises(B.SsdError) as e:
        B.Context([16], hp, w, mom, wl, pre, wdv)
    assert e.value.status == status


def test_init_rejects_bad_pointers():
    K = 2
    hp = B.make_hparams(K, 0.1, 0.9, 2, 4)
    w, mom, wl, pre, wdv = fake_ptrs(K)
    with pytest.raises(B.SsdError) as e:
        B.Context([16], hp, w + 4, mom, wl, pre, wdv)
    assert e.value.status == B.SSD_ERR_ALIGN
    with pytest.raises(B.SsdError) as e:
        B.Context([16], hp, w, mom, [wl[0], wl[1] + 8], pre, wdv)
    assert e.value.status == B.SSD_ERR_ALIGN
    with pytest.raises(B.SsdError) as e:
        B.Context([16], hp, w, mom, wl, [pre[0], None], wdv)
    assert e.value.status == B.SSD_ERR_ARG
    with pytest.raises(B.SsdError) as e:                  # two state buffers at one address
        B.Context([16], hp, w, mom, [wl[0], wl[0]], pre, wdv)
    assert e.value.status == B.SSD_ERR_ARG
    with pytest.raises(B.SsdError) as e:
        B.Context([16], hp, w, mom, wl, [pre[0], wl[1]], wdv)
    assert e.value.status == B.SSD_ERR_ARG
    B.Context([16], hp, w, mom, wl, [pre[0], pre[0]], wdv)   # one shared pre_weight for all workers: allowed
    hp3 = B.make_hparams(3, 0.1, 0.9, 2, 4)
    w3, mom3, wl3, pre3, wdv3 = fake_ptrs(3)
    with pytest.raises(B.SsdError) as e:                  # shared by some workers only
        B.Context([16], hp3, w3, mom3, wl3, [pre3[0], pre3[0], pre3[2]], wdv3)
    assert e.value.status == B.SSD_ERR_ARG
    L = B.lib()
    assert L.ssd_init(None, None, None, None) == B.SSD_ERR_ARG
    h = C.c_void_p(123)
    assert L.ssd_init(C.byref(h), None, None, None) == B.SSD_ERR_ARG and not h.value


def test_defaults_and_derived_constants():
    ctx = make_ctx(K=8, W=8, k=4)
    hp, c = ctx.ssd_get_hparams()
    import numpy as np
    f32 = np.float32
    assert hp.lr_local == f32(4.0) * f32(0.1) and hp.alpha == 2.0 and hp.beta == 0.5
    assert hp.rescale == 0.125
    assert c == f32((1.0 - float(f32(0.9))) / (float(f32(0.1)) * 4))
    # the oracle derives the same constant on its own
    assert c == oracle.sync_scale(oracle.Hyper(K=8, lr=0.1, m=0.9, W=8, k=4))
    ctx = make_ctx(K=3, W=1, k=0)
    hp, c = ctx.ssd_get_hparams()
    assert c == 0.0 and hp.rescale == f32(1.0 / 3.0)
    ctx.ssd_set_lr(lr=0.5)
    assert ctx.ssd_get_hparams()[0].lr == 0.5 and ctx.ssd_get_hparams()[0].lr_local == f32(4.0) * f32(0.1)
    ctx = make_ctx(K=2, W=1, k=2, lr=0.5, momentum=0.5)
    assert ctx.ssd_get_hparams()[1] == 0.5
    ctx.ssd_set_lr(lr=0.25, lr_local=3.0)
    hp, c = ctx.ssd_get_hparams()
    assert (hp.lr, hp.lr_local, c) == (0.25, 3.0, 1.0)
    with pytest.raises(B.SsdError):
        ctx.ssd_set_lr(lr=-1.0)


def test_schedule_is_bit_exact_with_the_oracle():
    for W in range(0, 10):
        for k in range(0, 9):
            ctx = make_ctx(K=2, W=W, k=k)
            for n in range(W + 4 * max(k, 1) + 2):
                assert ctx.ssd_schedule(n) == oracle.schedule(n, W, k), (W, k, n)
    ctx = make_ctx()
    with pytest.raises(B.SsdError):
        ctx.ssd_schedule(-1)


def test_counters_advance_and_views():
    W, k = 2, 3
    ctx = make_ctx(K=2, W=W, k=k)
    _, _, wl, _, wdv = fake_ptrs(2)
    w = fake_ptrs(2)[0]
    assert ctx.ssd_get_counters() == (0, 0, B.SSD_STAGE_WARMUP, 0)
    assert ctx.ssd_worker_weights(1) == (w, B.SSD_VIEW_GLOBAL)
    expect_view = []
    for n in range(12):
        stage, flags = ctx.ssd_schedule(n)
        assert ctx.ssd_get_counters()[2:] == (stage, flags)
        ctx.ssd_advance()
        it, lu, _, _ = ctx.ssd_get_counters()
        assert it == n + 1 and lu == max(0, n + 1 - W)
        p, view = ctx.ssd_worker_weights(1)
        if stage == B.SSD_STAGE_WARMUP:
            want = B.SSD_VIEW_LOCAL if flags & B.SSD_FLAG_COPY else B.SSD_VIEW_GLOBAL
        else:
            want = B.SSD_VIEW_DEVICE if flags & B.SSD_FLAG_PULL else B.SSD_VIEW_LOCAL
        assert view == want and p == (w, wl[1], wdv[1])[view]
    # restore: loc_update must be consistent with iter
    ctx.ssd_set_counters(7, 5)
    assert ctx.ssd_get_counters()[:2] == (7, 5)
    with pytest.raises(B.SsdError) as e:
        ctx.ssd_set_counters(7, 4)
    assert e.value.status == B.SSD_ERR_STATE
    ctx0 = make_ctx(K=2, W=2, k=0)
    ctx0.ssd_set_counters(9, 0)
    with pytest.raises(B.SsdError):
        ctx0.ssd_set_counters(9, 7)


def test_call_validation_happens_before_any_launch():
    ctx = make_ctx(K=2, W=0, k=2)
    g = [0x20000000, 0x21000000]
    for bad in (None, [g[0], None]):
        with pytest.raises((B.SsdError, TypeError)):
            ctx.ssd_step(bad if bad is not None else [None, None])
    with pytest.raises(B.SsdError) as e:
        ctx.ssd_step([g[0], g[1] + 2])
    assert e.value.status == B.SSD_ERR_ALIGN
    with pytest.raises(B.SsdError) as e:
        ctx.ssd_worker_glu_update(2, g[0], 0)
    assert e.value.status == B.SSD_ERR_ARG
    with pytest.raises(B.SsdError) as e:
        ctx.ssd_worker_glu_update(0, g[0], 16)
    assert e.value.status == B.SSD_ERR_ARG
    with pytest.raises(B.SsdError) as e:
        ctx.ssd_worker_glu_update(0, g[0] + 1, 0)
    assert e.value.status == B.SSD_ERR_ALIGN
    with pytest.raises(B.SsdError) as e:
        make_ctx(K=2, W=0, k=0).ssd_worker_glu_update(0, g[0], 0)
    assert e.value.status == B.SSD_ERR_STATE
    for t, b in ((32, 1), (48, 1), (1024, 1), (256, 33), (256, -1)):
        with pytest.raises(B.SsdError):
            ctx.ssd_set_launch(t, b)
    ctx.ssd_set_launch(128, 4)
    assert ctx.ssd_get_counters()[0] == 0 and ctx.ssd_kernel_launches() == 0


def test_missing_library_is_a_loud_error(monkeypatch):
    monkeypatch.setattr(B, "_lib", None)
    monkeypatch.setattr(B, "LIB_PATH", "/nonexistent/libssd_sgd.so")
    with pytest.raises(RuntimeError, match="no fallback"):
        B.lib()


def test_tensor_table_size_and_validation():
    ctx = make_ctx(numels=(10, 7, 64))
    assert ctx.ssd_tensor_table_bytes() == 32 + 3 * 16          # 3 ends padded to 16 bytes + 3 float4
    table = 0x30000000
    for lr_mult, wd_mult, tbl, status in (
            ([1.0, 0.0, 1.0], None, table, B.SSD_ERR_ARG),        # a zero lr multiplier has no grad_sync scale
            ([1.0, -1.0, 1.0], None, table, B.SSD_ERR_ARG),
            (None, [1.0, math.inf, 0.0], table, B.SSD_ERR_ARG),
            (None, None, table + 8, B.SSD_ERR_ALIGN)):
        with pytest.raises(B.SsdError) as e:
            ctx.ssd_set_tensor_scales(lr_mult, wd_mult, tbl)
        assert e.value.status == status
    ctx.ssd_set_tensor_scales(None, None, None)                  # uniform: nothing to upload


def test_header_is_valid_c_and_cpp(tmp_path):
    import subprocess
    header = os.path.join(ROOT, "include", "ssd_sgd.h")
    c = tmp_path / "use.c"
    c.write_text('#include "ssd_sgd.h"\nint main(void) { ssd_hparams hp; hp.K = 1; return (int)sizeof(ssd_buffers) * 0 + hp.K - 1; }\n')
    subprocess.check_call(["gcc", "-std=c99", "-pedantic", "-Wall", "-Werror", "-I", os.path.dirname(header),
                           "-c", str(c), "-o", str(tmp_path / "use_c.o")])
    subprocess.check_call(["g++", "-std=c++11", "-Wall", "-Werror", "-I", os.path.dirname(header), "-x", "c++",
                           "-c", str(c), "-o", str(tmp_path / "use_cpp.o")])


def test_launch_overrides_are_set_and_reset_together():
    ctx = make_ctx()
    assert ctx.ssd_get_launch() == (0, 0, 0, 0)
    ctx.ssd_set_launch(256, 3)
    ctx.ssd_set_kernel_shape(16, 2)
    assert ctx.ssd_get_launch() == (256, 3, 16, 2)
    ctx.ssd_set_launch(0, 5)                       # 0 returns the thread count to the default
    assert ctx.ssd_get_launch() == (0, 5, 16, 2)
    ctx.ssd_set_launch(128, 0)
    assert ctx.ssd_get_launch() == (128, 0, 16, 2)
    ctx.ssd_set_launch()
    ctx.ssd_set_kernel_shape()
    assert ctx.ssd_get_launch() == (0, 0, 0, 0)
    with pytest.raises(B.SsdError):
        ctx.ssd_set_kernel_shape(32, 1)


def test_overlapping_buffers_are_rejected():
    K = 2
    hp = B.make_hparams(K, 0.1, 0.9, 2, 4)
    n = 1 << 20                                               # 4 MiB arenas
    w, mom, wl, pre, wdv = fake_ptrs(K, step=n * 4)           # back to back: allowed
    B.Context([n], hp, w, mom, wl, pre, wdv)
    for shift in (16, n * 4 - 16):                            # slices of one slab with a wrong stride
        with pytest.raises(B.SsdError) as e:
            B.Context([n], hp, w, mom + shift - n * 4, wl, pre, wdv)
        assert e.value.status == B.SSD_ERR_ARG
        with pytest.raises(B.SsdError) as e:
            B.Context([n], hp, w, mom, wl, pre, [wdv[0], wl[0] + shift])
        assert e.value.status == B.SSD_ERR_ARG
    ctx = B.Context([n], hp, w, mom, wl, pre, wdv)
    free = wdv[-1] + n * 4
    ok = [free, free + n * 4]
    inside = [[w + 64, ok[1]], [ok[0], pre[1] - 32], [wdv[1] + n * 4 - 16, ok[1]], [ok[0], w - n * 4 + 16]]
    for grads in inside:                                      # a gradient range that reaches into the state
        for call in (ctx.ssd_step, ctx.ssd_server_sync_update):
            with pytest.raises(B.SsdError) as e:
                call(grads)
            assert e.value.status == B.SSD_ERR_ARG
    assert ctx.ssd_kernel_launches() == 0 and ctx.ssd_get_counters()[0] == 0
    ctx0 = B.Context([n], B.make_hparams(K, 0.1, 0.9, 0, 4), w, mom, wl, pre, wdv)
    with pytest.raises(B.SsdError) as e:
        ctx0.ssd_worker_glu_update(0, mom + 4096, 0)
    assert e.value.status == B.SSD_ERR_ARG
    # bfloat16 gradient arenas are half as long: the same start address may be free of the state
    hp16 = B.make_hparams(K, 0.1, 0.9, 2, 4, grad_dtype=B.SSD_BF16)
    ctx16 = B.Context([n], hp16, w, mom, wl, pre, wdv)
    with pytest.raises(B.SsdError) as e:
        ctx16.ssd_server_sync_update([w - n * 2 + 16, ok[0]])
    assert e.value.status == B.SSD_ERR_ARG


def test_merged_device_weights_are_all_or_none():
    # w_dev[i] == w_loc[i] for every worker: accepted, and the view after a pull is the local weight;
    # for some workers only, or a w_dev that merely overlaps a w_loc: rejected
    K, W, k = 3, 1, 2
    hp = B.make_hparams(K, 0.1, 0.9, W, k)
    n = 1 << 12
    w, mom, wl, pre, wdv = fake_ptrs(K)
    ctx = B.Context([n], hp, w, mom, wl, pre, list(wl))
    for it in range(7):
        stage, flags = ctx.ssd_schedule(it)
        ctx.ssd_advance()
        p, view = ctx.ssd_worker_weights(2)
        want = B.SSD_VIEW_GLOBAL if stage == B.SSD_STAGE_WARMUP and not flags & B.SSD_FLAG_COPY else B.SSD_VIEW_LOCAL
        assert (p, view) == ((w, wl[2])[view], want)
    for bad in ([wl[0], wdv[1], wdv[2]], [wdv[0], wdv[1], wl[2]], [wl[1], wl[0], wl[2]], [wl[0] + 16, wdv[1], wdv[2]]):
        with pytest.raises(B.SsdError) as e:
            B.Context([n], hp, w, mom, wl, pre, bad)
        assert e.value.status == B.SSD_ERR_ARG
    # a gradient may not reach into the merged buffers either
    with pytest.raises(B.SsdError) as e:
        ctx.ssd_step([wl[0] + 64, wdv[1], wdv[2]])
    assert e.value.status == B.SSD_ERR_ARG and ctx.ssd_kernel_launches() == 0


def test_host_pre_weight_mode_is_validated():
    K, n = 2, 4096
    hp = B.make_hparams(K, 0.1, 0.9, 0, 2)
    w, mom, wl, pre, wdv = fake_ptrs(K)
    host, slices, grads = 0x7f0000000000, 0x50000000, [0x60000000, 0x61000000]
    with_pre = B.Context([n], hp, w, mom, wl, pre, wdv)
    with pytest.raises(B.SsdError) as e:                       # pre_weight already lives on the device
        with_pre.ssd_set_host_pre_weight(host, slices, 2)
    assert e.value.status == B.SSD_ERR_STATE
    ctx = B.Context([n], hp, w, mom, wl, None, wdv)            # created without pre_weight buffers
    for call in (lambda: ctx.ssd_step(grads), lambda: ctx.ssd_step_tensors(grads, 0, 1),
                 lambda: ctx.ssd_worker_glu_update(0, grads[0], 0), lambda: ctx.ssd_worker_local_step(0, grads[0]),
                 lambda: ctx.ssd_step_host(grads, grads)):
        with pytest.raises(B.SsdError) as e:
            call()
        assert e.value.status == B.SSD_ERR_STATE
    for args, status in (((host, slices, 0), B.SSD_ERR_ARG), ((host, slices, 9), B.SSD_ERR_ARG),
                         ((None, slices, 2), B.SSD_ERR_ARG), ((host, None, 2), B.SSD_ERR_ARG),
                         ((host + 4, slices, 2), B.SSD_ERR_ALIGN), ((host, slices + 8, 2), B.SSD_ERR_ALIGN),
                         ((host, wl[0] - 64, 1), B.SSD_ERR_ARG)):          # slices reaching into the state
        with pytest.raises(B.SsdError) as e:
            ctx.ssd_set_host_pre_weight(*args)
        assert e.value.status == status
    for bad in (1000, 1 << 31, -1024):
        with pytest.raises(B.SsdError):
            ctx.ssd_set_host_chunk(bad)
    ctx.ssd_set_host_chunk(2048)
    ctx.ssd_set_host_pre_weight(host, slices, 2)
    with pytest.raises(B.SsdError) as e:                       # the slices were sized for the chunk
        ctx.ssd_set_host_chunk(4096)
    assert e.value.status == B.SSD_ERR_STATE
    with pytest.raises(B.SsdError) as e:                       # still no device pre_weight for the fused step
        ctx.ssd_step(grads)
    assert e.value.status == B.SSD_ERR_STATE
    ctx.ssd_set_host_pre_weight(None, None, 0)
    ctx.ssd_set_host_chunk(0)
    # without a delay stage, or with the plain-SGD updater, there is no pre_weight to place
    with pytest.raises(B.SsdError) as e:
        B.Context([n], B.make_hparams(K, 0.1, 0.9, 0, 0), w, mom, wl, None, wdv).ssd_set_host_pre_weight(host, slices, 2)
    assert e.value.status == B.SSD_ERR_STATE
    assert ctx.ssd_kernel_launches() == 0


def test_guard_words_catch_a_store_outside_an_arena():
    import torch
    from paper_2012_05396_b200.state import ArenaSlab, GUARD_WORD
    slab = ArenaSlab(3, 1001, torch.float32, "cpu")
    assert all(a.numel() == 1001 and a.data_ptr() % 16 == 0 for a in slab.arenas)
    for a in slab.arenas:
        a.fill_(1.0)                                           # writes inside the arenas leave the guards alone
    assert slab.guards_intact()
    words = slab.raw.view(torch.int32)
    base = slab.raw.data_ptr()
    first_past = (slab.arenas[1].data_ptr() - base) // 4 + 1001
    words[first_past] = 0                                      # one element past the end of arena 1
    assert slab.damaged_gaps() == [2]
    words[first_past] = GUARD_WORD
    words[(slab.arenas[0].data_ptr() - base) // 4 - 1] = 7     # one element before arena 0
    words[-1] = 7                                              # the last word of the allocation
    assert slab.damaged_gaps() == [0, 3]
