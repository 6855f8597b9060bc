"""Pins for the CPU oracle: what the paper and the mathematics fix, not the oracle itself.

Each test names the passage of arXiv 2012.05396 it is derived from.  None of them
touches a GPU or the CUDA library.
"""
import itertools

import numpy as np
import pytest
import torch

import oracle
from oracle import F_COPY, F_FIRST, F_PULL, F_REFRESH, STAGE_DELAY, STAGE_WARMUP, Hyper, State
from tests import golden_trace

f32 = np.float32


def rng_grads(rng, K, N, scale=1.0):
    return [(rng.standard_normal(N) * scale).astype(f32) for _ in range(K)]


# ---------------------------------------------------------------------------
# hand-computed traces (Algorithms 1 and 2, Sections 3.2.1 and 3.3 end to end)
# ---------------------------------------------------------------------------

@pytest.mark.parametrize("name", golden_trace.ALL)
def test_hand_trace(name):
    tr = golden_trace.load(name)
    h = tr.hp
    K = int(h["K"])
    hp = Hyper(K=K, lr=h["lr"], m=h["m"], W=int(h["W"]), k=int(h["k"]), wd=h["wd"],
               lr_loc=h["lr_loc"], alpha=h["alpha"], beta=h["beta"], rescale=h["rescale"])
    st = State(hp, tr.w0)
    for it in tr.iters:
        stage, flags = st.step([it.grads[i] for i in range(K)])
        assert stage == it.stage and flags == it.flags and st.view == it.view, (name, it.n)
        for key, exp in it.server.items():
            np.testing.assert_array_equal(getattr(st, key), exp, err_msg=f"{name} iter {it.n} {key}")
        for (key, i), exp in it.worker.items():
            np.testing.assert_array_equal(getattr(st, key)[i], exp,
                                          err_msg=f"{name} iter {it.n} {key}[{i}]")
    assert st.iter == len(tr.iters)
    assert st.loc_update == max(0, len(tr.iters) - hp.W)


# ---------------------------------------------------------------------------
# schedule: the d-relative tests equal the printed counters when (1+wp) % k == 0
# ---------------------------------------------------------------------------

def paper_counters(W, k, T):
    """Algorithm 1's `num` and Algorithm 2's `loc_update`, taken literally."""
    wp = W - 1
    num, loc_update, out = 0, 0, []
    for _ in range(T):
        if num <= wp:
            out.append((STAGE_WARMUP, F_COPY if num == wp else 0))
        else:
            flags = 0
            if loc_update == 0:
                flags |= F_FIRST                       # pre_weight initialised with w'
            if loc_update > 0 and loc_update % k == 0:
                flags |= F_REFRESH
            if num % k == k - 1:
                flags |= F_PULL
            loc_update += 1
            out.append((STAGE_DELAY, flags))
        num += 1
    return out


def test_schedule_equals_printed_counters():
    for k in range(1, 9):
        for W in range(k, 33, k):                      # the paper requires (1+wp) % k == 0
            ref = paper_counters(W, k, W + 5 * k + 3)
            got = [oracle.schedule(n, W, k) for n in range(len(ref))]
            assert got == ref, (W, k)


def test_schedule_zero_delay_is_ssgd_forever():
    for W in (0, 1, 5):
        assert all(oracle.schedule(n, W, 0) == (STAGE_WARMUP, 0) for n in range(40))


def test_schedule_period_and_counts():
    # In any window of k delay iterations exactly one pull and (after d=0) one refresh.
    for W, k in itertools.product(range(0, 7), range(1, 7)):
        flags = [oracle.schedule(n, W, k)[1] for n in range(W, W + 6 * k)]
        assert [bool(f & F_PULL) for f in flags] == [(d % k) == k - 1 for d in range(6 * k)]
        assert [bool(f & F_REFRESH) for f in flags] == [d > 0 and d % k == 0 for d in range(6 * k)]
        assert [bool(f & F_FIRST) for f in flags] == [d == 0 for d in range(6 * k)]
        # a refresh always directly follows a pull: it sees a freshly pulled global weight
        for d in range(1, 6 * k):
            if flags[d] & F_REFRESH:
                assert flags[d - 1] & F_PULL


# ---------------------------------------------------------------------------
# server rule: closed forms and library cross-checks (Section 3.2.1, Eq. 1 / Eq. 6)
# ---------------------------------------------------------------------------

def test_server_constant_gradient_closed_form():
    # mom_t = -lr*g*(1-m^(t+1))/(1-m) for constant g, wd = 0 (geometric series of Section 3.2.1)
    lr, m, g0, K, T = 0.1, 0.9, 0.37, 4, 60
    hp = Hyper(K=K, lr=lr, m=m, W=0, k=0)
    lr_, m_ = float(hp.lr), float(hp.m)
    for double, tol in ((True, 1e-13), (False, 2e-5)):
        st = State(hp, np.array([1.5, -0.25], f32), double=double)
        g = np.array([g0, -2 * g0], f32)
        gd = g.astype(np.float64)
        w_ref = st.w.astype(np.float64).copy()
        for t in range(T):
            st.step([g] * K)
            mom_ref = -lr_ * gd * (1 - m_ ** (t + 1)) / (1 - m_)
            w_ref = w_ref + mom_ref
            np.testing.assert_allclose(st.mom, mom_ref, rtol=tol, atol=tol)
            np.testing.assert_allclose(st.w, w_ref, rtol=tol, atol=tol)


def test_server_plain_sgd_special_case():
    # m = 0, wd = 0: Eq. 1 with the descent sign, w <- w - lr * mean_i g_i
    rng = np.random.default_rng(1)
    K, N, T = 5, 33, 7
    hp = Hyper(K=K, lr=0.05, m=0.0, W=0, k=0)
    st = State(hp, rng.standard_normal(N).astype(f32), double=True)
    ref = st.w.copy()
    for _ in range(T):
        gs = rng_grads(rng, K, N)
        st.step(gs)
        # the 1/K factor is the float32-typed `rescale` (0.2 is not a binary fraction)
        mean = np.sum(np.stack(gs).astype(np.float64), axis=0) * float(hp.rescale)
        ref = ref - float(hp.lr) * mean
        np.testing.assert_allclose(st.w, ref, rtol=1e-13, atol=1e-13)
        np.testing.assert_allclose(mean, np.mean(np.stack(gs).astype(np.float64), axis=0), rtol=1e-7)


def test_server_matches_torch_sgd_with_momentum_and_weight_decay():
    # For a constant learning rate torch.optim.SGD (buf = m*buf + g + wd*w; w -= lr*buf) and the
    # paper's rule (mom = m*mom - lr*(g + wd*w); w += mom) are the same recursion with mom = -lr*buf.
    rng = np.random.default_rng(2)
    K, N, T = 3, 17, 25
    hp = Hyper(K=K, lr=0.1, m=0.9, W=0, k=0, wd=0.01)
    w0 = rng.standard_normal(N).astype(f32)
    st = State(hp, w0, double=True)
    p = torch.nn.Parameter(torch.tensor(w0, dtype=torch.float64))
    opt = torch.optim.SGD([p], lr=float(hp.lr), momentum=float(hp.m), weight_decay=float(hp.wd))
    for _ in range(T):
        gs = rng_grads(rng, K, N)
        st.step(gs)
        p.grad = torch.tensor(np.sum(np.stack(gs).astype(np.float64), axis=0) * float(hp.rescale))
        opt.step()
        np.testing.assert_allclose(st.w, p.detach().numpy(), rtol=1e-12, atol=1e-12)


def test_aggregate_K1_and_power_of_two():
    rng = np.random.default_rng(3)
    N = 64
    g = rng.standard_normal(N).astype(f32)
    # K = 1: the aggregate is the single gradient; with lr = 1, m = 0: w = w0 - g exactly (w0 = 0)
    hp = Hyper(K=1, lr=1.0, m=0.0, W=0, k=0)
    st = State(hp, np.zeros(N, f32))
    st.step([g])
    np.testing.assert_array_equal(st.w, -g)
    # K = 2^p equal gradients with short mantissas: every partial sum and the 1/K scaling are exact
    g = np.round(g * 64).astype(f32) / f32(64)
    for K in (2, 4, 8, 16, 32):
        st = State(Hyper(K=K, lr=1.0, m=0.0, W=0, k=0), np.zeros(N, f32))
        st.step([g] * K)
        np.testing.assert_array_equal(st.w, -g)


def test_aggregate_is_left_to_right_and_uses_every_worker():
    # 2^24 + 1 + 1 differs from 1 + 1 + 2^24 in binary32: pins the summation order.
    big, one = f32(2.0 ** 24), f32(1.0)
    hp = Hyper(K=3, lr=1.0, m=0.0, W=0, k=0, rescale=1.0)
    st = State(hp, np.zeros(1, f32))
    st.step([np.array([big], f32), np.array([one], f32), np.array([one], f32)])
    assert st.w[0] == -(big)                           # (2^24 + 1) + 1 -> 2^24 (ties to even twice)
    st = State(hp, np.zeros(1, f32))
    st.step([np.array([one], f32), np.array([one], f32), np.array([big], f32)])
    assert st.w[0] == -(big + f32(2.0))
    # distinct weights per worker: dropping or repeating one changes the result
    st = State(Hyper(K=4, lr=1.0, m=0.0, W=0, k=0, rescale=1.0), np.zeros(1, f32))
    st.step([np.array([v], f32) for v in (1.0, 2.0, 4.0, 8.0)])
    assert st.w[0] == f32(-15.0)


def test_bf16_gradients_widen_exactly():
    rng = np.random.default_rng(4)
    N = 257
    gb = torch.tensor(rng.standard_normal(N).astype(f32)).to(torch.bfloat16)
    bits = gb.view(torch.int16).numpy().view(np.uint16)
    hp = Hyper(K=1, lr=1.0, m=0.0, W=0, k=0, grad_bf16=True)
    st = State(hp, np.zeros(N, f32))
    st.step([bits])
    np.testing.assert_array_equal(st.w, -gb.to(torch.float32).numpy())


# ---------------------------------------------------------------------------
# grad_sync and the GLU rule (Sections 3.2.1, 3.3; Algorithm 2)
# ---------------------------------------------------------------------------

def test_sync_scale():
    hp = Hyper(K=2, lr=0.5, m=0.5, W=1, k=2)
    assert oracle.sync_scale(hp) == 0.5
    hp = Hyper(K=2, lr=0.1, m=0.9, W=4, k=4)
    expect = (1.0 - float(f32(0.9))) / (float(f32(0.1)) * 4)
    assert oracle.sync_scale(hp, double=True) == expect
    assert oracle.sync_scale(hp) == f32(expect)


def test_grad_sync_closed_form_on_refresh_iterations():
    # Constant gradient g, wd = 0.  On a refresh iteration (d > 0, d % k == 0) the local weight is the
    # global weight after n updates and pre_weight the one after n-k updates, so (Section 3.3 with the
    # geometric series of Section 3.2.1)
    #   grad_sync = g * [1 - m^(n-k+1) * (1-m^k) / (k*(1-m))].
    # alpha = 0, beta = 1, lr_loc = 1 makes the GLU step equal to grad_sync itself.
    lr, m, k, W, K = 0.1, 0.9, 4, 4, 2
    hp = Hyper(K=K, lr=lr, m=m, W=W, k=k, lr_loc=1.0, alpha=0.0, beta=1.0)
    lr_, m_ = float(hp.lr), float(hp.m)
    g = np.array([0.3, -1.1, 2.0], f32)
    st = State(hp, np.array([1.0, 2.0, 3.0], f32), double=True)
    seen = 0
    for n in range(W + 6 * k + 1):
        before = [x.copy() for x in st.w_loc]
        _, flags = st.step([g] * K)
        if flags & F_REFRESH:
            factor = 1 - m_ ** (n - k + 1) * (1 - m_ ** k) / (k * (1 - m_))
            for i in range(K):
                # no pull on a refresh iteration when k > 1, so w_loc holds the GLU result
                np.testing.assert_allclose(before[i] - st.w_loc[i], g.astype(np.float64) * factor,
                                           rtol=1e-12, atol=1e-14)
            seen += 1
    assert seen == 6
    # the factor quoted for lr=0.1, m=0.9, k=4 and n=10 updates
    assert abs((1 - 0.9 ** 7 * (1 - 0.9 ** 4) / (4 * 0.1)) - 0.58878424) < 1e-6


def test_glu_sign_and_size_in_steady_state():
    # After a long warm-up with a constant gradient the server moves by -lr*g/(1-m) per step.  With
    # alpha + beta = 1 and lr_loc = lr/(1-m), the GLU step on a refresh iteration (grad_sync -> g)
    # must be that same move: same sign, same size.  The printed '+' would give the opposite.
    lr, m, k, W, K = 0.1, 0.5, 2, 60, 2
    hp = Hyper(K=K, lr=lr, m=m, W=W, k=k, lr_loc=lr / (1 - m), alpha=0.25, beta=0.75)
    g = np.array([0.7, -0.2], f32)
    st = State(hp, np.array([0.0, 5.0], f32), double=True)
    for n in range(W + 2 * k + 1):
        before_loc = st.w_loc[0].copy()
        before_w = st.w.copy()
        _, flags = st.step([g] * K)
        if flags & F_REFRESH:
            worker_move = st.w_loc[0] - before_loc
            server_move = st.w - before_w
            np.testing.assert_allclose(worker_move, server_move, rtol=1e-9)
            np.testing.assert_allclose(server_move,
                                       -float(hp.lr) * g.astype(np.float64) / (1 - float(hp.m)), rtol=1e-9)
            return
    raise AssertionError("no refresh iteration seen")


def test_grad_sync_drift_recurrence_between_pulls():
    # grad_sync is recomputed at every GLU call (Algorithm 2 has no condition on that line).  With
    # x_r = pre_weight - w' before the r-th update after pre_weight was set (x_1 = 0 on the first call):
    #   x_{r+1} = x_r * (1 + lr_loc*beta*c) + lr_loc*alpha*g      (wd = 0, constant own gradient g)
    lr, m, k, W = 0.1, 0.9, 8, 3
    hp = Hyper(K=1, lr=lr, m=m, W=W, k=k)               # lr_loc = 4 lr, alpha = 2, beta = 0.5
    c = oracle.sync_scale(hp, double=True)
    a = 1 + float(hp.lr_loc) * float(hp.beta) * c
    b = float(hp.lr_loc) * float(hp.alpha)
    assert abs(a - (1 + 2 * (1 - float(hp.m)) / k)) < 1e-12   # 1 + 2(1-m)/k for the paper's defaults
    g = np.array([0.01, -0.03], f32)
    st = State(hp, np.array([1.0, -1.0], f32), double=True)
    for _ in range(W):
        st.step([g])
    x = np.zeros(2)
    for d in range(k - 1):                               # up to, not including, the pull iteration
        st.step([g])
        x = x * a + b * g.astype(np.float64)
        np.testing.assert_allclose(st.pre[0] - st.w_loc[0], x, rtol=1e-12, atol=1e-15)


def test_glu_first_call_and_reductions():
    rng = np.random.default_rng(5)
    N = 19
    w0 = rng.standard_normal(N).astype(f32)
    g = rng.standard_normal(N).astype(f32)
    # first call: grad_sync = 0, pre_weight = w'  ->  w' - lr_loc*(alpha*g + wd*w')
    hp = Hyper(K=1, lr=0.1, m=0.9, W=0, k=3, wd=0.125, lr_loc=0.5, alpha=2.0, beta=0.5)
    wl, pre, wdv = w0.copy(), np.full(N, 77.0, f32), np.zeros(N, f32)
    oracle.glu_update(hp, g, wl, pre, wdv, None, F_FIRST)
    np.testing.assert_array_equal(pre, w0)
    np.testing.assert_array_equal(wl, w0 - f32(0.5) * (f32(2.0) * g + f32(0.125) * w0))
    # alpha = 1, beta = 0, wd = 0: Eq. 5, plain local SGD, independent of pre_weight
    hp = Hyper(K=1, lr=0.1, m=0.9, W=0, k=3, lr_loc=0.25, alpha=1.0, beta=0.0)
    for seed in (0, 1):
        wl = w0.copy()
        pre = np.random.default_rng(seed).standard_normal(N).astype(f32)
        oracle.glu_update(hp, g, wl, pre, wdv, None, 0)
        np.testing.assert_array_equal(wl, w0 - f32(0.25) * g)
    # general call against the formula evaluated in double
    hp = Hyper(K=1, lr=0.1, m=0.9, W=0, k=4, wd=0.01, lr_loc=0.4, alpha=2.0, beta=0.5)
    pre = rng.standard_normal(N).astype(f32)
    wl = w0.astype(np.float64)
    pre64 = pre.astype(np.float64)
    oracle.glu_update(hp, g, wl, pre64, wdv.astype(np.float64), None, 0)
    c = (1 - float(hp.m)) / (float(hp.lr) * 4)
    w64 = w0.astype(np.float64)
    ref = w64 - float(hp.lr_loc) * (2.0 * g.astype(np.float64) + float(hp.wd) * w64
                                    + 0.5 * (pre.astype(np.float64) - w64) * c)
    np.testing.assert_allclose(wl, ref, rtol=1e-13, atol=1e-13)
    np.testing.assert_array_equal(pre64, pre.astype(np.float64))     # no refresh: untouched


def test_refresh_uses_old_pre_weight_then_stores_pre_update_weight():
    hp = Hyper(K=1, lr=0.5, m=0.5, W=0, k=1, lr_loc=1.0, alpha=0.0, beta=1.0)   # c = 1
    wl, pre, wdv = np.array([3.0], f32), np.array([5.0], f32), np.zeros(1, f32)
    oracle.glu_update(hp, np.zeros(1, f32), wl, pre, wdv, None, F_REFRESH)
    assert wl[0] == 3.0 - (5.0 - 3.0) and pre[0] == 3.0


def test_pull_keeps_glu_result_for_devices_and_takes_global_weight():
    hp = Hyper(K=1, lr=0.5, m=0.5, W=0, k=1, lr_loc=1.0, alpha=1.0, beta=0.0)
    wl, pre, wdv = np.array([3.0], f32), np.array([3.0], f32), np.zeros(1, f32)
    oracle.glu_update(hp, np.array([0.5], f32), wl, pre, wdv, np.array([9.0], f32), F_PULL)
    assert wdv[0] == 2.5 and wl[0] == 9.0


# ---------------------------------------------------------------------------
# invariants of the whole schedule
# ---------------------------------------------------------------------------

def run_config(hp, w0, grads_per_iter, double=False):
    st = State(hp, w0, double=double)
    log = []
    for gs in grads_per_iter:
        stage, flags = st.step(gs)
        log.append((stage, flags, st.view, st.w.copy(), st.mom.copy(),
                    [x.copy() for x in st.w_loc], [x.copy() for x in st.pre]))
    return st, log


def test_server_trajectory_independent_of_delay_and_warmup():
    # "The process of parameter server keeps unchanged when compared to SSGD" (Section 3.4).
    rng = np.random.default_rng(6)
    K, N, T = 3, 21, 24
    w0 = rng.standard_normal(N).astype(f32)
    stream = [rng_grads(rng, K, N) for _ in range(T)]
    ref, _ = run_config(Hyper(K=K, lr=0.1, m=0.9, W=0, k=0, wd=0.001), w0, stream)
    for W, k in ((0, 1), (1, 1), (2, 4), (5, 4), (8, 8), (3, 2)):
        st, _ = run_config(Hyper(K=K, lr=0.1, m=0.9, W=W, k=k, wd=0.001), w0, stream)
        np.testing.assert_array_equal(st.w, ref.w)
        np.testing.assert_array_equal(st.mom, ref.mom)


def test_pull_and_pre_weight_invariants():
    rng = np.random.default_rng(7)
    K, N, T = 4, 13, 30
    w0 = rng.standard_normal(N).astype(f32)
    for W, k in ((2, 4), (5, 4), (1, 1), (4, 2), (0, 3)):
        hp = Hyper(K=K, lr=0.1, m=0.9, W=W, k=k, wd=0.01)
        stream = [rng_grads(rng, K, N, 1e-2) for _ in range(T)]
        _, log = run_config(hp, w0, stream)
        for n, (stage, flags, view, w, mom, w_loc, pre) in enumerate(log):
            if (stage == STAGE_WARMUP and flags & F_COPY) or flags & F_PULL:
                for i in range(K):
                    np.testing.assert_array_equal(w_loc[i], w)       # w' overwritten by the pull
            if stage == STAGE_DELAY:
                for i in range(1, K):
                    np.testing.assert_array_equal(pre[i], pre[0])    # "the same pre_weight"
            if stage == STAGE_DELAY and not flags & F_PULL and K > 1:
                assert any(not np.array_equal(w_loc[i], w_loc[0]) for i in range(1, K))


def test_device_weights_are_an_output_nothing_reads():
    # Algorithm 1 broadcasts the local update's result to the devices and, on a pull iteration,
    # overwrites the local weight right after.  Nothing in the method reads the device weights back,
    # so scrambling them after every iteration must leave w, mom, every local weight and every
    # pre_weight untouched.  (This is what lets a caller keep ONE buffer per worker for both: the
    # result of a pull iteration's local update is then simply never produced.)
    rng = np.random.default_rng(21)
    K, N, T = 3, 17, 26
    w0 = rng.standard_normal(N).astype(f32)
    for W, k in ((0, 1), (2, 1), (1, 3), (4, 4)):
        hp = Hyper(K=K, lr=0.1, m=0.9, W=W, k=k, wd=0.01)
        stream = [rng_grads(rng, K, N, 1e-2) for _ in range(T)]
        _, clean = run_config(hp, w0, stream)
        st = State(hp, w0)
        pulls = 0
        for n, gs in enumerate(stream):
            stage, flags = st.step(gs)
            if stage == STAGE_DELAY and flags & F_PULL:
                pulls += 1
                for i in range(K):                       # on a pull the two differ: GLU result vs pulled weight
                    assert not np.array_equal(st.w_dev[i], st.w_loc[i])
            for i in range(K):
                st.w_dev[i][:] = rng.standard_normal(N).astype(f32)
            _, _, _, w, mom, w_loc, pre = clean[n]
            np.testing.assert_array_equal(st.w, w)
            np.testing.assert_array_equal(st.mom, mom)
            for i in range(K):
                np.testing.assert_array_equal(st.w_loc[i], w_loc[i])
                np.testing.assert_array_equal(st.pre[i], pre[i])
        assert pulls >= 3


def test_zero_delay_reduces_to_ssgd():
    rng = np.random.default_rng(8)
    K, N, T = 2, 9, 10
    w0 = rng.standard_normal(N).astype(f32)
    stream = [rng_grads(rng, K, N) for _ in range(T)]
    st, log = run_config(Hyper(K=K, lr=0.1, m=0.9, W=3, k=0), w0, stream)
    assert all(stage == STAGE_WARMUP and flags == 0 and view == oracle.VIEW_GLOBAL
               for stage, flags, view, *_ in log)
    for i in range(K):
        np.testing.assert_array_equal(st.w_loc[i], w0)               # never written
    assert st.loc_update == 0 and st.iter == T


# ---------------------------------------------------------------------------
# brute force: an independent scalar re-implementation on tiny inputs
# ---------------------------------------------------------------------------

def brute_force(K, lr, m, wd, W, k, lr_loc, alpha, beta, w0, stream):
    """Scalar numpy.float32 loops written from the paper's equations, element by element."""
    lr, m, wd, lr_loc, alpha, beta = (f32(x) for x in (lr, m, wd, lr_loc, alpha, beta))
    inv_k = f32(1.0 / K)
    c = f32((1.0 - float(m)) / (float(lr) * k)) if k > 0 else f32(0)
    N = len(w0)
    w = [f32(x) for x in w0]
    mom = [f32(0)] * N
    w_loc = [[f32(x) for x in w0] for _ in range(K)]
    pre = [[None] * N for _ in range(K)]
    w_dev = [[None] * N for _ in range(K)]
    for n, grads in enumerate(stream):
        for j in range(N):
            acc = f32(grads[0][j])
            for i in range(1, K):
                acc = f32(acc + f32(grads[i][j]))
            grad = f32(acc * inv_k)
            mom[j] = f32(f32(m * mom[j]) - f32(lr * f32(grad + f32(wd * w[j]))))
            w[j] = f32(w[j] + mom[j])
        if k == 0 or n < W:
            if k != 0 and n == W - 1:
                for i in range(K):
                    w_loc[i] = list(w)
            continue
        d = n - W
        for i in range(K):
            for j in range(N):
                if d == 0:
                    pre[i][j] = w_loc[i][j]
                gsync = f32(f32(pre[i][j] - w_loc[i][j]) * c)
                if d > 0 and d % k == 0:
                    pre[i][j] = w_loc[i][j]
                inner = f32(f32(f32(alpha * f32(grads[i][j])) + f32(wd * w_loc[i][j])) + f32(beta * gsync))
                w_loc[i][j] = f32(w_loc[i][j] - f32(lr_loc * inner))
                if d % k == k - 1:
                    w_dev[i][j] = w_loc[i][j]
                    w_loc[i][j] = w[j]
    return w, mom, w_loc, pre, w_dev


def test_brute_force_all_small_schedules():
    rng = np.random.default_rng(9)
    N, T = 5, 12
    for W, k in itertools.product(range(5), range(5)):
        for K in (1, 2, 3, 4):
            w0 = rng.standard_normal(N).astype(f32)
            stream = [rng_grads(rng, K, N, 0.1) for _ in range(T)]
            hp = Hyper(K=K, lr=0.1, m=0.9, W=W, k=k, wd=0.01)
            st, _ = run_config(hp, w0, stream)
            w, mom, w_loc, pre, w_dev = brute_force(K, 0.1, 0.9, 0.01, W, k, float(hp.lr_loc), 2.0, 0.5,
                                                    w0, stream)
            np.testing.assert_array_equal(st.w, np.array(w, f32))
            np.testing.assert_array_equal(st.mom, np.array(mom, f32))
            for i in range(K):
                np.testing.assert_array_equal(st.w_loc[i], np.array(w_loc[i], f32))
                if pre[i][0] is not None:
                    np.testing.assert_array_equal(st.pre[i], np.array(pre[i], f32))
                if w_dev[i][0] is not None:
                    np.testing.assert_array_equal(st.w_dev[i], np.array(w_dev[i], f32))


def test_float32_tracks_double_shadow():
    # The fp32 oracle and its fp64 shadow stay within a few ulps per iteration of each other.
    rng = np.random.default_rng(10)
    K, N, T = 4, 101, 20
    w0 = rng.standard_normal(N).astype(f32)
    stream = [rng_grads(rng, K, N, 1e-2) for _ in range(T)]
    hp = Hyper(K=K, lr=0.1, m=0.9, W=2, k=4)
    a, _ = run_config(hp, w0, stream)
    b, _ = run_config(hp, w0, stream, double=True)
    np.testing.assert_allclose(a.w, b.w, rtol=1e-5, atol=1e-6)
    for i in range(K):
        np.testing.assert_allclose(a.w_loc[i], b.w_loc[i], rtol=1e-4, atol=1e-5)


# ---------------------------------------------------------------------------
# per-tensor multipliers: they must reduce to uniform runs on each tensor's slice
# ---------------------------------------------------------------------------

def per_tensor_composition_holds():
    """A run with per-tensor multipliers equals, tensor by tensor (padding included), a uniform run
    whose lr, lr_loc and wd are the tensor's products.  Returns False on the first mismatch."""
    rng = np.random.default_rng(11)
    K, W, k, T = 3, 2, 2, 9
    ends = np.array([8, 12, 24], np.int64)           # tensors of 5, 1 and 10 elements, padded to 4s
    lr_mult = np.array([1.0, 0.5, 2.0], f32)
    wd_mult = np.array([1.0, 0.0, 3.0], f32)
    N = int(ends[-1])
    w0 = rng.standard_normal(N).astype(f32)
    stream = [rng_grads(rng, K, N, 0.1) for _ in range(T)]
    hp = Hyper(K=K, lr=0.1, m=0.9, W=W, k=k, wd=0.01)
    hp.set_tensor_scales(ends, lr_mult, wd_mult)
    full = State(hp, w0)
    for gs in stream:
        full.step(gs)
    lo = 0
    for t, hi in enumerate(ends):
        hi = int(hi)
        one = Hyper(K=K, lr=f32(0.1) * lr_mult[t], m=0.9, W=W, k=k, wd=f32(0.01) * wd_mult[t],
                    lr_loc=hp.lr_loc * lr_mult[t])
        part = State(one, w0[lo:hi])
        for gs in stream:
            part.step([np.ascontiguousarray(g[lo:hi]) for g in gs])
        same = np.array_equal(full.w[lo:hi], part.w) and np.array_equal(full.mom[lo:hi], part.mom)
        for i in range(K):
            same = same and np.array_equal(full.w_loc[i][lo:hi], part.w_loc[i]) \
                and np.array_equal(full.pre[i][lo:hi], part.pre[i]) \
                and np.array_equal(full.w_dev[i][lo:hi], part.w_dev[i])
        if not same:
            return False
        lo = hi
    # a gathered sample of the arena, told where its elements sit, follows the same trajectories
    idx = np.array([0, 4, 7, 8, 11, 12, 23], np.int64)
    hs = Hyper(K=K, lr=0.1, m=0.9, W=W, k=k, wd=0.01)
    hs.set_tensor_scales(ends, lr_mult, wd_mult, arena_index=idx)
    samp = State(hs, w0[idx])
    for gs in stream:
        samp.step([np.ascontiguousarray(g[idx]) for g in gs])
    return bool(np.array_equal(samp.w, full.w[idx]) and np.array_equal(samp.w_loc[1], full.w_loc[1][idx])
                and np.array_equal(samp.pre[2], full.pre[2][idx]))


def test_per_tensor_multipliers_compose_from_uniform_runs():
    assert per_tensor_composition_holds()


def test_unit_multipliers_equal_the_uniform_path():
    rng = np.random.default_rng(12)
    K, N, T = 2, 16, 9
    w0 = rng.standard_normal(N).astype(f32)
    stream = [rng_grads(rng, K, N, 0.1) for _ in range(T)]
    a, _ = run_config(Hyper(K=K, lr=0.1, m=0.9, W=1, k=3, wd=0.01), w0, stream)
    hp = Hyper(K=K, lr=0.1, m=0.9, W=1, k=3, wd=0.01)
    hp.set_tensor_scales([4, 16], [1.0, 1.0], [1.0, 1.0])
    b, _ = run_config(hp, w0, stream)
    np.testing.assert_array_equal(a.w, b.w)
    for i in range(K):
        np.testing.assert_array_equal(a.w_loc[i], b.w_loc[i])
        np.testing.assert_array_equal(a.pre[i], b.pre[i])


def test_server_trajectory_independent_of_schedule_with_multipliers_and_lr_changes():
    # the server never sees the delay mechanism, also with per-tensor values and an lr schedule
    rng = np.random.default_rng(13)
    K, N, T = 2, 12, 15
    w0 = rng.standard_normal(N).astype(f32)
    stream = [rng_grads(rng, K, N) for _ in range(T)]

    def run(W, k):
        hp = Hyper(K=K, lr=0.1, m=0.9, W=W, k=k, wd=0.01)
        hp.set_tensor_scales([4, 12], [1.0, 0.25], [0.0, 1.0])
        st = State(hp, w0)
        for n, gs in enumerate(stream):
            if n == 6:
                hp.lr = f32(0.05)                     # a step of the learning-rate schedule
                hp.lr_loc = f32(0.2)
            st.step(gs)
        return st
    ref = run(0, 0)
    for W, k in ((2, 4), (3, 1), (0, 2)):
        st = run(W, k)
        np.testing.assert_array_equal(st.w, ref.w)
        np.testing.assert_array_equal(st.mom, ref.mom)


# ---------------------------------------------------------------------------
# plain SGD as the workers' local updater (Eq. 5; compared with GLU in Section 4.4)
# ---------------------------------------------------------------------------

def test_local_sgd_updater_is_eq5_and_never_touches_pre_weight():
    rng = np.random.default_rng(14)
    K, N, W, k, T = 3, 11, 2, 3, 12
    w0 = rng.standard_normal(N).astype(f32)
    stream = [rng_grads(rng, K, N, 0.1) for _ in range(T)]
    hp = Hyper(K=K, lr=0.1, m=0.9, W=W, k=k, wd=0.01, lr_loc=0.25, local_sgd=True)
    st = State(hp, w0, fill=123.0)
    shadow = None                                  # Eq. 5 in double, worker 1
    for n, gs in enumerate(stream):
        before = st.w_loc[1].astype(np.float64)
        stage, flags = st.step(gs)
        if stage == STAGE_DELAY:
            expect = before - 0.25 * (gs[1].astype(np.float64) + float(hp.wd) * before)
            got = st.w_dev[1] if flags & F_PULL else st.w_loc[1]
            np.testing.assert_allclose(got, expect, rtol=1e-6, atol=1e-7)
            if flags & F_PULL:
                np.testing.assert_array_equal(st.w_loc[1], st.w)
    for i in range(K):
        assert np.all(st.pre[i] == f32(123.0))      # no pre_weight in this updater
    # and the server does not care which local updater the workers use
    ref, _ = run_config(Hyper(K=K, lr=0.1, m=0.9, W=W, k=k, wd=0.01, lr_loc=0.25), w0, stream)
    np.testing.assert_array_equal(st.w, ref.w)
    np.testing.assert_array_equal(st.mom, ref.mom)


def test_local_sgd_equals_glu_with_alpha_one_beta_zero():
    rng = np.random.default_rng(15)
    K, N, T = 2, 64, 10
    w0 = rng.standard_normal(N).astype(f32)
    stream = [rng_grads(rng, K, N, 0.1) for _ in range(T)]
    a, _ = run_config(Hyper(K=K, lr=0.1, m=0.9, W=1, k=2, wd=0.01, lr_loc=0.3, local_sgd=True), w0, stream)
    b, _ = run_config(Hyper(K=K, lr=0.1, m=0.9, W=1, k=2, wd=0.01, lr_loc=0.3, alpha=1.0, beta=0.0), w0, stream)
    for i in range(K):
        np.testing.assert_array_equal(a.w_loc[i], b.w_loc[i])
        np.testing.assert_array_equal(a.w_dev[i], b.w_dev[i])


def test_brute_force_random_hyper_parameters():
    # the scalar rewrite against the oracle on random hyper-parameters, not only the paper's defaults
    rng = np.random.default_rng(16)
    for _ in range(25):
        K, N, T = int(rng.integers(1, 6)), int(rng.integers(1, 9)), 9
        W, k = int(rng.integers(0, 4)), int(rng.integers(0, 5))
        lr, m = float(rng.uniform(0.01, 0.5)), float(rng.uniform(0.0, 0.95))
        wd, lr_loc = float(rng.uniform(0.0, 0.1)), float(rng.uniform(0.01, 1.0))
        alpha, beta = float(rng.uniform(0.0, 3.0)), float(rng.uniform(0.0, 2.0))
        w0 = rng.standard_normal(N).astype(f32)
        stream = [rng_grads(rng, K, N, 0.1) for _ in range(T)]
        hp = Hyper(K=K, lr=lr, m=m, W=W, k=k, wd=wd, lr_loc=lr_loc, alpha=alpha, beta=beta)
        st, _ = run_config(hp, w0, stream)
        w, mom, w_loc, pre, w_dev = brute_force(K, lr, m, wd, W, k, lr_loc, alpha, beta, w0, stream)
        np.testing.assert_array_equal(st.w, np.array(w, f32))
        np.testing.assert_array_equal(st.mom, np.array(mom, f32))
        for i in range(K):
            np.testing.assert_array_equal(st.w_loc[i], np.array(w_loc[i], f32))
            if pre[i][0] is not None:
                np.testing.assert_array_equal(st.pre[i], np.array(pre[i], f32))
            if w_dev[i][0] is not None:
                np.testing.assert_array_equal(st.w_dev[i], np.array(w_dev[i], f32))


# ---------------------------------------------------------------------------
# the ends of the binary32 range: gradual underflow (no flush to zero), signed zeros,
# overflow to infinity.  The paper is silent on rounding; the reading is IEEE 754
# binary32, round to nearest even, every operation rounded on its own, subnormals kept.
# The expected values are exact rational arithmetic with that rounding written out.
# ---------------------------------------------------------------------------

from fractions import Fraction


def rn32(x: Fraction) -> float:
    """Round a rational to binary32, nearest even, with gradual underflow; overflow gives inf."""
    if x == 0:
        return 0.0
    sign = -1 if x < 0 else 1
    a = abs(x)
    e = -126                                   # exponent of the binade that holds a, subnormals share -126
    while a >= Fraction(2) ** (e + 1):
        e += 1
    quantum = Fraction(2) ** (e - 23)
    q = a / quantum
    n = q.numerator // q.denominator
    rem = q - n
    if rem > Fraction(1, 2) or (rem == Fraction(1, 2) and n % 2 == 1):
        n += 1
    r = n * quantum
    if r >= Fraction(2) ** 128:
        return sign * float("inf")
    return sign * float(r)                     # exact: r has at most 24 significant bits


def _finite(*xs):
    return all(np.isfinite(x) for x in xs)


def xmul(a, b) -> float:
    """binary32 product of two binary32 values (Python floats), exactly rounded."""
    a, b = float(a), float(b)
    if not _finite(a, b):
        with np.errstate(all="ignore"):
            return float(np.float64(a) * np.float64(b))         # inf and NaN rules do not depend on the width
    r = rn32(Fraction(a) * Fraction(b))
    negative = np.signbit(a) != np.signbit(b)
    return -abs(r) if negative else abs(r)                       # also fixes the sign of a zero product


def xadd(a, b) -> float:
    a, b = float(a), float(b)
    if not _finite(a, b):
        with np.errstate(all="ignore"):
            return float(np.float64(a) + np.float64(b))
    exact = Fraction(a) + Fraction(b)
    if exact == 0:                                               # x + (-x) = +0; (-0) + (-0) = -0
        return -0.0 if (a == 0 and b == 0 and np.signbit(a) and np.signbit(b)) else 0.0
    return rn32(exact)


def xsub(a, b) -> float:
    return xadd(a, -float(b))


def exact_server(g, w, mom, lr, m, wd, rescale):
    s = float(g[0])
    for gi in g[1:]:
        s = xadd(s, gi)
    grad = xmul(s, rescale)
    full = xadd(grad, xmul(wd, w))
    step = xmul(lr, full)
    keep = xmul(m, mom)
    mom2 = xsub(keep, step)
    return xadd(w, mom2), mom2


def exact_glu(g, wl, pre, lr_loc, alpha, beta, wd, c):
    gs = xmul(xsub(pre, wl), c)
    mix = xadd(xmul(alpha, g), xmul(wd, wl))
    mix = xadd(mix, xmul(beta, gs))
    return xsub(wl, xmul(lr_loc, mix))


def test_rounding_helper_against_known_values():
    tiny = 2.0 ** -149
    assert rn32(Fraction(1, 3)) == float(f32(1.0) / f32(3.0))
    assert rn32(Fraction(2) ** -150) == 0.0                       # tie between 0 and the smallest subnormal: even
    assert rn32(3 * Fraction(2) ** -150) == 2 * tiny              # tie between 1 and 2 quanta: even
    assert rn32(Fraction(2) ** -150 + Fraction(2) ** -200) == tiny
    assert rn32(Fraction(2) ** 128 - Fraction(2) ** 103) == float("inf")     # half a quantum above the largest
    assert rn32(Fraction(2) ** 128 - Fraction(2) ** 103 - 1) == float(np.finfo(f32).max)
    assert rn32(Fraction(16777217)) == 16777216.0 and rn32(Fraction(16777219)) == 16777220.0


def test_subnormals_are_kept_not_flushed_exact_dyadic_case():
    # every operand and every intermediate is a multiple of 2^-149 below 2^-126 or an exact dyadic
    # product, so nothing is rounded: the results are the exact values of the formulas of
    # Section 3.2.1 and 3.3 and are subnormal.  A flush to zero anywhere gives other numbers.
    u = 2.0 ** -149
    lr, m, wd, K = 0.5, 0.5, 0.25, 2
    g = [f32(24 * u), f32(40 * u)]                               # sum 64u, averaged 32u
    w, mom = f32(1024 * u), f32(-96 * u)                         # wd*w = 256u, lr*(32u+256u) = 144u, m*mom = -48u
    hp = Hyper(K=K, lr=lr, m=m, W=0, k=2, wd=wd, lr_loc=2.0, alpha=2.0, beta=0.5)
    wa, ma = np.array([w], f32), np.array([mom], f32)
    oracle.server_update(hp, [np.array([x], f32) for x in g], wa, ma)
    assert ma[0] == f32(-192 * u) and wa[0] == f32(832 * u)
    assert (float(wa[0]), float(ma[0])) == exact_server(g, w, mom, lr, m, wd, 1.0 / K)
    assert 0 < abs(float(ma[0])) < 2.0 ** -126                   # subnormal results, not zero
    # GLU: c = (1-m)/(lr*k) = 0.5; (pre - w') = 64u, grad_sync = 32u; alpha*g = 48u, wd*w' = 128u,
    # mix = 176u + beta*32u = 192u; w' - lr_loc*192u = 512u - 384u = 128u
    assert oracle.sync_scale(hp) == 0.5
    wl, pre, dev = np.array([512 * u], f32), np.array([576 * u], f32), np.zeros(1, f32)
    oracle.glu_update(hp, np.array([24 * u], f32), wl, pre, dev, None, 0)
    assert wl[0] == f32(128 * u) and pre[0] == f32(576 * u)
    assert float(wl[0]) == exact_glu(f32(24 * u), f32(512 * u), f32(576 * u), 2.0, 2.0, 0.5, wd, 0.5)


def test_range_ends_against_exact_rational_arithmetic():
    # operands drawn from both ends of the binary32 range, with rounding inside the subnormal
    # range, sums that cancel to +0, and overflow to infinity; expected values from exact
    # rational arithmetic rounded to nearest even operation by operation
    u = 2.0 ** -149
    big = float(np.finfo(f32).max)
    pool = [0.0, u, 3 * u, 5 * u, 2.0 ** -127, 2.0 ** -126, 1.5 * 2.0 ** -126, 7 * 2.0 ** -130, 1e-38, 1e-40,
            1.0, 0.1, big, big / 2, 2.0 ** 127, 1e38]
    rng = np.random.default_rng(12)
    lr, m, wd, lr_loc, alpha, beta = 0.1, 0.9, 0.01, 0.4, 2.0, 0.5
    n_sub = n_inf = n_zero = 0
    for K in (1, 2, 3):
        hp = Hyper(K=K, lr=lr, m=m, W=0, k=4, wd=wd, lr_loc=lr_loc, alpha=alpha, beta=beta)
        c = oracle.sync_scale(hp)
        for trial in range(400):
            draw = lambda: f32(rng.choice(pool) * rng.choice([-1.0, 1.0]))
            g = [draw() for _ in range(K)]
            w, mom, wl, pre = draw(), draw(), draw(), draw()
            if trial % 5 == 0:
                pre = wl                                         # grad_sync exactly +0
            exp_w, exp_mom = exact_server(g, w, mom, f32(lr), f32(m), f32(wd), hp.rescale)
            wa, ma = np.array([w], f32), np.array([mom], f32)
            with np.errstate(all="ignore"):
                oracle.server_update(hp, [np.array([x], f32) for x in g], wa, ma)
            if np.isnan(exp_mom) or np.isnan(exp_w):             # inf - inf: only "is a NaN" is defined
                assert np.isnan(ma[0]) or np.isnan(wa[0])
            else:
                assert (float(wa[0]), float(ma[0])) == (exp_w, exp_mom), (K, trial, g, w, mom)
                assert np.signbit(wa[0]) == np.signbit(f32(exp_w))           # the sign of a zero counts too
            exp_wl = exact_glu(g[0], wl, pre, f32(lr_loc), f32(alpha), f32(beta), f32(wd), f32(c))
            la, pa, da = np.array([wl], f32), np.array([pre], f32), np.zeros(1, f32)
            oracle.glu_update(hp, np.array([g[0]], f32), la, pa, da, None, 0)
            if np.isnan(exp_wl):
                assert np.isnan(la[0])
            else:
                assert float(la[0]) == exp_wl and np.signbit(la[0]) == np.signbit(f32(exp_wl)), (K, trial)
            for v in (exp_mom, exp_w, exp_wl):
                n_sub += 0 < abs(v) < 2.0 ** -126
                n_inf += np.isinf(v)
                n_zero += v == 0
    assert n_sub > 200 and n_inf > 50 and n_zero > 10            # the draw really reaches all three regimes
