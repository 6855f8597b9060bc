"""The pins must notice a plausible mistake anywhere in the oracle.

Each case plants one mistake in a copy of the oracle's C source (a dropped term, a wrong sign, a wrong
index, a swapped operand, an off-by-one in the schedule), builds it on the CPU and checks that the
hand-computed traces or the schedule pin fail.  Nothing here touches a GPU.
"""
import os
import subprocess

import numpy as np
import pytest

import oracle
from tests import golden_trace
from tests.test_oracle_pins import paper_counters, per_tensor_composition_holds
from tests import test_oracle_pins

SRC = os.path.join(os.path.dirname(oracle.__file__), "ssd_oracle.c")

MUTATIONS = [
    ("drops weight decay on the server", "real decay = wd * w[j];\n        real full", "real decay = 0 * w[j];\n        real full"),
    ("adds instead of subtracting the server step", "mom[j] = keep - step;", "mom[j] = keep + step;"),
    ("forgets the momentum term", "real keep = m * mom[j];", "real keep = 0 * mom[j];"),
    ("skips worker 0 in the sum twice", "s = s + grad_at(g[i], hp->grad_bf16, j);", "s = s + grad_at(g[i - 1], hp->grad_bf16, j);"),
    ("drops the rescale", "real grad = s * rescale;", "real grad = s;"),
    ("weight update uses the old momentum", "mom[j] = keep - step;\n        w[j] = w[j] + mom[j];", "w[j] = w[j] + mom[j];\n        mom[j] = keep - step;"),
    ("grad_sync with the wrong sign", "real diff = pre[j] - w_loc[j];", "real diff = w_loc[j] - pre[j];"),
    ("GLU adds instead of subtracting", "w_loc[j] = w_loc[j] - step;", "w_loc[j] = w_loc[j] + step;"),
    ("GLU drops beta * grad_sync", "real global = beta * grad_sync;", "real global = 0 * grad_sync;"),
    ("GLU swaps alpha and beta", "real local = alpha * grad_at(g, hp->grad_bf16, j);", "real local = beta * grad_at(g, hp->grad_bf16, j);"),
    ("GLU drops its weight decay", "real decay = wd * w_loc[j];", "real decay = 0 * w_loc[j];"),
    ("refresh before grad_sync", "real diff = pre[j] - w_loc[j];\n        real grad_sync = diff * c;\n        if (flags & F_REFRESH) pre[j] = w_loc[j];",
     "if (flags & F_REFRESH) pre[j] = w_loc[j];\n        real diff = pre[j] - w_loc[j];\n        real grad_sync = diff * c;"),
    ("refresh stores the updated weight", "if (flags & F_REFRESH) pre[j] = w_loc[j];\n        real local", "real local"),
    ("pull hands the global weight to the devices", "w_dev[j] = w_loc[j];\n            w_loc[j] = w_server[j];", "w_loc[j] = w_server[j];\n            w_dev[j] = w_loc[j];"),
    ("scale uses lr_loc", "s.c = sync_scale_for(hp->lr, hp->m, hp->k);", "s.c = sync_scale_for(hp->lr_loc, hp->m, hp->k);"),
    ("scale forgets k", "((double)lr * (double)k)", "((double)lr)"),
    ("workers use worker 0's gradient", "oracle_glu_update(st->N, hp, g[i],", "oracle_glu_update(st->N, hp, g[0],"),
    ("server runs after the workers", None, None),       # handled below: moves the call
    ("warm-up one iteration short", "n == W - 1) ? F_COPY", "n == W - 2) ? F_COPY"),
    ("pull one iteration early", "d % k == k - 1", "(d + 1) % k == k - 1"),
    ("refresh on the first call", "if (d > 0 && d % k == 0)", "if (d % k == 0)"),
    ("warm-up off by one", "if (k == 0 || n < W)", "if (k == 0 || n <= W)"),
    ("local SGD adds its step", "w_loc[j] = w_loc[j] - step_l;", "w_loc[j] = w_loc[j] + step_l;"),
    ("local SGD forgets weight decay", "real decay_l = wd * w_loc[j];", "real decay_l = 0 * w_loc[j];"),
    ("local SGD uses the server lr", "real step_l = lr_loc * full_l;", "real step_l = (real)hp->lr * full_l;"),
    ("local SGD pull keeps the local result", "w_dev[j] = w_loc[j];\n                w_loc[j] = w_server[j];\n            }\n            continue;", "w_dev[j] = w_server[j];\n            }\n            continue;"),
    ("tensor lookup off by one", "pos >= hp->tensor_end[t]", "pos > hp->tensor_end[t]"),
    ("local lr ignores the tensor's multiplier", "float lr_loc_t = hp->lr_loc * hp->lr_mult[t];", "float lr_loc_t = hp->lr_loc;"),
    ("decay multiplier taken from lr_mult", "float wd_t = hp->wd * hp->wd_mult[t];", "float wd_t = hp->wd * hp->lr_mult[t];"),
    ("server flushes subnormal momenta to zero", "mom[j] = keep - step;",
     "mom[j] = keep - step; if (mom[j] > -1.17549435e-38f && mom[j] < 1.17549435e-38f) mom[j] = 0;"),
    ("GLU flushes a subnormal grad_sync to zero", "real grad_sync = diff * c;",
     "real grad_sync = diff * c; if (grad_sync > -1.17549435e-38f && grad_sync < 1.17549435e-38f) grad_sync = 0;"),
    ("per-tensor scale from the global lr", "s.c = sync_scale_for(lr_t, hp->m, hp->k);", "s.c = sync_scale_for(hp->lr, hp->m, hp->k);"),
]


def mutate(src, old, new, name):
    if name == "server runs after the workers":
        call = "    oracle_server_update(st->N, hp, g, st->w, st->mom);\n"
        assert call in src
        src = src.replace(call, "")
        anchor = "    st->iter += 1;\n"
        return src.replace(anchor, call + anchor)
    if name == "refresh stores the updated weight":
        assert old in src
        src = src.replace(old, new)
        return src.replace("        w_loc[j] = w_loc[j] - step;\n",
                           "        w_loc[j] = w_loc[j] - step;\n        if (flags & F_REFRESH) pre[j] = w_loc[j];\n")
    assert src.count(old) >= 1, name
    return src.replace(old, new, 1)


def traces_pass(lib):
    """True when every hand trace matches with this oracle build."""
    saved = oracle._libs.get(False)
    oracle._libs[False] = lib
    try:
        for name in golden_trace.ALL:
            tr = golden_trace.load(name)
            h = tr.hp
            K = int(h["K"])
            hp = oracle.Hyper(K=K, lr=h["lr"], m=h["m"], W=int(h["W"]), k=int(h["k"]), wd=h["wd"],
                              lr_loc=h["lr_loc"], alpha=h["alpha"], beta=h["beta"], rescale=h["rescale"])
            st = oracle.State(hp, tr.w0)
            for it in tr.iters:
                stage, flags = st.step([it.grads[i] for i in range(K)])
                if (stage, flags, st.view) != (it.stage, it.flags, it.view):
                    return False
                for key, exp in it.server.items():
                    if not np.array_equal(getattr(st, key), exp):
                        return False
                for (key, i), exp in it.worker.items():
                    if not np.array_equal(getattr(st, key)[i], exp):
                        return False
        for k in range(1, 5):
            for W in range(k, 13, k):
                ref = paper_counters(W, k, W + 3 * k + 2)
                if [oracle.schedule(n, W, k) for n in range(len(ref))] != ref:
                    return False
        if not per_tensor_composition_holds():
            return False
        try:
            test_oracle_pins.test_local_sgd_updater_is_eq5_and_never_touches_pre_weight()
            test_oracle_pins.test_local_sgd_equals_glu_with_alpha_one_beta_zero()
            test_oracle_pins.test_subnormals_are_kept_not_flushed_exact_dyadic_case()
        except AssertionError:
            return False
        return True
    finally:
        if saved is not None:
            oracle._libs[False] = saved
        else:
            oracle._libs.pop(False, None)


def build_variant(tmp_path, text, tag):
    c = tmp_path / f"oracle_{tag}.c"
    so = tmp_path / f"oracle_{tag}.so"
    c.write_text(text)
    subprocess.check_call(["gcc", *oracle.CFLAGS, "-o", str(so), str(c)])
    return oracle.bind(str(so), False)


def test_unmodified_source_passes(tmp_path):
    assert traces_pass(build_variant(tmp_path, open(SRC).read(), "clean"))


@pytest.mark.parametrize("idx", range(len(MUTATIONS)))
def test_planted_mistake_is_caught(tmp_path, idx):
    name, old, new = MUTATIONS[idx]
    text = mutate(open(SRC).read(), old, new, name)
    assert text != open(SRC).read(), name
    assert not traces_pass(build_variant(tmp_path, text, str(idx))), f"pins did not notice: {name}"
