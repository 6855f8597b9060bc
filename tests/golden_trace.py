"""Reader for the hand-computed traces under tests/golden/.

File grammar (one record per line, '#' starts a comment):
  hp key=value ...          hyper-parameters and schedule
  w0 v v v ...              initial global weight
  iter n                    starts iteration n
  g i v v v ...             worker i's gradient for this iteration
  expect stage warmup|delay
  expect flags none|copy|first|refresh|pull ...
  expect view global|local|device
  expect w|mom v ...        server state after the iteration
  expect w_loc|pre|w_dev i v ...   worker i's state after the iteration
"""
import os

import numpy as np

GOLDEN_DIR = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
FLAG_BITS = {"none": 0, "first": 1, "refresh": 2, "pull": 4, "copy": 8}
STAGES = {"warmup": 0, "delay": 1}
VIEWS = {"global": 0, "local": 1, "device": 2}


class Iteration:
    def __init__(self, n):
        self.n = n
        self.grads = {}
        self.stage = None
        self.flags = None
        self.view = None
        self.server = {}      # name -> array
        self.worker = {}      # (name, i) -> array


class Trace:
    def __init__(self, name):
        self.name = name
        self.hp = {}
        self.w0 = None
        self.iters = []


def _vals(tokens):
    return np.array([float(t) for t in tokens], dtype=np.float32)


def load(name):
    tr = Trace(name)
    cur = None
    with open(os.path.join(GOLDEN_DIR, name)) as fh:
        for raw in fh:
            line = raw.split("#", 1)[0].strip()
            if not line:
                continue
            tok = line.split()
            if tok[0] == "hp":
                for kv in tok[1:]:
                    k, v = kv.split("=")
                    tr.hp[k] = float(v)
            elif tok[0] == "w0":
                tr.w0 = _vals(tok[1:])
            elif tok[0] == "iter":
                cur = Iteration(int(tok[1]))
                assert cur.n == len(tr.iters)
                tr.iters.append(cur)
            elif tok[0] == "g":
                cur.grads[int(tok[1])] = _vals(tok[2:])
            elif tok[0] == "expect":
                what = tok[1]
                if what == "stage":
                    cur.stage = STAGES[tok[2]]
                elif what == "flags":
                    cur.flags = sum(FLAG_BITS[t] for t in tok[2:])
                elif what == "view":
                    cur.view = VIEWS[tok[2]]
                elif what in ("w", "mom"):
                    cur.server[what] = _vals(tok[2:])
                elif what in ("w_loc", "pre", "w_dev"):
                    cur.worker[(what, int(tok[2]))] = _vals(tok[3:])
                else:
                    raise ValueError(line)
            else:
                raise ValueError(line)
    return tr


ALL = ("trace_wd0_K2_k2.txt", "trace_wd_K3_k1.txt")
