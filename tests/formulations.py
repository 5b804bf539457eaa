"""Two other ways to compute what a thread may attend to, used only to pin the oracle.

`TokenGraph` is the paper's own picture (Section 3 "Efficiency", Fig. 2b/2c): one token-granular
pool whose slots are filled in decode order, interleaved between threads, and a graph in which
every token points to "the very next token that may attend to it"; a token attends to itself and
to every ancestor reached by walking those edges backwards.  Attention is a dense masked softmax
over the whole pool.  No pages, no streams, no segment lists.

`NaiveRows` is the layout the paper's Appendix B describes in order to reject it: every thread is
a dense row, the prefix is duplicated into each fork's row, and at synchronisation each chunk is
copied into the main row right after its <promise/>.  Attention is plain causal attention over
the row.

Both replay the same workload scripts as the oracle, with their own bookkeeping.
"""
from __future__ import annotations

import numpy as np

from pasta_workloads import run_tensors, step_tensors


def _f64(t):
    import torch
    return t.detach().to("cpu", torch.float32).numpy().astype(np.float64)


def dense_softmax_attention(q, k, v, mask=None):
    """q [Hq, d], k/v [n, Hkv, d] fp64, mask [n] bool -> o [Hq, d], lse [Hq].  Masked dense softmax."""
    hq, d = q.shape
    group = hq // k.shape[1]
    o = np.zeros((hq, d))
    lse = np.zeros(hq)
    for h in range(hq):
        s = k[:, h // group, :] @ q[h] / np.sqrt(d)
        if mask is not None:
            s = np.where(mask, s, -np.inf)
        m = s.max()
        e = np.exp(s - m)
        o[h] = (e / e.sum()) @ v[:, h // group, :]
        lse[h] = m + np.log(e.sum())
    return o, lse


class TokenGraph:
    def __init__(self, script, layer=0):
        self.script, self.layer = script, layer
        geo = script.geometry
        self.parents = []          # node -> list of parent nodes
        self.slot_of = []          # node -> pool slot i, or -1 for a join node (not a token)
        self.k, self.v = [], []    # per slot
        self.last = {}             # (req, thread) -> node the thread's next token hangs from (or None)
        self.owner = []            # slot -> (req, thread)
        self.geo = geo
        self.finished, self.merged = set(), set()   # only to resolve "merge every finished fork"

    def _token(self, key, k, v):
        node = len(self.parents)
        self.parents.append([] if self.last[key] is None else [self.last[key]])
        self.slot_of.append(len(self.k))
        self.k.append(k); self.v.append(v); self.owner.append(key)
        self.last[key] = node
        return node

    def visible(self, key):
        """Pool slots the thread's newest token may attend to (itself included)."""
        seen, stack = set(), [] if self.last[key] is None else [self.last[key]]
        while stack:
            n = stack.pop()
            if n in seen:
                continue
            seen.add(n)
            stack.extend(self.parents[n])
        return sorted(self.slot_of[n] for n in seen if self.slot_of[n] >= 0)

    def apply(self, i):
        op = self.script.ops[i]
        kind = op[0]
        if kind == "begin":
            self.last[(op[1], 0)] = None
        elif kind == "end":
            for key in [k for k in self.last if k[0] == op[1]]:
                del self.last[key]
            self.finished = {k for k in self.finished if k[0] != op[1]}
            self.merged = {k for k in self.merged if k[0] != op[1]}
        elif kind == "spawn":
            self.last[(op[1], op[2])] = self.last[(op[1], 0)]
        elif kind == "finish":
            self.finished.add((op[1], op[2]))
        elif kind == "merge":
            req = op[1]
            forks = op[2]
            if forks is None:
                forks = self._finished_unmerged(req)
            node = len(self.parents)
            ps = [self.last[(req, t)] for t in (0,) + tuple(forks)]
            self.parents.append([p for p in ps if p is not None])
            self.slot_of.append(-1)
            self.last[(req, 0)] = node
            self.merged.update((req, t) for t in forks)
        elif kind == "run":
            k, v = run_tensors(self.script, i, self.layer)
            k, v = _f64(k), _f64(v)
            for j in range(op[3]):
                self._token((op[1], op[2]), k[j], v[j])
        elif kind == "step":
            k, v, q = step_tensors(self.script, i, self.layer)
            k, v, q = _f64(k), _f64(v), _f64(q)
            j = 0
            for req, t, n_new in op[1]:
                if n_new:
                    self._token((req, t), k[j], v[j]); j += 1
            K, V = np.stack(self.k), np.stack(self.v)
            outs, lses = [], []
            for row, (req, t, _n) in enumerate(op[1]):
                mask = np.zeros(len(self.k), dtype=bool)
                mask[self.visible((req, t))] = True
                o, l = dense_softmax_attention(q[row], K, V, mask)
                outs.append(o); lses.append(l)
            return np.stack(outs), np.stack(lses)
        return None

    def run_all(self):
        outs = {}
        for i, op in enumerate(self.script.ops):
            r = self.apply(i)
            if r is not None:
                outs[i] = r
        return outs

    def _finished_unmerged(self, req):
        return tuple(sorted(t for (r, t) in self.finished if r == req and (r, t) not in self.merged))


class NaiveRows:
    """One dense row of (k, v) per thread; prefix duplicated at spawn; chunks copied in at sync."""

    def __init__(self, script, layer=0):
        self.script, self.layer = script, layer
        self.rows = {}        # (req, thread) -> list of (k, v, tag); tag identifies promise positions
        self.cut = {}         # (req, fork) -> index in the main ROW right after its promise at spawn time
        self.own = {}         # (req, fork) -> number of own tokens at the end of its row
        self.finished, self.merged = set(), set()

    def run_all(self):
        outs = {}
        s = self.script
        for i, op in enumerate(s.ops):
            kind = op[0]
            if kind == "begin":
                self.rows[(op[1], 0)] = []
            elif kind == "end":
                for d in (self.rows, self.cut, self.own):
                    for key in [k for k in d if k[0] == op[1]]:
                        del d[key]
                self.finished = {k for k in self.finished if k[0] != op[1]}
                self.merged = {k for k in self.merged if k[0] != op[1]}
            elif kind == "spawn":
                key = (op[1], op[2])
                main = self.rows[(op[1], 0)]
                self.rows[key] = list(main)                 # the duplicated prefix
                self.cut[key] = len(main)
                self.own[key] = 0
            elif kind == "finish":
                self.finished.add((op[1], op[2]))
            elif kind == "merge":
                req = op[1]
                forks = op[2] if op[2] is not None else tuple(sorted(
                    t for (r, t) in self.finished if r == req and (r, t) not in self.merged))
                main = self.rows[(req, 0)]
                # insert later promises first so that earlier insertion points stay valid; among forks
                # with the same insertion point the smaller id must end up first
                for t in sorted(forks, key=lambda t: (self.cut[(req, t)], t), reverse=True):
                    key = (req, t)
                    n = self.own[key]
                    chunk = self.rows[key][len(self.rows[key]) - n:] if n else []
                    at = self.cut[key]
                    main[at:at] = chunk
                    # every insertion point at or after `at` that belongs to a later position moves right
                    for other in self.cut:
                        if other[0] == req and other != key and other not in self.merged and (
                                self.cut[other] > at or (self.cut[other] == at and other[1] > t)):
                            self.cut[other] += len(chunk)
                    self.merged.add(key)
            elif kind == "run":
                k, v = run_tensors(s, i, self.layer)
                k, v = _f64(k), _f64(v)
                key = (op[1], op[2])
                for j in range(op[3]):
                    self.rows[key].append((k[j], v[j]))
                if op[2] != 0:
                    self.own[key] += op[3]
            elif kind == "step":
                k, v, q = step_tensors(s, i, self.layer)
                k, v, q = _f64(k), _f64(v), _f64(q)
                j = 0
                for req, t, n_new in op[1]:
                    if n_new:
                        self.rows[(req, t)].append((k[j], v[j])); j += 1
                        if t != 0:
                            self.own[(req, t)] += 1
                o_all, l_all = [], []
                for row, (req, t, _n) in enumerate(op[1]):
                    r = self.rows[(req, t)]
                    K = np.stack([x[0] for x in r]); V = np.stack([x[1] for x in r])
                    o, l = dense_softmax_attention(q[row], K, V)
                    o_all.append(o); l_all.append(l)
                outs[i] = (np.stack(o_all), np.stack(l_all))
        return outs
