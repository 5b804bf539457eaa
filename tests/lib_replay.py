"""Replays a workload script on the CUDA library through its Python binding (tests only)."""
from __future__ import annotations

import numpy as np

from paper_2502_11517_b200 import binding
from pasta_workloads import Script, run_tensors, step_tensors


def make_pool(script: Script, host_only: bool = False, flags: int = 0, layers=None, **kw) -> binding.Pool:
    geo = script.geometry
    if host_only:
        flags |= binding.FLAG_HOST_ONLY
    return binding.Pool(geo.n_layers if layers is None else layers, geo.n_q_heads, geo.n_kv_heads, geo.head_dim,
                        script.n_pages, script.max_requests, script.max_threads_per_request,
                        script.max_segments_per_thread, free_order=script.free_order, flags=flags, **kw)


class LibReplay:
    """Applies operations one by one.  With a device pool, tensors of all layers are appended and
    `apply` returns (out, lse) as torch CUDA tensors [layers, n, Hq, d] / [layers, n, Hq] for steps."""

    def __init__(self, script: Script, pool: binding.Pool, layers=None, rope_theta=None):
        self.script, self.pool, self.rope_theta = script, pool, rope_theta
        self.layers = list(range(script.geometry.n_layers)) if layers is None else list(layers)
        self.last_slots = None

    def apply(self, i: int, attend: bool = True):
        import torch
        op = self.script.ops[i]
        kind, p = op[0], self.pool
        if kind == "begin":
            got = p.request_begin(); assert got == op[1], (got, op)
        elif kind == "end":
            p.request_end(op[1])
        elif kind == "spawn":
            got = p.thread_spawn_predicted(op[1], op[3], op[4] if len(op) > 4 else 0) if len(op) > 3 else p.thread_spawn(op[1])
            assert got == op[2], (got, op)
        elif kind == "finish":
            p.thread_finish(op[1], op[2])
        elif kind == "merge":
            p.sync_merge(op[1], None if op[2] is None else list(op[2]))
        elif kind == "run":
            if p.host_only or op[3] == 0:
                p.kv_append_run(op[1], op[2], op[3])
            else:
                ks, vs = zip(*[run_tensors(self.script, i, l) for l in self.layers])
                k = torch.stack(ks).cuda(); v = torch.stack(vs).cuda()
                if self.rope_theta:
                    p.kv_append_run_rope(op[1], op[2], op[3], k, v, self.rope_theta)
                else:
                    p.kv_append_run(op[1], op[2], op[3], k, v)
        elif kind == "step":
            reqs = [e[0] for e in op[1]]; thr = [e[1] for e in op[1]]; nn = [e[2] for e in op[1]]
            p.step_begin(reqs, thr, nn)
            self.last_slots = p.step_slots()
            if p.host_only:
                return None
            ks, vs, qs = zip(*[step_tensors(self.script, i, l) for l in self.layers])
            k = torch.stack(ks).cuda(); v = torch.stack(vs).cuda(); q = torch.stack(qs).cuda()
            if self.rope_theta:
                p.kv_append_rope(k, v, self.rope_theta)
                p.rope_queries(q, self.rope_theta)
            else:
                p.kv_append(k, v)
            if not attend:
                return None
            out = torch.empty(q.shape, dtype=torch.float32, device="cuda")
            lse = torch.empty(q.shape[:3], dtype=torch.float32, device="cuda")
            p.decode_attn(q, out, lse)
            return out, lse
        return None
