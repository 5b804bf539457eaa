"""Oracle, part 3: replay a workload script on the oracle.  TEST INFRASTRUCTURE — not a product path.

Applies the operations of a `pasta_workloads.Script` to a `PoolModel` and to one `KVStore` per
chosen layer, and evaluates `decode_attention` for the steps asked for.
"""
from __future__ import annotations

from typing import Callable, Dict, Iterable, List, Optional, Sequence

import numpy as np

from pasta_workloads import Script, run_tensors, step_tensors

from .attention import KVStore, decode_attention
from .pool_model import PoolModel


class OracleReplay:
    def __init__(self, script: Script, layers: Sequence[int] = (0,), with_kv: bool = True):
        geo = script.geometry
        self.script = script
        self.layers = list(layers)
        self.model = PoolModel(script.n_pages, geo.page_size, script.free_order,
                               script.max_requests, script.max_threads_per_request,
                               script.max_segments_per_thread)
        self.stores: Dict[int, KVStore] = (
            {l: KVStore(script.n_pages, geo.page_size, geo.n_kv_heads, geo.head_dim) for l in self.layers}
            if with_kv else {})
        self.next_op = 0

    def apply(self, op_index: int, attend: bool = True, tensors=None):
        """Apply operation `op_index`.  For a step, returns {layer: (out, lse)} (fp64) when attend=True.

        `tensors` optionally maps layer -> the tensors of this operation (as run_tensors /
        step_tensors would return them); by default they are regenerated from the script's seed."""
        assert op_index == self.next_op, "operations must be applied in order"
        self.next_op += 1
        op = self.script.ops[op_index]
        kind = op[0]
        m = self.model
        if kind == "begin":
            got = m.request_begin()
            assert got == op[1], (got, op)
        elif kind == "end":
            m.request_end(op[1])
        elif kind == "spawn":
            got = m.thread_spawn(op[1], op[3] if len(op) > 3 else 0, op[4] if len(op) > 4 else 0)
            assert got == op[2], (got, op)
        elif kind == "finish":
            m.thread_finish(op[1], op[2])
        elif kind == "merge":
            m.sync_merge(op[1], None if op[2] is None else list(op[2]))
        elif kind == "run":
            slots = m.append_run(op[1], op[2], op[3])
            for l, store in self.stores.items():
                k, v = tensors[l] if tensors else run_tensors(self.script, op_index, l)
                store.write(slots, k, v)
        elif kind == "step":
            slots = [s for s in m.reserve(op[1]) if s is not None]
            queries = m.queries_of(op[1])
            result = {}
            for l, store in self.stores.items():
                k, v, q = tensors[l] if tensors else step_tensors(self.script, op_index, l)
                store.write(slots, k, v)
                if attend:
                    result[l] = decode_attention(m, store, queries, q)
            return result
        else:
            raise ValueError(kind)
        return None

    def run_all(self, attend_steps: Optional[Iterable[int]] = None):
        """Apply every remaining operation; returns {op_index: {layer: (out, lse)}} for attended steps."""
        wanted = None if attend_steps is None else set(attend_steps)
        outputs = {}
        for i in range(self.next_op, len(self.script.ops)):
            is_step = self.script.ops[i][0] == "step"
            res = self.apply(i, attend=is_step and (wanted is None or i in wanted))
            if is_step and res:
                outputs[i] = res
        return outputs
