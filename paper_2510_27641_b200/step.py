"""One SpecAttn verification step as a reusable launch plan: the device buffers and the C
argument structs are prepared once, ``run()`` then issues one specattn_select_topp and one
specattn_sparse_verify per target layer on a stream (Alg. 1, blocks "Sparse Attention Mask
Creation" and "Verification with Sparse Attention").  Orchestration only; every computation
happens in the library's kernels."""
from __future__ import annotations

import ctypes as C
from typing import Sequence

import torch

from . import (SelectArgs, VerifyArgs, SpecAttnError, SELECT_FORM_CLUSTER, VERIFY_LISTS_STABLE, lib, make_select_args,
               make_verify_args, verify_plan, verify_plan_buffer, verify_plan_many,
               verify_step_host, verify_workspace, _stream_ptr)

__all__ = ["VerifyStep"]


class VerifyStep:
    def __init__(self, *, layer_map: Sequence[int], n_draft_layers: int, batch: int,
                 n_draft_heads: int, gamma: int, L_stride: int, n_q_heads: int, p: float,
                 kv_pools: Sequence[torch.Tensor], kv_len: torch.Tensor,
                 block_table: torch.Tensor | None, pages_per_seq: int | None = None,
                 n_groups: int = 1, head_group: Sequence[int] | None = None,
                 idx_stride: int | None = None, sm_scale: float = 0.0, verify_flags: int = 0,
                 use_plans: bool = True, select_workspace: bool = True, select_form: int = 0,
                 overlap_select: bool = False, device=None):
        dev = device or kv_pools[0].device
        self.layer_map = [int(x) for x in layer_map]
        self.n_layers = len(self.layer_map)
        assert len(kv_pools) == self.n_layers
        used = sorted({u for u in self.layer_map if u >= 0})
        self.used = used
        B, T = batch, gamma + 1
        d = kv_pools[0].shape[-1]
        self.draft_probs = [torch.zeros((B, n_draft_heads, gamma, L_stride), dtype=torch.float32, device=dev)
                            if u in used else None for u in range(n_draft_layers)]
        stride = int(L_stride if idx_stride is None else idx_stride)
        self.idx = torch.zeros((n_draft_layers, B, n_groups, stride), dtype=torch.int32, device=dev)
        self.counts = torch.full((n_draft_layers, B, n_groups), -1, dtype=torch.int32, device=dev)
        self.row_status = torch.full((n_draft_layers, B, n_groups), -1, dtype=torch.int32, device=dev)
        self.diag = torch.zeros((n_draft_layers, B, n_groups, 4), dtype=torch.float64, device=dev)
        self.kv_len, self.block_table, self.kv_pools = kv_len, block_table, list(kv_pools)
        self.q = [torch.zeros((B, T, n_q_heads, d), dtype=torch.bfloat16, device=dev) for _ in range(self.n_layers)]
        self.out = [torch.empty((B, T, n_q_heads, d), dtype=torch.float32, device=dev) for _ in range(self.n_layers)]
        self.lse = [torch.empty((B, T, n_q_heads), dtype=torch.float32, device=dev) for _ in range(self.n_layers)]
        self.status = torch.zeros((self.n_layers, B), dtype=torch.int32, device=dev)
        self.select_args, self._keep = None, None
        if used:   # a step whose layers are all dense has nothing to select
            self.select_args, self._keep = make_select_args(
                self.draft_probs, kv_len, self.layer_map, p, n_groups=n_groups, head_group=head_group,
                idx=self.idx, counts=self.counts, row_status=self.row_status, diag=self.diag,
                workspace=select_workspace, form=select_form)
        # overlapped schedule: one selection per used draft layer, so that all but the first run
        # on a second stream under the attention of the layers mapped to earlier draft layers
        self.overlap = bool(overlap_select) and len(used) > 1
        self.select_args_u, self._keep_u, self._side = {}, [], None
        if self.overlap:
            for u in used:
                a_u, keep_u = make_select_args(
                    self.draft_probs, kv_len, [u], p, n_groups=n_groups, head_group=head_group,
                    idx=self.idx, counts=self.counts, row_status=self.row_status, diag=self.diag,
                    workspace=False, form=SELECT_FORM_CLUSTER)
                self.select_args_u[u] = a_u
                self._keep_u.append(keep_u)
        self.verify_args: list[VerifyArgs] = []
        self.workspace = None
        self.plans: dict[int, tuple[torch.Tensor, int]] = {}   # draft layer (-1: dense) -> (plan, a layer using it)
        for j, u in enumerate(self.layer_map):
            a = make_verify_args(self.q[j], kv_pools[j], kv_len, block_table=block_table,
                                 pages_per_seq=pages_per_seq,
                                 idx=None if u < 0 else self.idx[u], counts=None if u < 0 else self.counts[u],
                                 n_groups=n_groups, dense=u < 0, sm_scale=sm_scale, out=self.out[j],
                                 lse=self.lse[j], status=self.status[j],
                                 # after the first layer the lists (written by select) and the
                                 # context's K/V rows predate the preceding launch
                                 flags=(VERIFY_LISTS_STABLE if j > 0 else 0) | int(verify_flags))
            if self.workspace is None:
                self.workspace = verify_workspace(a, dev)
            a.workspace, a.workspace_bytes = self.workspace.data_ptr(), self.workspace.numel()
            # target layers that share a draft layer's lists (or are dense) share a work partition;
            # a list set that a single layer uses is cheaper partitioned by that layer's own launch
            # than by a plan launch in front of it
            if use_plans and self.layer_map.count(u) > 1:
                if u not in self.plans:
                    self.plans[u] = (verify_plan_buffer(a, dev), j)
                a.plan = self.plans[u][0].data_ptr()
            self.verify_args.append(a)

    # ---- inputs -------------------------------------------------------------------------------
    def load_inputs(self, draft_probs_host: Sequence[torch.Tensor | None], q_host: Sequence[torch.Tensor]):
        """Plain (untimed) upload of a step's inputs into the plan's device buffers."""
        for u in self.used:
            self.draft_probs[u].copy_(draft_probs_host[u], non_blocking=True)
        for j in range(self.n_layers):
            self.q[j].copy_(q_host[j], non_blocking=True)

    # ---- launches -----------------------------------------------------------------------------
    def run_select(self, stream=None):
        if self.select_args is None:
            return
        rc = lib().specattn_select_topp(C.byref(self.select_args), _stream_ptr(stream))
        if rc != 0:
            raise SpecAttnError(rc, "specattn_select_topp")

    def run_plans(self, stream=None):
        """The work partitions that the verify launches of each distinct list set share: one
        small launch for up to eight of them."""
        if self.plans:
            verify_plan_many([self.verify_args[j] for _, j in self.plans.values()],
                             [plan for plan, _ in self.plans.values()], stream)

    def run_verify(self, j: int, stream=None):
        rc = lib().specattn_sparse_verify(C.byref(self.verify_args[j]), _stream_ptr(stream))
        if rc != 0:
            raise SpecAttnError(rc, "specattn_sparse_verify")

    def _run_overlapped(self, stream=None):
        """The selection of the first draft layer in use, then, on a second stream, the selections
        (and work partitions) of the others in the order of their first use, while the first
        stream runs the attention of the target layers: a layer waits for its draft layer's
        selection only (Alg. 1: every verifier layer needs the mask of its mapped draft layer)."""
        main = stream if stream is not None else torch.cuda.current_stream()
        if self._side is None:
            self._side = torch.cuda.Stream(device=main.device)
        L = lib()
        order = []
        for u in self.layer_map:
            if u >= 0 and u not in order:
                order.append(u)

        def select_and_plan(u, st):
            rc = L.specattn_select_topp(C.byref(self.select_args_u[u]), _stream_ptr(st))
            if rc != 0:
                raise SpecAttnError(rc, "specattn_select_topp")
            if u in self.plans:
                plan, j = self.plans[u]
                verify_plan(self.verify_args[j], plan, st)

        with torch.cuda.stream(main):
            select_and_plan(order[0], main)
            if -1 in self.plans:   # the dense layers' partition does not depend on any selection
                plan, j = self.plans[-1]
                verify_plan(self.verify_args[j], plan, main)
            fork = torch.cuda.Event()
            fork.record(main)
        ready = {order[0]}
        events = {}
        with torch.cuda.stream(self._side):
            self._side.wait_event(fork)
            for u in order[1:]:
                select_and_plan(u, self._side)
                events[u] = torch.cuda.Event()
                events[u].record(self._side)
        with torch.cuda.stream(main):
            sp = _stream_ptr(main)
            for j, a in enumerate(self.verify_args):
                u = self.layer_map[j]
                flags = a.flags
                if u >= 0 and u not in ready:
                    main.wait_event(events[u])
                    ready.add(u)
                    a.flags = flags & ~VERIFY_LISTS_STABLE   # lists and plan are new to this launch
                rc = L.specattn_sparse_verify(C.byref(a), sp)
                a.flags = flags
                if rc != 0:
                    raise SpecAttnError(rc, "specattn_sparse_verify")
            for u, ev in events.items():   # join (a draft layer whose layers were all visited is already waited for)
                if u not in ready:
                    main.wait_event(ev)

    def run(self, stream=None):
        """Device-resident step: 1 select launch + n_layers verify launches."""
        if self.overlap:
            return self._run_overlapped(stream)
        sp = _stream_ptr(stream)
        L = lib()
        self.run_select(stream)
        self.run_plans(stream)
        for a in self.verify_args:
            rc = L.specattn_sparse_verify(C.byref(a), sp)
            if rc != 0:
                raise SpecAttnError(rc, "specattn_sparse_verify")

    def run_host(self, draft_probs_host, q_host, out_host, lse_host, stream=None):
        """Whole step from pinned host tensors through specattn_verify_step_host."""
        verify_step_host(self.select_args, draft_probs_host, self.verify_args, q_host, out_host,
                         lse_host, stream)

    @property
    def launches_per_step(self) -> int:
        n_select = 0
        if self.overlap:
            return len(self.select_args_u) + len(self.plans) + self.n_layers
        if self.select_args is not None:
            n_select = 2 if self.select_args.workspace else 1   # aggregation + search, or the cluster form
        return n_select + (len(self.plans) + 7) // 8 + self.n_layers
