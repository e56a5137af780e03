"""Device buffers for one routing step and the four-stage call sequence.

Plumbing only: torch allocates the buffers once (the C library allocates nothing per call)
and every stage below is one C-ABI call into the CUDA kernels, enqueued on the current torch
stream.  `route()` works on data already resident on the device; `route_host()` is the same
step driven from pinned host buffers (inputs copied in, results copied out).
"""
from __future__ import annotations

from typing import Callable, Optional

import torch

from . import binding as cb


class RouteStep:
    def __init__(self, layout: "cb.Layout", T: int, K: int, H: int, device: Optional[torch.device] = None,
                 alias_expert_out: bool = True):
        self.layout, self.T, self.K, self.H = layout, T, K, H
        self.E, self.D, self.P = layout.E, layout.D, T * K
        dev = torch.device("cuda", torch.cuda.current_device()) if device is None else device
        self.device = dev

        def z(shape, dtype):
            return torch.zeros(shape, dtype=dtype, device=dev)

        # inputs
        self.topk_ids = z((T, K), torch.int32)
        self.gate_w = z((T, K), torch.float32)
        self.src_rank = z((T,), torch.int32)
        self.x = z((T, H), torch.bfloat16)
        # stage outputs
        self.coact = z((self.E, self.E), torch.int32)
        self.load = z((self.E,), torch.int32)
        self.assigned_slot = z((T, K), torch.int32)
        self.slot_load = z((self.D,), torch.int32)
        self.remote_nodes = z((T,), torch.uint8)
        self.totals = z((2,), torch.int64)
        self.dest_counts = z((self.D,), torch.int32)
        self.dest_offsets = z((self.D + 1,), torch.int32)
        self.row_of_pair = z((self.P,), torch.int32)
        self.pair_of_row = z((self.P,), torch.int32)
        self.send = z((self.P, H), torch.bfloat16)
        # without real experts between dispatch and combine, combine may read the send buffer
        self.expert_out = self.send if alias_expert_out else z((self.P, H), torch.bfloat16)
        self.y = z((T, H), torch.bfloat16)
        ws = max(cb.coact_stats_workspace_bytes(T, K, self.E), cb.assign_workspace_bytes(layout, T, K),
                 cb.permute_workspace_bytes(T, K, self.D), cb.route_index_workspace_bytes(layout, T, K), 256)
        self.workspace = torch.empty((ws,), dtype=torch.uint8, device=dev)

    # -- the four stages, device-resident --------------------------------------------------
    def stats(self, flags: int = 0) -> None:
        cb.coact_stats(self.topk_ids, self.E, self.coact, self.load, flags=flags, workspace=self.workspace)

    def assign(self, seed: int, flags: int = 0) -> None:
        cb.assign(self.layout, self.topk_ids, self.src_rank, seed, self.assigned_slot, slot_load=self.slot_load,
                  remote_nodes=self.remote_nodes, totals=self.totals, flags=flags, workspace=self.workspace)

    def permute(self, flags: int = 0) -> None:
        cb.permute(self.assigned_slot, self.D, self.x, self.send, self.dest_counts, self.dest_offsets,
                   self.row_of_pair, self.pair_of_row, self.workspace, flags=flags)

    def combine(self, flags: int = 0) -> None:
        cb.combine(self.expert_out, self.row_of_pair, self.gate_w, self.y, flags=flags)

    def route(self, seed: int, experts: Optional[Callable[[torch.Tensor, torch.Tensor], None]] = None,
              overlap_stats: bool = False) -> None:
        """stats -> assign -> permute -> [experts(send, expert_out)] -> combine on the current stream.

        Nothing in the step consumes the statistics (they feed the planner of later steps), so with
        `overlap_stats` they run on a side stream beside the other stages and are joined at the end.
        """
        main = torch.cuda.current_stream()
        if overlap_stats:
            if not hasattr(self, "_side"):
                self._side = torch.cuda.Stream()
            self._side.wait_stream(main)
            with torch.cuda.stream(self._side):
                self.stats()
        else:
            self.stats()
        self.assign(seed)
        self.permute()
        if experts is not None:
            experts(self.send, self.expert_out)
        self.combine()
        if overlap_stats:
            main.wait_stream(self._side)

    # -- the resident step replayed from a CUDA graph ------------------------------------------
    def capture(self, experts: Optional[Callable[[torch.Tensor, torch.Tensor], None]] = None,
                fused: bool = False) -> None:
        """Capture one step (the four stages, or the fused pass and the two row stages) into a CUDA
        graph.  The seed lives in a device word that the assignment kernels read when they run, so
        `replay(seed)` draws afresh every step.  The graph holds the addresses of this object's
        buffers: new inputs are copied into topk_ids / gate_w / src_rank / x before a replay."""
        self._seed_dev = torch.zeros(1, dtype=torch.int64, device=self.device)
        run = (lambda: self.route_fused(self._seed_dev, experts)) if fused else (lambda: self.route(self._seed_dev, experts))
        side = torch.cuda.Stream(device=self.device)
        side.wait_stream(torch.cuda.current_stream())
        with torch.cuda.stream(side):
            for _ in range(2):                     # first calls look up device attributes; not capturable
                run()
        torch.cuda.current_stream().wait_stream(side)
        torch.cuda.synchronize(self.device)
        self._graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(self._graph):
            run()

    def replay(self, seed: int) -> None:
        """One captured step with this seed, enqueued on the current stream."""
        self._seed_dev.fill_(seed if seed < 2**63 else seed - 2**64)
        self._graph.replay()

    def route_fused(self, seed: int, experts: Optional[Callable[[torch.Tensor, torch.Tensor], None]] = None) -> None:
        """The same step with stages 1, 2 and the permutation index fused into one pass over the ids
        (cobalt_route_index); slot_load is delivered as dest_counts."""
        cb.route_index(self.layout, self.topk_ids, self.src_rank, seed, self.coact, self.load, self.assigned_slot,
                       self.dest_counts, self.dest_offsets, self.row_of_pair, self.workspace,
                       remote_nodes=self.remote_nodes, totals=self.totals, pair_of_row=self.pair_of_row)
        cb.permute_rows(self.x, self.row_of_pair, self.K, self.send)
        if experts is not None:
            experts(self.send, self.expert_out)
        self.combine()

    # -- the same step from pinned host memory ----------------------------------------------
    def route_host(self, seed: int, ids_h: torch.Tensor, w_h: torch.Tensor, src_h: torch.Tensor,
                   x_h: torch.Tensor, y_h: torch.Tensor, coact_h: torch.Tensor, load_h: torch.Tensor,
                   slot_load_h: torch.Tensor, totals_h: torch.Tensor, chunks: int = 16, join: bool = True) -> None:
        """One step with inputs and results in pinned host memory.

        The gating output is small and goes first, so statistics, assignment and the permutation
        index run while the hidden rows are still on their way.  The rows then move in `chunks`
        token blocks: block c is copied in on one stream, fanned out to its send rows and (there
        being no expert computation between dispatch and combine here) combined on the compute
        stream, and its result copied out on a third stream, so both copy directions and the
        kernels overlap.  The C entry points take plain pointers, so a block is just an offset.

        With `join` the current stream waits for the last copy out, so the host buffers are valid once
        it has been synchronised.  Without it the call returns with copies still queued and
        `wait_host_results()` (or a device synchronise) must come before the host buffers are read;
        the next call may then start copying its inputs in while this one's last results are still
        on their way out, which keeps both copy directions busy across steps.
        """
        main = torch.cuda.current_stream()
        if not hasattr(self, "_h2d"):
            self._h2d, self._d2h = torch.cuda.Stream(), torch.cuda.Stream()
        h2d, d2h = self._h2d, self._d2h
        h2d.wait_stream(main)          # the previous step may still be reading x and the gating output
        d2h.wait_stream(main)
        # results of the previous call that may still be on their way out must not be overwritten
        prev_small = getattr(self, "_small_copied", None)
        prev_y = getattr(self, "_y_copied", [])
        T, K = self.T, self.K
        chunks = max(1, min(chunks, T)) if T > 0 else 1
        # block starts on multiples of 4 tokens keep every offset pointer 16-byte aligned for any K
        bounds = [min(T, ((T * c) // chunks + 3) // 4 * 4) for c in range(chunks)] + [T]
        # All copies of one direction go through one stream, the gating output ahead of the hidden
        # rows: copies in a direction share a copy engine, and a small copy issued from another
        # stream can end up queued behind every row block that is ready at the same moment.
        ready = []
        with torch.cuda.stream(h2d):
            self.topk_ids.copy_(ids_h, non_blocking=True)
            self.gate_w.copy_(w_h, non_blocking=True)
            self.src_rank.copy_(src_h, non_blocking=True)
            gating_ready = torch.cuda.Event()
            gating_ready.record(h2d)
            for c in range(chunks):
                t0, t1 = bounds[c], bounds[c + 1]
                self.x[t0:t1].copy_(x_h[t0:t1], non_blocking=True)
                ev = torch.cuda.Event()
                ev.record(h2d)
                ready.append(ev)
        main.wait_event(gating_ready)
        if prev_small is not None:
            main.wait_event(prev_small)
        if len(prev_y) != chunks:      # another block structure: wait for everything that is queued
            main.wait_stream(d2h)
            prev_y = []
        self.stats()
        self.assign(seed)
        cb.permute_index(self.assigned_slot, self.D, self.dest_counts, self.dest_offsets, self.row_of_pair,
                         self.pair_of_row, self.workspace)
        index_done = torch.cuda.Event()
        index_done.record(main)
        with torch.cuda.stream(d2h):
            d2h.wait_event(index_done)
            coact_h.copy_(self.coact, non_blocking=True)
            load_h.copy_(self.load, non_blocking=True)
            slot_load_h.copy_(self.slot_load, non_blocking=True)
            totals_h.copy_(self.totals, non_blocking=True)
            self._small_copied = torch.cuda.Event()
            self._small_copied.record(d2h)
        y_copied = [None] * chunks
        for c in range(chunks):
            t0, t1 = bounds[c], bounds[c + 1]
            if t1 == t0:
                continue
            main.wait_event(ready[c])
            rop = self.row_of_pair[t0 * K:t1 * K]
            # rows index the whole send buffer, so the full buffers are passed with a token offset
            cb.permute_rows_block(self.x, rop, K, self.send, t0, t1)
            if prev_y and prev_y[c] is not None:
                main.wait_event(prev_y[c])
            cb.combine_block(self.expert_out, rop, self.gate_w, self.y, t0, t1)
            done = torch.cuda.Event()
            done.record(main)
            with torch.cuda.stream(d2h):
                d2h.wait_event(done)
                y_h[t0:t1].copy_(self.y[t0:t1], non_blocking=True)
                y_copied[c] = torch.cuda.Event()
                y_copied[c].record(d2h)
        self._y_copied = y_copied
        self._host_done = torch.cuda.Event()
        self._host_done.record(d2h)
        if join:
            main.wait_stream(d2h)

    def wait_host_results(self) -> None:
        """Block the host until the results of the last route_host call are in the host buffers."""
        done = getattr(self, "_host_done", None)
        if done is not None:
            done.synchronize()

    def h2d_bytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in (self.topk_ids, self.gate_w, self.src_rank, self.x))

    def d2h_bytes(self) -> int:
        return sum(t.numel() * t.element_size() for t in (self.y, self.coact, self.load, self.slot_load, self.totals))
