"""The whole compression pass as a user calls it: phase A for every layer, the budget barrier,
phase B for every layer.  Only sequencing and buffer plumbing live here; every step is a C-ABI
call into libmeda.so (see binding.py) and nothing runs on the CPU in between."""
from __future__ import annotations

import torch

from . import binding
from .workloads import Workload


def owned_layers(n_layers: int, rank: int, world: int) -> list[int]:
    """Layers rank `rank` of `world` processes when ONE prompt is sharded by layer: round-robin, so that the
    layers a model's depth makes expensive (large budgets cluster) spread over the ranks."""
    return [l for l in range(n_layers) if l % world == rank]


def exchange_entropies(entropy: torch.Tensor, group=None) -> None:
    """The one exchange step of a layer-sharded pass (Eq. 7's softmax runs over ALL layers): `entropy` holds
    this rank's layers and zeros elsewhere; after the call every rank holds every layer's value (a sum over
    disjoint supports, so the result is exact and the same bits on every rank).  L floats: latency only."""
    import torch.distributed as dist
    if dist.is_available() and dist.is_initialized() and dist.get_world_size(group) > 1:
        dist.all_reduce(entropy, op=dist.ReduceOp.SUM, group=group)


class CompressionPass:
    """Buffers and call sequence of one prompt's pass on one GPU.

    Outputs are packed: layer l's compacted caches occupy rows [offset_l, offset_l + S_l) of
    `k_out` / `v_out` ([n_kv_heads] x rows x head_dim each), with offset_l = l * row_capacity.
    `row_capacity` bounds S_l per layer (n_tokens is always safe; a smaller value saves memory and
    makes a layer whose budget exceeds it report MEDA_ERR_WORKSPACE)."""

    def __init__(self, wl: Workload, row_capacity: int | None = None, device="cuda", n_streams: int = 8,
                 **ctx_overrides):
        self.wl = wl
        self.device = device
        # Layers are independent inside each phase, so they alternate between `n_streams` streams, each
        # with its own context (scratch memory): the short, latency-bound kernels of one layer
        # (selection, sort passes, reductions of partials) then run beside the long kernels of
        # the next instead of leaving the GPU idle.
        self.contexts = [binding.Context.for_workload(wl, **ctx_overrides) for _ in range(max(1, n_streams))]
        self.ctx = self.contexts[0]
        self.streams = [torch.cuda.Stream(device=device) for _ in self.contexts] if len(self.contexts) > 1 else []
        n, hkv, hq, w, d, L = wl.n_tokens, wl.n_kv_heads, wl.n_q_heads, wl.window, wl.head_dim, wl.n_layers
        self.cap = n if row_capacity is None else int(row_capacity)
        f32, i32 = torch.float32, torch.int32
        self.row_stats = [torch.empty((hq, w, 4), dtype=f32, device=device) for _ in self.contexts]
        self.scores = torch.empty((L, hkv, n), dtype=f32, device=device)
        self.entropy = torch.zeros(L, dtype=f32, device=device)
        self.budgets = torch.zeros((L, 3), dtype=i32, device=device)
        self.k_out = torch.empty((L, hkv, self.cap, d), dtype=wl.torch_dtype, device=device)
        self.v_out = torch.empty((L, hkv, self.cap, d), dtype=wl.torch_dtype, device=device)
        self.counts = torch.empty((L, hkv, self.cap), dtype=i32, device=device)
        self.idx_c = torch.empty((L, hkv, self.cap), dtype=i32, device=device)

    def close(self):
        for c in self.contexts:
            c.close()

    def check(self):
        """Synchronises and raises if any context recorded a device-side error."""
        torch.cuda.synchronize()
        for c in self.contexts:
            c.check()

    def launch_count(self) -> int:
        return sum(c.launch_count() for c in self.contexts)

    def _fork(self, main):
        ev = torch.cuda.Event()
        ev.record(main)
        for s in self.streams:
            s.wait_event(ev)

    def _join(self, main):
        for s in self.streams:
            ev = torch.cuda.Event()
            ev.record(s)
            main.wait_event(ev)

    def run(self, q_layers, k_layers, v_layers, stream=None, single_stream=False, qk_ready=None, v_ready=None,
            budgets_done=None, layer_done=None, max_lanes=None, layer_shard=None, exchange=None):
        """Enqueues the whole pass.  Inputs are lists of per-layer device tensors; results stay on the
        device in this object's buffers.  The work is ordered after what `stream` (default: torch's
        current stream) holds and `stream` waits for all of it.  With `single_stream` everything goes to
        `stream` through the first context (used when every launch is timed on its own).  `qk_ready` /
        `v_ready`: optional per-layer events after which a layer's (queries, keys) / values are in
        place (copies still in flight on another stream): phase A of a layer waits for the first,
        phase B for the second.  `budgets_done` (an event) is recorded once the budgets are written,
        `layer_done[l]` (events) once layer l's compressed cache is: a caller can start copying results
        out while later layers are still being compressed.  `max_lanes` limits the streams used.
        `layer_shard=(rank, world)`: this process runs only the layers `owned_layers` deals it (the other
        entries of the input lists are not read and may be None); the L entropies are exchanged between the
        two phases, so every rank computes the same budgets, and each rank's outputs hold its own layers
        only.  `exchange` replaces the collective (a callable taking the entropy tensor; used to emulate the
        other ranks on one GPU)."""
        L = self.wl.n_layers
        mine = list(range(L)) if layer_shard is None else owned_layers(L, *layer_shard)
        main = stream if stream is not None else torch.cuda.current_stream()
        if single_stream or not self.streams:
            lanes = [(self.contexts[0], main, self.row_stats[0])]
        else:
            lanes = list(zip(self.contexts, self.streams, self.row_stats))
            if max_lanes is not None:
                lanes = lanes[: max(1, max_lanes)]
            self._fork(main)
        if layer_shard is not None:
            with torch.cuda.stream(main):
                self.entropy.zero_()                  # the other ranks' layers must read as zero in the exchange
            if len(lanes) > 1:
                self._fork(main)
        for i, l in enumerate(mine):
            c, s, rs = lanes[i % len(lanes)]
            if qk_ready is not None:
                s.wait_event(qk_ready[l])
            c.window_scores(l, q_layers[l], k_layers[l], rs, self.scores[l], self.entropy, s)
        if len(lanes) > 1:
            self._join(main)
        if layer_shard is not None:
            with torch.cuda.stream(main):
                (exchange or exchange_entropies)(self.entropy)
        self.ctx.allocate_budgets(self.entropy, self.budgets, main)      # Eq. 7 needs every layer's entropy
        if budgets_done is not None:
            budgets_done.record(main)
        if len(lanes) > 1:
            self._fork(main)
        for i, l in enumerate(mine):
            c, s, _ = lanes[i % len(lanes)]
            if v_ready is not None:
                s.wait_event(v_ready[l])
            c.compress_layer(l, k_layers[l], v_layers[l], self.scores[l], self.budgets, self.k_out[l], self.v_out[l],
                             self.counts[l], self.idx_c[l], self.cap, s)
            if layer_done is not None:
                layer_done[l].record(s)
        if len(lanes) > 1:
            self._join(main)

    def capture(self, q_layers, k_layers, v_layers):
        """Records the whole pass (every launch of `run` on these buffers) into a CUDA graph, after one
        ordinary run that loads the kernels.  `replay()` then enqueues the pass with a single graph
        launch: no per-kernel launch cost on the host and shorter gaps between kernels on the device.
        Returns the number of kernels in the graph."""
        self.run(q_layers, k_layers, v_layers)
        torch.cuda.synchronize()
        before = self.launch_count()
        graph = torch.cuda.CUDAGraph()
        with torch.cuda.graph(graph):
            self.run(q_layers, k_layers, v_layers)
        self.graph = graph
        self.graph_kernels = self.launch_count() - before
        return self.graph_kernels

    def replay(self):
        """Enqueues the captured pass on torch's current stream."""
        self.graph.replay()

    def run_from_host(self, q_host, k_host, v_host, staging, out_host):
        """End-to-end variant: per-layer inputs in pinned HOST memory are copied to the device
        staging buffers, the pass runs, and the budgets plus the compacted caches (only the S_l live
        rows of each layer) are copied back to pinned host memory: out_host[name][l] has S_l rows per
        head (see `alloc_host_outputs`).  Returns (h2d_bytes, d2h_bytes)."""
        L = self.wl.n_layers
        h2d = 0
        # Copies run on their own stream, queries and keys of every layer first (phase A needs only
        # those), then the values; each layer's kernels wait for that layer's copies only, so the pass
        # overlaps with the transfer instead of following it.
        main = torch.cuda.current_stream()
        if not hasattr(self, "_copy_stream"):
            self._copy_stream = torch.cuda.Stream(device=self.device)
        cs = self._copy_stream
        cs.wait_stream(main)
        qk_ready, v_ready = [], []
        with torch.cuda.stream(cs):
            for l in range(L):
                for src, dst in ((q_host[l], staging["q"][l]), (k_host[l], staging["k"][l])):
                    dst.copy_(src, non_blocking=True)
                    h2d += src.numel() * src.element_size()
                ev = torch.cuda.Event()
                ev.record(cs)
                qk_ready.append(ev)
            for l in range(L):
                staging["v"][l].copy_(v_host[l], non_blocking=True)
                h2d += v_host[l].numel() * v_host[l].element_size()
                ev = torch.cuda.Event()
                ev.record(cs)
                v_ready.append(ev)
        budgets_done = torch.cuda.Event()
        layer_done = [torch.cuda.Event() for _ in range(L)]
        self.run(staging["q"], staging["k"], staging["v"], qk_ready=qk_ready, v_ready=v_ready,
                 budgets_done=budgets_done, layer_done=layer_done, max_lanes=4)
        # Results leave on a third stream: the budgets as soon as they exist (the live row counts decide
        # what comes back), then each layer's compacted cache as soon as that layer is done, while the
        # values of later layers are still arriving (the link carries both directions at once).
        if not hasattr(self, "_down_stream"):
            self._down_stream = torch.cuda.Stream(device=self.device)
        ds = self._down_stream
        with torch.cuda.stream(ds):
            ds.wait_event(budgets_done)
            out_host["budgets"].copy_(self.budgets, non_blocking=True)
            ds.synchronize()
            d2h = self.budgets.numel() * 4
            for l in range(L):
                s = int(out_host["budgets"][l, 0])
                ds.wait_event(layer_done[l])
                for name, src in (("k", self.k_out), ("v", self.v_out), ("counts", self.counts), ("idx", self.idx_c)):
                    out_host[name][l].copy_(src[l][:, :s], non_blocking=True)
                    d2h += src[l][:, :s].numel() * src.element_size()
        main.wait_stream(ds)
        main.synchronize()
        return h2d, d2h

    def alloc_host_outputs(self):
        """Pinned host buffers sized by the budgets of the last run (budgets are a deterministic
        function of the inputs, so a repeated run of the same prompt fits them exactly)."""
        b = self.budgets.cpu()
        wl = self.wl
        out = dict(budgets=torch.empty_like(b).pin_memory(), k=[], v=[], counts=[], idx=[])
        for l in range(wl.n_layers):
            s = int(b[l, 0])
            out["k"].append(torch.empty((wl.n_kv_heads, s, wl.head_dim), dtype=wl.torch_dtype).pin_memory())
            out["v"].append(torch.empty((wl.n_kv_heads, s, wl.head_dim), dtype=wl.torch_dtype).pin_memory())
            out["counts"].append(torch.empty((wl.n_kv_heads, s), dtype=torch.int32).pin_memory())
            out["idx"].append(torch.empty((wl.n_kv_heads, s), dtype=torch.int32).pin_memory())
        return out
