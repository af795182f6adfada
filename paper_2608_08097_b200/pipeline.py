"""Device buffers of one layer's sparse-decode state and the order of the library calls.

This is host-side bookkeeping only (allocation through torch, call sequencing, stream
choice); every step of the path runs inside liboasis.so through `binding`.
"""
import math

import torch

from . import binding as oasis


class DecodeLayer:
    """Working set of one layer: summaries, scores, selection, HBM slot pool, outputs.

    Fetch-all layout: row (b, h) owns the k + 2 consecutive pool slots
    (b * Hkv + h) * (k + 2) + c, column c holding the block sel[b][h][c].
    """

    def __init__(self, batch, n_q_heads, n_kv_heads, max_blocks, k, n_q_tokens, device="cuda",
                 want_lse=False):
        self.B, self.Hq, self.Hkv, self.mb = batch, n_q_heads, n_kv_heads, max_blocks
        self.k, self.T = k, n_q_tokens
        self.cols = k + 2
        self.dims = oasis.Dims(batch, n_q_heads, n_kv_heads, max_blocks)
        self.device = torch.device(device)
        dev = self.device
        rows = batch * n_kv_heads
        self.summaries = torch.zeros((batch, n_kv_heads, max_blocks, 2, 128), dtype=torch.bfloat16, device=dev)
        self.scores = torch.empty((batch, n_kv_heads, max_blocks), dtype=torch.float32, device=dev)
        self.sel = torch.empty((batch, n_kv_heads, self.cols), dtype=torch.int32, device=dev)
        self.stage_idx = torch.empty((batch, n_kv_heads, self.cols), dtype=torch.int64, device=dev)
        self.stage_slots = torch.empty((batch, n_kv_heads, self.cols), dtype=torch.int32, device=dev)
        self.pool = torch.zeros((rows * self.cols, 2, 16, 128), dtype=torch.bfloat16, device=dev)
        self.slot_tbl = torch.arange(rows * self.cols, dtype=torch.int32, device=dev).view(batch, n_kv_heads, self.cols)
        self.out = torch.empty((batch, n_q_tokens, n_q_heads, 128), dtype=torch.bfloat16, device=dev)
        self.lse = torch.empty((batch, n_q_tokens, n_q_heads), dtype=torch.float32, device=dev) if want_lse else None
        ws = oasis.attn_workspace_bytes(self.dims, n_q_tokens, self.cols)
        self.workspace = torch.empty((max(ws, 16),), dtype=torch.uint8, device=dev)
        self.scale = 1.0 / math.sqrt(128.0)

    # step 0
    def build_summaries(self, kv_pool, block_table, first_block, n_blocks, max_new_blocks, stream=None):
        oasis.build_summaries(self.dims, kv_pool, block_table, first_block, n_blocks, max_new_blocks,
                              self.summaries, stream=stream)

    # step 1: the draft tokens are rows 1..T-1 of the stacked verify-step queries
    def score(self, q, n_full, reduce_mode=oasis.REDUCE_MAX, stream=None):
        n_draft = self.T - 1
        q_draft = q[:, 1:]
        oasis.score_blocks(self.dims, q_draft, n_draft, self.summaries, n_full, self.scores,
                           reduce_mode=reduce_mode, q_batch_stride=self.T * self.Hq * 128, stream=stream)

    def score_queries(self, q_rows, n_full, reduce_mode=oasis.REDUCE_MAX, stream=None):
        """Scores with an explicit dense [B][Td][Hq][128] query tensor (e.g. the true queries)."""
        oasis.score_blocks(self.dims, q_rows, q_rows.shape[1], self.summaries, n_full, self.scores,
                           reduce_mode=reduce_mode, stream=stream)

    # step 2
    def select(self, n_full, seq_len, block_table, stream=None, sel=None):
        oasis.select_topk(self.dims, self.scores, n_full, seq_len, self.T, self.k, block_table,
                          self.sel if sel is None else sel,
                          self.stage_idx if sel is None else None,
                          self.stage_slots if sel is None else None, stream=stream)

    # step 3
    def stage(self, host_kv, stream=None):
        oasis.stage_blocks(host_kv, self.stage_idx, self.stage_slots, self.stage_idx.numel(), self.pool,
                           stream=stream)

    # step 4
    def attend(self, q, seq_len, blk_tbl=None, slot_tbl=None, stream=None):
        oasis.sparse_attn(self.dims, q, self.T, self.pool, self.slot_tbl if slot_tbl is None else slot_tbl,
                          self.sel if blk_tbl is None else blk_tbl, self.cols, seq_len, self.scale,
                          self.out, lse=self.lse, workspace=self.workspace, stream=stream)
        return self.out

    # steps 4 + 1 in one launch (shapes permitting)
    def attend_and_score(self, q, seq_len, n_full_next, blk_tbl=None, slot_tbl=None, stream=None):
        oasis.attn_and_score(self.dims, q, self.T, self.pool, self.slot_tbl if slot_tbl is None else slot_tbl,
                             self.sel if blk_tbl is None else blk_tbl, self.cols, seq_len, self.scale, self.out,
                             q[:, 1:], self.T - 1, self.summaries, n_full_next, self.scores, lse=self.lse,
                             q_batch_stride=self.T * self.Hq * 128, workspace=self.workspace, stream=stream)
        return self.out


class DecodeEngine:
    """Sequencing of one decode step across layers, after the paper's asynchronous prefetch
    pipeline (Sec. 4.2.2).  Four streams:
      foreground  attention of every layer over the working set that the previous step's
                  prediction staged;
      prediction  summary update for newly completed blocks and scoring with the draft queries;
      selection   top-k and (delta mode) the transfer plan -- the tables a layer's attention
                  reads are only rewritten after that attention has finished;
      transfer    the gather of what was selected, awaited, per layer, only by the next step's
                  attention of that same layer.
    In end-to-end mode a fifth stream uploads the step's queries (all layers, before the first
    gather) and downloads each layer's output.
    A whole step can be captured into a CUDA graph (`capture_step`) and replayed, which removes
    the host launch cost of its ~250 kernels.

    mode "fetch_all": every selected block is gathered each step (k + 2 requests per row).
    mode "delta": delta selection with capped eviction (Sec. 4.2.3) bounds the gather to
    `cap` blocks per (request, KV head) per step plus the local blocks.
    fused (default: whenever the library takes the shapes): a layer's attention and its scoring run
    as one launch on the foreground stream (`oasis_attn_and_score`); the summary updates of all
    layers are then issued at the start of the step on the prediction stream.
    transfer_streams: consecutive layers' gathers alternate between this many transfer streams (useful
    when the pool is in host memory: one gather's requests are in flight while the previous one's last
    ones come back).
    defer_tail: the last layer's prediction chain of a step is launched at the start of the next step
    (`flush()` launches a chain still pending); the state of that layer is then one step behind
    between steps.
    """

    def __init__(self, batch, n_q_heads, n_kv_heads, max_blocks, k, n_q_tokens, n_layers,
                 device="cuda", mode="fetch_all", cap=None, fused=None, transfer_streams=1, defer_tail=False):
        assert mode in ("fetch_all", "delta")
        self.mode, self.k, self.T, self.n_layers = mode, k, n_q_tokens, n_layers
        self.device = torch.device(device)
        self.layers = [DecodeLayer(batch, n_q_heads, n_kv_heads, max_blocks, k, n_q_tokens, device)
                       for _ in range(n_layers)]
        self.kv = [None] * n_layers
        self.table = [None] * n_layers
        self.main = torch.cuda.Stream(device=self.device)
        # The small kernels go to higher-priority streams: the block scheduler then places their few thread blocks
        # ahead of the big kernels' waiting ones instead of behind a partially dispatched grid.
        self.pred = torch.cuda.Stream(device=self.device, priority=-1)
        self.selq = torch.cuda.Stream(device=self.device, priority=-1)
        self.side = torch.cuda.Stream(device=self.device, priority=-1)
        self.copy = torch.cuda.Stream(device=self.device)     # end-to-end mode: query upload, output download
        # consecutive layers' gathers may alternate between several transfer streams, so that one gather's
        # requests are already in flight while the previous one's last ones come back over the host link
        self.xfer = [self.side] + [torch.cuda.Stream(device=self.device, priority=-1)
                                   for _ in range(max(1, int(transfer_streams)) - 1)]
        self.launches = 0
        self.cap = cap
        # defer_tail: the last layer's prediction chain (top-k, plan, gather) of a step is launched at the start of
        # the next step instead of at its end, where nothing would overlap it (the next step's attention of that
        # layer comes last and waits for it as usual); `flush()` launches a chain that is still pending.
        self.defer_tail = bool(defer_tail)
        self._deferred = None
        self._capturing = False
        can_fuse = n_layers > 0 and n_q_tokens > 1 and oasis.attn_and_score_supported(self.layers[0].dims, n_q_tokens, self.layers[0].cols, n_q_tokens - 1)
        self.fused = can_fuse if fused is None else (bool(fused) and can_fuse)
        self.stage_done = [None] * n_layers          # event of the layer's latest transfer
        self.sel_done = [None] * n_layers            # event of the layer's latest top-k (it reads the scores)
        if mode == "delta":
            assert cap is not None and 0 <= cap <= k
            dev, rows = self.device, (batch, n_kv_heads)
            self.resident = [torch.full(rows + (k + 2,), -1, dtype=torch.int32, device=dev) for _ in range(n_layers)]
            self.stamp = [torch.zeros(rows + (k + 2,), dtype=torch.int32, device=dev) for _ in range(n_layers)]
            self.plan_idx = [torch.empty(rows + (cap + 2,), dtype=torch.int64, device=dev) for _ in range(n_layers)]
            self.plan_slots = [torch.empty(rows + (cap + 2,), dtype=torch.int32, device=dev) for _ in range(n_layers)]
        self._splits = oasis.attn_workspace_bytes(self.layers[0].dims, n_q_tokens, k + 2) > 0 if n_layers else False

    def attach(self, layer, kv_src, block_table):
        """kv_src: the layer's full-KV pool (pinned host memory, or device memory)."""
        self.kv[layer], self.table[layer] = kv_src, block_table

    def blk_tbl(self, layer):
        return self.resident[layer] if self.mode == "delta" else self.layers[layer].sel

    @staticmethod
    def _tick(timers, name, stream):
        if timers is None or name not in timers:
            return None
        ev = torch.cuda.Event(enable_timing=True)
        ev.record(stream)
        return ev

    @staticmethod
    def _tock(timers, name, start, stream):
        if start is None:
            return
        ev = torch.cuda.Event(enable_timing=True)
        ev.record(stream)
        timers[name].append((start, ev))

    def _predict(self, l, q, first_block, n_new, max_new, n_full_next, seq_next, stamp, timers,
                 attn_done=None, plan=None, scored=None):
        """Prediction chain of one layer; returns the event after which the layer's gather may start.
        `scored`: the scores were already produced (by the fused launch) and this event marks them."""
        L, ps, qs = self.layers[l], self.pred, self.selq
        own_score = scored is None
        if own_score:
            with torch.cuda.stream(ps):
                # the scores buffer is rewritten: the previous step's top-k of this layer must have read it
                if self.sel_done[l] is not None:
                    ps.wait_event(self.sel_done[l])
                L.build_summaries(self.kv[l], self.table[l], first_block, n_new, max_new)
                t0 = self._tick(timers, "score", ps)
                L.score(q, n_full_next)
                self._tock(timers, "score", t0, ps)
                scored = torch.cuda.Event()
                scored.record(ps)
        # top-k and the transfer plan run on their own stream, so that waiting for this layer's attention does
        # not hold back the next layer's scoring
        with torch.cuda.stream(qs):
            if scored != "completed":                # (a chain deferred into the next captured step: all done)
                qs.wait_event(scored)
            if attn_done is not None:
                qs.wait_event(attn_done)            # sel / resident are read by this step's attention
            t0 = self._tick(timers, "select", qs)
            L.select(n_full_next, seq_next, self.table[l])
            self._tock(timers, "select", t0, qs)
            self.launches += 3 if own_score else 1      # (summary update, scoring,) top-k
            ev = torch.cuda.Event()
            ev.record(qs)
            self.sel_done[l] = ev
        if self.mode == "delta":
            # the transfer plan runs on the transfer stream, so the next layer's top-k does not queue behind it
            with torch.cuda.stream(self.side):
                self.side.wait_event(ev)
                plan_idx = self.plan_idx[l] if plan is None else plan[0]
                plan_slots = self.plan_slots[l] if plan is None else plan[1]
                oasis.plan_delta(L.dims, L.sel, self.k, self.table[l], self.resident[l], self.stamp[l],
                                 L.cols, plan_idx.shape[-1] - 2, stamp, plan_idx, plan_slots, n_local=2)
                self.launches += 1
                ev = torch.cuda.Event()
                ev.record(self.side)
        return ev

    def _transfer(self, l, ready, timers, plan=None):
        L, ss = self.layers[l], self.xfer[l % len(self.xfer)]
        with torch.cuda.stream(ss):
            ss.wait_event(ready)
            t0 = self._tick(timers, "stage", ss)
            if self.mode == "delta":
                plan_idx = self.plan_idx[l] if plan is None else plan[0]
                plan_slots = self.plan_slots[l] if plan is None else plan[1]
                oasis.stage_blocks(self.kv[l], plan_idx, plan_slots, plan_idx.numel(), L.pool)
            else:
                L.stage(self.kv[l])
            self._tock(timers, "stage", t0, ss)
            self.launches += 1
            ev = torch.cuda.Event()
            ev.record(ss)
        self.stage_done[l] = ev

    def handover(self, layer, dense_k, dense_v, gpu_table, seq_len):
        """Dense -> sparse transition of one layer (Sec. 4.3): every block of the dense GPU pool that
        holds tokens of a request is copied to the attached full-KV pool; the full blocks get their
        summaries on the way, the partially filled last block does not.  `prime(...,
        summaries_ready=True)` then selects and gathers the first working set."""
        L = self.layers[layer]
        torch.cuda.current_stream(self.device).synchronize()      # seq_len may still be in flight on the caller's stream
        with torch.cuda.stream(self.pred):                        # the small tensors are made on the stream that reads them
            n_full = (seq_len // 16).to(torch.int32)
            n_part = ((seq_len + 15) // 16).to(torch.int32) - n_full
            zeros = torch.zeros_like(n_full)
            oasis.offload_blocks(L.dims, dense_k, dense_v, gpu_table, self.table[layer], zeros, n_full, L.mb,
                                 self.kv[layer], L.summaries)
            oasis.offload_blocks(L.dims, dense_k, dense_v, gpu_table, self.table[layer], n_full, n_part, 1,
                                 self.kv[layer], None)
        self.launches += 2

    def prime(self, q_list, n_full_next, seq_next, step_stamp=0, summaries_ready=False):
        """Before the first step: build every summary (unless the hand-over already did) and run one
        prediction + transfer per layer, as the step before the first one would have done."""
        B = self.layers[0].B
        zeros = torch.zeros(B, dtype=torch.int32, device=self.device)
        n_build = zeros if summaries_ready else n_full_next
        torch.cuda.current_stream(self.device).synchronize()      # `zeros` is read on the engine's own streams
        plan = None
        if self.mode == "delta":        # the initial working set is admitted whole (cap = k)
            rows = (B, self.layers[0].Hkv, self.k + 2)
            plan = (torch.empty(rows, dtype=torch.int64, device=self.device),
                    torch.empty(rows, dtype=torch.int32, device=self.device))
        for l in range(self.n_layers):
            ready = self._predict(l, q_list[l], zeros, n_build, self.layers[l].mb, n_full_next, seq_next,
                                  step_stamp, None, plan=plan)
            self._transfer(l, ready, None, plan=plan)
            if plan is not None:
                for st in self.xfer:     # the shared priming plan is reused by the next layer
                    st.synchronize()
        torch.cuda.synchronize(self.device)
        self.stage_done = [None] * self.n_layers     # everything has completed
        self.sel_done = [None] * self.n_layers

    def step(self, q_list, seq_len, first_block, n_new, n_full_next, seq_next, step_stamp=0,
             timers=None, q_host=None, out_host=None):
        """One decode step over all layers.  seq_len: history tokens of this step; the
        prediction works on the next step's view (n_full_next, seq_next).  With q_host /
        out_host (pinned tensors per layer) the step's queries are copied in and its outputs
        copied out inside the step (end-to-end mode)."""
        ms, cs = self.main, self.copy
        self._launch_deferred(timers)
        q_ready = [None] * self.n_layers
        if q_host is not None or out_host is not None:
            # the copy stream starts after everything the previous step left on the other streams
            for st in (ms, self.pred):
                ev = torch.cuda.Event()
                ev.record(st)
                cs.wait_event(ev)
        if q_host is not None:
            # All of the step's queries cross the host link before its first gather: the zero-copy gathers keep
            # thousands of reads in flight on the link and would starve DMA copies queued beside them, which
            # would serialise gather(l) -> attention(l + 1).
            with torch.cuda.stream(cs):
                for l in range(self.n_layers):
                    q_list[l].copy_(q_host[l], non_blocking=True)
                    q_ready[l] = torch.cuda.Event()
                    q_ready[l].record(cs)
            for st in self.xfer:
                st.wait_event(q_ready[-1])
        summ_ready = [None] * self.n_layers
        if self.fused:
            # the summary updates (one newly completed block per request every 16 steps) only depend on this step's
            # KV append: all layers' updates go first, on the prediction stream
            with torch.cuda.stream(self.pred):
                for l0 in range(0, self.n_layers, oasis.MAX_LAYERS):       # one launch for (up to 128) layers
                    l1 = min(l0 + oasis.MAX_LAYERS, self.n_layers)
                    oasis.build_summaries_layers(self.layers[l0].dims, self.kv[l0:l1], self.table[l0:l1], first_block,
                                                 n_new, 1, [L.summaries for L in self.layers[l0:l1]])
                    self.launches += 1
                    # only the group's first fused launch waits for it: the later ones follow that launch on the
                    # foreground stream (a wait for the same, already awaited launch before every fused launch made
                    # the captured graph drop the programmatic edges between consecutive fused launches)
                    summ_ready[l0] = torch.cuda.Event()
                    summ_ready[l0].record(self.pred)
        for l in range(self.n_layers):
            L = self.layers[l]
            with torch.cuda.stream(ms):
                if q_ready[l] is not None:
                    ms.wait_event(q_ready[l])
                if self.stage_done[l] is not None:
                    ms.wait_event(self.stage_done[l])
                if self.fused:
                    if summ_ready[l] is not None:
                        ms.wait_event(summ_ready[l])
                    t0 = self._tick(timers, "layer", ms)
                    L.attend_and_score(q_list[l], seq_len, n_full_next, blk_tbl=self.blk_tbl(l))
                    self._tock(timers, "layer", t0, ms)
                    self.launches += 2 if self._splits else 1      # the fused launch (and the merge of split rows)
                else:
                    t0 = self._tick(timers, "attn", ms)
                    L.attend(q_list[l], seq_len, blk_tbl=self.blk_tbl(l))
                    self._tock(timers, "attn", t0, ms)
                    self.launches += 2 if self._splits else 1
                attn_done = torch.cuda.Event()
                attn_done.record(ms)
            if out_host is not None:
                cs.wait_event(attn_done)
                with torch.cuda.stream(cs):
                    out_host[l].copy_(L.out, non_blocking=True)
            if q_ready[l] is not None and not self.fused:
                self.pred.wait_event(q_ready[l])
            if self.defer_tail and self.fused and l == self.n_layers - 1:
                self._deferred = (l, q_list[l], first_block, n_new, n_full_next, seq_next, step_stamp, attn_done,
                                  self._capturing)
                continue
            ready = self._predict(l, q_list[l], first_block, n_new, 1, n_full_next, seq_next, step_stamp, timers,
                                  attn_done=attn_done, scored=attn_done if self.fused else None)
            self._transfer(l, ready, timers)
        if out_host is not None:
            ev = torch.cuda.Event()                  # the next step's attention overwrites the output buffers
            ev.record(cs)
            ms.wait_event(ev)

    def _launch_deferred(self, timers=None):
        if self._deferred is None:
            return
        l, q, first_block, n_new, n_full_next, seq_next, stamp, attn_done, was_captured = self._deferred
        self._deferred = None
        if self._capturing:
            attn_done = None                         # a graph starts after everything before it has completed
        elif was_captured:
            attn_done = torch.cuda.Event()           # the step was a graph replayed on the foreground stream
            attn_done.record(self.main)
        ready = self._predict(l, q, first_block, n_new, 1, n_full_next, seq_next, stamp, timers,
                              attn_done=attn_done, scored="completed")
        self._transfer(l, ready, timers)

    def flush(self):
        """Launches the prediction chain that `defer_tail` left pending (after the last step, or before reading the
        last layer's selection state)."""
        self._launch_deferred()

    def join(self):
        """Makes the foreground stream wait for everything the other streams have in flight."""
        for st in (self.pred, self.selq, self.copy, *self.xfer):
            ev = torch.cuda.Event()
            ev.record(st)
            self.main.wait_event(ev)
        self.stage_done = [None] * self.n_layers

    def capture_step(self, *args, **kwargs):
        """Captures one step (same arguments as `step`) into a CUDA graph on the foreground
        stream and returns it; `graph.replay()` must be issued on that stream, and a replay
        completes only when all streams' work of the step has completed."""
        torch.cuda.synchronize(self.device)
        self.stage_done = [None] * self.n_layers
        self.sel_done = [None] * self.n_layers
        before = self.launches
        g = torch.cuda.CUDAGraph()
        fork = torch.cuda.Event()
        self._capturing = True
        with torch.cuda.graph(g, stream=self.main, capture_error_mode="thread_local"):
            fork.record(self.main)
            self.pred.wait_event(fork)
            self.selq.wait_event(fork)
            for st in self.xfer:
                st.wait_event(fork)
            self.copy.wait_event(fork)
            self.step(*args, **kwargs)
            self.join()
        self._capturing = False
        self.sel_done = [None] * self.n_layers       # events recorded inside a capture mean nothing outside it
        g.launches = self.launches - before
        self.launches = before
        return g

    def replay(self, graph):
        with torch.cuda.stream(self.main):
            graph.replay()
        self.launches += graph.launches
