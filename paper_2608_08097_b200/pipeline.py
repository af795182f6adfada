"""Device buffers of one layer's sparse-decode state and the order of the library calls.

This is host-side bookkeeping only (allocation through torch, call sequencing, stream
choice); every step of the path runs inside liboasis.so through `binding`.
"""
import ctypes
import math

import torch

from . import binding as oasis


_libcuda = None                      # the driver library, loaded on the first DecodeEngine.upload


class DecodeLayer:
    """Working set of one layer: summaries, scores, selection, HBM slot pool, outputs.

    Fetch-all layout: row (b, h) owns the k + 2 consecutive pool slots
    (b * Hkv + h) * (k + 2) + c, column c holding the block sel[b][h][c].
    """

    def __init__(self, batch, n_q_heads, n_kv_heads, max_blocks, k, n_q_tokens, device="cuda",
                 want_lse=False, out=None):
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
        self.out = torch.empty((batch, n_q_tokens, n_q_heads, 128), dtype=torch.bfloat16, device=dev) if out is None else out
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
    """Sequencing of decode steps across layers, after the paper's asynchronous prefetch pipeline
    (Sec. 4.2.2).  Streams:
      foreground  attention of every layer over the working set that the previous step's
                  prediction staged;
      prediction  the step's KV append and summary update for newly completed blocks, and (unfused)
                  scoring with the draft queries;
      selection   top-k -- the tables a layer's attention reads are only rewritten after that
                  attention has finished;
      transfer    the transfer plan and the gather of what was selected, awaited, per layer, only by
                  the next step's attention of that same layer.
    In end-to-end mode an upload stream brings each layer's queries from pinned host memory and a
    download stream returns each layer's output.
    Every dependency is per layer and carries over from one step to the next, so consecutive steps
    overlap exactly as far as the data allows: a layer's gather may still be running while the next
    step's first layers attend.  Steps can be captured into CUDA graphs, one or several per graph
    (`capture_steps`); only the end of a graph is a synchronisation point.

    mode "fetch_all": every selected block is gathered each step (k + 2 requests per row).
    mode "delta": delta selection with capped eviction (Sec. 4.2.3) bounds the gather to
    `cap` blocks per (request, KV head) per step.
    append (delta mode): every step is given its new keys and values (`new_kv`), which `oasis_append_kv`
    writes into the GPU-resident local window (the committed token also through to the full-KV pool),
    so the local blocks never cross the host link; without it the local blocks are gathered from the
    full-KV pool like selected ones.
    fused (default: whenever the library takes the shapes): a layer's attention and its scoring run
    as one launch on the foreground stream (`oasis_attn_and_score`); the summary updates of all
    layers are then issued at the start of the step on the prediction stream.
    transfer_streams: consecutive layers' gathers alternate between this many transfer streams (useful
    when the pool is in host memory: one gather's requests are in flight while the previous one's last
    ones come back).
    transfer_group: the gathers of this many consecutive layers are one launch (`oasis_stage_blocks_layers`): a
    few large gathers keep the host link busier than many small ones; a layer's next-step attention then waits
    for its group's launch.
    transfer_kind: "warp" = the warp-per-entry zero-copy gather, "bulk" = `oasis_stage_blocks_bulk` (8 KiB bulk copies
    through shared memory: the faster one where the host link bounds the step).
    wait_group: the foreground stream picks up the other streams' events (a layer's transfer, query
    upload and output download of the previous step) for `wait_group` layers at a time, in front of the
    group's first launch.  A fused launch that follows a cross-stream wait is fully serialised behind
    its predecessor, the others overlap it through programmatic dependent launch; so fewer waits keep
    more of that overlap, at the price of a coarser dependency.
    """

    def __init__(self, batch, n_q_heads, n_kv_heads, max_blocks, k, n_q_tokens, n_layers,
                 device="cuda", mode="fetch_all", cap=None, fused=None, transfer_streams=1, wait_group=8,
                 append=False, transfer_group=1, plan_stream="own", n_commit=1, transfer_ctas=0, transfer_kind="warp"):
        assert mode in ("fetch_all", "delta")
        assert not append or mode == "delta", "the KV append goes with delta selection"
        self.append = bool(append)
        self.transfer_ctas = int(transfer_ctas)  # thread blocks per gather launch (0: the library's default)
        if transfer_kind not in ("warp", "bulk"):
            raise ValueError("transfer_kind must be 'warp' or 'bulk'")
        self.transfer_kind = transfer_kind       # warp-per-entry zero-copy gather, or bulk copies through shared memory
        self.n_commit = int(n_commit)            # tokens per step that the KV append also writes to the full-KV pool
        self.mode, self.k, self.T, self.n_layers = mode, k, n_q_tokens, n_layers
        self.device = torch.device(device)
        # the layers' outputs are slices of one tensor, so that several layers' outputs can leave in one copy
        self.out_all = torch.empty((n_layers, batch, n_q_tokens, n_q_heads, 128), dtype=torch.bfloat16, device=self.device)
        self.layers = [DecodeLayer(batch, n_q_heads, n_kv_heads, max_blocks, k, n_q_tokens, device, out=self.out_all[l])
                       for l in range(n_layers)]
        self.kv = [None] * n_layers
        self.table = [None] * n_layers
        self.main = torch.cuda.Stream(device=self.device)
        # The small kernels go to higher-priority streams: the block scheduler then places their few thread blocks
        # ahead of the big kernels' waiting ones instead of behind a partially dispatched grid.
        self.pred = torch.cuda.Stream(device=self.device, priority=-1)
        self.selq = torch.cuda.Stream(device=self.device, priority=-1)
        self.side = torch.cuda.Stream(device=self.device, priority=-1)
        # transfer plans: a stream of their own (never queued behind a gather), or the first transfer stream
        self.planq = torch.cuda.Stream(device=self.device, priority=-1) if plan_stream == "own" else self.side
        self.up = torch.cuda.Stream(device=self.device)       # end-to-end mode: query upload
        self.down = torch.cuda.Stream(device=self.device)     # end-to-end mode: output download
        # consecutive layers' gathers may alternate between several transfer streams, so that one gather's
        # requests are already in flight while the previous one's last ones come back over the host link
        self.xfer = [self.side] + [torch.cuda.Stream(device=self.device, priority=-1)
                                   for _ in range(max(1, int(transfer_streams)) - 1)]
        self.launches = 0
        self.cap = cap
        self.wait_group = max(1, int(wait_group))
        self.transfer_group = max(1, min(int(transfer_group), oasis.MAX_STAGE_LAYERS))
        can_fuse = n_layers > 0 and n_q_tokens > 1 and oasis.attn_and_score_supported(self.layers[0].dims, n_q_tokens, self.layers[0].cols, n_q_tokens - 1)
        self.fused = can_fuse if fused is None else (bool(fused) and can_fuse)
        self._reset_events()
        if mode == "delta":
            assert cap is not None and 0 <= cap <= k
            dev, rows = self.device, (batch, n_kv_heads)
            self.resident = [torch.full(rows + (k + 2,), -1, dtype=torch.int32, device=dev) for _ in range(n_layers)]
            self.stamp = [torch.zeros(rows + (k + 2,), dtype=torch.int32, device=dev) for _ in range(n_layers)]
            n_req = cap + (0 if append else 2)       # requests per row: the admitted pairs (and the local blocks)
            self.plan_idx = [torch.empty(rows + (n_req,), dtype=torch.int64, device=dev) for _ in range(n_layers)]
            self.plan_slots = [torch.empty(rows + (n_req,), dtype=torch.int32, device=dev) for _ in range(n_layers)]
        self._splits = oasis.attn_workspace_bytes(self.layers[0].dims, n_q_tokens, k + 2) > 0 if n_layers else False

    def _reset_events(self):
        """Forgets the previous step's events (everything before has completed)."""
        n = self.n_layers
        self.stage_done = [None] * n         # the layer's latest transfer
        self.sel_done = [None] * n           # the layer's latest top-k (it reads the scores)
        self.attn_done = [None] * n          # the layer's latest attention (it reads q, the tables and the pool)
        self.score_done = [None] * n         # unfused: the layer's latest scoring (it reads q)
        self.out_done = [None] * n           # end to end: the download of the layer's latest output

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

    @staticmethod
    def _event(stream):
        ev = torch.cuda.Event()
        ev.record(stream)
        return ev

    def _predict(self, l, q, first_block, n_new, max_new, n_full_next, seq_next, stamp, timers,
                 attn_done=None, plan=None, scored=None, n_local=2, sel_log=None):
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
                scored = self._event(ps)
                self.score_done[l] = scored
        # top-k and the transfer plan run on their own streams, so that waiting for this layer's attention does
        # not hold back the next layer's scoring
        with torch.cuda.stream(qs):
            qs.wait_event(scored)
            if attn_done is not None:
                qs.wait_event(attn_done)            # sel / resident are read by this step's attention
            t0 = self._tick(timers, "select", qs)
            L.select(n_full_next, seq_next, self.table[l])
            self._tock(timers, "select", t0, qs)
            if sel_log is not None:
                sel_log.copy_(L.sel, non_blocking=True)  # a record of this step's selection (tests, analysis)
            self.launches += 3 if own_score else 1      # (summary update, scoring,) top-k
            ev = self._event(qs)
            self.sel_done[l] = ev
        if self.mode == "delta":
            # the transfer plan runs on a stream of its own, so neither the next layer's top-k nor this plan queues
            # behind a gather
            with torch.cuda.stream(self.planq):
                self.planq.wait_event(ev)
                plan_idx = self.plan_idx[l] if plan is None else plan[0]
                plan_slots = self.plan_slots[l] if plan is None else plan[1]
                oasis.plan_delta(L.dims, L.sel, self.k, self.table[l], self.resident[l], self.stamp[l],
                                 L.cols, plan_idx.shape[-1] - n_local, stamp, plan_idx, plan_slots, n_local=n_local,
                                 n_res=self.k)
                self.launches += 1
                ev = self._event(self.planq)
        return ev

    def _transfer(self, ls, readies, timers, plan=None):
        """The gather of the consecutive layers `ls` (one launch), after their plans / selections `readies`."""
        ss = self.xfer[(ls[0] // self.transfer_group) % len(self.xfer)]
        with torch.cuda.stream(ss):
            for ev in readies:
                ss.wait_event(ev)
            t0 = self._tick(timers, "stage", ss)
            if self.mode == "delta":
                idx = [self.plan_idx[l] if plan is None else plan[0] for l in ls]
                slots = [self.plan_slots[l] if plan is None else plan[1] for l in ls]
            else:
                idx = [self.layers[l].stage_idx for l in ls]
                slots = [self.layers[l].stage_slots for l in ls]
            if self.transfer_kind == "bulk":
                oasis.stage_blocks_bulk([self.kv[l] for l in ls], idx, slots, idx[0].numel(),
                                        [self.layers[l].pool for l in ls], max_streams=self.transfer_ctas)
            elif len(ls) == 1 and self.transfer_ctas == 0:
                oasis.stage_blocks(self.kv[ls[0]], idx[0], slots[0], idx[0].numel(), self.layers[ls[0]].pool)
            else:
                oasis.stage_blocks_layers([self.kv[l] for l in ls], idx, slots, idx[0].numel(),
                                          [self.layers[l].pool for l in ls], max_ctas=self.transfer_ctas)
            self._tock(timers, "stage", t0, ss)
            self.launches += 1
            ev = self._event(ss)
            for l in ls:
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
        prediction + transfer per layer, as the step before the first one would have done.  With the KV
        append the (partially filled) local block is loaded from the full-KV pool into the local window
        once, here."""
        B = self.layers[0].B
        zeros = torch.zeros(B, dtype=torch.int32, device=self.device)
        n_build = zeros if summaries_ready else n_full_next
        torch.cuda.current_stream(self.device).synchronize()      # `zeros` is read on the engine's own streams
        plan = None
        n_local = 0 if self.append else 2
        if self.mode == "delta":        # the initial working set is admitted whole (cap = k)
            rows = (B, self.layers[0].Hkv, self.k + n_local)
            plan = (torch.empty(rows, dtype=torch.int64, device=self.device),
                    torch.empty(rows, dtype=torch.int32, device=self.device))
        for l in range(self.n_layers):
            L = self.layers[l]
            ready = self._predict(l, q_list[l], zeros, n_build, L.mb, n_full_next, seq_next,
                                  step_stamp, None, plan=plan, n_local=n_local)
            self._transfer([l], [ready], None, plan=plan)
            if self.append:
                with torch.cuda.stream(self.side):
                    self.side.wait_event(self.stage_done[l])
                    idx = torch.empty((B, L.Hkv, 2), dtype=torch.int64, device=self.device)
                    slots = torch.empty((B, L.Hkv, 2), dtype=torch.int32, device=self.device)
                    oasis.local_window(L.dims, seq_next, self.T, self.table[l], self.resident[l], self.k, L.cols, idx, slots)
                    oasis.stage_blocks(self.kv[l], idx, slots, idx.numel(), L.pool)
                    self.launches += 2
            if plan is not None:
                for st in self.xfer:     # the shared priming plan is reused by the next layer
                    st.synchronize()
        torch.cuda.synchronize(self.device)
        self._reset_events()                         # everything has completed

    def step(self, q_list, seq_len, first_block, n_new, n_full_next, seq_next, step_stamp=0,
             timers=None, q_host=None, out_host=None, new_kv=None, sel_log=None):
        """One decode step over all layers.  seq_len: history tokens of this step; the
        prediction works on the next step's view (n_full_next, seq_next).  With q_host /
        out_host (pinned tensors per layer) the step's queries are copied in and its outputs
        copied out inside the step (end-to-end mode).  When q_list / q_host / out_host are each ONE tensor stacked
        over the layers ([n_layers][B][T][Hq][128]) the copies are made for `wait_group` layers at a time: a few
        large copies disturb the gathers on the host link less than many small ones.  new_kv (one [B][T][Hkv][2][128] tensor per
        layer; engines built with append=True): the step's new keys and values.  sel_log (one tensor like
        `layers[l].sel` per layer): receives a copy of each layer's selection of this step."""
        ms, n = self.main, self.n_layers
        if self.append != (new_kv is not None):
            raise ValueError("new_kv must be given exactly when the engine was built with append=True")
        q_ready = [None] * n
        stacked = isinstance(q_list, torch.Tensor)
        if q_host is not None:
            # a layer's queries are uploaded as soon as the previous step no longer reads the staging tensor
            with torch.cuda.stream(self.up):
                grp = self.wait_group if (stacked and isinstance(q_host, torch.Tensor)) else 1
                for l0 in range(0, n, grp):
                    l1 = min(l0 + grp, n)
                    for l in range(l0, l1):
                        for ev in (self.attn_done[l], self.score_done[l]):
                            if ev is not None:
                                self.up.wait_event(ev)
                    if grp == 1:
                        q_list[l0].copy_(q_host[l0], non_blocking=True)
                    else:
                        q_list[l0:l1].copy_(q_host[l0:l1], non_blocking=True)
                    ev = self._event(self.up)
                    for l in range(l0, l1):
                        q_ready[l] = ev
        # Per group of `wait_group` layers, on the prediction stream: the KV append (the previous step's attention of
        # the group's layers read the local window and the local columns that are rewritten now) and, for the fused
        # launch, the summary updates (one newly completed block per request every 16 steps), which only depend on the
        # append.  Only the group's first launch on the foreground stream waits for them.
        head_ready = {}
        if self.append or self.fused:
            with torch.cuda.stream(self.pred):
                for l0 in range(0, n, self.wait_group):
                    l1 = min(l0 + self.wait_group, n)
                    if self.append:
                        if self.attn_done[l1 - 1] is not None:
                            self.pred.wait_event(self.attn_done[l1 - 1])
                        for a0 in range(l0, l1, oasis.MAX_APPEND_LAYERS):
                            a1 = min(a0 + oasis.MAX_APPEND_LAYERS, l1)
                            oasis.append_kv_layers(self.layers[a0].dims, new_kv[a0:a1], self.n_commit, seq_len, self.table[a0:a1],
                                                   [L.slot_tbl for L in self.layers[a0:a1]], self.resident[a0:a1], self.k,
                                                   [L.pool for L in self.layers[a0:a1]], self.kv[a0:a1])
                            self.launches += 1
                    if self.fused:
                        for a0 in range(l0, l1, oasis.MAX_LAYERS):
                            a1 = min(a0 + oasis.MAX_LAYERS, l1)
                            oasis.build_summaries_layers(self.layers[a0].dims, self.kv[a0:a1], self.table[a0:a1], first_block,
                                                         n_new, 1, [L.summaries for L in self.layers[a0:a1]])
                            self.launches += 1
                    head_ready[l0] = self._event(self.pred)
        pending, readies = [], []
        for l in range(n):
            L = self.layers[l]
            with torch.cuda.stream(ms):
                if l % self.wait_group == 0:
                    # what the other streams did for the layers of this group: queries uploaded, the previous step's
                    # transfer landed, the previous step's output downloaded, this step's tokens appended
                    for g in range(l, min(l + self.wait_group, n)):
                        for ev in (q_ready[g], self.stage_done[g], self.out_done[g]):
                            if ev is not None:
                                ms.wait_event(ev)
                    if l in head_ready:
                        ms.wait_event(head_ready[l])
                if self.fused:
                    t0 = self._tick(timers, "layer", ms)
                    L.attend_and_score(q_list[l], seq_len, n_full_next, blk_tbl=self.blk_tbl(l))
                    self._tock(timers, "layer", t0, ms)
                else:
                    t0 = self._tick(timers, "attn", ms)
                    L.attend(q_list[l], seq_len, blk_tbl=self.blk_tbl(l))
                    self._tock(timers, "attn", t0, ms)
                self.launches += 2 if self._splits else 1      # the launch (and the merge of split rows)
                attn_done = self._event(ms)
                self.attn_done[l] = attn_done
            if out_host is not None:
                with torch.cuda.stream(self.down):
                    self.down.wait_event(attn_done)
                    if not isinstance(out_host, torch.Tensor):
                        out_host[l].copy_(L.out, non_blocking=True)
                        self.out_done[l] = self._event(self.down)
                    elif (l + 1) % self.wait_group == 0 or l == n - 1:
                        l0 = l - l % self.wait_group
                        out_host[l0:l + 1].copy_(self.out_all[l0:l + 1], non_blocking=True)
                        ev = self._event(self.down)
                        for g in range(l0, l + 1):
                            self.out_done[g] = ev
            if q_ready[l] is not None and not self.fused:
                self.pred.wait_event(q_ready[l])
            ready = self._predict(l, q_list[l], first_block, n_new, 1, n_full_next, seq_next, step_stamp, timers,
                                  attn_done=attn_done, scored=attn_done if self.fused else None,
                                  n_local=0 if self.append else 2, sel_log=None if sel_log is None else sel_log[l])
            pending.append(l)
            readies.append(ready)
            if len(pending) == self.transfer_group or l == n - 1:
                self._transfer(pending, readies, timers)
                pending, readies = [], []

    def join(self):
        """Makes the foreground stream wait for everything the other streams have in flight."""
        for st in (self.pred, self.selq, self.planq, self.up, self.down, *self.xfer):
            self.main.wait_event(self._event(st))

    def capture_steps(self, steps):
        """Captures consecutive steps -- a list of (args, kwargs) of `step` -- into one CUDA graph on the
        foreground stream and returns it.  Inside the graph the steps overlap as far as their per-layer
        dependencies allow; `graph.replay()` must be issued on that stream, and a replay completes only when
        all streams' work of its last step has completed."""
        torch.cuda.synchronize(self.device)
        self._reset_events()
        before = self.launches
        g = torch.cuda.CUDAGraph()
        fork = torch.cuda.Event()
        with torch.cuda.graph(g, stream=self.main, capture_error_mode="thread_local"):
            fork.record(self.main)
            for st in (self.pred, self.selq, self.planq, self.up, self.down, *self.xfer):
                st.wait_event(fork)
            for args, kwargs in steps:
                self.step(*args, **kwargs)
            self.join()
        self._reset_events()                         # events recorded inside a capture mean nothing outside it
        g.launches = self.launches - before
        g.n_steps = len(steps)
        self.launches = before
        return g

    def capture_step(self, *args, **kwargs):
        """One step (same arguments as `step`) as a CUDA graph."""
        return self.capture_steps([(args, kwargs)])

    def upload(self, graph):
        """Makes an instantiated graph resident on the device ahead of its first replay (the driver's cuGraphUpload
        on the foreground stream): the first replay of a graph of some thousand nodes otherwise spends milliseconds
        on the host before the device sees its first node.  Returns False, having done nothing, where the driver
        library or the graph's handle cannot be had (the replay then uploads the graph itself)."""
        global _libcuda
        if _libcuda is None:
            try:
                lib = ctypes.CDLL("libcuda.so.1")
                lib.cuGraphUpload.argtypes = [ctypes.c_void_p, ctypes.c_void_p]
                lib.cuGraphUpload.restype = ctypes.c_int
                _libcuda = lib
            except (OSError, AttributeError):
                _libcuda = False
        if not _libcuda or not hasattr(graph, "raw_cuda_graph_exec"):
            return False
        rc = _libcuda.cuGraphUpload(ctypes.c_void_p(graph.raw_cuda_graph_exec()), ctypes.c_void_p(self.main.cuda_stream))
        if rc != 0:
            raise RuntimeError("cuGraphUpload failed with CUresult %d" % rc)
        return True

    def replay(self, graph):
        with torch.cuda.stream(self.main):
            graph.replay()
        self.launches += graph.launches
