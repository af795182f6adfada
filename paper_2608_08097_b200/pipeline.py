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
