"""ctypes/numpy front end of the CPU oracle (test infrastructure only).

Every function takes and returns numpy arrays; bf16 tensors travel as uint16 bit
patterns.  Nothing here may be imported by the product package: only tests, the smoke
check and the benchmark's CPU-baseline leg use it.  The arithmetic lives in
oasis_oracle.c; this file only marshals arguments.
"""
import ctypes
import os

import numpy as np

from . import build as _build

_LIB = None


def lib():
    global _LIB
    if _LIB is None:
        _LIB = ctypes.CDLL(_build.build())
        _LIB.oasis_oracle_topk_recall.restype = ctypes.c_double
    return _LIB


def _p(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


def _i32(a):
    return np.ascontiguousarray(a, dtype=np.int32)


def _u16(a):
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def f32_to_bf16(x):
    x = np.ascontiguousarray(x, dtype=np.float32)
    out = np.empty(x.shape, dtype=np.uint16)
    lib().oasis_oracle_f32_to_bf16(_p(x), _p(out), ctypes.c_int64(x.size))
    return out


def bf16_to_f32(x):
    x = _u16(x)
    out = np.empty(x.shape, dtype=np.float32)
    lib().oasis_oracle_bf16_to_f32(_p(x), _p(out), ctypes.c_int64(x.size))
    return out


def build_summaries(kv_pool, block_table, first_block, n_blocks, summaries=None):
    """kv_pool [P][Hkv][2][bs][d] u16, block_table [B][max_blocks] -> summaries
    [B][Hkv][max_blocks][2][d] u16 (updated in place when given)."""
    kv_pool = _u16(kv_pool)
    block_table = _i32(block_table)
    _, Hkv, _, bs, d = kv_pool.shape
    B, max_blocks = block_table.shape
    if summaries is None:
        summaries = np.zeros((B, Hkv, max_blocks, 2, d), dtype=np.uint16)
    assert summaries.flags.c_contiguous and summaries.dtype == np.uint16
    first_block, n_blocks = _i32(first_block), _i32(n_blocks)
    lib().oasis_oracle_build_summaries(B, Hkv, d, bs, max_blocks, _p(kv_pool), _p(block_table),
                                       _p(first_block), _p(n_blocks), _p(summaries))
    return summaries


def score_blocks(q_draft, summaries, n_full, reduce_mode=0):
    """q_draft [B][Td][Hq][d] u16 -> (scores fp32, scores fp64), each [B][Hkv][max_blocks]."""
    q_draft, summaries, n_full = _u16(q_draft), _u16(summaries), _i32(n_full)
    B, Td, Hq, d = q_draft.shape
    _, Hkv, max_blocks, _, _ = summaries.shape
    s32 = np.empty((B, Hkv, max_blocks), dtype=np.float32)
    s64 = np.empty((B, Hkv, max_blocks), dtype=np.float64)
    lib().oasis_oracle_score_blocks(B, Hq, Hkv, d, max_blocks, _p(q_draft), Td, _p(summaries),
                                    _p(n_full), int(reduce_mode), _p(s32), _p(s64))
    return s32, s64


def select_topk(scores, n_full, seq_len, n_q_tokens, k, block_table, bs=16, want_stage=True):
    """-> sel [B][Hkv][k+2] (and stage_idx int64, stage_slots int32, same shape)."""
    scores = np.ascontiguousarray(scores, dtype=np.float32)
    B, Hkv, max_blocks = scores.shape
    n_full, seq_len, block_table = _i32(n_full), _i32(seq_len), _i32(block_table)
    sel = np.empty((B, Hkv, k + 2), dtype=np.int32)
    idx = np.empty((B, Hkv, k + 2), dtype=np.int64) if want_stage else None
    slots = np.empty((B, Hkv, k + 2), dtype=np.int32) if want_stage else None
    lib().oasis_oracle_select_topk(B, Hkv, max_blocks, bs, _p(scores), _p(n_full), _p(seq_len),
                                   int(n_q_tokens), int(k), _p(block_table), _p(sel), _p(idx),
                                   _p(slots))
    return (sel, idx, slots) if want_stage else sel


def stage_blocks(host_kv, idx, slots, pool):
    """pool[slots[i]] = host_kv[idx[i]]; both pools u16 arrays whose leading axes index
    entries ([..., 2, bs, d]); pool is modified in place and returned."""
    host_kv, pool = _u16(host_kv), pool
    assert pool.flags.c_contiguous and pool.dtype == np.uint16
    entry_bytes = int(np.prod(host_kv.shape[-3:])) * 2
    idx = np.ascontiguousarray(idx, dtype=np.int64).reshape(-1)
    slots = _i32(slots).reshape(-1)
    lib().oasis_oracle_stage_blocks(_p(host_kv), _p(idx), _p(slots), int(idx.size),
                                    ctypes.c_int64(entry_bytes), _p(pool))
    return pool


def sparse_attn(q, pool, slot_tbl, blk_tbl, seq_len, scale, Hkv):
    """q [B][T][Hq][d] u16, pool [n_slots][2][bs][d] u16, tables [B][Hkv][n_cols]
    -> dict(out32, out64, out_bf16, lse, out_abs); out_abs = sum_p softmax_p * |v_p| (fp64), the scale of the
    terms behind each output element."""
    q, pool = _u16(q), _u16(pool)
    B, T, Hq, d = q.shape
    bs = pool.shape[-2]
    slot_tbl, blk_tbl, seq_len = _i32(slot_tbl), _i32(blk_tbl), _i32(seq_len)
    n_cols = blk_tbl.shape[-1]
    out32 = np.empty((B, T, Hq, d), dtype=np.float32)
    out64 = np.empty((B, T, Hq, d), dtype=np.float64)
    out16 = np.empty((B, T, Hq, d), dtype=np.uint16)
    lse = np.empty((B, T, Hq), dtype=np.float32)
    out_abs = np.empty((B, T, Hq, d), dtype=np.float64)
    lib().oasis_oracle_sparse_attn_abs(B, T, Hq, int(Hkv), d, bs, _p(q), _p(pool), _p(slot_tbl),
                                       _p(blk_tbl), n_cols, _p(seq_len), ctypes.c_float(scale),
                                       _p(out32), _p(out64), _p(out16), _p(lse), _p(out_abs))
    return dict(out32=out32, out64=out64, out_bf16=out16, lse=lse, out_abs=out_abs)


def topk_recall(sel_draft, sel_true, k):
    sel_draft, sel_true = _i32(sel_draft), _i32(sel_true)
    cols = sel_draft.shape[-1]
    rows = sel_draft.size // cols
    return float(lib().oasis_oracle_topk_recall(rows, cols, int(k), _p(sel_draft), _p(sel_true)))


def plan_delta(sel, block_table, resident, stamp, k, cap, step, slot_stride, n_res=None, n_local=0):
    """Updates resident/stamp [B][Hkv][res_stride] in place (n_res eviction-managed columns,
    then n_local local-block columns); returns (plan_idx int64 [B][Hkv][cap+n_local],
    plan_slots int32 (same shape), n_admitted [B][Hkv])."""
    sel, block_table = _i32(sel), _i32(block_table)
    assert resident.dtype == np.int32 and resident.flags.c_contiguous
    assert stamp.dtype == np.int32 and stamp.flags.c_contiguous
    B, Hkv, sel_cols = sel.shape
    res_stride = resident.shape[-1]
    n_res = res_stride - n_local if n_res is None else n_res
    max_blocks = block_table.shape[-1]
    plan_idx = np.empty((B, Hkv, max(cap, 0) + n_local), dtype=np.int64)
    plan_slots = np.empty((B, Hkv, max(cap, 0) + n_local), dtype=np.int32)
    n_adm = np.empty((B, Hkv), dtype=np.int32)
    lib().oasis_oracle_plan_delta(B, Hkv, max_blocks, int(k), sel_cols, int(n_res), int(res_stride),
                                  int(n_local), int(slot_stride), int(cap), int(step), _p(sel),
                                  _p(block_table), _p(resident), _p(stamp), _p(plan_idx),
                                  _p(plan_slots), _p(n_adm))
    return plan_idx, plan_slots, n_adm


def union_blocks(sel, k, max_blocks, max_union):
    """sel [B][Hkv][cols] -> (union_idx [B][max_union] ascending, -1 padded; n_union [B])."""
    sel = _i32(sel)
    B, Hkv, cols = sel.shape
    idx = np.empty((B, max_union), dtype=np.int32)
    n = np.empty((B,), dtype=np.int32)
    lib().oasis_oracle_union_blocks(B, Hkv, int(max_blocks), cols, int(k), _p(sel), int(max_union), _p(idx), _p(n))
    return idx, n


def offload_blocks(dense_k, dense_v, gpu_table, block_table, first_block, n_blocks, host_kv, summaries=None):
    """dense_k / dense_v [P_gpu][Hkv][bs][d] u16 -> entries of host_kv [P_cpu][Hkv][2][bs][d] u16 (in
    place); summaries [B][Hkv][max_blocks][2][d] u16 are updated in place when given."""
    dense_k, dense_v = _u16(dense_k), _u16(dense_v)
    gpu_table, block_table = _i32(gpu_table), _i32(block_table)
    first_block, n_blocks = _i32(first_block), _i32(n_blocks)
    _, Hkv, bs, d = dense_k.shape
    B, max_blocks = block_table.shape
    assert host_kv.dtype == np.uint16 and host_kv.flags.c_contiguous
    if summaries is not None:
        assert summaries.dtype == np.uint16 and summaries.flags.c_contiguous
    lib().oasis_oracle_offload_blocks(B, Hkv, d, bs, max_blocks, _p(dense_k), _p(dense_v), _p(gpu_table),
                                      _p(block_table), _p(first_block), _p(n_blocks), _p(host_kv), _p(summaries))
    return host_kv


def local_window(seq_len, n_q_tokens, block_table, blk_tbl, local_col, slot_stride, want_stage=True, bs=16):
    """Sets the two local columns of blk_tbl [B][Hkv][n_cols] (in place) by block parity; returns
    (stage_idx int64 [B][Hkv][2], stage_slots int32 [B][Hkv][2]) that reload them from the CPU pool."""
    seq_len, block_table = _i32(seq_len), _i32(block_table)
    assert blk_tbl.dtype == np.int32 and blk_tbl.flags.c_contiguous
    B, Hkv, n_cols = blk_tbl.shape
    max_blocks = block_table.shape[-1]
    idx = np.empty((B, Hkv, 2), dtype=np.int64) if want_stage else None
    slots = np.empty((B, Hkv, 2), dtype=np.int32) if want_stage else None
    lib().oasis_oracle_local_window(B, Hkv, bs, max_blocks, _p(seq_len), int(n_q_tokens), _p(block_table),
                                    _p(blk_tbl), n_cols, int(local_col), int(slot_stride), _p(idx), _p(slots))
    return idx, slots


def append_kv(new_kv, n_commit, seq_len, block_table, slot_tbl, blk_tbl, local_col, pool, host_kv=None):
    """new_kv [B][T][Hkv][2][d] u16; pool [n_slots][2][bs][d] and host_kv [P][Hkv][2][bs][d] u16 and blk_tbl
    [B][Hkv][n_cols] int32 are updated in place."""
    new_kv = _u16(new_kv)
    B, T, Hkv, _, d = new_kv.shape
    seq_len, block_table, slot_tbl = _i32(seq_len), _i32(block_table), _i32(slot_tbl)
    assert blk_tbl.dtype == np.int32 and blk_tbl.flags.c_contiguous
    assert pool.dtype == np.uint16 and pool.flags.c_contiguous
    if host_kv is not None:
        assert host_kv.dtype == np.uint16 and host_kv.flags.c_contiguous
    bs = pool.shape[-2]
    n_cols = blk_tbl.shape[-1]
    max_blocks = block_table.shape[-1]
    lib().oasis_oracle_append_kv(B, T, Hkv, d, bs, max_blocks, int(n_commit), _p(new_kv), _p(seq_len),
                                 _p(block_table), _p(slot_tbl), _p(blk_tbl), n_cols, int(local_col), _p(pool),
                                 _p(host_kv))


def block_mass(q_true, kv_pool, block_table, seq_len, scale):
    """q_true [B][Tq][Hq][d] u16 (row t at position seq_len[b] + t), kv_pool [P][Hkv][2][bs][d] u16 ->
    mass [B][Hkv][max_blocks] fp64: the largest share of a sharing query row's dense attention that falls on
    each block."""
    q_true, kv_pool = _u16(q_true), _u16(kv_pool)
    block_table, seq_len = _i32(block_table), _i32(seq_len)
    B, Tq, Hq, d = q_true.shape
    _, Hkv, _, bs, _ = kv_pool.shape
    max_blocks = block_table.shape[-1]
    mass = np.empty((B, Hkv, max_blocks), dtype=np.float64)
    lib().oasis_oracle_block_mass(B, Tq, Hq, Hkv, d, bs, max_blocks, _p(q_true), _p(kv_pool), _p(block_table),
                                  _p(seq_len), ctypes.c_float(scale), _p(mass))
    return mass
