"""Python names for the C-ABI calls of include/oasis.h -- argument marshalling only.

Every function takes torch tensors (device memory, or pinned host memory for the full-KV
pool), checks dtype / contiguity, hands raw pointers to liboasis.so and raises
`OasisError` when the library reports a failure.  All arithmetic happens in the CUDA
kernels; there is no CPU fallback: if liboasis.so has not been built
(`python -m paper_2608_08097_b200.build`), the first call raises.
"""
import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
# OASIS_LIB selects another build of the library for the whole process (the bounds-check build liboasis_checked.so)
LIB_PATH = os.environ.get("OASIS_LIB") or os.path.join(_HERE, "liboasis.so")

REDUCE_MAX, REDUCE_SUM = 0, 1
ENTRY_BYTES = 8192
SYMBOLS = ("oasis_build_summaries", "oasis_score_blocks", "oasis_select_topk",
           "oasis_stage_blocks", "oasis_sparse_attn", "oasis_attn_workspace_bytes",
           "oasis_plan_delta", "oasis_last_error", "oasis_version",
           "oasis_sparse_attn_static_scratch", "oasis_static_scratch_bytes", "oasis_set_error_word", "oasis_union_blocks",
           "oasis_offload_blocks", "oasis_attn_and_score", "oasis_attn_and_score_supported",
           "oasis_build_summaries_layers", "oasis_selftest_wait_timeout",
           "oasis_local_window", "oasis_append_kv", "oasis_append_kv_layers", "oasis_stage_blocks_layers", "oasis_stage_blocks_bulk",
           "oasis_set_extents", "oasis_bounds_checked")


class OasisError(RuntimeError):
    pass


class _Dims(ctypes.Structure):
    _fields_ = [(n, ctypes.c_int32) for n in
                ("batch", "n_q_heads", "n_kv_heads", "head_dim", "block_size", "max_blocks")]


@dataclass(frozen=True)
class Dims:
    batch: int
    n_q_heads: int
    n_kv_heads: int
    max_blocks: int
    head_dim: int = 128
    block_size: int = 16

    def c(self):
        return _Dims(self.batch, self.n_q_heads, self.n_kv_heads, self.head_dim, self.block_size,
                     self.max_blocks)


_lib = None


def lib():
    """Loads liboasis.so once; raises OasisError if it is missing."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise OasisError("%s not found: build it with `python -m paper_2608_08097_b200.build` "
                             "(there is no CPU fallback)" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, i32, i64, f32, sz = (ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64, ctypes.c_float,
                                 ctypes.c_size_t)
        dp = ctypes.POINTER(_Dims)
        L.oasis_build_summaries.argtypes = [dp, vp, vp, vp, vp, i32, vp, vp]
        L.oasis_score_blocks.argtypes = [dp, vp, i64, i32, vp, vp, i32, vp, vp]
        L.oasis_select_topk.argtypes = [dp, vp, vp, vp, i32, i32, vp, vp, vp, vp, vp]
        L.oasis_stage_blocks.argtypes = [vp, vp, vp, i32, vp, vp]
        L.oasis_sparse_attn.argtypes = [dp, vp, i32, vp, vp, vp, i32, vp, f32, vp, vp, vp, sz, vp]
        L.oasis_sparse_attn_static_scratch.argtypes = [dp, vp, i32, vp, vp, vp, i32, vp, f32, vp, vp, vp]
        L.oasis_sparse_attn_static_scratch.restype = ctypes.c_int
        L.oasis_static_scratch_bytes.argtypes = []
        L.oasis_static_scratch_bytes.restype = sz
        L.oasis_attn_workspace_bytes.argtypes = [dp, i32, i32]
        L.oasis_attn_workspace_bytes.restype = sz
        L.oasis_plan_delta.argtypes = [dp, vp, i32, i32, vp, vp, vp, i32, i32, i32, i32, i32, i32, vp, vp, vp, vp]
        for name in ("oasis_build_summaries", "oasis_score_blocks", "oasis_select_topk",
                     "oasis_stage_blocks", "oasis_sparse_attn", "oasis_plan_delta"):
            getattr(L, name).restype = ctypes.c_int
        L.oasis_union_blocks.argtypes = [dp, vp, i32, i32, i32, vp, vp, vp]
        L.oasis_offload_blocks.argtypes = [dp, vp, vp, vp, vp, vp, vp, i32, vp, vp, vp]
        L.oasis_offload_blocks.restype = ctypes.c_int
        L.oasis_attn_and_score.argtypes = [dp, vp, i32, vp, vp, vp, i32, vp, ctypes.c_float, vp, vp, vp, ctypes.c_int64, i32, vp, vp,
                                           i32, vp, vp, ctypes.c_size_t, vp]
        L.oasis_attn_and_score.restype = ctypes.c_int
        L.oasis_build_summaries_layers.argtypes = [dp, i32, vp, vp, vp, vp, i32, vp, vp]
        L.oasis_build_summaries_layers.restype = ctypes.c_int
        L.oasis_attn_and_score_supported.argtypes = [dp, i32, i32, i32]
        L.oasis_attn_and_score_supported.restype = ctypes.c_int
        L.oasis_union_blocks.restype = ctypes.c_int
        L.oasis_stage_blocks_layers.argtypes = [i32, vp, vp, vp, i32, vp, i32, vp]
        L.oasis_stage_blocks_layers.restype = ctypes.c_int
        L.oasis_stage_blocks_bulk.argtypes = [i32, vp, vp, vp, i32, vp, i32, vp]
        L.oasis_stage_blocks_bulk.restype = ctypes.c_int
        L.oasis_local_window.argtypes = [dp, vp, i32, vp, vp, i32, i32, i32, vp, vp, vp]
        L.oasis_local_window.restype = ctypes.c_int
        L.oasis_append_kv.argtypes = [dp, vp, i32, i32, vp, vp, vp, vp, i32, i32, vp, vp, vp]
        L.oasis_append_kv.restype = ctypes.c_int
        L.oasis_append_kv_layers.argtypes = [dp, i32, vp, i32, i32, vp, vp, vp, vp, i32, i32, vp, vp, vp]
        L.oasis_append_kv_layers.restype = ctypes.c_int
        L.oasis_selftest_wait_timeout.argtypes = [ctypes.c_uint32, vp, vp]
        L.oasis_selftest_wait_timeout.restype = ctypes.c_int
        L.oasis_set_extents.argtypes = [i64, i64]
        L.oasis_set_extents.restype = ctypes.c_int
        L.oasis_bounds_checked.argtypes = []
        L.oasis_bounds_checked.restype = ctypes.c_int
        L.oasis_set_error_word.argtypes = [vp]
        L.oasis_set_error_word.restype = ctypes.c_int
        L.oasis_last_error.restype = ctypes.c_char_p
        L.oasis_version.restype = ctypes.c_char_p
        _lib = L
    return _lib


def set_error_word(word):
    """Registers an int32 device tensor (one element, zero) that kernels flag on an internal
    wait time-out; None unregisters."""
    _check(lib().oasis_set_error_word(None if word is None else ctypes.c_void_p(word.data_ptr())),
           "oasis_set_error_word")


def set_extents(n_host_entries, n_slots):
    """Declares the sizes the bounds-check build checks indices against (entries of the full-KV pool, slots of
    the working-set pool; 0 = unknown)."""
    _check(lib().oasis_set_extents(int(n_host_entries), int(n_slots)), "oasis_set_extents")


def bounds_checked() -> bool:
    """Whether the loaded library is the bounds-check build."""
    return bool(lib().oasis_bounds_checked())


def selftest_wait_timeout(probes, result=None, stream=None):
    """Runs the bounded-wait self-test: a wait of `probes` polls that nothing completes.  result: int32[2]
    device tensor receiving (gave_up, code)."""
    _check(lib().oasis_selftest_wait_timeout(int(probes), _ptr(result, torch.int32, "result"), _stream(stream)),
           "oasis_selftest_wait_timeout")


def last_error() -> str:
    return lib().oasis_last_error().decode()


def _check(rc, name):
    if rc != 0:
        raise OasisError("%s failed with status %d: %s" % (name, rc, last_error()))


def _ptr(t, dtype=None, name="tensor"):
    if t is None:
        return None
    if dtype is not None and t.dtype != dtype:
        raise TypeError("%s: expected %s, got %s" % (name, dtype, t.dtype))
    if not t.is_contiguous():
        raise ValueError("%s must be contiguous" % name)
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    if stream is None:
        stream = torch.cuda.current_stream()
    return ctypes.c_void_p(stream.cuda_stream if hasattr(stream, "cuda_stream") else int(stream))


def build_summaries(dims, kv_pool, block_table, first_block, n_blocks, max_new_blocks, summaries,
                    stream=None):
    d = dims.c()
    _check(lib().oasis_build_summaries(
        ctypes.byref(d), _ptr(kv_pool, torch.bfloat16, "kv_pool"),
        _ptr(block_table, torch.int32, "block_table"), _ptr(first_block, torch.int32, "first_block"),
        _ptr(n_blocks, torch.int32, "n_blocks"), int(max_new_blocks),
        _ptr(summaries, torch.bfloat16, "summaries"), _stream(stream)), "oasis_build_summaries")


MAX_LAYERS = 128


def build_summaries_layers(dims, kv_pools, block_tables, first_block, n_blocks, max_new_blocks, summaries,
                           stream=None):
    """oasis_build_summaries for several layers in one launch: lists of per-layer tensors."""
    n = len(kv_pools)
    if not (len(block_tables) == n and len(summaries) == n):
        raise ValueError("kv_pools, block_tables and summaries must have one tensor per layer")
    d = dims.c()
    arr = ctypes.c_void_p * max(n, 1)
    kv = arr(*[_ptr(t, torch.bfloat16, "kv_pools").value for t in kv_pools])
    bt = arr(*[_ptr(t, torch.int32, "block_tables").value for t in block_tables])
    sm = arr(*[_ptr(t, torch.bfloat16, "summaries").value for t in summaries])
    _check(lib().oasis_build_summaries_layers(
        ctypes.byref(d), n, kv, bt, _ptr(first_block, torch.int32, "first_block"),
        _ptr(n_blocks, torch.int32, "n_blocks"), int(max_new_blocks), sm, _stream(stream)),
        "oasis_build_summaries_layers")


def score_blocks(dims, q_draft, n_draft, summaries, n_full_blocks, scores, reduce_mode=REDUCE_MAX,
                 q_batch_stride=None, stream=None):
    """q_draft may be a view into the stacked queries (q[:, 1:]): only its batch stride may
    differ from the dense layout."""
    if q_draft.dtype != torch.bfloat16:
        raise TypeError("q_draft: expected bfloat16")
    if q_batch_stride is None:
        if q_draft.dim() != 4 or q_draft.stride()[1:] != (q_draft.shape[2] * q_draft.shape[3], q_draft.shape[3], 1):
            raise ValueError("q_draft must be [B][Td][Hq][128] with dense inner dimensions")
        q_batch_stride = q_draft.stride(0) if q_draft.shape[0] > 1 else q_draft[0].numel()
    d = dims.c()
    _check(lib().oasis_score_blocks(
        ctypes.byref(d), ctypes.c_void_p(q_draft.data_ptr()), int(q_batch_stride), int(n_draft),
        _ptr(summaries, torch.bfloat16, "summaries"), _ptr(n_full_blocks, torch.int32, "n_full_blocks"),
        int(reduce_mode), _ptr(scores, torch.float32, "scores"), _stream(stream)), "oasis_score_blocks")


def select_topk(dims, scores, n_full_blocks, seq_len, n_q_tokens, k, block_table, sel,
                stage_idx=None, stage_slots=None, stream=None):
    d = dims.c()
    _check(lib().oasis_select_topk(
        ctypes.byref(d), _ptr(scores, torch.float32, "scores"),
        _ptr(n_full_blocks, torch.int32, "n_full_blocks"), _ptr(seq_len, torch.int32, "seq_len"),
        int(n_q_tokens), int(k), _ptr(block_table, torch.int32, "block_table"),
        _ptr(sel, torch.int32, "sel"), _ptr(stage_idx, torch.int64, "stage_idx"),
        _ptr(stage_slots, torch.int32, "stage_slots"), _stream(stream)), "oasis_select_topk")


def stage_blocks(host_kv, idx, slots, n, hbm_pool, stream=None):
    _check(lib().oasis_stage_blocks(
        _ptr(host_kv, torch.bfloat16, "host_kv"), _ptr(idx, torch.int64, "idx"),
        _ptr(slots, torch.int32, "slots"), int(n), _ptr(hbm_pool, torch.bfloat16, "hbm_pool"),
        _stream(stream)), "oasis_stage_blocks")


def attn_workspace_bytes(dims, n_q_tokens, n_cols) -> int:
    d = dims.c()
    return int(lib().oasis_attn_workspace_bytes(ctypes.byref(d), int(n_q_tokens), int(n_cols)))


def sparse_attn(dims, q, n_q_tokens, hbm_pool, slot_tbl, blk_tbl, n_cols, seq_len, scale, out,
                lse=None, workspace=None, stream=None):
    d = dims.c()
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    _check(lib().oasis_sparse_attn(
        ctypes.byref(d), _ptr(q, torch.bfloat16, "q"), int(n_q_tokens),
        _ptr(hbm_pool, torch.bfloat16, "hbm_pool"), _ptr(slot_tbl, torch.int32, "slot_tbl"),
        _ptr(blk_tbl, torch.int32, "blk_tbl"), int(n_cols), _ptr(seq_len, torch.int32, "seq_len"),
        float(scale), _ptr(out, torch.bfloat16, "out"), _ptr(lse, torch.float32, "lse"),
        _ptr(workspace, None, "workspace"), ws_bytes, _stream(stream)), "oasis_sparse_attn")


def union_blocks(dims, sel, k, union_idx, n_union, stream=None):
    """union_idx [B][max_union] int32, n_union [B] int32: distinct selected blocks over all KV heads."""
    d = dims.c()
    _check(lib().oasis_union_blocks(
        ctypes.byref(d), _ptr(sel, torch.int32, "sel"), int(sel.shape[-1]), int(k), int(union_idx.shape[-1]),
        _ptr(union_idx, torch.int32, "union_idx"), _ptr(n_union, torch.int32, "n_union"), _stream(stream)),
        "oasis_union_blocks")


def offload_blocks(dims, dense_k, dense_v, gpu_table, block_table, first_block, n_blocks, max_new_blocks,
                   host_kv, summaries=None, stream=None):
    """Dense -> sparse hand-over: dense_k / dense_v [P_gpu][Hkv][16][128] -> entries of host_kv (and the
    copied blocks' summaries when given)."""
    d = dims.c()
    _check(lib().oasis_offload_blocks(
        ctypes.byref(d), _ptr(dense_k, torch.bfloat16, "dense_k"), _ptr(dense_v, torch.bfloat16, "dense_v"),
        _ptr(gpu_table, torch.int32, "gpu_table"), _ptr(block_table, torch.int32, "block_table"),
        _ptr(first_block, torch.int32, "first_block"), _ptr(n_blocks, torch.int32, "n_blocks"), int(max_new_blocks),
        _ptr(host_kv, torch.bfloat16, "host_kv"), _ptr(summaries, torch.bfloat16, "summaries"), _stream(stream)),
        "oasis_offload_blocks")


def attn_and_score(dims, q, n_q_tokens, hbm_pool, slot_tbl, blk_tbl, n_cols, seq_len, scale, out, q_draft, n_draft,
                   summaries, n_full_blocks, scores, lse=None, reduce_mode=REDUCE_MAX, q_batch_stride=None, workspace=None,
                   stream=None):
    """Steps 4 and 1 of one layer in one launch; raises OasisError (status 2) for shapes outside the fused
    launch, which take sparse_attn + score_blocks instead.  `workspace`: attn_workspace_bytes() bytes where
    that is not zero (few rows: the column lists are split)."""
    d = dims.c()
    ws_bytes = 0 if workspace is None else workspace.numel() * workspace.element_size()
    if q_batch_stride is None:
        q_batch_stride = n_draft * dims.n_q_heads * 128
    _check(lib().oasis_attn_and_score(
        ctypes.byref(d), _ptr(q, torch.bfloat16, "q"), int(n_q_tokens), _ptr(hbm_pool, torch.bfloat16, "hbm_pool"),
        _ptr(slot_tbl, torch.int32, "slot_tbl"), _ptr(blk_tbl, torch.int32, "blk_tbl"), int(n_cols),
        _ptr(seq_len, torch.int32, "seq_len"), ctypes.c_float(scale), _ptr(out, torch.bfloat16, "out"),
        _ptr(lse, torch.float32, "lse"), ctypes.c_void_p(q_draft.data_ptr()), ctypes.c_int64(int(q_batch_stride)),
        int(n_draft), _ptr(summaries, torch.bfloat16, "summaries"), _ptr(n_full_blocks, torch.int32, "n_full_blocks"),
        int(reduce_mode), _ptr(scores, torch.float32, "scores"), _ptr(workspace, None, "workspace"), ws_bytes,
        _stream(stream)), "oasis_attn_and_score")


def attn_and_score_supported(dims, n_q_tokens, n_cols, n_draft) -> bool:
    """Whether oasis_attn_and_score takes these shapes on the current device."""
    d = dims.c()
    return bool(lib().oasis_attn_and_score_supported(ctypes.byref(d), int(n_q_tokens), int(n_cols), int(n_draft)))


def static_scratch_bytes() -> int:
    return int(lib().oasis_static_scratch_bytes())


def sparse_attn_static_scratch(dims, q, n_q_tokens, hbm_pool, slot_tbl, blk_tbl, n_cols, seq_len, scale,
                               out, lse=None, stream=None):
    """oasis_sparse_attn for callers that cannot hand over scratch memory (no free device memory
    left to allocate from, or no cudaMalloc allowed in the decode loop): the partial results go
    to a 4 MiB array built into the library.  Calls sharing a GPU must not overlap."""
    d = dims.c()
    _check(lib().oasis_sparse_attn_static_scratch(
        ctypes.byref(d), _ptr(q, torch.bfloat16, "q"), int(n_q_tokens),
        _ptr(hbm_pool, torch.bfloat16, "hbm_pool"), _ptr(slot_tbl, torch.int32, "slot_tbl"),
        _ptr(blk_tbl, torch.int32, "blk_tbl"), int(n_cols), _ptr(seq_len, torch.int32, "seq_len"),
        float(scale), _ptr(out, torch.bfloat16, "out"), _ptr(lse, torch.float32, "lse"),
        _stream(stream)), "oasis_sparse_attn_static_scratch")


def plan_delta(dims, sel, k, block_table, resident, stamp, slot_stride, cap, step, plan_idx,
               plan_slots, n_admitted=None, n_local=0, n_res=None, stream=None):
    """resident / stamp are [B][Hkv][res_stride] with the n_res eviction-managed columns first (default:
    all but the last n_local); plan lists [B][Hkv][cap + n_local]."""
    d = dims.c()
    res_stride = int(resident.shape[-1])
    n_res = res_stride - int(n_local) if n_res is None else int(n_res)
    _check(lib().oasis_plan_delta(
        ctypes.byref(d), _ptr(sel, torch.int32, "sel"), int(sel.shape[-1]), int(k),
        _ptr(block_table, torch.int32, "block_table"), _ptr(resident, torch.int32, "resident"),
        _ptr(stamp, torch.int32, "stamp"), n_res, res_stride, int(n_local),
        int(slot_stride), int(cap), int(step), _ptr(plan_idx, torch.int64, "plan_idx"),
        _ptr(plan_slots, torch.int32, "plan_slots"), _ptr(n_admitted, torch.int32, "n_admitted"),
        _stream(stream)), "oasis_plan_delta")


MAX_APPEND_LAYERS = 64


def local_window(dims, seq_len, n_q_tokens, block_table, blk_tbl, local_col, slot_stride=0, stage_idx=None,
                 stage_slots=None, stream=None):
    """Sets the two local columns of blk_tbl [B][Hkv][n_cols] (block parity picks the column) and, when the
    lists [B][Hkv][2] are given, emits the gather requests that load the local blocks from the CPU pool."""
    d = dims.c()
    _check(lib().oasis_local_window(
        ctypes.byref(d), _ptr(seq_len, torch.int32, "seq_len"), int(n_q_tokens),
        _ptr(block_table, torch.int32, "block_table"), _ptr(blk_tbl, torch.int32, "blk_tbl"), int(blk_tbl.shape[-1]),
        int(local_col), int(slot_stride), _ptr(stage_idx, torch.int64, "stage_idx"),
        _ptr(stage_slots, torch.int32, "stage_slots"), _stream(stream)), "oasis_local_window")


def append_kv(dims, new_kv, n_commit, seq_len, block_table, slot_tbl, blk_tbl, local_col, hbm_pool, host_kv=None,
              stream=None):
    """KV append of one step: new_kv [B][T][Hkv][2][128] into the local window of hbm_pool, its first n_commit
    tokens also into the CPU pool host_kv."""
    d = dims.c()
    _check(lib().oasis_append_kv(
        ctypes.byref(d), _ptr(new_kv, torch.bfloat16, "new_kv"), int(new_kv.shape[1]), int(n_commit),
        _ptr(seq_len, torch.int32, "seq_len"), _ptr(block_table, torch.int32, "block_table"),
        _ptr(slot_tbl, torch.int32, "slot_tbl"), _ptr(blk_tbl, torch.int32, "blk_tbl"), int(blk_tbl.shape[-1]),
        int(local_col), _ptr(hbm_pool, torch.bfloat16, "hbm_pool"), _ptr(host_kv, torch.bfloat16, "host_kv"),
        _stream(stream)), "oasis_append_kv")


def append_kv_layers(dims, new_kv, n_commit, seq_len, block_tables, slot_tbls, blk_tbls, local_col, hbm_pools,
                     host_kvs, stream=None):
    """oasis_append_kv for several layers in one launch: lists of per-layer tensors."""
    n = len(new_kv)
    if not all(len(x) == n for x in (block_tables, slot_tbls, blk_tbls, hbm_pools, host_kvs)):
        raise ValueError("one tensor per layer is needed in every list")
    d = dims.c()
    arr = ctypes.c_void_p * max(n, 1)
    mk = lambda ts, dt, nm: arr(*[None if t is None else _ptr(t, dt, nm).value for t in ts])
    _check(lib().oasis_append_kv_layers(
        ctypes.byref(d), n, mk(new_kv, torch.bfloat16, "new_kv"), int(new_kv[0].shape[1]) if n else 1, int(n_commit),
        _ptr(seq_len, torch.int32, "seq_len"), mk(block_tables, torch.int32, "block_tables"),
        mk(slot_tbls, torch.int32, "slot_tbls"), mk(blk_tbls, torch.int32, "blk_tbls"),
        int(blk_tbls[0].shape[-1]) if n else 2, int(local_col), mk(hbm_pools, torch.bfloat16, "hbm_pools"),
        mk(host_kvs, torch.bfloat16, "host_kvs"), _stream(stream)), "oasis_append_kv_layers")


MAX_STAGE_LAYERS = 64


def stage_blocks_layers(host_kvs, idx, slots, n, hbm_pools, max_ctas=0, stream=None):
    """oasis_stage_blocks for several layers in one launch: lists of per-layer tensors, every list of length n."""
    nl = len(host_kvs)
    if not all(len(x) == nl for x in (idx, slots, hbm_pools)):
        raise ValueError("one tensor per layer is needed in every list")
    arr = ctypes.c_void_p * max(nl, 1)
    mk = lambda ts, dt, nm: arr(*[_ptr(t, dt, nm).value for t in ts])
    _check(lib().oasis_stage_blocks_layers(
        nl, mk(host_kvs, torch.bfloat16, "host_kvs"), mk(idx, torch.int64, "idx"), mk(slots, torch.int32, "slots"), int(n),
        mk(hbm_pools, torch.bfloat16, "hbm_pools"), int(max_ctas), _stream(stream)), "oasis_stage_blocks_layers")


def stage_blocks_bulk(host_kvs, idx, slots, n, hbm_pools, max_streams=0, stream=None):
    """oasis_stage_blocks_bulk: the several-layers gather through the copy unit (same arguments and result as
    stage_blocks_layers; `max_streams` entry streams, 0 = the library's default)."""
    nl = len(host_kvs)
    if not all(len(x) == nl for x in (idx, slots, hbm_pools)):
        raise ValueError("one tensor per layer is needed in every list")
    arr = ctypes.c_void_p * max(nl, 1)
    mk = lambda ts, dt, nm: arr(*[_ptr(t, dt, nm).value for t in ts])
    _check(lib().oasis_stage_blocks_bulk(
        nl, mk(host_kvs, torch.bfloat16, "host_kvs"), mk(idx, torch.int64, "idx"), mk(slots, torch.int32, "slots"), int(n),
        mk(hbm_pools, torch.bfloat16, "hbm_pools"), int(max_streams), _stream(stream)), "oasis_stage_blocks_bulk")
