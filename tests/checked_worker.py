"""Worker of test_gpu_checked_build.py: runs in a process of its own with OASIS_LIB pointing at the bounds-check
build (liboasis_checked.so).  (1) Tiny configurations -- 3 to 7 blocks, K 1 to 3 -- through the whole path against
the oracle, with the real extents declared: the error word must stay zero.  (2) Every kind of index, once, between
a DECLARED extent and the (larger) size really allocated: the kernel must flag the right code, skip the access
(canaries intact) and do the rest of its work.  Nothing here can leave an allocation even if a check were wrong."""
import json
import math
import os
import sys

import numpy as np
import torch

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
sys.path.insert(0, ROOT)

from paper_2608_08097_b200 import binding, pipeline, synth  # noqa: E402
from oracle import oracle  # noqa: E402
from tests import parity_util as pu  # noqa: E402

HOST_ENTRY, SLOT, BLOCK_ID, BLOCK_COUNT = 201, 202, 203, 204
dev = torch.device("cuda")
word = torch.zeros(1, dtype=torch.int32, device=dev)


def take_code():
    torch.cuda.synchronize()
    c = int(word.item())
    word.zero_()
    return c


def tiny_parity():
    n = 0
    for batch, context, k, td in ((2, 56, 1, 1), (1, 48, 2, 2), (3, 112, 3, 1), (2, 37, 3, 4)):
        cfg = synth.scaled(synth.C1, batch=batch, context=context, k_blocks=k, n_draft=td)
        lay = synth.make_layer(cfg, seed=60 + n, ragged=True, permute_table=True)
        T = cfg.n_q_tokens
        L = pipeline.DecodeLayer(batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.max_blocks, k, T, dev, want_lse=True)
        binding.set_extents(lay.host_kv.shape[0] * cfg.n_kv_heads, L.pool.shape[0])
        kv = lay.host_kv.pin_memory()
        table, n_full, seq, q = (t.to(dev) for t in (lay.block_table, lay.n_full, lay.seq_len, lay.q))
        L.build_summaries(kv, table, torch.zeros_like(n_full), n_full, cfg.max_blocks)
        L.score(q, n_full)
        L.select(n_full, seq, table)
        L.stage(kv)
        L.attend(q, seq)
        torch.cuda.synchronize()
        ref = pu.oracle_layer(oracle, lay, k)
        pu.assert_summaries_equal(pu.np_u16(L.summaries), ref["summ"], ref["n_full"])
        pu.assert_scores_close(L.scores.cpu().numpy(), ref["s32"], ref["s64"], ref["n_full"])
        assert pu.assert_sel_parity(L.sel.cpu().numpy(), ref["sel"], ref["s64"], k) == 0
        assert np.array_equal(pu.np_u16(L.pool), ref["pool"])
        pu.assert_attn_close(pu.bf16_to_f32_np(L.out), ref["attn"])
        if binding.attn_and_score_supported(L.dims, T, L.cols, T - 1):
            L.out.zero_()
            L.attend_and_score(q, seq, n_full)
            torch.cuda.synchronize()
            pu.assert_attn_close(pu.bf16_to_f32_np(L.out), ref["attn"])
            pu.assert_scores_close(L.scores.cpu().numpy(), ref["s32"], ref["s64"], ref["n_full"])
        assert take_code() == 0, "a check fired on valid indices"
        n += 1
    return n


def flag_each_kind():
    seen = {}
    Hkv = 8
    canary = 0x1234
    bf = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
    rng = np.random.default_rng(3)
    # --- gather: 16 entries / 16 slots really allocated, 8 / 8 declared
    host = bf(rng.integers(0, 0x7f00, (16, 2, 16, 128)).astype(np.uint16)).pin_memory()
    pool = torch.full((16, 2, 16, 128), 0, dtype=torch.bfloat16, device=dev)
    pool.view(torch.int16).fill_(canary)
    binding.set_extents(8, 8)
    idx = torch.tensor([3, 12, 5, -1], dtype=torch.int64, device=dev)        # 12: beyond the declared 8 entries
    slots = torch.tensor([0, 1, 2, 3], dtype=torch.int32, device=dev)
    binding.stage_blocks(host, idx, slots, 4, pool)
    seen["gather source entry"] = take_code()
    p16 = pool.view(torch.int16).cpu()
    assert torch.equal(p16[0], host.view(torch.int16)[3]) and torch.equal(p16[2], host.view(torch.int16)[5])
    assert (p16[1] == canary).all() and (p16[3:] == canary).all()
    idx = torch.tensor([1, 2], dtype=torch.int64, device=dev)
    slots = torch.tensor([11, 4], dtype=torch.int32, device=dev)              # 11: beyond the declared 8 slots
    binding.stage_blocks_layers([host], [idx], [slots], 2, [pool])
    seen["gather slot"] = take_code()
    p16 = pool.view(torch.int16).cpu()
    assert (p16[11] == canary).all() and torch.equal(p16[4], host.view(torch.int16)[2])

    # --- summaries: a block table entry beyond the declared pool
    dims = binding.Dims(1, 32, Hkv, 8)
    kv = bf(rng.integers(0, 0x7f00, (4, Hkv, 2, 16, 128)).astype(np.uint16)).to(dev)      # 32 entries allocated
    binding.set_extents(2 * Hkv, 64)                                                       # 16 declared
    table = torch.tensor([[0, 1, 3, 0, 0, 0, 0, 0]], dtype=torch.int32, device=dev)       # block 3: entries 24..31
    summ = torch.zeros((1, Hkv, 8, 2, 128), dtype=torch.bfloat16, device=dev)
    summ.view(torch.int16).fill_(canary)
    binding.build_summaries(dims, kv, table, torch.zeros(1, dtype=torch.int32, device=dev),
                            torch.tensor([3], dtype=torch.int32, device=dev), 3, summ)
    seen["summary source entry"] = take_code()
    s16 = summ.view(torch.int16).cpu()
    assert (s16[0, :, 2] == canary).all() and not (s16[0, :, 1] == canary).all()

    # --- top-k: a block count beyond max_blocks is clamped and reported; a plan with a block id beyond max_blocks
    binding.set_extents(1 << 20, 1 << 20)
    scores = torch.randn((1, Hkv, 8), device=dev)
    sel = torch.empty((1, Hkv, 5), dtype=torch.int32, device=dev)
    n_big = torch.tensor([11], dtype=torch.int32, device=dev)
    seq = torch.tensor([8 * 16], dtype=torch.int32, device=dev)
    binding.select_topk(dims, scores, n_big, seq, 2, 3, table, sel)
    seen["block count"] = take_code()
    s = sel.cpu().numpy()
    assert ((s[..., :3] >= 0) & (s[..., :3] < 8)).all()
    sel_bad = sel.clone()
    sel_bad[..., 0] = 9                                                  # >= max_blocks = 8
    sel_bad[..., 3:] = -1
    resident = torch.full((1, Hkv, 3), -1, dtype=torch.int32, device=dev)
    stamp = torch.zeros((1, Hkv, 3), dtype=torch.int32, device=dev)
    plan_idx = torch.empty((1, Hkv, 3), dtype=torch.int64, device=dev)
    plan_slots = torch.empty((1, Hkv, 3), dtype=torch.int32, device=dev)
    binding.plan_delta(dims, sel_bad, 3, table, resident, stamp, 3, 3, 1, plan_idx, plan_slots)
    seen["block id"] = take_code()
    assert (resident.cpu().numpy() != 9).all()

    # --- attention: a slot beyond the declared pool is treated as a missing column
    cfg = synth.scaled(synth.C1, batch=1, context=64, k_blocks=3, n_draft=1)
    lay = synth.make_layer(cfg, seed=77)
    T, k = cfg.n_q_tokens, 3
    L = pipeline.DecodeLayer(1, cfg.n_q_heads, Hkv, cfg.max_blocks, k, T, dev)
    big_pool = torch.zeros((2 * L.pool.shape[0], 2, 16, 128), dtype=torch.bfloat16, device=dev)   # twice the declared slots
    n_decl = L.pool.shape[0]
    binding.set_extents(lay.host_kv.shape[0] * Hkv, n_decl)
    kvp = lay.host_kv.pin_memory()
    table, n_full, seq, q = (t.to(dev) for t in (lay.block_table, lay.n_full, lay.seq_len, lay.q))
    L.build_summaries(kvp, table, torch.zeros_like(n_full), n_full, cfg.max_blocks)
    L.score(q, n_full)
    L.select(n_full, seq, table)
    L.stage(kvp)
    assert take_code() == 0
    big_pool[:n_decl].copy_(L.pool)
    slot_bad = L.slot_tbl.clone()
    slot_bad[0, 2, 1] = n_decl + 5                                       # inside big_pool, outside the declared extent
    binding.sparse_attn(L.dims, q, T, big_pool, slot_bad, L.sel, L.cols, seq, L.scale, L.out, workspace=L.workspace)
    seen["attention slot"] = take_code()
    sel_ref = L.sel.cpu().numpy().copy()
    sel_ref[0, 2, 1] = -1                                                # what the kernel must have computed
    ref = oracle.sparse_attn(pu.np_u16(lay.q), pu.np_u16(L.pool), L.slot_tbl.cpu().numpy(), sel_ref, lay.seq_len.numpy(),
                             np.float32(1.0 / math.sqrt(128.0)), Hkv)
    pu.assert_attn_close(pu.bf16_to_f32_np(L.out), ref)

    # --- KV append: local slot beyond the declared pool, committed token into an entry beyond the declared CPU pool
    new_kv = bf(rng.integers(0, 0x7f00, (1, T, Hkv, 2, 128)).astype(np.uint16)).to(dev)
    blk = torch.full((1, Hkv, L.cols), -1, dtype=torch.int32, device=dev)
    big_pool.view(torch.int16).fill_(canary)
    binding.append_kv(L.dims, new_kv, 0, seq, table, slot_bad * 0 + (n_decl + 3), blk, k, big_pool, None)
    seen["append slot"] = take_code()
    assert (big_pool.view(torch.int16).cpu() == canary).all()
    host2 = torch.zeros((2 * lay.host_kv.shape[0], Hkv, 2, 16, 128), dtype=torch.bfloat16).pin_memory()
    host2.view(torch.int16).fill_(canary)
    table_bad = table + lay.host_kv.shape[0]                             # every block beyond the declared entries
    binding.append_kv(L.dims, new_kv, 1, seq, table_bad, L.slot_tbl, blk, k, big_pool, host2)
    seen["append host entry"] = take_code()
    assert (host2.view(torch.int16) == canary).all()
    return seen


def main():
    assert binding.bounds_checked(), "this worker must run on the bounds-check build (OASIS_LIB)"
    oracle.lib()
    binding.set_error_word(word)
    n = tiny_parity()
    seen = flag_each_kind()
    want = {"gather source entry": HOST_ENTRY, "gather slot": SLOT, "summary source entry": HOST_ENTRY,
            "block count": BLOCK_COUNT, "block id": BLOCK_ID, "attention slot": SLOT, "append slot": SLOT,
            "append host entry": HOST_ENTRY}
    assert seen == want, (seen, want)
    # and a normal call still works afterwards
    binding.set_extents(0, 0)
    assert tiny_parity() > 0
    binding.set_error_word(None)
    print(json.dumps({"ok": True, "tiny_configs": n, "flagged": seen}))


if __name__ == "__main__":
    main()
