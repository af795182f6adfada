"""The decode engine against the oracle, step by step: shared by the small engine tests and the full-size ones.

Every step's attention output must equal the oracle's attention over the working set that the previous step's
prediction staged; every step's selection must equal the oracle's (near-ties adjudicated, after which the
oracle-side simulation follows the GPU's selection); tables, working-set pool and -- with the KV append -- the CPU
pool must be identical at every synchronisation point."""
import math

import numpy as np
import torch

from paper_2608_08097_b200 import synth
from tests import parity_util as pu

SCALE = np.float32(1.0 / math.sqrt(128.0))


def check_engine(oracle, pipeline, cfg, lays, mode, cap, append, chunk, graph, e2e, fused, wait_group=2, transfer_group=1,
                 max_adjudicated=16, light=False):
    """cfg.layers layers (`lays`: one synth.Layer each, host_kv on the CPU), cfg.steps steps; `chunk` steps run between
    synchronisations -- one CUDA graph of `chunk` steps when `graph`, else eager steps launched back to back.
    light (full-size pools): the layers' pools are used in place and the CPU pool is compared on the blocks the steps
    can have touched instead of as a whole."""
    dev = torch.device("cuda")
    n_layers, S = cfg.layers, cfg.steps
    k, B, Hkv, T = cfg.k_blocks, cfg.batch, cfg.n_kv_heads, cfg.n_q_tokens
    eng = pipeline.DecodeEngine(B, cfg.n_q_heads, Hkv, cfg.max_blocks, k, T, n_layers, dev,
                                mode=mode, cap=cap, append=append, fused=fused, transfer_streams=2, wait_group=wait_group,
                                transfer_group=transfer_group)
    new_kv = [synth.new_kv_steps(lay) for lay in lays] if append else None     # [S][B][T][Hkv][2][128] per layer
    # with the KV append the pools start without the tokens that the steps will produce
    if light:
        kvs = [synth.blank_future(lay.host_kv, lay) if append else lay.host_kv for lay in lays]
        kvs = [kv if kv.is_pinned() else kv.pin_memory() for kv in kvs]
    else:
        kvs = [(synth.blank_future(lay.host_kv.clone(), lay) if append else lay.host_kv).pin_memory() for lay in lays]
    kv_ref = [pu.np_u16(kv).copy() for kv in kvs]                              # oracle-side copy of the CPU pool
    for l, lay in enumerate(lays):
        eng.attach(l, kvs[l], lay.block_table.to(dev))
    seq = lays[0].seq_len_steps                                   # [S][B]
    q_dev = [lay.q_steps.to(dev) for lay in lays]
    new_dev = [t.to(dev) for t in new_kv] if append else None
    to_dev = lambda t: t.to(torch.int32).contiguous().to(dev)
    # end-to-end mode: the step uploads its queries from pinned memory and downloads its outputs (one pinned output
    # buffer per step and layer, so every step's result can be read after a chunk)
    stacked = e2e and chunk in (4, 19)           # one tensor over the layers: grouped uploads / downloads
    q_pin = [lay.q_steps.pin_memory() for lay in lays] if e2e else None
    q_stage = [torch.empty_like(q_dev[l][0]) for l in range(n_layers)] if e2e else None
    out_pin = [[torch.zeros((B, T, cfg.n_q_heads, 128), dtype=torch.bfloat16).pin_memory() for _ in range(n_layers)]
               for _ in range(S)] if e2e else None
    if stacked:
        q_pin_all = torch.stack([lay.q_steps for lay in lays], dim=1).pin_memory()       # [S][n_layers][B][T][Hq][128]
        q_stage = torch.empty_like(q_pin_all[0], device=dev)
        out_pin = [torch.zeros((n_layers, B, T, cfg.n_q_heads, 128), dtype=torch.bfloat16).pin_memory() for _ in range(S)]
    eng.prime([q_dev[l][0] for l in range(n_layers)], to_dev(seq[0] // 16), to_dev(seq[0]))

    # oracle-side state
    pools = [np.zeros((B * Hkv * (k + 2), 2, 16, 128), np.uint16) for _ in range(n_layers)]
    slot_tbl = np.arange(B * Hkv * (k + 2), dtype=np.int32).reshape(B, Hkv, k + 2)
    res = [np.full((B, Hkv, k + 2), -1, np.int32) for _ in range(n_layers)]
    stp = [np.zeros((B, Hkv, k + 2), np.int32) for _ in range(n_layers)]
    blk = [None] * n_layers
    tables = [lay.block_table.numpy() for lay in lays]

    summ_cache = [None] * n_layers                # full build once, then only the blocks completed since the first step
    n_full0 = (seq[0] // 16).numpy().astype(np.int32)

    def oracle_prediction_on(l, q_step, n_full, sq):
        if summ_cache[l] is None:
            summ_cache[l] = oracle.build_summaries(kv_ref[l], tables[l], np.zeros(B, np.int32), n_full0)
        summ = oracle.build_summaries(kv_ref[l], tables[l], n_full0, (n_full - n_full0).astype(np.int32), summ_cache[l])
        q = pu.np_u16(lays[l].q_steps[q_step])
        s32, s64 = oracle.score_blocks(q[:, 1:], summ, n_full)
        sel, idx, slots = oracle.select_topk(s32, n_full, sq, T, k, tables[l])
        return sel, idx, slots, s64

    def oracle_transfer(l, sel, cap_now, stamp):
        kv = kv_ref[l].reshape(-1, 2, 16, 128)
        if mode == "delta":
            pidx, pslots, _ = oracle.plan_delta(sel, tables[l], res[l], stp[l], k, cap_now, stamp,
                                                k + 2, n_res=k, n_local=0 if append else 2)
            oracle.stage_blocks(kv, pidx, pslots, pools[l])
            blk[l] = res[l]
        else:
            idx = np.where(sel < 0, -1, np.take_along_axis(
                np.broadcast_to(tables[l][:, None, :], (B, Hkv, tables[l].shape[1])), np.maximum(sel, 0), axis=2)
                .astype(np.int64) * Hkv + np.arange(Hkv)[None, :, None])
            oracle.stage_blocks(kv, idx, slot_tbl, pools[l])
            blk[l] = sel.copy()

    for l in range(n_layers):
        sel, idx, slots, s64 = oracle_prediction_on(l, 0, (seq[0] // 16).numpy(), seq[0].numpy())
        gsel = eng.layers[l].sel.cpu().numpy()      # the oracle follows the GPU's selection wherever the two differ
        pu.assert_sel_parity(gsel, sel, s64, k)     # by a near-tie (scores within 1e-5 relative); anything else fails
        oracle_transfer(l, gsel, k, 0)
        if append:
            lidx, lslots = oracle.local_window(seq[0].numpy(), T, tables[l], res[l], k, k + 2)
            oracle.stage_blocks(kv_ref[l].reshape(-1, 2, 16, 128), lidx, lslots, pools[l])

    keep = []                                        # tensors and graphs captured so far stay alive
    sel_log = [[torch.empty_like(eng.layers[l].sel) for l in range(n_layers)] for _ in range(S)]
    n_adjudicated = 0
    want_out = {}                                    # (step, layer) -> oracle attention
    got_out = {}
    for s0 in range(0, S, chunk):
        steps = list(range(s0, min(s0 + chunk, S)))
        calls = []
        for s in steps:
            args = (q_stage if e2e else [q_dev[l][s] for l in range(n_layers)], to_dev(seq[s]), to_dev(seq[s] // 16),
                    to_dev((seq[s] + 1) // 16 - seq[s] // 16), to_dev((seq[s] + 1) // 16), to_dev(seq[s] + 1))
            kw = dict(step_stamp=s + 1, sel_log=sel_log[s])
            if e2e:
                kw.update(q_host=q_pin_all[s] if stacked else [q_pin[l][s] for l in range(n_layers)], out_host=out_pin[s])
            if append:
                kw.update(new_kv=[new_dev[l][s] for l in range(n_layers)])
            calls.append((args, kw))
        keep.append(calls)
        if graph:
            g = eng.capture_steps(calls)
            keep.append(g)
            eng.upload(g)                            # as the benchmark does ahead of its timed region
            eng.replay(g)
        else:
            for s, (args, kw) in zip(steps, calls):
                eng.step(*args, **kw)                # no join, no synchronisation between the steps of a chunk
                if not e2e:
                    with torch.cuda.stream(eng.main):
                        for l in range(n_layers):
                            got_out[(s, l)] = eng.layers[l].out.clone()
            eng.join()
        torch.cuda.synchronize()
        for s in steps:
            for l in range(n_layers):
                if e2e:
                    got_out[(s, l)] = out_pin[s][l]
                elif graph:
                    assert chunk == 1
                    got_out[(s, l)] = eng.layers[l].out.clone()
        # the oracle takes the same steps
        for s in steps:
            for l in range(n_layers):
                if append:
                    oracle.append_kv(pu.np_u16(new_kv[l][s]), 1, seq[s].numpy(), tables[l], slot_tbl, res[l], k, pools[l],
                                     kv_ref[l])
                # attention of this step ran over the working set predicted one step earlier
                ref = oracle.sparse_attn(pu.np_u16(lays[l].q_steps[s]), pools[l], slot_tbl, blk[l], seq[s].numpy(), SCALE, Hkv)
                pu.assert_attn_close(pu.bf16_to_f32_np(got_out[(s, l)]), ref)
                # this step's prediction and transfer, for the next step
                sel, idx, slots, s64 = oracle_prediction_on(l, s, ((seq[s] + 1) // 16).numpy(), (seq[s] + 1).numpy())
                gsel = sel_log[s][l].cpu().numpy()
                n_adjudicated += pu.assert_sel_parity(gsel, sel, s64, k)
                oracle_transfer(l, gsel, cap if cap is not None else k, s + 1)
                if s == steps[-1]:
                    # state at the synchronisation point
                    assert np.array_equal(eng.layers[l].sel.cpu().numpy(), gsel)
                    assert np.array_equal(eng.blk_tbl(l).cpu().numpy(), blk[l])
                    assert np.array_equal(pu.np_u16(eng.layers[l].pool), pools[l])
                    if e2e:
                        assert torch.equal(q_stage[l].cpu(), lays[l].q_steps[s])
                    if append and not light:
                        assert np.array_equal(pu.np_u16(kvs[l]), kv_ref[l])
                    elif append:
                        for b in range(B):                   # the blocks the steps so far can have written
                            j0, j1 = int(seq[0][b]) // 16, (int(seq[s][b]) + T) // 16 + 1
                            phys = tables[l][b, j0:j1]
                            assert np.array_equal(pu.np_u16(kvs[l][torch.from_numpy(phys.astype(np.int64))]), kv_ref[l][phys])
    assert n_adjudicated <= max_adjudicated, "too many near-ties for rounding order alone: %d" % n_adjudicated
    if append and not light:      # the write-through rebuilt, in the CPU pool, every committed position of the generator's pool
        for l, lay in enumerate(lays):
            for b in range(B):
                for p in range(int(seq[0][b]), int(seq[S - 1][b]) + 1):
                    assert torch.equal(kvs[l][lay.block_table[b][p // 16], :, :, p % 16], lay.host_kv[lay.block_table[b][p // 16], :, :, p % 16])
