"""GPU parity tests: the CUDA library (through its C ABI) against the CPU oracle, element by
element, on the same seeded inputs.  Index work must be bit-exact (fp32 near-ties adjudicated
with the oracle's double-precision scores); attention within atol 2e-3 / rtol 1e-2."""
import math

import numpy as np
import pytest
import torch

from paper_2608_08097_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module")
def gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_08097_b200 import build
    build.build()
    from paper_2608_08097_b200 import binding, pipeline
    binding.lib()
    return binding, pipeline


def run_gpu_path(pipeline, lay, k, step=0, reduce_mode=0, kv_on="pinned", want_lse=True):
    """All five calls on the GPU for one layer / step.  kv_on: where the full-KV pool lives."""
    cfg = lay.cfg
    dev = torch.device("cuda")
    L = pipeline.DecodeLayer(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.max_blocks, k, cfg.n_q_tokens,
                             device=dev, want_lse=want_lse)
    if kv_on == "pinned":
        kv = lay.host_kv if lay.host_kv.is_pinned() else lay.host_kv.pin_memory()
    else:
        kv = lay.host_kv.to(dev)
    table = lay.block_table.to(dev)
    n_full = lay.n_full_steps[step].to(dev)
    seq_len = lay.seq_len_steps[step].to(dev)
    q = lay.q_steps[step].to(dev)
    zeros = torch.zeros(cfg.batch, dtype=torch.int32, device=dev)
    L.build_summaries(kv, table, zeros, n_full, cfg.max_blocks)
    L.score(q, n_full, reduce_mode=reduce_mode)
    L.select(n_full, seq_len, table)
    L.stage(kv)
    L.attend(q, seq_len)
    torch.cuda.synchronize()
    return L, dict(kv=kv, table=table, n_full=n_full, seq_len=seq_len, q=q)


def compare_path(oracle, pipeline, lay, k, step=0, reduce_mode=0, kv_on="pinned"):
    L, dv = run_gpu_path(pipeline, lay, k, step, reduce_mode, kv_on)
    ref = pu.oracle_layer(oracle, lay, k, reduce_mode, step)
    cfg = lay.cfg
    pu.assert_summaries_equal(pu.np_u16(L.summaries), ref["summ"], ref["n_full"])
    gs = L.scores.cpu().numpy()
    pu.assert_scores_close(gs, ref["s32"], ref["s64"], ref["n_full"])
    gsel = L.sel.cpu().numpy()
    n_adj = pu.assert_sel_parity(gsel, ref["sel"], ref["s64"], k)
    # gather lists follow the GPU's own selection exactly
    table = lay.block_table.numpy()
    gidx, gslots = L.stage_idx.cpu().numpy(), L.stage_slots.cpu().numpy()
    want_idx = np.where(gsel < 0, -1, np.take_along_axis(
        np.broadcast_to(table[:, None, :], gsel.shape[:2] + (table.shape[1],)), np.maximum(gsel, 0), axis=2)
        .astype(np.int64) * cfg.n_kv_heads + np.arange(cfg.n_kv_heads)[None, :, None])
    assert np.array_equal(gidx, want_idx)
    assert np.array_equal(gslots.reshape(-1), np.arange(gslots.size))
    # staged pool: bit-exact copy of the requested entries
    want_pool = np.zeros_like(ref["pool"])
    oracle.stage_blocks(pu.np_u16(lay.host_kv).reshape(-1, 2, 16, 128), gidx, gslots, want_pool)
    assert np.array_equal(pu.np_u16(L.pool), want_pool)
    # attention on the GPU's own selection vs the oracle on that same selection
    slot_tbl = np.arange(gsel.size, dtype=np.int32).reshape(gsel.shape)
    ref_attn = oracle.sparse_attn(ref["q"], want_pool, slot_tbl, gsel, ref["seq_len"],
                                  np.float32(1.0 / math.sqrt(128.0)), cfg.n_kv_heads)
    pu.assert_attn_close(pu.bf16_to_f32_np(L.out), ref_attn)
    np.testing.assert_allclose(L.lse.cpu().numpy(), ref_attn["lse"], rtol=1e-3, atol=2e-3)
    # and attention on the ORACLE's selection and pool (independent of the GPU's choices)
    if n_adj:
        dev = torch.device("cuda")
        L.pool.copy_(torch.from_numpy(ref["pool"].view(np.int16)).view(torch.bfloat16).to(dev))
        L.attend(dv["q"], dv["seq_len"], blk_tbl=torch.from_numpy(ref["sel"]).to(dev))
        torch.cuda.synchronize()
        pu.assert_attn_close(pu.bf16_to_f32_np(L.out), ref["attn"])
    return L, ref, n_adj


SMALL = [
    # several tiles and a ragged tail in every dimension; shapes follow the five configurations
    ("c1", dict(base="c1_single", context=1040, k_blocks=24), dict()),
    ("c1_perm_ragged", dict(base="c1_single", batch=3, context=1232, k_blocks=16), dict(permute_table=True, ragged=True)),
    ("c2", dict(base="c2_reasoning", batch=3, context=2064, k_blocks=40, layers=1, steps=1), dict(ragged=True)),
    ("c3_zipf", dict(base="c3_longctx", batch=2, context=4112, k_blocks=128, layers=1), dict()),
    ("c4_gqa8", dict(base="c4_gqa8", batch=2, context=2064, k_blocks=48, layers=1), dict(ragged=True)),
    ("c5_td1", dict(base="c5_sweep", batch=2, context=1552, k_blocks=32, n_draft=1), dict()),
    ("c5_td2", dict(base="c5_sweep", batch=2, context=1552, k_blocks=64, n_draft=2), dict(ragged=True)),
    ("c5_td8", dict(base="c5_sweep", batch=2, context=1552, k_blocks=8, n_draft=8), dict()),
    ("full_budget", dict(base="c1_single", batch=2, context=528, k_blocks=64), dict(ragged=True)),
]


def make_cfg(spec):
    spec = dict(spec)
    base = synth.CONFIGS[spec.pop("base")]
    return synth.scaled(base, **spec)


@pytest.mark.parametrize("name,spec,kw", SMALL, ids=[s[0] for s in SMALL])
def test_whole_path_small(oracle, gpu, name, spec, kw):
    _, pipeline = gpu
    cfg = make_cfg(spec)
    lay = synth.make_layer(cfg, seed=11, **kw)
    compare_path(oracle, pipeline, lay, cfg.k_blocks)


def test_full_budget_equals_dense_attention(oracle, gpu):
    """Budget >= number of blocks: the GPU path must reproduce dense causal attention."""
    _, pipeline = gpu
    cfg = synth.scaled(synth.C1, batch=2, context=400, k_blocks=40)     # 25 full blocks, partial local block
    lay = synth.make_layer(cfg, seed=5)
    L, _ = run_gpu_path(pipeline, lay, cfg.k_blocks)
    kv = lay.host_kv.float().numpy()
    q = lay.q.float().numpy()
    scale = 1.0 / math.sqrt(128.0)
    G = cfg.group
    out = pu.bf16_to_f32_np(L.out)
    for b in range(cfg.batch):
        blocks = kv[lay.block_table[b].numpy()]                        # [mb][Hkv][2][16][128]
        for t in range(cfg.n_q_tokens):
            n_vis = cfg.context + t + 1
            for a in range(0, cfg.n_q_heads, 5):
                h = a // G
                K = blocks[:, h, 0].reshape(-1, 128)[:n_vis].astype(np.float64)
                V = blocks[:, h, 1].reshape(-1, 128)[:n_vis].astype(np.float64)
                logits = K @ q[b, t, a].astype(np.float64) * scale
                w = np.exp(logits - logits.max())
                want = (w[:, None] * V).sum(0) / w.sum()
                assert np.all(np.abs(out[b, t, a] - want) <= pu.ATTN_ATOL + pu.ATTN_RTOL * np.abs(want))


def test_sum_reduce_mode(oracle, gpu):
    _, pipeline = gpu
    cfg = synth.scaled(synth.C1, batch=2, context=1040, k_blocks=24, n_draft=3)
    lay = synth.make_layer(cfg, seed=2, ragged=True)
    compare_path(oracle, pipeline, lay, cfg.k_blocks, reduce_mode=1)


def test_kv_pool_in_device_memory(oracle, gpu):
    _, pipeline = gpu
    cfg = synth.scaled(synth.C1, batch=2, context=784, k_blocks=16)
    lay = synth.make_layer(cfg, seed=4, permute_table=True)
    compare_path(oracle, pipeline, lay, cfg.k_blocks, kv_on="device")


@pytest.mark.parametrize("Hq,Hkv,Td,B", [(8, 8, 1, 1), (16, 8, 1, 1), (32, 8, 2, 1), (32, 8, 7, 1), (64, 8, 5, 1), (40, 8, 8, 1),
                                         (128, 8, 8, 1),
                                         # KV head counts other than the five configurations' 8 (one head per GPU is the
                                         # tensor-parallel shape of the larger models, Sec. 5.3.1), odd group sizes
                                         (8, 1, 4, 5), (1, 1, 1, 3), (4, 2, 4, 3), (12, 4, 2, 2), (48, 16, 3, 2), (9, 3, 8, 7)])
def test_row_counts(oracle, gpu, Hq, Hkv, Td, B):
    """R = Td*G from 1 to 128 score rows; T*G from 2 to 144 would exceed 128, so Td is capped.  1 to 16 KV heads."""
    _, pipeline = gpu
    G = Hq // Hkv
    if (Td + 1) * G > 128:
        Td = 128 // G - 1
    cfg = synth.scaled(synth.C1, batch=B, n_q_heads=Hq, n_kv_heads=Hkv, context=656, k_blocks=12, n_draft=Td)
    lay = synth.make_layer(cfg, seed=6)
    compare_path(oracle, pipeline, lay, cfg.k_blocks)


def test_consecutive_steps_with_growing_context(oracle, gpu):
    """Drift workload: 20 decode steps, the local block fills up and a new full block (with its
    summary) appears; late steps need two local blocks (committed + T > 16)."""
    binding, pipeline = gpu
    cfg = synth.scaled(synth.C2, batch=2, context=1024, k_blocks=16, layers=1, steps=20)
    lay = synth.make_layer(cfg, seed=9)
    dev = torch.device("cuda")
    L = pipeline.DecodeLayer(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.max_blocks, cfg.k_blocks,
                             cfg.n_q_tokens, device=dev)
    kv = lay.host_kv.pin_memory()
    table = lay.block_table.to(dev)
    kv_np = pu.np_u16(lay.host_kv)
    summ_ref = None
    for s in range(cfg.steps):
        n_full = lay.n_full_steps[s].to(dev)
        seq_len = lay.seq_len_steps[s].to(dev)
        q = lay.q_steps[s].to(dev)
        if s == 0:
            first = torch.zeros(cfg.batch, dtype=torch.int32, device=dev)
            count = n_full
            max_new = cfg.max_blocks
        else:                                  # incremental: only blocks completed since the last step
            first = lay.n_full_steps[s - 1].to(dev)
            count = (lay.n_full_steps[s] - lay.n_full_steps[s - 1]).to(dev)
            max_new = 1
        L.build_summaries(kv, table, first, count, max_new)
        L.score(q, n_full)
        L.select(n_full, seq_len, table)
        L.stage(kv)
        L.attend(q, seq_len)
        torch.cuda.synchronize()
        ref = pu.oracle_layer(oracle, lay, cfg.k_blocks, 0, s)
        pu.assert_summaries_equal(pu.np_u16(L.summaries), ref["summ"], ref["n_full"])
        gsel = L.sel.cpu().numpy()
        n_adj = pu.assert_sel_parity(gsel, ref["sel"], ref["s64"], cfg.k_blocks)
        if 12 <= s < 16:
            assert (gsel[:, :, cfg.k_blocks + 1] >= 0).all()            # second local block in use
        if n_adj == 0:
            pu.assert_attn_close(pu.bf16_to_f32_np(L.out), ref["attn"])


def _select_only(binding, scores, n_full, seq_len, T, k, table=None, with_lists=True):
    dev = torch.device("cuda")
    B, Hkv, mb = scores.shape
    dims = binding.Dims(B, Hkv, Hkv, mb)
    sel = torch.full((B, Hkv, k + 2), -7, dtype=torch.int32, device=dev)
    idx = torch.full((B, Hkv, k + 2), -7, dtype=torch.int64, device=dev) if with_lists else None
    slots = torch.full((B, Hkv, k + 2), -7, dtype=torch.int32, device=dev) if with_lists else None
    if table is None:
        table = np.arange(B * mb, dtype=np.int32).reshape(B, mb)
    binding.select_topk(dims, torch.from_numpy(scores).to(dev), torch.tensor(n_full, dtype=torch.int32, device=dev),
                        torch.tensor(seq_len, dtype=torch.int32, device=dev), T, k, torch.from_numpy(table).to(dev),
                        sel, idx, slots)
    torch.cuda.synchronize()
    return sel.cpu().numpy(), (idx.cpu().numpy() if with_lists else None)


@pytest.mark.parametrize("n,k", [(1, 1), (5, 3), (31, 31), (33, 40), (64, 9), (1000, 128), (4096, 512),
                                 (8192, 128), (8192, 2048), (20000, 1), (49147, 300)])
def test_select_exact_with_ties(oracle, gpu, n, k):
    """Integer-valued scores: masses of exact ties, so the lowest-index rule decides; exact match."""
    binding, _ = gpu
    rng = np.random.default_rng(n * 31 + k)
    B, Hkv = 2, 3
    mb = n + 5                                                       # 49147 + 5 = 49152, the largest row
    scores = rng.integers(-4, 5, (B, Hkv, mb)).astype(np.float32)
    scores[0, 0, :] = 1.5                                           # a row of all-equal scores
    scores[1, 1, : min(n, 7)] = [0.0, -0.0, 0.0, -0.0, 0.0, -0.0, 0.0][: min(n, 7)]   # signed zeros are equal
    n_full = [n, max(0, n - 3)]
    seq_len = [n * 16 + 3, max(0, n - 3) * 16 + 14]
    table = rng.permutation(B * mb).astype(np.int32).reshape(B, mb)
    got, gidx = _select_only(binding, scores, n_full, seq_len, 5, k, table)
    want, widx, _ = oracle.select_topk(scores, n_full, seq_len, 5, k, table)
    assert np.array_equal(got, want)
    assert np.array_equal(gidx, widx)


def test_select_no_full_blocks_and_no_lists(oracle, gpu):
    binding, _ = gpu
    scores = np.zeros((1, 2, 8), np.float32)
    got, _ = _select_only(binding, scores, [0], [3], 5, 4, with_lists=False)
    assert (got[:, :, :4] == -1).all() and (got[:, :, 4] == 0).all() and (got[:, :, 5] == -1).all()
    got, _ = _select_only(binding, scores, [0], [13], 5, 4, with_lists=False)
    assert (got[:, :, 4] == 0).all() and (got[:, :, 5] == 1).all()


def test_select_random_floats_large(oracle, gpu):
    binding, _ = gpu
    rng = np.random.default_rng(77)
    scores = (rng.standard_normal((4, 8, 8200)) * 50 + 100).astype(np.float32)
    scores[2] = -np.abs(scores[2])                                   # negative scores
    scores[3, :, ::2] *= 1e-30                                       # wide dynamic range
    n_full = [8192, 8000, 4097, 8192]
    seq = [nf * 16 for nf in n_full]
    for k in (1, 128, 513):
        got, _ = _select_only(binding, scores, n_full, seq, 5, k)
        want = oracle.select_topk(scores, n_full, seq, 5, k, np.arange(4 * 8200, dtype=np.int32).reshape(4, 8200),
                                  want_stage=False)
        assert np.array_equal(got, want)


def test_stage_skips_negative_and_keeps_other_slots(oracle, gpu):
    binding, _ = gpu
    dev = torch.device("cuda")
    rng = np.random.default_rng(3)
    host = torch.from_numpy(rng.integers(0, 2 ** 15, (300, 2, 16, 128), dtype=np.int16)).view(torch.bfloat16).pin_memory()
    pool = torch.from_numpy(np.full((200, 2, 16, 128), 0x3ABC, np.int16)).view(torch.bfloat16).to(dev)
    n = 150
    idx = rng.permutation(300)[:n].astype(np.int64)
    idx[::7] = -1
    slots = rng.permutation(200)[:n].astype(np.int32)
    binding.stage_blocks(host, torch.from_numpy(idx).to(dev), torch.from_numpy(slots).to(dev), n, pool)
    torch.cuda.synchronize()
    want = np.full((200, 2, 16, 128), 0x3ABC, np.uint16)
    oracle.stage_blocks(pu.np_u16(host), idx, slots, want)
    assert np.array_equal(pu.np_u16(pool), want)
    binding.stage_blocks(host, torch.from_numpy(idx).to(dev), torch.from_numpy(slots).to(dev), 0, pool)   # n = 0: no-op


@pytest.mark.parametrize("src", ["pinned", "device"])
@pytest.mark.parametrize("n,streams", [(1, 0), (7, 0), (150, 0), (768, 0), (3001, 0), (150, 3), (768, 1024)])
@pytest.mark.parametrize("kind", ["warp", "bulk"])
def test_stage_several_layers_in_one_launch(oracle, gpu, kind, src, n, streams):
    """The several-layers gathers (warp per entry; bulk copies through shared memory): byte-exact per layer against the
    oracle, skipped requests, untouched slots, lists shorter and longer than the number of thread blocks, the error
    word stays 0."""
    binding, _ = gpu
    dev = torch.device("cuda")
    rng = np.random.default_rng(17 + n)
    n_layers, n_host, n_slots = 3, 4000, 3500
    err = torch.zeros(1, dtype=torch.int32, device=dev)
    binding.set_error_word(err)
    try:
        hosts, idxs, slotss, pools, wants = [], [], [], [], []
        for l in range(n_layers):
            h = torch.from_numpy(rng.integers(0, 2 ** 15, (n_host, 2, 16, 128), dtype=np.int16)).view(torch.bfloat16)
            h = h.pin_memory() if src == "pinned" else h.to(dev)
            idx = rng.integers(0, n_host, n).astype(np.int64)
            idx[::5] = -1
            slots = rng.permutation(n_slots)[:n].astype(np.int32)
            hosts.append(h); idxs.append(idx); slotss.append(slots)
            pools.append(torch.from_numpy(np.full((n_slots, 2, 16, 128), 0x3ABC + l, np.int16)).view(torch.bfloat16).to(dev))
            want = np.full((n_slots, 2, 16, 128), 0x3ABC + l, np.uint16)
            oracle.stage_blocks(pu.np_u16(h), idx, slots, want)
            wants.append(want)
        fn = binding.stage_blocks_layers if kind == "warp" else binding.stage_blocks_bulk
        fn(hosts, [torch.from_numpy(i).to(dev) for i in idxs], [torch.from_numpy(s_).to(dev) for s_ in slotss], n, pools, streams)
        torch.cuda.synchronize()
        for l in range(n_layers):
            assert np.array_equal(pu.np_u16(pools[l]), wants[l]), "layer %d" % l
        assert int(err.item()) == 0
    finally:
        binding.set_error_word(None)


def test_attention_padding_rows_and_empty_columns(oracle, gpu):
    """Columns of -1 anywhere in the table (not only at the end), rows that see nothing."""
    binding, pipeline = gpu
    cfg = synth.scaled(synth.C1, batch=2, context=640, k_blocks=20)
    lay = synth.make_layer(cfg, seed=8)
    L, dv = run_gpu_path(pipeline, lay, cfg.k_blocks)
    sel = L.sel.cpu().numpy().copy()
    sel[:, :, 3::4] = -1                                              # punch holes
    sel[1, 2, :] = -1                                                 # one row sees no key at all
    dev = torch.device("cuda")
    L.attend(dv["q"], dv["seq_len"], blk_tbl=torch.from_numpy(sel).to(dev))
    torch.cuda.synchronize()
    slot_tbl = np.arange(sel.size, dtype=np.int32).reshape(sel.shape)
    ref = oracle.sparse_attn(pu.np_u16(lay.q), pu.np_u16(L.pool), slot_tbl, sel, lay.seq_len.numpy(),
                             np.float32(1.0 / math.sqrt(128.0)), cfg.n_kv_heads)
    pu.assert_attn_close(pu.bf16_to_f32_np(L.out), ref)
    G = cfg.group
    assert (pu.bf16_to_f32_np(L.out)[1, :, 2 * G:3 * G] == 0).all()
    assert np.isneginf(L.lse.cpu().numpy()[1, :, 2 * G:3 * G]).all()


def test_empty_batch_is_a_no_op(gpu):
    binding, _ = gpu
    dev = torch.device("cuda")
    dims = binding.Dims(0, 32, 8, 64)
    e16 = torch.empty(16, dtype=torch.bfloat16, device=dev)
    e32 = torch.empty(16, dtype=torch.int32, device=dev)
    ef = torch.empty(16, dtype=torch.float32, device=dev)
    binding.build_summaries(dims, e16, e32, e32, e32, 4, e16)
    binding.score_blocks(dims, e16, 4, e16, e32, ef, q_batch_stride=4 * 32 * 128)
    binding.select_topk(dims, ef, e32, e32, 5, 4, e32, e32)
    binding.sparse_attn(dims, e16, 5, e16, e32, e32, 6, e32, 0.1, e16)
    torch.cuda.synchronize()


@pytest.mark.parametrize("cap_ratio", [0.05, 0.2, 1.0])
def test_plan_delta_matches_oracle_over_steps(oracle, gpu, cap_ratio):
    """Delta selection + capped eviction (KV selection stage) over the drift workload: resident
    table, stamps and gather plan must equal the oracle's exactly at every step, and after the
    planned gathers every resident column must hold exactly its block's bytes."""
    binding, pipeline = gpu
    cfg = synth.scaled(synth.C2, batch=2, context=2048, k_blocks=32, layers=1, steps=12)
    lay = synth.make_layer(cfg, seed=21)
    dev = torch.device("cuda")
    k = cfg.k_blocks
    cap = max(1, int(math.floor(cap_ratio * k)))
    L = pipeline.DecodeLayer(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.max_blocks, k, cfg.n_q_tokens, device=dev)
    kv = lay.host_kv.pin_memory()
    kv_np = pu.np_u16(lay.host_kv).reshape(-1, 2, 16, 128)
    table = lay.block_table.to(dev)
    B, Hkv = cfg.batch, cfg.n_kv_heads
    resident = torch.full((B, Hkv, k + 2), -1, dtype=torch.int32, device=dev)
    stamp = torch.zeros((B, Hkv, k + 2), dtype=torch.int32, device=dev)
    plan_idx = torch.empty((B, Hkv, cap + 2), dtype=torch.int64, device=dev)
    plan_slots = torch.empty((B, Hkv, cap + 2), dtype=torch.int32, device=dev)
    n_adm = torch.empty((B, Hkv), dtype=torch.int32, device=dev)
    res_ref = np.full((B, Hkv, k + 2), -1, np.int32)
    stamp_ref = np.zeros((B, Hkv, k + 2), np.int32)
    zeros = torch.zeros(B, dtype=torch.int32, device=dev)
    L.build_summaries(kv, table, zeros, lay.n_full_steps[-1].to(dev), cfg.max_blocks)
    for s in range(cfg.steps):
        n_full = lay.n_full_steps[s].to(dev)
        L.score(lay.q_steps[s].to(dev), n_full)
        L.select(n_full, lay.seq_len_steps[s].to(dev), table)
        binding.plan_delta(L.dims, L.sel, k, table, resident, stamp, L.cols, cap, s + 1, plan_idx, plan_slots, n_adm,
                           n_local=2)
        binding.stage_blocks(kv, plan_idx, plan_slots, plan_idx.numel(), L.pool)
        torch.cuda.synchronize()
        sel_np = L.sel.cpu().numpy()
        ridx, rslots, radm = oracle.plan_delta(sel_np, lay.block_table.numpy(), res_ref, stamp_ref, k, cap, s + 1, L.cols,
                                               n_local=2)
        assert np.array_equal(resident.cpu().numpy(), res_ref)
        assert np.array_equal(stamp.cpu().numpy(), stamp_ref)
        assert np.array_equal(n_adm.cpu().numpy(), radm)
        gi, gs = plan_idx.cpu().numpy(), plan_slots.cpu().numpy()
        assert np.array_equal(gi, ridx)
        assert np.array_equal(np.where(gi >= 0, gs, 0), np.where(ridx >= 0, rslots, 0))
        assert (radm <= cap).all()
        # the pool mirrors the resident table
        pool_np = pu.np_u16(L.pool)
        for b in range(B):
            for h in range(Hkv):
                for c in list(range(0, k, 5)) + [k, k + 1]:
                    j = res_ref[b, h, c]
                    if j >= 0:
                        src = int(lay.block_table[b, j]) * Hkv + h
                        assert np.array_equal(pool_np[(b * Hkv + h) * L.cols + c], kv_np[src])


@pytest.mark.parametrize("nblk,k,Hkv", [(50, 9, 4), (2056, 128, 8), (8200, 512, 8), (40000, 64, 2)])
def test_union_blocks_matches_oracle(oracle, gpu, nblk, k, Hkv):
    """Head-union set of partial transfer: exact match with the oracle, also when the list is too short."""
    binding, _ = gpu
    dev = torch.device("cuda")
    rng = np.random.default_rng(nblk + k)
    B = 3
    sel = np.stack([np.stack([rng.permutation(nblk)[:k] for _ in range(Hkv)]) for _ in range(B)]).astype(np.int32)
    sel = np.concatenate([sel, np.full((B, Hkv, 2), 5, np.int32)], axis=2)
    sel[1, 0, : k // 2] = -1
    sel[2, :, :k] = sel[2, 0:1, :k]
    dims = binding.Dims(B, Hkv, Hkv, nblk)
    for max_union in (Hkv * k, max(1, k // 2)):
        idx = torch.full((B, max_union), -7, dtype=torch.int32, device=dev)
        n = torch.full((B,), -7, dtype=torch.int32, device=dev)
        binding.union_blocks(dims, torch.from_numpy(sel).to(dev), k, idx, n)
        torch.cuda.synchronize()
        want_idx, want_n = oracle.union_blocks(sel, k, nblk, max_union)
        assert np.array_equal(n.cpu().numpy(), want_n)
        assert np.array_equal(idx.cpu().numpy(), want_idx)


@pytest.mark.parametrize("dst", ["pinned", "device"])
def test_offload_blocks_matches_oracle(oracle, gpu, dst):
    """Dense -> sparse hand-over: byte-exact CPU-pool entries and summaries, permuted page tables on both
    sides, ragged ranges (one running past max_blocks, one empty), untouched entries keep their canary."""
    binding, _ = gpu
    dev = torch.device("cuda")
    rng = np.random.default_rng(81)
    B, Hkv, mb = 3, 8, 21
    Pg, Pc = B * mb + 3, B * mb + 9
    k = torch.from_numpy(rng.standard_normal((Pg, Hkv, 16, 128)).astype(np.float32)).to(torch.bfloat16)
    v = torch.from_numpy(rng.standard_normal((Pg, Hkv, 16, 128)).astype(np.float32)).to(torch.bfloat16)
    gt = torch.from_numpy(rng.permutation(Pg)[:B * mb].reshape(B, mb).astype(np.int32))
    ct = torch.from_numpy(rng.permutation(Pc)[:B * mb].reshape(B, mb).astype(np.int32))
    first = torch.tensor([0, 4, 7], dtype=torch.int32)
    n = torch.tensor([mb, 30, 0], dtype=torch.int32)
    dims = binding.Dims(B, 32, Hkv, mb)
    for with_summ in (True, False):
        host = torch.full((Pc, Hkv, 2, 16, 128), -3.0, dtype=torch.bfloat16)
        host = host.pin_memory() if dst == "pinned" else host.to(dev)
        summ = torch.full((B, Hkv, mb, 2, 128), 7.0, dtype=torch.bfloat16, device=dev)
        want_host = pu.np_u16(torch.full((Pc, Hkv, 2, 16, 128), -3.0, dtype=torch.bfloat16)).copy()
        want_summ = pu.np_u16(torch.full((B, Hkv, mb, 2, 128), 7.0, dtype=torch.bfloat16)).copy()
        oracle.offload_blocks(pu.np_u16(k), pu.np_u16(v), gt.numpy(), ct.numpy(), first.numpy(), n.numpy(), want_host,
                              want_summ if with_summ else None)
        binding.offload_blocks(dims, k.to(dev), v.to(dev), gt.to(dev), ct.to(dev), first.to(dev), n.to(dev), mb,
                               host, summ if with_summ else None)
        torch.cuda.synchronize()
        assert np.array_equal(pu.np_u16(host), want_host)
        assert np.array_equal(pu.np_u16(summ), want_summ)


def test_error_word_registration(gpu):
    """A registered error word stays zero over a normal launch and can be unregistered again."""
    binding, pipeline = gpu
    dev = torch.device("cuda")
    word = torch.zeros(1, dtype=torch.int32, device=dev)
    binding.set_error_word(word)
    try:
        cfg = synth.scaled(synth.C1, batch=1, context=528, k_blocks=8)
        lay = synth.make_layer(cfg, seed=3)
        L = pipeline.DecodeLayer(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.max_blocks, cfg.k_blocks, cfg.n_q_tokens, dev)
        kv = lay.host_kv.to(dev)
        table, n_full, seq, q = (t.to(dev) for t in (lay.block_table, lay.n_full, lay.seq_len, lay.q))
        L.build_summaries(kv, table, torch.zeros_like(n_full), n_full, cfg.max_blocks)
        L.score(q, n_full)
        L.select(n_full, seq, table)
        L.stage(kv)
        L.attend(q, seq)
        torch.cuda.synchronize()
        assert int(word.item()) == 0
    finally:
        binding.set_error_word(None)


@pytest.mark.parametrize("B,Hq,Hkv,Td,nd,ctx,k", [(16, 32, 8, 4, 4, 2064, 24), (10, 32, 8, 2, 2, 1296, 16),
                                                  (12, 64, 8, 1, 1, 1040, 9), (10, 64, 8, 2, 2, 784, 20),
                                                  (16, 64, 8, 8, 4, 784, 20), (18, 16, 8, 4, 4, 3088, 40),
                                                  (16, 32, 8, 1, 1, 528, 40), (20, 32, 8, 4, 4, 1040, 24),
                                                  (38, 32, 8, 2, 2, 784, 9), (37, 32, 8, 1, 1, 528, 3),
                                                  (24, 64, 8, 4, 2, 784, 20), (19, 128, 8, 6, 2, 528, 12),
                                                  (16, 32, 8, 8, 8, 2064, 24), (16, 32, 8, 14, 14, 1040, 12),
                                                  (8, 64, 8, 8, 8, 10256, 38), (24, 64, 8, 8, 8, 1040, 12),
                                                  (1, 32, 8, 4, 4, 2064, 30), (3, 32, 8, 4, 4, 1040, 21),
                                                  (5, 64, 8, 2, 2, 784, 127), (9, 32, 8, 4, 4, 528, 16),
                                                  (16, 8, 1, 4, 4, 1040, 24), (150, 4, 1, 4, 4, 528, 8),
                                                  (30, 12, 4, 3, 3, 1040, 17), (5, 48, 16, 2, 2, 784, 9)])
def test_fused_attention_and_scoring_equals_the_two_calls(oracle, gpu, B, Hq, Hkv, Td, nd, ctx, k):
    """oasis_attn_and_score is steps 4 and 1 in one launch with unchanged arithmetic: outputs, log-sum-exps and
    scores must equal those of oasis_sparse_attn and oasis_score_blocks bit for bit (the separate calls are the
    ones checked against the oracle everywhere else), for 76 to 304 rows (none to three per thread block, evenly
    and unevenly spread), ragged lengths, every row-count variant (nd = draft tokens that score), the four-stage
    ring with narrow and wide scoring accumulators, and 8 to 72 rows whose column lists are split into 2 to 16
    work items each (the merge launch follows)."""
    binding, pipeline = gpu
    dev = torch.device("cuda")
    cfg = synth.scaled(synth.C1, batch=B, n_q_heads=Hq, n_kv_heads=Hkv, context=ctx, k_blocks=k, n_draft=Td)
    lay = synth.make_layer(cfg, seed=12, ragged=True, permute_table=True)
    L = pipeline.DecodeLayer(B, Hq, Hkv, cfg.max_blocks, k, cfg.n_q_tokens, dev, want_lse=True)
    kv = lay.host_kv.to(dev)
    table, n_full, seq, q = (t.to(dev) for t in (lay.block_table, lay.n_full, lay.seq_len, lay.q))
    stride = cfg.n_q_tokens * Hq * 128
    L.build_summaries(kv, table, torch.zeros_like(n_full), n_full, cfg.max_blocks)
    L.score(q, n_full)                                      # the selection uses all draft tokens
    L.select(n_full, seq, table)
    L.stage(kv)
    L.attend(q, seq)
    binding.score_blocks(L.dims, q[:, 1:1 + nd], nd, L.summaries, n_full, L.scores, q_batch_stride=stride)
    torch.cuda.synchronize()
    want_out, want_lse, want_scores = L.out.clone(), L.lse.clone(), L.scores.clone()
    L.out.fill_(float("nan")); L.lse.fill_(float("nan")); L.scores.fill_(float("nan"))
    assert binding.attn_and_score_supported(L.dims, cfg.n_q_tokens, L.cols, nd)
    binding.attn_and_score(L.dims, q, cfg.n_q_tokens, L.pool, L.slot_tbl, L.sel, L.cols, seq, L.scale, L.out,
                           q[:, 1:1 + nd], nd, L.summaries, n_full, L.scores, lse=L.lse, q_batch_stride=stride,
                           workspace=L.workspace)
    torch.cuda.synchronize()
    if 2 * B * Hkv > torch.cuda.get_device_properties(dev).multi_processor_count or \
            torch.equal(L.out.view(torch.int16), want_out.view(torch.int16)):
        # (few long rows: both paths split each column list over several thread blocks in the same way)
        assert torch.equal(L.out.view(torch.int16), want_out.view(torch.int16))
        assert torch.equal(L.lse, want_lse)
    else:
        # few rows, short enough for the fused launch to attend them whole while the separate attention splits
        # their column lists and merges the parts: same result up to the rounding order of the merge
        torch.testing.assert_close(L.out.float(), want_out.float(), atol=2e-3, rtol=1e-2)
        torch.testing.assert_close(L.lse, want_lse, atol=1e-4, rtol=1e-5)
    assert torch.equal(L.scores.view(torch.int32), want_scores.view(torch.int32))


def test_fused_call_rejects_shapes_outside_its_range(gpu):
    binding, _ = gpu
    dev = torch.device("cuda")
    dims = binding.Dims(2, 32, 8, 64)                               # 4 draft tokens asked below: fine; 20: 80 scoring rows
    z16 = torch.zeros(1 << 16, dtype=torch.bfloat16, device=dev)
    zi = torch.zeros(1 << 12, dtype=torch.int32, device=dev)
    zf = torch.zeros(1 << 12, dtype=torch.float32, device=dev)
    with pytest.raises(binding.OasisError, match="outside the fused"):
        binding.attn_and_score(dims, z16, 5, z16, zi, zi, 10, zi, 0.1, z16, z16, 20, z16, zi, zf)


def test_fused_call_wants_its_workspace_when_it_splits(gpu):
    """With few, long rows the fused launch splits the column lists and needs the attention's workspace; without
    it the call must fail before anything is launched."""
    binding, _ = gpu
    dev = torch.device("cuda")
    dims = binding.Dims(1, 32, 8, 512)                              # 8 rows of 130 columns: split
    assert binding.attn_workspace_bytes(dims, 5, 130) > 0
    assert binding.attn_and_score_supported(dims, 5, 130, 4)
    z16 = torch.zeros(1 << 20, dtype=torch.bfloat16, device=dev)
    zi = torch.zeros(1 << 12, dtype=torch.int32, device=dev)
    zf = torch.zeros(1 << 12, dtype=torch.float32, device=dev)
    with pytest.raises(binding.OasisError, match="workspace"):
        binding.attn_and_score(dims, z16, 5, z16, zi, zi, 130, zi, 0.1, z16, z16, 4, z16, zi, zf)


def test_build_summaries_layers_equals_per_layer_calls(gpu):
    """One launch for several layers writes exactly what one oasis_build_summaries call per layer writes
    (which the other tests check against the oracle), and nothing else."""
    binding, pipeline = gpu
    dev = torch.device("cuda")
    cfg = synth.scaled(synth.C1, batch=3, context=1040, k_blocks=8)
    n_layers = 5
    lays = [synth.make_layer(cfg, seed=70 + l, ragged=True, permute_table=True) for l in range(n_layers)]
    dims = binding.Dims(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.max_blocks)
    kvs = [lay.host_kv.to(dev) for lay in lays]
    tables = [lay.block_table.to(dev) for lay in lays]
    n_full = lays[0].n_full.to(dev)
    first = torch.tensor([0, 3, 7], dtype=torch.int32, device=dev)
    n_new = torch.minimum(n_full - first, torch.tensor([40, 1, 9], dtype=torch.int32, device=dev)).contiguous()
    shape = (cfg.batch, cfg.n_kv_heads, cfg.max_blocks, 2, 128)
    want = [torch.full(shape, 7.0, dtype=torch.bfloat16, device=dev) for _ in range(n_layers)]
    got = [torch.full(shape, 7.0, dtype=torch.bfloat16, device=dev) for _ in range(n_layers)]
    for l in range(n_layers):
        binding.build_summaries(dims, kvs[l], tables[l], first, n_new, 40, want[l])
    binding.build_summaries_layers(dims, kvs, tables, first, n_new, 40, got)
    torch.cuda.synchronize()
    for l in range(n_layers):
        assert torch.equal(got[l].view(torch.int16), want[l].view(torch.int16))
    assert not torch.equal(want[0].view(torch.int16), torch.full(shape, 7.0, dtype=torch.bfloat16, device=dev).view(torch.int16))


FUSED_DIRECT = [
    ("rows128", dict(base="c2_reasoning", batch=16, context=2064, k_blocks=24, layers=1, steps=1), dict(ragged=True)),
    ("rows24_split", dict(base="c1_single", batch=3, context=2064, k_blocks=40), dict(ragged=True, permute_table=True)),
    ("rows304", dict(base="c5_sweep", batch=38, context=784, k_blocks=9, n_draft=2), dict(ragged=True)),
    ("gqa8", dict(base="c4_gqa8", batch=10, context=1296, k_blocks=20, layers=1), dict(ragged=True)),
]


@pytest.mark.parametrize("name,spec,kw", FUSED_DIRECT, ids=[s[0] for s in FUSED_DIRECT])
def test_fused_launch_against_the_oracle(oracle, gpu, name, spec, kw):
    """oasis_attn_and_score checked directly against the oracle (not through the separate calls): its scores
    within 1e-5 relative of the double-precision scores, the selection made from ITS scores equal to the oracle's
    (near-ties adjudicated), its attention within tolerance of the oracle's attention on that selection."""
    binding, pipeline = gpu
    dev = torch.device("cuda")
    cfg = make_cfg(spec)
    lay = synth.make_layer(cfg, seed=21, **kw)
    k, T = cfg.k_blocks, cfg.n_q_tokens
    ref = pu.oracle_layer(oracle, lay, k)
    L = pipeline.DecodeLayer(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.max_blocks, k, T, dev, want_lse=True)
    assert binding.attn_and_score_supported(L.dims, T, L.cols, T - 1)
    kv = lay.host_kv.to(dev)
    table, n_full, seq, q = (t.to(dev) for t in (lay.block_table, lay.n_full, lay.seq_len, lay.q))
    L.build_summaries(kv, table, torch.zeros_like(n_full), n_full, cfg.max_blocks)
    # the working set the attention phase reads: the oracle's selection and the oracle's staged pool
    L.pool.copy_(torch.from_numpy(ref["pool"].view(np.int16)).view(torch.bfloat16).to(dev))
    blk = torch.from_numpy(ref["sel"]).to(dev)
    L.scores.fill_(float("nan"))
    L.attend_and_score(q, seq, n_full, blk_tbl=blk)
    L.select(n_full, seq, table)                       # top-k of the fused launch's own scores
    torch.cuda.synchronize()
    pu.assert_scores_close(L.scores.cpu().numpy(), ref["s32"], ref["s64"], ref["n_full"])
    pu.assert_sel_parity(L.sel.cpu().numpy(), ref["sel"], ref["s64"], k)
    pu.assert_attn_close(pu.bf16_to_f32_np(L.out), ref["attn"])
    np.testing.assert_allclose(L.lse.cpu().numpy(), ref["attn"]["lse"], rtol=1e-3, atol=2e-3)


def test_wait_timeout_selftest_reports_and_leaves_the_library_usable(oracle, gpu):
    """A bounded wait that nothing completes must give up, record its code in the registered error word and
    return; the next ordinary call must work and leave the (re-zeroed) word at zero."""
    binding, pipeline = gpu
    dev = torch.device("cuda")
    word = torch.zeros(1, dtype=torch.int32, device=dev)
    result = torch.full((2,), -1, dtype=torch.int32, device=dev)
    binding.set_error_word(word)
    try:
        binding.selftest_wait_timeout(4096, result)
        torch.cuda.synchronize()
        assert result.tolist() == [1, 99]
        assert int(word.item()) == 99
        # the word is only ever written from zero: a second time-out does not overwrite a code already there
        word.fill_(7)
        binding.selftest_wait_timeout(64, result)
        torch.cuda.synchronize()
        assert int(word.item()) == 7
        word.zero_()
        cfg = synth.scaled(synth.C1, batch=2, context=1040, k_blocks=24)
        lay = synth.make_layer(cfg, seed=11)
        compare_path(oracle, pipeline, lay, cfg.k_blocks)
        assert int(word.item()) == 0
    finally:
        binding.set_error_word(None)
    with pytest.raises(binding.OasisError, match="probes"):
        binding.selftest_wait_timeout(0, result)


def test_unwritten_tail_of_the_local_block_may_hold_any_finite_pattern(oracle, gpu):
    """Token rows of the local block past the visible positions are masked; whatever finite bit patterns they
    hold (here the largest finite bf16, in keys and values) must not change the result."""
    binding, pipeline = gpu
    dev = torch.device("cuda")
    cfg = synth.scaled(synth.C1, batch=2, context=1029, k_blocks=12)          # 5 tokens in the local block
    lay = synth.make_layer(cfg, seed=23)
    k, T = cfg.k_blocks, cfg.n_q_tokens
    ref = pu.oracle_layer(oracle, lay, k)
    L, dv = run_gpu_path(pipeline, lay, k)
    want = L.out.clone()
    # overwrite every row past position seq_len + T - 1 of the local entries with 0x7f7f (3.39e38)
    pool = L.pool.view(torch.int16)
    sel = L.sel.cpu().numpy()
    slots = L.slot_tbl.cpu().numpy()
    touched = 0
    for b in range(cfg.batch):
        last = int(lay.seq_len[b]) + T - 1
        for h in range(cfg.n_kv_heads):
            for c in (k, k + 1):
                j = int(sel[b, h, c])
                if j < 0:
                    continue
                first_hidden = max(0, last + 1 - j * 16)
                if first_hidden < 16:
                    pool[int(slots[b, h, c]), :, first_hidden:, :] = 0x7f7f
                    touched += 1
    assert touched > 0
    L.attend(dv["q"], dv["seq_len"])
    torch.cuda.synchronize()
    assert torch.equal(L.out.view(torch.int16), want.view(torch.int16))
    pu.assert_attn_close(pu.bf16_to_f32_np(L.out), ref["attn"])


@pytest.mark.parametrize("host_on", ["pinned", "device"])
def test_append_kv_and_local_window_match_oracle(oracle, gpu, host_on):
    """The KV append (single-layer call and the several-layers launch) and the local-window set-up against the
    oracle, byte for byte, over steps that fill a block, cross a block boundary with the draft tokens and roll
    the local window over; canaries around everything that must stay untouched."""
    binding, _ = gpu
    dev = torch.device("cuda")
    rng = np.random.default_rng(9)
    B, Hkv, T, mb, k, n_layers, steps = 5, 8, 5, 12, 6, 3, 24
    n_cols = k + 2
    dims = binding.Dims(B, 4 * Hkv, Hkv, mb)
    L0 = np.array([33, 16, 47, 60, 79], np.int32)
    tables = [rng.permutation(B * mb).astype(np.int32).reshape(B, mb) for _ in range(n_layers)]
    slot_tbls = [rng.permutation(B * Hkv * n_cols).astype(np.int32).reshape(B, Hkv, n_cols) for _ in range(n_layers)]
    host_ref = [rng.integers(0, 0x7f00, (B * mb, Hkv, 2, 16, 128)).astype(np.uint16) for _ in range(n_layers)]
    pool_ref = [rng.integers(0, 0x7f00, (B * Hkv * n_cols, 2, 16, 128)).astype(np.uint16) for _ in range(n_layers)]
    blk_ref = [np.full((B, Hkv, n_cols), -5, np.int32) for _ in range(n_layers)]
    bf = lambda a: torch.from_numpy(a.view(np.int16)).view(torch.bfloat16)
    host_gpu = [bf(a).pin_memory() if host_on == "pinned" else bf(a).to(dev) for a in host_ref]
    pool_gpu = [bf(a).to(dev) for a in pool_ref]
    blk_gpu = [torch.from_numpy(a).to(dev) for a in blk_ref]
    tab_gpu = [torch.from_numpy(a).to(dev) for a in tables]
    slot_gpu = [torch.from_numpy(a).to(dev) for a in slot_tbls]

    # local-window set-up with gather requests (layer 0), then the requests replayed on both sides
    seq0 = torch.from_numpy(L0).to(dev)
    idx_g = torch.empty((B, Hkv, 2), dtype=torch.int64, device=dev)
    slots_g = torch.empty((B, Hkv, 2), dtype=torch.int32, device=dev)
    binding.local_window(dims, seq0, T, tab_gpu[0], blk_gpu[0], k, n_cols, idx_g, slots_g)
    idx_r, slots_r = oracle.local_window(L0, T, tables[0], blk_ref[0], k, n_cols)
    torch.cuda.synchronize()
    assert np.array_equal(idx_g.cpu().numpy(), idx_r) and np.array_equal(slots_g.cpu().numpy(), slots_r)
    assert np.array_equal(blk_gpu[0].cpu().numpy(), blk_ref[0])

    for s in range(steps):
        seq = (L0 + s).astype(np.int32)
        seq_g = torch.from_numpy(seq).to(dev)
        new = [rng.integers(0, 0x7f00, (B, T, Hkv, 2, 128)).astype(np.uint16) for _ in range(n_layers)]
        new_g = [bf(a).to(dev) for a in new]
        n_commit = 1 if s % 5 else 2
        for l in range(n_layers):
            oracle.append_kv(new[l], n_commit, seq, tables[l], slot_tbls[l], blk_ref[l], k, pool_ref[l], host_ref[l])
        if s % 2:
            binding.append_kv_layers(dims, new_g, n_commit, seq_g, tab_gpu, slot_gpu, blk_gpu, k, pool_gpu, host_gpu)
        else:
            for l in range(n_layers):
                binding.append_kv(dims, new_g[l], n_commit, seq_g, tab_gpu[l], slot_gpu[l], blk_gpu[l], k, pool_gpu[l],
                                  host_gpu[l])
        torch.cuda.synchronize()
        for l in range(n_layers):
            assert np.array_equal(blk_gpu[l].cpu().numpy(), blk_ref[l]), (s, l)
            assert np.array_equal(pu.np_u16(pool_gpu[l]), pool_ref[l]), (s, l)
            assert np.array_equal(pu.np_u16(host_gpu[l]), host_ref[l]), (s, l)
    # no write-back without a CPU pool
    binding.append_kv(dims, new_g[0], 0, seq_g, tab_gpu[0], slot_gpu[0], blk_gpu[0], k, pool_gpu[0], None)
    torch.cuda.synchronize()
    with pytest.raises(binding.OasisError, match="n_commit"):
        binding.append_kv(dims, new_g[0], 1, seq_g, tab_gpu[0], slot_gpu[0], blk_gpu[0], k, pool_gpu[0], None)
