"""GPU parity at the full sizes of the five benchmark configurations, in the launch
configuration bench.py times (full batch): one layer is generated at full size, the whole
path runs on the GPU, and EVERY request of the batch is checked against the CPU oracle element
by element (summaries and gather exactly, indices with the fp32 near-tie rule, attention within
atol 2e-3 / rtol 1e-2).  The oracle handles one request at a time (0.1 - 1 s each)."""
import math

import numpy as np
import pytest
import torch

from paper_2608_08097_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu
SCALE = np.float32(1.0 / math.sqrt(128.0))


@pytest.fixture(scope="module")
def gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_08097_b200 import build
    build.build()
    from paper_2608_08097_b200 import binding, pipeline
    binding.lib()
    return binding, pipeline


def check_request(oracle, cfg, lay, L, b, k, q_cpu, n_draft_rows=None):
    """Oracle on request b alone (identity block table => its blocks are one contiguous slab)."""
    mb, Hkv = cfg.max_blocks, cfg.n_kv_heads
    kv = pu.np_u16(lay.host_kv[b * mb:(b + 1) * mb])
    table = np.arange(mb, dtype=np.int32).reshape(1, mb)
    n_full = lay.n_full.numpy()[b:b + 1]
    seq = lay.seq_len.numpy()[b:b + 1]
    q = pu.np_u16(q_cpu[b:b + 1])
    T = q.shape[1]
    summ = oracle.build_summaries(kv, table, np.zeros(1, np.int32), n_full)
    pu.assert_summaries_equal(pu.np_u16(L.summaries[b:b + 1]), summ, n_full)
    s32, s64 = oracle.score_blocks(q[:, 1:], summ, n_full)
    pu.assert_scores_close(L.scores[b:b + 1].cpu().numpy(), s32, s64, n_full)
    sel, idx, slots = oracle.select_topk(s32, n_full, seq, T, k, table)
    gsel = L.sel[b:b + 1].cpu().numpy()
    n_adj = pu.assert_sel_parity(gsel, sel, s64, k)
    # gather: the GPU's own requests for this request, replayed by the oracle
    gidx = L.stage_idx[b:b + 1].cpu().numpy()
    want_idx = np.where(gsel < 0, -1, (gsel.astype(np.int64) + b * mb) * Hkv + np.arange(Hkv)[None, :, None])
    assert np.array_equal(gidx, want_idx)
    pool = np.zeros((Hkv * (k + 2), 2, 16, 128), np.uint16)
    local_idx = np.where(gsel < 0, -1, gsel.astype(np.int64) * Hkv + np.arange(Hkv)[None, :, None])
    oracle.stage_blocks(kv.reshape(-1, 2, 16, 128), local_idx, slots, pool)
    rows = slice(b * Hkv * (k + 2), (b + 1) * Hkv * (k + 2))
    assert np.array_equal(pu.np_u16(L.pool[rows]), pool)
    ref = oracle.sparse_attn(q, pool, slots, gsel, seq, SCALE, Hkv)
    pu.assert_attn_close(pu.bf16_to_f32_np(L.out[b:b + 1]), ref)
    return n_adj


def run_full(pipeline, cfg, lay, k, q_dev, kv):
    dev = torch.device("cuda")
    T = q_dev.shape[1]
    L = pipeline.DecodeLayer(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.max_blocks, k, T, device=dev)
    table, n_full, seq_len = (t.to(dev) for t in (lay.block_table, lay.n_full, lay.seq_len))
    return L, table, n_full, seq_len


FULL = [("c1", synth.C1), ("c2", synth.C2), ("c3", synth.C3), ("c4", synth.C4)]


@pytest.mark.parametrize("name,cfg", FULL, ids=[f[0] for f in FULL])
def test_full_size_config(oracle, gpu, name, cfg):
    _, pipeline = gpu
    dev = torch.device("cuda")
    cfg = synth.scaled(cfg, layers=1, steps=1)
    lay = synth.make_layer(cfg, seed=0, layer=0, device=dev, pin=True)
    k = cfg.k_blocks
    q_dev = lay.q.to(dev)
    L, table, n_full, seq_len = run_full(pipeline, cfg, lay, k, q_dev, lay.host_kv)
    L.build_summaries(lay.host_kv, table, torch.zeros_like(n_full), n_full, cfg.max_blocks)
    L.score(q_dev, n_full)
    L.select(n_full, seq_len, table)
    L.stage(lay.host_kv)
    L.attend(q_dev, seq_len)
    torch.cuda.synchronize()
    for b in range(cfg.batch):
        check_request(oracle, cfg, lay, L, b, k, lay.q)
    # properties that hold for every row, checked over the whole batch
    sel = L.sel.cpu().numpy()
    assert (sel[:, :, :k] >= 0).all() and (sel[:, :, :k] < cfg.context // 16).all()
    assert (np.sort(sel[:, :, :k], axis=-1)[..., 1:] != np.sort(sel[:, :, :k], axis=-1)[..., :-1]).all()
    sc = L.scores.cpu().numpy()
    picked = np.take_along_axis(sc, sel[:, :, :k].astype(np.int64), axis=2)
    assert (np.diff(picked, axis=-1) <= 0).all()                       # rank order
    kth = picked[..., -1:]
    assert ((sc > kth).sum(-1) <= k - 1).all()                        # nothing better was left out
    assert np.isfinite(pu.bf16_to_f32_np(L.out)).all()
    # the fused attention + scoring launch (what the decode engine and bench.py run) at the same full size:
    # scores bit for bit, outputs bit for bit unless it attends whole rows where the separate call splits them
    binding = gpu[0]
    T = q_dev.shape[1]
    if binding.attn_and_score_supported(L.dims, T, L.cols, T - 1):
        want_out, want_scores = L.out.clone(), L.scores.clone()
        L.out.fill_(float("nan"))
        L.scores.fill_(float("nan"))
        L.attend_and_score(q_dev, seq_len, n_full)
        torch.cuda.synchronize()
        assert torch.equal(L.scores.view(torch.int32), want_scores.view(torch.int32))
        if not torch.equal(L.out.view(torch.int16), want_out.view(torch.int16)):
            assert 2 * cfg.batch * cfg.n_kv_heads <= torch.cuda.get_device_properties(dev).multi_processor_count
            torch.testing.assert_close(L.out.float(), want_out.float(), atol=2e-3, rtol=1e-2)
        # and the fused launch's own scores and outputs directly against the oracle, every request
        for b in range(cfg.batch):
            check_request(oracle, cfg, lay, L, b, k, lay.q)


def test_full_size_budget_and_draft_sweep(oracle, gpu):
    """configs[4]: budget {512 .. 8,192} tokens x draft length {1, 2, 4, 8} at batch 16, context 65,536."""
    _, pipeline = gpu
    dev = torch.device("cuda")
    cfg = synth.scaled(synth.C5, n_draft=8)
    lay = synth.make_layer(cfg, seed=0, layer=0, device=dev, pin=True)
    table, n_full, seq_len = (t.to(dev) for t in (lay.block_table, lay.n_full, lay.seq_len))
    first = True
    for budget in (512, 1024, 2048, 4096, 8192):
        k = budget // 16
        for td in (1, 2, 4, 8):
            q_cpu = lay.q[:, :td + 1].contiguous()
            q_dev = q_cpu.to(dev)
            L = pipeline.DecodeLayer(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.max_blocks, k, td + 1, device=dev)
            L.build_summaries(lay.host_kv, table, torch.zeros_like(n_full), n_full, cfg.max_blocks)
            L.score(q_dev, n_full)
            L.select(n_full, seq_len, table)
            L.stage(lay.host_kv)
            L.attend(q_dev, seq_len)
            torch.cuda.synchronize()
            for b in range(cfg.batch):
                check_request(oracle, cfg, lay, L, b, k, q_cpu)
            del L


ENGINE_FULL = [("c2", synth.C2, 2, 3), ("c3", synth.C3, 1, 2), ("c4", synth.C4, 1, 2)]


@pytest.mark.parametrize("name,base,n_layers,S", ENGINE_FULL, ids=[e[0] for e in ENGINE_FULL])
def test_full_size_engine_steps(oracle, gpu, name, base, n_layers, S):
    """configs[1], [2] and [3] at full size through the multi-layer engine (full batch, consecutive eager steps, every
    selected block gathered): every request's selection (near-ties adjudicated with the oracle's double-precision
    scores) and attention outputs against the oracle.  The fused launch runs in its three arrangements here: one row
    per thread block (128 rows), several rows per thread block (256 rows), 128 MMA rows with row-less scoring blocks
    (64 rows of 72 query rows)."""
    _, pipeline = gpu
    dev = torch.device("cuda")
    cfg = synth.scaled(base, layers=n_layers, steps=S)
    k, B, Hkv, mb = cfg.k_blocks, cfg.batch, cfg.n_kv_heads, cfg.max_blocks
    lays = [synth.make_layer(cfg, seed=0, layer=l, device=dev, pin=True) for l in range(n_layers)]
    eng = pipeline.DecodeEngine(B, cfg.n_q_heads, Hkv, mb, k, cfg.n_q_tokens, n_layers, dev)
    for l, lay in enumerate(lays):
        eng.attach(l, lay.host_kv, lay.block_table.to(dev))
    seq = lays[0].seq_len_steps
    q_dev = [lay.q_steps.to(dev) for lay in lays]
    to_dev = lambda t: t.to(torch.int32).contiguous().to(dev)
    eng.prime([q_dev[l][0] for l in range(n_layers)], to_dev(seq[0] // 16), to_dev(seq[0]))
    torch.cuda.synchronize()
    used_sel = [eng.layers[l].sel.cpu().numpy() for l in range(n_layers)]     # what the next attention reads
    prev_q = 0
    table = np.arange(mb, dtype=np.int32).reshape(1, mb)
    for s in range(S):
        eng.step([q_dev[l][s] for l in range(n_layers)], to_dev(seq[s]), to_dev(seq[s] // 16),
                 to_dev((seq[s] + 1) // 16 - seq[s] // 16), to_dev((seq[s] + 1) // 16), to_dev(seq[s] + 1))
        eng.join()
        torch.cuda.synchronize()
        for l in range(n_layers):
            for b in range(B):
                kv = pu.np_u16(lays[l].host_kv[b * mb:(b + 1) * mb])
                n_full = (seq[s][b:b + 1] // 16).numpy()
                sq = seq[s][b:b + 1].numpy()
                summ = oracle.build_summaries(kv, table, np.zeros(1, np.int32), n_full)
                qp = pu.np_u16(lays[l].q_steps[prev_q][b:b + 1])            # the drafts that predicted this step
                s32, s64 = oracle.score_blocks(qp[:, 1:], summ, n_full)
                sel, idx, slots = oracle.select_topk(s32, n_full, sq, cfg.n_q_tokens, k, table)
                gsel = used_sel[l][b:b + 1]
                pu.assert_sel_parity(gsel, sel, s64, k)
                # the attention ran over the GPU's own (adjudicated) selection
                gidx = np.where(gsel < 0, -1, gsel.astype(np.int64) * Hkv + np.arange(Hkv)[None, :, None])
                pool = np.zeros((Hkv * (k + 2), 2, 16, 128), np.uint16)
                oracle.stage_blocks(kv.reshape(-1, 2, 16, 128), gidx, slots, pool)
                ref = oracle.sparse_attn(pu.np_u16(lays[l].q_steps[s][b:b + 1]), pool, slots, gsel, sq, SCALE, Hkv)
                pu.assert_attn_close(pu.bf16_to_f32_np(eng.layers[l].out[b:b + 1]), ref)
        used_sel = [eng.layers[l].sel.cpu().numpy() for l in range(n_layers)]
        prev_q = s


def test_full_size_engine_delta_append_graph(oracle, gpu):
    """configs[1] at full size the way bench.py runs it: delta selection with the paper's default cap, the KV append,
    three decode steps in ONE CUDA graph, queries uploaded and outputs downloaded inside the steps; every request,
    two layers, against the oracle (attention of every step, selections, tables, working-set pool, and the blocks of
    the CPU pool that the write-through can have touched)."""
    from tests import engine_util
    _, pipeline = gpu
    dev = torch.device("cuda")
    cfg = synth.scaled(synth.C2, layers=2, steps=3)
    lays = [synth.make_layer(cfg, seed=0, layer=l, device=dev, pin=True) for l in range(cfg.layers)]
    engine_util.check_engine(oracle, pipeline, cfg, lays, "delta", int(0.05 * cfg.k_blocks), True, 3, True, True, True,
                             wait_group=1, transfer_group=2, max_adjudicated=64, light=True)
