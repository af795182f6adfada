"""GPU parity of the multi-layer decode engine (the launch sequence bench.py times): at every
step each layer's attention must equal the oracle's attention over the working set that the
previous step's lookahead prediction selected, in fetch-all and in capped-delta mode."""
import math

import numpy as np
import pytest
import torch

from paper_2608_08097_b200 import synth
from tests import engine_util, parity_util as pu

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


def oracle_prediction(oracle, lay, summ_cache, q_step, n_full, seq):
    """Selection made from the draft queries of step q_step for a step whose view is (n_full, seq)."""
    cfg = lay.cfg
    kv = pu.np_u16(lay.host_kv)
    table = lay.block_table.numpy()
    summ = oracle.build_summaries(kv, table, np.zeros(cfg.batch, np.int32), n_full)
    q = pu.np_u16(lay.q_steps[q_step])
    s32, s64 = oracle.score_blocks(q[:, 1:], summ, n_full)
    sel, idx, slots = oracle.select_topk(s32, n_full, seq, cfg.n_q_tokens, cfg.k_blocks, table)
    return sel, idx, slots, s64


# (mode, cap, append, chunk, graph, e2e): `chunk` steps run between synchronisations -- one CUDA graph of `chunk`
# steps when `graph`, else eager steps launched back to back without any synchronisation in between.
ENGINE_CASES = [
    ("fetch_all", None, False, 1, False, False), ("delta", 3, False, 1, False, False), ("delta", 16, False, 1, False, False),
    ("fetch_all", None, False, 1, True, False), ("delta", 3, False, 1, True, False), ("delta", 3, False, 1, False, True),
    ("delta", 3, False, 1, True, True),
    ("delta", 3, True, 1, False, False), ("delta", 3, True, 1, True, True), ("delta", 16, True, 1, True, False),
    ("delta", 3, True, 4, True, True), ("delta", 3, False, 5, True, True), ("fetch_all", None, False, 3, True, True),
    ("delta", 3, True, 19, False, False), ("delta", 3, True, 19, False, True), ("fetch_all", None, False, 19, False, False),
]


@pytest.mark.parametrize("fused", [True, False], ids=["fused", "unfused"])
@pytest.mark.parametrize("mode,cap,append,chunk,graph,e2e", ENGINE_CASES)
def test_engine_steps_match_oracle(oracle, gpu, mode, cap, append, chunk, graph, e2e, fused):
    binding, pipeline = gpu
    n_layers, S = 3, 19
    cfg = synth.scaled(synth.C2, batch=2, context=1544 if append else 1536, k_blocks=16, layers=n_layers, steps=S)
    lays = [synth.make_layer(cfg, seed=31, layer=l) for l in range(n_layers)]
    engine_util.check_engine(oracle, pipeline, cfg, lays, mode, cap, append, chunk, graph, e2e, fused, wait_group=2,
                             transfer_group=2 if (append or chunk == 3) else 1)


def test_handover_from_dense_pool_then_decode(oracle, gpu):
    """Dense -> sparse transition (Sec. 4.3): the engine starts from dense GPU key / value pools behind their
    own (permuted) page table, copies them to an empty pinned CPU pool with the summaries built on the way,
    then selects, gathers and attends.  The CPU pool must equal the generator's pool byte for byte and the
    first sparse step must match the oracle."""
    binding, pipeline = gpu
    dev = torch.device("cuda")
    cfg = synth.scaled(synth.C2, batch=2, context=1544, k_blocks=16, layers=1, steps=2)    # 96 full blocks + 8 tokens
    k, B, Hkv, mb = cfg.k_blocks, cfg.batch, cfg.n_kv_heads, cfg.max_blocks
    lay = synth.make_layer(cfg, seed=33, layer=0, permute_table=True)
    seq = lay.seq_len_steps
    # the dense pool: the same blocks, keys and values apart, at permuted physical positions
    g = torch.Generator()
    g.manual_seed(5)
    P = lay.host_kv.shape[0]
    perm = torch.randperm(P, generator=g)
    inv = torch.empty_like(perm)
    inv[perm] = torch.arange(P)
    dense_k = lay.host_kv[perm][:, :, 0].contiguous().to(dev)                # dense block p holds CPU block perm[p]
    dense_v = lay.host_kv[perm][:, :, 1].contiguous().to(dev)
    gpu_table = inv[lay.block_table.long()].to(torch.int32).to(dev)          # logical -> dense physical
    host = torch.zeros_like(lay.host_kv).pin_memory()

    eng = pipeline.DecodeEngine(B, cfg.n_q_heads, Hkv, mb, k, cfg.n_q_tokens, 1, dev, mode="fetch_all")
    eng.attach(0, host, lay.block_table.to(dev))
    to_dev = lambda t: t.to(torch.int32).contiguous().to(dev)
    eng.handover(0, dense_k, dense_v, gpu_table, to_dev(seq[0]))
    q_dev = lay.q_steps.to(dev)
    eng.prime([q_dev[0]], to_dev(seq[0] // 16), to_dev(seq[0]), summaries_ready=True)
    torch.cuda.synchronize()

    n_any = (int(seq[0].max()) + 15) // 16
    used = lay.block_table[:, :n_any].reshape(-1).long()
    assert torch.equal(host[used], lay.host_kv[used])
    kv = pu.np_u16(lay.host_kv)
    n_full0 = (seq[0] // 16).numpy()
    summ = oracle.build_summaries(kv, lay.block_table.numpy(), np.zeros(B, np.int32), n_full0)
    pu.assert_summaries_equal(pu.np_u16(eng.layers[0].summaries), summ, n_full0)

    sel, idx, slots, _ = oracle_prediction(oracle, lay, None, 0, n_full0, seq[0].numpy())
    pool = np.zeros((B * Hkv * (k + 2), 2, 16, 128), np.uint16)
    oracle.stage_blocks(kv.reshape(-1, 2, 16, 128), idx, slots, pool)
    slot_tbl = np.arange(B * Hkv * (k + 2), dtype=np.int32).reshape(B, Hkv, k + 2)
    args = ([q_dev[0]], to_dev(seq[0]), to_dev(seq[0] // 16), to_dev((seq[0] + 1) // 16 - seq[0] // 16),
            to_dev((seq[0] + 1) // 16), to_dev(seq[0] + 1))
    eng.step(*args, step_stamp=1)
    eng.join()
    torch.cuda.synchronize()
    ref = oracle.sparse_attn(pu.np_u16(lay.q_steps[0]), pool, slot_tbl, sel, seq[0].numpy(), SCALE, Hkv)
    pu.assert_attn_close(pu.bf16_to_f32_np(eng.layers[0].out), ref)


@pytest.mark.parametrize("mode,cap", [("fetch_all", None), ("delta", 2)])
def test_fused_engine_equals_unfused_engine(gpu, mode, cap):
    """With 128 (request, KV head) rows the engine makes one fused launch per layer (attention + scoring,
    overlapping consecutive layers through programmatic dependent launch); its outputs, selections and working
    sets must equal, bit for bit, those of the engine that makes the two separate launches."""
    binding, pipeline = gpu
    dev = torch.device("cuda")
    n_layers, S = 3, 6
    cfg = synth.scaled(synth.C2, batch=16, context=1040, k_blocks=12, layers=n_layers, steps=S)
    lays = [synth.make_layer(cfg, seed=51, layer=l, device=dev) for l in range(n_layers)]
    seq = lays[0].seq_len_steps
    to_dev = lambda t: t.to(torch.int32).contiguous().to(dev)
    engines = []
    for fused in (True, False):
        # the fused engine also alternates its gathers between three transfer streams
        eng = pipeline.DecodeEngine(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.max_blocks, cfg.k_blocks,
                                    cfg.n_q_tokens, n_layers, dev, mode=mode, cap=cap, fused=fused,
                                    transfer_streams=3 if fused else 1)
        assert eng.fused == fused
        for l, lay in enumerate(lays):
            eng.attach(l, lay.host_kv.to(dev), lay.block_table.to(dev))
        engines.append(eng)
    q_dev = [lay.q_steps.to(dev) for lay in lays]
    for eng in engines:
        eng.prime([q_dev[l][0] for l in range(n_layers)], to_dev(seq[0] // 16), to_dev(seq[0]))
    for s in range(S):
        args = ([q_dev[l][s] for l in range(n_layers)], to_dev(seq[s]), to_dev(seq[s] // 16),
                to_dev((seq[s] + 1) // 16 - seq[s] // 16), to_dev((seq[s] + 1) // 16), to_dev(seq[s] + 1))
        graphs = [eng.capture_step(*args, step_stamp=s + 1) for eng in engines]
        for eng, g in zip(engines, graphs):
            eng.replay(g)
        torch.cuda.synchronize()
        a, b = engines
        for l in range(n_layers):
            assert torch.equal(a.layers[l].out.view(torch.int16), b.layers[l].out.view(torch.int16))
            assert torch.equal(a.layers[l].scores.view(torch.int32), b.layers[l].scores.view(torch.int32))
            assert torch.equal(a.layers[l].sel, b.layers[l].sel)
            assert torch.equal(a.blk_tbl(l), b.blk_tbl(l))
            assert torch.equal(a.layers[l].pool.view(torch.int16), b.layers[l].pool.view(torch.int16))
