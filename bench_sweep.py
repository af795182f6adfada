"""Secondary measurements of the sparse-decode path on one B200 (not part of the `bench.py` contract).

    python bench_sweep.py [--what c5,stage,shapes]

Kernels alone (the whole step, every configuration and the fetch-ratio sweep are `bench.py --config / --sweep-ratios`).
Prints one JSON line per section:
  c5      the budget x draft-length sweep (configs[4]): solo kernel times and roofline fractions of
          scoring / top-k / attention and of the fused attention + scoring launch, and lookahead recall per cell.
  stage   the gather kernel alone on random entries of a pinned pool, against the DMA copy peak, and the
          dense -> sparse hand-over (device blocks -> pinned entries + summaries) alone.
  shapes  the kernels alone at the shapes of configs[0] to configs[3] (one layer, random
          summaries and pools): scoring, top-k, attention, and the fused attention + scoring launch where
          it takes the shape, each against the measured copy peak.
Inputs are synthetic (the generators of `synth`); nothing here touches the CPU oracle.
"""
import argparse
import json
import math
import os
import sys

import torch

ROOT = os.path.dirname(os.path.abspath(__file__))
sys.path.insert(0, ROOT)

import bench as B                                        # noqa: E402
from paper_2608_08097_b200 import synth                  # noqa: E402


def graph_time(fn, n_rot, iters=32, warm=4):
    """Median of 5 graph replays of `iters` launches rotating over `n_rot` working sets (us per launch)."""
    st = torch.cuda.Stream()
    with torch.cuda.stream(st):
        for i in range(warm):
            fn(i % n_rot)
    torch.cuda.synchronize()
    g = torch.cuda.CUDAGraph()
    with torch.cuda.graph(g, stream=st):
        for i in range(iters):
            fn(i % n_rot)
    ts = []
    for _ in range(5):
        a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        a.record()
        g.replay()
        b.record()
        torch.cuda.synchronize()
        ts.append(a.elapsed_time(b) * 1e3 / iters)
    ts.sort()
    return ts[2]


def section_c5(args, dev, hbm_peak):
    """Budget x draft-length sweep: kernels alone (graph replay over rotating working sets) and recall."""
    from paper_2608_08097_b200 import binding, pipeline
    base = synth.scaled(synth.C5, n_draft=8, layers=1, steps=1)
    lay = synth.make_layer(base, seed=args.seed, layer=0, device=dev)
    kv = lay.host_kv.to(dev)
    table, n_full, seq = lay.block_table.to(dev), lay.n_full.to(dev), lay.seq_len.to(dev)
    Bq, Hq, Hkv, mb = base.batch, base.n_q_heads, base.n_kv_heads, base.max_blocks
    zeros = torch.zeros(Bq, dtype=torch.int32, device=dev)
    nf = int(lay.n_full[0])
    n_rot = 3                                                            # 3 x 268 MB of summaries > 2 x L2
    cells = []
    for K in (32, 64, 128, 256, 512):
        for Td in (1, 2, 4, 8):
            T = Td + 1
            Ls = [pipeline.DecodeLayer(Bq, Hq, Hkv, mb, K, T, dev) for _ in range(n_rot)]
            q = lay.q[:, :T].contiguous().to(dev)
            q_true = lay.q_true[:, :Td].contiguous().to(dev)
            for L in Ls:
                L.build_summaries(kv, table, zeros, n_full, mb)
                L.score(q, n_full)
                L.select(n_full, seq, table)
                L.stage(kv)
            torch.cuda.synchronize()
            t_score = graph_time(lambda i: Ls[i].score(q, n_full), n_rot)
            t_sel = graph_time(lambda i: Ls[i].select(n_full, seq, table), n_rot)
            t_attn = graph_time(lambda i: Ls[i].attend(q, seq), n_rot)
            t_layer = None
            if binding.attn_and_score_supported(Ls[0].dims, T, Ls[0].cols, Td):
                t_layer = graph_time(lambda i: Ls[i].attend_and_score(q, seq, n_full), n_rot)
            sel_draft = Ls[0].sel.clone()
            sel_true = torch.empty_like(sel_draft)
            Ls[0].score_queries(q_true, n_full)
            Ls[0].select(n_full, seq, table, sel=sel_true)
            torch.cuda.synchronize()
            a, b = sel_draft[..., :K], sel_true[..., :K]
            recall = (a[..., :, None] == b[..., None, :]).any(-1).float().mean().item()
            sb = Bq * Hkv * nf * 516
            ab = Bq * Hkv * (min(K, nf) + 1) * 8192 + 2 * Bq * T * Hq * 256
            cells.append({"K": K, "Td": Td, "score_us": round(t_score, 1), "score_frac": round(sb / t_score / 1e3 / hbm_peak, 3),
                          "select_us": round(t_sel, 1), "attn_us": round(t_attn, 1),
                          "attn_frac": round(ab / t_attn / 1e3 / hbm_peak, 3),
                          "layer_us": None if t_layer is None else round(t_layer, 1),
                          "layer_frac": None if t_layer is None else round((sb + ab) / t_layer / 1e3 / hbm_peak, 3),
                          "tokens_per_s_per_layer": round(Bq / ((t_score + t_sel + t_attn) * 1e-6), 1),
                          "tokens_per_s_per_layer_fused": None if t_layer is None else round(Bq / ((t_layer + t_sel) * 1e-6), 1),
                          "recall": round(recall, 4)})
            del Ls
            torch.cuda.empty_cache()
    print(json.dumps({"section": "c5", "workload": "configs[4]: batch 16, 32q/8kv heads, context 65536, one layer "
                      "(3 rotating copies of the summaries and pools), kernels alone; frac = algorithmic bytes / time / "
                      "measured copy peak; layer = the fused attention + scoring launch; tokens/s/layer from the serial sum score + "
                      "top-k + attention (and fused launch + top-k)",
                      "hbm_peak_GBps": hbm_peak, "cells": cells}))


def section_stage(args, dev, hbm_peak):
    """The gather kernels alone: random 8 KiB entries of a 2 GiB pinned pool into HBM slots."""
    from paper_2608_08097_b200 import binding as oasis
    h2d_peak = B.time_pinned_h2d(dev)
    P = 262144
    host = torch.empty((P, 2, 16, 128), dtype=torch.bfloat16, pin_memory=True)
    host.view(torch.int16).random_(0, 1000)
    pool = torch.zeros((4 * 16640, 2, 16, 128), dtype=torch.bfloat16, device=dev)
    g = torch.Generator()
    g.manual_seed(args.seed)
    rows = []
    for n, pad in ((896, 1024), (4096, 4096), (16640, 16640)):
        idxs, slots = [], []
        for _ in range(8):
            idx = torch.full((pad,), -1, dtype=torch.int64)
            idx[torch.randperm(pad, generator=g)[:n]] = torch.randint(0, P, (n,), generator=g)
            idxs.append(idx.to(dev))
            slots.append(torch.arange(pad, dtype=torch.int32, device=dev))
        us = graph_time(lambda i: oasis.stage_blocks(host, idxs[i], slots[i], pad, pool), 8, iters=8, warm=8)
        rows.append({"kernel": "warp per entry", "requests": n, "list_length": pad, "us": round(us, 1),
                     "GBps": round(n * 8192 / us / 1e3, 2), "frac_of_h2d_peak": round(n * 8192 / us / 1e3 / h2d_peak, 3)})
        slots4 = [torch.arange(j * pad, (j + 1) * pad, dtype=torch.int32, device=dev) for j in range(4)]
        # the same lists through the copy unit: one launch carries four layers' lists (here four of the eight lists)
        us = graph_time(lambda i: oasis.stage_blocks_bulk([host] * 4, [idxs[(i + j) % 8] for j in range(4)],
                                                          slots4, pad, [pool] * 4),
                        8, iters=8, warm=8)
        rows.append({"kernel": "bulk copies, 4 lists per launch", "requests": 4 * n, "list_length": pad, "us": round(us, 1),
                     "GBps": round(4 * n * 8192 / us / 1e3, 2), "frac_of_h2d_peak": round(4 * n * 8192 / us / 1e3 / h2d_peak, 3)})
    # the hand-over in the other direction: dense key / value blocks (HBM) -> entries of the pinned pool + summaries
    Bq, Hkv, mb = 8, 8, 2048                                            # 16,384 blocks x 8 heads x 8 KiB = 1 GiB
    dims = oasis.Dims(Bq, 32, Hkv, mb)
    dk = torch.randn((Bq * mb, Hkv, 16, 128), device=dev).to(torch.bfloat16)
    dv = torch.randn((Bq * mb, Hkv, 16, 128), device=dev).to(torch.bfloat16)
    tbl = torch.arange(Bq * mb, dtype=torch.int32, device=dev).view(Bq, mb)
    summ = torch.empty((Bq, Hkv, mb, 2, 128), dtype=torch.bfloat16, device=dev)
    first = torch.zeros(Bq, dtype=torch.int32, device=dev)
    n = torch.full((Bq,), mb, dtype=torch.int32, device=dev)
    host1 = host.view(-1)[:Bq * mb * Hkv * 2 * 16 * 128].view(Bq * mb, Hkv, 2, 16, 128)
    us = graph_time(lambda i: oasis.offload_blocks(dims, dk, dv, tbl, tbl, first, n, mb, host1, summ), 1, iters=2, warm=1)
    gb = Bq * mb * Hkv * 8192 / 1e9
    offload = {"blocks": Bq * mb, "GB": round(gb, 3), "ms": round(us / 1e3, 2), "GBps_to_host": round(gb / (us * 1e-6), 2)}
    print(json.dumps({"section": "stage", "pinned_h2d_peak_GBps": round(h2d_peak, 2), "rows": rows, "offload": offload}))


def section_shapes(args, dev, hbm_peak):
    """Kernels alone at the shapes of configs[0..3] (graph replay over 3 rotating working sets)."""
    from paper_2608_08097_b200 import binding, pipeline
    rows = []
    for name, base in (("configs[0]", synth.C1), ("configs[1]", synth.C2), ("configs[2]", synth.C3), ("configs[3]", synth.C4)):
        cfg = synth.scaled(base, layers=1, steps=1)
        Bq, Hq, Hkv, T, mb, K = cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.n_q_tokens, cfg.max_blocks, cfg.k_blocks
        n_rot = 3
        Ls = [pipeline.DecodeLayer(Bq, Hq, Hkv, mb, K, T, dev) for _ in range(n_rot)]
        g = torch.Generator(device=dev)
        g.manual_seed(args.seed)
        q = torch.randn((Bq, T, Hq, 128), device=dev, generator=g).to(torch.bfloat16)
        nf = cfg.context // 16
        n_full = torch.full((Bq,), nf, dtype=torch.int32, device=dev)
        seq = torch.full((Bq,), cfg.context, dtype=torch.int32, device=dev)
        table = torch.arange(Bq * mb, dtype=torch.int32, device=dev).view(Bq, mb)
        for L in Ls:
            L.summaries.copy_(torch.randn(L.summaries.shape, device=dev, generator=g).to(torch.bfloat16))
            L.pool.copy_(torch.randn(L.pool.shape, device=dev, generator=g).to(torch.bfloat16))
            L.score(q, n_full)
            L.select(n_full, seq, table)
        torch.cuda.synchronize()
        Td, stride = T - 1, T * Hq * 128
        sb = Bq * Hkv * nf * 516
        ab = Bq * Hkv * (K + 1) * 8192 + 2 * Bq * T * Hq * 256
        t_score = graph_time(lambda i: Ls[i].score(q, n_full), n_rot)
        t_sel = graph_time(lambda i: Ls[i].select(n_full, seq, table), n_rot)
        t_attn = graph_time(lambda i: Ls[i].attend(q, seq), n_rot)
        row = {"shape": name, "batch": Bq, "rows": Bq * Hkv, "context": cfg.context, "K": K, "Td": Td, "G": Hq // Hkv,
               "score_us": round(t_score, 1), "score_frac": round(sb / t_score / 1e3 / hbm_peak, 3),
               "select_us": round(t_sel, 1), "attn_us": round(t_attn, 1),
               "attn_frac": round(ab / t_attn / 1e3 / hbm_peak, 3), "layer_us": None, "layer_frac": None}
        if binding.attn_and_score_supported(Ls[0].dims, T, Ls[0].cols, Td):
            def fused(i):
                L = Ls[i]
                binding.attn_and_score(L.dims, q, T, L.pool, L.slot_tbl, L.sel, L.cols, seq, L.scale, L.out, q[:, 1:], Td,
                                       L.summaries, n_full, L.scores, q_batch_stride=stride, workspace=L.workspace)
            t_layer = graph_time(fused, n_rot)
            row["layer_us"] = round(t_layer, 1)
            row["layer_frac"] = round((sb + ab) / t_layer / 1e3 / hbm_peak, 3)
        if name == "configs[1]":
            # step 0 at full size: the summaries of every full block of the layer from a device-resident pool
            kvs = [torch.randn((Bq * mb, Hkv, 2, 16, 128), device=dev, generator=g, dtype=torch.float32).to(torch.bfloat16)
                   for _ in range(n_rot)]
            zeros = torch.zeros(Bq, dtype=torch.int32, device=dev)
            torch.cuda.synchronize()
            t_sum = graph_time(lambda i: Ls[i].build_summaries(kvs[i], table, zeros, n_full, mb), n_rot, iters=12)
            row["summaries_full_build_us"] = round(t_sum, 1)
            row["summaries_full_build_frac"] = round(Bq * Hkv * nf * (4096 + 512) / t_sum / 1e3 / hbm_peak, 3)
            del kvs
        rows.append(row)
        del Ls
        torch.cuda.empty_cache()
    print(json.dumps({"section": "shapes", "workload": "one layer of configs[0..3], 3 rotating copies of summaries and "
                      "pools (random contents), kernels alone by graph replay; frac = algorithmic bytes / time / measured "
                      "copy peak; layer = the fused attention + scoring launch (null where it does not take the shape)",
                      "hbm_peak_GBps": hbm_peak, "rows": rows}))


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--seed", type=int, default=0)
    ap.add_argument("--what", default="c5,stage,shapes")
    args = ap.parse_args()
    if not torch.cuda.is_available():
        raise SystemExit("bench_sweep.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(0)
    dev = torch.device("cuda", 0)
    from paper_2608_08097_b200 import build
    build.build()
    hbm_peak, _ = B.measured_peaks()
    for what in args.what.split(","):
        {"c5": section_c5, "stage": section_stage, "shapes": section_shapes}[what](args, dev, hbm_peak)
        torch.cuda.empty_cache()


if __name__ == "__main__":
    main()
