"""oasis_sparse_attn_static_scratch: attention for callers that cannot allocate scratch memory
(all free device memory already belongs to the engine's KV pool, or cudaMalloc is not allowed
in the decode loop).  It runs the same kernels with the same split plan as oasis_sparse_attn, so
its output must equal that call's bit for bit on the same inputs -- also on a second call that
finds the previous call's partials still in the built-in array -- and both must agree with the CPU
oracle within the attention tolerance.  This file sorts last on purpose, so a run that stops at
the first failure has already run the others."""
import math

import numpy as np
import pytest
import torch

from paper_2608_08097_b200 import synth
from tests import parity_util as pu

pytestmark = pytest.mark.gpu


def test_static_scratch_attention_matches_workspace_attention_twice(oracle):
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_08097_b200 import build
    build.build()
    from paper_2608_08097_b200 import binding, pipeline
    dev = torch.device("cuda")
    scale = 1.0 / math.sqrt(128.0)
    # two different workloads, both split over the column list (so both use scratch)
    cases = [synth.scaled(synth.C1, batch=2, context=2064, k_blocks=48),
             synth.scaled(synth.C5, batch=3, context=1040, k_blocks=30, n_draft=2)]
    for call, cfg in enumerate(cases):
        lay = synth.make_layer(cfg, seed=40 + call, ragged=True)
        L = pipeline.DecodeLayer(cfg.batch, cfg.n_q_heads, cfg.n_kv_heads, cfg.max_blocks, cfg.k_blocks,
                                 cfg.n_q_tokens, device=dev, want_lse=True)
        need = binding.attn_workspace_bytes(L.dims, cfg.n_q_tokens, L.cols)
        assert 0 < need <= binding.static_scratch_bytes()
        kv = lay.host_kv.to(dev)
        table, n_full, seq_len, q = (t.to(dev) for t in (lay.block_table, lay.n_full, lay.seq_len, lay.q))
        L.build_summaries(kv, table, torch.zeros_like(n_full), n_full, cfg.max_blocks)
        L.score(q, n_full)
        L.select(n_full, seq_len, table)
        L.stage(kv)
        want = L.attend(q, seq_len).clone()                       # existing entry point, caller workspace
        want_lse = L.lse.clone()
        got = torch.full_like(want, float("nan"))
        got_lse = torch.full_like(want_lse, float("nan"))
        binding.sparse_attn_static_scratch(L.dims, q, cfg.n_q_tokens, L.pool, L.slot_tbl, L.sel, L.cols,
                                           seq_len, scale, got, lse=got_lse)
        torch.cuda.synchronize()
        assert torch.isfinite(got.float()).all()
        assert torch.equal(got.view(torch.int16), want.view(torch.int16)), "call %d differs" % call
        assert torch.equal(got_lse.view(torch.int32), want_lse.view(torch.int32)), "call %d: lse differs" % call
        # and against the oracle, on the selection and working set the GPU produced
        ref = oracle.sparse_attn(pu.np_u16(lay.q), pu.np_u16(L.pool), L.slot_tbl.cpu().numpy(), L.sel.cpu().numpy(),
                                 lay.seq_len.numpy(), np.float32(scale), cfg.n_kv_heads)
        pu.assert_attn_close(pu.bf16_to_f32_np(got), ref)
        np.testing.assert_allclose(got_lse.cpu().numpy(), ref["lse"], rtol=1e-3, atol=2e-3)


def test_static_scratch_rejects_oversized_shapes():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    from paper_2608_08097_b200 import binding
    dev = torch.device("cuda")
    # 128 query rows per KV head on one GPU split far enough to need more than the built-in 4 MiB
    dims = binding.Dims(1, 128, 1, 4096)
    n_cols = 2050
    assert binding.attn_workspace_bytes(dims, 1, n_cols) > binding.static_scratch_bytes()
    t16 = torch.zeros(128 * 128, dtype=torch.bfloat16, device=dev)
    ti = torch.zeros(n_cols, dtype=torch.int32, device=dev)
    with pytest.raises(binding.OasisError, match="built-in array holds"):
        binding.sparse_attn_static_scratch(dims, t16, 1, t16, ti, ti, n_cols, ti, 0.1, t16)
