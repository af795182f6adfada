"""Shared helpers of the GPU parity tests: run the oracle on a synthetic layer, and the
adjudication rules for indices (bit-exact, or fp32-tie within 1e-5 relative of the oracle's
double-precision scores) and for attention outputs (atol 2e-3, rtol 1e-2)."""
import numpy as np
import torch

from paper_2608_08097_b200 import synth

ATTN_ATOL, ATTN_RTOL = 2e-3, 1e-2
SCORE_RTOL = 1e-5


def np_u16(t):
    return synth.u16(t.detach().cpu())


def oracle_layer(oracle, lay, k, reduce_mode=0, step=0, sel_override=None):
    """The whole path on the CPU for one layer / step.  Returns every intermediate."""
    cfg = lay.cfg
    B, Hkv, T = cfg.batch, cfg.n_kv_heads, cfg.n_q_tokens
    kv = np_u16(lay.host_kv)
    table = lay.block_table.numpy()
    n_full = lay.n_full_steps[step].numpy()
    seq_len = lay.seq_len_steps[step].numpy()
    q = np_u16(lay.q_steps[step])
    summ = oracle.build_summaries(kv, table, np.zeros(B, np.int32), n_full)
    s32, s64 = oracle.score_blocks(q[:, 1:], summ, n_full, reduce_mode)
    sel, idx, slots = oracle.select_topk(s32, n_full, seq_len, T, k, table)
    if sel_override is not None:
        sel = sel_override
        idx = np.where(sel < 0, -1, np.take_along_axis(
            np.broadcast_to(table[:, None, :], (B, Hkv, table.shape[1])), np.maximum(sel, 0), axis=2).astype(np.int64)
            * Hkv + np.arange(Hkv)[None, :, None])
    pool = np.zeros((B * Hkv * (k + 2), 2, 16, 128), np.uint16)
    oracle.stage_blocks(kv.reshape(-1, 2, 16, 128), idx, slots, pool)
    slot_tbl = np.arange(B * Hkv * (k + 2), dtype=np.int32).reshape(B, Hkv, k + 2)
    attn = oracle.sparse_attn(q, pool, slot_tbl, sel, seq_len, np.float32(1.0 / np.sqrt(128.0)), Hkv)
    return dict(summ=summ, s32=s32, s64=s64, sel=sel, idx=idx, slots=slots, pool=pool, attn=attn,
                n_full=n_full, seq_len=seq_len, q=q)


def assert_summaries_equal(gpu_summ, ref_summ, n_full):
    """Exact equality of the bf16 values (a +0 / -0 difference is not a value difference)."""
    g = torch.from_numpy(np.ascontiguousarray(gpu_summ).view(np.int16)).view(torch.bfloat16).float().numpy()
    r = torch.from_numpy(np.ascontiguousarray(ref_summ).view(np.int16)).view(torch.bfloat16).float().numpy()
    for b, nf in enumerate(n_full):
        assert np.array_equal(g[b, :, :nf], r[b, :, :nf]), "summaries differ for request %d" % b


def assert_scores_close(gpu_scores, s32, s64, n_full):
    for b, nf in enumerate(n_full):
        g = gpu_scores[b, :, :nf].astype(np.float64)
        ref = s64[b, :, :nf]
        err = np.abs(g - ref) / np.maximum(np.abs(ref), 1e-30)
        assert err.max(initial=0.0) <= SCORE_RTOL, "score rel err %.3g (request %d)" % (err.max(), b)
        assert np.isneginf(gpu_scores[b, :, nf:]).all(), "scores past n_full must be -inf"


def assert_sel_parity(gpu_sel, ref_sel, s64, k):
    """Element-wise equality; a differing position is tolerated only if the two block ids have
    oracle double-precision scores within 1e-5 relative of each other.  Returns the number of
    adjudicated positions."""
    assert gpu_sel.shape == ref_sel.shape
    assert np.array_equal(gpu_sel[..., k:], ref_sel[..., k:]), "local block columns differ"
    diff = np.argwhere(gpu_sel[..., :k] != ref_sel[..., :k])
    for b, h, r in diff:
        jg, jr = gpu_sel[b, h, r], ref_sel[b, h, r]
        assert jg >= 0 and jr >= 0, "padding differs at %s" % ((b, h, r),)
        sg, sr = s64[b, h, jg], s64[b, h, jr]
        assert abs(sg - sr) <= SCORE_RTOL * max(abs(sg), abs(sr)), \
            "row (%d,%d) rank %d: gpu block %d (%.9g) vs oracle block %d (%.9g)" % (b, h, r, jg, sg, jr, sr)
    # each row must still be a set of distinct blocks
    for b in range(gpu_sel.shape[0]):
        for h in range(gpu_sel.shape[1]):
            row = gpu_sel[b, h, :k]
            row = row[row >= 0]
            assert len(set(row.tolist())) == len(row), "duplicate block in row (%d,%d)" % (b, h)
    return len(diff)


BF16_HALF_ULP = 2.0 ** -9           # relative rounding error of a value kept to 8 significant bits
MAX_BOUND_FRACTION = 1e-5           # share of the elements that may need the arithmetic bound instead of the tolerance


def assert_attn_close(gpu_out, ref):
    """ref: the oracle's result dict (or just its fp32 output).  Every element must lie within
    atol 2e-3 + rtol 1e-2 of the oracle.  The tensor core takes the softmax weights as bf16, which perturbs an
    output element by up to 2^-9 * sum_p w_p |v_p| whatever the element's own size; in rows whose softmax is carried
    by a few keys with large values that can exceed atol at a small element.  Such elements -- at most 1e-5 of
    all -- must then lie within the worst case of that arithmetic, 2^-9 * (2 * sum_p w_p |v_p| + |out|) (weights
    rounded in the numerator, exact in the denominator, output rounded to bf16), which the oracle's out_abs gives."""
    ref32 = ref["out32"] if isinstance(ref, dict) else ref
    g = gpu_out.astype(np.float64)
    r = ref32.astype(np.float64)
    err = np.abs(g - r)
    over = err - (ATTN_ATOL + ATTN_RTOL * np.abs(r))
    worst = over.max(initial=-1.0)
    if worst <= 0:
        return
    assert isinstance(ref, dict) and "out_abs" in ref, \
        "attention off by %.3g beyond tolerance (max abs err %.3g)" % (worst, err.max())
    bad = over > 0
    bound = BF16_HALF_ULP * (2.0 * ref["out_abs"] + np.abs(r)) + 1e-6
    assert (err[bad] <= bound[bad]).all(), \
        "attention off by %.3g beyond tolerance and beyond the bf16-weight bound (max abs err %.3g)" % (worst, err.max())
    assert bad.sum() <= max(1, int(MAX_BOUND_FRACTION * bad.size)), \
        "%d of %d elements beyond tolerance (worst by %.3g): more than rounding of the weights explains" % (bad.sum(), bad.size, worst)


def bf16_to_f32_np(t):
    return t.detach().float().cpu().numpy()
