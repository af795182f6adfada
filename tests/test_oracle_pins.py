"""Pins the CPU oracle to things other than itself: brute force on tiny inputs,
invariants, closed forms and library routines (numpy / torch CPU), chosen so that a
dropped term, a wrong sign or index, or a transposed operand fails at least one test.
"""
import math
import os

import numpy as np
import pytest
import torch

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def rand_bf16(rng, shape, scale=1.0):
    """Random values that are exactly representable in bf16, as (uint16 bits, float32)."""
    x = torch.from_numpy((rng.standard_normal(shape) * scale).astype(np.float32)).to(torch.bfloat16)
    bits = x.view(torch.int16).numpy().view(np.uint16).copy()
    return bits, x.to(torch.float32).numpy()


def make_pool(rng, P, Hkv, bs, d, scale=1.0):
    return rand_bf16(rng, (P, Hkv, 2, bs, d), scale)


# --------------------------------------------------------------------------- bf16


def test_bf16_roundtrip_matches_torch(oracle):
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(4096) * 10.0 ** rng.integers(-6, 6, 4096)).astype(np.float32)
    x[:4] = [0.0, -0.0, 1.0 + 2.0 ** -8, 1.0 + 3 * 2.0 ** -8]      # exact ties: round to even
    ours = oracle.f32_to_bf16(x)
    ref = torch.from_numpy(x).to(torch.bfloat16).view(torch.int16).numpy().view(np.uint16)
    assert np.array_equal(ours, ref)
    assert np.array_equal(oracle.bf16_to_f32(ours), torch.from_numpy(x).to(torch.bfloat16).float().numpy())


# --------------------------------------------------------------------------- summaries


def test_summaries_match_numpy_minmax_and_bounds(oracle):
    rng = np.random.default_rng(1)
    B, Hkv, bs, d, mb = 2, 3, 4, 5, 6
    bits, vals = make_pool(rng, B * mb, Hkv, bs, d)
    table = rng.permutation(B * mb).astype(np.int32).reshape(B, mb)
    summ = oracle.build_summaries(bits, table, np.zeros(B, np.int32), np.full(B, mb, np.int32))
    s = oracle.bf16_to_f32(summ)
    for b in range(B):
        for j in range(mb):
            keys = vals[table[b, j], :, 0]                       # [Hkv][bs][d]
            assert np.array_equal(s[b, :, j, 0], keys.min(axis=1))
            assert np.array_equal(s[b, :, j, 1], keys.max(axis=1))
            assert (s[b, :, j, 0][:, None, :] <= keys).all() and (keys <= s[b, :, j, 1][:, None, :]).all()
    # two summary rows per block of bs tokens of K and V: 2 / (2*bs) of the KV size (1/16 at bs=16)
    assert summ.size * 2 * bs == bits.size * 2


def test_summaries_use_keys_not_values_and_respect_range(oracle):
    rng = np.random.default_rng(2)
    B, Hkv, bs, d, mb = 1, 2, 4, 3, 5
    bits, vals = make_pool(rng, mb, Hkv, bs, d)
    bits[:, :, 1] = oracle.f32_to_bf16(np.full((mb, Hkv, bs, d), 1000.0, np.float32))   # V part
    table = np.arange(mb, dtype=np.int32).reshape(1, mb)
    summ = np.full((B, Hkv, mb, 2, d), 0x7FC0, np.uint16)                              # canary
    oracle.build_summaries(bits, table, np.array([1], np.int32), np.array([2], np.int32), summ)
    s = oracle.bf16_to_f32(summ)
    assert (np.abs(s[0, :, 1:3]) < 100).all()                      # V never enters
    assert (summ[0, :, 0] == 0x7FC0).all() and (summ[0, :, 3:] == 0x7FC0).all()  # outside the range untouched


def test_summaries_identical_keys_collapse(oracle):
    rng = np.random.default_rng(3)
    bs, d = 16, 8
    kbits, _ = rand_bf16(rng, (d,))
    pool = np.zeros((1, 1, 2, bs, d), np.uint16)
    pool[0, 0, 0] = kbits[None, :]
    summ = oracle.build_summaries(pool, np.zeros((1, 1), np.int32), [0], [1])
    assert np.array_equal(summ[0, 0, 0, 0], kbits) and np.array_equal(summ[0, 0, 0, 1], kbits)


# --------------------------------------------------------------------------- scores


def _score_setup(rng, B=2, Hq=4, Hkv=2, Td=3, d=16, bs=4, mb=7):
    bits, vals = make_pool(rng, B * mb, Hkv, bs, d)
    table = np.arange(B * mb, dtype=np.int32).reshape(B, mb)
    n_full = np.array([mb, mb - 2][:B], np.int32)
    summ = oracle_mod.build_summaries(bits, table, np.zeros(B, np.int32), n_full)
    qbits, q = rand_bf16(rng, (B, Td, Hq, d))
    return bits, vals, table, n_full, summ, qbits, q


@pytest.fixture(autouse=True)
def _bind_oracle(oracle):
    global oracle_mod
    oracle_mod = oracle


def test_score_toy_example(oracle):
    # hand-made: keys (1,-2),(3,0) -> min (1,-2), max (3,0); q = (2,-1):
    # max(2*1, 2*3) + max(-1*-2, -1*0) = 6 + 2 = 8, which bounds max(q.k) = max(4, 6) = 6
    pool = np.zeros((1, 1, 2, 2, 2), np.float32)
    pool[0, 0, 0] = [[1, -2], [3, 0]]
    bits = oracle.f32_to_bf16(pool)
    summ = oracle.build_summaries(bits, np.zeros((1, 1), np.int32), [0], [1])
    q = oracle.f32_to_bf16(np.array([2, -1], np.float32).reshape(1, 1, 1, 2))
    s32, s64 = oracle.score_blocks(q, summ, [1])
    assert s32[0, 0, 0] == 8.0 and s64[0, 0, 0] == 8.0


def test_score_equals_qplus_max_plus_qminus_min_matmul(oracle):
    """U(q,j) = q+ . M_j + q- . m_j, evaluated with numpy matmul in float64; then the
    reduce over the (t, g) rows sharing a KV head, for both reduce modes."""
    rng = np.random.default_rng(4)
    _, _, _, n_full, summ, qbits, q = _score_setup(rng)
    B, Td, Hq, d = q.shape
    Hkv, mb = summ.shape[1], summ.shape[2]
    G = Hq // Hkv
    s = oracle.bf16_to_f32(summ).astype(np.float64)
    qd = q.astype(np.float64)
    for mode in (0, 1):
        s32, s64 = oracle.score_blocks(qbits, summ, n_full, mode)
        for b in range(B):
            for h in range(Hkv):
                rows = qd[b, :, h * G:(h + 1) * G].reshape(Td * G, d)
                U = np.maximum(rows, 0) @ s[b, h, :, 1].T + np.minimum(rows, 0) @ s[b, h, :, 0].T
                want = U.max(axis=0) if mode == 0 else U.sum(axis=0)
                nf = n_full[b]
                np.testing.assert_allclose(s64[b, h, :nf], want[:nf], rtol=1e-13, atol=1e-13)
                np.testing.assert_allclose(s32[b, h, :nf], want[:nf], rtol=2e-6)
                assert np.isneginf(s32[b, h, nf:]).all() and np.isneginf(s64[b, h, nf:]).all()


def test_score_is_upper_bound_and_tight_for_identical_keys(oracle):
    rng = np.random.default_rng(5)
    bits, vals, table, n_full, summ, qbits, q = _score_setup(rng, B=1, Hq=2, Hkv=2, Td=1)
    _, s64 = oracle.score_blocks(qbits, summ, n_full)
    for h in range(2):
        for j in range(n_full[0]):
            dots = vals[table[0, j], h, 0].astype(np.float64) @ q[0, 0, h].astype(np.float64)
            assert s64[0, h, j] >= dots.max() - 1e-12
    # a block of identical keys makes the bound exact
    bs, d = 4, 16
    kb, kv = rand_bf16(rng, (d,))
    pool = np.zeros((1, 1, 2, bs, d), np.uint16)
    pool[0, 0, 0] = kb
    summ1 = oracle.build_summaries(pool, np.zeros((1, 1), np.int32), [0], [1])
    qb, qv = rand_bf16(rng, (1, 1, 1, d))
    s32, s64 = oracle.score_blocks(qb, summ1, [1])
    assert s64[0, 0, 0] == pytest.approx(float(kv.astype(np.float64) @ qv.reshape(-1).astype(np.float64)), abs=1e-12)


def test_score_unit_queries_and_power_of_two_scaling(oracle):
    rng = np.random.default_rng(6)
    _, _, _, n_full, summ, qbits, q = _score_setup(rng, B=1, Hq=1, Hkv=1, Td=1, d=8)
    s = oracle.bf16_to_f32(summ)
    for x in range(8):
        for sign in (1.0, -1.0):
            e = np.zeros((1, 1, 1, 8), np.float32)
            e[..., x] = sign
            s32, _ = oracle.score_blocks(oracle.f32_to_bf16(e), summ, n_full)
            want = s[0, 0, :, 1, x] if sign > 0 else -s[0, 0, :, 0, x]
            assert np.array_equal(s32[0, 0, :n_full[0]], want[:n_full[0]])
    base, _ = oracle.score_blocks(qbits, summ, n_full)
    scaled_q = oracle.f32_to_bf16(q * 8.0)
    big, _ = oracle.score_blocks(scaled_q, summ, n_full)
    assert np.array_equal(big[0, 0, :n_full[0]], base[0, 0, :n_full[0]] * 8.0)


def test_score_query_head_to_kv_head_mapping(oracle):
    rng = np.random.default_rng(7)
    _, _, _, n_full, summ, _, _ = _score_setup(rng, B=1, Hq=6, Hkv=3, Td=2, mb=5)
    q = np.zeros((1, 2, 6, 16), np.float32)
    q[0, 1, 3] = rng.standard_normal(16)                      # query head 3 -> KV head 3 // 2 = 1
    s32, _ = oracle.score_blocks(oracle.f32_to_bf16(q), summ, n_full)
    nf = n_full[0]
    assert (s32[0, 0, :nf] == 0).all() and (s32[0, 2, :nf] == 0).all()
    assert (s32[0, 1, :nf] != 0).all()


# --------------------------------------------------------------------------- selection


def test_select_matches_stable_sort_with_ties(oracle):
    rng = np.random.default_rng(8)
    for n, k in [(1, 1), (5, 3), (17, 17), (33, 40), (64, 9)]:
        B, Hkv, mb = 2, 2, n + 3
        scores = rng.integers(-3, 4, (B, Hkv, mb)).astype(np.float32)      # many ties
        n_full = np.array([n, max(1, n - 1)], np.int32)
        seq = (n_full * 16).astype(np.int32)
        table = np.arange(B * mb, dtype=np.int32).reshape(B, mb)
        sel = oracle.select_topk(scores, n_full, seq, 3, k, table, want_stage=False)
        for b in range(B):
            for h in range(Hkv):
                nf = n_full[b]
                order = np.argsort(-scores[b, h, :nf], kind="stable")[:min(k, nf)]
                assert np.array_equal(sel[b, h, :len(order)], order)
                assert (sel[b, h, len(order):k] == -1).all()
                assert sel[b, h, k] == nf and sel[b, h, k + 1] == -1       # one local block


def test_select_constant_scores_full_budget_and_permutation(oracle):
    n, k = 40, 12
    table = np.arange(n + 2, dtype=np.int32).reshape(1, n + 2)
    const = np.zeros((1, 1, n + 2), np.float32)
    sel = oracle.select_topk(const, [n], [n * 16], 1, k, table, want_stage=False)
    assert np.array_equal(sel[0, 0, :k], np.arange(k))
    rng = np.random.default_rng(9)
    s = rng.standard_normal((1, 1, n + 2)).astype(np.float32)
    full = oracle.select_topk(s, [n], [n * 16], 1, n + 5, table, want_stage=False)
    assert sorted(full[0, 0, :n].tolist()) == list(range(n)) and (full[0, 0, n:n + 5] == -1).all()
    assert (np.diff(s[0, 0, full[0, 0, :n]]) <= 0).all()
    perm = rng.permutation(n)
    sp = s.copy()
    sp[0, 0, :n] = s[0, 0, perm]                                            # block i now holds score of perm[i]
    selp = oracle.select_topk(sp, [n], [n * 16], 1, k, table, want_stage=False)
    sel0 = oracle.select_topk(s, [n], [n * 16], 1, k, table, want_stage=False)
    assert np.array_equal(perm[selp[0, 0, :k]], sel0[0, 0, :k])


def test_select_working_set_size_and_local_blocks(oracle):
    with open(os.path.join(GOLD, "working_set.txt")) as f:
        gold = dict(line.split("=") for line in f.read().split() if "=" in line)
    K, bs = int(gold["K"]), int(gold["block"])
    n = 512
    s = np.random.default_rng(10).standard_normal((1, 1, n + 8)).astype(np.float32)
    table = np.arange(n + 8, dtype=np.int32).reshape(1, -1)
    sel = oracle.select_topk(s, [n], [n * bs], 5, K, table, bs=bs, want_stage=False)
    kept = sel[0, 0][sel[0, 0] >= 0]
    assert len(kept) == int(gold["blocks_attended"]) and len(kept) * bs == int(gold["tokens_attended"])
    # history of n*16 + 13 tokens and 5 new ones: 13 + 5 > 16 -> two local blocks
    sel2 = oracle.select_topk(s, [n], [n * bs + 13], 5, K, table, bs=bs, want_stage=False)
    assert sel2[0, 0, K] == n and sel2[0, 0, K + 1] == n + 1
    sel3 = oracle.select_topk(s, [n], [n * bs + 11], 5, K, table, bs=bs, want_stage=False)
    assert sel3[0, 0, K] == n and sel3[0, 0, K + 1] == -1


def test_select_stage_lists(oracle):
    rng = np.random.default_rng(11)
    B, Hkv, n, k = 2, 3, 10, 4
    mb = n + 2
    s = rng.standard_normal((B, Hkv, mb)).astype(np.float32)
    table = rng.permutation(B * mb).astype(np.int32).reshape(B, mb)
    sel, idx, slots = oracle.select_topk(s, [n, n - 3], [n * 16, (n - 3) * 16 + 4], 2, k, table)
    assert np.array_equal(slots.reshape(-1), np.arange(B * Hkv * (k + 2)))
    for b in range(B):
        for h in range(Hkv):
            for c in range(k + 2):
                j = sel[b, h, c]
                assert idx[b, h, c] == (-1 if j < 0 else int(table[b, j]) * Hkv + h)


# --------------------------------------------------------------------------- gather


def test_stage_is_indexed_copy_and_leaves_other_slots(oracle):
    rng = np.random.default_rng(12)
    host, _ = rand_bf16(rng, (20, 2, 4, 8))                   # 20 entries of [2][bs=4][d=8]
    pool = np.full((9, 2, 4, 8), 0xABCD, np.uint16)
    idx = np.array([5, -1, 19, 0], np.int64)
    slots = np.array([7, 3, 0, 2], np.int32)
    oracle.stage_blocks(host, idx, slots, pool)
    assert np.array_equal(pool[[7, 0, 2]], host[[5, 19, 0]])
    assert (pool[[1, 3, 4, 5, 6, 8]] == 0xABCD).all()


# --------------------------------------------------------------------------- attention


def dense_attention_f64(q, K, V, L, scale):
    """Brute-force causal attention over contiguous K/V (no blocks, no tables).
    q [T][Hq][d], K/V [Hkv][N][d]; query t sits at position L+t and sees positions <= L+t."""
    T, Hq, d = q.shape
    Hkv = K.shape[0]
    G = Hq // Hkv
    out = np.zeros((T, Hq, d))
    lse = np.zeros((T, Hq))
    for t in range(T):
        for a in range(Hq):
            h = a // G
            n = L + t + 1
            logits = (K[h, :n].astype(np.float64) @ q[t, a].astype(np.float64)) * scale
            m = logits.max()
            w = np.exp(logits - m)
            out[t, a] = (w[:, None] * V[h, :n].astype(np.float64)).sum(0) / w.sum()
            lse[t, a] = m + math.log(w.sum())
    return out, lse


def contiguous_kv(vals, table_row, Hkv):
    """[blocks][Hkv][2][bs][d] values of one request -> K, V [Hkv][N][d]."""
    blocks = vals[table_row]                                   # [mb][Hkv][2][bs][d]
    K = np.concatenate([blocks[j, :, 0] for j in range(len(table_row))], axis=1)
    V = np.concatenate([blocks[j, :, 1] for j in range(len(table_row))], axis=1)
    return K, V


def identity_tables(B, Hkv, n_cols):
    return np.arange(B * Hkv * n_cols, dtype=np.int32).reshape(B, Hkv, n_cols)


def run_pipeline(oracle, bits, table, seq_len, n_full, qbits, k, Hkv, scale, bs):
    B, mb = table.shape
    summ = oracle.build_summaries(bits, table, np.zeros(B, np.int32), n_full)
    s32, _ = oracle.score_blocks(qbits[:, 1:], summ, n_full)
    T = qbits.shape[1]
    sel, idx, slots = oracle.select_topk(s32, n_full, seq_len, T, k, table, bs=bs)
    pool = np.zeros((B * Hkv * (k + 2),) + bits.shape[2:], np.uint16)
    oracle.stage_blocks(bits.reshape((-1,) + bits.shape[2:]), idx, slots, pool)
    res = oracle.sparse_attn(qbits, pool, identity_tables(B, Hkv, k + 2), sel, seq_len, scale, Hkv)
    return sel, res


@pytest.mark.parametrize("L0", [32, 37, 45])
def test_full_budget_pipeline_equals_dense_attention(oracle, L0):
    """With a budget that covers every full block, summaries -> scores -> top-k -> gather ->
    sparse attention must reproduce dense causal attention (Sec. 5.2: K blocks plus the
    local block; nothing else is dropped).  L0 = 45 with T = 4 needs two local blocks."""
    rng = np.random.default_rng(13 + L0)
    B, Hq, Hkv, d, bs, T = 2, 4, 2, 8, 4, 4
    mb = 16
    bits, vals = make_pool(rng, B * mb, Hkv, bs, d)
    table = rng.permutation(B * mb).astype(np.int32).reshape(B, mb)
    seq_len = np.array([L0, L0 - 9], np.int32)
    n_full = seq_len // bs
    qbits, q = rand_bf16(rng, (B, T, Hq, d))
    scale = float(np.float32(1.0 / math.sqrt(d)))          # the C side receives an fp32 scale
    sel, res = run_pipeline(oracle, bits, table, seq_len, n_full, qbits, mb, Hkv, scale, bs)
    for b in range(B):
        K, V = contiguous_kv(vals, table[b], Hkv)
        want, want_lse = dense_attention_f64(q[b], K, V, int(seq_len[b]), scale)
        np.testing.assert_allclose(res["out64"][b], want, rtol=1e-12, atol=1e-12)
        np.testing.assert_allclose(res["out32"][b], want, rtol=1e-5, atol=1e-6)
        np.testing.assert_allclose(res["lse"][b], want_lse, rtol=1e-5, atol=1e-5)
        assert np.array_equal(res["out_bf16"][b], oracle.f32_to_bf16(res["out32"][b]))


def test_sparse_attention_equals_dense_over_the_selected_keys_torch_sdpa(oracle):
    """Library second opinion: torch CPU SDPA over the gathered keys of a sparse selection."""
    rng = np.random.default_rng(20)
    B, Hq, Hkv, d, bs, T, k = 1, 4, 2, 16, 4, 1, 3
    mb = 12
    bits, vals = make_pool(rng, mb, Hkv, bs, d)
    table = np.arange(mb, dtype=np.int32).reshape(1, mb)
    seq_len = np.array([40], np.int32)                          # 10 full blocks, local block empty before the step
    n_full = seq_len // bs
    qbits, q = rand_bf16(rng, (B, T, Hq, d))
    scale = 0.375
    sel, res = run_pipeline(oracle, bits, table, seq_len, n_full, qbits, k, Hkv, scale, bs)
    assert (sel[0, :, :k] >= 0).all() and (sel[0, :, k] == 10).all()
    for a in range(Hq):
        h = a // (Hq // Hkv)
        keys, values = [], []
        for j in sel[0, h]:
            if j < 0:
                continue
            n_vis = bs if j < 10 else 1                          # local block: only the new token itself
            keys.append(vals[j, h, 0, :n_vis])
            values.append(vals[j, h, 1, :n_vis])
        Kt = torch.from_numpy(np.concatenate(keys)).double()[None, None]
        Vt = torch.from_numpy(np.concatenate(values)).double()[None, None]
        qt = torch.from_numpy(q[0, 0, a]).double()[None, None, None]
        want = torch.nn.functional.scaled_dot_product_attention(qt, Kt, Vt, scale=scale)[0, 0, 0].numpy()
        np.testing.assert_allclose(res["out64"][0, 0, a], want, rtol=1e-10, atol=1e-12)


def _single_block_attn(oracle, kvals, vvals, qvals, L, scale=1.0, blk=0):
    """One request, one KV head, blocks given explicitly as float arrays [n][bs][d]."""
    n, bs, d = kvals.shape
    pool = np.stack([kvals, vvals], axis=1).astype(np.float32)            # [n][2][bs][d]
    bits = oracle.f32_to_bf16(pool)
    q = oracle.f32_to_bf16(qvals.astype(np.float32))                       # [1][T][Hq][d]
    slot = np.arange(n, dtype=np.int32).reshape(1, 1, n)
    blkt = (np.arange(n, dtype=np.int32) + blk).reshape(1, 1, n)
    return oracle.sparse_attn(q, bits, slot, blkt, np.array([L], np.int32), scale, 1)


def test_attention_closed_forms(oracle):
    rng = np.random.default_rng(21)
    bs, d, n = 4, 8, 3
    v = rng.integers(-8, 9, (n, bs, d)).astype(np.float64)
    q = rng.integers(-3, 4, (1, 1, 2, d)).astype(np.float64)
    # all keys equal -> uniform softmax -> mean of the visible values
    k_same = np.broadcast_to(rng.integers(-2, 3, d).astype(np.float64), (n, bs, d))
    r = _single_block_attn(oracle, k_same, v, q, L=n * bs - 1)              # every position visible
    np.testing.assert_allclose(r["out64"][0, 0, 0], v.reshape(-1, d).mean(0), rtol=1e-13)
    np.testing.assert_allclose(r["lse"][0, 0], (k_same[0, 0] @ q[0, 0].T) + math.log(n * bs), rtol=1e-6)
    # causal limit: with L = 5 the query at position 5 sees positions 0..5 only
    r = _single_block_attn(oracle, k_same, v, q, L=5)
    np.testing.assert_allclose(r["out64"][0, 0, 1], v.reshape(-1, d)[:6].mean(0), rtol=1e-13)
    # one dominant key (logit 64 above the rest) -> its value
    k_dom = np.zeros((n, bs, d))
    k_dom[1, 2, 0] = 64.0
    qd = np.zeros((1, 1, 1, d))
    qd[..., 0] = 1.0
    r = _single_block_attn(oracle, k_dom, v, qd, L=n * bs - 1)
    np.testing.assert_allclose(r["out64"][0, 0, 0], v[1, 2], atol=1e-12)
    np.testing.assert_allclose(r["out32"][0, 0, 0], v[1, 2], atol=1e-6)
    # adding the same vector to every key shifts every logit equally: same output
    k_any = rng.integers(-2, 3, (n, bs, d)).astype(np.float64)
    r0 = _single_block_attn(oracle, k_any, v, q, L=n * bs - 1, scale=0.25)
    r1 = _single_block_attn(oracle, k_any + 3.0, v, q, L=n * bs - 1, scale=0.25)
    np.testing.assert_allclose(r0["out64"], r1["out64"], rtol=1e-12)


def test_attention_causal_among_verify_tokens_and_block_ids(oracle):
    """Token t of the step sits at position L+t: it sees the new tokens 0..t, not t+1.."""
    rng = np.random.default_rng(22)
    bs, d, T = 4, 8, 3
    k = rng.integers(-2, 3, (2, bs, d)).astype(np.float64)
    v = rng.integers(-8, 9, (2, bs, d)).astype(np.float64)
    q = rng.integers(-2, 3, (1, T, 1, d)).astype(np.float64)
    L = 6                                                          # blocks 1 (pos 4..7) and 2 (pos 8..11) as ids 1,2
    r = _single_block_attn(oracle, k, v, q, L=L, scale=0.5, blk=1)
    K = k.reshape(-1, d)
    V = v.reshape(-1, d)
    for t in range(T):
        n_vis = L + t + 1 - 4                                      # positions 4..L+t
        logits = K[:n_vis] @ q[0, t, 0] * 0.5
        w = np.exp(logits - logits.max())
        np.testing.assert_allclose(r["out64"][0, t, 0], (w[:, None] * V[:n_vis]).sum(0) / w.sum(), rtol=1e-12)


def test_attention_lse_merge_of_disjoint_halves(oracle):
    rng = np.random.default_rng(23)
    bs, d, n = 4, 8, 6
    k = rng.standard_normal((n, bs, d))
    v = rng.standard_normal((n, bs, d))
    q = rng.standard_normal((1, 2, 2, d))
    whole = _single_block_attn(oracle, k, v, q, L=n * bs + 5)
    a = _single_block_attn(oracle, k[:2], v[:2], q, L=n * bs + 5)
    b = _single_block_attn(oracle, k[2:], v[2:], q, L=n * bs + 5, blk=2)
    wa = np.exp(a["lse"].astype(np.float64))[..., None]
    wb = np.exp(b["lse"].astype(np.float64))[..., None]
    merged = (wa * a["out64"] + wb * b["out64"]) / (wa + wb)
    np.testing.assert_allclose(merged, whole["out64"], rtol=1e-5, atol=1e-6)
    np.testing.assert_allclose(np.log(wa + wb)[..., 0], whole["lse"], rtol=1e-5)


def test_attention_skips_padding_columns(oracle):
    rng = np.random.default_rng(24)
    bs, d = 4, 8
    k = rng.standard_normal((3, bs, d))
    v = rng.standard_normal((3, bs, d))
    q = rng.standard_normal((1, 1, 1, d))
    pool = oracle.f32_to_bf16(np.stack([k, v], axis=1).astype(np.float32))
    qb = oracle.f32_to_bf16(q.astype(np.float32))
    slot = np.array([[[0, 1, 2]]], np.int32)
    full = oracle.sparse_attn(qb, pool, slot, np.array([[[0, -1, 2]]], np.int32), [100], 1.0, 1)
    two = oracle.sparse_attn(qb, pool[[0, 2]], np.array([[[0, 1]]], np.int32),
                             np.array([[[0, 2]]], np.int32), [100], 1.0, 1)
    assert np.array_equal(full["out32"], two["out32"])
    none = oracle.sparse_attn(qb, pool, slot, np.array([[[-1, -1, -1]]], np.int32), [100], 1.0, 1)
    assert (none["out32"] == 0).all() and np.isneginf(none["lse"]).all()


# --------------------------------------------------------------------------- recall


def test_recall_extremes(oracle):
    rng = np.random.default_rng(25)
    rows, n, k = 64, 400, 40
    a = np.stack([rng.permutation(n)[:k] for _ in range(rows)]).astype(np.int32)
    pad = np.full((rows, 2), -1, np.int32)
    sel_a = np.concatenate([a, pad], axis=1)
    assert oracle.topk_recall(sel_a, sel_a, k) == 1.0
    shuffled = np.concatenate([a[:, ::-1], pad], axis=1)
    assert oracle.topk_recall(shuffled, sel_a, k) == 1.0                    # order does not matter
    b = np.stack([rng.permutation(n)[:k] for _ in range(rows)]).astype(np.int32)
    r = oracle.topk_recall(np.concatenate([b, pad], axis=1), sel_a, k)
    assert abs(r - k / n) < 0.03                                             # chance level K/n
    disjoint = np.concatenate([a + n, pad], axis=1)
    assert oracle.topk_recall(disjoint, sel_a, k) == 0.0


def test_recall_of_noiseless_drafts_is_one(oracle):
    from paper_2608_08097_b200 import synth
    cfg = synth.scaled(synth.C1, context=1024, k_blocks=16, noise=0.0)
    lay = synth.make_layer(cfg, seed=3)
    summ = oracle.build_summaries(synth.u16(lay.host_kv), lay.block_table.numpy(),
                                  np.zeros(1, np.int32), lay.n_full.numpy())
    sd, _ = oracle.score_blocks(synth.u16(lay.q[:, 1:]), summ, lay.n_full.numpy())
    st, _ = oracle.score_blocks(synth.u16(lay.q_true), summ, lay.n_full.numpy())
    args = (lay.n_full.numpy(), lay.seq_len.numpy(), cfg.n_q_tokens, cfg.k_blocks, lay.block_table.numpy())
    seld = oracle.select_topk(sd, *args, want_stage=False)
    selt = oracle.select_topk(st, *args, want_stage=False)
    assert oracle.topk_recall(seld, selt, cfg.k_blocks) == 1.0


# --------------------------------------------------------------------------- delta plan


def _plan(oracle, pred, resident, stamp, cap, step, k=None, Hkv=1):
    pred = np.asarray(pred, np.int32).reshape(1, Hkv, -1)
    k = pred.shape[-1] if k is None else k
    res = np.asarray(resident, np.int32).reshape(1, Hkv, -1).copy()
    stp = np.asarray(stamp, np.int32).reshape(1, Hkv, -1).copy()
    table = (np.arange(100, dtype=np.int32) + 1000).reshape(1, 100)
    idx, slots, n = oracle.plan_delta(pred, table, res, stp, k, cap, step, slot_stride=res.shape[-1])
    return res, stp, idx, slots, n


def test_plan_delta_hand_worked_example(oracle):
    # resident columns hold blocks 10,11,12,13 last selected at steps 5,2,7,3; prediction
    # (rank order) 12, 20, 10, 21, 22.  10 and 12 stay; 11 (stamp 2) then 13 (stamp 3) are the
    # least recently selected; cap 2 admits 20 -> column 1 and 21 -> column 3; 22 waits.
    res, stp, idx, slots, n = _plan(oracle, [12, 20, 10, 21, 22], [10, 11, 12, 13], [5, 2, 7, 3], cap=2, step=9)
    assert res.reshape(-1).tolist() == [10, 20, 12, 21]
    assert stp.reshape(-1).tolist() == [9, 9, 9, 9]
    assert n.reshape(-1).tolist() == [2]
    assert idx.reshape(-1).tolist() == [1020, 1021] and slots.reshape(-1).tolist() == [1, 3]
    # cap 1: only the best-ranked missing block comes in, into the least recently selected column
    res, stp, idx, slots, n = _plan(oracle, [12, 20, 10, 21, 22], [10, 11, 12, 13], [5, 2, 7, 3], cap=1, step=9)
    assert res.reshape(-1).tolist() == [10, 20, 12, 13] and stp.reshape(-1).tolist() == [9, 9, 9, 3]
    # cap larger than what is missing: three admissions, but only two eviction targets exist
    res, stp, idx, slots, n = _plan(oracle, [12, 20, 10, 21, 22], [10, 11, 12, 13], [5, 2, 7, 3], cap=4, step=9)
    assert n.reshape(-1).tolist() == [2] and idx.reshape(-1).tolist() == [1020, 1021, -1, -1]


def test_plan_delta_local_window(oracle):
    # two local columns after three managed ones: the ids in sel[k..k+2) are mirrored and always requested
    pred = np.array([[[7, 8, 9, 40, -1]]], np.int32)                      # k = 3, locals 40 and none
    res = np.array([[[7, 5, 6, 99, 99]]], np.int32)
    stp = np.array([[[4, 1, 2, 77, 78]]], np.int32)
    table = (np.arange(100, dtype=np.int32) + 1000).reshape(1, 100)
    idx, slots, n = oracle.plan_delta(pred, table, res, stp, 3, 1, 9, slot_stride=8, n_local=2)
    assert res.reshape(-1).tolist() == [7, 8, 6, 40, -1]                   # 8 replaces the oldest (block 5)
    assert stp.reshape(-1).tolist() == [9, 9, 2, 77, 78]                   # local stamps untouched
    assert idx.reshape(-1).tolist() == [1008, 1040, -1] and slots.reshape(-1).tolist()[:2] == [1, 3]
    assert slots.reshape(-1).tolist()[2] == 4 and n.reshape(-1).tolist() == [1]


def test_plan_delta_invariants(oracle):
    rng = np.random.default_rng(26)
    Hkv, k, n_res, nblk = 3, 12, 12, 60
    res = np.full((1, Hkv, n_res), -1, np.int32)
    stp = np.zeros((1, Hkv, n_res), np.int32)
    table = rng.permutation(nblk).astype(np.int32).reshape(1, nblk)
    # cold start with an unbounded cap: the resident set becomes the prediction
    pred = np.stack([rng.permutation(nblk)[:k] for _ in range(Hkv)]).astype(np.int32).reshape(1, Hkv, k)
    idx, slots, n = oracle.plan_delta(pred, table, res, stp, k, k, 1, n_res)
    assert (n == k).all()
    for h in range(Hkv):
        assert sorted(res[0, h].tolist()) == sorted(pred[0, h].tolist())
        assert np.array_equal(idx[0, h], table[0, pred[0, h]].astype(np.int64) * Hkv + h)
        assert np.array_equal(slots[0, h], h * n_res + np.arange(k))       # empty columns fill in order
    for step in range(2, 12):
        cap = int(rng.integers(0, 5))
        pred = np.stack([rng.permutation(nblk)[:k] for _ in range(Hkv)]).astype(np.int32).reshape(1, Hkv, k)
        before, before_stamp = res.copy(), stp.copy()
        idx, slots, n = oracle.plan_delta(pred, table, res, stp, k, cap, step, n_res)
        for h in range(Hkv):
            P, R0 = set(pred[0, h].tolist()), before[0, h]
            missing = [j for j in pred[0, h] if j not in set(R0.tolist())]
            outside = [c for c in range(n_res) if R0[c] not in P]
            assert n[0, h] == min(cap, len(missing), len(outside))
            assert len(set(res[0, h].tolist())) == n_res                      # no duplicates
            changed = np.nonzero(res[0, h] != R0)[0]
            assert len(changed) == n[0, h] and set(changed.tolist()) <= set(outside)
            assert sorted(res[0, h][changed].tolist()) == sorted(missing[:n[0, h]])   # best-ranked first
            # evicted columns are the least recently selected ones among those outside the prediction
            if len(changed):
                worst_evicted = before_stamp[0, h][changed].max()
                kept_outside = [c for c in outside if c not in set(changed.tolist())]
                assert all(before_stamp[0, h][c] >= worst_evicted for c in kept_outside)
            hits = [c for c in range(n_res) if R0[c] in P]
            assert (stp[0, h][hits] == step).all() and (stp[0, h][changed] == step).all()
            untouched = [c for c in outside if c not in set(changed.tolist())]
            assert np.array_equal(stp[0, h][untouched], before_stamp[0, h][untouched])


def test_union_blocks_matches_numpy_unique(oracle):
    rng = np.random.default_rng(27)
    B, Hkv, k, nblk = 3, 4, 9, 50
    sel = np.stack([np.stack([rng.permutation(nblk)[:k] for _ in range(Hkv)]) for _ in range(B)]).astype(np.int32)
    sel = np.concatenate([sel, np.full((B, Hkv, 2), 7, np.int32)], axis=2)          # local columns are not part of it
    sel[1, 2, 3:6] = -1                                                              # unused ranks
    sel[2, :, :k] = sel[2, 0:1, :k]                                                  # all heads agree: the union is one set
    idx, n = oracle.union_blocks(sel, k, nblk, Hkv * k)
    for b in range(B):
        want = np.unique(sel[b, :, :k][sel[b, :, :k] >= 0])
        assert n[b] == len(want) and np.array_equal(idx[b, :n[b]], want) and (idx[b, n[b]:] == -1).all()
    assert n[2] == k and k <= n[0] <= Hkv * k
    # a list shorter than the union: truncated, but the count is the true size
    idx2, n2 = oracle.union_blocks(sel, k, nblk, 5)
    assert np.array_equal(idx2[0], idx[0, :5]) and n2[0] == n[0]


def test_fetch_cap_reading_against_the_papers_table(oracle):
    """Table 'Fetch-cap ablation' (Sec. 5.5.1): GB per step, GB/s and tok/s per fetch ratio.
    With one committed token per request per step, requests = tok/s * (GB per step / GB/s).
    Bytes per request per step must equal layers * KV heads * C * entry bytes with
    C = floor(ratio * K) and an 8 KiB (16 tokens x 128 dims x K,V x bf16) entry."""
    rows = []
    with open(os.path.join(GOLD, "fetch_cap_table.txt")) as f:
        for line in f:
            if line.startswith("#") or not line.strip():
                continue
            ratio, gb_step, gbs, tps = (float(x) for x in line.split())
            rows.append((ratio, gb_step, gbs, tps))
    layers, heads, K, entry = 36, 8, 128, 16 * 128 * 2 * 2
    for ratio, gb_step, gbs, tps in rows:
        if ratio > 0.021:
            continue                                   # beyond that the cap no longer binds every head
        requests = tps * (gb_step / gbs)
        per_request = gb_step * 1e9 / requests
        C = math.floor(ratio * K)
        assert per_request == pytest.approx(layers * heads * C * entry, rel=0.05)
        assert per_request != pytest.approx(layers * heads * math.ceil(ratio * K) * entry, rel=0.2)


def test_kv_footprint_worked_numbers():
    """Eq. 1-2 and the worked numbers below them: 256 KiB per token, about 8.6 GB at 32.7K
    tokens, nine requests in 80 GB -- pins the bytes-per-token accounting (K and V, bf16)."""
    with open(os.path.join(GOLD, "kv_footprint.txt")) as f:
        gold = dict(line.split("=") for line in f.read().split() if "=" in line)
    layers, n_kv, d_h, s = 64, 8, 128, 2                    # the 32B-class GQA model of Sec. 2.1
    per_token = layers * 2 * n_kv * d_h * s
    assert per_token == int(gold["per_token_KiB"]) * 1024
    req = per_token * float(gold["context_tokens"])
    assert req / 1e9 == pytest.approx(float(gold["request_GB"]), abs=0.05)
    assert math.floor(float(gold["hbm_GB"]) / float(gold["request_GB"])) == int(gold["b_max"])


# --------------------------------------------------------------------------- dense -> sparse hand-over


def _handover_case(rng, B=3, Hkv=4, bs=16, d=128, mb=12):
    Pg, Pc = B * mb + 5, B * mb + 7
    kb, kf = rand_bf16(rng, (Pg, Hkv, bs, d))
    vb, _ = rand_bf16(rng, (Pg, Hkv, bs, d))
    gpu_table = rng.permutation(Pg)[:B * mb].reshape(B, mb).astype(np.int32)
    cpu_table = rng.permutation(Pc)[:B * mb].reshape(B, mb).astype(np.int32)
    return kb, kf, vb, gpu_table, cpu_table, Pc


def test_offload_matches_numpy_definition_and_leaves_other_entries_alone(oracle):
    """Entry (cpu block, head) = [K | V] of (gpu block, head), written out with numpy fancy indexing;
    entries outside the requested ranges keep their canary."""
    rng = np.random.default_rng(70)
    kb, _, vb, gt, ct, Pc = _handover_case(rng)
    B, mb = gt.shape
    Hkv = kb.shape[1]
    first = np.array([0, 3, 5], np.int32)
    n = np.array([mb, 4, 0], np.int32)                              # whole request / a middle range / nothing
    host = np.full((Pc, Hkv, 2, 16, 128), 0xBEEF, np.uint16)
    oracle.offload_blocks(kb, vb, gt, ct, first, n, host)
    want = np.full_like(host, 0xBEEF)
    for b in range(B):
        js = np.arange(first[b], first[b] + n[b])
        want[ct[b, js]] = np.stack([kb[gt[b, js]], vb[gt[b, js]]], axis=2)
    assert np.array_equal(host, want)
    # a transposed K / V or a swapped table would show here: the two halves differ and the tables are permutations
    assert not np.array_equal(kb, vb) and not np.array_equal(gt, ct)


def test_offload_then_gather_returns_the_dense_blocks(oracle):
    """Round trip: what the hand-over wrote to the CPU pool, gathered back by step 3, is the dense data."""
    rng = np.random.default_rng(71)
    kb, _, vb, gt, ct, Pc = _handover_case(rng, B=2, Hkv=2, mb=6)
    B, mb = gt.shape
    Hkv = kb.shape[1]
    host = np.zeros((Pc, Hkv, 2, 16, 128), np.uint16)
    oracle.offload_blocks(kb, vb, gt, ct, np.zeros(B, np.int32), np.full(B, mb, np.int32), host)
    b, h = 1, 1
    idx = (ct[b].astype(np.int64) * Hkv + h)
    pool = np.zeros((mb, 2, 16, 128), np.uint16)
    oracle.stage_blocks(host.reshape(-1, 2, 16, 128), idx, np.arange(mb, dtype=np.int32), pool)
    assert np.array_equal(pool[:, 0], kb[gt[b], h]) and np.array_equal(pool[:, 1], vb[gt[b], h])


def test_offload_summaries_are_the_min_and_max_of_the_copied_keys(oracle):
    rng = np.random.default_rng(72)
    kb, kf, vb, gt, ct, Pc = _handover_case(rng)
    B, mb = gt.shape
    Hkv = kb.shape[1]
    first = np.array([0, 2, 1], np.int32)
    n = np.array([mb, 5, 20], np.int32)                             # the last range runs past max_blocks: clipped
    host = np.zeros((Pc, Hkv, 2, 16, 128), np.uint16)
    summ = np.full((B, Hkv, mb, 2, 128), 0x7FC0, np.uint16)         # NaN canary
    oracle.offload_blocks(kb, vb, gt, ct, first, n, host, summ)
    got = oracle.bf16_to_f32(summ)
    for b in range(B):
        for j in range(mb):
            inside = first[b] <= j < first[b] + n[b]
            for h in range(Hkv):
                if inside:
                    keys = kf[gt[b, j], h]                          # [16][128]
                    assert np.array_equal(got[b, h, j, 0], keys.min(axis=0))
                    assert np.array_equal(got[b, h, j, 1], keys.max(axis=0))
                else:
                    assert np.all(summ[b, h, j] == 0x7FC0)
    # and they agree with step 0 run on the pool the hand-over filled
    again = oracle.build_summaries(host, ct, np.zeros(B, np.int32), np.full(B, mb, np.int32))
    sel = [(b, j) for b in range(B) for j in range(mb) if first[b] <= j < first[b] + n[b]]
    for b, j in sel:
        assert np.array_equal(summ[b, :, j], again[b, :, j])


# --------------------------------------------------------------------------- local window, KV append


def test_local_window_hand_worked_columns_and_requests(oracle):
    """bs = 16, T = 3, local columns 4 and 5 (block parity picks the column).
    L = 30: tokens at 30, 31 (block 1) and 32 (block 2)  -> column 5 = block 1, column 4 = block 2.
    L = 32: tokens 32..34, all in block 2                -> column 4 = block 2, column 5 = -1.
    L = 45: tokens 45..47, all in block 2                -> as before (a block keeps its column).
    L = 46: tokens 46, 47 (block 2) and 48 (block 3)     -> column 4 = block 2, column 5 = block 3."""
    Hkv, n_cols, mb = 2, 6, 8
    seq = np.array([30, 32, 45, 46], np.int32)
    table = (np.arange(4 * mb, dtype=np.int32).reshape(4, mb) * 3 + 1)            # some non-identity table
    blk = np.full((4, Hkv, n_cols), 77, np.int32)
    idx, slots = oracle.local_window(seq, 3, table, blk, 4, 10)
    assert blk[:, :, :4].tolist() == np.full((4, Hkv, 4), 77).tolist()            # other columns untouched
    assert blk[:, 0, 4:].tolist() == [[2, 1], [2, -1], [2, -1], [2, 3]]
    assert np.array_equal(blk[:, 0], blk[:, 1])
    for b, (c4, c5) in enumerate([(2, 1), (2, -1), (2, -1), (2, 3)]):
        for h in range(Hkv):
            row = b * Hkv + h
            assert slots[b, h].tolist() == [row * 10 + 4, row * 10 + 5]
            want = [(table[b, j] * Hkv + h) if j >= 0 else -1 for j in (c4, c5)]
            assert idx[b, h].tolist() == want


def _token_stream(rng, n_tok, Hkv, d):
    """A contiguous per-request K/V sequence [n_tok][Hkv][2][d] as (bits, values)."""
    return rand_bf16(rng, (n_tok, Hkv, 2, d))


def test_append_over_many_steps_rebuilds_the_blocks_in_the_cpu_pool(oracle):
    """Tokens appended one committed token per step (T = 5 written, 1 committed) over 40 steps: every position
    that was committed must sit in the CPU pool exactly where a plain numpy reshape of the contiguous token
    sequence into [block][head][K,V][row][dim] puts it, nothing else in the CPU pool may change, and the GPU
    working set's local slots must hold the tokens written last at each position."""
    rng = np.random.default_rng(5)
    B, Hkv, d, bs, T, mb, k = 2, 3, 8, 16, 5, 8, 2
    n_cols, steps = k + 2, 40
    L0 = np.array([21, 48], np.int32)
    table = rng.permutation(B * mb).astype(np.int32).reshape(B, mb)
    n_tok = mb * bs
    sbits, _ = _token_stream(rng, B * n_tok, Hkv, d)
    sbits = sbits.reshape(B, n_tok, Hkv, 2, d)
    # the layout a reshape gives: [block][row][head][part][d] -> [block][head][part][row][d]
    want_blocks = sbits.reshape(B, mb, bs, Hkv, 2, d).transpose(0, 1, 3, 4, 2, 5)
    canary = np.uint16(0xABCD)
    host = np.full((B * mb, Hkv, 2, bs, d), canary, np.uint16)
    pool = np.full((B * Hkv * n_cols, 2, bs, d), canary, np.uint16)
    slot_tbl = rng.permutation(B * Hkv * n_cols).astype(np.int32).reshape(B, Hkv, n_cols)
    blk = np.full((B, Hkv, n_cols), -1, np.int32)
    latest = {}                                     # (b, position) -> step that wrote it last
    for s in range(steps):
        seq = (L0 + s).astype(np.int32)
        new = np.stack([sbits[b, seq[b]:seq[b] + T] for b in range(B)])           # [B][T][Hkv][2][d]
        new = new + np.uint16(s % 3)                # drafts differ from what is committed later (bit noise)
        new[:, 0] = np.stack([sbits[b, seq[b]] for b in range(B)])                # the committed token is the true one
        oracle.append_kv(new, 1, seq, table, slot_tbl, blk, k, pool, host)
        for b in range(B):
            lo, hi = seq[b] // bs, (seq[b] + T - 1) // bs
            assert blk[b, 0, k + (lo & 1)] == lo
            assert blk[b, 0, k + 1 - (lo & 1)] == (hi if hi > lo else -1)
            for t in range(T):
                latest[(b, int(seq[b]) + t)] = (s, t, new[b, t].copy())
    for b in range(B):
        first, last = int(L0[b]), int(L0[b]) + steps - 1
        for j in range(mb):
            got = host[table[b, j]]                                               # [Hkv][2][bs][d]
            for i in range(bs):
                p = j * bs + i
                if first <= p <= last:
                    assert np.array_equal(got[:, :, i], want_blocks[b, j][:, :, i]), (b, p)
                else:
                    assert (got[:, :, i] == canary).all(), (b, p)
        # local slots: the last two local blocks hold, row by row, what was written last
        seq = int(L0[b]) + steps - 1
        for j in range(seq // bs, (seq + T - 1) // bs + 1):
            for h in range(Hkv):
                e = pool[slot_tbl[b, h, k + (j & 1)]]
                for i in range(bs):
                    p = j * bs + i
                    if (b, p) in latest and p >= seq - bs:     # still inside the two-block window
                        assert np.array_equal(e[:, i], latest[(b, p)][2][h]), (b, p, h)
    # slots of the k selected columns were never touched
    for b in range(B):
        for h in range(Hkv):
            for c in range(k):
                assert (pool[slot_tbl[b, h, c]] == canary).all()


@pytest.mark.parametrize("L0", [33, 45, 47])
def test_append_then_attention_equals_dense_attention(oracle, L0):
    """The local window written by the append (not gathered from the CPU pool) together with a full budget of
    gathered blocks must reproduce brute-force dense causal attention over the contiguous token sequence;
    L0 = 45 and 47 with T = 4 put tokens into two local blocks, and the steps before cross a block boundary."""
    rng = np.random.default_rng(17 + L0)
    B, Hq, Hkv, d, bs, T = 2, 4, 2, 8, 16, 4
    mb, k = 6, 6
    n_cols = k + 2
    n_tok = mb * bs
    sbits, svals = _token_stream(rng, B * n_tok, Hkv, d)
    sbits, svals = sbits.reshape(B, n_tok, Hkv, 2, d), svals.reshape(B, n_tok, Hkv, 2, d)
    table = rng.permutation(B * mb).astype(np.int32).reshape(B, mb)
    host = np.zeros((B * mb, Hkv, 2, bs, d), np.uint16)
    pool = np.zeros((B * Hkv * n_cols, 2, bs, d), np.uint16)
    slot_tbl = identity_tables(B, Hkv, n_cols)
    blk = np.full((B, Hkv, n_cols), -1, np.int32)
    start = np.array([L0 - 20, L0 - 20 - 7], np.int32)
    # history before `start` is already in the CPU pool (as after a hand-over)
    for b in range(B):
        for p in range(int(start[b])):
            host[table[b, p // bs], :, :, p % bs] = sbits[b, p]
    # the partially filled block at `start` is loaded into its local slot once
    idx, slots = oracle.local_window(start, T, table, blk, k, n_cols)
    oracle.stage_blocks(host.reshape(-1, 2, bs, d), idx, slots, pool)
    scale = float(np.float32(1.0 / math.sqrt(d)))
    qbits, q = rand_bf16(rng, (B, T, Hq, d))
    for s in range(21):
        seq = (start + s).astype(np.int32)
        new = np.stack([sbits[b, seq[b]:seq[b] + T] for b in range(B)])
        oracle.append_kv(new, 1, seq, table, slot_tbl, blk, k, pool, host)
        # full budget: every full block is selected and gathered from the CPU pool
        n_full = seq // bs
        for b in range(B):
            for h in range(Hkv):
                blk[b, h, :k] = -1
                blk[b, h, :n_full[b]] = np.arange(n_full[b])
        gidx = np.where(blk[:, :, :k] < 0, -1,
                        np.take_along_axis(np.broadcast_to(table[:, None, :], (B, Hkv, mb)), np.maximum(blk[:, :, :k], 0), axis=2)
                        .astype(np.int64) * Hkv + np.arange(Hkv)[None, :, None])
        oracle.stage_blocks(host.reshape(-1, 2, bs, d), gidx, slot_tbl[:, :, :k].copy(), pool)
        res = oracle.sparse_attn(qbits, pool, slot_tbl, blk, seq, scale, Hkv)
        for b in range(B):
            K = svals[b, :, :, 0].transpose(1, 0, 2)
            V = svals[b, :, :, 1].transpose(1, 0, 2)
            want, want_lse = dense_attention_f64(q[b], K, V, int(seq[b]), scale)
            np.testing.assert_allclose(res["out64"][b], want, rtol=1e-12, atol=1e-12)
            np.testing.assert_allclose(res["lse"][b], want_lse, rtol=1e-5, atol=1e-5)


# --------------------------------------------------------------------------- attention mass per block


def test_block_mass_equals_dense_softmax_summed_per_block(oracle):
    """Brute force with numpy on contiguous keys: softmax over the visible prefix, reshaped into blocks and
    summed, then the maximum over the query rows that share the KV head."""
    rng = np.random.default_rng(29)
    B, Tq, Hq, Hkv, d, bs, mb = 2, 3, 4, 2, 8, 4, 9
    bits, vals = make_pool(rng, B * mb, Hkv, bs, d)
    table = rng.permutation(B * mb).astype(np.int32).reshape(B, mb)
    seq = np.array([22, 13], np.int32)
    qbits, q = rand_bf16(rng, (B, Tq, Hq, d), scale=2.0)
    scale = float(np.float32(0.37))
    got = oracle.block_mass(qbits, bits, table, seq, scale)
    G = Hq // Hkv
    for b in range(B):
        K, _ = contiguous_kv(vals, table[b], Hkv)                       # [Hkv][mb*bs][d]
        want = np.zeros((Hkv, mb))
        for t in range(Tq):
            n = int(seq[b]) + t + 1
            for a in range(Hq):
                h = a // G
                logits = (K[h, :n].astype(np.float64) @ q[b, t, a].astype(np.float64)) * scale
                w = np.exp(logits - logits.max())
                prob = np.zeros(mb * bs)
                prob[:n] = w / w.sum()
                want[h] = np.maximum(want[h], prob.reshape(mb, bs).sum(1))
        np.testing.assert_allclose(got[b], want, rtol=1e-12, atol=1e-15)


def test_block_mass_closed_form_for_identical_keys(oracle):
    """All keys equal: every visible key gets 1/n, so a full block's mass is bs/n for the row that sees the
    fewest keys (t = 0, the maximum over rows), and the partially visible last block gets its visible share
    at the row that sees the most."""
    B, Tq, Hq, Hkv, d, bs, mb = 1, 2, 2, 1, 4, 4, 5
    key = rand_bf16(np.random.default_rng(1), (d,))[0]
    bits = np.zeros((mb, Hkv, 2, bs, d), np.uint16)
    bits[:, :, 0] = key
    table = np.arange(mb, dtype=np.int32).reshape(1, mb)
    seq = np.array([13], np.int32)                                       # rows see 14 and 15 keys
    qbits, _ = rand_bf16(np.random.default_rng(2), (B, Tq, Hq, d))
    got = oracle.block_mass(qbits, bits, table, seq, 1.0)[0, 0]
    np.testing.assert_allclose(got, [4 / 14, 4 / 14, 4 / 14, 3 / 15, 0.0], rtol=1e-12)


def test_attention_abs_weighted_output(oracle):
    """out_abs = sum_p softmax_p |v_p|: equals the output itself when no value is negative, never lies below
    |output|, and equals the brute-force sum on contiguous keys."""
    rng = np.random.default_rng(41)
    B, Hq, Hkv, d, bs, T, mb = 1, 2, 1, 8, 4, 2, 5
    bits, vals = make_pool(rng, mb, Hkv, bs, d)
    table = np.arange(mb, dtype=np.int32).reshape(1, mb)
    seq = np.array([14], np.int32)
    qbits, q = rand_bf16(rng, (B, T, Hq, d))
    blk = np.arange(mb, dtype=np.int32).reshape(1, 1, mb)
    slots = np.arange(mb, dtype=np.int32).reshape(1, 1, mb)
    res = oracle.sparse_attn(qbits, bits.reshape(-1, 2, bs, d), slots, blk, seq, 0.5, Hkv)
    assert (res["out_abs"] >= np.abs(res["out64"]) - 1e-15).all()
    K, V = contiguous_kv(vals, table[0], Hkv)
    for t in range(T):
        for a in range(Hq):
            n = int(seq[0]) + t + 1
            logits = (K[0, :n].astype(np.float64) @ q[0, t, a].astype(np.float64)) * 0.5
            w = np.exp(logits - logits.max())
            want = (w[:, None] * np.abs(V[0, :n].astype(np.float64))).sum(0) / w.sum()
            np.testing.assert_allclose(res["out_abs"][0, t, a], want, rtol=1e-12)
    pos_bits = bits.copy()
    pos_bits[:, :, 1] &= 0x7fff                                         # clear the sign bit of every value
    res2 = oracle.sparse_attn(qbits, pos_bits.reshape(-1, 2, bs, d), slots, blk, seq, 0.5, Hkv)
    np.testing.assert_allclose(res2["out_abs"], res2["out64"], rtol=1e-12)
