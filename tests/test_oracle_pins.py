"""Pins of the CPU oracle against things other than itself (no GPU needed).

Each test checks one oracle function against a closed form, an invariant, a library routine
(torch SDPA on the CPU, numpy reductions), a hand-derived fixture or brute-force enumeration,
chosen so that a dropped term, a wrong sign or index, or a transposed operand fails somewhere.
"""
import itertools
import math
from pathlib import Path

import numpy as np
import pytest
import torch

import oracle
from paper_2512_02337_b200 import workloads as wl

GOLDEN = Path(__file__).resolve().parent / "golden"


def bf16_bits(x: np.ndarray) -> np.ndarray:
    return wl.to_numpy(torch.from_numpy(np.asarray(x, dtype=np.float32)).to(torch.bfloat16))


def make_cache(rng, n_blocks, Hkv, bs, d, dtype="fp32", shuffle=False, extra_pages=0):
    n_pages = n_blocks + extra_pages
    k = rng.standard_normal((n_pages, Hkv, bs, d)).astype(np.float32)
    v = rng.standard_normal((n_pages, Hkv, bs, d)).astype(np.float32)
    table = np.arange(n_blocks, dtype=np.int32)
    if shuffle:
        table = rng.permutation(n_pages)[:n_blocks].astype(np.int32)
    if dtype == "bf16":
        k, v = bf16_bits(k), bf16_bits(v)
    return k, v, table


def logical_tokens(pool, table, seq_len):
    """[seq_len][Hkv][d] float64 view of a paged pool (test-side helper, plain indexing)."""
    w = oracle.widen(pool)
    bs = pool.shape[2]
    return np.stack([w[table[t // bs], :, t % bs, :] for t in range(seq_len)])


# ----------------------------------------------------------------------------- tree mask
def test_tree_mask_golden_fixture():
    vals = {}
    for line in (GOLDEN / "tree_mask_small.txt").read_text().splitlines():
        if line and not line.startswith("#"):
            key, *rest = line.split()
            vals[key] = [int(x, 0) for x in rest]
    parents = np.array(vals["parents"], dtype=np.int32)
    assert oracle.tree_mask(parents)[:, 0].tolist() == vals["mask"]
    assert oracle.tree_mask(parents, n_chain=vals["chain"][0])[:, 0].tolist() == vals["mask_chain"]


@pytest.mark.parametrize("M,depth,branch,chain", [(16, 4, 4, 0), (60, 6, 4, 0), (64, 6, 4, 0),
                                                  (48, 5, 4, 42), (100, 8, 3, 27), (1, 0, 1, 0)])
def test_tree_mask_brute_force_parent_walk(M, depth, branch, chain):
    rng = np.random.default_rng(M * 131 + chain)
    parents = wl.make_tree(M, depth, branch, rng)
    mask = oracle.tree_mask(parents, n_chain=chain)
    total = M + chain
    combined = np.concatenate([np.arange(-1, chain - 1), np.where(parents < 0, chain - 1, parents + chain)])
    for j in range(total):
        seen = set()
        a = j
        while a >= 0:
            seen.add(a)
            a = int(combined[a])
        got = {a for a in range(total) if (int(mask[j, a // 64]) >> (a % 64)) & 1}
        assert got == seen


def test_tree_mask_chain_is_lower_triangular_and_bad_tree_rejected():
    M = 70
    mask = oracle.tree_mask(np.arange(-1, M - 1, dtype=np.int32))
    for j in range(M):
        for a in range(M):
            assert ((int(mask[j, a // 64]) >> (a % 64)) & 1) == (a <= j)
    with pytest.raises(ValueError):
        oracle.tree_mask(np.array([-1, 2, 1], dtype=np.int32))
    with pytest.raises(ValueError):
        oracle.tree_mask(np.array([-1, -1], dtype=np.int32))


# ----------------------------------------------------------------------------- Eq. 1 summaries
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_block_summaries_match_numpy_reductions(dtype):
    rng = np.random.default_rng(1)
    bs, Hkv, d, seq_len = 16, 3, 8, 16 * 5 + 7  # ragged last block
    k, _, table = make_cache(rng, 6, Hkv, bs, d, dtype, shuffle=True, extra_pages=3)
    kmax, kmin = oracle.block_summaries(k, table, seq_len)
    toks = logical_tokens(k, table, seq_len)
    for i in range(6):
        blk = toks[i * bs:min((i + 1) * bs, seq_len)]
        assert np.array_equal(kmax[:, i], blk.max(axis=0))
        assert np.array_equal(kmin[:, i], blk.min(axis=0))
    assert np.all(kmax >= kmin)


# ----------------------------------------------------------------------------- Eq. 2-3 scores
def test_block_scores_closed_form_constant_blocks():
    # all keys of a block identical => Kmax = Kmin = k and s_{i,j} = q_j . k exactly (Eq. 2 collapses)
    rng = np.random.default_rng(2)
    Hq, Hkv, d, nb, M = 4, 2, 8, 5, 3
    keys = rng.integers(-4, 5, size=(Hkv, nb, d)).astype(np.float64)
    q = rng.integers(-4, 5, size=(M, Hq, d)).astype(np.float32)
    s = oracle.block_scores(q, keys, keys, Hkv, reduce=0)
    G = Hq // Hkv
    for h in range(Hkv):
        for i in range(nb):
            rows = [float(q[j, h * G + g].astype(np.float64) @ keys[h, i]) for j in range(M) for g in range(G)]
            assert s[h, i] == pytest.approx(np.mean(rows), abs=1e-12)
            assert oracle.block_scores(q, keys, keys, Hkv, reduce=1)[h, i] == max(rows)


@pytest.mark.parametrize("reduce", [0, 1, 2])
def test_block_scores_match_independent_einsum(reduce):
    rng = np.random.default_rng(3)
    Hq, Hkv, d, nb, M = 8, 2, 16, 7, 5
    G = Hq // Hkv
    kmax = rng.standard_normal((Hkv, nb, d))
    kmin = kmax - np.abs(rng.standard_normal((Hkv, nb, d)))
    q = bf16_bits(rng.standard_normal((M, Hq, d)))
    qw = oracle.widen(q).reshape(M, Hkv, G, d)
    per_query = np.maximum(np.einsum("mhgc,hic->hmgi", qw, kmax), np.einsum("mhgc,hic->hmgi", qw, kmin))
    last = 3
    want = {0: per_query.mean(axis=(1, 2)), 1: per_query.max(axis=(1, 2)),
            2: per_query[:, last].mean(axis=1)}[reduce]
    got = oracle.block_scores(q, kmax, kmin, Hkv, reduce=reduce, last_query=last)
    np.testing.assert_allclose(got, want, rtol=1e-12, atol=1e-12)


def test_channelwise_scores_closed_form_bound_and_separation():
    """score_mode 1 (the channel-wise form of Quest, cited by Section 3.2): three pins that do not retype it."""
    rng = np.random.default_rng(21)
    M, Hq, Hkv, d, nb, bs = 5, 4, 2, 16, 6, 8
    G = Hq // Hkv
    q = rng.standard_normal((M, Hq, d)).astype(np.float32)
    keys = rng.standard_normal((Hkv, nb, bs, d))
    kmax, kmin = keys.max(axis=2), keys.min(axis=2)
    got = oracle.block_scores(q, kmax, kmin, Hkv, reduce=1, score_mode=1)  # max over the rows
    qw = q.astype(np.float64).reshape(M, Hkv, G, d)
    # (a) sign split: for q_c >= 0 the channel takes Kmax, for q_c < 0 it takes Kmin, so the score is two plain
    #     contractions, q+ . Kmax + q- . Kmin
    split = np.einsum("mhgc,hic->hmgi", np.maximum(qw, 0), kmax) + np.einsum("mhgc,hic->hmgi", np.minimum(qw, 0), kmin)
    np.testing.assert_allclose(got, split.max(axis=(1, 2)), rtol=1e-12, atol=1e-12)
    # (b) it bounds the true score of every key of the block from above (the reason Quest uses it)
    true = np.einsum("mhgc,hitc->hmgit", qw, keys)
    assert np.all(split[..., None] >= true - 1e-12)
    # (c) it is never below Eq. 2 as printed, and strictly above when the channels disagree in sign
    printed = oracle.block_scores(q, kmax, kmin, Hkv, reduce=1, score_mode=0)
    assert np.all(got >= printed - 1e-12) and np.any(got > printed + 1e-6)
    one = oracle.block_scores(np.array([[[1.0, -1.0]]], dtype=np.float32), np.array([[[1.0, 1.0]]]),
                              np.array([[[0.0, 0.0]]]), 1, score_mode=1)
    assert one[0, 0] == 1.0  # 1*1 + max(-1*1, -1*0) = 1, where the printed form gives 0
    # blocks of one repeated key: both forms equal q . k
    same = np.repeat(keys[:, :, :1], bs, axis=2)
    eq = oracle.block_scores(q, same.max(axis=2), same.min(axis=2), Hkv, reduce=0, score_mode=1)
    np.testing.assert_allclose(eq, np.einsum("mhgc,hic->hmgi", qw, same[:, :, 0]).mean(axis=(1, 2)), rtol=1e-12, atol=1e-12)


def test_block_scores_is_max_of_full_dot_products_not_channelwise():
    # q = (1, -1), Kmax = (1, 1), Kmin = (0, 0): Eq. 2 as printed gives max(0, 0) = 0,
    # the channel-wise variant would give 1*1 + (-1)*0 = 1.
    q = np.array([[[1.0, -1.0]]], dtype=np.float32)
    kmax = np.array([[[1.0, 1.0]]])
    kmin = np.array([[[0.0, 0.0]]])
    assert oracle.block_scores(q, kmax, kmin, 1)[0, 0] == 0.0
    # and the max really picks the larger product: q = (-1,-1) => max(-2, 0) = 0 ; q = (1,1) => 2
    assert oracle.block_scores(-np.abs(q), kmax, kmin, 1)[0, 0] == 0.0
    assert oracle.block_scores(np.abs(q), kmax, kmin, 1)[0, 0] == 2.0


# ----------------------------------------------------------------------------- selection
def brute_force_select(scores, sink, local, budget):
    nb = len(scores)
    if nb <= budget:
        return list(range(nb))
    cand = list(range(sink, nb - local))
    k = budget - sink - local
    best = None
    for sub in itertools.combinations(cand, k):  # ascending tuples, lexicographic order
        total = sum(scores[i] for i in sub)
        if best is None or total > best[0]:
            best = (total, sub)
    return list(range(sink)) + list(best[1]) + list(range(nb - local, nb))


@pytest.mark.parametrize("seed", range(6))
def test_select_equals_best_subset_enumeration(seed):
    rng = np.random.default_rng(seed)
    nb, sink, local, budget = 12, 1, 2, 7
    # distinct dyadic scores: subset sums are exact and the best subset is unique
    scores = rng.permutation(nb).astype(np.float64) / 4.0 - 1.0
    got = oracle.select(scores, sink, local, budget).tolist()
    assert got == brute_force_select(scores, sink, local, budget)
    assert got == sorted(got) and len(set(got)) == budget
    assert got[:sink] == list(range(sink)) and got[-local:] == list(range(nb - local, nb))


def test_select_ties_nan_and_small_contexts():
    # ties -> lower index (also the lexicographically smallest best subset)
    scores = np.array([9, 1, 1, 1, 1, 1, 9, 9], dtype=np.float64)
    assert oracle.select(scores, 1, 2, 5).tolist() == [0, 1, 2, 6, 7]
    assert oracle.select(scores, 1, 2, 5).tolist() == brute_force_select(scores, 1, 2, 5)
    # sink/local scores are irrelevant; a high score inside the candidate range wins
    scores = np.array([-100, 0, 5, 0, 7, 0, -100, -100], dtype=np.float64)
    assert oracle.select(scores, 1, 2, 5).tolist() == [0, 2, 4, 6, 7]
    # NaN ranks below every number, including -inf
    scores = np.array([0, np.nan, -np.inf, 3, np.nan, 0, 0], dtype=np.float64)
    assert oracle.select(scores, 1, 1, 4).tolist() == [0, 3, 5, 6]        # 3 and 0 beat -inf and NaN
    assert oracle.select(scores, 1, 1, 5).tolist() == [0, 2, 3, 5, 6]     # then -inf beats NaN
    assert oracle.select(scores, 1, 1, 6).tolist() == [0, 1, 2, 3, 5, 6]  # then the lower-index NaN
    # nb <= budget: every block, whatever the scores (Section 3.3: no partial below the budget)
    assert oracle.select(np.zeros(5), 1, 2, 8).tolist() == [0, 1, 2, 3, 4]
    assert oracle.select(np.zeros(8), 1, 2, 8).tolist() == list(range(8))
    # exactly one more block than the budget: the single worst candidate is dropped
    s = np.array([0, 4, 3, 1, 2, 0, 0, 0, 0], dtype=np.float64)
    assert oracle.select(s, 1, 2, 8).tolist() == [0, 1, 2, 3, 4, 5, 7, 8]


# ----------------------------------------------------------------------------- attention
def sdpa_reference(qw, k_all, v_all, attn_mask):
    """torch CPU scaled_dot_product_attention in float64 with an explicit boolean mask (library witness)."""
    M, Hq, d = qw.shape
    Hkv = k_all.shape[1]
    G = Hq // Hkv
    qt = torch.from_numpy(qw).permute(1, 0, 2)[None]                              # [1][Hq][M][d]
    kt = torch.from_numpy(k_all).permute(1, 0, 2).repeat_interleave(G, 0)[None]   # [1][Hq][T][d]
    vt = torch.from_numpy(v_all).permute(1, 0, 2).repeat_interleave(G, 0)[None]
    out = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, attn_mask=torch.from_numpy(attn_mask))
    return out[0].permute(1, 0, 2).numpy()


def step_tensors(rng, M, Hq, Hkv, d, dtype):
    q = rng.standard_normal((M, Hq, d)).astype(np.float32)
    kn = rng.standard_normal((M, Hkv, d)).astype(np.float32)
    vn = rng.standard_normal((M, Hkv, d)).astype(np.float32)
    if dtype == "bf16":
        q, kn, vn = bf16_bits(q), bf16_bits(kn), bf16_bits(vn)
    return q, kn, vn


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_chain_tree_equals_causal_attention_library(dtype):
    # a chain-shaped tree is ordinary causal attention of the last M positions of a sequence
    rng = np.random.default_rng(5)
    Hq, Hkv, d, bs, M, seq_len = 6, 2, 16, 16, 9, 16 * 3 + 5
    k, v, table = make_cache(rng, 4, Hkv, bs, d, dtype, shuffle=True, extra_pages=2)
    q, kn, vn = step_tensors(rng, M, Hq, Hkv, d, dtype)
    mask = oracle.tree_mask(np.arange(-1, M - 1, dtype=np.int32))
    out, lse = oracle.tree_attention(q, kn, vn, mask, k, v, table, seq_len)
    T = seq_len + M
    k_all = np.concatenate([logical_tokens(k, table, seq_len), oracle.widen(kn)])
    v_all = np.concatenate([logical_tokens(v, table, seq_len), oracle.widen(vn)])
    # library call on the whole sequence with is_causal; rows of the first seq_len positions are dummies
    Gq = Hq // Hkv
    q_full = np.concatenate([rng.standard_normal((seq_len, Hq, d)), oracle.widen(q)])
    qt = torch.from_numpy(q_full).permute(1, 0, 2)[None]
    kt = torch.from_numpy(k_all).permute(1, 0, 2).repeat_interleave(Gq, 0)[None]
    vt = torch.from_numpy(v_all).permute(1, 0, 2).repeat_interleave(Gq, 0)[None]
    want = torch.nn.functional.scaled_dot_product_attention(qt, kt, vt, is_causal=True)[0]
    want = want.permute(1, 0, 2).numpy()[seq_len:]
    np.testing.assert_allclose(out, want, rtol=1e-10, atol=1e-12)
    assert T == k_all.shape[0]


def test_random_tree_equals_sdpa_with_explicit_mask_and_lse_closed_form():
    rng = np.random.default_rng(6)
    Hq, Hkv, d, bs, M, seq_len = 8, 2, 8, 16, 13, 16 * 2 + 1
    k, v, table = make_cache(rng, 3, Hkv, bs, d)
    q, kn, vn = step_tensors(rng, M, Hq, Hkv, d, "fp32")
    parents = wl.make_tree(M, 4, 3, rng)
    mask = oracle.tree_mask(parents)
    out, lse, probs = oracle.tree_attention(q, kn, vn, mask, k, v, table, seq_len, want_probs=True)
    vis = np.ones((M, seq_len + M), dtype=bool)
    for j in range(M):
        for a in range(M):
            vis[j, seq_len + a] = (int(mask[j, 0]) >> a) & 1
    k_all = np.concatenate([logical_tokens(k, table, seq_len), oracle.widen(kn)])
    v_all = np.concatenate([logical_tokens(v, table, seq_len), oracle.widen(vn)])
    want = sdpa_reference(oracle.widen(q), k_all, v_all, vis[None, None])
    np.testing.assert_allclose(out, want, rtol=1e-10, atol=1e-12)
    # every softmax row sums to 1 and masked keys contribute exactly 0
    np.testing.assert_allclose(probs.sum(-1), 1.0, rtol=0, atol=1e-12)
    for j in range(M):
        assert np.all(probs[j][:, ~vis[j]] == 0.0)
        assert np.all(probs[j][:, vis[j]] > 0.0)
    # lse against log-sum-exp written with numpy on the visible logits
    G = Hq // Hkv
    for j in range(M):
        for n in range(Hq):
            logits = (k_all[vis[j], n // G] @ oracle.widen(q)[j, n]) / math.sqrt(d)
            assert lse[j, n] == pytest.approx(np.log(np.exp(logits - logits.max()).sum()) + logits.max(), abs=1e-12)


def test_tiny_case_brute_force_loops():
    # pure-Python enumeration on a case small enough to follow by hand
    rng = np.random.default_rng(7)
    Hq, Hkv, d, bs, M, seq_len = 2, 1, 2, 2, 3, 3
    k, v, table = make_cache(rng, 2, Hkv, bs, d)
    q, kn, vn = step_tensors(rng, M, Hq, Hkv, d, "fp32")
    parents = np.array([-1, 0, 0], dtype=np.int32)
    out, lse = oracle.tree_attention(q, kn, vn, oracle.tree_mask(parents), k, v, table, seq_len, scale=0.5)
    visible_new = {0: [0], 1: [0, 1], 2: [0, 2]}
    for j in range(M):
        for n in range(Hq):
            keys, vals = [], []
            for t in range(seq_len):
                keys.append(k[table[t // bs], 0, t % bs].astype(float))
                vals.append(v[table[t // bs], 0, t % bs].astype(float))
            for a in visible_new[j]:
                keys.append(kn[a, 0].astype(float))
                vals.append(vn[a, 0].astype(float))
            w = [math.exp(0.5 * sum(float(q[j, n, c]) * kk[c] for c in range(d))) for kk in keys]
            z = sum(w)
            for c in range(d):
                assert out[j, n, c] == pytest.approx(sum(wi / z * vv[c] for wi, vv in zip(w, vals)), abs=1e-13)
            assert lse[j, n] == pytest.approx(math.log(z), abs=1e-13)


def test_single_node_tree_is_decode_attention_and_shift_invariance():
    rng = np.random.default_rng(8)
    Hq, Hkv, d, bs, seq_len = 4, 2, 8, 16, 40
    k, v, table = make_cache(rng, 3, Hkv, bs, d)
    q, kn, vn = step_tensors(rng, 1, Hq, Hkv, d, "fp32")
    # keys with few mantissa bits, so that adding the shift below is exact in float32
    k, kn = np.round(k * 16) / np.float32(16), np.round(kn * 16) / np.float32(16)
    mask = oracle.tree_mask(np.array([-1], dtype=np.int32))
    out, lse = oracle.tree_attention(q, kn, vn, mask, k, v, table, seq_len)
    k_all = np.concatenate([logical_tokens(k, table, seq_len), oracle.widen(kn)])
    v_all = np.concatenate([logical_tokens(v, table, seq_len), oracle.widen(vn)])
    want = sdpa_reference(oracle.widen(q), k_all, v_all, np.ones((1, 1, 1, seq_len + 1), dtype=bool))
    np.testing.assert_allclose(out, want, rtol=1e-10, atol=1e-12)
    # adding one vector to every key shifts each row's logits by a constant: the output is unchanged
    # and lse moves by q.shift*scale (softmax shift invariance)
    shift = np.arange(d, dtype=np.float32) / 8.0
    out2, lse2 = oracle.tree_attention(q, kn + shift, vn, mask, k + shift, v, table, seq_len)
    np.testing.assert_allclose(out2, out, rtol=1e-9, atol=1e-11)
    np.testing.assert_allclose((lse2 - lse)[0], (oracle.widen(q)[0] @ shift.astype(np.float64)) / math.sqrt(d),
                               rtol=1e-9, atol=1e-11)


def test_page_permutation_invariance():
    rng = np.random.default_rng(9)
    Hq, Hkv, d, bs, M, seq_len = 4, 2, 8, 16, 6, 16 * 4 - 3
    k, v, table = make_cache(rng, 4, Hkv, bs, d, extra_pages=3)
    q, kn, vn = step_tensors(rng, M, Hq, Hkv, d, "fp32")
    mask = oracle.tree_mask(wl.make_tree(M, 3, 3, rng))
    out, lse = oracle.tree_attention(q, kn, vn, mask, k, v, table, seq_len)
    perm = rng.permutation(k.shape[0])
    k2, v2 = np.empty_like(k), np.empty_like(v)
    k2[perm], v2[perm] = k, v
    out2, lse2 = oracle.tree_attention(q, kn, vn, mask, k2, v2, perm[table].astype(np.int32), seq_len)
    assert np.array_equal(out, out2) and np.array_equal(lse, lse2)


# ----------------------------------------------------------------------------- gather / partial == full
@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_selecting_every_block_equals_full_verification(dtype):
    rng = np.random.default_rng(10)
    Hq, Hkv, d, bs, M, seq_len = 4, 2, 8, 16, 7, 16 * 5 + 9
    nb = 6
    k, v, table = make_cache(rng, nb, Hkv, bs, d, dtype, shuffle=True, extra_pages=1)
    q, kn, vn = step_tensors(rng, M, Hq, Hkv, d, dtype)
    mask = oracle.tree_mask(wl.make_tree(M, 3, 3, rng))
    full_out, full_lse = oracle.tree_attention(q, kn, vn, mask, k, v, table, seq_len)
    kmax, kmin = oracle.block_summaries(k, table, seq_len)
    scores = oracle.block_scores(q, kmax, kmin, Hkv)
    idx = np.stack([oracle.select(scores[h], 1, 2, budget_blocks=nb) for h in range(Hkv)])
    assert idx.tolist() == [list(range(nb))] * Hkv
    pk, pv = np.zeros((nb + 2, Hkv, bs, d), k.dtype), np.zeros((nb + 2, Hkv, bs, d), k.dtype)
    plen = oracle.gather(k, v, table, seq_len, idx, pk, pv, first_page=1)
    assert plen == seq_len
    ptable = np.arange(1, nb + 1, dtype=np.int32)
    part_out, part_lse = oracle.tree_attention(q, kn, vn, mask, pk, pv, ptable, plen)
    assert np.array_equal(part_out, full_out) and np.array_equal(part_lse, full_lse)


def test_gather_per_head_lists_and_partial_attention_is_attention_over_kept_tokens():
    rng = np.random.default_rng(11)
    Hq, Hkv, d, bs, M, seq_len = 4, 2, 8, 8, 5, 8 * 9 + 3
    nb = 10
    k, v, table = make_cache(rng, nb, Hkv, bs, d, shuffle=True)
    q, kn, vn = step_tensors(rng, M, Hq, Hkv, d, "fp32")
    mask = oracle.tree_mask(wl.make_tree(M, 3, 2, rng))
    idx = np.array([[0, 2, 5, 8, 9], [0, 3, 4, 8, 9]], dtype=np.int32)
    pk, pv = np.zeros((6, Hkv, bs, d), np.float32), np.zeros((6, Hkv, bs, d), np.float32)
    plen = oracle.gather(k, v, table, seq_len, idx, pk, pv, first_page=0)
    assert plen == 4 * bs + 3
    kt, vt = logical_tokens(k, table, seq_len), logical_tokens(v, table, seq_len)
    pkt = logical_tokens(pk, np.arange(6, dtype=np.int32), plen)
    for h in range(Hkv):
        kept = np.concatenate([np.arange(i * bs, min((i + 1) * bs, seq_len)) for i in idx[h]])
        assert np.array_equal(pkt[:, h], kt[kept, h])
    out, _ = oracle.tree_attention(q, kn, vn, mask, pk, pv, np.arange(6, dtype=np.int32), plen)
    # reference: SDPA over the full sequence with the dropped tokens masked out, per KV head
    G = Hq // Hkv
    for h in range(Hkv):
        kept = np.zeros(seq_len, dtype=bool)
        for i in idx[h]:
            kept[i * bs:(i + 1) * bs] = True
        vis = np.ones((M, seq_len + M), dtype=bool)
        vis[:, :seq_len] = kept
        for j in range(M):
            for a in range(M):
                vis[j, seq_len + a] = (int(mask[j, 0]) >> a) & 1
        k_all = np.concatenate([kt[:, h:h + 1], oracle.widen(kn)[:, h:h + 1]])
        v_all = np.concatenate([vt[:, h:h + 1], oracle.widen(vn)[:, h:h + 1]])
        want = sdpa_reference(oracle.widen(q)[:, h * G:(h + 1) * G], k_all, v_all, vis[None, None])
        np.testing.assert_allclose(out[:, h * G:(h + 1) * G], want, rtol=1e-10, atol=1e-12)


# ----------------------------------------------------------------------------- commit / mode rule
def test_commit_appends_accepted_rows_bit_exact():
    rng = np.random.default_rng(12)
    Hq, Hkv, d, bs, M, seq_len = 4, 2, 8, 8, 6, 8 * 2 + 6
    k, v, table = make_cache(rng, 4, Hkv, bs, d, "bf16", shuffle=True)
    q, kn, vn = step_tensors(rng, M, Hq, Hkv, d, "bf16")
    k0, v0 = k.copy(), v.copy()
    accepted = np.array([0, 2, 5], dtype=np.int32)
    new_len = oracle.commit(kn, vn, accepted, k, v, table, seq_len)
    assert new_len == seq_len + 3
    for a, row in enumerate(accepted):
        t = seq_len + a  # crosses from block 2 into block 3
        assert np.array_equal(k[table[t // bs], :, t % bs], kn[row])
        assert np.array_equal(v[table[t // bs], :, t % bs], vn[row])
    # nothing else changed
    changed = (k != k0) | (v != v0)
    touched = np.zeros_like(changed)
    for a in range(3):
        t = seq_len + a
        touched[table[t // bs], :, t % bs] = True
    assert not np.any(changed & ~touched)
    # attending the grown cache with a 1-node tree == attending old cache + chain of the accepted tokens
    q1, kn1, vn1 = step_tensors(rng, 1, Hq, Hkv, d, "bf16")
    one = oracle.tree_mask(np.array([-1], dtype=np.int32))
    out_a, _ = oracle.tree_attention(q1, kn1, vn1, one, k, v, table, new_len)
    qc = np.concatenate([np.zeros((3, Hq, d), np.uint16), q1])
    knc, vnc = np.concatenate([kn[accepted], kn1]), np.concatenate([vn[accepted], vn1])
    chain = oracle.tree_mask(np.array([-1], dtype=np.int32), n_chain=3)
    out_b, _ = oracle.tree_attention(qc, knc, vnc, chain, k0, v0, table, seq_len)
    np.testing.assert_allclose(out_a[0], out_b[3], rtol=1e-12, atol=1e-14)


def test_mode_rule_follows_section_3_3():
    F, P, R = oracle.FULL, oracle.PARTIAL, oracle.REFRESH
    budget, buf = 4096, 68
    assert oracle.select_mode(1000, budget, 0, 48, buf, False) == F      # shorter than the budget
    assert oracle.select_mode(4095, budget, 0, 48, buf, True) == F
    assert oracle.select_mode(4096, budget, 0, 48, buf, False) == R      # first crossing initialises
    assert oracle.select_mode(5000, budget, 0, 48, buf, True) == P
    assert oracle.select_mode(5000, budget, 20, 48, buf, True) == P      # 68 fits exactly
    assert oracle.select_mode(5000, budget, 21, 48, buf, True) == R      # exceeds the buffer


def test_planted_mistakes_are_caught():
    """A wrong sign / transposed operand in a copy of the definition must disagree with the oracle."""
    rng = np.random.default_rng(13)
    Hq, Hkv, d, bs, M, seq_len = 2, 1, 4, 4, 3, 10
    k, v, table = make_cache(rng, 3, Hkv, bs, d)
    q, kn, vn = step_tensors(rng, M, Hq, Hkv, d, "fp32")
    mask = oracle.tree_mask(np.array([-1, 0, 1], dtype=np.int32))
    out, _ = oracle.tree_attention(q, kn, vn, mask, k, v, table, seq_len)
    swapped, _ = oracle.tree_attention(q, kn, vn, mask, v, k, table, seq_len)  # K and V exchanged
    negated, _ = oracle.tree_attention(q, kn, vn, mask, k, v, table, seq_len, scale=-1 / math.sqrt(d))
    unmasked, _ = oracle.tree_attention(q, kn, vn, oracle.tree_mask(np.array([-1, 0, 0])), k, v, table, seq_len)
    for wrong in (swapped, negated, unmasked):
        assert np.abs(wrong - out).max() > 1e-3


def test_head_shared_scores_is_the_mean_over_heads():
    # hand values: three heads, four blocks
    s = np.array([[1.0, 2.0, -3.0, 0.5], [3.0, 2.0, 3.0, 0.25], [2.0, 5.0, 0.0, 0.0]])
    got = oracle.head_shared_scores(s)
    assert got.dtype == np.float64
    assert np.array_equal(got, np.array([2.0, 3.0, 0.0, 0.25]))
    rng = np.random.default_rng(5)
    r = rng.standard_normal((8, 300)).astype(np.float32) * 30
    assert np.array_equal(oracle.head_shared_scores(r[:1]), r[0].astype(np.float64))  # a single head is left as it is
    # the mean is linear: a constant added to one head moves every block's shared score by constant / heads
    r2 = r.astype(np.float64)
    r2[3] += 8.0
    np.testing.assert_allclose(oracle.head_shared_scores(r2), oracle.head_shared_scores(r) + 1.0, rtol=0, atol=1e-12)
    # selection on it is ordinary selection: with identical heads the shared list equals every head's own list
    same = np.repeat(r[:1], 4, axis=0)
    assert np.array_equal(oracle.select(oracle.head_shared_scores(same), 1, 2, 16),
                          oracle.select(r[0].astype(np.float64), 1, 2, 16))


def test_shared_selection_check_accepts_rounding_ties_and_rejects_wrong_lists():
    """The GPU-side check of head-shared lists (tests/util.check_shared_selection) against planted lists."""
    from tests import util
    rng = np.random.default_rng(11)
    s = rng.standard_normal((8, 64)).astype(np.float32) * 10
    want = oracle.select(oracle.head_shared_scores(s), 1, 2, 16)
    util.check_shared_selection(want, s, 1, 2, 16)                       # the oracle's own list
    mean = oracle.head_shared_scores(s)
    kept = [i for i in want if 1 <= i < 62]
    dropped = [i for i in range(1, 62) if i not in want]
    worst_kept, best_dropped = min(kept, key=lambda i: mean[i]), max(dropped, key=lambda i: mean[i])
    swapped = np.array(sorted((set(want.tolist()) - {worst_kept}) | {best_dropped}), dtype=np.int32)
    with pytest.raises(AssertionError):                                  # far apart: the swap is a mistake
        util.check_shared_selection(swapped, s, 1, 2, 16)
    tie = s.copy()
    tie[:, best_dropped] = tie[:, worst_kept]                            # equal means: either block may be kept
    want_tie = oracle.select(oracle.head_shared_scores(tie), 1, 2, 16)
    other = np.array(sorted((set(want_tie.tolist()) - {min(worst_kept, best_dropped)}) | {max(worst_kept, best_dropped)}),
                     dtype=np.int32)
    util.check_shared_selection(other, tie, 1, 2, 16)
    with pytest.raises(AssertionError):                                  # a sink block left out
        util.check_shared_selection(np.array(sorted(set(want.tolist()) - {0} | {dropped[0]}), dtype=np.int32), s, 1, 2, 16)


# ---- the linear maps either side of the attention (Algorithm 1 "TreeDecode") ------------------------------------
def test_rope_closed_form_pairs_channel_c_with_c_plus_half():
    """d = 4, theta = 10000, position 1: channel 0 turns by 1 rad into channel 2, channel 1 by 0.01 rad into 3.

    The numbers are cos/sin of 1 and 0.01 typed from tables, so a wrong pairing (neighbouring channels), a wrong
    sign of the sine or a wrong frequency exponent each miss."""
    x = np.array([[1, 0, 0, 0], [0, 1, 0, 0], [0, 0, 1, 0]], dtype=np.float32)
    w = np.tile(np.eye(4, dtype=np.float32), (3, 1))  # q, k and v heads all copy the input
    q, k, v = oracle.qkv_rope(x, w, 1, 1, 4, [1, 1, 1], 10000.0)
    want_q = np.array([[0.5403023058681398, 0, 0.8414709848078965, 0],
                       [0, 0.9999500004166653, 0, 0.009999833334166664],
                       [-0.8414709848078965, 0, 0.5403023058681398, 0]])
    np.testing.assert_allclose(q.reshape(3, 4), want_q, atol=1e-15)
    np.testing.assert_allclose(k.reshape(3, 4), want_q, atol=1e-15)
    np.testing.assert_array_equal(v.reshape(3, 4), x.astype(np.float64))  # values are never rotated


def test_rope_is_a_rotation_that_depends_on_relative_position_only():
    rng = np.random.default_rng(11)
    T, H, d = 6, 3, 16
    a = rng.standard_normal((T, H, d))
    b = rng.standard_normal((T, H, d))
    pos = np.array([0, 1, 5, 70000, 131071, 131072], dtype=np.int32)
    ra, rb = oracle.rope(a, pos, 500000.0), oracle.rope(b, pos, 500000.0)
    np.testing.assert_array_equal(ra[0], a[0])  # position 0 is the identity
    np.testing.assert_allclose((ra ** 2).sum(-1), (a ** 2).sum(-1), rtol=1e-12)  # norms kept per head
    # <R_m a, R_n b> depends on m - n only: shift every position by the same amount
    for shift in (1, 977, 60000):
        sa, sb = oracle.rope(a, pos + shift, 500000.0), oracle.rope(b, pos + shift, 500000.0)
        g0 = np.einsum("thd,uhd->htu", ra, rb)
        g1 = np.einsum("thd,uhd->htu", sa, sb)
        np.testing.assert_allclose(g1, g0, atol=1e-8)
    # and it is not the identity elsewhere
    assert np.abs(ra[2] - a[2]).max() > 0.1


def test_linear_matches_library_matmul_and_is_not_transposed():
    rng = np.random.default_rng(5)
    T, n_in, n_out = 7, 48, 20
    x = rng.standard_normal((T, n_in)).astype(np.float32)
    w = rng.standard_normal((n_out, n_in)).astype(np.float32)
    r = rng.standard_normal((T, n_out)).astype(np.float32)
    np.testing.assert_allclose(oracle.linear(x, w), x.astype(np.float64) @ w.astype(np.float64).T, atol=1e-12)
    np.testing.assert_allclose(oracle.linear(x, w, r), x.astype(np.float64) @ w.astype(np.float64).T + r, atol=1e-12)
    # a weight whose row f has a single one at column perm[f] picks input channel perm[f]
    perm = rng.integers(0, n_in, size=n_out)
    sel = np.zeros((n_out, n_in), dtype=np.float32)
    sel[np.arange(n_out), perm] = 1
    np.testing.assert_array_equal(oracle.linear(x, sel), x[:, perm].astype(np.float64))
    # bfloat16 inputs are widened exactly
    xb, wb = bf16_bits(x), bf16_bits(w)
    np.testing.assert_allclose(oracle.linear(xb, wb), oracle.widen(xb) @ oracle.widen(wb).T, atol=1e-12)


def test_qkv_rope_splits_heads_in_q_k_v_order():
    rng = np.random.default_rng(6)
    T, hidden, Hq, Hkv, d = 5, 32, 4, 2, 8
    x = rng.standard_normal((T, hidden)).astype(np.float32)
    w = rng.standard_normal(((Hq + 2 * Hkv) * d, hidden)).astype(np.float32)
    pos = np.array([3, 4, 4, 5, 9], dtype=np.int32)
    q, k, v = oracle.qkv_rope(x, w, Hq, Hkv, d, pos, 10000.0)
    y = x.astype(np.float64) @ w.astype(np.float64).T
    np.testing.assert_allclose(v, y[:, (Hq + Hkv) * d:].reshape(T, Hkv, d), atol=1e-12)
    np.testing.assert_allclose(q, oracle.rope(y[:, :Hq * d].reshape(T, Hq, d), pos, 10000.0), atol=1e-12)
    np.testing.assert_allclose(k, oracle.rope(y[:, Hq * d:(Hq + Hkv) * d].reshape(T, Hkv, d), pos, 10000.0), atol=1e-12)
    # at position 0 nothing is rotated
    q0, k0, _ = oracle.qkv_rope(x, w, Hq, Hkv, d, np.zeros(T, np.int32), 10000.0)
    np.testing.assert_allclose(q0.reshape(T, -1), y[:, :Hq * d], atol=1e-12)
    np.testing.assert_allclose(k0.reshape(T, -1), y[:, Hq * d:(Hq + Hkv) * d], atol=1e-12)


def test_step_positions_are_base_plus_depth():
    parents = np.array([-1, 0, 0, 1, 3, 2, 5, 6], dtype=np.int32)
    # depths by hand: 0, 1, 1, 2, 3, 2, 3, 4
    np.testing.assert_array_equal(oracle.step_positions(parents, 0, 1000),
                                  1000 + np.array([0, 1, 1, 2, 3, 2, 3, 4]))
    np.testing.assert_array_equal(oracle.step_positions(parents, 3, 50),
                                  np.concatenate([[50, 51, 52], 53 + np.array([0, 1, 1, 2, 3, 2, 3, 4])]))
    # the depth of a row is also the number of step tokens it sees, minus one
    m = oracle.tree_mask(parents, 3)
    seen = np.array([sum(bin(int(wd)).count("1") for wd in row) for row in m])
    np.testing.assert_array_equal(oracle.step_positions(parents, 3, 0), seen - 1)
    with pytest.raises(ValueError):
        oracle.step_positions(np.array([-1, 2, 1], dtype=np.int32))


def test_attention_over_own_keys_ignores_where_the_step_starts():
    """Rotary q and k followed by the tree attention with an empty cache: only position differences enter, so moving
    the whole step elsewhere in the sequence leaves the output unchanged."""
    rng = np.random.default_rng(8)
    T, hidden, Hq, Hkv, d = 9, 24, 4, 2, 16
    parents = np.array([-1, 0, 0, 1, 1, 2, 4, 4, 6], dtype=np.int32)
    x = rng.standard_normal((T, hidden)).astype(np.float32)
    w = (rng.standard_normal(((Hq + 2 * Hkv) * d, hidden)) / np.sqrt(hidden)).astype(np.float32)
    mask = oracle.tree_mask(parents)
    empty_k = np.zeros((1, Hkv, 16, d), dtype=np.float32)
    outs = []
    for base in (0, 4096, 100000):
        q, k, v = oracle.qkv_rope(x, w, Hq, Hkv, d, oracle.step_positions(parents, 0, base), 10000.0)
        out, _ = oracle.tree_attention(q.astype(np.float32), k.astype(np.float32), v.astype(np.float32), mask,
                                       empty_k, empty_k, np.zeros(1, np.int32), 0)
        outs.append(out)
    np.testing.assert_allclose(outs[1], outs[0], atol=2e-5)
    np.testing.assert_allclose(outs[2], outs[0], atol=2e-5)
