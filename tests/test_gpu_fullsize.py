"""GPU parity at the full sizes of the benchmark configurations, in the launch configuration the
benchmark times (all layers in one layer-batched call), on sampled outputs the oracle computes one by
one: a few layers, every head, the rows of root-to-leaf paths of the draft tree (a row only sees its
ancestors among the step's tokens, so its output does not depend on the rows left out).  Selection is
checked on every (layer, sequence, head); summaries, scores, the gathered partial cache and the partial
verification on the sampled layers.  The last test runs the 64-step decode loop (partial verification
every step, refresh every 8th, cache growing by the accepted tokens) against an oracle loop that mirrors
the state of two layers."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_02337_b200 import binding as B
from paper_2512_02337_b200 import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu


def sample_rows(parents, rng, n_extra=2):
    """Deepest root-to-leaf path plus a few random nodes (closure is taken by the oracle helper)."""
    M = len(parents)
    depth = [len(wl.path_to(parents, n)) for n in range(M)]
    rows = set(int(r) for r in wl.path_to(parents, int(np.argmax(depth))))
    rows.update(int(r) for r in rng.integers(0, M, size=n_extra))
    return sorted(rows)


def check_rows(got_out, got_lse, q, kn, vn, parents, rows, kp, vp, table, seq_len, what, n_chain=0):
    closed, o_out, o_lse = util.oracle_attention_rows(q, kn, vn, parents, n_chain, rows, kp, vp, table, seq_len)
    util.compare(got_out[closed], o_out, "bf16", what)
    np.testing.assert_allclose(got_lse[closed], o_lse, atol=5e-3, err_msg=what)


def run_full_size(name, layers, budgets, score_mode=0):
    dev = torch.device("cuda")
    w = wl.make_workload(name, device=dev, spare_tokens=64)
    c = w.cfg
    L, Hq, Hkv, d, bs, M, batch = c["n_layers"], c["Hq"], c["Hkv"], c["d"], c["bs"], c["M"], w.batch
    rng = np.random.default_rng(c["index"])
    cfg = util.config_for(w, score_mode=score_mode)
    full = util.full_cache(w)
    full.max_seq_len = int(max(c["ctx"])) + 64
    ws = B.new_workspace(cfg, L, batch, full.max_seq_len, M)
    mask = util.device_masks(w.parents, M)
    kmax = torch.zeros((L, batch, Hkv, w.max_blocks, d), dtype=torch.bfloat16, device=dev)
    kmin = torch.zeros_like(kmax)
    scores = torch.zeros((L, batch, Hkv, w.max_blocks), dtype=torch.float32, device=dev)
    out = torch.zeros((L, batch, M, Hq, d), dtype=torch.float32, device=dev)
    lse = torch.zeros((L, batch, M, Hq), dtype=torch.float32, device=dev)
    last_query = torch.zeros(batch, dtype=torch.int32, device=dev)
    B.specpv_update_block_summaries(cfg, 0, L, full, None, w.max_blocks, kmax, kmin, ws)
    B.specpv_score_blocks(cfg, 0, L, w.q, None, M, last_query, kmax, kmin, full, scores, ws)
    B.specpv_verify_full(cfg, 0, L, w.q, w.k_new, w.v_new, mask, None, M, full, out, lse, ws)
    util.sync_status(ws)

    seq_lens, table = w.seq_lens.cpu().numpy(), w.block_table.cpu().numpy()
    scores_g = scores.cpu().numpy()
    sink, local = cfg.sink_blocks, cfg.local_blocks
    host = {}
    for l in layers:  # host copies of the sampled layers (the same bytes the kernels read)
        host[l] = (wl.to_numpy(w.k_pool[l]), wl.to_numpy(w.v_pool[l]), wl.to_numpy(w.q[l]), wl.to_numpy(w.k_new[l]),
                   wl.to_numpy(w.v_new[l]))
    rows = [sample_rows(w.parents[b], rng) for b in range(batch)]
    for l in layers:
        kp, vp, qn, knn, vnn = host[l]
        got_out, got_lse = out[l].cpu().numpy(), lse[l].cpu().numpy()
        for b in range(batch):
            sl = int(seq_lens[b])
            nb = (sl + bs - 1) // bs
            okmax, okmin = oracle.block_summaries(kp, table[b], sl)
            assert np.array_equal(util.widen_t(kmax[l, b])[:, :nb], okmax)
            assert np.array_equal(util.widen_t(kmin[l, b])[:, :nb], okmin)
            osc = oracle.block_scores(qn[b], okmax, okmin, Hkv, reduce=0, last_query=0, score_mode=score_mode)
            np.testing.assert_allclose(scores_g[l, b, :, :nb], osc, rtol=2e-3, atol=2e-2)
            check_rows(got_out[b], got_lse[b], qn[b], knn[b], vnn[b], w.parents[b], rows[b], kp, vp, table[b], sl,
                       f"{name} full l{l} b{b}")

    # selection / gather / partial verification for every budget of the sweep
    for budget in budgets:
        cfgb = util.config_for(w, budget_blocks=budget, score_mode=score_mode)
        idx = torch.full((L, batch, Hkv, budget), -7, dtype=torch.int32, device=dev)
        count = torch.zeros(batch, dtype=torch.int32, device=dev)
        ppb = budget + (cfgb.buffer_tokens + bs - 1) // bs + 1
        pk = torch.zeros((L, batch * ppb, Hkv, bs, d), dtype=torch.bfloat16, device=dev)
        pv = torch.zeros_like(pk)
        ptable = torch.arange(batch * ppb, dtype=torch.int32, device=dev).reshape(batch, ppb).contiguous()
        plens = torch.zeros(batch, dtype=torch.int32, device=dev)
        partial = B.Cache(pk, pv, ptable, plens, budget * bs + cfgb.buffer_tokens)
        B.specpv_select_partial_kv(cfgb, L, scores, w.seq_lens, batch, w.max_blocks, idx, count, ws)
        B.specpv_refresh_partial(cfgb, full, idx, count, partial, plens, ws)
        B.specpv_verify_partial(cfgb, 0, L, w.q, w.k_new, w.v_new, mask, None, M, partial, out, lse, ws)
        util.sync_status(ws)
        idx_g, count_g, plens_g = idx.cpu().numpy(), count.cpu().numpy(), plens.cpu().numpy()
        for l in range(L):  # bit-exact on every (layer, sequence, head), given the kernel's float32 scores
            for b in range(batch):
                nb = (int(seq_lens[b]) + bs - 1) // bs
                assert count_g[b] == min(nb, budget)
                for h in range(Hkv):
                    want = oracle.select(scores_g[l, b, h, :nb].astype(np.float64), sink, local, budget)
                    assert np.array_equal(idx_g[l, b, h, :len(want)], want), (name, budget, l, b, h)
        for l in layers:
            kp, vp, qn, knn, vnn = host[l]
            pk_g, pv_g = wl.to_numpy(pk[l]), wl.to_numpy(pv[l])
            got_out, got_lse = out[l].cpu().numpy(), lse[l].cpu().numpy()
            for b in range(batch):
                sl = int(seq_lens[b])
                opk, opv = np.zeros_like(pk_g), np.zeros_like(pv_g)
                oplen = oracle.gather(kp, vp, table[b], sl, idx_g[l, b], opk, opv, first_page=b * ppb)
                assert plens_g[b] == oplen
                n_keep = int(count_g[b])
                first = b * ppb
                gk, gv = pk_g[first:first + n_keep].copy(), pv_g[first:first + n_keep].copy()
                tail = oplen - (n_keep - 1) * bs
                gk[-1, :, tail:], gv[-1, :, tail:] = 0, 0  # tokens past the ragged end are unspecified
                assert np.array_equal(gk, opk[first:first + n_keep]) and np.array_equal(gv, opv[first:first + n_keep])
                check_rows(got_out[b], got_lse[b], qn[b], knn[b], vnn[b], w.parents[b], rows[b], opk, opv,
                           ptable[b].cpu().numpy(), oplen, f"{name} partial budget {budget} l{l} b{b}")


def test_llama_32k_all_layers_sampled():
    run_full_size("llama_32k", layers=[0, 31], budgets=[64])


def test_llama_32k_all_layers_sampled_on_the_pair_kernel(monkeypatch):
    """The same full-size check with the CTA-pair attention kernel (persistent launch, shared KV ranges merged in the
    kernel) in place of the default one."""
    monkeypatch.setenv("SPECPV_ATTN_KERNEL", "pair")
    run_full_size("llama_32k", layers=[0, 31], budgets=[64])


def test_stress_batch4_on_the_pair_kernel(monkeypatch):
    monkeypatch.setenv("SPECPV_ATTN_KERNEL", "pair")
    run_full_size("stress_b4", layers=[0, 31], budgets=[64])


def test_llama_32k_channelwise_scores_several_tiles_per_cta():
    # the channel-wise form of Eq. 2 at full size: 256 heads leave two CTAs per head, two 128-block tiles each
    run_full_size("llama_32k", layers=[3, 31], budgets=[64], score_mode=1)


def test_llama_128k_all_layers_sampled_budget_sweep():
    run_full_size("llama_128k", layers=[0, 17, 31], budgets=[32, 64, 128])


def test_stress_batch4_ragged_shuffled_all_layers_sampled():
    run_full_size("stress_b4", layers=[9, 31], budgets=[64])


def test_qwen3_64k_decode_loop_64_steps():
    """Config "qwen3_64k_loop": 36 layers, 64K context, 48-node trees, 64 steps; partial verification
    every step, full verification with refresh every 8th step over the chain of partially verified tokens
    plus the tree, accepted path lengths 1..6 drawn from the seed.  An oracle loop mirrors layers 0 and 35."""
    run_decode_loop("qwen3_64k_loop", n_steps=64, period=8)


def test_decode_loop_paper_geometry_refresh_on_buffer_overflow():
    """The paper's own settings (Appendix "Generation Settings"): 16-token blocks, 32 sink and 128 local tokens,
    a 512-token budget and a buffer of 20 tokens beyond the tree; the refresh is triggered by the mode rule
    alone (partially verified + candidate tokens exceed the buffer), not by a fixed period."""
    run_decode_loop("llama_32k", n_steps=24, period=None, n_layers=2, ctx=[16 * 300 + 7], bs=16, M=12, depth=4,
                    branch=3, budget_blocks=32, buffer_tokens=20 + 12)


def run_decode_loop(name, n_steps, period, **over):
    dev = torch.device("cuda")
    c0 = wl.CONFIGS[name]
    spare = n_steps * 6 + 64
    w = wl.make_workload(name, device=dev, spare_tokens=spare, **over)
    c = w.cfg
    L, Hq, Hkv, d, bs, M = c["n_layers"], c["Hq"], c["Hkv"], c["d"], c["bs"], c["M"]
    rng = np.random.default_rng(c0["index"])
    cfg = util.config_for(w)
    sink, local, budget = cfg.sink_blocks, cfg.local_blocks, cfg.budget_blocks
    M_max = min(cfg.buffer_tokens + 6, 128)  # the longest chain of partially verified tokens plus the tree
    full = util.full_cache(w)
    full.max_seq_len = int(c["ctx"][0]) + spare
    ws = B.new_workspace(cfg, L, 1, full.max_seq_len, M_max)
    kmax = torch.zeros((L, 1, Hkv, w.max_blocks, d), dtype=torch.bfloat16, device=dev)
    kmin = torch.zeros_like(kmax)
    scores = torch.zeros((L, 1, Hkv, w.max_blocks), dtype=torch.float32, device=dev)
    idx = torch.zeros((L, 1, Hkv, budget), dtype=torch.int32, device=dev)
    count = torch.zeros(1, dtype=torch.int32, device=dev)
    ppb = budget + (cfg.buffer_tokens + bs - 1) // bs + 1
    pk = torch.zeros((L, ppb, Hkv, bs, d), dtype=torch.bfloat16, device=dev)
    pv = torch.zeros_like(pk)
    ptable = torch.arange(ppb, dtype=torch.int32, device=dev)[None].contiguous()
    plens = torch.zeros(1, dtype=torch.int32, device=dev)
    partial = B.Cache(pk, pv, ptable, plens, budget * bs + cfg.buffer_tokens)
    out = torch.zeros((L, 1, M_max, Hq, d), dtype=torch.float32, device=dev)
    lse = torch.zeros((L, 1, M_max, Hq), dtype=torch.float32, device=dev)
    B.specpv_update_block_summaries(cfg, 0, L, full, None, w.max_blocks, kmax, kmin, ws)

    # the oracle's mirror of two layers
    mirror = sorted({0, L - 1})
    table = w.block_table[0].cpu().numpy()
    ptab = ptable[0].cpu().numpy()
    o_k = {l: wl.to_numpy(w.k_pool[l]).copy() for l in mirror}
    o_v = {l: wl.to_numpy(w.v_pool[l]).copy() for l in mirror}
    o_pk = {l: np.zeros_like(wl.to_numpy(pk[l])) for l in mirror}
    o_pv = {l: np.zeros_like(wl.to_numpy(pv[l])) for l in mirror}
    o_len, o_plen = int(c["ctx"][0]), 0
    chain_k = {l: [] for l in mirror}  # K/V of the partially verified tokens as last computed (host copies)

    g = torch.Generator(device=dev).manual_seed(c0["index"] + 77)
    initialised = False
    pending = []  # per partially verified token: nothing but a count is needed on the GPU side
    for step in range(1, n_steps + 1):
        parents = wl.make_tree(M, c["depth"], c["branch"], rng)
        accept_len = int(rng.integers(1, min(6, c["depth"] + 1) + 1))
        depth = [len(wl.path_to(parents, n)) for n in range(M)]
        path = wl.path_to(parents, depth.index(accept_len))  # the accepted root-to-node path
        n_pv = len(pending)
        mode = B.specpv_select_mode(o_len, budget * bs, n_pv, M, cfg.buffer_tokens, initialised)
        assert mode in (B.MODE_REFRESH, B.MODE_PARTIAL)
        assert mode == oracle.select_mode(o_len, budget * bs, n_pv, M, cfg.buffer_tokens, initialised)
        refresh = mode == B.MODE_REFRESH or (period is not None and step % period == 0)
        if period is not None and mode == B.MODE_REFRESH:
            assert step % period == 0 or not initialised  # the buffer is sized so that the rule never forces an earlier refresh
        n_chain = n_pv if refresh else 0
        m_rows = n_chain + M
        q = torch.randn((L, 1, M_max, Hq, d), generator=g, device=dev).to(torch.bfloat16)
        kn = torch.randn((L, 1, M_max, Hkv, d), generator=g, device=dev).to(torch.bfloat16)
        vn = torch.randn((L, 1, M_max, Hkv, d), generator=g, device=dev).to(torch.bfloat16)
        W = (M_max + 63) // 64
        mask_np = np.zeros((1, M_max, W), dtype=np.uint64)
        mask_np[0, :m_rows] = B.specpv_build_tree_mask(parents, n_chain, W)
        mask = torch.from_numpy(mask_np.view(np.int64)).to(dev)
        q_lens = torch.tensor([m_rows], dtype=torch.int32, device=dev)
        rows = sorted(set(range(n_chain)) | set(n_chain + int(r) for r in path) |
                      set(n_chain + int(r) for r in rng.integers(0, M, size=2)))
        if refresh:
            # full verification over the whole cache; the chain's K/V are recomputed by this pass
            B.specpv_verify_full(cfg, 0, L, q, kn, vn, mask, q_lens, M_max, full, out, lse, ws)
            acc = np.concatenate([np.arange(n_chain), n_chain + path]).astype(np.int32)
        else:
            B.specpv_verify_partial(cfg, 0, L, q, kn, vn, mask, q_lens, M_max, partial, out, lse, ws)
            acc = path.astype(np.int32)
        util.sync_status(ws)
        # ---- oracle attention on the sampled rows of the mirrored layers, before any state changes
        for l in mirror:
            qn, knn, vnn = wl.to_numpy(q[l, 0, :m_rows]), wl.to_numpy(kn[l, 0, :m_rows]), wl.to_numpy(vn[l, 0, :m_rows])
            if refresh:
                kpool, vpool, tab, ln = o_k[l], o_v[l], table, o_len
            else:
                kpool, vpool, tab, ln = o_pk[l], o_pv[l], ptab, o_plen
            closed, o_out, o_lse = util.oracle_attention_rows(qn, knn, vnn, parents, n_chain, rows, kpool, vpool, tab, ln)
            util.compare(out[l, 0].cpu().numpy()[closed], o_out, "bf16", f"step {step} layer {l} {'refresh' if refresh else 'partial'}")
            np.testing.assert_allclose(lse[l, 0].cpu().numpy()[closed], o_lse, atol=5e-3)
        # ---- state update
        A_max = 64
        acc_t = torch.zeros((1, A_max), dtype=torch.int32, device=dev)
        acc_t[0, :len(acc)] = torch.from_numpy(acc).to(dev)
        n_acc = torch.tensor([len(acc)], dtype=torch.int32, device=dev)
        if refresh:
            B.specpv_commit_accepted(cfg, 0, L, kn, vn, M_max, acc_t, n_acc, A_max, full, kmax, kmin, ws)
            B.specpv_score_blocks(cfg, 0, L, q, q_lens, M_max, torch.tensor([n_chain], dtype=torch.int32, device=dev),
                                  kmax, kmin, full, scores, ws)
            B.specpv_select_partial_kv(cfg, L, scores, w.seq_lens, 1, w.max_blocks, idx, count, ws)
            B.specpv_refresh_partial(cfg, full, idx, count, partial, plens, ws)
            util.sync_status(ws)
            new_len = o_len + len(acc)
            nb = (new_len + bs - 1) // bs
            scores_g, idx_g = scores.cpu().numpy(), idx.cpu().numpy()
            for l in range(L):  # selection: bit-exact on every layer and head
                for h in range(Hkv):
                    want = oracle.select(scores_g[l, 0, h, :nb].astype(np.float64), sink, local, budget)
                    assert np.array_equal(idx_g[l, 0, h, :len(want)], want), (step, l, h)
            for l in mirror:
                knn, vnn = wl.to_numpy(kn[l, 0, :m_rows]), wl.to_numpy(vn[l, 0, :m_rows])
                assert oracle.commit(knn, vnn, acc, o_k[l], o_v[l], table, o_len) == new_len
                okmax, okmin = oracle.block_summaries(o_k[l], table, new_len)
                assert np.array_equal(util.widen_t(kmax[l, 0])[:, :nb], okmax)
                assert np.array_equal(util.widen_t(kmin[l, 0])[:, :nb], okmin)
                osc = oracle.block_scores(wl.to_numpy(q[l, 0, :m_rows]), okmax, okmin, Hkv, reduce=0, last_query=n_chain)
                np.testing.assert_allclose(scores_g[l, 0, :, :nb], osc, rtol=2e-3, atol=2e-2)
                o_pk[l][:], o_pv[l][:] = 0, 0
                plen = oracle.gather(o_k[l], o_v[l], table, new_len, idx_g[l, 0], o_pk[l], o_pv[l], first_page=0)
                n_keep = min(nb, budget)
                gk, gv = wl.to_numpy(pk[l, :n_keep]).copy(), wl.to_numpy(pv[l, :n_keep]).copy()
                tail = plen - (n_keep - 1) * bs
                gk[-1, :, tail:], gv[-1, :, tail:] = 0, 0
                assert np.array_equal(gk, o_pk[l][:n_keep]) and np.array_equal(gv, o_pv[l][:n_keep])
            o_len, o_plen = new_len, plen
            assert int(w.seq_lens[0]) == o_len and int(plens[0]) == o_plen
            pending, initialised = [], True
        else:
            B.specpv_commit_accepted(cfg, 0, L, kn, vn, M_max, acc_t, n_acc, A_max, partial, None, None, ws)
            util.sync_status(ws)
            for l in mirror:
                knn, vnn = wl.to_numpy(kn[l, 0, :m_rows]), wl.to_numpy(vn[l, 0, :m_rows])
                o_new = oracle.commit(knn, vnn, acc, o_pk[l], o_pv[l], ptab, o_plen)
            o_plen = o_new
            assert int(plens[0]) == o_plen
            pending.extend([0] * len(acc))
    assert o_len > int(c["ctx"][0]) and initialised  # the cache has grown by the accepted tokens


@pytest.mark.parametrize("reduce,score_mode", [(0, 0), (1, 0), (2, 0), (0, 1)])
def test_block_scores_repeat_bit_for_bit_under_back_to_back_launches(reduce, score_mode):
    """The score kernel's CTAs each walk a share of all tiles with several warps that meet only on shared-memory
    barriers; a barrier phase that one of them missed shows up as a rare wrong tile, not as a steady error.  Thirty
    back-to-back launches on the ragged batch-4 shape (shares that cross heads, sequences and layers; 8 layers) must
    give the same bits every time, and the first of them the scores the oracle computes for sampled heads."""
    dev = torch.device("cuda")
    w = wl.make_workload("stress_b4", device=dev, n_layers=8)
    c = w.cfg
    L, Hkv, d, bs, M, batch = c["n_layers"], c["Hkv"], c["d"], c["bs"], c["M"], w.batch
    cfg = util.config_for(w, reduce=reduce, score_mode=score_mode)
    full = util.full_cache(w)
    ws = B.new_workspace(cfg, L, batch, full.max_seq_len, M)
    kmax = torch.zeros((L, batch, Hkv, w.max_blocks, d), dtype=torch.bfloat16, device=dev)
    kmin = torch.zeros_like(kmax)
    last_query = torch.tensor([0, 3, M - 1, 7], dtype=torch.int32, device=dev)
    B.specpv_update_block_summaries(cfg, 0, L, full, None, w.max_blocks, kmax, kmin, ws)
    runs = [torch.full((L, batch, Hkv, w.max_blocks), 7.0, dtype=torch.float32, device=dev) for _ in range(30)]
    for s in runs:
        B.specpv_score_blocks(cfg, 0, L, w.q, None, M, last_query, kmax, kmin, full, s, ws)
    util.sync_status(ws)
    for i, s in enumerate(runs[1:], 1):
        assert torch.equal(s, runs[0]), f"launch {i} differs from launch 0"
    got = runs[0].cpu().numpy()
    seq_lens = w.seq_lens.cpu().numpy()
    qn = wl.to_numpy(w.q)
    for (l, b) in [(0, 0), (3, 1), (7, 3), (5, 2)]:  # the oracle on whole (layer, sequence) pairs, every KV head
        nb = (int(seq_lens[b]) + bs - 1) // bs
        want = oracle.block_scores(qn[l, b], util.widen_t(kmax[l, b])[:, :nb], util.widen_t(kmin[l, b])[:, :nb], Hkv, reduce=reduce,
                                   last_query=int(last_query[b]), score_mode=score_mode)
        np.testing.assert_allclose(got[l, b, :, :nb], want, rtol=2e-3, atol=2e-2, err_msg=f"scores l{l} b{b}")
        assert np.all(got[l, b, :, nb:] == 7.0), "blocks past the context must be left alone"
