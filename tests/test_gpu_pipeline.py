"""GPU parity of the whole hot path on the tiny float32 config and on a small bfloat16 shape:
summaries, scores, selection, gather, partial and full verification, commit -- each compared with the
CPU oracle through the C ABI."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_02337_b200 import binding as B
from paper_2512_02337_b200 import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu


def run_pipeline(name, n_layers=None, reduce=0, score_mode=0, select_shared=0, **over):
    w = wl.make_workload(name, device="cuda", n_layers=n_layers, spare_tokens=256, **over)
    c = w.cfg
    L, Hq, Hkv, d, bs, M = c["n_layers"], c["Hq"], c["Hkv"], c["d"], c["bs"], c["M"]
    batch = w.batch
    cfg = util.config_for(w, reduce=reduce, score_mode=score_mode, select_shared=select_shared)
    full = util.full_cache(w)
    full.max_seq_len = int(max(c["ctx"])) + 256
    ws = B.new_workspace(cfg, L, batch, full.max_seq_len, M)
    dt = wl.torch_dtype(c["dtype"])
    dev = w.device
    mask = util.device_masks(w.parents, M)
    last_query = torch.zeros(batch, dtype=torch.int32, device=dev)

    # ---- Eq. 1 summaries: bit-exact
    kmax = torch.zeros((L, batch, Hkv, w.max_blocks, d), dtype=dt, device=dev)
    kmin = torch.zeros_like(kmax)
    B.specpv_update_block_summaries(cfg, 0, L, full, None, w.max_blocks, kmax, kmin, ws)
    # ---- Eq. 2-3 scores
    scores = torch.full((L, batch, Hkv, w.max_blocks), float("nan"), dtype=torch.float32, device=dev)
    B.specpv_score_blocks(cfg, 0, L, w.q, None, M, last_query, kmax, kmin, full, scores, ws)
    # ---- selection
    idx = torch.full((L, batch, Hkv, cfg.budget_blocks), -7, dtype=torch.int32, device=dev)
    count = torch.zeros(batch, dtype=torch.int32, device=dev)
    B.specpv_select_partial_kv(cfg, L, scores, w.seq_lens, batch, w.max_blocks, idx, count, ws)
    # ---- gather into the partial cache (pages of sequence b: [b*ppb, (b+1)*ppb), identity table)
    ppb = cfg.budget_blocks + (cfg.buffer_tokens + bs - 1) // bs + 1
    pk = torch.zeros((L, batch * ppb, Hkv, bs, d), dtype=dt, device=dev)
    pv = torch.zeros_like(pk)
    ptable = torch.arange(batch * ppb, dtype=torch.int32, device=dev).reshape(batch, ppb)
    plens = torch.zeros(batch, dtype=torch.int32, device=dev)
    partial = B.Cache(pk, pv, ptable, plens, cfg.budget_blocks * bs + cfg.buffer_tokens)
    B.specpv_refresh_partial(cfg, full, idx, count, partial, plens, ws)
    # ---- verification
    out_full = torch.zeros((L, batch, M, Hq, d), dtype=torch.float32, device=dev)
    lse_full = torch.zeros((L, batch, M, Hq), dtype=torch.float32, device=dev)
    out_part, lse_part = torch.zeros_like(out_full), torch.zeros_like(lse_full)
    B.specpv_verify_full(cfg, 0, L, w.q, w.k_new, w.v_new, mask, None, M, full, out_full, lse_full, ws)
    B.specpv_verify_partial(cfg, 0, L, w.q, w.k_new, w.v_new, mask, None, M, partial, out_part, lse_part, ws)
    if c["dtype"] == "bf16":  # the bfloat16 output is the float32 one, rounded
        cfg16 = util.config_for(w, reduce=reduce, score_mode=score_mode, select_shared=select_shared, out_f32=0)
        o16f, o16p = torch.zeros_like(out_full, dtype=dt), torch.zeros_like(out_full, dtype=dt)
        B.specpv_verify_full(cfg16, 0, L, w.q, w.k_new, w.v_new, mask, None, M, full, o16f, None, ws)
        B.specpv_verify_partial(cfg16, 0, L, w.q, w.k_new, w.v_new, mask, None, M, partial, o16p, None, ws)
        util.same_as_rounded(o16f, out_full)
        util.same_as_rounded(o16p, out_part)
    util.sync_status(ws)

    seq_lens = w.seq_lens.cpu().numpy()
    table = w.block_table.cpu().numpy()
    kp, vp = wl.to_numpy(w.k_pool), wl.to_numpy(w.v_pool)
    qn, knn, vnn = wl.to_numpy(w.q), wl.to_numpy(w.k_new), wl.to_numpy(w.v_new)
    kmax_g, kmin_g = util.widen_t(kmax), util.widen_t(kmin)
    scores_g, idx_g, count_g = scores.cpu().numpy(), idx.cpu().numpy(), count.cpu().numpy()
    pk_g, pv_g, plens_g = wl.to_numpy(pk), wl.to_numpy(pv), plens.cpu().numpy()
    sink, local = cfg.sink_blocks, cfg.local_blocks
    for l in range(L):
        for b in range(batch):
            sl = int(seq_lens[b])
            nb = (sl + bs - 1) // bs
            okmax, okmin = oracle.block_summaries(kp[l], table[b], sl)
            assert np.array_equal(kmax_g[l, b, :, :nb], okmax) and np.array_equal(kmin_g[l, b, :, :nb], okmin)
            osc = oracle.block_scores(qn[l, b], okmax, okmin, Hkv, reduce=reduce, last_query=0, score_mode=score_mode)
            np.testing.assert_allclose(scores_g[l, b, :, :nb], osc, rtol=2e-3 if c["dtype"] == "bf16" else 2e-5,
                                       atol=2e-2 if c["dtype"] == "bf16" else 2e-4)
            assert np.all(np.isnan(scores_g[l, b, :, nb:]))  # untouched beyond the context
            n_keep = min(nb, cfg.budget_blocks)
            assert count_g[b] == n_keep
            if select_shared:  # one list per (layer, sequence), ranked on the mean over the heads
                for h in range(1, Hkv):
                    assert np.array_equal(idx_g[l, b, h, :n_keep], idx_g[l, b, 0, :n_keep])
                util.check_shared_selection(idx_g[l, b, 0, :n_keep], scores_g[l, b, :, :nb], sink, local,
                                            cfg.budget_blocks, f"shared selection l{l} b{b}")
                oidx = idx_g[l, b, :, :n_keep].copy()  # the list the gather below has to follow
            else:
                oidx = np.stack([oracle.select(scores_g[l, b, h, :nb].astype(np.float64), sink, local, cfg.budget_blocks)
                                 for h in range(Hkv)])
                assert np.array_equal(idx_g[l, b, :, :n_keep], oidx)  # bit-exact given the same float32 scores
            opk, opv = np.zeros_like(pk_g[l]), np.zeros_like(pv_g[l])
            oplen = oracle.gather(kp[l], vp[l], table[b], sl, oidx, opk, opv, first_page=b * ppb)
            assert plens_g[b] == oplen
            first, last = b * ppb, b * ppb + n_keep
            gk, gv = pk_g[l, first:last].copy(), pv_g[l, first:last].copy()
            tail = oplen - (n_keep - 1) * bs
            gk[-1, :, tail:], gv[-1, :, tail:] = 0, 0   # tokens past the ragged end are unspecified
            assert np.array_equal(gk, opk[first:last]) and np.array_equal(gv, opv[first:last])
            omask = oracle.tree_mask(w.parents[b])
            assert np.array_equal(omask, B.specpv_build_tree_mask(w.parents[b]))
            o_out, o_lse = oracle.tree_attention(qn[l, b], knn[l, b], vnn[l, b], omask, kp[l], vp[l], table[b], sl)
            util.compare(util.widen_t(out_full[l, b]), o_out, c["dtype"], f"full out l{l} b{b}")
            np.testing.assert_allclose(lse_full[l, b].cpu().numpy(), o_lse, atol=2e-5 if c["dtype"] == "fp32" else 5e-3)
            p_out, p_lse = oracle.tree_attention(qn[l, b], knn[l, b], vnn[l, b], omask, opk, opv,
                                                 ptable[b].cpu().numpy(), oplen)
            util.compare(util.widen_t(out_part[l, b]), p_out, c["dtype"], f"partial out l{l} b{b}")
            np.testing.assert_allclose(lse_part[l, b].cpu().numpy(), p_lse, atol=2e-5 if c["dtype"] == "fp32" else 5e-3)
    return w, cfg, full, partial, ws, (kmax, kmin)


def test_tiny_fp32_config_every_step_matches_oracle():
    run_pipeline("tiny_fp32")


@pytest.mark.parametrize("reduce", [1, 2])
def test_tiny_fp32_other_reductions(reduce):
    run_pipeline("tiny_fp32", reduce=reduce)


def test_small_bf16_llama_shape_pipeline():
    # the 32K LLaMA geometry cut down to 2 layers and 6K tokens so that the oracle covers every row
    run_pipeline("llama_32k", n_layers=2, ctx=[6144 + 37], M=60)


@pytest.mark.parametrize("reduce", [1, 2])
def test_small_bf16_other_reductions(reduce):
    # max / last reductions through the tensor-core score kernel, M = 20 (80 query rows: one Q tile)
    run_pipeline("llama_32k", n_layers=1, reduce=reduce, ctx=[64 * 150 + 11], M=20)


@pytest.mark.parametrize("reduce", [0, 1])
def test_channelwise_score_mode_fp32_and_bf16(reduce):
    # score_mode 1: the maximum is taken per channel; selection, gather and partial verification follow from it
    run_pipeline("tiny_fp32", reduce=reduce, score_mode=1)
    run_pipeline("llama_32k", n_layers=1, reduce=reduce, score_mode=1, ctx=[64 * 90 + 3], M=33)


def test_head_shared_selection_fp32_and_bf16():
    # one block set per (layer, sequence): every head gathers and attends the blocks ranked on the heads' mean score
    run_pipeline("tiny_fp32", select_shared=1)
    run_pipeline("llama_32k", n_layers=2, select_shared=1, ctx=[64 * 120 + 9], M=25)


def test_ragged_batch_shuffled_table_pipeline():
    run_pipeline("stress_b4", n_layers=1, ctx=[4096 + 5, 4800, 5120 - 1, 5120], M=64)


def test_commit_appends_and_updates_summaries():
    w, cfg, full, partial, ws, (kmax, kmin) = run_pipeline("tiny_fp32")
    c = w.cfg
    L, Hkv, d, bs, M = c["n_layers"], c["Hkv"], c["d"], c["bs"], c["M"]
    dev = w.device
    path = wl.path_to(w.parents[0], int(np.argmax([len(wl.path_to(w.parents[0], n)) for n in range(M)])))
    A_max = 8
    acc = torch.zeros((1, A_max), dtype=torch.int32, device=dev)
    acc[0, :len(path)] = torch.from_numpy(path).to(dev)
    n_acc = torch.tensor([len(path)], dtype=torch.int32, device=dev)
    kp0, vp0 = wl.to_numpy(w.k_pool).copy(), wl.to_numpy(w.v_pool).copy()
    sl0 = int(w.seq_lens[0])
    pl0 = int(partial.seq_lens[0])
    ppk0, ppv0 = wl.to_numpy(partial.k_pool).copy(), wl.to_numpy(partial.v_pool).copy()
    # full cache (with summaries) and partial cache (buffer append, no summaries)
    B.specpv_commit_accepted(cfg, 0, L, w.k_new, w.v_new, M, acc, n_acc, A_max, full, kmax, kmin, ws)
    B.specpv_commit_accepted(cfg, 0, L, w.k_new, w.v_new, M, acc, n_acc, A_max, partial, None, None, ws)
    util.sync_status(ws)
    assert int(w.seq_lens[0]) == sl0 + len(path) and int(partial.seq_lens[0]) == pl0 + len(path)
    table = w.block_table.cpu().numpy()
    knn, vnn = wl.to_numpy(w.k_new), wl.to_numpy(w.v_new)
    for l in range(L):
        new_len = oracle.commit(knn[l, 0], vnn[l, 0], path, kp0[l], vp0[l], table[0], sl0)
        assert new_len == sl0 + len(path)
        oracle.commit(knn[l, 0], vnn[l, 0], path, ppk0[l], ppv0[l], partial.block_table[0].cpu().numpy(), pl0)
        okmax, okmin = oracle.block_summaries(kp0[l], table[0], new_len)
        nb = (new_len + bs - 1) // bs
        assert np.array_equal(util.widen_t(kmax[l, 0])[:, :nb], okmax)
        assert np.array_equal(util.widen_t(kmin[l, 0])[:, :nb], okmin)
    assert np.array_equal(wl.to_numpy(w.k_pool), kp0) and np.array_equal(wl.to_numpy(w.v_pool), vp0)
    assert np.array_equal(wl.to_numpy(partial.k_pool), ppk0) and np.array_equal(wl.to_numpy(partial.v_pool), ppv0)
    # incremental summaries == full recompute
    kmax2, kmin2 = torch.zeros_like(kmax), torch.zeros_like(kmin)
    B.specpv_update_block_summaries(cfg, 0, L, full, None, w.max_blocks, kmax2, kmin2, ws)
    nb = (sl0 + len(path) + bs - 1) // bs
    assert torch.equal(kmax[:, :, :, :nb], kmax2[:, :, :, :nb]) and torch.equal(kmin[:, :, :, :nb], kmin2[:, :, :, :nb])


def test_commit_in_layer_groups_matches_the_oracle():
    """A step's commit issued in two layer groups, in ascending order: every group writes its rows at the lengths as
    they stand and the lengths advance with the group that holds the model's last layer."""
    w = wl.make_workload("llama_32k", device="cuda", n_layers=3, spare_tokens=64, ctx=[64 * 20 + 9], M=20)
    c = w.cfg
    L, M = c["n_layers"], c["M"]
    cfg = util.config_for(w)
    full = util.full_cache(w)
    ws = B.new_workspace(cfg, L, 1, int(max(c["ctx"])) + 64, M)
    path = wl.path_to(w.parents[0], int(np.argmax([len(wl.path_to(w.parents[0], n)) for n in range(M)])))
    acc = torch.zeros((1, 8), dtype=torch.int32, device="cuda")
    acc[0, :len(path)] = torch.from_numpy(path).cuda()
    n_acc = torch.tensor([len(path)], dtype=torch.int32, device="cuda")
    kp0, vp0 = wl.to_numpy(w.k_pool).copy(), wl.to_numpy(w.v_pool).copy()
    sl0 = int(w.seq_lens[0])
    B.specpv_commit_accepted(cfg, 0, 2, w.k_new[0:2], w.v_new[0:2], M, acc, n_acc, 8, full, None, None, ws)
    torch.cuda.synchronize()
    assert int(w.seq_lens[0]) == sl0                      # not yet: the last layer is not in this group
    B.specpv_commit_accepted(cfg, 2, 1, w.k_new[2:3], w.v_new[2:3], M, acc, n_acc, 8, full, None, None, ws)
    util.sync_status(ws)
    assert int(w.seq_lens[0]) == sl0 + len(path)
    table = w.block_table.cpu().numpy()
    knn, vnn = wl.to_numpy(w.k_new), wl.to_numpy(w.v_new)
    for l in range(L):
        assert oracle.commit(knn[l, 0], vnn[l, 0], path, kp0[l], vp0[l], table[0], sl0) == sl0 + len(path)
    assert np.array_equal(wl.to_numpy(w.k_pool), kp0) and np.array_equal(wl.to_numpy(w.v_pool), vp0)


@pytest.mark.parametrize("nb,budget", [(300, 40), (2048, 64), (4099, 128), (9000, 1000)])
def test_selection_alone_on_synthetic_scores_with_ties_and_nan(nb, budget):
    """The selection kernel on its own: more candidate blocks than it keeps in registers (nb > 4096), repeated
    scores (ties go to the lower index), NaN (ranks last), -0 / +0; bit-exact against the oracle."""
    dev = "cuda"
    rng = np.random.default_rng(nb)
    Hkv, L, batch, bs = 3, 2, 2, 64
    sc = rng.standard_normal((L, batch, Hkv, nb)).astype(np.float32)
    sc[:, :, 0] = np.round(sc[:, :, 0] * 4) / 4          # many exact ties
    sc[0, 0, 1, rng.integers(0, nb, size=nb // 7)] = np.nan
    sc[1, 1, 2, ::5] = -0.0
    sc[1, 1, 2, 1::5] = 0.0
    lens = np.array([nb * bs - 3, (nb - 5) * bs], dtype=np.int32)  # ragged last block; a shorter second sequence
    cfg = B.make_config(L, 8 * Hkv, Hkv, 128, bs, "bf16", 1, 2, budget, 64)
    scores = torch.from_numpy(sc).to(dev)
    idx = torch.full((L, batch, Hkv, budget), -7, dtype=torch.int32, device=dev)
    count = torch.zeros(batch, dtype=torch.int32, device=dev)
    ws = torch.zeros(4096, dtype=torch.uint8, device=dev)
    B.specpv_select_partial_kv(cfg, L, scores, torch.from_numpy(lens).to(dev), batch, nb, idx, count, ws)
    util.sync_status(ws)
    got = idx.cpu().numpy()
    for b in range(batch):
        n = (int(lens[b]) + bs - 1) // bs
        assert int(count[b]) == min(n, budget)
        for l in range(L):
            for h in range(Hkv):
                want = oracle.select(sc[l, b, h, :n].astype(np.float64), 1, 2, budget)
                assert np.array_equal(got[l, b, h, :len(want)], want), (l, b, h)


@pytest.mark.parametrize("name,L,over", [("tiny_fp32", 1, {}), ("llama_32k", 5, dict(ctx=[5000])),
                                         ("llama_32k", 11, dict(ctx=[1500])), ("stress_b4", 3, dict(ctx=[900, 2100, 64, 1300]))])
def test_verify_host_matches_the_device_call_and_the_oracle(name, L, over):
    """The end-to-end entry point (pinned host step tensors in, host outputs back; layers pipelined in groups of
    1 and 2 with a short last group) against the device-pointer call and, on one layer, the oracle."""
    w = wl.make_workload(name, device="cuda", n_layers=L, spare_tokens=256, **over)  # the bytes of run_pipeline's caches
    c = w.cfg
    Hq, d, M, batch = c["Hq"], c["d"], c["M"], w.batch
    cfg = util.config_for(w)
    full = util.full_cache(w)
    ws = B.new_workspace(cfg, L, batch, int(max(c["ctx"])) + 256, M)
    mask = util.device_masks(w.parents, M)
    out_d = torch.zeros((L, batch, M, Hq, d), dtype=torch.float32, device="cuda")
    lse_d = torch.zeros((L, batch, M, Hq), dtype=torch.float32, device="cuda")
    B.specpv_verify_full(cfg, 0, L, w.q, w.k_new, w.v_new, mask, None, M, full, out_d, lse_d, ws)
    host = [t.cpu().pin_memory() for t in (w.q, w.k_new, w.v_new)]
    mask_h = mask.cpu().pin_memory()
    out_h = torch.full((L, batch, M, Hq, d), float("nan"), dtype=torch.float32).pin_memory()
    lse_h = torch.full((L, batch, M, Hq), float("nan"), dtype=torch.float32).pin_memory()
    for _ in range(2):  # twice: the staging area and the copy streams are reused
        B.specpv_verify_host(cfg, B.MODE_FULL, 0, L, host[0], host[1], host[2], mask_h, M, full, out_h, lse_h, ws)
    util.sync_status(ws)
    # the layer groups may be split over the KV range differently from the one-launch call: two results that are each
    # within the bar of the oracle, not bit-equal to each other
    tol = 2e-5 if c["dtype"] == "fp32" else 4e-2
    assert torch.isfinite(out_h).all() and torch.isfinite(lse_h).all()
    assert (out_h - out_d.cpu()).abs().max().item() <= tol
    assert (lse_h - lse_d.cpu()).abs().max().item() <= tol
    l, b = L - 1, batch - 1
    o_out, o_lse = oracle.tree_attention(wl.to_numpy(w.q[l, b]), wl.to_numpy(w.k_new[l, b]), wl.to_numpy(w.v_new[l, b]),
                                         oracle.tree_mask(w.parents[b]), wl.to_numpy(w.k_pool[l]),
                                         wl.to_numpy(w.v_pool[l]), wl.to_numpy(w.block_table[b]), int(c["ctx"][b]))
    util.compare(out_h[l, b].numpy(), o_out, c["dtype"], "verify_host")
    np.testing.assert_allclose(lse_h[l, b].numpy(), o_lse, atol=5e-3)


@pytest.mark.parametrize("score_mode", [0, 1])
@pytest.mark.parametrize("reduce", [B.REDUCE_MEAN, B.REDUCE_MAX, B.REDUCE_LAST])
def test_scores_of_a_refresh_step_with_more_rows_than_one_accumulator(reduce, score_mode):
    """A refresh scores with the chain and the tree together: 90 and 77 tokens x 4 heads = 360 and 308 query rows per
    KV head, which the tensor-core kernel takes in two passes of 64 tokens (the second sequence's second pass is
    ragged); the "last" row sits in the second pass for one sequence and in the first for the other."""
    w = wl.make_workload("llama_32k", device="cuda", n_layers=2, M=90, ctx=[64 * 140 + 9, 64 * 300 + 1])
    c = w.cfg
    Hkv, d, M, batch, L = c["Hkv"], c["d"], c["M"], w.batch, c["n_layers"]
    cfg = util.config_for(w, reduce=reduce, score_mode=score_mode)
    full = util.full_cache(w)
    ws = B.new_workspace(cfg, L, batch, int(max(c["ctx"])), M)
    kmax = torch.zeros((L, batch, Hkv, w.max_blocks, d), dtype=torch.bfloat16, device="cuda")
    kmin = torch.zeros_like(kmax)
    B.specpv_update_block_summaries(cfg, 0, L, full, None, w.max_blocks, kmax, kmin, ws)
    q_lens = torch.tensor([90, 77], dtype=torch.int32, device="cuda")
    last = torch.tensor([71, 5], dtype=torch.int32, device="cuda")
    scores = torch.full((L, batch, Hkv, w.max_blocks), float("nan"), dtype=torch.float32, device="cuda")
    B.specpv_score_blocks(cfg, 0, L, w.q, q_lens, M, last, kmax, kmin, full, scores, ws)
    util.sync_status(ws)
    for l in range(L):
        for b in range(batch):
            sl = int(c["ctx"][b])
            nb = (sl + c["bs"] - 1) // c["bs"]
            okmax, okmin = oracle.block_summaries(wl.to_numpy(w.k_pool[l]), wl.to_numpy(w.block_table[b]), sl)
            m = int(q_lens[b])
            osc = oracle.block_scores(wl.to_numpy(w.q[l, b, :m]), okmax, okmin, Hkv, reduce=reduce, last_query=int(last[b]),
                                      score_mode=score_mode)
            got = scores[l, b, :, :nb].cpu().numpy().astype(np.float64)
            assert np.isfinite(got).all()
            np.testing.assert_allclose(got, osc, rtol=2e-3, atol=2e-2, err_msg=f"layer {l} seq {b}")
            assert torch.isnan(scores[l, b, :, nb:]).all()  # blocks past the context are left alone
