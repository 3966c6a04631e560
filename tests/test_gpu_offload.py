"""GPU parity of a refresh step whose FULL cache lives in page-locked host memory (Section 3.3, last paragraph):
full verification staged layer by layer with the next layer's copy in flight, commit of the accepted rows into the
host pools in place, selection on the device-resident summaries and the gather of only the selected blocks from
host memory.  The attention output is checked against the oracle; every other result must equal, bit for bit, the
one the same calls give on a device-resident copy of the cache."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_02337_b200 import binding as B
from paper_2512_02337_b200 import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu


def refresh_tail(cfg, w, cache, q, mask, accepted, n_accepted, A_max, kmax, kmin, ws):
    """commit -> scores -> select -> gather on `cache` (resident or host pools); returns what it produced."""
    c = w.cfg
    L, Hkv, d, bs, M, batch = c["n_layers"], c["Hkv"], c["d"], c["bs"], c["M"], w.batch
    dev = w.device
    dt = wl.torch_dtype(c["dtype"])
    B.specpv_commit_accepted(cfg, 0, L, w.k_new, w.v_new, M, accepted, n_accepted, A_max, cache, kmax, kmin, ws)
    scores = torch.zeros((L, batch, Hkv, w.max_blocks), dtype=torch.float32, device=dev)
    last_query = torch.zeros(batch, dtype=torch.int32, device=dev)
    B.specpv_score_blocks(cfg, 0, L, q, None, M, last_query, kmax, kmin, cache, scores, ws)
    idx = torch.zeros((L, batch, Hkv, cfg.budget_blocks), dtype=torch.int32, device=dev)
    count = torch.zeros(batch, dtype=torch.int32, device=dev)
    B.specpv_select_partial_kv(cfg, L, scores, cache.seq_lens, batch, w.max_blocks, idx, count, ws)
    ppb = cfg.budget_blocks + (cfg.buffer_tokens + bs - 1) // bs + 1
    pk = torch.zeros((L, batch * ppb, Hkv, bs, d), dtype=dt, device=dev)
    pv = torch.zeros_like(pk)
    ptable = torch.arange(batch * ppb, dtype=torch.int32, device=dev).reshape(batch, ppb).contiguous()
    plens = torch.zeros(batch, dtype=torch.int32, device=dev)
    partial = B.Cache(pk, pv, ptable, plens, cfg.budget_blocks * bs + cfg.buffer_tokens)
    B.specpv_refresh_partial(cfg, cache, idx, count, partial, plens, ws)
    return scores, idx, count, pk, pv, plens


@pytest.mark.parametrize("name,over,L", [("llama_32k", dict(ctx=[9000]), 5), ("llama_32k", dict(ctx=[700]), 2),
                                         ("tiny_fp32", dict(), 1),
                                         ("stress_b4", dict(ctx=[3000, 4100, 2000, 3900]), 3)])
def test_refresh_step_with_the_full_cache_in_host_memory(name, over, L):
    w = wl.make_workload(name, device="cuda", n_layers=L, spare_tokens=128, **over)
    c = w.cfg
    Hq, Hkv, d, bs, M, batch = c["Hq"], c["Hkv"], c["d"], c["bs"], c["M"], w.batch
    dev = w.device
    dt = wl.torch_dtype(c["dtype"])
    cfg = util.config_for(w)
    max_len = int(max(c["ctx"])) + 128
    ws = B.new_workspace(cfg, L, batch, max_len, M)
    mask = util.device_masks(w.parents, M)

    # resident reference state and the offloaded one (the same bytes in page-locked host memory)
    lens_res, lens_off = w.seq_lens.clone(), w.seq_lens.clone()
    resident = B.Cache(w.k_pool.clone(), w.v_pool.clone(), w.block_table, lens_res, max_len)
    off = B.OffloadedCache(w.k_pool.cpu().pin_memory(), w.v_pool.cpu().pin_memory(),
                           torch.zeros((2,) + tuple(w.k_pool.shape[1:]), dtype=dt, device=dev),
                           torch.zeros((2,) + tuple(w.k_pool.shape[1:]), dtype=dt, device=dev),
                           w.block_table, lens_off, max_len)
    kmax_r = torch.zeros((L, batch, Hkv, w.max_blocks, d), dtype=dt, device=dev)
    kmin_r = torch.zeros_like(kmax_r)
    B.specpv_update_block_summaries(cfg, 0, L, resident, None, w.max_blocks, kmax_r, kmin_r, ws)
    kmax_o, kmin_o = kmax_r.clone(), kmin_r.clone()

    # ---- full verification: staged from host memory vs resident, and vs the oracle
    out_r = torch.zeros((L, batch, M, Hq, d), dtype=torch.float32, device=dev)
    lse_r = torch.zeros((L, batch, M, Hq), dtype=torch.float32, device=dev)
    out_o, lse_o = torch.full_like(out_r, float("nan")), torch.full_like(lse_r, float("nan"))
    for l in range(L):  # one layer per call, as the staged path issues them: the KV split, and with it the rounding, is the same
        B.specpv_verify_full(cfg, l, 1, w.q[l:l + 1], w.k_new[l:l + 1], w.v_new[l:l + 1], mask, None, M, resident,
                             out_r[l:l + 1], lse_r[l:l + 1], ws)
    copy_stream = torch.cuda.Stream(device=dev)
    for _ in range(2):  # twice: the second call reuses the slots the first one filled
        B.specpv_verify_full_offloaded(cfg, 0, L, w.q, w.k_new, w.v_new, mask, None, M, off, out_o, lse_o, ws,
                                       copy_stream=copy_stream)
    util.sync_status(ws)
    assert torch.equal(out_o, out_r) and torch.equal(lse_o, lse_r)
    # a sub-range of layers lands at the right place too
    if L >= 3:
        out_s = torch.full_like(out_r[1:3], float("nan"))
        B.specpv_verify_full_offloaded(cfg, 1, 2, w.q[1:3], w.k_new[1:3], w.v_new[1:3], mask, None, M, off, out_s, None,
                                       ws, copy_stream=copy_stream)
        util.sync_status(ws)
        assert torch.equal(out_s, out_r[1:3])
    l, b = L - 1, batch - 1
    o_out, o_lse = oracle.tree_attention(wl.to_numpy(w.q[l, b]), wl.to_numpy(w.k_new[l, b]), wl.to_numpy(w.v_new[l, b]),
                                         oracle.tree_mask(w.parents[b]), wl.to_numpy(w.k_pool[l]),
                                         wl.to_numpy(w.v_pool[l]), wl.to_numpy(w.block_table[b]), int(c["ctx"][b]))
    util.compare(out_o[l, b].cpu().numpy(), o_out, c["dtype"], "offloaded full verification")

    # ---- commit the accepted path, re-score, select, gather: host pools in place vs resident
    A_max = 8
    acc = np.zeros((batch, A_max), dtype=np.int32)
    n_acc = np.zeros(batch, dtype=np.int32)
    for bb in range(batch):
        depth = [len(wl.path_to(w.parents[bb], n)) for n in range(M)]
        path = wl.path_to(w.parents[bb], int(np.argmax(depth)))[:A_max]
        acc[bb, :len(path)] = path
        n_acc[bb] = len(path)
    accepted = torch.from_numpy(acc).to(dev)
    n_accepted = torch.from_numpy(n_acc).to(dev)
    res = refresh_tail(cfg, w, resident, w.q, mask, accepted, n_accepted, A_max, kmax_r, kmin_r, ws)
    got = refresh_tail(cfg, w, off.as_cache(), w.q, mask, accepted, n_accepted, A_max, kmax_o, kmin_o, ws)
    util.sync_status(ws)
    assert torch.equal(lens_off, lens_res) and torch.equal(lens_off.cpu(), w.seq_lens.cpu() + torch.from_numpy(n_acc))
    assert torch.equal(off.k_host, resident.k_pool.cpu()) and torch.equal(off.v_host, resident.v_pool.cpu())
    assert torch.equal(kmax_o, kmax_r) and torch.equal(kmin_o, kmin_r)
    for a, r, what in zip(got, res, ("scores", "idx", "count", "partial K", "partial V", "partial lengths")):
        assert torch.equal(a, r), what
    # and the host pools hold what the oracle's commit writes
    kp, vp = wl.to_numpy(w.k_pool[0]).copy(), wl.to_numpy(w.v_pool[0]).copy()
    oracle.commit(wl.to_numpy(w.k_new[0, 0]), wl.to_numpy(w.v_new[0, 0]), acc[0, :n_acc[0]], kp, vp,
                  wl.to_numpy(w.block_table[0]), int(c["ctx"][0]))
    if batch == 1:
        np.testing.assert_array_equal(wl.to_numpy(off.k_host[0]), kp)
        np.testing.assert_array_equal(wl.to_numpy(off.v_host[0]), vp)
