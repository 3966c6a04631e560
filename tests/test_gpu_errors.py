"""Device-detected faults are reported through the status word, never by a trap: a page id outside
the pool, a commit that would overflow the cache.  Every fault here is made on the host (bad
arguments); the kernels skip the offending work item and keep the context usable."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_02337_b200 import binding as B
from paper_2512_02337_b200 import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu


def small(dtype="fp32"):
    dev = "cuda"
    Hq, Hkv, d, bs, L, M = 8, 2, 64, 64, 64 * 4, 6
    dt = torch.float32 if dtype == "fp32" else torch.bfloat16
    n_pages = 6
    k_pool = torch.randn((1, n_pages, Hkv, bs, d), device=dev).to(dt)
    v_pool = torch.randn((1, n_pages, Hkv, bs, d), device=dev).to(dt)
    q = torch.randn((1, 1, M, Hq, d), device=dev).to(dt)
    k_new = torch.randn((1, 1, M, Hkv, d), device=dev).to(dt)
    v_new = torch.randn((1, 1, M, Hkv, d), device=dev).to(dt)
    table = torch.arange(5, dtype=torch.int32, device=dev)[None].contiguous()
    cfg = B.make_config(1, Hq, Hkv, d, bs, dtype, 1, 1, 3, 64)
    cache = B.Cache(k_pool, v_pool, table, torch.tensor([L], dtype=torch.int32, device=dev), L)
    ws = B.new_workspace(cfg, 1, 1, L + 64, M)
    mask = util.device_masks([np.arange(-1, M - 1, dtype=np.int32)], M)
    return cfg, cache, ws, (q, k_new, v_new, mask, M)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_bad_page_id_is_reported_and_context_survives(dtype):
    cfg, cache, ws, (q, k_new, v_new, mask, M) = small(dtype)
    out = torch.zeros_like(q)
    cache.block_table[0, 2] = 1000  # outside the pool
    B.specpv_verify_full(cfg, 0, 1, q, k_new, v_new, mask, None, M, cache, out, None, ws)
    st, info = B.specpv_poll_status(ws)
    assert st == 6 and info[2] == 1000
    cache.block_table[0, 2] = -1
    B.specpv_verify_full(cfg, 0, 1, q, k_new, v_new, mask, None, M, cache, out, None, ws)
    assert B.specpv_poll_status(ws)[0] == 6
    # the status was cleared and a valid call works afterwards
    cache.block_table[0, 2] = 2
    B.specpv_verify_full(cfg, 0, 1, q, k_new, v_new, mask, None, M, cache, out, None, ws)
    util.sync_status(ws)
    assert torch.isfinite(out.float()).all()


def test_commit_overflow_is_reported_and_skipped():
    cfg, cache, ws, (q, k_new, v_new, mask, M) = small()
    dev = q.device
    cache.seq_lens[0] = 5 * 64 - 2  # room for two more tokens
    before_k = cache.k_pool.clone()
    acc = torch.tensor([[0, 1, 2, 3]], dtype=torch.int32, device=dev)
    n_acc = torch.tensor([4], dtype=torch.int32, device=dev)
    cache.max_seq_len = 5 * 64
    B.specpv_commit_accepted(cfg, 0, 1, k_new, v_new, M, acc, n_acc, 4, cache, None, None, ws)
    st, info = B.specpv_poll_status(ws)
    assert st == 4
    assert int(cache.seq_lens[0]) == 5 * 64 - 2 and torch.equal(cache.k_pool, before_k)
    n_acc[0] = 2
    B.specpv_commit_accepted(cfg, 0, 1, k_new, v_new, M, acc, n_acc, 4, cache, None, None, ws)
    util.sync_status(ws)
    assert int(cache.seq_lens[0]) == 5 * 64


def test_a_bounded_wait_that_runs_out_reports_timeout_and_the_context_survives():
    """The give-up path of the kernels' barrier waits, on the self-test kernel whose barrier nobody ever arrives on:
    the wait ends after its limit, SPECPV_ERR_TIMEOUT lands in the status word with the self-test's marker, the kernel
    frees its tensor memory and returns, the stream drains, and ordinary calls on the same workspace work afterwards
    (tensor-core and plain kernels)."""
    import time
    cfg, cache, ws, (q, k_new, v_new, mask, M) = small("bf16")
    observed = torch.zeros(1, dtype=torch.int64, device="cuda")
    t0 = time.time()
    B.specpv_selftest_wait_timeout(ws, 1000, observed)          # one millisecond
    st, info = B.specpv_poll_status(ws)                          # synchronises the stream
    assert time.time() - t0 < 5.0
    assert st == 9 and info[0] == B.SELFTEST_WHERE               # SPECPV_ERR_TIMEOUT, recorded by the self-test
    assert 1_000_000 <= int(observed[0]) < 100_000_000           # it waited its limit, not much longer
    assert B.specpv_poll_status(ws)[0] == 0                      # the status was cleared by the poll
    out = torch.zeros_like(q)
    B.specpv_verify_full(cfg, 0, 1, q, k_new, v_new, mask, None, M, cache, out, None, ws)
    util.sync_status(ws)
    assert torch.isfinite(out.float()).all()
    # a tensor-core call (bfloat16, head_dim 128) on a workspace that has seen a time-out
    Hq, Hkv, d, bs, L, M2 = 32, 8, 128, 64, 64 * 6 + 5, 40
    g = torch.Generator().manual_seed(5)
    mk = lambda *shape: torch.randn(shape, generator=g).to(torch.bfloat16).cuda()  # noqa: E731
    k_pool, v_pool = mk(1, 8, Hkv, bs, d), mk(1, 8, Hkv, bs, d)
    q2, kn2, vn2 = mk(1, 1, M2, Hq, d), mk(1, 1, M2, Hkv, d), mk(1, 1, M2, Hkv, d)
    cfg2 = B.make_config(1, Hq, Hkv, d, bs, "bf16", 1, 1, 3, 64, out_f32=1)
    cache2 = B.Cache(k_pool, v_pool, torch.arange(8, dtype=torch.int32, device="cuda")[None].contiguous(),
                     torch.tensor([L], dtype=torch.int32, device="cuda"), L)
    ws2 = B.new_workspace(cfg2, 1, 1, L, M2)
    B.specpv_selftest_wait_timeout(ws2, 500)
    assert B.specpv_poll_status(ws2)[0] == 9
    parents = [wl.make_tree(M2, 5, 4, np.random.default_rng(2))]
    mask2 = util.device_masks(parents, M2)
    out2 = torch.zeros((1, 1, M2, Hq, d), dtype=torch.float32, device="cuda")
    B.specpv_verify_full(cfg2, 0, 1, q2, kn2, vn2, mask2, None, M2, cache2, out2, None, ws2)
    util.sync_status(ws2)
    o_out, _ = oracle.tree_attention(wl.to_numpy(q2[0, 0]), wl.to_numpy(kn2[0, 0]), wl.to_numpy(vn2[0, 0]), oracle.tree_mask(parents[0]),
                                     wl.to_numpy(k_pool[0]), wl.to_numpy(v_pool[0]), np.arange(8, dtype=np.int32), L)
    util.compare(out2[0, 0].cpu().numpy(), o_out, "bf16", "after a time-out")
