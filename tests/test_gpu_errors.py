"""Device-detected faults are reported through the status word, never by a trap: a page id outside
the pool, a commit that would overflow the cache.  Every fault here is made on the host (bad
arguments); the kernels skip the offending work item and keep the context usable."""
import numpy as np
import pytest
import torch

from paper_2512_02337_b200 import binding as B
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
