"""The allocation-free entry point, specpv_verify_partial_static, against specpv_verify_partial and the oracle.

Some users of this library cannot pass a workspace because they cannot allocate device memory where
they call it (a server whose memory pool already owns the whole GPU, a plug-in inside a decode loop
where an allocation would stall the device).  For them the library carries a fixed scratch array; this
test checks that the call which uses it gives the same attention output as the ordinary entry point
(and, on one layer and sequence, as the float64 oracle), twice in a row with different inputs (the array
keeps the first call's contents), and that it refuses
a request that does not fit the array.  The file sorts last on purpose: a run that stops at the first
failure has then already run every other test.
"""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_02337_b200 import binding as B
from paper_2512_02337_b200 import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu


def _case(seed, Hq=32, Hkv=8, d=128, bs=64, n_layers=2, ctx=(64 * 40 + 17, 64 * 33), Ms=(60, 41)):
    """A partial cache long enough to be split over several CTAs, with ragged lengths and tree sizes."""
    dev = "cuda"
    rng = np.random.default_rng(seed)
    g = torch.Generator().manual_seed(seed)
    batch, M_max = len(ctx), max(Ms)
    blocks = [(c + bs - 1) // bs + 2 for c in ctx]
    n_pages, max_blocks = sum(blocks), max(blocks)
    table = np.zeros((batch, max_blocks), dtype=np.int32)
    pages, off = rng.permutation(n_pages), 0
    for b in range(batch):
        table[b, :blocks[b]] = pages[off:off + blocks[b]]
        off += blocks[b]
    mk = lambda *shape, s=1.0: (torch.randn(shape, generator=g) * s).to(torch.bfloat16).to(dev)  # noqa: E731
    k_pool, v_pool = mk(n_layers, n_pages, Hkv, bs, d), mk(n_layers, n_pages, Hkv, bs, d)
    q, k_new, v_new = mk(n_layers, batch, M_max, Hq, d, s=1.5), mk(n_layers, batch, M_max, Hkv, d), mk(n_layers, batch, M_max, Hkv, d)
    parents = [wl.make_tree(m, min(5, m - 1), 4, rng) for m in Ms]
    mask = util.device_masks(parents, M_max)
    q_lens = torch.tensor(Ms, dtype=torch.int32, device=dev)
    budget = max(blocks) - 2
    cfg = B.make_config(n_layers, Hq, Hkv, d, bs, "bf16", 1, 2, budget, bs, out_f32=1)
    cache = B.Cache(k_pool, v_pool, torch.from_numpy(table).to(dev), torch.tensor(ctx, dtype=torch.int32, device=dev),
                    max(ctx))
    return cfg, n_layers, q, k_new, v_new, mask, q_lens, M_max, cache, Ms, parents, table


def test_static_scratch_matches_workspace_entry_point_twice():
    for seed in (11, 12):  # two calls in a row on the same scratch array, different inputs
        cfg, L, q, k_new, v_new, mask, q_lens, M_max, cache, Ms, parents, table = _case(seed)
        shape = (L, len(Ms), M_max, cfg.n_q_heads, cfg.head_dim)
        want = torch.full(shape, 77.0, dtype=torch.float32, device="cuda")
        want_lse = torch.full(shape[:-1], 77.0, dtype=torch.float32, device="cuda")
        ws = B.new_workspace(cfg, L, len(Ms), cache.max_seq_len, M_max)
        B.specpv_verify_partial(cfg, 0, L, q, k_new, v_new, mask, q_lens, M_max, cache, want, want_lse, ws)
        util.sync_status(ws)

        got = torch.full(shape, 77.0, dtype=torch.float32, device="cuda")
        got_lse = torch.full(shape[:-1], 77.0, dtype=torch.float32, device="cuda")
        status = torch.full((5,), -1, dtype=torch.int32, device="cuda")
        B.specpv_verify_partial_static(cfg, 0, L, q, k_new, v_new, mask, q_lens, M_max, cache, got, got_lse, status)
        torch.cuda.synchronize()
        assert status.tolist() == [0, 0, 0, 0, 0]
        for b, m in enumerate(Ms):
            # the two entry points must agree
            util.compare(got[:, b, :m].cpu().numpy(), want[:, b, :m].double().cpu().numpy(), "bf16", f"seed {seed} seq {b}")
            np.testing.assert_allclose(got_lse[:, b, :m].cpu().numpy(), want_lse[:, b, :m].cpu().numpy(), atol=5e-3)
            assert torch.all(got[:, b, m:] == 77.0)  # rows past q_lens are not written
        # and the allocation-free call on its own against the oracle: last layer, second sequence
        l, b, m = L - 1, 1, Ms[1]
        o_out, o_lse = oracle.tree_attention(wl.to_numpy(q[l, b, :m]), wl.to_numpy(k_new[l, b, :m]), wl.to_numpy(v_new[l, b, :m]),
                                             oracle.tree_mask(parents[b]), wl.to_numpy(cache.k_pool[l]),
                                             wl.to_numpy(cache.v_pool[l]), table[b], int(cache.seq_lens[b]))
        util.compare(got[l, b, :m].cpu().numpy(), o_out, "bf16", f"seed {seed} against the oracle")
        np.testing.assert_allclose(got_lse[l, b, :m].cpu().numpy(), o_lse, atol=5e-3)


def test_static_scratch_rejects_requests_beyond_the_array():
    # one split's partial results of 48 layers x 4 sequences do not fit twice into the fixed array
    cfg, L, q, k_new, v_new, mask, q_lens, M_max, cache, Ms, _, _ = _case(13, n_layers=1)
    per_split = 48 * 4 * cfg.n_kv_heads * 256 * (cfg.head_dim + 2) * 4
    assert 2 * per_split > B.STATIC_SCRATCH_BYTES - B.WORKSPACE_HEAD_BYTES
    big = B.make_config(48, cfg.n_q_heads, cfg.n_kv_heads, cfg.head_dim, cfg.block_tokens, "bf16", 1, 2,
                        cfg.budget_blocks, cfg.buffer_tokens, out_f32=1)
    wide = B.Cache(cache.k_pool, cache.v_pool, cache.block_table.repeat(2, 1).contiguous(),
                   cache.seq_lens.repeat(2).contiguous(), cache.max_seq_len)
    out = torch.zeros(1, device="cuda")
    with pytest.raises(B.SpecPVError) as err:
        # nothing is launched on a refusal, so the undersized tensors are never touched
        B.specpv_verify_partial_static(big, 0, 48, q, k_new, v_new, mask, None, M_max, wide, out, None, None)
    assert err.value.status == 4  # SPECPV_ERR_CAPACITY
