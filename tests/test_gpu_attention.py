"""GPU parity of the verification attention over a sweep of small shapes and edge cases
(ragged last block, empty context, one-node trees, M not a multiple of 8, refresh chains,
per-sequence row counts, every group size and block size), element by element against the oracle."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_02337_b200 import binding as B
from paper_2512_02337_b200 import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu


@pytest.fixture(autouse=True, params=["single", "pair"])
def attention_kernel(request, monkeypatch):
    """Every case runs on both tensor-core kernels: the default (one CTA per KV range) and the CTA-pair kernel,
    which the library uses on request for shapes with more than 128 query rows per KV head."""
    if request.param == "pair":
        monkeypatch.setenv("SPECPV_ATTN_KERNEL", "pair")
    else:
        monkeypatch.delenv("SPECPV_ATTN_KERNEL", raising=False)
    return request.param


def run_case(dtype, Hq, Hkv, d, bs, ctx, Ms, depth=4, branch=3, n_chain=0, n_layers=1, shuffle=True, seed=0,
             partial_entry=False):
    """One verify call on random data; Ms lists the tree size of every sequence (ragged q_lens)."""
    rng = np.random.default_rng(seed)
    dev = "cuda"
    batch = len(ctx)
    dt = wl.torch_dtype(dtype)
    M_max = max(Ms) + n_chain
    blocks = [(c + bs - 1) // bs + 1 for c in ctx]
    n_pages = sum(blocks) + 2
    max_blocks = max(blocks)
    pages = rng.permutation(n_pages) if shuffle else np.arange(n_pages)
    table = np.zeros((batch, max_blocks), dtype=np.int32)
    off = 0
    for b in range(batch):
        table[b, :blocks[b]] = pages[off:off + blocks[b]]
        off += blocks[b]
    g = torch.Generator(device="cpu").manual_seed(seed)
    k_pool = torch.randn((n_layers, n_pages, Hkv, bs, d), generator=g).to(dt).to(dev)
    v_pool = torch.randn((n_layers, n_pages, Hkv, bs, d), generator=g).to(dt).to(dev)
    q = (torch.randn((n_layers, batch, M_max, Hq, d), generator=g) * 1.5).to(dt).to(dev)
    k_new = torch.randn((n_layers, batch, M_max, Hkv, d), generator=g).to(dt).to(dev)
    v_new = torch.randn((n_layers, batch, M_max, Hkv, d), generator=g).to(dt).to(dev)
    parents = [wl.make_tree(m, min(depth, m - 1), branch, rng) for m in Ms]
    W = (M_max + 63) // 64
    masks = np.zeros((batch, M_max, W), dtype=np.uint64)
    for b in range(batch):
        m = B.specpv_build_tree_mask(parents[b], n_chain, W)
        masks[b, :m.shape[0]] = m
    q_lens = torch.tensor([m + n_chain for m in Ms], dtype=torch.int32, device=dev)
    seq_lens = torch.tensor(ctx, dtype=torch.int32, device=dev)
    cfg = B.make_config(n_layers, Hq, Hkv, d, bs, dtype, 1, 1, 3, bs, out_f32=1)
    cache = B.Cache(k_pool, v_pool, torch.from_numpy(table).to(dev), seq_lens, max(ctx))
    ws = B.new_workspace(cfg, n_layers, batch, max(max(ctx), 1), M_max)
    out = torch.full((n_layers, batch, M_max, Hq, d), 77.0, dtype=torch.float32, device=dev)
    lse = torch.full((n_layers, batch, M_max, Hq), 77.0, dtype=torch.float32, device=dev)
    fn = B.specpv_verify_partial if partial_entry else B.specpv_verify_full
    mask_dev = torch.from_numpy(masks.view(np.int64)).to(dev)
    fn(cfg, 0, n_layers, q, k_new, v_new, mask_dev, q_lens, M_max, cache, out, lse, ws)
    if dtype == "bf16":  # the bfloat16 output is the float32 one, rounded
        cfg16 = B.make_config(n_layers, Hq, Hkv, d, bs, dtype, 1, 1, 3, bs, out_f32=0)
        out16 = torch.full((n_layers, batch, M_max, Hq, d), 77.0, dtype=dt, device=dev)
        fn(cfg16, 0, n_layers, q, k_new, v_new, mask_dev, q_lens, M_max, cache, out16, None, ws)
        util.same_as_rounded(out16, out)
    util.sync_status(ws)
    kp, vp = wl.to_numpy(k_pool), wl.to_numpy(v_pool)
    qn, knn, vnn = wl.to_numpy(q), wl.to_numpy(k_new), wl.to_numpy(v_new)
    for l in range(n_layers):
        for b in range(batch):
            m = Ms[b] + n_chain
            omask = oracle.tree_mask(parents[b], n_chain)
            assert np.array_equal(omask, masks[b, :m, :omask.shape[1]])
            o_out, o_lse = oracle.tree_attention(qn[l, b, :m], knn[l, b, :m], vnn[l, b, :m], omask, kp[l], vp[l],
                                                 table[b], ctx[b])
            util.compare(util.widen_t(out[l, b, :m]), o_out, dtype, f"out l{l} b{b}")
            np.testing.assert_allclose(lse[l, b, :m].cpu().numpy(), o_lse, atol=2e-5 if dtype == "fp32" else 5e-3)
            # rows past q_lens[b] are not written
            assert torch.all(out[l, b, m:].float() == 77.0)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
@pytest.mark.parametrize("Hq,Hkv,d,bs", [(8, 2, 64, 64), (32, 8, 128, 64), (4, 4, 128, 16), (16, 2, 64, 32),
                                          (8, 4, 128, 64)])
def test_shapes_ragged_context(dtype, Hq, Hkv, d, bs):
    run_case(dtype, Hq, Hkv, d, bs, ctx=[bs * 9 + 5, bs * 4], Ms=[13, 7], seed=Hq + d + bs)


@pytest.mark.parametrize("bs", [16, 32])
def test_small_pages_on_the_tensor_core_path(bs):
    """16- and 32-token pages (the paper's block size is 16): eight or four pages per 128-token tile, shuffled
    table, a context long enough to be split over many CTAs with a ragged last page, two layers, refresh rows."""
    run_case("bf16", 32, 8, 128, bs, ctx=[bs * 531 + bs - 3, bs * 7 + 1, 0], Ms=[60, 9, 2], depth=6, branch=4,
             n_layers=2, seed=40 + bs)
    run_case("bf16", 8, 2, 128, bs, ctx=[128 * 20 + 5], Ms=[48], depth=5, branch=4, n_chain=20, seed=41 + bs)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_empty_context_and_single_node_tree(dtype):
    run_case(dtype, 8, 2, 128, 64, ctx=[0, 1, 64], Ms=[5, 1, 1], seed=3)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_refresh_rows_chain_plus_tree(dtype):
    # partially verified chain of 42 tokens in front of a 48-node tree: 90 rows, two mask words
    run_case(dtype, 32, 8, 128, 64, ctx=[64 * 40 + 17], Ms=[48], depth=5, branch=4, n_chain=42, seed=4)


@pytest.mark.parametrize("dtype", ["fp32", "bf16"])
def test_maximum_rows_and_long_split_context(dtype):
    # M_max = 128 (the kernels' limit) and a context long enough to be split across many CTAs
    run_case(dtype, 8, 2, 128, 64, ctx=[64 * 300 + 63], Ms=[128], depth=8, branch=4, seed=5)


def test_partial_entry_point_multi_layer_bf16():
    run_case("bf16", 32, 8, 128, 64, ctx=[64 * 64 + 20, 64 * 70], Ms=[60, 33], depth=6, branch=4, n_layers=3,
             seed=6, partial_entry=True)


def test_chain_tree_matches_torch_causal_sdpa():
    # independent witness on the GPU side as well: a chain tree is causal attention (library SDPA)
    dev = "cuda"
    Hq, Hkv, d, bs, L, M = 8, 2, 64, 64, 64 * 5 + 9, 12
    g = torch.Generator().manual_seed(1)
    n_pages = (L + bs - 1) // bs
    k_pool = torch.randn((1, n_pages, Hkv, bs, d), generator=g).to(dev)
    v_pool = torch.randn((1, n_pages, Hkv, bs, d), generator=g).to(dev)
    q = torch.randn((1, 1, M, Hq, d), generator=g).to(dev)
    k_new = torch.randn((1, 1, M, Hkv, d), generator=g).to(dev)
    v_new = torch.randn((1, 1, M, Hkv, d), generator=g).to(dev)
    mask = util.device_masks([np.arange(-1, M - 1, dtype=np.int32)], M)
    cfg = B.make_config(1, Hq, Hkv, d, bs, "fp32", 1, 1, 3, 64)
    cache = B.Cache(k_pool, v_pool, torch.arange(n_pages, dtype=torch.int32, device=dev)[None],
                    torch.tensor([L], dtype=torch.int32, device=dev), L)
    ws = B.new_workspace(cfg, 1, 1, L, M)
    out = torch.zeros_like(q)
    B.specpv_verify_full(cfg, 0, 1, q, k_new, v_new, mask, None, M, cache, out, None, ws)
    util.sync_status(ws)
    k_all = torch.cat([k_pool[0].permute(0, 2, 1, 3).reshape(-1, Hkv, d)[:L], k_new[0, 0]]).double().cpu()
    v_all = torch.cat([v_pool[0].permute(0, 2, 1, 3).reshape(-1, Hkv, d)[:L], v_new[0, 0]]).double().cpu()
    q_full = torch.cat([torch.zeros((L, Hq, d), dtype=torch.float64), q[0, 0].double().cpu()])
    G = Hq // Hkv
    want = torch.nn.functional.scaled_dot_product_attention(
        q_full.permute(1, 0, 2)[None], k_all.permute(1, 0, 2).repeat_interleave(G, 0)[None],
        v_all.permute(1, 0, 2).repeat_interleave(G, 0)[None], is_causal=True)[0].permute(1, 0, 2)[L:]
    assert (out[0, 0].double().cpu() - want).abs().max() < 1e-5


@pytest.mark.parametrize("where", ["late", "early", "middle_twice"])
def test_large_score_jumps_take_the_general_path(where):
    """The tensor-core kernel keeps a row's reference maximum across full context tiles and only checks the row sum
    for overflow; keys whose scores exceed the reference by hundreds of nats (far beyond float32 range of the
    weights) must send it back over the tile, rescale, and still match the oracle."""
    dev = "cuda"
    Hq, Hkv, d, bs, M = 32, 8, 128, 64, 40
    L_ctx = 64 * 48 + 21
    g = torch.Generator().manual_seed(17)
    n_pages = (L_ctx + bs - 1) // bs + 1
    k_pool = torch.randn((1, n_pages, Hkv, bs, d), generator=g)
    v_pool = torch.randn((1, n_pages, Hkv, bs, d), generator=g)
    q = torch.randn((1, 1, M, Hq, d), generator=g)
    # blocks whose keys are the queries' mean direction, scaled: their logits jump by hundreds of nats
    direction = q[0, 0].mean(dim=(0, 1))
    direction = direction / direction.norm()
    q = q + 8.0 * direction
    boost = {"late": [(40, 400.0)], "early": [(0, 400.0)], "middle_twice": [(9, 150.0), (30, 500.0)]}[where]
    for page, scale in boost:
        k_pool[0, page, :, 5:9] = scale * direction
    to = lambda t: t.to(torch.bfloat16).to(dev)  # noqa: E731
    k_pool, v_pool, q = to(k_pool), to(v_pool), to(q)
    k_new = to(torch.randn((1, 1, M, Hkv, d), generator=g))
    v_new = to(torch.randn((1, 1, M, Hkv, d), generator=g))
    rng = np.random.default_rng(3)
    parents = [wl.make_tree(M, 5, 4, rng)]
    mask = util.device_masks(parents, M)
    cfg = B.make_config(1, Hq, Hkv, d, bs, "bf16", 1, 1, 3, bs, out_f32=1)
    table = torch.arange(n_pages, dtype=torch.int32, device=dev)[None].contiguous()
    cache = B.Cache(k_pool, v_pool, table, torch.tensor([L_ctx], dtype=torch.int32, device=dev), L_ctx)
    ws = B.new_workspace(cfg, 1, 1, L_ctx, M)
    out = torch.zeros((1, 1, M, Hq, d), dtype=torch.float32, device=dev)
    lse = torch.zeros((1, 1, M, Hq), dtype=torch.float32, device=dev)
    B.specpv_verify_full(cfg, 0, 1, q, k_new, v_new, mask, None, M, cache, out, lse, ws)
    util.sync_status(ws)
    o_out, o_lse = oracle.tree_attention(wl.to_numpy(q[0, 0]), wl.to_numpy(k_new[0, 0]), wl.to_numpy(v_new[0, 0]),
                                         oracle.tree_mask(parents[0]), wl.to_numpy(k_pool[0]), wl.to_numpy(v_pool[0]),
                                         table[0].cpu().numpy(), L_ctx)
    assert np.abs(o_lse).max() > 200  # the jump really is beyond what unscaled float32 weights could hold
    util.compare(out[0, 0].cpu().numpy(), o_out, "bf16", f"jump {where}")
    np.testing.assert_allclose(lse[0, 0].cpu().numpy(), o_lse, rtol=2e-5, atol=5e-3)
