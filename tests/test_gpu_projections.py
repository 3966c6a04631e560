"""GPU parity of the linear maps either side of the attention (QKV projection with rotary embedding, step positions,
output projection) against the oracle, through the C ABI: the tensor-core path (bfloat16, head size 128) with one
and several input-feature ranges per tile, several layers, more rows than one accumulator holds, and the plain path
(float32, head size 64, odd hidden sizes)."""
import numpy as np
import pytest
import torch

import oracle
from paper_2512_02337_b200 import binding as B
from paper_2512_02337_b200 import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu


def make_cfg(dtype, Hq, Hkv, d, n_layers):
    return B.make_config(n_layers=n_layers, n_q_heads=Hq, n_kv_heads=Hkv, head_dim=d, block_tokens=64, dtype=dtype,
                         sink_blocks=1, local_blocks=2, budget_blocks=8, buffer_tokens=64)


def rand(shape, dt, g, scale=1.0):
    return (torch.randn(shape, generator=g) * scale).to(dt).to("cuda")


def oracle_cos_sin(pos, d, theta):
    """(cos, sin) [T][d/2] read off the oracle's rotation of the vector (1, .., 1, 0, .., 0)."""
    T = len(pos)
    a = np.zeros((T, 1, d))
    a[:, :, : d // 2] = 1.0
    r = oracle.rope(a, pos, theta)
    return r[:, 0, : d // 2], r[:, 0, d // 2:]


def step_tables(cfg, parents, n_chain, q_lens, base, M_max, d, theta):
    """Device rope table of a step through the C ABI, plus the oracle's positions per sequence."""
    batch = len(parents)
    masks = util.device_masks(parents, M_max, n_chain)
    ql = torch.tensor(q_lens, dtype=torch.int32, device="cuda")
    bp = torch.tensor(base, dtype=torch.int32, device="cuda")
    cos_sin = torch.zeros((batch, M_max, d // 2, 2), dtype=torch.float32, device="cuda")
    B.specpv_rope_table(cfg, masks, ql, bp, batch, M_max, theta, cos_sin)
    pos = [oracle.step_positions(parents[b], n_chain, base[b]) for b in range(batch)]
    return masks, ql, cos_sin, pos


@pytest.mark.parametrize("d,theta", [(128, 5.0e5), (64, 1.0e4)])
def test_rope_table_positions_and_angles(d, theta):
    rng = np.random.default_rng(3)
    n_chain, Ms = 5, [23, 9, 1]
    M_max = max(Ms) + n_chain
    parents = [wl.make_tree(m, min(4, m - 1), 3, rng) for m in Ms]
    cfg = make_cfg("fp32", 4, 2, d, 1)
    base = [131072, 98304 + 17, 0]
    _, _, cos_sin, pos = step_tables(cfg, parents, n_chain, [m + n_chain for m in Ms], base, M_max, d, theta)
    torch.cuda.synchronize()
    got = cos_sin.cpu().numpy()
    for b, m in enumerate(Ms):
        c, s = oracle_cos_sin(pos[b], d, theta)
        # the table is the double-precision angle's cosine and sine rounded once to float32
        np.testing.assert_allclose(got[b, : m + n_chain, :, 0], c, atol=1e-7)
        np.testing.assert_allclose(got[b, : m + n_chain, :, 1], s, atol=1e-7)


CASES = [
    # dtype, Hq, Hkv, d, hidden, batch, M, n_layers (pool), layer0, n_call
    ("fp32", 8, 2, 64, 512, 1, 16, 1, 0, 1),        # plain path, the tiny config's geometry
    ("bf16", 4, 2, 64, 192, 2, 9, 2, 1, 1),         # plain path in bfloat16, second layer of the pool
    ("bf16", 32, 8, 128, 4096, 1, 60, 1, 0, 1),     # tensor cores, one layer: six input ranges per tile
    ("bf16", 8, 2, 128, 448, 1, 37, 3, 1, 2),       # seven 64-wide input steps over seven ranges, layers 1-2 of 3
    ("bf16", 8, 4, 128, 1024, 4, 64, 10, 0, 10),    # 160 tiles: one range per tile, 256 rows per tile
    ("bf16", 4, 2, 128, 256, 5, 64, 1, 0, 1),       # 320 rows: two row chunks
    ("bf16", 2, 2, 128, 64, 1, 1, 1, 0, 1),         # one row, one 64-wide input step, no grouping of heads
    ("bf16", 16, 2, 128, 2048, 3, 43, 2, 0, 2),     # 129 rows: the 128-row staging limit is passed by one
]


@pytest.mark.parametrize("dtype,Hq,Hkv,d,hidden,batch,M,L,layer0,n_call", CASES)
def test_qkv_rope_and_o_proj_match_the_oracle(dtype, Hq, Hkv, d, hidden, batch, M, L, layer0, n_call):
    dt = wl.torch_dtype(dtype)
    g = torch.Generator(device="cpu").manual_seed(hidden + M)
    rng = np.random.default_rng(hidden + M)
    theta = 5.0e5
    cfg = make_cfg(dtype, Hq, Hkv, d, L)
    x = rand((n_call, batch, M, hidden), dt, g)
    res = rand((n_call, batch, M, hidden), dt, g)
    w_qkv = rand((L, (Hq + 2 * Hkv) * d, hidden), dt, g, hidden ** -0.5)
    w_o = rand((L, hidden, Hq * d), dt, g, (Hq * d) ** -0.5)
    attn = rand((n_call, batch, M, Hq, d), dt, g)
    parents = [wl.make_tree(M, min(5, M - 1), 3, rng) for _ in range(batch)]
    base = [int(v) for v in rng.integers(0, 131072, size=batch)]
    _, _, cos_sin, pos = step_tables(cfg, parents, 0, [M] * batch, base, M, d, theta)
    ws = B.new_workspace(cfg, n_call, batch, 4096, M)
    # poisoned outputs: every element must be written
    q = torch.full((n_call, batch, M, Hq, d), float("nan"), dtype=dt, device="cuda")
    k_new = torch.full((n_call, batch, M, Hkv, d), float("nan"), dtype=dt, device="cuda")
    v_new = torch.full_like(k_new, float("nan"))
    y = torch.full((n_call, batch, M, hidden), float("nan"), dtype=dt, device="cuda")
    y_res = torch.full_like(y, float("nan"))
    B.specpv_qkv_rope(cfg, layer0, n_call, x, hidden, w_qkv, cos_sin, batch, M, q, k_new, v_new, ws)
    B.specpv_o_proj(cfg, layer0, n_call, attn, w_o, hidden, None, batch, M, y, ws)
    B.specpv_o_proj(cfg, layer0, n_call, attn, w_o, hidden, res, batch, M, y_res, ws)
    util.sync_status(ws)
    xn, wn, won = wl.to_numpy(x), wl.to_numpy(w_qkv), wl.to_numpy(w_o)
    an, rn = wl.to_numpy(attn), wl.to_numpy(res)
    for l in range(n_call):
        for b in range(batch):
            oq, ok, ov = oracle.qkv_rope(xn[l, b], wn[layer0 + l], Hq, Hkv, d, pos[b], theta)
            util.compare(util.widen_t(q[l, b]), oq, dtype, f"q layer {l} seq {b}")
            util.compare(util.widen_t(k_new[l, b]), ok, dtype, f"k layer {l} seq {b}")
            util.compare(util.widen_t(v_new[l, b]), ov, dtype, f"v layer {l} seq {b}")
            a2 = an[l, b].reshape(M, Hq * d)
            util.compare(util.widen_t(y[l, b]), oracle.linear(a2, won[layer0 + l]), dtype, f"o layer {l} seq {b}")
            util.compare(util.widen_t(y_res[l, b]), oracle.linear(a2, won[layer0 + l], rn[l, b]), dtype,
                         f"o + residual layer {l} seq {b}")


def test_attention_block_of_a_refresh_step_stage_by_stage():
    """rope table -> QKV -> full verification -> output projection on the LLaMA head geometry with a partially
    verified chain in front of the tree; each stage is checked against the oracle run on the previous stage's
    device output (the bytes the next kernel reads)."""
    w = wl.make_workload("llama_32k", device="cuda", n_layers=1, ctx=[3000])
    c = w.cfg
    Hq, Hkv, d, M = c["Hq"], c["Hkv"], c["d"], c["M"]
    n_chain = 7
    M_max = M + n_chain
    bw = wl.make_block_weights("llama_32k", device="cuda", n_layers=1, M=M_max, ctx=[3000])
    cfg = util.config_for(w, out_f32=0)
    cache = util.full_cache(w)
    masks, ql, cos_sin, pos = step_tables(cfg, [w.parents[0]], n_chain, [M_max], [3000], M_max, d, bw.rope_theta)
    ws = B.new_workspace(cfg, 1, 1, 3000, M_max)
    dt = torch.bfloat16
    q = torch.empty((1, 1, M_max, Hq, d), dtype=dt, device="cuda")
    k_new = torch.empty((1, 1, M_max, Hkv, d), dtype=dt, device="cuda")
    v_new = torch.empty_like(k_new)
    out = torch.empty_like(q)
    y = torch.empty((1, 1, M_max, bw.hidden), dtype=dt, device="cuda")
    B.specpv_qkv_rope(cfg, 0, 1, bw.x, bw.hidden, bw.w_qkv, cos_sin, 1, M_max, q, k_new, v_new, ws)
    B.specpv_verify_full(cfg, 0, 1, q, k_new, v_new, masks, ql, M_max, cache, out, None, ws)
    B.specpv_o_proj(cfg, 0, 1, out, bw.w_o, bw.hidden, bw.residual, 1, M_max, y, ws)
    util.sync_status(ws)
    oq, ok, ov = oracle.qkv_rope(wl.to_numpy(bw.x[0, 0]), wl.to_numpy(bw.w_qkv[0]), Hq, Hkv, d, pos[0], bw.rope_theta)
    util.compare(util.widen_t(q[0, 0]), oq, "bf16", "q")
    util.compare(util.widen_t(k_new[0, 0]), ok, "bf16", "k")
    util.compare(util.widen_t(v_new[0, 0]), ov, "bf16", "v")
    mask = oracle.tree_mask(w.parents[0], n_chain)
    o_attn, _ = oracle.tree_attention(wl.to_numpy(q[0, 0]), wl.to_numpy(k_new[0, 0]), wl.to_numpy(v_new[0, 0]), mask,
                                      wl.to_numpy(w.k_pool[0]), wl.to_numpy(w.v_pool[0]),
                                      wl.to_numpy(w.block_table[0]), 3000)
    # the attention output is rounded to bfloat16 here: add half a unit in the last place of its largest value
    tol = 2e-2 + float(np.abs(o_attn).max()) * 2.0 ** -9
    assert np.abs(util.widen_t(out[0, 0]) - o_attn).max() <= tol
    oy = oracle.linear(wl.to_numpy(out[0, 0]).reshape(M_max, Hq * d), wl.to_numpy(bw.w_o[0]),
                       wl.to_numpy(bw.residual[0, 0]))
    util.compare(util.widen_t(y[0, 0]), oy, "bf16", "block output")


@pytest.mark.parametrize("name,layers", [("llama_128k", (0, 13, 31)), ("stress_b4", (0, 31))])
def test_projections_at_full_size_in_the_benchmark_launch(name, layers):
    """All 32 layers of the LLaMA-3.1-8B block shapes in one layer-batched launch each (the configuration the
    benchmark times: 2.7 GB of weights, one input range per tile; batch 4 x 64 rows = one 256-row tile for the
    stress shape).  Checked on sampled layers: every output of every row against the oracle."""
    c = wl.CONFIGS[name]
    L, Hq, Hkv, d, M, batch = c["n_layers"], c["Hq"], c["Hkv"], c["d"], c["M"], len(c["ctx"])
    bw = wl.make_block_weights(name, device="cuda")
    hid = bw.hidden
    cfg = make_cfg("bf16", Hq, Hkv, d, L)
    rng = np.random.default_rng(c["index"])
    parents = [wl.make_tree(M, c["depth"], c["branch"], rng) for _ in range(batch)]
    _, _, cos_sin, pos = step_tables(cfg, parents, 0, [M] * batch, list(c["ctx"]), M, d, bw.rope_theta)
    ws = B.new_workspace(cfg, L, batch, 4096, M)
    dt = torch.bfloat16
    q = torch.full((L, batch, M, Hq, d), float("nan"), dtype=dt, device="cuda")
    k_new = torch.full((L, batch, M, Hkv, d), float("nan"), dtype=dt, device="cuda")
    v_new = torch.full_like(k_new, float("nan"))
    y = torch.full((L, batch, M, hid), float("nan"), dtype=dt, device="cuda")
    attn = bw.x  # any bfloat16 tensor of the right size serves as the attention output here (Hq d = hidden)
    assert Hq * d == hid
    B.specpv_qkv_rope(cfg, 0, L, bw.x, hid, bw.w_qkv, cos_sin, batch, M, q, k_new, v_new, ws)
    B.specpv_o_proj(cfg, 0, L, attn, bw.w_o, hid, bw.residual, batch, M, y, ws)
    util.sync_status(ws)
    assert not torch.isnan(q.float()).any() and not torch.isnan(k_new.float()).any()
    assert not torch.isnan(v_new.float()).any() and not torch.isnan(y.float()).any()
    for l in layers:
        wq, wo = wl.to_numpy(bw.w_qkv[l]), wl.to_numpy(bw.w_o[l])
        for b in range(batch):
            xb = wl.to_numpy(bw.x[l, b])
            oq, ok, ov = oracle.qkv_rope(xb, wq, Hq, Hkv, d, pos[b], bw.rope_theta)
            util.compare(util.widen_t(q[l, b]), oq, "bf16", f"q layer {l} seq {b}")
            util.compare(util.widen_t(k_new[l, b]), ok, "bf16", f"k layer {l} seq {b}")
            util.compare(util.widen_t(v_new[l, b]), ov, "bf16", f"v layer {l} seq {b}")
            util.compare(util.widen_t(y[l, b]), oracle.linear(xb, wo, wl.to_numpy(bw.residual[l, b])), "bf16",
                         f"block output layer {l} seq {b}")
