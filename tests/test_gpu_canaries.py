"""Out-of-bounds writes without a memory checker: every output of the path is a window inside a larger buffer whose
margins hold a sentinel; after the calls the margins must be untouched and the windows fully written.  Runs the
tensor-core and the plain kernels (bfloat16 LLaMA shape, float32 tiny shape) with ragged row counts."""
import numpy as np
import pytest
import torch

from paper_2512_02337_b200 import binding as B
from paper_2512_02337_b200 import workloads as wl
from tests import util

pytestmark = pytest.mark.gpu

GUARD = 4096  # elements of margin on either side


class Guarded:
    """A tensor of `shape` carved out of the middle of a sentinel-filled buffer."""

    def __init__(self, shape, dtype, sentinel, fill):
        n = int(np.prod(shape))
        self.buf = torch.full((n + 2 * GUARD,), sentinel, dtype=dtype, device="cuda")
        self.t = self.buf[GUARD:GUARD + n].view(shape)
        self.t.fill_(fill)
        self.sentinel = sentinel

    def margins_intact(self):
        lo, hi = self.buf[:GUARD], self.buf[-GUARD:]
        if self.buf.dtype.is_floating_point:
            return bool((lo == self.sentinel).all() and (hi == self.sentinel).all())
        return bool(torch.equal(lo, torch.full_like(lo, self.sentinel)) and torch.equal(hi, torch.full_like(hi, self.sentinel)))


@pytest.mark.parametrize("name,over,L", [("llama_32k", dict(ctx=[64 * 150 + 7, 64 * 20]), 2), ("tiny_fp32", dict(), 1)])
def test_no_call_writes_outside_its_outputs(name, over, L):
    w = wl.make_workload(name, device="cuda", n_layers=L, spare_tokens=64, **over)
    c = w.cfg
    Hq, Hkv, d, bs, M, batch = c["Hq"], c["Hkv"], c["d"], c["bs"], c["M"], w.batch
    dt = wl.torch_dtype(c["dtype"])
    cfg = util.config_for(w, out_f32=0)
    full = util.full_cache(w)
    full.max_seq_len = int(max(c["ctx"])) + 64
    ws = B.new_workspace(cfg, L, batch, full.max_seq_len, M)
    mask = util.device_masks(w.parents, M)
    q_lens = torch.tensor([M] + [max(M - 5, 1)] * (batch - 1), dtype=torch.int32, device="cuda")
    nan = float("nan")

    kmax = Guarded((L, batch, Hkv, w.max_blocks, d), dt, 777.0, nan)
    kmin = Guarded((L, batch, Hkv, w.max_blocks, d), dt, 777.0, nan)
    scores = Guarded((L, batch, Hkv, w.max_blocks), torch.float32, 777.0, nan)
    idx = Guarded((L, batch, Hkv, cfg.budget_blocks), torch.int32, -99, -1)
    count = Guarded((batch,), torch.int32, -99, -1)
    ppb = cfg.budget_blocks + (cfg.buffer_tokens + bs - 1) // bs + 1
    pk = Guarded((L, batch * ppb, Hkv, bs, d), dt, 777.0, 0.0)
    pv = Guarded((L, batch * ppb, Hkv, bs, d), dt, 777.0, 0.0)
    plens = Guarded((batch,), torch.int32, -99, -1)
    out_f = Guarded((L, batch, M, Hq, d), dt, 777.0, nan)
    lse_f = Guarded((L, batch, M, Hq), torch.float32, 777.0, nan)
    out_p = Guarded((L, batch, M, Hq, d), dt, 777.0, nan)
    lse_p = Guarded((L, batch, M, Hq), torch.float32, 777.0, nan)
    ptable = torch.arange(batch * ppb, dtype=torch.int32, device="cuda").reshape(batch, ppb).contiguous()
    partial = B.Cache(pk.t, pv.t, ptable, plens.t, cfg.budget_blocks * bs + cfg.buffer_tokens)
    last_query = torch.zeros(batch, dtype=torch.int32, device="cuda")

    B.specpv_update_block_summaries(cfg, 0, L, full, None, w.max_blocks, kmax.t, kmin.t, ws)
    B.specpv_score_blocks(cfg, 0, L, w.q, q_lens, M, last_query, kmax.t, kmin.t, full, scores.t, ws)
    B.specpv_select_partial_kv(cfg, L, scores.t, w.seq_lens, batch, w.max_blocks, idx.t, count.t, ws)
    B.specpv_refresh_partial(cfg, full, idx.t, count.t, partial, plens.t, ws)
    B.specpv_verify_full(cfg, 0, L, w.q, w.k_new, w.v_new, mask, q_lens, M, full, out_f.t, lse_f.t, ws)
    B.specpv_verify_partial(cfg, 0, L, w.q, w.k_new, w.v_new, mask, q_lens, M, partial, out_p.t, lse_p.t, ws)
    util.sync_status(ws)
    for g, what in ((kmax, "kmax"), (kmin, "kmin"), (scores, "scores"), (idx, "idx"), (count, "count"), (pk, "partial K"),
                    (pv, "partial V"), (plens, "partial lengths"), (out_f, "full out"), (lse_f, "full lse"),
                    (out_p, "partial out"), (lse_p, "partial lse")):
        assert g.margins_intact(), f"{what}: a margin was overwritten"
    # the rows in use are fully written, the rows past a sequence's q_len are left alone
    for b in range(batch):
        m = int(q_lens[b])
        for g in (out_f, out_p, lse_f, lse_p):
            assert torch.isfinite(g.t[:, b, :m].float()).all()
            assert torch.isnan(g.t[:, b, m:].float()).all()
        nb = (int(c["ctx"][b]) + bs - 1) // bs
        assert torch.isfinite(scores.t[:, b, :, :nb]).all() and torch.isnan(scores.t[:, b, :, nb:]).all()
        assert torch.isfinite(kmax.t[:, b, :, :nb].float()).all() and torch.isnan(kmax.t[:, b, :, nb:].float()).all()
        n_keep = min(nb, cfg.budget_blocks)
        assert int(count.t[b]) == n_keep and (idx.t[:, b, :, :n_keep] >= 0).all()

    # the linear maps either side of the attention (hidden size of the block shape)
    bw = wl.make_block_weights(name, device="cuda", n_layers=L, **over)
    qg = Guarded((L, batch, M, Hq, d), dt, 777.0, nan)
    kg = Guarded((L, batch, M, Hkv, d), dt, 777.0, nan)
    vg = Guarded((L, batch, M, Hkv, d), dt, 777.0, nan)
    yg = Guarded((L, batch, M, bw.hidden), dt, 777.0, nan)
    cs = Guarded((batch, M, d // 2, 2), torch.float32, 777.0, nan)
    B.specpv_rope_table(cfg, mask, q_lens, w.seq_lens, batch, M, bw.rope_theta, cs.t)
    B.specpv_qkv_rope(cfg, 0, L, bw.x, bw.hidden, bw.w_qkv, cs.t, batch, M, qg.t, kg.t, vg.t, ws)
    attn = torch.randn((L, batch, M, Hq, d), device="cuda").to(dt)
    B.specpv_o_proj(cfg, 0, L, attn, bw.w_o, bw.hidden, bw.residual, batch, M, yg.t, ws)
    util.sync_status(ws)
    for g, what in ((qg, "q"), (kg, "k"), (vg, "v"), (yg, "block output"), (cs, "rope table")):
        assert g.margins_intact(), f"{what}: a margin was overwritten"
        assert torch.isfinite(g.t.float()).all(), f"{what}: not fully written"
