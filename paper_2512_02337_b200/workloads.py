"""Seeded synthetic workloads shaped like the paper's (no method arithmetic lives here).

The paper measures on PG-19 continuations and LongBench with trained models (Section 4.1); none
of that is available, so these generators stand in for it with the same shapes: head geometry
of LLaMA-3.1-8B / Qwen3-8B, contexts of 2K..128K tokens in paged blocks, draft trees of 16..64
nodes, partial budgets of 512..8192 tokens, and an attention-sparsity structure (a few heavy
hitter tokens, a minority of "hot" blocks the queries are biased towards).

Everything is drawn from ``torch.Generator`` streams keyed by (seed, tensor, layer) so the same
bytes can be handed both to the CUDA library (device tensors) and, copied to the host, to the
CPU oracle.  bfloat16 tensors are converted for the oracle with :func:`to_numpy` (raw uint16 bits).
"""
from __future__ import annotations

from dataclasses import dataclass, field

import numpy as np
import torch

BASE_SEED = 251202337

# name -> parameters.  `ctx` lists the context length of every sequence of the batch.
CONFIGS = {
    # 0: tiny fp32 single layer (the oracle finishes in seconds)
    "tiny_fp32": dict(index=0, n_layers=1, Hq=8, Hkv=2, d=64, bs=64, dtype="fp32", ctx=[2048],
                      M=16, depth=4, branch=4, budget_blocks=8, buffer_tokens=64,
                      heavy=("count", 16, 4.0), hot=None, shuffle=False),
    # 1: LLaMA-3.1-8B attention shape, 32K context
    "llama_32k": dict(index=1, n_layers=32, Hq=32, Hkv=8, d=128, bs=64, dtype="bf16", ctx=[32768],
                      M=60, depth=6, branch=4, budget_blocks=64, buffer_tokens=80,
                      heavy=("frac", 0.02, 3.0), hot=(0.10, 6.0), shuffle=False),
    # 2: same at 128K (budgets 32/64/128 blocks are swept by the caller)
    "llama_128k": dict(index=2, n_layers=32, Hq=32, Hkv=8, d=128, bs=64, dtype="bf16", ctx=[131072],
                       M=60, depth=6, branch=4, budget_blocks=64, buffer_tokens=80,
                       heavy=("frac", 0.02, 3.0), hot=(0.10, 6.0), shuffle=False),
    # 3: Qwen3-8B-like decode loop at 64K
    "qwen3_64k_loop": dict(index=3, n_layers=36, Hq=32, Hkv=8, d=128, bs=64, dtype="bf16", ctx=[65536],
                           M=48, depth=5, branch=4, budget_blocks=64, buffer_tokens=7 * 6 + 48,
                           heavy=("frac", 0.02, 3.0), hot=(0.10, 6.0), shuffle=False),
    # 4: ragged batch-4 stress with a shuffled block table
    "stress_b4": dict(index=4, n_layers=32, Hq=32, Hkv=8, d=128, bs=64, dtype="bf16",
                      ctx=[98304, 114688, 122880, 131072], M=64, depth=6, branch=4, budget_blocks=64,
                      buffer_tokens=84, heavy=("frac", 0.02, 3.0), hot=(0.10, 6.0), shuffle=True),
}


def sink_local_blocks(bs: int) -> tuple[int, int]:
    """Blocks that cover the paper's 32 sink tokens and 128-token local window (Appendix D)."""
    return (32 + bs - 1) // bs, (128 + bs - 1) // bs


def torch_dtype(name: str) -> torch.dtype:
    return {"fp32": torch.float32, "bf16": torch.bfloat16}[name]


def to_numpy(t: torch.Tensor) -> np.ndarray:
    """Host copy in the oracle's convention: float32 as is, bfloat16 as raw uint16 bits."""
    t = t.detach().cpu().contiguous()
    if t.dtype == torch.bfloat16:
        return t.view(torch.int16).numpy().view(np.uint16)
    return t.numpy()


def from_numpy_bits(a: np.ndarray, device) -> torch.Tensor:
    """Inverse of :func:`to_numpy`."""
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).view(torch.bfloat16).to(device)
    return torch.from_numpy(a).to(device)


def make_tree(n_nodes: int, depth: int, branch: int, rng: np.random.Generator) -> np.ndarray:
    """Random draft tree: parents[0] = -1, parents[i] < i, node depth <= depth, children <= branch.

    A spine 0 -> 1 -> ... -> depth guarantees that every path length 1..depth+1 exists."""
    parents = np.full(n_nodes, -1, dtype=np.int32)
    node_depth = np.zeros(n_nodes, dtype=np.int32)
    children = np.zeros(n_nodes, dtype=np.int32)
    for i in range(1, n_nodes):
        if i <= depth:
            p = i - 1
        else:
            ok = np.nonzero((node_depth[:i] < depth) & (children[:i] < branch))[0]
            p = int(ok[rng.integers(len(ok))])
        parents[i] = p
        node_depth[i] = node_depth[p] + 1
        children[p] += 1
    return parents


def path_to(parents: np.ndarray, node: int) -> np.ndarray:
    """Root-to-node path (the accepted tokens of a step when `node` is the last accepted one)."""
    path = []
    while node >= 0:
        path.append(node)
        node = int(parents[node])
    return np.asarray(path[::-1], dtype=np.int32)


@dataclass
class Workload:
    name: str
    cfg: dict
    device: torch.device
    n_pages: int
    max_blocks: int
    k_pool: torch.Tensor        # [n_layers][n_pages][Hkv][bs][d]
    v_pool: torch.Tensor
    block_table: torch.Tensor   # [batch][max_blocks] int32
    seq_lens: torch.Tensor      # [batch] int32
    q: torch.Tensor             # [n_layers][batch][M][Hq][d]
    k_new: torch.Tensor         # [n_layers][batch][M][Hkv][d]
    v_new: torch.Tensor
    parents: np.ndarray         # [batch][M] int32 (host)
    extra: dict = field(default_factory=dict)

    @property
    def batch(self) -> int:
        return len(self.cfg["ctx"])


def _gen(seed: int, tensor_id: int, layer: int, device) -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed((seed * 1000003 + tensor_id * 10007 + layer) % (2 ** 63 - 1))
    return g


def make_workload(name: str, device="cpu", n_layers: int | None = None, spare_tokens: int = 0,
                  **overrides) -> Workload:
    """Build the caches and one step's tensors of a named config.

    ``n_layers`` truncates the layer count (parity tests on a subset of layers);
    ``spare_tokens`` adds room in every sequence's block table for tokens appended later."""
    cfg = dict(CONFIGS[name])
    cfg.update(overrides)
    if n_layers is not None:
        cfg["n_layers"] = n_layers
    device = torch.device(device)
    seed = BASE_SEED + cfg["index"]
    L, Hq, Hkv, d, bs = cfg["n_layers"], cfg["Hq"], cfg["Hkv"], cfg["d"], cfg["bs"]
    dt = torch_dtype(cfg["dtype"])
    ctx = list(cfg["ctx"])
    batch = len(ctx)
    M = cfg["M"]
    blocks_per_seq = [(c + spare_tokens + bs - 1) // bs for c in ctx]
    max_blocks = max(blocks_per_seq)
    n_pages = sum(blocks_per_seq)
    host_rng = np.random.default_rng(seed)

    # block table: consecutive pages per sequence, optionally a seeded shuffle of all pages
    page_ids = np.arange(n_pages, dtype=np.int32)
    if cfg["shuffle"]:
        page_ids = host_rng.permutation(n_pages).astype(np.int32)
    table = np.zeros((batch, max_blocks), dtype=np.int32)
    off = 0
    for b in range(batch):
        table[b, :blocks_per_seq[b]] = page_ids[off:off + blocks_per_seq[b]]
        off += blocks_per_seq[b]
    table_t = torch.from_numpy(table).to(device)

    k_pool = torch.empty((L, n_pages, Hkv, bs, d), dtype=dt, device=device)
    v_pool = torch.empty_like(k_pool)
    q = torch.empty((L, batch, M, Hq, d), dtype=dt, device=device)
    k_new = torch.empty((L, batch, M, Hkv, d), dtype=dt, device=device)
    v_new = torch.empty_like(k_new)
    G = Hq // Hkv

    for layer in range(L):
        g = _gen(seed, 1, layer, device)
        kf = torch.randn((n_pages, Hkv, bs, d), generator=g, device=device, dtype=torch.float32)
        vf = torch.randn((n_pages, Hkv, bs, d), generator=g, device=device, dtype=torch.float32)
        qf = torch.randn((batch, M, Hq, d), generator=g, device=device, dtype=torch.float32)
        knf = torch.randn((batch, M, Hkv, d), generator=g, device=device, dtype=torch.float32)
        vnf = torch.randn((batch, M, Hkv, d), generator=g, device=device, dtype=torch.float32)
        # heavy hitters: a token subset per (layer, kv head) with K and V rows scaled
        kind, amount, scale = cfg["heavy"]
        if kind == "count":
            for h in range(Hkv):
                flat = torch.randperm(n_pages * bs, generator=g, device=device)[: int(amount)]
                kf[flat // bs, h, flat % bs] *= scale
                vf[flat // bs, h, flat % bs] *= scale
        else:
            hit = torch.rand((n_pages, Hkv, bs), generator=g, device=device) < amount
            mult = torch.where(hit, torch.tensor(scale, device=device), torch.tensor(1.0, device=device))
            kf *= mult[..., None]
            vf *= mult[..., None]
            del hit, mult
        # hot blocks: a direction u per (layer, kv head); keys of 10% of the pages and all queries shifted
        if cfg["hot"] is not None:
            frac, shift = cfg["hot"]
            u = torch.randn((Hkv, d), generator=g, device=device)
            u = u / u.norm(dim=-1, keepdim=True)
            hot = torch.rand((n_pages, Hkv), generator=g, device=device) < frac
            kf += (hot[..., None, None] * shift) * u[None, :, None, :]
            qf += shift * u.repeat_interleave(G, dim=0)[None, None]
            del hot
        k_pool[layer] = kf.to(dt)
        v_pool[layer] = vf.to(dt)
        q[layer] = qf.to(dt)
        k_new[layer] = knf.to(dt)
        v_new[layer] = vnf.to(dt)
        del kf, vf, qf, knf, vnf

    parents = np.stack([make_tree(M, cfg["depth"], cfg["branch"], host_rng) for _ in range(batch)])
    return Workload(name=name, cfg=cfg, device=device, n_pages=n_pages, max_blocks=max_blocks,
                    k_pool=k_pool, v_pool=v_pool, block_table=table_t,
                    seq_lens=torch.tensor(ctx, dtype=torch.int32, device=device),
                    q=q, k_new=k_new, v_new=v_new, parents=parents)


# hidden size and rotary base of the attention block each config's head geometry comes from
# (LLaMA-3.1-8B: 4096 / 5e5, Qwen3-8B: 4096 / 1e6; the tiny config: Hq * d / 1e4)
BLOCK_SHAPES = {
    "tiny_fp32": (512, 1.0e4),
    "llama_32k": (4096, 5.0e5),
    "llama_128k": (4096, 5.0e5),
    "qwen3_64k_loop": (4096, 1.0e6),
    "stress_b4": (4096, 5.0e5),
}


@dataclass
class BlockWeights:
    """Synthetic inputs of the linear maps either side of the attention (random-init weights)."""
    hidden: int
    rope_theta: float
    x: torch.Tensor         # [n_layers][batch][M][hidden]   hidden states entering the block
    residual: torch.Tensor  # [n_layers][batch][M][hidden]
    w_qkv: torch.Tensor     # [n_layers][(Hq + 2 Hkv) d][hidden]
    w_o: torch.Tensor       # [n_layers][hidden][Hq d]


def make_block_weights(name: str, device="cpu", n_layers: int | None = None, M: int | None = None,
                       hidden: int | None = None, **overrides) -> BlockWeights:
    """x ~ N(0, 1); weights ~ N(0, 1 / fan-in) so that q, k, v and the block output stay near unit scale."""
    cfg = dict(CONFIGS[name])
    cfg.update(overrides)
    L = cfg["n_layers"] if n_layers is None else n_layers
    M = cfg["M"] if M is None else M
    hid, theta = BLOCK_SHAPES[name]
    hid = hid if hidden is None else hidden
    Hq, Hkv, d = cfg["Hq"], cfg["Hkv"], cfg["d"]
    batch = len(cfg["ctx"])
    dt = torch_dtype(cfg["dtype"])
    device = torch.device(device)
    seed = BASE_SEED + cfg["index"]
    x = torch.empty((L, batch, M, hid), dtype=dt, device=device)
    res = torch.empty_like(x)
    w_qkv = torch.empty((L, (Hq + 2 * Hkv) * d, hid), dtype=dt, device=device)
    w_o = torch.empty((L, hid, Hq * d), dtype=dt, device=device)
    for layer in range(L):
        g = _gen(seed, 2, layer, device)
        x[layer] = torch.randn((batch, M, hid), generator=g, device=device).to(dt)
        res[layer] = torch.randn((batch, M, hid), generator=g, device=device).to(dt)
        w_qkv[layer] = (torch.randn(((Hq + 2 * Hkv) * d, hid), generator=g, device=device) / hid ** 0.5).to(dt)
        w_o[layer] = (torch.randn((hid, Hq * d), generator=g, device=device) / (Hq * d) ** 0.5).to(dt)
    return BlockWeights(hidden=hid, rope_theta=theta, x=x, residual=res, w_qkv=w_qkv, w_o=w_o)
