"""CPU-only checks: the C-ABI library loads and exports every symbol the header declares, the host
functions (tree mask, mode rule) agree bit-for-bit with the oracle, and argument validation rejects
bad requests before anything is launched."""
import ctypes
import re
from pathlib import Path

import numpy as np
import pytest

import oracle
from paper_2512_02337_b200 import binding as B
from paper_2512_02337_b200 import build as build_mod
from paper_2512_02337_b200 import workloads as wl

ROOT = Path(__file__).resolve().parent.parent


@pytest.fixture(scope="module", autouse=True)
def built():
    build_mod.build()


def test_library_exports_every_declared_symbol():
    header = (ROOT / "include" / "specpv.h").read_text()
    declared = set(re.findall(r"\b(specpv_[a-z_0-9]+)\s*\(", header))
    assert declared == set(B.EXPORTS)
    selftest = (ROOT / "include" / "specpv_selftest.h").read_text()
    declared_selftest = set(re.findall(r"\b(specpv_[a-z_0-9]+)\s*\(", selftest))
    assert declared_selftest == set(B.SELFTEST_EXPORTS)
    lib = B.lib()
    for name in declared | declared_selftest:
        assert getattr(lib, name) is not None


@pytest.mark.parametrize("M,depth,branch,chain", [(1, 0, 1, 0), (16, 4, 4, 0), (60, 6, 4, 0), (64, 6, 4, 0),
                                                  (48, 5, 4, 42), (100, 8, 3, 28), (128, 10, 2, 0), (5, 4, 1, 123)])
def test_tree_mask_bit_exact_with_oracle(M, depth, branch, chain):
    rng = np.random.default_rng(M + chain)
    for _ in range(5):
        parents = wl.make_tree(M, depth, branch, rng)
        assert np.array_equal(B.specpv_build_tree_mask(parents, chain), oracle.tree_mask(parents, chain))
    wide = B.specpv_build_tree_mask(parents, chain, row_words=4)
    assert np.array_equal(wide[:, : (M + chain + 63) // 64], oracle.tree_mask(parents, chain))
    assert not wide[:, (M + chain + 63) // 64:].any()


def test_tree_mask_rejects_bad_trees():
    for bad in ([0], [-1, 1], [-1, 0, 5], [-1, -1], [-1, 0, -2]):
        with pytest.raises(B.SpecPVError) as e:
            B.specpv_build_tree_mask(np.array(bad, dtype=np.int32))
        assert e.value.status == 5
    with pytest.raises(B.SpecPVError) as e:
        B.specpv_build_tree_mask(np.arange(-1, 69, dtype=np.int32), row_words=1)
    assert e.value.status == 4


def test_mode_rule_matches_oracle_on_a_grid():
    for ctx in (0, 100, 4095, 4096, 4097, 100000):
        for budget in (512, 4096):
            for npv in (0, 1, 20, 21, 60):
                for ncand in (1, 48, 60):
                    for buf in (20, 68, 80):
                        for init in (0, 1):
                            assert B.specpv_select_mode(ctx, budget, npv, ncand, buf, init) == \
                                oracle.select_mode(ctx, budget, npv, ncand, buf, init)


def test_config_validation_happens_on_the_host():
    good = dict(n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=64, block_tokens=64, dtype="fp32", sink_blocks=1,
                local_blocks=2, budget_blocks=8, buffer_tokens=64)
    assert B.specpv_workspace_bytes(B.make_config(**good), 2, 1, 2048, 16) > 256
    for key, val in [("n_q_heads", 7), ("head_dim", 96), ("block_tokens", 48), ("dtype", 5), ("budget_blocks", 3),
                     ("local_blocks", 0), ("reduce", 3), ("score_mode", 2), ("softmax_scale", -1.0)]:
        assert B.specpv_workspace_bytes(B.make_config(**{**good, key: val}), 2, 1, 2048, 16) == 0, key
    # null pointers / bad layer ranges are refused before any CUDA call (works without a GPU)
    cfg = B.make_config(**good)
    lib = B.lib()
    kv = B.PagedKV(0, 0, 0, 0, 1, 4, 4, 256)
    st = lib.specpv_verify_full(ctypes.byref(cfg), 0, 1, None, None, None, None, None, 16, ctypes.byref(kv), None,
                                None, None, ctypes.c_size_t(0), None)
    assert st == 1
    assert B.specpv_status_string(0) == "ok" and "capacity" in B.specpv_status_string(4)


def test_projection_and_offload_calls_validate_on_the_host():
    """Bad shapes and null pointers of the linear maps and of the offloaded verification are refused before any CUDA
    call (so this runs without a GPU); 16-byte aligned host buffers stand in for device pointers."""
    cfg = B.make_config(n_layers=2, n_q_heads=8, n_kv_heads=2, head_dim=64, block_tokens=64, dtype="fp32", sink_blocks=1,
                        local_blocks=2, budget_blocks=8, buffer_tokens=64)
    lib = B.lib()
    buf = np.zeros(4096, dtype=np.float32)
    ptr = ctypes.c_void_p(buf.ctypes.data + (-buf.ctypes.data) % 16)
    size = ctypes.c_size_t(1024)

    def qkv(hidden=512, layer0=0, n_layers=1, x=ptr, cos_sin=ptr, ws=ptr):
        return lib.specpv_qkv_rope(ctypes.byref(cfg), layer0, n_layers, x, hidden, ptr, cos_sin, 1, 16, ptr, ptr, ptr, ws,
                                   size, None)
    assert qkv(hidden=100) == 2          # hidden not a multiple of 16
    assert qkv(hidden=0) == 2
    assert qkv(x=None) == 1
    assert qkv(cos_sin=None) == 1
    assert qkv(ws=None) == 1
    assert qkv(layer0=2) == 1            # outside the two layers of the pool
    assert qkv(n_layers=3) == 1
    assert qkv(x=ctypes.c_void_p(ptr.value + 4)) == 1  # misaligned

    def o_proj(hidden=512, attn=ptr, y=ptr):
        return lib.specpv_o_proj(ctypes.byref(cfg), 0, 1, attn, ptr, hidden, None, 1, 16, y, ptr, size, None)
    assert o_proj(hidden=24) == 2
    assert o_proj(attn=None) == 1 and o_proj(y=None) == 1

    def table(theta=1.0e4, batch=1, M=16, mask=ptr):
        return lib.specpv_rope_table(ctypes.byref(cfg), mask, None, ptr, batch, M, ctypes.c_double(theta), ptr, None)
    assert table(theta=1.0) == 1 and table(theta=float("inf")) == 1 and table(theta=float("nan")) == 1
    assert table(batch=0) == 1 and table(mask=None) == 1
    assert table(M=129) == 4             # more rows than the mask words the kernels handle

    off = B.OffloadedKV(ptr, ptr, ptr, ptr, ptr, ptr, 1, 4, 4, 256)
    def staged(kv=off, q=ptr, layer0=0, n_layers=1, M=16):
        return lib.specpv_verify_full_offloaded(ctypes.byref(cfg), layer0, n_layers, q, ptr, ptr, ptr, None, M,
                                                ctypes.byref(kv) if kv is not None else None, ptr, None, ptr, size, None,
                                                None)
    assert staged(kv=None) == 1 and staged(q=None) == 1 and staged(n_layers=3) == 1
    assert staged(kv=B.OffloadedKV(None, ptr, ptr, ptr, ptr, ptr, 1, 4, 4, 256)) == 1
    assert staged(kv=B.OffloadedKV(ptr, ptr, ptr, ptr, ptr, ptr, 1, 4, 4, 257)) == 4   # longer than the table covers
    assert staged(M=129) == 4
    assert staged() == 4                 # a 1 KB workspace cannot hold the split partials


def test_workspace_grows_with_the_request():
    cfg = B.make_config(32, 32, 8, 128, 64, "bf16", 1, 2, 64, 80)
    a = B.specpv_workspace_bytes(cfg, 1, 1, 131072, 60)
    b = B.specpv_workspace_bytes(cfg, 32, 1, 131072, 60)
    c = B.specpv_workspace_bytes(cfg, 32, 4, 131072, 64)
    assert 256 < a < b < c


def _rank_main(rank, world, port, q):
    import torch.distributed as dist
    import torch

    import bench
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    try:
        # each replica reports its own device-timed figures; the job's figure is the slowest replica's
        got = bench.max_over_ranks([10.0 + rank, 5.0 - rank], torch.device("cpu"))
        q.put((rank, got))
    finally:
        dist.destroy_process_group()


def test_replica_timings_are_reduced_with_max_over_ranks_gloo():
    """bench.py --gpus N runs N independent replicas (the path has no exchange step); the only multi-rank
    logic is the MAX reduction of the timings, exercised here with two gloo ranks on the CPU."""
    import socket
    import torch.multiprocessing as mp
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        port = s.getsockname()[1]
    ctx = mp.get_context("spawn")
    q = ctx.Queue()
    procs = [ctx.Process(target=_rank_main, args=(r, 2, port, q)) for r in range(2)]
    for p in procs:
        p.start()
    results = dict(q.get(timeout=120) for _ in range(2))
    for p in procs:
        p.join(timeout=60)
        assert p.exitcode == 0
    assert results[0] == results[1] == [11.0, 5.0]
