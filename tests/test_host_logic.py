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
    lib = B.lib()
    for name in declared:
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
