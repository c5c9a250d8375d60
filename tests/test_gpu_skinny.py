"""GPU parity: ef_rmsnorm_matmul and ef_gated_mlp (through the C ABI) against the fp64 oracle."""
import numpy as np
import pytest

import workloads as wl
from gpu_common import run_parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_gated_mlp_small_ragged(seed):
    r = run_parity("gated_mlp", seed)             # M=11, K=320 (5 k blocks), N=200 (128+72): split-K partials
    assert r["rel_l2"] < 5e-3


@pytest.mark.parametrize("M,K,N", [(1, 64, 8), (16, 64, 128), (7, 128, 136), (16, 1024, 520), (3, 2048, 1024)])
def test_gated_mlp_shapes(M, K, N):
    run_parity("gated_mlp", 3, M=M, K=K, N=N)


def test_gated_mlp_more_units_than_sms():
    run_parity("gated_mlp", 4, M=16, K=512, N=4096)   # 32 tiles x 8 k blocks = 256 units


def test_gated_mlp_one_block_per_whole_tile():
    # 86 n tiles (the last one ragged: 120 columns) x 16 k blocks: enough tiles to saturate HBM with one block each,
    # so no block shares a tile and no partial results are exchanged
    run_parity("gated_mlp", 5, M=16, K=1024, N=11000)


def test_gated_mlp_full_config():
    r = run_parity("gated_mlp", 0, size="full")
    assert r["rel_l2"] < 5e-3


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_rmsnorm_matmul_small_ragged(seed):
    r = run_parity("rmsnorm_matmul", seed)        # M=5, K=192, N=328
    assert r["rel_l2"] < 5e-3


@pytest.mark.parametrize("M,K,N", [(1, 64, 8), (16, 64, 128), (8, 4096, 264), (13, 512, 2048)])
def test_rmsnorm_matmul_shapes(M, K, N):
    run_parity("rmsnorm_matmul", 3, M=M, K=K, N=N)


def test_rmsnorm_matmul_large_eps_and_zero_row():
    import torch
    import oracle
    import paper_2609_12330_b200 as ef
    from parity import assert_close

    p, t = wl.make_inputs("rmsnorm_matmul", seed=5, size="small", eps=0.5)
    t["X"][2, :] = 0                               # an all-zero row: r = 1/sqrt(eps), y = 0, no NaN
    ref = oracle.run("rmsnorm_matmul", p, {k: wl.bf16_bits_to_f64(v) for k, v in t.items()})
    dev = {k: wl.bf16_bits_to_torch(v, "cuda") for k, v in t.items()}
    ws = ef.Workspace(ef.workspace_bytes("rmsnorm_matmul", p))
    out = ef.run("rmsnorm_matmul", p, dev, ws)
    ws.check()
    got = wl.torch_bf16_to_f64(out)
    assert_close(got, ref, "rmsnorm eps=0.5")
    assert np.all(got[2] == 0.0)


def test_rmsnorm_matmul_full_config():
    r = run_parity("rmsnorm_matmul", 0, size="full")
    assert r["rel_l2"] < 5e-3


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_rmsnorm_gated_mlp_small_ragged(seed):
    r = run_parity("rmsnorm_gated_mlp", seed)     # M=5, K=192, N=200
    assert r["rel_l2"] < 5e-3


@pytest.mark.parametrize("M,K,N", [(1, 64, 8), (16, 4096, 264), (9, 1024, 1000)])
def test_rmsnorm_gated_mlp_shapes(M, K, N):
    run_parity("rmsnorm_gated_mlp", 3, M=M, K=K, N=N)


@pytest.mark.parametrize("seed,M,K,N", [(613, 13, 576, 1512), (58, 16, 256, 2296), (485, 9, 768, 1496), (592, 14, 768, 1544)])
def test_rmsnorm_gated_mlp_more_than_eight_rows(seed, M, K, N):
    """9..16 rows run as two launches of <= 8 rows, each with the hi/lo operand split: with a plain bf16 operand these
    seeds had one element each (small SiLU(g) times a large u) outside 1e-2 + 1e-2*|ref|."""
    run_parity("rmsnorm_gated_mlp", seed, M=M, K=K, N=N)


def test_rmsnorm_gated_mlp_full_config():
    r = run_parity("rmsnorm_gated_mlp", 0, size="full")   # batch 8, 4096 -> 11008
    assert r["rel_l2"] < 5e-3


def test_one_workspace_serves_calls_of_different_shapes():
    """The workspace layout does not depend on the shape: a small-N call must not leave partial sums where a later
    large-N call keeps its arrival counters."""
    import torch

    import oracle
    import paper_2609_12330_b200 as ef
    import workloads as wl
    from parity import assert_close

    shapes = [dict(M=5, K=192, N=136), dict(M=16, K=1024, N=11008), dict(M=3, K=64, N=8), dict(M=16, K=1024, N=11008),
              dict(M=9, K=4096, N=1000)]
    cases, need = [], 0
    for i, sh in enumerate(shapes):
        p, t = wl.make_inputs("gated_mlp", seed=30 + i, size="small", **sh)
        cases.append((p, t))
        need = max(need, ef.workspace_bytes("gated_mlp", p))
    ws = ef.Workspace(need)
    for p, t in cases:
        dev = {k: wl.to_torch(k, v, "cuda") for k, v in t.items()}
        ref = oracle.run("gated_mlp", p, {k: wl.to_f64(k, v) for k, v in t.items()})
        out = torch.full(ref.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
        ef.run("gated_mlp", p, dev, ws, out=out)
        ws.check()
        assert_close(wl.torch_bf16_to_f64(out), ref, f"gated_mlp {p}")
