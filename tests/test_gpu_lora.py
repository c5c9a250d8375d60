"""GPU parity: ef_lora_linear (through the C ABI) against the fp64 oracle, element by element."""
import numpy as np
import pytest

import workloads as wl
from gpu_common import run_parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_lora_small_ragged(seed):
    r = run_parity("lora_linear", seed)          # M=200 (128+72), K=192 (3 k blocks), N=328 (256+72)
    assert r["rel_l2"] < 5e-3


@pytest.mark.parametrize("M,K,N", [(1, 64, 8), (128, 64, 256), (129, 128, 264), (300, 512, 1000), (64, 1024, 512)])
def test_lora_shapes(M, K, N):
    run_parity("lora_linear", 3, M=M, K=K, N=N)


def test_lora_alpha_zero_is_plain_gemm():
    run_parity("lora_linear", 4, alpha=0.0)


def test_lora_adapter_dominates():
    # alpha = 25: the rank-16 slab carries as much of the output as the main product, so T and Bm operand layouts are exercised
    run_parity("lora_linear", 5, alpha=25.0)


def test_lora_many_tiles_persistent_loop():
    run_parity("lora_linear", 6, M=1500, K=256, N=3080)   # 12 x 13 = 156 tiles > 148 SMs


def test_lora_full_config():
    r = run_parity("lora_linear", 0, size="full")
    assert r["rel_l2"] < 5e-3


@pytest.mark.parametrize("M", [1, 5, 8, 16, 17])
def test_lora_few_rows_take_the_weight_streaming_tail(M):
    # M <= 16: second kernel = skinny projection with the rank-16 update as one extra k block; 17: the tiled kernel
    run_parity("lora_linear", seed=7, size="small", M=M, K=512, N=1000)


def test_lora_decode_shape():
    # the B=1 LoRA case of Section 7.2 at the benchmark's layer size
    run_parity("lora_linear", seed=8, size="full", M=1)


def test_lora_few_rows_adapter_dominates():
    run_parity("lora_linear", seed=9, size="small", M=4, K=256, N=264, alpha=25.0)


@pytest.mark.parametrize("M,K,N", [(512, 256, 9728), (400, 192, 9736), (300, 128, 19464)])
def test_lora_256_row_block_tiles(M, K, N):
    # enough 128x256 tiles for two waves of the grid: the kernel instance with 256-row block tiles runs,
    # with ragged rows in the last tile and a ragged last column tile
    run_parity("lora_linear", seed=10, size="small", M=M, K=K, N=N, check_repeat=False)


def test_lora_workspace_reused_across_shapes_and_calls():
    """One workspace, calls of different shapes in a row: the in-kernel hand-over of T (per-piece ready words keyed by
    an epoch) must not be confused by words a differently shaped earlier call left behind."""
    import numpy as np
    import torch

    import oracle
    import paper_2609_12330_b200 as ef
    import workloads as wl
    from parity import assert_close

    shapes = [dict(M=256, K=128, N=264), dict(M=700, K=192, N=520), dict(M=130, K=64, N=256), dict(M=700, K=192, N=520),
              dict(M=9, K=128, N=264), dict(M=512, K=256, N=9728), dict(M=256, K=128, N=264)]
    need = 0
    cases = []
    for i, sh in enumerate(shapes):
        p, t = wl.make_inputs("lora_linear", seed=20 + i, size="small", **sh)
        need = max(need, ef.workspace_bytes("lora_linear", p))
        cases.append((p, t))
    ws = ef.Workspace(need)
    for p, t in cases:
        dev = {k: wl.to_torch(k, v, "cuda") for k, v in t.items()}
        ref = oracle.run("lora_linear", p, {k: wl.to_f64(k, v) for k, v in t.items()})
        for _ in range(2):
            out = torch.full(ref.shape, float("nan"), dtype=torch.bfloat16, device="cuda")
            ef.run("lora_linear", p, dev, ws, out=out)
            ws.check()
            assert_close(wl.torch_bf16_to_f64(out), ref, f"lora {p}")
