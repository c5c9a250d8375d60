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
