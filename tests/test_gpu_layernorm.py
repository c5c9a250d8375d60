"""GPU parity of ef_layernorm_matmul (LayerNorm fused into a projection, one kernel) against the fp64 oracle."""
import pytest

from gpu_common import run_parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_small(seed):
    run_parity("layernorm_matmul", seed=seed, size="small")


@pytest.mark.parametrize("M", [1, 2, 7, 8, 11, 15])
def test_row_counts_across_the_split_threshold(M):
    # M <= 7: hi/lo operand rows with beta in row 7; M >= 8: single rows with beta in row 15
    run_parity("layernorm_matmul", seed=3, size="small", M=M, K=320, N=264)


@pytest.mark.parametrize("K,N", [(64, 8), (64, 136), (1024, 4096), (4096, 1000), (768, 3072)])
def test_shapes(K, N):
    run_parity("layernorm_matmul", seed=4, size="small", M=6, K=K, N=N)


def test_full_config():
    run_parity("layernorm_matmul", seed=0, size="full")


def test_large_mean_rows():
    """Rows whose mean dwarfs their spread: the deviations, not the raw values, feed the tensor core."""
    import numpy as np
    import torch

    import oracle
    import paper_2609_12330_b200 as ef
    import workloads as wl
    from parity import assert_close

    p, t = wl.make_inputs("layernorm_matmul", seed=5, size="small", M=4, K=512, N=256)
    x = wl.bf16_bits_to_f64(t["X"]) * 0.25 + 8.0     # mean 8, spread 0.25 (bf16 keeps 3 fractional bits at 8)
    t["X"] = wl.f32_to_bf16_bits(x.astype(np.float32))
    f64 = {k: wl.to_f64(k, v) for k, v in t.items()}
    ref = oracle.run("layernorm_matmul", p, f64)
    dev = {k: wl.to_torch(k, v, "cuda") for k, v in t.items()}
    ws = ef.Workspace(ef.workspace_bytes("layernorm_matmul", p))
    out = ef.run("layernorm_matmul", p, dev, ws)
    ws.check()
    assert_close(wl.torch_bf16_to_f64(out), ref, "layernorm large mean")


def test_unsupported_row_count_is_refused():
    import torch

    import paper_2609_12330_b200 as ef
    import workloads as wl

    p, t = wl.make_inputs("layernorm_matmul", seed=6, size="small", M=16)
    dev = {k: wl.to_torch(k, v, "cuda") for k, v in t.items()}
    ws = ef.Workspace(1 << 22)
    with pytest.raises(ef.EquiforgeError):
        ef.run("layernorm_matmul", p, dev, ws)
