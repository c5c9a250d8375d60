"""GPU parity on seeded random shapes: every program, shapes drawn over the whole supported range (odd sizes, ragged tiles,
one row / one key, more and fewer units than SMs), element by element against the fp64 oracle.

The fixed cases of the other files pin the known corners; this sweep is what found the one accuracy problem the fixed cases
had missed (the gated product for more than eight rows), so a slice of it stays in the suite."""
import random

import pytest

from gpu_common import run_parity

pytestmark = pytest.mark.gpu


def _draw(rng):
    g = rng.choice([1, 2, 4, 8])
    hkv = rng.randint(1, 8)
    L = rng.randint(50, 3000)
    S = rng.randint(1, 700)
    w = rng.randint(1, S)
    return [
        ("gated_mlp", dict(M=rng.randint(1, 16), K=64 * rng.randint(1, 40), N=8 * rng.randint(1, 1500))),
        ("rmsnorm_matmul", dict(M=rng.randint(1, 16), K=64 * rng.randint(1, 24), N=8 * rng.randint(1, 500))),
        ("rmsnorm_gated_mlp", dict(M=rng.randint(1, 16), K=64 * rng.randint(1, 24), N=8 * rng.randint(1, 300))),
        ("layernorm_matmul", dict(M=rng.randint(1, 15), K=64 * rng.randint(1, 24), N=8 * rng.randint(1, 300))),
        ("gqa_decode", dict(B=rng.randint(1, 24), Hq=g * hkv, Hkv=hkv, L=rng.randint(1, 3000))),
        ("gqa_decode_varlen", dict(B=rng.randint(1, 24), Hq=g * hkv, Hkv=hkv, L=rng.randint(1, 3000))),
        ("gqa_decode_window", dict(B=rng.randint(1, 10), Hq=g * hkv, Hkv=hkv, L=L, window=rng.randint(1, L),
                                   sinks=rng.randint(0, 40))),
        ("lora_linear", dict(M=rng.randint(1, 300), K=64 * rng.randint(1, 12), N=8 * rng.randint(2, 200))),
        ("qknorm_attn", dict(B=rng.randint(1, 3), H=rng.randint(1, 6), S=S, causal=rng.randint(0, 1))),
        ("qknorm_attn_ex", dict(B=rng.randint(1, 2), Hq=g * min(hkv, 3), Hkv=min(hkv, 3), S=S, window=w,
                                sinks=rng.choice([0, 0, 3, 64, 128]) if w < S else 0)),
    ]


@pytest.mark.parametrize("sweep_seed", [1, 2, 3])
def test_random_shapes(sweep_seed):
    rng = random.Random(sweep_seed)
    for _ in range(4):
        for program, over in _draw(rng):
            run_parity(program, seed=rng.randrange(1000), size="small", check_repeat=False, **over)
