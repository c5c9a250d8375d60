"""GPU parity of ef_gqa_decode_varlen (decode attention with per-sequence key lengths) against the fp64 oracle."""
import numpy as np
import pytest

from gpu_common import run_parity

pytestmark = pytest.mark.gpu


def test_small_mix_with_empty_entry():
    # lengths 333 (full), 1, 0 (output defined as zero), and two random ones; padding rows hold NaN
    run_parity("gqa_decode_varlen", seed=0, size="small")


@pytest.mark.parametrize("seed", [1, 2])
def test_small_other_seeds(seed):
    run_parity("gqa_decode_varlen", seed=seed, size="small")


@pytest.mark.parametrize("lens", [
    [128, 128, 128],          # exactly one chunk each
    [129, 127, 1],            # one key past / short of a chunk boundary
    [0, 0, 5],                # leading empty entries
    [7, 0, 0],                # trailing empty entries
    [0, 0, 0],                # nothing to attend anywhere: all zeros
    [640, 3, 257],
])
def test_length_patterns(lens):
    run_parity("gqa_decode_varlen", seed=3, size="small", B=3, L=640, lens=lens)


def test_lengths_beyond_lmax_and_negative_are_clamped():
    run_parity("gqa_decode_varlen", seed=4, size="small", B=3, L=200, lens=[5000, -3, 77])


def test_uniform_lengths_agree_with_the_plain_entry_point():
    """With every length equal to Lmax both entry points compute the same function; the item lists differ (the
    per-sequence variant adds one empty item per unit, so blocks split the key range elsewhere), hence not bit for
    bit: both must match the oracle, and each other to a rounding of the bf16 output."""
    import numpy as np
    import torch

    import oracle
    import paper_2609_12330_b200 as ef
    import workloads as wl
    from parity import assert_close

    p, t = wl.make_inputs("gqa_decode_varlen", seed=5, size="small", B=4, L=500, lens=[500] * 4)
    dev = {k: wl.to_torch(k, v, "cuda") for k, v in t.items()}
    ws = ef.Workspace(ef.workspace_bytes("gqa_decode_varlen", p))
    a = ef.gqa_decode_varlen(dev["Q"], dev["K"], dev["V"], dev["seq_lens"], p["scale"], ws)
    b = ef.gqa_decode(dev["Q"], dev["K"], dev["V"], p["scale"], ws)
    ws.check()
    ref = oracle.run("gqa_decode_varlen", p, {k: wl.to_f64(k, v) for k, v in t.items()})
    fa, fb = wl.torch_bf16_to_f64(a), wl.torch_bf16_to_f64(b)
    assert_close(fa, ref, "varlen, uniform lengths")
    assert_close(fb, ref, "plain")
    assert np.max(np.abs(fa - fb)) <= 2.0 ** -8 * np.max(np.abs(ref))


@pytest.mark.parametrize("group", [1, 4, 8])
def test_group_sizes(group):
    run_parity("gqa_decode_varlen", seed=6, size="small", B=4, Hq=2 * group, Hkv=2, L=400)


def test_many_short_sequences():
    # more (batch, kv head) units than blocks, most blocks own several whole units
    run_parity("gqa_decode_varlen", seed=7, size="small", B=200, Hq=8, Hkv=2, L=96)


@pytest.mark.parametrize("lens", [
    [6000, 40, 900],          # one sequence far longer than a block's share: equal ranges, units split and merged
    [5000, 5000, 5000],       # long and even: split as well (few units)
    [1500, 700, 1, 0],        # short enough for one block per whole unit
])
def test_both_partitions(lens):
    """The kernel decides from the lengths whether every block takes one whole (batch, kv head) unit or the item list is
    cut into equal ranges with partial states merged across blocks."""
    run_parity("gqa_decode_varlen", seed=8, size="small", B=len(lens), L=6016, lens=lens)


def test_full_serving_batch():
    run_parity("gqa_decode_varlen", seed=0, size="full")
