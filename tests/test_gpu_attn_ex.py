"""GPU parity of ef_qknorm_attn_ex (grouped KV heads, sliding window, attention sinks) against the fp64 oracle."""
import pytest

from gpu_common import run_parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", [0, 1])
def test_small_window_sinks_gqa(seed):
    run_parity("qknorm_attn_ex", seed=seed, size="small")


@pytest.mark.parametrize("window,sinks", [
    (0, 0),        # no window: the plain causal kernel instance, grouped heads only
    (1, 0),        # every query sees itself only
    (1, 4),        # ... plus the sink keys
    (64, 0),       # window inside one tile
    (128, 0),      # exactly one tile wide: two tiles per row block
    (129, 4),
    (200, 4),
    (300, 128),    # a whole tile of sinks
    (256, 1),
    (699, 4),      # almost everything
    (5000, 4),     # wider than the sequence: treated as no window
])
def test_window_sizes(window, sinks):
    run_parity("qknorm_attn_ex", seed=2, size="small", window=window, sinks=sinks)


@pytest.mark.parametrize("S", [1, 127, 128, 129, 256, 257, 513, 1000])
def test_sequence_lengths(S):
    run_parity("qknorm_attn_ex", seed=3, size="small", S=S, window=150, sinks=3)


@pytest.mark.parametrize("Hq,Hkv", [(1, 1), (8, 1), (8, 2), (6, 3), (4, 4)])
def test_head_groupings(Hq, Hkv):
    run_parity("qknorm_attn_ex", seed=4, size="small", Hq=Hq, Hkv=Hkv, S=400, window=130, sinks=2)


def test_gqa_without_window_noncausal():
    run_parity("qknorm_attn_ex", seed=5, size="small", causal=0, window=0, sinks=0, S=300)


def test_running_max_path_under_a_window():
    """A large scale defeats the a-priori logit bound, so the running maximum with lazy repair runs; rows whose
    first visited tile holds none of their keys must not poison the state."""
    run_parity("qknorm_attn_ex", seed=6, size="small", scale=0.6, S=600, window=140, sinks=0)
    run_parity("qknorm_attn_ex", seed=6, size="small", scale=0.6, S=600, window=140, sinks=5)


def test_batch_and_many_items():
    run_parity("qknorm_attn_ex", seed=7, size="small", B=3, Hq=8, Hkv=2, S=520, window=256, sinks=4)


def test_unsupported_combinations_are_refused():
    import paper_2609_12330_b200 as ef
    import workloads as wl

    ws = ef.Workspace(1 << 24)
    for over in (dict(causal=0, window=100, sinks=0), dict(window=0, sinks=4), dict(window=300, sinks=129)):
        p, t = wl.make_inputs("qknorm_attn_ex", seed=8, size="small", **over)
        dev = {k: wl.to_torch(k, v, "cuda") for k, v in t.items()}
        with pytest.raises(ef.EquiforgeError):
            ef.run("qknorm_attn_ex", p, dev, ws)


def test_long_context_config():
    # B=1, 32 query heads on 8 KV heads, S=8192, window 1024, 4 sinks: the oracle takes a few seconds
    run_parity("qknorm_attn_ex", seed=0, size="full", check_repeat=False)
