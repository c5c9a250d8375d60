"""GPU parity of ef_gqa_decode_window (decode attention over a sliding window with attention sinks)."""
import pytest

from gpu_common import run_parity

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("seed", [0, 1, 2])
def test_small(seed):
    run_parity("gqa_decode_window", seed=seed, size="small")


@pytest.mark.parametrize("window,sinks", [
    (0, 0), (0, 4),          # no window: the plain program (sinks ignored)
    (1, 0), (1, 4),          # the last key only (+ sinks)
    (127, 0), (128, 4), (129, 4),
    (333, 0), (333, 1), (333, 128), (333, 200), (333, 1400),   # sinks inside one chunk, across chunks, reaching the window
    (1499, 4), (1500, 4), (9999, 4),                          # (almost) everything
])
def test_window_and_sink_sizes(window, sinks):
    run_parity("gqa_decode_window", seed=3, size="small", window=window, sinks=sinks)


@pytest.mark.parametrize("L", [1, 100, 128, 129, 1024, 4097])
def test_history_lengths(L):
    run_parity("gqa_decode_window", seed=4, size="small", L=L, window=200, sinks=4)


@pytest.mark.parametrize("group", [1, 4, 8])
def test_group_sizes(group):
    run_parity("gqa_decode_window", seed=5, size="small", Hq=2 * group, Hkv=2)


def test_many_units():
    run_parity("gqa_decode_window", seed=6, size="small", B=40, Hq=8, Hkv=4, L=900, window=300, sinks=4)


def test_long_history_config():
    # B=8, 32K history, 4 sinks + the last 4096 keys: 1/8 of the cache is read
    run_parity("gqa_decode_window", seed=0, size="full")
