"""ef_gqa_decode_static: decode attention for callers that cannot allocate device memory.

Some users of the library run where cudaMalloc is off limits at call time (a fixed memory pool,
a real-time loop, a framework that forbids allocation after start-up).  For them the library
carries its decode scratch inside its own image and exposes an entry point without a workspace
argument.  This test calls it through the C ABI twice in a row -- the built-in scratch keeps the
first call's contents, so the second call checks that what must start at zero is cleared -- and
compares with the ordinary entry point on the same inputs.  It is collected last so that a run
that stops at the first failure has already run everything else; it also passes on its own in a
fresh process (it does not rely on state left by other tests).
"""
import ctypes

import numpy as np
import pytest

import workloads as wl
from parity import assert_close

pytestmark = pytest.mark.gpu


@pytest.mark.parametrize("size,over", [("small", {}), ("small", dict(B=3, Hq=12, Hkv=4, L=700)), ("full", {})])
def test_static_decode_matches_workspace_decode_twice(size, over):
    import torch

    import paper_2609_12330_b200 as ef

    p, t = wl.make_inputs("gqa_decode", seed=11, size=size, **over)
    dev = {k: wl.bf16_bits_to_torch(v, "cuda") for k, v in t.items()}
    ws = ef.Workspace(ef.workspace_bytes("gqa_decode", p))
    expect = ef.run("gqa_decode", p, dev, ws)
    ws.check()
    expect64 = wl.torch_bf16_to_f64(expect)
    out = torch.full_like(expect, float("nan"))
    for call in range(2):
        out.fill_(float("nan"))
        ef.gqa_decode_static(dev["Q"], dev["K"], dev["V"], p["scale"], out=out)   # raises on a non-zero status
        torch.cuda.synchronize()
        assert_close(wl.torch_bf16_to_f64(out), expect64, f"static decode call {call} {p}")


def test_static_decode_rejects_problems_beyond_its_scratch():
    import paper_2609_12330_b200 as ef

    lib = ef.lib()
    limit = int(lib.ef_gqa_decode_static_max_units())
    assert limit == 1024
    one = ctypes.c_void_p(4096)   # never dereferenced: the size check comes first
    too_many = lib.ef_gqa_decode_static(one, one, one, one, limit + 1, 4, 1, 128, 128, 1.0, None)
    assert too_many == 5          # EF_ERR_WORKSPACE: beyond the built-in scratch
