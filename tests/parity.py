"""Comparator shared by the GPU parity tests: the tolerance stated for bf16 outputs with fp32
accumulation, |gpu - ref| <= 1e-2 + 1e-2*|ref| per element, plus the paper's own validity gate
(relative L2 error <= 0.01, Section 7.1 "Hardware and measurement")."""
import numpy as np

ATOL = 1e-2
RTOL = 1e-2
REL_L2 = 1e-2


def compare(gpu_f64: np.ndarray, ref_f64: np.ndarray):
    assert gpu_f64.shape == ref_f64.shape
    assert np.all(np.isfinite(gpu_f64)), "non-finite GPU output"
    err = np.abs(gpu_f64 - ref_f64)
    bound = ATOL + RTOL * np.abs(ref_f64)
    worst = np.unravel_index(np.argmax(err - bound), err.shape)
    rel_l2 = float(np.linalg.norm(gpu_f64 - ref_f64) / max(np.linalg.norm(ref_f64), 1e-300))
    return dict(ok=bool(np.all(err <= bound)) and rel_l2 <= REL_L2, max_abs=float(err.max()), rel_l2=rel_l2,
                worst=tuple(int(i) for i in worst), worst_gpu=float(gpu_f64[worst]), worst_ref=float(ref_f64[worst]))


def assert_close(gpu_f64, ref_f64, what=""):
    r = compare(gpu_f64, ref_f64)
    assert r["ok"], f"{what}: parity failed {r}"
    return r
