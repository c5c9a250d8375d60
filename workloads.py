"""Seeded synthetic inputs for the five fused tensor programs.

This module is the only code shared by the CPU oracle's tests and the CUDA
path's tests/benchmark.  It holds no arithmetic of the method itself: it draws
normal variates from a counter-based generator (Philox), scales and shifts
them, rounds to bfloat16 (round-to-nearest-even) and hands out the resulting
bit patterns.  Both sides consume the identical bits.

Reading of the workload notation "~N(mu, s)": the second parameter is the
standard deviation (1/32 = 1/sqrt(1024) and 1/64 = 1/sqrt(4096) are fan-in
scalings that give unit-variance products).

The paper evaluates on the Mirage/Prism benchmark definitions with Llama-2 and
BERT shapes (Section 7.1, "Workloads"); those shapes are not printed in the
paper, so the shapes below (bf16 activations at batch 8/16 tokens, a
4096->11008 gated MLP, 32x128 attention heads, a rank-16 adapter) stand in
for them.
"""
from __future__ import annotations

import numpy as np

PROGRAMS = ("rmsnorm_matmul", "gated_mlp", "gqa_decode", "qknorm_attn", "lora_linear")
# programs beyond the five benchmark configurations (the "next" rows of the scope table)
EXTRA_PROGRAMS = ("rmsnorm_gated_mlp", "gqa_decode_varlen", "layernorm_matmul", "qknorm_attn_ex", "gqa_decode_window")
_PROGRAM_ID = {name: i for i, name in enumerate(PROGRAMS + EXTRA_PROGRAMS)}


# ----------------------------------------------------------------------------
# bf16 bit handling (storage format only)
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 values to bfloat16 (nearest-even); return uint16 bit patterns."""
    u = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = u + np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f64(bits: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns to float64."""
    u = np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def bf16_bits_to_torch(bits: np.ndarray, device="cpu"):
    """bfloat16 torch tensor holding exactly these bit patterns."""
    import torch

    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16).copy())
    return t.view(torch.bfloat16).to(device)


INT_TENSORS = ("seq_lens",)   # tensor names that are int32, not bf16 bit patterns


def to_torch(name: str, arr: np.ndarray, device="cpu"):
    """Torch tensor for one entry of make_inputs()'s tensor dict (bf16 bits, or int32 for INT_TENSORS)."""
    if name in INT_TENSORS:
        import torch

        return torch.from_numpy(np.ascontiguousarray(arr, dtype=np.int32).copy()).to(device)
    return bf16_bits_to_torch(arr, device)


def to_f64(name: str, arr: np.ndarray) -> np.ndarray:
    """Oracle-side view of one entry of the tensor dict (exact widening; int tensors stay int32)."""
    if name in INT_TENSORS:
        return np.ascontiguousarray(arr, dtype=np.int32)
    return bf16_bits_to_f64(arr)


def torch_bf16_to_f64(t) -> np.ndarray:
    """Exact widening of a torch bfloat16 tensor (any device) to a float64 numpy array."""
    import torch

    bits = t.detach().contiguous().cpu().view(torch.int16).numpy().view(np.uint16)
    return bf16_bits_to_f64(bits)


# ----------------------------------------------------------------------------
# generator
# ----------------------------------------------------------------------------
def _normal_bf16(seed: int, program: str, tensor_index: int, shape, mean: float, std: float) -> np.ndarray:
    ss = np.random.SeedSequence([int(seed), _PROGRAM_ID[program], int(tensor_index)])
    rng = np.random.Generator(np.random.Philox(ss))
    a = rng.standard_normal(size=shape, dtype=np.float32)
    a = a * np.float32(std) + np.float32(mean)
    return f32_to_bf16_bits(a)


# ----------------------------------------------------------------------------
# workload shapes
# ----------------------------------------------------------------------------
# "full" entries are the benchmark configurations; "small" entries are sized so
# the oracle finishes in well under a second while still spanning several
# tiles and ragged tails of the kernels.
SHAPES = {
    "rmsnorm_matmul": {
        "full": dict(M=8, K=1024, N=4096, eps=1e-6),
        "small": dict(M=5, K=192, N=328, eps=1e-6),
    },
    "gated_mlp": {
        "full": dict(M=16, K=4096, N=11008),
        "small": dict(M=11, K=320, N=200),
    },
    "rmsnorm_gated_mlp": {  # RMSNorm-MLP at batch 8 (Section 7.2), Llama-2-7B MLP shape
        "full": dict(M=8, K=4096, N=11008, eps=1e-6),
        "small": dict(M=5, K=192, N=200, eps=1e-6),
    },
    "layernorm_matmul": {  # LayerNorm+GEMM at batch 8, BERT-large hidden size into its 4x intermediate layer
        "full": dict(M=8, K=1024, N=4096, eps=1e-5),
        "small": dict(M=5, K=192, N=328, eps=1e-5),
    },
    "gqa_decode": {
        "full": dict(B=8, Hq=32, Hkv=8, L=4096, D=128, scale=1.0 / np.sqrt(128.0)),
        "small": dict(B=2, Hq=8, Hkv=2, L=333, D=128, scale=1.0 / np.sqrt(128.0)),
    },
    "gqa_decode_window": {  # one query token over a 32K history: 4 sink tokens + the last 4096 (Section 7.3), batch 8
        "full": dict(B=8, Hq=32, Hkv=8, L=32768, D=128, scale=1.0 / np.sqrt(128.0), window=4096, sinks=4),
        "small": dict(B=2, Hq=8, Hkv=2, L=1500, D=128, scale=1.0 / np.sqrt(128.0), window=333, sinks=4),
    },
    "gqa_decode_varlen": {  # serving batch with a length mix: lengths uniform in [1, L], one full, one of length 1
        "full": dict(B=16, Hq=32, Hkv=8, L=4096, D=128, scale=1.0 / np.sqrt(128.0)),
        "small": dict(B=5, Hq=8, Hkv=2, L=333, D=128, scale=1.0 / np.sqrt(128.0)),
    },
    "qknorm_attn": {
        "full": dict(B=2, H=32, S=2048, D=128, eps=1e-6, scale=1.0 / np.sqrt(128.0), causal=1),
        "small": dict(B=1, H=2, S=300, D=128, eps=1e-6, scale=1.0 / np.sqrt(128.0), causal=1),
    },
    "qknorm_attn_ex": {  # long-context prefill: grouped KV heads, sliding window with sink tokens (Section 7.3)
        "full": dict(B=1, Hq=32, Hkv=8, S=8192, D=128, eps=1e-6, scale=1.0 / np.sqrt(128.0), causal=1, window=1024, sinks=4),
        "small": dict(B=1, Hq=4, Hkv=2, S=700, D=128, eps=1e-6, scale=1.0 / np.sqrt(128.0), causal=1, window=200, sinks=4),
    },
    "lora_linear": {
        "full": dict(M=2048, K=4096, N=4096, R=16, alpha=2.0),
        "small": dict(M=200, K=192, N=328, R=16, alpha=2.0),
    },
}


def make_inputs(program: str, seed: int = 0, size: str = "full", **overrides):
    """Return (params, tensors): params is the shape/scalar dict, tensors maps the
    argument name to a uint16 array of bfloat16 bit patterns, in signature order."""
    p = dict(SHAPES[program][size])
    p.update(overrides)
    g = lambda idx, shape, mean, std: _normal_bf16(seed, program, idx, shape, mean, std)
    if program == "rmsnorm_matmul":
        M, K, N = p["M"], p["K"], p["N"]
        t = {
            "X": g(0, (M, K), 0.0, 1.0),
            "gamma": g(1, (K,), 1.0, 0.1),
            "W": g(2, (K, N), 0.0, 1.0 / np.sqrt(K)),
        }
    elif program == "gated_mlp":
        M, K, N = p["M"], p["K"], p["N"]
        t = {
            "X": g(0, (M, K), 0.0, 1.0),
            "Wgate": g(1, (K, N), 0.0, 1.0 / np.sqrt(K)),
            "Wup": g(2, (K, N), 0.0, 1.0 / np.sqrt(K)),
        }
    elif program == "rmsnorm_gated_mlp":
        M, K, N = p["M"], p["K"], p["N"]
        t = {
            "X": g(0, (M, K), 0.0, 1.0),
            "gamma": g(1, (K,), 1.0, 0.1),
            "Wgate": g(2, (K, N), 0.0, 1.0 / np.sqrt(K)),
            "Wup": g(3, (K, N), 0.0, 1.0 / np.sqrt(K)),
        }
    elif program == "layernorm_matmul":
        M, K, N = p["M"], p["K"], p["N"]
        t = {
            "X": g(0, (M, K), 0.3, 1.0),      # a non-zero mean: the subtraction must matter
            "gamma": g(1, (K,), 1.0, 0.1),
            "beta": g(2, (K,), 0.0, 0.1),
            "W": g(3, (K, N), 0.0, 1.0 / np.sqrt(K)),
        }
    elif program == "gqa_decode":
        B, Hq, Hkv, L, D = p["B"], p["Hq"], p["Hkv"], p["L"], p["D"]
        t = {
            "Q": g(0, (B, Hq, D), 0.0, 1.0),
            "K": g(1, (B, Hkv, L, D), 0.0, 1.0),
            "V": g(2, (B, Hkv, L, D), 0.0, 1.0),
        }
    elif program == "gqa_decode_window":
        B, Hq, Hkv, L, D = p["B"], p["Hq"], p["Hkv"], p["L"], p["D"]
        t = {
            "Q": g(0, (B, Hq, D), 0.0, 1.0),
            "K": g(1, (B, Hkv, L, D), 0.0, 1.0),
            "V": g(2, (B, Hkv, L, D), 0.0, 1.0),
        }
    elif program == "gqa_decode_varlen":
        B, Hq, Hkv, L, D = p["B"], p["Hq"], p["Hkv"], p["L"], p["D"]
        lens = p.pop("lens", None)
        pad_nan = p.pop("pad_nan", True)
        if lens is None:
            ss = np.random.SeedSequence([int(seed), _PROGRAM_ID[program], 99])
            lens = np.random.Generator(np.random.Philox(ss)).integers(1, L + 1, size=B)
            lens[0] = L
            if B > 1:
                lens[1] = 1
            if B > 2 and size == "small":
                lens[2] = 0          # an entry without keys: its output is defined as zero
        lens = np.asarray(lens, dtype=np.int32)
        K, V = g(1, (B, Hkv, L, D), 0.0, 1.0), g(2, (B, Hkv, L, D), 0.0, 1.0)
        for b in range(B if pad_nan else 0):   # padding rows hold NaN: neither side may let them reach the output
            n = int(np.clip(lens[b], 0, L))
            K[b, :, n:, :] = 0x7FC0
            V[b, :, n:, :] = 0x7FC0
        p["lens_sum"] = int(np.clip(lens, 0, L).sum())
        t = {"Q": g(0, (B, Hq, D), 0.0, 1.0), "K": K, "V": V, "seq_lens": lens}
    elif program == "qknorm_attn":
        B, H, S, D = p["B"], p["H"], p["S"], p["D"]
        t = {
            "Q": g(0, (B, H, S, D), 0.0, 1.0),
            "K": g(1, (B, H, S, D), 0.0, 1.0),
            "V": g(2, (B, H, S, D), 0.0, 1.0),
            "gamma_q": g(3, (D,), 1.0, 0.1),
            "gamma_k": g(4, (D,), 1.0, 0.1),
        }
    elif program == "qknorm_attn_ex":
        B, Hq, Hkv, S, D = p["B"], p["Hq"], p["Hkv"], p["S"], p["D"]
        t = {
            "Q": g(0, (B, Hq, S, D), 0.0, 1.0),
            "K": g(1, (B, Hkv, S, D), 0.0, 1.0),
            "V": g(2, (B, Hkv, S, D), 0.0, 1.0),
            "gamma_q": g(3, (D,), 1.0, 0.1),
            "gamma_k": g(4, (D,), 1.0, 0.1),
        }
    elif program == "lora_linear":
        M, K, N, R = p["M"], p["K"], p["N"], p["R"]
        t = {
            "X": g(0, (M, K), 0.0, 1.0),
            "W": g(1, (K, N), 0.0, 1.0 / np.sqrt(K)),
            "A": g(2, (K, R), 0.0, 1.0 / np.sqrt(K)),
            "Bm": g(3, (R, N), 0.0, 0.01),
        }
    else:
        raise KeyError(program)
    return p, t


def algorithmic_work(program: str, p: dict) -> dict:
    """Flops and compulsory HBM bytes of one call (bf16 storage), from the shapes only."""
    if program == "rmsnorm_matmul":
        M, K, N = p["M"], p["K"], p["N"]
        return dict(flops=2 * M * K * N, bytes=2 * (K * N + M * K + K + M * N))
    if program == "layernorm_matmul":
        M, K, N = p["M"], p["K"], p["N"]
        return dict(flops=2 * M * K * N, bytes=2 * (K * N + M * K + 2 * K + M * N))
    if program == "gated_mlp":
        M, K, N = p["M"], p["K"], p["N"]
        return dict(flops=4 * M * K * N, bytes=2 * (2 * K * N + M * K + M * N))
    if program == "rmsnorm_gated_mlp":
        M, K, N = p["M"], p["K"], p["N"]
        return dict(flops=4 * M * K * N, bytes=2 * (2 * K * N + M * K + K + M * N))
    if program == "gqa_decode":
        B, Hq, Hkv, L, D = p["B"], p["Hq"], p["Hkv"], p["L"], p["D"]
        return dict(flops=4 * B * Hq * L * D, bytes=2 * (2 * B * Hkv * L * D + 2 * B * Hq * D))
    if program == "gqa_decode_window":   # visible keys only
        B, Hq, Hkv, L, D = p["B"], p["Hq"], p["Hkv"], p["L"], p["D"]
        w, sk = p["window"], p["sinks"]
        vis = L if (w <= 0 or w >= L) else w + min(sk, L - w)
        return dict(flops=4 * B * Hq * vis * D, bytes=2 * (2 * B * Hkv * vis * D + 2 * B * Hq * D))
    if program == "gqa_decode_varlen":   # needs the lengths: p["lens_sum"] = sum of clamped lengths
        Hq, Hkv, D = p["Hq"], p["Hkv"], p["D"]
        tot = int(p["lens_sum"])
        return dict(flops=4 * Hq * tot * D, bytes=2 * (2 * Hkv * tot * D + 2 * p["B"] * Hq * D))
    if program == "qknorm_attn":
        B, H, S, D = p["B"], p["H"], p["S"], p["D"]
        pairs = S * (S + 1) // 2 if p.get("causal", 1) else S * S
        return dict(flops=4 * B * H * D * pairs, bytes=2 * (4 * B * H * S * D + 2 * D))
    if program == "qknorm_attn_ex":
        B, Hq, Hkv, S, D = p["B"], p["Hq"], p["Hkv"], p["S"], p["D"]
        w, sk = p.get("window", 0), p.get("sinks", 0)
        if not p.get("causal", 1):
            pairs = S * S
        elif w <= 0 or w >= S:
            pairs = S * (S + 1) // 2
        else:   # row i sees min(i + 1, w) window keys plus the sink keys that lie below its window
            pairs = sum(min(i + 1, w) + min(sk, max(0, i + 1 - w)) for i in range(S))
        return dict(flops=4 * B * Hq * D * pairs, bytes=2 * (2 * B * Hq * S * D + 2 * B * Hkv * S * D + 2 * D))
    if program == "lora_linear":
        M, K, N, R = p["M"], p["K"], p["N"], p["R"]
        return dict(flops=2 * M * K * N + 2 * M * K * R + 2 * M * R * N,
                    bytes=2 * (M * K + K * N + K * R + R * N + M * N))
    raise KeyError(program)
