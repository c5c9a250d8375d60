"""ctypes access to the fp64 CPU oracle (oracle/ef_oracle.c).

TEST INFRASTRUCTURE ONLY.  Importers: tests/, the smoke check, and the
benchmark's cpu_baseline / reference legs.  The CUDA library and its Python
binding never import this package and share nothing with it.

Each wrapper takes float64 numpy arrays (bf16 inputs are widened exactly by the
caller) and returns the unrounded float64 result of the unfused definition.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "ef_oracle.c")
_LIB = os.path.join(_HERE, "libef_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (OpenMP, strict IEEE arithmetic); return the .so path."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c11", "-fopenmp", "-fPIC", "-shared", "-fno-fast-math",
               "-o", _LIB, _SRC, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        _lib = ctypes.CDLL(build())
        _lib.ef_oracle_num_threads.restype = ctypes.c_int
    return _lib


def num_threads() -> int:
    return int(_load().ef_oracle_num_threads())


def _d(a):
    a = np.ascontiguousarray(a, dtype=np.float64)
    return a, a.ctypes.data_as(ctypes.POINTER(ctypes.c_double))


def rmsnorm_matmul(X, gamma, W, eps):
    X, pX = _d(X); gamma, pg = _d(gamma); W, pW = _d(W)
    M, K = X.shape; N = W.shape[1]
    assert W.shape[0] == K and gamma.shape == (K,)
    Y = np.empty((M, N), dtype=np.float64)
    _load().ef_oracle_rmsnorm_matmul(pX, pg, pW, _d(Y)[1], M, K, N, ctypes.c_double(eps))
    return Y


def layernorm_matmul(X, gamma, beta, W, eps):
    X, pX = _d(X); gamma, pg = _d(gamma); beta, pb = _d(beta); W, pW = _d(W)
    M, K = X.shape; N = W.shape[1]
    assert W.shape[0] == K and gamma.shape == (K,) and beta.shape == (K,)
    Y = np.empty((M, N), dtype=np.float64)
    _load().ef_oracle_layernorm_matmul(pX, pg, pb, pW, _d(Y)[1], M, K, N, ctypes.c_double(eps))
    return Y


def gated_mlp(X, Wgate, Wup):
    X, pX = _d(X); Wgate, pG = _d(Wgate); Wup, pU = _d(Wup)
    M, K = X.shape; N = Wgate.shape[1]
    assert Wgate.shape == (K, N) and Wup.shape == (K, N)
    Y = np.empty((M, N), dtype=np.float64)
    _load().ef_oracle_gated_mlp(pX, pG, pU, _d(Y)[1], M, K, N)
    return Y


def rmsnorm_gated_mlp(X, gamma, Wgate, Wup, eps):
    X, pX = _d(X); gamma, pg = _d(gamma); Wgate, pG = _d(Wgate); Wup, pU = _d(Wup)
    M, K = X.shape; N = Wgate.shape[1]
    assert Wgate.shape == (K, N) and Wup.shape == (K, N) and gamma.shape == (K,)
    Y = np.empty((M, N), dtype=np.float64)
    _load().ef_oracle_rmsnorm_gated_mlp(pX, pg, pG, pU, _d(Y)[1], M, K, N, ctypes.c_double(eps))
    return Y


def gqa_decode(Q, K, V, scale):
    Q, pQ = _d(Q); K, pK = _d(K); V, pV = _d(V)
    B, Hq, D = Q.shape; _, Hkv, L, _ = K.shape
    assert K.shape == (B, Hkv, L, D) and V.shape == K.shape and Hq % Hkv == 0
    O = np.empty((B, Hq, D), dtype=np.float64)
    _load().ef_oracle_gqa_decode(pQ, pK, pV, _d(O)[1], B, Hq, Hkv, L, D, ctypes.c_double(scale))
    return O


def gqa_decode_window(Q, K, V, scale, window, sinks):
    Q, pQ = _d(Q); K, pK = _d(K); V, pV = _d(V)
    B, Hq, D = Q.shape; _, Hkv, L, _ = K.shape
    assert K.shape == (B, Hkv, L, D) and V.shape == K.shape and Hq % Hkv == 0
    O = np.empty((B, Hq, D), dtype=np.float64)
    _load().ef_oracle_gqa_decode_window(pQ, pK, pV, _d(O)[1], B, Hq, Hkv, L, D, ctypes.c_double(scale), int(window), int(sinks))
    return O


def gqa_decode_varlen(Q, K, V, seq_lens, scale):
    Q, pQ = _d(Q); K, pK = _d(K); V, pV = _d(V)
    B, Hq, D = Q.shape; _, Hkv, L, _ = K.shape
    assert K.shape == (B, Hkv, L, D) and V.shape == K.shape and Hq % Hkv == 0
    lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    assert lens.shape == (B,)
    O = np.empty((B, Hq, D), dtype=np.float64)
    _load().ef_oracle_gqa_decode_varlen(pQ, pK, pV, lens.ctypes.data_as(ctypes.POINTER(ctypes.c_int)), _d(O)[1],
                                        B, Hq, Hkv, L, D, ctypes.c_double(scale))
    return O


def qknorm_attn(Q, K, V, gamma_q, gamma_k, eps, scale, causal=1):
    Q, pQ = _d(Q); K, pK = _d(K); V, pV = _d(V)
    gamma_q, pgq = _d(gamma_q); gamma_k, pgk = _d(gamma_k)
    B, H, S, D = Q.shape
    assert K.shape == Q.shape and V.shape == Q.shape and gamma_q.shape == (D,) and gamma_k.shape == (D,)
    O = np.empty((B, H, S, D), dtype=np.float64)
    _load().ef_oracle_qknorm_attn(pQ, pK, pV, pgq, pgk, _d(O)[1], B, H, S, D,
                                  ctypes.c_double(eps), ctypes.c_double(scale), int(causal))
    return O


def qknorm_attn_ex(Q, K, V, gamma_q, gamma_k, eps, scale, causal=1, window=0, sinks=0):
    Q, pQ = _d(Q); K, pK = _d(K); V, pV = _d(V)
    gamma_q, pgq = _d(gamma_q); gamma_k, pgk = _d(gamma_k)
    B, Hq, S, D = Q.shape
    Hkv = K.shape[1]
    assert K.shape == (B, Hkv, S, D) and V.shape == K.shape and Hq % Hkv == 0
    assert gamma_q.shape == (D,) and gamma_k.shape == (D,)
    O = np.empty((B, Hq, S, D), dtype=np.float64)
    _load().ef_oracle_qknorm_attn_ex(pQ, pK, pV, pgq, pgk, _d(O)[1], B, Hq, Hkv, S, D, ctypes.c_double(eps),
                                     ctypes.c_double(scale), int(causal), int(window), int(sinks))
    return O


def lora_linear(X, W, A, Bm, alpha):
    X, pX = _d(X); W, pW = _d(W); A, pA = _d(A); Bm, pB = _d(Bm)
    M, K = X.shape; N = W.shape[1]; R = A.shape[1]
    assert W.shape == (K, N) and A.shape == (K, R) and Bm.shape == (R, N)
    Y = np.empty((M, N), dtype=np.float64)
    _load().ef_oracle_lora_linear(pX, pW, pA, pB, _d(Y)[1], M, K, N, R, ctypes.c_double(alpha))
    return Y


def run(program: str, params: dict, tensors_f64: dict) -> np.ndarray:
    """Dispatch by program name; tensors_f64 maps argument names to float64 arrays."""
    t, p = tensors_f64, params
    if program == "rmsnorm_matmul":
        return rmsnorm_matmul(t["X"], t["gamma"], t["W"], p["eps"])
    if program == "layernorm_matmul":
        return layernorm_matmul(t["X"], t["gamma"], t["beta"], t["W"], p["eps"])
    if program == "gated_mlp":
        return gated_mlp(t["X"], t["Wgate"], t["Wup"])
    if program == "rmsnorm_gated_mlp":
        return rmsnorm_gated_mlp(t["X"], t["gamma"], t["Wgate"], t["Wup"], p["eps"])
    if program == "gqa_decode":
        return gqa_decode(t["Q"], t["K"], t["V"], p["scale"])
    if program == "gqa_decode_window":
        return gqa_decode_window(t["Q"], t["K"], t["V"], p["scale"], p["window"], p["sinks"])
    if program == "gqa_decode_varlen":
        return gqa_decode_varlen(t["Q"], t["K"], t["V"], t["seq_lens"], p["scale"])
    if program == "qknorm_attn":
        return qknorm_attn(t["Q"], t["K"], t["V"], t["gamma_q"], t["gamma_k"], p["eps"], p["scale"], p.get("causal", 1))
    if program == "qknorm_attn_ex":
        return qknorm_attn_ex(t["Q"], t["K"], t["V"], t["gamma_q"], t["gamma_k"], p["eps"], p["scale"], p.get("causal", 1),
                              p.get("window", 0), p.get("sinks", 0))
    if program == "lora_linear":
        return lora_linear(t["X"], t["W"], t["A"], t["Bm"], p["alpha"])
    raise KeyError(program)
