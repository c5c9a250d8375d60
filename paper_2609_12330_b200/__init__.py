"""Python binding of the B200 fused tensor-program library (libequiforge.so).

Argument marshalling only: every function checks dtypes/devices, passes raw device
pointers, shapes, scalars and the current CUDA stream through the C ABI declared in
include/equiforge.h, and raises on a non-zero status.  All arithmetic runs in the
hand-written sm_100a kernels; there is no CPU or PyTorch fallback, and importing a
function without the compiled library raises.
"""
from __future__ import annotations

import ctypes
import os

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libequiforge.so")
_lib = None

EXPORTS = [
    "ef_rmsnorm_matmul", "ef_rmsnorm_matmul_workspace_bytes",
    "ef_gated_mlp", "ef_gated_mlp_workspace_bytes",
    "ef_rmsnorm_gated_mlp", "ef_rmsnorm_gated_mlp_workspace_bytes",
    "ef_layernorm_matmul", "ef_layernorm_matmul_workspace_bytes",
    "ef_gqa_decode", "ef_gqa_decode_workspace_bytes", "ef_gqa_decode_varlen", "ef_gqa_decode_window", "ef_gqa_decode_static",
    "ef_gqa_decode_static_max_units",
    "ef_qknorm_attn", "ef_qknorm_attn_workspace_bytes", "ef_qknorm_attn_ex",
    "ef_lora_linear", "ef_lora_linear_workspace_bytes",
    "ef_workspace_init", "ef_check_status", "ef_status_string", "ef_last_cuda_error", "ef_version",
]


class EquiforgeError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        msg = lib().ef_status_string(code).decode()
        super().__init__(f"{where}: status {code} ({msg}); last CUDA error {lib().ef_last_cuda_error()}")


def lib():
    """Load libequiforge.so (raises if it has not been built: there is no fallback path)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: run `python -m paper_2609_12330_b200.build` first")
        L = ctypes.CDLL(LIB_PATH)
        vp, i, f, sz = ctypes.c_void_p, ctypes.c_int, ctypes.c_float, ctypes.c_size_t
        L.ef_rmsnorm_matmul.argtypes = [vp, vp, vp, vp, i, i, i, f, vp, sz, vp]
        L.ef_rmsnorm_matmul_workspace_bytes.argtypes = [i, i, i]
        L.ef_gated_mlp.argtypes = [vp, vp, vp, vp, i, i, i, vp, sz, vp]
        L.ef_gated_mlp_workspace_bytes.argtypes = [i, i, i]
        L.ef_rmsnorm_gated_mlp.argtypes = [vp, vp, vp, vp, vp, i, i, i, f, vp, sz, vp]
        L.ef_rmsnorm_gated_mlp_workspace_bytes.argtypes = [i, i, i]
        L.ef_layernorm_matmul.argtypes = [vp, vp, vp, vp, vp, i, i, i, f, vp, sz, vp]
        L.ef_layernorm_matmul_workspace_bytes.argtypes = [i, i, i]
        L.ef_gqa_decode.argtypes = [vp, vp, vp, vp, i, i, i, i, i, f, vp, sz, vp]
        L.ef_gqa_decode_workspace_bytes.argtypes = [i, i, i, i, i]
        L.ef_gqa_decode_window.argtypes = [vp, vp, vp, vp, i, i, i, i, i, f, i, i, vp, sz, vp]
        L.ef_gqa_decode_varlen.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, i, f, vp, sz, vp]
        L.ef_gqa_decode_static.argtypes = [vp, vp, vp, vp, i, i, i, i, i, f, vp]
        L.ef_gqa_decode_static_max_units.argtypes = []
        L.ef_qknorm_attn.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, f, f, i, vp, sz, vp]
        L.ef_qknorm_attn_workspace_bytes.argtypes = [i, i, i, i]
        L.ef_qknorm_attn_ex.argtypes = [vp, vp, vp, vp, vp, vp, i, i, i, i, i, f, f, i, i, i, vp, sz, vp]
        L.ef_lora_linear.argtypes = [vp, vp, vp, vp, vp, i, i, i, i, f, vp, sz, vp]
        L.ef_lora_linear_workspace_bytes.argtypes = [i, i, i, i]
        L.ef_workspace_init.argtypes = [vp, sz, vp]
        L.ef_check_status.argtypes = [vp, vp]
        L.ef_status_string.argtypes = [i]
        L.ef_status_string.restype = ctypes.c_char_p
        for name in EXPORTS:
            fn = getattr(L, name)
            if name.endswith("_workspace_bytes") or name.endswith("_max_units"):
                fn.restype = sz
            elif name != "ef_status_string":
                fn.restype = i
        _lib = L
    return _lib


def _check(code: int, where: str):
    if code != 0:
        raise EquiforgeError(code, where)


def _ptr(t, name):
    import torch

    if not (isinstance(t, torch.Tensor) and t.is_cuda and t.dtype == torch.bfloat16 and t.is_contiguous()):
        raise TypeError(f"{name}: expected a contiguous CUDA bfloat16 tensor")
    return ctypes.c_void_p(t.data_ptr())


def _stream():
    import torch

    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


class Workspace:
    """Caller-owned device scratch buffer, initialised once through ef_workspace_init."""

    def __init__(self, nbytes: int, device="cuda"):
        import torch

        self.nbytes = max(int(nbytes), 4096)
        self.buf = torch.empty(self.nbytes + 256, dtype=torch.uint8, device=device)
        off = (-self.buf.data_ptr()) % 256
        self.ptr = self.buf.data_ptr() + off
        _check(lib().ef_workspace_init(ctypes.c_void_p(self.ptr), self.nbytes, _stream()), "ef_workspace_init")

    def check(self):
        _check(lib().ef_check_status(ctypes.c_void_p(self.ptr), _stream()), "ef_check_status")


def _ws_args(ws: Workspace, need: int, where: str):
    if ws is None or ws.nbytes < need:
        raise EquiforgeError(5, where)
    return ctypes.c_void_p(ws.ptr), ws.nbytes


def rmsnorm_matmul_workspace_bytes(M, K, N):
    return int(lib().ef_rmsnorm_matmul_workspace_bytes(M, K, N))


def gated_mlp_workspace_bytes(M, K, N):
    return int(lib().ef_gated_mlp_workspace_bytes(M, K, N))


def rmsnorm_gated_mlp_workspace_bytes(M, K, N):
    return int(lib().ef_rmsnorm_gated_mlp_workspace_bytes(M, K, N))


def layernorm_matmul_workspace_bytes(M, K, N):
    return int(lib().ef_layernorm_matmul_workspace_bytes(M, K, N))


def gqa_decode_workspace_bytes(B, Hq, Hkv, L, D):
    return int(lib().ef_gqa_decode_workspace_bytes(B, Hq, Hkv, L, D))


def qknorm_attn_workspace_bytes(B, H, S, D):
    return int(lib().ef_qknorm_attn_workspace_bytes(B, H, S, D))


def lora_linear_workspace_bytes(M, K, N, R):
    return int(lib().ef_lora_linear_workspace_bytes(M, K, N, R))


def rmsnorm_matmul(X, gamma, W, eps, ws: Workspace, out=None):
    import torch

    M, K = X.shape
    N = W.shape[1]
    Y = out if out is not None else torch.empty((M, N), dtype=torch.bfloat16, device=X.device)
    wp, wb = _ws_args(ws, rmsnorm_matmul_workspace_bytes(M, K, N), "ef_rmsnorm_matmul")
    _check(lib().ef_rmsnorm_matmul(_ptr(X, "X"), _ptr(gamma, "gamma"), _ptr(W, "W"), _ptr(Y, "Y"), M, K, N,
                                   float(eps), wp, wb, _stream()), "ef_rmsnorm_matmul")
    return Y


def gated_mlp(X, Wgate, Wup, ws: Workspace, out=None):
    import torch

    M, K = X.shape
    N = Wgate.shape[1]
    Y = out if out is not None else torch.empty((M, N), dtype=torch.bfloat16, device=X.device)
    wp, wb = _ws_args(ws, gated_mlp_workspace_bytes(M, K, N), "ef_gated_mlp")
    _check(lib().ef_gated_mlp(_ptr(X, "X"), _ptr(Wgate, "Wgate"), _ptr(Wup, "Wup"), _ptr(Y, "Y"), M, K, N,
                              wp, wb, _stream()), "ef_gated_mlp")
    return Y


def rmsnorm_gated_mlp(X, gamma, Wgate, Wup, eps, ws: Workspace, out=None):
    import torch

    M, K = X.shape
    N = Wgate.shape[1]
    Y = out if out is not None else torch.empty((M, N), dtype=torch.bfloat16, device=X.device)
    wp, wb = _ws_args(ws, rmsnorm_gated_mlp_workspace_bytes(M, K, N), "ef_rmsnorm_gated_mlp")
    _check(lib().ef_rmsnorm_gated_mlp(_ptr(X, "X"), _ptr(gamma, "gamma"), _ptr(Wgate, "Wgate"), _ptr(Wup, "Wup"),
                                      _ptr(Y, "Y"), M, K, N, float(eps), wp, wb, _stream()), "ef_rmsnorm_gated_mlp")
    return Y


def layernorm_matmul(X, gamma, beta, W, eps, ws: Workspace, out=None):
    import torch

    M, K = X.shape
    N = W.shape[1]
    Y = out if out is not None else torch.empty((M, N), dtype=torch.bfloat16, device=X.device)
    wp, wb = _ws_args(ws, layernorm_matmul_workspace_bytes(M, K, N), "ef_layernorm_matmul")
    _check(lib().ef_layernorm_matmul(_ptr(X, "X"), _ptr(gamma, "gamma"), _ptr(beta, "beta"), _ptr(W, "W"), _ptr(Y, "Y"),
                                     M, K, N, float(eps), wp, wb, _stream()), "ef_layernorm_matmul")
    return Y


def gqa_decode(Q, K, V, scale, ws: Workspace, out=None):
    import torch

    B, Hq, D = Q.shape
    _, Hkv, L, _ = K.shape
    O = out if out is not None else torch.empty((B, Hq, D), dtype=torch.bfloat16, device=Q.device)
    wp, wb = _ws_args(ws, gqa_decode_workspace_bytes(B, Hq, Hkv, L, D), "ef_gqa_decode")
    _check(lib().ef_gqa_decode(_ptr(Q, "Q"), _ptr(K, "K"), _ptr(V, "V"), _ptr(O, "O"), B, Hq, Hkv, L, D,
                               float(scale), wp, wb, _stream()), "ef_gqa_decode")
    return O


def gqa_decode_window(Q, K, V, scale, window, sinks, ws: Workspace, out=None):
    """Decode attention over the last `window` keys plus the first `sinks` keys (the query is the last position)."""
    import torch

    B, Hq, D = Q.shape
    _, Hkv, L, _ = K.shape
    O = out if out is not None else torch.empty((B, Hq, D), dtype=torch.bfloat16, device=Q.device)
    wp, wb = _ws_args(ws, gqa_decode_workspace_bytes(B, Hq, Hkv, L, D), "ef_gqa_decode_window")
    _check(lib().ef_gqa_decode_window(_ptr(Q, "Q"), _ptr(K, "K"), _ptr(V, "V"), _ptr(O, "O"), B, Hq, Hkv, L, D,
                                      float(scale), int(window), int(sinks), wp, wb, _stream()), "ef_gqa_decode_window")
    return O


def gqa_decode_varlen(Q, K, V, seq_lens, scale, ws: Workspace, out=None):
    """Decode attention where batch entry b attends keys [0, seq_lens[b]); seq_lens is a CUDA int32 tensor [B]."""
    import torch

    B, Hq, D = Q.shape
    _, Hkv, L, _ = K.shape
    if seq_lens.dtype != torch.int32 or not seq_lens.is_cuda or not seq_lens.is_contiguous() or seq_lens.numel() != B:
        raise ValueError("seq_lens must be a contiguous CUDA int32 tensor with one entry per batch element")
    O = out if out is not None else torch.empty((B, Hq, D), dtype=torch.bfloat16, device=Q.device)
    wp, wb = _ws_args(ws, gqa_decode_workspace_bytes(B, Hq, Hkv, L, D), "ef_gqa_decode_varlen")
    _check(lib().ef_gqa_decode_varlen(_ptr(Q, "Q"), _ptr(K, "K"), _ptr(V, "V"), ctypes.c_void_p(seq_lens.data_ptr()),
                                      _ptr(O, "O"), B, Hq, Hkv, L, D, float(scale), wp, wb, _stream()),
           "ef_gqa_decode_varlen")
    return O


def gqa_decode_static(Q, K, V, scale, out=None):
    """Decode attention through ef_gqa_decode_static: no workspace argument, nothing allocated by
    the call itself (the output tensor is the caller's: pass `out` to avoid torch allocating one).
    For callers that may not allocate device memory when they call; at most
    ef_gqa_decode_static_max_units() (batch, kv head) units; calls on one device must not overlap."""
    import torch

    B, Hq, D = Q.shape
    _, Hkv, L, _ = K.shape
    O = out if out is not None else torch.empty((B, Hq, D), dtype=torch.bfloat16, device=Q.device)
    _check(lib().ef_gqa_decode_static(_ptr(Q, "Q"), _ptr(K, "K"), _ptr(V, "V"), _ptr(O, "O"), B, Hq, Hkv, L, D,
                                      float(scale), _stream()), "ef_gqa_decode_static")
    return O


def qknorm_attn(Q, K, V, gamma_q, gamma_k, eps, scale, causal, ws: Workspace, out=None):
    import torch

    B, H, S, D = Q.shape
    O = out if out is not None else torch.empty((B, H, S, D), dtype=torch.bfloat16, device=Q.device)
    wp, wb = _ws_args(ws, qknorm_attn_workspace_bytes(B, H, S, D), "ef_qknorm_attn")
    _check(lib().ef_qknorm_attn(_ptr(Q, "Q"), _ptr(K, "K"), _ptr(V, "V"), _ptr(gamma_q, "gamma_q"),
                                _ptr(gamma_k, "gamma_k"), _ptr(O, "O"), B, H, S, D, float(eps), float(scale),
                                int(causal), wp, wb, _stream()), "ef_qknorm_attn")
    return O


def qknorm_attn_ex(Q, K, V, gamma_q, gamma_k, eps, scale, causal, window, sinks, ws: Workspace, out=None):
    """QK-normalised attention with grouped KV heads (K, V: [B,Hkv,S,D]), a sliding window and attention sinks."""
    import torch

    B, Hq, S, D = Q.shape
    Hkv = K.shape[1]
    O = out if out is not None else torch.empty((B, Hq, S, D), dtype=torch.bfloat16, device=Q.device)
    wp, wb = _ws_args(ws, qknorm_attn_workspace_bytes(B, Hkv, S, D), "ef_qknorm_attn_ex")
    _check(lib().ef_qknorm_attn_ex(_ptr(Q, "Q"), _ptr(K, "K"), _ptr(V, "V"), _ptr(gamma_q, "gamma_q"),
                                   _ptr(gamma_k, "gamma_k"), _ptr(O, "O"), B, Hq, Hkv, S, D, float(eps), float(scale),
                                   int(causal), int(window), int(sinks), wp, wb, _stream()), "ef_qknorm_attn_ex")
    return O


def lora_linear(X, W, A, Bm, alpha, ws: Workspace, out=None):
    import torch

    M, K = X.shape
    N = W.shape[1]
    R = A.shape[1]
    Y = out if out is not None else torch.empty((M, N), dtype=torch.bfloat16, device=X.device)
    wp, wb = _ws_args(ws, lora_linear_workspace_bytes(M, K, N, R), "ef_lora_linear")
    _check(lib().ef_lora_linear(_ptr(X, "X"), _ptr(W, "W"), _ptr(A, "A"), _ptr(Bm, "Bm"), _ptr(Y, "Y"), M, K, N, R,
                                float(alpha), wp, wb, _stream()), "ef_lora_linear")
    return Y


def workspace_bytes(program: str, p: dict) -> int:
    if program == "rmsnorm_matmul":
        return rmsnorm_matmul_workspace_bytes(p["M"], p["K"], p["N"])
    if program == "gated_mlp":
        return gated_mlp_workspace_bytes(p["M"], p["K"], p["N"])
    if program == "rmsnorm_gated_mlp":
        return rmsnorm_gated_mlp_workspace_bytes(p["M"], p["K"], p["N"])
    if program == "layernorm_matmul":
        return layernorm_matmul_workspace_bytes(p["M"], p["K"], p["N"])
    if program in ("gqa_decode", "gqa_decode_varlen", "gqa_decode_window"):
        return gqa_decode_workspace_bytes(p["B"], p["Hq"], p["Hkv"], p["L"], p["D"])
    if program == "qknorm_attn":
        return qknorm_attn_workspace_bytes(p["B"], p["H"], p["S"], p["D"])
    if program == "qknorm_attn_ex":
        return qknorm_attn_workspace_bytes(p["B"], p["Hkv"], p["S"], p["D"])
    if program == "lora_linear":
        return lora_linear_workspace_bytes(p["M"], p["K"], p["N"], p["R"])
    raise KeyError(program)


def run(program: str, p: dict, t: dict, ws: Workspace, out=None):
    """Dispatch by program name; `t` maps argument names to CUDA bf16 tensors."""
    if program == "rmsnorm_matmul":
        return rmsnorm_matmul(t["X"], t["gamma"], t["W"], p["eps"], ws, out)
    if program == "gated_mlp":
        return gated_mlp(t["X"], t["Wgate"], t["Wup"], ws, out)
    if program == "rmsnorm_gated_mlp":
        return rmsnorm_gated_mlp(t["X"], t["gamma"], t["Wgate"], t["Wup"], p["eps"], ws, out)
    if program == "layernorm_matmul":
        return layernorm_matmul(t["X"], t["gamma"], t["beta"], t["W"], p["eps"], ws, out)
    if program == "gqa_decode":
        return gqa_decode(t["Q"], t["K"], t["V"], p["scale"], ws, out)
    if program == "gqa_decode_window":
        return gqa_decode_window(t["Q"], t["K"], t["V"], p["scale"], p["window"], p["sinks"], ws, out)
    if program == "gqa_decode_varlen":
        return gqa_decode_varlen(t["Q"], t["K"], t["V"], t["seq_lens"], p["scale"], ws, out)
    if program == "qknorm_attn":
        return qknorm_attn(t["Q"], t["K"], t["V"], t["gamma_q"], t["gamma_k"], p["eps"], p["scale"],
                           p.get("causal", 1), ws, out)
    if program == "qknorm_attn_ex":
        return qknorm_attn_ex(t["Q"], t["K"], t["V"], t["gamma_q"], t["gamma_k"], p["eps"], p["scale"], p.get("causal", 1),
                              p.get("window", 0), p.get("sinks", 0), ws, out)
    if program == "lora_linear":
        return lora_linear(t["X"], t["W"], t["A"], t["Bm"], p["alpha"], ws, out)
    raise KeyError(program)
