"""ctypes binding of the C-ABI library.  Argument marshalling only: every step of the
forward pass runs inside the library's CUDA kernels.  PyTorch supplies device memory and the
current stream.  There is no CPU fallback: if the shared library is missing, loading fails."""
from __future__ import annotations

import ctypes as C
import os

import numpy as np
import torch

_LIB_PATH = os.environ.get("HYPERATTN_LIB") or os.path.join(os.path.dirname(os.path.abspath(__file__)), "libhyperattn.so")
_lib = None

BF16, FP32 = 0, 1
STAGE_NAMES = ["convert", "hash", "sample", "sort_scan", "sort_scatter", "attention", "merge", "backward"]
NUM_STAGES = len(STAGE_NAMES)          # HYPERATTN_NUM_STAGES
EXPORTS = ["hyperattn_forward", "hyperattn_forward_ex", "hyperattn_forward_host", "hyperattn_workspace_bytes",
           "hyperattn_backward", "hyperattn_backward_workspace_bytes",
           "hyperattn_get_projections", "hyperattn_last_device_status", "hyperattn_profile_enable",
           "hyperattn_profile_reset", "hyperattn_profile_read", "hyperattn_release",
           "hyperattn_status_string", "hyperattn_version", "hyperattn_sortlsh_noalloc",
           "hyperattn_alpha", "hyperattn_alpha_workspace_bytes", "hyperattn_get_node_projections"]


class HyperAttnError(RuntimeError):
    pass


class _Debug(C.Structure):
    _fields_ = [("q_ids", C.c_void_p), ("k_ids", C.c_void_p), ("perm_q", C.c_void_p), ("perm_k", C.c_void_p),
                ("rank_k", C.c_void_p), ("samples", C.c_void_p), ("near_zero_bits", C.c_void_p),
                ("row_subset", C.c_void_p), ("log2_tau", C.c_void_p), ("sample_log2w", C.c_void_p)]


class _Params(C.Structure):
    _fields_ = [("q", C.c_void_p), ("k", C.c_void_p), ("v", C.c_void_p), ("out", C.c_void_p), ("lse", C.c_void_p),
                ("B", C.c_int), ("H", C.c_int), ("n", C.c_int), ("d", C.c_int),
                ("block", C.c_int), ("samples", C.c_int), ("hash_bits", C.c_int), ("causal", C.c_int),
                ("n0", C.c_int), ("seed", C.c_uint64), ("dtype", C.c_int), ("out_dtype", C.c_int),
                ("softmax_scale", C.c_float), ("workspace", C.c_void_p), ("workspace_bytes", C.c_size_t),
                ("debug", C.POINTER(_Debug)), ("stream", C.c_void_p),
                ("precise", C.c_int), ("n_k", C.c_int), ("capped", C.c_int), ("cap_scale", C.c_float), ("kappa", C.c_float),
                ("sampling", C.c_int), ("node_directions", C.c_int)]


class _StageTimes(C.Structure):
    _fields_ = [("ms", C.c_float * NUM_STAGES), ("launches", C.c_int * NUM_STAGES), ("calls", C.c_int)]


def lib() -> C.CDLL:
    """Loads libhyperattn.so (built in-tree by paper_2310_05869_b200/build.py)."""
    global _lib
    if _lib is None:
        if not os.path.exists(_LIB_PATH):
            raise HyperAttnError(f"{_LIB_PATH} is missing: build it with `python -m paper_2310_05869_b200.build`")
        L = C.CDLL(_LIB_PATH)
        L.hyperattn_forward.restype = C.c_int
        L.hyperattn_forward.argtypes = [C.c_void_p] * 5 + [C.c_int] * 9 + [C.c_uint64, C.c_void_p]
        for name in ("hyperattn_forward_ex", "hyperattn_forward_host"):
            getattr(L, name).restype = C.c_int
            getattr(L, name).argtypes = [C.POINTER(_Params)]
        L.hyperattn_workspace_bytes.restype = C.c_int
        L.hyperattn_workspace_bytes.argtypes = [C.POINTER(_Params), C.POINTER(C.c_size_t)]
        L.hyperattn_get_projections.restype = C.c_int
        L.hyperattn_get_projections.argtypes = [C.c_int, C.c_int, C.c_uint64, C.c_void_p]
        L.hyperattn_get_node_projections.restype = C.c_int
        L.hyperattn_get_node_projections.argtypes = [C.c_int, C.c_int, C.c_uint64, C.c_int, C.c_void_p]
        L.hyperattn_last_device_status.restype = C.c_int
        L.hyperattn_last_device_status.argtypes = [C.c_void_p, C.POINTER(C.c_int)]
        L.hyperattn_profile_enable.argtypes = [C.c_int]
        L.hyperattn_profile_read.argtypes = [C.POINTER(_StageTimes)]
        L.hyperattn_sortlsh_noalloc.restype = C.c_int
        L.hyperattn_sortlsh_noalloc.argtypes = [C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_uint64,
                                                C.c_void_p, C.c_void_p, C.c_void_p, C.c_void_p]
        L.hyperattn_alpha.restype = C.c_int
        L.hyperattn_alpha.argtypes = [C.c_void_p, C.c_void_p, C.c_int, C.c_int, C.c_int, C.c_int, C.c_int, C.c_float, C.c_int, C.c_int,
                                      C.c_void_p, C.c_void_p, C.c_size_t, C.c_void_p]
        L.hyperattn_alpha_workspace_bytes.restype = C.c_int
        L.hyperattn_alpha_workspace_bytes.argtypes = [C.c_int, C.c_int, C.c_int, C.c_int, C.POINTER(C.c_size_t)]
        L.hyperattn_backward.restype = C.c_int
        L.hyperattn_backward.argtypes = [C.POINTER(_Params), C.POINTER(_Grads)]
        L.hyperattn_backward_workspace_bytes.restype = C.c_int
        L.hyperattn_backward_workspace_bytes.argtypes = [C.POINTER(_Params), C.c_int, C.POINTER(C.c_size_t)]
        L.hyperattn_status_string.restype = C.c_char_p
        L.hyperattn_status_string.argtypes = [C.c_int]
        _lib = L
    return _lib


def _check(rc: int, what: str):
    if rc != 0:
        raise HyperAttnError(f"{what}: {lib().hyperattn_status_string(rc).decode()} ({rc})")


def _dtype_code(t: torch.dtype) -> int:
    if t == torch.bfloat16:
        return BF16
    if t == torch.float32:
        return FP32
    raise HyperAttnError(f"unsupported dtype {t}")


def _fill(p: _Params, B, H, n, d, block, samples, hash_bits, causal, n0, seed, dtype, out_dtype, scale, n_k=0):
    p.B, p.H, p.n, p.d = B, H, n, d
    p.n_k = 0 if n_k == n else n_k
    p.block, p.samples, p.hash_bits, p.causal, p.n0 = block, samples, hash_bits, int(bool(causal)), n0
    p.seed = seed
    p.dtype, p.out_dtype, p.softmax_scale = dtype, out_dtype, float(scale)


def _debug_shapes(B, H, n, block, samples, causal, n0, n_k=None):
    """Shapes of the exported intermediates (see hyperattn_debug in the header)."""
    G = B * H
    n_k = n if n_k is None else n_k
    if not causal:
        LV, NL, NODES = 1, max(n, n_k), 1
    elif n <= n0:
        LV, NL, NODES = 1, n, 0
    else:
        L = 0
        while -((-n) >> L) > n0:                  # Alg. 4: halve until a part is not longer than n0
            L += 1
        leaf = -((-n) >> L)
        LV, NL, NODES = L, (leaf << L) // 2, (1 << L) - 1
    return G, LV, NL, NODES


def forward(q, k, v, block, samples, hash_bits, causal=False, n0=0, seed=0, out_dtype=None, scale=0.0,
            workspace=None, debug=False, stream=None, precise=False, caps=None, value_norm_sampling=False,
            node_directions=False):
    """HyperAttention forward on CUDA tensors q [B, H, n, d] and k, v [B, H, n_k, d] (bf16 or fp32).
    caps = (cap_scale, kappa) runs the row-sum estimate with the caps of Alg. 2.
    Returns (out, lse) or (out, lse, intermediates) when debug=True."""
    if not (q.is_cuda and k.is_cuda and v.is_cuda):
        raise HyperAttnError("q, k, v must be CUDA tensors (there is no CPU path)")
    q, k, v = q.contiguous(), k.contiguous(), v.contiguous()
    B, H, n, d = q.shape
    n_k = k.shape[2]
    if k.shape != (B, H, n_k, d) or v.shape != k.shape:
        raise HyperAttnError("k and v must be [B, H, n_k, d] with the batch, heads and d of q")
    out_dtype = out_dtype or q.dtype
    out = torch.empty((B, H, n, d), dtype=out_dtype, device=q.device)
    lse = torch.empty((B, H, n), dtype=torch.float32, device=q.device)
    p = _Params()
    _fill(p, B, H, n, d, block, samples, hash_bits, causal, n0, seed, _dtype_code(q.dtype), _dtype_code(out_dtype), scale, n_k)
    p.q, p.k, p.v, p.out, p.lse = q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lse.data_ptr()
    if workspace is not None:
        p.workspace, p.workspace_bytes = workspace.data_ptr(), workspace.numel() * workspace.element_size()
    p.stream = stream if stream is not None else torch.cuda.current_stream(q.device).cuda_stream
    p.precise = int(bool(precise))
    if caps is not None:
        p.capped, p.cap_scale, p.kappa = 1, float(caps[0]), float(caps[1])
    p.sampling = int(bool(value_norm_sampling))
    p.node_directions = int(bool(node_directions))
    inter = None
    if debug:
        G, LV, NL, NODES = _debug_shapes(B, H, n, block, samples, causal, n0, n_k)
        dev = q.device
        id_sets = (LV,) if (node_directions and causal and NODES > 0) else ()
        inter = {
            "q_ids": torch.zeros(id_sets + (G, n), dtype=torch.uint8, device=dev),
            "k_ids": torch.zeros(id_sets + (G, n_k), dtype=torch.uint8, device=dev),
            "perm_q": torch.full((LV, G, NL), -1, dtype=torch.int32, device=dev),
            "perm_k": torch.full((LV, G, NL), -1, dtype=torch.int32, device=dev),
            "rank_k": torch.full((LV, G, NL), -1, dtype=torch.int32, device=dev),
            "samples": torch.full((G, max(NODES, 1), max(samples, 1)), -1, dtype=torch.int32, device=dev),
            "near_zero_bits": torch.zeros(1, dtype=torch.int64, device=dev),
            "row_subset": torch.full((G, max(NODES, 1), max(samples, 1)), -1, dtype=torch.int32, device=dev),
            "log2_tau": torch.full((G, max(NODES, 1)), float("nan"), dtype=torch.float32, device=dev),
            "sample_log2w": torch.full((G, max(NODES, 1), max(samples, 1)), float("nan"), dtype=torch.float32, device=dev),
        }
        dbg = _Debug(*(inter[f].data_ptr() for f, _ in _Debug._fields_))
        p.debug = C.pointer(dbg)
    with torch.cuda.device(q.device):
        _check(lib().hyperattn_forward_ex(C.byref(p)), "hyperattn_forward_ex")
    return (out, lse, inter) if debug else (out, lse)


class _Grads(C.Structure):
    _fields_ = [("dout", C.c_void_p), ("dq", C.c_void_p), ("dk", C.c_void_p), ("dv", C.c_void_p), ("grad_dtype", C.c_int)]


def backward(q, k, v, out, lse, dout, block, samples, hash_bits, causal=False, n0=0, seed=0, grad_dtype=None, scale=0.0,
             stream=None):
    """Backward pass of `forward` (same shape arguments and seed as the forward call; out and lse are its
    results).  q, k, v, dout: bf16 CUDA tensors [B, H, n, d].  Returns (dq, dk, dv) of grad_dtype (default bf16)."""
    if not all(t.is_cuda for t in (q, k, v, out, lse, dout)):
        raise HyperAttnError("all tensors must be CUDA tensors (there is no CPU path)")
    q, k, v, out, lse, dout = (t.contiguous() for t in (q, k, v, out, lse, dout))
    B, H, n, d = q.shape
    grad_dtype = grad_dtype or torch.bfloat16
    dq, dk, dv = (torch.empty((B, H, n, d), dtype=grad_dtype, device=q.device) for _ in range(3))
    p = _Params()
    _fill(p, B, H, n, d, block, samples, hash_bits, causal, n0, seed, _dtype_code(q.dtype), _dtype_code(out.dtype), scale)
    p.q, p.k, p.v, p.out, p.lse = q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lse.data_ptr()
    p.stream = stream if stream is not None else torch.cuda.current_stream(q.device).cuda_stream
    g = _Grads(dout.data_ptr(), dq.data_ptr(), dk.data_ptr(), dv.data_ptr(), _dtype_code(grad_dtype))
    with torch.cuda.device(q.device):
        _check(lib().hyperattn_backward(C.byref(p), C.byref(g)), "hyperattn_backward")
    return dq, dk, dv


def forward_host(q, k, v, out, lse, block, samples, hash_bits, causal=False, n0=0, seed=0, scale=0.0, stream=None):
    """Host-buffer entry: q, k, v, out, lse are CPU tensors (pinned for asynchronous copies).
    Enqueues H2D copies, the forward pass and D2H copies on the stream; the caller synchronises."""
    B, H, n, d = q.shape
    p = _Params()
    _fill(p, B, H, n, d, block, samples, hash_bits, causal, n0, seed, _dtype_code(q.dtype), _dtype_code(out.dtype), scale, k.shape[2])
    p.q, p.k, p.v, p.out, p.lse = q.data_ptr(), k.data_ptr(), v.data_ptr(), out.data_ptr(), lse.data_ptr()
    p.stream = stream if stream is not None else torch.cuda.current_stream().cuda_stream
    _check(lib().hyperattn_forward_host(C.byref(p)), "hyperattn_forward_host")


NOALLOC_MAX_ROWS = 262144


def sortlsh_noalloc(x, hash_bits, seed=0, stream=None):
    """sortLSH of one CUDA bf16 matrix x[n, d] through the entry point that allocates nothing
    inside the library (its scratch is a fixed array in the library image; n is capped at
    NOALLOC_MAX_ROWS).  The three result tensors are allocated here, by the caller.
    Returns (ids uint8[n], perm int32[n], rank int32[n])."""
    if not x.is_cuda or x.dtype != torch.bfloat16 or x.dim() != 2:
        raise HyperAttnError("x must be a 2-D CUDA bf16 tensor")
    x = x.contiguous()
    n, d = x.shape
    ids = torch.empty(n, dtype=torch.uint8, device=x.device)
    perm = torch.empty(n, dtype=torch.int32, device=x.device)
    rank = torch.empty(n, dtype=torch.int32, device=x.device)
    s = stream if stream is not None else torch.cuda.current_stream(x.device).cuda_stream
    with torch.cuda.device(x.device):
        _check(lib().hyperattn_sortlsh_noalloc(x.data_ptr(), n, d, hash_bits, seed, ids.data_ptr(), perm.data_ptr(),
                                               rank.data_ptr(), s), "hyperattn_sortlsh_noalloc")
    return ids, perm, rank


def alpha(q, k, causal=False, skip_cols=0, scale=0.0, stream=None):
    """n times the largest squared column norm of the exact softmax matrix of every (batch, head) (the alpha
    of the paper's Theorem 1): CUDA bf16 tensors q [B, H, n, d], k [B, H, n_k, d] -> float tensor [B, H]."""
    if not (q.is_cuda and k.is_cuda) or q.dtype != torch.bfloat16 or k.dtype != torch.bfloat16:
        raise HyperAttnError("q and k must be CUDA bf16 tensors")
    q, k = q.contiguous(), k.contiguous()
    B, H, n, d = q.shape
    n_k = k.shape[2]
    nbytes = C.c_size_t(0)
    _check(lib().hyperattn_alpha_workspace_bytes(B, H, n, n_k, C.byref(nbytes)), "hyperattn_alpha_workspace_bytes")
    ws = torch.empty(int(nbytes.value), dtype=torch.uint8, device=q.device)
    out = torch.empty((B, H), dtype=torch.float32, device=q.device)
    s = stream if stream is not None else torch.cuda.current_stream(q.device).cuda_stream
    with torch.cuda.device(q.device):
        _check(lib().hyperattn_alpha(q.data_ptr(), k.data_ptr(), B, H, n, 0 if n_k == n else n_k, d, float(scale), int(bool(causal)),
                                     int(skip_cols), out.data_ptr(), ws.data_ptr(), ws.numel(), s), "hyperattn_alpha")
    return out


def workspace_bytes(B, H, n, d, block, samples, hash_bits, causal=False, n0=0, dtype=BF16, out_dtype=BF16, n_k=0) -> int:
    p = _Params()
    _fill(p, B, H, n, d, block, samples, hash_bits, causal, n0, 0, dtype, out_dtype, 0.0, n_k or n)
    nbytes = C.c_size_t(0)
    _check(lib().hyperattn_workspace_bytes(C.byref(p), C.byref(nbytes)), "hyperattn_workspace_bytes")
    return int(nbytes.value)


def get_projections(d: int, hash_bits: int, seed: int, node: int = 0) -> np.ndarray:
    w = np.zeros((d, hash_bits), dtype=np.float32)
    if node:
        _check(lib().hyperattn_get_node_projections(d, hash_bits, C.c_uint64(seed), node, w.ctypes.data), "hyperattn_get_node_projections")
    else:
        _check(lib().hyperattn_get_projections(d, hash_bits, seed, w.ctypes.data), "hyperattn_get_projections")
    return w


def last_device_status(stream=None) -> int:
    st = C.c_int(0)
    s = stream if stream is not None else torch.cuda.current_stream().cuda_stream
    _check(lib().hyperattn_last_device_status(s, C.byref(st)), "hyperattn_last_device_status")
    return int(st.value)


def profile_enable(on: bool, stages=None):
    """Stage timing on/off; `stages` (names from STAGE_NAMES) restricts it to those stages."""
    code = int(bool(on))
    if on and stages is not None:
        code = 0
        for name in stages:
            code |= 1 << (STAGE_NAMES.index(name) + 1)
    lib().hyperattn_profile_enable(code)


def profile_reset():
    lib().hyperattn_profile_reset()


def profile_read() -> dict:
    t = _StageTimes()
    _check(lib().hyperattn_profile_read(C.byref(t)), "hyperattn_profile_read")
    return {"calls": t.calls, "ms": {STAGE_NAMES[i]: float(t.ms[i]) for i in range(NUM_STAGES)},
            "launches": {STAGE_NAMES[i]: int(t.launches[i]) for i in range(NUM_STAGES)}}


def release():
    lib().hyperattn_release()


def version() -> int:
    return int(lib().hyperattn_version())
