"""ctypes binding of libpsk.so: same names as the C ABI, argument marshalling only."""
from __future__ import annotations

import ctypes
import os
from ctypes import c_int, c_int32, c_int64, c_size_t, c_void_p, c_char_p, POINTER, Structure, byref

import torch

PATH_AUTO, PATH_CUDA_CORES, PATH_TENSOR_CORES = 0, 1, 2
FLAG_KEEP_STATES = 1
FLAG_LOCAL_EXACT = 2
FLAG_NONCAUSAL = 4
_DTYPES = {torch.float32: 0, torch.bfloat16: 1}
_PKG = os.path.dirname(os.path.abspath(__file__))


class PskError(RuntimeError):
    def __init__(self, code, where):
        self.code = code
        super().__init__("%s: %s (%d)" % (where, status_string(code), code))


class Shape(Structure):
    """Mirror of `psk_shape`."""
    _fields_ = [("B", c_int32), ("H", c_int32), ("n", c_int32), ("h", c_int32), ("r", c_int32),
                ("p", c_int32), ("b", c_int32), ("dtype", c_int32),
                ("stride_b", c_int64), ("stride_h", c_int64), ("stride_n", c_int64),
                ("g_heads", c_int32), ("path", c_int32), ("flags", c_int32), ("seq_segments", c_int32)]


_lib = None


def library_path() -> str:
    """libpsk.so beside this file, or the library the environment variable PSK_LIBRARY names."""
    return os.environ.get("PSK_LIBRARY") or os.path.join(_PKG, "libpsk.so")


def lib():
    """Loads libpsk.so (built in-tree by `python -m paper_2310_01655_b200.build`)."""
    global _lib
    if _lib is not None:
        return _lib
    path = library_path()
    if not os.path.exists(path):
        raise RuntimeError("libpsk.so is not built: run `python -m paper_2310_01655_b200.build` "
                           "(there is no fallback implementation)")
    L = ctypes.CDLL(path)
    P = POINTER(Shape)
    L.psk_version.restype = c_int
    L.psk_status_string.restype = c_char_p
    L.psk_status_string.argtypes = [c_int]
    L.psk_workspace_bytes.restype = c_size_t
    L.psk_workspace_bytes.argtypes = [P, c_int]
    L.psk_sketch.restype = c_int
    L.psk_sketch.argtypes = [P] + [c_void_p] * 6
    L.psk_causal_attn_fwd.restype = c_int
    L.psk_causal_attn_fwd.argtypes = [P] + [c_void_p] * 8 + [c_size_t, c_void_p]
    L.psk_causal_attn_bwd.restype = c_int
    L.psk_causal_attn_bwd.argtypes = [P] + [c_void_p] * 12 + [c_size_t, c_void_p]
    L.psk_static_scratch_bytes.restype = c_size_t
    L.psk_causal_attn_fwd_static.restype = c_int
    L.psk_causal_attn_fwd_static.argtypes = [P] + [c_void_p] * 8
    L.psk_check.restype = c_int
    L.psk_check.argtypes = [c_void_p, c_void_p]
    L.psk_selftest_wait_timeout.restype = c_int
    L.psk_selftest_wait_timeout.argtypes = [c_void_p, c_size_t, ctypes.c_uint64, c_void_p]
    L.psk_last_launch_count.restype = c_int
    L.psk_lt_multiply_workspace_bytes.restype = c_size_t
    L.psk_lt_multiply_workspace_bytes.argtypes = [c_int] * 5
    L.psk_lt_multiply.restype = c_int
    L.psk_lt_multiply.argtypes = [c_int] * 5 + [c_void_p] * 5 + [c_size_t, c_void_p]
    L.psk_lt_multiply_bf16_workspace_bytes.restype = c_size_t
    L.psk_lt_multiply_bf16_workspace_bytes.argtypes = [c_int] * 5
    L.psk_lt_multiply_bf16.restype = c_int
    L.psk_lt_multiply_bf16.argtypes = [c_int] * 5 + [c_void_p] * 5 + [c_size_t, c_void_p]
    L.psk_decode_state_bytes.restype = c_size_t
    L.psk_decode_state_bytes.argtypes = [POINTER(Shape)]
    L.psk_decode_step.restype = c_int
    L.psk_decode_step.argtypes = [POINTER(Shape)] + [c_void_p] * 9
    L.psk_learned_param_count.restype = c_size_t
    L.psk_learned_param_count.argtypes = [c_int, c_int]
    L.psk_learned_workspace_bytes.restype = c_size_t
    L.psk_learned_workspace_bytes.argtypes = [P, c_int]
    L.psk_learned_sketch.restype = c_int
    L.psk_learned_sketch.argtypes = [P] + [c_void_p] * 5
    L.psk_learned_attn_fwd.restype = c_int
    L.psk_learned_attn_fwd.argtypes = [P] + [c_void_p] * 7 + [c_size_t, c_void_p]
    L.psk_learned_attn_bwd.restype = c_int
    L.psk_learned_attn_bwd.argtypes = [P] + [c_void_p] * 12 + [c_size_t, c_void_p]
    L.psk_profile_enable.restype = c_int
    L.psk_profile_enable.argtypes = [c_int]
    L.psk_profile_count.restype = c_int
    L.psk_feature_table.restype = c_int
    L.psk_feature_table.argtypes = [c_int, c_void_p, c_void_p, c_void_p, c_int]
    L.psk_profile_get.restype = c_int
    L.psk_profile_get.argtypes = [c_int, ctypes.c_char_p, c_size_t, POINTER(ctypes.c_float)]
    _lib = L
    return L


def status_string(code: int) -> str:
    return lib().psk_status_string(int(code)).decode()


def _require_cuda(*ts):
    for t in ts:
        if t is not None and not t.is_cuda:
            raise RuntimeError("psk: tensors must live on a CUDA device (no CPU path exists)")


def _ptr(t):
    return c_void_p(t.data_ptr()) if t is not None else c_void_p(0)


def _contig(t):
    return t.contiguous() if t is not None else None


def _sketch_r(G1, x):
    return G1.shape[-1] if G1 is not None else x.shape[-1]      # p = 2: the half sketch is the row, r = h


def _stream():
    return c_void_p(torch.cuda.current_stream().cuda_stream)


def make_shape(x: torch.Tensor, G1: torch.Tensor, r: int, b: int, p: int = 4, path: int = PATH_AUTO,
               flags: int = 0, seq_segments: int = 0) -> Shape:
    """Shape descriptor for a [B,H,n,h] tensor `x` (its strides are used for all eight tensors)."""
    if x.dim() != 4 or x.stride(3) != 1:
        raise ValueError("expected a [B,H,n,h] tensor with a contiguous last dimension")
    if x.dtype not in _DTYPES:
        raise ValueError("unsupported storage dtype %s" % x.dtype)
    B, H, n, h = x.shape
    g_heads = G1.shape[0] if (G1 is not None and G1.dim() == 3) else 1
    return Shape(B, H, n, h, r, p, b, _DTYPES[x.dtype], x.stride(0), x.stride(1), x.stride(2), g_heads, path, flags,
                 seq_segments)


def workspace_bytes(shape: Shape, for_backward: bool) -> int:
    return int(lib().psk_workspace_bytes(byref(shape), 1 if for_backward else 0))


def _workspace(shape, for_backward, workspace):
    need = workspace_bytes(shape, for_backward)
    if need == 0:
        # let the library report the precise reason
        return None, 0
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device="cuda")
    return workspace, workspace.numel()


def _check_sketch_matrices(*gs):
    for g in gs:
        if g is not None and not g.is_contiguous():
            raise ValueError("G1 and G2 must be contiguous [g_heads, h, r] tensors")


def _check_keep_states(flags, workspace):
    if (flags & FLAG_KEEP_STATES) and workspace is None:
        raise ValueError("FLAG_KEEP_STATES needs a caller-owned workspace shared by the forward and the backward call")


def _same_layout(ref, *ts):
    for t in ts:
        if t is not None and (t.shape != ref.shape or t.stride() != ref.stride() or t.dtype != ref.dtype):
            raise ValueError("all [B,H,n,h] tensors must share shape, strides and dtype")


def _empty_like(x):
    """Uninitialised tensor with exactly x's shape AND strides (views included)."""
    return torch.empty_strided(x.shape, x.stride(), dtype=x.dtype, device=x.device)


def sketch(X, G1, G2, r=None, b=128, want_phi=False, path=PATH_AUTO):
    """psk_sketch: returns (M [B,H,n,r] fp32, Phi [B,H,n,r*r] fp32 or None)."""
    _require_cuda(X, G1, G2)
    p = 4 if G1 is not None else 2             # no sketch matrices: degree 2, M = X
    r = (G1.shape[-1] if G1 is not None else X.shape[-1]) if r is None else r
    shp = make_shape(X, G1, r, b, p, path=path)
    B, H, n, _ = X.shape
    M = torch.empty((B, H, n, r), dtype=torch.float32, device=X.device)
    Phi = torch.empty((B, H, n, r * r), dtype=torch.float32, device=X.device) if want_phi else None
    st = lib().psk_sketch(byref(shp), _ptr(X), _ptr(_contig(G1)), _ptr(_contig(G2)), _ptr(M), _ptr(Phi),
                          _stream())
    if st != 0:
        raise PskError(st, "psk_sketch")
    return M, Phi


def causal_attn_fwd(Q, K, V, G1, G2, b, p=4, path=PATH_AUTO, workspace=None, out=None, denom=None, flags=0,
                    seq_segments=0):
    """psk_causal_attn_fwd: returns (O, denom)."""
    _require_cuda(Q, K, V, G1, G2)
    _check_sketch_matrices(G1, G2)
    _check_keep_states(flags, workspace)
    _same_layout(Q, K, V, out)
    shp = make_shape(Q, G1, _sketch_r(G1, Q), b, p, path, flags, seq_segments)
    O = _empty_like(Q) if out is None else out
    B, H, n, _ = Q.shape
    if denom is None:
        denom = torch.empty((B, H, n), dtype=torch.float32, device=Q.device)
    ws, nbytes = _workspace(shp, False, workspace)
    st = lib().psk_causal_attn_fwd(byref(shp), _ptr(Q), _ptr(K), _ptr(V), _ptr(G1), _ptr(G2), _ptr(O),
                                   _ptr(denom), _ptr(ws), nbytes, _stream())
    if st != 0:
        raise PskError(st, "psk_causal_attn_fwd")
    return O, denom


def static_scratch_bytes() -> int:
    return int(lib().psk_static_scratch_bytes())


def causal_attn_fwd_static(Q, K, V, G1, G2, b, p=4, out=None, denom=None):
    """psk_causal_attn_fwd_static: the forward for callers that cannot allocate device
    memory.  The library uses its built-in 16 MiB scratch array, so no workspace is passed
    and nothing is allocated by the call itself; `out` and `denom` must be supplied by such
    a caller (they are created here only as a convenience when omitted)."""
    _require_cuda(Q, K, V, G1, G2)
    _check_sketch_matrices(G1, G2)
    _same_layout(Q, K, V, out)
    shp = make_shape(Q, G1, _sketch_r(G1, Q), b, p, PATH_CUDA_CORES)
    O = _empty_like(Q) if out is None else out
    B, H, n, _ = Q.shape
    if denom is None:
        denom = torch.empty((B, H, n), dtype=torch.float32, device=Q.device)
    st = lib().psk_causal_attn_fwd_static(byref(shp), _ptr(Q), _ptr(K), _ptr(V), _ptr(G1), _ptr(G2), _ptr(O),
                                          _ptr(denom), _stream())
    if st != 0:
        raise PskError(st, "psk_causal_attn_fwd_static")
    return O, denom


def causal_attn_bwd(Q, K, V, G1, G2, O, denom, dO, b, p=4, path=PATH_AUTO, workspace=None, out=None, flags=0,
                    seq_segments=0):
    """psk_causal_attn_bwd: returns (dQ, dK, dV)."""
    _require_cuda(Q, K, V, G1, G2, O, denom, dO)
    _check_sketch_matrices(G1, G2)
    _check_keep_states(flags, workspace)
    _same_layout(Q, K, V, O, dO)
    shp = make_shape(Q, G1, _sketch_r(G1, Q), b, p, path, flags, seq_segments)
    dQ, dK, dV = out if out is not None else (_empty_like(Q), _empty_like(Q), _empty_like(Q))
    _same_layout(Q, dQ, dK, dV)
    ws, nbytes = _workspace(shp, True, workspace)
    st = lib().psk_causal_attn_bwd(byref(shp), _ptr(Q), _ptr(K), _ptr(V), _ptr(G1), _ptr(G2), _ptr(O),
                                   _ptr(denom), _ptr(dO), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(ws), nbytes,
                                   _stream())
    if st != 0:
        raise PskError(st, "psk_causal_attn_bwd")
    return dQ, dK, dV


def check(workspace) -> int:
    """psk_check: synchronises the current stream and returns the device-side status."""
    return int(lib().psk_check(_ptr(workspace), _stream()))


def selftest_wait_timeout(workspace, limit_ns: int):
    """psk_selftest_wait_timeout: makes a bounded device-side wait run out (nothing hangs or traps).
    Returns (ns of the first wait, ns of the second wait, threads failed first, threads failed second)
    after synchronising; psk_check(workspace) then reports the timeout."""
    st = lib().psk_selftest_wait_timeout(_ptr(workspace), workspace.numel(), int(limit_ns), _stream())
    if st != 0:
        raise PskError(st, "psk_selftest_wait_timeout")
    torch.cuda.current_stream().synchronize()
    rep = workspace[64:96].view(torch.int64).cpu().tolist()
    return tuple(int(x) for x in rep)


def last_launch_count() -> int:
    return int(lib().psk_last_launch_count())


def profile_enable(on: bool) -> None:
    """psk_profile_enable: start (discarding old records) or stop per-kernel event timing."""
    lib().psk_profile_enable(1 if on else 0)


def profile_records():
    """All launches recorded since profile_enable(True): list of (kernel name, ms)."""
    L = lib()
    out = []
    buf = ctypes.create_string_buffer(64)
    ms = ctypes.c_float()
    for i in range(L.psk_profile_count()):
        st = L.psk_profile_get(i, buf, 64, byref(ms))
        if st != 0:
            raise PskError(st, "psk_profile_get")
        out.append((buf.value.decode(), float(ms.value)))
    return out


def feature_table(r: int):
    """psk_feature_table: (a, b, w) numpy arrays of the tensor-core path's stored features (host only)."""
    import numpy as np
    cap = 4096
    a = np.zeros(cap, dtype=np.int32)
    b = np.zeros(cap, dtype=np.int32)
    w = np.zeros(cap, dtype=np.float32)
    n = lib().psk_feature_table(int(r), a.ctypes.data, b.ctypes.data, w.ctypes.data, cap)
    if n < 0:
        raise PskError(n, "psk_feature_table")
    return a[:n].copy(), b[:n].copy(), w[:n].copy()


def lt_multiply(A, B, C, b, workspace=None):
    """psk_lt_multiply: lt(A B^T) C for fp32 CUDA tensors A, B [batch, n, m] and C [batch, n, k]."""
    _require_cuda(A, B, C)
    for t in (A, B, C):
        if t.dtype != torch.float32 or t.dim() != 3 or not t.is_contiguous():
            raise ValueError("lt_multiply expects contiguous fp32 [batch, n, *] tensors")
    batch, n, m = A.shape
    k = C.shape[2]
    if B.shape != A.shape or C.shape[:2] != A.shape[:2]:
        raise ValueError("lt_multiply: A, B [batch, n, m] and C [batch, n, k] must agree")
    need = int(lib().psk_lt_multiply_workspace_bytes(batch, n, m, k, b))
    if workspace is None and need:
        workspace = torch.empty(need, dtype=torch.uint8, device=A.device)
    out = torch.empty_like(C)
    st = lib().psk_lt_multiply(batch, n, m, k, b, _ptr(A), _ptr(B), _ptr(C), _ptr(out), _ptr(workspace),
                               workspace.numel() if workspace is not None else 0, _stream())
    if st != 0:
        raise PskError(st, "psk_lt_multiply")
    return out


def lt_multiply_bf16(A, B, C, b, workspace=None):
    """psk_lt_multiply_bf16: lt(A B^T) C on the tensor cores for bf16 CUDA tensors A, B [batch, n, m] and
    C [batch, n, 64]; returns (Out fp32 [batch, n, 64], workspace) - pass the workspace to check()."""
    _require_cuda(A, B, C)
    for t in (A, B, C):
        if t.dtype != torch.bfloat16 or t.dim() != 3 or not t.is_contiguous():
            raise ValueError("lt_multiply_bf16 expects contiguous bf16 [batch, n, *] tensors")
    batch, n, m = A.shape
    k = C.shape[2]
    if B.shape != A.shape or C.shape[:2] != A.shape[:2]:
        raise ValueError("lt_multiply_bf16: A, B [batch, n, m] and C [batch, n, k] must agree")
    need = int(lib().psk_lt_multiply_bf16_workspace_bytes(batch, n, m, k, b))
    if workspace is None:
        workspace = torch.empty(max(need, 256), dtype=torch.uint8, device=A.device)
    out = torch.empty((batch, n, k), dtype=torch.float32, device=A.device)
    st = lib().psk_lt_multiply_bf16(batch, n, m, k, b, _ptr(A), _ptr(B), _ptr(C), _ptr(out), _ptr(workspace),
                                    workspace.numel() if need else 0, _stream())
    if st != 0:
        raise PskError(st, "psk_lt_multiply_bf16")
    return out, workspace


# ---- learnable sketch (Algorithm 2): parameter packing and the three calls ----
LEARNED_KEYS = ("g0", "c0", "W1", "b1", "g1", "c1", "W2", "b2", "W3", "b3", "W4", "b4")


def learned_param_count(h: int, r: int) -> int:
    """Floats in one network's packed parameter vector (0 for unsupported h, r)."""
    return int(lib().psk_learned_param_count(int(h), int(r)))


def learned_shapes(h: int, r: int):
    m = 8 * r
    return {"g0": (h,), "c0": (h,), "W1": (h, m), "b1": (m,), "g1": (m,), "c1": (m,), "W2": (m, r), "b2": (r,),
            "W3": (r, m), "b3": (m,), "W4": (m, r), "b4": (r,)}


def pack_learned_params(P1, P2, device="cuda"):
    """Two dicts of arrays (keys LEARNED_KEYS) -> the fp32 [2, count] tensor the library reads."""
    rows = []
    for P in (P1, P2):
        rows.append(torch.cat([torch.as_tensor(P[k], dtype=torch.float32).reshape(-1) for k in LEARNED_KEYS]))
    return torch.stack(rows).to(device).contiguous()


def unpack_learned_params(flat, h: int, r: int):
    """The inverse of pack_learned_params (for gradients): a pair of dicts of tensors."""
    out = []
    for row in flat:
        o, P = 0, {}
        for k, shp in learned_shapes(h, r).items():
            cnt = 1
            for x in shp:
                cnt *= x
            P[k] = row[o:o + cnt].reshape(shp)
            o += cnt
        out.append(P)
    return out[0], out[1]


def _learned_shape(x, r, b, flags, path=PATH_AUTO):
    return make_shape(x, None, r, b, 4, path, flags)


def learned_sketch(X, params, r, want_phi=False):
    """psk_learned_sketch: (M [B,H,n,r] fp32, Phi [B,H,n,r*r] fp32 or None)."""
    _require_cuda(X, params)
    B, H, n, _ = X.shape
    shp = _learned_shape(X, r, 128, 0)
    M = torch.empty((B, H, n, r), dtype=torch.float32, device=X.device)
    Phi = torch.empty((B, H, n, r * r), dtype=torch.float32, device=X.device) if want_phi else None
    st = lib().psk_learned_sketch(byref(shp), _ptr(X), _ptr(params), _ptr(M), _ptr(Phi), _stream())
    if st != 0:
        raise PskError(st, "psk_learned_sketch")
    return M, Phi


def learned_workspace_bytes(Q, r, b, flags=0, for_backward=True, path=PATH_AUTO):
    """psk_learned_workspace_bytes for tensors laid out like Q (the backward's covers the forward's)."""
    shp = _learned_shape(Q, r, b, flags, path)
    return int(lib().psk_learned_workspace_bytes(byref(shp), 1 if for_backward else 0))


def learned_attn_fwd(Q, K, V, params, r, b, flags=0, workspace=None, path=PATH_AUTO):
    """psk_learned_attn_fwd: returns (O, denom)."""
    _require_cuda(Q, K, V, params)
    _same_layout(Q, K, V)
    shp = _learned_shape(Q, r, b, flags, path)
    need = int(lib().psk_learned_workspace_bytes(byref(shp), 0))
    ws = workspace if workspace is not None else torch.empty(max(need, 256), dtype=torch.uint8, device=Q.device)
    B, H, n, _ = Q.shape
    O = _empty_like(Q)
    den = torch.empty((B, H, n), dtype=torch.float32, device=Q.device)
    st = lib().psk_learned_attn_fwd(byref(shp), _ptr(Q), _ptr(K), _ptr(V), _ptr(params), _ptr(O), _ptr(den), _ptr(ws),
                                    ws.numel() if need else 0, _stream())
    if st != 0:
        raise PskError(st, "psk_learned_attn_fwd")
    return O, den


def learned_attn_bwd(Q, K, V, params, O, denom, dO, r, b, flags=0, workspace=None, path=PATH_AUTO):
    """psk_learned_attn_bwd: returns (dQ, dK, dV, dparams [2, count] fp32)."""
    _require_cuda(Q, K, V, params, O, denom, dO)
    _same_layout(Q, K, V, O, dO)
    shp = _learned_shape(Q, r, b, flags, path)
    need = int(lib().psk_learned_workspace_bytes(byref(shp), 1))
    ws = workspace if workspace is not None else torch.empty(max(need, 256), dtype=torch.uint8, device=Q.device)
    dQ, dK, dV = _empty_like(Q), _empty_like(Q), _empty_like(Q)
    dparams = torch.empty_like(params)
    st = lib().psk_learned_attn_bwd(byref(shp), _ptr(Q), _ptr(K), _ptr(V), _ptr(params), _ptr(O), _ptr(denom), _ptr(dO),
                                    _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(dparams), _ptr(ws), ws.numel() if need else 0,
                                    _stream())
    if st != 0:
        raise PskError(st, "psk_learned_attn_bwd")
    return dQ, dK, dV, dparams


def decode_state(B, H, r, device="cuda"):
    """Zero state for decode_step: [B, H, r*r, 65] fp32."""
    return torch.zeros((B, H, r * r, 65), dtype=torch.float32, device=device)


def decode_step(q, k, v, G1, G2, state):
    """psk_decode_step: q, k, v [B, H, h]; updates `state` in place; returns (o [B, H, h], denom [B, H])."""
    _require_cuda(q, k, v, G1, G2, state)
    B, H, h = q.shape
    r = G1.shape[-1]
    g_heads = G1.shape[0] if G1.dim() == 3 else 1
    if not (q.is_contiguous() and k.is_contiguous() and v.is_contiguous() and state.is_contiguous()):
        raise ValueError("decode_step expects contiguous tensors")
    shp = Shape(B, H, 1, h, r, 4, 128, _DTYPES[q.dtype], H * h, h, h, g_heads, PATH_AUTO, 0, 0)
    if state.numel() * 4 != int(lib().psk_decode_state_bytes(byref(shp))):
        raise ValueError("decode_step: state must be [B, H, r*r, 65] fp32")
    o = torch.empty_like(q)
    den = torch.empty((B, H), dtype=torch.float32, device=q.device)
    st = lib().psk_decode_step(byref(shp), _ptr(q), _ptr(k), _ptr(v), _ptr(_contig(G1)), _ptr(_contig(G2)),
                               _ptr(state), _ptr(o), _ptr(den), _stream())
    if st != 0:
        raise PskError(st, "psk_decode_step")
    return o, den
