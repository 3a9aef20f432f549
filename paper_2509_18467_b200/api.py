"""Thin ctypes binding of ``liblawcat.so``: argument marshalling only, every step of the layer runs in the CUDA kernels.

The functions carry the names of the C entry points declared in ``include/lawcat.h`` and take ``torch`` CUDA tensors
(PyTorch serves as the device allocator and stream provider). Outputs that the caller does not pass are allocated with
``torch.empty``. A missing library is a hard error: there is no CPU path.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "liblawcat.so")

F32, BF16 = 0, 1
PHI_SOFTMAX, PHI_ELU1, PHI_IDENTITY = 0, 1, 2
GATE_LOGITS, GATE_LOGDECAY = 0, 1
OP_CONV_FWD, OP_CONV_BWD, OP_GLA_FWD, OP_GLA_BWD, OP_LAYER_FWD, OP_DECODE_STEP, OP_LAYER_BWD = range(7)

EXPORTS = ["lawcat_workspace_bytes", "lawcat_status_string", "lawcat_version", "lawcat_launch_count",
           "lawcat_trace_begin", "lawcat_trace_end", "lawcat_test_set_wait_limit", "lawcat_conv_fwd", "lawcat_conv_bwd", "lawcat_gla_fwd",
           "lawcat_gla_bwd", "lawcat_layer_fwd", "lawcat_layer_fwd_varlen_workspace_bytes",
           "lawcat_layer_fwd_varlen", "lawcat_layer_bwd", "lawcat_decode_step", "lawcat_layer_fwd_host_arena_bytes",
           "lawcat_layer_fwd_host", "lawcat_noalloc_scratch_bytes", "lawcat_layer_fwd_noalloc", "lawcat_last_cuda_error", "lawcat_gate_fn_workspace_bytes",
           "lawcat_gate_fn_fwd"]


class LawcatError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = ""
        if status == 3:  # LAWCAT_ERR_CUDA: the runtime's own message, when a launch produced it
            f = lib().lawcat_last_cuda_error
            f.restype = ctypes.c_char_p
            detail = (f() or b"").decode()
        super().__init__(f"{where}: {status_string(status)} (status {status})" + (f": {detail}" if detail else ""))


class Params(ctypes.Structure):
    """Mirror of ``lawcat_params``."""
    _fields_ = [("B", ctypes.c_int32), ("T", ctypes.c_int32), ("H", ctypes.c_int32), ("H_kv", ctypes.c_int32),
                ("d_k", ctypes.c_int32), ("d_v", ctypes.c_int32), ("conv_k", ctypes.c_int32),
                ("gate_dim", ctypes.c_int32), ("chunk", ctypes.c_int32), ("dtype", ctypes.c_int32),
                ("phi", ctypes.c_int32), ("gate_mode", ctypes.c_int32), ("gate_tau", ctypes.c_float),
                ("eps", ctypes.c_float), ("normalize", ctypes.c_int32), ("mix_unshared", ctypes.c_int32)]


def params(B, T, H, H_kv, d_k, d_v, conv_k=4, gate_dim=0, chunk=0, dtype=BF16, phi=PHI_SOFTMAX,
           gate_mode=GATE_LOGITS, gate_tau=16.0, eps=0.0, normalize=1, mix_unshared=0) -> Params:
    if isinstance(dtype, str):
        dtype = {"f32": F32, "bf16": BF16}[dtype]
    return Params(B, T, H, H_kv, d_k, d_v, conv_k, gate_dim or d_k, chunk, dtype, phi, gate_mode, gate_tau, eps,
                  normalize, mix_unshared)


_lib = None


def lib() -> ctypes.CDLL:
    """Open the CUDA library; fail loudly when it has not been built."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2509_18467_b200.build` "
                               "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        L.lawcat_workspace_bytes.restype = ctypes.c_size_t
        L.lawcat_workspace_bytes.argtypes = [ctypes.POINTER(Params), ctypes.c_int]
        L.lawcat_status_string.restype = ctypes.c_char_p
        L.lawcat_status_string.argtypes = [ctypes.c_int]
        L.lawcat_version.restype = ctypes.c_int
        L.lawcat_launch_count.restype = ctypes.c_ulonglong
        L.lawcat_layer_fwd_host_arena_bytes.restype = ctypes.c_size_t
        L.lawcat_layer_fwd_host_arena_bytes.argtypes = [ctypes.POINTER(Params)]
        L.lawcat_noalloc_scratch_bytes.restype = ctypes.c_size_t
        L.lawcat_layer_fwd_noalloc.restype = ctypes.c_int
        L.lawcat_layer_fwd_noalloc.argtypes = [ctypes.POINTER(Params)] + [ctypes.c_void_p] * 18
        L.lawcat_layer_fwd_host.restype = ctypes.c_int
        L.lawcat_layer_fwd_host.argtypes = [ctypes.POINTER(Params)] + [ctypes.c_void_p] * 9 + \
                                           [ctypes.c_size_t, ctypes.c_void_p]
        L.lawcat_trace_end.argtypes = [ctypes.c_char_p, ctypes.c_size_t]
        for name, nptr in (("lawcat_conv_fwd", 9), ("lawcat_conv_bwd", 14), ("lawcat_gla_fwd", 10),
                           ("lawcat_gla_bwd", 13), ("lawcat_layer_fwd", 16), ("lawcat_layer_bwd", 19),
                           ("lawcat_decode_step", 12)):
            f = getattr(L, name)
            f.restype = ctypes.c_int
            f.argtypes = [ctypes.POINTER(Params)] + [ctypes.c_void_p] * nptr + \
                         [ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p]
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().lawcat_status_string(status).decode()


def launch_count() -> int:
    return int(lib().lawcat_launch_count())


def trace_begin() -> None:
    lib().lawcat_trace_begin()


def trace_end() -> dict:
    """Stop tracing; returns {kernel name: (launches, total device milliseconds)}."""
    buf = ctypes.create_string_buffer(1 << 16)
    st = lib().lawcat_trace_end(buf, len(buf))
    if st != 0:
        raise LawcatError(st, "lawcat_trace_end")
    out = {}
    for line in buf.value.decode().splitlines():
        name, n, ms = line.split()
        out[name] = (int(n), float(ms))
    return out


def test_set_wait_limit(cycles: int) -> None:
    """Test hook: bound (clock cycles) of the device-side waits of the tensor-core layer kernels; 0 = default."""
    f = lib().lawcat_test_set_wait_limit
    f.argtypes, f.restype = [ctypes.c_longlong], None
    f(cycles)


def workspace_bytes(p: Params, op: int) -> int:
    return int(lib().lawcat_workspace_bytes(ctypes.byref(p), op))


def torch_dtype(p: Params):
    return torch.float32 if p.dtype == F32 else torch.bfloat16


def _ptr(t: Optional[torch.Tensor]):
    if t is None or t.numel() == 0:
        return None
    assert t.is_cuda and t.is_contiguous(), "tensors must be contiguous CUDA tensors"
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _ws(p: Params, op: int, ws: Optional[torch.Tensor], dev):
    need = workspace_bytes(p, op)
    if ws is None and need:
        ws = torch.empty(need, dtype=torch.uint8, device=dev)
    return ws, (0 if ws is None else ws.numel() * ws.element_size())


def _call(name, p, ptrs, ws, ws_bytes, stream, dev_status):
    st = getattr(lib(), name)(ctypes.byref(p), *[_ptr(t) for t in ptrs], _ptr(ws), ws_bytes, _stream(stream),
                              _ptr(dev_status))
    if st != 0:
        raise LawcatError(st, name)


def lawcat_conv_fwd(p: Params, q, k, w_q, w_k, W=None, cache_q=None, cache_k=None, qdot=None, kdot=None, ws=None,
                    stream=None, dev_status=None):
    dt, dev = torch_dtype(p), q.device
    if qdot is None:
        qdot = torch.empty(p.B, p.T, p.H, p.d_k, dtype=dt, device=dev)
    if kdot is None:
        kdot = torch.empty(p.B, p.T, p.H if W is not None else p.H_kv, p.d_k, dtype=dt, device=dev)
    ws, nb = _ws(p, OP_CONV_FWD, ws, dev)
    _call("lawcat_conv_fwd", p, [q, k, w_q, w_k, W, cache_q, cache_k, qdot, kdot], ws, nb, stream, dev_status)
    return qdot, kdot


def lawcat_gate_fn_fwd(p: Params, d_model: int, rank: int, x, A1, A2, bias=None, gate=None, ws=None, stream=None,
                       dev_status=None):
    """x [B,T,d_model], A1 [rank,d_model], A2 [H*gate_dim,rank], bias [H*gate_dim] -> gate logits [B,T,H,gate_dim]."""
    dt, dev = torch_dtype(p), x.device
    if gate is None:
        gate = torch.empty(p.B, p.T, p.H, p.gate_dim, dtype=dt, device=dev)
    f = lib().lawcat_gate_fn_workspace_bytes
    f.restype = ctypes.c_size_t
    f.argtypes = [ctypes.POINTER(Params), ctypes.c_int32, ctypes.c_int32]
    need = f(ctypes.byref(p), d_model, rank)
    if ws is None and need:
        ws = torch.empty(need, dtype=torch.uint8, device=dev)
    nb = 0 if ws is None else ws.numel() * ws.element_size()
    st = lib().lawcat_gate_fn_fwd(ctypes.byref(p), ctypes.c_int32(d_model), ctypes.c_int32(rank), _ptr(x), _ptr(A1),
                                  _ptr(A2), _ptr(bias), _ptr(gate), _ptr(ws), ctypes.c_size_t(nb), _stream(stream),
                                  _ptr(dev_status))
    if st != 0:
        raise LawcatError(st, "lawcat_gate_fn_fwd")
    return gate


def lawcat_conv_bwd(p: Params, q, k, w_q, w_k, W, d_qdot, d_kdot, cache_q=None, cache_k=None, ws=None, stream=None,
                    dev_status=None):
    dev = q.device
    dq, dk = torch.empty_like(q), torch.empty_like(k)
    dw_q = torch.empty(w_q.shape, dtype=torch.float32, device=dev)
    dw_k = torch.empty(w_k.shape, dtype=torch.float32, device=dev)
    dW = None if W is None else torch.empty(W.shape, dtype=torch.float32, device=dev)
    ws, nb = _ws(p, OP_CONV_BWD, ws, dev)
    _call("lawcat_conv_bwd", p, [q, k, w_q, w_k, W, cache_q, cache_k, d_qdot, d_kdot, dq, dk, dw_q, dw_k, dW], ws,
          nb, stream, dev_status)
    return dict(dq=dq, dk=dk, dw_q=dw_q, dw_k=dw_k, dW=dW)


def lawcat_gla_fwd(p: Params, qdot, kdot, v, gate, S0=None, z0=None, o=None, want_den=True, want_state=True, ws=None,
                   stream=None, dev_status=None):
    dt, dev = torch_dtype(p), qdot.device
    if o is None:
        o = torch.empty(p.B, p.T, p.H, p.d_v, dtype=dt, device=dev)
    den = torch.empty(p.B, p.T, p.H, dtype=torch.float32, device=dev) if want_den else None
    S_T = torch.empty(p.B, p.H, p.d_k, p.d_v, dtype=torch.float32, device=dev) if want_state else None
    z_T = torch.empty(p.B, p.H, p.d_k, dtype=torch.float32, device=dev) if want_state else None
    ws, nb = _ws(p, OP_GLA_FWD, ws, dev)
    _call("lawcat_gla_fwd", p, [qdot, kdot, v, gate, S0, z0, o, den, S_T, z_T], ws, nb, stream, dev_status)
    return dict(o=o, den=den, S_T=S_T, z_T=z_T)


def lawcat_gla_bwd(p: Params, qdot, kdot, v, gate, o, den, dO, S0=None, z0=None, ws=None, stream=None,
                   dev_status=None):
    dev = qdot.device
    d_qdot, d_kdot, dv, dgate = (torch.empty_like(x) for x in (qdot, kdot, v, gate))
    ws, nb = _ws(p, OP_GLA_BWD, ws, dev)
    _call("lawcat_gla_bwd", p, [qdot, kdot, v, gate, S0, z0, o, den, dO, d_qdot, d_kdot, dv, dgate], ws, nb, stream,
          dev_status)
    return dict(d_qdot=d_qdot, d_kdot=d_kdot, dv=dv, dgate=dgate)


def lawcat_layer_fwd(p: Params, q, k, v, gate, w_q, w_k, W, cache_q=None, cache_k=None, S0=None, z0=None, o=None,
                     want_state=True, want_cache=True, ws=None, stream=None, dev_status=None):
    dt, dev = torch_dtype(p), q.device
    if o is None:
        o = torch.empty(p.B, p.T, p.H, p.d_v, dtype=dt, device=dev)
    # want_state: True / False, or "S" / "z" for one of the two state outputs alone (each is optional on its own)
    S_T = torch.empty(p.B, p.H, p.d_k, p.d_v, dtype=torch.float32, device=dev) if want_state in (True, "S") else None
    z_T = torch.empty(p.B, p.H, p.d_k, dtype=torch.float32, device=dev) if want_state in (True, "z") else None
    cq = torch.empty(p.B, p.conv_k - 1, p.H * p.d_k, dtype=dt, device=dev) if want_cache else None
    ck = torch.empty(p.B, p.conv_k - 1, p.H_kv * p.d_k, dtype=dt, device=dev) if want_cache else None
    ws, nb = _ws(p, OP_LAYER_FWD, ws, dev)
    _call("lawcat_layer_fwd", p, [q, k, v, gate, w_q, w_k, W, cache_q, cache_k, S0, z0, o, cq, ck, S_T, z_T], ws, nb,
          stream, dev_status)
    return dict(o=o, cache_q=cq, cache_k=ck, S_T=S_T, z_T=z_T)


def lawcat_layer_fwd_varlen(p: Params, cu_seqlens, q, k, v, gate, w_q, w_k, W, cache_q=None, cache_k=None, S0=None, z0=None,
                            stream=None, dev_status=None):
    """Packed sequences (B = 1): cu_seqlens is a host sequence of nseq + 1 token offsets. Returns dict(o, cache_q, cache_k,
    S_T, z_T) with the state outputs per sequence."""
    L = lib()
    nseq = len(cu_seqlens) - 1
    cu = (ctypes.c_int32 * (nseq + 1))(*[int(x) for x in cu_seqlens])
    dt, dev = torch_dtype(p), q.device
    o = torch.empty(1, p.T, p.H, p.d_v, dtype=dt, device=dev)
    S_T = torch.empty(nseq, p.H, p.d_k, p.d_v, dtype=torch.float32, device=dev)
    z_T = torch.empty(nseq, p.H, p.d_k, dtype=torch.float32, device=dev)
    cq = torch.empty(nseq, p.conv_k - 1, p.H * p.d_k, dtype=dt, device=dev)
    ck = torch.empty(nseq, p.conv_k - 1, p.H_kv * p.d_k, dtype=dt, device=dev)
    L.lawcat_layer_fwd_varlen_workspace_bytes.restype = ctypes.c_size_t
    L.lawcat_layer_fwd_varlen_workspace_bytes.argtypes = [ctypes.POINTER(Params), ctypes.c_void_p, ctypes.c_int]
    need = int(L.lawcat_layer_fwd_varlen_workspace_bytes(ctypes.byref(p), cu, nseq))
    ws = torch.empty(max(need, 16), dtype=torch.uint8, device=dev)
    f = L.lawcat_layer_fwd_varlen
    f.restype = ctypes.c_int
    f.argtypes = [ctypes.POINTER(Params), ctypes.c_void_p, ctypes.c_int] + [ctypes.c_void_p] * 17 + \
                 [ctypes.c_size_t, ctypes.c_void_p, ctypes.c_void_p]
    st = f(ctypes.byref(p), cu, nseq, *[_ptr(t) for t in (q, k, v, gate, w_q, w_k, W, cache_q, cache_k, S0, z0, o, cq, ck,
                                                          S_T, z_T)], _ptr(ws), ws.numel(), _stream(stream),
           _ptr(dev_status))
    if st != 0:
        raise LawcatError(st, "lawcat_layer_fwd_varlen")
    return dict(o=o, cache_q=cq, cache_k=ck, S_T=S_T, z_T=z_T)


def lawcat_layer_bwd(p: Params, q, k, v, gate, w_q, w_k, W, dO, cache_q=None, cache_k=None, S0=None, z0=None, ws=None,
                     stream=None, dev_status=None):
    """Gradients of the whole layer for the upstream gradient dO: dict(dq, dk, dv, dgate, dw_q, dw_k, dW)."""
    dev = q.device
    dq, dk, dv, dgate = (torch.empty_like(x) for x in (q, k, v, gate))
    dw_q = torch.empty(w_q.shape, dtype=torch.float32, device=dev)
    dw_k = torch.empty(w_k.shape, dtype=torch.float32, device=dev)
    dW = torch.empty(W.shape, dtype=torch.float32, device=dev)
    ws, nb = _ws(p, OP_LAYER_BWD, ws, dev)
    _call("lawcat_layer_bwd", p, [q, k, v, gate, w_q, w_k, W, cache_q, cache_k, S0, z0, dO, dq, dk, dv, dgate, dw_q, dw_k,
                                  dW], ws, nb, stream, dev_status)
    return dict(dq=dq, dk=dk, dv=dv, dgate=dgate, dw_q=dw_q, dw_k=dw_k, dW=dW)


def lawcat_decode_step(p: Params, q_t, k_t, v_t, gate_t, w_q, w_k, W, S, z, cache_q, cache_k, o_t=None, ws=None,
                       stream=None, dev_status=None):
    """S, z, cache_q, cache_k are updated in place; returns o_t [B,H,d_v]."""
    if o_t is None:
        o_t = torch.empty(p.B, p.H, p.d_v, dtype=torch_dtype(p), device=q_t.device)
    ws, nb = _ws(p, OP_DECODE_STEP, ws, q_t.device)
    _call("lawcat_decode_step", p, [q_t, k_t, v_t, gate_t, w_q, w_k, W, S, z, cache_q, cache_k, o_t], ws, nb, stream,
          dev_status)
    return o_t


def lawcat_layer_fwd_host(p: Params, h_q, h_k, h_v, h_gate, h_w_q, h_w_k, h_W, h_o, arena, stream=None):
    """Host tensors in (pinned for asynchronous copies), host tensor h_o out; `arena` is a CUDA uint8 tensor of at
    least ``lawcat_layer_fwd_host_arena_bytes`` bytes. Enqueues copies + layer + copy back; does not synchronize."""
    hp = lambda t: ctypes.c_void_p(t.data_ptr())
    st = lib().lawcat_layer_fwd_host(ctypes.byref(p), *[hp(t) for t in (h_q, h_k, h_v, h_gate, h_w_q, h_w_k, h_W, h_o)],
                                     _ptr(arena), arena.numel(), _stream(stream))
    if st != 0:
        raise LawcatError(st, "lawcat_layer_fwd_host")
    return h_o


def lawcat_layer_fwd_noalloc(p: Params, q, k, v, gate, w_q, w_k, W, cache_q=None, cache_k=None, S0=None, z0=None,
                             o=None, cache_q_out=None, cache_k_out=None, S_T=None, z_T=None, stream=None,
                             dev_status=None):
    """The layer forward for callers that cannot allocate: no workspace argument, the scratch is a fixed array inside
    the library (see the header for its size limit and the sharing rules). Every output must be passed in by the
    caller; only `o` is required. Returns o."""
    ptrs = [q, k, v, gate, w_q, w_k, W, cache_q, cache_k, S0, z0, o, cache_q_out, cache_k_out, S_T, z_T]
    st = lib().lawcat_layer_fwd_noalloc(ctypes.byref(p), *[_ptr(t) for t in ptrs], _stream(stream), _ptr(dev_status))
    if st != 0:
        raise LawcatError(st, "lawcat_layer_fwd_noalloc")
    return o


def host_arena_bytes(p: Params) -> int:
    return int(lib().lawcat_layer_fwd_host_arena_bytes(ctypes.byref(p)))


def to_device(x, dtype, device="cuda"):
    """numpy float32 array (already bf16-representable when dtype is bf16) -> CUDA tensor of the storage type."""
    t = torch.from_numpy(x)
    if dtype in (BF16, "bf16", torch.bfloat16):
        return t.to(device).to(torch.bfloat16)
    return t.to(device)
