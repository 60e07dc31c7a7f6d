"""Thin binding over the C ABI of ``libl2a.so`` (declared in ``include/l2a.h``).

Argument marshalling only: every step of the path runs in the CUDA kernels of the library.  There is
no fallback -- if the library has not been built (``python -m paper_2603_17484_b200.build``) or
cannot be loaded, the first call raises.  torch is used for device memory and streams.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libl2a.so")

L2A_OK = 0
FLAG_SAVE_FOR_BWD = 1
FLAG_SKIP_LOCAL = 2
FLAG_SKIP_GLOBAL = 4
FLAG_FORCE_ALL_GLOBAL = 8
FLAG_GLOBAL_PHASE = 16
FLAG_SHARED_WINDOW = 64
ROUTER_MASK_U8 = 0
ROUTER_LOGITS_F32 = 1
ROUTER_LOGITS_BF16 = 2

EXPORTS = (
    "l2a_version", "l2a_status_string", "l2a_workspace_bytes", "l2a_workspace_status",
    "l2a_route_compact", "l2a_forward", "l2a_backward", "l2a_step_host", "l2a_profile_next_call",
    "l2a_route_compact_static", "l2a_router_logits", "l2a_decode_workspace_bytes", "l2a_decode",
    "l2a_backward_split", "l2a_router_backward", "l2a_forward_routed", "l2a_selftest_wait_timeout",
    "l2a_forward_sets", "l2a_backward_sets", "l2a_pack_sequences", "l2a_step_host_async", "l2a_step_host_wait",
)


class L2AParams(ctypes.Structure):
    _fields_ = [
        ("B", ctypes.c_int32), ("Lq", ctypes.c_int32), ("Lk", ctypes.c_int32),
        ("Hq", ctypes.c_int32), ("Hkv", ctypes.c_int32), ("D", ctypes.c_int32),
        ("window", ctypes.c_int32), ("q_pos_offset", ctypes.c_int32),
        ("softmax_scale", ctypes.c_float), ("flags", ctypes.c_uint32),
        ("q_stride", ctypes.c_int64 * 2), ("k_stride", ctypes.c_int64 * 2),
        ("v_stride", ctypes.c_int64 * 2), ("o_stride", ctypes.c_int64 * 2),
        ("seq_bounds", ctypes.c_void_p),
    ]


class L2AError(RuntimeError):
    def __init__(self, code: int, where: str):
        self.code = code
        super().__init__(f"{where}: {status_string(code)} ({code})")


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libl2a.so; raises if it is missing (there is no CPU or eager fallback)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} not built: run `python -m paper_2603_17484_b200.build`")
        L = ctypes.CDLL(LIB_PATH)
        L.l2a_version.restype = ctypes.c_char_p
        L.l2a_status_string.restype = ctypes.c_char_p
        L.l2a_status_string.argtypes = [ctypes.c_int]
        for name in EXPORTS[2:]:
            getattr(L, name).restype = ctypes.c_int
        _lib = L
    return _lib


def version() -> str:
    return lib().l2a_version().decode()


def status_string(code: int) -> str:
    return lib().l2a_status_string(code).decode()


def params(B, Lq, Lk, Hq, Hkv, D, window, q_pos_offset=None, softmax_scale=0.0, flags=0, q_stride=None,
           k_stride=None, v_stride=None, o_stride=None, seq_bounds=None) -> L2AParams:
    """Strides: optional (batch stride, token stride) in elements; None = dense (see include/l2a.h).
    seq_bounds: the int32 [Lq, 2] device table of l2a_pack_sequences for a packed variable-length batch (the caller
    keeps the tensor alive while the parameters are in use)."""
    two = ctypes.c_int64 * 2
    st = [two(*(s if s is not None else (0, 0))) for s in (q_stride, k_stride, v_stride, o_stride)]
    return L2AParams(B, Lq, Lk, Hq, Hkv, D, window, Lk - Lq if q_pos_offset is None else q_pos_offset,
                     softmax_scale, flags, *st, None if seq_bounds is None else seq_bounds.data_ptr())


def _ptr(t):
    if t is None:
        return ctypes.c_void_p(0)
    if isinstance(t, torch.Tensor):
        # strided views (slices of a fused buffer) are described by the strides in L2AParams; only the base
        # address is passed
        return ctypes.c_void_p(t.data_ptr())
    return ctypes.c_void_p(int(t))


def _stream(stream=None):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _check(code: int, where: str):
    if code != L2A_OK:
        raise L2AError(code, where)


def l2a_workspace_bytes(p: L2AParams) -> tuple[int, int, int]:
    r, f, b = ctypes.c_size_t(0), ctypes.c_size_t(0), ctypes.c_size_t(0)
    _check(lib().l2a_workspace_bytes(ctypes.byref(p), ctypes.byref(r), ctypes.byref(f), ctypes.byref(b)),
           "l2a_workspace_bytes")
    return r.value, f.value, b.value


def l2a_workspace_status(ws: torch.Tensor, stream=None) -> int:
    return lib().l2a_workspace_status(_ptr(ws), _stream(stream))


def l2a_selftest_wait_timeout(ws: torch.Tensor, limit_us: int, stream=None, check=True) -> int:
    """Runs the bounded-wait self-test kernel (a wait that nothing satisfies, limited to limit_us microseconds)."""
    code = lib().l2a_selftest_wait_timeout(_ptr(ws), ctypes.c_uint(limit_us), _stream(stream))
    if check:
        _check(code, "l2a_selftest_wait_timeout")
    return code


def l2a_route_compact(p, router, router_kind, logit_threshold, d_mask, q_idx, n_routed, prefix, route_ws,
                      stream=None, check=True) -> int:
    code = lib().l2a_route_compact(ctypes.byref(p), _ptr(router), ctypes.c_int(router_kind),
                                   ctypes.c_float(logit_threshold), _ptr(d_mask), _ptr(q_idx), _ptr(n_routed),
                                   _ptr(prefix), _ptr(route_ws),
                                   ctypes.c_size_t(route_ws.numel() * route_ws.element_size() if route_ws is not None else 0),
                                   _stream(stream))
    if check:
        _check(code, "l2a_route_compact")
    return code


def l2a_pack_sequences(cu_seqlens, Lq, seq_bounds=None, stream=None):
    """cu_seqlens: int32 device tensor [n_seq + 1]; returns the int32 [Lq, 2] table for `params(seq_bounds=...)`."""
    if seq_bounds is None:
        seq_bounds = torch.empty((Lq, 2), dtype=torch.int32, device=cu_seqlens.device)
    _check(lib().l2a_pack_sequences(_ptr(cu_seqlens), ctypes.c_int(cu_seqlens.numel() - 1), ctypes.c_int(Lq),
                                    _ptr(seq_bounds), _stream(stream)), "l2a_pack_sequences")
    return seq_bounds


def l2a_route_compact_static(p, router, router_kind, logit_threshold, d_mask, q_idx, n_routed, prefix, stream=None,
                             check=True) -> int:
    """Routing + compaction with the scratch held in the library's own fixed device array: for callers that
    cannot hand over (or allocate) a workspace.  Limits and sharing rules are in include/l2a.h."""
    code = lib().l2a_route_compact_static(ctypes.byref(p), _ptr(router), ctypes.c_int(router_kind),
                                          ctypes.c_float(logit_threshold), _ptr(d_mask), _ptr(q_idx),
                                          _ptr(n_routed), _ptr(prefix), _stream(stream))
    if check:
        _check(code, "l2a_route_compact_static")
    return code


def l2a_decode_workspace_bytes(p) -> int:
    n = ctypes.c_size_t(0)
    _check(lib().l2a_decode_workspace_bytes(ctypes.byref(p), ctypes.byref(n)), "l2a_decode_workspace_bytes")
    return n.value


def l2a_decode(p, q, K, V, d, O, ws, stream=None, check=True) -> int:
    """Decode step: one new token per sequence against the K/V cache (local window always, whole cache if d = 1)."""
    code = lib().l2a_decode(ctypes.byref(p), _ptr(q), _ptr(K), _ptr(V), _ptr(d), _ptr(O), _ptr(ws),
                            ctypes.c_size_t(ws.numel() if ws is not None else 0), _stream(stream))
    if check:
        _check(code, "l2a_decode")
    return code


def l2a_router_logits(p, S, w, bias, logits, sum_sq=None, stream=None, check=True) -> int:
    """Router logits z_t = w . s_t + bias from the local output (Eq. 3); optional sum of sigmoid(z)^2 per batch entry."""
    code = lib().l2a_router_logits(ctypes.byref(p), _ptr(S), _ptr(w), ctypes.c_float(bias), _ptr(logits), _ptr(sum_sq),
                                   _stream(stream))
    if check:
        _check(code, "l2a_router_logits")
    return code


def l2a_forward(p, Q, K, V, d_mask, q_idx, n_routed, prefix, O, S_save, A_c, lse_loc, lse_glb, fwd_ws,
                stream=None, check=True) -> int:
    code = lib().l2a_forward(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(d_mask), _ptr(q_idx), _ptr(n_routed),
                             _ptr(prefix), _ptr(O), _ptr(S_save), _ptr(A_c), _ptr(lse_loc), _ptr(lse_glb),
                             _ptr(fwd_ws),
                             ctypes.c_size_t(fwd_ws.numel() * fwd_ws.element_size() if fwd_ws is not None else 0),
                             _stream(stream))
    if check:
        _check(code, "l2a_forward")
    return code


def l2a_backward(p, Q, K, V, d_mask, q_idx, n_routed, prefix, dO, S_save, A_c, lse_loc, lse_glb, dQ, dK, dV,
                 dgate, bwd_ws, stream=None, check=True) -> int:
    code = lib().l2a_backward(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(d_mask), _ptr(q_idx),
                              _ptr(n_routed), _ptr(prefix), _ptr(dO), _ptr(S_save), _ptr(A_c), _ptr(lse_loc),
                              _ptr(lse_glb), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(dgate), _ptr(bwd_ws),
                              ctypes.c_size_t(bwd_ws.numel() * bwd_ws.element_size() if bwd_ws is not None else 0),
                              _stream(stream))
    if check:
        _check(code, "l2a_backward")
    return code


def _nbytes(t):
    return ctypes.c_size_t(t.numel() * t.element_size() if t is not None else 0)


def l2a_forward_sets(p, Q, K, V, Qg, Kg, Vg, d_mask, q_idx, n_routed, prefix, O, S_save, A_c, lse_loc, lse_glb, fwd_ws,
                     stream=None, check=True) -> int:
    """l2a_forward with a second Q/K/V set for the Global Attention module (None, None, None = one set)."""
    code = lib().l2a_forward_sets(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(Qg), _ptr(Kg), _ptr(Vg), _ptr(d_mask),
                                  _ptr(q_idx), _ptr(n_routed), _ptr(prefix), _ptr(O), _ptr(S_save), _ptr(A_c),
                                  _ptr(lse_loc), _ptr(lse_glb), _ptr(fwd_ws), _nbytes(fwd_ws), _stream(stream))
    if check:
        _check(code, "l2a_forward_sets")
    return code


def l2a_backward_sets(p, Q, K, V, Qg, Kg, Vg, d_mask, q_idx, n_routed, prefix, dO, S_save, A_c, lse_loc, lse_glb, dQ, dK,
                      dV, dQg, dKg, dVg, dgate, bwd_ws, stream=None, check=True) -> int:
    """l2a_backward with a second Q/K/V set: gradients of the local module's set and of the global module's set."""
    code = lib().l2a_backward_sets(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(Qg), _ptr(Kg), _ptr(Vg),
                                   _ptr(d_mask), _ptr(q_idx), _ptr(n_routed), _ptr(prefix), _ptr(dO), _ptr(S_save),
                                   _ptr(A_c), _ptr(lse_loc), _ptr(lse_glb), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(dQg),
                                   _ptr(dKg), _ptr(dVg), _ptr(dgate), _ptr(bwd_ws), _nbytes(bwd_ws), _stream(stream))
    if check:
        _check(code, "l2a_backward_sets")
    return code


def l2a_backward_split(p, Q, K, V, d_mask, q_idx, n_routed, prefix, dO, dS_loc, S_save, A_c, lse_loc, lse_glb, dQ,
                       dK, dV, dgate, bwd_ws, stream=None, check=True) -> int:
    """l2a_backward with a separate gradient dS_loc for the local output (dO + the router path)."""
    code = lib().l2a_backward_split(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(d_mask), _ptr(q_idx),
                                    _ptr(n_routed), _ptr(prefix), _ptr(dO), _ptr(dS_loc), _ptr(S_save), _ptr(A_c),
                                    _ptr(lse_loc), _ptr(lse_glb), _ptr(dQ), _ptr(dK), _ptr(dV), _ptr(dgate),
                                    _ptr(bwd_ws),
                                    ctypes.c_size_t(bwd_ws.numel() * bwd_ws.element_size() if bwd_ws is not None else 0),
                                    _stream(stream))
    if check:
        _check(code, "l2a_backward_split")
    return code


def l2a_router_backward(p, S, w, logits, dgate, reg_coeff, dO=None, dz=None, dw=None, dbias=None, dS_loc=None,
                        stream=None, check=True) -> int:
    """Router backward (Eq. 7 + regulariser gradient): dz, dw, dbias and dS_loc = dO + dz * w."""
    code = lib().l2a_router_backward(ctypes.byref(p), _ptr(S), _ptr(w), _ptr(logits), _ptr(dgate),
                                     ctypes.c_float(reg_coeff), _ptr(dO), _ptr(dz), _ptr(dw), _ptr(dbias),
                                     _ptr(dS_loc), _stream(stream))
    if check:
        _check(code, "l2a_router_backward")
    return code


def l2a_forward_routed(p, Q, K, V, router_w, router_bias, logit_threshold, logits, sum_sq, d_mask, q_idx, n_routed,
                       prefix, O, S_save, A_c, lse_loc, lse_glb, route_ws, fwd_ws, stream=None, check=True) -> int:
    """Layer forward in its defining order in one call: local -> router -> route/compact -> global (Eq. 2-5)."""
    nbytes = lambda t: ctypes.c_size_t(t.numel() * t.element_size() if t is not None else 0)
    code = lib().l2a_forward_routed(ctypes.byref(p), _ptr(Q), _ptr(K), _ptr(V), _ptr(router_w),
                                    ctypes.c_float(router_bias), ctypes.c_float(logit_threshold), _ptr(logits),
                                    _ptr(sum_sq), _ptr(d_mask), _ptr(q_idx), _ptr(n_routed), _ptr(prefix), _ptr(O),
                                    _ptr(S_save), _ptr(A_c), _ptr(lse_loc), _ptr(lse_glb), _ptr(route_ws),
                                    nbytes(route_ws), _ptr(fwd_ws), nbytes(fwd_ws), _stream(stream))
    if check:
        _check(code, "l2a_forward_routed")
    return code


class HostIO(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("Q", "K", "V", "router", "dO", "O", "dQ", "dK", "dV")]


class DeviceIO(ctypes.Structure):
    _fields_ = [(n, ctypes.c_void_p) for n in ("Q", "K", "V", "router", "dO", "d_mask", "q_idx", "n_routed", "prefix",
                                                "O", "S_save", "A_c", "lse_loc", "lse_glb", "dQ", "dK", "dV")] + [
        ("route_ws", ctypes.c_void_p), ("route_ws_bytes", ctypes.c_size_t),
        ("fwd_ws", ctypes.c_void_p), ("fwd_ws_bytes", ctypes.c_size_t),
        ("bwd_ws", ctypes.c_void_p), ("bwd_ws_bytes", ctypes.c_size_t)]


def _addr(t):
    return None if t is None else (t.data_ptr() if isinstance(t, torch.Tensor) else int(t))


def l2a_step_host(p, host: dict, bufs: "Buffers", router_kind=ROUTER_MASK_U8, logit_threshold=0.0, stream=None,
                  check=True, pipelined=False) -> int:
    """Whole step from HOST tensors (dict with Q, K, V, router, O and, for a backward, dO, dQ, dK, dV):
    copies in, routes, runs forward (+ backward), copies the results out, synchronises."""
    h = HostIO(*[_addr(host.get(n)) for n in ("Q", "K", "V", "router", "dO", "O", "dQ", "dK", "dV")])
    names = ("Q", "K", "V", "router", "dO", "d_mask", "q_idx", "n_routed", "prefix", "O", "S_save", "A_c",
             "lse_loc", "lse_glb", "dQ", "dK", "dV")
    d = DeviceIO(*[_addr(getattr(bufs, n)) for n in names],
                 _addr(bufs.route_ws), bufs.route_ws.numel(), _addr(bufs.fwd_ws), bufs.fwd_ws.numel(),
                 _addr(bufs.bwd_ws), 0 if bufs.bwd_ws is None else bufs.bwd_ws.numel())
    fn = lib().l2a_step_host_async if pipelined else lib().l2a_step_host
    code = fn(ctypes.byref(p), ctypes.byref(h), ctypes.byref(d), ctypes.c_int(router_kind),
              ctypes.c_float(logit_threshold), _stream(stream))
    if check:
        _check(code, "l2a_step_host_async" if pipelined else "l2a_step_host")
    return code


def l2a_step_host_async(p, host: dict, bufs: "Buffers", router_kind=ROUTER_MASK_U8, logit_threshold=0.0, stream=None,
                        check=True) -> int:
    """The same step, enqueued only (two steps in flight on alternating Buffers; see include/l2a.h)."""
    return l2a_step_host(p, host, bufs, router_kind, logit_threshold, stream, check, pipelined=True)


def l2a_step_host_wait(stream=None) -> int:
    code = lib().l2a_step_host_wait(_stream(stream))
    _check(code, "l2a_step_host_wait")
    return code


def l2a_profile_next_call(events) -> int:
    """events: sequence of raw cudaEvent_t handles (ints); see include/l2a.h for the phase boundaries."""
    arr = (ctypes.c_void_p * len(events))(*[ctypes.c_void_p(int(e)) for e in events])
    code = lib().l2a_profile_next_call(arr, ctypes.c_int(len(events)))
    _check(code, "l2a_profile_next_call")
    return code


@dataclass
class Buffers:
    """Device buffers for one shape (allocation helper for tests and benchmarks; torch owns the memory)."""
    p: L2AParams
    Q: torch.Tensor = None
    K: torch.Tensor = None
    V: torch.Tensor = None
    router: torch.Tensor = None
    d_mask: torch.Tensor = None
    q_idx: torch.Tensor = None
    n_routed: torch.Tensor = None
    prefix: torch.Tensor = None
    O: torch.Tensor = None
    S_save: torch.Tensor = None
    A_c: torch.Tensor = None
    lse_loc: torch.Tensor = None
    lse_glb: torch.Tensor = None
    dO: torch.Tensor = None
    dQ: torch.Tensor = None
    dK: torch.Tensor = None
    dV: torch.Tensor = None
    dgate: torch.Tensor = None
    route_ws: torch.Tensor = None
    fwd_ws: torch.Tensor = None
    bwd_ws: torch.Tensor = None

    GUARD_BYTES = 4096
    GUARD_BYTE = 0xA5

    @staticmethod
    def allocate(p: L2AParams, backward: bool = False, device="cuda", router_dtype=torch.uint8,
                 guard: bool = False) -> "Buffers":
        """guard: every tensor sits between two 4 KB regions filled with a byte pattern; check_guards() tells whether a
        kernel wrote outside a buffer (the stand-in for a memory checker in the GPU tests)."""
        B, Lq, Lk, Hq, Hkv, D = p.B, p.Lq, p.Lk, p.Hq, p.Hkv, p.D
        bf, dev = torch.bfloat16, device
        r, f, w = l2a_workspace_bytes(p)
        b = Buffers(p)
        b._raw = []
        G = Buffers.GUARD_BYTES

        def new(shape, dtype):
            if not guard:
                return torch.empty(shape, dtype=dtype, device=dev)
            n = 1
            for x in shape:
                n *= x
            nbytes = n * torch.empty((), dtype=dtype).element_size()
            pad = (-nbytes) % 256                                  # the back guard starts right after the last byte
            raw = torch.full((G + nbytes + pad + G,), Buffers.GUARD_BYTE, dtype=torch.uint8, device=dev)
            b._raw.append((raw, nbytes))
            return raw[G:G + nbytes].view(dtype).view(shape)

        b.Q = new((B, Lq, Hq, D), bf)
        b.K = new((B, Lk, Hkv, D), bf)
        b.V = new((B, Lk, Hkv, D), bf)
        b.router = new((B, Lq), router_dtype)
        b.d_mask = new((B, Lq), torch.uint8)
        b.q_idx = new((B, Lq), torch.int32)
        b.n_routed = new((B,), torch.int32)
        b.prefix = new((B, Lq + 1), torch.int32)
        b.O = new((B, Lq, Hq, D), bf)
        b.route_ws = new((r,), torch.uint8)
        b.fwd_ws = new((f,), torch.uint8)
        if backward:
            b.S_save = new((B, Lq, Hq, D), bf)
            b.A_c = new((B, Lq, Hq, D), bf)
            b.lse_loc = new((B, Hq, Lq), torch.float32)
            b.lse_glb = new((B, Hq, Lq), torch.float32)
            b.dO = new((B, Lq, Hq, D), bf)
            b.dQ = new((B, Lq, Hq, D), bf)
            b.dK = new((B, Lk, Hkv, D), bf)
            b.dV = new((B, Lk, Hkv, D), bf)
            b.dgate = new((B, Lq), torch.float32)
            b.bwd_ws = new((w,), torch.uint8)
        return b

    def check_guards(self) -> bool:
        """True if no guard byte around any buffer changed (always True without guard=True)."""
        G = Buffers.GUARD_BYTES
        for raw, nbytes in getattr(self, "_raw", []):
            if not bool((raw[:G] == Buffers.GUARD_BYTE).all()) or not bool((raw[G + nbytes:] == Buffers.GUARD_BYTE).all()):
                return False
        return True

    def route(self, router_kind=ROUTER_MASK_U8, threshold=0.0, stream=None):
        return l2a_route_compact(self.p, self.router, router_kind, threshold, self.d_mask, self.q_idx,
                                 self.n_routed, self.prefix, self.route_ws, stream)

    def forward(self, stream=None):
        return l2a_forward(self.p, self.Q, self.K, self.V, self.d_mask, self.q_idx, self.n_routed, self.prefix,
                           self.O, self.S_save, self.A_c, self.lse_loc, self.lse_glb, self.fwd_ws, stream)

    def backward(self, stream=None, with_dgate=False):
        return l2a_backward(self.p, self.Q, self.K, self.V, self.d_mask, self.q_idx, self.n_routed, self.prefix,
                            self.dO, self.S_save, self.A_c, self.lse_loc, self.lse_glb, self.dQ, self.dK, self.dV,
                            self.dgate if with_dgate else None, self.bwd_ws, stream)
