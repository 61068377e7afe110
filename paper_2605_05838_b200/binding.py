"""Thin Python binding of libmdn (argument marshalling only).

Every step of the path runs in the CUDA kernels behind the C ABI declared in
include/mdn.h; this module turns torch tensors into pointers and sizes.  There is
no CPU fallback: if the library is missing or was not built, importing the symbols
raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Tuple

import torch

_PKG = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_PKG, "libmdn.so")

MDN_F32, MDN_BF16 = 0, 1
PATH_AUTO, PATH_SIMT, PATH_TENSOR = 0, 1, 2
_PATHS = {"auto": PATH_AUTO, "simt": PATH_SIMT, "tensor": PATH_TENSOR}
PATH_NAMES = {PATH_AUTO: "auto", PATH_SIMT: "simt", PATH_TENSOR: "tensor"}
NUM_COEF = 12
CHUNK = 64
NUM_STAGE_EVENTS = 4
STAGE_NAMES = ["coeff_scan", "intra_chunk", "chain"]


class MdnParams(ctypes.Structure):
    _fields_ = [("B", ctypes.c_int32), ("T", ctypes.c_int32), ("H", ctypes.c_int32),
                ("dk", ctypes.c_int32), ("dv", ctypes.c_int32), ("chunk", ctypes.c_int32),
                ("num_seqs", ctypes.c_int32), ("io_dtype", ctypes.c_int32), ("o_dtype", ctypes.c_int32),
                ("path", ctypes.c_int32), ("scale", ctypes.c_float), ("segments", ctypes.c_int32)]


class MdnWsLayout(ctypes.Structure):
    _fields_ = [("num_slots", ctypes.c_int32), ("mat_dtype", ctypes.c_int32),
                ("off_status", ctypes.c_uint64), ("off_chunk_off", ctypes.c_uint64),
                ("off_slot_map", ctypes.c_uint64), ("off_coef", ctypes.c_uint64),
                ("off_T", ctypes.c_uint64), ("off_W", ctypes.c_uint64), ("total_bytes", ctypes.c_uint64),
                ("off_seg", ctypes.c_uint64), ("segments", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class MdnLayerOps(ctypes.Structure):
    """mdn_layer_ops of include/mdn.h (Section 3.3 element-wise operations absorbed by the forward)."""
    _fields_ = [("raw_gates", ctypes.c_int32),
                ("decay_a_alpha", ctypes.c_void_p), ("decay_b_alpha", ctypes.c_void_p),
                ("decay_a_mu", ctypes.c_void_p), ("decay_b_mu", ctypes.c_void_p),
                ("s", ctypes.c_float), ("tau", ctypes.c_float), ("log_mu_min", ctypes.c_float),
                ("qk_norm", ctypes.c_int32), ("d", ctypes.c_void_p), ("qk_eps", ctypes.c_float),
                ("out_norm_gate", ctypes.c_int32), ("g", ctypes.c_void_p), ("w", ctypes.c_void_p),
                ("rms_eps", ctypes.c_float), ("placement", ctypes.c_int32)]


class MdnError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        detail = ""
        if status == 4:
            detail = ": " + lib().mdn_last_cuda_error_string().decode()
        super().__init__("%s: %s (status %d)%s" % (where, status_string(status), status, detail))


_lib = None


def lib() -> ctypes.CDLL:
    """Loads libmdn.so (built in-tree by paper_2605_05838_b200.build); raises if absent."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError("libmdn.so not found at %s: run `python -m paper_2605_05838_b200.build`" % LIB_PATH)
        L = ctypes.CDLL(LIB_PATH)
        vp, P = ctypes.c_void_p, ctypes.POINTER(MdnParams)
        L.mdn_chunk_fwd_workspace_bytes.restype = ctypes.c_size_t
        L.mdn_chunk_fwd_workspace_bytes.argtypes = [P]
        L.mdn_chunk_fwd_host_arena_bytes.restype = ctypes.c_size_t
        L.mdn_chunk_fwd_host_arena_bytes.argtypes = [P]
        L.mdn_chunk_fwd.restype = ctypes.c_int
        L.mdn_chunk_fwd.argtypes = [P] + [vp] * 13 + [vp, ctypes.c_size_t, vp]
        L.mdn_chunk_fwd_fused.restype = ctypes.c_int
        L.mdn_chunk_fwd_fused.argtypes = [P, ctypes.POINTER(MdnLayerOps)] + [vp] * 13 + [vp, ctypes.c_size_t, vp]
        L.mdn_chunk_fwd_fused_workspace_bytes.restype = ctypes.c_size_t
        L.mdn_chunk_fwd_fused_workspace_bytes.argtypes = [P, ctypes.POINTER(MdnLayerOps)]
        L.mdn_chunk_states_bytes.restype = ctypes.c_size_t
        L.mdn_chunk_states_bytes.argtypes = [P]
        L.mdn_chunk_fwd_keep_states.restype = ctypes.c_int
        L.mdn_chunk_fwd_keep_states.argtypes = [P] + [vp] * 14 + [vp, ctypes.c_size_t, vp]
        L.mdn_bwd_state_chain_workspace_bytes.restype = ctypes.c_size_t
        L.mdn_bwd_state_chain_workspace_bytes.argtypes = [P]
        L.mdn_bwd_adjoint_states_bytes.restype = ctypes.c_size_t
        L.mdn_bwd_adjoint_states_bytes.argtypes = [P]
        L.mdn_bwd_state_chain.restype = ctypes.c_int
        L.mdn_bwd_state_chain.argtypes = [P] + [vp] * 7 + [ctypes.c_size_t] + [vp] * 4 + [ctypes.c_size_t, vp]
        L.mdn_chunk_bwd_chunked_workspace_bytes.restype = ctypes.c_size_t
        L.mdn_chunk_bwd_chunked_workspace_bytes.argtypes = [P]
        L.mdn_chunk_bwd_chunked.restype = ctypes.c_int
        L.mdn_chunk_bwd_chunked.argtypes = [P] + [vp] * 22 + [vp, ctypes.c_size_t, vp]
        L.mdn_chunk_bwd_saved_workspace_bytes.restype = ctypes.c_size_t
        L.mdn_chunk_bwd_saved_workspace_bytes.argtypes = [P]
        L.mdn_chunk_bwd_saved.restype = ctypes.c_int
        L.mdn_chunk_bwd_saved.argtypes = [P] + [vp] * 9 + [ctypes.c_size_t] + [vp] * 13 + [vp, ctypes.c_size_t, vp]
        L.mdn_chunk_bwd.restype = ctypes.c_int
        L.mdn_chunk_bwd.argtypes = [P] + [vp] * 22 + [vp, ctypes.c_size_t, vp]
        L.mdn_chunk_bwd_workspace_bytes.restype = ctypes.c_size_t
        L.mdn_chunk_bwd_workspace_bytes.argtypes = [P]
        L.mdn_chunk_fwd_host.restype = ctypes.c_int
        L.mdn_chunk_fwd_host.argtypes = [P] + [vp] * 13 + [vp, ctypes.c_size_t, vp]
        L.mdn_chunk_fwd_static_scratch.restype = ctypes.c_int
        L.mdn_chunk_fwd_static_scratch.argtypes = [P] + [vp] * 13 + [vp]
        L.mdn_decode_step.restype = ctypes.c_int
        L.mdn_decode_step.argtypes = [P] + [vp] * 10 + [vp]
        L.mdn_decode_step_fused.restype = ctypes.c_int
        L.mdn_decode_step_fused.argtypes = [P, ctypes.POINTER(MdnLayerOps)] + [vp] * 10 + [vp]
        L.mdn_workspace_layout.restype = ctypes.c_int
        L.mdn_workspace_layout.argtypes = [P, ctypes.POINTER(MdnWsLayout)]
        L.mdn_coeff_scan.restype = ctypes.c_int
        L.mdn_coeff_scan.argtypes = [P] + [vp] * 5 + [vp, ctypes.c_size_t, vp]
        L.mdn_intra_chunk.restype = ctypes.c_int
        L.mdn_intra_chunk.argtypes = [P] + [vp] * 3 + [vp, ctypes.c_size_t, vp]
        L.mdn_read_status.restype = ctypes.c_int
        L.mdn_read_status.argtypes = [P, vp, vp]
        L.mdn_status_string.restype = ctypes.c_char_p
        L.mdn_status_string.argtypes = [ctypes.c_int]
        L.mdn_set_stage_events.restype = ctypes.c_int
        L.mdn_set_stage_events.argtypes = [ctypes.POINTER(vp), ctypes.c_int32]
        L.mdn_last_cuda_error_string.restype = ctypes.c_char_p
        L.mdn_last_cuda_error_string.argtypes = []
        L.mdn_last_launch_count.restype = ctypes.c_int32
        L.mdn_last_launch_count.argtypes = []
        _lib = L
    return _lib


def status_string(status: int) -> str:
    return lib().mdn_status_string(int(status)).decode()


def last_launch_count() -> int:
    return int(lib().mdn_last_launch_count())


def set_stage_events(events) -> None:
    """events: NUM_STAGE_EVENTS torch.cuda.Event(enable_timing=True), or None to clear the hooks."""
    if events is None:
        st = lib().mdn_set_stage_events(None, 0)
    else:
        for e in events:
            if not e.cuda_event:      # torch creates the handle lazily, on the first record
                e.record()
        arr = (ctypes.c_void_p * len(events))(*[ctypes.c_void_p(e.cuda_event) for e in events])
        st = lib().mdn_set_stage_events(arr, len(events))
    if st != 0:
        raise MdnError(st, "mdn_set_stage_events")


def resolved_path(p: "MdnParams") -> str:
    """Which chain kernels a call with these parameters runs ("simt" or "tensor")."""
    lay = workspace_layout(p)
    return "tensor" if lay.mat_dtype == MDN_BF16 else "simt"


def _dtype_code(dt: torch.dtype) -> int:
    if dt == torch.float32:
        return MDN_F32
    if dt == torch.bfloat16:
        return MDN_BF16
    raise TypeError("q, k, v, o must be float32 or bfloat16, got %s" % dt)


def _ptr(t: Optional[torch.Tensor]):
    return None if t is None else ctypes.c_void_p(t.data_ptr())


def _stream() -> ctypes.c_void_p:
    return ctypes.c_void_p(torch.cuda.current_stream().cuda_stream)


def make_params(q: torch.Tensor, v: torch.Tensor, *, num_seqs: int = 0, scale: Optional[float] = None,
                o_dtype: Optional[torch.dtype] = None, path: str = "auto", segments: int = 0) -> MdnParams:
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    return MdnParams(B, T, H, dk, dv, CHUNK, int(num_seqs), _dtype_code(q.dtype),
                     _dtype_code(o_dtype or q.dtype), _PATHS[path],
                     float(dk) ** -0.5 if scale is None else float(scale), int(segments))


def workspace_bytes(p: MdnParams) -> int:
    return int(lib().mdn_chunk_fwd_workspace_bytes(ctypes.byref(p)))


def host_arena_bytes(p: MdnParams) -> int:
    return int(lib().mdn_chunk_fwd_host_arena_bytes(ctypes.byref(p)))


def workspace_layout(p: MdnParams) -> MdnWsLayout:
    lay = MdnWsLayout()
    st = lib().mdn_workspace_layout(ctypes.byref(p), ctypes.byref(lay))
    if st != 0:
        raise MdnError(st, "mdn_workspace_layout")
    return lay


def _f32_vec(name, t, n):
    if t is None:
        return None
    if t.device.type != "cuda" or t.dtype != torch.float32 or not t.is_contiguous() or t.numel() != n:
        raise ValueError("%s must be a contiguous float32 cuda tensor of %d elements" % (name, n))
    return ctypes.c_void_p(t.data_ptr())


def make_layer_ops(q, v, *, gate_param=None, qk_norm=None, out_norm_gate=None, placement="fused"):
    """Builds mdn_layer_ops from tensors (marshalling only; keep the tensors alive until the call returns).
      gate_param    = dict(a_alpha, b_alpha, a_mu, b_mu: float32 [H]; s, tau: float; log_mu_min=-1.0): the gate
                      arguments of the call are then the raw projections x_beta, x_alpha, x_mu, x_eta
      qk_norm       = dict(d: float32 [H] or None, eps: float)
      out_norm_gate = dict(g: [B,T,H,dv] in q's dtype, w: float32 [dv] or None, eps: float)
      placement     = "fused" (inside the forward's kernels) or "separate" (kernels of their own)"""
    H, dv = q.shape[2], v.shape[-1]
    ops = MdnLayerOps()
    if gate_param is not None:
        ops.raw_gates = 1
        ops.decay_a_alpha = _f32_vec("a_alpha", gate_param["a_alpha"], H)
        ops.decay_b_alpha = _f32_vec("b_alpha", gate_param["b_alpha"], H)
        ops.decay_a_mu = _f32_vec("a_mu", gate_param["a_mu"], H)
        ops.decay_b_mu = _f32_vec("b_mu", gate_param["b_mu"], H)
        ops.s, ops.tau = float(gate_param["s"]), float(gate_param["tau"])
        ops.log_mu_min = float(gate_param.get("log_mu_min", -1.0))
    if qk_norm is not None:
        ops.qk_norm = 1
        ops.d = _f32_vec("d", qk_norm.get("d"), H)
        ops.qk_eps = float(qk_norm["eps"])
    if out_norm_gate is not None:
        g = out_norm_gate["g"]
        if g.device.type != "cuda" or g.dtype != q.dtype or not g.is_contiguous() or tuple(g.shape) != tuple(v.shape):
            raise ValueError("g must be a contiguous cuda tensor with v's shape and dtype")
        ops.out_norm_gate = 1
        ops.g = ctypes.c_void_p(g.data_ptr())
        ops.w = _f32_vec("w", out_norm_gate.get("w"), dv)
        ops.rms_eps = float(out_norm_gate["eps"])
    ops.placement = {"fused": 0, "separate": 1}[placement]
    return ops


def _check_inputs(q, k, v, gates, device_type: str):
    for name, t in (("q", q), ("k", k), ("v", v)):
        if t.device.type != device_type or not t.is_contiguous() or t.dim() != 4:
            raise ValueError("%s must be a contiguous 4-d %s tensor" % (name, device_type))
    if q.shape != k.shape or q.shape[:3] != v.shape[:3] or q.dtype != k.dtype or q.dtype != v.dtype:
        raise ValueError("q, k, v shapes/dtypes disagree")
    for name, t in gates:
        if t is None:
            continue
        if t.device.type != device_type or not t.is_contiguous() or t.dtype != torch.float32 \
                or tuple(t.shape) != tuple(q.shape[:3]):
            raise ValueError("%s must be a contiguous float32 [B,T,H] %s tensor" % (name, device_type))


def _check_state(name, t, shape, device_type):
    if t is None:
        return
    if t.device.type != device_type or not t.is_contiguous() or t.dtype != torch.float32 or tuple(t.shape) != shape:
        raise ValueError("%s must be a contiguous float32 %s tensor of shape %s" % (name, device_type, shape))


def chunk_fwd(q, k, v, beta, log_alpha, log_mu, eta=None, *, initial_S=None, initial_M=None,
              cu_seqlens=None, scale: Optional[float] = None, o_dtype: Optional[torch.dtype] = None,
              path: str = "auto", output_final_state: bool = True, workspace: Optional[torch.Tensor] = None,
              out: Optional[torch.Tensor] = None, segments: int = 0, layer_ops: Optional[MdnLayerOps] = None,
              keep_chunk_states: bool = False):
    """mdn_chunk_fwd (mdn_chunk_fwd_fused when layer_ops is given) on CUDA tensors, current stream.
    Returns (o, final_S, final_M).
    segments: 0 = automatic, 1 = plain serial chain, >= 3 = force the parallel inter-chunk scan.
    layer_ops: from make_layer_ops; with its gate_param set, beta / log_alpha / log_mu / eta are the raw
    projections x_beta / x_alpha / x_mu / x_eta.
    keep_chunk_states: mdn_chunk_fwd_keep_states; returns (o, final_S, final_M, chunk_states, workspace) where
    chunk_states is the raw uint8 buffer (unpack_chunk_states turns it into float tensors)."""
    _check_inputs(q, k, v, (("beta", beta), ("log_alpha", log_alpha), ("log_mu", log_mu), ("eta", eta)), "cuda")
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    N = 0
    if cu_seqlens is not None:
        if cu_seqlens.device.type != "cuda" or cu_seqlens.dtype != torch.int32 or not cu_seqlens.is_contiguous():
            raise ValueError("cu_seqlens must be a contiguous int32 cuda tensor")
        N = cu_seqlens.numel() - 1
    p = make_params(q, v, num_seqs=N, scale=scale, o_dtype=o_dtype, path=path, segments=segments)
    nst = N if N > 0 else B
    _check_state("initial_S", initial_S, (nst, H, dk, dv), "cuda")
    _check_state("initial_M", initial_M, (nst, H, dk, dv), "cuda")
    if layer_ops is None:
        need = workspace_bytes(p)
    else:
        need = int(lib().mdn_chunk_fwd_fused_workspace_bytes(ctypes.byref(p), ctypes.byref(layer_ops)))
    if need == 0:
        raise MdnError(2, "mdn_chunk_fwd_workspace_bytes")
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    o = out if out is not None else torch.empty((B, T, H, dv), dtype=o_dtype or q.dtype, device=q.device)
    Sf = Mf = None
    if output_final_state:
        Sf = torch.empty((nst, H, dk, dv), dtype=torch.float32, device=q.device)
        Mf = torch.empty((nst, H, dk, dv), dtype=torch.float32, device=q.device)
    tail = (_ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(log_alpha), _ptr(log_mu), _ptr(eta), _ptr(initial_S),
            _ptr(initial_M), _ptr(cu_seqlens), _ptr(o), _ptr(Sf), _ptr(Mf), _ptr(workspace), workspace.numel(),
            _stream())
    if keep_chunk_states:
        if layer_ops is not None:
            raise ValueError("keep_chunk_states and layer_ops exclude each other")
        nbytes = int(lib().mdn_chunk_states_bytes(ctypes.byref(p)))
        if nbytes == 0:
            raise MdnError(2, "mdn_chunk_states_bytes")
        states = torch.empty(nbytes, dtype=torch.uint8, device=q.device)
        st = lib().mdn_chunk_fwd_keep_states(ctypes.byref(p), *tail[:13], _ptr(states), *tail[13:])
        if st != 0:
            raise MdnError(st, "mdn_chunk_fwd_keep_states")
        return o, Sf, Mf, states, workspace
    if layer_ops is None:
        st = lib().mdn_chunk_fwd(ctypes.byref(p), *tail)
    else:
        st = lib().mdn_chunk_fwd_fused(ctypes.byref(p), ctypes.byref(layer_ops), *tail)
    if st != 0:
        raise MdnError(st, "mdn_chunk_fwd_fused" if layer_ops is not None else "mdn_chunk_fwd")
    return o, Sf, Mf


_IMAGE_BYTES, _VT_BYTES = 65536, 64 * 128 * 4


def _states_parts(states: torch.Tensor, H: int):
    """(state images, V~ part, slots) of a kept-states buffer: per (slot, head) a 64 KB state image, and behind all
    images one fp32 [64, H, 128] block per slot."""
    nbytes = states.numel()
    slots = nbytes // (H * (_IMAGE_BYTES + _VT_BYTES))
    if slots * H * (_IMAGE_BYTES + _VT_BYTES) != nbytes:
        raise ValueError("not a kept-states buffer for H = %d" % H)
    cut = slots * H * _IMAGE_BYTES
    return states[:cut], states[cut:], slots


def unpack_chunk_states(states: torch.Tensor, H: int):
    """The state images of a mdn_chunk_fwd_keep_states (or mdn_bwd_state_chain) buffer as float32 tensors (S, M) of
    shape [slots, H, dk, dv] (dk = dv = 128): undoes the transposition and the 128-byte swizzle of the shared-memory
    image."""
    images, _, _ = _states_parts(states, H)
    raw = images.view(torch.bfloat16).view(-1, H, 2, 2, 128, 8, 8)          # slot, head, S|M, key half, row, piece, elem
    rows = torch.arange(128, device=states.device)
    piece = torch.arange(8, device=states.device)
    src = (piece[None, :] ^ (rows[:, None] & 7))                            # where logical piece c of row r lies
    idx = src[None, None, None, None, :, :, None].expand(raw.shape[0], H, 2, 2, 128, 8, 8)
    logical = torch.gather(raw, 5, idx).reshape(-1, H, 2, 2, 128, 64)       # [.., row = value index, 64 key indices]
    full = torch.cat([logical[:, :, :, 0], logical[:, :, :, 1]], dim=-1)    # [slot, H, 2, value, key]
    full = full.transpose(-1, -2).float()                                   # [slot, H, 2, key, value]
    return full[:, :, 0].contiguous(), full[:, :, 1].contiguous()


def unpack_chunk_vt(states: torch.Tensor, H: int):
    """The second part of a kept-states buffer: V~ of every chunk slot as float32 [slots, 64, H, 128] (rows past a
    short chunk's end are unwritten); for the adjoint chain's buffer, dR = T^T dV~ in the chain's mirrored order."""
    _, vt, _ = _states_parts(states, H)
    return vt.view(torch.float32).view(-1, 64, H, 128)


def bwd_state_chain(q, k, d_o, fwd_workspace, *, v_dim: int, d_final_S=None, d_final_M=None, cu_seqlens=None,
                    scale: Optional[float] = None, want_initial: bool = True):
    """mdn_bwd_state_chain after a chunk_fwd(..., keep_chunk_states=True) call whose workspace is `fwd_workspace`.
    Returns (adjoint_states, d_initial_S, d_initial_M): the raw adjoint-state buffer (one entry per chunk, a
    sequence's chunks in reverse order, see include/mdn.h; unpack_chunk_states gives (dM, dS) per entry) and the
    initial states' gradients."""
    B, T, H, dk = q.shape
    N = 0 if cu_seqlens is None else cu_seqlens.numel() - 1
    nst = N if N > 0 else B
    p = make_params(q, d_o, num_seqs=N, scale=scale, o_dtype=torch.bfloat16, path="tensor")
    nbytes = int(lib().mdn_bwd_adjoint_states_bytes(ctypes.byref(p)))
    need = int(lib().mdn_bwd_state_chain_workspace_bytes(ctypes.byref(p)))
    if nbytes == 0 or need == 0:
        raise MdnError(2, "mdn_bwd_state_chain_workspace_bytes")
    adj = torch.empty(nbytes, dtype=torch.uint8, device=q.device)
    ws = torch.empty(need, dtype=torch.uint8, device=q.device)
    dS0 = torch.empty((nst, H, dk, v_dim), dtype=torch.float32, device=q.device) if want_initial else None
    dM0 = torch.empty((nst, H, dk, v_dim), dtype=torch.float32, device=q.device) if want_initial else None
    st = lib().mdn_bwd_state_chain(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(d_o), _ptr(d_final_S), _ptr(d_final_M),
                                   _ptr(cu_seqlens), _ptr(fwd_workspace), fwd_workspace.numel(), _ptr(adj), _ptr(dS0), _ptr(dM0),
                                   _ptr(ws), ws.numel(), _stream())
    if st != 0:
        raise MdnError(st, "mdn_bwd_state_chain")
    return adj, dS0, dM0


def chunk_bwd(q, k, v, beta, log_alpha, log_mu, eta, d_o, *, initial_S=None, initial_M=None, cu_seqlens=None,
              d_final_S=None, d_final_M=None, scale: Optional[float] = None, workspace: Optional[torch.Tensor] = None,
              method: str = "stepwise", saved=None):
    """mdn_chunk_bwd (method="stepwise": exact, fp32, token by token) or mdn_chunk_bwd_chunked (method="chunked":
    chunk-parallel on the tensor cores; bf16 inputs, dk = dv = 128, fixed length) on CUDA tensors (current stream):
    gradients of mdn_chunk_fwd's outputs' loss.  saved = (fwd_workspace, chunk_states) of a chunk_fwd(...,
    keep_chunk_states=True) call with the same inputs: mdn_chunk_bwd_saved (method="chunked" only).
    d_o: [B,T,H,dv] (its dtype is taken as the forward's o_dtype).  Returns a dict of float32 tensors
    dq, dk, dv, dbeta, dlog_alpha, dlog_mu, deta (None when eta is None), d_initial_S, d_initial_M."""
    _check_inputs(q, k, v, (("beta", beta), ("log_alpha", log_alpha), ("log_mu", log_mu), ("eta", eta)), "cuda")
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    if d_o.device.type != "cuda" or not d_o.is_contiguous() or tuple(d_o.shape) != (B, T, H, dv):
        raise ValueError("d_o must be a contiguous cuda tensor of o's shape")
    N = 0
    if cu_seqlens is not None:
        if cu_seqlens.device.type != "cuda" or cu_seqlens.dtype != torch.int32 or not cu_seqlens.is_contiguous():
            raise ValueError("cu_seqlens must be a contiguous int32 cuda tensor")
        N = cu_seqlens.numel() - 1
    p = make_params(q, v, num_seqs=N, scale=scale, o_dtype=d_o.dtype)
    nst = N if N > 0 else B
    for name, t in (("initial_S", initial_S), ("initial_M", initial_M), ("d_final_S", d_final_S), ("d_final_M", d_final_M)):
        _check_state(name, t, (nst, H, dk, dv), "cuda")
    if method not in ("stepwise", "chunked"):
        raise ValueError("method")
    chunked = method == "chunked"
    if chunked:
        p = make_params(q, v, num_seqs=N, scale=scale, o_dtype=d_o.dtype, path="tensor")
        need = int(lib().mdn_chunk_bwd_saved_workspace_bytes(ctypes.byref(p)) if saved is not None
                   else lib().mdn_chunk_bwd_chunked_workspace_bytes(ctypes.byref(p)))
    else:
        need = int(lib().mdn_chunk_bwd_workspace_bytes(ctypes.byref(p)))
    if need == 0:
        raise MdnError(2, "mdn_chunk_bwd_workspace_bytes")
    if workspace is None:
        workspace = torch.empty(need, dtype=torch.uint8, device=q.device)
    f32 = dict(dtype=torch.float32, device=q.device)
    g = dict(dq=torch.empty((B, T, H, dk), **f32), dk=torch.empty((B, T, H, dk), **f32),
             dv=torch.empty((B, T, H, dv), **f32), dbeta=torch.empty((B, T, H), **f32),
             dlog_alpha=torch.empty((B, T, H), **f32), dlog_mu=torch.empty((B, T, H), **f32),
             deta=torch.empty((B, T, H), **f32) if eta is not None else None,
             d_initial_S=torch.empty((nst, H, dk, dv), **f32), d_initial_M=torch.empty((nst, H, dk, dv), **f32))
    if chunked and saved is not None:
        fws, fstates = saved
        st = lib().mdn_chunk_bwd_saved(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(log_alpha), _ptr(log_mu),
                                       _ptr(eta), _ptr(cu_seqlens), _ptr(fws), fws.numel(), _ptr(fstates), _ptr(d_o),
                                       _ptr(d_final_S), _ptr(d_final_M), _ptr(g["dq"]), _ptr(g["dk"]), _ptr(g["dv"]),
                                       _ptr(g["dbeta"]), _ptr(g["dlog_alpha"]), _ptr(g["dlog_mu"]), _ptr(g["deta"]),
                                       _ptr(g["d_initial_S"]), _ptr(g["d_initial_M"]), _ptr(workspace),
                                       workspace.numel(), _stream())
        if st != 0:
            raise MdnError(st, "mdn_chunk_bwd_saved")
        return g
    if chunked:
        st = lib().mdn_chunk_bwd_chunked(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(log_alpha),
                                         _ptr(log_mu), _ptr(eta), _ptr(initial_S), _ptr(initial_M), _ptr(cu_seqlens),
                                         _ptr(d_o), _ptr(d_final_S), _ptr(d_final_M), _ptr(g["dq"]), _ptr(g["dk"]), _ptr(g["dv"]),
                                         _ptr(g["dbeta"]), _ptr(g["dlog_alpha"]), _ptr(g["dlog_mu"]), _ptr(g["deta"]),
                                         _ptr(g["d_initial_S"]), _ptr(g["d_initial_M"]), _ptr(workspace),
                                         workspace.numel(), _stream())
        if st != 0:
            raise MdnError(st, "mdn_chunk_bwd_chunked")
        return g
    st = lib().mdn_chunk_bwd(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(log_alpha), _ptr(log_mu),
                             _ptr(eta), _ptr(initial_S), _ptr(initial_M), _ptr(cu_seqlens), _ptr(d_o), _ptr(d_final_S),
                             _ptr(d_final_M), _ptr(g["dq"]), _ptr(g["dk"]), _ptr(g["dv"]), _ptr(g["dbeta"]),
                             _ptr(g["dlog_alpha"]), _ptr(g["dlog_mu"]), _ptr(g["deta"]), _ptr(g["d_initial_S"]),
                             _ptr(g["d_initial_M"]), _ptr(workspace), workspace.numel(), _stream())
    if st != 0:
        raise MdnError(st, "mdn_chunk_bwd")
    return g


class _ChunkAttention(torch.autograd.Function):
    """Autograd glue around mdn_chunk_fwd_keep_states / mdn_chunk_bwd_saved (no arithmetic here)."""

    @staticmethod
    def forward(ctx, q, k, v, beta, log_alpha, log_mu, eta, initial_S, initial_M, cu_seqlens, scale):
        o, Sf, Mf, states, ws = chunk_fwd(q, k, v, beta, log_alpha, log_mu, eta, initial_S=initial_S,
                                          initial_M=initial_M, cu_seqlens=cu_seqlens, scale=scale, path="tensor",
                                          keep_chunk_states=True)
        ctx.save_for_backward(q, k, v, beta, log_alpha, log_mu, eta, initial_S, initial_M, cu_seqlens, states, ws)
        ctx.scale = scale
        return o, Sf, Mf

    @staticmethod
    def backward(ctx, d_o, d_Sf, d_Mf):
        q, k, v, beta, log_alpha, log_mu, eta, initial_S, initial_M, cu_seqlens, states, ws = ctx.saved_tensors
        g = chunk_bwd(q, k, v, beta, log_alpha, log_mu, eta, d_o.contiguous().to(q.dtype), initial_S=initial_S,
                      initial_M=initial_M, cu_seqlens=cu_seqlens,
                      d_final_S=None if d_Sf is None else d_Sf.contiguous().float(),
                      d_final_M=None if d_Mf is None else d_Mf.contiguous().float(), scale=ctx.scale,
                      method="chunked", saved=(ws, states))
        return (g["dq"].to(q.dtype), g["dk"].to(k.dtype), g["dv"].to(v.dtype), g["dbeta"], g["dlog_alpha"], g["dlog_mu"],
                g["deta"], None if initial_S is None else g["d_initial_S"], None if initial_M is None else g["d_initial_M"],
                None, None)


def chunk_attention(q, k, v, beta, log_alpha, log_mu, eta, *, initial_S=None, initial_M=None, cu_seqlens=None,
                    scale: Optional[float] = None):
    """The forward as a differentiable torch function (tensor path: bf16 q, k, v, dk = dv = 128): returns
    (o, final_S, final_M); gradients come from the chunk-parallel backward on the states the forward kept."""
    return _ChunkAttention.apply(q, k, v, beta, log_alpha, log_mu, eta, initial_S, initial_M, cu_seqlens, scale)


def decode_step(q, k, v, beta, log_alpha, log_mu, eta, S, M, *, scale: Optional[float] = None,
                o_dtype: Optional[torch.dtype] = None, out: Optional[torch.Tensor] = None,
                layer_ops: Optional[MdnLayerOps] = None) -> torch.Tensor:
    """mdn_decode_step (mdn_decode_step_fused when layer_ops is given): one token per sequence (q, k: [B,1,H,dk];
    v: [B,1,H,dv]; gates [B,1,H]); the fp32 states S, M [B,H,dk,dv] are updated in place.  Returns o [B,1,H,dv]."""
    _check_inputs(q, k, v, (("beta", beta), ("log_alpha", log_alpha), ("log_mu", log_mu), ("eta", eta)), "cuda")
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    if T != 1:
        raise ValueError("decode_step takes exactly one token per sequence")
    _check_state("S", S, (B, H, dk, dv), "cuda")
    _check_state("M", M, (B, H, dk, dv), "cuda")
    p = make_params(q, v, scale=scale, o_dtype=o_dtype, path="auto")
    o = out if out is not None else torch.empty((B, 1, H, dv), dtype=o_dtype or q.dtype, device=q.device)
    tail = (_ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(log_alpha), _ptr(log_mu), _ptr(eta), _ptr(S), _ptr(M), _ptr(o),
            _stream())
    if layer_ops is None:
        st = lib().mdn_decode_step(ctypes.byref(p), *tail)
    else:
        st = lib().mdn_decode_step_fused(ctypes.byref(p), ctypes.byref(layer_ops), *tail)
    if st != 0:
        raise MdnError(st, "mdn_decode_step")
    return o


STATIC_SCRATCH_BYTES = 32 << 20


def chunk_fwd_static_scratch(q, k, v, beta, log_alpha, log_mu, eta=None, *, out, final_S=None, final_M=None,
                             initial_S=None, initial_M=None, cu_seqlens=None, scale: Optional[float] = None,
                             path: str = "auto") -> None:
    """mdn_chunk_fwd_static_scratch: the forward without a workspace argument, for callers that
    cannot allocate device memory.  This wrapper allocates nothing either: `out` (and the optional
    `final_S`, `final_M`) are tensors the caller already owns and are written in place.  Raises
    MdnError (status 6) when the problem needs more than STATIC_SCRATCH_BYTES of scratch.  Calls share
    one built-in scratch array: do not let two of them overlap on the GPU."""
    _check_inputs(q, k, v, (("beta", beta), ("log_alpha", log_alpha), ("log_mu", log_mu), ("eta", eta)), "cuda")
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    N = 0 if cu_seqlens is None else cu_seqlens.numel() - 1
    p = make_params(q, v, num_seqs=N, scale=scale, o_dtype=out.dtype, path=path)
    nst = N if N > 0 else B
    for name, t in (("initial_S", initial_S), ("initial_M", initial_M), ("final_S", final_S), ("final_M", final_M)):
        _check_state(name, t, (nst, H, dk, dv), "cuda")
    if tuple(out.shape) != (B, T, H, dv) or not out.is_contiguous() or out.device.type != "cuda":
        raise ValueError("out must be a contiguous cuda tensor of shape [B,T,H,dv]")
    st = lib().mdn_chunk_fwd_static_scratch(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(log_alpha),
                                            _ptr(log_mu), _ptr(eta), _ptr(initial_S), _ptr(initial_M),
                                            _ptr(cu_seqlens), _ptr(out), _ptr(final_S), _ptr(final_M), _stream())
    if st != 0:
        raise MdnError(st, "mdn_chunk_fwd_static_scratch")


def chunk_fwd_host(q, k, v, beta, log_alpha, log_mu, eta=None, *, initial_S=None, initial_M=None,
                   cu_seqlens=None, scale: Optional[float] = None, o_dtype: Optional[torch.dtype] = None,
                   path: str = "auto", output_final_state: bool = True, arena: Optional[torch.Tensor] = None,
                   out=None, device="cuda:0"):
    """mdn_chunk_fwd_host: all tensors are HOST tensors (pinned for async copies); `arena` is a
    CUDA uint8 buffer of host_arena_bytes(p).  Returns host (o, final_S, final_M); synchronises."""
    _check_inputs(q, k, v, (("beta", beta), ("log_alpha", log_alpha), ("log_mu", log_mu), ("eta", eta)), "cpu")
    B, T, H, dk = q.shape
    dv = v.shape[-1]
    N = 0 if cu_seqlens is None else cu_seqlens.numel() - 1
    p = make_params(q, v, num_seqs=N, scale=scale, o_dtype=o_dtype, path=path)
    nst = N if N > 0 else B
    _check_state("initial_S", initial_S, (nst, H, dk, dv), "cpu")
    _check_state("initial_M", initial_M, (nst, H, dk, dv), "cpu")
    need = host_arena_bytes(p)
    if need == 0:
        raise MdnError(2, "mdn_chunk_fwd_host_arena_bytes")
    if arena is None:
        arena = torch.empty(need, dtype=torch.uint8, device=device)
    if out is None:
        o = torch.empty((B, T, H, dv), dtype=o_dtype or q.dtype).pin_memory()
        Sf = torch.empty((nst, H, dk, dv), dtype=torch.float32).pin_memory() if output_final_state else None
        Mf = torch.empty((nst, H, dk, dv), dtype=torch.float32).pin_memory() if output_final_state else None
    else:
        o, Sf, Mf = out
    with torch.cuda.device(arena.device):
        st = lib().mdn_chunk_fwd_host(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(v), _ptr(beta), _ptr(log_alpha),
                                      _ptr(log_mu), _ptr(eta), _ptr(initial_S), _ptr(initial_M), _ptr(cu_seqlens),
                                      _ptr(o), _ptr(Sf), _ptr(Mf), _ptr(arena), arena.numel(), _stream())
        if st != 0:
            raise MdnError(st, "mdn_chunk_fwd_host")
        torch.cuda.current_stream().synchronize()
    return o, Sf, Mf


def coeff_scan(p: MdnParams, beta, log_alpha, log_mu, eta, cu_seqlens, workspace) -> None:
    st = lib().mdn_coeff_scan(ctypes.byref(p), _ptr(beta), _ptr(log_alpha), _ptr(log_mu), _ptr(eta),
                              _ptr(cu_seqlens), _ptr(workspace), workspace.numel(), _stream())
    if st != 0:
        raise MdnError(st, "mdn_coeff_scan")


def intra_chunk(p: MdnParams, q, k, cu_seqlens, workspace) -> None:
    st = lib().mdn_intra_chunk(ctypes.byref(p), _ptr(q), _ptr(k), _ptr(cu_seqlens), _ptr(workspace),
                               workspace.numel(), _stream())
    if st != 0:
        raise MdnError(st, "mdn_intra_chunk")


def read_status(p: MdnParams, workspace) -> int:
    return int(lib().mdn_read_status(ctypes.byref(p), _ptr(workspace), _stream()))
