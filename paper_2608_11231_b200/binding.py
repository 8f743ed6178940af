"""ctypes binding of the lkv C ABI (see include/lkv.h): argument marshalling only.

Functions carry the names of the C entry points and take torch CUDA tensors for
device buffers; torch is used for device memory and streams, nothing else.
Every step of the computation runs in the CUDA library.  There is no fallback:
if ``liblkv.so`` is missing, the first call raises.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import numpy as np
import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "liblkv.so")

# constants of include/lkv.h
LKV_OK = 0
LKV_ERR_NULL, LKV_ERR_DIM, LKV_ERR_MODE, LKV_ERR_INDEX, LKV_ERR_ALIGN = -1, -2, -3, -4, -5
LKV_ERR_UNSUPPORTED, LKV_ERR_WORKSPACE, LKV_ERR_CUDA, LKV_ERR_DEVICE_TIMEOUT, LKV_ERR_OVERLAP = -6, -7, -8, -9, -10
LKV_FAMILY_MAMBA2, LKV_FAMILY_GDN = 0, 1
LKV_DTYPE_F32, LKV_DTYPE_BF16 = 0, 1
LKV_INIT_LAST, LKV_INIT_INDEX, LKV_INIT_EXACT = 0, 1, 2
LKV_COMPUTE_AUTO, LKV_COMPUTE_FP32, LKV_COMPUTE_TENSOR = 0, 1, 2
LKV_WS_INIT, LKV_WS_GDN, LKV_WS_SSD = 0, 1, 2

EXPORTS = ("lkv_init_state", "lkv_init_state_batched", "lkv_init_state_batched_static", "lkv_gdn_fwd", "lkv_ssd_fwd",
           "lkv_gdn_chunk_transition", "lkv_mamba_chunk_logdecay", "lkv_init_state_fold", "lkv_gdn_fwd_segmented",
           "lkv_gdn_segmented_scratch_bytes", "lkv_stage_chunks", "lkv_gdn_chunk_artifacts", "lkv_state_rel_error",
           "lkv_state_rel_error_workspace_bytes", "lkv_workspace_bytes", "lkv_device_status", "lkv_device_status_static",
           "lkv_selftest_bounded_wait", "lkv_status_string", "lkv_version")


class lkv_init_desc(ctypes.Structure):
    _fields_ = [("family", ctypes.c_int32), ("H", ctypes.c_int32), ("d_k", ctypes.c_int32), ("d_v", ctypes.c_int32),
                ("n_chunks", ctypes.c_int32), ("state_dtype", ctypes.c_int32), ("sel_index", ctypes.c_int32),
                ("compute", ctypes.c_int32), ("chunk_ids", ctypes.c_void_p), ("workspace", ctypes.c_void_p),
                ("workspace_bytes", ctypes.c_size_t)]


class lkv_gdn_desc(ctypes.Structure):
    _fields_ = [("T_total", ctypes.c_int32), ("n_seq", ctypes.c_int32), ("cu_seqlens", ctypes.c_void_p),
                ("H_k", ctypes.c_int32), ("H_v", ctypes.c_int32), ("d_k", ctypes.c_int32), ("d_v", ctypes.c_int32),
                ("io_dtype", ctypes.c_int32), ("compute", ctypes.c_int32), ("scale", ctypes.c_float),
                ("state_dtype", ctypes.c_int32), ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t)]


class lkv_ssd_desc(ctypes.Structure):
    _fields_ = [("T_total", ctypes.c_int32), ("n_seq", ctypes.c_int32), ("cu_seqlens", ctypes.c_void_p),
                ("H", ctypes.c_int32), ("P", ctypes.c_int32), ("N", ctypes.c_int32), ("G", ctypes.c_int32),
                ("io_dtype", ctypes.c_int32), ("compute", ctypes.c_int32), ("state_dtype", ctypes.c_int32),
                ("workspace", ctypes.c_void_p), ("workspace_bytes", ctypes.c_size_t)]


class LkvError(RuntimeError):
    def __init__(self, status: int, where: str):
        self.status = status
        super().__init__(f"{where}: {status_string(status)} ({status})")


_lib = None


def load() -> ctypes.CDLL:
    """Load liblkv.so (built in-tree by build.py).  Raises if it is missing: there is no fallback path."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise RuntimeError(f"{LIB_PATH} is missing: build it with `python -m paper_2608_11231_b200.build` "
                               "(or __graft_entry__.build()); the library has no CPU or PyTorch fallback")
        lib = ctypes.CDLL(LIB_PATH)
        vp, ci = ctypes.c_void_p, ctypes.c_int
        lib.lkv_init_state.argtypes = [vp, vp, ci, ci, vp, ctypes.POINTER(lkv_init_desc), vp]
        lib.lkv_init_state_batched.argtypes = [vp, vp, vp, vp, ci, ci, vp, vp, ctypes.POINTER(lkv_init_desc), vp]
        lib.lkv_init_state_batched_static.argtypes = lib.lkv_init_state_batched.argtypes
        lib.lkv_init_state_batched_static.restype = ci
        lib.lkv_gdn_fwd.argtypes = [vp] * 8 + [ctypes.POINTER(lkv_gdn_desc), vp]
        lib.lkv_ssd_fwd.argtypes = [vp] * 8 + [ctypes.POINTER(lkv_ssd_desc), vp]
        lib.lkv_gdn_chunk_transition.argtypes = [vp] * 4 + [ctypes.POINTER(lkv_gdn_desc), vp]
        lib.lkv_mamba_chunk_logdecay.argtypes = [vp] * 3 + [ctypes.POINTER(lkv_ssd_desc), vp]
        lib.lkv_init_state_fold.argtypes = [vp, vp, vp, vp, vp, ci, vp, ctypes.POINTER(lkv_init_desc), ci, ci, vp]
        lib.lkv_init_state_fold.restype = ci
        lib.lkv_gdn_chunk_artifacts.argtypes = [vp] * 6 + [ctypes.POINTER(lkv_gdn_desc), vp]
        lib.lkv_gdn_chunk_artifacts.restype = ci
        lib.lkv_stage_chunks.argtypes = [vp, vp, vp, ci, vp, vp, ci, vp, vp, ctypes.POINTER(lkv_init_desc), vp]
        lib.lkv_stage_chunks.restype = ci
        lib.lkv_gdn_fwd_segmented.argtypes = [vp] * 8 + [ctypes.POINTER(lkv_gdn_desc), ci, vp, ctypes.c_size_t, vp]
        lib.lkv_gdn_fwd_segmented.restype = ci
        lib.lkv_gdn_segmented_scratch_bytes.argtypes = [ctypes.POINTER(lkv_gdn_desc), ci]
        lib.lkv_gdn_segmented_scratch_bytes.restype = ctypes.c_size_t
        lib.lkv_state_rel_error.argtypes = [vp, vp, vp, ci, ctypes.c_size_t, vp, ctypes.c_size_t, vp]
        lib.lkv_state_rel_error_workspace_bytes.argtypes = [ci, ctypes.c_size_t]
        lib.lkv_state_rel_error_workspace_bytes.restype = ctypes.c_size_t
        lib.lkv_workspace_bytes.argtypes = [ci, vp, ci, ci]
        lib.lkv_workspace_bytes.restype = ctypes.c_size_t
        lib.lkv_device_status.argtypes = [vp, vp]
        lib.lkv_device_status_static.argtypes = [vp]
        lib.lkv_selftest_bounded_wait.argtypes = [ci, vp, vp]
        lib.lkv_status_string.argtypes = [ci]
        lib.lkv_status_string.restype = ctypes.c_char_p
        for name in ("lkv_init_state", "lkv_init_state_batched", "lkv_gdn_fwd", "lkv_ssd_fwd",
                     "lkv_device_status", "lkv_device_status_static", "lkv_selftest_bounded_wait", "lkv_version"):
            getattr(lib, name).restype = ci
        _lib = lib
    return _lib


def status_string(status: int) -> str:
    return load().lkv_status_string(int(status)).decode()


def lkv_version() -> int:
    return int(load().lkv_version())


def _dtype_code(t: torch.Tensor) -> int:
    if t.dtype == torch.float32:
        return LKV_DTYPE_F32
    if t.dtype == torch.bfloat16:
        return LKV_DTYPE_BF16
    raise TypeError(f"unsupported dtype {t.dtype}")


def _ptr(t: Optional[torch.Tensor]):
    if t is None:
        return None
    if not t.is_cuda or not t.is_contiguous():
        raise ValueError("device buffers must be contiguous CUDA tensors")
    return ctypes.c_void_p(t.data_ptr())


def _stream(stream):
    s = torch.cuda.current_stream() if stream is None else stream
    return ctypes.c_void_p(s.cuda_stream)


def _host_i32(a) -> Optional[np.ndarray]:
    if a is None:
        return None
    if isinstance(a, torch.Tensor):
        a = a.cpu().numpy()
    return np.ascontiguousarray(a, dtype=np.int32)


def _hp(a: Optional[np.ndarray]):
    return None if a is None else ctypes.c_void_p(a.ctypes.data)


_ws_cache = {}
_err_ws_cache = {}


def workspace(device, nbytes: int) -> torch.Tensor:
    """A zero-initialised, cached device workspace of at least nbytes (one per device and stream)."""
    key = (torch.device(device).index, torch.cuda.current_stream().cuda_stream)
    ws = _ws_cache.get(key)
    if ws is None or ws.numel() < nbytes:
        ws = torch.zeros(max(int(nbytes), 4096), dtype=torch.uint8, device=device)
        _ws_cache[key] = ws
    return ws


def lkv_workspace_bytes(which: int, desc, n_units: int, n_index: int = 0) -> int:
    return int(load().lkv_workspace_bytes(which, ctypes.cast(ctypes.pointer(desc), ctypes.c_void_p), n_units, n_index))


def lkv_device_status(ws: torch.Tensor, stream=None) -> int:
    return int(load().lkv_device_status(_ptr(ws), _stream(stream)))


def lkv_device_status_static(stream=None) -> int:
    """Status of the scratch of lkv_init_state_batched_static on the current device (cleared after a time-out)."""
    return int(load().lkv_device_status_static(_stream(stream)))


def lkv_selftest_bounded_wait(poll_limit: int, ws: torch.Tensor, stream=None) -> int:
    """Launches the kernel whose only job is to let a bounded wait run out; the status word of ws is set."""
    return int(load().lkv_selftest_bounded_wait(int(poll_limit), _ptr(ws), _stream(stream)))


def _init_desc(states, family, compute, ws_t, n_units, n_index, chunk_ids_np=None, sel_index=0):
    n, H, d_k, d_v = states.shape
    d = lkv_init_desc(family=family, H=H, d_k=d_k, d_v=d_v, n_chunks=n, state_dtype=_dtype_code(states),
                      sel_index=int(sel_index), compute=compute,
                      chunk_ids=None if chunk_ids_np is None else chunk_ids_np.ctypes.data, workspace=None,
                      workspace_bytes=0)
    if ws_t is None:
        ws_t = workspace(states.device, lkv_workspace_bytes(LKV_WS_INIT, d, n_units, n_index))
    d.workspace = ws_t.data_ptr()
    d.workspace_bytes = ws_t.numel()
    return d, ws_t


def lkv_init_state(states: torch.Tensor, transitions: Optional[torch.Tensor], K: int, mode: int,
                   S0: Optional[torch.Tensor] = None, *, family: int, chunk_ids=None, sel_index: int = 0,
                   compute: int = LKV_COMPUTE_AUTO, workspace_t: Optional[torch.Tensor] = None, stream=None):
    """State initialisation for one request.  states: pool [n, H, d_k, d_v]; returns S0 [H, d_k, d_v] fp32."""
    ids = _host_i32(chunk_ids)
    d, ws_t = _init_desc(states, family, compute, workspace_t, 1, int(K), ids, sel_index)
    if S0 is None:
        S0 = torch.empty(states.shape[1:], dtype=torch.float32, device=states.device)
    st = load().lkv_init_state(_ptr(states), _ptr(transitions), int(K), int(mode), _ptr(S0), ctypes.byref(d),
                               _stream(stream))
    if st != LKV_OK:
        raise LkvError(st, "lkv_init_state")
    return S0


def lkv_init_state_batched(states: torch.Tensor, transitions: Optional[torch.Tensor], chunk_ids, cu_k, n_req: int,
                           mode: int, sel_index=None, S0: Optional[torch.Tensor] = None, *, family: int,
                           compute: int = LKV_COMPUTE_AUTO, workspace_t: Optional[torch.Tensor] = None, stream=None):
    """State initialisation for n_req requests in one launch; returns S0 [n_req, H, d_k, d_v] fp32."""
    ids, cu, sel = _host_i32(chunk_ids), _host_i32(cu_k), _host_i32(sel_index)
    d, ws_t = _init_desc(states, family, compute, workspace_t, int(n_req), 0 if ids is None else ids.size)
    if S0 is None:
        S0 = torch.empty((n_req,) + tuple(states.shape[1:]), dtype=torch.float32, device=states.device)
    st = load().lkv_init_state_batched(_ptr(states), _ptr(transitions), _hp(ids), _hp(cu), int(n_req), int(mode),
                                       _hp(sel), _ptr(S0), ctypes.byref(d), _stream(stream))
    if st != LKV_OK:
        raise LkvError(st, "lkv_init_state_batched")
    return S0


LKV_STATIC_MAX_INDEX = 16384


def lkv_init_state_batched_static(states: torch.Tensor, transitions: Optional[torch.Tensor], chunk_ids, cu_k,
                                  n_req: int, mode: int, sel_index=None, S0: Optional[torch.Tensor] = None, *,
                                  family: int, compute: int = LKV_COMPUTE_AUTO, stream=None):
    """lkv_init_state_batched for callers that cannot allocate: no workspace is passed or created.

    The library keeps its scratch in a fixed array of its own (see the header for the size limit, the
    first-call rule and why overlapping calls race).  Pass S0 to keep this wrapper allocation-free too;
    if it is None the wrapper creates the output tensor, which a caller that cannot allocate would not do.
    """
    ids, cu, sel = _host_i32(chunk_ids), _host_i32(cu_k), _host_i32(sel_index)
    n, H, d_k, d_v = states.shape
    d = lkv_init_desc(family=family, H=H, d_k=d_k, d_v=d_v, n_chunks=n, state_dtype=_dtype_code(states),
                      sel_index=0, compute=compute, chunk_ids=None, workspace=None, workspace_bytes=0)
    if S0 is None:
        S0 = torch.empty((n_req,) + tuple(states.shape[1:]), dtype=torch.float32, device=states.device)
    st = load().lkv_init_state_batched_static(_ptr(states), _ptr(transitions), _hp(ids), _hp(cu), int(n_req),
                                              int(mode), _hp(sel), _ptr(S0), ctypes.byref(d), _stream(stream))
    if st != LKV_OK:
        raise LkvError(st, "lkv_init_state_batched_static")
    return S0


def lkv_gdn_fwd(q, k, v, g, beta, S0=None, o=None, S_T=None, *, cu_seqlens=None, scale: float = 0.0,
                compute: int = LKV_COMPUTE_AUTO, want_final_state: bool = True, want_outputs: bool = True,
                state_dtype=torch.float32, workspace_t: Optional[torch.Tensor] = None, stream=None):
    """Gated DeltaNet scan.  q, k: [T, H_k, d_k]; v: [T, H_v, d_v]; g, beta: [T, H_v] fp32.

    Returns (o [T, H_v, d_v] in the dtype of v, or None with want_outputs=False; S_T [n_seq, H_v, d_k, d_v] in
    state_dtype (fp32 or bf16; the dtype of S_T if one is passed) or None).
    """
    T, H_k, d_k = q.shape
    _, H_v, d_v = v.shape
    cu = _host_i32(cu_seqlens)
    n_seq = 1 if cu is None else cu.size - 1
    d = lkv_gdn_desc(T_total=T, n_seq=n_seq, cu_seqlens=None if cu is None else cu.ctypes.data, H_k=H_k, H_v=H_v,
                     d_k=d_k, d_v=d_v, io_dtype=_dtype_code(v), compute=compute, scale=float(scale), state_dtype=0,
                     workspace=None, workspace_bytes=0)
    ws_t = workspace_t if workspace_t is not None else workspace(v.device, lkv_workspace_bytes(LKV_WS_GDN, d, n_seq))
    d.workspace, d.workspace_bytes = ws_t.data_ptr(), ws_t.numel()
    if o is None and want_outputs:
        o = torch.empty_like(v)
    if S_T is None and want_final_state:
        S_T = torch.empty((n_seq, H_v, d_k, d_v), dtype=state_dtype, device=v.device)
    if S_T is not None:
        d.state_dtype = _dtype_code(S_T)
    st = load().lkv_gdn_fwd(_ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(S0), _ptr(o), _ptr(S_T),
                            ctypes.byref(d), _stream(stream))
    if st != LKV_OK:
        raise LkvError(st, "lkv_gdn_fwd")
    return o, S_T


def lkv_gdn_fwd_segmented(q, k, v, g, beta, S0=None, o=None, S_T=None, *, n_segments: int, scale: float = 0.0,
                          compute: int = LKV_COMPUTE_AUTO, scratch: Optional[torch.Tensor] = None,
                          workspace_t: Optional[torch.Tensor] = None, stream=None):
    """lkv_gdn_fwd for one long sequence, its n_segments segments scanned in parallel (states and transitions of the
    segments, exact composition, then all segments at once).  S0: [1, H_v, d, d] fp32 or None.  Returns (o, S_T)."""
    T, H_k, d_k = q.shape
    _, H_v, d_v = v.shape
    d = lkv_gdn_desc(T_total=T, n_seq=1, cu_seqlens=None, H_k=H_k, H_v=H_v, d_k=d_k, d_v=d_v, io_dtype=_dtype_code(v),
                     compute=compute, scale=float(scale), state_dtype=0, workspace=None, workspace_bytes=0)
    ws_t = workspace_t if workspace_t is not None else workspace(v.device, lkv_workspace_bytes(LKV_WS_GDN, d, 2 * n_segments))
    d.workspace, d.workspace_bytes = ws_t.data_ptr(), ws_t.numel()
    need = int(load().lkv_gdn_segmented_scratch_bytes(ctypes.byref(d), int(n_segments)))
    if scratch is None:
        scratch = torch.empty(max(need, 16), dtype=torch.uint8, device=v.device)
    if o is None:
        o = torch.empty_like(v)
    if S_T is None:
        S_T = torch.empty((1, H_v, d_k, d_v), dtype=torch.float32, device=v.device)
    st = load().lkv_gdn_fwd_segmented(_ptr(q), _ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(S0), _ptr(o), _ptr(S_T),
                                      ctypes.byref(d), int(n_segments), _ptr(scratch), scratch.numel(), _stream(stream))
    if st != LKV_OK:
        raise LkvError(st, "lkv_gdn_fwd_segmented")
    return o, S_T


def lkv_ssd_fwd(x, dt, A, B, C, S0=None, y=None, S_T=None, *, cu_seqlens=None, compute: int = LKV_COMPUTE_AUTO,
                want_final_state: bool = True, want_outputs: bool = True, state_dtype=torch.float32,
                workspace_t: Optional[torch.Tensor] = None, stream=None):
    """Mamba-2 (SSD) scan.  x: [T, H, P]; dt: [T, H] fp32; A: [H] fp32; B, C: [T, G, N].

    Returns (y [T, H, P] in the dtype of x, S_T [n_seq, H, N, P] in state_dtype (fp32 or bf16) or None).
    """
    T, H, P = x.shape
    _, G, N = B.shape
    cu = _host_i32(cu_seqlens)
    n_seq = 1 if cu is None else cu.size - 1
    d = lkv_ssd_desc(T_total=T, n_seq=n_seq, cu_seqlens=None if cu is None else cu.ctypes.data, H=H, P=P, N=N, G=G,
                     io_dtype=_dtype_code(x), compute=compute, workspace=None, workspace_bytes=0)
    ws_t = workspace_t if workspace_t is not None else workspace(x.device, lkv_workspace_bytes(LKV_WS_SSD, d, n_seq))
    d.workspace, d.workspace_bytes = ws_t.data_ptr(), ws_t.numel()
    if y is None and want_outputs:
        y = torch.empty_like(x)
    if S_T is None and want_final_state:
        S_T = torch.empty((n_seq, H, N, P), dtype=state_dtype, device=x.device)
    if S_T is not None:
        d.state_dtype = _dtype_code(S_T)
    st = load().lkv_ssd_fwd(_ptr(x), _ptr(dt), _ptr(A), _ptr(B), _ptr(C), _ptr(S0), _ptr(y), _ptr(S_T),
                            ctypes.byref(d), _stream(stream))
    if st != LKV_OK:
        raise LkvError(st, "lkv_ssd_fwd")
    return y, S_T


def lkv_init_state_fold(states: torch.Tensor, k, g, beta, cu_tokens, K: int, chunk_ids=None,
                        S0: Optional[torch.Tensor] = None, *, compute: int = LKV_COMPUTE_AUTO,
                        workspace_t: Optional[torch.Tensor] = None, stream=None):
    """GDN exact composition of one request from the cached key / gate streams (no materialised transitions).

    states: fp32 pool [n_chunks, H, d, d]; k: [total_tokens, H_k, d]; g, beta: [total_tokens, H] fp32;
    cu_tokens: host int32[n_chunks + 1].  Returns S0 [H, d, d] fp32.
    """
    ids, cu = _host_i32(chunk_ids), _host_i32(cu_tokens)
    d, ws_t = _init_desc(states, LKV_FAMILY_GDN, compute, workspace_t, 1, int(K), ids)
    if S0 is None:
        S0 = torch.empty(tuple(states.shape[1:]), dtype=torch.float32, device=states.device)
    st = load().lkv_init_state_fold(_ptr(states), _ptr(k), _ptr(g), _ptr(beta), _hp(cu), int(K), _ptr(S0),
                                    ctypes.byref(d), int(k.shape[1]), _dtype_code(k), _stream(stream))
    if st != LKV_OK:
        raise LkvError(st, "lkv_init_state_fold")
    return S0


def lkv_stage_chunks(host_states: torch.Tensor, host_transitions: Optional[torch.Tensor], chunk_ids, dev_states: torch.Tensor,
                     dev_transitions: Optional[torch.Tensor], *, family: int, stream=None):
    """Copies the distinct chunks named by chunk_ids from host pools (pinned CPU tensors) into the device staging pools.
    Returns (staged_ids int32 numpy array for lkv_init_state_batched, number of chunks copied)."""
    ids = _host_i32(chunk_ids)
    n, H, d_k, d_v = host_states.shape
    d = lkv_init_desc(family=family, H=H, d_k=d_k, d_v=d_v, n_chunks=n, state_dtype=_dtype_code(host_states), sel_index=0,
                      compute=LKV_COMPUTE_AUTO, chunk_ids=None, workspace=None, workspace_bytes=0)
    staged = np.empty(ids.size, dtype=np.int32)
    n_staged = ctypes.c_int32(0)
    st = load().lkv_stage_chunks(host_states.data_ptr(), None if host_transitions is None else host_transitions.data_ptr(),
                                 _hp(ids), ids.size, _ptr(dev_states), _ptr(dev_transitions), int(dev_states.shape[0]),
                                 staged.ctypes.data, ctypes.addressof(n_staged), ctypes.byref(d), _stream(stream))
    if st != LKV_OK:
        raise LkvError(st, "lkv_stage_chunks")
    return staged, int(n_staged.value)


def lkv_gdn_chunk_transition(k, g, beta, transitions=None, *, cu_seqlens=None, H_v: Optional[int] = None,
                             compute: int = LKV_COMPUTE_AUTO, workspace_t: Optional[torch.Tensor] = None, stream=None):
    """Accumulated transition of every chunk (sequence of cu_seqlens) and value head.

    k: [T, H_k, d]; g, beta: [T, H_v] fp32.  Returns transitions [n_seq, H_v, d, d] fp32.
    """
    T, H_k, d_k = k.shape
    H_v = g.shape[1] if H_v is None else H_v
    cu = _host_i32(cu_seqlens)
    n_seq = 1 if cu is None else cu.size - 1
    d = lkv_gdn_desc(T_total=T, n_seq=n_seq, cu_seqlens=None if cu is None else cu.ctypes.data, H_k=H_k, H_v=H_v,
                     d_k=d_k, d_v=d_k, io_dtype=_dtype_code(k), compute=compute, scale=0.0, state_dtype=0,
                     workspace=None, workspace_bytes=0)
    ws_t = workspace_t if workspace_t is not None else workspace(k.device, lkv_workspace_bytes(LKV_WS_GDN, d, n_seq))
    d.workspace, d.workspace_bytes = ws_t.data_ptr(), ws_t.numel()
    if transitions is None:
        transitions = torch.empty((n_seq, H_v, d_k, d_k), dtype=torch.float32, device=k.device)
    st = load().lkv_gdn_chunk_transition(_ptr(k), _ptr(g), _ptr(beta), _ptr(transitions), ctypes.byref(d), _stream(stream))
    if st != LKV_OK:
        raise LkvError(st, "lkv_gdn_chunk_transition")
    return transitions


def lkv_gdn_chunk_artifacts(k, v, g, beta, states=None, transitions=None, *, cu_seqlens=None,
                            compute: int = LKV_COMPUTE_AUTO, workspace_t: Optional[torch.Tensor] = None, stream=None):
    """S_local and T_C of every chunk (sequence of cu_seqlens) in one launch.  Returns (states, transitions),
    fp32 [n_seq, H_v, d, d] each."""
    T, H_k, d_k = k.shape
    _, H_v, d_v = v.shape
    cu = _host_i32(cu_seqlens)
    n_seq = 1 if cu is None else cu.size - 1
    d = lkv_gdn_desc(T_total=T, n_seq=n_seq, cu_seqlens=None if cu is None else cu.ctypes.data, H_k=H_k, H_v=H_v,
                     d_k=d_k, d_v=d_v, io_dtype=_dtype_code(k), compute=compute, scale=0.0, state_dtype=0,
                     workspace=None, workspace_bytes=0)
    ws_t = workspace_t if workspace_t is not None else workspace(k.device, lkv_workspace_bytes(LKV_WS_GDN, d, 2 * n_seq))
    d.workspace, d.workspace_bytes = ws_t.data_ptr(), ws_t.numel()
    if states is None:
        states = torch.empty((n_seq, H_v, d_k, d_v), dtype=torch.float32, device=k.device)
    if transitions is None:
        transitions = torch.empty((n_seq, H_v, d_k, d_k), dtype=torch.float32, device=k.device)
    st = load().lkv_gdn_chunk_artifacts(_ptr(k), _ptr(v), _ptr(g), _ptr(beta), _ptr(states), _ptr(transitions),
                                        ctypes.byref(d), _stream(stream))
    if st != LKV_OK:
        raise LkvError(st, "lkv_gdn_chunk_artifacts")
    return states, transitions


def lkv_mamba_chunk_logdecay(dt, A, logdecay=None, *, cu_seqlens=None, workspace_t: Optional[torch.Tensor] = None,
                             stream=None):
    """lambda[c][h] = A[h] * sum of dt over chunk c.  dt: [T, H] fp32; A: [H] fp32.  Returns [n_seq, H] fp32."""
    T, H = dt.shape
    cu = _host_i32(cu_seqlens)
    n_seq = 1 if cu is None else cu.size - 1
    d = lkv_ssd_desc(T_total=T, n_seq=n_seq, cu_seqlens=None if cu is None else cu.ctypes.data, H=H, P=1, N=1, G=1,
                     io_dtype=LKV_DTYPE_F32, compute=LKV_COMPUTE_AUTO, workspace=None, workspace_bytes=0)
    ws_t = workspace_t if workspace_t is not None else workspace(dt.device, lkv_workspace_bytes(LKV_WS_SSD, d, n_seq))
    d.workspace, d.workspace_bytes = ws_t.data_ptr(), ws_t.numel()
    if logdecay is None:
        logdecay = torch.empty((n_seq, H), dtype=torch.float32, device=dt.device)
    st = load().lkv_mamba_chunk_logdecay(_ptr(dt), _ptr(A), _ptr(logdecay), ctypes.byref(d), _stream(stream))
    if st != LKV_OK:
        raise LkvError(st, "lkv_mamba_chunk_logdecay")
    return logdecay


def lkv_state_rel_error(S_init, S_ref, n_states: Optional[int] = None, rel_err=None, *, stream=None):
    """||S_init_i - S_ref_i|| / ||S_ref_i|| per state; the tensors are split into n_states equal runs
    (default: along the leading axis).  Returns rel_err [n_states] fp32."""
    assert S_init.shape == S_ref.shape and S_init.dtype == torch.float32 and S_ref.dtype == torch.float32
    n = S_init.shape[0] if n_states is None else int(n_states)
    elems = S_init.numel() // max(n, 1)
    if rel_err is None:
        rel_err = torch.empty((n,), dtype=torch.float32, device=S_init.device)
    nbytes = load().lkv_state_rel_error_workspace_bytes(n, elems)
    # scratch of its own: this call keeps partial sums from byte 0 on, it has no status header
    key = torch.device(S_init.device).index
    ws_t = _err_ws_cache.get(key)
    if ws_t is None or ws_t.numel() < nbytes:
        ws_t = _err_ws_cache[key] = torch.empty(max(int(nbytes), 256), dtype=torch.uint8, device=S_init.device)
    st = load().lkv_state_rel_error(_ptr(S_init), _ptr(S_ref), _ptr(rel_err), n, elems, ws_t.data_ptr(), ws_t.numel(),
                                    _stream(stream))
    if st != LKV_OK:
        raise LkvError(st, "lkv_state_rel_error")
    return rel_err

