"""fp64 CPU oracle for the recurrent-layer hot path -- TEST INFRASTRUCTURE.

Only the tests, the smoke check and the benchmark's CPU-baseline leg may import
this package.  It does not import the CUDA library or its Python binding and
shares no code with them; inputs arrive as numpy arrays and every function
widens them to float64 before computing.

The arithmetic lives in ``lkv_oracle.c`` (plain C, token-by-token recurrences,
compiled here with gcc); this module only marshals arrays.

Functions and the passage of the paper each one states:

``gdn_seq``            Eq. 1 with the GDN transition of Eq. 3, token by token
``ssd_seq``            Eq. 1 with the Mamba-2 scalar transition of Eq. 2
``gdn_transition``     the accumulated chunk transition T_C of Eq. 5 (GDN)
``mamba_logdecay``     the same for Mamba-2, as log of the scalar decay
``init_exact_gdn``     Eq. 6 through repeated use of Eq. 5 (dense transitions)
``init_exact_mamba``   Eq. 6 with scalar transitions
``init_single``        the single-block initialiser S_init = S_b (Section 3.2,
                       "Single-block initialization"; Appendix A for b != K)
``state_rel_error``    the per-state relative error ||S_init - S*|| / ||S*|| of
                       Section 3.2, "Diagnosis via relative error" (numpy)

Parity status: every function above is pinned by the CPU tests (brute force on
the concatenated prefix, literal Eq. 3 matrices, closed forms and library
limits).  Two conventions the paper does not state stay "parity unpinned": the
read-out (o_t = scale * S_t^T q_t, y_t = S_t^T C_t, post-update state) and the
grouped-head mapping (value head h reads q/k head h // (H_v // H_k)).
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "lkv_oracle.c")
_LIB = os.path.join(_HERE, "liblkv_oracle.so")

_lib = None


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (-O2, OpenMP, no fast-math)."""
    stale = (not os.path.exists(_LIB)) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.run(
            ["gcc", "-O2", "-fopenmp", "-shared", "-fPIC", "-std=c11", "-o", tmp, _SRC, "-lm"],
            check=True,
        )
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.lkvo_num_threads.restype = ctypes.c_int
    return _lib


def _f64(a):
    return np.ascontiguousarray(np.asarray(a, dtype=np.float64))


def _p(a):
    return a.ctypes.data_as(ctypes.c_void_p) if a is not None else None


def num_threads() -> int:
    return int(_load().lkvo_num_threads())


def set_num_threads(n: int) -> None:
    _load().lkvo_set_num_threads(ctypes.c_int(int(n)))


def gdn_seq(q, k, v, g, beta, S0=None, scale=None):
    """Token-by-token Gated DeltaNet over one sequence.

    q, k: [T, Hk, dk]; v: [T, Hv, dv]; g, beta: [T, Hv]; S0: [Hv, dk, dv] or None.
    Returns (o [T, Hv, dv], S_T [Hv, dk, dv]) in float64.
    """
    q, k, v, g, beta = _f64(q), _f64(k), _f64(v), _f64(g), _f64(beta)
    T, Hk, dk = q.shape
    _, Hv, dv = v.shape
    assert k.shape == (T, Hk, dk) and g.shape == (T, Hv) and beta.shape == (T, Hv)
    assert Hv % Hk == 0
    if scale is None:
        scale = dk ** -0.5
    s0 = _f64(S0) if S0 is not None else None
    if s0 is not None:
        assert s0.shape == (Hv, dk, dv)
    o = np.empty((T, Hv, dv), dtype=np.float64)
    S_T = np.empty((Hv, dk, dv), dtype=np.float64)
    _load().lkvo_gdn_seq(_p(q), _p(k), _p(v), _p(g), _p(beta), _p(s0), ctypes.c_double(scale),
                         T, Hk, Hv, dk, dv, _p(o), _p(S_T))
    return o, S_T


def ssd_seq(x, dt, A, B, C, S0=None):
    """Token-by-token Mamba-2 (SSD) over one sequence.

    x: [T, H, P]; dt: [T, H]; A: [H]; B, C: [T, G, N]; S0: [H, N, P] or None.
    Returns (y [T, H, P], S_T [H, N, P]) in float64.
    """
    x, dt, A, B, C = _f64(x), _f64(dt), _f64(A), _f64(B), _f64(C)
    T, H, P = x.shape
    _, G, N = B.shape
    assert dt.shape == (T, H) and A.shape == (H,) and C.shape == (T, G, N) and H % G == 0
    s0 = _f64(S0) if S0 is not None else None
    if s0 is not None:
        assert s0.shape == (H, N, P)
    y = np.empty((T, H, P), dtype=np.float64)
    S_T = np.empty((H, N, P), dtype=np.float64)
    _load().lkvo_ssd_seq(_p(x), _p(dt), _p(A), _p(B), _p(C), _p(s0), T, H, P, N, G, _p(y), _p(S_T))
    return y, S_T


def gdn_transition(k, g, beta):
    """Accumulated GDN transition of one chunk, [Hv, dk, dk] float64."""
    k, g, beta = _f64(k), _f64(g), _f64(beta)
    T, Hk, dk = k.shape
    Hv = g.shape[1]
    assert g.shape == (T, Hv) and beta.shape == (T, Hv) and Hv % Hk == 0
    Tc = np.empty((Hv, dk, dk), dtype=np.float64)
    _load().lkvo_gdn_transition(_p(k), _p(g), _p(beta), T, Hk, Hv, dk, _p(Tc))
    return Tc


def mamba_logdecay(dt, A):
    """Log of the accumulated Mamba-2 scalar decay of one chunk, [H] float64."""
    dt, A = _f64(dt), _f64(A)
    T, H = dt.shape
    lam = np.empty((H,), dtype=np.float64)
    _load().lkvo_mamba_logdecay(_p(dt), _p(A), T, H, _p(lam))
    return lam


def _ids(chunk_ids, K, n_chunks):
    ids = np.arange(K, dtype=np.int32) if chunk_ids is None else np.ascontiguousarray(chunk_ids, dtype=np.int32)
    assert ids.shape == (K,)
    assert K == 0 or (ids.min() >= 0 and ids.max() < n_chunks)
    return ids


def init_exact_gdn(states, transitions, chunk_ids=None, K=None):
    """Exact composition of K cached GDN chunk states in context order.

    states: pool [n, H, dk, dv]; transitions: pool [n, H, dk, dk];
    chunk_ids: the request's K pool indices (None = 0..K-1).
    """
    states, transitions = _f64(states), _f64(transitions)
    n, H, dk, dv = states.shape
    assert transitions.shape == (n, H, dk, dk)
    if K is None:
        K = n if chunk_ids is None else len(chunk_ids)
    ids = _ids(chunk_ids, K, n)
    S0 = np.empty((H, dk, dv), dtype=np.float64)
    _load().lkvo_init_exact_gdn(_p(states), _p(transitions), _p(ids), K, H, dk, dv, _p(S0))
    return S0


def init_exact_mamba(states, logdecay, chunk_ids=None, K=None):
    """Exact composition of K cached Mamba-2 chunk states in context order.

    states: pool [n, H, N, P]; logdecay: pool [n, H].
    """
    states, logdecay = _f64(states), _f64(logdecay)
    n, H, N, P = states.shape
    assert logdecay.shape == (n, H)
    if K is None:
        K = n if chunk_ids is None else len(chunk_ids)
    ids = _ids(chunk_ids, K, n)
    S0 = np.empty((H, N, P), dtype=np.float64)
    _load().lkvo_init_exact_mamba(_p(states), _p(logdecay), _p(ids), K, H, N, P, _p(S0))
    return S0


def init_single(states, chunk_ids=None, K=None, b=None):
    """Single-block initialiser: a copy of the stored state of block b.

    ``b`` is a position in the request (0-based); None selects the last block.
    The stored values are returned untouched, in the pool's own dtype, so the
    comparison with the library can be bitwise.  Returns (S0, pool index used).
    """
    states = np.asarray(states)
    n = states.shape[0]
    if K is None:
        K = n if chunk_ids is None else len(chunk_ids)
    ids = _ids(chunk_ids, K, n)
    if K == 0:
        return np.zeros(states.shape[1:], dtype=states.dtype), -1
    if b is None:
        b = K - 1
    assert 0 <= b < K
    return states[ids[b]].copy(), int(ids[b])


def state_rel_error(S_init, S_ref, n_states=None):
    """Relative error of constructed states against reference states, one number per state:
    ||S_init_i - S_ref_i|| / ||S_ref_i|| in the Frobenius norm (Section 3.2, "Diagnosis via relative error").

    The arrays are split into ``n_states`` equal parts along the flattened leading order (default: the
    leading axis).  A zero reference gives inf, or nan when the constructed state is zero too.
    """
    a, r = _f64(S_init), _f64(S_ref)
    assert a.shape == r.shape
    n = a.shape[0] if n_states is None else int(n_states)
    a, r = a.reshape(n, -1), r.reshape(n, -1)
    with np.errstate(divide="ignore", invalid="ignore"):
        return np.sqrt(((a - r) ** 2).sum(axis=1)) / np.sqrt((r ** 2).sum(axis=1))

