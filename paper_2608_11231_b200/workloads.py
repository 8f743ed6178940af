"""Seeded synthetic inputs shaped like the paper's 8K-32K hybrid workloads.

This module only draws random numbers and shapes them; it holds none of the
method's arithmetic (no recurrence, no composition).  The tests hand the same
arrays to the CPU oracle and to the CUDA library, and the benchmark uses them
as stand-ins for real activations, which are not available offline.

All arrays are float32 numpy arrays whose values are already rounded to the
I/O dtype they will be fed in (bf16 values are exactly representable in fp32),
so both sides of a parity test see identical numbers.

Draw order is fixed: for a GDN chunk q, k, v, beta-logits, g-logits; for a
Mamba-2 chunk x, dt-logits, B, C (A is drawn once per layer before any chunk).
"""
from __future__ import annotations

import numpy as np

# The five benchmark configurations (shapes only; distributions are in the
# generator functions below).
CONFIGS = {
    0: dict(family="gdn", io="f32", H_k=2, H_v=2, d_k=64, d_v=64, K=4, chunk_len=256, suffix=64, seed=0),
    1: dict(family="mamba2", io="bf16", H=80, P=64, N=128, G=1, K=8, chunk_len=1024, suffix=1024, seed=1),
    2: dict(family="gdn", io="bf16", H_k=16, H_v=32, d_k=128, d_v=128, K=16, chunk_len=1024, suffix=0, seed=2),
    3: dict(family="gdn", io="bf16", H_k=16, H_v=32, d_k=128, d_v=128, K=32, chunk_len=1024, suffix=2048,
            n_req=8, seed=3),
    4: dict(family="mixed", io="bf16", n_req=64, K_lo=2, K_hi=32, len_lo=256, len_hi=2048,
            total_lo=8192, total_hi=32768, recompute_ratio=0.2, seed=4),
}


def bf16_round(a) -> np.ndarray:
    """Round to the nearest bfloat16 (ties to even); result is float32."""
    x = np.ascontiguousarray(a, dtype=np.float32)
    u = x.view(np.uint32)
    u = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) & np.uint32(0xFFFF0000)
    return u.view(np.float32).reshape(x.shape)


def _io_round(a, io: str) -> np.ndarray:
    a32 = np.asarray(a, dtype=np.float32)
    return bf16_round(a32) if io == "bf16" else np.ascontiguousarray(a32)


def _softplus(z):
    return np.logaddexp(0.0, z)


def _sigmoid(z):
    return 1.0 / (1.0 + np.exp(-z))


def gdn_tokens(rng, T, H_k, H_v, d_k, d_v, io="bf16", live_chunk_len=None):
    """T tokens of post-convolution GDN layer inputs.

    q, k ~ N(0,1) then L2-normalised per (token, head); v ~ N(0,1);
    beta = sigmoid(N(0,1)); g = -0.1 * softplus(N(0,1)).
    ``live_chunk_len`` = L switches to the weak-decay variant
    (g * 4 / L, beta / 8) in which states carried across a cache chunk of L
    tokens stay well inside fp32 range, so that composition is observable.
    """
    q = rng.standard_normal((T, H_k, d_k), dtype=np.float32)
    k = rng.standard_normal((T, H_k, d_k), dtype=np.float32)
    v = rng.standard_normal((T, H_v, d_v), dtype=np.float32)
    b_logit = rng.standard_normal((T, H_v))
    g_logit = rng.standard_normal((T, H_v))
    q /= np.linalg.norm(q, axis=-1, keepdims=True)
    k /= np.linalg.norm(k, axis=-1, keepdims=True)
    beta = _sigmoid(b_logit)
    g = -0.1 * _softplus(g_logit)
    if live_chunk_len is not None:
        g = g * (4.0 / float(live_chunk_len))
        beta = beta / 8.0
    return dict(
        q=_io_round(q, io), k=_io_round(k, io), v=_io_round(v, io),
        g=np.ascontiguousarray(g, dtype=np.float32), beta=np.ascontiguousarray(beta, dtype=np.float32),
    )


def ssd_A(rng, H, live_chunk_len=None):
    """Per-head A = -exp(U(0,2)); the live variant scales it by 4 / L."""
    A = -np.exp(rng.uniform(0.0, 2.0, size=(H,)))
    if live_chunk_len is not None:
        A = A * (4.0 / float(live_chunk_len))
    return np.ascontiguousarray(A, dtype=np.float32)


def ssd_tokens(rng, T, H, P, N, G, io="bf16"):
    """T tokens of post-convolution Mamba-2 inputs.

    x ~ N(0,1); dt = softplus(N(-2, sd 0.5)) (already activated);
    B, C ~ N(0,1) / sqrt(N).
    """
    x = rng.standard_normal((T, H, P), dtype=np.float32)
    dt = _softplus(-2.0 + 0.5 * rng.standard_normal((T, H)))
    B = rng.standard_normal((T, G, N), dtype=np.float32) / np.float32(np.sqrt(N))
    C = rng.standard_normal((T, G, N), dtype=np.float32) / np.float32(np.sqrt(N))
    return dict(x=_io_round(x, io), dt=np.ascontiguousarray(dt, dtype=np.float32),
                B=_io_round(B, io), C=_io_round(C, io))


def synthetic_states(rng, n, H, d_k, d_v):
    """A pool of stand-in cached states, N(0,1) fp32, [n, H, d_k, d_v]."""
    return rng.standard_normal((n, H, d_k, d_v), dtype=np.float32)


def synthetic_gdn_transitions(rng, n, H, d_k, rho_lo=0.9, rho_hi=1.0):
    """Stand-in chunk transitions rho * Q with Q random orthogonal, [n, H, d_k, d_k] fp32.

    Every chunk keeps most of what it is handed and the matrices do not commute,
    so a composition that drops, reorders or transposes a factor is visible.
    """
    out = np.empty((n, H, d_k, d_k), dtype=np.float32)
    for c in range(n):
        for h in range(H):
            qm, r = np.linalg.qr(rng.standard_normal((d_k, d_k)))
            qm = qm * np.sign(np.diag(r))
            out[c, h] = (rng.uniform(rho_lo, rho_hi) * qm).astype(np.float32)
    return out


def cheap_gdn_transitions(rng, n, H, d_k, gain=0.45):
    """Large pools for timing only: i.i.d. N(0, gain^2 / d_k) entries (spectral radius about 2*gain)."""
    t = rng.standard_normal((n, H, d_k, d_k), dtype=np.float32)
    t *= np.float32(gain / np.sqrt(d_k))
    return t


def synthetic_logdecay(rng, n, H, lo=-2.0, hi=0.0):
    """Stand-in Mamba-2 chunk log-decays, U(lo, hi) fp32, [n, H]."""
    return rng.uniform(lo, hi, size=(n, H)).astype(np.float32)


def request_permutation(seed, r, K):
    """Chunk order of request r over a shared pool of K chunks (request 0 = context order)."""
    if r == 0:
        return np.arange(K, dtype=np.int32)
    return np.random.default_rng(seed * 1000 + r).permutation(K).astype(np.int32)


def ragged_mix(seed=4, n_req=64, K_lo=2, K_hi=32, len_lo=256, len_hi=2048,
               total_lo=8192, total_hi=32768, recompute_ratio=0.2):
    """The ragged serving mix: per request a family, chunk lengths and a recompute length.

    K ~ U{K_lo..K_hi}, chunk lengths ~ U{len_lo..len_hi}, redrawn until the
    total lies in [total_lo, total_hi]; the first half of the requests are
    Mamba-2 layers, the second half GDN layers; each request recomputes
    round(ratio * total) tokens.
    """
    rng = np.random.default_rng(seed)
    reqs = []
    for r in range(n_req):
        while True:
            K = int(rng.integers(K_lo, K_hi + 1))
            lens = rng.integers(len_lo, len_hi + 1, size=K).astype(np.int64)
            total = int(lens.sum())
            if total_lo <= total <= total_hi:
                break
        reqs.append(dict(index=r, family="mamba2" if r < n_req // 2 else "gdn", K=K,
                         chunk_lens=lens, total=total, recompute=int(round(recompute_ratio * total))))
    return reqs
