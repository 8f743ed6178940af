"""Shared test helpers: error metrics, tensor conversion, oracle-built cache pools."""
from __future__ import annotations

import numpy as np

import oracle
from paper_2608_11231_b200 import workloads as wl

# Tolerances: fp32 paths (fp32 I/O, fp32 FMA); bf16 I/O with fp32 accumulation and fp32 state.
TOL_F32 = 1e-4
TOL_BF16 = 2e-2


# every maxrel() value of the running test, in call order (conftest.py writes them out on request)
ERRORS: list = []


def maxrel(x, ref) -> float:
    """max |x - ref| / max |ref| over one tensor (elementwise-relative is undefined at zeros)."""
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.abs(ref).max()
    err = float(np.abs(x).max()) if den == 0.0 else float(np.abs(x - ref).max() / den)
    ERRORS.append(err)
    return err


def maxrel_per_head(x, ref, head_axis: int) -> float:
    """The worst head's own max-norm relative error: max over h of max|x - ref|_h / max|ref|_h.

    A head (or a head of one sequence, with the sequences split by the caller) whose values are small cannot
    hide behind a large one, as it can in maxrel() over the whole tensor.
    """
    x = np.moveaxis(np.asarray(x, dtype=np.float64), head_axis, 0)
    ref = np.moveaxis(np.asarray(ref, dtype=np.float64), head_axis, 0)
    worst = 0.0
    for xh, rh in zip(x, ref):
        den = np.abs(rh).max()
        worst = max(worst, float(np.abs(xh).max()) if den == 0.0 else float(np.abs(xh - rh).max() / den))
    ERRORS.append(worst)
    return worst


def frobrel(x, ref) -> float:
    x = np.asarray(x, dtype=np.float64)
    ref = np.asarray(ref, dtype=np.float64)
    den = np.linalg.norm(ref)
    return float(np.linalg.norm(x - ref) / den) if den else float(np.linalg.norm(x))


def dev(a, dtype=None):
    """numpy float32 array -> CUDA tensor (values already representable in the target dtype)."""
    import torch
    t = torch.from_numpy(np.ascontiguousarray(a)).cuda()
    return t if dtype is None else t.to(dtype)


def host(t):
    import torch
    return t.detach().to(torch.float32).cpu().numpy()


def gdn_pool_from_tokens(chunks):
    """Cached artefacts of GDN chunks, built by the oracle from raw tokens and stored as fp32.

    Each chunk is scanned from the empty state to get its local state and its accumulated
    transition.  Storage rounding (fp32) happens here, before either side composes.
    """
    states = np.stack([oracle.gdn_seq(c["q"], c["k"], c["v"], c["g"], c["beta"])[1] for c in chunks])
    trans = np.stack([oracle.gdn_transition(c["k"], c["g"], c["beta"]) for c in chunks])
    return states.astype(np.float32), trans.astype(np.float32)


def mamba_pool_from_tokens(chunks, A):
    states = np.stack([oracle.ssd_seq(c["x"], c["dt"], A, c["B"], c["C"])[1] for c in chunks])
    lam = np.stack([oracle.mamba_logdecay(c["dt"], A) for c in chunks])
    return states.astype(np.float32), lam.astype(np.float32)


def slice_gdn_heads(tok, v_heads, H_k, H_v):
    """Restrict GDN tokens to a set of value heads whose q/k heads are kept once each, in order.

    v_heads must cover whole groups (all value heads of each q/k head they touch).
    """
    rep = H_v // H_k
    k_heads = sorted({h // rep for h in v_heads})
    assert list(v_heads) == [kh * rep + i for kh in k_heads for i in range(rep)]
    return dict(q=tok["q"][:, k_heads], k=tok["k"][:, k_heads], v=tok["v"][:, list(v_heads)],
                g=tok["g"][:, list(v_heads)], beta=tok["beta"][:, list(v_heads)])


def cat_tokens(chunks, keys):
    return {n: np.concatenate([c[n] for c in chunks], axis=0) for n in keys}
