"""Parity of the CUDA library (through the C ABI) against the fp64 oracle on seeded inputs.

Bars: bit-exact for the single-state copy and the K = 1 identity; max-norm relative error
<= 1e-4 on fp32 paths and <= 2e-2 with bf16 I/O (fp32 accumulation, fp32 state).
"""
import numpy as np
import pytest

import oracle
from helpers import (TOL_BF16, TOL_F32, cat_tokens, dev, gdn_pool_from_tokens, host, mamba_pool_from_tokens, maxrel)
from paper_2608_11231_b200 import binding as b
from paper_2608_11231_b200 import workloads as wl

pytestmark = pytest.mark.gpu

COMPUTES = [b.LKV_COMPUTE_FP32, b.LKV_COMPUTE_AUTO]


def _torch():
    import torch
    return torch


# ------------------------------------------------------------------ single-state init

@pytest.mark.parametrize("family", [b.LKV_FAMILY_GDN, b.LKV_FAMILY_MAMBA2])
@pytest.mark.parametrize("pool_bf16", [False, True])
def test_single_state_is_a_bitwise_copy(family, pool_bf16):
    torch = _torch()
    rng = np.random.default_rng(7)
    n, H, dk, dv = 6, 3, 32, 64
    pool = wl.synthetic_states(rng, n, H, dk, dv)
    if pool_bf16:
        pool = wl.bf16_round(pool)
    pool_t = dev(pool, torch.bfloat16 if pool_bf16 else None)
    ids = np.array([4, 1, 1, 5, 0], dtype=np.int32)
    last = b.lkv_init_state(pool_t, None, 5, b.LKV_INIT_LAST, family=family, chunk_ids=ids)
    ref, idx = oracle.init_single(pool, ids)
    assert idx == 0 and last.cpu().numpy().tobytes() == ref.tobytes()
    for pos in range(5):
        got = b.lkv_init_state(pool_t, None, 5, b.LKV_INIT_INDEX, family=family, chunk_ids=ids, sel_index=pos)
        ref, idx = oracle.init_single(pool, ids, b=pos)
        assert idx == ids[pos] and got.cpu().numpy().tobytes() == ref.tobytes()
    # implicit ids 0..K-1, K smaller than the pool
    got = b.lkv_init_state(pool_t, None, 3, b.LKV_INIT_LAST, family=family)
    assert got.cpu().numpy().tobytes() == pool[2].tobytes()
    # K = 0: empty state
    assert not b.lkv_init_state(pool_t, None, 0, b.LKV_INIT_LAST, family=family).any().item()
    assert not b.lkv_init_state(pool_t, None, 0, b.LKV_INIT_EXACT, family=family).any().item()


def test_single_state_batched_random_block():
    """The random-block control: a seeded position per request, passed by the caller."""
    rng = np.random.default_rng(11)
    n, H, dk, dv = 9, 2, 16, 32
    pool = wl.synthetic_states(rng, n, H, dk, dv)
    ks = [3, 0, 9, 1, 5]
    cu = np.concatenate([[0], np.cumsum(ks)]).astype(np.int32)
    ids = np.concatenate([rng.integers(0, n, size=k) for k in ks]).astype(np.int32)
    sel = np.array([rng.integers(0, k) if k else 0 for k in ks], dtype=np.int32)
    got = b.lkv_init_state_batched(dev(pool), None, ids, cu, len(ks), b.LKV_INIT_INDEX, sel,
                                   family=b.LKV_FAMILY_GDN).cpu().numpy()
    last = b.lkv_init_state_batched(dev(pool), None, ids, cu, len(ks), b.LKV_INIT_LAST, None,
                                    family=b.LKV_FAMILY_GDN).cpu().numpy()
    for r, k in enumerate(ks):
        rid = ids[cu[r]:cu[r + 1]]
        ref, _ = oracle.init_single(pool, rid, b=int(sel[r]) if k else None)
        assert got[r].tobytes() == ref.tobytes()
        ref, _ = oracle.init_single(pool, rid)
        assert last[r].tobytes() == ref.tobytes()


# ------------------------------------------------------------------ Mamba-2 exact composition

def _carried(S0, S0_ref, last):
    """Error of the part of S0 that was carried across chunk boundaries, and its share of S0."""
    c_ref = np.asarray(S0_ref, np.float64) - last
    c = np.asarray(S0, np.float64) - last
    share = np.abs(c_ref).max() / np.abs(S0_ref).max()
    return maxrel(c, c_ref), share


@pytest.mark.parametrize("N", [32, 128])     # 128 x 64: heads are whole 16 KB tiles, the streaming kernel runs
@pytest.mark.parametrize("pool_bf16", [False, True])
def test_mamba_exact_synthetic_transitions(pool_bf16, N):
    torch = _torch()
    rng = np.random.default_rng(3)
    n, H, P = 12, 5, 64
    pool = wl.synthetic_states(rng, n, H, N, P)
    if pool_bf16:
        pool = wl.bf16_round(pool)
    lam = wl.synthetic_logdecay(rng, n, H)
    pool_t, lam_t = dev(pool, torch.bfloat16 if pool_bf16 else None), dev(lam)
    for K in (1, 2, 7, 9, 12, 20):
        ids = rng.integers(0, n, size=K).astype(np.int32)
        got = b.lkv_init_state(pool_t, lam_t, K, b.LKV_INIT_EXACT, family=b.LKV_FAMILY_MAMBA2, chunk_ids=ids)
        ref = oracle.init_exact_mamba(pool, lam, ids)
        assert maxrel(host(got), ref) <= 1e-5
        if K == 1:
            assert host(got).tobytes() == pool[ids[0]].astype(np.float32).tobytes()
        else:
            err, share = _carried(host(got), ref, pool[ids[-1]].astype(np.float64))
            assert share > 0.05 and err <= 1e-4


def test_mamba_exact_batched_ragged_and_limits():
    rng = np.random.default_rng(5)
    n, H, N, P = 40, 4, 16, 32
    pool = wl.synthetic_states(rng, n, H, N, P)
    lam = wl.synthetic_logdecay(rng, n, H)
    lam[3] = 0.0          # identity transition
    lam[4] = -800.0       # underflows exp(): everything before chunk 4 is forgotten
    ks = [5, 1, 0, 32, 2, 17]
    cu = np.concatenate([[0], np.cumsum(ks)]).astype(np.int32)
    ids = np.concatenate([rng.integers(0, n, size=k) for k in ks]).astype(np.int32)
    ids[0:5] = [7, 8, 3, 3, 9]
    ids[cu[4]:cu[5]] = [6, 4]
    got = host(b.lkv_init_state_batched(dev(pool), dev(lam), ids, cu, len(ks), b.LKV_INIT_EXACT, None,
                                        family=b.LKV_FAMILY_MAMBA2))
    for r, k in enumerate(ks):
        ref = oracle.init_exact_mamba(pool, lam, ids[cu[r]:cu[r + 1]])
        assert maxrel(got[r], ref) <= 1e-5, (r, k)
    assert got[4].tobytes() == pool[4].tobytes()      # zero transition: exactly the last block
    assert not got[2].any()


def test_mamba_exact_from_tokens_equals_sequential_pass():
    """Eq. 6 end to end: states cached per chunk, composed on the GPU, against one pass over the prefix."""
    rng = np.random.default_rng(1)
    H, P, N, G = 6, 64, 128, 1
    A = wl.ssd_A(rng, H, live_chunk_len=64)
    chunks = [wl.ssd_tokens(rng, L, H, P, N, G) for L in (64, 40, 72, 64)]
    states, lam = mamba_pool_from_tokens(chunks, A)
    got = host(b.lkv_init_state(dev(states), dev(lam), 4, b.LKV_INIT_EXACT, family=b.LKV_FAMILY_MAMBA2))
    cat = cat_tokens(chunks, ["x", "dt", "B", "C"])
    _, S_full = oracle.ssd_seq(cat["x"], cat["dt"], A, cat["B"], cat["C"])
    assert maxrel(got, S_full) <= 1e-5
    err, share = _carried(got, S_full, states[-1].astype(np.float64))
    assert share > 0.05 and err <= 1e-4


# ------------------------------------------------------------------ GDN exact composition

@pytest.mark.parametrize("compute", COMPUTES)
@pytest.mark.parametrize("dims", [(64, 64), (128, 128), (24, 40), (128, 64)])
def test_gdn_exact_synthetic_transitions(dims, compute):
    dk, dv = dims
    rng = np.random.default_rng(dk + dv)
    n, H = 6, 3
    pool = wl.synthetic_states(rng, n, H, dk, dv)
    trans = wl.synthetic_gdn_transitions(rng, n, H, dk)
    tol = TOL_F32 if compute == b.LKV_COMPUTE_FP32 else 2e-3
    for K in (1, 2, 5, 9):
        ids = rng.integers(0, n, size=K).astype(np.int32)
        got = host(b.lkv_init_state(dev(pool), dev(trans), K, b.LKV_INIT_EXACT, family=b.LKV_FAMILY_GDN,
                                    chunk_ids=ids, compute=compute))
        ref = oracle.init_exact_gdn(pool, trans, ids)
        assert maxrel(got, ref) <= tol, (K, maxrel(got, ref))
        if K == 1:
            assert got.tobytes() == pool[ids[0]].tobytes()
        else:
            err, share = _carried(got, ref, pool[ids[-1]].astype(np.float64))
            assert share > 0.2 and err <= 2 * tol


@pytest.mark.parametrize("compute", COMPUTES)
def test_gdn_exact_batched_shared_pool_permutations(compute):
    """Eight requests over one shared pool, each with its own chunk order (chunk reuse at different positions)."""
    rng = np.random.default_rng(33)
    n, H, dk, dv = 8, 2, 128, 128
    pool = wl.synthetic_states(rng, n, H, dk, dv)
    trans = wl.synthetic_gdn_transitions(rng, n, H, dk)
    perms = [wl.request_permutation(3, r, n) for r in range(8)]
    ids = np.concatenate(perms).astype(np.int32)
    cu = (np.arange(9) * n).astype(np.int32)
    got = host(b.lkv_init_state_batched(dev(pool), dev(trans), ids, cu, 8, b.LKV_INIT_EXACT, None,
                                        family=b.LKV_FAMILY_GDN, compute=compute))
    tol = TOL_F32 if compute == b.LKV_COMPUTE_FP32 else 2e-3
    for r in range(8):
        ref = oracle.init_exact_gdn(pool, trans, perms[r])
        assert maxrel(got[r], ref) <= tol, r
    assert maxrel(got[1], got[0]) > 0.1     # order matters: different permutations give different states


def test_gdn_identity_and_zero_transition_limits():
    rng = np.random.default_rng(2)
    n, H, dk, dv = 4, 2, 64, 64
    pool = wl.synthetic_states(rng, n, H, dk, dv)
    eye = np.broadcast_to(np.eye(dk, dtype=np.float32), (n, H, dk, dk)).copy()
    got = host(b.lkv_init_state(dev(pool), dev(eye), n, b.LKV_INIT_EXACT, family=b.LKV_FAMILY_GDN,
                                compute=b.LKV_COMPUTE_FP32))
    assert maxrel(got, pool.astype(np.float64).sum(0)) <= 1e-6
    got = host(b.lkv_init_state(dev(pool), dev(np.zeros_like(eye)), n, b.LKV_INIT_EXACT, family=b.LKV_FAMILY_GDN,
                                compute=b.LKV_COMPUTE_FP32))
    assert got.tobytes() == pool[-1].tobytes()     # exact composition coincides with last-block init


# ------------------------------------------------------------------ scans

def _run_gdn(tok, S0, io, cu=None, compute=b.LKV_COMPUTE_AUTO, scale=0.0):
    torch = _torch()
    dt = torch.bfloat16 if io == "bf16" else None
    o, ST = b.lkv_gdn_fwd(dev(tok["q"], dt), dev(tok["k"], dt), dev(tok["v"], dt), dev(tok["g"]), dev(tok["beta"]),
                          None if S0 is None else dev(S0.astype(np.float32)), cu_seqlens=cu, compute=compute,
                          scale=scale)
    return host(o), host(ST)


def _oracle_gdn_varlen(tok, S0, cu, scale=None):
    outs, finals = [], []
    for s in range(len(cu) - 1):
        sl = slice(cu[s], cu[s + 1])
        o, ST = oracle.gdn_seq(tok["q"][sl], tok["k"][sl], tok["v"][sl], tok["g"][sl], tok["beta"][sl],
                               None if S0 is None else S0[s], scale)
        outs.append(o)
        finals.append(ST)
    return np.concatenate(outs), np.stack(finals)


@pytest.mark.parametrize("compute", COMPUTES)
@pytest.mark.parametrize("shape", [(2, 2, 64, 64, "f32"), (1, 2, 32, 16, "f32"), (2, 4, 128, 128, "f32"),
                                   (2, 4, 128, 128, "bf16"), (1, 1, 64, 128, "bf16")])
def test_gdn_scan_matches_token_recurrence(shape, compute):
    H_k, H_v, dk, dv, io = shape
    rng = np.random.default_rng(H_v * dk + dv)
    lens = [77, 0, 5, 200, 64, 129]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    tok = wl.gdn_tokens(rng, int(cu[-1]), H_k, H_v, dk, dv, io=io, live_chunk_len=64)
    S0 = rng.standard_normal((len(lens), H_v, dk, dv)).astype(np.float32)
    o, ST = _run_gdn(tok, S0, io, cu, compute, scale=0.25)
    o_ref, ST_ref = _oracle_gdn_varlen(tok, S0, cu, 0.25)
    tol = TOL_BF16 if io == "bf16" else TOL_F32
    assert maxrel(o, o_ref) <= tol and maxrel(ST, ST_ref) <= tol, (maxrel(o, o_ref), maxrel(ST, ST_ref))
    for s, L in enumerate(lens):
        if L == 0:
            assert ST[s].tobytes() == S0[s].tobytes()   # an empty sequence hands its state through
    # strongly decaying inputs as the configs draw them, empty start, default scale
    tok2 = wl.gdn_tokens(rng, 300, H_k, H_v, dk, dv, io=io)
    o2, ST2 = _run_gdn(tok2, None, io, None, compute)
    o2_ref, ST2_ref = oracle.gdn_seq(tok2["q"], tok2["k"], tok2["v"], tok2["g"], tok2["beta"])
    assert maxrel(o2, o2_ref) <= tol and maxrel(ST2[0], ST2_ref) <= tol


def _run_ssd(tok, A, S0, io, cu=None, compute=b.LKV_COMPUTE_AUTO):
    torch = _torch()
    dt = torch.bfloat16 if io == "bf16" else None
    y, ST = b.lkv_ssd_fwd(dev(tok["x"], dt), dev(tok["dt"]), dev(A), dev(tok["B"], dt), dev(tok["C"], dt),
                          None if S0 is None else dev(S0.astype(np.float32)), cu_seqlens=cu, compute=compute)
    return host(y), host(ST)


@pytest.mark.parametrize("compute", COMPUTES)
@pytest.mark.parametrize("shape", [(4, 64, 128, 1, "bf16"), (6, 64, 128, 2, "f32"), (3, 32, 16, 1, "f32"),
                                   (2, 128, 64, 2, "bf16")])
def test_ssd_scan_matches_token_recurrence(shape, compute):
    H, P, N, G, io = shape
    rng = np.random.default_rng(H * P + N)
    lens = [130, 0, 3, 257, 64]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    A = wl.ssd_A(rng, H)
    tok = wl.ssd_tokens(rng, int(cu[-1]), H, P, N, G, io=io)
    S0 = rng.standard_normal((len(lens), H, N, P)).astype(np.float32)
    y, ST = _run_ssd(tok, A, S0, io, cu, compute)
    ys, fs = [], []
    for s in range(len(lens)):
        sl = slice(cu[s], cu[s + 1])
        yr, fr = oracle.ssd_seq(tok["x"][sl], tok["dt"][sl], A, tok["B"][sl], tok["C"][sl], S0[s])
        ys.append(yr)
        fs.append(fr)
    tol = TOL_BF16 if io == "bf16" else TOL_F32
    assert maxrel(y, np.concatenate(ys)) <= tol and maxrel(ST, np.stack(fs)) <= tol
    assert ST[1].tobytes() == S0[1].tobytes()
    # weak decay, empty start, single sequence
    A2 = wl.ssd_A(rng, H, live_chunk_len=256)
    tok2 = wl.ssd_tokens(rng, 300, H, P, N, G, io=io)
    y2, ST2 = _run_ssd(tok2, A2, None, io, None, compute)
    y2_ref, ST2_ref = oracle.ssd_seq(tok2["x"], tok2["dt"], A2, tok2["B"], tok2["C"])
    assert maxrel(y2, y2_ref) <= tol and maxrel(ST2[0], ST2_ref) <= tol


def test_scans_are_deterministic_and_state_may_alias():
    torch = _torch()
    rng = np.random.default_rng(9)
    tok = wl.gdn_tokens(rng, 150, 2, 4, 128, 128, io="bf16", live_chunk_len=64)
    S0 = rng.standard_normal((1, 4, 128, 128)).astype(np.float32)
    a = _run_gdn(tok, S0, "bf16")
    c = _run_gdn(tok, S0, "bf16")
    assert a[0].tobytes() == c[0].tobytes() and a[1].tobytes() == c[1].tobytes()
    bf = torch.bfloat16
    S = dev(S0)
    _, ST = b.lkv_gdn_fwd(dev(tok["q"], bf), dev(tok["k"], bf), dev(tok["v"], bf), dev(tok["g"]), dev(tok["beta"]),
                          S, S_T=S)
    assert host(ST).tobytes() == a[1].tobytes()


def test_split_and_chain_equals_one_call():
    rng = np.random.default_rng(10)
    tok = wl.gdn_tokens(rng, 210, 1, 2, 64, 64, io="f32", live_chunk_len=64)
    o_full, ST_full = _run_gdn(tok, None, "f32")
    cut = 83
    a = {n: x[:cut] for n, x in tok.items()}
    c = {n: x[cut:] for n, x in tok.items()}
    o_a, ST_a = _run_gdn(a, None, "f32")
    o_c, ST_c = _run_gdn(c, ST_a, "f32")
    assert maxrel(np.concatenate([o_a, o_c]), o_full) <= 1e-5 and maxrel(ST_c, ST_full) <= 1e-5


# ------------------------------------------------------------------ configuration 0, whole path

def test_config0_whole_path():
    """Tiny GDN layer, fp32: both init modes, then the suffix scanned from S0; tolerance 1e-4.
    Also the paper's identity at this scale: composed state == state of one pass over the prefix."""
    cfg = wl.CONFIGS[0]
    for live in (None, cfg["chunk_len"]):
        rng = np.random.default_rng(cfg["seed"])
        mk = lambda T: wl.gdn_tokens(rng, T, cfg["H_k"], cfg["H_v"], cfg["d_k"], cfg["d_v"], io="f32",
                                     live_chunk_len=live)
        chunks = [mk(cfg["chunk_len"]) for _ in range(cfg["K"])]
        suffix = mk(cfg["suffix"])
        states, trans = gdn_pool_from_tokens(chunks)
        S0_ex = host(b.lkv_init_state(dev(states), dev(trans), cfg["K"], b.LKV_INIT_EXACT, family=b.LKV_FAMILY_GDN))
        S0_lb = host(b.lkv_init_state(dev(states), None, cfg["K"], b.LKV_INIT_LAST, family=b.LKV_FAMILY_GDN))
        assert S0_lb.tobytes() == states[-1].tobytes()
        ref_ex = oracle.init_exact_gdn(states, trans)
        assert maxrel(S0_ex, ref_ex) <= TOL_F32
        if live is not None:
            err, share = _carried(S0_ex, ref_ex, states[-1].astype(np.float64))
            assert share > 0.1 and err <= TOL_F32
        cat = cat_tokens(chunks + [suffix], ["q", "k", "v", "g", "beta"])
        o_all, ST_all = oracle.gdn_seq(cat["q"], cat["k"], cat["v"], cat["g"], cat["beta"])
        for S0 in (S0_ex, S0_lb):
            o, ST = _run_gdn(suffix, S0[None], "f32")
            o_ref, ST_ref = oracle.gdn_seq(suffix["q"], suffix["k"], suffix["v"], suffix["g"], suffix["beta"], S0)
            assert maxrel(o, o_ref) <= TOL_F32 and maxrel(ST[0], ST_ref) <= TOL_F32
        o, ST = _run_gdn(suffix, S0_ex[None], "f32")
        n_pre = cfg["K"] * cfg["chunk_len"]
        assert maxrel(o, o_all[n_pre:]) <= TOL_F32 and maxrel(ST[0], ST_all) <= TOL_F32


def test_batched_init_with_index_list_in_workspace():
    """More chunk ids than fit in the kernel parameters: the list travels through the workspace."""
    rng = np.random.default_rng(21)
    n, H, N, P = 24, 2, 16, 32
    pool = wl.synthetic_states(rng, n, H, N, P)
    lam = wl.synthetic_logdecay(rng, n, H, lo=-0.5)
    n_req, K = 160, 30
    ids = rng.integers(0, n, size=n_req * K).astype(np.int32)
    cu = (np.arange(n_req + 1) * K).astype(np.int32)
    assert ids.size + 2 * n_req + 1 > 4000
    got = host(b.lkv_init_state_batched(dev(pool), dev(lam), ids, cu, n_req, b.LKV_INIT_EXACT, None,
                                        family=b.LKV_FAMILY_MAMBA2))
    for r in (0, 1, 77, n_req - 1):
        assert maxrel(got[r], oracle.init_exact_mamba(pool, lam, ids[cu[r]:cu[r + 1]])) <= 1e-5
    sel = rng.integers(0, K, size=n_req).astype(np.int32)
    got = host(b.lkv_init_state_batched(dev(pool), None, ids, cu, n_req, b.LKV_INIT_INDEX, sel,
                                        family=b.LKV_FAMILY_MAMBA2))
    for r in (0, 5, n_req - 1):
        assert got[r].tobytes() == pool[ids[cu[r] + sel[r]]].tobytes()


def test_gdn_exact_tensor_many_heads_ragged():
    """Enough (request, head) pairs that the tensor-core kernel takes its wide column blocks; ragged K
    including the K = 1 identity and the empty request; the device status word must stay clean."""
    rng = np.random.default_rng(44)
    n, H, dk, dv = 10, 8, 128, 128
    pool = wl.synthetic_states(rng, n, H, dk, dv)
    trans = wl.synthetic_gdn_transitions(rng, n, H, dk)
    ks = [4, 1, 0, 9, 2, 3, 7, 5]
    cu = np.concatenate([[0], np.cumsum(ks)]).astype(np.int32)
    ids = np.concatenate([rng.integers(0, n, size=k) for k in ks]).astype(np.int32)
    ws = _torch().zeros(4096, dtype=_torch().uint8, device="cuda")
    got = host(b.lkv_init_state_batched(dev(pool), dev(trans), ids, cu, len(ks), b.LKV_INIT_EXACT, None,
                                        family=b.LKV_FAMILY_GDN, compute=b.LKV_COMPUTE_TENSOR, workspace_t=ws))
    assert b.lkv_device_status(ws) == b.LKV_OK
    for r, k in enumerate(ks):
        ref = oracle.init_exact_gdn(pool, trans, ids[cu[r]:cu[r + 1]])
        assert maxrel(got[r], ref) <= 2e-3, (r, k, maxrel(got[r], ref))
    assert got[1].tobytes() == pool[ids[cu[1]]].tobytes()
    assert not got[2].any()


def test_scans_with_violent_decay_take_the_exact_exponent_path():
    """Decay so strong that a 16-token group spans more than 2^100: the tensor-core kernels must fall back to
    per-element exponents (the grouped form would overflow) and still match the token recurrence."""
    torch = _torch()
    bf = torch.bfloat16
    rng = np.random.default_rng(77)
    tok = wl.gdn_tokens(rng, 200, 2, 4, 128, 128)
    tok["g"] = (tok["g"] * 80.0).astype(np.float32)            # about -6 per token
    assert (tok["g"].min() * 16 * 1.4427) < -100
    S0 = rng.standard_normal((1, 4, 128, 128)).astype(np.float32)
    o, ST = _run_gdn(tok, S0, "bf16")
    o_ref, ST_ref = oracle.gdn_seq(tok["q"], tok["k"], tok["v"], tok["g"], tok["beta"], S0[0])
    assert maxrel(o, o_ref) <= TOL_BF16 and maxrel(ST[0], ST_ref) <= TOL_BF16
    H, P, N, G = 4, 64, 128, 1
    A = (wl.ssd_A(rng, H) * 12.0).astype(np.float32)          # dt * A about -6 per token and more
    st = wl.ssd_tokens(rng, 300, H, P, N, G)
    assert (st["dt"].max() * A.min() * 16 * 1.4427) < -100
    y, hT = _run_ssd(st, A, rng.standard_normal((1, H, N, P)).astype(np.float32) * 0 + 1.0, "bf16")
    y_ref, hT_ref = oracle.ssd_seq(st["x"], st["dt"], A, st["B"], st["C"], np.ones((H, N, P)))
    assert maxrel(y, y_ref) <= TOL_BF16 and maxrel(hT[0], hT_ref) <= TOL_BF16


def test_scans_with_more_sequences_than_fit_the_parameter_block():
    """1100 short sequences: cu_seqlens no longer fits the kernel parameter block and travels through the
    workspace.  Every sequence's final state and a sample of outputs are checked against the oracle."""
    torch = _torch()
    bf = torch.bfloat16
    rng = np.random.default_rng(31)
    n_seq = 1100
    lens = rng.integers(0, 40, size=n_seq)
    lens[[5, 500, 1099]] = [130, 70, 200]          # a few that span several blocks
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T = int(cu[-1])
    g = wl.gdn_tokens(rng, T, 1, 2, 128, 128)
    o, ST = b.lkv_gdn_fwd(dev(g["q"], bf), dev(g["k"], bf), dev(g["v"], bf), dev(g["g"]), dev(g["beta"]), cu_seqlens=cu)
    o, ST = host(o), host(ST)
    m = wl.ssd_tokens(rng, T, 2, 64, 128, 1)
    A = wl.ssd_A(rng, 2)
    y, MT = b.lkv_ssd_fwd(dev(m["x"], bf), dev(m["dt"]), dev(A), dev(m["B"], bf), dev(m["C"], bf), cu_seqlens=cu)
    y, MT = host(y), host(MT)
    for s in [0, 5, 499, 500, 777, 1098, 1099] + list(rng.integers(0, n_seq, size=8)):
        a0, a1 = int(cu[s]), int(cu[s + 1])
        if a1 == a0:
            assert not ST[s].any() and not MT[s].any()
            continue
        o_ref, S_ref = oracle.gdn_seq(*[g[n][a0:a1] for n in ("q", "k", "v", "g", "beta")])
        assert maxrel(o[a0:a1], o_ref) <= TOL_BF16 and maxrel(ST[s], S_ref) <= TOL_BF16
        y_ref, M_ref = oracle.ssd_seq(m["x"][a0:a1], m["dt"][a0:a1], A, m["B"][a0:a1], m["C"][a0:a1])
        assert maxrel(y[a0:a1], y_ref) <= TOL_BF16 and maxrel(MT[s], M_ref) <= TOL_BF16


@pytest.mark.parametrize("compute", COMPUTES)
def test_gdn_exact_with_bf16_stored_states(compute):
    """Cached states stored as bf16 (the paper's storage format), fp32 transitions, fp32 result: single request and
    ragged batch, tensor-core and fp32 paths; K = 1 hands the stored values through exactly."""
    torch = _torch()
    rng = np.random.default_rng(41)
    n, H, d = 10, 3, 128
    pool = wl.bf16_round(wl.synthetic_states(rng, n, H, d, d))
    trans = wl.synthetic_gdn_transitions(rng, n, H, d)
    pool_t, trans_t = dev(pool, torch.bfloat16), dev(trans)
    tol = TOL_F32 if compute == b.LKV_COMPUTE_FP32 else 2e-3
    for K in (1, 2, 7):
        ids = rng.integers(0, n, size=K).astype(np.int32)
        got = host(b.lkv_init_state(pool_t, trans_t, K, b.LKV_INIT_EXACT, family=b.LKV_FAMILY_GDN, chunk_ids=ids,
                                    compute=compute))
        ref = oracle.init_exact_gdn(pool, trans, ids)
        assert maxrel(got, ref) <= tol, (K, maxrel(got, ref))
        if K == 1:
            assert got.tobytes() == pool[ids[0]].astype(np.float32).tobytes()
    ks = [3, 0, 1, 6]
    cu = np.concatenate([[0], np.cumsum(ks)]).astype(np.int32)
    ids = rng.integers(0, n, size=int(cu[-1])).astype(np.int32)
    got = host(b.lkv_init_state_batched(pool_t, trans_t, ids, cu, len(ks), b.LKV_INIT_EXACT, None,
                                        family=b.LKV_FAMILY_GDN, compute=compute))
    for r, K in enumerate(ks):
        if K == 0:
            assert not got[r].any()
        else:
            assert maxrel(got[r], oracle.init_exact_gdn(pool, trans, ids[cu[r]:cu[r + 1]])) <= tol, r
