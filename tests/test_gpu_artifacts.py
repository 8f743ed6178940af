"""Producers of the cached artefacts (chunk transitions, log-decays, final-state-only scans) against the oracle,
and the whole cache-building pipeline on the GPU: chunk tokens -> (S_local, T_C) -> exact composition, which must
equal one sequential pass of the oracle over the concatenated prefix (Eq. 5, Eq. 6)."""
import numpy as np
import pytest

import oracle
from helpers import TOL_BF16, TOL_F32, dev, host, maxrel
from paper_2608_11231_b200 import binding as b
from paper_2608_11231_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _t():
    import torch
    return torch


def _cat(chunks, names):
    return {n: np.concatenate([c[n] for c in chunks]) for n in names}


@pytest.mark.parametrize("shape", [
    dict(H_k=2, H_v=4, d=64, io="f32", lens=[70, 0, 33, 128], tol=TOL_F32),
    dict(H_k=2, H_v=4, d=128, io="bf16", lens=[200, 64, 0, 131], tol=TOL_BF16),
    dict(H_k=1, H_v=2, d=128, io="bf16", lens=[1024], tol=TOL_BF16),
])
@pytest.mark.parametrize("live", [False, True])
def test_gdn_chunk_transition_matches_oracle(shape, live):
    torch = _t()
    H_k, H_v, d, io = shape["H_k"], shape["H_v"], shape["d"], shape["io"]
    rng = np.random.default_rng(11)
    chunks = [wl.gdn_tokens(rng, L, H_k, H_v, d, d, io=io, live_chunk_len=256 if live else None) for L in shape["lens"]]
    cat = _cat(chunks, ("k", "g", "beta"))
    cu = np.concatenate([[0], np.cumsum(shape["lens"])]).astype(np.int32)
    dt = torch.bfloat16 if io == "bf16" else None
    T = host(b.lkv_gdn_chunk_transition(dev(cat["k"], dt), dev(cat["g"]), dev(cat["beta"]), cu_seqlens=cu))
    assert T.shape == (len(chunks), H_v, d, d)
    for c, ch in enumerate(chunks):
        if len(ch["k"]) == 0:
            assert T[c].tobytes() == np.broadcast_to(np.eye(d, dtype=np.float32), (H_v, d, d)).tobytes()
            continue
        ref = oracle.gdn_transition(ch["k"], ch["g"], ch["beta"])
        assert maxrel(T[c], ref) <= shape["tol"], (c, maxrel(T[c], ref))


def test_mamba_chunk_logdecay_matches_oracle():
    rng = np.random.default_rng(12)
    H, lens = 80, [1024, 0, 77, 300]
    A = wl.ssd_A(rng, H)
    dts = [wl.ssd_tokens(rng, L, H, 8, 16, 1, io="f32")["dt"] for L in lens]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    lam = host(b.lkv_mamba_chunk_logdecay(dev(np.concatenate(dts)), dev(A), cu_seqlens=cu))
    assert lam.shape == (len(lens), H)
    for c, d in enumerate(dts):
        ref = oracle.mamba_logdecay(d, A) if len(d) else np.zeros(H)
        assert np.abs(lam[c] - ref).max() <= 1e-5 * max(1.0, np.abs(ref).max())


def test_final_state_only_scans_equal_full_scans():
    torch = _t()
    bf = torch.bfloat16
    rng = np.random.default_rng(13)
    lens = [300, 64, 129]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    g = wl.gdn_tokens(rng, sum(lens), 2, 4, 128, 128)
    args = (dev(g["q"], bf), dev(g["k"], bf), dev(g["v"], bf), dev(g["g"]), dev(g["beta"]))
    o, ST = b.lkv_gdn_fwd(*args, cu_seqlens=cu)
    o2, ST2 = b.lkv_gdn_fwd(*args, cu_seqlens=cu, want_outputs=False)
    assert o2 is None and host(ST2).tobytes() == host(ST).tobytes()
    m = wl.ssd_tokens(rng, sum(lens), 8, 64, 128, 1)
    A = wl.ssd_A(rng, 8)
    margs = (dev(m["x"], bf), dev(m["dt"]), dev(A), dev(m["B"], bf), dev(m["C"], bf))
    y, MT = b.lkv_ssd_fwd(*margs, cu_seqlens=cu)
    y2, MT2 = b.lkv_ssd_fwd(*margs, cu_seqlens=cu, want_outputs=False)
    assert y2 is None and host(MT2).tobytes() == host(MT).tobytes()


def test_cache_building_pipeline_gdn_reproduces_the_full_prefix_state():
    """Artefacts made by the library from raw chunk tokens, composed by the library, against one oracle pass."""
    torch = _t()
    bf = torch.bfloat16
    H_k, H_v, d, lens = 2, 4, 128, [256, 192, 320, 256]
    rng = np.random.default_rng(14)
    chunks = [wl.gdn_tokens(rng, L, H_k, H_v, d, d, live_chunk_len=256) for L in lens]
    cat = _cat(chunks, ("q", "k", "v", "g", "beta"))
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    q, k, v, g, beta = dev(cat["q"], bf), dev(cat["k"], bf), dev(cat["v"], bf), dev(cat["g"]), dev(cat["beta"])
    _, states = b.lkv_gdn_fwd(q, k, v, g, beta, cu_seqlens=cu, want_outputs=False)      # S_local of every chunk
    trans = b.lkv_gdn_chunk_transition(k, g, beta, cu_seqlens=cu)                        # T_C of every chunk
    S0 = host(b.lkv_init_state(states, trans, len(lens), b.LKV_INIT_EXACT, family=b.LKV_FAMILY_GDN))
    _, S_ref = oracle.gdn_seq(cat["q"], cat["k"], cat["v"], cat["g"], cat["beta"])
    assert maxrel(S0, S_ref) <= TOL_BF16, maxrel(S0, S_ref)
    # the carried part (everything but the last chunk's own state) is what composition adds
    last = host(states)[-1].astype(np.float64)
    carried_ref = S_ref - oracle.gdn_seq(*[chunks[-1][n] for n in ("q", "k", "v", "g", "beta")])[1]
    assert np.abs(carried_ref).max() > 0.05 * np.abs(S_ref).max()
    assert maxrel(S0 - last, carried_ref) <= 2 * TOL_BF16


def test_cache_building_pipeline_mamba_reproduces_the_full_prefix_state():
    torch = _t()
    bf = torch.bfloat16
    H, P, N, lens = 8, 64, 128, [256, 128, 384]
    rng = np.random.default_rng(15)
    A = wl.ssd_A(rng, H, live_chunk_len=256)
    chunks = [wl.ssd_tokens(rng, L, H, P, N, 1) for L in lens]
    cat = _cat(chunks, ("x", "dt", "B", "C"))
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    x, dt, Bm, Cm = dev(cat["x"], bf), dev(cat["dt"]), dev(cat["B"], bf), dev(cat["C"], bf)
    _, states = b.lkv_ssd_fwd(x, dt, dev(A), Bm, Cm, cu_seqlens=cu, want_outputs=False)
    lam = b.lkv_mamba_chunk_logdecay(dt, dev(A), cu_seqlens=cu)
    S0 = host(b.lkv_init_state(states, lam, len(lens), b.LKV_INIT_EXACT, family=b.LKV_FAMILY_MAMBA2))
    _, S_ref = oracle.ssd_seq(cat["x"], cat["dt"], A, cat["B"], cat["C"])
    assert maxrel(S0, S_ref) <= TOL_BF16, maxrel(S0, S_ref)


@pytest.mark.parametrize("n,shape", [(5, (2, 64, 64)), (3, (32, 128, 128)), (1, (4,))])
def test_state_rel_error_matches_oracle(n, shape):
    rng = np.random.default_rng(16)
    ref = rng.standard_normal((n,) + shape).astype(np.float32)
    init = (ref + 0.01 * rng.standard_normal(ref.shape)).astype(np.float32)
    init[0] = ref[0]                                   # exact -> 0
    if n > 1:
        init[1] = 0.0                                  # empty-state initialiser -> 1
    err = host(b.lkv_state_rel_error(dev(init), dev(ref)))
    want = oracle.state_rel_error(init, ref)
    assert err[0] == 0.0
    assert np.abs(err - want).max() <= 1e-5 * max(1.0, want.max())
    # whole layer as one state, and per head
    one = host(b.lkv_state_rel_error(dev(init), dev(ref), n_states=1))
    assert abs(one[0] - oracle.state_rel_error(init, ref, n_states=1)[0]) <= 1e-5
    if len(shape) == 3:
        per_head = host(b.lkv_state_rel_error(dev(init), dev(ref), n_states=n * shape[0]))
        assert np.abs(per_head - oracle.state_rel_error(init, ref, n_states=n * shape[0])).max() <= 1e-5


def test_state_rel_error_of_the_two_initialisers():
    """The paper's diagnostic on the library's own initialisers: exact composition sits at the rounding floor,
    the last-block state differs from the full-prefix state by the carried part."""
    torch = _t()
    bf = torch.bfloat16
    H_k, H_v, d, lens = 2, 4, 128, [256, 256, 256]
    rng = np.random.default_rng(17)
    chunks = [wl.gdn_tokens(rng, L, H_k, H_v, d, d, live_chunk_len=256) for L in lens]
    cat = _cat(chunks, ("q", "k", "v", "g", "beta"))
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    q, k, v, g, beta = dev(cat["q"], bf), dev(cat["k"], bf), dev(cat["v"], bf), dev(cat["g"]), dev(cat["beta"])
    _, states = b.lkv_gdn_fwd(q, k, v, g, beta, cu_seqlens=cu, want_outputs=False)
    trans = b.lkv_gdn_chunk_transition(k, g, beta, cu_seqlens=cu)
    S_ex = b.lkv_init_state(states, trans, 3, b.LKV_INIT_EXACT, family=b.LKV_FAMILY_GDN)
    S_lb = b.lkv_init_state(states, None, 3, b.LKV_INIT_LAST, family=b.LKV_FAMILY_GDN)
    S_star = dev(oracle.gdn_seq(cat["q"], cat["k"], cat["v"], cat["g"], cat["beta"])[1].astype(np.float32))
    e_ex = host(b.lkv_state_rel_error(S_ex, S_star, n_states=1))[0]
    e_lb = host(b.lkv_state_rel_error(S_lb, S_star, n_states=1))[0]
    assert e_ex <= 2e-2 and e_lb > 5 * e_ex



def test_online_fold_equals_exact_composition_and_one_pass():
    """Eq. 6 without materialised transitions: S <- scan_{v=0}(chunk j's keys and gates; from S) + S_j.
    Equals the composition over materialised transitions and, by the paper's identity, the state of one pass over
    the concatenated prefix."""
    import torch
    from helpers import TOL_BF16, dev, host, maxrel
    rng = np.random.default_rng(41)
    H_k, H_v, d = 2, 4, 128
    lens = [200, 64, 0, 131, 77]                      # cached chunks in pool order (one of them empty)
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    tok = wl.gdn_tokens(rng, int(cu[-1]), H_k, H_v, d, d, io="bf16", live_chunk_len=128)
    bf = torch.bfloat16
    k, g, beta = dev(tok["k"], bf), dev(tok["g"]), dev(tok["beta"])
    # the cache as the library builds it: local states (scan from the empty state) and transitions, fp32
    _, states = b.lkv_gdn_fwd(dev(tok["q"], bf), k, dev(tok["v"], bf), g, beta, cu_seqlens=cu, want_outputs=False)
    trans = b.lkv_gdn_chunk_transition(k, g, beta, cu_seqlens=cu)
    ids = np.array([3, 0, 2, 4, 1], dtype=np.int32)   # a request that uses the chunks in another order
    for compute in (b.LKV_COMPUTE_AUTO, b.LKV_COMPUTE_FP32):
        S_fold = b.lkv_init_state_fold(states, k, g, beta, cu, len(ids), ids, compute=compute)
        S_mat = b.lkv_init_state(states, trans, len(ids), b.LKV_INIT_EXACT, family=b.LKV_FAMILY_GDN, chunk_ids=ids)
        assert maxrel(host(S_fold), host(S_mat)) <= TOL_BF16
        # one pass of the oracle over the chunks' tokens in request order
        order = np.concatenate([np.arange(cu[c], cu[c + 1]) for c in ids])
        _, S_ref = oracle.gdn_seq(tok["q"][order], tok["k"][order], tok["v"][order], tok["g"][order], tok["beta"][order])
        assert maxrel(host(S_fold), S_ref) <= TOL_BF16
    # K = 1 is the stored state, K = 0 the zero state
    assert torch.equal(b.lkv_init_state_fold(states, k, g, beta, cu, 1, ids[:1]), states[3])
    assert float(b.lkv_init_state_fold(states, k, g, beta, cu, 0, None).abs().max()) == 0.0


def test_final_states_stored_as_bf16_are_the_rounded_fp32_ones():
    import torch
    from helpers import dev, host
    rng = np.random.default_rng(42)
    bf = torch.bfloat16
    lens = [150, 0, 64]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    tok = wl.gdn_tokens(rng, int(cu[-1]), 2, 4, 128, 128, io="bf16", live_chunk_len=64)
    S0 = dev(rng.standard_normal((3, 4, 128, 128)).astype(np.float32))
    a = (dev(tok["q"], bf), dev(tok["k"], bf), dev(tok["v"], bf), dev(tok["g"]), dev(tok["beta"]), S0)
    for compute in (b.LKV_COMPUTE_TENSOR, b.LKV_COMPUTE_FP32):
        _, S32 = b.lkv_gdn_fwd(*a, cu_seqlens=cu, compute=compute, want_outputs=False)
        _, S16 = b.lkv_gdn_fwd(*a, cu_seqlens=cu, compute=compute, want_outputs=False, state_dtype=bf)
        assert S16.dtype == bf and torch.equal(S16, S32.to(bf))
    A = wl.ssd_A(rng, 3, live_chunk_len=64)
    mt = wl.ssd_tokens(rng, int(cu[-1]), 3, 64, 128, 1)
    M0 = dev(rng.standard_normal((3, 3, 128, 64)).astype(np.float32))
    m = (dev(mt["x"], bf), dev(mt["dt"]), dev(A), dev(mt["B"], bf), dev(mt["C"], bf), M0)
    for compute in (b.LKV_COMPUTE_TENSOR, b.LKV_COMPUTE_FP32):
        _, S32 = b.lkv_ssd_fwd(*m, cu_seqlens=cu, compute=compute, want_outputs=False)
        _, S16 = b.lkv_ssd_fwd(*m, cu_seqlens=cu, compute=compute, want_outputs=False, state_dtype=bf)
        assert S16.dtype == bf and torch.equal(S16, S32.to(bf))
    # a bf16 pool built this way feeds the initialisers
    S_last = b.lkv_init_state(S16, None, 3, b.LKV_INIT_LAST, family=b.LKV_FAMILY_MAMBA2)
    assert torch.equal(S_last, S16[2].float())


@pytest.mark.parametrize("case", [dict(T=1000, n=3, d=128, io="bf16", compute="auto", tol=TOL_BF16),
                                  dict(T=700, n=4, d=128, io="bf16", compute="auto", tol=TOL_BF16),
                                  dict(T=130, n=2, d=128, io="bf16", compute="auto", tol=TOL_BF16),
                                  dict(T=50, n=3, d=128, io="bf16", compute="auto", tol=TOL_BF16),
                                  dict(T=500, n=3, d=64, io="f32", compute="fp32", tol=TOL_F32)])
def test_segmented_prefill_equals_the_plain_scan_and_the_oracle(case):
    """One sequence cut into segments scanned in parallel (states and transitions of the segments, exact composition,
    all segments at once) == the plain scan == the oracle's token recurrence."""
    import torch
    rng = np.random.default_rng(43 + case["T"])
    T, d, H_k, H_v = case["T"], case["d"], 2, 4
    tok = wl.gdn_tokens(rng, T, H_k, H_v, d, d, io=case["io"], live_chunk_len=256)
    S0 = rng.standard_normal((1, H_v, d, d)).astype(np.float32)
    dt = torch.bfloat16 if case["io"] == "bf16" else None
    compute = b.LKV_COMPUTE_AUTO if case["compute"] == "auto" else b.LKV_COMPUTE_FP32
    args = (dev(tok["q"], dt), dev(tok["k"], dt), dev(tok["v"], dt), dev(tok["g"]), dev(tok["beta"]))
    o_ref, ST_ref = oracle.gdn_seq(tok["q"], tok["k"], tok["v"], tok["g"], tok["beta"], S0[0])
    for s0 in (S0, None):
        o, ST = b.lkv_gdn_fwd_segmented(*args, None if s0 is None else dev(s0), n_segments=case["n"], compute=compute)
        o_p, ST_p = b.lkv_gdn_fwd(*args, None if s0 is None else dev(s0), compute=compute)
        assert maxrel(host(o), host(o_p)) <= case["tol"] and maxrel(host(ST), host(ST_p)) <= case["tol"]
        if s0 is not None:
            assert maxrel(host(o), o_ref) <= case["tol"] and maxrel(host(ST)[0], ST_ref) <= case["tol"]
    # the first segment is the same blocks from the same state: its outputs are the plain scan's, bit for bit
    per = ((T + case["n"] - 1) // case["n"] + 63) // 64 * 64
    assert torch.equal(o[:per], o_p[:per])


@pytest.mark.parametrize("family", ["gdn", "mamba2"])
def test_staging_from_a_host_pool_feeds_the_initialisers(family):
    """The cache lives in (pinned) host memory; the chunks a batch names are staged once each into a compact device pool
    and the ids rewritten: composing from the staged pool == composing from the whole pool on the device, bit for bit."""
    import torch
    rng = np.random.default_rng(44)
    n, H = 40, 3
    if family == "gdn":
        code, dk, dv = b.LKV_FAMILY_GDN, 128, 128
        trans = wl.synthetic_gdn_transitions(rng, n, H, dk)
    else:
        code, dk, dv = b.LKV_FAMILY_MAMBA2, 128, 64
        trans = wl.synthetic_logdecay(rng, n, H)
    states = wl.synthetic_states(rng, n, H, dk, dv)
    h_states, h_trans = torch.from_numpy(states).pin_memory(), torch.from_numpy(trans).pin_memory()
    n_req, K = 6, 5
    ids = rng.integers(0, n, size=n_req * K).astype(np.int32)     # repeats across and inside requests
    cu_k = (np.arange(n_req + 1) * K).astype(np.int32)
    distinct = len(set(ids.tolist()))
    d_states = torch.empty((distinct,) + states.shape[1:], device="cuda")
    d_trans = torch.empty((distinct,) + trans.shape[1:], device="cuda")
    staged, n_staged = b.lkv_stage_chunks(h_states, h_trans, ids, d_states, d_trans, family=code)
    assert n_staged == distinct and staged.max() == distinct - 1
    torch.cuda.synchronize()
    for slot, c in {int(s): int(c) for s, c in zip(staged, ids)}.items():
        assert torch.equal(d_states[slot].cpu(), h_states[c]) and torch.equal(d_trans[slot].cpu(), h_trans[c])
    got = b.lkv_init_state_batched(d_states, d_trans, staged, cu_k, n_req, b.LKV_INIT_EXACT, family=code)
    ref = b.lkv_init_state_batched(dev(states), dev(trans), ids, cu_k, n_req, b.LKV_INIT_EXACT, family=code)
    assert torch.equal(got, ref)
    with pytest.raises(b.LkvError) as e:       # a staging pool that is too small is refused before anything is copied
        b.lkv_stage_chunks(h_states, h_trans, ids, d_states[: distinct - 1], d_trans[: distinct - 1], family=code)
    assert e.value.status == b.LKV_ERR_WORKSPACE


@pytest.mark.parametrize("compute", [b.LKV_COMPUTE_AUTO, b.LKV_COMPUTE_FP32])
def test_one_launch_producer_equals_the_two_calls_bit_for_bit(compute):
    import torch
    rng = np.random.default_rng(45)
    lens = [200, 64, 0, 131, 77, 1024]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    tok = wl.gdn_tokens(rng, int(cu[-1]), 2, 4, 128, 128, io="bf16", live_chunk_len=128)
    bf = torch.bfloat16
    k, v, g, beta = dev(tok["k"], bf), dev(tok["v"], bf), dev(tok["g"]), dev(tok["beta"])
    states, trans = b.lkv_gdn_chunk_artifacts(k, v, g, beta, cu_seqlens=cu, compute=compute)
    _, states2 = b.lkv_gdn_fwd(k, k, v, g, beta, cu_seqlens=cu, want_outputs=False, compute=compute)
    trans2 = b.lkv_gdn_chunk_transition(k, g, beta, cu_seqlens=cu, compute=compute)
    assert torch.equal(states, states2) and torch.equal(trans, trans2)
    assert float(states[2].abs().max()) == 0.0 and torch.equal(trans[2, 0], torch.eye(128, device="cuda"))   # the empty chunk
