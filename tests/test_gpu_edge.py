"""Edge cases, invariances and failure reporting of the CUDA library on the tensor-core paths.

Empty batches, sequences shorter than a block, run-to-run determinism of every kernel, cutting a sequence at a
point that is not a block boundary, appended identity tokens, permuted value heads, the per-head error metric,
the give-up path of the bounded device waits, and index lists under stream capture.
"""
import numpy as np
import pytest

import oracle
from helpers import TOL_BF16, dev, host, maxrel, maxrel_per_head
from paper_2608_11231_b200 import binding as b
from paper_2608_11231_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _torch():
    import torch
    return torch


def _gdn(tok, S0=None, cu=None, **kw):
    bf = _torch().bfloat16
    return b.lkv_gdn_fwd(dev(tok["q"], bf), dev(tok["k"], bf), dev(tok["v"], bf), dev(tok["g"]), dev(tok["beta"]),
                         None if S0 is None else dev(S0), cu_seqlens=cu, **kw)


def _ssd(tok, A, S0=None, cu=None, **kw):
    bf = _torch().bfloat16
    return b.lkv_ssd_fwd(dev(tok["x"], bf), dev(tok["dt"]), dev(A), dev(tok["B"], bf), dev(tok["C"], bf),
                         None if S0 is None else dev(S0), cu_seqlens=cu, **kw)


# ------------------------------------------------------------------ empty batches and short sequences

def test_all_empty_batch_hands_states_through_on_the_tensor_paths():
    torch = _torch()
    rng = np.random.default_rng(21)
    cu = np.zeros(3, dtype=np.int32)                      # two sequences, no token at all
    bf = torch.bfloat16
    # GDN, tensor-path shape
    S0 = rng.standard_normal((2, 4, 128, 128)).astype(np.float32)
    e = lambda *shape, dt=bf: torch.empty(shape, dtype=dt, device="cuda")
    o, ST = b.lkv_gdn_fwd(e(0, 2, 128), e(0, 2, 128), e(0, 4, 128), e(0, 4, dt=torch.float32), e(0, 4, dt=torch.float32),
                          dev(S0), cu_seqlens=cu, compute=b.LKV_COMPUTE_TENSOR)
    assert o.shape[0] == 0 and host(ST).tobytes() == S0.tobytes()
    # chunk transitions of empty chunks: the identity
    T = b.lkv_gdn_chunk_transition(e(0, 2, 128), e(0, 4, dt=torch.float32), e(0, 4, dt=torch.float32), H_v=4,
                                   cu_seqlens=cu, compute=b.LKV_COMPUTE_TENSOR)
    assert np.array_equal(host(T), np.broadcast_to(np.eye(128, dtype=np.float32), (2, 4, 128, 128)))
    # SSD, tensor-path shape
    M0 = rng.standard_normal((2, 3, 128, 64)).astype(np.float32)
    y, MT = b.lkv_ssd_fwd(e(0, 3, 64), e(0, 3, dt=torch.float32), dev(-np.ones(3, np.float32)), e(0, 1, 128), e(0, 1, 128),
                          dev(M0), cu_seqlens=cu, compute=b.LKV_COMPUTE_TENSOR)
    assert y.shape[0] == 0 and host(MT).tobytes() == M0.tobytes()


@pytest.mark.parametrize("T", [1, 37, 63])
def test_single_sequence_shorter_than_a_block(T):
    rng = np.random.default_rng(100 + T)
    tok = wl.gdn_tokens(rng, T, 2, 4, 128, 128, io="bf16", live_chunk_len=64)
    S0 = rng.standard_normal((1, 4, 128, 128)).astype(np.float32)
    o, ST = _gdn(tok, S0, compute=b.LKV_COMPUTE_TENSOR)
    o_ref, ST_ref = oracle.gdn_seq(tok["q"], tok["k"], tok["v"], tok["g"], tok["beta"], S0[0])
    assert maxrel(host(o), o_ref) <= TOL_BF16 and maxrel(host(ST)[0], ST_ref) <= TOL_BF16
    assert maxrel_per_head(host(o), o_ref, 1) <= TOL_BF16 and maxrel_per_head(host(ST)[0], ST_ref, 0) <= TOL_BF16
    A = wl.ssd_A(rng, 3, live_chunk_len=64)
    mt = wl.ssd_tokens(rng, T, 3, 64, 128, 1)
    M0 = rng.standard_normal((1, 3, 128, 64)).astype(np.float32)
    y, MT = _ssd(mt, A, M0, compute=b.LKV_COMPUTE_TENSOR)
    y_ref, MT_ref = oracle.ssd_seq(mt["x"], mt["dt"], A, mt["B"], mt["C"], M0[0])
    assert maxrel(host(y), y_ref) <= TOL_BF16 and maxrel(host(MT)[0], MT_ref) <= TOL_BF16
    assert maxrel_per_head(host(y), y_ref, 1) <= TOL_BF16 and maxrel_per_head(host(MT)[0], MT_ref, 0) <= TOL_BF16


# ------------------------------------------------------------------ determinism

def test_every_kernel_is_run_to_run_deterministic():
    torch = _torch()
    rng = np.random.default_rng(22)
    # SSD scan (tensor path), ragged
    lens = [300, 0, 129, 64]
    cu = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    A = wl.ssd_A(rng, 4, live_chunk_len=128)
    mt = wl.ssd_tokens(rng, int(cu[-1]), 4, 64, 128, 1)
    M0 = rng.standard_normal((4, 4, 128, 64)).astype(np.float32)
    r1, r2 = _ssd(mt, A, M0, cu), _ssd(mt, A, M0, cu)
    assert all(host(x).tobytes() == host(z).tobytes() for x, z in zip(r1, r2))
    # Mamba-2 composition (streaming kernel) and GDN composition (tensor cores and fp32), batched
    n_req, K = 5, 7
    cu_k = (np.arange(n_req + 1) * K).astype(np.int32)
    ids = rng.integers(0, 12, size=n_req * K).astype(np.int32)
    pool_m = dev(wl.synthetic_states(rng, 12, 3, 128, 64))
    lam = dev(wl.synthetic_logdecay(rng, 12, 3))
    f = lambda: b.lkv_init_state_batched(pool_m, lam, ids, cu_k, n_req, b.LKV_INIT_EXACT, family=b.LKV_FAMILY_MAMBA2)
    assert host(f()).tobytes() == host(f()).tobytes()
    pool_g = dev(wl.synthetic_states(rng, 12, 3, 128, 128))
    tr = dev(wl.synthetic_gdn_transitions(rng, 12, 3, 128))
    for compute in (b.LKV_COMPUTE_TENSOR, b.LKV_COMPUTE_FP32):
        f = lambda: b.lkv_init_state_batched(pool_g, tr, ids, cu_k, n_req, b.LKV_INIT_EXACT, family=b.LKV_FAMILY_GDN,
                                             compute=compute)
        assert host(f()).tobytes() == host(f()).tobytes()
    # state-error diagnostic
    x = torch.randn(6, 3, 128, 128, device="cuda")
    r = torch.randn(6, 3, 128, 128, device="cuda")
    e1 = b.lkv_state_rel_error(x, r, 6)
    e2 = b.lkv_state_rel_error(x, r, 6)
    assert host(e1).tobytes() == host(e2).tobytes()


# ------------------------------------------------------------------ invariances on the tensor paths

def test_split_and_chain_at_a_ragged_cut_on_the_tensor_paths():
    """One call over a sequence == two chained calls cut inside a block (Eq. 1 holds for any run of tokens)."""
    rng = np.random.default_rng(23)
    T, cut = 330, 147
    tok = wl.gdn_tokens(rng, T, 2, 4, 128, 128, io="bf16", live_chunk_len=128)
    S0 = rng.standard_normal((1, 4, 128, 128)).astype(np.float32)
    o_full, ST_full = _gdn(tok, S0)
    first = {n: x[:cut] for n, x in tok.items()}
    second = {n: x[cut:] for n, x in tok.items()}
    o_a, ST_a = _gdn(first, S0)
    o_c, ST_c = _gdn(second, host(ST_a))
    o_ref, ST_ref = oracle.gdn_seq(tok["q"], tok["k"], tok["v"], tok["g"], tok["beta"], S0[0])
    o_cat = np.concatenate([host(o_a), host(o_c)])
    # the two evaluations round differently (the blocks do not line up): both sit inside the bf16 bound of the
    # oracle, and within it of each other
    assert maxrel(o_cat, o_ref) <= TOL_BF16 and maxrel(host(ST_c)[0], ST_ref) <= TOL_BF16
    assert maxrel(o_cat, host(o_full)) <= TOL_BF16 and maxrel(host(ST_c), host(ST_full)) <= TOL_BF16
    A = wl.ssd_A(rng, 3, live_chunk_len=128)
    mt = wl.ssd_tokens(rng, T, 3, 64, 128, 1)
    M0 = rng.standard_normal((1, 3, 128, 64)).astype(np.float32)
    y_full, MT_full = _ssd(mt, A, M0)
    y_a, MT_a = _ssd({n: x[:cut] for n, x in mt.items()}, A, M0)
    y_c, MT_c = _ssd({n: x[cut:] for n, x in mt.items()}, A, host(MT_a))
    y_ref, MT_ref = oracle.ssd_seq(mt["x"], mt["dt"], A, mt["B"], mt["C"], M0[0])
    y_cat = np.concatenate([host(y_a), host(y_c)])
    assert maxrel(y_cat, y_ref) <= TOL_BF16 and maxrel(host(MT_c)[0], MT_ref) <= TOL_BF16
    assert maxrel(y_cat, host(y_full)) <= TOL_BF16 and maxrel(host(MT_c), host(MT_full)) <= TOL_BF16


def test_appended_identity_tokens_change_nothing_on_the_tensor_paths():
    """A token with g = 0, beta = 0 (GDN) or dt = 0 (SSD) is the identity step: T = I, u = 0."""
    rng = np.random.default_rng(24)
    T, pad = 150, 41
    tok = wl.gdn_tokens(rng, T + pad, 2, 4, 128, 128, io="bf16", live_chunk_len=128)
    tok["g"][T:] = 0.0
    tok["beta"][T:] = 0.0
    S0 = rng.standard_normal((1, 4, 128, 128)).astype(np.float32)
    o_p, ST_p = _gdn(tok, S0)
    o, ST = _gdn({n: x[:T] for n, x in tok.items()}, S0)
    # same blocks, same arithmetic for the first T tokens: the outputs agree bit for bit, the state within rounding of
    # nothing (the padded block adds exact zeros)
    assert host(o_p)[:T].tobytes() == host(o).tobytes()
    assert maxrel(host(ST_p), host(ST)) <= 1e-6
    A = wl.ssd_A(rng, 3, live_chunk_len=128)
    mt = wl.ssd_tokens(rng, T + pad, 3, 64, 128, 1)
    mt["dt"][T:] = 0.0
    M0 = rng.standard_normal((1, 3, 128, 64)).astype(np.float32)
    y_p, MT_p = _ssd(mt, A, M0)
    y, MT = _ssd({n: x[:T] for n, x in mt.items()}, A, M0)
    assert host(y_p)[:T].tobytes() == host(y).tobytes()
    assert maxrel(host(MT_p), host(MT)) <= 1e-6


def test_permuting_value_heads_permutes_outputs_and_states():
    """Value head h reads q/k head h // (H_v / H_k): value heads that share a q/k head may be swapped freely."""
    rng = np.random.default_rng(25)
    H_k, H_v, T = 2, 6, 200
    tok = wl.gdn_tokens(rng, T, H_k, H_v, 128, 128, io="bf16", live_chunk_len=128)
    S0 = rng.standard_normal((1, H_v, 128, 128)).astype(np.float32)
    perm = np.array([2, 0, 1, 4, 5, 3])                   # stays inside the two groups {0,1,2} and {3,4,5}
    o, ST = _gdn(tok, S0)
    tok_p = dict(tok, v=np.ascontiguousarray(tok["v"][:, perm]), g=np.ascontiguousarray(tok["g"][:, perm]),
                 beta=np.ascontiguousarray(tok["beta"][:, perm]))
    o_p, ST_p = _gdn(tok_p, np.ascontiguousarray(S0[:, perm]))
    assert host(o_p).tobytes() == np.ascontiguousarray(host(o)[:, perm]).tobytes()
    assert host(ST_p).tobytes() == np.ascontiguousarray(host(ST)[:, perm]).tobytes()
    # and moving a value head to the other group does change its result (it now reads other keys)
    cross = np.array([3, 1, 2, 0, 4, 5])
    tok_x = dict(tok, v=np.ascontiguousarray(tok["v"][:, cross]), g=np.ascontiguousarray(tok["g"][:, cross]),
                 beta=np.ascontiguousarray(tok["beta"][:, cross]))
    o_x, _ = _gdn(tok_x, np.ascontiguousarray(S0[:, cross]))
    assert maxrel(host(o_x)[:, 0], host(o)[:, 3]) > 0.1


# ------------------------------------------------------------------ failure reporting

def test_bounded_wait_runs_out_and_is_reported():
    """The give-up path of the device-side waits: a wait nobody will ever satisfy ends by itself and is reported."""
    torch = _torch()
    ws = torch.zeros(4096, dtype=torch.uint8, device="cuda")
    assert b.lkv_device_status(ws) == b.LKV_OK
    assert b.lkv_selftest_bounded_wait(2000, ws) == b.LKV_OK          # the launch itself succeeds
    assert b.lkv_device_status(ws) == b.LKV_ERR_DEVICE_TIMEOUT
    assert b.lkv_device_status(ws) == b.LKV_ERR_DEVICE_TIMEOUT         # sticky until the caller clears it
    assert int(ws.view(torch.int32)[1].item()) == 0                    # no wait claimed success
    # the context is intact: clear the header and run a normal call on the same workspace
    ws.zero_()
    rng = np.random.default_rng(26)
    tok = wl.gdn_tokens(rng, 130, 1, 2, 128, 128, io="bf16", live_chunk_len=64)
    o, ST = _gdn(tok, workspace_t=ws)
    assert b.lkv_device_status(ws) == b.LKV_OK
    o_ref, ST_ref = oracle.gdn_seq(tok["q"], tok["k"], tok["v"], tok["g"], tok["beta"])
    assert maxrel(host(o), o_ref) <= TOL_BF16 and maxrel(host(ST)[0], ST_ref) <= TOL_BF16


def test_long_index_list_is_refused_under_stream_capture():
    """An index list too long for the kernel parameters needs a copy from a host array that dies with the call."""
    torch = _torch()
    rng = np.random.default_rng(27)
    n_req, K = 150, 30
    pool = dev(wl.synthetic_states(rng, 16, 2, 16, 32))
    lam = dev(wl.synthetic_logdecay(rng, 16, 2))
    ids = rng.integers(0, 16, size=n_req * K).astype(np.int32)
    cu = (np.arange(n_req + 1) * K).astype(np.int32)
    S0 = torch.empty((n_req, 2, 16, 32), device="cuda")
    ws = torch.zeros(1 << 16, dtype=torch.uint8, device="cuda")
    ref = b.lkv_init_state_batched(pool, lam, ids, cu, n_req, b.LKV_INIT_EXACT, None, S0, family=b.LKV_FAMILY_MAMBA2,
                                   workspace_t=ws).clone()
    g = torch.cuda.CUDAGraph()
    s = torch.cuda.Stream()
    with torch.cuda.stream(s):
        with torch.cuda.graph(g, stream=s):
            with pytest.raises(b.LkvError) as e:
                b.lkv_init_state_batched(pool, lam, ids, cu, n_req, b.LKV_INIT_EXACT, None, S0,
                                         family=b.LKV_FAMILY_MAMBA2, workspace_t=ws)
            # a short list travels in the kernel parameters: this one is captured
            b.lkv_init_state_batched(pool, lam, ids[: 10 * K], cu[:11], 10, b.LKV_INIT_EXACT, None, S0,
                                     family=b.LKV_FAMILY_MAMBA2, workspace_t=ws)
    assert e.value.status == b.LKV_ERR_UNSUPPORTED
    S0.zero_()
    g.replay()
    torch.cuda.synchronize()
    assert torch.equal(S0[:10], ref[:10])
