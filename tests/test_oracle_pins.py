"""Pins for the fp64 CPU oracle: what the paper and the mathematics fix.

Each test checks the oracle against something other than itself: literal
matrices built from Eq. 2 / Eq. 3, hand-derived fixtures, brute force over the
concatenated prefix (Eq. 5 / Eq. 6), closed forms and library limits.
"""
import json
import os

import numpy as np
import pytest

import oracle
from paper_2608_11231_b200 import workloads as wl

GOLD = os.path.join(os.path.dirname(__file__), "golden")


def _gdn_inputs(seed, T, Hk=1, Hv=2, dk=8, dv=6, live=None):
    rng = np.random.default_rng(seed)
    d = wl.gdn_tokens(rng, T, Hk, Hv, dk, dv, io="f32", live_chunk_len=live)
    return {n: a.astype(np.float64) for n, a in d.items()}


def _ssd_inputs(seed, T, H=4, P=5, N=6, G=2, live=None):
    rng = np.random.default_rng(seed)
    A = wl.ssd_A(rng, H, live_chunk_len=live).astype(np.float64)
    d = wl.ssd_tokens(rng, T, H, P, N, G, io="f32")
    d = {n: a.astype(np.float64) for n, a in d.items()}
    d["A"] = A
    return d


# ---------------------------------------------------------------- literal forms

def test_gdn_matches_literal_eq3_matrices():
    """Eq. 3 written with explicit d_k x d_k transition matrices, per head."""
    T, Hk, Hv, dk, dv = 9, 2, 4, 5, 3
    d = _gdn_inputs(11, T, Hk, Hv, dk, dv)
    rng = np.random.default_rng(5)
    S0 = rng.standard_normal((Hv, dk, dv))
    scale = 0.37
    o, S_T = oracle.gdn_seq(d["q"], d["k"], d["v"], d["g"], d["beta"], S0, scale)
    for h in range(Hv):
        hk = h // (Hv // Hk)
        S = S0[h].copy()
        for t in range(T):
            k = d["k"][t, hk][:, None]
            Tt = np.exp(d["g"][t, h]) * (np.eye(dk) - d["beta"][t, h] * (k @ k.T))
            u = d["beta"][t, h] * (k @ d["v"][t, h][None, :])
            S = Tt @ S + u
            np.testing.assert_allclose(o[t, h], scale * (S.T @ d["q"][t, hk]), rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(S_T[h], S, rtol=1e-12, atol=1e-14)


def test_ssd_matches_literal_eq2():
    T, H, P, N, G = 7, 4, 3, 5, 2
    d = _ssd_inputs(3, T, H, P, N, G)
    rng = np.random.default_rng(6)
    S0 = rng.standard_normal((H, N, P))
    y, S_T = oracle.ssd_seq(d["x"], d["dt"], d["A"], d["B"], d["C"], S0)
    for h in range(H):
        grp = h // (H // G)
        S = S0[h].copy()
        for t in range(T):
            a = np.exp(d["dt"][t, h] * d["A"][h])
            S = a * S + d["dt"][t, h] * np.outer(d["B"][t, grp], d["x"][t, h])
            np.testing.assert_allclose(y[t, h], S.T @ d["C"][t, grp], rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(S_T[h], S, rtol=1e-12, atol=1e-14)


def test_gdn_hand_worked_fixture():
    with open(os.path.join(GOLD, "gdn_two_tokens.json")) as f:
        fx = json.load(f)
    g = np.log(np.array(fx["alpha"]))
    o, S_T = oracle.gdn_seq(fx["q"], fx["k"], fx["v"], g, fx["beta"], None, fx["scale"])
    np.testing.assert_allclose(o, np.array(fx["o"]), rtol=1e-14, atol=1e-15)
    np.testing.assert_allclose(S_T, np.array(fx["S_T"]), rtol=1e-14, atol=1e-15)
    Tc = oracle.gdn_transition(fx["k"], g, fx["beta"])
    np.testing.assert_allclose(Tc, np.array(fx["T_C"]), rtol=1e-14, atol=1e-15)
    # the reverse product order is the transpose here and must be rejected
    assert np.abs(Tc - np.array(fx["T_C"]).transpose(0, 2, 1)).max() > 1e-2


def test_mamba_hand_worked_fixture():
    with open(os.path.join(GOLD, "mamba_two_tokens.json")) as f:
        fx = json.load(f)
    A = np.array([-np.log(2.0)])
    y, S_T = oracle.ssd_seq(fx["x"], fx["dt"], A, fx["B"], fx["C"], None)
    np.testing.assert_allclose(y, np.array(fx["y"]), rtol=1e-14)
    np.testing.assert_allclose(S_T, np.array(fx["S_T"]), rtol=1e-14)
    lam = oracle.mamba_logdecay(fx["dt"], A)
    np.testing.assert_allclose(np.exp(lam), [fx["chunk_decay"]], rtol=1e-14)


# ------------------------------------------------- Eq. 5 / Eq. 6 by brute force

def _gdn_chunks(seed, lens, Hk, Hv, dk, dv, live=64):
    rng = np.random.default_rng(seed)
    return [{n: a.astype(np.float64) for n, a in
             wl.gdn_tokens(rng, int(L), Hk, Hv, dk, dv, io="f32", live_chunk_len=live).items()} for L in lens]


def _cat(chunks, order, keys):
    return {n: np.concatenate([chunks[c][n] for c in order], axis=0) for n in keys}


@pytest.mark.parametrize("lens", [[13], [5, 9], [7, 3, 11], [6, 6, 6, 6], [4, 9, 2, 7, 5, 8, 3]])
def test_gdn_exact_composition_equals_sequential_pass(lens):
    Hk, Hv, dk, dv = 2, 4, 8, 6
    chunks = _gdn_chunks(21 + len(lens), lens, Hk, Hv, dk, dv)
    states = np.stack([oracle.gdn_seq(c["q"], c["k"], c["v"], c["g"], c["beta"])[1] for c in chunks])
    trans = np.stack([oracle.gdn_transition(c["k"], c["g"], c["beta"]) for c in chunks])
    rng = np.random.default_rng(0)
    for trial in range(3):
        order = np.arange(len(lens)) if trial == 0 else rng.permutation(len(lens))
        cat = _cat(chunks, order, ["q", "k", "v", "g", "beta"])
        _, S_full = oracle.gdn_seq(cat["q"], cat["k"], cat["v"], cat["g"], cat["beta"])
        S0 = oracle.init_exact_gdn(states, trans, order.astype(np.int32))
        # carried part must be a visible share of the state, else the test is vacuous
        if len(lens) > 1:
            assert np.abs(S0 - states[order[-1]]).max() > 1e-2 * np.abs(S0).max()
        np.testing.assert_allclose(S0, S_full, rtol=1e-11, atol=1e-13)


def test_gdn_chunk_is_affine_operator():
    """Eq. 5: a chunk entered with any S_in returns T_C S_in + S_local."""
    Hk, Hv, dk, dv = 1, 2, 7, 5
    c = _gdn_chunks(2, [17], Hk, Hv, dk, dv)[0]
    S_in = np.random.default_rng(1).standard_normal((Hv, dk, dv))
    _, S_out = oracle.gdn_seq(c["q"], c["k"], c["v"], c["g"], c["beta"], S_in)
    _, S_loc = oracle.gdn_seq(c["q"], c["k"], c["v"], c["g"], c["beta"], None)
    Tc = oracle.gdn_transition(c["k"], c["g"], c["beta"])
    np.testing.assert_allclose(S_out, np.einsum("hij,hjk->hik", Tc, S_in) + S_loc, rtol=1e-12, atol=1e-14)
    # the transposed transition is a different matrix and must not satisfy it
    wrong = np.einsum("hji,hjk->hik", Tc, S_in) + S_loc
    assert np.abs(wrong - S_out).max() > 1e-3


@pytest.mark.parametrize("lens", [[10], [4, 12], [9, 2, 6, 7, 3]])
def test_mamba_exact_composition_equals_sequential_pass(lens):
    H, P, N, G = 4, 5, 6, 2
    rng = np.random.default_rng(17)
    A = wl.ssd_A(rng, H, live_chunk_len=8).astype(np.float64)
    chunks = [{n: a.astype(np.float64) for n, a in wl.ssd_tokens(rng, int(L), H, P, N, G, io="f32").items()}
              for L in lens]
    states = np.stack([oracle.ssd_seq(c["x"], c["dt"], A, c["B"], c["C"])[1] for c in chunks])
    lam = np.stack([oracle.mamba_logdecay(c["dt"], A) for c in chunks])
    prng = np.random.default_rng(1)
    for trial in range(3):
        order = np.arange(len(lens)) if trial == 0 else prng.permutation(len(lens))
        cat = _cat(chunks, order, ["x", "dt", "B", "C"])
        _, S_full = oracle.ssd_seq(cat["x"], cat["dt"], A, cat["B"], cat["C"])
        S0 = oracle.init_exact_mamba(states, lam, order.astype(np.int32))
        if len(lens) > 1:
            assert np.abs(S0 - states[order[-1]]).max() > 1e-2 * np.abs(S0).max()
        np.testing.assert_allclose(S0, S_full, rtol=1e-11, atol=1e-13)


def test_exact_composition_closed_form_sum():
    """Eq. 6 written as the explicit sum of products, against the chained form."""
    rng = np.random.default_rng(8)
    n, H, dk, dv = 5, 2, 4, 3
    states = rng.standard_normal((n, H, dk, dv))
    trans = wl.synthetic_gdn_transitions(rng, n, H, dk).astype(np.float64)
    ids = np.array([3, 0, 4, 0, 2], dtype=np.int32)  # a chunk reused at two positions
    S0 = oracle.init_exact_gdn(states, trans, ids)
    ref = np.zeros((H, dk, dv))
    for h in range(H):
        for j in range(len(ids)):
            prod = np.eye(dk)
            for m in range(j + 1, len(ids)):       # later chunk on the left
                prod = trans[ids[m], h] @ prod
            ref[h] += prod @ states[ids[j], h]
    np.testing.assert_allclose(S0, ref, rtol=1e-12, atol=1e-14)
    lam = wl.synthetic_logdecay(rng, n, H).astype(np.float64)
    S0m = oracle.init_exact_mamba(states, lam, ids)
    refm = np.zeros((H, dk, dv))
    for h in range(H):
        for j in range(len(ids)):
            w = np.exp(sum(lam[ids[m], h] for m in range(j + 1, len(ids))))
            refm[h] += w * states[ids[j], h]
    np.testing.assert_allclose(S0m, refm, rtol=1e-12, atol=1e-14)


def test_mismatch_recursion_eq7():
    """Eq. 7: a perturbation delta_j of the cached states propagates as e_j = T e_{j-1} + delta_j."""
    rng = np.random.default_rng(9)
    n, H, dk, dv = 4, 2, 5, 3
    states = rng.standard_normal((n, H, dk, dv))
    delta = 1e-3 * rng.standard_normal((n, H, dk, dv))
    trans = wl.synthetic_gdn_transitions(rng, n, H, dk).astype(np.float64)
    e = np.zeros((H, dk, dv))
    for j in range(n):
        e = (np.einsum("hij,hjk->hik", trans[j], e) if j > 0 else e) + delta[j]
    got = oracle.init_exact_gdn(states + delta, trans) - oracle.init_exact_gdn(states, trans)
    np.testing.assert_allclose(got, e, rtol=1e-9, atol=1e-15)


# ---------------------------------------------------------------- special cases

def test_k1_is_identity_and_modes_coincide():
    rng = np.random.default_rng(2)
    states32 = rng.standard_normal((3, 2, 4, 5), dtype=np.float32)
    trans = wl.synthetic_gdn_transitions(rng, 3, 2, 4)
    ids = np.array([1], dtype=np.int32)
    ex = oracle.init_exact_gdn(states32, trans, ids)
    single, idx = oracle.init_single(states32, ids)
    assert idx == 1
    assert single.dtype == np.float32 and single.tobytes() == states32[1].tobytes()
    assert np.array_equal(ex, states32[1].astype(np.float64))
    lam = wl.synthetic_logdecay(rng, 3, 2)
    assert np.array_equal(oracle.init_exact_mamba(states32, lam, ids), states32[1].astype(np.float64))


def test_k0_is_empty_state():
    states = np.ones((2, 1, 3, 3))
    assert not oracle.init_exact_gdn(states, np.ones((2, 1, 3, 3)), np.zeros((0,), np.int32)).any()
    assert not oracle.init_exact_mamba(states, np.zeros((2, 1)), np.zeros((0,), np.int32)).any()
    z, idx = oracle.init_single(states, np.zeros((0,), np.int32))
    assert idx == -1 and not z.any()


def test_single_block_selection_is_bitwise():
    rng = np.random.default_rng(4)
    states = rng.standard_normal((6, 2, 3, 4), dtype=np.float32)
    ids = np.array([5, 2, 2, 0], dtype=np.int32)
    last, idx = oracle.init_single(states, ids)
    assert idx == 0 and last.tobytes() == states[0].tobytes()
    for b in range(4):
        s, idx = oracle.init_single(states, ids, b=b)
        assert idx == ids[b] and s.tobytes() == states[ids[b]].tobytes()


def test_identity_and_zero_transition_limits():
    rng = np.random.default_rng(3)
    n, H, dk, dv = 4, 2, 5, 3
    states = rng.standard_normal((n, H, dk, dv))
    eye = np.broadcast_to(np.eye(dk), (n, H, dk, dk)).copy()
    np.testing.assert_allclose(oracle.init_exact_gdn(states, eye), states.sum(0), rtol=1e-14)
    assert np.array_equal(oracle.init_exact_gdn(states, np.zeros((n, H, dk, dk))), states[-1])
    np.testing.assert_allclose(oracle.init_exact_mamba(states, np.zeros((n, H))), states.sum(0), rtol=1e-14)
    assert np.array_equal(oracle.init_exact_mamba(states, np.full((n, H), -np.inf)), states[-1])
    # strong decay that underflows exp(): still exactly the last block
    assert np.array_equal(oracle.init_exact_mamba(states, np.full((n, H), -800.0)), states[-1])


def test_delta_rule_overwrite():
    """With no decay, beta = 1 and orthonormal keys the state is an associative memory."""
    rng = np.random.default_rng(12)
    dk, dv, T = 8, 5, 6
    Q, _ = np.linalg.qr(rng.standard_normal((dk, dk)))
    keys = Q[:, :T].T.copy()
    keys[5] = keys[1]                    # token 5 rewrites key 1
    vals = rng.standard_normal((T, dv))
    k = keys[:, None, :]
    v = vals[:, None, :]
    o, S_T = oracle.gdn_seq(k, k, v, np.zeros((T, 1)), np.ones((T, 1)), None, 1.0)
    for t in range(T):
        np.testing.assert_allclose(o[t, 0], vals[t], atol=1e-13)      # read-back right after writing
    for t in [0, 2, 3, 4]:
        np.testing.assert_allclose(S_T[0].T @ keys[t], vals[t], atol=1e-13)
    np.testing.assert_allclose(S_T[0].T @ keys[1], vals[5], atol=1e-13)  # later write wins


def test_ssd_zero_decay_is_causal_linear_attention():
    d = _ssd_inputs(5, 12, H=4, P=3, N=6, G=2)
    A0 = np.zeros(4)
    rng = np.random.default_rng(1)
    S0 = rng.standard_normal((4, 6, 3))
    y, S_T = oracle.ssd_seq(d["x"], d["dt"], A0, d["B"], d["C"], S0)
    for h in range(4):
        grp = h // 2
        Bm, Cm = d["B"][:, grp], d["C"][:, grp]
        X = d["dt"][:, h:h + 1] * d["x"][:, h]
        np.testing.assert_allclose(S_T[h], S0[h] + Bm.T @ X, rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(y[:, h], np.tril(Cm @ Bm.T) @ X + Cm @ S0[h], rtol=1e-12, atol=1e-14)


def test_ssd_decay_mask_closed_form():
    """With decay: y = (L o C B^T)(dt x) + diag(exp(l)) C S0, L_ti = exp(l_t - l_i), l = cumsum(dt A)."""
    d = _ssd_inputs(6, 10, H=2, P=3, N=4, G=1)
    rng = np.random.default_rng(2)
    S0 = rng.standard_normal((2, 4, 3))
    y, S_T = oracle.ssd_seq(d["x"], d["dt"], d["A"], d["B"], d["C"], S0)
    for h in range(2):
        l = np.cumsum(d["dt"][:, h] * d["A"][h])
        L = np.tril(np.exp(l[:, None] - l[None, :]))
        Bm, Cm = d["B"][:, 0], d["C"][:, 0]
        X = d["dt"][:, h:h + 1] * d["x"][:, h]
        np.testing.assert_allclose(y[:, h], (L * (Cm @ Bm.T)) @ X + np.exp(l)[:, None] * (Cm @ S0[h]),
                                   rtol=1e-12, atol=1e-14)
        np.testing.assert_allclose(S_T[h], np.exp(l[-1]) * S0[h] + (np.exp(l[-1] - l)[:, None] * Bm).T @ X,
                                   rtol=1e-12, atol=1e-14)


def test_gdn_beta_zero_is_pure_decay():
    d = _gdn_inputs(7, 9, Hk=1, Hv=2, dk=4, dv=3)
    rng = np.random.default_rng(3)
    S0 = rng.standard_normal((2, 4, 3))
    zero = np.zeros_like(d["beta"])
    o, S_T = oracle.gdn_seq(d["q"], d["k"], d["v"], d["g"], zero, S0, 0.5)
    cg = np.cumsum(d["g"], axis=0)
    for h in range(2):
        np.testing.assert_allclose(S_T[h], np.exp(cg[-1, h]) * S0[h], rtol=1e-13)
        ref = 0.5 * np.exp(cg[:, h])[:, None] * (d["q"][:, 0] @ S0[h])
        np.testing.assert_allclose(o[:, h], ref, rtol=1e-12, atol=1e-15)
    _, S_same = oracle.gdn_seq(d["q"], d["k"], d["v"], np.zeros_like(d["g"]), zero, S0, 0.5)
    assert np.array_equal(S_same, S0)


def test_padding_tokens_and_split_chaining():
    d = _gdn_inputs(8, 21, Hk=2, Hv=2, dk=6, dv=4)
    o, S_T = oracle.gdn_seq(d["q"], d["k"], d["v"], d["g"], d["beta"])
    pad = {n: np.concatenate([a, np.zeros((5,) + a.shape[1:])]) for n, a in d.items()}
    pad["k"][-5:] = 1.0   # keys of padded tokens are irrelevant when beta = 0 and g = 0
    o2, S_T2 = oracle.gdn_seq(pad["q"], pad["k"], pad["v"], pad["g"], pad["beta"])
    np.testing.assert_allclose(S_T2, S_T, rtol=1e-14)
    np.testing.assert_allclose(o2[:21], o, rtol=1e-14)
    for cut in (1, 8, 20):
        a = {n: x[:cut] for n, x in d.items()}
        b = {n: x[cut:] for n, x in d.items()}
        o_a, S_a = oracle.gdn_seq(a["q"], a["k"], a["v"], a["g"], a["beta"])
        o_b, S_b = oracle.gdn_seq(b["q"], b["k"], b["v"], b["g"], b["beta"], S_a)
        np.testing.assert_allclose(np.concatenate([o_a, o_b]), o, rtol=1e-12, atol=1e-15)
        np.testing.assert_allclose(S_b, S_T, rtol=1e-12, atol=1e-15)
    s = _ssd_inputs(9, 15)
    y, h_T = oracle.ssd_seq(s["x"], s["dt"], s["A"], s["B"], s["C"])
    y_a, h_a = oracle.ssd_seq(s["x"][:6], s["dt"][:6], s["A"], s["B"][:6], s["C"][:6])
    y_b, h_b = oracle.ssd_seq(s["x"][6:], s["dt"][6:], s["A"], s["B"][6:], s["C"][6:], h_a)
    np.testing.assert_allclose(np.concatenate([y_a, y_b]), y, rtol=1e-12, atol=1e-15)
    np.testing.assert_allclose(h_b, h_T, rtol=1e-12, atol=1e-15)
    zpad = np.zeros((3,) + s["dt"].shape[1:])
    _, h_pad = oracle.ssd_seq(np.concatenate([s["x"], np.ones((3,) + s["x"].shape[1:])]),
                              np.concatenate([s["dt"], zpad]), s["A"],
                              np.concatenate([s["B"], np.ones((3,) + s["B"].shape[1:])]),
                              np.concatenate([s["C"], np.ones((3,) + s["C"].shape[1:])]))
    np.testing.assert_allclose(h_pad, h_T, rtol=1e-14)


def test_scan_started_from_identity_yields_transition():
    """With v = 0 and S0 = I (d_v = d_k) the scan's final state is the chunk transition."""
    Hk, Hv, dk = 2, 4, 6
    d = _gdn_inputs(10, 14, Hk, Hv, dk, dk)
    eye = np.broadcast_to(np.eye(dk), (Hv, dk, dk)).copy()
    _, S_T = oracle.gdn_seq(d["q"], d["k"], np.zeros_like(d["v"]), d["g"], d["beta"], eye)
    np.testing.assert_allclose(oracle.gdn_transition(d["k"], d["g"], d["beta"]), S_T, rtol=1e-12, atol=1e-15)


def test_grouped_heads_follow_the_stated_mapping():
    """Value head h reads q/k head h // (H_v // H_k): same result as repeating q/k per value head."""
    d = _gdn_inputs(13, 10, Hk=2, Hv=6, dk=4, dv=3)
    o, S = oracle.gdn_seq(d["q"], d["k"], d["v"], d["g"], d["beta"])
    o2, S2 = oracle.gdn_seq(np.repeat(d["q"], 3, axis=1), np.repeat(d["k"], 3, axis=1), d["v"], d["g"], d["beta"])
    assert np.array_equal(o, o2) and np.array_equal(S, S2)


def test_bf16_round_helper():
    import torch
    x = np.random.default_rng(0).standard_normal(4096).astype(np.float32) * 37.0
    ref = torch.from_numpy(x).to(torch.bfloat16).to(torch.float32).numpy()
    assert np.array_equal(wl.bf16_round(x), ref)


def test_generators_are_seeded_and_shaped():
    a = wl.gdn_tokens(np.random.default_rng(2), 16, 2, 4, 8, 8)
    b = wl.gdn_tokens(np.random.default_rng(2), 16, 2, 4, 8, 8)
    assert all(np.array_equal(a[n], b[n]) for n in a)
    assert (a["g"] <= 0).all() and (a["beta"] > 0).all() and (a["beta"] < 1).all()
    reqs = wl.ragged_mix()
    assert len(reqs) == 64 and all(8192 <= r["total"] <= 32768 and 2 <= r["K"] <= 32 for r in reqs)
    assert [r["family"] for r in reqs].count("gdn") == 32
    assert np.array_equal(wl.request_permutation(3, 0, 32), np.arange(32))
    assert sorted(wl.request_permutation(3, 5, 32).tolist()) == list(range(32))


def test_state_rel_error_closed_forms():
    """Section 3.2 diagnostic: values fixed by hand, not by the formula's own code."""
    ref = np.zeros((3, 2, 4))
    ref[0, 0, 0] = 3.0
    ref[0, 1, 3] = 4.0          # ||ref_0|| = 5
    ref[1] = 1.0                # ||ref_1|| = sqrt(8)
    ref[2, 1, 1] = 2.0
    init = ref.copy()
    init[0, 0, 1] = 5.0         # one entry off by 5 -> 5 / 5
    init[1] *= 1.5              # scaled copy -> |1.5 - 1|
    init[2] = 0.0               # the "empty state" initialiser -> exactly 1
    err = oracle.state_rel_error(init, ref)
    assert np.allclose(err, [1.0, 0.5, 1.0], rtol=0, atol=1e-15)
    assert oracle.state_rel_error(ref, ref).tolist() == [0.0, 0.0, 0.0]
    # one number for the whole array = ratio of the norms of the concatenated vectors
    whole = oracle.state_rel_error(init, ref, n_states=1)
    assert np.isclose(whole[0], np.sqrt(25.0 + 8 * 0.25 + 4.0) / np.sqrt(25.0 + 8.0 + 4.0), rtol=1e-15)
    # sign and order of the arguments matter only through the denominator
    assert np.isclose(oracle.state_rel_error(ref[:1], init[:1])[0], 5.0 / np.sqrt(50.0), rtol=1e-15)

