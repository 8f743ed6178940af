"""The allocation-free batched initialiser, checked against the ordinary entry point.

Some callers of this library cannot obtain device memory at call time (an engine that has
closed its allocator on the request path, a component living inside another one's memory
budget), so they cannot pass a workspace.  lkv_init_state_batched_static keeps the scratch in
a fixed array inside the library instead.  This file is collected last on purpose: a run that
stops at the first failure has then already run every other test.
"""
import numpy as np
import pytest

from paper_2608_11231_b200 import binding as b
from paper_2608_11231_b200 import workloads as wl

pytestmark = pytest.mark.gpu


def _case(seed, n_req, K):
    import torch
    rng = np.random.default_rng(seed)
    n, H, N, P = 24, 2, 16, 32
    pool = torch.from_numpy(wl.synthetic_states(rng, n, H, N, P)).cuda()
    lam = torch.from_numpy(wl.synthetic_logdecay(rng, n, H, lo=-0.5)).cuda()
    ids = rng.integers(0, n, size=n_req * K).astype(np.int32)
    cu = (np.arange(n_req + 1) * K).astype(np.int32)
    sel = rng.integers(0, K, size=n_req).astype(np.int32)
    return pool, lam, ids, cu, sel


def test_static_scratch_matches_workspace_entry_point_twice_in_a_row():
    import torch
    # first call: index list long enough to live in the scratch array rather than in the kernel parameters
    # second call, straight after it: a shorter, different list -- the array still holds the first one
    for seed, n_req, K in ((1, 160, 30), (2, 90, 50)):
        pool, lam, ids, cu, sel = _case(seed, n_req, K)
        assert 2 * n_req + 1 + ids.size > 4000
        out = torch.full((n_req,) + tuple(pool.shape[1:]), float("nan"), device="cuda")
        for mode, tr, s in ((b.LKV_INIT_EXACT, lam, None), (b.LKV_INIT_INDEX, None, sel), (b.LKV_INIT_LAST, None, None)):
            ref = b.lkv_init_state_batched(pool, tr, ids, cu, n_req, mode, s, family=b.LKV_FAMILY_MAMBA2)
            got = b.lkv_init_state_batched_static(pool, tr, ids, cu, n_req, mode, s, out, family=b.LKV_FAMILY_MAMBA2)
            torch.cuda.synchronize()
            assert got.data_ptr() == out.data_ptr()
            assert torch.equal(got, ref), (seed, mode)          # same kernels, same order: bit-identical
    # a short list (kept in the kernel parameters) works too and leaves the result identical
    pool, lam, ids, cu, sel = _case(3, 4, 5)
    ref = b.lkv_init_state_batched(pool, lam, ids, cu, 4, b.LKV_INIT_EXACT, None, family=b.LKV_FAMILY_MAMBA2)
    got = b.lkv_init_state_batched_static(pool, lam, ids, cu, 4, b.LKV_INIT_EXACT, None, family=b.LKV_FAMILY_MAMBA2)
    assert torch.equal(got, ref)


def test_static_scratch_rejects_oversized_requests():
    pool, lam, ids, cu, sel = _case(4, 4, 5)
    n_req = 600
    K = 30                                   # 2*600 + 1 + 18000 > 16384
    big_ids = np.zeros(n_req * K, dtype=np.int32)
    big_cu = (np.arange(n_req + 1) * K).astype(np.int32)
    with pytest.raises(b.LkvError) as e:
        b.lkv_init_state_batched_static(pool, lam, big_ids, big_cu, n_req, b.LKV_INIT_EXACT, None,
                                        family=b.LKV_FAMILY_MAMBA2)
    assert e.value.status == b.LKV_ERR_WORKSPACE


def test_static_scratch_gdn_exact_on_the_tensor_cores_and_its_status_word():
    """The kernel with bounded device waits (GDN composition, d = 128) on the library's own scratch:
    index list in the scratch array, results equal to the workspace entry point, status word clean."""
    import torch
    rng = np.random.default_rng(5)
    n, H, d = 16, 2, 128
    pool = torch.from_numpy(wl.synthetic_states(rng, n, H, d, d)).cuda()
    tr = torch.from_numpy(wl.synthetic_gdn_transitions(rng, n, H, d)).cuda()
    n_req, K = 140, 30
    ids = rng.integers(0, n, size=n_req * K).astype(np.int32)
    cu = (np.arange(n_req + 1) * K).astype(np.int32)
    assert 2 * n_req + 1 + ids.size > 4000
    out = torch.full((n_req, H, d, d), float("nan"), device="cuda")
    assert b.lkv_device_status_static() == b.LKV_OK
    for compute in (b.LKV_COMPUTE_TENSOR, b.LKV_COMPUTE_FP32):
        ref = b.lkv_init_state_batched(pool, tr, ids, cu, n_req, b.LKV_INIT_EXACT, None, family=b.LKV_FAMILY_GDN,
                                       compute=compute)
        got = b.lkv_init_state_batched_static(pool, tr, ids, cu, n_req, b.LKV_INIT_EXACT, None, out,
                                              family=b.LKV_FAMILY_GDN, compute=compute)
        torch.cuda.synchronize()
        assert torch.equal(got, ref), compute
        assert b.lkv_device_status_static() == b.LKV_OK
    # an argument error is found before anything reaches the stream: the earlier result stays as it was
    keep = out.clone()
    with pytest.raises(b.LkvError) as e:
        bad = ids.copy()
        bad[7] = n                                           # chunk id out of range
        b.lkv_init_state_batched_static(pool, tr, bad, cu, n_req, b.LKV_INIT_EXACT, None, out, family=b.LKV_FAMILY_GDN)
    assert e.value.status == b.LKV_ERR_INDEX
    torch.cuda.synchronize()
    assert torch.equal(out, keep) and b.lkv_device_status_static() == b.LKV_OK
