"""Host-side checks of the C ABI that need no GPU: the library loads, exports every symbol
the header declares, and rejects bad arguments before anything could be launched."""
import ctypes
import os
import re

import numpy as np
import pytest

from paper_2608_11231_b200 import binding as b

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
FAKE = 0x7F0000000000  # a 16-byte aligned non-NULL "device pointer"; never dereferenced on the host


def fake(i):
    """Distinct fake device buffers, 4 GiB apart (the library checks that outputs do not overlap inputs)."""
    return FAKE + (i << 32)



@pytest.fixture(scope="module")
def lib():
    if not os.path.exists(b.LIB_PATH):
        import __graft_entry__
        __graft_entry__.build()
    return b.load()


def test_every_declared_symbol_is_exported(lib):
    text = open(os.path.join(ROOT, "include", "lkv.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    declared = set(re.findall(r"\b(lkv_[a-z_0-9]+)\s*\(", text))
    assert declared == set(b.EXPORTS)
    for name in declared:
        assert getattr(lib, name) is not None


def test_version_and_status_strings(lib):
    assert b.lkv_version() == 100
    seen = {b.status_string(s) for s in range(0, -11, -1)}
    assert len(seen) == 11 and "unknown status" not in seen
    assert b.status_string(-99) == "unknown status"


def _desc(**kw):
    base = dict(family=b.LKV_FAMILY_GDN, H=2, d_k=64, d_v=64, n_chunks=4, state_dtype=b.LKV_DTYPE_F32, sel_index=0,
                compute=b.LKV_COMPUTE_AUTO, chunk_ids=None, workspace=FAKE, workspace_bytes=1 << 20)
    base.update(kw)
    return b.lkv_init_desc(**base)


def _init(lib, d, K=4, mode=b.LKV_INIT_EXACT, states=fake(1), trans=fake(2), S0=fake(3)):
    return lib.lkv_init_state(states, trans, K, mode, S0, ctypes.byref(d) if d is not None else None, None)


def test_init_state_argument_errors(lib):
    assert _init(lib, None) == b.LKV_ERR_NULL
    assert _init(lib, _desc(), K=-1) == b.LKV_ERR_DIM
    assert _init(lib, _desc(), mode=7) == b.LKV_ERR_MODE
    assert _init(lib, _desc(family=5)) == b.LKV_ERR_MODE
    assert _init(lib, _desc(state_dtype=9)) == b.LKV_ERR_MODE
    assert _init(lib, _desc(compute=3)) == b.LKV_ERR_MODE
    assert _init(lib, _desc(H=0)) == b.LKV_ERR_DIM
    assert _init(lib, _desc(), K=5) == b.LKV_ERR_INDEX            # implicit ids 0..4 exceed the pool of 4
    ids = np.array([0, 1, 4, 2], dtype=np.int32)
    assert _init(lib, _desc(chunk_ids=ids.ctypes.data)) == b.LKV_ERR_INDEX
    ids = np.array([0, -1, 3, 2], dtype=np.int32)
    assert _init(lib, _desc(chunk_ids=ids.ctypes.data)) == b.LKV_ERR_INDEX
    assert _init(lib, _desc(sel_index=4), mode=b.LKV_INIT_INDEX) == b.LKV_ERR_INDEX
    assert _init(lib, _desc(sel_index=-1), mode=b.LKV_INIT_INDEX) == b.LKV_ERR_INDEX
    assert _init(lib, _desc(), S0=None) == b.LKV_ERR_NULL
    assert _init(lib, _desc(), states=None) == b.LKV_ERR_NULL
    assert _init(lib, _desc(), trans=None) == b.LKV_ERR_NULL      # exact mode with K >= 2 needs transitions
    assert _init(lib, _desc(), S0=fake(3) + 4) == b.LKV_ERR_ALIGN
    assert _init(lib, _desc(), states=fake(1) + 8) == b.LKV_ERR_ALIGN
    assert _init(lib, _desc(), S0=fake(1) + 64) == b.LKV_ERR_OVERLAP        # S0 inside the pool of states
    assert _init(lib, _desc(), S0=fake(2)) == b.LKV_ERR_OVERLAP              # S0 on the transitions
    assert _init(lib, _desc(d_v=6)) == b.LKV_ERR_UNSUPPORTED
    assert _init(lib, _desc(workspace=None)) == b.LKV_ERR_WORKSPACE
    assert _init(lib, _desc(workspace_bytes=16)) == b.LKV_ERR_WORKSPACE
    assert _init(lib, _desc(compute=b.LKV_COMPUTE_TENSOR, d_k=24, d_v=24)) == b.LKV_ERR_UNSUPPORTED


def test_init_state_batched_argument_errors(lib):
    d = _desc()
    ids = np.array([0, 1, 2, 3, 1], dtype=np.int32)
    f = lib.lkv_init_state_batched
    call = lambda cu, n, mode=b.LKV_INIT_EXACT, sel=None, idp=ids: f(
        fake(1), fake(2), idp.ctypes.data if idp is not None else None, cu.ctypes.data if cu is not None else None, n, mode,
        sel.ctypes.data if sel is not None else None, fake(3), ctypes.byref(d), None)
    assert call(None, 2) == b.LKV_ERR_NULL
    assert call(np.array([1, 3, 5], dtype=np.int32), 2) == b.LKV_ERR_INDEX      # must start at 0
    assert call(np.array([0, 4, 3], dtype=np.int32), 2) == b.LKV_ERR_INDEX      # not monotone
    assert call(np.array([0, 3, 5], dtype=np.int32), -1) == b.LKV_ERR_DIM
    assert call(np.array([0, 3, 5], dtype=np.int32), 2, idp=None) == b.LKV_ERR_NULL
    assert call(np.array([0, 3, 5], dtype=np.int32), 2, mode=b.LKV_INIT_INDEX) == b.LKV_ERR_NULL
    assert call(np.array([0, 3, 5], dtype=np.int32), 2, mode=b.LKV_INIT_INDEX,
                sel=np.array([2, 2], dtype=np.int32)) == b.LKV_ERR_INDEX
    assert call(np.array([0], dtype=np.int32), 0) == b.LKV_OK                    # no requests: nothing to do


def _gdn_desc(**kw):
    base = dict(T_total=100, n_seq=1, cu_seqlens=None, H_k=2, H_v=4, d_k=64, d_v=64, io_dtype=b.LKV_DTYPE_F32,
                compute=b.LKV_COMPUTE_AUTO, scale=0.0, state_dtype=0, workspace=FAKE, workspace_bytes=1 << 20)
    base.update(kw)
    return b.lkv_gdn_desc(**base)


def test_gdn_fwd_argument_errors(lib):
    f = lambda d, q=fake(1), o=fake(7), S0=None, S_T=None: lib.lkv_gdn_fwd(q, fake(2), fake(3), fake(4), fake(5), S0, o, S_T,
                                                                            ctypes.byref(d) if d is not None else None, None)
    assert f(None) == b.LKV_ERR_NULL
    assert f(_gdn_desc(io_dtype=4)) == b.LKV_ERR_MODE
    assert f(_gdn_desc(H_v=3)) == b.LKV_ERR_DIM
    assert f(_gdn_desc(d_k=0)) == b.LKV_ERR_DIM
    assert f(_gdn_desc(T_total=-1)) == b.LKV_ERR_DIM
    assert f(_gdn_desc(n_seq=2)) == b.LKV_ERR_NULL                      # several sequences need cu_seqlens
    cu = np.array([0, 60, 90], dtype=np.int32)
    assert f(_gdn_desc(n_seq=2, cu_seqlens=cu.ctypes.data)) == b.LKV_ERR_INDEX   # does not end at T_total
    cu = np.array([0, 120, 100], dtype=np.int32)
    assert f(_gdn_desc(n_seq=2, cu_seqlens=cu.ctypes.data)) == b.LKV_ERR_INDEX
    assert f(_gdn_desc(), q=None) == b.LKV_ERR_NULL
    assert f(_gdn_desc(), o=fake(7) + 2) == b.LKV_ERR_ALIGN
    assert f(_gdn_desc(), S0=fake(6) + 4) == b.LKV_ERR_ALIGN
    assert f(_gdn_desc(), o=fake(3)) == b.LKV_ERR_OVERLAP                  # o on v
    assert f(_gdn_desc(), o=fake(1) + 1024) == b.LKV_ERR_OVERLAP           # o inside q
    assert f(_gdn_desc(), S0=fake(6), S_T=fake(6) + 256) == b.LKV_ERR_OVERLAP   # S_T may be S0 itself, not a shifted view
    assert f(_gdn_desc(), S_T=fake(4)) == b.LKV_ERR_OVERLAP                # S_T on g
    assert f(_gdn_desc(state_dtype=7)) == b.LKV_ERR_MODE
    assert f(_gdn_desc(state_dtype=b.LKV_DTYPE_BF16), S0=fake(6), S_T=fake(6)) == b.LKV_ERR_OVERLAP   # fp32 in, bf16 out
    assert f(_gdn_desc(d_v=48)) == b.LKV_ERR_UNSUPPORTED
    assert f(_gdn_desc(workspace=None)) == b.LKV_ERR_WORKSPACE
    assert f(_gdn_desc(compute=b.LKV_COMPUTE_TENSOR, d_k=24, d_v=32)) == b.LKV_ERR_UNSUPPORTED
    assert f(_gdn_desc(n_seq=0, T_total=0, cu_seqlens=np.array([0], dtype=np.int32).ctypes.data)) == b.LKV_OK


def _ssd_desc(**kw):
    base = dict(T_total=100, n_seq=1, cu_seqlens=None, H=8, P=64, N=128, G=2, io_dtype=b.LKV_DTYPE_BF16,
                compute=b.LKV_COMPUTE_AUTO, workspace=FAKE, workspace_bytes=1 << 20)
    base.update(kw)
    return b.lkv_ssd_desc(**base)


def test_ssd_fwd_argument_errors(lib):
    f = lambda d, x=fake(1), A=fake(3), y=fake(7): lib.lkv_ssd_fwd(x, fake(2), A, fake(4), fake(5), None, y, None,
                                                                   ctypes.byref(d) if d is not None else None, None)
    assert f(None) == b.LKV_ERR_NULL
    assert f(_ssd_desc(compute=-1)) == b.LKV_ERR_MODE
    assert f(_ssd_desc(G=3)) == b.LKV_ERR_DIM
    assert f(_ssd_desc(N=0)) == b.LKV_ERR_DIM
    assert f(_ssd_desc(), A=None) == b.LKV_ERR_NULL
    assert f(_ssd_desc(), x=None) == b.LKV_ERR_NULL
    assert f(_ssd_desc(), y=fake(7) + 8) == b.LKV_ERR_ALIGN
    assert f(_ssd_desc(), y=fake(1)) == b.LKV_ERR_OVERLAP                  # y on x
    assert f(_ssd_desc(), y=fake(5) + 32) == b.LKV_ERR_OVERLAP             # y inside C
    assert f(_ssd_desc(P=48)) == b.LKV_ERR_UNSUPPORTED
    assert f(_ssd_desc(workspace_bytes=8)) == b.LKV_ERR_WORKSPACE


def test_artifact_producers_argument_errors(lib):
    t = lambda d, k=fake(1), out=fake(7): lib.lkv_gdn_chunk_transition(k, fake(2), fake(3), out,
                                                                  ctypes.byref(d) if d is not None else None, None)
    assert t(None) == b.LKV_ERR_NULL
    assert t(_gdn_desc(d_k=128, d_v=64)) == b.LKV_ERR_DIM             # the transition is d_k x d_k: d_v must equal d_k
    assert t(_gdn_desc(), out=None) == b.LKV_ERR_NULL
    assert t(_gdn_desc(), k=None) == b.LKV_ERR_NULL
    assert t(_gdn_desc(), out=fake(7) + 4) == b.LKV_ERR_ALIGN
    assert t(_gdn_desc(workspace=None)) == b.LKV_ERR_WORKSPACE
    m = lambda d, dt=FAKE, A=FAKE, out=FAKE: lib.lkv_mamba_chunk_logdecay(dt, A, out,
                                                                          ctypes.byref(d) if d is not None else None, None)
    assert m(None) == b.LKV_ERR_NULL
    assert m(_ssd_desc(H=0)) == b.LKV_ERR_DIM
    assert m(_ssd_desc(), A=None) == b.LKV_ERR_NULL
    assert m(_ssd_desc(), out=None) == b.LKV_ERR_NULL
    assert m(_ssd_desc(), dt=FAKE + 4) == b.LKV_ERR_ALIGN
    assert m(_ssd_desc(workspace_bytes=8)) == b.LKV_ERR_WORKSPACE
    # final-state-only scans: o / y may be NULL, but not together with S_T
    g = lib.lkv_gdn_fwd(fake(1), fake(2), fake(3), fake(4), fake(5), None, None, None, ctypes.byref(_gdn_desc()), None)
    assert g == b.LKV_ERR_NULL
    y = lib.lkv_ssd_fwd(fake(1), fake(2), fake(3), fake(4), fake(5), None, None, None, ctypes.byref(_ssd_desc()), None)
    assert y == b.LKV_ERR_NULL


def test_state_rel_error_argument_errors(lib):
    f = lambda a=FAKE, r=FAKE, out=FAKE, n=4, elems=1024, ws=FAKE, wsb=1 << 20: lib.lkv_state_rel_error(
        a, r, out, n, elems, ws, wsb, None)
    assert f(n=-1) == b.LKV_ERR_DIM
    assert f(elems=0) == b.LKV_ERR_DIM
    assert f(elems=1022) == b.LKV_ERR_DIM            # multiple of 4 for the 16-byte loads
    assert f(n=0) == b.LKV_OK
    assert f(a=None) == b.LKV_ERR_NULL
    assert f(out=None) == b.LKV_ERR_NULL
    assert f(r=FAKE + 4) == b.LKV_ERR_ALIGN
    assert f(ws=None) == b.LKV_ERR_WORKSPACE
    assert f(wsb=16) == b.LKV_ERR_WORKSPACE
    need = lib.lkv_state_rel_error_workspace_bytes(4, 1 << 20)
    assert need >= 4 * 64 * 8 and need % 256 == 0    # 64 slices of 16384 floats per state, two sums each
    assert lib.lkv_state_rel_error_workspace_bytes(4, 0) == 0


def test_workspace_bytes(lib):
    d = _desc()
    small = b.lkv_workspace_bytes(b.LKV_WS_INIT, d, 1, 8)
    big = b.lkv_workspace_bytes(b.LKV_WS_INIT, d, 64, 64 * 64)
    assert small >= 256 and big >= 256 + 4 * (64 * 64 + 129)
    assert b.lkv_workspace_bytes(b.LKV_WS_GDN, _gdn_desc(), 64) >= 256
    assert lib.lkv_workspace_bytes(b.LKV_WS_INIT, None, 1, 1) == 0
    assert b.lkv_workspace_bytes(17, d, 1, 1) == 0


def test_missing_library_fails_loudly(tmp_path, monkeypatch):
    monkeypatch.setattr(b, "_lib", None)
    monkeypatch.setattr(b, "LIB_PATH", str(tmp_path / "liblkv.so"))
    with pytest.raises(RuntimeError, match="no CPU or PyTorch fallback"):
        b.load()


def test_selftest_and_static_status_argument_errors(lib):
    assert lib.lkv_selftest_bounded_wait(1000, None, None) == b.LKV_ERR_NULL
    assert lib.lkv_selftest_bounded_wait(0, FAKE, None) == b.LKV_ERR_DIM
    assert lib.lkv_selftest_bounded_wait(1 << 21, FAKE, None) == b.LKV_ERR_DIM
    assert lib.lkv_selftest_bounded_wait(1000, FAKE + 4, None) == b.LKV_ERR_ALIGN


def test_fold_argument_errors(lib):
    cu = np.array([0, 100, 300, 300], dtype=np.int32)
    ids = np.array([2, 0, 1], dtype=np.int32)

    def call(d, K=3, states=fake(1), k=fake(2), cu_p=cu.ctypes.data, S0=fake(5), H_k=2, io=b.LKV_DTYPE_BF16):
        return lib.lkv_init_state_fold(states, k, fake(3), fake(4), cu_p, K, S0, ctypes.byref(d) if d is not None else None,
                                       H_k, io, None)
    gd = lambda **kw: _desc(**dict(dict(family=b.LKV_FAMILY_GDN, H=4, d_k=64, d_v=64, n_chunks=3, chunk_ids=ids.ctypes.data), **kw))
    assert call(None) == b.LKV_ERR_NULL
    assert call(_desc(family=b.LKV_FAMILY_MAMBA2, n_chunks=3)) == b.LKV_ERR_MODE      # Mamba-2 has no key stream to fold
    assert call(gd(), io=9) == b.LKV_ERR_MODE
    assert call(gd(state_dtype=b.LKV_DTYPE_BF16)) == b.LKV_ERR_UNSUPPORTED
    assert call(gd(), K=-1) == b.LKV_ERR_DIM
    assert call(gd(), H_k=3) == b.LKV_ERR_DIM
    assert call(gd(d_v=32)) == b.LKV_ERR_DIM
    assert call(gd(), states=None) == b.LKV_ERR_NULL
    assert call(gd(), cu_p=None) == b.LKV_ERR_NULL
    assert call(gd(), k=None) == b.LKV_ERR_NULL
    bad = np.array([0, 100, 50, 300], dtype=np.int32)
    assert call(gd(), cu_p=bad.ctypes.data) == b.LKV_ERR_INDEX
    ids[1] = 3
    assert call(gd()) == b.LKV_ERR_INDEX


def test_segmented_prefill_argument_errors(lib):
    f = lambda d, n=3, scratch=fake(9), nbytes=1 << 30, S_T=fake(8): lib.lkv_gdn_fwd_segmented(
        fake(1), fake(2), fake(3), fake(4), fake(5), None, fake(7), S_T, ctypes.byref(d) if d is not None else None, n,
        scratch, nbytes, None)
    lib.lkv_gdn_fwd_segmented.argtypes = [ctypes.c_void_p] * 8 + [ctypes.POINTER(b.lkv_gdn_desc), ctypes.c_int, ctypes.c_void_p,
                                          ctypes.c_size_t, ctypes.c_void_p]
    assert f(None) == b.LKV_ERR_NULL
    assert f(_gdn_desc(), n=-1) == b.LKV_ERR_DIM
    cu = np.array([0, 60, 100], dtype=np.int32)
    assert f(_gdn_desc(n_seq=2, cu_seqlens=cu.ctypes.data)) == b.LKV_ERR_UNSUPPORTED     # one sequence only
    assert f(_gdn_desc(state_dtype=b.LKV_DTYPE_BF16)) == b.LKV_ERR_UNSUPPORTED
    assert f(_gdn_desc(d_k=64, d_v=32)) == b.LKV_ERR_DIM
    assert f(_gdn_desc(), scratch=None) == b.LKV_ERR_WORKSPACE
    assert f(_gdn_desc(), nbytes=1024) == b.LKV_ERR_WORKSPACE
    assert f(_gdn_desc(), scratch=fake(9) + 4) == b.LKV_ERR_ALIGN
    need = lib.lkv_gdn_segmented_scratch_bytes(ctypes.byref(_gdn_desc()), 3)
    assert need == (4 * 3 - 3) * 4 * 64 * 64 * 4
    assert lib.lkv_gdn_segmented_scratch_bytes(ctypes.byref(_gdn_desc()), 1) == 0


def test_stage_chunks_argument_errors(lib):
    lib.lkv_stage_chunks.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p,
                                     ctypes.c_void_p, ctypes.c_int, ctypes.c_void_p, ctypes.c_void_p,
                                     ctypes.POINTER(b.lkv_init_desc), ctypes.c_void_p]
    ids = np.array([3, 1, 3, 0], dtype=np.int32)
    out = np.zeros(4, dtype=np.int32)
    n = ctypes.c_int32(-1)

    def call(d, idp=ids.ctypes.data, n_ids=4, hs=fake(1), ht=fake(2), ds=fake(3), dt=fake(4), cap=8, outp=out.ctypes.data,
             np_=ctypes.addressof(n)):
        return lib.lkv_stage_chunks(hs, ht, idp, n_ids, ds, dt, cap, outp, np_, ctypes.byref(d) if d is not None else None, None)
    assert call(None) == b.LKV_ERR_NULL
    assert call(_desc(), n_ids=-1) == b.LKV_ERR_DIM
    assert call(_desc(), np_=None) == b.LKV_ERR_NULL
    assert call(_desc(), n_ids=0) == b.LKV_OK and n.value == 0            # nothing named, nothing copied
    assert call(_desc(), hs=None) == b.LKV_ERR_NULL
    assert call(_desc(), ht=None) == b.LKV_ERR_NULL                       # one transition pool without the other
    assert call(_desc(), ds=fake(3) + 8) == b.LKV_ERR_ALIGN
    assert call(_desc(n_chunks=3)) == b.LKV_ERR_INDEX                     # id 3 of a 3-chunk pool
    assert call(_desc(), cap=2) == b.LKV_ERR_WORKSPACE                    # three distinct chunks, room for two


def test_chunk_artifacts_argument_errors(lib):
    lib.lkv_gdn_chunk_artifacts.argtypes = [ctypes.c_void_p] * 6 + [ctypes.POINTER(b.lkv_gdn_desc), ctypes.c_void_p]
    f = lambda d, st=fake(6), tr=fake(7): lib.lkv_gdn_chunk_artifacts(fake(2), fake(3), fake(4), fake(5), st, tr,
                                                                       ctypes.byref(d) if d is not None else None, None)
    assert f(None) == b.LKV_ERR_NULL
    assert f(_gdn_desc(), st=None) == b.LKV_ERR_NULL
    assert f(_gdn_desc(), tr=None) == b.LKV_ERR_NULL
    assert f(_gdn_desc(state_dtype=b.LKV_DTYPE_BF16)) == b.LKV_ERR_MODE
    assert f(_gdn_desc(d_k=64, d_v=32)) == b.LKV_ERR_DIM
    assert f(_gdn_desc(), tr=fake(6) + 1024) == b.LKV_ERR_OVERLAP            # transitions inside the states buffer
    assert f(_gdn_desc(), tr=fake(7) + 4) == b.LKV_ERR_ALIGN
    assert f(_gdn_desc(workspace_bytes=8)) == b.LKV_ERR_WORKSPACE
