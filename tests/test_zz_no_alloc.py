"""The allocation-free attention entry point (aflex_attn_decode_static) against the regular one.

Some users of this library cannot allocate GPU memory when they call it -- their own memory pool
owns the device, or they run under a host application's allocator rules -- so they cannot create
a context (which owns a workspace).  For them the library carries one entry point whose scratch is
a fixed array inside the library itself.  This test calls it through the C ABI, twice in a row (the
second call finds the first call's leftovers in the shared scratch), and checks both results against
aflex_attn_decode on the same inputs.  It also checks that a batch beyond the scratch's stated
capacity is refused.  The file sorts last on purpose: if it fails under `-x`, every other test has
already run.  Both calls are also compared with the fp64 oracle (the static path cuts the work into
its own shares, so agreement with the regular entry point alone would not show a defect the two
share), and the status reader that goes with the entry point is checked on a clamped length, a
redirected page id and a sequence of length 0 between valid rows."""
import ctypes

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2608_01891_b200 import aflex as AF
from paper_2608_01891_b200 import inputs as IN
from tests.helpers import TOL_ATTN, TOL_LSE, f64, row_rel_err, u16

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(Hq, Hkv, D, lens, cid):
    cfg = IN.LayerConfig(cid, "no-alloc", len(lens), Hq, Hkv, D, 0, 0)
    kvh = IN.make_paged_kv(cfg, np.asarray(lens, dtype=np.int32), poison=True)
    qh = IN.make_q(cfg)
    q = qh.to(DEV)
    kv = AF.make_kv(kvh.k_cache.to(DEV), kvh.v_cache.to(DEV), kvh.page_table.to(DEV), kvh.seq_lens.to(DEV), kvh.seq_lens)
    return q, kv, qh, kvh


def _oracle(qh, kvh, rows=None):
    rows = np.arange(qh.shape[0]) if rows is None else rows
    return O.attn_decode(u16(qh[rows]), u16(kvh.k_cache), u16(kvh.v_cache), kvh.page_table.numpy()[rows],
                         kvh.seq_lens.numpy()[rows])


@pytest.mark.parametrize("Hq,Hkv,D", [(64, 8, 128), (8, 2, 64)])
def test_static_scratch_entry_point_matches_regular_one_twice_in_a_row(Hq, Hkv, D):
    torch.cuda.set_device(0)
    desc = AF.attn_desc(Hq, Hkv, D)
    # two different problems back to back: the second call must not be disturbed by what the first left behind
    cases = [_case(Hq, Hkv, D, [1, 17, 64, 65, 300, 1025, 2500, 4096, 777, 33], 95),
             _case(Hq, Hkv, D, [3000, 5, 129, 2048, 640], 96)]
    ctx = AF.Context(0, 64 << 20)
    try:
        for q, kv, qh, kvh in cases:
            want = torch.full_like(q, float("nan"))
            want_lse = torch.full((q.shape[0], Hq), float("nan"), device=DEV)
            ctx.attn_decode(desc, q, kv, want, want_lse)
            got = torch.full_like(q, float("nan"))
            got_lse = torch.full((q.shape[0], Hq), float("nan"), device=DEV)
            AF.attn_decode_static(desc, q, kv, got, got_lse)
            torch.cuda.synchronize()
            assert torch.isfinite(got.float()).all()
            assert row_rel_err(f64(got), f64(want)) <= TOL_ATTN
            assert np.abs(f64(got_lse) - f64(want_lse)).max() <= TOL_LSE
            ref, ref_lse = _oracle(qh, kvh)
            assert row_rel_err(f64(got), ref) <= TOL_ATTN
            assert np.abs(f64(got_lse) - ref_lse).max() <= TOL_LSE
            assert AF.attn_decode_static_status() == AF.OK
        assert ctx.device_status() == AF.OK
    finally:
        ctx.close()


def test_static_scratch_status_reports_what_the_kernel_met():
    """Without a context there is no device status to poll, so the entry point has a reader of its own.  A page id
    beyond the pool (the load goes to page 0 instead), a length beyond the page-table row (clamped) and a length
    of 0 between valid rows (no output for that row) each read back as ERR_BOUNDS; no case faults, the valid rows
    of the last case match the oracle, and a clean call afterwards reads OK again."""
    torch.cuda.set_device(0)
    Hq, Hkv, D = 8, 2, 64
    desc = AF.attn_desc(Hq, Hkv, D)
    q, kv, qh, kvh = _case(Hq, Hkv, D, [40, 70, 900], 98)
    out = torch.empty_like(q)
    AF.attn_decode_static(desc, q, kv, out)
    assert AF.attn_decode_static_status() == AF.OK
    table = kvh.page_table.clone()
    table[1, 2] = kvh.num_pages + 12345
    kv_bad = AF.make_kv(kvh.k_cache.to(DEV), kvh.v_cache.to(DEV), table.to(DEV), kvh.seq_lens.to(DEV), None)
    AF.attn_decode_static(desc, q, kv_bad, out)
    assert AF.attn_decode_static_status() == AF.ERR_BOUNDS
    lens = kvh.seq_lens.clone()
    lens[1] = 16 * kvh.page_table.shape[1] + 500
    kv_bad = AF.make_kv(kvh.k_cache.to(DEV), kvh.v_cache.to(DEV), kvh.page_table.to(DEV), lens.to(DEV), None)
    AF.attn_decode_static(desc, q, kv_bad, out)
    assert AF.attn_decode_static_status() == AF.ERR_BOUNDS
    # lengths of 0 in front, in the middle (a run of three) and at the end of a batch whose other rows are split over CTAs
    rng = np.random.default_rng(3)
    n_seq = 40
    true_lens = rng.integers(300, 2500, size=n_seq)
    zero = rng.random(n_seq) < 0.35
    zero[0] = zero[-1] = True
    zero[20:23] = True
    for (hq, hkv, d) in ((8, 2, 64), (64, 8, 128)):
        desc = AF.attn_desc(hq, hkv, d)
        q, kv, qh, kvh = _case(hq, hkv, d, true_lens.tolist(), 99)
        lens = kvh.seq_lens.clone()
        lens[torch.from_numpy(zero)] = 0
        kv0 = AF.make_kv(kvh.k_cache.to(DEV), kvh.v_cache.to(DEV), kvh.page_table.to(DEV), lens.to(DEV), None)
        got = torch.full_like(q, float("nan"))
        got_lse = torch.full((n_seq, hq), float("nan"), device=DEV)
        AF.attn_decode_static(desc, q, kv0, got, got_lse)
        assert AF.attn_decode_static_status() == AF.ERR_BOUNDS
        valid = np.flatnonzero(~zero)
        ref, ref_lse = _oracle(qh, kvh, valid)
        assert row_rel_err(f64(got)[valid], ref) <= TOL_ATTN
        assert np.abs(f64(got_lse)[valid] - ref_lse).max() <= TOL_LSE
        assert torch.isnan(got.float()[torch.from_numpy(zero).to(DEV)]).all()
        AF.attn_decode_static(desc, q, kv, got)
        assert AF.attn_decode_static_status() == AF.OK
        assert row_rel_err(f64(got), _oracle(qh, kvh)[0]) <= TOL_ATTN


def test_static_scratch_entry_point_refuses_what_does_not_fit():
    torch.cuda.set_device(0)
    q, kv, _, _ = _case(8, 2, 64, [5, 6], 97)
    out = torch.empty_like(q)
    lib = AF.load_library()
    st = torch.cuda.current_stream().cuda_stream
    desc = AF.attn_desc(8, 2, 64)
    too_many = 16384 // 2 + 1                      # batch * Hkv > 16384: validated before any pointer is used
    assert lib.aflex_attn_decode_static(ctypes.byref(desc), q.data_ptr(), ctypes.byref(kv), too_many, out.data_ptr(),
                                        None, st) == AF.ERR_WORKSPACE
    bad = AF.attn_desc(8, 2, 96)
    assert lib.aflex_attn_decode_static(ctypes.byref(bad), q.data_ptr(), ctypes.byref(kv), 2, out.data_ptr(),
                                        None, st) == AF.ERR_UNSUPPORTED
    with pytest.raises(AF.AflexError):
        AF.attn_decode_static(desc, q, kv, None)
    torch.cuda.synchronize()
