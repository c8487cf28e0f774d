"""The allocation-free attention entry point (aflex_attn_decode_static) against the regular one.

Some users of this library cannot allocate GPU memory when they call it -- their own memory pool
owns the device, or they run under a host application's allocator rules -- so they cannot create
a context (which owns a workspace).  For them the library carries one entry point whose scratch is
a fixed array inside the library itself.  This test calls it through the C ABI, twice in a row (the
second call finds the first call's leftovers in the shared scratch), and checks both results against
aflex_attn_decode on the same inputs.  It also checks that a batch beyond the scratch's stated
capacity is refused.  The file sorts last on purpose: if it fails under `-x`, every other test has
already run."""
import ctypes

import numpy as np
import pytest
import torch

from paper_2608_01891_b200 import aflex as AF
from paper_2608_01891_b200 import inputs as IN
from tests.helpers import TOL_ATTN, TOL_LSE, f64, row_rel_err

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def _case(Hq, Hkv, D, lens, cid):
    cfg = IN.LayerConfig(cid, "no-alloc", len(lens), Hq, Hkv, D, 0, 0)
    kvh = IN.make_paged_kv(cfg, np.asarray(lens, dtype=np.int32), poison=True)
    q = IN.make_q(cfg).to(DEV)
    kv = AF.make_kv(kvh.k_cache.to(DEV), kvh.v_cache.to(DEV), kvh.page_table.to(DEV), kvh.seq_lens.to(DEV), kvh.seq_lens)
    return q, kv


@pytest.mark.parametrize("Hq,Hkv,D", [(64, 8, 128), (8, 2, 64)])
def test_static_scratch_entry_point_matches_regular_one_twice_in_a_row(Hq, Hkv, D):
    torch.cuda.set_device(0)
    desc = AF.attn_desc(Hq, Hkv, D)
    # two different problems back to back: the second call must not be disturbed by what the first left behind
    cases = [_case(Hq, Hkv, D, [1, 17, 64, 65, 300, 1025, 2500, 4096, 777, 33], 95),
             _case(Hq, Hkv, D, [3000, 5, 129, 2048, 640], 96)]
    ctx = AF.Context(0, 64 << 20)
    try:
        for q, kv in cases:
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
        assert ctx.device_status() == AF.OK
    finally:
        ctx.close()


def test_static_scratch_entry_point_refuses_what_does_not_fit():
    torch.cuda.set_device(0)
    q, kv = _case(8, 2, 64, [5, 6], 97)
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
