"""Parity of prefill (causal) attention against the fp64 oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2608_01891_b200 import aflex as AF
from paper_2608_01891_b200 import inputs as IN
from tests.helpers import TOL_ATTN, f64, row_rel_err, u16

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def run_case(ctx, Hq, Hkv, D, lens, q_lens, seed, poison=True):
    cfg = IN.LayerConfig(20 + seed, "prefill", len(lens), Hq, Hkv, D, 64, 64)
    lens = np.asarray(lens, dtype=np.int32)
    kvh = IN.make_paged_kv(cfg, lens, poison=poison)
    q_off = np.concatenate([[0], np.cumsum(q_lens)]).astype(np.int32)
    T = int(q_off[-1])
    g = torch.Generator().manual_seed(seed)
    q = torch.randn(T, Hq, D, generator=g).to(torch.bfloat16)
    kv = AF.make_kv(kvh.k_cache.to(DEV), kvh.v_cache.to(DEV), kvh.page_table.to(DEV), kvh.seq_lens.to(DEV), kvh.seq_lens)
    out = torch.full((T, Hq, D), float("nan"), dtype=torch.bfloat16, device=DEV)
    qo = torch.from_numpy(q_off)
    ctx.attn_prefill(AF.attn_desc(Hq, Hkv, D), q.to(DEV), kv, qo.to(DEV), qo, out)
    torch.cuda.synchronize()
    assert ctx.device_status() == AF.OK
    ko, vo = u16(kvh.k_cache), u16(kvh.v_cache)
    if poison:      # the oracle never reads unreferenced slots, but keep its inputs finite anyway
        ko, vo = ko.copy(), vo.copy()
    want = O.attn_prefill(u16(q), ko, vo, kvh.page_table.numpy(), lens, q_off)
    return f64(out), want


@pytest.fixture(scope="module")
def ctx():
    c = AF.Context(0, 1 << 26)
    yield c
    c.close()


@pytest.mark.parametrize("Hq,Hkv,D", [(8, 2, 128), (4, 4, 64), (16, 2, 64)])
def test_prefill_whole_prompts_ragged(ctx, Hq, Hkv, D):
    lens = [1, 17, 128, 129, 300, 64, 255]
    got, want = run_case(ctx, Hq, Hkv, D, lens, lens, seed=1)
    assert row_rel_err(got, want) <= TOL_ATTN


def test_prefill_chunk_behind_existing_context(ctx):
    lens = [500, 130, 1000, 77]
    q_lens = [100, 130, 1, 33]          # a chunk, a whole prompt, a single token (decode), a short tail
    got, want = run_case(ctx, 8, 2, 128, lens, q_lens, seed=2)
    assert row_rel_err(got, want) <= TOL_ATTN


def test_prefill_single_token_rows_equal_decode_attention(ctx):
    lens = [40, 200, 9]
    got, want = run_case(ctx, 8, 2, 128, lens, [1, 1, 1], seed=3)
    assert row_rel_err(got, want) <= TOL_ATTN
    # and the decode kernel agrees on the same inputs
    cfg = IN.LayerConfig(23, "prefill", 3, 8, 2, 128, 64, 64)
    kvh = IN.make_paged_kv(cfg, np.asarray(lens, dtype=np.int32), poison=True)
    g = torch.Generator().manual_seed(3)
    q = torch.randn(3, 8, 128, generator=g).to(torch.bfloat16)
    kv = AF.make_kv(kvh.k_cache.to(DEV), kvh.v_cache.to(DEV), kvh.page_table.to(DEV), kvh.seq_lens.to(DEV), kvh.seq_lens)
    out = torch.empty(3, 8, 128, dtype=torch.bfloat16, device=DEV)
    ctx.attn_decode(AF.attn_desc(8, 2, 128), q.to(DEV), kv, out)
    torch.cuda.synchronize()
    assert row_rel_err(f64(out), got) <= TOL_ATTN


def test_prefill_long_prompt_and_empty_sequence_and_determinism(ctx):
    lens = [2100, 5, 700]
    q_lens = [2100, 0, 700]             # the middle sequence contributes no query
    got, want = run_case(ctx, 8, 2, 128, lens, q_lens, seed=4)
    assert row_rel_err(got, want) <= TOL_ATTN
    got2, _ = run_case(ctx, 8, 2, 128, lens, q_lens, seed=4)
    assert (got == got2).all()


def test_prefill_argument_checks(ctx):
    cfg = IN.LayerConfig(29, "prefill", 2, 8, 2, 128, 64, 64)
    lens = np.asarray([20, 30], dtype=np.int32)
    kvh = IN.make_paged_kv(cfg, lens)
    kv = AF.make_kv(kvh.k_cache.to(DEV), kvh.v_cache.to(DEV), kvh.page_table.to(DEV), kvh.seq_lens.to(DEV), kvh.seq_lens)
    q = torch.zeros(60, 8, 128, dtype=torch.bfloat16, device=DEV)
    out = torch.zeros_like(q)
    bad = torch.tensor([0, 40, 60], dtype=torch.int32)          # 40 queries for 20 cached tokens
    with pytest.raises(AF.AflexError):
        ctx.attn_prefill(AF.attn_desc(8, 2, 128), q, kv, bad.to(DEV), bad, out)
    bad = torch.tensor([0, 10, 5], dtype=torch.int32)
    with pytest.raises(AF.AflexError):
        ctx.attn_prefill(AF.attn_desc(8, 2, 128), q, kv, bad.to(DEV), bad, out)
    assert ctx.device_status() == AF.OK
