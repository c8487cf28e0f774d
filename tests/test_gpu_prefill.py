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


@pytest.mark.parametrize("direction", ["rising", "falling"])
def test_prefill_scores_that_ramp_along_the_sequence(ctx, direction):
    """Keys built so that every query's score ramps by about 37 (base 2) per 128 cached tokens.  Rising: each step's
    maximum outgrows the standing reference, so the accumulator is rescaled at every step; falling: everything after
    the first steps underflows to zero.  Both are exact cases for an online softmax, and a worst case for one that
    moves its reference lazily."""
    Hq, Hkv, D = 8, 2, 128
    lens = np.asarray([1000, 333], dtype=np.int32)
    cfg = IN.LayerConfig(41, "prefill-ramp", len(lens), Hq, Hkv, D, 64, 64)
    kvh = IN.make_paged_kv(cfg, lens, poison=True)
    g = torch.Generator().manual_seed(41)
    u = torch.randn(Hkv, D, generator=g)
    u = u / u.norm(dim=-1, keepdim=True)
    table = kvh.page_table.numpy()
    for b, n in enumerate(lens):
        j = torch.arange(int(n), dtype=torch.float32)
        ramp = 0.29 * 11.3 * (j if direction == "rising" else (float(n) - j))      # q.k * scale grows by 0.2 per token
        k = (u[None, :, :] * ramp[:, None, None] / 8.0 + 0.05 * torch.randn(int(n), Hkv, D, generator=g)).to(torch.bfloat16)
        pages = torch.from_numpy(table[b, : (int(n) + 15) // 16].astype(np.int64))
        for t0 in range(0, int(n), 16):
            w = min(16, int(n) - t0)
            kvh.k_cache[pages[t0 // 16], :, :w, :] = k[t0:t0 + w].transpose(0, 1)
    q_off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T = int(q_off[-1])
    q = (8.0 * u.repeat_interleave(Hq // Hkv, dim=0)[None, :, :] + 0.1 * torch.randn(T, Hq, D, generator=g)).to(torch.bfloat16)
    kv = AF.make_kv(kvh.k_cache.to(DEV), kvh.v_cache.to(DEV), kvh.page_table.to(DEV), kvh.seq_lens.to(DEV), kvh.seq_lens)
    out = torch.full((T, Hq, D), float("nan"), dtype=torch.bfloat16, device=DEV)
    qo = torch.from_numpy(q_off)
    ctx.attn_prefill(AF.attn_desc(Hq, Hkv, D), q.to(DEV), kv, qo.to(DEV), qo, out)
    torch.cuda.synchronize()
    assert ctx.device_status() == AF.OK
    want = O.attn_prefill(u16(q), u16(kvh.k_cache), u16(kvh.v_cache), table, lens, q_off)
    assert row_rel_err(f64(out), want) <= TOL_ATTN


def test_prefill_full_size_sampled_rows(ctx):
    """The head shape and prompt lengths bench.py times (64 query heads, 8 KV heads, head size 128; 16 384 and 4 099
    tokens), checked on sampled query rows: a prefill row is decode attention over the sequence cut after that row."""
    Hq, Hkv, D = 64, 8, 128
    lens = np.asarray([16384, 4099], dtype=np.int32)
    cfg = IN.LayerConfig(42, "prefill-full", len(lens), Hq, Hkv, D, 64, 64)
    kvh = IN.make_paged_kv(cfg, lens, device=DEV)
    q_off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T = int(q_off[-1])
    g = torch.Generator(device=DEV).manual_seed(42)
    q = torch.randn(T, Hq, D, generator=g, device=DEV).to(torch.bfloat16)
    kv = AF.make_kv(kvh.k_cache, kvh.v_cache, kvh.page_table.to(DEV), kvh.seq_lens.to(DEV), kvh.seq_lens)
    out = torch.full((T, Hq, D), float("nan"), dtype=torch.bfloat16, device=DEV)
    qo = torch.from_numpy(q_off)
    ctx.attn_prefill(AF.attn_desc(Hq, Hkv, D), q, kv, qo.to(DEV), qo, out)
    torch.cuda.synchronize()
    assert ctx.device_status() == AF.OK
    assert torch.isfinite(out.float()).all()
    rng = np.random.default_rng(42)
    rows = [(0, 0), (0, 1), (0, 127), (0, 128), (0, 255), (0, 256), (0, 16383), (1, 0), (1, 4095), (1, 4096), (1, 4098)]
    rows += [(0, int(r)) for r in rng.integers(0, 16384, size=12)] + [(1, int(r)) for r in rng.integers(0, 4099, size=6)]
    table = kvh.page_table.numpy()
    q_s = torch.stack([q[int(q_off[b]) + r] for b, r in rows]).cpu()
    got = torch.stack([out[int(q_off[b]) + r] for b, r in rows]).cpu()
    want, _ = O.attn_decode(u16(q_s), u16(kvh.k_cache.cpu()), u16(kvh.v_cache.cpu()),
                            np.stack([table[b] for b, _ in rows]), np.asarray([r + 1 for _, r in rows], dtype=np.int32))
    assert row_rel_err(f64(got), want) <= TOL_ATTN


def test_prefill_lengths_on_tile_and_step_boundaries(ctx):
    """Prompt lengths that end exactly on the kernel's natural boundaries (16-token pages, 128-token steps, 128-row
    query tiles, 256-row blocks) and one token beyond them; a non-default softmax scale."""
    lens = [128, 129, 256, 257, 512, 16, 127, 384]
    Hq, Hkv, D = 8, 2, 128
    cfg = IN.LayerConfig(43, "prefill-bounds", len(lens), Hq, Hkv, D, 64, 64)
    l = np.asarray(lens, dtype=np.int32)
    kvh = IN.make_paged_kv(cfg, l, poison=True)
    q_off = np.concatenate([[0], np.cumsum(l)]).astype(np.int32)
    T = int(q_off[-1])
    g = torch.Generator().manual_seed(43)
    q = torch.randn(T, Hq, D, generator=g).to(torch.bfloat16)
    kv = AF.make_kv(kvh.k_cache.to(DEV), kvh.v_cache.to(DEV), kvh.page_table.to(DEV), kvh.seq_lens.to(DEV), kvh.seq_lens)
    out = torch.full((T, Hq, D), float("nan"), dtype=torch.bfloat16, device=DEV)
    qo = torch.from_numpy(q_off)
    desc = AF.attn_desc(Hq, Hkv, D, sm_scale=0.05)
    ctx.attn_prefill(desc, q.to(DEV), kv, qo.to(DEV), qo, out)
    torch.cuda.synchronize()
    assert ctx.device_status() == AF.OK
    want = O.attn_prefill(u16(q), u16(kvh.k_cache), u16(kvh.v_cache), kvh.page_table.numpy(), l, q_off, scale=0.05)
    assert row_rel_err(f64(out), want) <= TOL_ATTN


def test_prefill_with_equal_keys_is_the_running_mean_of_the_values(ctx):
    """Closed form, no oracle: when every cached key of a sequence is the same vector, every query weighs the tokens
    it may see equally, so row i of the output is the mean of V over positions 0 .. pos_i."""
    Hq, Hkv, D = 4, 2, 64
    lens = np.asarray([300, 45], dtype=np.int32)
    new = np.asarray([300, 20], dtype=np.int32)
    cfg = IN.LayerConfig(44, "prefill-mean", len(lens), Hq, Hkv, D, 64, 64)
    kvh = IN.make_paged_kv(cfg, lens)
    kvh.k_cache[:] = torch.randn(D, generator=torch.Generator().manual_seed(44)).to(torch.bfloat16)
    q_off = np.concatenate([[0], np.cumsum(new)]).astype(np.int32)
    T = int(q_off[-1])
    q = torch.randn(T, Hq, D, generator=torch.Generator().manual_seed(45)).to(torch.bfloat16)
    kv = AF.make_kv(kvh.k_cache.to(DEV), kvh.v_cache.to(DEV), kvh.page_table.to(DEV), kvh.seq_lens.to(DEV), kvh.seq_lens)
    out = torch.full((T, Hq, D), float("nan"), dtype=torch.bfloat16, device=DEV)
    qo = torch.from_numpy(q_off)
    ctx.attn_prefill(AF.attn_desc(Hq, Hkv, D), q.to(DEV), kv, qo.to(DEV), qo, out)
    torch.cuda.synchronize()
    assert ctx.device_status() == AF.OK
    table = kvh.page_table.numpy()
    v = kvh.v_cache.to(torch.float64).numpy()
    want = np.zeros((T, Hq, D))
    for b in range(2):
        vs = np.stack([v[table[b, j // 16], :, j % 16, :] for j in range(int(lens[b]))])      # [n, Hkv, D]
        run = np.cumsum(vs, axis=0) / np.arange(1, int(lens[b]) + 1)[:, None, None]
        for i in range(int(new[b])):
            pos = int(lens[b] - new[b]) + i
            want[q_off[b] + i] = np.repeat(run[pos], Hq // Hkv, axis=0)
    assert row_rel_err(f64(out), want) <= TOL_ATTN


def test_prefill_random_shapes(ctx):
    """Seeded sweep over head shapes (D 64 / 128, 1 - 4 KV heads, group sizes 1 - 8), batch sizes, ragged cached
    lengths and query counts (whole prompts, arbitrary chunks, short tails, sequences without a query), with and
    without the host copy of the lengths."""
    rng = np.random.default_rng(7)
    worst = 0.0
    for case in range(24):
        D, Hkv, G = int(rng.choice([64, 128])), int(rng.choice([1, 2, 4])), int(rng.choice([1, 2, 4, 8]))
        B = int(rng.integers(1, 6))
        lens = rng.integers(1, 700, size=B).astype(np.int32)
        mode = int(rng.integers(0, 3))
        if mode == 0:
            new = lens.copy()
        elif mode == 1:
            new = np.array([int(rng.integers(0, n + 1)) for n in lens], dtype=np.int32)
        else:
            new = np.minimum(lens, rng.integers(1, 40, size=B)).astype(np.int32)
        if new.sum() == 0:
            new[0] = 1
        cfg = IN.LayerConfig(100 + case, "prefill-sweep", B, Hkv * G, Hkv, D, 64, 64)
        kvh = IN.make_paged_kv(cfg, lens, poison=True)
        q_off = np.concatenate([[0], np.cumsum(new)]).astype(np.int32)
        T = int(q_off[-1])
        q = torch.randn(T, Hkv * G, D, generator=torch.Generator().manual_seed(case)).to(torch.bfloat16)
        kv = AF.make_kv(kvh.k_cache.to(DEV), kvh.v_cache.to(DEV), kvh.page_table.to(DEV), kvh.seq_lens.to(DEV),
                        kvh.seq_lens if case % 2 else None)
        out = torch.full((T, Hkv * G, D), float("nan"), dtype=torch.bfloat16, device=DEV)
        qo = torch.from_numpy(q_off)
        ctx.attn_prefill(AF.attn_desc(Hkv * G, Hkv, D), q.to(DEV), kv, qo.to(DEV), qo, out)
        torch.cuda.synchronize()
        assert ctx.device_status() == AF.OK, case
        want = O.attn_prefill(u16(q), u16(kvh.k_cache), u16(kvh.v_cache), kvh.page_table.numpy(), lens, q_off)
        worst = max(worst, row_rel_err(f64(out), want))
    assert worst <= TOL_ATTN
