"""Full-size parity: configurations 2-5 at their real sizes, in the launch configuration the
benchmark times (aflex_layer_step with the configuration's microbatch depths).  The attention
output of EVERY sequence is compared with the fp64 oracle; the layer output is compared on batch
rows chosen to cover every token tile of every GEMM launch and, for the MoE layers, both ends of
every expert's row segment (rows are independent, so the oracle computes them one by one); plus
properties that hold at any size."""
import numpy as np
import pytest
import torch

import bench
from oracle import oracle as O
from paper_2608_01891_b200 import aflex as AF
from paper_2608_01891_b200 import inputs as IN
from tests.helpers import TOL_ATTN, TOL_FFN, compact_kv, f64, row_rel_err, u16

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def near_equal_offsets(batch: int, M: int):
    """The library's default microbatch split: near-equal, the first batch % M microbatches one row larger."""
    base, extra = divmod(batch, M)
    offs = [0]
    for i in range(M):
        offs.append(offs[-1] + base + (1 if i < extra else 0))
    return offs


def token_tile(rows: int) -> int:
    """Token rows per GEMM tile as the library picks them: the fewest tiles of at most 256 rows, equal widths,
    rounded up to 16 (grouped GEMMs cap a tile at 128 rows at decode sizes)."""
    rows = max(rows, 16)
    tiles = (rows + 255) // 256
    return min(256, -(-(-(-rows // tiles)) // 16) * 16)


def coverage_rows(cfg, lens: np.ndarray, logits):
    """Batch rows chosen so that, for every microbatch depth the configuration is run at, every token tile of
    every GEMM launch holds a compared row: the first and last row of every microbatch and of every token tile
    inside it; for the MoE layers also the first and last assignment of every expert's row segment in every
    microbatch and both sides of every 128-row chunk boundary inside a segment.  Plus the shortest and longest
    context, a seeded random row and eight evenly spread rows."""
    rows = {int(np.argmin(lens)), int(np.argmax(lens)), int(np.random.default_rng(12345).integers(len(lens)))}
    rows.update(range(0, len(lens), max(1, len(lens) // 8)))                  # evenly spread as well
    idx = O.moe_route(logits, cfg.top_k)[0] if cfg.num_experts else None
    for M in cfg.microbatch_depths:
        offs = near_equal_offsets(cfg.batch, M)
        for r0, r1 in zip(offs, offs[1:]):
            nt = token_tile(r1 - r0)
            for t0 in range(r0, r1, nt):
                rows.update((t0, min(r1, t0 + nt) - 1))
            if idx is None:
                continue
            chunk = min(128, nt)
            for e in range(cfg.num_experts):
                seg = [t for t in range(r0, r1) if e in idx[t]]         # the segment's rows, in token order
                for c0 in range(0, len(seg), chunk):
                    rows.update((seg[c0], seg[min(len(seg), c0 + chunk) - 1]))
    return sorted(rows)


def oracle_rows(cfg, wl, rows):
    kvh = wl["kvh"]
    k, v, table, lens = compact_kv(kvh.k_cache, kvh.v_cache, kvh.page_table.numpy(), kvh.seq_lens.numpy(), rows)
    q = u16(wl["q"][rows])
    logits = wl["logits"][rows].cpu().numpy() if cfg.num_experts else None
    return O.layer_step(q, k, v, table, lens, u16(wl["wo"]), u16(wl["wg"]), u16(wl["wu"]), u16(wl["wd"]),
                        logits=logits, top_k=cfg.top_k)


def oracle_attention_all_rows(wl):
    """The oracle's attention for EVERY sequence of the workload (the whole paged cache goes to the host)."""
    kvh = wl["kvh"]
    out, _ = O.attn_decode(u16(wl["q"]), u16(kvh.k_cache), u16(kvh.v_cache), kvh.page_table.numpy(), kvh.seq_lens.numpy())
    return out


@pytest.mark.parametrize("cid", [2, 3, 4, 5])
def test_layer_step_full_size_all_attention_rows_and_tile_covering_ffn_rows(cid):
    cfg = IN.CONFIGS[cid]
    torch.cuda.set_device(0)
    wl = bench.build_workload(cfg, DEV)
    lens = wl["kvh"].seq_lens.numpy()
    ctx = AF.Context(0, AF.workspace_bytes(wl["layer"], cfg.batch, wl["kvh"].max_pages_per_seq))
    try:
        rows = coverage_rows(cfg, lens, wl["logits"].cpu().numpy() if cfg.num_experts else None)
        assert len(rows) >= (8 if cfg.num_experts == 0 else 16)
        _, want_y = oracle_rows(cfg, wl, rows)
        want_a_all = oracle_attention_all_rows(wl)
        a = torch.full_like(wl["q"], float("nan"))
        results = {}
        for M in cfg.microbatch_depths:
            wl["y"].fill_(float("nan"))
            a.fill_(float("nan"))
            ctx.layer_step(wl["layer"], wl["q"], wl["kv"], wl["y"], M, None, wl["logits"], a)
            torch.cuda.synchronize()
            assert ctx.device_status() == AF.OK
            assert row_rel_err(f64(a), want_a_all) <= TOL_ATTN, (cid, M)        # every sequence, every head
            assert row_rel_err(f64(wl["y"][rows]), want_y) <= TOL_FFN, (cid, M)
            assert torch.isfinite(wl["y"].float()).all()
            results[M] = wl["y"].float().cpu().numpy().astype(np.float64)
        # the result does not depend on the microbatch depth (to bf16 rounding of different GEMM plans)
        base = results[cfg.microbatch_depths[0]]
        for M, y in results.items():
            assert row_rel_err(y, base) <= 1e-2, (cid, M)
        # run-to-run determinism at full size
        ctx.layer_step(wl["layer"], wl["q"], wl["kv"], wl["y"], cfg.microbatch_depths[0], None, wl["logits"], a)
        torch.cuda.synchronize()
        y1 = wl["y"].clone()
        ctx.layer_step(wl["layer"], wl["q"], wl["kv"], wl["y"], cfg.microbatch_depths[0], None, wl["logits"], a)
        torch.cuda.synchronize()
        assert torch.equal(y1.view(torch.int16), wl["y"].view(torch.int16))
    finally:
        ctx.close()
        del wl
        torch.cuda.empty_cache()


def test_moe_routing_full_size_is_bit_exact_and_zipf_loaded():
    """Configuration 5's routing (T = 256, skewed logits): indices and counts bit-exact, gates to 1e-6,
    and the per-expert load follows the Zipf(1.2) recipe."""
    cfg = IN.CONFIGS[5]
    torch.cuda.set_device(0)
    T, H, E = cfg.batch, 256, cfg.num_experts            # routing does not depend on the hidden size
    logits = IN.make_router_logits(cfg)
    g = torch.Generator().manual_seed(3)
    x = torch.randn(T, H, generator=g).to(torch.bfloat16)
    mk = lambda *s: (torch.randn(*s, generator=g) * 0.05).to(torch.bfloat16)
    wg, wu, wd = mk(E, 128, H), mk(E, 128, H), mk(E, H, 128)
    ctx = AF.Context(0, 1 << 28)
    try:
        y = torch.zeros(T, H, dtype=torch.bfloat16, device=DEV)
        idx = torch.zeros(T, 2, dtype=torch.int32, device=DEV)
        gate = torch.zeros(T, 2, dtype=torch.float32, device=DEV)
        counts = torch.zeros(E, dtype=torch.int32, device=DEV)
        ctx.ffn_moe(x.to(DEV), wg.to(DEV), wu.to(DEV), wd.to(DEV), 2, y, router_logits=logits.to(DEV),
                    topk_idx=idx, topk_gate=gate, expert_counts=counts)
        torch.cuda.synchronize()
        want_y, want_idx, want_gate = O.ffn_moe(u16(x), logits.numpy(), u16(wg), u16(wu), u16(wd), 2)
        assert (idx.cpu().numpy() == want_idx).all()
        assert (counts.cpu().numpy() == np.bincount(want_idx.ravel(), minlength=E)).all()
        assert np.abs(f64(gate) - want_gate).max() <= 1e-6
        assert row_rel_err(f64(y), want_y) <= TOL_FFN
        share = counts.cpu().numpy()[IN.zipf_rank_to_expert(cfg)] / (2.0 * T)
        assert share[0] > 0.3 and share[0] > share[-1] * 4          # hot expert vs coldest, 512 samples
    finally:
        ctx.close()
