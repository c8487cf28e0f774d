"""Full-size parity: configurations 2-5 at their real sizes, in the launch configuration the
benchmark times (aflex_layer_step with the configuration's microbatch depths), checked on
sampled batch rows that the fp64 oracle computes one by one (rows are independent), plus
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


def sampled_rows(lens: np.ndarray, extra: int = 1):
    """Shortest, longest and `extra` seeded random rows."""
    rows = {int(np.argmin(lens)), int(np.argmax(lens))}
    rng = np.random.default_rng(12345)
    while len(rows) < min(len(lens), 2 + extra):
        rows.add(int(rng.integers(len(lens))))
    return sorted(rows)


def oracle_rows(cfg, wl, rows):
    kvh = wl["kvh"]
    k, v, table, lens = compact_kv(kvh.k_cache, kvh.v_cache, kvh.page_table.numpy(), kvh.seq_lens.numpy(), rows)
    q = u16(wl["q"][rows])
    logits = wl["logits"][rows].cpu().numpy() if cfg.num_experts else None
    return O.layer_step(q, k, v, table, lens, u16(wl["wo"]), u16(wl["wg"]), u16(wl["wu"]), u16(wl["wd"]),
                        logits=logits, top_k=cfg.top_k)


@pytest.mark.parametrize("cid", [2, 3, 4, 5])
def test_layer_step_full_size_sampled_rows(cid):
    cfg = IN.CONFIGS[cid]
    torch.cuda.set_device(0)
    wl = bench.build_workload(cfg, DEV)
    lens = wl["kvh"].seq_lens.numpy()
    ctx = AF.Context(0, AF.workspace_bytes(wl["layer"], cfg.batch, wl["kvh"].max_pages_per_seq))
    try:
        rows = sampled_rows(lens)
        want_a, want_y = oracle_rows(cfg, wl, rows)
        a = torch.full_like(wl["q"], float("nan"))
        results = {}
        for M in cfg.microbatch_depths:
            wl["y"].fill_(float("nan"))
            a.fill_(float("nan"))
            ctx.layer_step(wl["layer"], wl["q"], wl["kv"], wl["y"], M, None, wl["logits"], a)
            torch.cuda.synchronize()
            assert ctx.device_status() == AF.OK
            ya, yy = f64(a[rows]), f64(wl["y"][rows])
            assert row_rel_err(ya, want_a) <= TOL_ATTN, (cid, M)
            assert row_rel_err(yy, want_y) <= TOL_FFN, (cid, M)
            # any-size properties: every output finite; attention output inside the convex hull bound
            assert torch.isfinite(wl["y"].float()).all() and torch.isfinite(a.float()).all()
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
