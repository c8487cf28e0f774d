"""Parity of the whole-decoder-layer entry points (aflex_add_rmsnorm, aflex_rope_append,
aflex_decoder_layers) against the fp64 oracle, through the C ABI."""
import dataclasses

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2608_01891_b200 import aflex as AF
from paper_2608_01891_b200 import inputs as IN
from tests.helpers import TOL_ATTN, TOL_FFN, compact_kv, f64, row_rel_err, u16

pytestmark = pytest.mark.gpu
DEV = "cuda:0"

TINY_MOE = IN.LayerConfig(11, "tiny-moe", 6, 8, 2, 64, 256, 384, num_experts=4, top_k=2,
                          len_dist="uniform", len_lo=16, len_hi=128, rms_eps=1e-5, qk_norm=False)
TINY_D128 = IN.LayerConfig(12, "tiny-d128", 5, 8, 1, 128, 384, 640, len_dist="uniform", len_lo=1, len_hi=70)


def bf16_to_f64(a: np.ndarray) -> np.ndarray:
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def oracle_weights(w: IN.DecoderWeights) -> dict:
    g = lambda t: None if t is None else u16(t)
    return {"ln_attn": g(w.ln_attn), "qkv": g(w.qkv), "q_norm": g(w.q_norm), "k_norm": g(w.k_norm), "o": g(w.o),
            "ln_ffn": g(w.ln_ffn), "gate": g(w.gate), "up": g(w.up), "down": g(w.down), "router": g(w.router)}


class Chain:
    """L decoder layers of configuration `cfg` on the device, with one KV cache per layer."""

    def __init__(self, cfg, num_layers: int, seq_lens=None, gen: str = "cpu"):
        # gen = "cuda:0" draws the multi-GB tensors on the device (the oracle reads them back)
        self.cfg, self.L = cfg, num_layers
        self.kvh = IN.make_paged_kv(cfg, seq_lens, device=gen)
        self.table = self.kvh.page_table.to(DEV)
        self.lens = self.kvh.seq_lens.to(DEV)
        self.weights = [IN.make_decoder_weights(cfg, l, device=gen) for l in range(num_layers)]
        self.dev_w, self.descs, self.kvs, self.caches = [], [], [], []
        attn = AF.attn_desc(cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim)
        for l, w in enumerate(self.weights):
            dw = {f.name: (None if getattr(w, f.name) is None else getattr(w, f.name).to(DEV)) for f in dataclasses.fields(w)}
            self.dev_w.append(dw)
            layer = AF.layer_desc(attn, cfg.hidden, cfg.inter, dw["o"], dw["gate"], dw["up"], dw["down"],
                                  cfg.num_experts, cfg.top_k, dw["router"])
            self.descs.append(AF.decoder_desc(layer, dw["qkv"], dw["ln_attn"], dw["ln_ffn"], dw["q_norm"],
                                              dw["k_norm"], cfg.rms_eps, cfg.rope_theta))
            kc, vc = self.kvh.k_cache.to(DEV, copy=True), self.kvh.v_cache.to(DEV, copy=True)
            self.caches.append((kc, vc))
            self.kvs.append(AF.make_kv(kc, vc, self.table, self.lens, self.kvh.seq_lens))
        self.x = IN.make_hidden(cfg)

    def reset_caches(self):
        for kc, vc in self.caches:
            kc.copy_(self.kvh.k_cache)
            vc.copy_(self.kvh.v_cache)

    def workspace(self) -> int:
        return max(AF.decoder_workspace_bytes(d, self.cfg.batch) for d in self.descs)

    def oracle(self, rows=None):
        """fp64 chain on all rows (or the sampled `rows`, with their pages compacted).  Returns the
        hidden states after every layer, the caches after the appends, and per-layer router margins."""
        cfg = self.cfg
        rows = list(range(cfg.batch)) if rows is None else list(rows)
        x = bf16_to_f64(u16(self.x))[rows]
        outs, caches, margins = [], [], []
        for l, w in enumerate(self.weights):
            k, v, table, lens = compact_kv(self.kvh.k_cache, self.kvh.v_cache, self.kvh.page_table.numpy(),
                                           self.kvh.seq_lens.numpy(), rows)
            k, v = k.copy(), v.copy()
            ow = oracle_weights(w)
            _, h1, x = O.decoder_layer(x, ow, k, v, table, lens, cfg.num_q_heads, cfg.rms_eps, cfg.rope_theta,
                                       top_k=cfg.top_k)
            if cfg.num_experts:
                lg = np.sort(O.router_logits(O.rmsnorm(h1, ow["ln_ffn"], cfg.rms_eps), ow["router"]), axis=1)
                margins.append(lg[:, -cfg.top_k] - lg[:, -cfg.top_k - 1])
            outs.append(x)
            caches.append((k, v, table, lens))
        return outs, caches, margins


# --------------------------------------------------------------------------- the small operators
@pytest.mark.parametrize("T,H", [(1, 512), (37, 5120), (4, 8), (3, 4104)])
def test_add_rmsnorm_matches_oracle(T, H):
    g = torch.Generator().manual_seed(100 + H)
    res = torch.randn(T, H, generator=g).to(torch.bfloat16)
    add = (torch.randn(T, H, generator=g) * 3).to(torch.bfloat16)
    w = (1 + 0.1 * torch.randn(H, generator=g)).to(torch.bfloat16)
    eps = 1e-6
    ctx = AF.Context(0, 1 << 24)
    try:
        s_want = bf16_to_f64(u16(res)) + bf16_to_f64(u16(add))
        y_want = O.rmsnorm(s_want, u16(w), eps)
        r_d, a_d, w_d = res.to(DEV), add.to(DEV), w.to(DEV)
        r_out = torch.full((T, H), float("nan"), dtype=torch.bfloat16, device=DEV)
        y = torch.full((T, H), float("nan"), dtype=torch.bfloat16, device=DEV)
        ctx.add_rmsnorm(r_d, a_d, w_d, eps, r_out, y)
        torch.cuda.synchronize()
        # the residual is the fp32 sum rounded once more: at most one bf16 step from the exact sum
        assert row_rel_err(f64(r_out), s_want) <= 2.0 ** -8
        assert row_rel_err(f64(y), y_want) <= TOL_ATTN
        # without an addend the residual passes through bit for bit
        y0 = torch.empty_like(y)
        r0 = torch.empty_like(y)
        ctx.add_rmsnorm(r_d, None, w_d, eps, r0, y0)
        torch.cuda.synchronize()
        assert torch.equal(r0.view(torch.int16), r_d.view(torch.int16))
        assert row_rel_err(f64(y0), O.rmsnorm(bf16_to_f64(u16(res)), u16(w), eps)) <= TOL_ATTN
        # in place (outputs alias inputs) gives the same bits
        r_alias = r_d.clone()
        ctx.add_rmsnorm(r_alias, a_d, w_d, eps, r_alias, None)
        a_alias = a_d.clone()
        ctx.add_rmsnorm(r_d, a_alias, w_d, eps, None, a_alias)
        torch.cuda.synchronize()
        assert torch.equal(r_alias.view(torch.int16), r_out.view(torch.int16))
        assert torch.equal(a_alias.view(torch.int16), y.view(torch.int16))
        assert ctx.device_status() == AF.OK
    finally:
        ctx.close()


@pytest.mark.parametrize("cfg", [IN.CONFIGS[1], TINY_MOE, TINY_D128], ids=lambda c: c.name)
def test_attention_front_matches_oracle(cfg):
    """rmsnorm -> QKV projection -> q/k norm, rotary embedding, K/V append, operator by operator."""
    ch = Chain(cfg, 1)
    w, dw = ch.weights[0], ch.dev_w[0]
    B, H, Hq, Hkv, D = cfg.batch, cfg.hidden, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim
    ctx = AF.Context(0, 1 << 26)
    try:
        x = ch.x.to(DEV)
        xn = torch.empty_like(x)
        qkv = torch.empty(B, (Hq + 2 * Hkv) * D, dtype=torch.bfloat16, device=DEV)
        q = torch.full((B, Hq, D), float("nan"), dtype=torch.bfloat16, device=DEV)
        kc, vc = ch.caches[0]
        k_before, v_before = kc.clone(), vc.clone()
        ctx.add_rmsnorm(x, None, dw["ln_attn"], cfg.rms_eps, None, xn)
        ctx.linear(xn, dw["qkv"], qkv)
        ctx.rope_append(AF.attn_desc(Hq, Hkv, D), qkv, ch.kvs[0], q, dw["q_norm"], dw["k_norm"], cfg.rms_eps,
                        cfg.rope_theta)
        torch.cuda.synchronize()
        assert ctx.device_status() == AF.OK
        ko, vo = u16(ch.kvh.k_cache).copy(), u16(ch.kvh.v_cache).copy()
        ow = oracle_weights(w)
        q_want = O.qkv_rope_append(bf16_to_f64(u16(ch.x)), ow["ln_attn"], ow["qkv"], ow["q_norm"], ow["k_norm"],
                                   cfg.rms_eps, cfg.rope_theta, ko, vo, ch.kvh.page_table.numpy(),
                                   ch.kvh.seq_lens.numpy(), Hq)
        assert row_rel_err(f64(q), q_want) <= TOL_ATTN
        # exactly the decoded tokens' slots changed, and they hold the oracle's keys / values
        changed_k = (kc.view(torch.int16) != k_before.view(torch.int16)).any(dim=-1).cpu().numpy()
        changed_v = (vc.view(torch.int16) != v_before.view(torch.int16)).any(dim=-1).cpu().numpy()
        want_slots = np.zeros(changed_k.shape, dtype=bool)
        lens, table = ch.kvh.seq_lens.numpy(), ch.kvh.page_table.numpy()
        for b in range(B):
            pos = int(lens[b]) - 1
            want_slots[table[b, pos // 16], :, pos % 16] = True
        assert (changed_k == want_slots).all() and (changed_v == want_slots).all()
        kg, vg = bf16_to_f64(u16(kc)), bf16_to_f64(u16(vc))
        assert row_rel_err(kg[want_slots], bf16_to_f64(ko)[want_slots]) <= TOL_ATTN
        assert row_rel_err(vg[want_slots], bf16_to_f64(vo)[want_slots]) <= TOL_ATTN
    finally:
        ctx.close()


def test_rope_append_reports_bad_lengths_and_pages():
    cfg = IN.CONFIGS[1]
    ch = Chain(cfg, 1)
    B, Hq, Hkv, D = cfg.batch, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim
    ctx = AF.Context(0, 1 << 26)
    try:
        qkv = torch.zeros(B, (Hq + 2 * Hkv) * D, dtype=torch.bfloat16, device=DEV)
        q = torch.zeros(B, Hq, D, dtype=torch.bfloat16, device=DEV)
        kc, vc = ch.caches[0]
        before = kc.clone()
        bad_lens = ch.lens.clone()
        bad_lens[1] = 0
        bad_lens[2] = ch.kvh.max_pages_per_seq * 16 + 1
        kv = AF.make_kv(kc, vc, ch.table, bad_lens)
        ctx.rope_append(AF.attn_desc(Hq, Hkv, D), qkv, kv, q, None, None, 1e-6, 1e4)
        torch.cuda.synchronize()
        assert ctx.device_status() == AF.ERR_BOUNDS
        bad_table = ch.table.clone()
        bad_table[0, (int(ch.kvh.seq_lens[0]) - 1) // 16] = ch.kvh.num_pages + 5
        kc.copy_(before)
        kv = AF.make_kv(kc, vc, bad_table, ch.lens)
        ctx.rope_append(AF.attn_desc(Hq, Hkv, D), qkv, kv, q, None, None, 1e-6, 1e4)
        torch.cuda.synchronize()
        assert ctx.device_status() == AF.ERR_BOUNDS
        assert ctx.device_status() == AF.OK          # the status word was cleared by the read
    finally:
        ctx.close()


# --------------------------------------------------------------------------- whole layers, chained
def _run_chain(ctx, ch, M, offsets=None):
    ch.reset_caches()
    x_out = torch.full_like(ch.x, float("nan"), device=DEV)
    ctx.decoder_layers(ch.descs, ch.kvs, ch.x.to(DEV), x_out, M, offsets)
    torch.cuda.synchronize()
    assert ctx.device_status() == AF.OK
    return x_out


@pytest.mark.parametrize("cfg,L", [(IN.CONFIGS[1], 1), (IN.CONFIGS[1], 3), (TINY_D128, 2), (TINY_MOE, 1), (TINY_MOE, 2)],
                         ids=lambda v: getattr(v, "name", str(v)))
def test_decoder_layers_match_oracle(cfg, L):
    ch = Chain(cfg, L)
    ctx = AF.Context(0, ch.workspace())
    try:
        outs, caches, margins = ch.oracle()
        keep = np.ones(cfg.batch, dtype=bool)
        for m in margins:                  # rows whose top-k choice hangs on a near-tie are not unique
            keep &= m > 0.02
        assert keep.sum() >= cfg.batch - 3
        depths = [1, 2, cfg.batch] if cfg.batch >= 2 else [1]
        for M in depths:
            offsets = None
            if M == 2 and cfg.batch >= 3:
                offsets = [0, 1, cfg.batch]          # ragged split
            x_out = _run_chain(ctx, ch, M, offsets)
            assert torch.isfinite(x_out.float()).all()
            # tolerance: the FFN bound, once per layer
            assert row_rel_err(f64(x_out)[keep], outs[-1][keep]) <= TOL_FFN * L, (cfg.name, L, M)
            for l in range(L):
                k_want, v_want, _, _ = caches[l]
                kc, vc = ch.caches[l]
                kk, vv = bf16_to_f64(u16(kc)), bf16_to_f64(u16(vc))
                # compact_kv renumbers pages in table order; map them back
                ids = np.concatenate([ch.kvh.page_table.numpy()[b, :(int(n) + 15) // 16]
                                      for b, n in enumerate(ch.kvh.seq_lens.numpy())])
                tol = TOL_ATTN if l == 0 else TOL_FFN * l + TOL_ATTN
                rows_ok = np.repeat(keep, [(int(n) + 15) // 16 for n in ch.kvh.seq_lens.numpy()])
                assert row_rel_err(kk[ids][rows_ok], bf16_to_f64(k_want)[rows_ok]) <= tol, (l, M)
                assert row_rel_err(vv[ids][rows_ok], bf16_to_f64(v_want)[rows_ok]) <= tol, (l, M)
        # same call twice: identical bits
        a = _run_chain(ctx, ch, min(2, cfg.batch))
        b = _run_chain(ctx, ch, min(2, cfg.batch))
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
    finally:
        ctx.close()


def test_decoder_layers_with_planner_chosen_unequal_split_match_oracle():
    """The split aflex_plan_microbatches picks is handed to aflex_decoder_layers as it comes.  With stage times
    proportional to the work, the FFN side twice as slow as the attention side and one layer on separate pools, the
    best two-microbatch split puts a third of the rows first (closed form pinned in the control-oracle tests): an
    unequal, planner-made split.  The chain's result with it equals the oracle's, and (to rounding of the differently
    sized GEMM launches) the depth-1 result."""
    cfg = IN.LayerConfig(13, "tiny-plan", 12, 8, 2, 64, 256, 384, len_dist="uniform", len_lo=20, len_hi=90)
    ch = Chain(cfg, 2)
    lens = ch.kvh.seq_lens.numpy().tolist()
    tokens = float(sum(lens))
    model = AF.pipeline_model(([0.0, tokens], [0.0, 120.0]), ([0.0], [0.0]), ([0.0, 12.0], [0.0, 240.0]))
    M, offsets, _ = AF.plan_microbatches(model, lens, 1, [2])
    assert M == 2 and offsets[0] == 0 and offsets[2] == cfg.batch and 0 < offsets[1] < cfg.batch
    assert offsets[1] != cfg.batch // 2                     # not the equal split
    ctx = AF.Context(0, ch.workspace())
    try:
        outs, _, _ = ch.oracle()
        got = _run_chain(ctx, ch, M, offsets)
        assert row_rel_err(f64(got), outs[-1]) <= TOL_FFN * 2
        one = _run_chain(ctx, ch, 1)
        assert row_rel_err(f64(got), f64(one)) <= 1e-2
    finally:
        ctx.close()


def test_decoder_layers_attention_sees_the_token_it_just_appended():
    """Sequences of 1-3 tokens: the appended K/V carries most of the softmax weight, so an attention
    that read the cache before the append would be far off."""
    cfg = IN.CONFIGS[1]
    ch = Chain(cfg, 2, seq_lens=np.array([1, 2, 1, 3], dtype=np.int32))
    ctx = AF.Context(0, ch.workspace())
    try:
        outs, _, _ = ch.oracle()
        for M in (1, 2, 4):
            x_out = _run_chain(ctx, ch, M)
            assert row_rel_err(f64(x_out), outs[-1]) <= TOL_FFN * 2, M
        # the stand-alone attention after a stand-alone append agrees with the oracle on the same cache
        ch.reset_caches()
        B, Hq, Hkv, D = cfg.batch, cfg.num_q_heads, cfg.num_kv_heads, cfg.head_dim
        g = torch.Generator().manual_seed(9)
        qkv = torch.randn(B, (Hq + 2 * Hkv) * D, generator=g).to(torch.bfloat16).to(DEV)
        q = torch.empty(B, Hq, D, dtype=torch.bfloat16, device=DEV)
        out = torch.empty_like(q)
        desc = AF.attn_desc(Hq, Hkv, D)
        ctx.rope_append(desc, qkv, ch.kvs[0], q, None, None, cfg.rms_eps, cfg.rope_theta)
        ctx.attn_decode(desc, q, ch.kvs[0], out)
        torch.cuda.synchronize()
        kc, vc = ch.caches[0]
        want, _ = O.attn_decode(u16(q), u16(kc), u16(vc), ch.kvh.page_table.numpy(), ch.kvh.seq_lens.numpy())
        assert row_rel_err(f64(out), want) <= TOL_ATTN
        # sequences of one token return exactly the value rows just stored
        v_new = qkv.view(B, Hq + 2 * Hkv, D)[:, Hq + Hkv:, :]
        for b in (0, 2):
            got = out[b].view(Hkv, Hq // Hkv, D)
            assert torch.equal(got, v_new[b][:, None, :].expand(Hkv, Hq // Hkv, D))
    finally:
        ctx.close()


@pytest.mark.parametrize("cfg,L", [(IN.CONFIGS[1], 3), (TINY_MOE, 2)], ids=lambda v: getattr(v, "name", str(v)))
def test_af_pair_matches_oracle_and_single_context_chain(cfg, L):
    """Attention side and FFN side in two contexts (here on the same GPU: the peer copies are then
    device-local), hidden states handed over once each way per layer and microbatch."""
    ch = Chain(cfg, L)
    ctx = AF.Context(0, ch.workspace())
    ca = AF.Context(0, max(AF.af_workspace_bytes(d, cfg.batch, False) for d in ch.descs))
    cf = AF.Context(0, max(AF.af_workspace_bytes(d, cfg.batch, True) for d in ch.descs))
    try:
        outs, _, margins = ch.oracle()
        keep = np.ones(cfg.batch, dtype=bool)
        for m in margins:
            keep &= m > 0.02
        single = _run_chain(ctx, ch, 1)
        for M in (1, 2, cfg.batch):
            ch.reset_caches()
            x_out = torch.full_like(ch.x, float("nan"), device=DEV)
            AF.af_decoder_layers(ca, cf, ch.descs, ch.kvs, ch.x.to(DEV), x_out, M)
            torch.cuda.synchronize()
            assert ca.device_status() == AF.OK and cf.device_status() == AF.OK
            assert row_rel_err(f64(x_out)[keep], outs[-1][keep]) <= TOL_FFN * L, (cfg.name, M)
            assert row_rel_err(f64(x_out)[keep], f64(single)[keep]) <= 1e-2 * L, (cfg.name, M)
        # the same call twice gives the same bits
        ch.reset_caches()
        a = torch.empty_like(x_out)
        AF.af_decoder_layers(ca, cf, ch.descs, ch.kvs, ch.x.to(DEV), a, 2)
        ch.reset_caches()
        b = torch.empty_like(x_out)
        AF.af_decoder_layers(ca, cf, ch.descs, ch.kvs, ch.x.to(DEV), b, 2)
        torch.cuda.synchronize()
        assert torch.equal(a.view(torch.int16), b.view(torch.int16))
        with pytest.raises(AF.AflexError):
            AF.af_decoder_layers(ca, ca, ch.descs, ch.kvs, ch.x.to(DEV), a, 1)
        small = AF.Context(0, 1 << 16)
        try:
            with pytest.raises(AF.AflexError) as ei:
                AF.af_decoder_layers(ca, small, ch.descs, ch.kvs, ch.x.to(DEV), a, 1)
            assert ei.value.status == AF.ERR_WORKSPACE
        finally:
            small.close()
    finally:
        ctx.close()
        ca.close()
        cf.close()


def test_decoder_layers_in_place_and_argument_checks():
    cfg = IN.CONFIGS[1]
    ch = Chain(cfg, 2)
    ctx = AF.Context(0, ch.workspace())
    try:
        want = _run_chain(ctx, ch, 1)
        ch.reset_caches()
        x = ch.x.to(DEV).clone()
        ctx.decoder_layers(ch.descs, ch.kvs, x, x, 2)           # x_out aliases x_in
        torch.cuda.synchronize()
        assert row_rel_err(f64(x), f64(want)) <= 1e-2
        with pytest.raises(AF.AflexError):
            ctx.decoder_layers(ch.descs, ch.kvs, x, x, cfg.batch + 1)
        with pytest.raises(AF.AflexError):
            ctx.decoder_layers(ch.descs, ch.kvs, x, x, 2, [0, 3, 3])
        bad = AF.decoder_desc(ch.descs[0].layer, None, ch.dev_w[0]["ln_attn"], ch.dev_w[0]["ln_ffn"], None, None,
                              1e-6, 1e4)
        with pytest.raises(AF.AflexError):
            ctx.decoder_layers([bad], ch.kvs[:1], x, x, 1)
        small = AF.Context(0, 1 << 16)
        try:
            with pytest.raises(AF.AflexError) as ei:
                small.decoder_layers(ch.descs, ch.kvs, x, x, 1)
            assert ei.value.status == AF.ERR_WORKSPACE
        finally:
            small.close()
        assert ctx.device_status() == AF.OK
    finally:
        ctx.close()


@pytest.mark.parametrize("cid,L", [(2, 2), (4, 1)])
def test_decoder_layers_full_size_sampled_rows(cid, L):
    """Configurations 2 (dense) and 4 (MoE) at full size: sampled sequences against the oracle
    (sequences are independent through the whole chain)."""
    cfg = IN.CONFIGS[cid]
    torch.cuda.set_device(0)
    ch = Chain(cfg, L, gen=DEV)
    ctx = AF.Context(0, ch.workspace())
    try:
        lens = ch.kvh.seq_lens.numpy()
        rows = sorted({int(np.argmin(lens)), int(np.argmax(lens)), 7})
        outs, _, margins = ch.oracle(rows)
        keep = np.ones(len(rows), dtype=bool)
        for m in margins:
            keep &= m > 0.02
        assert keep.any()
        for M in (1, 2):
            x_out = _run_chain(ctx, ch, M)
            assert torch.isfinite(x_out.float()).all()
            assert row_rel_err(f64(x_out[rows])[keep], outs[-1][keep]) <= TOL_FFN * L, (cid, M)
    finally:
        ctx.close()
        del ch
        torch.cuda.empty_cache()
