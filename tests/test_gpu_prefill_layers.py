"""Parity of aflex_prefill_layers (whole decoder layers over the tokens being prefilled) against the fp64
oracle, through the C ABI."""
import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2608_01891_b200 import aflex as AF
from paper_2608_01891_b200 import inputs as IN
from tests.helpers import TOL_ATTN, TOL_FFN, f64, row_rel_err, u16
from tests.test_gpu_decoder import TINY_D128, TINY_MOE, Chain, bf16_to_f64, oracle_weights

pytestmark = pytest.mark.gpu
DEV = "cuda:0"


def prompt_hidden(T, H, seed):
    g = torch.Generator().manual_seed(seed)
    return torch.randn(T, H, generator=g).to(torch.bfloat16)


def run_gpu(ctx, ch, x, q_off):
    ch.reset_caches()
    qo = torch.from_numpy(q_off)
    x_out = torch.full_like(x, float("nan"), device=DEV)
    ctx.prefill_layers(ch.descs, ch.kvs, x.to(DEV), qo.to(DEV), qo, x_out)
    torch.cuda.synchronize()
    assert ctx.device_status() == AF.OK
    return x_out


def run_oracle(ch, x, q_off):
    """fp64 chain; returns the hidden states after the last layer, the caches after every layer's appends and the
    rows whose top-k choice does not hang on a near-tie in any layer."""
    cfg = ch.cfg
    h = bf16_to_f64(u16(x))
    lens, table = ch.kvh.seq_lens.numpy(), ch.kvh.page_table.numpy()
    keep = np.ones(h.shape[0], dtype=bool)
    caches = []
    for w in ch.weights:
        k, v = u16(ch.kvh.k_cache).copy(), u16(ch.kvh.v_cache).copy()
        ow = oracle_weights(w)
        _, h1, h = O.prefill_layer(h, ow, k, v, table, lens, q_off, cfg.num_q_heads, cfg.rms_eps, cfg.rope_theta,
                                   top_k=cfg.top_k)
        if cfg.num_experts:
            lg = np.sort(O.router_logits(O.rmsnorm(h1, ow["ln_ffn"], cfg.rms_eps), ow["router"]), axis=1)
            keep &= (lg[:, -cfg.top_k] - lg[:, -cfg.top_k - 1]) > 0.02
        caches.append((k, v))
    return h, caches, keep


def written_slots(ch, q_off):
    lens, table = ch.kvh.seq_lens.numpy(), ch.kvh.page_table.numpy()
    m = np.zeros(tuple(ch.kvh.k_cache.shape[:3]), dtype=bool)
    for b in range(len(lens)):
        new = int(q_off[b + 1] - q_off[b])
        for pos in range(int(lens[b]) - new, int(lens[b])):
            m[table[b, pos // 16], :, pos % 16] = True
    return m


CASES = [
    (IN.CONFIGS[1], 2, [40, 1, 129, 300], [40, 1, 129, 300]),          # whole prompts, ragged
    (IN.CONFIGS[1], 1, [500, 130, 77, 64], [100, 130, 1, 0]),           # chunks behind prefixes, a decode row, nothing
    (TINY_D128, 2, [257, 16, 33, 5, 700], [257, 16, 20, 5, 188]),
    (IN.CONFIGS[1], 1, [1100, 30, 5, 200], [1100, 30, 5, 200]),        # more than 1024 rows: several heads per warp in the append kernel
    (TINY_MOE, 1, [90, 17, 128, 3, 260, 31], [90, 17, 100, 3, 200, 31]),
]


@pytest.mark.parametrize("cfg,L,lens,new", CASES, ids=lambda v: getattr(v, "name", None))
def test_prefill_layers_match_oracle(cfg, L, lens, new):
    ch = Chain(cfg, L, seq_lens=np.asarray(lens, dtype=np.int32))
    q_off = np.concatenate([[0], np.cumsum(new)]).astype(np.int32)
    T = int(q_off[-1])
    x = prompt_hidden(T, cfg.hidden, 7 + L)
    ctx = AF.Context(0, max(AF.prefill_workspace_bytes(d, T) for d in ch.descs))
    try:
        want, caches, keep = run_oracle(ch, x, q_off)
        assert keep.sum() >= 0.85 * T      # rows whose top-k choice hangs on a near-tie are not unique
        got = run_gpu(ctx, ch, x, q_off)
        assert torch.isfinite(got.float()).all()
        assert row_rel_err(f64(got)[keep], want[keep]) <= TOL_FFN * L, (cfg.name, L)
        slots = written_slots(ch, q_off)
        for l in range(L):
            kc, vc = ch.caches[l]
            k_want, v_want = caches[l]
            # exactly the prefilled tokens' slots changed
            changed = (kc.view(torch.int16) != ch.kvh.k_cache.to(DEV).view(torch.int16)).any(dim=-1).cpu().numpy()
            assert not (changed & ~slots).any()
            if l == 0:      # layer 0's keys do not depend on any routing
                tol = TOL_ATTN
                assert row_rel_err(bf16_to_f64(u16(kc))[slots], bf16_to_f64(k_want)[slots]) <= tol
                assert row_rel_err(bf16_to_f64(u16(vc))[slots], bf16_to_f64(v_want)[slots]) <= tol
        again = run_gpu(ctx, ch, x, q_off)
        assert torch.equal(again.view(torch.int16), got.view(torch.int16))
    finally:
        ctx.close()


def test_prefill_in_two_chunks_equals_the_oracle_of_the_whole():
    """Prompts prefilled in two calls on the same caches (the second call's tokens attend to what the first one
    appended, in every layer): the rows of both calls match the oracle of the one-pass prefill."""
    cfg = IN.CONFIGS[1]
    full = np.asarray([150, 64, 37, 260], dtype=np.int32)
    first = np.asarray([100, 64, 10, 129], dtype=np.int32)
    ch = Chain(cfg, 2, seq_lens=full)
    T = int(full.sum())
    x = prompt_hidden(T, cfg.hidden, 99)
    q_all = np.concatenate([[0], np.cumsum(full)]).astype(np.int32)
    want, _, _ = run_oracle(ch, x, q_all)
    rows_a = np.concatenate([np.arange(q_all[b], q_all[b] + first[b]) for b in range(4)])
    rows_b = np.concatenate([np.arange(q_all[b] + first[b], q_all[b + 1]) for b in range(4)])
    ctx = AF.Context(0, max(AF.prefill_workspace_bytes(d, T) for d in ch.descs))
    try:
        ch.reset_caches()
        lens_a = torch.from_numpy(first.copy())
        kvs_a = [AF.make_kv(kc, vc, ch.table, lens_a.to(DEV), lens_a) for kc, vc in ch.caches]
        qa = torch.from_numpy(np.concatenate([[0], np.cumsum(first)]).astype(np.int32))
        out_a = torch.empty(len(rows_a), cfg.hidden, dtype=torch.bfloat16, device=DEV)
        ctx.prefill_layers(ch.descs, kvs_a, x[rows_a].to(DEV), qa.to(DEV), qa, out_a)
        qb = torch.from_numpy(np.concatenate([[0], np.cumsum(full - first)]).astype(np.int32))
        out_b = torch.empty(len(rows_b), cfg.hidden, dtype=torch.bfloat16, device=DEV)
        ctx.prefill_layers(ch.descs, ch.kvs, x[rows_b].to(DEV), qb.to(DEV), qb, out_b)
        torch.cuda.synchronize()
        assert ctx.device_status() == AF.OK
        assert row_rel_err(f64(out_a), want[rows_a]) <= TOL_FFN * 2
        assert row_rel_err(f64(out_b), want[rows_b]) <= TOL_FFN * 2
    finally:
        ctx.close()


def test_prefill_layers_argument_checks():
    cfg = IN.CONFIGS[1]
    ch = Chain(cfg, 1, seq_lens=np.asarray([20, 30, 5, 9], dtype=np.int32))
    ctx = AF.Context(0, 1 << 26)
    try:
        x = torch.zeros(64, cfg.hidden, dtype=torch.bfloat16, device=DEV)
        bad = torch.tensor([0, 40, 50, 55, 64], dtype=torch.int32)       # 40 new tokens in a 20-token sequence
        with pytest.raises(AF.AflexError):
            ctx.prefill_layers(ch.descs, ch.kvs, x, bad.to(DEV), bad, x)
        bad = torch.tensor([0, 10, 5, 7, 9], dtype=torch.int32)
        with pytest.raises(AF.AflexError):
            ctx.prefill_layers(ch.descs, ch.kvs, x, bad.to(DEV), bad, x)
        small = AF.Context(0, 1 << 16)
        ok = torch.tensor([0, 20, 50, 55, 64], dtype=torch.int32)
        with pytest.raises(AF.AflexError):
            small.prefill_layers(ch.descs, ch.kvs, x, ok.to(DEV), ok, x)
        small.close()
        assert ctx.device_status() == AF.OK
    finally:
        ctx.close()


def test_prefill_layers_replay_from_a_cuda_graph():
    """The prefill chain only enqueues work on the caller's stream (tensor maps are kernel parameters, no
    synchronisation, no allocation): captured into a CUDA graph after a warm-up call and replayed, it gives the
    bits of the eager call."""
    cfg = IN.CONFIGS[1]
    lens = np.asarray([70, 33, 129, 16], dtype=np.int32)
    ch = Chain(cfg, 2, seq_lens=lens)
    q_off = np.concatenate([[0], np.cumsum(lens)]).astype(np.int32)
    T = int(q_off[-1])
    x = prompt_hidden(T, cfg.hidden, 5).to(DEV)
    qo = torch.from_numpy(q_off)
    qod = qo.to(DEV)
    out = torch.zeros(T, cfg.hidden, dtype=torch.bfloat16, device=DEV)
    ctx = AF.Context(0, max(AF.prefill_workspace_bytes(d, T) for d in ch.descs))
    try:
        s = torch.cuda.Stream()
        with torch.cuda.stream(s):
            ch.reset_caches()
            ctx.prefill_layers(ch.descs, ch.kvs, x, qod, qo, out, s)        # warm-up: sets kernel attributes
            s.synchronize()
            want = out.clone()
            g = torch.cuda.CUDAGraph()
            with torch.cuda.graph(g, stream=s):
                ctx.prefill_layers(ch.descs, ch.kvs, x, qod, qo, out, s)
            for _ in range(2):
                out.zero_()
                g.replay()
                s.synchronize()
                assert torch.equal(out.view(torch.int16), want.view(torch.int16))
        assert ctx.device_status() == AF.OK
    finally:
        ctx.close()
