"""Pins for the fp64 CPU oracle: closed forms, hand-computed cases, invariants,
special cases that reduce to a library routine, and brute force on tiny inputs.
A dropped term, wrong sign/index or transposed operand anywhere in the oracle
fails at least one of these.  No GPU needed."""
import itertools
import json
import math
import os

import numpy as np
import pytest
import torch

from oracle import oracle as O
from paper_2608_01891_b200 import inputs as IN

GOLD = json.load(open(os.path.join(os.path.dirname(__file__), "golden", "hand_cases.json")))


def bf16(a) -> np.ndarray:
    """float array -> bf16 bit patterns (RNE)."""
    t = torch.as_tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    return IN.bf16_bits(t).copy()


def bf16_to_f64(u16: np.ndarray) -> np.ndarray:
    return (u16.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


# --------------------------------------------------------------------------- attention
def test_attn_hand_two_keys():
    c = GOLD["attention_two_keys"]
    out, lse = O.attn_one_query_f64(c["q"], c["keys"], c["vals"], c["scale"])
    np.testing.assert_allclose(out, c["out"], rtol=0, atol=1e-14)
    assert abs(lse - c["lse"]) < 1e-14


def test_attn_hand_three_keys():
    c = GOLD["attention_three_keys"]
    out, lse = O.attn_one_query_f64(c["q"], c["keys"], c["vals"], c["scale"])
    np.testing.assert_allclose(out, c["out"], rtol=0, atol=1e-13)
    assert abs(lse - c["lse"]) < 1e-14


def test_attn_single_token_returns_v_exactly():
    rng = np.random.default_rng(1)
    q, k, v = rng.standard_normal(8), rng.standard_normal((1, 8)), rng.standard_normal((1, 8))
    out, lse = O.attn_one_query_f64(q, k, v, 0.3)
    assert (out == v[0]).all()
    assert abs(lse - 0.3 * float(q @ k[0])) < 1e-14


def test_attn_identical_keys_gives_mean_of_v():
    rng = np.random.default_rng(2)
    n, D = 16, 8
    q = rng.standard_normal(D)
    k = np.tile(rng.standard_normal(D), (n, 1))
    v = rng.integers(-8, 9, size=(n, D)).astype(np.float64) / 4.0  # coarse grid: mean is exact
    out, lse = O.attn_one_query_f64(q, k, v, 0.5)
    assert (out == v.mean(axis=0)).all()
    assert abs(lse - (0.5 * float(q @ k[0]) + math.log(n))) < 1e-12


def test_attn_zero_query_is_mean_and_lse_is_log_n():
    rng = np.random.default_rng(3)
    n, D = 37, 16
    k, v = rng.standard_normal((n, D)), rng.standard_normal((n, D))
    out, lse = O.attn_one_query_f64(np.zeros(D), k, v, 1.0)
    np.testing.assert_allclose(out, v.mean(axis=0), rtol=0, atol=1e-14)
    assert abs(lse - math.log(n)) < 1e-14


def test_attn_matches_numpy_softmax():
    rng = np.random.default_rng(4)
    n, D = 50, 32
    q, k, v = rng.standard_normal(D), rng.standard_normal((n, D)), rng.standard_normal((n, D))
    scale = 1 / math.sqrt(D)
    s = scale * (k @ q)
    p = np.exp(s - s.max())
    p /= p.sum()
    out, lse = O.attn_one_query_f64(q, k, v, scale)
    np.testing.assert_allclose(out, p @ v, rtol=0, atol=1e-13)
    assert abs(lse - (s.max() + math.log(np.exp(s - s.max()).sum()))) < 1e-13


def test_attn_invariants_convexity_duplication_order():
    rng = np.random.default_rng(5)
    n, D = 23, 8
    q, k, v = rng.standard_normal(D), rng.standard_normal((n, D)), rng.standard_normal((n, D))
    out, lse = O.attn_one_query_f64(q, k, v, 0.7)
    assert (out <= v.max(axis=0) + 1e-15).all() and (out >= v.min(axis=0) - 1e-15).all()
    out2, lse2 = O.attn_one_query_f64(q, np.vstack([k, k]), np.vstack([v, v]), 0.7)
    np.testing.assert_allclose(out2, out, rtol=0, atol=1e-14)
    assert abs(lse2 - (lse + math.log(2))) < 1e-13
    perm = rng.permutation(n)
    out3, lse3 = O.attn_one_query_f64(q, k[perm], v[perm], 0.7)
    np.testing.assert_allclose(out3, out, rtol=0, atol=1e-14)
    assert abs(lse3 - lse) < 1e-13


def test_attn_large_scores_do_not_overflow():
    q = np.array([100.0, 0.0])
    k = np.array([[10.0, 0.0], [9.0, 0.0]])
    v = np.array([[1.0, 0.0], [0.0, 1.0]])
    out, lse = O.attn_one_query_f64(q, k, v, 1.0)
    assert np.isfinite(out).all() and abs(out[0] - 1.0) < 1e-12 and abs(lse - 1000.0) < 1e-9


def _tiny_paged(rng, B, Hq, Hkv, D, lens, num_pages=None, shuffle=True):
    P = IN.PAGE_SIZE
    lens = np.asarray(lens, dtype=np.int32)
    table, npg = IN.make_page_table(lens, seed=int(rng.integers(1 << 30)), fill=0)
    if not shuffle:
        o = 0
        for b, n in enumerate((lens + P - 1) // P):
            table[b, :n] = np.arange(o, o + n)
            o += n
    k = bf16(rng.standard_normal((npg, Hkv, P, D)))
    v = bf16(rng.standard_normal((npg, Hkv, P, D)))
    q = bf16(rng.standard_normal((B, Hq, D)))
    return q, k, v, table, lens


def test_paged_attention_matches_gather_plus_single_query():
    """The page-table walk, the HND layout and the GQA head->group map, checked by
    gathering each sequence with numpy indexing written independently here."""
    rng = np.random.default_rng(6)
    B, Hq, Hkv, D, P = 3, 4, 2, 8, IN.PAGE_SIZE
    q, k, v, table, lens = _tiny_paged(rng, B, Hq, Hkv, D, [1, 16, 45])
    out, lse = O.attn_decode(q, k, v, table, lens)
    kf, vf, qf = bf16_to_f64(k), bf16_to_f64(v), bf16_to_f64(q)
    for b in range(B):
        toks = np.arange(lens[b])
        pages = table[b, toks // P]
        for h in range(Hq):
            g = h // (Hq // Hkv)
            K = kf[pages, g, toks % P, :]
            V = vf[pages, g, toks % P, :]
            s = (K @ qf[b, h]) / math.sqrt(D)
            p = np.exp(s - s.max())
            p /= p.sum()
            np.testing.assert_allclose(out[b, h], p @ V, rtol=0, atol=1e-13)
            assert abs(lse[b, h] - (s.max() + math.log(np.exp(s - s.max()).sum()))) < 1e-12
    # n = 1: output is that token's V row, exactly
    assert (out[0, :, :] == vf[table[0, 0], np.arange(Hq) // 2, 0, :]).all()


def test_paged_attention_page_relocation_and_poison_invariance():
    """Moving pages physically (and updating the table) leaves the result
    bit-identical; NaNs in unreferenced slots/pages never reach the output."""
    rng = np.random.default_rng(7)
    B, Hq, Hkv, D = 2, 4, 2, 8
    q, k, v, table, lens = _tiny_paged(rng, B, Hq, Hkv, D, [19, 33])
    out, lse = O.attn_decode(q, k, v, table, lens)
    perm = rng.permutation(k.shape[0])            # new_page = perm[old_page]
    k2, v2 = np.empty_like(k), np.empty_like(v)
    k2[perm], v2[perm] = k, v
    out2, lse2 = O.attn_decode(q, k2, v2, perm[table].astype(np.int32), lens)
    assert (out2 == out).all() and (lse2 == lse).all()
    # poison everything that is not referenced
    used = np.zeros(k.shape[0] * IN.PAGE_SIZE, dtype=bool).reshape(-1, IN.PAGE_SIZE)
    for b in range(B):
        for j in range(lens[b]):
            used[table[b, j // 16], j % 16] = True
    kp, vp = k.copy(), v.copy()
    nan = bf16([float("nan")])[0]
    mask = np.broadcast_to(~used[:, None, :, None], k.shape)
    kp[mask] = nan
    vp[mask] = nan
    out3, lse3 = O.attn_decode(q, kp, vp, table, lens)
    assert (out3 == out).all() and (lse3 == lse).all()


def test_gqa_heads_of_one_group_share_kv():
    rng = np.random.default_rng(8)
    B, Hq, Hkv, D = 1, 8, 2, 8
    q, k, v, table, lens = _tiny_paged(rng, B, Hq, Hkv, D, [40])
    q[0, :, :] = q[0, 0, :]                         # same query in every head
    out, _ = O.attn_decode(q, k, v, table, lens)
    for h in range(1, 4):
        assert (out[0, h] == out[0, 0]).all()       # heads 0..3 -> KV head 0
    for h in range(5, 8):
        assert (out[0, h] == out[0, 4]).all()       # heads 4..7 -> KV head 1
    assert not np.allclose(out[0, 0], out[0, 4])


# --------------------------------------------------------------------------- dense FFN
def test_silu_identities():
    for z in [0.0, 0.5, 1.0, 3.25, 17.0]:
        assert abs(O.silu(z) - O.silu(-z) - z) < 1e-14
    assert O.silu(0.0) == 0.0
    assert abs(O.silu(40.0) - 40.0) < 1e-12 and abs(O.silu(-40.0)) < 1e-12
    assert math.isfinite(O.silu(-800.0)) or O.silu(-800.0) == 0.0
    assert abs(O.silu(1.0) - 1.0 / (1.0 + math.exp(-1.0))) < 1e-16


def test_swiglu_scalar_hand_case():
    c = GOLD["swiglu_scalar"]
    y = O.ffn_dense(bf16([[c["x"]]]), bf16([[c["w_gate"]]]), bf16([[c["w_up"]]]), bf16([[c["w_down"]]]))
    assert abs(y[0, 0] - c["y"]) < 1e-14


def _tiny_ffn(rng, T, H, I, E=0):
    lead = (E,) if E else ()
    x = bf16(rng.standard_normal((T, H)))
    wg = bf16(0.5 * rng.standard_normal(lead + (I, H)))
    wu = bf16(0.5 * rng.standard_normal(lead + (I, H)))
    wd = bf16(0.5 * rng.standard_normal(lead + (H, I)))
    return x, wg, wu, wd


def test_dense_ffn_matches_numpy_float64():
    """Catches a transposed operand (H != I and T > 1) or gate/up swapped."""
    rng = np.random.default_rng(10)
    T, H, I = 3, 8, 24
    x, wg, wu, wd = _tiny_ffn(rng, T, H, I)
    X, G, U, Dn = map(bf16_to_f64, (x, wg, wu, wd))
    g, u = X @ G.T, X @ U.T
    want = ((g / (1 + np.exp(-g))) * u) @ Dn.T
    np.testing.assert_allclose(O.ffn_dense(x, wg, wu, wd), want, rtol=0, atol=1e-12)
    swapped = O.ffn_dense(x, wu, wg, wd)
    assert np.abs(swapped - want).max() > 1e-3


def test_dense_ffn_zero_and_scaling_properties():
    rng = np.random.default_rng(11)
    T, H, I = 2, 8, 16
    x, wg, wu, wd = _tiny_ffn(rng, T, H, I)
    y = O.ffn_dense(x, wg, wu, wd)
    assert (O.ffn_dense(x, np.zeros_like(wg), wu, wd) == 0).all()       # silu(0) = 0
    assert (O.ffn_dense(np.zeros_like(x), wg, wu, wd) == 0).all()
    two = lambda w: bf16(2.0 * bf16_to_f64(w))                           # exact in bf16
    assert (O.ffn_dense(x, wg, two(wu), wd) == 2.0 * y).all()
    assert (O.ffn_dense(x, wg, wu, two(wd)) == 2.0 * y).all()


def test_linear_matches_numpy():
    rng = np.random.default_rng(12)
    x = rng.standard_normal((3, 10))
    w = bf16(rng.standard_normal((7, 10)))
    np.testing.assert_allclose(O.linear(x, w), x @ bf16_to_f64(w).T, rtol=0, atol=1e-13)


# --------------------------------------------------------------------------- MoE routing
def _brute_force_top2(l):
    """Best pair under (value descending, index ascending), by enumerating all pairs."""
    E = len(l)
    best = None
    for a, b in itertools.permutations(range(E), 2):
        key = (-l[a], a, -l[b], b)
        ok_order = (l[a] > l[b]) or (l[a] == l[b] and a < b)
        if ok_order and (best is None or key < best[0]):
            best = (key, (a, b))
    return best[1]


@pytest.mark.parametrize("grid", [False, True])
def test_routing_matches_exhaustive_top2(grid):
    rng = np.random.default_rng(13)
    T, E = 400, 8
    if grid:   # three-valued logits force ties everywhere
        logits = rng.integers(-1, 2, size=(T, E)).astype(np.float32)
    else:
        logits = rng.standard_normal((T, E)).astype(np.float32)
    idx, gate = O.moe_route(logits, 2)
    for t in range(T):
        assert tuple(idx[t]) == _brute_force_top2(logits[t]), (t, logits[t])
        assert idx[t, 0] != idx[t, 1]
    np.testing.assert_allclose(gate.sum(axis=1), 1.0, rtol=0, atol=1e-15)
    assert (gate[:, 0] >= gate[:, 1]).all()


def test_routing_hand_cases():
    c = GOLD["gates_two_experts"]
    idx, gate = O.moe_route(np.array([c["logits"]], dtype=np.float32), 2)
    assert idx[0].tolist() == c["idx"]
    np.testing.assert_allclose(gate[0], c["gate"], rtol=0, atol=1e-7)   # fp32 ln 3 as input
    idx, gate = O.moe_route(np.full((1, 8), 0.25, dtype=np.float32), 2)
    assert idx[0].tolist() == [0, 1] and gate[0].tolist() == [0.5, 0.5]
    idx, gate = O.moe_route(np.array([[1, 5, 5, 2]], dtype=np.float32), 1)
    assert idx[0].tolist() == [1] and gate[0].tolist() == [1.0]
    # softmax over all experts then renormalised over the selected two gives the same gates
    l = np.random.default_rng(14).standard_normal((1, 8)).astype(np.float32)
    idx, gate = O.moe_route(l, 2)
    p = np.exp(l[0].astype(np.float64)); p /= p.sum()
    np.testing.assert_allclose(gate[0], p[idx[0]] / p[idx[0]].sum(), rtol=0, atol=1e-15)


def test_permutation_is_stable_bijection():
    rng = np.random.default_rng(15)
    T, E, K = 61, 8, 2
    idx, _ = O.moe_route(rng.standard_normal((T, E)).astype(np.float32), K)
    counts, offsets, pos = O.moe_permute(idx, E)
    assert counts.sum() == T * K and (counts == np.bincount(idx.ravel(), minlength=E)).all()
    assert (offsets == np.concatenate([[0], np.cumsum(counts)])).all()
    assert sorted(pos.ravel().tolist()) == list(range(T * K))
    order = np.argsort(idx.ravel(), kind="stable")          # numpy's stable sort = (expert, t, k) order
    want = np.empty(T * K, dtype=np.int32)
    want[order] = np.arange(T * K)
    assert (pos.ravel() == want).all()


# --------------------------------------------------------------------------- MoE values
def test_moe_with_identical_experts_equals_dense():
    rng = np.random.default_rng(16)
    T, H, I, E = 3, 8, 16, 4
    x, wg, wu, wd = _tiny_ffn(rng, T, H, I)
    logits = rng.standard_normal((T, E)).astype(np.float32)
    rep = lambda w: np.ascontiguousarray(np.broadcast_to(w, (E,) + w.shape))
    y, _, _ = O.ffn_moe(x, logits, rep(wg), rep(wu), rep(wd), 2)
    np.testing.assert_allclose(y, O.ffn_dense(x, wg, wu, wd), rtol=0, atol=1e-13)


def test_moe_single_expert_and_dominant_logit():
    rng = np.random.default_rng(17)
    T, H, I, E = 2, 8, 16, 4
    x, wg, wu, wd = _tiny_ffn(rng, T, H, I, E)
    y, idx, gate = O.ffn_moe(x, np.zeros((T, 1), np.float32), wg[:1], wu[:1], wd[:1], 1)
    assert (y == O.ffn_dense(x, wg[0], wu[0], wd[0])).all()
    logits = np.zeros((T, E), np.float32)
    logits[:, 2] = 50.0
    y, idx, gate = O.ffn_moe(x, logits, wg, wu, wd, 1)
    assert (idx == 2).all() and (y == O.ffn_dense(x, wg[2], wu[2], wd[2])).all()


def test_moe_matches_explicit_gated_sum():
    rng = np.random.default_rng(18)
    T, H, I, E = 5, 8, 16, 8
    x, wg, wu, wd = _tiny_ffn(rng, T, H, I, E)
    logits = rng.standard_normal((T, E)).astype(np.float32)
    y, idx, gate = O.ffn_moe(x, logits, wg, wu, wd, 2)
    for t in range(T):
        want = sum(gate[t, k] * O.ffn_dense(x[t:t + 1], wg[idx[t, k]], wu[idx[t, k]], wd[idx[t, k]])[0]
                   for k in range(2))
        np.testing.assert_allclose(y[t], want, rtol=0, atol=1e-13)


# --------------------------------------------------------------------------- layer step, Eq. 2
def test_layer_step_is_the_composition():
    rng = np.random.default_rng(19)
    B, Hq, Hkv, D, H, I = 3, 4, 2, 8, 16, 24
    q, k, v, table, lens = _tiny_paged(rng, B, Hq, Hkv, D, [5, 16, 31])
    wo = bf16(0.3 * rng.standard_normal((H, Hq * D)))
    _, wg, wu, wd = _tiny_ffn(rng, B, H, I)
    a, y = O.layer_step(q, k, v, table, lens, wo, wg, wu, wd)
    a2, _ = O.attn_decode(q, k, v, table, lens)
    assert (a == a2).all()
    x = O.linear(a2.reshape(B, Hq * D), wo)
    np.testing.assert_allclose(x, a2.reshape(B, -1) @ bf16_to_f64(wo).T, rtol=0, atol=1e-13)
    assert (y == O.ffn_dense(x, wg, wu, wd)).all()
    # rows are independent: any split of the batch into microbatches gives the same rows
    for lo, hi in [(0, 1), (1, 3)]:
        _, ys = O.layer_step(q[lo:hi], k, v, table[lo:hi], lens[lo:hi], wo, wg, wu, wd)
        assert (ys == y[lo:hi]).all()


def test_layer_step_moe_and_identity_projection():
    rng = np.random.default_rng(20)
    B, Hq, Hkv, D, I, E = 2, 4, 2, 4, 8, 4
    H = Hq * D
    q, k, v, table, lens = _tiny_paged(rng, B, Hq, Hkv, D, [9, 20])
    _, wg, wu, wd = _tiny_ffn(rng, B, H, I, E)
    logits = rng.standard_normal((B, E)).astype(np.float32)
    a, y = O.layer_step(q, k, v, table, lens, None, wg, wu, wd, logits=logits, top_k=2)
    y2, _, _ = O.ffn_moe(a.reshape(B, H), logits, wg, wu, wd, 2)
    assert (y == y2).all()


def test_eq2_pipeline_latency_model():
    for c in GOLD["eq2"]["cases"]:
        assert O.eq2_layer_time(c["t_a"], c["t_f"], c["t_comm"], c["M"]) == c["t_layer"]
    assert O.eq2_layer_time(2.0, 9.0, 0.0, 3) == 9.0


# --------------------------------------------------------------------------- input recipe checks
def test_zipf_biases_give_zipf_expert_shares():
    """The skewed-load recipe: shares of the T*K assignments per expert follow
    Zipf(1.2) by rank (checked with the oracle's routing on a large sample)."""
    cfg = IN.CONFIGS[5]
    logits = IN.make_router_logits(cfg, tokens=40000).numpy()
    idx, _ = O.moe_route(logits, 2)
    share = np.bincount(idx.ravel(), minlength=8) / idx.size
    r2e = IN.zipf_rank_to_expert(cfg)
    np.testing.assert_allclose(share[r2e], IN.zipf_shares(8, 1.2), rtol=0, atol=0.012)


def test_context_length_recipes():
    for cid, cfg in IN.CONFIGS.items():
        lens = IN.make_seq_lens(cfg)
        assert lens.shape == (cfg.batch,) and lens.min() >= cfg.len_lo and lens.max() <= cfg.len_hi
    big = IN.make_seq_lens(IN.CONFIGS[3], batch=20000)
    assert abs(np.median(big) - 2048) < 60
    kv = IN.make_paged_kv(IN.CONFIGS[1], poison=True)
    tab, lens = kv.page_table.numpy(), kv.seq_lens.numpy()
    used = [tab[b, j] for b in range(len(lens)) for j in range((lens[b] + 15) // 16)]
    assert len(set(used)) == len(used) and max(used) < kv.num_pages
