"""Pins for the oracle's whole-decoder-layer operators (RMS normalisation, rotary embedding,
bf16 storage rounding, K/V append, residual blocks): closed forms, hand cases, invariants and
special cases that reduce to functions pinned elsewhere.  No GPU needed."""
import math

import numpy as np
import torch

from oracle import oracle as O
from paper_2608_01891_b200 import inputs as IN


def bf16(a) -> np.ndarray:
    t = torch.as_tensor(np.asarray(a, dtype=np.float32)).to(torch.bfloat16)
    return IN.bf16_bits(t).copy()


def bf16_to_f64(u16: np.ndarray) -> np.ndarray:
    return (u16.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


# --------------------------------------------------------------------------- bf16 storage rounding
def test_f64_to_bf16_matches_library_rounding_on_floats():
    rng = np.random.default_rng(0)
    x = (rng.standard_normal(4000) * np.exp(rng.uniform(-20, 20, 4000))).astype(np.float32)
    want = bf16(x)                                   # torch's fp32 -> bf16 (round to nearest even)
    got = O.f64_to_bf16(x.astype(np.float64))
    assert (got == want).all()


def test_f64_to_bf16_hand_cases():
    # ties go to the even neighbour; one rounding only (a value just above a tie rounds up even
    # though its fp32 image is the tie itself); subnormals, overflow, signed zero
    cases = [(1.0, 0x3F80), (1.0 + 2.0 ** -8, 0x3F80), (1.0 + 3 * 2.0 ** -8, 0x3F82),
             (1.0 + 2.0 ** -8 + 2.0 ** -40, 0x3F81), (-2.5, 0xC020), (2.0 ** -133, 0x0001),
             (2.0 ** -134, 0x0000), (3 * 2.0 ** -134, 0x0002), (1e39, 0x7F80), (-0.0, 0x8000)]
    got = O.f64_to_bf16(np.array([c[0] for c in cases]))
    assert got.tolist() == [c[1] for c in cases]


# --------------------------------------------------------------------------- RMS normalisation
def test_rmsnorm_hand_case():
    y = O.rmsnorm(np.array([[3.0, 4.0]]), None, 0.0)
    np.testing.assert_allclose(y, np.array([[3.0, 4.0]]) / math.sqrt(12.5), rtol=0, atol=1e-15)


def test_rmsnorm_constant_vector_closed_form():
    c, eps, H = -1.75, 1e-3, 37
    y = O.rmsnorm(np.full((1, H), c), None, eps)
    np.testing.assert_allclose(y, np.full((1, H), c / math.sqrt(c * c + eps)), rtol=0, atol=1e-15)


def test_rmsnorm_invariants_and_weights():
    rng = np.random.default_rng(3)
    x = rng.standard_normal((5, 64))
    y = O.rmsnorm(x, None, 0.0)
    np.testing.assert_allclose((y * y).mean(axis=1), 1.0, rtol=0, atol=1e-14)     # unit mean square
    np.testing.assert_allclose(O.rmsnorm(7.5 * x, None, 0.0), y, rtol=0, atol=1e-14)   # scale-free
    w = bf16(rng.uniform(0.5, 2.0, 64))
    np.testing.assert_allclose(O.rmsnorm(x, w, 0.0), y * bf16_to_f64(w)[None, :], rtol=0, atol=1e-14)
    # rows are independent
    np.testing.assert_array_equal(O.rmsnorm(x[2:3], w, 1e-6), O.rmsnorm(x, w, 1e-6)[2:3])
    # eps is added to the mean square, not to the sum or to the root
    x1 = np.array([[2.0, 0.0, 0.0, 0.0]])
    np.testing.assert_allclose(O.rmsnorm(x1, None, 3.0)[0, 0], 2.0 / math.sqrt(1.0 + 3.0), rtol=0, atol=1e-15)


# --------------------------------------------------------------------------- rotary embedding
def test_rope_position_zero_is_identity():
    v = np.random.default_rng(1).standard_normal(16)
    np.testing.assert_array_equal(O.rope(v, 0.0, 1e6), v)


def test_rope_two_dims_is_a_plane_rotation():
    for pos in (1.0, 2.5, 100.0):
        out = O.rope(np.array([1.0, 0.0]), pos, 1e4)
        np.testing.assert_allclose(out, [math.cos(pos), math.sin(pos)], rtol=0, atol=1e-15)
        out = O.rope(np.array([0.0, 1.0]), pos, 1e4)
        np.testing.assert_allclose(out, [-math.sin(pos), math.cos(pos)], rtol=0, atol=1e-15)


def test_rope_pairs_and_frequencies():
    # D = 4, theta = 10^4: pair (0, 2) turns by pos, pair (1, 3) by pos * theta^(-2/4) = pos / 100
    pos = 50.0
    out = O.rope(np.array([1.0, 0.0, 0.0, 0.0]), pos, 1e4)
    np.testing.assert_allclose(out, [math.cos(pos), 0.0, math.sin(pos), 0.0], rtol=0, atol=1e-15)
    out = O.rope(np.array([0.0, 1.0, 0.0, 0.0]), pos, 1e4)
    np.testing.assert_allclose(out, [0.0, math.cos(0.5), 0.0, math.sin(0.5)], rtol=0, atol=1e-14)
    out = O.rope(np.array([0.0, 0.0, 0.0, 2.0]), pos, 1e4)
    np.testing.assert_allclose(out, [0.0, -2 * math.sin(0.5), 0.0, 2 * math.cos(0.5)], rtol=0, atol=1e-14)


def test_rope_preserves_norm_and_depends_on_relative_position():
    rng = np.random.default_rng(2)
    q, k = rng.standard_normal(64), rng.standard_normal(64)
    for m, n in ((7, 3), (1000, 990), (5, 5)):
        qm, kn = O.rope(q, m, 1e6), O.rope(k, n, 1e6)
        assert abs(np.linalg.norm(qm) - np.linalg.norm(q)) < 1e-12
        want = float(O.rope(q, m - n, 1e6) @ k)
        assert abs(float(qm @ kn) - want) < 1e-10


# --------------------------------------------------------------------------- attention with f64 queries
def test_attn_f64q_equals_bf16_query_version_on_representable_queries():
    cfg = IN.CONFIGS[1]
    kv = IN.make_paged_kv(cfg)
    q = IN.make_q(cfg)
    k, v = IN.bf16_bits(kv.k_cache), IN.bf16_bits(kv.v_cache)
    a0, l0 = O.attn_decode(IN.bf16_bits(q), k, v, kv.page_table.numpy(), kv.seq_lens.numpy())
    a1, l1 = O.attn_decode_f64q(bf16_to_f64(IN.bf16_bits(q)), k, v, kv.page_table.numpy(), kv.seq_lens.numpy())
    np.testing.assert_array_equal(a0, a1)
    np.testing.assert_array_equal(l0, l1)


# --------------------------------------------------------------------------- QKV, rope, append
def _tiny_layer(rng, B=2, Hq=4, Hkv=2, D=8, H=32, I=24, E=0, lens=(1, 17), qk_norm=True):
    P = IN.PAGE_SIZE
    lens = np.asarray(lens, dtype=np.int32)
    pages = (lens + P - 1) // P
    num_pages = int(pages.sum()) + 3
    perm = rng.permutation(num_pages)
    table = np.zeros((B, int(pages.max())), dtype=np.int32)
    o = 0
    for b in range(B):
        table[b, :pages[b]] = perm[o:o + pages[b]]
        o += int(pages[b])
    k = bf16(rng.standard_normal((num_pages, Hkv, P, D)))
    v = bf16(rng.standard_normal((num_pages, Hkv, P, D)))
    lead = (E,) if E else ()
    w = {
        "ln_attn": bf16(rng.uniform(0.5, 1.5, H)), "qkv": bf16(rng.standard_normal(((Hq + 2 * Hkv) * D, H)) * 0.2),
        "q_norm": bf16(rng.uniform(0.5, 1.5, D)) if qk_norm else None,
        "k_norm": bf16(rng.uniform(0.5, 1.5, D)) if qk_norm else None,
        "o": bf16(rng.standard_normal((H, Hq * D)) * 0.2), "ln_ffn": bf16(rng.uniform(0.5, 1.5, H)),
        "gate": bf16(rng.standard_normal(lead + (I, H)) * 0.2), "up": bf16(rng.standard_normal(lead + (I, H)) * 0.2),
        "down": bf16(rng.standard_normal(lead + (H, I)) * 0.2),
        "router": bf16(rng.standard_normal((E, H))) if E else None,
    }
    x = rng.standard_normal((B, H))
    return x, w, k, v, table, lens


def test_qkv_rope_append_writes_one_slot_per_head_with_rotated_keys():
    rng = np.random.default_rng(5)
    Hq, Hkv, D, H, P = 4, 2, 8, 32, IN.PAGE_SIZE
    x, w, k, v, table, lens = _tiny_layer(rng, Hq=Hq, Hkv=Hkv, D=D, H=H, lens=(1, 17))
    k0, v0 = k.copy(), v.copy()
    eps, theta = 1e-5, 1e4
    q = O.qkv_rope_append(x, w["ln_attn"], w["qkv"], w["q_norm"], w["k_norm"], eps, theta, k, v, table, lens, Hq)
    # expected, from functions pinned on their own
    qkv = O.linear(O.rmsnorm(x, w["ln_attn"], eps), w["qkv"])
    touched = np.zeros(k.shape[:3], dtype=bool)
    for b in range(2):
        pos = int(lens[b]) - 1
        page, slot = int(table[b, pos // P]), pos % P
        for h in range(Hq):
            want = O.rope(O.rmsnorm(qkv[b:b + 1, h * D:(h + 1) * D], w["q_norm"], eps)[0], pos, theta)
            np.testing.assert_allclose(q[b, h], want, rtol=0, atol=1e-14)
        for g in range(Hkv):
            kk = O.rope(O.rmsnorm(qkv[b:b + 1, (Hq + g) * D:(Hq + g + 1) * D], w["k_norm"], eps)[0], pos, theta)
            vv = qkv[b, (Hq + Hkv + g) * D:(Hq + Hkv + g + 1) * D]
            assert (k[page, g, slot] == O.f64_to_bf16(kk)).all()
            assert (v[page, g, slot] == O.f64_to_bf16(vv)).all()      # values are not rotated
            touched[page, g, slot] = True
    # sequence 0 has length 1: position 0, so its key is only normalised, not turned
    assert touched.sum() == 2 * Hkv
    assert (k[~touched] == k0[~touched]).all() and (v[~touched] == v0[~touched]).all()
    # without the per-head gains the normalisation step is skipped entirely
    k2, v2 = k0.copy(), v0.copy()
    q2 = O.qkv_rope_append(x, w["ln_attn"], w["qkv"], None, None, eps, theta, k2, v2, table, lens, Hq)
    np.testing.assert_allclose(q2[1, 0], O.rope(qkv[1, 0:D], 16, theta), rtol=0, atol=1e-14)


# --------------------------------------------------------------------------- whole layer
def test_decoder_layer_zero_output_weights_pass_the_residual_through():
    rng = np.random.default_rng(6)
    x, w, k, v, table, lens = _tiny_layer(rng)
    w["o"] = np.zeros_like(w["o"])
    w["down"] = np.zeros_like(w["down"])
    _, h1, out = O.decoder_layer(x, w, k, v, table, lens, 4, 1e-6, 1e4)
    np.testing.assert_array_equal(h1, x)
    np.testing.assert_array_equal(out, x)


def test_decoder_layer_single_token_sequences_closed_form():
    # With one cached token the softmax weight is 1: the attention output is the value just
    # appended (after its bf16 storage rounding), whatever q and k are.
    rng = np.random.default_rng(7)
    Hq, Hkv, D, H = 4, 2, 8, 32
    x, w, k, v, table, lens = _tiny_layer(rng, lens=(1, 1))
    eps, theta = 1e-6, 1e4
    _, h1, out = O.decoder_layer(x, w, k, v, table, lens, Hq, eps, theta)
    qkv = O.linear(O.rmsnorm(x, w["ln_attn"], eps), w["qkv"])
    vals = bf16_to_f64(O.f64_to_bf16(qkv[:, (Hq + Hkv) * D:]))           # [B, Hkv*D]
    a = np.repeat(vals.reshape(2, Hkv, D), Hq // Hkv, axis=1).reshape(2, Hq * D)   # head h reads KV head h // G
    h1_want = x + O.linear(a, w["o"])
    np.testing.assert_allclose(h1, h1_want, rtol=0, atol=1e-13)
    out_want = h1_want + O.ffn_dense(O.rmsnorm(h1_want, w["ln_ffn"], eps), w["gate"], w["up"], w["down"])
    np.testing.assert_allclose(out, out_want, rtol=0, atol=1e-12)


def test_decoder_layer_general_case_from_pinned_parts():
    rng = np.random.default_rng(8)
    Hq = 4
    x, w, k, v, table, lens = _tiny_layer(rng, lens=(9, 40))
    ka, va = k.copy(), v.copy()
    eps, theta = 1e-5, 1e6
    q, h1, out = O.decoder_layer(x, w, k, v, table, lens, Hq, eps, theta)
    q_want = O.qkv_rope_append(x, w["ln_attn"], w["qkv"], w["q_norm"], w["k_norm"], eps, theta, ka, va, table, lens, Hq)
    assert (ka == k).all() and (va == v).all()
    np.testing.assert_array_equal(q, q_want)
    a, _ = O.attn_decode_f64q(q_want, ka, va, table, lens)
    h1_want = x + O.linear(a.reshape(2, -1), w["o"])
    np.testing.assert_allclose(h1, h1_want, rtol=0, atol=1e-13)
    out_want = h1_want + O.ffn_dense(O.rmsnorm(h1_want, w["ln_ffn"], eps), w["gate"], w["up"], w["down"])
    np.testing.assert_allclose(out, out_want, rtol=0, atol=1e-12)
    # the appended token takes part in the attention: removing it changes the result
    a_short, _ = O.attn_decode_f64q(q_want, ka, va, table, lens - 1)
    assert np.abs(a_short - a).max() > 1e-3


def test_decoder_layer_moe_routes_on_the_normalised_ffn_input():
    rng = np.random.default_rng(9)
    x, w, k, v, table, lens = _tiny_layer(rng, E=4, lens=(5, 20))
    eps, theta = 1e-5, 1e6
    _, h1, out = O.decoder_layer(x, w, k, v, table, lens, 4, eps, theta, top_k=2)
    xn = O.rmsnorm(h1, w["ln_ffn"], eps)
    logits = O.router_logits(xn, w["router"]).astype(np.float32)
    f, _, _ = O.ffn_moe(xn, logits, w["gate"], w["up"], w["down"], 2)
    np.testing.assert_allclose(out, h1 + f, rtol=0, atol=1e-12)
    # with the logits given by the caller the router weight is not used
    w2 = dict(w, router=None)
    k2, v2 = k.copy(), v.copy()
    given = rng.standard_normal((2, 4)).astype(np.float32)
    _, h1b, outb = O.decoder_layer(x, w2, k2, v2, table, lens, 4, eps, theta, top_k=2, logits=given)
    fb, _, _ = O.ffn_moe(O.rmsnorm(h1b, w["ln_ffn"], eps), given, w["gate"], w["up"], w["down"], 2)
    np.testing.assert_allclose(outb, h1b + fb, rtol=0, atol=1e-12)


def test_decoder_layer_one_expert_equals_dense():
    rng = np.random.default_rng(10)
    x, w, k, v, table, lens = _tiny_layer(rng, E=1, lens=(3, 33))
    k2, v2 = k.copy(), v.copy()
    _, _, out_moe = O.decoder_layer(x, w, k, v, table, lens, 4, 1e-6, 1e4, top_k=1)
    wd = dict(w, gate=w["gate"][0], up=w["up"][0], down=w["down"][0], router=None)
    _, _, out_dense = O.decoder_layer(x, wd, k2, v2, table, lens, 4, 1e-6, 1e4)
    np.testing.assert_allclose(out_moe, out_dense, rtol=0, atol=1e-13)


# --------------------------------------------------------------------------- prefill (causal) attention
def _prefill_case(rng, lens, q_lens, Hq=4, Hkv=2, D=8):
    P = IN.PAGE_SIZE
    lens = np.asarray(lens, dtype=np.int32)
    pages = (lens + P - 1) // P
    num_pages = int(pages.sum()) + 2
    perm = rng.permutation(num_pages)
    table = np.zeros((len(lens), int(pages.max())), dtype=np.int32)
    o = 0
    for b in range(len(lens)):
        table[b, :pages[b]] = perm[o:o + pages[b]]
        o += int(pages[b])
    k = bf16(rng.standard_normal((num_pages, Hkv, P, D)))
    v = bf16(rng.standard_normal((num_pages, Hkv, P, D)))
    q_off = np.concatenate([[0], np.cumsum(q_lens)]).astype(np.int32)
    q = bf16(rng.standard_normal((int(q_off[-1]), Hq, D)))
    return q, k, v, table, lens, q_off


def test_prefill_with_one_query_per_sequence_is_decode_attention():
    rng = np.random.default_rng(20)
    q, k, v, table, lens, q_off = _prefill_case(rng, (5, 33, 16), (1, 1, 1))
    got = O.attn_prefill(q, k, v, table, lens, q_off)
    want, _ = O.attn_decode(q, k, v, table, lens)
    np.testing.assert_array_equal(got, want)


def test_prefill_is_causal_row_by_row():
    # query i of a sequence sees exactly the cached tokens up to its own position: the same as decoding with a
    # sequence length cut at that position
    rng = np.random.default_rng(21)
    q, k, v, table, lens, q_off = _prefill_case(rng, (20, 37), (20, 9))
    got = O.attn_prefill(q, k, v, table, lens, q_off)
    for b in range(2):
        m = int(q_off[b + 1] - q_off[b])
        for i in range(m):
            row = int(q_off[b]) + i
            cut = np.array([int(lens[b]) - m + i + 1], dtype=np.int32)
            want, _ = O.attn_decode(q[row:row + 1], k, v, table[b:b + 1], cut)
            np.testing.assert_array_equal(got[row], want[0])
    # the first token of a full prefill attends to itself only: its output is its own value row
    vals = bf16_to_f64(v)
    first = vals[table[0, 0], :, 0, :]                      # [Hkv, D]
    np.testing.assert_array_equal(got[0], np.repeat(first, 2, axis=0))
    # a later key cannot influence an earlier query
    k2, v2 = k.copy(), v.copy()
    last_page, last_slot = table[0, 19 // 16], 19 % 16
    k2[last_page, :, last_slot] = bf16(np.full((2, 8), 50.0))
    v2[last_page, :, last_slot] = bf16(np.full((2, 8), -7.0))
    got2 = O.attn_prefill(q, k2, v2, table, lens, q_off)
    np.testing.assert_array_equal(got2[:19], got[:19])
    assert np.abs(got2[19] - got[19]).max() > 1e-3


# --------------------------------------------------------------------------- prefill layer
def _prompt_rows(q_off, b, i):
    return int(q_off[b]) + i


def test_prefill_layer_equals_the_decode_layer_fed_one_token_at_a_time():
    """A layer's output for a prompt token depends on the earlier tokens only through the cache, so prefilling a
    prompt must give, row by row, what the (separately pinned) decode layer gives when the same rows are fed one
    position at a time.  Dense and mixture-of-experts FFN, two ragged prompts, one of them behind a cached prefix."""
    for E in (0, 4):
        rng = np.random.default_rng(21 + E)
        Hq, eps, theta = 4, 1e-5, 1e4
        lens = np.asarray([7, 21], dtype=np.int32)
        new = np.asarray([7, 5], dtype=np.int32)            # sequence 1 already holds 16 cached tokens
        _, w, k, v, table, _ = _tiny_layer(rng, lens=tuple(lens), E=E)
        q_off = np.concatenate([[0], np.cumsum(new)]).astype(np.int32)
        T = int(q_off[-1])
        x = rng.standard_normal((T, 32))
        kp, vp = k.copy(), v.copy()
        q, h1, out = O.prefill_layer(x, w, kp, vp, table, lens, q_off, Hq, eps, theta, top_k=2 if E else 0)
        kd, vd = k.copy(), v.copy()
        for b in range(2):
            for i in range(int(new[b])):
                r = _prompt_rows(q_off, b, i)
                cur = np.asarray([lens[b] - new[b] + i + 1], dtype=np.int32)
                q1, h11, out1 = O.decoder_layer(x[r:r + 1], w, kd, vd, table[b:b + 1], cur, Hq, eps, theta,
                                                top_k=2 if E else 0)
                np.testing.assert_allclose(q[r], q1[0], rtol=0, atol=1e-13)
                np.testing.assert_allclose(h1[r], h11[0], rtol=0, atol=1e-12)
                np.testing.assert_allclose(out[r], out1[0], rtol=0, atol=1e-11)
        assert (kp == kd).all() and (vp == vd).all()         # the same cache slots, bit for bit
        assert (kp != k).any()


def test_prefill_layer_in_two_chunks_equals_one_pass():
    rng = np.random.default_rng(31)
    Hq, eps, theta = 4, 1e-5, 1e6
    lens = np.asarray([19, 6], dtype=np.int32)
    _, w, k, v, table, _ = _tiny_layer(rng, lens=tuple(lens))
    q_off = np.asarray([0, 19, 25], dtype=np.int32)
    x = rng.standard_normal((25, 32))
    k1, v1 = k.copy(), v.copy()
    _, _, out = O.prefill_layer(x, w, k1, v1, table, lens, q_off, Hq, eps, theta)
    # first 11 / 2 tokens, then the rest
    first = np.asarray([11, 2], dtype=np.int32)
    k2, v2 = k.copy(), v.copy()
    rows_a = np.r_[0:11, 19:21]
    rows_b = np.r_[11:19, 21:25]
    _, _, out_a = O.prefill_layer(x[rows_a], w, k2, v2, table, first, np.asarray([0, 11, 13], dtype=np.int32), Hq, eps, theta)
    _, _, out_b = O.prefill_layer(x[rows_b], w, k2, v2, table, lens, np.asarray([0, 8, 12], dtype=np.int32), Hq, eps, theta)
    np.testing.assert_allclose(out[rows_a], out_a, rtol=0, atol=1e-12)
    np.testing.assert_allclose(out[rows_b], out_b, rtol=0, atol=1e-12)
    assert (k1 == k2).all() and (v1 == v2).all()
