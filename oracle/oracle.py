"""ctypes front end of the fp64 CPU oracle (``aflex_oracle.c``).

TEST INFRASTRUCTURE ONLY: imported by ``tests/``, by the smoke check and by the
benchmark's CPU-baseline leg.  The CUDA library and its Python binding never
import this module, and this module imports nothing of theirs.

All array arguments are numpy arrays: bf16 tensors as ``uint16`` bit patterns,
logits as ``float32``, integer tables as ``int32``; results come back as
``float64`` / ``int32`` arrays.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from typing import Optional, Tuple

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "aflex_oracle.c")
_LIB = os.path.join(_HERE, "libaflex_oracle.so")
_lib = None


def build(force: bool = False) -> str:
    """Compile the oracle with gcc (strict fp: no -ffast-math)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        cmd = ["gcc", "-O2", "-std=c99", "-fopenmp", "-fvisibility=hidden", "-shared", "-fPIC",
               _SRC, "-o", _LIB, "-lm"]
        subprocess.run(cmd, check=True)
    return _LIB


_u16p = ctypes.POINTER(ctypes.c_uint16)
_i32p = ctypes.POINTER(ctypes.c_int32)
_f32p = ctypes.POINTER(ctypes.c_float)
_f64p = ctypes.POINTER(ctypes.c_double)


def _load():
    global _lib
    if _lib is None:
        build()
        _lib = ctypes.CDLL(_LIB)
        _lib.oracle_num_threads.restype = ctypes.c_int
        _lib.oracle_silu.restype = ctypes.c_double
        _lib.oracle_silu.argtypes = [ctypes.c_double]
        _lib.oracle_eq2_layer_time.restype = ctypes.c_double
        _lib.oracle_eq2_layer_time.argtypes = [ctypes.c_double, ctypes.c_double, ctypes.c_double, ctypes.c_int]
    return _lib


def _p(a: Optional[np.ndarray], ty):
    if a is None:
        return None
    assert a.flags["C_CONTIGUOUS"], "oracle arrays must be C-contiguous"
    return a.ctypes.data_as(ty)


def _u16(a) -> np.ndarray:
    a = np.ascontiguousarray(a)
    assert a.dtype == np.uint16, a.dtype
    return a


def num_threads() -> int:
    return int(_load().oracle_num_threads())


def set_num_threads(n: int) -> None:
    _load().oracle_set_num_threads(ctypes.c_int(n))


def silu(z: float) -> float:
    return float(_load().oracle_silu(float(z)))


def eq2_layer_time(t_a: float, t_f: float, t_comm: float, M: int) -> float:
    return float(_load().oracle_eq2_layer_time(t_a, t_f, t_comm, int(M)))


def attn_one_query_f64(q, keys, vals, scale: float) -> Tuple[np.ndarray, float]:
    q = np.ascontiguousarray(q, dtype=np.float64)
    keys = np.ascontiguousarray(keys, dtype=np.float64)
    vals = np.ascontiguousarray(vals, dtype=np.float64)
    n, D = keys.shape
    assert q.shape == (D,) and vals.shape == (n, D) and n >= 1
    out = np.zeros(D, dtype=np.float64)
    lse = ctypes.c_double(0.0)
    _load().oracle_attn_one_query_f64(_p(q, _f64p), _p(keys, _f64p), _p(vals, _f64p), n, D,
                                      ctypes.c_double(scale), _p(out, _f64p), ctypes.byref(lse))
    return out, float(lse.value)


def attn_decode(q, k_cache, v_cache, page_table, seq_lens, scale: Optional[float] = None):
    """q u16 [B,Hq,D]; caches u16 [num_pages,Hkv,P,D]; page_table i32 [B,max_pages];
    seq_lens i32 [B] -> (out f64 [B,Hq,D], lse f64 [B,Hq])."""
    q, k_cache, v_cache = _u16(q), _u16(k_cache), _u16(v_cache)
    page_table = np.ascontiguousarray(page_table, dtype=np.int32)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    B, Hq, D = q.shape
    _, Hkv, P, D2 = k_cache.shape
    assert D2 == D and v_cache.shape == k_cache.shape and Hq % Hkv == 0
    assert page_table.shape[0] == B and seq_lens.shape == (B,) and (seq_lens >= 1).all()
    if scale is None:
        scale = 1.0 / np.sqrt(float(D))
    out = np.zeros((B, Hq, D), dtype=np.float64)
    lse = np.zeros((B, Hq), dtype=np.float64)
    _load().oracle_attn_decode(_p(q, _u16p), _p(k_cache, _u16p), _p(v_cache, _u16p),
                               _p(page_table, _i32p), int(page_table.shape[1]), _p(seq_lens, _i32p),
                               B, Hq, Hkv, D, P, ctypes.c_double(scale), _p(out, _f64p), _p(lse, _f64p))
    return out, lse


def linear(x, w) -> np.ndarray:
    """x f64 [T,K], w u16 [N,K] -> f64 [T,N]."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    w = _u16(w)
    T, K = x.shape
    N, K2 = w.shape
    assert K == K2
    y = np.zeros((T, N), dtype=np.float64)
    _load().oracle_linear(_p(x, _f64p), _p(w, _u16p), T, K, N, _p(y, _f64p))
    return y


def ffn_dense(x, w_gate, w_up, w_down) -> np.ndarray:
    """x u16 or f64 [T,H]; w_gate,w_up u16 [I,H]; w_down u16 [H,I] -> f64 [T,H]."""
    w_gate, w_up, w_down = _u16(w_gate), _u16(w_up), _u16(w_down)
    I, H = w_gate.shape
    assert w_up.shape == (I, H) and w_down.shape == (H, I)
    x = np.ascontiguousarray(x)
    T = x.shape[0]
    assert x.shape == (T, H)
    y = np.zeros((T, H), dtype=np.float64)
    if x.dtype == np.uint16:
        _load().oracle_ffn_dense(_p(x, _u16p), _p(w_gate, _u16p), _p(w_up, _u16p), _p(w_down, _u16p),
                                 T, H, I, _p(y, _f64p))
    else:
        x = np.ascontiguousarray(x, dtype=np.float64)
        _load().oracle_ffn_dense_f64x(_p(x, _f64p), _p(w_gate, _u16p), _p(w_up, _u16p), _p(w_down, _u16p),
                                      T, H, I, _p(y, _f64p))
    return y


def moe_route(logits, top_k: int):
    """logits f32 [T,E] -> (idx i32 [T,K], gate f64 [T,K])."""
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    T, E = logits.shape
    idx = np.zeros((T, top_k), dtype=np.int32)
    gate = np.zeros((T, top_k), dtype=np.float64)
    _load().oracle_moe_route(_p(logits, _f32p), T, E, top_k, _p(idx, _i32p), _p(gate, _f64p))
    return idx, gate


def moe_permute(idx, num_experts: int):
    """idx i32 [T,K] -> (counts i32 [E], offsets i32 [E+1], pos i32 [T,K])."""
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    T, K = idx.shape
    counts = np.zeros(num_experts, dtype=np.int32)
    offsets = np.zeros(num_experts + 1, dtype=np.int32)
    pos = np.zeros((T, K), dtype=np.int32)
    _load().oracle_moe_permute(_p(idx, _i32p), T, num_experts, K, _p(counts, _i32p), _p(offsets, _i32p),
                               _p(pos, _i32p))
    return counts, offsets, pos


def ffn_moe(x, logits, w_gate, w_up, w_down, top_k: int):
    """x u16 or f64 [T,H]; logits f32 [T,E]; w_gate,w_up u16 [E,I,H]; w_down u16 [E,H,I]
    -> (y f64 [T,H], idx i32 [T,K], gate f64 [T,K])."""
    w_gate, w_up, w_down = _u16(w_gate), _u16(w_up), _u16(w_down)
    E, I, H = w_gate.shape
    assert w_up.shape == (E, I, H) and w_down.shape == (E, H, I)
    logits = np.ascontiguousarray(logits, dtype=np.float32)
    x = np.ascontiguousarray(x)
    T = x.shape[0]
    assert x.shape == (T, H) and logits.shape == (T, E)
    y = np.zeros((T, H), dtype=np.float64)
    idx = np.zeros((T, top_k), dtype=np.int32)
    gate = np.zeros((T, top_k), dtype=np.float64)
    if x.dtype == np.uint16:
        _load().oracle_ffn_moe(_p(x, _u16p), _p(logits, _f32p), _p(w_gate, _u16p), _p(w_up, _u16p),
                               _p(w_down, _u16p), T, H, I, E, top_k, _p(y, _f64p), _p(idx, _i32p),
                               _p(gate, _f64p))
    else:
        x = np.ascontiguousarray(x, dtype=np.float64)
        _load().oracle_ffn_moe_f64x(_p(x, _f64p), _p(logits, _f32p), _p(w_gate, _u16p), _p(w_up, _u16p),
                                    _p(w_down, _u16p), T, H, I, E, top_k, _p(y, _f64p), _p(idx, _i32p),
                                    _p(gate, _f64p))
    return y, idx, gate


def router_logits(x, w_router) -> np.ndarray:
    """x f64 [T,H], w_router u16 [E,H] -> f64 [T,E]."""
    return linear(x, w_router)


def layer_step(q, k_cache, v_cache, page_table, seq_lens, w_o, w_gate, w_up, w_down,
               logits=None, top_k: int = 0, scale: Optional[float] = None):
    """One decoder-layer decode step (attention -> W_o -> FFN) in fp64.
    Returns (attn_out f64 [B,Hq,D], y f64 [B,H])."""
    q, k_cache, v_cache = _u16(q), _u16(k_cache), _u16(v_cache)
    page_table = np.ascontiguousarray(page_table, dtype=np.int32)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    w_gate, w_up, w_down = _u16(w_gate), _u16(w_up), _u16(w_down)
    B, Hq, D = q.shape
    _, Hkv, P, _ = k_cache.shape
    if w_gate.ndim == 3:
        E, I, H = w_gate.shape
        assert logits is not None and top_k >= 1
        logits = np.ascontiguousarray(logits, dtype=np.float32)
        assert logits.shape == (B, E)
    else:
        E = 0
        I, H = w_gate.shape
    if w_o is not None:
        w_o = _u16(w_o)
        assert w_o.shape == (H, Hq * D)
    else:
        assert Hq * D == H
    if scale is None:
        scale = 1.0 / np.sqrt(float(D))
    a = np.zeros((B, Hq, D), dtype=np.float64)
    y = np.zeros((B, H), dtype=np.float64)
    _load().oracle_layer_step(_p(q, _u16p), _p(k_cache, _u16p), _p(v_cache, _u16p),
                              _p(page_table, _i32p), int(page_table.shape[1]), _p(seq_lens, _i32p),
                              B, Hq, Hkv, D, P, ctypes.c_double(scale),
                              _p(w_o, _u16p), H, I, E, int(top_k),
                              _p(w_gate, _u16p), _p(w_up, _u16p), _p(w_down, _u16p),
                              _p(logits, _f32p) if E else None, _p(a, _f64p), _p(y, _f64p))
    return a, y


# --------------------------------------------------------------------------- whole decoder layer
def f64_to_bf16(values) -> np.ndarray:
    """f64 array -> bf16 bit patterns (u16), round to nearest even in one rounding."""
    values = np.ascontiguousarray(values, dtype=np.float64)
    lib = _load()
    lib.oracle_f64_to_bf16.restype = ctypes.c_uint16
    lib.oracle_f64_to_bf16.argtypes = [ctypes.c_double]
    out = np.zeros(values.shape, dtype=np.uint16)
    flat_in, flat_out = values.reshape(-1), out.reshape(-1)
    for i in range(flat_in.size):
        flat_out[i] = lib.oracle_f64_to_bf16(float(flat_in[i]))
    return out


def rmsnorm(x, w, eps: float) -> np.ndarray:
    """x f64 [T,H]; w u16 [H] or None (ones) -> f64 [T,H]."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    T, H = x.shape
    if w is not None:
        w = _u16(w)
        assert w.shape == (H,)
    y = np.zeros((T, H), dtype=np.float64)
    _load().oracle_rmsnorm(_p(x, _f64p), _p(w, _u16p), T, H, ctypes.c_double(eps), _p(y, _f64p))
    return y


def rope(v, pos: float, theta: float) -> np.ndarray:
    """One head vector f64 [D] rotated to position pos (rotate-half convention)."""
    v = np.ascontiguousarray(v, dtype=np.float64)
    (D,) = v.shape
    assert D % 2 == 0
    out = np.zeros(D, dtype=np.float64)
    _load().oracle_rope(_p(v, _f64p), D, ctypes.c_double(pos), ctypes.c_double(theta), _p(out, _f64p))
    return out


def attn_decode_f64q(q, k_cache, v_cache, page_table, seq_lens, scale: Optional[float] = None):
    """As attn_decode with the queries in f64 [B,Hq,D]."""
    q = np.ascontiguousarray(q, dtype=np.float64)
    k_cache, v_cache = _u16(k_cache), _u16(v_cache)
    page_table = np.ascontiguousarray(page_table, dtype=np.int32)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    B, Hq, D = q.shape
    _, Hkv, P, _ = k_cache.shape
    if scale is None:
        scale = 1.0 / np.sqrt(float(D))
    out = np.zeros((B, Hq, D), dtype=np.float64)
    lse = np.zeros((B, Hq), dtype=np.float64)
    _load().oracle_attn_decode_f64q(_p(q, _f64p), _p(k_cache, _u16p), _p(v_cache, _u16p),
                                    _p(page_table, _i32p), int(page_table.shape[1]), _p(seq_lens, _i32p),
                                    B, Hq, Hkv, D, P, ctypes.c_double(scale), _p(out, _f64p), _p(lse, _f64p))
    return out, lse


def qkv_rope_append(x, w_ln, w_qkv, w_qn, w_kn, eps: float, theta: float, k_cache, v_cache, page_table,
                    seq_lens, num_q_heads: int) -> np.ndarray:
    """Attention-group operators in front of the attention itself.  x f64 [B,H]; w_ln u16 [H];
    w_qkv u16 [(Hq+2Hkv)*D, H]; w_qn, w_kn u16 [D] or None.  Updates k_cache / v_cache (u16
    [num_pages,Hkv,P,D]) IN PLACE at position seq_lens[b]-1 and returns q f64 [B,Hq,D]."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    B, H = x.shape
    assert k_cache.dtype == np.uint16 and k_cache.flags["C_CONTIGUOUS"] and k_cache.flags["WRITEABLE"]
    assert v_cache.dtype == np.uint16 and v_cache.flags["C_CONTIGUOUS"] and v_cache.flags["WRITEABLE"]
    _, Hkv, P, D = k_cache.shape
    Hq = int(num_q_heads)
    w_ln, w_qkv = _u16(w_ln), _u16(w_qkv)
    assert w_qkv.shape == ((Hq + 2 * Hkv) * D, H) and w_ln.shape == (H,)
    w_qn = None if w_qn is None else _u16(w_qn)
    w_kn = None if w_kn is None else _u16(w_kn)
    page_table = np.ascontiguousarray(page_table, dtype=np.int32)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    q = np.zeros((B, Hq, D), dtype=np.float64)
    _load().oracle_qkv_rope_append(_p(x, _f64p), _p(w_ln, _u16p), _p(w_qkv, _u16p), _p(w_qn, _u16p),
                                   _p(w_kn, _u16p), ctypes.c_double(eps), ctypes.c_double(theta),
                                   _p(k_cache, _u16p), _p(v_cache, _u16p), _p(page_table, _i32p),
                                   int(page_table.shape[1]), _p(seq_lens, _i32p), B, H, Hq, Hkv, D, P,
                                   _p(q, _f64p))
    return q


def decoder_layer(x, w, k_cache, v_cache, page_table, seq_lens, num_q_heads: int, eps: float, theta: float,
                  top_k: int = 0, logits=None, scale: Optional[float] = None):
    """One whole pre-norm decoder layer (decode step) in fp64.

    x f64 [B,H] (the residual stream); ``w`` is a dict of u16 arrays: ln_attn [H], qkv
    [(Hq+2Hkv)*D,H], q_norm / k_norm [D] or None, o [H,Hq*D], ln_ffn [H], gate / up ([I,H] dense,
    [E,I,H] MoE), down ([H,I] / [E,H,I]), router [E,H] or None (then ``logits`` f32 [B,E] is used).
    The caches are updated IN PLACE.  Returns (q f64 [B,Hq,D], h1 f64 [B,H], out f64 [B,H])."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    B, H = x.shape
    assert k_cache.dtype == np.uint16 and k_cache.flags["C_CONTIGUOUS"] and k_cache.flags["WRITEABLE"]
    assert v_cache.dtype == np.uint16 and v_cache.flags["C_CONTIGUOUS"] and v_cache.flags["WRITEABLE"]
    _, Hkv, P, D = k_cache.shape
    Hq = int(num_q_heads)
    page_table = np.ascontiguousarray(page_table, dtype=np.int32)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    g = {k: (None if v is None else _u16(v)) for k, v in w.items()}
    assert g["qkv"].shape == ((Hq + 2 * Hkv) * D, H) and g["o"].shape == (H, Hq * D)
    if g["gate"].ndim == 3:
        E, I, _ = g["gate"].shape
        assert top_k >= 1
        if g.get("router") is None:
            logits = np.ascontiguousarray(logits, dtype=np.float32)
            assert logits.shape == (B, E)
    else:
        E = 0
        I = g["gate"].shape[0]
    if scale is None:
        scale = 1.0 / np.sqrt(float(D))
    q = np.zeros((B, Hq, D), dtype=np.float64)
    h1 = np.zeros((B, H), dtype=np.float64)
    out = np.zeros((B, H), dtype=np.float64)
    _load().oracle_decoder_layer(_p(x, _f64p), _p(g["ln_attn"], _u16p), _p(g["qkv"], _u16p),
                                 _p(g.get("q_norm"), _u16p), _p(g.get("k_norm"), _u16p),
                                 ctypes.c_double(eps), ctypes.c_double(theta),
                                 _p(k_cache, _u16p), _p(v_cache, _u16p), _p(page_table, _i32p),
                                 int(page_table.shape[1]), _p(seq_lens, _i32p), B, H, Hq, Hkv, D, P,
                                 ctypes.c_double(scale), _p(g["o"], _u16p), _p(g["ln_ffn"], _u16p),
                                 I, E, int(top_k), _p(g["gate"], _u16p), _p(g["up"], _u16p), _p(g["down"], _u16p),
                                 _p(g.get("router"), _u16p) if E else None,
                                 _p(logits, _f32p) if (E and g.get("router") is None) else None,
                                 _p(q, _f64p), _p(h1, _f64p), _p(out, _f64p))
    return q, h1, out


def prefill_layer(x, w, k_cache, v_cache, page_table, seq_lens, q_offsets, num_q_heads: int, eps: float, theta: float,
                  top_k: int = 0, logits=None, scale: Optional[float] = None):
    """One whole pre-norm decoder layer over the tokens being prefilled, in fp64.

    x f64 [T,H] (T = q_offsets[-1]): row q_offsets[b] + i is token i of the last q_offsets[b+1] - q_offsets[b]
    tokens of sequence b (seq_lens counts them already).  ``w`` as for decoder_layer; ``logits`` f32 [T,E].
    The caches are updated IN PLACE.  Returns (q f64 [T,Hq,D], h1 f64 [T,H], out f64 [T,H])."""
    x = np.ascontiguousarray(x, dtype=np.float64)
    T, H = x.shape
    assert k_cache.dtype == np.uint16 and k_cache.flags["C_CONTIGUOUS"] and k_cache.flags["WRITEABLE"]
    assert v_cache.dtype == np.uint16 and v_cache.flags["C_CONTIGUOUS"] and v_cache.flags["WRITEABLE"]
    _, Hkv, P, D = k_cache.shape
    Hq = int(num_q_heads)
    page_table = np.ascontiguousarray(page_table, dtype=np.int32)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    q_offsets = np.ascontiguousarray(q_offsets, dtype=np.int32)
    B = seq_lens.shape[0]
    assert q_offsets.shape == (B + 1,) and q_offsets[0] == 0 and q_offsets[-1] == T
    m = q_offsets[1:] - q_offsets[:-1]
    assert (m >= 0).all() and (m <= seq_lens).all()
    g = {k: (None if v is None else _u16(v)) for k, v in w.items()}
    assert g["qkv"].shape == ((Hq + 2 * Hkv) * D, H) and g["o"].shape == (H, Hq * D)
    if g["gate"].ndim == 3:
        E, I, _ = g["gate"].shape
        assert top_k >= 1
        if g.get("router") is None:
            logits = np.ascontiguousarray(logits, dtype=np.float32)
            assert logits.shape == (T, E)
    else:
        E = 0
        I = g["gate"].shape[0]
    if scale is None:
        scale = 1.0 / np.sqrt(float(D))
    q = np.zeros((T, Hq, D), dtype=np.float64)
    h1 = np.zeros((T, H), dtype=np.float64)
    out = np.zeros((T, H), dtype=np.float64)
    _load().oracle_prefill_layer(_p(x, _f64p), _p(g["ln_attn"], _u16p), _p(g["qkv"], _u16p),
                                 _p(g.get("q_norm"), _u16p), _p(g.get("k_norm"), _u16p),
                                 ctypes.c_double(eps), ctypes.c_double(theta),
                                 _p(k_cache, _u16p), _p(v_cache, _u16p), _p(page_table, _i32p),
                                 int(page_table.shape[1]), _p(seq_lens, _i32p), _p(q_offsets, _i32p), B, H, Hq, Hkv, D, P,
                                 ctypes.c_double(scale), _p(g["o"], _u16p), _p(g["ln_ffn"], _u16p),
                                 I, E, int(top_k), _p(g["gate"], _u16p), _p(g["up"], _u16p), _p(g["down"], _u16p),
                                 _p(g.get("router"), _u16p) if E else None,
                                 _p(logits, _f32p) if (E and g.get("router") is None) else None,
                                 _p(q, _f64p), _p(h1, _f64p), _p(out, _f64p))
    return q, h1, out


def attn_prefill(q, k_cache, v_cache, page_table, seq_lens, q_offsets, scale: Optional[float] = None) -> np.ndarray:
    """Causal attention of the last q_len tokens of every sequence over its paged cache.
    q u16 [T,Hq,D] (T = q_offsets[-1]); seq_lens i32 [B] (cached tokens incl. the prefilled ones);
    q_offsets i32 [B+1] -> out f64 [T,Hq,D]."""
    q, k_cache, v_cache = _u16(q), _u16(k_cache), _u16(v_cache)
    page_table = np.ascontiguousarray(page_table, dtype=np.int32)
    seq_lens = np.ascontiguousarray(seq_lens, dtype=np.int32)
    q_offsets = np.ascontiguousarray(q_offsets, dtype=np.int32)
    T, Hq, D = q.shape
    _, Hkv, P, _ = k_cache.shape
    B = seq_lens.shape[0]
    assert q_offsets.shape == (B + 1,) and q_offsets[0] == 0 and q_offsets[-1] == T
    assert ((q_offsets[1:] - q_offsets[:-1]) <= seq_lens).all() and ((q_offsets[1:] - q_offsets[:-1]) >= 0).all()
    if scale is None:
        scale = 1.0 / np.sqrt(float(D))
    out = np.zeros((T, Hq, D), dtype=np.float64)
    _load().oracle_attn_prefill(_p(q, _u16p), _p(k_cache, _u16p), _p(v_cache, _u16p), _p(page_table, _i32p),
                                int(page_table.shape[1]), _p(seq_lens, _i32p), _p(q_offsets, _i32p), B, Hq, Hkv, D, P,
                                ctypes.c_double(scale), _p(out, _f64p))
    return out
