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
