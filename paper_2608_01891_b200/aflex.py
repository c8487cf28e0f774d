"""Thin ctypes binding over the C-ABI CUDA library (``include/aflex.h``).

Argument marshalling only: every step of the hot path runs inside libaflex's
kernels.  PyTorch tensors are used as device-memory handles (``data_ptr()``) and
for the current stream.  There is no CPU fallback: if the library cannot be
loaded, or a call returns a non-OK status, an exception is raised.
"""
from __future__ import annotations

import ctypes
import os
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libaflex.so")

OK, ERR_INVALID_ARG, ERR_UNSUPPORTED, ERR_WORKSPACE, ERR_CUDA, ERR_TIMEOUT, ERR_BOUNDS = range(7)

# Every symbol include/aflex.h declares.
EXPORTS = (
    "aflex_status_string", "aflex_version", "aflex_create", "aflex_destroy", "aflex_last_error",
    "aflex_get_device_status", "aflex_attn_decode", "aflex_ffn_dense", "aflex_ffn_moe", "aflex_moe_route", "aflex_layer_step",
    "aflex_workspace_bytes", "aflex_linear", "aflex_set_attn_ctas", "aflex_set_attn_q_final", "aflex_set_interleave_streams", "aflex_num_kernel_kinds",
    "aflex_kernel_name", "aflex_launch_count", "aflex_profile_enable", "aflex_profile_read",
    "aflex_trace_read", "aflex_attn_decode_static", "aflex_attn_decode_static_status", "aflex_decoder_layers", "aflex_decoder_workspace_bytes",
    "aflex_add_rmsnorm", "aflex_rope_append", "aflex_attn_prefill", "aflex_af_decoder_layers", "aflex_af_workspace_bytes",
    "aflex_prefill_layers", "aflex_prefill_workspace_bytes",
    "aflex_eq2_layer_time", "aflex_curve_eval",
    "aflex_pipeline_makespan", "aflex_plan_microbatches", "aflex_dvfs_window", "aflex_dvfs_decode_step",
    "aflex_dvfs_prefill_pair",
)


class AttnDesc(ctypes.Structure):
    _fields_ = [("num_q_heads", ctypes.c_int), ("num_kv_heads", ctypes.c_int), ("head_dim", ctypes.c_int),
                ("page_size", ctypes.c_int), ("sm_scale", ctypes.c_float)]


class KV(ctypes.Structure):
    _fields_ = [("k_cache", ctypes.c_void_p), ("v_cache", ctypes.c_void_p), ("num_pages", ctypes.c_int64),
                ("page_table", ctypes.c_void_p), ("max_pages_per_seq", ctypes.c_int),
                ("seq_lens", ctypes.c_void_p), ("seq_lens_host", ctypes.c_void_p)]


class LayerDesc(ctypes.Structure):
    _fields_ = [("attn", AttnDesc), ("hidden", ctypes.c_int), ("inter", ctypes.c_int),
                ("num_experts", ctypes.c_int), ("top_k", ctypes.c_int), ("w_o", ctypes.c_void_p),
                ("w_gate", ctypes.c_void_p), ("w_up", ctypes.c_void_p), ("w_down", ctypes.c_void_p),
                ("w_router", ctypes.c_void_p)]


class DecoderDesc(ctypes.Structure):
    _fields_ = [("layer", LayerDesc), ("w_qkv", ctypes.c_void_p), ("w_ln_attn", ctypes.c_void_p),
                ("w_ln_ffn", ctypes.c_void_p), ("w_q_norm", ctypes.c_void_p), ("w_k_norm", ctypes.c_void_p),
                ("rms_eps", ctypes.c_float), ("rope_theta", ctypes.c_float)]


class Curve(ctypes.Structure):
    _fields_ = [("n", ctypes.c_int), ("x", ctypes.POINTER(ctypes.c_double)), ("y", ctypes.POINTER(ctypes.c_double))]


class PipelineModel(ctypes.Structure):
    _fields_ = [("attn_vs_tokens", Curve), ("attn_vs_rows", Curve), ("ffn_vs_rows", Curve),
                ("comm_fixed", ctypes.c_double), ("comm_per_row", ctypes.c_double),
                ("shared_memory_system", ctypes.c_int)]


class DvfsParams(ctypes.Structure):
    _fields_ = [("n_da", ctypes.c_int), ("n_df", ctypes.c_int), ("tau", ctypes.c_double),
                ("delta_b", ctypes.c_double), ("window", ctypes.c_int), ("t_switch", ctypes.c_double)]


class DvfsState(ctypes.Structure):
    _fields_ = [("i_da", ctypes.c_int), ("i_df", ctypes.c_int), ("w", ctypes.c_int), ("b_last", ctypes.c_int)]


DVFS_ESCALATED, DVFS_INFEASIBLE = 1, 2


class AflexError(RuntimeError):
    def __init__(self, status: int, name: str, detail: str):
        super().__init__(f"{name} ({status}): {detail}")
        self.status = status


_lib = None


def load_library() -> ctypes.CDLL:
    """dlopen libaflex.so (built in-tree by ``build.py``).  Raises if missing."""
    global _lib
    if _lib is not None:
        return _lib
    if not os.path.exists(LIB_PATH):
        raise RuntimeError(f"{LIB_PATH} not found: build it with `python -m paper_2608_01891_b200.build` "
                           "(there is no fallback path)")
    lib = ctypes.CDLL(LIB_PATH)
    vp, ci, cs = ctypes.c_void_p, ctypes.c_int, ctypes.c_size_t
    lib.aflex_status_string.restype = ctypes.c_char_p
    lib.aflex_status_string.argtypes = [ci]
    lib.aflex_version.restype = ci
    lib.aflex_create.restype = ci
    lib.aflex_create.argtypes = [ctypes.POINTER(vp), ci, cs]
    lib.aflex_destroy.restype = ci
    lib.aflex_destroy.argtypes = [vp]
    lib.aflex_last_error.restype = ctypes.c_char_p
    lib.aflex_last_error.argtypes = [vp]
    lib.aflex_get_device_status.restype = ci
    lib.aflex_get_device_status.argtypes = [vp, vp]
    lib.aflex_set_attn_ctas.restype = ci
    lib.aflex_set_attn_ctas.argtypes = [vp, ci]
    lib.aflex_set_attn_q_final.restype = ci
    lib.aflex_set_attn_q_final.argtypes = [vp, ci]
    lib.aflex_set_interleave_streams.restype = ci
    lib.aflex_set_interleave_streams.argtypes = [vp, ci]
    lib.aflex_attn_decode.restype = ci
    lib.aflex_attn_decode.argtypes = [vp, ctypes.POINTER(AttnDesc), vp, ctypes.POINTER(KV), ci, vp, vp, vp]
    lib.aflex_attn_prefill.restype = ci
    lib.aflex_attn_prefill.argtypes = [vp, ctypes.POINTER(AttnDesc), vp, ctypes.POINTER(KV), ci, vp, vp, vp, vp]
    lib.aflex_linear.restype = ci
    lib.aflex_linear.argtypes = [vp, vp, vp, ci, ci, ci, vp, vp]
    lib.aflex_ffn_dense.restype = ci
    lib.aflex_ffn_dense.argtypes = [vp, vp, vp, vp, vp, ci, ci, ci, vp, vp]
    lib.aflex_ffn_moe.restype = ci
    lib.aflex_ffn_moe.argtypes = [vp, vp, vp, vp, vp, vp, vp, ci, ci, ci, ci, ci, vp, vp, vp, vp, vp]
    lib.aflex_moe_route.restype = ci
    lib.aflex_moe_route.argtypes = [vp, vp, ci, ci, ci, vp, vp, vp, vp, vp, vp]
    lib.aflex_layer_step.restype = ci
    lib.aflex_layer_step.argtypes = [vp, ctypes.POINTER(LayerDesc), vp, ctypes.POINTER(KV), ci, vp, ci,
                                     ctypes.POINTER(ctypes.c_int32), vp, vp, vp]
    lib.aflex_workspace_bytes.restype = cs
    lib.aflex_workspace_bytes.argtypes = [ctypes.POINTER(LayerDesc), ci, ci]
    lib.aflex_num_kernel_kinds.restype = ci
    lib.aflex_kernel_name.restype = ctypes.c_char_p
    lib.aflex_kernel_name.argtypes = [ci]
    lib.aflex_launch_count.restype = ctypes.c_longlong
    lib.aflex_launch_count.argtypes = [vp, ci]
    lib.aflex_profile_enable.restype = ci
    lib.aflex_profile_enable.argtypes = [vp, ci]
    lib.aflex_profile_read.restype = ci
    lib.aflex_profile_read.argtypes = [vp, ci, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_longlong)]
    lib.aflex_decoder_layers.restype = ci
    lib.aflex_decoder_layers.argtypes = [vp, ctypes.POINTER(DecoderDesc), ctypes.POINTER(KV), ci, vp, ci, ci,
                                         ctypes.POINTER(ctypes.c_int32), vp, vp]
    lib.aflex_decoder_workspace_bytes.restype = cs
    lib.aflex_decoder_workspace_bytes.argtypes = [ctypes.POINTER(DecoderDesc), ci]
    lib.aflex_prefill_layers.restype = ci
    lib.aflex_prefill_layers.argtypes = [vp, ctypes.POINTER(DecoderDesc), ctypes.POINTER(KV), ci, vp, ci, vp, vp, vp, vp]
    lib.aflex_prefill_workspace_bytes.restype = cs
    lib.aflex_prefill_workspace_bytes.argtypes = [ctypes.POINTER(DecoderDesc), ci]
    lib.aflex_af_decoder_layers.restype = ci
    lib.aflex_af_decoder_layers.argtypes = [vp, vp, ctypes.POINTER(DecoderDesc), ctypes.POINTER(KV), ci, vp, ci, ci,
                                            ctypes.POINTER(ctypes.c_int32), vp, vp]
    lib.aflex_af_workspace_bytes.restype = cs
    lib.aflex_af_workspace_bytes.argtypes = [ctypes.POINTER(DecoderDesc), ci, ci]
    lib.aflex_add_rmsnorm.restype = ci
    lib.aflex_add_rmsnorm.argtypes = [vp, vp, vp, vp, ci, ci, ctypes.c_float, vp, vp, vp]
    lib.aflex_rope_append.restype = ci
    lib.aflex_rope_append.argtypes = [vp, ctypes.POINTER(AttnDesc), vp, ctypes.POINTER(KV), ci, vp, vp,
                                      ctypes.c_float, ctypes.c_float, vp, vp]
    cd, dp, ip = ctypes.c_double, ctypes.POINTER(ctypes.c_double), ctypes.POINTER(ctypes.c_int32)
    lib.aflex_eq2_layer_time.restype = cd
    lib.aflex_eq2_layer_time.argtypes = [cd, cd, cd, ci]
    lib.aflex_curve_eval.restype = cd
    lib.aflex_curve_eval.argtypes = [ctypes.POINTER(Curve), cd]
    lib.aflex_pipeline_makespan.restype = cd
    lib.aflex_pipeline_makespan.argtypes = [ctypes.POINTER(PipelineModel), ip, ci, ci, ip, ci]
    lib.aflex_plan_microbatches.restype = ci
    lib.aflex_plan_microbatches.argtypes = [ctypes.POINTER(PipelineModel), ip, ci, ci, ctypes.POINTER(ci), ci, ci,
                                            ctypes.POINTER(ci), ip, dp]
    lib.aflex_dvfs_window.restype = ci
    lib.aflex_dvfs_window.argtypes = [ci, cd, cd, cd]
    lib.aflex_dvfs_decode_step.restype = ci
    lib.aflex_dvfs_decode_step.argtypes = [ctypes.POINTER(DvfsParams), dp, dp, ci, cd, ctypes.POINTER(DvfsState)]
    lib.aflex_dvfs_prefill_pair.restype = ci
    lib.aflex_dvfs_prefill_pair.argtypes = [ci, ci, dp, dp, cd, cd, ci, ci, ci, ci, ctypes.POINTER(ci),
                                            ctypes.POINTER(ci)]
    lib.aflex_attn_decode_static.restype = ci
    lib.aflex_attn_decode_static.argtypes = [ctypes.POINTER(AttnDesc), vp, ctypes.POINTER(KV), ci, vp, vp, vp]
    lib.aflex_attn_decode_static_status.restype = ci
    lib.aflex_attn_decode_static_status.argtypes = [ctypes.POINTER(ci), vp]
    _lib = lib
    return lib


def _ptr(t: Optional[torch.Tensor]) -> Optional[int]:
    if t is None:
        return None
    assert t.is_contiguous(), "tensors passed to aflex must be contiguous"
    return t.data_ptr()


def _stream(stream: Optional[torch.cuda.Stream]) -> int:
    return (stream or torch.cuda.current_stream()).cuda_stream


def attn_desc(num_q_heads: int, num_kv_heads: int, head_dim: int, sm_scale: float = 0.0) -> AttnDesc:
    return AttnDesc(num_q_heads, num_kv_heads, head_dim, 16, sm_scale)


def make_kv(k_cache: torch.Tensor, v_cache: torch.Tensor, page_table: torch.Tensor, seq_lens: torch.Tensor,
            seq_lens_host: Optional[torch.Tensor] = None) -> KV:
    """k_cache/v_cache bf16 CUDA [num_pages,Hkv,16,D]; page_table i32 CUDA [B,max_pages]; seq_lens i32 CUDA [B];
    seq_lens_host optional i32 CPU [B].  The returned struct borrows the tensors: keep them alive."""
    assert k_cache.dtype == torch.bfloat16 and v_cache.dtype == torch.bfloat16
    assert page_table.dtype == torch.int32 and seq_lens.dtype == torch.int32
    kv = KV(_ptr(k_cache), _ptr(v_cache), k_cache.shape[0], _ptr(page_table), page_table.shape[1],
            _ptr(seq_lens), None)
    if seq_lens_host is not None:
        assert seq_lens_host.dtype == torch.int32 and seq_lens_host.device.type == "cpu"
        kv.seq_lens_host = _ptr(seq_lens_host)
    kv._keep = (k_cache, v_cache, page_table, seq_lens, seq_lens_host)
    return kv


def layer_desc(attn: AttnDesc, hidden: int, inter: int, w_o, w_gate, w_up, w_down, num_experts: int = 0,
               top_k: int = 0, w_router=None) -> LayerDesc:
    d = LayerDesc(attn, hidden, inter, num_experts, top_k, _ptr(w_o), _ptr(w_gate), _ptr(w_up), _ptr(w_down),
                  _ptr(w_router))
    d._keep = (w_o, w_gate, w_up, w_down, w_router)
    return d


def decoder_desc(layer: LayerDesc, w_qkv, w_ln_attn, w_ln_ffn, w_q_norm, w_k_norm, rms_eps: float,
                 rope_theta: float) -> DecoderDesc:
    d = DecoderDesc(layer, _ptr(w_qkv), _ptr(w_ln_attn), _ptr(w_ln_ffn), _ptr(w_q_norm), _ptr(w_k_norm),
                    rms_eps, rope_theta)
    d._keep = (layer, w_qkv, w_ln_attn, w_ln_ffn, w_q_norm, w_k_norm)
    return d


def decoder_workspace_bytes(layer: DecoderDesc, max_batch: int) -> int:
    return int(load_library().aflex_decoder_workspace_bytes(ctypes.byref(layer), max_batch))


def prefill_workspace_bytes(layer: DecoderDesc, max_tokens: int) -> int:
    return int(load_library().aflex_prefill_workspace_bytes(ctypes.byref(layer), max_tokens))


def af_workspace_bytes(layer: DecoderDesc, max_batch: int, ffn_side: bool) -> int:
    return int(load_library().aflex_af_workspace_bytes(ctypes.byref(layer), max_batch, 1 if ffn_side else 0))


def af_decoder_layers(ctx_a: "Context", ctx_f: "Context", layers: Sequence[DecoderDesc], kvs: Sequence[KV], x_in, x_out,
                      microbatch_depth: int = 1, mb_offsets: Optional[Sequence[int]] = None, stream=None) -> None:
    """Chained decoder layers with the Attention side on ctx_a's GPU and the FFN side on ctx_f's (see the header
    for which weights live where).  `stream` is a stream of ctx_a's device (default: its current stream)."""
    assert len(layers) == len(kvs) and len(layers) >= 1
    offs = None
    if mb_offsets is not None:
        offs = (ctypes.c_int32 * len(mb_offsets))(*[int(v) for v in mb_offsets])
    la = (DecoderDesc * len(layers))(*layers)
    ka = (KV * len(kvs))(*kvs)
    st = stream.cuda_stream if stream is not None else torch.cuda.current_stream(x_in.device).cuda_stream
    ctx_a._check(ctx_a._lib.aflex_af_decoder_layers(ctx_a._h, ctx_f._h, la, ka, len(layers), _ptr(x_in), x_in.shape[0],
                                                    microbatch_depth, offs, _ptr(x_out), st))


def workspace_bytes(layer: LayerDesc, max_batch: int, max_pages_per_seq: int) -> int:
    return int(load_library().aflex_workspace_bytes(ctypes.byref(layer), max_batch, max_pages_per_seq))


_STATIC_ERRORS = {
    ERR_INVALID_ARG: "null / misaligned pointer, batch < 1, or Hkv does not divide Hq",
    ERR_UNSUPPORTED: "outside the supported envelope (head_dim 64|128, page_size 16, Hq/Hkv in 1,2,4,8)",
    ERR_WORKSPACE: "batch * num_kv_heads exceeds the fixed scratch capacity (16384)",
    ERR_CUDA: "a CUDA call failed",
}


def attn_decode_static(desc: AttnDesc, q: torch.Tensor, kv: KV, out: torch.Tensor,
                       lse: Optional[torch.Tensor] = None, stream=None) -> None:
    """Decode attention through the allocation-free entry point: no Context, no workspace; the
    kernel's scratch is a fixed array inside the library.  For callers that cannot allocate device
    memory (a pool that owns the whole GPU, a host application's allocator rules, a path that must not
    synchronise).  Calls must not overlap on the GPU: they share that one scratch array."""
    lib = load_library()
    st = lib.aflex_attn_decode_static(ctypes.byref(desc), _ptr(q), ctypes.byref(kv), q.shape[0], _ptr(out), _ptr(lse),
                                      _stream(stream))
    if st != OK:
        raise AflexError(st, lib.aflex_status_string(st).decode(), _STATIC_ERRORS.get(st, "unknown error"))


def attn_decode_static_status(stream=None) -> int:
    """What the kernel of the last attn_decode_static call on this device recorded while it ran (OK,
    ERR_BOUNDS for a clamped length or a redirected page id, ERR_TIMEOUT); synchronises the stream."""
    lib = load_library()
    v = ctypes.c_int(-1)
    st = lib.aflex_attn_decode_static_status(ctypes.byref(v), _stream(stream))
    if st != OK:
        raise AflexError(st, lib.aflex_status_string(st).decode(), _STATIC_ERRORS.get(st, "unknown error"))
    return int(v.value)


# --------------------------------------------------------------------------- host-side decisions
def _dbl(values):
    return (ctypes.c_double * len(values))(*[float(v) for v in values])


def curve(xs, ys) -> Curve:
    assert len(xs) == len(ys) >= 1
    ax, ay = _dbl(xs), _dbl(ys)
    c = Curve(len(xs), ax, ay)
    c._keep = (ax, ay)
    return c


def pipeline_model(attn_vs_tokens, attn_vs_rows, ffn_vs_rows, comm_fixed=0.0, comm_per_row=0.0,
                   shared_memory_system=False) -> PipelineModel:
    """Each curve is an (xs, ys) pair of profiled points."""
    cs = [curve(*attn_vs_tokens), curve(*attn_vs_rows), curve(*ffn_vs_rows)]
    m = PipelineModel(cs[0], cs[1], cs[2], comm_fixed, comm_per_row, 1 if shared_memory_system else 0)
    m._keep = cs
    return m


def eq2_layer_time(t_a: float, t_f: float, t_comm: float, depth: int) -> float:
    return float(load_library().aflex_eq2_layer_time(t_a, t_f, t_comm, depth))


def curve_eval(c: Curve, x: float) -> float:
    return float(load_library().aflex_curve_eval(ctypes.byref(c), x))


def pipeline_makespan(model: PipelineModel, seq_lens, offsets, layers: int) -> float:
    lens = (ctypes.c_int32 * len(seq_lens))(*[int(v) for v in seq_lens])
    offs = (ctypes.c_int32 * len(offsets))(*[int(v) for v in offsets])
    return float(load_library().aflex_pipeline_makespan(ctypes.byref(model), lens, len(seq_lens), len(offsets) - 1,
                                                        offs, layers))


def plan_microbatches(model: PipelineModel, seq_lens, layers: int, depths, granularity: int = 1):
    """-> (depth, offsets, predicted time).  Raises AflexError on a non-OK status."""
    lib = load_library()
    lens = (ctypes.c_int32 * len(seq_lens))(*[int(v) for v in seq_lens])
    ds = (ctypes.c_int * len(depths))(*[int(v) for v in depths])
    best = ctypes.c_int(0)
    offs = (ctypes.c_int32 * (max(depths) + 1))()
    pred = ctypes.c_double(0.0)
    st = lib.aflex_plan_microbatches(ctypes.byref(model), lens, len(seq_lens), layers, ds, len(depths), granularity,
                                     ctypes.byref(best), offs, ctypes.byref(pred))
    if st != OK:
        raise AflexError(st, lib.aflex_status_string(st).decode(), "aflex_plan_microbatches")
    return best.value, list(offs[:best.value + 1]), pred.value


def dvfs_window(w_min: int, kappa: float, t_switch: float, t_iter: float) -> int:
    return int(load_library().aflex_dvfs_window(w_min, kappa, t_switch, t_iter))


def dvfs_decode_step(params: DvfsParams, t_hat, e_hat, batch_now: int, t_iter: float, state: DvfsState) -> int:
    """t_hat / e_hat: nested [n_da][n_df] lists.  Updates `state` in place; returns the library's code."""
    flat_t = _dbl([v for row in t_hat for v in row])
    flat_e = _dbl([v for row in e_hat for v in row])
    return int(load_library().aflex_dvfs_decode_step(ctypes.byref(params), flat_t, flat_e, batch_now, t_iter,
                                                     ctypes.byref(state)))


def dvfs_prefill_pair(t_hat, e_hat, budget: float, t_switch: float, current, base):
    """-> ((pa, pf), flags)."""
    flat_t = _dbl([v for row in t_hat for v in row])
    flat_e = _dbl([v for row in e_hat for v in row])
    pa, pf = ctypes.c_int(0), ctypes.c_int(0)
    flags = load_library().aflex_dvfs_prefill_pair(len(t_hat), len(t_hat[0]), flat_t, flat_e, budget, t_switch,
                                                   current[0], current[1], base[0], base[1], ctypes.byref(pa),
                                                   ctypes.byref(pf))
    return (pa.value, pf.value), int(flags)


class Context:
    """Owns an aflex_ctx (device workspace, internal streams/events, status word)."""

    def __init__(self, device: int = 0, workspace_bytes: int = 0):
        self._lib = load_library()
        self._h = ctypes.c_void_p()
        st = self._lib.aflex_create(ctypes.byref(self._h), device, workspace_bytes)
        if st != OK:
            raise AflexError(st, self._lib.aflex_status_string(st).decode(), "aflex_create failed")
        self.device = device

    def close(self) -> None:
        if getattr(self, "_h", None) and self._h.value:
            self._lib.aflex_destroy(self._h)
            self._h = ctypes.c_void_p()

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _check(self, st: int) -> None:
        if st != OK:
            raise AflexError(st, self._lib.aflex_status_string(st).decode(),
                             self._lib.aflex_last_error(self._h).decode())

    def raw_call(self, name: str, *args) -> int:
        """Call an entry point and return the raw status (for error-path tests)."""
        return int(getattr(self._lib, name)(self._h, *args))

    def last_error(self) -> str:
        return self._lib.aflex_last_error(self._h).decode()

    def device_status(self, stream=None) -> int:
        return int(self._lib.aflex_get_device_status(self._h, _stream(stream)))

    def launch_count(self, kind: int = -1) -> int:
        return int(self._lib.aflex_launch_count(self._h, kind))

    def profile_enable(self, on: bool) -> None:
        self._check(self._lib.aflex_profile_enable(self._h, 1 if on else 0))

    def profile_read(self) -> dict:
        """{kernel kind name: (total device ms, launches)} for the launches collected since enable."""
        out = {}
        for k in range(self._lib.aflex_num_kernel_kinds()):
            ms, n = ctypes.c_double(0.0), ctypes.c_longlong(0)
            self._check(self._lib.aflex_profile_read(self._h, k, ctypes.byref(ms), ctypes.byref(n)))
            if n.value:
                out[self._lib.aflex_kernel_name(k).decode()] = (ms.value, n.value)
        return out

    def trace_read(self, launches: int):
        """(records uint64 [launches, 4096, 8], launches recorded since the last read); needs AFLEX_TRACE=1."""
        import numpy as np
        buf = np.zeros((launches, 4096, 8), dtype=np.uint64)
        n = ctypes.c_int(0)
        self._lib.aflex_trace_read.restype = ctypes.c_int
        self._check(self._lib.aflex_trace_read(self._h, ctypes.c_void_p(buf.ctypes.data), launches, ctypes.byref(n)))
        return buf, n.value

    def set_attn_q_final(self, on: bool) -> None:
        """Promise that q is never produced by the library kernel enqueued directly before an attention call."""
        self._check(self._lib.aflex_set_attn_q_final(self._h, 1 if on else 0))

    def set_interleave_streams(self, on: bool) -> None:
        """layer_step with M >= 2: A side and F side on the ctx's two streams (True) or everything on the caller's stream."""
        self._check(self._lib.aflex_set_interleave_streams(self._h, 1 if on else 0))

    def set_attn_ctas(self, ctas: int) -> None:
        self._check(self._lib.aflex_set_attn_ctas(self._h, ctas))

    def attn_decode(self, desc: AttnDesc, q: torch.Tensor, kv: KV, out: torch.Tensor,
                    lse: Optional[torch.Tensor] = None, stream=None) -> None:
        self._check(self._lib.aflex_attn_decode(self._h, ctypes.byref(desc), _ptr(q), ctypes.byref(kv),
                                                q.shape[0], _ptr(out), _ptr(lse), _stream(stream)))

    def attn_prefill(self, desc: AttnDesc, q: torch.Tensor, kv: KV, q_offsets: torch.Tensor,
                     q_offsets_host: torch.Tensor, out: torch.Tensor, stream=None) -> None:
        """Causal attention of the last q_len tokens of every sequence over its paged cache.  q, out bf16
        [T,Hq,D]; q_offsets i32 CUDA [B+1]; q_offsets_host the same on the CPU."""
        assert q_offsets.dtype == torch.int32 and q_offsets_host.dtype == torch.int32 and q_offsets_host.device.type == "cpu"
        self._check(self._lib.aflex_attn_prefill(self._h, ctypes.byref(desc), _ptr(q), ctypes.byref(kv),
                                                 q_offsets_host.shape[0] - 1, _ptr(q_offsets), _ptr(q_offsets_host),
                                                 _ptr(out), _stream(stream)))

    def linear(self, x: torch.Tensor, w: torch.Tensor, y: torch.Tensor, stream=None) -> None:
        T, K = x.shape
        N = w.shape[0]
        self._check(self._lib.aflex_linear(self._h, _ptr(x), _ptr(w), T, K, N, _ptr(y), _stream(stream)))

    def ffn_dense(self, x, w_gate, w_up, w_down, y, stream=None) -> None:
        T, H = x.shape
        I = w_gate.shape[0]
        self._check(self._lib.aflex_ffn_dense(self._h, _ptr(x), _ptr(w_gate), _ptr(w_up), _ptr(w_down), T, H, I,
                                              _ptr(y), _stream(stream)))

    def ffn_moe(self, x, w_gate, w_up, w_down, top_k: int, y, router_logits=None, w_router=None,
                topk_idx=None, topk_gate=None, expert_counts=None, stream=None) -> None:
        T, H = x.shape
        E, I, _ = w_gate.shape
        self._check(self._lib.aflex_ffn_moe(self._h, _ptr(x), _ptr(router_logits), _ptr(w_router), _ptr(w_gate),
                                            _ptr(w_up), _ptr(w_down), T, H, I, E, top_k, _ptr(y), _ptr(topk_idx),
                                            _ptr(topk_gate), _ptr(expert_counts), _stream(stream)))

    def moe_route(self, router_logits, top_k: int, topk_idx, topk_gate, expert_counts, expert_offsets, pos,
                  stream=None) -> None:
        """Routing + permutation alone: idx/gate [T,K], counts [E], offsets [E+1], pos [T,K] (device tensors)."""
        T, E = router_logits.shape
        self._check(self._lib.aflex_moe_route(self._h, _ptr(router_logits), T, E, top_k, _ptr(topk_idx), _ptr(topk_gate),
                                              _ptr(expert_counts), _ptr(expert_offsets), _ptr(pos), _stream(stream)))

    def layer_step(self, layer: LayerDesc, q, kv: KV, y, microbatch_depth: int = 1,
                   mb_offsets: Optional[Sequence[int]] = None, router_logits=None, attn_out=None,
                   stream=None) -> None:
        offs = None
        if mb_offsets is not None:
            offs = (ctypes.c_int32 * len(mb_offsets))(*[int(v) for v in mb_offsets])
        self._check(self._lib.aflex_layer_step(self._h, ctypes.byref(layer), _ptr(q), ctypes.byref(kv), q.shape[0],
                                               _ptr(router_logits), microbatch_depth, offs, _ptr(attn_out),
                                               _ptr(y), _stream(stream)))

    def decoder_layers(self, layers: Sequence[DecoderDesc], kvs: Sequence[KV], x_in, x_out,
                       microbatch_depth: int = 1, mb_offsets: Optional[Sequence[int]] = None, stream=None) -> None:
        """Runs len(layers) whole decoder layers on x_in bf16 [B,H] -> x_out; kvs[l] is layer l's cache
        (its decoded-token slots are written)."""
        assert len(layers) == len(kvs) and len(layers) >= 1
        offs = None
        if mb_offsets is not None:
            offs = (ctypes.c_int32 * len(mb_offsets))(*[int(v) for v in mb_offsets])
        la = (DecoderDesc * len(layers))(*layers)
        ka = (KV * len(kvs))(*kvs)
        self._check(self._lib.aflex_decoder_layers(self._h, la, ka, len(layers), _ptr(x_in), x_in.shape[0],
                                                   microbatch_depth, offs, _ptr(x_out), _stream(stream)))

    def prefill_layers(self, layers: Sequence[DecoderDesc], kvs: Sequence[KV], x_in, q_offsets: torch.Tensor,
                       q_offsets_host: torch.Tensor, x_out, stream=None) -> None:
        """Runs len(layers) whole decoder layers over the tokens being prefilled: x_in bf16 [T,H] -> x_out, row
        q_offsets[b] + i = token i of the last q_offsets[b+1] - q_offsets[b] tokens of sequence b (the caches'
        seq_lens count them already; their K / V slots are written).  q_offsets i32 CUDA [B+1], q_offsets_host
        the same on the CPU."""
        assert len(layers) == len(kvs) and len(layers) >= 1
        assert q_offsets.dtype == torch.int32 and q_offsets_host.dtype == torch.int32 and q_offsets_host.device.type == "cpu"
        la = (DecoderDesc * len(layers))(*layers)
        ka = (KV * len(kvs))(*kvs)
        self._check(self._lib.aflex_prefill_layers(self._h, la, ka, len(layers), _ptr(x_in), q_offsets_host.shape[0] - 1,
                                                   _ptr(q_offsets), _ptr(q_offsets_host), _ptr(x_out), _stream(stream)))

    def add_rmsnorm(self, res, add, w, eps: float, res_out=None, y=None, stream=None) -> None:
        self._check(self._lib.aflex_add_rmsnorm(self._h, _ptr(res), _ptr(add), _ptr(w), res.shape[0], res.shape[1],
                                                eps, _ptr(res_out), _ptr(y), _stream(stream)))

    def rope_append(self, desc: AttnDesc, qkv, kv: KV, q_out, w_q_norm, w_k_norm, rms_eps: float, rope_theta: float,
                    stream=None) -> None:
        self._check(self._lib.aflex_rope_append(self._h, ctypes.byref(desc), _ptr(qkv), ctypes.byref(kv),
                                                qkv.shape[0], _ptr(w_q_norm), _ptr(w_k_norm), rms_eps, rope_theta,
                                                _ptr(q_out), _stream(stream)))
