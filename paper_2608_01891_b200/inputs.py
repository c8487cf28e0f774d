"""Seeded synthetic inputs for the A/F decode-layer hot path.

This module only draws random tensors and lays them out; it holds none of the
method's arithmetic (no attention, no FFN, no routing).  Both the CUDA library's
tests/benchmarks and the CPU oracle's tests read the bytes produced here, so the
two sides always see identical bf16 inputs.

Workload shapes follow the five benchmark configurations (a tiny layer, two
Qwen3-32B-shaped dense layers, two Mixtral-8x7B-shaped MoE layers).  Context
lengths stand in for the conversation-like (uniform) and coding-like (lognormal)
request traces used in the paper's evaluation (Section 6.1); weights ~N(0, 0.02)
stand in for the trained checkpoints.

Every tensor k of configuration c is drawn from its own generator seeded
``1000*c + k`` (configuration 1 uses seed 0 for its context lengths), in fp32,
then rounded to bf16 with round-to-nearest-even.  Draws can be made on the CPU
(default; bit-reproducible everywhere) or on a CUDA device (fast path for the
multi-GB tensors; reproducible per device type).
"""
from __future__ import annotations

import dataclasses
import math
from typing import Optional, Tuple

import numpy as np
import torch

PAGE_SIZE = 16


@dataclasses.dataclass(frozen=True)
class LayerConfig:
    """Shape of one decoder-layer decode step."""
    cfg_id: int
    name: str
    batch: int
    num_q_heads: int
    num_kv_heads: int
    head_dim: int
    hidden: int
    inter: int
    num_experts: int = 0          # 0 => dense SwiGLU FFN
    top_k: int = 0
    len_dist: str = "uniform"     # "uniform" | "lognormal"
    len_lo: int = 16
    len_hi: int = 128
    len_median: int = 0           # lognormal only
    len_sigma: float = 0.7        # lognormal only
    microbatch_depths: Tuple[int, ...] = (1,)
    zipf_s: float = 0.0           # > 0 => skewed expert load
    # the rest of the decoder layer (whole-layer entry points)
    rms_eps: float = 1e-6
    rope_theta: float = 1.0e6
    qk_norm: bool = True          # per-head RMS normalisation of queries and keys

    @property
    def group(self) -> int:
        return self.num_q_heads // self.num_kv_heads

    @property
    def kv_bytes_per_token(self) -> int:
        return 2 * self.num_kv_heads * self.head_dim * 2


CONFIGS = {
    1: LayerConfig(1, "tiny-dense", 4, 8, 2, 64, 512, 1376,
                   len_dist="uniform", len_lo=16, len_hi=128, rope_theta=1.0e4),
    2: LayerConfig(2, "qwen3-32b-shape", 32, 64, 8, 128, 5120, 25600,
                   len_dist="uniform", len_lo=512, len_hi=4096),
    3: LayerConfig(3, "qwen3-32b-shape-interleaved", 128, 64, 8, 128, 5120, 25600,
                   len_dist="lognormal", len_lo=256, len_hi=8192, len_median=2048,
                   microbatch_depths=(1, 2, 4)),
    4: LayerConfig(4, "mixtral-8x7b-shape", 64, 32, 8, 128, 4096, 14336,
                   num_experts=8, top_k=2,
                   len_dist="uniform", len_lo=1024, len_hi=8192, rms_eps=1e-5, qk_norm=False),
    5: LayerConfig(5, "mixtral-8x7b-shape-loaded", 256, 32, 8, 128, 4096, 14336,
                   num_experts=8, top_k=2,
                   len_dist="lognormal", len_lo=512, len_hi=16384, len_median=4096,
                   microbatch_depths=(1, 2, 3, 4), zipf_s=1.2, rms_eps=1e-5, qk_norm=False),
}

# Tensor indices k inside a configuration (seed = 1000*cfg + k).
_K_LENS, _K_PAGES, _K_Q, _K_KC, _K_VC, _K_X, _K_WG, _K_WU, _K_WD, _K_WO, _K_LOGITS, _K_WR, _K_RANKMAP = range(13)

# Router-logit biases that make per-expert shares of the T*K assignments follow
# Zipf(s=1.2) over ranks 1..8 under top-2 routing of N(0,1)+b logits.  They were
# fitted once, offline, by a fixed-point iteration on the bias vector against a
# large N(0,1) sample; they are plain constants of the input recipe.
ZIPF12_RANK_BIAS = (1.765, 0.449, 0.060, -0.176, -0.345, -0.474, -0.589, -0.689)


def zipf_shares(n: int, s: float) -> np.ndarray:
    """Target share of rank r = 1..n: r^-s, normalised."""
    w = np.arange(1, n + 1, dtype=np.float64) ** (-s)
    return w / w.sum()


def _seed(cfg: LayerConfig, k: int) -> int:
    if cfg.cfg_id == 1 and k == _K_LENS:
        return 0
    return 1000 * cfg.cfg_id + k


def _gen(seed: int, device: str = "cpu") -> torch.Generator:
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    return g


def _randn_bf16(shape, std: float, seed: int, device: str = "cpu", chunk: int = 1 << 27) -> torch.Tensor:
    """fp32 normal draw scaled by std, rounded (RNE) to bf16.  Drawn in chunks so
    multi-GB tensors never hold a full fp32 copy."""
    g = _gen(seed, device)
    n = int(np.prod(shape))
    out = torch.empty(n, dtype=torch.bfloat16, device=device)
    for s in range(0, n, chunk):
        e = min(n, s + chunk)
        t = torch.randn(e - s, generator=g, device=device, dtype=torch.float32)
        if std != 1.0:
            t.mul_(std)
        out[s:e] = t.to(torch.bfloat16)
    return out.view(*shape)


def make_seq_lens(cfg: LayerConfig, batch: Optional[int] = None) -> np.ndarray:
    """Context length of every sequence in the decode batch (int32, >= 1).  The
    length counts the token being decoded (its K/V is already in the cache)."""
    B = cfg.batch if batch is None else batch
    rng = np.random.default_rng(_seed(cfg, _K_LENS))
    if cfg.len_dist == "uniform":
        lens = rng.integers(cfg.len_lo, cfg.len_hi + 1, size=B)
    elif cfg.len_dist == "lognormal":
        z = rng.standard_normal(B)
        lens = np.rint(np.exp(math.log(cfg.len_median) + cfg.len_sigma * z))
        lens = np.clip(lens, cfg.len_lo, cfg.len_hi)
    else:
        raise ValueError(cfg.len_dist)
    return lens.astype(np.int32)


@dataclasses.dataclass
class PagedKV:
    k_cache: torch.Tensor      # bf16 [num_pages, Hkv, PAGE_SIZE, D]
    v_cache: torch.Tensor      # bf16 [num_pages, Hkv, PAGE_SIZE, D]
    page_table: torch.Tensor   # int32 [B, max_pages_per_seq] (CPU)
    seq_lens: torch.Tensor     # int32 [B] (CPU)
    num_pages: int
    max_pages_per_seq: int


def make_page_table(seq_lens: np.ndarray, seed: int, spare_frac: float = 0.25,
                    spare_min: int = 8, fill: int = 0) -> Tuple[np.ndarray, int]:
    """Allocate ceil(len/16) physical pages per sequence from a pool that is
    (1+spare_frac) times larger, through a seeded random permutation, so a
    sequence's pages are physically scattered and non-monotone.  Table entries
    beyond a sequence's last page hold `fill`."""
    pages_per_seq = (seq_lens.astype(np.int64) + PAGE_SIZE - 1) // PAGE_SIZE
    need = int(pages_per_seq.sum())
    num_pages = need + max(spare_min, int(math.ceil(need * spare_frac)))
    rng = np.random.default_rng(seed)
    perm = rng.permutation(num_pages)[:need]
    max_pages = int(pages_per_seq.max()) if len(pages_per_seq) else 1
    table = np.full((len(seq_lens), max_pages), fill, dtype=np.int32)
    o = 0
    for b, n in enumerate(pages_per_seq):
        table[b, :n] = perm[o:o + n]
        o += int(n)
    return table, num_pages


def make_paged_kv(cfg: LayerConfig, seq_lens: Optional[np.ndarray] = None, device: str = "cpu",
                  poison: bool = False) -> PagedKV:
    """K and V pools ~N(0,1) in the library's HND page layout, plus the shuffled
    page table.  With poison=True every slot that no sequence references (spare
    pages, tail slots of last pages) is overwritten with NaN: such slots must
    never influence the output."""
    if seq_lens is None:
        seq_lens = make_seq_lens(cfg)
    table, num_pages = make_page_table(seq_lens, _seed(cfg, _K_PAGES))
    shape = (num_pages, cfg.num_kv_heads, PAGE_SIZE, cfg.head_dim)
    k = _randn_bf16(shape, 1.0, _seed(cfg, _K_KC), device)
    v = _randn_bf16(shape, 1.0, _seed(cfg, _K_VC), device)
    if poison:
        used = torch.zeros(num_pages, PAGE_SIZE, dtype=torch.bool)
        for b, n in enumerate(seq_lens):
            n = int(n)
            npg = (n + PAGE_SIZE - 1) // PAGE_SIZE
            pg = torch.from_numpy(table[b, :npg].astype(np.int64))
            used[pg] = True
            if n % PAGE_SIZE:
                used[int(table[b, npg - 1]), n % PAGE_SIZE:] = False
        mask = (~used).to(k.device)[:, None, :, None].expand(shape)
        nan = torch.tensor(float("nan"), dtype=torch.bfloat16, device=k.device)
        k = torch.where(mask, nan, k)
        v = torch.where(mask, nan, v)
    return PagedKV(k, v, torch.from_numpy(table), torch.from_numpy(seq_lens.astype(np.int32)),
                   num_pages, table.shape[1])


def make_q(cfg: LayerConfig, device: str = "cpu", batch: Optional[int] = None) -> torch.Tensor:
    B = cfg.batch if batch is None else batch
    return _randn_bf16((B, cfg.num_q_heads, cfg.head_dim), 1.0, _seed(cfg, _K_Q), device)


def make_x(cfg: LayerConfig, device: str = "cpu", tokens: Optional[int] = None) -> torch.Tensor:
    """Activations ~N(0,1) entering the FFN side when it is run on its own."""
    T = cfg.batch if tokens is None else tokens
    return _randn_bf16((T, cfg.hidden), 1.0, _seed(cfg, _K_X), device)


def make_wo(cfg: LayerConfig, device: str = "cpu") -> torch.Tensor:
    """Attention output projection [H, Hq*D] ~N(0,0.02)."""
    return _randn_bf16((cfg.hidden, cfg.num_q_heads * cfg.head_dim), 0.02, _seed(cfg, _K_WO), device)


def make_ffn_weights(cfg: LayerConfig, device: str = "cpu"):
    """(w_gate, w_up, w_down) ~N(0,0.02).  Dense: [I,H],[I,H],[H,I].  MoE: the
    same with a leading expert dimension."""
    H, I, E = cfg.hidden, cfg.inter, cfg.num_experts
    lead = (E,) if E > 0 else ()
    wg = _randn_bf16(lead + (I, H), 0.02, _seed(cfg, _K_WG), device)
    wu = _randn_bf16(lead + (I, H), 0.02, _seed(cfg, _K_WU), device)
    wd = _randn_bf16(lead + (H, I), 0.02, _seed(cfg, _K_WD), device)
    return wg, wu, wd


def make_router_weight(cfg: LayerConfig, device: str = "cpu") -> torch.Tensor:
    return _randn_bf16((cfg.num_experts, cfg.hidden), 0.02, _seed(cfg, _K_WR), device)


@dataclasses.dataclass
class DecoderWeights:
    """Weights of one whole decoder layer (bf16).  Index 100*layer + k seeds tensor k of a layer."""
    ln_attn: torch.Tensor                 # [H]            ~ 1 + N(0, 0.1)
    qkv: torch.Tensor                     # [(Hq+2Hkv)*D, H] rows: query heads, key heads, value heads
    q_norm: Optional[torch.Tensor]        # [D] or None    ~ 1 + N(0, 0.1)
    k_norm: Optional[torch.Tensor]        # [D] or None
    o: torch.Tensor                       # [H, Hq*D]
    ln_ffn: torch.Tensor                  # [H]
    gate: torch.Tensor
    up: torch.Tensor
    down: torch.Tensor
    router: Optional[torch.Tensor]        # [E, H] (MoE only)


def _gain_bf16(n: int, seed: int, device: str) -> torch.Tensor:
    g = _gen(seed, device)
    t = torch.randn(n, generator=g, device=device, dtype=torch.float32).mul_(0.1).add_(1.0)
    return t.to(torch.bfloat16)


def make_decoder_weights(cfg: LayerConfig, layer: int = 0, device: str = "cpu") -> DecoderWeights:
    """All weights of decoder layer `layer`: projections ~N(0,0.02), normalisation gains ~1+N(0,0.1).
    Layer 0 reuses the FFN and W_o draws of the hot-path benchmarks; further layers get their own."""
    H, I, E, D = cfg.hidden, cfg.inter, cfg.num_experts, cfg.head_dim
    base = 1000 * cfg.cfg_id + 100 * (layer + 1)
    n_qkv = (cfg.num_q_heads + 2 * cfg.num_kv_heads) * D
    lead = (E,) if E > 0 else ()
    if layer == 0:
        gate, up, down = make_ffn_weights(cfg, device)
        o = make_wo(cfg, device)
        router = make_router_weight(cfg, device) if E > 0 else None
    else:
        gate = _randn_bf16(lead + (I, H), 0.02, base + 0, device)
        up = _randn_bf16(lead + (I, H), 0.02, base + 1, device)
        down = _randn_bf16(lead + (H, I), 0.02, base + 2, device)
        o = _randn_bf16((H, cfg.num_q_heads * D), 0.02, base + 3, device)
        router = _randn_bf16((E, H), 0.02, base + 4, device) if E > 0 else None
    qkv = _randn_bf16((n_qkv, H), 0.02, base + 5, device)
    ln_attn = _gain_bf16(H, base + 6, device)
    ln_ffn = _gain_bf16(H, base + 7, device)
    q_norm = _gain_bf16(D, base + 8, device) if cfg.qk_norm else None
    k_norm = _gain_bf16(D, base + 9, device) if cfg.qk_norm else None
    return DecoderWeights(ln_attn, qkv, q_norm, k_norm, o, ln_ffn, gate, up, down, router)


def make_hidden(cfg: LayerConfig, device: str = "cpu", batch: Optional[int] = None) -> torch.Tensor:
    """Residual-stream input [B, H] ~N(0,1) of the first decoder layer."""
    B = cfg.batch if batch is None else batch
    return _randn_bf16((B, cfg.hidden), 1.0, 1000 * cfg.cfg_id + 50, device)


def make_router_logits(cfg: LayerConfig, tokens: Optional[int] = None) -> torch.Tensor:
    """fp32 router logits [T, E] ~N(0,1) (CPU tensor).  With cfg.zipf_s > 0 a
    per-expert bias is added so expert loads are skewed; the rank -> expert id
    map is a seeded permutation so the hot expert is not always id 0."""
    T = cfg.batch if tokens is None else tokens
    E = cfg.num_experts
    logits = torch.randn(T, E, generator=_gen(_seed(cfg, _K_LOGITS)), dtype=torch.float32)
    if cfg.zipf_s > 0:
        if not (E == 8 and abs(cfg.zipf_s - 1.2) < 1e-12):
            raise ValueError("bias constants are provided for E=8, s=1.2 only")
        rank_to_expert = np.random.default_rng(_seed(cfg, _K_RANKMAP)).permutation(E)
        bias = np.zeros(E, dtype=np.float32)
        bias[rank_to_expert] = np.asarray(ZIPF12_RANK_BIAS, dtype=np.float32)
        logits = logits + torch.from_numpy(bias)
    return logits.contiguous()


def zipf_rank_to_expert(cfg: LayerConfig) -> np.ndarray:
    return np.random.default_rng(_seed(cfg, _K_RANKMAP)).permutation(cfg.num_experts)


def default_mb_offsets(batch: int, depth: int) -> np.ndarray:
    """Near-equal contiguous split of `batch` rows into `depth` microbatches;
    the first batch % depth microbatches get one extra row."""
    base, extra = divmod(batch, depth)
    sizes = [base + (1 if i < extra else 0) for i in range(depth)]
    return np.concatenate([[0], np.cumsum(sizes)]).astype(np.int32)


def bf16_bits(t: torch.Tensor) -> np.ndarray:
    """The raw bf16 bit patterns of a CPU tensor as a uint16 numpy array (no copy)."""
    assert t.dtype == torch.bfloat16 and t.device.type == "cpu"
    return t.contiguous().view(torch.int16).numpy().view(np.uint16)
