// FFN-side GEMMs on the 5th-generation tensor cores (tcgen05.mma, accumulators in TMEM,
// operands staged by TMA with the 128-byte swizzle).
//
// Orientation ("weights are the M operand"): every product here is  out[t][n] = sum_k x[t][k] * w[n][k]
// with a weight matrix w[N][K] that is far larger than the activation x[T][K] at decode batch
// sizes.  The MMA's 128-row M operand is therefore a tile of 128 weight rows and its N operand
// is a tile of n_tile token rows (16..256), so a decode batch of 32 tokens costs one N=32 MMA
// per 128 weight rows instead of a 128-row tile that is three quarters padding.  At small T the
// kernel is a weight-streaming kernel (HBM-bound), at large T a tensor-core kernel; the same
// code serves both.  The accumulator in TMEM is out^T: lane = weight row (output feature),
// column = token.
//
// Variants (template MODE):
//   kLinear : out = x w^T                                   (W_o projection, down projection)
//   kGateUp : out = silu(x w_gate^T) .* (x w_up^T)          (two accumulators, fused SwiGLU epilogue)
// Both have a grouped form for the mixture-of-experts FFN: the rows of x are the permuted
// assignments, expert e owns rows [offsets[e], offsets[e+1]) and its own weight matrices.
// kLinear optionally splits K across CTAs (fp32 partials + a fixed-order reduction kernel) so
// that small-N projections still occupy every SM; the reduction order is fixed => deterministic.
//
// CTA = 6 warps: warp 0 TMA producer, warp 1 MMA issuer (owns TMEM), warps 2..5 epilogue.
// Persistent over a static round-robin tile list.  All waits are bounded.
#include <cuda_bf16.h>
#include <stdio.h>

#include "internal.h"
#include "ptx.cuh"

namespace aflex {

enum GemmMode { kLinear = 0, kGateUp = 1 };

constexpr int kBlockM = 128;   // weight rows per tile (UMMA M)
constexpr int kBlockK = 64;    // bf16 elements per 128-byte swizzled row
constexpr int kGemmThreads = 192;
constexpr int kMaxStages = 8;
constexpr int kMaxExperts = 64;

struct GemmParams {
    int T;            // token rows of x (all experts' rows together for the grouped form)
    int N;            // weight rows (output features) per expert
    int K;
    int n_tile;       // token rows per tile, multiple of 16, <= 256
    int m_tiles;      // ceil(N / 128)
    int n_tiles;      // ceil(T / n_tile) (non-grouped)
    int splits;       // K splits (kLinear only)
    int kblocks;      // ceil(K / 64)
    int stages;       // smem pipeline depth
    int nbuf;         // TMEM accumulator buffers (1 or 2)
    int num_experts;  // 0 => not grouped
    int tmem_cols;    // power of two >= 32
    const int32_t* offsets;   // grouped: device [E+1]
    __nv_bfloat16* out_bf16;  // [T][N] (direct bf16 output) or nullptr
    float* out_f32;           // [splits][T][N] fp32 partial sums, or nullptr
    int* status;
};

struct TileCoord {
    int m_tile;     // weight-row tile inside the expert
    int a_row0;     // first row in the 2-D [(E*N)][K] weight view
    int b_row0;     // first token row
    int b_rows;     // valid token rows in this tile (<= n_tile)
    int split;
    int out_row_limit;  // exclusive bound on token rows that may be stored
};

// Work list shared by all roles of a CTA.  Non-grouped: item = (m_tile, n_tile, split), n fastest.
// Grouped: item = (expert, m_tile, chunk, split) over the experts' row segments, chunk fastest.
struct TileIter {
    const GemmParams& p;
    const int* seg;       // smem copy of offsets (grouped)
    int total;
    __device__ TileIter(const GemmParams& p_, const int* seg_) : p(p_), seg(seg_) {
        if (p.num_experts == 0) {
            total = p.m_tiles * p.n_tiles * p.splits;
        } else {
            int chunks = 0;
            for (int e = 0; e < p.num_experts; ++e) chunks += (seg[e + 1] - seg[e] + p.n_tile - 1) / p.n_tile;
            total = chunks * p.m_tiles * p.splits;
        }
    }
    __device__ TileCoord get(int w) const {
        TileCoord c;
        c.split = w % p.splits;
        w /= p.splits;
        if (p.num_experts == 0) {
            int nt = w % p.n_tiles;
            c.m_tile = w / p.n_tiles;
            c.a_row0 = c.m_tile * kBlockM;
            c.b_row0 = nt * p.n_tile;
            c.b_rows = min(p.n_tile, p.T - c.b_row0);
            c.out_row_limit = p.T;
        } else {
            int e = 0;
            for (; e < p.num_experts; ++e) {
                int items = ((seg[e + 1] - seg[e] + p.n_tile - 1) / p.n_tile) * p.m_tiles;
                if (w < items) break;
                w -= items;
            }
            int chunks = (seg[e + 1] - seg[e] + p.n_tile - 1) / p.n_tile;
            int ch = w % chunks;
            c.m_tile = w / chunks;
            c.a_row0 = e * p.N + c.m_tile * kBlockM;
            c.b_row0 = seg[e] + ch * p.n_tile;
            c.b_rows = min(p.n_tile, seg[e + 1] - c.b_row0);
            c.out_row_limit = seg[e + 1];
        }
        return c;
    }
};

struct __align__(8) GemmBarriers {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint32_t tmem_base;
    volatile int abort;
    int seg[kMaxExperts + 1];
};

__device__ __forceinline__ float silu_f32(float z) { return z / (1.0f + __expf(-z)); }

template <int MODE>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmap_a0, const __grid_constant__ CUtensorMap tmap_a1,
            const __grid_constant__ CUtensorMap tmap_b, const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment: the 128-byte swizzle pattern is a function of address bits [7,10).
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int kNumA = (MODE == kGateUp) ? 2 : 1;
    constexpr int kABytes = kBlockM * kBlockK * 2;           // 16 KB
    const int b_bytes = p.n_tile * kBlockK * 2;
    const int stage_bytes = kNumA * kABytes + ((b_bytes + 1023) & ~1023);
    GemmBarriers* bars = reinterpret_cast<GemmBarriers*>(smem + (size_t)p.stages * stage_bytes);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&bars->tmem_full[b], 1); mbar_init(&bars->tmem_empty[b], 4); }
        bars->abort = 0;
        fence_mbar_init();
    }
    if (p.num_experts > 0) {
        for (int i = threadIdx.x; i <= p.num_experts; i += blockDim.x) bars->seg[i] = p.offsets[i];
    }
    if (warp == 1) {
        tmem_alloc(&bars->tmem_base, (uint32_t)p.tmem_cols);
        tmem_relinquish();
    }
    if (warp == 0 && lane == 0) {
        prefetch_tmap(&tmap_a0);
        if (MODE == kGateUp) prefetch_tmap(&tmap_a1);
        prefetch_tmap(&tmap_b);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    const uint32_t tmem_base = bars->tmem_base;
    const TileIter tiles(p, bars->seg);
    const int acc_cols = (MODE == kGateUp ? 2 : 1) * p.n_tile;   // TMEM columns per accumulator buffer

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            const uint64_t pol_w = policy_evict_first();   // weights: streamed once
            const uint64_t pol_x = policy_evict_last();    // activations: re-read by every tile
            int s = 0; uint32_t ph = 0;
            const uint32_t tx = (uint32_t)(kNumA * kABytes + b_bytes);
            for (int w = blockIdx.x; w < tiles.total && !bars->abort; w += gridDim.x) {
                const TileCoord c = tiles.get(w);
                const int kb0 = (int)(((long long)c.split * p.kblocks) / p.splits);
                const int kb1 = (int)(((long long)(c.split + 1) * p.kblocks) / p.splits);
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!mbar_wait(&bars->empty[s], ph ^ 1)) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); break; }
                    uint8_t* st = smem + (size_t)s * stage_bytes;
                    mbar_expect_tx(&bars->full[s], tx);
                    tma_load_2d_hint(st, &tmap_a0, kb * kBlockK, c.a_row0, &bars->full[s], pol_w);
                    if (MODE == kGateUp) tma_load_2d_hint(st + kABytes, &tmap_a1, kb * kBlockK, c.a_row0, &bars->full[s], pol_w);
                    tma_load_2d_hint(st + kNumA * kABytes, &tmap_b, kb * kBlockK, c.b_row0, &bars->full[s], pol_x);
                    if (++s == p.stages) { s = 0; ph ^= 1; }
                }
            }
            // Drain: every load issued above has a consumer waiting on its full barrier unless the
            // kernel aborted; on abort wait (bounded) for the loads in flight before leaving.
            if (bars->abort) {
                for (int i = 0; i < p.stages; ++i) (void)mbar_wait(&bars->full[i], 0);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = umma_idesc_bf16(kBlockM, (uint32_t)p.n_tile);
            int s = 0; uint32_t ph = 0;
            int buf = 0; uint32_t acc_ph = 0;
            bool issued_any = false;
            for (int w = blockIdx.x; w < tiles.total && !bars->abort; w += gridDim.x) {
                const TileCoord c = tiles.get(w);
                const int kb0 = (int)(((long long)c.split * p.kblocks) / p.splits);
                const int kb1 = (int)(((long long)(c.split + 1) * p.kblocks) / p.splits);
                if (!mbar_wait(&bars->tmem_empty[buf], acc_ph ^ 1)) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); break; }
                tc_fence_after();
                const uint32_t d0 = tmem_base + (uint32_t)(buf * acc_cols);
                for (int kb = kb0; kb < kb1; ++kb) {
                    if (!mbar_wait(&bars->full[s], ph)) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); break; }
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(smem + (size_t)s * stage_bytes);
                    const uint64_t da0 = umma_desc_k_sw128(a_addr);
                    const uint64_t db = umma_desc_k_sw128(a_addr + kNumA * kABytes);
#pragma unroll
                    for (int k = 0; k < kBlockK / 16; ++k) {
                        const uint32_t acc = (kb > kb0 || k > 0) ? 1u : 0u;
                        // advancing 16 bf16 along K inside the swizzled row = +32 bytes = +2 in 16-byte units
                        umma_bf16(d0, da0 + 2 * k, db + 2 * k, idesc, acc);
                        if (MODE == kGateUp) {
                            const uint64_t da1 = umma_desc_k_sw128(a_addr + kABytes);
                            umma_bf16(d0 + (uint32_t)p.n_tile, da1 + 2 * k, db + 2 * k, idesc, acc);
                        }
                    }
                    umma_commit(&bars->empty[s]);   // smem stage reusable once these MMAs retire
                    issued_any = true;
                    if (++s == p.stages) { s = 0; ph ^= 1; }
                }
                if (bars->abort) break;
                umma_commit(&bars->tmem_full[buf]);  // accumulator complete
                if (++buf == p.nbuf) { buf = 0; acc_ph ^= 1; }
            }
            (void)issued_any;
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..5)
        const int lane_grp = warp & 3;                 // TMEM lanes [32*lane_grp, +32) belong to this warp
        int buf = 0; uint32_t acc_ph = 0;
        for (int w = blockIdx.x; w < tiles.total && !bars->abort; w += gridDim.x) {
            const TileCoord c = tiles.get(w);
            if (!mbar_wait(&bars->tmem_full[buf], acc_ph)) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); break; }
            tc_fence_after();
            const int n_local = c.m_tile * kBlockM + lane_grp * 32 + lane;    // output feature inside the expert
            const bool n_ok = n_local < p.N;
            const uint32_t t0 = tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(buf * acc_cols);
            for (int c0 = 0; c0 < c.b_rows; c0 += 16) {
                uint32_t g[16];
                tmem_ld_32x32b_x16(t0 + (uint32_t)c0, g);
                if (MODE == kGateUp) {
                    uint32_t u[16];
                    tmem_ld_32x32b_x16(t0 + (uint32_t)(p.n_tile + c0), u);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int t = c.b_row0 + c0 + j;
                        if (n_ok && t < c.out_row_limit) {
                            const float hv = silu_f32(__uint_as_float(g[j])) * __uint_as_float(u[j]);
                            p.out_bf16[(size_t)t * p.N + n_local] = __float2bfloat16_rn(hv);
                        }
                    }
                } else {
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int t = c.b_row0 + c0 + j;
                        if (n_ok && t < c.out_row_limit) {
                            const float v = __uint_as_float(g[j]);
                            if (p.out_f32) p.out_f32[((size_t)c.split * p.T + t) * p.N + n_local] = v;
                            else p.out_bf16[(size_t)t * p.N + n_local] = __float2bfloat16_rn(v);
                        }
                    }
                }
            }
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&bars->tmem_empty[buf]);
            if (++buf == p.nbuf) { buf = 0; acc_ph ^= 1; }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// out[t][n] = sum_s part[s][t][n]  (fixed order s = 0,1,..) -> bf16 or fp32
__global__ void splitk_reduce_kernel(const float* __restrict__ part, int splits, size_t TN, __nv_bfloat16* out_bf16,
                                     float* out_f32) {
    const size_t i4 = ((size_t)blockIdx.x * blockDim.x + threadIdx.x) * 4;
    if (i4 >= TN) return;
    float4 acc = *reinterpret_cast<const float4*>(part + i4);
    for (int s = 1; s < splits; ++s) {
        const float4 v = *reinterpret_cast<const float4*>(part + (size_t)s * TN + i4);
        acc.x += v.x; acc.y += v.y; acc.z += v.z; acc.w += v.w;
    }
    if (out_bf16) {
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
        uint2 pk;
        pk.x = *reinterpret_cast<uint32_t*>(&lo);
        pk.y = *reinterpret_cast<uint32_t*>(&hi);
        *reinterpret_cast<uint2*>(out_bf16 + i4) = pk;
    } else {
        *reinterpret_cast<float4*>(out_f32 + i4) = acc;
    }
}

// ----------------------------------------------------------------------------------------- host side
static int round_up(int a, int b) { return (a + b - 1) / b * b; }

static int pick_n_tile(int rows_max) {
    int n = round_up(rows_max < 16 ? 16 : rows_max, 16);
    return n > 256 ? 256 : n;
}

// Choose the K split so that the static round-robin list fills whole waves of CTAs.
static int pick_splits(int base_items, int kblocks, int num_sms, bool allow) {
    if (!allow || base_items >= 2 * num_sms) return 1;
    int best = 1;
    double best_score = -1.0;
    for (int s = 1; s <= 16; ++s) {
        if (kblocks / s < 8) break;
        const int items = base_items * s;
        const int waves = (items + num_sms - 1) / num_sms;
        double eff = (double)items / ((double)waves * num_sms);
        // prefer fewer splits when efficiency is close (partials cost traffic)
        const double score = eff - 0.004 * s;
        if (score > best_score) { best_score = score; best = s; }
    }
    return best;
}

struct GemmConfig {
    GemmParams p;
    size_t smem_bytes;
    int grid;
};

static bool make_config(int mode, int T, int N, int K, int rows_max, int E, int num_sms, bool allow_split,
                        GemmConfig* cfg) {
    GemmParams& p = cfg->p;
    p.T = T; p.N = N; p.K = K;
    p.n_tile = pick_n_tile(rows_max);
    p.m_tiles = (N + kBlockM - 1) / kBlockM;
    p.n_tiles = (T + p.n_tile - 1) / p.n_tile;
    p.kblocks = (K + kBlockK - 1) / kBlockK;
    p.num_experts = E;
    const int base_items = (E == 0) ? p.m_tiles * p.n_tiles : p.m_tiles * E * ((rows_max + p.n_tile - 1) / p.n_tile);
    p.splits = (mode == kLinear) ? pick_splits(base_items, p.kblocks, num_sms, allow_split) : 1;
    const int acc_cols = (mode == kGateUp ? 2 : 1) * p.n_tile;
    p.nbuf = (2 * acc_cols <= 512) ? 2 : 1;
    int cols = 32;
    while (cols < p.nbuf * acc_cols) cols <<= 1;
    p.tmem_cols = cols;
    const int a_bytes = (mode == kGateUp ? 2 : 1) * kBlockM * kBlockK * 2;
    const int stage_bytes = a_bytes + round_up(p.n_tile * kBlockK * 2, 1024);
    const int budget = 227 * 1024 - 1024 /*alignment slack*/ - (int)sizeof(GemmBarriers) - 256;
    int stages = budget / stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) return false;
    p.stages = stages;
    cfg->smem_bytes = (size_t)stages * stage_bytes + sizeof(GemmBarriers) + 1024 + 128;
    int items = base_items * p.splits;
    cfg->grid = items < num_sms ? items : num_sms;
    if (cfg->grid < 1) cfg->grid = 1;
    return true;
}

template <int MODE>
static aflex_status launch_gemm(aflex_ctx* ctx, const GemmConfig& cfg, const CUtensorMap& ta0, const CUtensorMap& ta1,
                                const CUtensorMap& tb, cudaStream_t st, int kind) {
    if (!ctx->gemm_attr_set[MODE]) {
        cudaError_t e = cudaFuncSetAttribute(gemm_kernel<MODE>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kMaxDynamicSmem);
        if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(gemm)");
        ctx->gemm_attr_set[MODE] = true;
    }
    KernelScope scope(ctx, kind, st);
    gemm_kernel<MODE><<<cfg.grid, kGemmThreads, cfg.smem_bytes, st>>>(ta0, ta1, tb, cfg.p);
    return check_cuda(ctx, cudaGetLastError(), "gemm_kernel launch");
}

static aflex_status run_reduce(aflex_ctx* ctx, const float* part, int splits, size_t TN, void* out_bf16, float* out_f32,
                               cudaStream_t st) {
    const int threads = 256;
    const size_t n4 = (TN + 3) / 4;
    const int blocks = (int)((n4 + threads - 1) / threads);
    KernelScope scope(ctx, kKSplitKReduce, st);
    splitk_reduce_kernel<<<blocks, threads, 0, st>>>(part, splits, TN, (__nv_bfloat16*)out_bf16, out_f32);
    return check_cuda(ctx, cudaGetLastError(), "splitk_reduce launch");
}

size_t linear_workspace_bytes(int T, int K, int N, int num_sms) {
    GemmConfig cfg;
    if (!make_config(kLinear, T, N, K, T, 0, num_sms, true, &cfg)) return 0;
    return cfg.p.splits > 1 ? align256((size_t)cfg.p.splits * T * N * sizeof(float)) : 0;
}

aflex_status linear_launch(aflex_ctx* ctx, const void* x, const void* w, int T, int K, int N, void* y, char* ws,
                           size_t ws_bytes, cudaStream_t st, int kind) {
    GemmConfig cfg;
    if (!make_config(kLinear, T, N, K, T, 0, ctx->num_sms, true, &cfg))
        return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "linear: no tile configuration fits");
    GemmParams& p = cfg.p;
    p.offsets = nullptr;
    p.status = ctx->dev_status;
    if (p.splits > 1) {
        const size_t need = (size_t)p.splits * T * N * sizeof(float);
        if (need > ws_bytes) return set_error(ctx, AFLEX_ERR_WORKSPACE, "linear: need %zu workspace bytes, have %zu", need, ws_bytes);
        p.out_f32 = reinterpret_cast<float*>(ws);
        p.out_bf16 = nullptr;
    } else {
        p.out_f32 = nullptr;
        p.out_bf16 = reinterpret_cast<__nv_bfloat16*>(y);
    }
    CUtensorMap ta, tb;
    if (!encode_tmap_2d_bf16(&ta, w, (uint64_t)N, (uint64_t)K, (uint64_t)K * 2, kBlockM, kBlockK, true) ||
        !encode_tmap_2d_bf16(&tb, x, (uint64_t)T, (uint64_t)K, (uint64_t)K * 2, (uint32_t)p.n_tile, kBlockK, false))
        return set_error(ctx, AFLEX_ERR_CUDA, "linear: cuTensorMapEncodeTiled failed");
    aflex_status s = launch_gemm<kLinear>(ctx, cfg, ta, ta, tb, st, kind);
    if (s != AFLEX_OK) return s;
    if (p.splits > 1) return run_reduce(ctx, p.out_f32, p.splits, (size_t)T * N, y, nullptr, st);
    return AFLEX_OK;
}

size_t gateup_workspace_bytes(int, int, int, int) { return 0; }

aflex_status gateup_launch(aflex_ctx* ctx, const void* x, const void* w_gate, const void* w_up, int T, int H, int I,
                           void* h, char*, size_t, cudaStream_t st) {
    GemmConfig cfg;
    if (!make_config(kGateUp, T, I, H, T, 0, ctx->num_sms, false, &cfg))
        return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "gate/up: no tile configuration fits");
    GemmParams& p = cfg.p;
    p.offsets = nullptr;
    p.status = ctx->dev_status;
    p.out_f32 = nullptr;
    p.out_bf16 = reinterpret_cast<__nv_bfloat16*>(h);
    CUtensorMap tg, tu, tb;
    if (!encode_tmap_2d_bf16(&tg, w_gate, (uint64_t)I, (uint64_t)H, (uint64_t)H * 2, kBlockM, kBlockK, true) ||
        !encode_tmap_2d_bf16(&tu, w_up, (uint64_t)I, (uint64_t)H, (uint64_t)H * 2, kBlockM, kBlockK, true) ||
        !encode_tmap_2d_bf16(&tb, x, (uint64_t)T, (uint64_t)H, (uint64_t)H * 2, (uint32_t)p.n_tile, kBlockK, false))
        return set_error(ctx, AFLEX_ERR_CUDA, "gate/up: cuTensorMapEncodeTiled failed");
    return launch_gemm<kGateUp>(ctx, cfg, tg, tu, tb, st, kKGateUpGemm);
}

size_t grouped_workspace_bytes(int rows_total, int rows_max, int K, int N, int E, int num_sms) {
    GemmConfig cfg;
    if (!make_config(kLinear, rows_total, N, K, rows_max, E, num_sms, true, &cfg)) return 0;
    return cfg.p.splits > 1 ? align256((size_t)cfg.p.splits * rows_total * N * sizeof(float)) : 0;
}

aflex_status grouped_gateup_launch(aflex_ctx* ctx, const void* xp, const void* w_gate, const void* w_up,
                                   const int32_t* offsets, int rows_total, int rows_max, int H, int I, int E,
                                   void* hp, char*, size_t, cudaStream_t st) {
    if (E > kMaxExperts) return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "num_experts > %d", kMaxExperts);
    GemmConfig cfg;
    if (!make_config(kGateUp, rows_total, I, H, rows_max, E, ctx->num_sms, false, &cfg))
        return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "grouped gate/up: no tile configuration fits");
    GemmParams& p = cfg.p;
    p.offsets = offsets;
    p.status = ctx->dev_status;
    p.out_f32 = nullptr;
    p.out_bf16 = reinterpret_cast<__nv_bfloat16*>(hp);
    CUtensorMap tg, tu, tb;
    if (!encode_tmap_2d_bf16(&tg, w_gate, (uint64_t)E * I, (uint64_t)H, (uint64_t)H * 2, kBlockM, kBlockK, true) ||
        !encode_tmap_2d_bf16(&tu, w_up, (uint64_t)E * I, (uint64_t)H, (uint64_t)H * 2, kBlockM, kBlockK, true) ||
        !encode_tmap_2d_bf16(&tb, xp, (uint64_t)rows_total, (uint64_t)H, (uint64_t)H * 2, (uint32_t)p.n_tile, kBlockK, false))
        return set_error(ctx, AFLEX_ERR_CUDA, "grouped gate/up: cuTensorMapEncodeTiled failed");
    return launch_gemm<kGateUp>(ctx, cfg, tg, tu, tb, st, kKMoeGateUpGemm);
}

aflex_status grouped_linear_launch(aflex_ctx* ctx, const void* hp, const void* w_down, const int32_t* offsets,
                                   int rows_total, int rows_max, int K, int N, int E, float* yp, char* ws,
                                   size_t ws_bytes, cudaStream_t st) {
    if (E > kMaxExperts) return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "num_experts > %d", kMaxExperts);
    GemmConfig cfg;
    if (!make_config(kLinear, rows_total, N, K, rows_max, E, ctx->num_sms, true, &cfg))
        return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "grouped linear: no tile configuration fits");
    GemmParams& p = cfg.p;
    p.offsets = offsets;
    p.status = ctx->dev_status;
    p.out_bf16 = nullptr;
    if (p.splits > 1) {
        const size_t need = (size_t)p.splits * rows_total * N * sizeof(float);
        if (need > ws_bytes) return set_error(ctx, AFLEX_ERR_WORKSPACE, "grouped linear: need %zu workspace bytes, have %zu", need, ws_bytes);
        p.out_f32 = reinterpret_cast<float*>(ws);
    } else {
        p.out_f32 = yp;
    }
    CUtensorMap ta, tb;
    if (!encode_tmap_2d_bf16(&ta, w_down, (uint64_t)E * N, (uint64_t)K, (uint64_t)K * 2, kBlockM, kBlockK, true) ||
        !encode_tmap_2d_bf16(&tb, hp, (uint64_t)rows_total, (uint64_t)K, (uint64_t)K * 2, (uint32_t)p.n_tile, kBlockK, false))
        return set_error(ctx, AFLEX_ERR_CUDA, "grouped linear: cuTensorMapEncodeTiled failed");
    aflex_status s = launch_gemm<kLinear>(ctx, cfg, ta, ta, tb, st, kKMoeDownGemm);
    if (s != AFLEX_OK) return s;
    if (p.splits > 1) return run_reduce(ctx, p.out_f32, p.splits, (size_t)rows_total * N, nullptr, yp, st);
    return AFLEX_OK;
}

}  // namespace aflex
