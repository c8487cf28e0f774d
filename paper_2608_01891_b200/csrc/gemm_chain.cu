// A chain of dependent decode-batch GEMMs as ONE persistent tcgen05 kernel, software-pipelined
// across the GEMMs.
//
// At decode batch sizes (<= 64 token rows by default) the FFN side and the W_o projection are weight-streaming
// kernels: the boundary projection x = a W_o^T, h = silu(x W_gate^T) .* (x W_up^T) and y = h W_down^T
// each read their weights once and are bound by HBM.  Run as separate kernels, every boundary between
// two of them leaves DRAM idle: the last CTAs of one kernel finish their shared-tile reduction (a chain
// of half a dozen dependent L2 round trips, each 1 - 2 us while the memory system is busy) while the
// next kernel's CTAs cannot become resident beside them (shared memory), set up, and only then request
// their first bytes.  Here the GEMMs are PHASES of one kernel, and no phase waits for the whole of its
// predecessor:
//
//   * one CTA per SM stays resident for all phases; barriers, TMEM and the shared-memory ring are set
//     up once and the ring keeps turning across phase boundaries;
//   * the weight producer (warp 0) never waits for anything but a free ring stage: weights are inputs
//     that no kernel writes;
//   * every phase produces its output tiles in up to four SEGMENTS, one after the other (remainder tiles
//     that are shared along K first, whole tiles second; a phase whose tiles are all shared is cut into
//     equal groups of tiles).  A segment's output is completed - its shared-tile reductions included -
//     while the next segment streams, and is announced through an epoch word;
//   * the reductions run on warps of their own (7..10): the epilogue warps only park fp32 partials and
//     post a job through a shared-memory barrier, so a segment's reduction (waiting for the other
//     contributors, summing in CTA order) never delays the parking of the next accumulators, and no
//     epilogue thread ever executes a device-wide fence; a publisher thread releases each parked
//     partial to the other CTAs at once, whatever the reducers are busy with;
//   * a K step of phase p+1 reads 64 or 128 columns of phase p's output, i.e. the output of ONE tile of
//     phase p.  Every piece of work of phase p+1 (a run of K steps of one tile in one CTA) visits its
//     share of the K steps fed by segment 0 of phase p first, then of segment 1, and so on (any K order
//     gives the same sum up to rounding; the order is a fixed function of the piece, so results are
//     bit-deterministic).  The activation producer (warp 6) waits (bounded) for a segment's epoch only
//     before the first step that needs it - by which time the reduction and the slowest CTA of that
//     segment have had the earlier steps' streaming time to finish;
//   * per segment the tiles are dealt exactly like the stand-alone GEMM (gemm_sched.cuh): equal,
//     contiguous shares of K steps, partials reduced in CTA order.
//
// Orientation as in gemm_tcgen05.cu: 128 weight rows are the MMA's M operand, the token rows its N
// operand; the accumulator in TMEM is out^T (lane = weight row, column = token).
//
// A ring stage holds two 128x64 weight tiles and two activation tiles.  A gate/up phase uses them as
// (gate tile, up tile, x tile) of one 64-wide K block with two accumulators; a linear phase as two
// consecutive K blocks (w, w', x, x') of one accumulator, so that both phase kinds keep the whole ring
// in flight.
//
// CTA = 12 warps: 0 weight producer, 1 MMA issuer (owns TMEM), 2..5 epilogue, 6 activation producer,
// 7..10 reducers, 11 publisher (releases parked partials to the other CTAs).  Every wait is bounded; on expiry the CTA raises AFLEX_ERR_TIMEOUT, drains and leaves.
#include <cuda_bf16.h>
#include <stdlib.h>

#include "internal.h"
#include "ptx.cuh"
#include "gemm_sched.cuh"

namespace aflex {

constexpr int kChainThreads = 384;
constexpr int kChainBlockM = 128;
constexpr int kChainBlockK = 64;
constexpr int kChainTileBytes = kChainBlockM * kChainBlockK * 2;   // one weight tile: 16 KB
constexpr int kChainMaxStages = 8;
constexpr int kChainMaxPhases = 4;
constexpr int kChainMaxSegs = 4;
constexpr long long kChainIdleCycles = 4000;   // a wait for a free ring stage this long (~2 us) is a stall, not back-pressure
constexpr int kChainSlots = 2 * kChainMaxSegs * 2;   // partial slots per CTA: [phase parity][segment][first / later unit]
constexpr int kChainCounterInts = 8192;   // per half of the double-buffered counter array: per-tile counters, then the epoch words
constexpr int kChainEpochBase = kChainCounterInts - 16;
constexpr int kChainMaxStatTiles = 512;    // tiles of a phase with the residual + normalisation epilogue (N <= 65536)
constexpr int kChainStageTokens = 32;       // token rows of an output tile staged per round (the staging buffers' height)
constexpr int kChainMaxJobs = 64;          // reduce jobs one CTA can post in a launch (<= 2 per segment, plus markers)

struct ChainPhase {
    int gateup;        // 1: two weight matrices, SwiGLU epilogue; 0: plain linear
    int N;             // weight rows (output features)
    int K;             // reduction length
    int ksteps;        // ring stages per tile: ceil(K / 64) (gate/up) or ceil(K / 128) (linear)
    int nseg;          // segments in use (1..4)
    int seg_tiles[kChainMaxSegs];   // output tiles per segment; segment g owns tile ids [sum of the earlier ones, + seg_tiles[g])
    int cls_end[kChainMaxSegs];     // K steps [cls_end[g-1], cls_end[g]) read what segment g of the previous phase wrote
                                    // (non-decreasing, last = ksteps; first phase: everything is class 0)
    int counter_base;  // first per-tile arrival counter of this phase
    __nv_bfloat16* out;   // [T][N]
    // Residual + normalisation epilogue (a linear phase in front of a normalised consumer): with o = bf16(in . w^T),
    //   resid_out = bf16(o + resid_in),  out = bf16(resid_out * gain),  ss[tile][t] = sum over the tile's features of resid_out^2
    // and the NEXT phase multiplies its accumulators by rsqrt(sum_tiles ss / N + eps) per token row: RMS normalisation
    // with the row scale moved behind the GEMM, where it commutes ((r x) W^T = r (x W^T)).  gain == nullptr: off.
    const __nv_bfloat16* resid_in;    // [T][N] (may alias resid_out)
    __nv_bfloat16* resid_out;         // [T][N]
    const __nv_bfloat16* gain;        // [N]
    float eps;
    int scale_rows;    // 1: this phase's accumulators take the per-row scale from the previous phase's statistics
};

struct ChainParams {
    int T;             // token rows (<= n_tile)
    int n_tile;        // accumulator columns per matrix: T rounded up to 16
    int box;           // token rows per activation box (TMA) = MMA N
    int nphase;
    int stages;
    int tmem_cols;
    int l2_first_phase;   // first phase whose weights may be prefetched that way
    int l2_ahead;      // ring stages' worth of weights the idle weight producer may prefetch into L2 beyond the ring (0 = off)
    ChainPhase ph[kChainMaxPhases];
    float* partials;   // [grid][kChainSlots][2 * n_tile / 4][128 rows] float4
    float* ss_part;    // [tiles of the normalised phase][n_tile]: per-tile sums of squares of the residual stream rows
    int* counters;     // two halves of kChainCounterInts ints, then the generation word.  A launch of generation g counts
                       // in half g & 1 (per-tile arrival counters and, at kChainEpochBase, its epoch words: (phase, segment)
                       // finished by so many CTAs; all zero on entry), zeroes the other half for its
                       // successor and bumps g
    int* status;
    unsigned long long* trace;   // optional [grid][32] timestamps (ns), or nullptr
};

struct ChainMaps {
    CUtensorMap a0[kChainMaxPhases];   // weights (gate/up: W_gate)
    CUtensorMap a1[kChainMaxPhases];   // gate/up: W_up; linear: unused (a0 again)
    CUtensorMap b[kChainMaxPhases];    // the phase's input activations
};

struct __align__(8) ChainBarriers {
    uint64_t full[kChainMaxStages];     // 2 arrivals (weight producer, activation producer) + their bytes
    uint64_t empty[kChainMaxStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint32_t tmem_base;
    volatile int abort;
    volatile int gen;       // this launch's generation, published by the epilogue once the grid dependency has resolved (-1 before)
    uint64_t job_bar[kChainMaxJobs];    // job n is posted when the 128 epilogue threads have arrived on job_bar[n] (used once each)
    volatile int cur_job, cur_gen;   // the reducers' current job and the generation, handed from their thread 0 to the others
    volatile int job[kChainMaxJobs];   // (phase << 24) | (segment << 20) | kind << 16 | tile in the segment
};
static_assert(sizeof(ChainBarriers) <= 1024, "the staging buffers start 1 KB behind the barriers");
constexpr int kJobReduce = 0, kJobSegEnd = 1, kJobExit = 2;

// The order in which a piece (logical K positions [j0, j1) of a tile with nK steps) visits the actual K steps:
// its share of class 0's steps first, then of class 1's, ... (class g = actual steps [E[g-1], E[g])).  The shares
// are defined by halving twice - classes {0,1} against {2,3}, then inside each half - with the rule
// "positions [0, j) hold floor(j * n / m) steps of the first part", which is monotone in j, so over the pieces
// of a tile the shares partition every class exactly.
struct StepOrder {
    int lo[kChainMaxSegs], len[kChainMaxSegs];
    __device__ static int part(int j, int n, int m) { return m > 0 ? (int)((long long)j * n / m) : 0; }
    __device__ StepOrder(int j0, int j1, int nK, const int* E) {
        const int x0 = part(j0, E[1], nK), x1 = part(j1, E[1], nK);       // classes 0,1: index range [x0, x1) of [0, E1)
        const int y0 = j0 - x0, y1 = j1 - x1;                              // classes 2,3: index range [y0, y1) of [0, nK - E1)
        const int a0 = part(x0, E[0], E[1]), a1 = part(x1, E[0], E[1]);
        lo[0] = a0; len[0] = a1 - a0;
        lo[1] = E[0] + (x0 - a0); len[1] = (x1 - a1) - (x0 - a0);
        const int c0 = part(y0, E[2] - E[1], nK - E[1]), c1 = part(y1, E[2] - E[1], nK - E[1]);
        lo[2] = E[1] + c0; len[2] = c1 - c0;
        lo[3] = E[2] + (y0 - c0); len[3] = (y1 - c1) - (y0 - c0);
    }
    __device__ int actual(int i) const {
#pragma unroll
        for (int g = 0; g < kChainMaxSegs - 1; ++g) {
            if (i < len[g]) return lo[g] + i;
            i -= len[g];
        }
        return lo[kChainMaxSegs - 1] + i;
    }
};

__device__ __forceinline__ float chain_silu(float z) { return __fdividef(z, 1.0f + __expf(-z)); }
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ int seg_tile0(const ChainPhase& P, int seg) {
    int t = 0;
    for (int g = 0; g < seg; ++g) t += P.seg_tiles[g];
    return t;
}

__global__ void __launch_bounds__(kChainThreads, 1)
gemm_chain_kernel(const __grid_constant__ ChainMaps maps, const ChainParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    const int b_bytes = (p.n_tile * kChainBlockK * 2 + 1023) & ~1023;       // one activation tile slot
    const int stage_bytes = 2 * kChainTileBytes + 2 * b_bytes;
    ChainBarriers* bars = reinterpret_cast<ChainBarriers*>(smem + (size_t)p.stages * stage_bytes);
    // output staging, one buffer for the epilogue warps and one for the reducer warps: the output tile as
    // [token][128 features] bf16, so that it leaves the SM in 16-byte pieces
    __nv_bfloat16* stage_epi = reinterpret_cast<__nv_bfloat16*>(smem + (size_t)p.stages * stage_bytes + 1024);
    __nv_bfloat16* stage_red = stage_epi + (size_t)kChainStageTokens * kChainBlockM;
    float* rinv_epi = reinterpret_cast<float*>(stage_red + (size_t)kChainStageTokens * kChainBlockM);   // per-row scales, one copy per group
    float* rinv_red = rinv_epi + kChainMaxRows;

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int grid = (int)gridDim.x;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(&bars->full[s], 2); mbar_init(&bars->empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&bars->tmem_full[b], 1); mbar_init(&bars->tmem_empty[b], 4); }
        bars->abort = 0;
        bars->gen = -1;
        for (int i = 0; i < kChainMaxJobs; ++i) mbar_init(&bars->job_bar[i], 128);
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(&bars->tmem_base, (uint32_t)p.tmem_cols);
        tmem_relinquish();
    }
    if (warp == 0 && lane == 0) {
        for (int i = 0; i < p.nphase; ++i) { prefetch_tmap(&maps.a0[i]); if (p.ph[i].gateup) prefetch_tmap(&maps.a1[i]); }
    }
    if (warp == 6 && lane == 0) {
        for (int i = 0; i < p.nphase; ++i) prefetch_tmap(&maps.b[i]);
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();

    const uint32_t tmem_base = bars->tmem_base;
    const int buf_cols = 2 * p.n_tile;                   // TMEM columns per accumulator buffer (room for gate and up)
    const size_t slot_floats = (size_t)2 * p.n_tile * kChainBlockM;
    pdl_launch_dependents();
    unsigned long long* tr = p.trace ? p.trace + (size_t)blockIdx.x * 32 : nullptr;
    if (tr && threadIdx.x == 0) { tr[0] = global_timer_ns(); unsigned smid; asm volatile("mov.u32 %0, %%smid;" : "=r"(smid)); tr[3] = smid; }   // CTA running

    // The launch's generation, read from global memory by the epilogue after the grid dependency has resolved.
    auto wait_gen = [&]() -> int {
        const long long t_start = clock64();
        int gen;
        while ((gen = bars->gen) < 0 && !bars->abort && clock64() - t_start < kWaitBudgetCycles) __nanosleep(20);
        if (gen < 0 && !bars->abort) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); }
        return gen;
    };

    // Token rows [t_lo, t_hi) of a staged output tile -> memory, 16 bytes per thread and store.  `tid` = 0..127 inside
    // the calling group (epilogue or reducers).  With the residual + normalisation epilogue the same pass adds the
    // residual rows, writes them back, writes the gain-weighted rows for the next phase and reduces every row's sum of
    // squares over the tile's 128 features (16 lanes hold one token row: a fixed-order shuffle reduction).
    // (the staging buffer holds token rows t_lo .. : row t of the tile sits in staged row t - t_lo)
    auto store_tokens = [&](const ChainPhase& P, const __nv_bfloat16* stage_at_t0, int tile_g, int t_lo, int t_hi, int tid) {
        const __nv_bfloat16* stage = stage_at_t0 - (size_t)t_lo * kChainBlockM;
        if (t_hi > p.T) t_hi = p.T;
        if (P.gain == nullptr) {
            for (int c = t_lo * 16 + tid; c < t_hi * 16; c += 128) {
                const int t = c >> 4, part = c & 15;
                const int n = tile_g * kChainBlockM + part * 8;
                if (n < P.N)
                    *reinterpret_cast<uint4*>(P.out + (size_t)t * P.N + n) = *reinterpret_cast<const uint4*>(stage + t * kChainBlockM + part * 8);
            }
            return;
        }
        for (int c0 = t_lo * 16; c0 < t_hi * 16; c0 += 128) {
            const int c = c0 + tid;
            const int t = c >> 4, part = c & 15;
            const int n = tile_g * kChainBlockM + part * 8;
            const bool on = c < t_hi * 16 && n < P.N;
            float ss = 0.f;
            if (on) {
                const uint4 o8 = *reinterpret_cast<const uint4*>(stage + t * kChainBlockM + part * 8);
                const uint4 r8 = __ldcg(reinterpret_cast<const uint4*>(P.resid_in + (size_t)t * P.N + n));
                const uint4 g8 = *reinterpret_cast<const uint4*>(P.gain + n);
                const __nv_bfloat162* po = reinterpret_cast<const __nv_bfloat162*>(&o8);
                const __nv_bfloat162* pr = reinterpret_cast<const __nv_bfloat162*>(&r8);
                const __nv_bfloat162* pg = reinterpret_cast<const __nv_bfloat162*>(&g8);
                uint4 res, xg;
                __nv_bfloat162* ps = reinterpret_cast<__nv_bfloat162*>(&res);
                __nv_bfloat162* px = reinterpret_cast<__nv_bfloat162*>(&xg);
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    const float2 fo = __bfloat1622float2(po[k]), fr = __bfloat1622float2(pr[k]), fg = __bfloat1622float2(pg[k]);
                    ps[k] = __floats2bfloat162_rn(fo.x + fr.x, fo.y + fr.y);
                    const float2 v = __bfloat1622float2(ps[k]);        // the residual stream as stored
                    ss = fmaf(v.x, v.x, ss);
                    ss = fmaf(v.y, v.y, ss);
                    px[k] = __floats2bfloat162_rn(v.x * fg.x, v.y * fg.y);
                }
                *reinterpret_cast<uint4*>(P.resid_out + (size_t)t * P.N + n) = res;
                *reinterpret_cast<uint4*>(P.out + (size_t)t * P.N + n) = xg;
            }
#pragma unroll
            for (int off = 8; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
            if (c < t_hi * 16 && part == 0) p.ss_part[(size_t)tile_g * p.n_tile + t] = ss;
        }
    };
    // The per-row scales of a phase whose input was left un-normalised by the previous phase: waits (bounded) until every
    // segment of that phase is complete everywhere, then sums each row's per-tile statistics in tile order.  Called by
    // all 128 threads of a group; false = gave up (uniformly).
    auto load_row_scales = [&](int pi, const int* ctr, float* rinv, int tid, int bar_id) -> bool {
        const ChainPhase& Q = p.ph[pi - 1];
        bool failed = false;
        if (tid == 0) {
            for (int g = 0; g < Q.nseg && !failed; ++g) {
                const long long t_start = clock64();
                int seen;
                do {
                    asm volatile("ld.acquire.gpu.b32 %0, [%1];" : "=r"(seen) : "l"(ctr + kChainEpochBase + (pi - 1) * kChainMaxSegs + g) : "memory");
                    if (seen >= grid) break;
                    __nanosleep(40);
                } while (clock64() - t_start < kWaitBudgetCycles && !bars->abort);
                if (seen < grid) { failed = true; if (!bars->abort) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); } }
            }
        }
        if (bar_or(bar_id, 128, failed)) return false;
        if (tid < p.n_tile) {
            int tiles = 0;
            for (int g = 0; g < Q.nseg; ++g) tiles += Q.seg_tiles[g];
            float ssum = 0.f;
            for (int m = 0; m < tiles; ++m) ssum += __ldcg(p.ss_part + (size_t)m * p.n_tile + tid);
            rinv[tid] = rsqrtf(ssum / (float)Q.N + Q.eps);
        }
        if (bar_id == 2) asm volatile("bar.sync 2, 128;" ::: "memory");
        else asm volatile("bar.sync 3, 128;" ::: "memory");
        return true;
    };

    if (warp == 0) {
        // ------------------------------------------------------------ weight producer
        if (lane == 0) {
            const uint64_t pol_w = policy_evict_first();      // every weight byte is read once
            int s = 0; uint32_t ph = 0;
            for (int pi = 0; pi < p.nphase && !bars->abort; ++pi) {
                const ChainPhase& P = p.ph[pi];
                for (int seg = 0; seg < P.nseg && !bars->abort; ++seg) {
                    const Schedule sched(P.ksteps, 1, P.seg_tiles[seg], grid);
                    const int tile0 = seg_tile0(P, seg);
                    UnitCursor cur(sched, blockIdx.x);
                    WorkUnit wu;
                    while (!bars->abort && cur.next(wu)) {
                        const int row0 = (tile0 + wu.tile) * kChainBlockM;
                        const StepOrder ord(wu.kb0, wu.kb1, P.ksteps, P.cls_end);
                        const int L = wu.kb1 - wu.kb0;
                        int pf = 0;                                   // steps of this unit already asked into L2
                        for (int i = 0; i < L; ++i) {
                            const int ks = ord.actual(i);
                            if (!mbar_try_wait(&bars->empty[s], ph ^ 1)) {
                                // No free stage.  In steady state one frees up every ~0.7 us.  A longer wait means the
                                // consumers are held up (a phase's input is not there yet): nobody on this SM asks DRAM
                                // for anything, so the wait can be spent pulling the next steps' weight tiles into L2.
                                const long long t0w = clock64();
                                bool ok = false;
                                while (!(ok = mbar_try_wait(&bars->empty[s], ph ^ 1))) {
                                    const long long dt = clock64() - t0w;
                                    if (dt > kWaitBudgetCycles || bars->abort) break;
                                    if (p.l2_ahead > 0 && pi >= p.l2_first_phase && dt > kChainIdleCycles) {
                                        if (pf < i) pf = i;
                                        if (pf < L && pf < i + p.l2_ahead) {
                                            const int kp = ord.actual(pf);
                                            if (P.gateup) {
                                                tma_prefetch_l2_2d(&maps.a0[pi], kp * kChainBlockK, row0);
                                                tma_prefetch_l2_2d(&maps.a1[pi], kp * kChainBlockK, row0);
                                            } else {
                                                tma_prefetch_l2_2d(&maps.a0[pi], 2 * kp * kChainBlockK, row0);
                                                tma_prefetch_l2_2d(&maps.a0[pi], (2 * kp + 1) * kChainBlockK, row0);
                                            }
                                            ++pf;
                                        }
                                    }
                                }
                                if (!ok) { if (!bars->abort) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); } break; }
                            }
                            uint8_t* st = smem + (size_t)s * stage_bytes;
                            mbar_expect_tx(&bars->full[s], 2u * kChainTileBytes);
                            if (P.gateup) {
                                tma_load_2d_hint(st, &maps.a0[pi], ks * kChainBlockK, row0, &bars->full[s], pol_w);
                                tma_load_2d_hint(st + kChainTileBytes, &maps.a1[pi], ks * kChainBlockK, row0, &bars->full[s], pol_w);
                            } else {
                                tma_load_2d_hint(st, &maps.a0[pi], 2 * ks * kChainBlockK, row0, &bars->full[s], pol_w);
                                tma_load_2d_hint(st + kChainTileBytes, &maps.a0[pi], (2 * ks + 1) * kChainBlockK, row0, &bars->full[s], pol_w);
                            }
                            if (++s == p.stages) { s = 0; ph ^= 1; }
                        }
                    }
                }
                if (tr) tr[4 + pi * 8 + 0] = global_timer_ns();       // phase's weight loads all issued
            }
            if (bars->abort) {
                for (int i = 0; i < 200; ++i) __nanosleep(1000);     // loads land within microseconds; their barriers may never complete
            }
        }
    } else if (warp == 6) {
        // ------------------------------------------------------------ activation producer
        if (lane == 0) {
            const uint64_t pol_x = policy_evict_last();       // activations are re-read by every CTA
            const uint32_t box_bytes = (uint32_t)(p.box * kChainBlockK * 2);
            int s = 0; uint32_t ph = 0;
            pdl_wait();                                       // the first phase's input comes from the preceding kernel
            if (tr) tr[1] = global_timer_ns();
            bool bumped = false;
            for (int pi = 0; pi < p.nphase && !bars->abort; ++pi) {
                const ChainPhase& P = p.ph[pi];
                int ready = pi == 0 ? kChainMaxSegs : 0;      // classes [0, ready) of this phase's input are complete
                // Segment e of the previous phase complete in every CTA, and visible to the TMA reads that follow.
                auto need = [&](int e) -> bool {
                    while (ready <= e) {
                        const int gen = wait_gen();
                        if (gen < 0) return false;
                        const int* word = p.counters + (size_t)(gen & 1) * kChainCounterInts + kChainEpochBase + (pi - 1) * kChainMaxSegs + ready;
                        const long long t_start = clock64();
                        int seen;
                        do {
                            asm volatile("ld.acquire.gpu.b32 %0, [%1];" : "=r"(seen) : "l"(word) : "memory");
                            if (seen >= grid) break;
                            __nanosleep(20);
                        } while (clock64() - t_start < kWaitBudgetCycles && !bars->abort);
                        if (seen < grid) { if (!bars->abort) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); } return false; }
                        fence_proxy_async_all();
                        // every CTA's epilogue has read the generation by now (it signs off only afterwards): one thread of
                        // the grid moves it on for the next launch
                        if (blockIdx.x == 0 && !bumped) { p.counters[2 * kChainCounterInts] = (gen + 1) & 0x3fffffff; bumped = true; }
                        if (tr && ready < 2) tr[4 + pi * 8 + 1 + ready] = global_timer_ns();   // input from segment `ready` available
                        ++ready;
                    }
                    return true;
                };
                for (int seg = 0; seg < P.nseg && !bars->abort; ++seg) {
                    const Schedule sched(P.ksteps, 1, P.seg_tiles[seg], grid);
                    UnitCursor cur(sched, blockIdx.x);
                    WorkUnit wu;
                    while (!bars->abort && cur.next(wu)) {
                        const StepOrder ord(wu.kb0, wu.kb1, P.ksteps, P.cls_end);
                        for (int i = 0; i < wu.kb1 - wu.kb0; ++i) {
                            const int ks = ord.actual(i);
                            const int cls = ks < P.cls_end[0] ? 0 : ks < P.cls_end[1] ? 1 : ks < P.cls_end[2] ? 2 : 3;
                            if (!need(cls)) break;
                            if (!mbar_wait(&bars->empty[s], ph ^ 1)) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); break; }
                            uint8_t* st = smem + (size_t)s * stage_bytes + 2 * kChainTileBytes;
                            if (P.gateup) {
                                mbar_expect_tx(&bars->full[s], box_bytes);
                                tma_load_2d_hint(st, &maps.b[pi], ks * kChainBlockK, 0, &bars->full[s], pol_x);
                            } else {
                                mbar_expect_tx(&bars->full[s], 2u * box_bytes);
                                tma_load_2d_hint(st, &maps.b[pi], 2 * ks * kChainBlockK, 0, &bars->full[s], pol_x);
                                tma_load_2d_hint(st + b_bytes, &maps.b[pi], (2 * ks + 1) * kChainBlockK, 0, &bars->full[s], pol_x);
                            }
                            if (++s == p.stages) { s = 0; ph ^= 1; }
                        }
                    }
                }
            }
            // a grid without any later phase step in CTA 0 still has to move the generation on
            if (blockIdx.x == 0 && !bumped && !bars->abort && p.nphase > 1) {
                const int gen = wait_gen();
                if (gen >= 0) {
                    const int* word = p.counters + (size_t)(gen & 1) * kChainCounterInts + kChainEpochBase;
                    const long long t_start = clock64();
                    int seen;
                    do {
                        asm volatile("ld.acquire.gpu.b32 %0, [%1];" : "=r"(seen) : "l"(word) : "memory");
                        if (seen >= grid) break;
                        __nanosleep(20);
                    } while (clock64() - t_start < kWaitBudgetCycles && !bars->abort);
                    if (seen >= grid) p.counters[2 * kChainCounterInts] = (gen + 1) & 0x3fffffff;
                }
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            int s = 0; uint32_t ph = 0;
            int buf = 0; uint32_t acc_ph = 0;
            const uint32_t idesc = umma_idesc_bf16(kChainBlockM, (uint32_t)p.box);
            for (int pi = 0; pi < p.nphase && !bars->abort; ++pi) {
                const ChainPhase& P = p.ph[pi];
                for (int seg = 0; seg < P.nseg && !bars->abort; ++seg) {
                    const Schedule sched(P.ksteps, 1, P.seg_tiles[seg], grid);
                    UnitCursor cur(sched, blockIdx.x);
                    WorkUnit wu;
                    while (!bars->abort && cur.next(wu)) {
                        if (!mbar_wait(&bars->tmem_empty[buf], acc_ph ^ 1)) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); break; }
                        tc_fence_after();
                        const uint32_t d0 = tmem_base + (uint32_t)(buf * buf_cols);
                        for (int i = 0; i < wu.kb1 - wu.kb0; ++i) {
                            if (!mbar_wait(&bars->full[s], ph)) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); break; }
                            tc_fence_after();
                            const uint32_t a_addr = smem_u32(smem + (size_t)s * stage_bytes);
                            const uint64_t da0 = umma_desc_k_sw128(a_addr);
                            const uint64_t da1 = umma_desc_k_sw128(a_addr + kChainTileBytes);
                            const uint64_t db0 = umma_desc_k_sw128(a_addr + 2 * kChainTileBytes);
                            const uint64_t db1 = umma_desc_k_sw128(a_addr + 2 * kChainTileBytes + b_bytes);
                            if (P.gateup) {
#pragma unroll
                                for (int k = 0; k < kChainBlockK / 16; ++k) {
                                    const uint32_t acc = (i > 0 || k > 0) ? 1u : 0u;
                                    umma_bf16(d0, da0 + 2 * k, db0 + 2 * k, idesc, acc);
                                    umma_bf16(d0 + (uint32_t)p.n_tile, da1 + 2 * k, db0 + 2 * k, idesc, acc);
                                }
                            } else {
#pragma unroll
                                for (int k = 0; k < kChainBlockK / 16; ++k)
                                    umma_bf16(d0, da0 + 2 * k, db0 + 2 * k, idesc, (i > 0 || k > 0) ? 1u : 0u);
#pragma unroll
                                for (int k = 0; k < kChainBlockK / 16; ++k)
                                    umma_bf16(d0, da1 + 2 * k, db1 + 2 * k, idesc, 1u);
                            }
                            umma_commit(&bars->empty[s]);
                            if (++s == p.stages) { s = 0; ph ^= 1; }
                        }
                        if (bars->abort) break;
                        umma_commit(&bars->tmem_full[buf]);
                        if (++buf == 2) { buf = 0; acc_ph ^= 1; }
                    }
                }
                if (tr) tr[4 + pi * 8 + 3] = global_timer_ns();       // phase's last MMA issued
            }
        }
    } else if (warp >= 2 && warp <= 5) {
        // ------------------------------------------------------------ epilogue (warps 2..5)
        // Whole tiles go from TMEM through the staging buffer to the output; partial accumulators are parked in the
        // workspace and handed to the reducer warps as a job.  These warps never wait for another CTA.
        const int lane_grp = warp & 3;
        const int row = lane_grp * 32 + lane;
        const int etid = threadIdx.x - 64;
        int buf = 0; uint32_t acc_ph = 0;
        int njobs = 0;
        // Every epilogue thread calls this after its own stores of the job's data: the barrier's release / acquire hands
        // those stores on to the publisher and the reducers, who put their device-wide fence behind them.
        auto post = [&](int job) {
            if (njobs < kChainMaxJobs) {
                if (etid == 0) bars->job[njobs] = job;
                mbar_arrive(&bars->job_bar[njobs]);
                ++njobs;
            }
        };
        pdl_wait();   // nothing is written (outputs, partials, counters) before the preceding kernels have completed
        // The counters are double-buffered over launches: this launch counts in half (generation & 1), zero on entry,
        // and zeroes the other half, which the launch before it used and the launch after it will use.  Both
        // neighbours are ordered against these stores by the grid dependency (the wait above; the next launch's own).
        if (etid == 0) {
            int g;
            asm volatile("ld.relaxed.gpu.b32 %0, [%1];" : "=r"(g) : "l"(p.counters + 2 * kChainCounterInts) : "memory");
            bars->gen = g;
        }
        asm volatile("bar.sync 2, 128;" ::: "memory");
        int* const ctr = p.counters + (size_t)(bars->gen & 1) * kChainCounterInts;
        {
            int* other = p.counters + (size_t)((bars->gen & 1) ^ 1) * kChainCounterInts;
            for (int i = (int)blockIdx.x * 128 + etid; i < kChainCounterInts; i += grid * 128) other[i] = 0;
        }

        bool gave_up = false;
        for (int pi = 0; pi < p.nphase && !gave_up; ++pi) {
            const ChainPhase& P = p.ph[pi];
            const int accs = P.gateup ? 2 : 1;
            if (P.scale_rows && !load_row_scales(pi, ctr, rinv_epi, etid, 2)) { gave_up = true; break; }
            for (int seg = 0; seg < P.nseg && !gave_up; ++seg) {
                const Schedule sched(P.ksteps, 1, P.seg_tiles[seg], grid);
                const int tile0 = seg_tile0(P, seg);
                const int slot0 = ((pi & 1) * kChainMaxSegs + seg) * 2;    // this (phase parity, segment)'s pair of partial slots
                UnitCursor cur(sched, blockIdx.x);
                WorkUnit wu;
                // (the four warps leave this loop together: every exit is decided on a predicate OR-ed across them)
                while (cur.next(wu)) {
                    if (bar_or(2, 128, bars->abort != 0)) { gave_up = true; break; }
                    const bool ok = mbar_wait(&bars->tmem_full[buf], acc_ph);
                    if (bar_or(2, 128, !ok)) {
                        if (etid == 0) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); }
                        gave_up = true;
                        break;
                    }
                    tc_fence_after();
                    const uint32_t t0 = tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(buf * buf_cols);
                    if (wu.slot < 0) {
                        for (int tc = 0; tc < p.T; tc += kChainStageTokens) {          // kChainStageTokens token columns per round
                            const int ntok = min(kChainStageTokens, p.T - tc);
                            for (int c0 = 0; c0 < ntok; c0 += 16) {
                                uint32_t g[16], u[16];
                                tmem_ld_32x32b_x16(t0 + (uint32_t)(tc + c0), g);
                                if (P.gateup) tmem_ld_32x32b_x16(t0 + (uint32_t)(p.n_tile + tc + c0), u);
                                tmem_ld_wait();
#pragma unroll
                                for (int j = 0; j < 16; ++j) {
                                    const float r = P.scale_rows ? rinv_epi[tc + c0 + j] : 1.0f;
                                    const float gv = r * __uint_as_float(g[j]);
                                    const float v = P.gateup ? chain_silu(gv) * (r * __uint_as_float(u[j])) : gv;
                                    stage_epi[(c0 + j) * kChainBlockM + row] = __float2bfloat16_rn(v);
                                }
                            }
                            if (tc + kChainStageTokens >= p.T) {
                                // the accumulator has been read in full: hand the TMEM buffer back before the stores
                                tc_fence_before();
                                __syncwarp();
                                if (lane == 0) mbar_arrive(&bars->tmem_empty[buf]);
                            }
                            asm volatile("bar.sync 2, 128;" ::: "memory");
                            store_tokens(P, stage_epi, tile0 + wu.tile, tc, tc + ntok, etid);
                            asm volatile("bar.sync 2, 128;" ::: "memory");
                        }
                    } else {
                        uint4* mine = reinterpret_cast<uint4*>(p.partials + ((size_t)blockIdx.x * kChainSlots + slot0 + wu.slot) * slot_floats) + row;
                        for (int a = 0; a < accs; ++a) {
                            for (int c0 = 0; c0 < p.T; c0 += 16) {
                                uint32_t g[16];
                                tmem_ld_32x32b_x16(t0 + (uint32_t)(a * p.n_tile + c0), g);
                                tmem_ld_wait();
#pragma unroll
                                for (int j = 0; j < 16; j += 4)
                                    mine[(size_t)((a * p.n_tile + c0 + j) >> 2) * kChainBlockM] = make_uint4(g[j], g[j + 1], g[j + 2], g[j + 3]);
                            }
                        }
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&bars->tmem_empty[buf]);
                        post((pi << 24) | (seg << 20) | (kJobReduce << 16) | wu.tile);
                    }
                    if (++buf == 2) { buf = 0; acc_ph ^= 1; }
                }
                // ---- this CTA's whole tiles of the segment are written (behind a barrier): sign off for the epilogue, and
                //      tell the reducers that the segment has no more jobs
                if (!gave_up) {
                    post((pi << 24) | (seg << 20) | (kJobSegEnd << 16));
                    if (tr && etid == 0 && seg < 2) tr[4 + pi * 8 + 4 + seg] = global_timer_ns();    // segment parked / written by this CTA's epilogue
                }
            }
        }
        post(kJobExit << 16);
    } else if (warp >= 7 && warp <= 10) {
        // ------------------------------------------------------------ reducers (warps 7..10)
        // One job at a time, in the order the epilogue posted them: this CTA's slice of a shared tile, summed over the
        // contributors' pieces in CTA order (bit-deterministic), staged and written; at a segment's end marker, the
        // sign-off for the reducers.
        const int rtid = threadIdx.x - 224;
        volatile int& s_job = bars->cur_job;
        volatile int& s_gen = bars->cur_gen;
        pdl_wait();
        int* ctr = nullptr;
        int taken = 0;
        int scales_of = -1;      // phase whose per-row scales sit in rinv_red
        // (the four warps move together: thread 0 takes every decision and hands it on through shared memory or an
        // OR-ing barrier, so no exit can split the group in front of a barrier)
        while (true) {
            const bool got = taken < kChainMaxJobs && mbar_wait(&bars->job_bar[taken], 0);
            if (rtid == 0) {
                if (!got && !bars->abort) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); }
                s_job = (!got || bars->abort) ? (kJobExit << 16) : bars->job[taken];
                if (ctr == nullptr) s_gen = (!got || bars->abort) ? -1 : wait_gen();
            }
            asm volatile("bar.sync 3, 128;" ::: "memory");
            const int job = s_job, gen = s_gen;
            asm volatile("bar.sync 3, 128;" ::: "memory");     // everybody has read them before they are overwritten
            ++taken;
            const int kind = (job >> 16) & 0xf, pi = job >> 24, seg = (job >> 20) & 0xf, tile = job & 0xffff;
            if (kind == kJobExit || gen < 0) break;
            if (ctr == nullptr) ctr = p.counters + (size_t)(gen & 1) * kChainCounterInts;
            const ChainPhase& P = p.ph[pi];
            if (kind == kJobSegEnd) {
                // The segment is complete in this CTA: its whole tiles were stored by the epilogue threads before they posted
                // this marker, every reduce job ended with a barrier behind its last output store.  One sign-off for both.
                if (rtid == 0 && pi + 1 < p.nphase) {
                    __threadfence();
                    atomicAdd(ctr + kChainEpochBase + pi * kChainMaxSegs + seg, 1);
                }
                if (tr && rtid == 0 && seg < 2) tr[26 + seg] = global_timer_ns();
                continue;
            }
            const int accs = P.gateup ? 2 : 1;
            if (P.scale_rows && scales_of != pi) {
                if (!load_row_scales(pi, ctr, rinv_red, rtid, 3)) break;
                scales_of = pi;
            }
            const Schedule sched(P.ksteps, 1, P.seg_tiles[seg], grid);
            const int tile0 = seg_tile0(P, seg);
            const int* counters = ctr + P.counter_base + tile0;
            const int slot0 = ((pi & 1) * kChainMaxSegs + seg) * 2;
            const long long x0 = (long long)tile * P.ksteps;
            const int cf = sched.cta_of(x0);
            const int cl = sched.cta_of(x0 + P.ksteps - 1);
            const int np = cl - cf + 1, me = (int)blockIdx.x - cf;
            // A last contributor whose share runs on into the next tile has that tile to finish as well: it is excused here.
            const int nred = (np > 1 && sched.share_begin(cl + 1) > x0 + P.ksteps) ? np - 1 : np;
            if (me >= nred) continue;
            bool failed = false;
            if (rtid == 0) {
                const long long t_start = clock64();
                int seen;
                do {
                    asm volatile("ld.acquire.gpu.b32 %0, [%1];" : "=r"(seen) : "l"(counters + tile) : "memory");
                    if (seen >= np) break;
                    __nanosleep(40);
                } while (clock64() - t_start < kWaitBudgetCycles && !bars->abort);
                if (seen < np) { failed = true; if (!bars->abort) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); } }
            }
            // the barrier hands thread 0's acquire on to the other 127 threads, and its decision with it
            if (bar_or(3, 128, failed)) break;
            const bool cf_early = sched.share_begin(cf) < x0;
            // The parked accumulator is [column group of 4 tokens][128 rows] float4: reducer `me` takes whole column
            // groups, thread = weight row.  kE groups per round, every piece's loads of a round in flight together
            // (the loop is a chain of L2 round trips, not bandwidth).
            const int ncg = ((p.T + 15) / 16) * 4;
            const int cg_lo = ncg * me / nred, cg_hi = ncg * (me + 1) / nred;
            const int up_off = (p.n_tile >> 2) * kChainBlockM;
            constexpr int kE = 4;
            constexpr int kCgPerFlush = kChainStageTokens / 4;
            for (int f0 = cg_lo; f0 < cg_hi; f0 += kCgPerFlush) {
            const int f1 = min(cg_hi, f0 + kCgPerFlush);
            for (int c0 = f0; c0 < f1; c0 += kE) {
                float4 g[kE], u[kE];
#pragma unroll
                for (int e = 0; e < kE; ++e) g[e] = u[e] = make_float4(0.f, 0.f, 0.f, 0.f);
                for (int cb = cf; cb <= cl; cb += 4) {
                    float4 a[kE][4];
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        const int cc = cb + q;
                        if (cc <= cl) {
                            const int sl = slot0 + ((cc == cf && cf_early) ? 1 : 0);
                            const float4* part = reinterpret_cast<const float4*>(p.partials + ((size_t)cc * kChainSlots + sl) * slot_floats) + rtid;
#pragma unroll
                            for (int e = 0; e < kE; ++e)
                                if (c0 + e < f1) a[e][q] = __ldcg(part + (c0 + e) * kChainBlockM);
                        }
                    }
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        if (cb + q <= cl) {
#pragma unroll
                            for (int e = 0; e < kE; ++e)
                                if (c0 + e < f1) { g[e].x += a[e][q].x; g[e].y += a[e][q].y; g[e].z += a[e][q].z; g[e].w += a[e][q].w; }
                        }
                    }
                    if (accs == 2) {
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const int cc = cb + q;
                            if (cc <= cl) {
                                const int sl = slot0 + ((cc == cf && cf_early) ? 1 : 0);
                                const float4* part = reinterpret_cast<const float4*>(p.partials + ((size_t)cc * kChainSlots + sl) * slot_floats) + up_off + rtid;
#pragma unroll
                                for (int e = 0; e < kE; ++e)
                                    if (c0 + e < f1) a[e][q] = __ldcg(part + (c0 + e) * kChainBlockM);
                            }
                        }
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            if (cb + q <= cl) {
#pragma unroll
                                for (int e = 0; e < kE; ++e)
                                    if (c0 + e < f1) { u[e].x += a[e][q].x; u[e].y += a[e][q].y; u[e].z += a[e][q].z; u[e].w += a[e][q].w; }
                            }
                        }
                    }
                }
#pragma unroll
                for (int e = 0; e < kE; ++e) {
                    if (c0 + e >= f1) break;
                    const float gf[4] = {g[e].x, g[e].y, g[e].z, g[e].w}, uf[4] = {u[e].x, u[e].y, u[e].z, u[e].w};
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        const int t = (c0 + e) * 4 + k;
                        const float r = P.scale_rows ? rinv_red[t] : 1.0f;
                        stage_red[(t - f0 * 4) * kChainBlockM + rtid] = __float2bfloat16_rn(P.gateup ? chain_silu(r * gf[k]) * (r * uf[k]) : r * gf[k]);
                    }
                }
            }
            asm volatile("bar.sync 3, 128;" ::: "memory");
            store_tokens(P, stage_red, tile0 + tile, f0 * 4, f1 * 4, rtid);
            asm volatile("bar.sync 3, 128;" ::: "memory");
            }
        }
    }

    else if (warp == 11) {
        // ------------------------------------------------------------ publisher
        // Releases every parked partial to the other CTAs as soon as the epilogue has posted it: the arrival counter of
        // its tile is bumped behind a device-wide fence.  Kept apart from the reducers, which may be waiting for another
        // CTA's partial at that moment - a wait that must never hold back this CTA's own partials.
        if (lane == 0) {
            pdl_wait();
            int* ctr = nullptr;
            for (int n = 0; n < kChainMaxJobs && !bars->abort; ++n) {
                if (!mbar_wait(&bars->job_bar[n], 0)) { if (!bars->abort) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); } break; }
                const int job = bars->job[n];
                const int kind = (job >> 16) & 0xf, pi = job >> 24, seg = (job >> 20) & 0xf, tile = job & 0xffff;
                if (kind == kJobExit) break;
                if (kind != kJobReduce) continue;
                if (ctr == nullptr) {
                    const int gen = wait_gen();
                    if (gen < 0) break;
                    ctr = p.counters + (size_t)(gen & 1) * kChainCounterInts;
                }
                __threadfence();
                atomicAdd(ctr + p.ph[pi].counter_base + seg_tile0(p.ph[pi], seg) + tile, 1);
            }
        }
    }

    if (tr && threadIdx.x == 0) tr[2] = global_timer_ns();
    tc_fence_before();
    __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// ----------------------------------------------------------------------------------------- host side
static int chain_enabled() {
    static int v = -1;
    if (v < 0) { const char* e = getenv("AFLEX_FFN_CHAIN"); v = e ? atoi(e) : 1; }
    return v;
}

// Groups of tiles a phase is cut into when all its tiles are shared along K and another phase follows: the later
// groups stream while the earlier ones are reduced, and the next phase starts on the earlier groups' columns.
// Measured on the Qwen3-32B-shaped layer (W_o: 40 tiles, 12 us of streaming): 1 / 2 / 4 groups -> 194.6 / 197.0 /
// 213.0 us per step.  The phase is too short for it: every group adds up to two parked partials per CTA, and a group's
// tile is then shared by 15 CTAs instead of 4.  One group is the default; AFLEX_CHAIN_SPLIT = 2 / 4 cuts (tuning).
static int chain_split() {
    static int v = -1;
    if (v < 0) { const char* e = getenv("AFLEX_CHAIN_SPLIT"); v = e ? atoi(e) : 1; if (v < 1) v = 1; if (v > kChainMaxSegs) v = kChainMaxSegs; }
    return v;
}

// The largest batch that takes the chain kernel.  The kernel itself handles up to kChainMaxRows = 128 token rows, but
// above 64 a ring stage is 64 KB and only three fit: measured at the Qwen3-32B shape with 128 rows, 152.9 us for the FFN
// against 142.4 us as two launches of the stand-alone GEMM, and 403.9 against 397.3 us for the configuration-3 step.
// So 64 is the default; AFLEX_CHAIN_MAX_ROWS (<= 128) moves it (tuning / comparison).
static int chain_max_rows() {
    static int v = -1;
    if (v < 0) { const char* e = getenv("AFLEX_CHAIN_MAX_ROWS"); v = e ? atoi(e) : 64; if (v > kChainMaxRows) v = kChainMaxRows; if (v < 0) v = 0; }
    return v;
}

bool chain_supported(int T) { return chain_enabled() != 0 && T >= 1 && T <= chain_max_rows(); }

static int chain_n_tile(int T) { return ((T < 16 ? 16 : T) + 15) / 16 * 16; }

size_t chain_counter_ints() { return 2 * (size_t)kChainCounterInts + 64; }

size_t chain_workspace_bytes(int T, int num_sms) {
    return align256((size_t)num_sms * kChainSlots * 2 * chain_n_tile(T) * kChainBlockM * sizeof(float)) +
           align256((size_t)kChainMaxStatTiles * chain_n_tile(T) * sizeof(float));
}

aflex_status chain_launch(aflex_ctx* ctx, const ChainStep* steps, int nsteps, int T, char* ws, size_t ws_bytes,
                          cudaStream_t st, int* counters) {
    if (nsteps < 1 || nsteps > kChainMaxPhases || !chain_supported(T))
        return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "gemm chain: %d steps at %d rows", nsteps, T);
    ChainParams p;
    ChainMaps maps;
    p.T = T;
    p.n_tile = chain_n_tile(T);
    p.box = p.n_tile;
    p.nphase = nsteps;
    { static int v = -1; if (v < 0) { const char* e = getenv("AFLEX_CHAIN_L2_PHASE"); v = e ? atoi(e) : 1; } p.l2_first_phase = v; }
    { static int v = -1; if (v < 0) { const char* e = getenv("AFLEX_CHAIN_L2_AHEAD"); v = e ? atoi(e) : 0; if (v < 0) v = 0; if (v > 64) v = 64; } p.l2_ahead = v; }
    int cols = 32;
    while (cols < 2 * 2 * p.n_tile) cols <<= 1;
    p.tmem_cols = cols;
    const int b_bytes = (p.n_tile * kChainBlockK * 2 + 1023) & ~1023;
    const int stage_bytes = 2 * kChainTileBytes + 2 * b_bytes;
    const int stage_out_bytes = 2 * kChainStageTokens * kChainBlockM * 2 + 2 * kChainMaxRows * 4;      // one staging buffer each for epilogue and reducers, and their per-row scales
    const int budget = kMaxDynamicSmem - 1024 - 1024 - stage_out_bytes - 256;
    p.stages = budget / stage_bytes;
    if (p.stages > kChainMaxStages) p.stages = kChainMaxStages;
    { static int v = -1; if (v < 0) { const char* e = getenv("AFLEX_CHAIN_STAGES"); v = e ? atoi(e) : 0; } if (v >= 2 && v < p.stages) p.stages = v; }
    if (p.stages < 2) return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "gemm chain: no ring fits");
    const size_t smem_bytes = (size_t)p.stages * stage_bytes + 1024 + stage_out_bytes + 1024 + 128;
    const size_t need = chain_workspace_bytes(T, ctx->num_sms);
    if (need > ws_bytes || ws == nullptr)
        return set_error(ctx, AFLEX_ERR_WORKSPACE, "gemm chain: need %zu workspace bytes, have %zu", need, ws_bytes);
    int base = 0;
    const void* in = nullptr;
    for (int i = 0; i < nsteps; ++i) {
        const ChainStep& s = steps[i];
        ChainPhase& P = p.ph[i];
        P.gateup = s.w1 != nullptr;
        P.N = s.N; P.K = s.K;
        const int m_tiles = (s.N + kChainBlockM - 1) / kChainBlockM;
        P.ksteps = P.gateup ? (s.K + kChainBlockK - 1) / kChainBlockK : (s.K + 2 * kChainBlockK - 1) / (2 * kChainBlockK);
        // Segments: the remainder tiles (shared along K) first and the whole tiles second; when no CTA gets a whole
        // tile, equal groups of tiles - except in the last phase, whose output nobody in this kernel waits for.
        const int grid = ctx->num_sms, whole = m_tiles / grid * grid, rem = m_tiles - whole;
        for (int g = 0; g < kChainMaxSegs; ++g) P.seg_tiles[g] = 0;
        if (whole > 0) { P.nseg = 2; P.seg_tiles[0] = rem; P.seg_tiles[1] = whole; }
        else {
            int ns = (i + 1 < nsteps) ? chain_split() : 1;
            if (ns > m_tiles) ns = m_tiles;
            P.nseg = ns;
            for (int g = 0; g < ns; ++g) P.seg_tiles[g] = m_tiles * (g + 1) / ns - m_tiles * g / ns;
        }
        // K steps fed by the previous phase's segments (its tile t is this phase's K columns [128 t, 128 t + 128))
        if (i == 0) { for (int g = 0; g < kChainMaxSegs; ++g) P.cls_end[g] = P.ksteps; }
        else {
            int tiles = 0;
            for (int g = 0; g < kChainMaxSegs; ++g) {
                tiles += p.ph[i - 1].seg_tiles[g];
                const int e = (P.gateup ? 2 : 1) * tiles;
                P.cls_end[g] = (e < P.ksteps && g + 1 < kChainMaxSegs) ? e : P.ksteps;
            }
        }
        P.counter_base = base;
        base += m_tiles;
        P.out = reinterpret_cast<__nv_bfloat16*>(s.out);
        P.resid_in = reinterpret_cast<const __nv_bfloat16*>(s.resid_in);
        P.resid_out = reinterpret_cast<__nv_bfloat16*>(s.resid_out);
        P.gain = reinterpret_cast<const __nv_bfloat16*>(s.gain);
        P.eps = s.eps;
        P.scale_rows = (i > 0 && steps[i - 1].gain != nullptr) ? 1 : 0;
        if (P.gain && (P.gateup || !P.resid_in || !P.resid_out || i + 1 >= nsteps || m_tiles > kChainMaxStatTiles))
            return set_error(ctx, AFLEX_ERR_INVALID_ARG, "gemm chain: the residual + normalisation epilogue needs a linear step with a successor");
        in = s.in;
        if (!encode_tmap_2d_bf16(&maps.a0[i], s.w0, (uint64_t)s.N, (uint64_t)s.K, (uint64_t)s.K * 2, kChainBlockM, kChainBlockK, true) ||
            !encode_tmap_2d_bf16(&maps.a1[i], P.gateup ? s.w1 : s.w0, (uint64_t)s.N, (uint64_t)s.K, (uint64_t)s.K * 2, kChainBlockM, kChainBlockK, true) ||
            !encode_tmap_2d_bf16(&maps.b[i], in, (uint64_t)T, (uint64_t)s.K, (uint64_t)s.K * 2, (uint32_t)p.box, kChainBlockK, false))
            return set_error(ctx, AFLEX_ERR_CUDA, "gemm chain: cuTensorMapEncodeTiled failed");
    }
    for (int i = nsteps; i < kChainMaxPhases; ++i) { p.ph[i] = p.ph[0]; maps.a0[i] = maps.a0[0]; maps.a1[i] = maps.a1[0]; maps.b[i] = maps.b[0]; }
    p.partials = reinterpret_cast<float*>(ws);
    p.ss_part = reinterpret_cast<float*>(ws + align256((size_t)ctx->num_sms * kChainSlots * 2 * p.n_tile * kChainBlockM * sizeof(float)));
    if (base > kChainEpochBase) return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "gemm chain: too many tiles");
    p.counters = counters;
    p.status = ctx->dev_status;
    p.trace = ctx->trace ? ctx->trace + (size_t)(ctx->trace_slot++ % kTraceKernels) * kTraceStride : nullptr;

    if (!ctx->chain_attr_set) {
        cudaError_t e = cudaFuncSetAttribute(gemm_chain_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, kMaxDynamicSmem);
        if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(gemm chain)");
        ctx->chain_attr_set = true;
    }
    KernelScope scope(ctx, kKGemmChain, st);
    return check_cuda(ctx, launch_pdl(gemm_chain_kernel, dim3((unsigned)ctx->num_sms), dim3(kChainThreads), smem_bytes, st, maps, p),
                      "gemm_chain_kernel launch");
}

}  // namespace aflex
