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
//   kLinear2: kLinear with two weight-row tiles (256 rows) per CTA tile sharing one activation tile:
//             half the activation traffic per weight byte, used at 64..128 token rows
// Both have a grouped form for the mixture-of-experts FFN: the rows of x are the permuted
// assignments, expert e owns rows [offsets[e], offsets[e+1]) and its own weight matrices.
//
// Scheduling.  A persistent CTA per SM.  With many tiles per CTA, whole tiles are taken
// round-robin.  With few (the decode case: 200 gate/up tiles or 40 down-projection tiles on 148
// SMs) the tile count is written as W * G + R for G CTAs: the R remainder tiles are cut along K
// into one equal, contiguous share of 64-wide K blocks per CTA and are processed FIRST; then every
// CTA takes its W whole tiles.  Every SM therefore streams the same number of weight bytes.  A
// remainder tile whose K range is shared by several CTAs is finished by those CTAs together: each
// contributor stores its fp32 partial accumulator to the workspace and bumps the tile's counter;
// when all pieces are there, contributor i sums the i-th slice of the tile over the pieces IN CTA
// ORDER (bit-deterministic), applies the epilogue and writes that slice.  Because the shared tiles
// come first, this fix-up overlaps the main loop of the CTA's next tile.
//
// Programmatic dependent launch: the kernel lets its successor start early and itself starts
// before its predecessor has drained; weight tiles (which no kernel writes) are prefetched into
// the pipeline before the grid-dependency wait, activation tiles only after it.
//
// CTA = 10 warps: warp 0 TMA producer, warp 1 MMA issuer (owns TMEM), warps 2..9 epilogue (a warp reads the TMEM lanes
// of its quadrant, warp index mod 4; the two warps of a quadrant take alternate groups of 16 token columns).
// All waits are bounded.
#include <cuda_bf16.h>
#include <stdio.h>
#include <stdlib.h>

#include "internal.h"
#include "ptx.cuh"
#include "gemm_sched.cuh"

namespace aflex {

enum GemmMode { kLinear = 0, kGateUp = 1, kLinear2 = 2 };

constexpr int kBlockM = 128;   // weight rows per tile (UMMA M)
constexpr int kBlockK = 64;    // bf16 elements per 128-byte swizzled row
constexpr int kEpiWarps = 8;                                 // epilogue warps: two per TMEM lane quadrant, each pair splits the token columns
constexpr int kEpiThreads = kEpiWarps * 32;
constexpr int kGemmThreads = 64 + kEpiThreads;
constexpr int kMaxStages = 8;
constexpr int kMaxExperts = 64;
constexpr int kStageTokens = 32;                             // token rows staged per round of the epilogue

struct GemmParams {
    int T;            // token rows of x (all experts' rows together for the grouped form)
    int N;            // weight rows (output features) per expert
    int K;
    int n_tile;       // token rows per tile, multiple of 16, <= 256
    int m_tiles;      // ceil(N / tile_rows)
    int tile_rows;    // weight rows per tile: 128, or 256 in kLinear2
    int n_tiles;      // ceil(T / n_tile) (non-grouped)
    int kblocks;      // ceil(K / 64)
    int stages;       // smem pipeline depth
    int nbuf;         // TMEM accumulator buffers (1 or 2)
    int num_experts;  // 0 => not grouped
    int tmem_cols;    // power of two >= 32
    int streamk;      // 1 => equal contiguous shares of (tile, k-block) units per CTA
    int w_reuse;      // 1 => keep weight tiles in L2 (normal eviction priority) for a second reader
    const int32_t* offsets;   // grouped: device [E+1]
    __nv_bfloat16* out_bf16;  // [T][N] bf16 output, or nullptr
    float* out_f32;           // [T][N] fp32 output (MoE down projection), or nullptr
    float* partials;          // shared tiles: [grid][2 slots][accumulators * n_tile / 4][128 rows] float4
    int* counters;            // shared tiles: [2][kStreamKMaxTiles] arrival / completion counters, zero on entry and exit
    int* status;
    unsigned long long* trace;   // optional [grid][8] timestamps (ns) for timeline debugging, or nullptr
};

struct TileCoord {
    int m_tile;     // weight-row tile inside the expert
    int a_row0;     // first row in the 2-D [(E*N)][K] weight view
    int b_row0;     // first token row
    int b_rows;     // valid token rows in this tile (<= n_tile)
    int out_row_limit;  // exclusive bound on token rows that may be stored
};

// Tile list shared by all roles of a CTA.  Non-grouped: tile = (m_tile, n_tile), n fastest.
// Grouped: tile = (expert, m_tile, chunk) over the experts' row segments, chunk fastest.
struct TileIter {
    const GemmParams& p;
    const int* seg;       // smem copy of offsets (grouped)
    int total;
    __device__ TileIter(const GemmParams& p_, const int* seg_) : p(p_), seg(seg_) {
        if (p.num_experts == 0) {
            total = p.m_tiles * p.n_tiles;
        } else {
            int chunks = 0;
            for (int e = 0; e < p.num_experts; ++e) chunks += (seg[e + 1] - seg[e] + p.n_tile - 1) / p.n_tile;
            total = chunks * p.m_tiles;
        }
    }
    __device__ TileCoord get(int w) const {
        TileCoord c;
        if (p.num_experts == 0) {
            int nt = w % p.n_tiles;
            c.m_tile = w / p.n_tiles;
            c.a_row0 = c.m_tile * p.tile_rows;
            c.b_row0 = nt * p.n_tile;
            c.b_rows = min(p.n_tile, p.T - c.b_row0);
            c.out_row_limit = p.T;
        } else {
            int e = 0;
            for (; e < p.num_experts - 1; ++e) {
                int items = ((seg[e + 1] - seg[e] + p.n_tile - 1) / p.n_tile) * p.m_tiles;
                if (w < items) break;
                w -= items;
            }
            int chunks = (seg[e + 1] - seg[e] + p.n_tile - 1) / p.n_tile;
            if (chunks < 1) chunks = 1;
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

// Activation (B operand) tensor maps with box heights 16, 32, 64, 128, 256 token rows: a tile loads
// (and multiplies) only as many token rows as it has, rounded up to the next of these sizes; a cold
// expert with 18 rows costs an N = 32 MMA and a 4 KB load per K block, not the widest tile's.
struct TmapSetB {
    CUtensorMap m[5];
};
__host__ __device__ __forceinline__ int box_index(int rows) { return rows <= 16 ? 0 : rows <= 32 ? 1 : rows <= 64 ? 2 : rows <= 128 ? 3 : 4; }
// Box height actually used for a tile with `rows` token rows: never more than the tile (the stage's
// activation buffer and the TMEM accumulator are sized for n_tile rows).
__host__ __device__ __forceinline__ int box_rows(int rows, int n_tile) { const int b = 16 << box_index(rows); return b < n_tile ? b : n_tile; }

struct __align__(8) GemmBarriers {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full[2];
    uint64_t tmem_empty[2];
    uint32_t tmem_base;
    volatile int abort;
    int seg[kMaxExperts + 1];
};

__device__ __forceinline__ float silu_f32(float z) { return __fdividef(z, 1.0f + __expf(-z)); }

template <int MODE, bool PAIR>
__global__ void __launch_bounds__(kGemmThreads, 1)
gemm_kernel(const __grid_constant__ CUtensorMap tmap_a0, const __grid_constant__ CUtensorMap tmap_a1,
            const __grid_constant__ TmapSetB tmaps_b, const GemmParams p) {
    extern __shared__ uint8_t smem_raw[];
    // 1024-byte alignment: the 128-byte swizzle pattern is a function of address bits [7,10).
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    constexpr int kNumA = (MODE == kLinear) ? 1 : 2;
    constexpr int kABytes = kBlockM * kBlockK * 2;           // 16 KB
    // (a CTA of a pair holds half of the token rows of the activation tile)
    const int stage_bytes = kNumA * kABytes + (((PAIR ? p.n_tile / 2 : p.n_tile) * kBlockK * 2 + 1023) & ~1023);
    // Pair form: CTAs 2c and 2c + 1 are pair c of the schedule; rank 0 issues the MMAs of both.
    const int rank = PAIR ? (int)cluster_cta_rank() : 0;
    const int cid = PAIR ? (int)(blockIdx.x >> 1) : (int)blockIdx.x;
    GemmBarriers* bars = reinterpret_cast<GemmBarriers*>(smem + (size_t)p.stages * stage_bytes);
    // Epilogue staging: kStageTokens token rows of the output tile, [token][tile's weight rows] in the output type, so
    // that results leave the SM as 16-byte stores of consecutive features instead of one 2-byte store per value.
    uint8_t* stage_out = smem + (size_t)p.stages * stage_bytes + ((sizeof(GemmBarriers) + 127) & ~(size_t)127);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < p.stages; ++s) { mbar_init(&bars->full[s], 1); mbar_init(&bars->empty[s], 1); }
        for (int b = 0; b < 2; ++b) { mbar_init(&bars->tmem_full[b], 1); mbar_init(&bars->tmem_empty[b], (PAIR ? 2 : 1) * kEpiWarps); }
        bars->abort = 0;
        fence_mbar_init();
    }
    if (p.num_experts > 0) {
        // the expert segment offsets come from an earlier kernel of the same chain: they are only
        // valid once the grid dependency has resolved (so the grouped form cannot prefetch weights early)
        pdl_wait();
        for (int i = threadIdx.x; i <= p.num_experts; i += blockDim.x) bars->seg[i] = p.offsets[i];
    }
    if (warp == 1) {
        if (PAIR) { tmem_alloc_pair(&bars->tmem_base, (uint32_t)p.tmem_cols); tmem_relinquish_pair(); }
        else { tmem_alloc(&bars->tmem_base, (uint32_t)p.tmem_cols); tmem_relinquish(); }
    }
    if (warp == 0 && lane == 0) {
        prefetch_tmap(&tmap_a0);
        if (MODE == kGateUp) prefetch_tmap(&tmap_a1);
        for (int i = 0; i <= box_index(p.n_tile); ++i) prefetch_tmap(&tmaps_b.m[i]);
    }
    tc_fence_before();
    if (PAIR) cluster_sync_all();      // the peer's barriers are initialised before anything signals them
    else __syncthreads();
    tc_fence_after();

    const uint32_t tmem_base = bars->tmem_base;
    const TileIter tiles(p, bars->seg);
    constexpr int kAccs = (MODE == kLinear) ? 1 : 2;
    const int acc_cols = kAccs * p.n_tile;   // TMEM columns per accumulator buffer
    const Schedule sched(p.kblocks, p.streamk, tiles.total, PAIR ? (int)(gridDim.x >> 1) : (int)gridDim.x);
    pdl_launch_dependents();
    unsigned long long* tr = p.trace ? p.trace + (size_t)blockIdx.x * 8 : nullptr;
    if (tr && threadIdx.x == 0) tr[0] = global_timer_ns();           // CTA running

    if (warp == 0) {
        // ------------------------------------------------------------ TMA producer
        if (lane == 0) {
            // weights: streamed once (evict first), unless a second chunk of the same expert re-reads them
            const uint64_t pol_w = p.w_reuse ? policy_evict_normal() : policy_evict_first();
            const uint64_t pol_x = policy_evict_last();    // activations: re-read by every tile
            int s = 0; uint32_t ph = 0;
            UnitCursor cur(sched, cid);
            WorkUnit wu;
            // Pair form: both CTAs' loads of a stage are counted on the even CTA's barrier (it issues the MMAs).
            auto load = [&](void* dst, const CUtensorMap* tm, int x, int y, int stage, uint64_t pol) {
                if (PAIR) tma_load_2d_hint_pair(dst, tm, x, y, cluster_map_shared(smem_u32(&bars->full[stage]), 0), pol);
                else tma_load_2d_hint(dst, tm, x, y, &bars->full[stage], pol);
            };
            const int a_off = rank * kBlockM;                      // this CTA's weight rows inside a pair tile
            // The first `stages` K blocks find the ring empty: their weight tiles are requested at once,
            // before the grid-dependency wait; their activation tiles follow after it.
            int primed = 0;
            int pend_kb[kMaxStages], pend_row[kMaxStages], pend_box[kMaxStages];
            bool waited = false;
            while (!bars->abort && cur.next(wu)) {
                const TileCoord c = tiles.get(wu.tile);
                const int bi = box_index(c.b_rows);
                const int box = box_rows(c.b_rows, p.n_tile);
                const uint32_t tx = (uint32_t)((PAIR ? 2 : 1) * kNumA * kABytes + box * kBlockK * 2);   // both CTAs' bytes
                const int b_row = c.b_row0 + (PAIR ? rank * (box >> 1) : 0);
                for (int kb = wu.kb0; kb < wu.kb1; ++kb) {
                    if (primed < p.stages) {
                        uint8_t* st = smem + (size_t)primed * stage_bytes;
                        if (rank == 0) mbar_expect_tx(&bars->full[primed], tx);
                        load(st, &tmap_a0, kb * kBlockK, c.a_row0 + a_off, primed, pol_w);
                        if (kNumA == 2) load(st + kABytes, MODE == kGateUp ? &tmap_a1 : &tmap_a0, kb * kBlockK,
                                             c.a_row0 + a_off + (MODE == kGateUp ? 0 : kBlockM), primed, pol_w);
                        pend_kb[primed] = kb; pend_row[primed] = b_row; pend_box[primed] = bi;
                        ++primed;
                        if (++s == p.stages) { s = 0; ph ^= 1; }
                        continue;
                    }
                    if (!waited) {
                        if (tr) tr[1] = global_timer_ns();           // weights primed, about to wait
                        pdl_wait();
                        if (tr) tr[2] = global_timer_ns();           // dependency satisfied
                        for (int i = 0; i < primed; ++i)
                            load(smem + (size_t)i * stage_bytes + kNumA * kABytes, &tmaps_b.m[pend_box[i]],
                                 pend_kb[i] * kBlockK, pend_row[i], i, pol_x);
                        waited = true;
                    }
                    if (!mbar_wait(&bars->empty[s], ph ^ 1)) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); break; }
                    uint8_t* st = smem + (size_t)s * stage_bytes;
                    if (rank == 0) mbar_expect_tx(&bars->full[s], tx);
                    load(st, &tmap_a0, kb * kBlockK, c.a_row0 + a_off, s, pol_w);
                    if (kNumA == 2) load(st + kABytes, MODE == kGateUp ? &tmap_a1 : &tmap_a0, kb * kBlockK,
                                         c.a_row0 + a_off + (MODE == kGateUp ? 0 : kBlockM), s, pol_w);
                    load(st + kNumA * kABytes, &tmaps_b.m[bi], kb * kBlockK, b_row, s, pol_x);
                    if (++s == p.stages) { s = 0; ph ^= 1; }
                }
            }
            if (tr) tr[3] = global_timer_ns();                       // all loads issued
            if (!waited) {
                pdl_wait();
                for (int i = 0; i < primed; ++i)
                    load(smem + (size_t)i * stage_bytes + kNumA * kABytes, &tmaps_b.m[pend_box[i]],
                         pend_kb[i] * kBlockK, pend_row[i], i, pol_x);
            }
            // On abort wait (bounded) for loads still in flight before the CTA leaves (the even CTA of a pair waits
            // for its peer's too: they are counted on its barriers, and the peer leaves after it).
            if (bars->abort && rank == 0) {
                for (int i = 0; i < p.stages; ++i) (void)mbar_wait(&bars->full[i], 0);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------ MMA issuer
        if (lane == 0 && rank == 0) {
            int s = 0; uint32_t ph = 0;
            int buf = 0; uint32_t acc_ph = 0;
            UnitCursor cur(sched, cid);
            WorkUnit wu;
            while (!bars->abort && cur.next(wu)) {
                const uint32_t idesc = umma_idesc_bf16(PAIR ? 2 * kBlockM : kBlockM, (uint32_t)box_rows(tiles.get(wu.tile).b_rows, p.n_tile));
                if (!mbar_wait(&bars->tmem_empty[buf], acc_ph ^ 1)) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); break; }
                tc_fence_after();
                const uint32_t d0 = tmem_base + (uint32_t)(buf * acc_cols);
                for (int kb = wu.kb0; kb < wu.kb1; ++kb) {
                    if (!mbar_wait(&bars->full[s], ph)) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); break; }
                    tc_fence_after();
                    const uint32_t a_addr = smem_u32(smem + (size_t)s * stage_bytes);
                    const uint64_t da0 = umma_desc_k_sw128(a_addr);
                    const uint64_t db = umma_desc_k_sw128(a_addr + kNumA * kABytes);
#pragma unroll
                    for (int k = 0; k < kBlockK / 16; ++k) {
                        const uint32_t acc = (kb > wu.kb0 || k > 0) ? 1u : 0u;
                        // advancing 16 bf16 along K inside the swizzled row = +32 bytes = +2 in 16-byte units
                        if (PAIR) umma_bf16_pair(d0, da0 + 2 * k, db + 2 * k, idesc, acc);
                        else umma_bf16(d0, da0 + 2 * k, db + 2 * k, idesc, acc);
                        if (kNumA == 2) {
                            const uint64_t da1 = umma_desc_k_sw128(a_addr + kABytes);
                            if (PAIR) umma_bf16_pair(d0 + (uint32_t)p.n_tile, da1 + 2 * k, db + 2 * k, idesc, acc);
                            else umma_bf16(d0 + (uint32_t)p.n_tile, da1 + 2 * k, db + 2 * k, idesc, acc);
                        }
                    }
                    // smem stage reusable once these MMAs retire (in both CTAs of a pair)
                    if (PAIR) umma_commit_pair(&bars->empty[s]); else umma_commit(&bars->empty[s]);
                    if (++s == p.stages) { s = 0; ph ^= 1; }
                }
                if (bars->abort) break;
                if (PAIR) umma_commit_pair(&bars->tmem_full[buf]); else umma_commit(&bars->tmem_full[buf]);  // accumulator complete
                if (tr) tr[4] = global_timer_ns();                   // last MMA of the unit issued
                if (++buf == p.nbuf) { buf = 0; acc_ph ^= 1; }
            }
        }
    } else {
        // ------------------------------------------------------------ epilogue (warps 2..9)
        const int lane_grp = warp & 3;                 // TMEM lanes [32*lane_grp, +32) belong to this warp
        const int chalf = (warp - 2) >> 2;             // which of the quadrant's two warps: takes column groups chalf, chalf + 2, ..
        const int row = lane_grp * 32 + lane;          // accumulator row = weight row inside the tile
        const int etid = threadIdx.x - 64;             // 0..255 among the epilogue threads
        const int cols = kAccs * p.n_tile;             // fp32 values per accumulator row
        const size_t slot_floats = (size_t)cols * kBlockM;
        int buf = 0; uint32_t acc_ph = 0;
        UnitCursor cur(sched, cid);
        WorkUnit wu;
        // Handing an accumulator buffer back: to the MMA issuer's barrier, which in a pair is the even CTA's.
        auto release_tmem = [&](int b) {
            if (PAIR) mbar_arrive_cluster(cluster_map_shared(smem_u32(&bars->tmem_empty[b]), 0));
            else mbar_arrive(&bars->tmem_empty[b]);
        };
        // Counters of a shared tile: in a pair each CTA finishes its own 128 rows with the same-rank CTAs of the other pairs.
        auto ctile = [&](int tile) { return PAIR ? tile * 2 + rank : tile; };
        pdl_wait();   // nothing is written before the predecessor grid has completed

        // Geometry of the output tile in the staging buffer and in memory.
        constexpr int kTileCols = (MODE == kLinear2) ? 2 * kBlockM : kBlockM;    // weight rows (output features) per tile
        const int es = p.out_f32 ? 4 : 2;                                        // bytes per output element
        const int per16 = 16 / es;                                               // elements per 16-byte store
        const int cpr = kTileCols / per16;                                       // 16-byte pieces per staged token row
        auto stage_put = [&](int tl, int col, float v) {                         // token row tl of the round, feature col of the tile
            if (p.out_f32) reinterpret_cast<float*>(stage_out)[tl * kTileCols + col] = v;
            else reinterpret_cast<__nv_bfloat16*>(stage_out)[tl * kTileCols + col] = __float2bfloat16_rn(v);
        };
        // Staged token rows [0, ntok) -> output rows t0 + .. (bounded by t_limit), features 128 * .. of the tile; the
        // barriers order the staging writes before the reads and free the buffer for its next user.
        auto stage_flush = [&](const TileCoord& c, int t0, int ntok) {
            asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads) : "memory");
            const int n0 = c.m_tile * p.tile_rows + rank * kBlockM;
            for (int i = etid; i < ntok * cpr; i += kEpiThreads) {
                const int tl = i / cpr, part = i - tl * cpr;
                const int t = t0 + tl, n = n0 + part * per16;
                if (t < c.out_row_limit && n < p.N) {
                    const uint4 v = *reinterpret_cast<const uint4*>(stage_out + ((size_t)tl * kTileCols + part * per16) * es);
                    uint8_t* dst = p.out_f32 ? reinterpret_cast<uint8_t*>(p.out_f32 + (size_t)t * p.N + n)
                                             : reinterpret_cast<uint8_t*>(p.out_bf16 + (size_t)t * p.N + n);
                    *reinterpret_cast<uint4*>(dst) = v;
                }
            }
            asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads) : "memory");
        };

        // A shared tile is finished by its contributors together (all of them but a last one that has another
        // shared tile to finish): once every piece is published (arrival counter == number of pieces; bounded
        // spin), reducer i sums the i-th slice of the tile over all pieces, in CTA order, and writes that slice
        // of the output.  A second counter tells the last finisher to reset both counters.  Contributors of a tile run concurrently (the
        // grid never exceeds the SM count and shared tiles are everyone's first units), so the spin is short.
        struct PendingTile { int tile; TileCoord c; };
        PendingTile pend[2];
        int npend = 0;
        bool gave_up = false;
        auto run_reduce = [&](const PendingTile& pd) {
            const long long x0 = (long long)pd.tile * p.kblocks;
            const int cf = sched.cta_of(x0);
            const int cl = sched.cta_of(x0 + p.kblocks - 1);
            const int np = cl - cf + 1, me = cid - cf;
            // A last contributor whose share runs on into the next tile has a second shared tile to finish (as that
            // tile's first contributor): it is excused here, so that no CTA does two reductions one after the other
            // at the very end, where everybody else waits for the kernel's last CTA.
            const int nred = (np > 1 && sched.share_begin(cl + 1) > x0 + p.kblocks) ? np - 1 : np;
            if (me >= nred) return;
            bool failed = false;
            if (etid == 0) {
                const long long t_start = clock64();
                int seen;
                do {
                    asm volatile("ld.acquire.gpu.b32 %0, [%1];" : "=r"(seen) : "l"(p.counters + ctile(pd.tile)) : "memory");
                    if (seen >= np) break;
                    __nanosleep(64);
                } while (clock64() - t_start < kWaitBudgetCycles);
                if (seen < np) { failed = true; bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); }
            }
            // the barrier hands thread 0's acquire on to the other epilogue threads, and its decision with it: the warps
            // leave together or not at all (there are barriers further down)
            if (bar_or(2, kEpiThreads, failed)) { gave_up = true; return; }
            const bool cf_early = sched.share_begin(cf) < x0;
            // The parked accumulators are [column group of 4 tokens][128 rows] float4.  Reducer `me` takes whole column
            // groups, thread = accumulator row; kElems groups per round with every piece's loads of a round in flight
            // together (the loop is bound by L2 latency, not bandwidth); kStageTokens tokens are staged per flush.
            const int ncg = ((pd.c.b_rows + 15) / 16) * 4;
            const int cg_lo = ncg * me / nred, cg_hi = ncg * (me + 1) / nred;
            const int up_off = (p.n_tile >> 2) * kBlockM;               // float4 offset of the second accumulator
            constexpr int kElems = (kAccs == 1) ? 4 : 2;
            constexpr int kCgPerFlush = kStageTokens / 4;
            for (int f0 = cg_lo; f0 < cg_hi; f0 += kCgPerFlush) {
                const int f1 = min(cg_hi, f0 + kCgPerFlush);
                for (int c0 = f0 + chalf * kElems; c0 < f1; c0 += 2 * kElems) {
                    float4 g[kElems], u[kElems];
#pragma unroll
                    for (int e = 0; e < kElems; ++e) g[e] = u[e] = make_float4(0.f, 0.f, 0.f, 0.f);
                    for (int cb = cf; cb <= cl; cb += 4) {
                        float4 a[kElems][4], b[kElems][4];
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            const int cc = cb + q;
                            if (cc <= cl) {
                                // only the first contributor's share can begin before the tile: then its piece is a
                                // later unit of that CTA (slot 1); every other piece is a first unit (slot 0)
                                const int sl = (cc == cf && cf_early) ? 1 : 0;
                                const size_t who = PAIR ? (size_t)cc * 2 + rank : (size_t)cc;      // the CTA that parked the piece
                                const float4* part = reinterpret_cast<const float4*>(p.partials + (who * 2 + sl) * slot_floats) + row;
#pragma unroll
                                for (int e = 0; e < kElems; ++e) {
                                    if (c0 + e < f1) {
                                        a[e][q] = __ldcg(part + (size_t)(c0 + e) * kBlockM);
                                        if (kAccs == 2) b[e][q] = __ldcg(part + up_off + (size_t)(c0 + e) * kBlockM);
                                    }
                                }
                            }
                        }
#pragma unroll
                        for (int q = 0; q < 4; ++q) {
                            if (cb + q <= cl) {
#pragma unroll
                                for (int e = 0; e < kElems; ++e) {
                                    if (c0 + e < f1) {
                                        g[e].x += a[e][q].x; g[e].y += a[e][q].y; g[e].z += a[e][q].z; g[e].w += a[e][q].w;
                                        if (kAccs == 2) { u[e].x += b[e][q].x; u[e].y += b[e][q].y; u[e].z += b[e][q].z; u[e].w += b[e][q].w; }
                                    }
                                }
                            }
                        }
                    }
#pragma unroll
                    for (int e = 0; e < kElems; ++e) {
                        if (c0 + e >= f1) break;
                        const float gf[4] = {g[e].x, g[e].y, g[e].z, g[e].w}, uf[4] = {u[e].x, u[e].y, u[e].z, u[e].w};
#pragma unroll
                        for (int k = 0; k < 4; ++k) {
                            const int tl = (c0 + e - f0) * 4 + k;
                            if (MODE == kGateUp) stage_put(tl, row, silu_f32(gf[k]) * uf[k]);
                            else {
                                stage_put(tl, row, gf[k]);
                                if (MODE == kLinear2) stage_put(tl, row + kBlockM, uf[k]);
                            }
                        }
                    }
                }
                stage_flush(pd.c, pd.c.b_row0 + f0 * 4, (f1 - f0) * 4);
            }
            asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads) : "memory");
            if (etid == 0) {
                const int done = atomicAdd(&p.counters[kStreamKMaxTiles + ctile(pd.tile)], 1);
                if (done == nred - 1) {   // every reducer has read what it needs: clean up for the next launch
                    p.counters[ctile(pd.tile)] = 0;
                    p.counters[kStreamKMaxTiles + ctile(pd.tile)] = 0;
                }
            }
        };

        // (every exit from this loop is decided on a predicate OR-ed across the four epilogue warps: the loop body holds
        // barriers, and a warp that left alone would leave the others waiting at one for good)
        while (cur.next(wu)) {
            if (bar_or(2, kEpiThreads, bars->abort != 0)) { gave_up = true; break; }
            const TileCoord c = tiles.get(wu.tile);
            if (wu.slot < 0 && npend > 0) {
                // shared tiles come first: before waiting for the first whole tile, finish this CTA's part
                // of the shared tiles (the main loop of the whole tile runs meanwhile)
                for (int i = 0; i < npend && !gave_up; ++i) run_reduce(pend[i]);
                npend = 0;
                if (gave_up) break;
            }
            const bool full_ok = mbar_wait(&bars->tmem_full[buf], acc_ph);
            if (bar_or(2, kEpiThreads, !full_ok)) {
                if (etid == 0) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); }
                gave_up = true;
                break;
            }
            tc_fence_after();
            const uint32_t t0 = tmem_base + ((uint32_t)(lane_grp * 32) << 16) + (uint32_t)(buf * acc_cols);
            if (wu.slot < 0) {
                // ---- whole K range in this CTA: epilogue straight from TMEM, kStageTokens token columns per round
                for (int tc = 0; tc < c.b_rows; tc += kStageTokens) {
                    const int ntok = min(kStageTokens, c.b_rows - tc);
                    for (int c0 = 16 * chalf; c0 < ntok; c0 += 32) {
                        uint32_t g[16];
                        tmem_ld_32x32b_x16(t0 + (uint32_t)(tc + c0), g);
                        if (MODE != kLinear) {
                            uint32_t u[16];
                            tmem_ld_32x32b_x16(t0 + (uint32_t)(p.n_tile + tc + c0), u);
                            tmem_ld_wait();
#pragma unroll
                            for (int j = 0; j < 16; ++j) {
                                if (MODE == kGateUp) stage_put(c0 + j, row, silu_f32(__uint_as_float(g[j])) * __uint_as_float(u[j]));
                                else { stage_put(c0 + j, row, __uint_as_float(g[j])); stage_put(c0 + j, row + kBlockM, __uint_as_float(u[j])); }
                            }
                        } else {
                            tmem_ld_wait();
#pragma unroll
                            for (int j = 0; j < 16; ++j) stage_put(c0 + j, row, __uint_as_float(g[j]));
                        }
                    }
                    if (tc + kStageTokens >= c.b_rows) {
                        // the accumulator has been read in full: hand the TMEM buffer back before the stores
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) release_tmem(buf);
                    }
                    stage_flush(c, c.b_row0 + tc, ntok);
                }
            } else {
                // ---- partial K range: park the fp32 accumulator as [column group of 4][row] float4 (a warp
                //      stores / loads 512 contiguous bytes per instruction); the last arriver finishes the tile
                uint4* mine = reinterpret_cast<uint4*>(p.partials + ((size_t)blockIdx.x * 2 + wu.slot) * slot_floats) + row;
                for (int c0 = 16 * chalf; c0 < cols; c0 += 32) {
                    if ((c0 % p.n_tile) >= c.b_rows) continue;   // token columns beyond the tile's valid rows
                    uint32_t g[16];
                    tmem_ld_32x32b_x16(t0 + (uint32_t)c0, g);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; j += 4)
                        mine[(size_t)((c0 + j) >> 2) * kBlockM] = make_uint4(g[j], g[j + 1], g[j + 2], g[j + 3]);
                }
                tc_fence_before();
                __syncwarp();
                if (lane == 0) release_tmem(buf);   // TMEM buffer is free again
                // publish: all 128 rows stored (CTA barrier), then one thread releases them device-wide
                // and bumps the tile counter.  The reduction itself is deferred (see run_reduce).
                asm volatile("bar.sync 2, %0;" ::"n"(kEpiThreads) : "memory");
                if (etid == 0) {
                    if (tr) tr[6] = global_timer_ns();               // partial stored, about to publish
                    __threadfence();
                    atomicAdd(&p.counters[ctile(wu.tile)], 1);
                    if (tr) tr[7] = global_timer_ns();               // published
                }
                pend[npend].tile = wu.tile;
                pend[npend].c = c;
                ++npend;
            }
            if (++buf == p.nbuf) { buf = 0; acc_ph ^= 1; }
        }
        for (int i = 0; i < npend && !gave_up; ++i) run_reduce(pend[i]);
    }

    if (tr && threadIdx.x == 64) tr[5] = global_timer_ns();          // epilogue finished
    tc_fence_before();
    // A pair leaves together: the peer's shared memory, barriers and TMEM are in use until both are done.
    if (PAIR) cluster_sync_all();
    else __syncthreads();
    if (warp == 1) {
        tc_fence_after();
        if (PAIR) tmem_dealloc_pair(tmem_base, (uint32_t)p.tmem_cols);
        else tmem_dealloc(tmem_base, (uint32_t)p.tmem_cols);
    }
}

// ----------------------------------------------------------------------------------------- host side
static int round_up(int a, int b) { return (a + b - 1) / b * b; }

// Token-tile width: the fewest tiles of at most 256 rows, all of (nearly) the same width, so that
// e.g. 384 rows become 192 + 192 rather than 256 + 128.
constexpr int kGroupedWideRowsLinear = 128, kGroupedWideRowsGateUp = 512;
static int pick_n_tile(int rows_max) {
    const int rows = rows_max < 16 ? 16 : rows_max;
    const int tiles = (rows + 255) / 256;
    const int n = round_up((rows + tiles - 1) / tiles, 16);
    return n > 256 ? 256 : n;
}

struct GemmConfig {
    GemmParams p;
    bool pair;          // CTA pairs (cta_group::2): a 256-weight-row tile per pair, half of the token rows loaded by each CTA
    size_t smem_bytes;
    size_t partial_bytes;
    int grid;
};

// Shared-memory budget of a CTA in the few-tiles (weight-streaming) regime.  Half of the SM, so the
// first CTAs of the next kernel in the stream can become resident (and prefetch weights) while this
// kernel's CTAs are still in their epilogue.  AFLEX_GEMM_SMEM_KB overrides it (tuning).
static int streaming_smem_budget() {
    static int kb = -1;
    if (kb < 0) {
        const char* e = getenv("AFLEX_GEMM_SMEM_KB");
        kb = e ? atoi(e) : 150;
        if (kb < 48) kb = 48;
        if (kb > 227) kb = 227;
    }
    return kb * 1024;
}

// Plain linear GEMMs take two weight-row tiles per CTA tile (kLinear2) when the activation tile is as
// large as a weight tile's K slice or close to it (64..128 token rows) and the weight matrix is large:
// the activation bytes that go from L2 to shared memory per weight byte are halved.  AFLEX_GEMM_DUAL = 0 / 1 forces it off / on (tuning).
// CTA pairs pay where the activation tile takes a large part of a pipeline stage, so that too few weight bytes are in
// flight per SM to cover the DRAM latency: from this token-tile width on (dense form).  AFLEX_GEMM_PAIR: 0 = never,
// n >= 16 = from n token rows per tile on (tuning).
static int pair_from_rows() {
    static int v = -1;
    if (v < 0) { const char* e = getenv("AFLEX_GEMM_PAIR"); v = e ? atoi(e) : 192; }
    return v;
}
static bool use_pair(int T, int N, int E, int num_sms) {
    const int from = pair_from_rows();
    return from >= 16 && E == 0 && pick_n_tile(T) >= from && N >= 2 * kBlockM && num_sms >= 2;
}

static int linear_mode(int T, int N, int K) {
    static int force = -2;
    if (force == -2) { const char* e = getenv("AFLEX_GEMM_DUAL"); force = e ? atoi(e) : -1; }
    if (N < 2 * kBlockM) return kLinear;
    if (force == 0) return kLinear;
    if (force == 1) return kLinear2;
    const int n_tile = pick_n_tile(T);
    if (pair_from_rows() >= 16 && n_tile >= pair_from_rows()) return kLinear;   // the pair form halves the activation bytes itself
    // measured at the Qwen3-32B shapes: pays on the long down projection (70.6 -> 66.3 us at 128 rows), not on
    // the short W_o / QKV projections, whose time is fixed cost rather than streaming
    return (n_tile >= 64 && n_tile <= 128 && (long long)N * K >= (64LL << 20)) ? kLinear2 : kLinear;
}

static bool make_config(int mode, int T, int N, int K, int rows_max, int E, int num_sms, GemmConfig* cfg, bool out_f32 = false) {
    GemmParams& p = cfg->p;
    p.T = T; p.N = N; p.K = K;
    p.n_tile = pick_n_tile(rows_max);
    // Grouped form: cap the tile at 128 token rows so the two gate/up accumulators stay double-buffered
    // in TMEM; a hot expert with more rows becomes two adjacent tiles whose weight tiles are read by
    // neighbouring CTAs at the same time (the second read is an L2 hit).
    // That is the decode regime (tens of rows per expert).  With hundreds of rows per expert (prefill) the grouped
    // form is a tensor-core kernel like the dense one, and a 128-row tile's MMAs read as many shared-memory bytes per
    // cycle as the SM delivers.  Measured at the Mixtral shape: the down projection (one accumulator, still double-
    // buffered at 256 rows) gains from an average of 128 rows per expert on (328 -> 289 us at 256, 2388 -> 1582 us at
    // 2048); gate/up (two accumulators: 256 rows fill TMEM, no double buffering) only from about 512 on
    // (536 -> 593 us at 256 rows per expert, 3612 -> 3384 us at 2048).  AFLEX_GEMM_GROUP_WIDE overrides both (tuning).
    {
        static int wide = -1;
        if (wide < 0) { const char* e = getenv("AFLEX_GEMM_GROUP_WIDE"); wide = e ? atoi(e) : 0; }
        const int from = wide > 0 ? wide : (mode == kGateUp ? kGroupedWideRowsGateUp : kGroupedWideRowsLinear);
        if (E > 0 && p.n_tile > 128 && T / E < from) p.n_tile = 128;
    }
    {
        static int cap = -1;
        if (cap < 0) { const char* e = getenv("AFLEX_GEMM_NTILE_CAP"); cap = e ? atoi(e) : 0; }
        if (cap >= 16 && p.n_tile > cap) p.n_tile = cap / 16 * 16;
    }
    cfg->pair = mode != kLinear2 && use_pair(rows_max, N, E, num_sms) && p.n_tile >= pair_from_rows();
    p.tile_rows = (mode == kLinear2 || cfg->pair) ? 2 * kBlockM : kBlockM;
    p.m_tiles = (N + p.tile_rows - 1) / p.tile_rows;
    p.n_tiles = (T + p.n_tile - 1) / p.n_tile;
    p.kblocks = (K + kBlockK - 1) / kBlockK;
    p.num_experts = E;
    {
        // Measured: the dense form is fastest with evict-first weights at every token count (the token
        // tiles of one weight tile run side by side); the grouped form gains 3 % on the loaded
        // Mixtral-shaped configuration from normal priority when an expert's rows can span two chunks.
        // AFLEX_GEMM_WPOL = 0 / 1 forces evict-first / normal (tuning).
        static int pol = -1;
        if (pol < 0) { const char* e = getenv("AFLEX_GEMM_WPOL"); pol = e ? atoi(e) : 2; }
        p.w_reuse = pol == 2 ? ((E > 0 && rows_max > p.n_tile) ? 1 : 0) : (pol ? 1 : 0);
    }
    // upper bound on tiles (exact for the non-grouped form; the grouped form knows its tile count
    // only on the device: every expert can add one ragged chunk)
    const long long tiles_hi = (E == 0) ? (long long)p.m_tiles * p.n_tiles
                                        : (long long)p.m_tiles * ((T + p.n_tile - 1) / p.n_tile + E);
    const int accs = (mode == kLinear ? 1 : 2);
    const int acc_cols = accs * p.n_tile;
    p.nbuf = (2 * acc_cols <= 512) ? 2 : 1;
    int cols = 32;
    while (cols < p.nbuf * acc_cols) cols <<= 1;
    p.tmem_cols = cols;
    const int a_bytes = accs * kBlockM * kBlockK * 2;
    const int stage_bytes = a_bytes + round_up((cfg->pair ? p.n_tile / 2 : p.n_tile) * kBlockK * 2, 1024);
    // few tiles per SM: share the remainder tiles along K; many: whole tiles round-robin.  Wide tiles
    // (large T, compute-bound) make the shared tiles' partials big, so they are shared only when whole
    // tiles alone would leave most SMs idle.
    static int nostream = -1;   // AFLEX_GEMM_NOSTREAMK=1: whole tiles only (measurement of per-SM streaming rates)
    if (nostream < 0) { const char* e = getenv("AFLEX_GEMM_NOSTREAMK"); nostream = e ? atoi(e) : 0; }
    const long long workers = cfg->pair ? num_sms / 2 : num_sms;      // CTAs, or CTA pairs, that share the tile list
    // ... or, for the dense single-accumulator form (128 KB partials, double-buffered TMEM), when whole tiles in rounds
    // would leave more than a tenth of the last round's CTAs idle: the down projection at 2048 tokens is 160 tiles on 74
    // pairs, three rounds for 2.16 rounds of work (465 -> 380 us with the remainder shared along K).  Gate/up (two
    // accumulators: 256 KB partials, no second buffer) and the grouped form measured slower that way.
    // AFLEX_GEMM_STREAMK_WIDE=0 switches it off (tuning).
    static int wide_sk = -1;
    if (wide_sk < 0) { const char* e = getenv("AFLEX_GEMM_STREAMK_WIDE"); wide_sk = e ? atoi(e) : 1; }
    const long long rounds = (tiles_hi + workers - 1) / workers;
    const bool wide_share = wide_sk != 0 && E == 0 && mode == kLinear && tiles_hi * 10 < rounds * workers * 9;
    p.streamk = nostream ? 0 : (tiles_hi < 8LL * workers && tiles_hi <= kStreamKMaxTiles && (p.n_tile <= 128 || wide_share || tiles_hi < 2LL * workers)) ? 1 : 0;
    // epilogue staging: kStageTokens token rows of the tile in the output type
    const int stage_out_bytes = kStageTokens * (mode == kLinear2 ? 2 : 1) * kBlockM * (out_f32 ? 4 : 2);
    int cap = (p.streamk && p.n_tile <= 64 && mode != kLinear2) ? streaming_smem_budget() + stage_out_bytes : kMaxDynamicSmem;
    if (cap > kMaxDynamicSmem) cap = kMaxDynamicSmem;
    const int budget = cap - 1024 /*alignment slack*/ - (int)sizeof(GemmBarriers) - 256 - stage_out_bytes;
    int stages = budget / stage_bytes;
    if (stages > kMaxStages) stages = kMaxStages;
    if (stages < 2) stages = 2;
    p.stages = stages;
    cfg->smem_bytes = (size_t)stages * stage_bytes + sizeof(GemmBarriers) + 1024 + 256 + stage_out_bytes;
    if (cfg->smem_bytes > (size_t)kMaxDynamicSmem) return false;
    long long units = tiles_hi * p.kblocks;
    if (cfg->pair) {
        const int pairs = num_sms / 2;
        cfg->grid = 2 * (int)(units < pairs ? units : pairs);
        if (2 * tiles_hi > kStreamKMaxTiles) return false;             // each CTA of a pair has its own tile counters
    } else {
        cfg->grid = (int)(units < num_sms ? units : num_sms);
    }
    if (cfg->grid < 1) cfg->grid = 1;
    cfg->partial_bytes = p.streamk ? align256((size_t)cfg->grid * 2 * accs * p.n_tile * kBlockM * sizeof(float)) : 0;
    return true;
}

static bool encode_b_set(TmapSetB* set, const void* base, uint64_t rows, uint64_t K, int n_tile, bool pair = false) {
    for (int i = 0; i < 5; ++i) {
        uint32_t box = (uint32_t)((16 << i) < n_tile ? (16 << i) : n_tile);   // same rule as box_rows()
        if (pair) box >>= 1;                                                  // each CTA of a pair loads half of the rows
        if (!encode_tmap_2d_bf16(&set->m[i], base, rows, K, K * 2, box, kBlockK, false)) return false;
    }
    return true;
}

template <int MODE, bool PAIR = false>
static aflex_status launch_gemm(aflex_ctx* ctx, const GemmConfig& cfg, const CUtensorMap& ta0, const CUtensorMap& ta1,
                                const TmapSetB& tb, cudaStream_t st, int kind) {
    if (!ctx->gemm_attr_set[MODE + (PAIR ? 3 : 0)]) {
        cudaError_t e = cudaFuncSetAttribute(gemm_kernel<MODE, PAIR>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                             kMaxDynamicSmem);
        if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(gemm)");
        ctx->gemm_attr_set[MODE + (PAIR ? 3 : 0)] = true;
    }
    KernelScope scope(ctx, kind, st);
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)cfg.grid);
    lc.blockDim = dim3(kGemmThreads);
    lc.dynamicSmemBytes = cfg.smem_bytes;
    lc.stream = st;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    if (PAIR) {
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = 2;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        lc.numAttrs = 2;
    }
    return check_cuda(ctx, cudaLaunchKernelEx(&lc, gemm_kernel<MODE, PAIR>, ta0, ta1, tb, cfg.p), "gemm_kernel launch");
}

static aflex_status bind_scratch(aflex_ctx* ctx, GemmConfig& cfg, char* ws, size_t ws_bytes, int* counters,
                                 const char* who) {
    GemmParams& p = cfg.p;
    p.status = ctx->dev_status;
    p.trace = ctx->trace ? ctx->trace + (size_t)(ctx->trace_slot++ % kTraceKernels) * kTraceStride : nullptr;
    p.counters = counters;
    p.partials = nullptr;
    if (p.streamk) {
        if (cfg.partial_bytes > ws_bytes || ws == nullptr)
            return set_error(ctx, AFLEX_ERR_WORKSPACE, "%s: need %zu workspace bytes, have %zu", who, cfg.partial_bytes, ws_bytes);
        p.partials = reinterpret_cast<float*>(ws);
    }
    return AFLEX_OK;
}

size_t linear_workspace_bytes(int T, int K, int N, int num_sms) {
    GemmConfig cfg;
    if (!make_config(linear_mode(T, N, K), T, N, K, T, 0, num_sms, &cfg)) return 0;
    return cfg.partial_bytes;
}

aflex_status linear_launch(aflex_ctx* ctx, const void* x, const void* w, int T, int K, int N, void* y, char* ws,
                           size_t ws_bytes, cudaStream_t st, int kind, int* counters) {
    GemmConfig cfg;
    const int mode = linear_mode(T, N, K);
    if (!make_config(mode, T, N, K, T, 0, ctx->num_sms, &cfg))
        return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "linear: no tile configuration fits");
    GemmParams& p = cfg.p;
    p.offsets = nullptr;
    p.out_f32 = nullptr;
    p.out_bf16 = reinterpret_cast<__nv_bfloat16*>(y);
    aflex_status s = bind_scratch(ctx, cfg, ws, ws_bytes, counters, "linear");
    if (s != AFLEX_OK) return s;
    CUtensorMap ta;
    TmapSetB tb;
    if (!encode_tmap_2d_bf16(&ta, w, (uint64_t)N, (uint64_t)K, (uint64_t)K * 2, kBlockM, kBlockK, true) ||
        !encode_b_set(&tb, x, (uint64_t)T, (uint64_t)K, p.n_tile, cfg.pair))
        return set_error(ctx, AFLEX_ERR_CUDA, "linear: cuTensorMapEncodeTiled failed");
    if (cfg.pair) return launch_gemm<kLinear, true>(ctx, cfg, ta, ta, tb, st, kind);
    if (mode == kLinear2) return launch_gemm<kLinear2>(ctx, cfg, ta, ta, tb, st, kind);
    return launch_gemm<kLinear>(ctx, cfg, ta, ta, tb, st, kind);
}

size_t gateup_workspace_bytes(int T, int H, int I, int num_sms) {
    GemmConfig cfg;
    if (!make_config(kGateUp, T, I, H, T, 0, num_sms, &cfg)) return 0;
    return cfg.partial_bytes;
}

aflex_status gateup_launch(aflex_ctx* ctx, const void* x, const void* w_gate, const void* w_up, int T, int H, int I,
                           void* h, char* ws, size_t ws_bytes, cudaStream_t st, int* counters) {
    GemmConfig cfg;
    if (!make_config(kGateUp, T, I, H, T, 0, ctx->num_sms, &cfg))
        return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "gate/up: no tile configuration fits");
    GemmParams& p = cfg.p;
    p.offsets = nullptr;
    p.out_f32 = nullptr;
    p.out_bf16 = reinterpret_cast<__nv_bfloat16*>(h);
    aflex_status s = bind_scratch(ctx, cfg, ws, ws_bytes, counters, "gate/up");
    if (s != AFLEX_OK) return s;
    CUtensorMap tg, tu;
    TmapSetB tb;
    if (!encode_tmap_2d_bf16(&tg, w_gate, (uint64_t)I, (uint64_t)H, (uint64_t)H * 2, kBlockM, kBlockK, true) ||
        !encode_tmap_2d_bf16(&tu, w_up, (uint64_t)I, (uint64_t)H, (uint64_t)H * 2, kBlockM, kBlockK, true) ||
        !encode_b_set(&tb, x, (uint64_t)T, (uint64_t)H, p.n_tile, cfg.pair))
        return set_error(ctx, AFLEX_ERR_CUDA, "gate/up: cuTensorMapEncodeTiled failed");
    if (cfg.pair) return launch_gemm<kGateUp, true>(ctx, cfg, tg, tu, tb, st, kKGateUpGemm);
    return launch_gemm<kGateUp>(ctx, cfg, tg, tu, tb, st, kKGateUpGemm);
}

size_t grouped_workspace_bytes(int mode_gateup, int rows_total, int rows_max, int K, int N, int E, int num_sms) {
    GemmConfig cfg;
    if (!make_config(mode_gateup ? kGateUp : kLinear, rows_total, N, K, rows_max, E, num_sms, &cfg, !mode_gateup)) return 0;
    return cfg.partial_bytes;
}

aflex_status grouped_gateup_launch(aflex_ctx* ctx, const void* xp, const void* w_gate, const void* w_up,
                                   const int32_t* offsets, int rows_total, int rows_max, int H, int I, int E,
                                   void* hp, char* ws, size_t ws_bytes, cudaStream_t st, int* counters) {
    if (E > kMaxExperts) return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "num_experts > %d", kMaxExperts);
    GemmConfig cfg;
    if (!make_config(kGateUp, rows_total, I, H, rows_max, E, ctx->num_sms, &cfg))
        return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "grouped gate/up: no tile configuration fits");
    GemmParams& p = cfg.p;
    p.offsets = offsets;
    p.out_f32 = nullptr;
    p.out_bf16 = reinterpret_cast<__nv_bfloat16*>(hp);
    aflex_status s = bind_scratch(ctx, cfg, ws, ws_bytes, counters, "grouped gate/up");
    if (s != AFLEX_OK) return s;
    CUtensorMap tg, tu;
    TmapSetB tb;
    if (!encode_tmap_2d_bf16(&tg, w_gate, (uint64_t)E * I, (uint64_t)H, (uint64_t)H * 2, kBlockM, kBlockK, true) ||
        !encode_tmap_2d_bf16(&tu, w_up, (uint64_t)E * I, (uint64_t)H, (uint64_t)H * 2, kBlockM, kBlockK, true) ||
        !encode_b_set(&tb, xp, (uint64_t)rows_total, (uint64_t)H, p.n_tile))
        return set_error(ctx, AFLEX_ERR_CUDA, "grouped gate/up: cuTensorMapEncodeTiled failed");
    return launch_gemm<kGateUp>(ctx, cfg, tg, tu, tb, st, kKMoeGateUpGemm);
}

aflex_status grouped_linear_launch(aflex_ctx* ctx, const void* hp, const void* w_down, const int32_t* offsets,
                                   int rows_total, int rows_max, int K, int N, int E, float* yp, char* ws,
                                   size_t ws_bytes, cudaStream_t st, int* counters) {
    if (E > kMaxExperts) return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "num_experts > %d", kMaxExperts);
    GemmConfig cfg;
    if (!make_config(kLinear, rows_total, N, K, rows_max, E, ctx->num_sms, &cfg, true))
        return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "grouped linear: no tile configuration fits");
    GemmParams& p = cfg.p;
    p.offsets = offsets;
    p.out_bf16 = nullptr;
    p.out_f32 = yp;
    aflex_status s = bind_scratch(ctx, cfg, ws, ws_bytes, counters, "grouped linear");
    if (s != AFLEX_OK) return s;
    CUtensorMap ta;
    TmapSetB tb;
    if (!encode_tmap_2d_bf16(&ta, w_down, (uint64_t)E * N, (uint64_t)K, (uint64_t)K * 2, kBlockM, kBlockK, true) ||
        !encode_b_set(&tb, hp, (uint64_t)rows_total, (uint64_t)K, p.n_tile))
        return set_error(ctx, AFLEX_ERR_CUDA, "grouped linear: cuTensorMapEncodeTiled failed");
    return launch_gemm<kLinear>(ctx, cfg, ta, ta, tb, st, kKMoeDownGemm);
}

}  // namespace aflex
