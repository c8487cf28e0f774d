// Attention side: paged grouped-query decode attention as a persistent, balanced split-KV kernel.
//
// The operator is bound by streaming the KV cache from HBM once (the paper's Sections 1-2:
// decode attention is memory-bound on KV-cache reads), so the kernel is organised around
// keeping many page loads in flight on every SM for the whole launch and touching every K/V
// byte exactly once for all G = Hq/Hkv query heads of a group.
//
//   work        = the list of 64-token units (4 pages) of every (sequence, KV head) item, in
//                 (sequence, head, unit) order.  It is cut into one contiguous, equal share per CTA
//                 (2 CTAs per SM), located on the device from the sequence lengths: no host plan,
//                 no wave quantisation, no per-chunk launch overhead.  A CTA's share is a run of
//                 "pieces": unit ranges of consecutive items.
//   data path   = a producer warp walks the share and issues tiled TMA loads (128-byte swizzle) of
//                 whole pages (a page's K or V slab for one KV head is a contiguous [16][D] block)
//                 into a 3-stage mbarrier ring of 4-page stages; page ids are fetched one unit
//                 ahead.  The ring never drains between pieces.
//   arithmetic  = mma.sync m16n8k16 (bf16 -> fp32) with the 16 tokens of a page as the M dimension
//                 and the (<= 8) heads of the group as the N dimension, so no rows are wasted on
//                 padding: S^T = K Q^T, then O^T += V^T P^T with P^T obtained from the S^T
//                 accumulator by movmatrix.  The flop/byte ratio (8 at G = 8) is above what the
//                 fp32 pipes sustain at full HBM rate, which is the only reason MMAs are used.
//   softmax     = online, fp32, base-2 exponentials; each of the 4 compute warps owns one page of a
//                 unit and its own running (m, l, O).  At the last unit of a piece every compute warp
//                 parks its state in its own K/V pages of that stage and goes on to the next piece
//                 without waiting; an epilogue warp that walks the same pieces folds the four states
//                 (fixed order), releases the stage and does everything that touches global memory.
//   combine     = a piece that covers its whole item is written straight to the output.  Otherwise
//                 the piece's unnormalised (O, m, l) goes to one of the range's two partial slots and
//                 the item's arrival counter is bumped; the warp that arrives last merges the item's
//                 pieces, always in list order, so the result does not depend on which was last.
//   tail        = on launches large enough for one 16-unit chunk per CTA, the last quarter of the
//                 list is handed out as ticket-claimed chunks, so faster CTAs take more.
//
// Unreferenced slots (beyond a sequence's length) may hold NaN: scores of such tokens are
// replaced (not multiplied) by -inf and their V rows are zeroed in shared memory before use.
#include <cuda_bf16.h>
#include <math.h>
#include <stdlib.h>

#include "internal.h"
#include "ptx.cuh"

namespace aflex {

constexpr int kPage = 16;
constexpr int kPagesPerStage = 4;
constexpr int kUnitTokens = kPage * kPagesPerStage;   // 64
constexpr int kAttnStages = 3;
constexpr int kAttnConsumerWarps = 4;
constexpr int kAttnThreads = (kAttnConsumerWarps + 2) * 32;   // compute warps, producer warp, epilogue warp
constexpr float kNegBig = -1.0e30f;

struct AttnParams {
    const __nv_bfloat16* q;
    const int32_t* page_table;
    const int32_t* seq_lens;
    int batch;
    int max_pages;
    int Hq, Hkv, G;
    long long num_pages;
    float scale_log2;      // sm_scale * log2(e)
    float* o_part;         // [grid][2 slots][8 heads][D]  unnormalised sum_j p_j v_j of a piece
    float* ml_part;        // [grid][2 slots][8 heads][2]  (running max in log2 units, sum of p)
    __nv_bfloat16* out;    // [B][Hq][D]
    float* lse;            // [B][Hq] or nullptr
    int* counters;         // [B][Hkv] piece-arrival counters, zero on entry and on exit
    int* ticket;           // [2]: next dynamic chunk, CTAs finished; zero on entry and on exit, not shared with the launches
                           // next to this one in the stream (unused if dyn_pct == 0)
    int dyn_pct;           // percent of the unit list handed out dynamically (0 = static shares only)
    int dyn_chunks;        // target number of dynamic chunks per CTA
    int kv_policy;         // 0: evict-first KV loads, 1: normal priority (tuning)
    int q_final;           // 1: q is final when the kernel starts (its first loads need not wait for the grid dependency)
    int dyn_min;           // chunk size (units) the dynamic tail aims at
    int piece_cost;        // list positions charged per item start (balances the fixed cost of a piece)
    int* status;
    unsigned long long* trace;
};

// A contiguous run of the unit list handed to a CTA: its static share (rid = CTA index) or a
// dynamically claimed chunk (rid = grid + chunk index).  x0 == x1 ends the CTA's work.
struct AttnRange {
    long long x0, x1;        // unit positions
    long long prefix;        // units (per KV head) of the sequences before b
    int b;                   // sequence that contains x0
    int rid;                 // partial-slot owner id of the range
};
constexpr int kRangeRing = 4;

struct __align__(8) AttnShared {
    uint64_t full[kAttnStages];
    uint64_t empty[kAttnStages];
    uint64_t xready[kAttnStages];   // the compute warps' states of a finished piece are parked in this stage
    uint64_t rng_ready[kRangeRing];
    AttnRange rng[kRangeRing];
    volatile int abort;
    int scan[kAttnThreads];  // exclusive prefix (units per KV head) of the sequences before each thread's segment
};

// A sequence length as the kernel uses it: never beyond what the page-table row can address (a
// longer value would walk off the row).  Out-of-range lengths are reported by the prologue.
__device__ __forceinline__ int usable_len(int raw, int max_pages) {
    const int cap = max_pages * kPage;
    return raw < 0 ? 0 : (raw > cap ? cap : raw);
}

// Position in the (sequence, head, unit) list; every warp of a CTA walks the same sequence of pieces.
// The list is "virtual": every item is preceded by `cost` empty positions, so that cutting the list
// into equal shares balances units AND item starts (each start costs a warp merge, a publish, maybe a
// cross-CTA merge).  Position u of an item is real unit u - cost; positions below `cost` hold no work.
struct Walker {
    const int32_t* lens;
    int Hkv, cost, max_pages;
    long long pos, end;   // unit positions in the global list
    long long prefix;     // units (per head) of the sequences before b
    int b, g, u, nu, len;
    __device__ void init(const AttnParams& p, const AttnRange& r) {
        lens = p.seq_lens; Hkv = p.Hkv; cost = p.piece_cost; max_pages = p.max_pages; pos = r.x0; end = r.x1;
        b = r.b; prefix = r.prefix;
        len = usable_len(lens[b], max_pages); nu = (len + kUnitTokens - 1) / kUnitTokens + cost;
        const long long rel = pos - prefix * Hkv;
        if (nu > 0) { g = (int)(rel / nu); u = (int)(rel % nu); }
        else { g = 0; u = 0; }                  // an item without any position (length 0, cost 0): skip_empty() steps over it
    }
    __device__ bool done() const { return pos >= end; }
    // Step over list positions that hold no work: the `cost` empty positions charged in front of every item,
    // and items that have no position at all (a sequence whose usable length is 0 when cost is 0).
    __device__ void skip_empty() {
        while (!done()) {
            if (u < cost) advance(1);
            else if (u >= nu) advance(0);
            else break;
        }
    }
    // advance by n units inside the current item, moving to the next item / sequence when it ends
    __device__ void advance(int n) {
        pos += n; u += n;
        if (u >= nu) {
            u = 0;
            if (++g == Hkv) {
                g = 0; prefix += nu; ++b;
                if (pos < end) { len = usable_len(lens[b], max_pages); nu = (len + kUnitTokens - 1) / kUnitTokens + cost; }
            }
        }
    }
};

// How the unit list [0, U) is handed out: [0, U1) as one static share per CTA (Ge1 CTAs take part),
// [U1, U) as n2 chunks of K2 units claimed through a ticket counter by whichever CTA is free.
struct AttnSplit {
    long long U, U1;
    int Ge1, K2, n2;
    // dyn_pct: share of the list handed out dynamically; dyn_chunks: most chunks per CTA (bounds the partial
    // slots); dyn_units: chunk size aimed at.  A chunk costs a claim, a hand-over and an extra partial piece
    // to publish and merge, so chunks stay at dyn_units or more, and the tail is dynamic only when it yields
    // at least one chunk per CTA (small launches stay purely static).
    __device__ AttnSplit(long long U_, int grid, int dyn_pct, int dyn_chunks, int dyn_units = 16) {
        U = U_;
        long long U2 = dyn_pct > 0 ? U * dyn_pct / 100 : 0;
        K2 = 1; n2 = 0;
        if (U2 > 0) {
            long long k = (U2 + (long long)dyn_chunks * grid - 1) / ((long long)dyn_chunks * grid);
            if (k < dyn_units) k = dyn_units;
            if (k > (1 << 20)) k = 1 << 20;
            K2 = (int)k;
            n2 = (int)((U2 + K2 - 1) / K2);
            if (n2 < grid) { U2 = 0; n2 = 0; K2 = 1; }
        }
        U1 = U - U2;
        Ge1 = (int)min((long long)grid, U1);
    }
};

__device__ __forceinline__ long long share_begin(long long U, int c, int Ge) { return U * c / Ge; }
__device__ __forceinline__ int cta_of_unit(long long x, long long U, int Ge) {
    int c = (int)((x * Ge) / U);
    if (c >= Ge) c = Ge - 1;
    while (c > 0 && share_begin(U, c, Ge) > x) --c;
    while (c + 1 < Ge && share_begin(U, c + 1, Ge) <= x) ++c;
    return c;
}

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 2)
attn_decode_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                   const AttnParams p) {
    constexpr int kHalves = D / 64;                 // 128-byte column blocks per row
    constexpr int kPageBytes = kPage * D * 2;       // one page of K (or V) for one KV head
    constexpr int kQBytes = 8 * D * 2;              // the (at most 8) query heads of one group: the block behind the pages
    constexpr int kStageBytes = 2 * kPagesPerStage * kPageBytes + kQBytes;
    constexpr int kOpsPerStage = 2 * kPagesPerStage * kHalves;
    constexpr int kKSteps = D / 16;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    AttnShared* sh = reinterpret_cast<AttnShared*>(smem + kAttnStages * kStageBytes);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;
    const int cta = blockIdx.x;

    pdl_launch_dependents();
    unsigned long long* tr = (p.trace && cta < 4096) ? p.trace + (size_t)cta * 8 : nullptr;
    if (tr && threadIdx.x == 0) {
        tr[0] = global_timer_ns(); tr[3] = 0; tr[5] = 0;
        unsigned smid;
        asm volatile("mov.u32 %0, %%smid;" : "=r"(smid));
        tr[6] = smid;
    }
    if (threadIdx.x == 0) {
        for (int s = 0; s < kAttnStages; ++s) {
            mbar_init(&sh->full[s], 1);
            mbar_init(&sh->empty[s], kAttnConsumerWarps);
            mbar_init(&sh->xready[s], kAttnConsumerWarps);
        }
        for (int i = 0; i < kRangeRing; ++i) mbar_init(&sh->rng_ready[i], 1);
        sh->abort = 0;
        fence_mbar_init();
        prefetch_tmap(&tmap_k);
        prefetch_tmap(&tmap_v);
    }
    // The lengths and the page table are inputs of the step, never written by a kernel of this library,
    // so the plan (prefix scan, this CTA's share, its first page ids) is made while the preceding kernel
    // is still draining.  q and the KV cache may come from that kernel (the K/V append), and the partial
    // slots, counters and ticket may still be in use by an earlier attention launch: everything that
    // touches those waits for the grid dependency (pdl_wait below, per role).

    // ---- block-wide exclusive prefix over ceil(len/64): thread t owns sequences [t*per_thread, ...)
    const int per_thread = (p.batch + kAttnThreads - 1) / kAttnThreads;
    {
        const int b_lo = min(p.batch, (int)threadIdx.x * per_thread), b_hi = min(p.batch, b_lo + per_thread);
        int local = 0;
        for (int b = b_lo; b < b_hi; ++b) {
            const int raw = p.seq_lens[b];
            if ((raw < 1 || raw > p.max_pages * kPage) && cta == 0) atomicExch(p.status, AFLEX_ERR_BOUNDS);
            local += (usable_len(raw, p.max_pages) + kUnitTokens - 1) / kUnitTokens + p.piece_cost;
        }
        // inclusive warp scan, then warp totals through shared memory
        int incl = local;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const int v = __shfl_up_sync(0xffffffffu, incl, off);
            if (lane >= off) incl += v;
        }
        __shared__ int warp_tot[kAttnThreads / 32];
        if (lane == 31) warp_tot[warp] = incl;
        __syncthreads();
        int base = 0;
        for (int w = 0; w < warp; ++w) base += warp_tot[w];
        sh->scan[threadIdx.x] = base + incl - local;
        if (threadIdx.x == kAttnThreads - 1) sh->rng[0].x0 = base + incl;   // grand total, parked for everyone
        __syncthreads();
    }
    const long long U = sh->rng[0].x0 * (long long)p.Hkv;
    __syncthreads();
    const AttnSplit sp(U, (int)gridDim.x, p.dyn_pct, p.dyn_chunks, p.dyn_min);
    if (tr && threadIdx.x == 0) tr[1] = global_timer_ns();            // prefix ready

    // Sequence that contains unit position x (cooperative over the 32 lanes of one warp).
    auto locate = [&](long long x, int& b_out, long long& prefix_out) {
        int best = 0;
#pragma unroll
        for (int k = 0; k < kAttnThreads / 32; ++k) {
            const int t = lane * (kAttnThreads / 32) + k;
            if ((long long)sh->scan[t] * p.Hkv <= x) best = t;      // scan is non-decreasing
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) best = max(best, __shfl_xor_sync(0xffffffffu, best, off));
        int b = min(p.batch - 1, best * per_thread);
        long long pre = sh->scan[best];
        while (b + 1 < p.batch) {
            const int nu = (usable_len(p.seq_lens[b], p.max_pages) + kUnitTokens - 1) / kUnitTokens + p.piece_cost;
            if (x < (pre + nu) * p.Hkv) break;
            pre += nu; ++b;
        }
        b_out = b; prefix_out = pre;
    };

    if (warp == kAttnConsumerWarps) {
        // ------------------------------------------------------------------ producer warp
        const int pg = lane / (2 * kHalves);
        const int kv = (lane / kHalves) & 1;
        const int hf = lane % kHalves;
        const bool op_lane = lane < kOpsPerStage;
        auto page_id = [&](const Walker& w) -> int {
            const int idx = (w.u - w.cost) * kPagesPerStage + pg;
            return (op_lane && idx * kPage < w.len) ? p.page_table[(size_t)w.b * p.max_pages + idx] : 0;
        };
        const uint64_t pol_kv = p.kv_policy == 1 ? policy_evict_normal() : policy_evict_first();    // KV is read once: do not let it push reusable lines out of L2
        int s = 0;
        uint32_t ph = 0;
        int r = 0;                       // ranges published so far
        bool aborted = false;
        // range 0: the static share; later ranges: claimed chunks
        long long x0 = 0, x1 = 0;
        int rid = cta;
        if (cta < sp.Ge1) { x0 = share_begin(sp.U1, cta, sp.Ge1); x1 = share_begin(sp.U1, cta + 1, sp.Ge1); }
        int next_ticket = -1;
        // the static share's start, located before the grid dependency resolves
        AttnRange rg0;
        rg0.x0 = x0; rg0.x1 = x1; rg0.rid = rid; rg0.b = 0; rg0.prefix = 0;
        int pid0 = 0;
        if (x1 > x0) {
            locate(x0, rg0.b, rg0.prefix);
            Walker w0;
            w0.init(p, rg0);
            w0.skip_empty();
            pid0 = w0.done() ? 0 : page_id(w0);          // also warms the page-table line
        }
        // KV loads do not wait for the grid dependency: the only kernel of this library that writes the
        // cache (the K/V append) does not release its dependents early, so whatever precedes this launch
        // in the stream has left the cache final.  Neither do the chunk tickets: consecutive launches use
        // different ticket words (four pairs in rotation, picked by the host), and a launch cannot start
        // before the launch four back has completed, its words reset.
        bool waited = false;
        auto claim = [&]() {
            if (lane == 0) next_ticket = atomicAdd(&p.ticket[0], 1);
            next_ticket = __shfl_sync(0xffffffffu, next_ticket, 0);
        };
        bool first_range = true;
        while (true) {
            // claim the chunk after this range while the range streams (the round trip hides behind it);
            // in the first range only once the ring has been filled
            bool claimed = sp.n2 == 0;
            if (!claimed && !first_range) { claim(); claimed = true; }
            int issued = 0;
            if (x1 > x0) {
                AttnRange rg;
                if (first_range) { rg = rg0; }
                else { rg.x0 = x0; rg.x1 = x1; rg.rid = rid; locate(x0, rg.b, rg.prefix); }
                Walker wk;
                wk.init(p, rg);
                wk.skip_empty();                                         // positions without work
                // a range without any real unit is not handed to the consumers at all (every published
                // range then holds at least one ring stage, which is what bounds the range ring)
                if (!wk.done()) {
                    if (lane == 0) { sh->rng[r % kRangeRing] = rg; mbar_arrive(&sh->rng_ready[r % kRangeRing]); }
                    ++r;
                }
                int pid = wk.done() ? 0 : (first_range ? pid0 : page_id(wk));
                int piece_b = -1, piece_g = -1;           // item of the piece being loaded (a new range starts a new piece)
                while (!wk.done()) {
                    const int g = wk.g, u = wk.u - wk.cost, len = wk.len, b_now = wk.b;
                    const bool piece_start = (b_now != piece_b) || (g != piece_g);
                    piece_b = b_now; piece_g = g;
                    wk.advance(1);
                    wk.skip_empty();
                    const int pid_next = wk.done() ? 0 : page_id(wk);   // one unit ahead of the ring
                    if (!claimed && issued >= kAttnStages) { claim(); claimed = true; }
                    ++issued;
                    bool ok = mbar_wait(&sh->empty[s], ph ^ 1);
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok || sh->abort) {
                        if (lane == 0) { sh->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); }
                        aborted = true;
                        break;
                    }
                    const int np = min(kPagesPerStage, (len - u * kUnitTokens + kPage - 1) / kPage);
                    const uint32_t q_bytes = piece_start ? (uint32_t)(p.G * D * 2) : 0u;
                    if (lane == 0) mbar_expect_tx(&sh->full[s], (uint32_t)(np * 2 * kPageBytes) + q_bytes);
                    __syncwarp();
                    if (op_lane && pg < np) {
                        int id = pid;
                        if (id < 0 || id >= p.num_pages) { atomicExch(p.status, AFLEX_ERR_BOUNDS); id = 0; }
                        uint8_t* dst = smem + s * kStageBytes + kv * (kPagesPerStage * kPageBytes) + pg * kPageBytes + hf * (kPage * 128);
                        const int row = (id * p.Hkv + g) * kPage;
                        tma_load_2d_hint(dst, kv ? &tmap_v : &tmap_k, hf * 64, row, &sh->full[s], pol_kv);
                    }
                    if (piece_start) {
                        // The piece's queries (the G heads of the group are contiguous in q) travel with its first unit.
                        // q may be the output of the kernel just before this one: unless the launcher knows better, the
                        // first copy waits for the grid dependency (the KV loads above are already in flight).
                        if (!p.q_final && !waited) { pdl_wait(); waited = true; }
                        if (lane == 0)
                            bulk_load_1d(smem + s * kStageBytes + 2 * kPagesPerStage * kPageBytes,
                                         p.q + ((size_t)b_now * p.Hq + (size_t)g * p.G) * D, q_bytes, &sh->full[s]);
                    }
                    pid = pid_next;
                    if (++s == kAttnStages) { s = 0; ph ^= 1; }
                }
            }
            first_range = false;
            if (!claimed && !aborted) { claim(); claimed = true; }
            if (aborted || sp.n2 == 0 || next_ticket >= sp.n2) break;
            x0 = sp.U1 + (long long)next_ticket * sp.K2;
            x1 = min(sp.U, x0 + sp.K2);
            rid = (int)gridDim.x + next_ticket;
        }
        // end marker for the consumers
        if (lane == 0) {
            AttnRange rg;
            rg.x0 = 0; rg.x1 = 0; rg.prefix = 0; rg.b = 0; rg.rid = -1;
            sh->rng[r % kRangeRing] = rg;
            mbar_arrive(&sh->rng_ready[r % kRangeRing]);
            if (sp.n2 > 0) {
                // last CTA out resets the ticket counters (every CTA has made its final claim by now)
                __threadfence();
                if (atomicAdd(&p.ticket[1], 1) == (int)gridDim.x - 1) { p.ticket[0] = 0; p.ticket[1] = 0; }
            }
        }
    } else if (warp < kAttnConsumerWarps) {
        // ------------------------------------------------------------------ compute warps
        // q may be the output of the kernel just before this one (a projection GEMM of this library releases
        // its dependents early), so unless the launcher knows better (q written by the K/V append kernel, which
        // does not release early, or the caller's promise) these warps wait for the grid dependency before
        // their first q load; the ring fills meanwhile.  They never write to global memory: a finished
        // piece's state goes to the epilogue warp through the piece's last stage buffer.
        const int mi = lane >> 3, r8 = lane & 7;
        int s = 0;
        uint32_t ph = 0;
        bool aborted = false;

        for (int r = 0; !aborted; ++r) {
            // ---- next range of this CTA
            if (!mbar_wait(&sh->rng_ready[r % kRangeRing], (uint32_t)((r / kRangeRing) & 1))) {
                if (lane == 0) { sh->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); }
                break;
            }
            const AttnRange rg = sh->rng[r % kRangeRing];
            if (rg.x1 <= rg.x0) break;
            Walker wk;
            wk.init(p, rg);

        while (!wk.done() && !aborted) {
            // ---- one piece: units [u0, u0 + n) of one (sequence, KV head) item
            const int len = wk.len, cost = wk.cost;
            const int nv = (int)min((long long)(wk.nu - wk.u), wk.end - wk.pos);
            const int u0 = max(wk.u, cost) - cost;                           // real unit range [u0, u0 + n)
            const int n = max(wk.u + nv, cost) - cost - u0;
            wk.advance(nv);
            if (n <= 0) continue;                                            // only empty positions: no piece

            // Q^T as the MMA's B operand: lane holds head (lane/4), d = 16*ks + 2*(lane%4) + {0,1} (+8); read from the
            // piece's first stage, where the producer put the group's queries
            uint32_t qb[kKSteps][2];
            float o[kKSteps][4];
#pragma unroll
            for (int i = 0; i < kKSteps; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
            float m0 = kNegBig, m1 = kNegBig, l0 = 0.f, l1 = 0.f;

            for (int u = u0; u < u0 + n; ++u) {
                bool ok = mbar_wait(&sh->full[s], ph);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok || sh->abort) {
                    if (lane == 0) { sh->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); }
                    aborted = true;
                    break;
                }
                if (tr && threadIdx.x == 0 && tr[3] == 0) tr[3] = global_timer_ns();     // first data landed
                if (u == u0) {
                    const int h = lane >> 2;
                    const uint8_t* qs = smem + s * kStageBytes + 2 * kPagesPerStage * kPageBytes + (h < p.G ? h : 0) * (D * 2);
#pragma unroll
                    for (int ks = 0; ks < kKSteps; ++ks) {
                        const int d0 = ks * 16 + 2 * (lane & 3);
                        const uint32_t v0 = *reinterpret_cast<const uint32_t*>(qs + d0 * 2);
                        const uint32_t v1 = *reinterpret_cast<const uint32_t*>(qs + (d0 + 8) * 2);
                        qb[ks][0] = h < p.G ? v0 : 0u;
                        qb[ks][1] = h < p.G ? v1 : 0u;
                    }
                }
                const int nvalid = min(kPage, len - (u * kUnitTokens + warp * kPage));   // tokens of this warp's page
                if (nvalid > 0) {
                    const uint32_t kpage = smem_u32(smem + s * kStageBytes + warp * kPageBytes);
                    const uint32_t vpage = kpage + kPagesPerStage * kPageBytes;
                    if (nvalid < kPage) {
                        // zero the V rows of slots past the end of the sequence (they may hold NaN)
                        constexpr int kChunksPerRow = D / 8;
                        for (int i = lane; i < (kPage - nvalid) * kChunksPerRow; i += 32) {
                            const int row = nvalid + i / kChunksPerRow, cg = i % kChunksPerRow;
                            uint8_t* dst = smem + s * kStageBytes + (kPagesPerStage + warp) * kPageBytes + (cg >> 3) * (kPage * 128) +
                                           row * 128 + (cg & 7) * 16;
                            *reinterpret_cast<uint4*>(dst) = make_uint4(0, 0, 0, 0);
                        }
                        __syncwarp();
                    }
                    // ---- S^T[16 tokens][8 heads] = K Q^T
                    float sc[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                    for (int ks = 0; ks < kKSteps; ++ks) {
                        const int row = r8 + (mi & 1) * 8;
                        const int cg = ks * 2 + (mi >> 1);
                        const uint32_t addr = kpage + (cg >> 3) * (kPage * 128) + row * 128 + (((cg & 7) ^ (row & 7)) << 4);
                        uint32_t a0, a1, a2, a3;
                        ldmatrix_x4(addr, a0, a1, a2, a3);
                        mma_bf16_16816(sc, a0, a1, a2, a3, qb[ks][0], qb[ks][1]);
                    }
                    const int r0 = lane >> 2;
                    sc[0] = (r0 < nvalid) ? sc[0] * p.scale_log2 : -INFINITY;
                    sc[1] = (r0 < nvalid) ? sc[1] * p.scale_log2 : -INFINITY;
                    sc[2] = (r0 + 8 < nvalid) ? sc[2] * p.scale_log2 : -INFINITY;
                    sc[3] = (r0 + 8 < nvalid) ? sc[3] * p.scale_log2 : -INFINITY;
                    float mx0 = fmaxf(sc[0], sc[2]), mx1 = fmaxf(sc[1], sc[3]);
#pragma unroll
                    for (int off = 4; off < 32; off <<= 1) {
                        mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
                        mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
                    }
                    const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
                    const float c0 = fast_exp2(m0 - mn0), c1 = fast_exp2(m1 - mn1);
                    m0 = mn0; m1 = mn1;
                    const float p0 = fast_exp2(sc[0] - mn0), p1 = fast_exp2(sc[1] - mn1);
                    const float p2 = fast_exp2(sc[2] - mn0), p3 = fast_exp2(sc[3] - mn1);
                    l0 = l0 * c0 + p0 + p2;
                    l1 = l1 * c1 + p1 + p3;
                    // P^T as B operand: transpose the two 8x8 (token x head) blocks across the warp
                    const uint32_t pb0 = movmatrix_trans(pack_bf16x2(p0, p1));
                    const uint32_t pb1 = movmatrix_trans(pack_bf16x2(p2, p3));
                    // ---- O^T[D][8 heads] = O^T * corr + V^T P^T
#pragma unroll
                    for (int mt = 0; mt < kKSteps; ++mt) {
                        o[mt][0] *= c0; o[mt][1] *= c1; o[mt][2] *= c0; o[mt][3] *= c1;
                        const int trow = r8 + (mi >> 1) * 8;
                        const int cg = mt * 2 + (mi & 1);
                        const uint32_t addr = vpage + (cg >> 3) * (kPage * 128) + trow * 128 + (((cg & 7) ^ (trow & 7)) << 4);
                        uint32_t a0, a1, a2, a3;
                        ldmatrix_x4_trans(addr, a0, a1, a2, a3);
                        mma_bf16_16816(o[mt], a0, a1, a2, a3, pb0, pb1);
                    }
                    if (nvalid < kPage) fence_proxy_async();   // order the zeroing stores before the next TMA write
                }
                __syncwarp();
                if (u + 1 < u0 + n) {
                    if (lane == 0) mbar_arrive(&sh->empty[s]);
                } else {
                    // ---- last unit of the piece: park (O, m, l) in this warp's own pages of the stage (the O
                    // fragments fill the K page exactly, m and l go to the V page) and tell the epilogue warp;
                    // it releases the stage once it has read the four states.  No warp waits for another.
#pragma unroll
                    for (int off = 4; off < 32; off <<= 1) {
                        l0 += __shfl_xor_sync(0xffffffffu, l0, off);
                        l1 += __shfl_xor_sync(0xffffffffu, l1, off);
                    }
                    float* kdst = reinterpret_cast<float*>(smem + s * kStageBytes + warp * kPageBytes) + lane;
                    float* vdst = reinterpret_cast<float*>(smem + s * kStageBytes + (kPagesPerStage + warp) * kPageBytes) + lane;
#pragma unroll
                    for (int mt = 0; mt < kKSteps; ++mt) {
#pragma unroll
                        for (int j = 0; j < 4; ++j) kdst[(mt * 4 + j) * 32] = o[mt][j];
                    }
                    vdst[0] = m0; vdst[32] = m1; vdst[64] = l0; vdst[96] = l1;
                    fence_proxy_async();                 // these stores precede the stage's next TMA write
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&sh->xready[s]);
                }
                if (++s == kAttnStages) { s = 0; ph ^= 1; }
            }

            if (tr && threadIdx.x == 0) tr[4] = global_timer_ns();      // units of this piece consumed
        }
        }
    } else {
        // ------------------------------------------------------------------ epilogue warp
        // Walks the same ranges and pieces as the compute warps.  For every piece it waits until the four
        // states are parked in the piece's last stage, folds them (fixed order 0, 1, 2, 3), releases the
        // stage to the producer, and then does everything that touches global memory: the output row of a
        // whole item, or the partial slot, the arrival counter and - for the last arriver - the merge.
        // The compute warps stream on meanwhile; only the stage that holds the states waits for this warp.
        bool dep_ok = false;
        const int h0 = 2 * (lane & 3);          // this lane's two heads of the group: h0, h0 + 1
        int s = 0;
        uint32_t xph = 0;                       // phase bit of xready[] per stage
        bool aborted = false;
        const int G = (int)gridDim.x;

        for (int r = 0; !aborted; ++r) {
            // ---- next range of this CTA
            if (!mbar_wait(&sh->rng_ready[r % kRangeRing], (uint32_t)((r / kRangeRing) & 1))) {
                if (lane == 0) { sh->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); }
                break;
            }
            const AttnRange rg = sh->rng[r % kRangeRing];
            if (rg.x1 <= rg.x0) break;
            Walker wk;
            wk.init(p, rg);

        while (!wk.done() && !aborted) {
            // ---- one piece: units [u0, u0 + n) of item (b, g)
            const int b = wk.b, g = wk.g, cost = wk.cost;
            const int nu = wk.nu - cost;                                     // real units of the item
            const long long item_v0 = wk.prefix * p.Hkv + (long long)g * wk.nu;   // list position where the item starts
            const long long item_x0 = item_v0 + cost;                        // ... where its real units start
            const int nv = (int)min((long long)(wk.nu - wk.u), wk.end - wk.pos);
            const int u0 = max(wk.u, cost) - cost;                           // real unit range [u0, u0 + n)
            const int n = max(wk.u + nv, cost) - cost - u0;
            wk.advance(nv);
            if (n <= 0) continue;                                            // only empty positions: no piece
            // A range holds at most two partial pieces: one of an item that began before the range (slot 0) and one
            // of an item that begins inside it (slot 1).  The merge below locates a piece by the same predicate.
            const int slot = rg.x0 < item_v0 ? 1 : 0;

            const int s_last = (s + n - 1) % kAttnStages;
            s = (s + n) % kAttnStages;
            {
                bool ok = mbar_wait(&sh->xready[s_last], (xph >> s_last) & 1u);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok || sh->abort) {
                    if (lane == 0) { sh->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); }
                    aborted = true;
                    break;
                }
                xph ^= 1u << s_last;
            }
            float o[kKSteps][4];
            float m0, m1, l0, l1;
            {
                const float* ksrc = reinterpret_cast<const float*>(smem + s_last * kStageBytes) + lane;
                const float* vsrc = reinterpret_cast<const float*>(smem + s_last * kStageBytes + kPagesPerStage * kPageBytes) + lane;
#pragma unroll
                for (int mt = 0; mt < kKSteps; ++mt) {
#pragma unroll
                    for (int j = 0; j < 4; ++j) o[mt][j] = ksrc[(mt * 4 + j) * 32];
                }
                m0 = vsrc[0]; m1 = vsrc[32]; l0 = vsrc[64]; l1 = vsrc[96];
#pragma unroll
                for (int w = 1; w < kAttnConsumerWarps; ++w) {
                    const float* ks = ksrc + w * (kPageBytes / 4);
                    const float* vs = vsrc + w * (kPageBytes / 4);
                    const float om0 = vs[0], om1 = vs[32], ol0 = vs[64], ol1 = vs[96];
                    const float mn0 = fmaxf(m0, om0), mn1 = fmaxf(m1, om1);
                    const float a0 = fast_exp2(m0 - mn0), a1 = fast_exp2(m1 - mn1);
                    const float b0 = fast_exp2(om0 - mn0), b1 = fast_exp2(om1 - mn1);
                    m0 = mn0; m1 = mn1;
                    l0 = l0 * a0 + ol0 * b0;
                    l1 = l1 * a1 + ol1 * b1;
#pragma unroll
                    for (int mt = 0; mt < kKSteps; ++mt) {
                        o[mt][0] = o[mt][0] * a0 + ks[(mt * 4 + 0) * 32] * b0;
                        o[mt][1] = o[mt][1] * a1 + ks[(mt * 4 + 1) * 32] * b1;
                        o[mt][2] = o[mt][2] * a0 + ks[(mt * 4 + 2) * 32] * b0;
                        o[mt][3] = o[mt][3] * a1 + ks[(mt * 4 + 3) * 32] * b1;
                    }
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive_n(&sh->empty[s_last], kAttnConsumerWarps);    // the stage may be refilled
            if (!dep_ok) {
                pdl_wait();   // output rows, partial slots and counters may still be in use by earlier kernels
                dep_ok = true;
                if (tr && lane == 0) tr[2] = global_timer_ns();
            }
            const int dr = lane >> 2;
            const size_t hq0 = (size_t)g * p.G + h0;
            if (u0 == 0 && n == nu) {
                // the piece is the whole item: final result
                if (h0 < p.G) {
                    const float i0 = 1.0f / l0, i1 = 1.0f / l1;
                    __nv_bfloat16* out0 = p.out + ((size_t)b * p.Hq + hq0) * D;
#pragma unroll
                    for (int mt = 0; mt < kKSteps; ++mt) {
                        out0[mt * 16 + dr] = __float2bfloat16_rn(o[mt][0] * i0);
                        out0[mt * 16 + dr + 8] = __float2bfloat16_rn(o[mt][2] * i0);
                        if (h0 + 1 < p.G) {
                            out0[D + mt * 16 + dr] = __float2bfloat16_rn(o[mt][1] * i1);
                            out0[D + mt * 16 + dr + 8] = __float2bfloat16_rn(o[mt][3] * i1);
                        }
                    }
                    if (p.lse != nullptr && dr == 0) {
                        p.lse[(size_t)b * p.Hq + hq0] = (m0 + log2f(l0)) * 0.6931471805599453f;
                        if (h0 + 1 < p.G) p.lse[(size_t)b * p.Hq + hq0 + 1] = (m1 + log2f(l1)) * 0.6931471805599453f;
                    }
                }
                continue;
            }
            // ---- partial piece.  Pieces of this item: static shares cf..cl over [item_x0, min(item_x1, U1)), then
            // dynamic chunks jf..jl; `mine` is this piece's place in that list.
            const long long item_x1 = item_x0 + nu;
            int cf = 0, cl = -1, jf = 0, jl = -1;
            if (item_x0 < sp.U1) {
                cf = cta_of_unit(item_x0, sp.U1, sp.Ge1);
                cl = cta_of_unit(min(item_x1, sp.U1) - 1, sp.U1, sp.Ge1);
            }
            const long long dyn_x0 = max(item_x0, sp.U1);
            if (item_x1 > sp.U1) {
                jf = (int)((dyn_x0 - sp.U1) / sp.K2);
                jl = (int)((item_x1 - 1 - sp.U1) / sp.K2);
            }
            const int n_static = cl - cf + 1;
            const int expected = n_static + (jl - jf + 1);
            const int mine = rg.rid < G ? rg.rid - cf : n_static + (rg.rid - G - jf);
            int* counter = p.counters + b * p.Hkv + g;
            // Whoever finds all other pieces published finishes the item.  Usually that is known before anything is
            // written: the other pieces of an item that ends a CTA's share were computed at the start of the next
            // CTA's share, long ago.  Then this piece stays in registers: no partial store, no fence, no atomic.
            int seen = 0;
            if (lane == 0) asm volatile("ld.acquire.gpu.b32 %0, [%1];" : "=r"(seen) : "l"(counter) : "memory");
            seen = __shfl_sync(0xffffffffu, seen, 0);
            if (seen != expected - 1) {
                // park the piece in the range's slot (as the lanes hold it: [k step][lane][4]), bump the item's counter
                float4* op = reinterpret_cast<float4*>(p.o_part + ((size_t)rg.rid * 2 + slot) * 8 * D) + lane;
                float* mlp = p.ml_part + ((size_t)rg.rid * 2 + slot) * 8 * 2;
#pragma unroll
                for (int mt = 0; mt < kKSteps; ++mt) op[mt * 32] = make_float4(o[mt][0], o[mt][1], o[mt][2], o[mt][3]);
                if (dr == 0) *reinterpret_cast<float4*>(mlp + 2 * h0) = make_float4(m0, l0, m1, l1);
                __syncwarp();
                int last = 0;
                if (lane == 0) {
                    __threadfence();
                    last = (atomicAdd(counter, 1) == expected - 1) ? 1 : 0;
                }
                last = __shfl_sync(0xffffffffu, last, 0);
                if (!last) continue;
                __threadfence();
            }
            // ---- merge the item's pieces in list order (running maximum), this piece from registers, the others
            // from their slots.  A piece sits in slot 0 of its range unless other units of the range precede it
            // (slot 1): that can only happen for the first static share and for the first dynamic chunk.
            float acc[kKSteps][4];
#pragma unroll
            for (int mt = 0; mt < kKSteps; ++mt) { acc[mt][0] = acc[mt][1] = acc[mt][2] = acc[mt][3] = 0.f; }
            float M0 = kNegBig, M1 = kNegBig, L0 = 0.f, L1 = 0.f;
            for (int i = 0; i < expected; ++i) {
                float pm0, pl0, pm1, pl1;
                float4 po[kKSteps];
                if (i == mine) {
                    pm0 = m0; pl0 = l0; pm1 = m1; pl1 = l1;
#pragma unroll
                    for (int mt = 0; mt < kKSteps; ++mt) po[mt] = make_float4(o[mt][0], o[mt][1], o[mt][2], o[mt][3]);
                } else {
                    int rid_i, sl;
                    if (i < n_static) {
                        rid_i = cf + i;
                        sl = (i == 0 && share_begin(sp.U1, cf, sp.Ge1) < item_v0) ? 1 : 0;
                    } else {
                        const int j = jf + (i - n_static);
                        rid_i = G + j;
                        sl = (j == jf && sp.U1 + (long long)jf * sp.K2 < max(item_v0, sp.U1)) ? 1 : 0;
                    }
                    const size_t base = ((size_t)rid_i * 2 + sl) * 8;
                    const float4 ml = __ldcg(reinterpret_cast<const float4*>(p.ml_part + base * 2 + 2 * h0));
                    const float4* src = reinterpret_cast<const float4*>(p.o_part + base * D) + lane;
#pragma unroll
                    for (int mt = 0; mt < kKSteps; ++mt) po[mt] = __ldcg(src + mt * 32);
                    pm0 = ml.x; pl0 = ml.y; pm1 = ml.z; pl1 = ml.w;
                }
                const float mn0 = fmaxf(M0, pm0), mn1 = fmaxf(M1, pm1);
                const float a0 = fast_exp2(M0 - mn0), a1 = fast_exp2(M1 - mn1);
                const float b0 = fast_exp2(pm0 - mn0), b1 = fast_exp2(pm1 - mn1);
                M0 = mn0; M1 = mn1;
                L0 = L0 * a0 + pl0 * b0;
                L1 = L1 * a1 + pl1 * b1;
#pragma unroll
                for (int mt = 0; mt < kKSteps; ++mt) {
                    acc[mt][0] = acc[mt][0] * a0 + po[mt].x * b0;
                    acc[mt][1] = acc[mt][1] * a1 + po[mt].y * b1;
                    acc[mt][2] = acc[mt][2] * a0 + po[mt].z * b0;
                    acc[mt][3] = acc[mt][3] * a1 + po[mt].w * b1;
                }
            }
            if (h0 < p.G) {
                const float i0 = 1.0f / L0, i1 = 1.0f / L1;
                __nv_bfloat16* out0 = p.out + ((size_t)b * p.Hq + hq0) * D;
#pragma unroll
                for (int mt = 0; mt < kKSteps; ++mt) {
                    out0[mt * 16 + dr] = __float2bfloat16_rn(acc[mt][0] * i0);
                    out0[mt * 16 + dr + 8] = __float2bfloat16_rn(acc[mt][2] * i0);
                    if (h0 + 1 < p.G) {
                        out0[D + mt * 16 + dr] = __float2bfloat16_rn(acc[mt][1] * i1);
                        out0[D + mt * 16 + dr + 8] = __float2bfloat16_rn(acc[mt][3] * i1);
                    }
                }
                if (p.lse != nullptr && dr == 0) {
                    p.lse[(size_t)b * p.Hq + hq0] = (M0 + log2f(L0)) * 0.6931471805599453f;
                    if (h0 + 1 < p.G) p.lse[(size_t)b * p.Hq + hq0 + 1] = (M1 + log2f(L1)) * 0.6931471805599453f;
                }
            }
            __syncwarp();
            if (lane == 0) p.counters[b * p.Hkv + g] = 0;   // clean for the next launch
        }
        }
        if (tr && lane == 0) tr[5] = global_timer_ns();
    }
}

// ------------------------------------------------------------------------------------------ host
int attn_grid(const aflex_ctx* ctx) {
    int g = ctx->attn_ctas > 0 ? ctx->attn_ctas : 2 * ctx->num_sms;
    if (g > 4096) g = 4096;
    return g;
}

// Dynamic hand-out of the tail of the unit list (tuning: AFLEX_ATTN_DYN_PCT, AFLEX_ATTN_DYN_CHUNKS).
static int attn_dyn_pct() {
    static int v = -1;
    if (v < 0) { const char* e = getenv("AFLEX_ATTN_DYN_PCT"); v = e ? atoi(e) : 25; if (v < 0) v = 0; if (v > 90) v = 90; }
    return v;
}
static int attn_dyn_chunks() {
    static int v = -1;
    if (v < 0) { const char* e = getenv("AFLEX_ATTN_DYN_CHUNKS"); v = e ? atoi(e) : 8; if (v < 1) v = 1; if (v > 64) v = 64; }
    return v;
}

// List positions charged per item start when the unit list is cut into equal shares (tuning).
static int attn_piece_cost() {
    static int v = -1;
    if (v < 0) { const char* e = getenv("AFLEX_ATTN_PIECE_COST"); v = e ? atoi(e) : 1; if (v < 0) v = 0; if (v > 16) v = 16; }
    return v;
}

// Partial slots: two per range id; range ids = one static share per CTA plus at most
// dyn_chunks * grid + 1 dynamic chunks.
static size_t attn_slots(int grid) { return ((size_t)grid * (1 + attn_dyn_chunks()) + 2) * 2; }

size_t attn_workspace_bytes(const aflex_attn_desc* d, int grid) {
    return align256(attn_slots(grid) * 8 * d->head_dim * sizeof(float)) + align256(attn_slots(grid) * 8 * 2 * sizeof(float));
}

template <int D>
static aflex_status attn_launch_t(aflex_ctx* ctx, const aflex_attn_desc* d, const void* q, const aflex_kv* kv, int batch,
                                  void* out, float* lse, char* ws, size_t ws_bytes, cudaStream_t st) {
    const int grid = attn_grid(ctx);
    if ((long long)batch * d->num_kv_heads > kAttnCounterCap)
        return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "attention: batch * Hkv > %d", kAttnCounterCap);
    const size_t need = attn_workspace_bytes(d, grid);
    if (need > ws_bytes)
        return set_error(ctx, AFLEX_ERR_WORKSPACE, "attention: need %zu workspace bytes, have %zu", need, ws_bytes);
    Arena arena(ws, ws_bytes);
    AttnParams p;
    p.o_part = arena.take<float>(attn_slots(grid) * 8 * D);
    p.ml_part = arena.take<float>(attn_slots(grid) * 8 * 2);
    p.q = reinterpret_cast<const __nv_bfloat16*>(q);
    p.page_table = kv->page_table;
    p.seq_lens = kv->seq_lens;
    p.batch = batch;
    p.max_pages = kv->max_pages_per_seq;
    p.Hq = d->num_q_heads; p.Hkv = d->num_kv_heads; p.G = d->num_q_heads / d->num_kv_heads;
    p.num_pages = kv->num_pages;
    const float scale = d->sm_scale != 0.f ? d->sm_scale : 1.0f / sqrtf((float)D);
    p.scale_log2 = scale * 1.4426950408889634f;
    p.ticket = ctx->counters_attn + kAttnCounterCap + 2 * (ctx->attn_launch_seq++ & 3u);   // past the per-item counters
    p.dyn_pct = attn_dyn_pct();
    p.dyn_chunks = attn_dyn_chunks();
    p.piece_cost = attn_piece_cost();
    p.q_final = (ctx->attn_q_final || ctx->attn_q_final_once) ? 1 : 0;
    ctx->attn_q_final_once = false;
    { static int v = -1; if (v < 0) { const char* e = getenv("AFLEX_ATTN_DYN_UNITS"); v = e ? atoi(e) : 16; if (v < 1) v = 1; } p.dyn_min = v; }
    { static int v = -1; if (v < 0) { const char* e = getenv("AFLEX_ATTN_KVPOL"); v = e ? atoi(e) : 0; } p.kv_policy = v; }
    p.status = ctx->dev_status;
    p.out = reinterpret_cast<__nv_bfloat16*>(out);
    p.lse = lse;
    p.counters = ctx->counters_attn;
    p.trace = ctx->trace ? ctx->trace + (size_t)(ctx->trace_slot++ % kTraceKernels) * kTraceStride : nullptr;

    const uint64_t rows = (uint64_t)kv->num_pages * d->num_kv_heads * kPage;
    CUtensorMap tk, tv;
    if (!encode_tmap_2d_bf16(&tk, kv->k_cache, rows, D, (uint64_t)D * 2, kPage, 64, true) ||
        !encode_tmap_2d_bf16(&tv, kv->v_cache, rows, D, (uint64_t)D * 2, kPage, 64, true))
        return set_error(ctx, AFLEX_ERR_CUDA, "attention: cuTensorMapEncodeTiled failed");

    constexpr int kStageBytes = 2 * kPagesPerStage * kPage * D * 2 + 8 * D * 2;
    const size_t smem = (size_t)kAttnStages * kStageBytes + sizeof(AttnShared) + 1024;
    const int ti = (D == 128) ? 1 : 0;
    if (!ctx->attn_attr_set[ti]) {
        cudaError_t e = cudaFuncSetAttribute(attn_decode_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(attention)");
        ctx->attn_attr_set[ti] = true;
    }
    KernelScope scope(ctx, kKAttnDecode, st);
    cudaLaunchConfig_t lc = {};
    lc.gridDim = dim3((unsigned)grid);
    lc.blockDim = dim3(kAttnThreads);
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    return check_cuda(ctx, cudaLaunchKernelEx(&lc, attn_decode_kernel<D>, tk, tv, p), "attn_decode_kernel launch");
}

aflex_status attn_decode_launch(aflex_ctx* ctx, const aflex_attn_desc* d, const void* q, const aflex_kv* kv, int batch,
                                void* out, float* lse, char* ws, size_t ws_bytes, cudaStream_t st) {
    if (d->head_dim == 128) return attn_launch_t<128>(ctx, d, q, kv, batch, out, lse, ws, ws_bytes, st);
    return attn_launch_t<64>(ctx, d, q, kv, batch, out, lse, ws, ws_bytes, st);
}

}  // namespace aflex

// ------------------------------------------------------------------------------------------------
// Allocation-free decode attention.
//
// Some callers must not allocate device memory at all: a serving process whose memory pool has
// already claimed the whole GPU (every later cudaMalloc fails), a plugin that runs inside
// someone else's allocator discipline, or code on a latency-critical path where an allocation
// (an implicit device synchronisation) is not acceptable.  aflex_create allocates a workspace, so
// those callers cannot use the ctx-based entry points.  This entry point needs no ctx: the
// kernel's scratch (per-CTA partial results, arrival counters, a status word) lives in the
// file-scope device array below, which every GPU that loads the library holds until exit.
//
// Limits (stated maxima of the fixed scratch): at most kStaticMaxCtas persistent CTAs are
// launched and batch * num_kv_heads must not exceed kStaticMaxItems.  Everything else follows
// aflex_attn_decode (same kernel, same arithmetic).
namespace aflex {

constexpr int kStaticMaxCtas = 320;        // >= 2 CTAs per SM on a 148-SM part
constexpr int kStaticMaxItems = 16384;     // (sequence, KV head) pairs per call
constexpr size_t kStaticOPartFloats = (size_t)kStaticMaxCtas * 2 * 8 * 128;
constexpr size_t kStaticMlFloats = (size_t)kStaticMaxCtas * 2 * 8 * 2;
constexpr size_t kStaticScratchBytes =
    (kStaticOPartFloats + kStaticMlFloats) * sizeof(float) + (size_t)kStaticMaxItems * sizeof(int) + 256;   // ~2.7 MB

// Layout: [o_part floats | ml_part floats | counters ints | status word].
static __device__ __align__(256) unsigned char g_attn_static_scratch[kStaticScratchBytes];

struct StaticDeviceState {
    unsigned char* scratch = nullptr;   // device address of g_attn_static_scratch on this device
    int num_sms = 0;
    bool attr_set[2] = {false, false};
};
static StaticDeviceState g_static_state[64];

template <int D>
static aflex_status attn_static_launch(StaticDeviceState& stt, const aflex_attn_desc* d, const void* q, const aflex_kv* kv,
                                       int batch, void* out, float* lse, cudaStream_t st) {
    int grid = 2 * stt.num_sms;
    if (grid > kStaticMaxCtas) grid = kStaticMaxCtas;
    float* o_part = reinterpret_cast<float*>(stt.scratch);
    float* ml_part = o_part + kStaticOPartFloats;
    int* counters = reinterpret_cast<int*>(ml_part + kStaticMlFloats);
    int* status = counters + kStaticMaxItems;
    // The array keeps whatever the previous call left: the arrival counters and the status word must
    // start at zero (a call that was cut short could have left them dirty).
    cudaError_t e = cudaMemsetAsync(counters, 0, ((size_t)batch * d->num_kv_heads) * sizeof(int), st);
    if (e == cudaSuccess) e = cudaMemsetAsync(status, 0, sizeof(int), st);
    if (e != cudaSuccess) return AFLEX_ERR_CUDA;

    AttnParams p;
    p.o_part = o_part;
    p.ml_part = ml_part;
    p.q = reinterpret_cast<const __nv_bfloat16*>(q);
    p.page_table = kv->page_table;
    p.seq_lens = kv->seq_lens;
    p.batch = batch;
    p.max_pages = kv->max_pages_per_seq;
    p.Hq = d->num_q_heads; p.Hkv = d->num_kv_heads; p.G = d->num_q_heads / d->num_kv_heads;
    p.num_pages = kv->num_pages;
    const float scale = d->sm_scale != 0.f ? d->sm_scale : 1.0f / sqrtf((float)D);
    p.scale_log2 = scale * 1.4426950408889634f;
    p.status = status;
    p.out = reinterpret_cast<__nv_bfloat16*>(out);
    p.lse = lse;
    p.counters = counters;
    p.ticket = nullptr;     // static shares only: the fixed scratch has two slots per CTA
    p.dyn_pct = 0;
    p.dyn_chunks = 1;
    p.kv_policy = 0;
    p.q_final = 0;
    p.dyn_min = 12;
    p.piece_cost = 0;
    p.trace = nullptr;

    const uint64_t rows = (uint64_t)kv->num_pages * d->num_kv_heads * kPage;
    CUtensorMap tk, tv;
    if (!encode_tmap_2d_bf16(&tk, kv->k_cache, rows, D, (uint64_t)D * 2, kPage, 64, true) ||
        !encode_tmap_2d_bf16(&tv, kv->v_cache, rows, D, (uint64_t)D * 2, kPage, 64, true))
        return AFLEX_ERR_CUDA;
    constexpr int kStageBytes = 2 * kPagesPerStage * kPage * D * 2 + 8 * D * 2;
    const size_t smem = (size_t)kAttnStages * kStageBytes + sizeof(AttnShared) + 1024;
    const int ti = (D == 128) ? 1 : 0;
    if (!stt.attr_set[ti]) {
        e = cudaFuncSetAttribute(attn_decode_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return AFLEX_ERR_CUDA;
        stt.attr_set[ti] = true;
    }
    attn_decode_kernel<D><<<grid, kAttnThreads, smem, st>>>(tk, tv, p);
    return cudaGetLastError() == cudaSuccess ? AFLEX_OK : AFLEX_ERR_CUDA;
}

}  // namespace aflex

extern "C" aflex_status aflex_attn_decode_static(const aflex_attn_desc* desc, const void* q, const aflex_kv* kv, int batch,
                                                 void* out, float* lse, void* stream) {
    using namespace aflex;
    if (!desc || !q || !kv || !out || !kv->k_cache || !kv->v_cache || !kv->page_table || !kv->seq_lens)
        return AFLEX_ERR_INVALID_ARG;
    if (batch < 1 || kv->num_pages < 1 || kv->max_pages_per_seq < 1) return AFLEX_ERR_INVALID_ARG;
    if (desc->num_q_heads < 1 || desc->num_kv_heads < 1 || desc->num_q_heads % desc->num_kv_heads != 0)
        return AFLEX_ERR_INVALID_ARG;
    const int G = desc->num_q_heads / desc->num_kv_heads;
    if ((desc->head_dim != 64 && desc->head_dim != 128) || desc->page_size != 16 || (G != 1 && G != 2 && G != 4 && G != 8))
        return AFLEX_ERR_UNSUPPORTED;
    if ((long long)kv->num_pages * desc->num_kv_heads * 16 >= (1LL << 31)) return AFLEX_ERR_UNSUPPORTED;
    if ((reinterpret_cast<uintptr_t>(q) | reinterpret_cast<uintptr_t>(out) | reinterpret_cast<uintptr_t>(kv->k_cache) |
         reinterpret_cast<uintptr_t>(kv->v_cache)) & 15)
        return AFLEX_ERR_INVALID_ARG;
    // beyond the fixed scratch: refuse, never spill into an allocation
    if ((long long)batch * desc->num_kv_heads > kStaticMaxItems) return AFLEX_ERR_WORKSPACE;

    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return AFLEX_ERR_CUDA;
    StaticDeviceState& stt = g_static_state[dev];
    if (stt.scratch == nullptr) {
        // One-time set-up for this device (it is the current device): in host code the array's name is
        // only a stand-in, the kernel needs its device address.
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_attn_static_scratch) != cudaSuccess || ptr == nullptr) return AFLEX_ERR_CUDA;
        int sms = 0;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms < 1) return AFLEX_ERR_CUDA;
        stt.num_sms = sms;
        stt.scratch = static_cast<unsigned char*>(ptr);
    }
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    if (desc->head_dim == 128) return attn_static_launch<128>(stt, desc, q, kv, batch, out, lse, st);
    return attn_static_launch<64>(stt, desc, q, kv, batch, out, lse, st);
}

extern "C" aflex_status aflex_attn_decode_static_status(int* host_status, void* stream) {
    using namespace aflex;
    if (!host_status) return AFLEX_ERR_INVALID_ARG;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return AFLEX_ERR_CUDA;
    const StaticDeviceState& stt = g_static_state[dev];
    if (stt.scratch == nullptr) return AFLEX_ERR_INVALID_ARG;     // no static call on this device yet
    const int* status = reinterpret_cast<const int*>(reinterpret_cast<const float*>(stt.scratch) + kStaticOPartFloats + kStaticMlFloats) +
                        kStaticMaxItems;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(host_status, status, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    return e == cudaSuccess ? AFLEX_OK : AFLEX_ERR_CUDA;
}
