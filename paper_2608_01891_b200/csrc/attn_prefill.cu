// Prefill (causal) attention over the paged KV cache: the attention operator of the prefill phase
// (the paper's PA pool; Section 1: during prefill both operators are dominated by matrix
// multiplications).  Compute-bound, so it runs on the 5th-generation tensor cores:
//
//   CTA         = two tiles of 128 consecutive query tokens of one query head; both walk the same cached tokens,
//               128 at a step, share the K/V ring and alternate on the tensor pipe (one tile's softmax runs
//               while the other tile's MMAs do)
//   S = Q K^T   tcgen05.mma (128 x 128 x 16: issuing an MMA costs about as much as a 128-wide one takes, so
//               narrower steps starve the pipe), both operands K-major (Q tile and K rows of D contiguous
//               elements, 128-byte swizzle as TMA writes them), fp32 accumulator in TMEM, one per tile
//   softmax     four warps per tile, one query row per thread: tcgen05.ld of its S row, causal mask, online
//               max / sum in base 2, P rounded to bf16 and stored back over the S columns (tcgen05.st)
//   O += P V    tcgen05.mma with A = P read from TMEM and B = V exactly as the cache stores it ([token][D]:
//               an MN-major operand); accumulator in TMEM, rescaled in place only when a row's maximum
//               outgrows the reference by 2^8
//   pipeline    a producer warp issues the TMA loads of the K rows and the V rows of the coming steps into a
//               ring of slots (K(0) V(0) K(1) V(1) ...: a slot is free as soon as its own MMAs retire);
//               one thread issues MMAs in the order P V(t), S(t+1) per tile, so the pipe's in-order execution
//               keeps S(t+1) from landing on P(t) before it was read
//
// Query i of a sequence with n cached tokens of which the last m are being prefilled sits at position
// n - m + i and sees cached tokens 0 .. n - m + i.  Cache slots beyond n may hold anything (NaN too):
// their scores are replaced by -inf and their V rows are zeroed in shared memory before use.
#include <cuda_bf16.h>
#include <math.h>

#include "internal.h"
#include "ptx.cuh"

namespace aflex {
namespace pa {

constexpr int kBM = 128;          // query rows per tile
constexpr int kQT = 2;            // query tiles per CTA (they share the K/V stages and alternate on the tensor pipe)
constexpr int kBN = 128;          // cached tokens per step
constexpr int kPage = 16;
constexpr int kPagesPerStep = kBN / kPage;
constexpr int kMaxSlots = 6;
constexpr int slots_for(int D) { return D == 128 ? 5 : 6; }   // K or V rows of one step per slot (32 KB at D = 128)
constexpr int kSoftmaxWarps = 4 * kQT;         // warp groups 0 and 1: four softmax warps per query tile
constexpr int kThreads = (kSoftmaxWarps + 4) * 32;   // warp group 2: producer, MMA issuer, two idle warps
constexpr int kRegsSoftmax = 216, kRegsIssue = 72;   // registers per thread after the warp groups trade them
constexpr float kNegBig = -1.0e30f;

struct Params {
    const int32_t* page_table;
    const int32_t* seq_lens;      // cached tokens per sequence, the prefilled ones included
    const int32_t* q_offsets;     // [B+1] first query row of every sequence
    int batch, max_pages, Hq, Hkv, G;
    long long num_pages;
    int total_blocks;             // sum over sequences of ceil(q_len / 256)
    float scale_log2;
    __nv_bfloat16* out;           // [T][Hq][D]
    int* status;
};

struct __align__(8) Shared {
    uint64_t q_full;
    uint64_t kv_full[kMaxSlots], kv_empty[kMaxSlots];
    uint64_t s_ready[kQT], p_ready[kQT], pv_done[kQT];
    uint32_t tmem_base;
    volatile int abort;
};

__device__ __forceinline__ void tmem_st_32x32b_x16(uint32_t taddr, const uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.st.sync.aligned.32x32b.x16.b32 [%0], "
        "{%1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, %16};"
        ::"r"(taddr), "r"(r[0]), "r"(r[1]), "r"(r[2]), "r"(r[3]), "r"(r[4]), "r"(r[5]), "r"(r[6]), "r"(r[7]), "r"(r[8]),
          "r"(r[9]), "r"(r[10]), "r"(r[11]), "r"(r[12]), "r"(r[13]), "r"(r[14]), "r"(r[15])
        : "memory");
}
__device__ __forceinline__ void tmem_st_wait() { asm volatile("tcgen05.wait::st.sync.aligned;" ::: "memory"); }

// Shared-memory operand descriptors, all with the 128-byte swizzle TMA writes (8-row groups 1024 B apart: the
// stride byte offset).  K-major operands (Q, K: rows of 64 contiguous K elements) leave the leading byte offset at
// its unused value 16; the MN-major operand (V as the cache stores it, [token = K row][64 D columns] blocks) puts the
// distance between its 64-column blocks there and advances by 2048 B per 16 token rows.
// The MMA issuer keeps descriptors as a low word (start address in 16-byte units, leading byte offset at bit 16) that
// it advances by adding byte offsets >> 4, and one upper word shared by every operand here (8-row groups 1024 B apart,
// descriptor version 1, 128-byte swizzle).
constexpr uint32_t kDescHi = (1024u >> 4) | (1u << 14) | (2u << 29);
__device__ __forceinline__ uint32_t desc_lo(uint32_t smem_addr, uint32_t lbo_bytes) {
    return ((smem_addr & 0x3FFFF) >> 4) | ((lbo_bytes >> 4) << 16);
}
__device__ __forceinline__ void umma_ss(uint32_t tmem_d, uint32_t a_lo, uint32_t b_lo, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 da, db;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "mov.b64 da, {%1, %5};\n\t"
        "mov.b64 db, {%2, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], da, db, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(a_lo), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi)
        : "memory");
}
__device__ __forceinline__ void umma_ts(uint32_t tmem_d, uint32_t tmem_a, uint32_t b_lo, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t.reg .b64 db;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "mov.b64 db, {%2, %5};\n\t"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], [%1], db, %3, p;\n\t}"
        ::"r"(tmem_d), "r"(tmem_a), "r"(b_lo), "r"(idesc), "r"(accumulate), "r"(kDescHi)
        : "memory");
}

template <int D>
__global__ void __launch_bounds__(kThreads, 1)
attn_prefill_kernel(const __grid_constant__ CUtensorMap tmap_q, const __grid_constant__ CUtensorMap tmap_k,
                    const __grid_constant__ CUtensorMap tmap_v, const Params p) {
    constexpr int kHalves = D / 64;
    constexpr int kQHalf = kBM * 128;                    // 128 query rows of 128 B
    constexpr int kQBytes = kHalves * kQHalf;            // one query tile
    constexpr int kKVHalf = kBN * 128;                   // 128 cached tokens of 128 B
    constexpr int kSlotBytes = kHalves * kKVHalf;        // the K rows, or the V rows, of one step
    constexpr int kSlots = slots_for(D);                 // ring of K and V slots: K(0) V(0) K(1) V(1) ...
    constexpr uint32_t kOCol = kQT * kBN;                // TMEM: S[tile] (P over it) first, then O[tile]

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    uint8_t* sq = smem;
    uint8_t* skv = sq + kQT * kQBytes;
    Shared* sh = reinterpret_cast<Shared*>(skv + kSlots * kSlotBytes);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    // ---- which block of 256 query rows: query head fastest (the heads of a group share K/V in L2), long blocks first
    const int h = blockIdx.x % p.Hq;
    const int block_id = p.total_blocks - 1 - (int)(blockIdx.x / p.Hq);
    int b = 0, block_in_seq = 0;
    {
        int acc = 0;
        for (b = 0; b < p.batch; ++b) {
            const int m = p.q_offsets[b + 1] - p.q_offsets[b];
            const int nb = (m + kQT * kBM - 1) / (kQT * kBM);
            if (block_id < acc + nb) { block_in_seq = block_id - acc; break; }
            acc += nb;
        }
        if (b >= p.batch) return;                        // cannot happen with a consistent total_blocks
    }
    const int q_len = p.q_offsets[b + 1] - p.q_offsets[b];
    int n_cached = p.seq_lens[b];
    {
        const int cap = p.max_pages * kPage;
        if (n_cached > cap || n_cached < q_len) { if (threadIdx.x == 0) atomicExch(p.status, AFLEX_ERR_BOUNDS); n_cached = max(min(n_cached, cap), q_len); }
    }
    // per query tile: rows, position of the first query, cached tokens visible to the last query, steps
    int rows_valid[kQT], pos0[kQT], kv_end[kQT], n_steps[kQT];
#pragma unroll
    for (int i = 0; i < kQT; ++i) {
        const int first = (block_in_seq * kQT + i) * kBM;
        rows_valid[i] = max(0, min(kBM, q_len - first));
        pos0[i] = n_cached - q_len + first;
        kv_end[i] = rows_valid[i] > 0 ? pos0[i] + rows_valid[i] : 0;
        n_steps[i] = (kv_end[i] + kBN - 1) / kBN;
    }
    const int q_row0 = p.q_offsets[b] + block_in_seq * kQT * kBM;
    const int kv_end_all = max(kv_end[0], kv_end[1]);
    const int steps_all = max(n_steps[0], n_steps[1]);
    const int g = h / p.G;

    if (threadIdx.x == 0) {
        mbar_init(&sh->q_full, 1);
        for (int s = 0; s < kSlots; ++s) { mbar_init(&sh->kv_full[s], 1); mbar_init(&sh->kv_empty[s], 1); }
        for (int i = 0; i < kQT; ++i) {
            mbar_init(&sh->s_ready[i], 1);
            mbar_init(&sh->p_ready[i], 4);
            mbar_init(&sh->pv_done[i], 1);
        }
        sh->abort = 0;
        fence_mbar_init();
        prefetch_tmap(&tmap_q); prefetch_tmap(&tmap_k); prefetch_tmap(&tmap_v);
    }
    if (warp == kSoftmaxWarps + 1) { tmem_alloc(&sh->tmem_base, 512); tmem_relinquish(); }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh->tmem_base;
    pdl_launch_dependents();
    pdl_wait();

    if (warp >= kSoftmaxWarps) {
    asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(kRegsIssue));
    if (warp == kSoftmaxWarps) {
        // ------------------------------------------------------------------ producer warp
        if (lane == 0) {
            mbar_expect_tx(&sh->q_full, (uint32_t)(kQT * kQBytes));
            for (int i = 0; i < kQT; ++i)
                for (int hf = 0; hf < kHalves; ++hf)
                    tma_load_2d(sq + i * kQBytes + hf * kQHalf, &tmap_q, h * D + hf * 64, q_row0 + i * kBM, &sh->q_full);
        }
        // one lane per (64-column half, page) box of a slot; slot 2t holds the K rows of step t, slot 2t + 1 its V rows
        const int page = lane % kPagesPerStep;
        const int hf = lane / kPagesPerStep;
        const bool op_lane = lane < kHalves * kPagesPerStep;
        auto page_id = [&](int t) -> int {
            const int idx = t * kPagesPerStep + page;
            return (op_lane && idx * kPage < kv_end_all) ? p.page_table[(size_t)b * p.max_pages + idx] : 0;
        };
        int id = page_id(0);
        for (int t = 0; t < steps_all; ++t) {
            const int id_next = (t + 1 < steps_all) ? page_id(t + 1) : 0;     // one step ahead of the ring
            const int np = min(kPagesPerStep, (kv_end_all - t * kBN + kPage - 1) / kPage);
            int pid = id;
            if (op_lane && page < np && (pid < 0 || pid >= p.num_pages)) { atomicExch(p.status, AFLEX_ERR_BOUNDS); pid = 0; }
            bool ok = true;
            for (int isv = 0; isv < 2 && ok; ++isv) {
                const int j = 2 * t + isv, s = j % kSlots;
                ok = mbar_wait(&sh->kv_empty[s], ((j / kSlots) & 1) ^ 1);
                ok = __all_sync(0xffffffffu, ok) && !sh->abort;
                if (!ok) break;
                if (lane == 0) mbar_expect_tx(&sh->kv_full[s], (uint32_t)(np * kHalves * kPage * 128));
                __syncwarp();
                if (op_lane && page < np)
                    tma_load_2d(skv + s * kSlotBytes + hf * kKVHalf + page * (kPage * 128), isv ? &tmap_v : &tmap_k, hf * 64,
                                (pid * p.Hkv + g) * kPage, &sh->kv_full[s]);
            }
            if (!ok) { if (lane == 0) { sh->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); } break; }
            id = id_next;
        }
    } else if (warp == kSoftmaxWarps + 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc_s = umma_idesc_bf16(kBM, kBN);
            const uint32_t idesc_pv = umma_idesc_bf16(kBM, D) | (1u << 16);      // B operand (V) is MN-major
            bool ok = mbar_wait(&sh->q_full, 0);
            // S of step t of query tile i (needs the step's K rows; the tile's S / P columns are free once its
            // previous P V has been issued: the tensor pipe runs in order)
            auto issue_s = [&](int t, int i) {
                if (t >= n_steps[i]) return;
                const int j = 2 * t, s = j % kSlots;
                ok = ok && mbar_wait(&sh->kv_full[s], (j / kSlots) & 1);
                if (!ok) return;
                tc_fence_after();
                const uint32_t k_lo = desc_lo(smem_u32(skv + s * kSlotBytes), 16);
                const uint32_t q_lo = desc_lo(smem_u32(sq + i * kQBytes), 16);
#pragma unroll
                for (int ks = 0; ks < D / 16; ++ks)
                    umma_ss(tmem + (uint32_t)(i * kBN), q_lo + (uint32_t)(((ks / 4) * kQHalf + (ks % 4) * 32) >> 4),
                            k_lo + (uint32_t)(((ks / 4) * kKVHalf + (ks % 4) * 32) >> 4), idesc_s, ks > 0 ? 1u : 0u);
                umma_commit(&sh->s_ready[i]);
            };
            for (int i = 0; i < kQT; ++i) issue_s(0, i);
            if (steps_all > 0 && ok) umma_commit(&sh->kv_empty[0]);
            for (int t = 0; t < steps_all && ok && !sh->abort; ++t) {
                const int jv = 2 * t + 1, sv_ = jv % kSlots;
                for (int i = 0; i < kQT && ok; ++i) {
                    if (t >= n_steps[i]) continue;
                    ok = ok && mbar_wait(&sh->p_ready[i], t & 1);
                    ok = ok && mbar_wait(&sh->kv_full[sv_], (jv / kSlots) & 1);
                    if (!ok) break;
                    tc_fence_after();
                    const uint32_t v_lo = desc_lo(smem_u32(skv + sv_ * kSlotBytes), kKVHalf);
#pragma unroll
                    for (int ks = 0; ks < kBN / 16; ++ks)
                        umma_ts(tmem + kOCol + (uint32_t)(i * D), tmem + (uint32_t)(i * kBN + ks * 8), v_lo + (uint32_t)((ks * 2048) >> 4),
                                idesc_pv, (t > 0 || ks > 0) ? 1u : 0u);
                    umma_commit(&sh->pv_done[i]);
                    issue_s(t + 1, i);                                       // runs under the other tile's softmax
                }
                if (!ok) break;
                umma_commit(&sh->kv_empty[sv_]);                             // V of this step
                if (t + 1 < steps_all) umma_commit(&sh->kv_empty[(2 * t + 2) % kSlots]);   // K of the next
            }
            if (!ok) { sh->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); }
        }
    }
    } else {
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(kRegsSoftmax));
        // ------------------------------------------------------------------ softmax warps: one query row per thread
        const int i = warp / 4;                       // query tile of this warp
        const int w = warp & 3;                       // TMEM lane quadrant of this warp
        const int row = w * 32 + lane;
        const bool row_ok = row < rows_valid[i];
        const int pos = pos0[i] + row;                // position of this row's query
        const uint32_t lane_base = tmem + ((uint32_t)(w * 32) << 16);
        const uint32_t s_addr = lane_base + (uint32_t)(i * kBN);
        const uint32_t o_addr = lane_base + kOCol + (uint32_t)(i * D);
        const int steps = n_steps[i];
        const int tid = (warp & 3) * 32 + lane;       // 0..127 inside the tile's warps
        float m = kNegBig, l = 0.f;
        bool ok = true;
        for (int t = 0; t < steps; ++t) {
            ok = mbar_wait(&sh->s_ready[i], t & 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok || sh->abort) break;
            tc_fence_after();
            const int col0 = t * kBN;
            // ---- this thread's S row into registers (one wait for all loads)
            float sv[kBN];
#pragma unroll
            for (int c0 = 0; c0 < kBN; c0 += 16)
                tmem_ld_32x32b_x16(s_addr + (uint32_t)c0, *reinterpret_cast<uint32_t(*)[16]>(&sv[c0]));
            tmem_ld_wait();
            // causal mask: only steps that reach past the tile's first query need it
            if (col0 + kBN - 1 > pos0[i] || !row_ok) {
#pragma unroll
                for (int j = 0; j < kBN; ++j)
                    if (!(row_ok && col0 + j <= pos)) sv[j] = -INFINITY;
            }
            float mx0 = -INFINITY, mx1 = -INFINITY, mx2 = -INFINITY, mx3 = -INFINITY;
#pragma unroll
            for (int j = 0; j < kBN; j += 4) {
                mx0 = fmaxf(mx0, sv[j]); mx1 = fmaxf(mx1, sv[j + 1]); mx2 = fmaxf(mx2, sv[j + 2]); mx3 = fmaxf(mx3, sv[j + 3]);
            }
            const float mx = fmaxf(fmaxf(mx0, mx1), fmaxf(mx2, mx3)) * p.scale_log2;
            // The reference maximum m moves only when some row of the warp outgrows it by more than 2^8: until
            // then p = 2^(s - m) stays below 256 (harmless in bf16 / fp32) and O needs no rescaling.
            const bool grow = __any_sync(0xffffffffu, mx > m + 8.0f);
            const float m_new = grow ? fmaxf(m, mx) : m;
            const float corr = fast_exp2(m - m_new);
            // ---- O is rescaled only after the previous step's P V has retired (rare: see `grow`)
            if (t > 0 && grow) {
                ok = mbar_wait(&sh->pv_done[i], (t - 1) & 1);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
#pragma unroll
                for (int c0 = 0; c0 < D; c0 += 16) {
                    uint32_t r[16];
                    tmem_ld_32x32b_x16(o_addr + (uint32_t)c0, r);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 16; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) * corr);
                    tmem_st_32x32b_x16(o_addr + (uint32_t)c0, r);
                }
            }
            // ---- V rows that were not loaded or lie past the sequence's end: zero them, whatever they hold
            //      (by the warps of both query tiles: each tile's P V waits only for its own warps, zeros are idempotent)
            {
                const int np = min(kPagesPerStep, (kv_end_all - col0 + kPage - 1) / kPage);
                const int n_here = max(0, min(n_cached - col0, np * kPage));
                if (n_here < kBN) {
                    const int jv = 2 * t + 1, sv_ = jv % kSlots;
                    ok = mbar_wait(&sh->kv_full[sv_], (jv / kSlots) & 1);        // the loaded rows must have landed first
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    uint8_t* vbase = skv + sv_ * kSlotBytes;
                    for (int k = tid; k < (kBN - n_here) * kHalves * 8; k += 128) {
                        const int r_ = n_here + k / (kHalves * 8), c_ = k % (kHalves * 8);
                        *reinterpret_cast<uint4*>(vbase + (c_ / 8) * kKVHalf + r_ * 128 + (c_ % 8) * 16) = make_uint4(0, 0, 0, 0);
                    }
                    fence_proxy_async();
                }
            }
            // ---- p = 2^(s * scale - m), row sum; P (bf16, two per column) goes back over the S columns it came
            //      from as the A operand of P V (the tensor pipe runs in order: the next S lands there after P V read it)
            float l0 = 0.f, l1 = 0.f;
#pragma unroll
            for (int c0 = 0; c0 < kBN; c0 += 32) {
                uint32_t pk[16];
#pragma unroll
                for (int j = 0; j < 32; j += 2) {
                    const float p0 = fast_exp2(fmaf(sv[c0 + j], p.scale_log2, -m_new));
                    const float p1 = fast_exp2(fmaf(sv[c0 + j + 1], p.scale_log2, -m_new));
                    l0 += p0; l1 += p1;
                    pk[j >> 1] = pack_bf16x2(p0, p1);
                }
                tmem_st_32x32b_x16(s_addr + (uint32_t)(c0 / 2), pk);
            }
            tmem_st_wait();
            l = l * corr + (l0 + l1);
            m = m_new;
            // P (and zeroed V rows) written: hand them to the MMA issuer
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(&sh->p_ready[i]);
        }
        if (steps > 0 && ok && !sh->abort) {
            ok = mbar_wait(&sh->pv_done[i], (steps - 1) & 1);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (steps > 0 && ok && !sh->abort) {
            tc_fence_after();
            const float inv = row_ok ? 1.0f / l : 0.f;
            __nv_bfloat16* orow = p.out + ((size_t)(q_row0 + i * kBM + row) * p.Hq + h) * D;
#pragma unroll
            for (int c0 = 0; c0 < D; c0 += 16) {
                uint32_t r[16];
                tmem_ld_32x32b_x16(o_addr + (uint32_t)c0, r);
                tmem_ld_wait();
                if (row_ok) {
                    uint32_t pk[8];
#pragma unroll
                    for (int j = 0; j < 16; j += 2)
                        pk[j >> 1] = pack_bf16x2(__uint_as_float(r[j]) * inv, __uint_as_float(r[j + 1]) * inv);
                    *reinterpret_cast<uint4*>(orow + c0) = make_uint4(pk[0], pk[1], pk[2], pk[3]);
                    *reinterpret_cast<uint4*>(orow + c0 + 8) = make_uint4(pk[4], pk[5], pk[6], pk[7]);
                }
            }
        } else if (steps > 0 && lane == 0 && !sh->abort) {
            sh->abort = 1;
            atomicExch(p.status, AFLEX_ERR_TIMEOUT);
        }
    }
    tc_fence_before();
    __syncthreads();
    if (warp == kSoftmaxWarps + 1) { tc_fence_after(); tmem_dealloc(tmem, 512); }
}

template <int D>
static aflex_status launch_t(aflex_ctx* ctx, const aflex_attn_desc* d, const void* q, const aflex_kv* kv, int batch,
                             const int32_t* q_offsets, int total_rows, int total_blocks, void* out, cudaStream_t st) {
    Params p;
    p.page_table = kv->page_table;
    p.seq_lens = kv->seq_lens;
    p.q_offsets = q_offsets;
    p.batch = batch;
    p.max_pages = kv->max_pages_per_seq;
    p.Hq = d->num_q_heads; p.Hkv = d->num_kv_heads; p.G = d->num_q_heads / d->num_kv_heads;
    p.num_pages = kv->num_pages;
    p.total_blocks = total_blocks;
    const float scale = d->sm_scale != 0.f ? d->sm_scale : 1.0f / sqrtf((float)D);
    p.scale_log2 = scale * 1.4426950408889634f;
    p.out = reinterpret_cast<__nv_bfloat16*>(out);
    p.status = ctx->dev_status;
    CUtensorMap tq, tk, tv;
    const uint64_t rows = (uint64_t)kv->num_pages * d->num_kv_heads * kPage;
    const uint64_t qcols = (uint64_t)d->num_q_heads * D;
    if (!encode_tmap_2d_bf16(&tq, q, (uint64_t)total_rows, qcols, qcols * 2, kBM, 64, false) ||
        !encode_tmap_2d_bf16(&tk, kv->k_cache, rows, D, (uint64_t)D * 2, kPage, 64, true) ||
        !encode_tmap_2d_bf16(&tv, kv->v_cache, rows, D, (uint64_t)D * 2, kPage, 64, true))
        return set_error(ctx, AFLEX_ERR_CUDA, "prefill attention: cuTensorMapEncodeTiled failed");
    const size_t smem = (size_t)kQT * (D / 64) * kBM * 128 + (size_t)slots_for(D) * (D / 64) * kBN * 128 +
                        sizeof(Shared) + 1024;
    const int ti = (D == 128) ? 1 : 0;
    if (!ctx->prefill_attr_set[ti]) {
        cudaError_t e = cudaFuncSetAttribute(attn_prefill_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(prefill attention)");
        ctx->prefill_attr_set[ti] = true;
    }
    KernelScope scope(ctx, kKAttnPrefill, st);
    return check_cuda(ctx,
                      launch_pdl(attn_prefill_kernel<D>, dim3((unsigned)total_blocks * (unsigned)d->num_q_heads), dim3(kThreads),
                                 smem, st, tq, tk, tv, p),
                      "attn_prefill_kernel launch");
}

}  // namespace pa

aflex_status attn_prefill_launch(aflex_ctx* ctx, const aflex_attn_desc* d, const void* q, const aflex_kv* kv, int batch,
                                 const int32_t* q_offsets, const int32_t* q_offsets_host, void* out, cudaStream_t st) {
    long long tiles = 0;
    for (int b = 0; b < batch; ++b) {
        const int m = q_offsets_host[b + 1] - q_offsets_host[b];
        if (m < 0) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "prefill attention: q_offsets_host must not decrease");
        tiles += (m + pa::kQT * pa::kBM - 1) / (pa::kQT * pa::kBM);
    }
    const int total_rows = q_offsets_host[batch];
    if (q_offsets_host[0] != 0 || total_rows < 1 || tiles < 1)
        return set_error(ctx, AFLEX_ERR_INVALID_ARG, "prefill attention: q_offsets_host must start at 0 and hold at least one query");
    if (tiles * d->num_q_heads > 0x7fffffffLL) return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "prefill attention: too many tiles");
    if (d->head_dim == 128) return pa::launch_t<128>(ctx, d, q, kv, batch, q_offsets, total_rows, (int)tiles, out, st);
    return pa::launch_t<64>(ctx, d, q, kv, batch, q_offsets, total_rows, (int)tiles, out, st);
}

}  // namespace aflex
