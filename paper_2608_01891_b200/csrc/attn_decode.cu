// Attention side: paged grouped-query decode attention, split over KV chunks.
//
// The operator is bound by streaming the KV cache from HBM once (the paper's Sections 1-2:
// decode attention is memory-bound on KV-cache reads), so the kernel is organised around
// keeping many page loads in flight per SM and touching every K/V byte exactly once for all
// G = Hq/Hkv query heads of a group:
//
//   work item   = (sequence b, KV head g, chunk c of C tokens)  -> one CTA
//   data path   = TMA tiled loads (128-byte swizzle) of whole pages: a page's K (or V) slab for
//                 one KV head is a contiguous [16 tokens][D] block; a stage holds 4 pages of K and
//                 V; a 3-stage mbarrier ring per CTA and 2 CTAs per SM keep ~190 KB in flight per SM
//   arithmetic  = mma.sync m16n8k16 (bf16 -> fp32) with the 16 tokens of a page as the M dimension
//                 and the (<= 8) heads of the group as the N dimension, so no rows are wasted on
//                 padding: S^T = K Q^T, then O^T += V^T P^T with P^T obtained from the S^T
//                 accumulator by movmatrix.  The flop/byte ratio (8 at G = 8) is above what the
//                 fp32 pipes sustain at full HBM rate, which is the only reason MMAs are used.
//   softmax     = online, fp32, base-2 exponentials; each of the 4 consumer warps owns one page
//                 of a stage and its own running (m, l, O); the warps are merged through shared
//                 memory at the end of the chunk and the chunk's unnormalised (O, m, l) goes to
//                 the workspace
//   combine     = a second small kernel merges the chunks of a sequence in fixed order.
//
// Unreferenced slots (beyond a sequence's length) may hold NaN: scores of such tokens are
// replaced (not multiplied) by -inf and their V rows are zeroed in shared memory before use.
#include <cuda_bf16.h>
#include <math.h>

#include "internal.h"
#include "ptx.cuh"

namespace aflex {

constexpr int kPage = 16;
constexpr int kPagesPerStage = 4;
constexpr int kAttnStages = 3;
constexpr int kAttnConsumerWarps = 4;
constexpr int kAttnThreads = (kAttnConsumerWarps + 1) * 32;
constexpr float kNegBig = -1.0e30f;

struct AttnParams {
    const __nv_bfloat16* q;
    const int32_t* page_table;
    const int32_t* seq_lens;
    int max_pages;
    int Hq, Hkv, G;
    int chunk_tokens;
    int max_chunks;
    long long num_pages;
    float scale_log2;      // sm_scale * log2(e)
    float* o_part;         // [B][max_chunks][Hq][D]  unnormalised sum_j p_j v_j
    float* ml_part;        // [B][max_chunks][Hq][2]  (running max in log2 units, sum of p)
    int* status;
};

struct __align__(8) AttnBarriers {
    uint64_t full[kAttnStages];
    uint64_t empty[kAttnStages];
    volatile int abort;
};

template <int D>
__global__ void __launch_bounds__(kAttnThreads, 2)
attn_partial_kernel(const __grid_constant__ CUtensorMap tmap_k, const __grid_constant__ CUtensorMap tmap_v,
                    const AttnParams p) {
    constexpr int kHalves = D / 64;                 // 128-byte column blocks per row
    constexpr int kPageBytes = kPage * D * 2;       // one page of K (or V) for one KV head
    constexpr int kStageBytes = 2 * kPagesPerStage * kPageBytes;
    constexpr int kOpsPerStage = 2 * kPagesPerStage * kHalves;
    constexpr int kKSteps = D / 16;

    const int chunk = blockIdx.x, g = blockIdx.y, b = blockIdx.z;
    const int len = p.seq_lens[b];
    const int tok_begin = chunk * p.chunk_tokens;
    if (tok_begin >= len) return;
    const int tok_end = min(len, tok_begin + p.chunk_tokens);
    const int n_pages = (tok_end - tok_begin + kPage - 1) / kPage;
    const int n_iters = (n_pages + kPagesPerStage - 1) / kPagesPerStage;
    const int page0 = tok_begin / kPage;

    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~(uintptr_t)1023);
    AttnBarriers* bars = reinterpret_cast<AttnBarriers*>(smem + kAttnStages * kStageBytes);

    const int warp = threadIdx.x >> 5;
    const int lane = threadIdx.x & 31;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kAttnStages; ++s) {
            mbar_init(&bars->full[s], 1);
            mbar_init(&bars->empty[s], kAttnConsumerWarps);
        }
        bars->abort = 0;
        fence_mbar_init();
        prefetch_tmap(&tmap_k);
        prefetch_tmap(&tmap_v);
    }
    __syncthreads();

    if (warp == kAttnConsumerWarps) {
        // ------------------------------------------------------------------ producer warp
        const int32_t* table = p.page_table + (size_t)b * p.max_pages;
        const int seq_pages = (len + kPage - 1) / kPage;
        auto load_ids = [&](int batch) -> int {
            const int idx = page0 + batch * 32 + lane;
            return idx < seq_pages ? table[idx] : 0;
        };
        int ids = load_ids(0), ids_next = 0;
        int s = 0;
        uint32_t ph = 0;
        for (int it = 0; it < n_iters; ++it) {
            if ((it & 7) == 0) {
                if (it > 0) ids = ids_next;
                ids_next = load_ids((it >> 3) + 1);
            }
            bool ok = mbar_wait(&bars->empty[s], ph ^ 1);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok || bars->abort) {
                if (lane == 0) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); }
                break;
            }
            const int np = min(kPagesPerStage, n_pages - it * kPagesPerStage);
            if (lane == 0) mbar_expect_tx(&bars->full[s], (uint32_t)(np * 2 * kPageBytes));
            __syncwarp();
            const int pg = lane / (2 * kHalves);
            const int kv = (lane / kHalves) & 1;
            const int hf = lane % kHalves;
            int pid = __shfl_sync(0xffffffffu, ids, ((it & 7) * kPagesPerStage + pg) & 31);
            if (lane < kOpsPerStage && pg < np) {
                if (pid < 0 || pid >= p.num_pages) { atomicExch(p.status, AFLEX_ERR_BOUNDS); pid = 0; }
                uint8_t* dst = smem + s * kStageBytes + kv * (kPagesPerStage * kPageBytes) + pg * kPageBytes + hf * (kPage * 128);
                const int row = (pid * p.Hkv + g) * kPage;
                tma_load_2d(dst, kv ? &tmap_v : &tmap_k, hf * 64, row, &bars->full[s]);
            }
            if (++s == kAttnStages) { s = 0; ph ^= 1; }
        }
    } else {
        // ------------------------------------------------------------------ consumer warps
        // Q^T as the MMA's B operand: thread holds head (lane/4), d = 16*ks + 2*(lane%4) + {0,1} (+8).
        uint32_t qb[kKSteps][2];
        {
            const int h = lane >> 2;
            const __nv_bfloat16* qrow = p.q + ((size_t)b * p.Hq + (size_t)g * p.G + (h < p.G ? h : 0)) * D;
#pragma unroll
            for (int ks = 0; ks < kKSteps; ++ks) {
                const int d0 = ks * 16 + 2 * (lane & 3);
                uint32_t v0 = *reinterpret_cast<const uint32_t*>(qrow + d0);
                uint32_t v1 = *reinterpret_cast<const uint32_t*>(qrow + d0 + 8);
                qb[ks][0] = h < p.G ? v0 : 0u;
                qb[ks][1] = h < p.G ? v1 : 0u;
            }
        }
        float o[kKSteps][4];
#pragma unroll
        for (int i = 0; i < kKSteps; ++i) { o[i][0] = o[i][1] = o[i][2] = o[i][3] = 0.f; }
        float m0 = kNegBig, m1 = kNegBig, l0 = 0.f, l1 = 0.f;   // heads 2*(lane%4), +1

        const int mi = lane >> 3, r8 = lane & 7;
        int s = 0;
        uint32_t ph = 0;
        bool aborted = false;
        for (int it = 0; it < n_iters; ++it) {
            bool ok = mbar_wait(&bars->full[s], ph);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok || bars->abort) {
                if (lane == 0) { bars->abort = 1; atomicExch(p.status, AFLEX_ERR_TIMEOUT); }
                aborted = true;
                break;
            }
            const int pg = it * kPagesPerStage + warp;          // page of the chunk owned by this warp
            if (pg < n_pages) {
                const int nvalid = min(kPage, tok_end - (tok_begin + pg * kPage));
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
            if (lane == 0) mbar_arrive(&bars->empty[s]);
            if (++s == kAttnStages) { s = 0; ph ^= 1; }
        }

        // ---- merge the 4 warps, write the chunk's partial result
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
            l0 += __shfl_xor_sync(0xffffffffu, l0, off);
            l1 += __shfl_xor_sync(0xffffffffu, l1, off);
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kAttnConsumerWarps * 32));   // all stage reads done: reuse stage memory
        float* mO = reinterpret_cast<float*>(smem);                        // [4 warps][8 heads][D]
        float* mM = mO + kAttnConsumerWarps * 8 * D;                       // [4][8]
        float* mL = mM + kAttnConsumerWarps * 8;                           // [4][8]
        {
            const int h0 = 2 * (lane & 3), dr = lane >> 2;
#pragma unroll
            for (int mt = 0; mt < kKSteps; ++mt) {
                mO[(warp * 8 + h0) * D + mt * 16 + dr] = o[mt][0];
                mO[(warp * 8 + h0 + 1) * D + mt * 16 + dr] = o[mt][1];
                mO[(warp * 8 + h0) * D + mt * 16 + dr + 8] = o[mt][2];
                mO[(warp * 8 + h0 + 1) * D + mt * 16 + dr + 8] = o[mt][3];
            }
            if (lane < 4) {
                mM[warp * 8 + h0] = m0; mM[warp * 8 + h0 + 1] = m1;
                mL[warp * 8 + h0] = l0; mL[warp * 8 + h0 + 1] = l1;
            }
        }
        asm volatile("bar.sync 1, %0;" ::"n"(kAttnConsumerWarps * 32));
        if (!aborted && !bars->abort) {
            const int tid = threadIdx.x;                       // 0..127
            const int d = tid % D;
            const size_t item = (size_t)b * p.max_chunks + chunk;
            for (int h = tid / D; h < p.G; h += (kAttnConsumerWarps * 32) / D) {
                float M = mM[h];
#pragma unroll
                for (int w = 1; w < kAttnConsumerWarps; ++w) M = fmaxf(M, mM[w * 8 + h]);
                float acc = 0.f, L = 0.f;
#pragma unroll
                for (int w = 0; w < kAttnConsumerWarps; ++w) {
                    const float f = fast_exp2(mM[w * 8 + h] - M);
                    acc += f * mO[(w * 8 + h) * D + d];
                    L += f * mL[w * 8 + h];
                }
                const size_t hq = (size_t)g * p.G + h;
                p.o_part[(item * p.Hq + hq) * D + d] = acc;
                if (d == 0) {
                    p.ml_part[(item * p.Hq + hq) * 2 + 0] = M;
                    p.ml_part[(item * p.Hq + hq) * 2 + 1] = L;
                }
            }
        }
    }
}

// Merge the chunks of one (sequence, query head) in fixed order c = 0,1,...:
//   M = max_c m_c ; out = sum_c 2^(m_c-M) o_c / sum_c 2^(m_c-M) l_c ; lse = ln2 * (M + log2 sum)
template <int D>
__global__ void attn_combine_kernel(const float* __restrict__ o_part, const float* __restrict__ ml_part,
                                    const int32_t* __restrict__ seq_lens, int Hq, int chunk_tokens, int max_chunks,
                                    __nv_bfloat16* __restrict__ out, float* __restrict__ lse) {
    const int bh = blockIdx.x;
    const int b = bh / Hq, h = bh % Hq;
    const int d = threadIdx.x;
    const int len = seq_lens[b];
    const int nc = (len + chunk_tokens - 1) / chunk_tokens;
    float M = kNegBig;
    for (int c = 0; c < nc; ++c) M = fmaxf(M, ml_part[(((size_t)b * max_chunks + c) * Hq + h) * 2]);
    float acc = 0.f, L = 0.f;
    for (int c = 0; c < nc; ++c) {
        const size_t item = ((size_t)b * max_chunks + c) * Hq + h;
        const float f = fast_exp2(ml_part[item * 2] - M);
        acc += f * o_part[item * D + d];
        L += f * ml_part[item * 2 + 1];
    }
    out[((size_t)b * Hq + h) * D + d] = __float2bfloat16_rn(acc / L);
    if (lse != nullptr && d == 0) lse[(size_t)b * Hq + h] = (M + log2f(L)) * 0.6931471805599453f;
}

// ------------------------------------------------------------------------------------------ host
AttnPlan attn_make_plan(const aflex_ctx* ctx, const aflex_attn_desc* d, const aflex_kv* kv, int batch) {
    AttnPlan plan;
    const long long max_len = (long long)kv->max_pages_per_seq * kPage;
    int C = ctx->attn_chunk;
    if (C <= 0) {
        // Pick the largest chunk that still yields >= 3 waves of CTAs (2 resident per SM).
        double tokens = 0.0;
        if (kv->seq_lens_host) { for (int b = 0; b < batch; ++b) tokens += kv->seq_lens_host[b]; }
        else tokens = 0.6 * (double)batch * (double)max_len;
        const double want_items = 3.0 * 2.0 * ctx->num_sms;
        C = 2048;
        while (C > 128 && tokens / C * d->num_kv_heads < want_items) C >>= 1;
    }
    C = (C + 63) / 64 * 64;
    plan.chunk_tokens = C;
    plan.max_chunks = (int)((max_len + C - 1) / C);
    if (plan.max_chunks < 1) plan.max_chunks = 1;
    return plan;
}

size_t attn_workspace_bytes(const aflex_attn_desc* d, int batch, int max_chunks) {
    const size_t items = (size_t)batch * max_chunks * d->num_q_heads;
    return align256(items * d->head_dim * sizeof(float)) + align256(items * 2 * sizeof(float));
}

template <int D>
static aflex_status attn_launch_t(aflex_ctx* ctx, const aflex_attn_desc* d, const void* q, const aflex_kv* kv, int batch,
                                  void* out, float* lse, char* ws, size_t ws_bytes, cudaStream_t st) {
    const AttnPlan plan = attn_make_plan(ctx, d, kv, batch);
    const size_t need = attn_workspace_bytes(d, batch, plan.max_chunks);
    if (need > ws_bytes)
        return set_error(ctx, AFLEX_ERR_WORKSPACE, "attention: need %zu workspace bytes, have %zu", need, ws_bytes);
    Arena arena(ws, ws_bytes);
    const size_t items = (size_t)batch * plan.max_chunks * d->num_q_heads;
    AttnParams p;
    p.o_part = arena.take<float>(items * D);
    p.ml_part = arena.take<float>(items * 2);
    p.q = reinterpret_cast<const __nv_bfloat16*>(q);
    p.page_table = kv->page_table;
    p.seq_lens = kv->seq_lens;
    p.max_pages = kv->max_pages_per_seq;
    p.Hq = d->num_q_heads; p.Hkv = d->num_kv_heads; p.G = d->num_q_heads / d->num_kv_heads;
    p.chunk_tokens = plan.chunk_tokens;
    p.max_chunks = plan.max_chunks;
    p.num_pages = kv->num_pages;
    const float scale = d->sm_scale != 0.f ? d->sm_scale : 1.0f / sqrtf((float)D);
    p.scale_log2 = scale * 1.4426950408889634f;
    p.status = ctx->dev_status;

    const uint64_t rows = (uint64_t)kv->num_pages * d->num_kv_heads * kPage;
    CUtensorMap tk, tv;
    if (!encode_tmap_2d_bf16(&tk, kv->k_cache, rows, D, (uint64_t)D * 2, kPage, 64, true) ||
        !encode_tmap_2d_bf16(&tv, kv->v_cache, rows, D, (uint64_t)D * 2, kPage, 64, true))
        return set_error(ctx, AFLEX_ERR_CUDA, "attention: cuTensorMapEncodeTiled failed");

    constexpr int kStageBytes = 2 * kPagesPerStage * kPage * D * 2;
    const size_t smem = (size_t)kAttnStages * kStageBytes + sizeof(AttnBarriers) + 1024;
    const int ti = (D == 128) ? 1 : 0;
    if (!ctx->attn_attr_set[ti]) {
        cudaError_t e = cudaFuncSetAttribute(attn_partial_kernel<D>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return check_cuda(ctx, e, "cudaFuncSetAttribute(attention)");
        ctx->attn_attr_set[ti] = true;
    }
    dim3 grid((unsigned)plan.max_chunks, (unsigned)d->num_kv_heads, (unsigned)batch);
    {
        KernelScope scope(ctx, kKAttnPartial, st);
        attn_partial_kernel<D><<<grid, kAttnThreads, smem, st>>>(tk, tv, p);
    }
    aflex_status s = check_cuda(ctx, cudaGetLastError(), "attn_partial_kernel launch");
    if (s != AFLEX_OK) return s;
    KernelScope scope(ctx, kKAttnCombine, st);
    attn_combine_kernel<D><<<batch * d->num_q_heads, D, 0, st>>>(p.o_part, p.ml_part, kv->seq_lens, d->num_q_heads,
                                                               plan.chunk_tokens, plan.max_chunks,
                                                               reinterpret_cast<__nv_bfloat16*>(out), lse);
    return check_cuda(ctx, cudaGetLastError(), "attn_combine_kernel launch");
}

aflex_status attn_decode_launch(aflex_ctx* ctx, const aflex_attn_desc* d, const void* q, const aflex_kv* kv, int batch,
                                void* out, float* lse, char* ws, size_t ws_bytes, cudaStream_t st) {
    if (d->head_dim == 128) return attn_launch_t<128>(ctx, d, q, kv, batch, out, lse, ws, ws_bytes, st);
    return attn_launch_t<64>(ctx, d, q, kv, batch, out, lse, ws, ws_bytes, st);
}

}  // namespace aflex
