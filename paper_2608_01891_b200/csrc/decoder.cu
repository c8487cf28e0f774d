// The Attention group's small operators around the hot path, so that whole decoder layers chain:
//   add_rmsnorm_kernel  residual add + RMS normalisation of one token row per CTA
//   rope_append_kernel  per head: optional RMS normalisation of q / k, rotary embedding at the
//                       decoded token's position, q written out, k / v stored into the paged cache
// Both are row-local, bandwidth-trivial kernels (a few hundred KB per launch); they are chained with
// programmatic dependent launch so that their launch latency hides behind their neighbours.
#include <cuda_bf16.h>
#include <math.h>

#include "internal.h"
#include "ptx.cuh"

namespace aflex {

constexpr int kNormThreads = 256;

// s = res (+ add), both bf16, summed in fp32.  res_out = bf16(s) (when given; may alias res or add),
// y = bf16(s / sqrt(mean(s^2) + eps) * w) (when given).  One CTA per row; H % 8 == 0.
// Pass 1 reduces, pass 2 re-reads the (cache-resident) row and writes, so that aliasing outputs
// with inputs is safe: every element is read and written by the same thread, in pass 2 only.
__global__ void __launch_bounds__(kNormThreads)
add_rmsnorm_kernel(const __nv_bfloat16* res, const __nv_bfloat16* add, const __nv_bfloat16* __restrict__ w, int H,
                   float eps, __nv_bfloat16* res_out, __nv_bfloat16* y) {
    __shared__ float s_part[kNormThreads / 32];
    __shared__ float s_rinv;
    pdl_launch_dependents();
    pdl_wait();
    const size_t row = blockIdx.x;
    const uint4* r4 = reinterpret_cast<const uint4*>(res + row * H);
    const uint4* a4 = add ? reinterpret_cast<const uint4*>(add + row * H) : nullptr;
    const int chunks = H / 8;
    float rinv = 0.f;
    if (y != nullptr) {
        float ss = 0.f;
        for (int i = threadIdx.x; i < chunks; i += kNormThreads) {
            const uint4 r = r4[i];
            const __nv_bfloat162* pr = reinterpret_cast<const __nv_bfloat162*>(&r);
            uint4 a = make_uint4(0, 0, 0, 0);
            if (a4) a = a4[i];
            const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 fr = __bfloat1622float2(pr[j]), fa = __bfloat1622float2(pa[j]);
                const float s0 = fr.x + fa.x, s1 = fr.y + fa.y;
                ss = fmaf(s0, s0, ss);
                ss = fmaf(s1, s1, ss);
            }
        }
#pragma unroll
        for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
        if ((threadIdx.x & 31) == 0) s_part[threadIdx.x >> 5] = ss;
        __syncthreads();
        if (threadIdx.x == 0) {
            float tot = 0.f;
#pragma unroll
            for (int k = 0; k < kNormThreads / 32; ++k) tot += s_part[k];
            s_rinv = rsqrtf(tot / (float)H + eps);
        }
        __syncthreads();
        rinv = s_rinv;
    }
    const uint4* w4 = reinterpret_cast<const uint4*>(w);
    for (int i = threadIdx.x; i < chunks; i += kNormThreads) {
        const uint4 r = r4[i];
        const __nv_bfloat162* pr = reinterpret_cast<const __nv_bfloat162*>(&r);
        uint4 a = make_uint4(0, 0, 0, 0);
        if (a4) a = a4[i];
        const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
        float s[8];
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 fr = __bfloat1622float2(pr[j]), fa = __bfloat1622float2(pa[j]);
            s[2 * j] = fr.x + fa.x;
            s[2 * j + 1] = fr.y + fa.y;
        }
        if (res_out != nullptr) {
            uint4 o;
            __nv_bfloat162* po = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
            for (int j = 0; j < 4; ++j) po[j] = __floats2bfloat162_rn(s[2 * j], s[2 * j + 1]);
            reinterpret_cast<uint4*>(res_out + row * H)[i] = o;
        }
        if (y != nullptr) {
            uint4 g = w4[i];
            const __nv_bfloat162* pg = reinterpret_cast<const __nv_bfloat162*>(&g);
            uint4 o;
            __nv_bfloat162* po = reinterpret_cast<__nv_bfloat162*>(&o);
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const float2 fg = __bfloat1622float2(pg[j]);
                po[j] = __floats2bfloat162_rn(s[2 * j] * rinv * fg.x, s[2 * j + 1] * rinv * fg.y);
            }
            reinterpret_cast<uint4*>(y + row * H)[i] = o;
        }
    }
}

struct RopeParams {
    const __nv_bfloat16* qkv;      // [B][(Hq + 2 Hkv) * D]
    const __nv_bfloat16* w_qn;     // [D] or null
    const __nv_bfloat16* w_kn;     // [D] or null
    const int32_t* page_table;     // [B][max_pages]
    const int32_t* seq_lens;       // [B]
    const int32_t* q_offsets;      // null: one row per sequence, the token being decoded; else [B + 1]: row
                                   // q_offsets[b] + i is token i of the last q_offsets[b+1] - q_offsets[b] of sequence b
    int batch;
    __nv_bfloat16* q_out;          // [rows][Hq][D]
    __nv_bfloat16* k_cache;        // [num_pages][Hkv][16][D]
    __nv_bfloat16* v_cache;
    long long num_pages;
    int max_pages, Hq, Hkv, D;
    int heads_per_warp;            // 1 for a decode batch (every head its own warp); more for prompt rows, so that a
                                   // warp's position lookup and rotation serve several heads
    float eps;
    double inv_freq[64];           // theta^(-2 i / D), i < D / 2 (D <= 128), formed in double on the host
    int* status;
};

// One warp per (row, head) of the concatenated q | k | v heads.  Lane handles the rotary pairs
// (i, i + D/2), i = lane, lane + 32, ...  The angle pos * theta^(-2i/D) is formed and reduced to
// [-pi, pi] in double (at positions of 10^4 and more an fp32 angle would already be off by 10^-3 rad; the
// frequencies come from the host as doubles); only the sine and cosine of the remainder are fp32.
constexpr int kRopeWarps = 4;
__global__ void __launch_bounds__(kRopeWarps * 32) rope_append_kernel(const RopeParams p) {
    // No early release of the dependents here: the attention kernel streams the KV cache without waiting
    // for the grid dependency, which is sound only if the kernel that writes the cache has finished (and
    // flushed) before anything later in the stream starts.
    pdl_wait();
    const int lane = threadIdx.x & 31;
    const int head0 = (blockIdx.y * kRopeWarps + (threadIdx.x >> 5)) * p.heads_per_warp;
    const int row = blockIdx.x;
    const int heads = p.Hq + 2 * p.Hkv;
    if (head0 >= heads) return;
    const int D = p.D, half = D / 2;
    int b = row, back = 0;                         // sequence of this row; tokens of the sequence that follow it
    if (p.q_offsets != nullptr) {
        int lo = 0, hi = p.batch;                  // largest b with q_offsets[b] <= row
        while (hi - lo > 1) {
            const int mid = (lo + hi) / 2;
            if (p.q_offsets[mid] <= row) lo = mid; else hi = mid;
        }
        b = lo;
        back = p.q_offsets[b + 1] - 1 - row;
        if (back < 0) {                            // offsets that do not cover this row
            if (lane == 0) atomicExch(p.status, AFLEX_ERR_BOUNDS);
            return;
        }
    }
    const int len = p.seq_lens[b];
    if (len - back < 1 || len > p.max_pages * 16) {
        if (lane == 0) atomicExch(p.status, AFLEX_ERR_BOUNDS);
        return;                                    // no position to write to
    }
    const int pos = len - 1 - back;
    const int page = p.page_table[(size_t)b * p.max_pages + pos / 16];
    const bool page_ok = page >= 0 && page < p.num_pages;
    // the row's rotation: the same for every head (D <= 128: at most two pairs per lane)
    float cs[2], sn[2];
#pragma unroll
    for (int k = 0; k < 2; ++k) {
        const int i = lane + 32 * k;
        cs[k] = 1.f; sn[k] = 0.f;
        if (i < half) {
            // angle and its reduction to [-pi, pi] in double (two-term 2 pi), sine and cosine of the remainder in fp32
            const double ang = (double)pos * p.inv_freq[i];
            const double turns = rint(ang * 0.15915494309189535);
            const double red = fma(-turns, 2.4492935982947064e-16, fma(-turns, 6.283185307179586, ang));
            sincosf((float)red, &sn[k], &cs[k]);
        }
    }
    const int head_end = min(heads, head0 + p.heads_per_warp);
    for (int head = head0; head < head_end; ++head) {
        const __nv_bfloat16* src = p.qkv + ((size_t)row * heads + head) * D;
        const bool is_q = head < p.Hq, is_k = !is_q && head < p.Hq + p.Hkv;
        const __nv_bfloat16* gain = is_q ? p.w_qn : (is_k ? p.w_kn : nullptr);
        // destination row
        __nv_bfloat16* dst;
        if (is_q) {
            dst = p.q_out + ((size_t)row * p.Hq + head) * D;
        } else {
            if (!page_ok) {
                if (lane == 0) atomicExch(p.status, AFLEX_ERR_BOUNDS);
                continue;
            }
            const int g = is_k ? head - p.Hq : head - p.Hq - p.Hkv;
            dst = (is_k ? p.k_cache : p.v_cache) + (((size_t)page * p.Hkv + g) * 16 + (pos & 15)) * D;
        }
        if (!is_q && !is_k) {                      // values are stored as they are
            for (int i = lane; i < D / 2; i += 32)
                reinterpret_cast<uint32_t*>(dst)[i] = reinterpret_cast<const uint32_t*>(src)[i];
            continue;
        }
        float lo[2], hi[2];
        float ss = 0.f;
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int i = lane + 32 * k;
            lo[k] = hi[k] = 0.f;
            if (i < half) {
                lo[k] = __bfloat162float(src[i]);
                hi[k] = __bfloat162float(src[i + half]);
                ss = fmaf(lo[k], lo[k], ss);
                ss = fmaf(hi[k], hi[k], ss);
            }
        }
        if (gain != nullptr) {
#pragma unroll
            for (int off = 16; off > 0; off >>= 1) ss += __shfl_xor_sync(0xffffffffu, ss, off);
            const float rinv = rsqrtf(ss / (float)D + p.eps);
#pragma unroll
            for (int k = 0; k < 2; ++k) {
                const int i = lane + 32 * k;
                if (i < half) {
                    lo[k] = lo[k] * rinv * __bfloat162float(gain[i]);
                    hi[k] = hi[k] * rinv * __bfloat162float(gain[i + half]);
                }
            }
        }
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int i = lane + 32 * k;
            if (i < half) {
                dst[i] = __float2bfloat16_rn(lo[k] * cs[k] - hi[k] * sn[k]);
                dst[i + half] = __float2bfloat16_rn(hi[k] * cs[k] + lo[k] * sn[k]);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------ host
aflex_status add_rmsnorm_launch(aflex_ctx* ctx, const void* res, const void* add, const void* w, int T, int H, float eps,
                                void* res_out, void* y, cudaStream_t st) {
    KernelScope scope(ctx, kKAddRmsNorm, st);
    return check_cuda(ctx,
                      launch_pdl(add_rmsnorm_kernel, dim3(T), dim3(kNormThreads), 0, st, (const __nv_bfloat16*)res,
                                 (const __nv_bfloat16*)add, (const __nv_bfloat16*)w, H, eps, (__nv_bfloat16*)res_out,
                                 (__nv_bfloat16*)y),
                      "add_rmsnorm_kernel launch");
}

aflex_status rope_append_launch(aflex_ctx* ctx, const aflex_attn_desc* d, const void* qkv, const aflex_kv* kv, int batch,
                                const void* w_qn, const void* w_kn, float eps, float theta, void* q_out, cudaStream_t st,
                                const int32_t* q_offsets, int rows) {
    RopeParams p;
    p.q_offsets = q_offsets;
    p.batch = batch;
    p.qkv = (const __nv_bfloat16*)qkv;
    p.w_qn = (const __nv_bfloat16*)w_qn;
    p.w_kn = (const __nv_bfloat16*)w_kn;
    p.page_table = kv->page_table;
    p.seq_lens = kv->seq_lens;
    p.q_out = (__nv_bfloat16*)q_out;
    p.k_cache = (__nv_bfloat16*)const_cast<void*>(kv->k_cache);
    p.v_cache = (__nv_bfloat16*)const_cast<void*>(kv->v_cache);
    p.num_pages = kv->num_pages;
    p.max_pages = kv->max_pages_per_seq;
    p.Hq = d->num_q_heads; p.Hkv = d->num_kv_heads; p.D = d->head_dim;
    p.eps = eps;
    for (int i = 0; i < 64; ++i) p.inv_freq[i] = i < d->head_dim / 2 ? pow((double)theta, -2.0 * i / (double)d->head_dim) : 0.0;
    p.status = ctx->dev_status;
    const int heads = p.Hq + 2 * p.Hkv;
    p.heads_per_warp = (q_offsets && rows >= 1024) ? 8 : 1;
    const int warps = (heads + p.heads_per_warp - 1) / p.heads_per_warp;
    KernelScope scope(ctx, kKRopeAppend, st);
    return check_cuda(ctx,
                      launch_pdl(rope_append_kernel, dim3(q_offsets ? rows : batch, (warps + kRopeWarps - 1) / kRopeWarps), dim3(kRopeWarps * 32),
                                 0, st, p),
                      "rope_append_kernel launch");
}

}  // namespace aflex
