// Mixture-of-experts glue around the grouped GEMMs: router logits, top-k routing with gates,
// the stable expert-sorted permutation, row gather and the gate-weighted un-permute.
// Everything here is integer work or plain copies; nothing uses float atomics, so results are
// bit-reproducible.
#include <cuda_bf16.h>

#include "internal.h"
#include "ptx.cuh"

namespace aflex {

constexpr int kRouteThreads = 1024;
constexpr int kRouteWarps = kRouteThreads / 32;
constexpr int kRouteMaxExperts = 64;

// logits[t][e] = <x[t], w_router[e]>  (bf16 inputs, fp32 accumulation in a fixed lane-strided,
// then butterfly, order).  One warp per (t, e).
__global__ void router_logits_kernel(const __nv_bfloat16* __restrict__ x, const __nv_bfloat16* __restrict__ w,
                                     int T, int H, int E, float* __restrict__ logits) {
    pdl_launch_dependents();
    pdl_wait();
    const int gw = (blockIdx.x * blockDim.x + threadIdx.x) >> 5;
    const int lane = threadIdx.x & 31;
    if (gw >= T * E) return;
    const int t = gw / E, e = gw % E;
    const uint4* xr = reinterpret_cast<const uint4*>(x + (size_t)t * H);
    const uint4* wr = reinterpret_cast<const uint4*>(w + (size_t)e * H);
    float acc = 0.f;
    for (int i = lane; i < H / 8; i += 32) {
        const uint4 a = xr[i], b = wr[i];
        const __nv_bfloat162* pa = reinterpret_cast<const __nv_bfloat162*>(&a);
        const __nv_bfloat162* pb = reinterpret_cast<const __nv_bfloat162*>(&b);
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const float2 fa = __bfloat1622float2(pa[j]), fb = __bfloat1622float2(pb[j]);
            acc = fmaf(fa.x, fb.x, acc);
            acc = fmaf(fa.y, fb.y, acc);
        }
    }
#pragma unroll
    for (int off = 16; off > 0; off >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, off);
    if (lane == 0) logits[gw] = acc;
}

// One block does the whole routing problem:
//   A. per token: K rounds of "largest logit not yet taken, lowest index on ties, NaN never wins",
//      gates = softmax over the K selected logits (fp32); histogram of expert ids;
//   B. offsets = exclusive scan of counts;
//   C. pos(t,k) = offsets[e] + number of earlier assignments (in (t,k) order) with the same expert.
__global__ void __launch_bounds__(kRouteThreads)
moe_route_kernel(const float* __restrict__ logits, int T, int E, int K, int32_t* __restrict__ idx,
                 float* __restrict__ gate, int32_t* __restrict__ counts, int32_t* __restrict__ offsets,
                 int32_t* __restrict__ pos) {
    __shared__ int s_count[kRouteMaxExperts];
    __shared__ int s_offset[kRouteMaxExperts + 1];
    __shared__ int s_running[kRouteMaxExperts];
    __shared__ int s_warp[kRouteWarps][kRouteMaxExperts];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    pdl_launch_dependents();
    if (tid < kRouteMaxExperts) { s_count[tid] = 0; s_running[tid] = 0; }
    pdl_wait();
    __syncthreads();

    for (int t = tid; t < T; t += kRouteThreads) {
        const float* l = logits + (size_t)t * E;
        int sel[2] = {-1, -1};
        float lv[2] = {0.f, 0.f};
        for (int k = 0; k < K; ++k) {
            int best = -1;
            float bv = 0.f;
            for (int e = 0; e < E; ++e) {
                if (k == 1 && e == sel[0]) continue;
                const float v = l[e];
                if (best < 0) { best = e; bv = v; continue; }
                if (v > bv || (bv != bv && v == v)) { best = e; bv = v; }
            }
            sel[k] = best;
            lv[k] = bv;
        }
        float g0 = 1.f, g1 = 0.f;
        if (K == 2) {
            const float e1 = expf(lv[1] - lv[0]);       // <= 1
            const float den = 1.f + e1;
            g0 = 1.f / den;
            g1 = e1 / den;
        }
        idx[(size_t)t * K] = sel[0];
        gate[(size_t)t * K] = g0;
        atomicAdd(&s_count[sel[0]], 1);
        if (K == 2) {
            idx[(size_t)t * K + 1] = sel[1];
            gate[(size_t)t * K + 1] = g1;
            atomicAdd(&s_count[sel[1]], 1);
        }
    }
    __syncthreads();
    if (tid == 0) {
        int run = 0;
        for (int e = 0; e < E; ++e) { s_offset[e] = run; run += s_count[e]; }
        s_offset[E] = run;
    }
    __syncthreads();
    if (tid <= E) offsets[tid] = s_offset[tid];
    if (tid < E) counts[tid] = s_count[tid];

    const int total = T * K;
    for (int base = 0; base < total; base += kRouteThreads) {
        for (int i = tid; i < kRouteWarps * kRouteMaxExperts; i += kRouteThreads) (&s_warp[0][0])[i] = 0;
        __syncthreads();
        const int i = base + tid;
        const int e = (i < total) ? idx[i] : -1;
        const unsigned same = __match_any_sync(0xffffffffu, e);
        const int rank_in_warp = __popc(same & ((1u << lane) - 1u));
        if (e >= 0 && rank_in_warp == 0) s_warp[warp][e] = __popc(same);
        __syncthreads();
        if (tid < E) {   // exclusive prefix over warps for expert `tid`, then advance the running base
            int run = s_running[tid];
            for (int w = 0; w < kRouteWarps; ++w) { const int c = s_warp[w][tid]; s_warp[w][tid] = run; run += c; }
            s_running[tid] = run;
        }
        __syncthreads();
        if (e >= 0) pos[i] = s_offset[e] + s_warp[warp][e] + rank_in_warp;
        __syncthreads();
    }
}

// xp[pos[t][k]][:] = x[t][:]
__global__ void moe_gather_kernel(const __nv_bfloat16* __restrict__ x, const int32_t* __restrict__ pos, int K, int H,
                                  __nv_bfloat16* __restrict__ xp) {
    pdl_launch_dependents();
    pdl_wait();
    const int a = blockIdx.x;          // assignment index t*K + k
    const int t = a / K;
    const uint4* src = reinterpret_cast<const uint4*>(x + (size_t)t * H);
    uint4* dst = reinterpret_cast<uint4*>(xp + (size_t)pos[a] * H);
    for (int i = threadIdx.x; i < H / 8; i += blockDim.x) dst[i] = src[i];
}

// y[t][:] = sum_{k ascending} gate[t][k] * yp[pos[t][k]][:]   (fp32) -> bf16
__global__ void moe_combine_kernel(const float* __restrict__ yp, const int32_t* __restrict__ pos,
                                   const float* __restrict__ gate, int K, int H, __nv_bfloat16* __restrict__ y) {
    pdl_launch_dependents();
    pdl_wait();
    const int t = blockIdx.x;
    for (int i = threadIdx.x; i < H / 4; i += blockDim.x) {
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int k = 0; k < K; ++k) {
            const float g = gate[(size_t)t * K + k];
            const float4 v = reinterpret_cast<const float4*>(yp + (size_t)pos[(size_t)t * K + k] * H)[i];
            acc.x = fmaf(g, v.x, acc.x); acc.y = fmaf(g, v.y, acc.y);
            acc.z = fmaf(g, v.z, acc.z); acc.w = fmaf(g, v.w, acc.w);
        }
        __nv_bfloat162 lo = __floats2bfloat162_rn(acc.x, acc.y), hi = __floats2bfloat162_rn(acc.z, acc.w);
        uint2 pk;
        pk.x = *reinterpret_cast<uint32_t*>(&lo);
        pk.y = *reinterpret_cast<uint32_t*>(&hi);
        reinterpret_cast<uint2*>(y + (size_t)t * H)[i] = pk;
    }
}

aflex_status moe_router_logits_launch(aflex_ctx* ctx, const void* x, const void* w_router, int T, int H, int E,
                                      float* logits, cudaStream_t st) {
    const int warps = T * E;
    const int threads = 256;
    const int blocks = (warps * 32 + threads - 1) / threads;
    KernelScope scope(ctx, kKRouterLogits, st);
    return check_cuda(ctx, launch_pdl(router_logits_kernel, dim3(blocks), dim3(threads), 0, st, (const __nv_bfloat16*)x,
                                      (const __nv_bfloat16*)w_router, T, H, E, logits),
                      "router_logits_kernel launch");
}

aflex_status moe_route_launch(aflex_ctx* ctx, const float* logits, int T, int E, int K, const MoeBuffers& mb,
                              cudaStream_t st) {
    KernelScope scope(ctx, kKMoeRoute, st);
    return check_cuda(ctx, launch_pdl(moe_route_kernel, dim3(1), dim3(kRouteThreads), 0, st, logits, T, E, K, mb.idx, mb.gate,
                                      mb.counts, mb.offsets, mb.pos),
                      "moe_route_kernel launch");
}

aflex_status moe_gather_launch(aflex_ctx* ctx, const void* x, const int32_t* pos, int T, int K, int H, void* xp,
                               cudaStream_t st) {
    KernelScope scope(ctx, kKMoeGather, st);
    return check_cuda(ctx, launch_pdl(moe_gather_kernel, dim3(T * K), dim3(128), 0, st, (const __nv_bfloat16*)x, pos, K, H,
                                      (__nv_bfloat16*)xp),
                      "moe_gather_kernel launch");
}

aflex_status moe_combine_launch(aflex_ctx* ctx, const float* yp, const int32_t* pos, const float* gate, int T, int K,
                                int H, void* y, cudaStream_t st) {
    KernelScope scope(ctx, kKMoeCombine, st);
    return check_cuda(ctx, launch_pdl(moe_combine_kernel, dim3(T), dim3(256), 0, st, yp, pos, gate, K, H, (__nv_bfloat16*)y),
                      "moe_combine_kernel launch");
}

}  // namespace aflex
