// C-ABI entry points, the context and the A/F microbatch interleave.
#include <cuda_bf16.h>
#include <stdarg.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

#include <new>

#include "internal.h"

namespace aflex {

aflex_status set_error(aflex_ctx* ctx, aflex_status s, const char* fmt, ...) {
    if (ctx) {
        va_list ap;
        va_start(ap, fmt);
        vsnprintf(ctx->err, sizeof(ctx->err), fmt, ap);
        va_end(ap);
    }
    return s;
}

aflex_status check_cuda(aflex_ctx* ctx, cudaError_t e, const char* what) {
    if (e == cudaSuccess) return AFLEX_OK;
    return set_error(ctx, AFLEX_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn get_encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// Encoding a tensor map costs a driver call (~1-2 us) and a decode step launches ~20 loads' worth of
// maps over the same few tensors every time: keep the encoded maps in a small per-thread cache keyed
// by everything the encoding depends on (address, extents, stride, box, promotion).
namespace {
struct TmapKey {
    const void* base; uint64_t rows, cols, stride; uint32_t box_rows, box_cols; bool promote;
    bool operator==(const TmapKey& o) const {
        return base == o.base && rows == o.rows && cols == o.cols && stride == o.stride && box_rows == o.box_rows &&
               box_cols == o.box_cols && promote == o.promote;
    }
};
struct TmapCache {
    static constexpr int kEntries = 128;
    TmapKey keys[kEntries];
    CUtensorMap maps[kEntries];
    int used = 0, next = 0;
};
thread_local TmapCache g_tmap_cache;
}  // namespace

bool encode_tmap_2d_bf16(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint64_t row_stride_bytes,
                         uint32_t box_rows, uint32_t box_cols, bool promote_l2_256) {
    TmapCache& cache = g_tmap_cache;
    const TmapKey key{base, rows, cols, row_stride_bytes, box_rows, box_cols, promote_l2_256};
    for (int i = 0; i < cache.used; ++i) {
        if (cache.keys[i] == key) { *out = cache.maps[i]; return true; }
    }
    EncodeTiledFn fn = get_encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {row_stride_bytes};
    cuuint32_t box[2] = {box_cols, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                    promote_l2_256 ? CU_TENSOR_MAP_L2_PROMOTION_L2_256B : CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return false;
    const int slot = cache.used < TmapCache::kEntries ? cache.used++ : (cache.next = (cache.next + 1) % TmapCache::kEntries);
    cache.keys[slot] = key;
    cache.maps[slot] = *out;
    return true;
}

static bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15) == 0; }

static aflex_status validate_attn(aflex_ctx* ctx, const aflex_attn_desc* d, const void* q, const aflex_kv* kv, int batch,
                                  const void* out) {
    if (!ctx) return AFLEX_ERR_INVALID_ARG;
    if (!d || !q || !kv || !out) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "attention: null argument");
    if (!kv->k_cache || !kv->v_cache || !kv->page_table || !kv->seq_lens)
        return set_error(ctx, AFLEX_ERR_INVALID_ARG, "attention: null KV argument");
    if (batch < 1 || kv->num_pages < 1 || kv->max_pages_per_seq < 1)
        return set_error(ctx, AFLEX_ERR_INVALID_ARG, "attention: batch, num_pages and max_pages_per_seq must be >= 1");
    if (d->num_q_heads < 1 || d->num_kv_heads < 1 || d->num_q_heads % d->num_kv_heads != 0)
        return set_error(ctx, AFLEX_ERR_INVALID_ARG, "attention: Hkv must divide Hq");
    if (!aligned16(q) || !aligned16(out) || !aligned16(kv->k_cache) || !aligned16(kv->v_cache))
        return set_error(ctx, AFLEX_ERR_INVALID_ARG, "attention: pointers must be 16-byte aligned");
    const int G = d->num_q_heads / d->num_kv_heads;
    if (d->head_dim != 64 && d->head_dim != 128)
        return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "attention: head_dim %d (supported: 64, 128)", d->head_dim);
    if (d->page_size != 16) return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "attention: page_size %d (supported: 16)", d->page_size);
    if (G != 1 && G != 2 && G != 4 && G != 8)
        return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "attention: Hq/Hkv = %d (supported: 1, 2, 4, 8)", G);
    if (batch > 65535) return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "attention: batch > 65535");
    if ((long long)kv->num_pages * d->num_kv_heads * 16 >= (1LL << 31))
        return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "attention: KV pool has more than 2^31 token rows");
    if (kv->seq_lens_host) {
        const long long max_len = (long long)kv->max_pages_per_seq * 16;
        for (int b = 0; b < batch; ++b)
            if (kv->seq_lens_host[b] < 1 || kv->seq_lens_host[b] > max_len)
                return set_error(ctx, AFLEX_ERR_INVALID_ARG, "attention: seq_lens_host[%d] = %d outside [1, %lld]", b,
                                 kv->seq_lens_host[b], max_len);
    }
    return AFLEX_OK;
}

static aflex_status validate_ffn_dims(aflex_ctx* ctx, int T, int H, int I) {
    if (T < 1 || H < 1 || I < 1) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "ffn: T, H, I must be >= 1");
    if (H % 8 || I % 8) return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "ffn: H and I must be multiples of 8");
    return AFLEX_OK;
}

// ---- F side, shared by the stand-alone entry points and the layer step -----------------------
static size_t dense_ws_bytes(int T, int H, int I, int num_sms) {
    const size_t gu = gateup_workspace_bytes(T, H, I, num_sms), dn = linear_workspace_bytes(T, I, H, num_sms);
    const size_t ch = chain_supported(T) ? chain_workspace_bytes(T, num_sms) : 0;
    const size_t scratch = gu > dn ? (gu > ch ? gu : ch) : (dn > ch ? dn : ch);
    return align256((size_t)T * I * 2) + scratch;
}

static aflex_status dense_run(aflex_ctx* ctx, const void* x, const void* wg, const void* wu, const void* wd, int T,
                              int H, int I, void* y, char* ws, size_t ws_bytes, cudaStream_t st,
                              const ChainStep* pre = nullptr) {
    Arena arena(ws, ws_bytes);
    __nv_bfloat16* h = arena.take<__nv_bfloat16>((size_t)T * I);
    // the two GEMMs run back to back on one stream: they share one scratch region and one counter array
    const size_t gu = gateup_workspace_bytes(T, H, I, ctx->num_sms), dn = linear_workspace_bytes(T, I, H, ctx->num_sms);
    const size_t ch = chain_supported(T) ? chain_workspace_bytes(T, ctx->num_sms) : 0;
    const size_t scratch = gu > dn ? (gu > ch ? gu : ch) : (dn > ch ? dn : ch);
    char* sws = scratch ? arena.take<char>(scratch) : nullptr;
    if (arena.overflow)
        return set_error(ctx, AFLEX_ERR_WORKSPACE, "dense ffn: need %zu workspace bytes, have %zu",
                         dense_ws_bytes(T, H, I, ctx->num_sms), ws_bytes);
    if (chain_supported(T)) {
        // decode batch: gate/up and down as two phases of one persistent kernel (x_pre, when given, is a projection
        // that produces x and becomes a phase in front of them)
        ChainStep steps[3];
        int n = 0;
        if (pre) steps[n++] = *pre;
        steps[n++] = ChainStep{x, wg, wu, H, I, h};
        steps[n++] = ChainStep{h, wd, nullptr, I, H, y};
        return chain_launch(ctx, steps, n, T, sws, scratch, st, ctx->chain_counters);
    }
    if (pre) {
        aflex_status sp = linear_launch(ctx, pre->in, pre->w0, T, pre->K, pre->N, pre->out, sws, scratch, st, kKLinearGemm, ctx->counters_f);
        if (sp != AFLEX_OK) return sp;
    }
    aflex_status s = gateup_launch(ctx, x, wg, wu, T, H, I, h, sws, scratch, st, ctx->counters_f);
    if (s != AFLEX_OK) return s;
    return linear_launch(ctx, h, wd, T, I, H, y, sws, scratch, st, kKDownGemm, ctx->counters_f);
}

// Decode batch, dense FFN, whole decoder layer: the output projection, the residual add, the RMS normalisation in
// front of the FFN and the FFN itself as ONE chain launch.  a [T][A] is the attention output; resid [T][H] is updated in
// place (resid += a W_o^T); xg [T][H] is scratch (the gain-weighted residual rows, the FFN's input before the row scale).
// With next_qkv: the down projection's output is added to the residual rows as well, normalised for the NEXT layer
// (gain next_gain, rows left in xn) and pushed through that layer's QKV projection (w_qkv [NQ][H] -> qkv [T][NQ]); y is
// then not written.
static aflex_status dense_fused_run(aflex_ctx* ctx, const void* a, const void* w_o, int A, void* resid, const void* gain, float eps,
                                    void* xg, const void* wg, const void* wu, const void* wd, int T, int H, int I, void* y,
                                    char* ws, size_t ws_bytes, cudaStream_t st, const void* next_gain = nullptr,
                                    float next_eps = 0.f, void* xn = nullptr, const void* w_qkv = nullptr, int NQ = 0,
                                    void* qkv = nullptr) {
    Arena arena(ws, ws_bytes);
    __nv_bfloat16* h = arena.take<__nv_bfloat16>((size_t)T * I);
    const size_t scratch = chain_workspace_bytes(T, ctx->num_sms);
    char* sws = arena.take<char>(scratch);
    if (arena.overflow)
        return set_error(ctx, AFLEX_ERR_WORKSPACE, "fused dense layer: need %zu workspace bytes, have %zu",
                         dense_ws_bytes(T, H, I, ctx->num_sms), ws_bytes);
    ChainStep steps[4];
    steps[0] = ChainStep{a, w_o, nullptr, A, H, xg};
    steps[0].resid_in = resid; steps[0].resid_out = resid; steps[0].gain = gain; steps[0].eps = eps;
    steps[1] = ChainStep{xg, wg, wu, H, I, h};
    if (w_qkv == nullptr) {
        steps[2] = ChainStep{h, wd, nullptr, I, H, y};
        return chain_launch(ctx, steps, 3, T, sws, scratch, st, ctx->chain_counters);
    }
    steps[2] = ChainStep{h, wd, nullptr, I, H, xn};
    steps[2].resid_in = resid; steps[2].resid_out = resid; steps[2].gain = next_gain; steps[2].eps = next_eps;
    steps[3] = ChainStep{xn, w_qkv, nullptr, H, NQ, qkv};
    return chain_launch(ctx, steps, 4, T, sws, scratch, st, ctx->chain_counters);
}

static size_t moe_ws_bytes(int T, int H, int I, int E, int K, int num_sms) {
    const size_t R = (size_t)T * K;
    size_t b = 0;
    b += align256(R * 4) * 3;                   // idx, gate, pos
    b += align256((size_t)E * 4) + align256((size_t)(E + 1) * 4);
    b += align256((size_t)T * E * 4);           // logits
    b += align256(R * H * 2);                   // xp
    b += align256(R * I * 2);                   // hp
    b += align256(R * H * 4);                   // yp
    const size_t gu = grouped_workspace_bytes(1, (int)R, T, H, I, E, num_sms);
    const size_t dn = grouped_workspace_bytes(0, (int)R, T, I, H, E, num_sms);
    b += gu > dn ? gu : dn;
    return b;
}

static aflex_status moe_run(aflex_ctx* ctx, const void* x, const float* router_logits, const void* w_router,
                            const void* wg, const void* wu, const void* wd, int T, int H, int I, int E, int K, void* y,
                            int32_t* topk_idx, float* topk_gate, int32_t* expert_counts, char* ws, size_t ws_bytes,
                            cudaStream_t st) {
    const size_t R = (size_t)T * K;
    Arena arena(ws, ws_bytes);
    MoeBuffers mb;
    mb.idx = arena.take<int32_t>(R);
    mb.gate = arena.take<float>(R);
    mb.pos = arena.take<int32_t>(R);
    mb.counts = arena.take<int32_t>(E);
    mb.offsets = arena.take<int32_t>(E + 1);
    mb.logits = arena.take<float>((size_t)T * E);
    __nv_bfloat16* xp = arena.take<__nv_bfloat16>(R * H);
    __nv_bfloat16* hp = arena.take<__nv_bfloat16>(R * I);
    float* yp = arena.take<float>(R * H);
    const size_t gu = grouped_workspace_bytes(1, (int)R, T, H, I, E, ctx->num_sms);
    const size_t dn = grouped_workspace_bytes(0, (int)R, T, I, H, E, ctx->num_sms);
    const size_t gws = gu > dn ? gu : dn;
    char* gw = gws ? arena.take<char>(gws) : nullptr;
    if (arena.overflow)
        return set_error(ctx, AFLEX_ERR_WORKSPACE, "moe ffn: need %zu workspace bytes, have %zu",
                         moe_ws_bytes(T, H, I, E, K, ctx->num_sms), ws_bytes);
    aflex_status s;
    const float* logits = router_logits;
    if (!logits) {
        s = moe_router_logits_launch(ctx, x, w_router, T, H, E, mb.logits, st);
        if (s != AFLEX_OK) return s;
        logits = mb.logits;
    }
    s = moe_route_launch(ctx, logits, T, E, K, mb, st);
    if (s != AFLEX_OK) return s;
    s = moe_gather_launch(ctx, x, mb.pos, T, K, H, xp, st);
    if (s != AFLEX_OK) return s;
    // an expert receives at most one assignment per token => segments have at most T rows
    s = grouped_gateup_launch(ctx, xp, wg, wu, mb.offsets, (int)R, T, H, I, E, hp, gw, gws, st, ctx->counters_f);
    if (s != AFLEX_OK) return s;
    s = grouped_linear_launch(ctx, hp, wd, mb.offsets, (int)R, T, I, H, E, yp, gw, gws, st, ctx->counters_f);
    if (s != AFLEX_OK) return s;
    s = moe_combine_launch(ctx, yp, mb.pos, mb.gate, T, K, H, y, st);
    if (s != AFLEX_OK) return s;
    if (topk_idx) { s = check_cuda(ctx, cudaMemcpyAsync(topk_idx, mb.idx, R * 4, cudaMemcpyDeviceToDevice, st), "copy topk_idx"); if (s != AFLEX_OK) return s; }
    if (topk_gate) { s = check_cuda(ctx, cudaMemcpyAsync(topk_gate, mb.gate, R * 4, cudaMemcpyDeviceToDevice, st), "copy topk_gate"); if (s != AFLEX_OK) return s; }
    if (expert_counts) { s = check_cuda(ctx, cudaMemcpyAsync(expert_counts, mb.counts, (size_t)E * 4, cudaMemcpyDeviceToDevice, st), "copy expert_counts"); if (s != AFLEX_OK) return s; }
    return AFLEX_OK;
}

static aflex_status validate_moe(aflex_ctx* ctx, int T, int H, int I, int E, int K) {
    aflex_status s = validate_ffn_dims(ctx, T, H, I);
    if (s != AFLEX_OK) return s;
    if (E < 1 || K < 1) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "moe: E and top_k must be >= 1");
    if (K > E) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "moe: top_k > num_experts");
    if (E > 64 || K > 2) return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "moe: supported E <= 64, top_k in {1,2}");
    return AFLEX_OK;
}

}  // namespace aflex

using namespace aflex;

extern "C" {

const char* aflex_status_string(aflex_status s) {
    switch (s) {
        case AFLEX_OK: return "AFLEX_OK";
        case AFLEX_ERR_INVALID_ARG: return "AFLEX_ERR_INVALID_ARG";
        case AFLEX_ERR_UNSUPPORTED: return "AFLEX_ERR_UNSUPPORTED";
        case AFLEX_ERR_WORKSPACE: return "AFLEX_ERR_WORKSPACE";
        case AFLEX_ERR_CUDA: return "AFLEX_ERR_CUDA";
        case AFLEX_ERR_TIMEOUT: return "AFLEX_ERR_TIMEOUT";
        case AFLEX_ERR_BOUNDS: return "AFLEX_ERR_BOUNDS";
    }
    return "AFLEX_ERR_UNKNOWN";
}

int aflex_version(void) { return 100; }

aflex_status aflex_create(aflex_ctx** out, int device, size_t workspace_bytes) {
    if (!out) return AFLEX_ERR_INVALID_ARG;
    *out = nullptr;
    aflex_ctx* ctx = new (std::nothrow) aflex_ctx();
    if (!ctx) return AFLEX_ERR_CUDA;
    ctx->device = device;
    { const char* ev = getenv("AFLEX_MB_STREAMS"); ctx->mb_two_streams = ev && atoi(ev) == 2; }
    ctx->ws_bytes = workspace_bytes ? align256(workspace_bytes) : kDefaultWorkspace;
    cudaError_t e = cudaSetDevice(device);
    cudaDeviceProp prop;
    if (e == cudaSuccess) e = cudaGetDeviceProperties(&prop, device);
    if (e == cudaSuccess) {
        ctx->num_sms = prop.multiProcessorCount;
        if (prop.major != 10) {
            delete ctx;
            return AFLEX_ERR_UNSUPPORTED;   // kernels are built for sm_100a only
        }
    }
    if (e == cudaSuccess) e = cudaMalloc(&ctx->ws, ctx->ws_bytes);
    if (e == cudaSuccess) e = cudaMalloc(&ctx->dev_status, sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(ctx->dev_status, 0, sizeof(int));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->counters_attn, (kAttnCounterCap + 16) * sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(ctx->counters_attn, 0, (kAttnCounterCap + 16) * sizeof(int));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->counters_a, 2 * kStreamKMaxTiles * sizeof(int));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->counters_f, 2 * kStreamKMaxTiles * sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(ctx->counters_a, 0, 2 * kStreamKMaxTiles * sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(ctx->counters_f, 0, 2 * kStreamKMaxTiles * sizeof(int));
    if (e == cudaSuccess) e = cudaMalloc(&ctx->chain_counters, chain_counter_ints() * sizeof(int));
    if (e == cudaSuccess) e = cudaMemset(ctx->chain_counters, 0, chain_counter_ints() * sizeof(int));
    if (e == cudaSuccess && getenv("AFLEX_TRACE") && atoi(getenv("AFLEX_TRACE")) > 0) {
        const size_t tb = (size_t)kTraceKernels * kTraceStride * sizeof(unsigned long long);
        e = cudaMalloc(&ctx->trace, tb);
        if (e == cudaSuccess) e = cudaMemset(ctx->trace, 0, tb);
    }
    if (e == cudaSuccess) e = cudaMallocHost(&ctx->host_status, sizeof(int));
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->stream_a, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->stream_f, cudaStreamNonBlocking);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_entry, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_a_done, cudaEventDisableTiming);
    if (e == cudaSuccess) e = cudaEventCreateWithFlags(&ctx->ev_f_done, cudaEventDisableTiming);
    for (int i = 0; i < kMaxMicrobatches && e == cudaSuccess; ++i)
        e = cudaEventCreateWithFlags(&ctx->ev_a[i], cudaEventDisableTiming);
    for (int i = 0; i < kMaxMicrobatches && e == cudaSuccess; ++i)
        e = cudaEventCreateWithFlags(&ctx->ev_f[i], cudaEventDisableTiming);
    if (e != cudaSuccess || !get_encode_fn()) {
        aflex_destroy(ctx);
        return AFLEX_ERR_CUDA;
    }
    *out = ctx;
    return AFLEX_OK;
}

aflex_status aflex_destroy(aflex_ctx* ctx) {
    if (!ctx) return AFLEX_OK;
    cudaSetDevice(ctx->device);
    if (ctx->stream_a) cudaStreamSynchronize(ctx->stream_a);
    if (ctx->stream_f) cudaStreamSynchronize(ctx->stream_f);
    for (int i = 0; i < kMaxMicrobatches; ++i) if (ctx->ev_a[i]) cudaEventDestroy(ctx->ev_a[i]);
    for (int i = 0; i < kMaxMicrobatches; ++i) if (ctx->ev_f[i]) cudaEventDestroy(ctx->ev_f[i]);
    if (ctx->ev_entry) cudaEventDestroy(ctx->ev_entry);
    if (ctx->ev_a_done) cudaEventDestroy(ctx->ev_a_done);
    if (ctx->ev_f_done) cudaEventDestroy(ctx->ev_f_done);
    if (ctx->stream_a) cudaStreamDestroy(ctx->stream_a);
    if (ctx->stream_f) cudaStreamDestroy(ctx->stream_f);
    if (ctx->prof) {
        for (int i = 0; i < kProfMaxSlots; ++i) {
            if (ctx->prof[i].start) cudaEventDestroy(ctx->prof[i].start);
            if (ctx->prof[i].stop) cudaEventDestroy(ctx->prof[i].stop);
        }
        delete[] ctx->prof;
    }
    if (ctx->host_status) cudaFreeHost(ctx->host_status);
    if (ctx->dev_status) cudaFree(ctx->dev_status);
    if (ctx->trace) cudaFree(ctx->trace);
    if (ctx->counters_attn) cudaFree(ctx->counters_attn);
    if (ctx->counters_a) cudaFree(ctx->counters_a);
    if (ctx->counters_f) cudaFree(ctx->counters_f);
    if (ctx->chain_counters) cudaFree(ctx->chain_counters);
    if (ctx->ws) cudaFree(ctx->ws);
    delete ctx;
    return AFLEX_OK;
}

const char* aflex_last_error(const aflex_ctx* ctx) { return ctx ? ctx->err : "null context"; }

aflex_status aflex_get_device_status(aflex_ctx* ctx, void* stream) {
    if (!ctx) return AFLEX_ERR_INVALID_ARG;
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemcpyAsync(ctx->host_status, ctx->dev_status, sizeof(int), cudaMemcpyDeviceToHost, st);
    if (e == cudaSuccess) e = cudaMemsetAsync(ctx->dev_status, 0, sizeof(int), st);
    if (e == cudaSuccess) e = cudaStreamSynchronize(st);
    if (e != cudaSuccess) return check_cuda(ctx, e, "aflex_get_device_status");
    const int v = *ctx->host_status;
    if (v != 0) {
        // a kernel that gave up may have left arrival counters half-way: restore the all-zero state
        cudaMemsetAsync(ctx->counters_attn, 0, (kAttnCounterCap + 16) * sizeof(int), st);
        cudaMemsetAsync(ctx->counters_a, 0, 2 * kStreamKMaxTiles * sizeof(int), st);
        cudaMemsetAsync(ctx->counters_f, 0, 2 * kStreamKMaxTiles * sizeof(int), st);
        cudaMemsetAsync(ctx->chain_counters, 0, chain_counter_ints() * sizeof(int), st);
        cudaStreamSynchronize(st);
    }
    if (v != 0) set_error(ctx, (aflex_status)v, "device status word = %d (%s)", v, aflex_status_string((aflex_status)v));
    return (aflex_status)v;
}

static const char* kKernelNames[kKKindCount] = {
    "attn_decode", "linear_gemm", "down_gemm", "gateup_gemm", "router_logits",
    "moe_route", "moe_gather", "moe_gateup_gemm", "moe_down_gemm", "moe_combine",
    "add_rmsnorm", "qkv_gemm", "rope_append", "attn_prefill", "gemm_chain"};

int aflex_num_kernel_kinds(void) { return kKKindCount; }

const char* aflex_kernel_name(int kind) { return (kind >= 0 && kind < kKKindCount) ? kKernelNames[kind] : "?"; }

long long aflex_launch_count(const aflex_ctx* ctx, int kind) {
    if (!ctx) return 0;
    if (kind >= 0 && kind < kKKindCount) return ctx->launches[kind];
    long long t = 0;
    for (int i = 0; i < kKKindCount; ++i) t += ctx->launches[i];
    return t;
}

aflex_status aflex_profile_enable(aflex_ctx* ctx, int on) {
    if (!ctx) return AFLEX_ERR_INVALID_ARG;
    if (on && !ctx->prof) {
        ctx->prof = new (std::nothrow) ProfSlot[kProfMaxSlots]();
        if (!ctx->prof) return set_error(ctx, AFLEX_ERR_CUDA, "profile: out of host memory");
        for (int i = 0; i < kProfMaxSlots; ++i) {
            cudaError_t e = cudaEventCreate(&ctx->prof[i].start);
            if (e == cudaSuccess) e = cudaEventCreate(&ctx->prof[i].stop);
            if (e != cudaSuccess) return check_cuda(ctx, e, "profile: cudaEventCreate");
        }
    }
    if (on) ctx->prof_used = 0;
    ctx->profiling = on != 0;
    return AFLEX_OK;
}

aflex_status aflex_profile_read(aflex_ctx* ctx, int kind, double* total_ms, long long* launches) {
    if (!ctx || !total_ms || !launches || kind < 0 || kind >= kKKindCount) return AFLEX_ERR_INVALID_ARG;
    *total_ms = 0.0;
    *launches = 0;
    for (int i = 0; i < ctx->prof_used; ++i) {
        if (ctx->prof[i].kind != kind) continue;
        cudaError_t e = cudaEventSynchronize(ctx->prof[i].stop);
        float ms = 0.f;
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, ctx->prof[i].start, ctx->prof[i].stop);
        if (e != cudaSuccess) return check_cuda(ctx, e, "profile: event read");
        *total_ms += ms;
        *launches += 1;
    }
    return AFLEX_OK;
}

aflex_status aflex_trace_read(aflex_ctx* ctx, unsigned long long* host_out, int launches, int* next_slot) {
    if (!ctx || !host_out || launches < 1 || launches > kTraceKernels) return AFLEX_ERR_INVALID_ARG;
    if (!ctx->trace) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "tracing is off (create the ctx with AFLEX_TRACE=1)");
    cudaError_t e = cudaDeviceSynchronize();
    if (e == cudaSuccess)
        e = cudaMemcpy(host_out, ctx->trace, (size_t)launches * kTraceStride * sizeof(unsigned long long), cudaMemcpyDeviceToHost);
    if (next_slot) *next_slot = ctx->trace_slot;
    ctx->trace_slot = 0;
    return check_cuda(ctx, e, "aflex_trace_read");
}

aflex_status aflex_set_attn_q_final(aflex_ctx* ctx, int on) {
    if (!ctx) return AFLEX_ERR_INVALID_ARG;
    ctx->attn_q_final = on != 0;
    return AFLEX_OK;
}

aflex_status aflex_set_interleave_streams(aflex_ctx* ctx, int on) {
    if (!ctx) return AFLEX_ERR_INVALID_ARG;
    ctx->mb_two_streams = on != 0;
    return AFLEX_OK;
}

aflex_status aflex_set_attn_ctas(aflex_ctx* ctx, int ctas) {
    if (!ctx || ctas < 0 || ctas > 4096) return AFLEX_ERR_INVALID_ARG;
    ctx->attn_ctas = ctas;
    return AFLEX_OK;
}

aflex_status aflex_attn_decode(aflex_ctx* ctx, const aflex_attn_desc* desc, const void* q, const aflex_kv* kv, int batch,
                               void* out, float* lse, void* stream) {
    aflex_status s = validate_attn(ctx, desc, q, kv, batch, out);
    if (s != AFLEX_OK) return s;
    return attn_decode_launch(ctx, desc, q, kv, batch, out, lse, ctx->ws, ctx->ws_bytes,
                              reinterpret_cast<cudaStream_t>(stream));
}

aflex_status aflex_attn_prefill(aflex_ctx* ctx, const aflex_attn_desc* desc, const void* q, const aflex_kv* kv, int batch,
                                const int32_t* q_offsets, const int32_t* q_offsets_host, void* out, void* stream) {
    aflex_status s = validate_attn(ctx, desc, q, kv, batch, out);
    if (s != AFLEX_OK) return s;
    if (!q_offsets || !q_offsets_host) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "prefill attention: null q_offsets");
    if (kv->seq_lens_host) {
        for (int b = 0; b < batch; ++b)
            if (q_offsets_host[b + 1] - q_offsets_host[b] > kv->seq_lens_host[b])
                return set_error(ctx, AFLEX_ERR_INVALID_ARG, "prefill attention: sequence %d has more queries than cached tokens", b);
    }
    return attn_prefill_launch(ctx, desc, q, kv, batch, q_offsets, q_offsets_host, out, reinterpret_cast<cudaStream_t>(stream));
}

aflex_status aflex_linear(aflex_ctx* ctx, const void* x, const void* w, int T, int K, int N, void* y, void* stream) {
    if (!ctx) return AFLEX_ERR_INVALID_ARG;
    if (!x || !w || !y || T < 1 || K < 1 || N < 1) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "linear: bad argument");
    if (K % 8 || N % 8) return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "linear: K and N must be multiples of 8");
    if (!aligned16(x) || !aligned16(w) || !aligned16(y)) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "linear: pointers must be 16-byte aligned");
    return linear_launch(ctx, x, w, T, K, N, y, ctx->ws, ctx->ws_bytes, reinterpret_cast<cudaStream_t>(stream), kKLinearGemm, ctx->counters_a);
}

aflex_status aflex_ffn_dense(aflex_ctx* ctx, const void* x, const void* w_gate, const void* w_up, const void* w_down,
                             int T, int H, int I, void* y, void* stream) {
    if (!ctx) return AFLEX_ERR_INVALID_ARG;
    if (!x || !w_gate || !w_up || !w_down || !y) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "dense ffn: null argument");
    aflex_status s = validate_ffn_dims(ctx, T, H, I);
    if (s != AFLEX_OK) return s;
    if (!aligned16(x) || !aligned16(w_gate) || !aligned16(w_up) || !aligned16(w_down) || !aligned16(y))
        return set_error(ctx, AFLEX_ERR_INVALID_ARG, "dense ffn: pointers must be 16-byte aligned");
    return dense_run(ctx, x, w_gate, w_up, w_down, T, H, I, y, ctx->ws, ctx->ws_bytes,
                     reinterpret_cast<cudaStream_t>(stream));
}

aflex_status aflex_ffn_moe(aflex_ctx* ctx, const void* x, const float* router_logits, const void* w_router,
                           const void* w_gate, const void* w_up, const void* w_down, int T, int H, int I, int E, int top_k,
                           void* y, int32_t* topk_idx, float* topk_gate, int32_t* expert_counts, void* stream) {
    if (!ctx) return AFLEX_ERR_INVALID_ARG;
    if (!x || !w_gate || !w_up || !w_down || !y) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "moe ffn: null argument");
    if ((router_logits == nullptr) == (w_router == nullptr))
        return set_error(ctx, AFLEX_ERR_INVALID_ARG, "moe ffn: exactly one of router_logits and w_router must be given");
    aflex_status s = validate_moe(ctx, T, H, I, E, top_k);
    if (s != AFLEX_OK) return s;
    if (!aligned16(x) || !aligned16(w_gate) || !aligned16(w_up) || !aligned16(w_down) || !aligned16(y))
        return set_error(ctx, AFLEX_ERR_INVALID_ARG, "moe ffn: pointers must be 16-byte aligned");
    return moe_run(ctx, x, router_logits, w_router, w_gate, w_up, w_down, T, H, I, E, top_k, y, topk_idx, topk_gate,
                   expert_counts, ctx->ws, ctx->ws_bytes, reinterpret_cast<cudaStream_t>(stream));
}

aflex_status aflex_moe_route(aflex_ctx* ctx, const float* router_logits, int T, int E, int top_k, int32_t* topk_idx,
                             float* topk_gate, int32_t* expert_counts, int32_t* expert_offsets, int32_t* pos, void* stream) {
    if (!ctx) return AFLEX_ERR_INVALID_ARG;
    if (!router_logits || !topk_idx || !topk_gate || !expert_counts || !expert_offsets || !pos)
        return set_error(ctx, AFLEX_ERR_INVALID_ARG, "moe route: null argument");
    aflex_status s = validate_moe(ctx, T, 8, 8, E, top_k);
    if (s != AFLEX_OK) return s;
    MoeBuffers mb;
    mb.idx = topk_idx; mb.gate = topk_gate; mb.counts = expert_counts; mb.offsets = expert_offsets; mb.pos = pos;
    mb.logits = nullptr;
    return moe_route_launch(ctx, router_logits, T, E, top_k, mb, reinterpret_cast<cudaStream_t>(stream));
}

// Workspace layout of the layer step: [A region | attention output a | boundary x | F region].
// The A region (attention partials, W_o split-K partials) is used only on the attention stream,
// the F region only on the FFN stream; a and x are indexed by batch row, so microbatches touch
// disjoint slices.
namespace {
struct LayerWs {
    size_t a_attn, a_lin, a_total, attn_out, x, f_total, total;
};
// a_attn: bytes the attention partials need (the caller knows the chunk plan).
LayerWs layer_ws(const aflex_layer_desc* L, int max_batch, size_t a_attn, int num_sms) {
    LayerWs w;
    const int A = L->attn.num_q_heads * L->attn.head_dim;
    w.a_attn = a_attn;
    w.a_lin = L->w_o ? linear_workspace_bytes(max_batch, A, L->hidden, num_sms) : 0;
    // split-K plans depend on T; take the max over the microbatch sizes 1..max_batch that matter
    if (L->w_o) {
        for (int t = 1; t <= max_batch; t = t < 16 ? t + 1 : t + 16) {
            size_t b = linear_workspace_bytes(t, A, L->hidden, num_sms);
            if (b > w.a_lin) w.a_lin = b;
        }
    }
    w.a_total = w.a_attn + w.a_lin;
    w.attn_out = align256((size_t)max_batch * A * 2);
    w.x = L->w_o ? align256((size_t)max_batch * L->hidden * 2) : 0;
    size_t f = 0;
    for (int t = 1; t <= max_batch; t = t < 16 ? t + 1 : t + 16) {
        size_t b = L->num_experts == 0 ? dense_ws_bytes(t, L->hidden, L->inter, num_sms)
                                       : moe_ws_bytes(t, L->hidden, L->inter, L->num_experts, L->top_k, num_sms);
        if (b > f) f = b;
    }
    {
        size_t b = L->num_experts == 0 ? dense_ws_bytes(max_batch, L->hidden, L->inter, num_sms)
                                       : moe_ws_bytes(max_batch, L->hidden, L->inter, L->num_experts, L->top_k, num_sms);
        if (b > f) f = b;
    }
    w.f_total = f;
    w.total = w.a_total + w.attn_out + w.x + w.f_total + 1024;
    return w;
}
}  // namespace

// SM count the workspace queries size for: the current device's (the per-SM scratch of the persistent
// kernels scales with it, and the entry points size the same regions from their ctx's device), or 148
// when no device can be asked (a host without a GPU).
static int query_num_sms() {
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) == cudaSuccess && cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) == cudaSuccess && sms > 0)
        return sms;
    (void)cudaGetLastError();   // no device: not an error of this query
    return 148;
}

size_t aflex_workspace_bytes(const aflex_layer_desc* layer, int max_batch, int max_pages_per_seq) {
    if (!layer || max_batch < 1 || max_pages_per_seq < 1) return 0;
    (void)max_pages_per_seq;   // the attention scratch is per CTA, not per context token
    return layer_ws(layer, max_batch, attn_workspace_bytes(&layer->attn, 4096), query_num_sms()).total;
}

aflex_status aflex_layer_step(aflex_ctx* ctx, const aflex_layer_desc* L, const void* q, const aflex_kv* kv, int batch,
                              const float* router_logits, int M, const int32_t* mb_offsets, void* attn_out, void* y,
                              void* stream) {
    if (!ctx) return AFLEX_ERR_INVALID_ARG;
    if (!L || !y) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "layer step: null argument");
    aflex_status s = validate_attn(ctx, &L->attn, q, kv, batch, y);
    if (s != AFLEX_OK) return s;
    const int A = L->attn.num_q_heads * L->attn.head_dim;
    const int H = L->hidden, I = L->inter, E = L->num_experts, K = L->top_k;
    if (!L->w_gate || !L->w_up || !L->w_down) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "layer step: null FFN weights");
    if (!L->w_o && A != H) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "layer step: w_o is required when Hq*D != hidden");
    if (A % 8) return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "layer step: Hq*D must be a multiple of 8");
    if (E == 0) s = validate_ffn_dims(ctx, batch, H, I);
    else {
        s = validate_moe(ctx, batch, H, I, E, K);
        if (s == AFLEX_OK && (router_logits == nullptr) == (L->w_router == nullptr))
            s = set_error(ctx, AFLEX_ERR_INVALID_ARG, "layer step: exactly one of router_logits and w_router must be given");
    }
    if (s != AFLEX_OK) return s;
    if (M < 1 || M > batch || M > kMaxMicrobatches)
        return set_error(ctx, AFLEX_ERR_INVALID_ARG, "layer step: microbatch depth %d outside [1, min(batch, %d)]", M, kMaxMicrobatches);
    int32_t offs[kMaxMicrobatches + 1];
    if (mb_offsets) {
        for (int i = 0; i <= M; ++i) offs[i] = mb_offsets[i];
        if (offs[0] != 0 || offs[M] != batch) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "layer step: mb_offsets must run from 0 to batch");
        for (int i = 0; i < M; ++i)
            if (offs[i + 1] <= offs[i]) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "layer step: mb_offsets must be strictly increasing");
    } else {
        const int base = batch / M, extra = batch % M;
        offs[0] = 0;
        for (int i = 0; i < M; ++i) offs[i + 1] = offs[i] + base + (i < extra ? 1 : 0);
    }

    const size_t a_attn = attn_workspace_bytes(&L->attn, attn_grid(ctx));
    const LayerWs w = layer_ws(L, batch, a_attn, ctx->num_sms);
    if (w.total > ctx->ws_bytes)
        return set_error(ctx, AFLEX_ERR_WORKSPACE, "layer step: need %zu workspace bytes, have %zu", w.total, ctx->ws_bytes);
    char* ws_a = ctx->ws;
    char* ws_alin = ws_a + w.a_attn;
    __nv_bfloat16* a_buf = attn_out ? reinterpret_cast<__nv_bfloat16*>(attn_out)
                                    : reinterpret_cast<__nv_bfloat16*>(ctx->ws + w.a_total);
    __nv_bfloat16* x_buf = L->w_o ? reinterpret_cast<__nv_bfloat16*>(ctx->ws + w.a_total + w.attn_out) : a_buf;
    char* ws_f = ctx->ws + w.a_total + w.attn_out + w.x;

    cudaStream_t user = reinterpret_cast<cudaStream_t>(stream);
    // M = 1 is A then F in series (Eq. 2, first case): everything goes on the caller's stream, where
    // consecutive kernels chain through programmatic dependent launch.  So does M >= 2 by default, in the
    // order A_0, F_0, A_1, F_1, ...: on one GPU a kernel of either side fills every SM, so the sides cannot
    // run at the same time and the chained launches have the shorter boundaries.  On request M >= 2 uses the
    // ctx's attention and FFN streams, joined to the caller's stream on entry and exit.
    const bool serial = (M == 1) || !ctx->mb_two_streams;
    cudaStream_t sa = serial ? user : ctx->stream_a, sf = serial ? user : ctx->stream_f;
    cudaError_t e = cudaSuccess;
    if (!serial) {
        e = cudaEventRecord(ctx->ev_entry, user);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(sa, ctx->ev_entry, 0);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(sf, ctx->ev_entry, 0);
        if (e != cudaSuccess) return check_cuda(ctx, e, "layer step: entry join");
    }

    const int Hq = L->attn.num_q_heads, D = L->attn.head_dim;
    for (int i = 0; i < M; ++i) {
        const int r0 = offs[i], rows = offs[i + 1] - offs[i];
        // ---- A_i on the attention stream
        aflex_kv kvi = *kv;
        kvi.page_table = kv->page_table + (size_t)r0 * kv->max_pages_per_seq;
        kvi.seq_lens = kv->seq_lens + r0;
        kvi.seq_lens_host = kv->seq_lens_host ? kv->seq_lens_host + r0 : nullptr;
        const __nv_bfloat16* qi = reinterpret_cast<const __nv_bfloat16*>(q) + (size_t)r0 * Hq * D;
        s = attn_decode_launch(ctx, &L->attn, qi, &kvi, rows, a_buf + (size_t)r0 * A, nullptr, ws_a, w.a_attn, sa);
        if (s != AFLEX_OK) return s;
        // M = 1, dense FFN, decode batch: W_o, gate/up and down are the three phases of one persistent kernel
        const bool chain3 = serial && E == 0 && L->w_o && chain_supported(rows);
        if (L->w_o && !chain3) {
            s = linear_launch(ctx, a_buf + (size_t)r0 * A, L->w_o, rows, A, H, x_buf + (size_t)r0 * H, ws_alin, w.a_lin, sa, kKLinearGemm, ctx->counters_a);
            if (s != AFLEX_OK) return s;
        }
        if (!serial) {
            e = cudaEventRecord(ctx->ev_a[i], sa);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(sf, ctx->ev_a[i], 0);
            if (e != cudaSuccess) return check_cuda(ctx, e, "layer step: A->F event");
        }
        // ---- F_i on the FFN stream
        __nv_bfloat16* yi = reinterpret_cast<__nv_bfloat16*>(y) + (size_t)r0 * H;
        const __nv_bfloat16* xi = x_buf + (size_t)r0 * H;
        if (E == 0) {
            const ChainStep wo_step{a_buf + (size_t)r0 * A, L->w_o, nullptr, A, H, x_buf + (size_t)r0 * H};
            s = dense_run(ctx, xi, L->w_gate, L->w_up, L->w_down, rows, H, I, yi, ws_f, w.f_total, sf, chain3 ? &wo_step : nullptr);
        } else {
            s = moe_run(ctx, xi, router_logits ? router_logits + (size_t)r0 * E : nullptr, L->w_router, L->w_gate,
                        L->w_up, L->w_down, rows, H, I, E, K, yi, nullptr, nullptr, nullptr, ws_f, w.f_total, sf);
        }
        if (s != AFLEX_OK) return s;
    }
    if (serial) return AFLEX_OK;
    e = cudaEventRecord(ctx->ev_a_done, sa);
    if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_f_done, sf);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(user, ctx->ev_a_done, 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(user, ctx->ev_f_done, 0);
    return check_cuda(ctx, e, "layer step: exit join");
}

// AFLEX_DECODER_FUSE=0: keep W_o, the residual add + RMS normalisation and the FFN as separate launches (tuning / comparison).
static bool decoder_fuse() {
    static int v = -1;
    if (v < 0) { const char* e = getenv("AFLEX_DECODER_FUSE"); v = e ? atoi(e) : 1; }
    return v != 0;
}

// ---- whole decoder layers ------------------------------------------------------------------
// Workspace: [A scratch | resid | xn | qkv | q | a | o | xn2 | y | F scratch].  The row-indexed
// buffers are touched by microbatch i only in rows of i, in the order A_{l,i} -> F_{l,i} ->
// A_{l+1,i} that the events enforce; the A scratch is used on the attention stream only, the F
// scratch on the FFN stream only.
namespace {
struct DecoderWs {
    size_t a_attn, a_lin, rows_h, rows_qkv, rows_a, f_total, total;
};
DecoderWs decoder_ws(const aflex_decoder_desc* d, int max_batch, size_t a_attn, int num_sms) {
    const aflex_layer_desc* L = &d->layer;
    const int D = L->attn.head_dim, A = L->attn.num_q_heads * D, H = L->hidden;
    const int NQ = (L->attn.num_q_heads + 2 * L->attn.num_kv_heads) * D;
    DecoderWs w;
    w.a_attn = a_attn;
    w.a_lin = 0;
    for (int t = 1; t <= max_batch; t = (t < 16 ? t + 1 : t + 16)) {
        const size_t b0 = linear_workspace_bytes(t, A, H, num_sms), b1 = linear_workspace_bytes(t, H, NQ, num_sms);
        if (b0 > w.a_lin) w.a_lin = b0;
        if (b1 > w.a_lin) w.a_lin = b1;
    }
    {
        const size_t b0 = linear_workspace_bytes(max_batch, A, H, num_sms), b1 = linear_workspace_bytes(max_batch, H, NQ, num_sms);
        if (b0 > w.a_lin) w.a_lin = b0;
        if (b1 > w.a_lin) w.a_lin = b1;
    }
    w.rows_h = align256((size_t)max_batch * H * 2);
    w.rows_qkv = align256((size_t)max_batch * NQ * 2);
    w.rows_a = align256((size_t)max_batch * A * 2);
    w.f_total = layer_ws(L, max_batch, 0, num_sms).f_total;
    w.total = w.a_attn + w.a_lin + 5 * w.rows_h + w.rows_qkv + 2 * w.rows_a + w.f_total + 1024;
    return w;
}
}  // namespace

size_t aflex_decoder_workspace_bytes(const aflex_decoder_desc* layer, int max_batch) {
    if (!layer || max_batch < 1) return 0;
    return decoder_ws(layer, max_batch, attn_workspace_bytes(&layer->layer.attn, 4096), query_num_sms()).total;
}

aflex_status aflex_add_rmsnorm(aflex_ctx* ctx, const void* res, const void* add, const void* w, int T, int H, float eps,
                               void* res_out, void* y, void* stream) {
    if (!ctx) return AFLEX_ERR_INVALID_ARG;
    if (!res || (!res_out && !y) || (y && !w) || T < 1 || H < 1)
        return set_error(ctx, AFLEX_ERR_INVALID_ARG, "add_rmsnorm: bad argument");
    if (H % 8) return set_error(ctx, AFLEX_ERR_UNSUPPORTED, "add_rmsnorm: H must be a multiple of 8");
    if (!aligned16(res) || !aligned16(add) || !aligned16(w) || !aligned16(res_out) || !aligned16(y))
        return set_error(ctx, AFLEX_ERR_INVALID_ARG, "add_rmsnorm: pointers must be 16-byte aligned");
    return add_rmsnorm_launch(ctx, res, add, w, T, H, eps, res_out, y, reinterpret_cast<cudaStream_t>(stream));
}

aflex_status aflex_rope_append(aflex_ctx* ctx, const aflex_attn_desc* desc, const void* qkv, const aflex_kv* kv, int batch,
                               const void* w_q_norm, const void* w_k_norm, float rms_eps, float rope_theta, void* q_out,
                               void* stream) {
    aflex_status s = validate_attn(ctx, desc, qkv, kv, batch, q_out);
    if (s != AFLEX_OK) return s;
    if (!(rope_theta > 0.f)) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "rope_append: rope_theta must be > 0");
    return rope_append_launch(ctx, desc, qkv, kv, batch, w_q_norm, w_k_norm, rms_eps, rope_theta, q_out,
                              reinterpret_cast<cudaStream_t>(stream));
}

namespace {
// Argument checks shared by the single-GPU chain and the A/F pair.  Errors are recorded on ctx.
aflex_status validate_decoder_args(aflex_ctx* ctx, const aflex_decoder_desc* layers, const aflex_kv* kvs, int num_layers,
                                   const void* x_in, int batch, const void* x_out) {
    if (!layers || !kvs || !x_in || !x_out || num_layers < 1)
        return set_error(ctx, AFLEX_ERR_INVALID_ARG, "decoder layers: null argument or num_layers < 1");
    if (!aligned16(x_in) || !aligned16(x_out))
        return set_error(ctx, AFLEX_ERR_INVALID_ARG, "decoder layers: pointers must be 16-byte aligned");
    const int H = layers[0].layer.hidden;
    for (int l = 0; l < num_layers; ++l) {
        const aflex_decoder_desc* d = &layers[l];
        const aflex_layer_desc* L = &d->layer;
        aflex_status s = validate_attn(ctx, &L->attn, x_in, &kvs[l], batch, x_out);
        if (s != AFLEX_OK) return s;
        if (L->hidden != H) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "decoder layers: layer %d has another hidden size", l);
        if (!d->w_qkv || !d->w_ln_attn || !d->w_ln_ffn || !L->w_o || !L->w_gate || !L->w_up || !L->w_down)
            return set_error(ctx, AFLEX_ERR_INVALID_ARG, "decoder layers: layer %d has a null weight", l);
        if (!aligned16(d->w_qkv) || !aligned16(d->w_ln_attn) || !aligned16(d->w_ln_ffn) || !aligned16(L->w_o) ||
            !aligned16(L->w_gate) || !aligned16(L->w_up) || !aligned16(L->w_down))
            return set_error(ctx, AFLEX_ERR_INVALID_ARG, "decoder layers: pointers must be 16-byte aligned");
        if (!(d->rope_theta > 0.f) || !(d->rms_eps >= 0.f))
            return set_error(ctx, AFLEX_ERR_INVALID_ARG, "decoder layers: rope_theta must be > 0 and rms_eps >= 0");
        if (L->num_experts == 0) s = validate_ffn_dims(ctx, batch, H, L->inter);
        else {
            s = validate_moe(ctx, batch, H, L->inter, L->num_experts, L->top_k);
            if (s == AFLEX_OK && !L->w_router) s = set_error(ctx, AFLEX_ERR_INVALID_ARG, "decoder layers: MoE layer %d needs w_router", l);
        }
        if (s != AFLEX_OK) return s;
    }
    return AFLEX_OK;
}

// Microbatch offsets: the caller's (validated) or the near-equal split.
aflex_status make_offsets(aflex_ctx* ctx, int batch, int M, const int32_t* mb_offsets, int32_t* offs) {
    if (M < 1 || M > batch || M > kMaxMicrobatches)
        return set_error(ctx, AFLEX_ERR_INVALID_ARG, "microbatch depth %d outside [1, min(batch, %d)]", M, kMaxMicrobatches);
    if (mb_offsets) {
        for (int i = 0; i <= M; ++i) offs[i] = mb_offsets[i];
        if (offs[0] != 0 || offs[M] != batch) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "mb_offsets must run from 0 to batch");
        for (int i = 0; i < M; ++i)
            if (offs[i + 1] <= offs[i]) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "mb_offsets must be strictly increasing");
    } else {
        const int base = batch / M, extra = batch % M;
        offs[0] = 0;
        for (int i = 0; i < M; ++i) offs[i + 1] = offs[i] + base + (i < extra ? 1 : 0);
    }
    return AFLEX_OK;
}
}  // namespace

aflex_status aflex_decoder_layers(aflex_ctx* ctx, const aflex_decoder_desc* layers, const aflex_kv* kvs, int num_layers,
                                  const void* x_in, int batch, int M, const int32_t* mb_offsets, void* x_out,
                                  void* stream) {
    if (!ctx) return AFLEX_ERR_INVALID_ARG;
    aflex_status s = validate_decoder_args(ctx, layers, kvs, num_layers, x_in, batch, x_out);
    if (s != AFLEX_OK) return s;
    const int H = layers[0].layer.hidden;
    size_t need = 0;
    for (int l = 0; l < num_layers; ++l) {
        const DecoderWs w = decoder_ws(&layers[l], batch, attn_workspace_bytes(&layers[l].layer.attn, attn_grid(ctx)), ctx->num_sms);
        if (w.total > need) need = w.total;
    }
    if (need > ctx->ws_bytes)
        return set_error(ctx, AFLEX_ERR_WORKSPACE, "decoder layers: need %zu workspace bytes, have %zu", need, ctx->ws_bytes);
    int32_t offs[kMaxMicrobatches + 1];
    s = make_offsets(ctx, batch, M, mb_offsets, offs);
    if (s != AFLEX_OK) return s;

    cudaStream_t user = reinterpret_cast<cudaStream_t>(stream);
    // (always two streams at M >= 2 here: with the layer's small attention-side kernels between the big ones the
    //  two-stream form measured equal on the dense configurations and 4 - 5 % faster on the MoE ones)
    const bool serial = (M == 1);
    cudaStream_t sa = serial ? user : ctx->stream_a, sf = serial ? user : ctx->stream_f;
    cudaError_t e = cudaSuccess;
    if (!serial) {
        e = cudaEventRecord(ctx->ev_entry, user);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(sa, ctx->ev_entry, 0);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(sf, ctx->ev_entry, 0);
        if (e != cudaSuccess) return check_cuda(ctx, e, "decoder layers: entry join");
    }
    typedef __nv_bfloat16 bf;
    for (int l = 0; l < num_layers; ++l) {
        const aflex_decoder_desc* d = &layers[l];
        const aflex_layer_desc* L = &d->layer;
        const int Hq = L->attn.num_q_heads, Hkv = L->attn.num_kv_heads, D = L->attn.head_dim;
        const int A = Hq * D, NQ = (Hq + 2 * Hkv) * D, I = L->inter, E = L->num_experts;
        const DecoderWs w = decoder_ws(d, batch, attn_workspace_bytes(&L->attn, attn_grid(ctx)), ctx->num_sms);
        char* p = ctx->ws;
        char* ws_attn = p; p += w.a_attn;
        char* ws_lin = p; p += w.a_lin;
        bf* resid = reinterpret_cast<bf*>(p); p += w.rows_h;
        bf* xn = reinterpret_cast<bf*>(p); p += w.rows_h;
        bf* qkv = reinterpret_cast<bf*>(p); p += w.rows_qkv;
        bf* qb = reinterpret_cast<bf*>(p); p += w.rows_a;
        bf* ab = reinterpret_cast<bf*>(p); p += w.rows_a;
        bf* ob = reinterpret_cast<bf*>(p); p += w.rows_h;
        bf* xn2 = reinterpret_cast<bf*>(p); p += w.rows_h;
        bf* yb = reinterpret_cast<bf*>(p); p += w.rows_h;
        char* ws_f = p;
        for (int i = 0; i < M; ++i) {
            const int r0 = offs[i], rows = offs[i + 1] - offs[i];
            const size_t oh = (size_t)r0 * H;
            // ---- A_{l,i}
            if (l > 0 && !serial) {
                e = cudaStreamWaitEvent(sa, ctx->ev_f[i], 0);     // F_{l-1,i} has returned this microbatch
                if (e != cudaSuccess) return check_cuda(ctx, e, "decoder layers: F->A event");
            }
            // Decode batch with a dense FFN: W_o, the residual add, the FFN's RMS normalisation and the FFN are one chain
            // launch on the FFN stream (the hand-over event then sits behind the attention kernel); when the next layer is
            // of the same kind, the chain goes on through the FFN's residual add, that layer's first normalisation and its
            // QKV projection, so that a layer is three launches: rotary + append, attention, the chain.
            auto can_fuse = [&](int k) { return layers[k].layer.num_experts == 0 && chain_supported(rows) && decoder_fuse(); };
            auto same_shape = [&](int k0, int k1) {      // same workspace layout, so one layer's chain can fill the next one's buffers
                const aflex_layer_desc &x = layers[k0].layer, &y = layers[k1].layer;
                return x.attn.num_q_heads == y.attn.num_q_heads && x.attn.num_kv_heads == y.attn.num_kv_heads &&
                       x.attn.head_dim == y.attn.head_dim && x.hidden == y.hidden && x.inter == y.inter;
            };
            const bool fused = can_fuse(l);
            const bool qkv_done = l > 0 && can_fuse(l - 1) && fused && same_shape(l - 1, l);      // the previous layer's chain made xn and qkv
            const bool fuse_next = fused && l + 1 < num_layers && can_fuse(l + 1) && same_shape(l, l + 1);
            if (!qkv_done) {
                if (l == 0) s = add_rmsnorm_launch(ctx, reinterpret_cast<const bf*>(x_in) + oh, nullptr, d->w_ln_attn, rows, H, d->rms_eps, resid + oh, xn + oh, sa);
                else s = add_rmsnorm_launch(ctx, resid + oh, yb + oh, d->w_ln_attn, rows, H, d->rms_eps, resid + oh, xn + oh, sa);
                if (s != AFLEX_OK) return s;
                s = linear_launch(ctx, xn + oh, d->w_qkv, rows, H, NQ, qkv + (size_t)r0 * NQ, ws_lin, w.a_lin, sa, kKQkvGemm, ctx->counters_a);
                if (s != AFLEX_OK) return s;
            }
            aflex_kv kvi = kvs[l];
            kvi.page_table = kvs[l].page_table + (size_t)r0 * kvs[l].max_pages_per_seq;
            kvi.seq_lens = kvs[l].seq_lens + r0;
            kvi.seq_lens_host = kvs[l].seq_lens_host ? kvs[l].seq_lens_host + r0 : nullptr;
            s = rope_append_launch(ctx, &L->attn, qkv + (size_t)r0 * NQ, &kvi, rows, d->w_q_norm, d->w_k_norm, d->rms_eps, d->rope_theta, qb + (size_t)r0 * A, sa);
            if (s != AFLEX_OK) return s;
            ctx->attn_q_final_once = true;      // q was written by the append kernel, which does not release its dependents early
            s = attn_decode_launch(ctx, &L->attn, qb + (size_t)r0 * A, &kvi, rows, ab + (size_t)r0 * A, nullptr, ws_attn, w.a_attn, sa);
            if (s != AFLEX_OK) return s;
            if (!fused) {
                s = linear_launch(ctx, ab + (size_t)r0 * A, L->w_o, rows, A, H, ob + oh, ws_lin, w.a_lin, sa, kKLinearGemm, ctx->counters_a);
                if (s != AFLEX_OK) return s;
            }
            if (!serial) {
                e = cudaEventRecord(ctx->ev_a[i], sa);
                if (e == cudaSuccess) e = cudaStreamWaitEvent(sf, ctx->ev_a[i], 0);
                if (e != cudaSuccess) return check_cuda(ctx, e, "decoder layers: A->F event");
            }
            // ---- F_{l,i}
            if (fused) {
                const aflex_decoder_desc* dn = fuse_next ? &layers[l + 1] : nullptr;
                const int NQn = dn ? (dn->layer.attn.num_q_heads + 2 * dn->layer.attn.num_kv_heads) * dn->layer.attn.head_dim : 0;
                s = dense_fused_run(ctx, ab + (size_t)r0 * A, L->w_o, A, resid + oh, d->w_ln_ffn, d->rms_eps, xn2 + oh, L->w_gate, L->w_up,
                                    L->w_down, rows, H, I, yb + oh, ws_f, w.f_total, sf, dn ? dn->w_ln_attn : nullptr, dn ? dn->rms_eps : 0.f,
                                    xn + oh, dn ? dn->w_qkv : nullptr, NQn, dn ? qkv + (size_t)r0 * NQn : nullptr);
            } else {
                s = add_rmsnorm_launch(ctx, resid + oh, ob + oh, d->w_ln_ffn, rows, H, d->rms_eps, resid + oh, xn2 + oh, sf);
                if (s != AFLEX_OK) return s;
            }
            if (fused) {}
            else if (E == 0) s = dense_run(ctx, xn2 + oh, L->w_gate, L->w_up, L->w_down, rows, H, I, yb + oh, ws_f, w.f_total, sf);
            else s = moe_run(ctx, xn2 + oh, nullptr, L->w_router, L->w_gate, L->w_up, L->w_down, rows, H, I, E, L->top_k, yb + oh,
                             nullptr, nullptr, nullptr, ws_f, w.f_total, sf);
            if (s != AFLEX_OK) return s;
            if (l == num_layers - 1) {     // hidden states leaving the last layer
                s = add_rmsnorm_launch(ctx, resid + oh, yb + oh, nullptr, rows, H, 0.f, reinterpret_cast<bf*>(x_out) + oh, nullptr, sf);
                if (s != AFLEX_OK) return s;
            } else if (!serial) {
                e = cudaEventRecord(ctx->ev_f[i], sf);
                if (e != cudaSuccess) return check_cuda(ctx, e, "decoder layers: F event");
            }
        }
    }
    if (serial) return AFLEX_OK;
    e = cudaEventRecord(ctx->ev_a_done, sa);
    if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_f_done, sf);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(user, ctx->ev_a_done, 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(user, ctx->ev_f_done, 0);
    return check_cuda(ctx, e, "decoder layers: exit join");
}

// ---- whole decoder layers over the tokens being prefilled -----------------------------------
// Workspace: [linear scratch | resid | xn | qkv | q | a | o | xn2 | y | F scratch], rows = prompt tokens.
namespace {
struct PrefillWs {
    size_t a_lin, rows_h, rows_qkv, rows_a, f_total, total;
};
PrefillWs prefill_ws(const aflex_decoder_desc* d, int T, int num_sms) {
    const aflex_layer_desc* L = &d->layer;
    const int D = L->attn.head_dim, A = L->attn.num_q_heads * D, H = L->hidden;
    const int NQ = (L->attn.num_q_heads + 2 * L->attn.num_kv_heads) * D;
    PrefillWs w;
    const size_t b0 = linear_workspace_bytes(T, A, H, num_sms), b1 = linear_workspace_bytes(T, H, NQ, num_sms);
    w.a_lin = b0 > b1 ? b0 : b1;
    w.rows_h = align256((size_t)T * H * 2);
    w.rows_qkv = align256((size_t)T * NQ * 2);
    w.rows_a = align256((size_t)T * A * 2);
    w.f_total = L->num_experts == 0 ? dense_ws_bytes(T, H, L->inter, num_sms)
                                    : moe_ws_bytes(T, H, L->inter, L->num_experts, L->top_k, num_sms);
    w.total = w.a_lin + 5 * w.rows_h + w.rows_qkv + 2 * w.rows_a + w.f_total + 1024;
    return w;
}
}  // namespace

size_t aflex_prefill_workspace_bytes(const aflex_decoder_desc* layer, int max_tokens) {
    if (!layer || max_tokens < 1) return 0;
    return prefill_ws(layer, max_tokens, query_num_sms()).total;
}

aflex_status aflex_prefill_layers(aflex_ctx* ctx, const aflex_decoder_desc* layers, const aflex_kv* kvs, int num_layers,
                                  const void* x_in, int batch, const int32_t* q_offsets, const int32_t* q_offsets_host,
                                  void* x_out, void* stream) {
    if (!ctx) return AFLEX_ERR_INVALID_ARG;
    if (!q_offsets || !q_offsets_host) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "prefill layers: null q_offsets");
    if (batch < 1 || q_offsets_host[0] != 0)
        return set_error(ctx, AFLEX_ERR_INVALID_ARG, "prefill layers: batch must be >= 1 and q_offsets_host start at 0");
    for (int b = 0; b < batch; ++b)
        if (q_offsets_host[b + 1] < q_offsets_host[b])
            return set_error(ctx, AFLEX_ERR_INVALID_ARG, "prefill layers: q_offsets_host must not decrease");
    const int T = q_offsets_host[batch];
    if (T < 1) return set_error(ctx, AFLEX_ERR_INVALID_ARG, "prefill layers: no token to prefill");
    aflex_status s = validate_decoder_args(ctx, layers, kvs, num_layers, x_in, batch, x_out);
    if (s != AFLEX_OK) return s;
    const int H = layers[0].layer.hidden;
    size_t need = 0;
    for (int l = 0; l < num_layers; ++l) {
        if (kvs[l].seq_lens_host)
            for (int b = 0; b < batch; ++b)
                if (q_offsets_host[b + 1] - q_offsets_host[b] > kvs[l].seq_lens_host[b])
                    return set_error(ctx, AFLEX_ERR_INVALID_ARG, "prefill layers: sequence %d has more new tokens than cached tokens", b);
        const PrefillWs w = prefill_ws(&layers[l], T, ctx->num_sms);
        if (w.total > need) need = w.total;
    }
    if (need > ctx->ws_bytes)
        return set_error(ctx, AFLEX_ERR_WORKSPACE, "prefill layers: need %zu workspace bytes, have %zu", need, ctx->ws_bytes);
    cudaStream_t st = reinterpret_cast<cudaStream_t>(stream);
    typedef __nv_bfloat16 bf;
    for (int l = 0; l < num_layers; ++l) {
        const aflex_decoder_desc* d = &layers[l];
        const aflex_layer_desc* L = &d->layer;
        const int Hq = L->attn.num_q_heads, Hkv = L->attn.num_kv_heads, D = L->attn.head_dim;
        const int A = Hq * D, NQ = (Hq + 2 * Hkv) * D, I = L->inter, E = L->num_experts;
        const PrefillWs w = prefill_ws(d, T, ctx->num_sms);
        char* p = ctx->ws;
        char* ws_lin = p; p += w.a_lin;
        bf* resid = reinterpret_cast<bf*>(p); p += w.rows_h;
        bf* xn = reinterpret_cast<bf*>(p); p += w.rows_h;
        bf* qkv = reinterpret_cast<bf*>(p); p += w.rows_qkv;
        bf* qb = reinterpret_cast<bf*>(p); p += w.rows_a;
        bf* ab = reinterpret_cast<bf*>(p); p += w.rows_a;
        bf* ob = reinterpret_cast<bf*>(p); p += w.rows_h;
        bf* xn2 = reinterpret_cast<bf*>(p); p += w.rows_h;
        bf* yb = reinterpret_cast<bf*>(p); p += w.rows_h;
        char* ws_f = p;
        // ---- PA
        if (l == 0) s = add_rmsnorm_launch(ctx, x_in, nullptr, d->w_ln_attn, T, H, d->rms_eps, resid, xn, st);
        else s = add_rmsnorm_launch(ctx, resid, yb, d->w_ln_attn, T, H, d->rms_eps, resid, xn, st);
        if (s != AFLEX_OK) return s;
        s = linear_launch(ctx, xn, d->w_qkv, T, H, NQ, qkv, ws_lin, w.a_lin, st, kKQkvGemm, ctx->counters_a);
        if (s != AFLEX_OK) return s;
        s = rope_append_launch(ctx, &L->attn, qkv, &kvs[l], batch, d->w_q_norm, d->w_k_norm, d->rms_eps, d->rope_theta, qb, st,
                               q_offsets, T);
        if (s != AFLEX_OK) return s;
        s = attn_prefill_launch(ctx, &L->attn, qb, &kvs[l], batch, q_offsets, q_offsets_host, ab, st);
        if (s != AFLEX_OK) return s;
        s = linear_launch(ctx, ab, L->w_o, T, A, H, ob, ws_lin, w.a_lin, st, kKLinearGemm, ctx->counters_a);
        if (s != AFLEX_OK) return s;
        // ---- PF
        s = add_rmsnorm_launch(ctx, resid, ob, d->w_ln_ffn, T, H, d->rms_eps, resid, xn2, st);
        if (s != AFLEX_OK) return s;
        if (E == 0) s = dense_run(ctx, xn2, L->w_gate, L->w_up, L->w_down, T, H, I, yb, ws_f, w.f_total, st);
        else s = moe_run(ctx, xn2, nullptr, L->w_router, L->w_gate, L->w_up, L->w_down, T, H, I, E, L->top_k, yb, nullptr, nullptr,
                         nullptr, ws_f, w.f_total, st);
        if (s != AFLEX_OK) return s;
        if (l == num_layers - 1) {
            s = add_rmsnorm_launch(ctx, resid, yb, nullptr, T, H, 0.f, x_out, nullptr, st);
            if (s != AFLEX_OK) return s;
        }
    }
    return AFLEX_OK;
}

// ---- A/F pair: Attention side on ctx_a's device, FFN side on ctx_f's device ----------------
// A-side workspace: [attn scratch | linear scratch | xn | qkv | q | a | o | h1 | back]
// F-side workspace: [h1_f | xn2 | y | out_f | F scratch]
namespace {
struct PairWs {
    size_t a_attn, a_lin, rows_h, rows_qkv, rows_a, a_total, f_scratch, f_total;
};
PairWs pair_ws(const aflex_decoder_desc* d, int max_batch, size_t a_attn, int num_sms) {
    const DecoderWs w = decoder_ws(d, max_batch, a_attn, num_sms);
    PairWs p;
    p.a_attn = w.a_attn; p.a_lin = w.a_lin; p.rows_h = w.rows_h; p.rows_qkv = w.rows_qkv; p.rows_a = w.rows_a;
    p.a_total = w.a_attn + w.a_lin + 4 * w.rows_h + w.rows_qkv + 2 * w.rows_a + 1024;
    p.f_scratch = w.f_total;
    p.f_total = 4 * w.rows_h + w.f_total + 1024;
    return p;
}
struct DeviceGuard {
    int saved = -1;
    DeviceGuard() { cudaGetDevice(&saved); }
    ~DeviceGuard() { if (saved >= 0) cudaSetDevice(saved); }
};
}  // namespace

size_t aflex_af_workspace_bytes(const aflex_decoder_desc* layer, int max_batch, int ffn_side) {
    if (!layer || max_batch < 1) return 0;
    const PairWs w = pair_ws(layer, max_batch, attn_workspace_bytes(&layer->layer.attn, 4096), query_num_sms());
    return ffn_side ? w.f_total : w.a_total;
}

aflex_status aflex_af_decoder_layers(aflex_ctx* ca, aflex_ctx* cf, const aflex_decoder_desc* layers, const aflex_kv* kvs,
                                     int num_layers, const void* x_in, int batch, int M, const int32_t* mb_offsets,
                                     void* x_out, void* stream) {
    if (!ca || !cf) return AFLEX_ERR_INVALID_ARG;
    if (ca == cf) return set_error(ca, AFLEX_ERR_INVALID_ARG, "A/F pair: the two sides need separate contexts");
    aflex_status s = validate_decoder_args(ca, layers, kvs, num_layers, x_in, batch, x_out);
    if (s != AFLEX_OK) return s;
    const int H = layers[0].layer.hidden;
    size_t need_a = 0, need_f = 0;
    for (int l = 0; l < num_layers; ++l) {
        const PairWs w = pair_ws(&layers[l], batch, attn_workspace_bytes(&layers[l].layer.attn, attn_grid(ca)), ca->num_sms);
        if (w.a_total > need_a) need_a = w.a_total;
        if (w.f_total > need_f) need_f = w.f_total;
    }
    if (need_a > ca->ws_bytes)
        return set_error(ca, AFLEX_ERR_WORKSPACE, "A/F pair: attention side needs %zu workspace bytes, has %zu", need_a, ca->ws_bytes);
    if (need_f > cf->ws_bytes)
        return set_error(ca, AFLEX_ERR_WORKSPACE, "A/F pair: FFN side needs %zu workspace bytes, has %zu", need_f, cf->ws_bytes);
    int32_t offs[kMaxMicrobatches + 1];
    s = make_offsets(ca, batch, M, mb_offsets, offs);
    if (s != AFLEX_OK) return s;

    DeviceGuard guard;                                    // the caller's current device is restored on return
    const int dev_a = ca->device, dev_f = cf->device;
    cudaStream_t user = reinterpret_cast<cudaStream_t>(stream);
    cudaStream_t sa = ca->stream_a, sf = cf->stream_f;
    cudaError_t e = cudaSetDevice(dev_a);
    if (e == cudaSuccess) e = cudaEventRecord(ca->ev_entry, user);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(sa, ca->ev_entry, 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(sf, ca->ev_entry, 0);
    if (e != cudaSuccess) return check_cuda(ca, e, "A/F pair: entry join");

    typedef __nv_bfloat16 bf;
    for (int l = 0; l < num_layers; ++l) {
        const aflex_decoder_desc* d = &layers[l];
        const aflex_layer_desc* L = &d->layer;
        const int Hq = L->attn.num_q_heads, Hkv = L->attn.num_kv_heads, D = L->attn.head_dim;
        const int A = Hq * D, NQ = (Hq + 2 * Hkv) * D, I = L->inter, E = L->num_experts;
        const PairWs w = pair_ws(d, batch, attn_workspace_bytes(&L->attn, attn_grid(ca)), ca->num_sms);
        char* p = ca->ws;
        char* ws_attn = p; p += w.a_attn;
        char* ws_lin = p; p += w.a_lin;
        bf* xn = reinterpret_cast<bf*>(p); p += w.rows_h;
        bf* qkv = reinterpret_cast<bf*>(p); p += w.rows_qkv;
        bf* qb = reinterpret_cast<bf*>(p); p += w.rows_a;
        bf* ab = reinterpret_cast<bf*>(p); p += w.rows_a;
        bf* ob = reinterpret_cast<bf*>(p); p += w.rows_h;
        bf* h1 = reinterpret_cast<bf*>(p); p += w.rows_h;
        bf* back = reinterpret_cast<bf*>(p); p += w.rows_h;
        char* pf = cf->ws;
        bf* h1f = reinterpret_cast<bf*>(pf); pf += w.rows_h;
        bf* xn2 = reinterpret_cast<bf*>(pf); pf += w.rows_h;
        bf* yb = reinterpret_cast<bf*>(pf); pf += w.rows_h;
        bf* outf = reinterpret_cast<bf*>(pf); pf += w.rows_h;
        char* ws_f = pf;
        for (int i = 0; i < M; ++i) {
            const int r0 = offs[i], rows = offs[i + 1] - offs[i];
            const size_t oh = (size_t)r0 * H;
            const size_t row_bytes = (size_t)rows * H * sizeof(bf);
            // ---- A_{l,i} on the attention GPU
            e = cudaSetDevice(dev_a);
            if (e == cudaSuccess && l > 0) e = cudaStreamWaitEvent(sa, cf->ev_f[i], 0);   // the rows are back
            if (e != cudaSuccess) return check_cuda(ca, e, "A/F pair: F->A event");
            const bf* r = (l == 0 ? reinterpret_cast<const bf*>(x_in) : back) + oh;        // residual stream entering the layer
            s = add_rmsnorm_launch(ca, r, nullptr, d->w_ln_attn, rows, H, d->rms_eps, nullptr, xn + oh, sa);
            if (s != AFLEX_OK) return s;
            s = linear_launch(ca, xn + oh, d->w_qkv, rows, H, NQ, qkv + (size_t)r0 * NQ, ws_lin, w.a_lin, sa, kKQkvGemm, ca->counters_a);
            if (s != AFLEX_OK) return s;
            aflex_kv kvi = kvs[l];
            kvi.page_table = kvs[l].page_table + (size_t)r0 * kvs[l].max_pages_per_seq;
            kvi.seq_lens = kvs[l].seq_lens + r0;
            kvi.seq_lens_host = kvs[l].seq_lens_host ? kvs[l].seq_lens_host + r0 : nullptr;
            s = rope_append_launch(ca, &L->attn, qkv + (size_t)r0 * NQ, &kvi, rows, d->w_q_norm, d->w_k_norm, d->rms_eps, d->rope_theta, qb + (size_t)r0 * A, sa);
            if (s != AFLEX_OK) return s;
            ca->attn_q_final_once = true;
            s = attn_decode_launch(ca, &L->attn, qb + (size_t)r0 * A, &kvi, rows, ab + (size_t)r0 * A, nullptr, ws_attn, w.a_attn, sa);
            if (s != AFLEX_OK) return s;
            s = linear_launch(ca, ab + (size_t)r0 * A, L->w_o, rows, A, H, ob + oh, ws_lin, w.a_lin, sa, kKLinearGemm, ca->counters_a);
            if (s != AFLEX_OK) return s;
            s = add_rmsnorm_launch(ca, r, ob + oh, nullptr, rows, H, 0.f, h1 + oh, nullptr, sa);     // h1 = r + a W_o^T
            if (s != AFLEX_OK) return s;
            // what A sends to F: into the FFN GPU's own memory, then the event
            e = cudaMemcpyPeerAsync(h1f + oh, dev_f, h1 + oh, dev_a, row_bytes, sa);
            if (e == cudaSuccess) e = cudaEventRecord(ca->ev_a[i], sa);
            if (e != cudaSuccess) return check_cuda(ca, e, "A/F pair: A->F transfer");
            // ---- F_{l,i} on the FFN GPU
            e = cudaSetDevice(dev_f);
            if (e == cudaSuccess) e = cudaStreamWaitEvent(sf, ca->ev_a[i], 0);
            if (e != cudaSuccess) return check_cuda(ca, e, "A/F pair: A->F event");
            s = add_rmsnorm_launch(cf, h1f + oh, nullptr, d->w_ln_ffn, rows, H, d->rms_eps, nullptr, xn2 + oh, sf);
            if (s == AFLEX_OK) {
                if (E == 0) s = dense_run(cf, xn2 + oh, L->w_gate, L->w_up, L->w_down, rows, H, I, yb + oh, ws_f, w.f_scratch, sf);
                else s = moe_run(cf, xn2 + oh, nullptr, L->w_router, L->w_gate, L->w_up, L->w_down, rows, H, I, E, L->top_k, yb + oh,
                                 nullptr, nullptr, nullptr, ws_f, w.f_scratch, sf);
            }
            if (s == AFLEX_OK) s = add_rmsnorm_launch(cf, h1f + oh, yb + oh, nullptr, rows, H, 0.f, outf + oh, nullptr, sf);   // out = h1 + FFN
            if (s != AFLEX_OK) return set_error(ca, s, "A/F pair: FFN side: %s", cf->err);
            // what F returns: into the attention GPU's memory (the last layer's rows go straight to x_out)
            bf* dst = (l == num_layers - 1 ? reinterpret_cast<bf*>(x_out) : back) + oh;
            e = cudaMemcpyPeerAsync(dst, dev_a, outf + oh, dev_f, row_bytes, sf);
            if (e == cudaSuccess) e = cudaEventRecord(cf->ev_f[i], sf);
            if (e != cudaSuccess) return check_cuda(ca, e, "A/F pair: F->A transfer");
        }
    }
    e = cudaSetDevice(dev_a);
    if (e == cudaSuccess) e = cudaEventRecord(ca->ev_a_done, sa);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(user, ca->ev_a_done, 0);
    for (int i = 0; i < M && e == cudaSuccess; ++i) e = cudaStreamWaitEvent(user, cf->ev_f[i], 0);
    return check_cuda(ca, e, "A/F pair: exit join");
}

}  // extern "C"
