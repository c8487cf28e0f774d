// Host-side internals shared by the translation units of libaflex: the context,
// the workspace arena, tensor-map encoding and the launchers each .cu file exports.
#pragma once
#include <cuda.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/aflex.h"

namespace aflex {

constexpr int kMaxMicrobatches = 64;
constexpr size_t kDefaultWorkspace = (size_t)256 << 20;
constexpr int kMaxDynamicSmem = 227 * 1024;   // opt-in shared memory per CTA on sm_100
constexpr int kAttnCounterCap = 1 << 20;       // (sequence, KV head) arrival counters
constexpr int kTraceKernels = 64;              // timeline debugging: ring of per-launch records
constexpr int kTraceStride = 4096 * 8;         // u64 per launch record: [cta < 4096][8 stamps]
constexpr int kStreamKMaxTiles = 16384;       // capacity of each per-tile arrival-counter array


}  // namespace aflex

namespace aflex {
// Kernel kinds, for launch counting and optional per-kernel event timing.
enum KernelKind {
    kKAttnDecode = 0, kKLinearGemm, kKDownGemm, kKGateUpGemm, kKRouterLogits,
    kKMoeRoute, kKMoeGather, kKMoeGateUpGemm, kKMoeDownGemm, kKMoeCombine,
    kKAddRmsNorm, kKQkvGemm, kKRopeAppend, kKAttnPrefill, kKGemmChain, kKKindCount
};
constexpr int kProfMaxSlots = 8192;
struct ProfSlot { cudaEvent_t start, stop; int kind; };

}  // namespace aflex

struct aflex_ctx {
    int device = 0;
    int num_sms = 148;
    size_t ws_bytes = 0;
    char* ws = nullptr;           // device workspace
    int* dev_status = nullptr;    // device status word (0 = OK)
    int* host_status = nullptr;   // pinned mirror used by aflex_get_device_status
    int* counters_attn = nullptr; // per-(sequence, KV head) chunk arrival counters (zero between launches)
    int* counters_a = nullptr;    // per-tile arrival counters, attention-stream GEMMs (zero between launches)
    int* counters_f = nullptr;    // per-tile arrival counters, FFN-stream GEMMs
    int* chain_counters = nullptr;   // arrival counters and epoch words of the GEMM chain kernel, double-buffered over launches
    cudaStream_t stream_a = nullptr, stream_f = nullptr;
    cudaEvent_t ev_entry = nullptr;
    cudaEvent_t ev_a[aflex::kMaxMicrobatches] = {};
    cudaEvent_t ev_f[aflex::kMaxMicrobatches] = {};   // F_{l,i} done (decoder chain)
    cudaEvent_t ev_f_done = nullptr, ev_a_done = nullptr;
    int attn_ctas = 0;            // persistent attention CTAs per launch; 0 = two per SM
    unsigned attn_launch_seq = 0; // attention launches so far: picks the launch's pair of chunk-ticket words (four pairs in rotation)
    bool mb_two_streams = false;  // aflex_layer_step, M >= 2: A side and F side on the ctx's two streams (else all on the caller's)
    bool attn_q_final = false;    // caller's promise (aflex_set_attn_q_final): q is never the output of the kernel just before
    bool attn_q_final_once = false;   // set by the layer chains for their own attention launch (q comes from the append kernel)
    bool gemm_attr_set[6] = {false, false, false, false, false, false};   // [mode + 3 * pair form]
    bool chain_attr_set = false;
    bool attn_attr_set[2] = {false, false};
    bool prefill_attr_set[2] = {false, false};   // shared-memory limit raised for attn_prefill_kernel<64 / 128> on this device
    char err[512] = {0};
    // launch counters (always on) and event-pair timing of every launch (when profiling is enabled)
    long long launches[aflex::kKKindCount] = {};
    bool profiling = false;
    aflex::ProfSlot* prof = nullptr;   // kProfMaxSlots pre-created event pairs
    int prof_used = 0;
    unsigned long long* trace = nullptr;   // device buffer, allocated when AFLEX_TRACE=1
    int trace_slot = 0;
};

namespace aflex {

aflex_status set_error(aflex_ctx* ctx, aflex_status s, const char* fmt, ...);
aflex_status check_cuda(aflex_ctx* ctx, cudaError_t e, const char* what);

// Brackets one kernel launch: counts it, and records an event pair on its stream when profiling.
struct KernelScope {
    aflex_ctx* ctx; cudaStream_t st; int slot;
    KernelScope(aflex_ctx* c, int kind, cudaStream_t s) : ctx(c), st(s), slot(-1) {
        ctx->launches[kind]++;
        if (ctx->profiling && ctx->prof_used < kProfMaxSlots) {
            slot = ctx->prof_used++;
            ctx->prof[slot].kind = kind;
            cudaEventRecord(ctx->prof[slot].start, st);
        }
    }
    ~KernelScope() { if (slot >= 0) cudaEventRecord(ctx->prof[slot].stop, st); }
};

// Launch with programmatic stream serialization: the kernel may start while its predecessor in the
// stream is still draining; it must execute griddepcontrol.wait before touching the predecessor's output.
template <typename... KArgs, typename... Args>
inline cudaError_t launch_pdl(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t lc = {};
    lc.gridDim = grid;
    lc.blockDim = block;
    lc.dynamicSmemBytes = smem;
    lc.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = 1;
    return cudaLaunchKernelEx(&lc, kernel, static_cast<KArgs>(args)...);
}

// Bump allocator over a byte range of the ctx workspace (256-byte granules).
struct Arena {
    char* base;
    size_t size;
    size_t used = 0;
    bool overflow = false;
    Arena(char* b, size_t s) : base(b), size(s) {}
    template <typename T>
    T* take(size_t n) {
        size_t bytes = (n * sizeof(T) + 255) & ~(size_t)255;
        if (used + bytes > size) { overflow = true; return nullptr; }
        T* p = reinterpret_cast<T*>(base + used);
        used += bytes;
        return p;
    }
};
inline size_t align256(size_t b) { return (b + 255) & ~(size_t)255; }

// Encode a 2-D bf16 tiled tensor map: rows x cols (cols contiguous), box_rows x box_cols,
// 128-byte swizzle (box_cols * 2 must be 128).  Returns false on driver error.
bool encode_tmap_2d_bf16(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint64_t row_stride_bytes,
                         uint32_t box_rows, uint32_t box_cols, bool promote_l2_256);

// ---- attention (attn_decode.cu)
int attn_grid(const aflex_ctx* ctx);                                    // persistent CTAs per launch
size_t attn_workspace_bytes(const aflex_attn_desc* d, int grid);        // per-CTA partial slots
aflex_status attn_decode_launch(aflex_ctx* ctx, const aflex_attn_desc* d, const void* q, const aflex_kv* kv,
                                int batch, void* out, float* lse, char* ws, size_t ws_bytes, cudaStream_t st);

// ---- GEMM (gemm_tcgen05.cu)
// y[T][N] = x[T][K] . w[N][K]^T (bf16 in, fp32 accumulate, bf16 out).
// `counters`: kStreamKMaxTiles zeroed ints not used by any launch that may run concurrently.
size_t linear_workspace_bytes(int T, int K, int N, int num_sms);
aflex_status linear_launch(aflex_ctx* ctx, const void* x, const void* w, int T, int K, int N, void* y, char* ws,
                           size_t ws_bytes, cudaStream_t st, int kind, int* counters);
// h[T][I] = silu(x Wg^T) .* (x Wu^T)
size_t gateup_workspace_bytes(int T, int H, int I, int num_sms);
aflex_status gateup_launch(aflex_ctx* ctx, const void* x, const void* w_gate, const void* w_up, int T, int H, int I,
                           void* h, char* ws, size_t ws_bytes, cudaStream_t st, int* counters);

// ---- chain of dependent decode-batch GEMMs as one persistent kernel (gemm_chain.cu)
// Step i computes out = in . w0^T (w1 == nullptr) or out = silu(in . w0^T) .* (in . w1^T); step i + 1 reads
// step i's output.  in bf16 [T][K], w bf16 [N][K], out bf16 [T][N].  T <= kChainMaxRows.
constexpr int kChainMaxRows = 128;
struct ChainStep {
    const void* in; const void* w0; const void* w1; int K, N; void* out;
    // optional residual + normalisation epilogue of a linear step (w1 == nullptr) that has a successor:
    //   resid_out = o + resid_in (o = the step's product, rounded to bf16), out = resid_out * gain (NOT yet divided by the
    //   row's RMS), and the successor scales its accumulators by rsqrt(mean(resid_out^2) + eps) per row
    const void* resid_in = nullptr; void* resid_out = nullptr; const void* gain = nullptr; float eps = 0.f;
};
bool chain_supported(int T);
size_t chain_workspace_bytes(int T, int num_sms);
// `counters`: chain_counter_ints() zeroed ints reserved for the chain launches of one stream (double-buffered over
// launches by a generation word the kernel itself keeps there: a launch counts in one half and zeroes the other).
size_t chain_counter_ints();
aflex_status chain_launch(aflex_ctx* ctx, const ChainStep* steps, int nsteps, int T, char* ws, size_t ws_bytes,
                          cudaStream_t st, int* counters);

// Grouped (per-expert) variants over permuted rows.  `offsets` is a device array [E+1]
// (row segment of expert e = [offsets[e], offsets[e+1])); rows_max bounds any segment.
size_t grouped_workspace_bytes(int mode_gateup, int rows_total, int rows_max, int K, int N, int E, int num_sms);
aflex_status grouped_gateup_launch(aflex_ctx* ctx, const void* xp, const void* w_gate, const void* w_up,
                                   const int32_t* offsets, int rows_total, int rows_max, int H, int I, int E,
                                   void* hp, char* ws, size_t ws_bytes, cudaStream_t st, int* counters);
aflex_status grouped_linear_launch(aflex_ctx* ctx, const void* hp, const void* w_down, const int32_t* offsets,
                                   int rows_total, int rows_max, int K, int N, int E, float* yp, char* ws,
                                   size_t ws_bytes, cudaStream_t st, int* counters);

// ---- MoE glue (moe.cu)
struct MoeBuffers {
    int32_t* idx;      // [T][K]
    float* gate;       // [T][K]
    int32_t* counts;   // [E]
    int32_t* offsets;  // [E+1]
    int32_t* pos;      // [T][K]
    float* logits;     // [T][E] (router GEMM output when w_router is used)
};
aflex_status moe_router_logits_launch(aflex_ctx* ctx, const void* x, const void* w_router, int T, int H, int E,
                                      float* logits, cudaStream_t st);
aflex_status moe_route_launch(aflex_ctx* ctx, const float* logits, int T, int E, int K, const MoeBuffers& mb,
                              cudaStream_t st);
aflex_status moe_gather_launch(aflex_ctx* ctx, const void* x, const int32_t* pos, int T, int K, int H, void* xp,
                               cudaStream_t st);
aflex_status moe_combine_launch(aflex_ctx* ctx, const float* yp, const int32_t* pos, const float* gate, int T,
                                int K, int H, void* y, cudaStream_t st);


// ---- prefill attention (attn_prefill.cu)
aflex_status attn_prefill_launch(aflex_ctx* ctx, const aflex_attn_desc* d, const void* q, const aflex_kv* kv, int batch,
                                 const int32_t* q_offsets, const int32_t* q_offsets_host, void* out, cudaStream_t st);

// ---- decoder-layer glue (decoder.cu)
aflex_status add_rmsnorm_launch(aflex_ctx* ctx, const void* res, const void* add, const void* w, int T, int H, float eps,
                                void* res_out, void* y, cudaStream_t st);
aflex_status rope_append_launch(aflex_ctx* ctx, const aflex_attn_desc* d, const void* qkv, const aflex_kv* kv, int batch,
                                const void* w_qn, const void* w_kn, float eps, float theta, void* q_out, cudaStream_t st,
                                const int32_t* q_offsets = nullptr, int rows = 0);

}  // namespace aflex
