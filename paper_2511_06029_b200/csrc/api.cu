// C ABI of the Lethe hot path: argument checking, launch geometry, context-owned scratch and status word.
#include <math.h>
#include <stdio.h>
#include <string.h>

#include <new>

#include "common.cuh"
#include "prefill.cuh"

namespace lethe {
cudaError_t launch_attend_simt(const AttendArgs& a, int dtype, int D, bool paged, cudaStream_t stream);
size_t kv8_smem_bytes(int D, int shape, int chunk_tokens, int GP);
size_t kv8_stream_smem_bytes(int D, int shape, int chunk_tokens, int GP);
cudaError_t launch_attend_kv8_stream(const AttendArgs& a, int D, int shape, bool paged, int grid, cudaStream_t stream);
cudaError_t launch_attend_kv8(const AttendArgs& a, int D, int shape, bool paged, bool e5m2, cudaStream_t stream);
size_t kv8_tc_smem_bytes(int nslot, int G, int cap_pad, int ng);
size_t kv8_tc_maps_bytes();
bool build_kv8_tc_maps(void* encode, void* k, void* v, unsigned long long rows, bool paged, void* out_maps);
cudaError_t launch_attend_kv8_tc(const AttendArgs& a, const void* maps, bool paged, bool e5m2, int ng, int nslot, int cap_pad, int grid,
                                 cudaStream_t stream);
size_t simt_smem_bytes(int D, int chunk_tokens, int GP);
cudaError_t launch_attend_mma(const AttendArgs& a, int D, int shape, bool paged, cudaStream_t stream);
size_t mma_smem_bytes(int D, int shape, int chunk_tokens, int GP);
cudaError_t launch_attend_layer(const AttendArgs& a, int D, int shape, bool paged, cudaStream_t stream);
size_t kv8_layer_smem_bytes(int chunk_tokens, int GP);
cudaError_t launch_attend_kv8_layer(const AttendArgs& a, bool paged, bool e5m2, cudaStream_t stream);
size_t layer_smem_bytes(int D, int shape, int chunk_tokens, int GP);
cudaError_t launch_attend_stream(const AttendArgs& a, int D, int shape, bool paged, int grid, cudaStream_t stream);
size_t stream_smem_bytes(int D, int shape, int chunk_tokens, int GP);
cudaError_t launch_attend_async(const AttendArgs& a, int D, int shape, bool paged, int grid, cudaStream_t stream, bool tma,
                                const void* maps);
bool build_tma_maps(void* encode, void* k, void* v, unsigned long long rows, int D, void* out_maps);
size_t tma_maps_bytes();
size_t async_smem_bytes(int D, int shape, int chunk_tokens, int GP);
cudaError_t launch_sparsity(const CacheView& c, float* sparsity, cudaStream_t stream);
cudaError_t launch_budgets(int L, int B, const float* sparsity, const long long* total, int k_min, int32_t* budgets,
                           int32_t* status, cudaStream_t stream);
cudaError_t launch_segment_prune(const CacheView& c, int n_segments, float tau, int recent, int sink, int32_t* l_evict,
                                 int32_t* keep_idx, int max_k, int smem_tokens, int32_t* list_scratch, int32_t* status,
                                 cudaStream_t stream);
cudaError_t launch_order(const int32_t* len, int n_items, int cap_tokens, int32_t* order, cudaStream_t stream);
cudaError_t launch_collapsed_prune(const CacheView& c, const int32_t* budgets, int recent, int sink, int per_group,
                                   int32_t* keep_idx, int max_k, int smem_tokens, uint32_t* key_scratch,
                                   int32_t* lists, int32_t* plan, int32_t* status, cudaStream_t stream);
cudaError_t launch_rasr_prune(const CacheView& c, const int32_t* budgets, int recent, int sink, int32_t* keep_idx,
                              int max_k, int smem_tokens, int32_t* list_scratch, int32_t* status,
                              cudaStream_t stream);
}  // namespace lethe

using namespace lethe;

#include <map>
#include <mutex>
#include <utility>

namespace lethe {
cudaError_t prepare_kernel(const void* func, size_t smem_needed) {
    static std::mutex mu;
    static std::map<std::pair<const void*, int>, size_t> done;  // (function, device) -> opted-in bytes
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    std::lock_guard<std::mutex> lock(mu);
    auto it = done.find({func, dev});
    if (it != done.end()) return smem_needed <= it->second ? cudaSuccess : cudaErrorInvalidValue;
    int max_optin = 0;
    e = cudaDeviceGetAttribute(&max_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev);
    if (e != cudaSuccess) return e;
    cudaFuncAttributes fa;
    e = cudaFuncGetAttributes(&fa, func);
    if (e != cudaSuccess) return e;
    const int max_dyn = max_optin - (int)fa.sharedSizeBytes;  // static shared memory counts against the limit
    e = cudaFuncSetAttribute(func, cudaFuncAttributeMaxDynamicSharedMemorySize, max_dyn);
    if (e != cudaSuccess) return e;
    e = cudaFuncSetAttribute(func, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
    if (e != cudaSuccess) return e;
    done[{func, dev}] = (size_t)max_dyn;
    return smem_needed <= (size_t)max_dyn ? cudaSuccess : cudaErrorInvalidValue;
}
}  // namespace lethe

struct lethe_ctx {
    int device;
    int sm_count;
    size_t max_smem;  // opt-in dynamic shared memory per CTA
    int32_t* status;      // device: {code, item} followed by the persistent kernel's work-queue words
    unsigned int* sched;  // device: {next ticket, CTAs finished}; zero whenever no attend launch is running
    void* scratch;
    size_t scratch_bytes;
    // longest-first item order written by the last lethe_rasr_prune, and the cache it describes
    int32_t* order;
    size_t order_bytes;
    const int32_t* order_len;  // cache.len the order was computed from
    int order_items;
    void* flat;  // scratch-merged split mode: arrival counters (zero between launches), partials, logits
    size_t flat_bytes;
    void* staging;  // device staging of lethe_decode_attend_host
    size_t staging_bytes;
    // lethe_decode_attend_host: upload / download streams and the events that chain them to the caller's stream
    cudaStream_t up_stream, down_stream;
    cudaEvent_t ev_start, ev_up[8], ev_done[8], ev_down;
    bool host_pipeline_ready;
    int variant, splits;
    int wait_limit;  // poll limit of the kernels' bounded waits (0 = their defaults); lethe_set_wait_limit
    // layer pipelining (tuning 51): the last call enqueued through this context, if it was a decode call
    int pipeline_layers;
    const int32_t* last_len;  // cache.len of that call (NULL: the last call was something else)
    int last_l0, last_l1;
    void* last_stream;
    int prefill_engine;  // 0 = tcgen05 kernels (TMA producers when the cache is contiguous), 1 = mma.sync kernels, 2 = tcgen05 with cp.async producers
    // TMA variant: tensor maps of the last cache seen (rebuilt when k, v, the row count or D change)
    alignas(64) unsigned char tma_maps[512];
    const void* tma_k;
    const void* tma_v;
    unsigned long long tma_rows;
    int tma_d;
    void* tma_encode;  // cuTensorMapEncodeTiled, resolved on first use
    // tensor-memory kernel for byte caches: its tensor maps (byte rows) of the last cache seen
    alignas(64) unsigned char kv8_maps[512];
    const void* kv8_k;
    const void* kv8_v;
    unsigned long long kv8_rows;
    int kv8_paged;
    char err[256];
};

static lethe_status fail(lethe_ctx* ctx, lethe_status st, const char* fmt, const char* detail = "") {
    if (ctx) snprintf(ctx->err, sizeof(ctx->err), fmt, detail);
    return st;
}

static lethe_status cuda_fail(lethe_ctx* ctx, cudaError_t e, const char* where) {
    if (ctx) snprintf(ctx->err, sizeof(ctx->err), "%s: %s", where, cudaGetErrorString(e));
    return LETHE_ERR_CUDA;
}

namespace {
struct DeviceGuard {
    int prev = -1;
    bool ok;
    explicit DeviceGuard(int dev) {
        ok = cudaGetDevice(&prev) == cudaSuccess && (prev == dev || cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard() {
        int cur = -1;
        if (prev >= 0 && cudaGetDevice(&cur) == cudaSuccess && cur != prev) cudaSetDevice(prev);
    }
};

// Grow a context-owned buffer.  Growth synchronises the device and frees the old buffer, so it must not happen
// while `stream` is being captured (the capture would be invalidated, and a graph captured earlier may still name
// the old buffer): that case is refused.
lethe_status ensure(lethe_ctx* ctx, void** buf, size_t* have, size_t need, const char* what, void* stream = nullptr) {
    if (need <= *have) return LETHE_OK;
    cudaStreamCaptureStatus cap = cudaStreamCaptureStatusNone;
    if (cudaStreamIsCapturing((cudaStream_t)stream, &cap) != cudaSuccess) cudaGetLastError();
    else if (cap != cudaStreamCaptureStatusNone)
        return fail(ctx, LETHE_ERR_UNSUPPORTED, "%s would have to grow while the stream is being captured", what);
    cudaError_t e = cudaDeviceSynchronize();  // the old buffer may still be in use
    if (e != cudaSuccess) return cuda_fail(ctx, e, what);
    if (*buf) cudaFree(*buf);
    *buf = nullptr;
    *have = 0;
    size_t sz = need + need / 4;
    e = cudaMalloc(buf, sz);
    if (e != cudaSuccess) return cuda_fail(ctx, e, what);
    *have = sz;
    return LETHE_OK;
}

lethe_status check_cache(lethe_ctx* ctx, const lethe_cache* c) {
    if (!ctx) return LETHE_ERR_INVALID_ARG;
    if (!c) return fail(ctx, LETHE_ERR_INVALID_ARG, "cache is NULL");
    if (!c->k || !c->v || !c->rel || !c->pos || !c->len) return fail(ctx, LETHE_ERR_INVALID_ARG, "cache has a NULL tensor");
    if (c->n_layers < 1 || c->batch < 1 || c->n_kv_heads < 1 || c->n_q_heads < 1)
        return fail(ctx, LETHE_ERR_INVALID_ARG, "cache dimensions must be positive");
    if (c->n_q_heads % c->n_kv_heads) return fail(ctx, LETHE_ERR_INVALID_ARG, "n_q_heads must be a multiple of n_kv_heads");
    if (c->head_dim != 64 && c->head_dim != 128) return fail(ctx, LETHE_ERR_UNSUPPORTED, "head_dim must be 64 or 128");
    const bool bytes = c->dtype == LETHE_FP8_E4M3 || c->dtype == LETHE_FP8_E5M2;
    if (c->dtype != LETHE_F32 && c->dtype != LETHE_BF16 && !bytes)
        return fail(ctx, LETHE_ERR_INVALID_ARG, "unknown dtype");
    if (bytes)
        for (int l = 0; l < c->n_layers; ++l) {
            const float ks = c->k_scale ? c->k_scale[l] : 1.f, vs = c->v_scale ? c->v_scale[l] : 1.f;
            if (!(ks > 0.f && ks < 1e30f && vs > 0.f && vs < 1e30f)) return fail(ctx, LETHE_ERR_INVALID_ARG, "k_scale and v_scale must be positive and finite");
        }
    if (c->layout != LETHE_CONTIG && c->layout != LETHE_PAGED) return fail(ctx, LETHE_ERR_INVALID_ARG, "unknown layout");
    if (c->capacity < 1) return fail(ctx, LETHE_ERR_INVALID_ARG, "capacity must be positive");
    if (c->layout == LETHE_PAGED) {
        if (!c->page_table || c->page_tokens < 1 || c->n_pages < 1)
            return fail(ctx, LETHE_ERR_INVALID_ARG, "paged layout needs page_table, page_tokens and n_pages");
        if ((long long)c->capacity * c->page_tokens > 0x7fffffffLL) return fail(ctx, LETHE_ERR_INVALID_ARG, "capacity too large");
    }
    if (((uintptr_t)c->k | (uintptr_t)c->v | (uintptr_t)c->rel) & 15) return fail(ctx, LETHE_ERR_INVALID_ARG, "k, v, rel must be 16-byte aligned");
    const long long items = (long long)c->n_layers * c->batch * c->n_kv_heads;
    if (items > 0x7fffffffLL / 16) return fail(ctx, LETHE_ERR_UNSUPPORTED, "too many (layer, sequence, head) items");
    return LETHE_OK;
}

int cap_tokens_of(const lethe_cache* c) { return c->layout == LETHE_PAGED ? c->capacity * c->page_tokens : c->capacity; }

CacheView view_of(const lethe_cache* c) {
    CacheView v;
    v.k = c->k; v.v = c->v; v.rel = c->rel; v.pos = c->pos; v.len = c->len; v.page_table = c->page_table;
    v.n_pages = c->n_pages;
    v.L = c->n_layers; v.B = c->batch; v.Hkv = c->n_kv_heads; v.D = c->head_dim;
    v.elt_bytes = c->dtype == LETHE_BF16 ? 2 : (c->dtype == LETHE_F32 ? 4 : 1);
    v.capacity = c->capacity; v.cap_tokens = cap_tokens_of(c);
    v.page_tokens = c->layout == LETHE_PAGED ? c->page_tokens : 1;
    v.paged = c->layout == LETHE_PAGED;
    return v;
}
}  // namespace

extern "C" {

lethe_status lethe_create(lethe_ctx** out, int device, size_t scratch_bytes_hint) {
    if (!out) return LETHE_ERR_INVALID_ARG;
    *out = nullptr;
    int count = 0;
    if (cudaGetDeviceCount(&count) != cudaSuccess || device < 0 || device >= count) return LETHE_ERR_CUDA;
    DeviceGuard guard(device);
    if (!guard.ok) return LETHE_ERR_CUDA;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, device) != cudaSuccess) return LETHE_ERR_CUDA;
    if (prop.major != 10) return LETHE_ERR_CUDA;  // built for sm_100a only
    lethe_ctx* ctx = new (std::nothrow) lethe_ctx();
    if (!ctx) return LETHE_ERR_CUDA;
    memset(ctx, 0, sizeof(*ctx));
    ctx->device = device;
    ctx->sm_count = prop.multiProcessorCount;
    ctx->max_smem = prop.sharedMemPerBlockOptin;
    strcpy(ctx->err, "no error");
    if (cudaMalloc((void**)&ctx->status, 4 * sizeof(int32_t)) != cudaSuccess ||
        cudaMemset(ctx->status, 0, 4 * sizeof(int32_t)) != cudaSuccess) {
        delete ctx;
        return LETHE_ERR_CUDA;
    }
    ctx->sched = reinterpret_cast<unsigned int*>(ctx->status + 2);
    if (scratch_bytes_hint) {
        if (ensure(ctx, &ctx->scratch, &ctx->scratch_bytes, scratch_bytes_hint, "scratch") != LETHE_OK) {
            cudaFree(ctx->status);
            delete ctx;
            return LETHE_ERR_CUDA;
        }
    }
    *out = ctx;
    return LETHE_OK;
}

void lethe_destroy(lethe_ctx* ctx) {
    if (!ctx) return;
    DeviceGuard guard(ctx->device);
    cudaDeviceSynchronize();
    if (ctx->status) cudaFree(ctx->status);
    if (ctx->scratch) cudaFree(ctx->scratch);
    if (ctx->staging) cudaFree(ctx->staging);
    if (ctx->host_pipeline_ready) {
        cudaStreamDestroy(ctx->up_stream);
        cudaStreamDestroy(ctx->down_stream);
        cudaEventDestroy(ctx->ev_start);
        cudaEventDestroy(ctx->ev_down);
        for (int i = 0; i < 8; ++i) {
            cudaEventDestroy(ctx->ev_up[i]);
            cudaEventDestroy(ctx->ev_done[i]);
        }
    }
    if (ctx->order) cudaFree(ctx->order);
    if (ctx->flat) cudaFree(ctx->flat);
    delete ctx;
}

const char* lethe_last_error(const lethe_ctx* ctx) { return ctx ? ctx->err : "context is NULL"; }

lethe_status lethe_poll_status(lethe_ctx* ctx, void* stream, int32_t* info) {
    if (!ctx) return LETHE_ERR_INVALID_ARG;
    DeviceGuard guard(ctx->device);
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "poll_status: synchronize");
    int32_t h[2] = {0, 0};
    e = cudaMemcpyAsync(h, ctx->status, sizeof(h), cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "poll_status: read");
    if (h[0] != 0) {
        e = cudaMemsetAsync(ctx->status, 0, sizeof(h), s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "poll_status: clear");
        snprintf(ctx->err, sizeof(ctx->err), "device-side status %d at item %d", h[0], h[1]);
    }
    if (info) {
        info[0] = h[0];
        info[1] = h[1];
    }
    return (lethe_status)h[0];
}


// cuTensorMapEncodeTiled through the runtime (no link-time dependency on the driver library); resolved once.
static bool resolve_tma_encode(lethe_ctx* ctx) {
    if (ctx->tma_encode) return true;
    cudaDriverEntryPointQueryResult qres;
    if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &ctx->tma_encode, cudaEnableDefault, &qres) != cudaSuccess ||
        qres != cudaDriverEntryPointSuccess || !ctx->tma_encode) {
        ctx->tma_encode = nullptr;
        return false;
    }
    return true;
}

lethe_status lethe_set_tuning(lethe_ctx* ctx, int variant, int splits) {
    if (!ctx) return LETHE_ERR_INVALID_ARG;
    if (variant >= 40 && variant <= 42) {  // engine of lethe_prefill_seed; the attend tuning is left as it is
        ctx->prefill_engine = variant - 40;
        return LETHE_OK;
    }
    if (variant == 50 || variant == 51) {  // layer pipelining of the one-layer-per-launch kernel; nothing else changes
        ctx->pipeline_layers = variant - 50;
        return LETHE_OK;
    }
    const bool layer_variant = variant >= 44 && variant <= 49;
    if ((variant < 0 || variant > 37) && !layer_variant)
        return fail(ctx, LETHE_ERR_INVALID_ARG, "variant must be 0..37, 40..42 or 44..51");
    const bool flat_variant = variant >= 32 && variant <= 37;
    if (flat_variant ? (splits < 0 || splits > 16)
                     : !(splits == 0 || splits == 1 || splits == 2 || splits == 4 || splits == 8 || splits == 16))
        return fail(ctx, LETHE_ERR_INVALID_ARG, "splits must be 0, 1, 2, 4, 8 or 16 (0..16 for the scratch-merged variants)");
    ctx->variant = variant;
    ctx->splits = splits;
    return LETHE_OK;
}

// Everything about a decode call that the host can check, for the device and the host entry points alike (the
// host entry point checks before it sizes staging or enqueues a copy).  Alignment is a matter of device pointers.
static lethe_status check_attend_args(lethe_ctx* ctx, const lethe_cache* c, int layer_begin, int layer_end, const void* q,
                                      const void* k_new, const void* v_new, const int32_t* token_pos, const float* scale,
                                      float gamma, const void* out, bool device_pointers) {
    lethe_status st = check_cache(ctx, c);
    if (st != LETHE_OK) return st;
    if (!q || !out || !scale) return fail(ctx, LETHE_ERR_INVALID_ARG, "q, out and scale are required");
    if (layer_begin < 0 || layer_end > c->n_layers || layer_begin >= layer_end)
        return fail(ctx, LETHE_ERR_INVALID_ARG, "bad layer range");
    if ((k_new == nullptr) != (v_new == nullptr)) return fail(ctx, LETHE_ERR_INVALID_ARG, "k_new and v_new go together");
    if (k_new && !token_pos) return fail(ctx, LETHE_ERR_INVALID_ARG, "token_pos is required when appending");
    if (!(gamma > 0.f && gamma <= 1.f)) return fail(ctx, LETHE_ERR_INVALID_ARG, "gamma must be in (0, 1]");
    if (c->n_layers > kMaxLayers) return fail(ctx, LETHE_ERR_UNSUPPORTED, "more than 128 layers");
    if (c->n_q_heads / c->n_kv_heads > kMaxGroup) return fail(ctx, LETHE_ERR_UNSUPPORTED, "more than 8 query heads per KV head");
    if (device_pointers && (((uintptr_t)q | (uintptr_t)out | (uintptr_t)k_new | (uintptr_t)v_new) & 15))
        return fail(ctx, LETHE_ERR_INVALID_ARG, "q, k_new, v_new, out must be 16-byte aligned");
    for (int l = layer_begin; l < layer_end; ++l)
        if (!(scale[l] == scale[l]) || fabsf(scale[l]) > 1e30f) return fail(ctx, LETHE_ERR_INVALID_ARG, "scale must be finite");
    const bool bytes = c->dtype == LETHE_FP8_E4M3 || c->dtype == LETHE_FP8_E5M2;
    if (bytes && c->layout == LETHE_PAGED && c->page_tokens != kGroupTokens)
        return fail(ctx, LETHE_ERR_UNSUPPORTED, "quantised caches need 16-token pages");
    return LETHE_OK;
}

lethe_status lethe_set_wait_limit(lethe_ctx* ctx, int32_t polls) {
    if (!ctx) return LETHE_ERR_INVALID_ARG;
    if (polls < 0) return fail(ctx, LETHE_ERR_INVALID_ARG, "the poll limit must be >= 0 (0 = default)");
    ctx->wait_limit = polls;
    return LETHE_OK;
}

lethe_status lethe_decode_attend(lethe_ctx* ctx, const lethe_cache* c, int layer_begin, int layer_end, const void* q,
                                 const void* k_new, const void* v_new, const int32_t* token_pos, const float* scale,
                                 float gamma, void* out, float* lse, void* stream) {
    lethe_status st = check_attend_args(ctx, c, layer_begin, layer_end, q, k_new, v_new, token_pos, scale, gamma, out, true);
    if (st != LETHE_OK) return st;
    const int G = c->n_q_heads / c->n_kv_heads;

    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, LETHE_ERR_CUDA, "cannot select the context's device");

    AttendArgs a;
    memset(&a, 0, sizeof(a));
    a.k = c->k; a.v = c->v; a.rel = c->rel; a.pos = c->pos; a.len = c->len; a.page_table = c->page_table;
    a.q = q; a.k_new = k_new; a.v_new = v_new; a.token_pos = token_pos; a.out = out; a.lse = lse;
    a.status = ctx->status;
    a.sched = ctx->sched;
    // Work-queue order from the last prune round: usable while the call covers the same items (all layers of the
    // same cache).  Appends lengthen every item alike, so the order stays longest-first between rounds.
    if (ctx->order && ctx->order_len == c->len && layer_begin == 0 && layer_end == c->n_layers &&
        ctx->order_items == c->n_layers * c->batch * c->n_kv_heads)
        a.order = ctx->order;
    a.n_pages = c->n_pages;
    a.B = c->batch; a.Hq = c->n_q_heads; a.Hkv = c->n_kv_heads; a.G = G; a.GP = (G + 1) & ~1;
    a.capacity = c->capacity; a.cap_tokens = cap_tokens_of(c);
    a.page_tokens = c->layout == LETHE_PAGED ? c->page_tokens : 1;
    a.layer_begin = layer_begin;
    a.n_items = (layer_end - layer_begin) * c->batch * c->n_kv_heads;
    a.gamma = gamma;
    a.wait_limit = ctx->wait_limit;
    // Layer pipelining: the kernel may fetch cached K / V tiles before the previous kernel of the stream is done only
    // if that kernel cannot have written this call's items: it was this context's previous call, a decode call on
    // the same cache and stream, over layers disjoint from this call's.
    a.early_prefetch = ctx->pipeline_layers && ctx->last_len == c->len && ctx->last_stream == stream &&
                       (layer_end <= ctx->last_l0 || layer_begin >= ctx->last_l1);
    ctx->last_len = c->len;
    ctx->last_l0 = layer_begin;
    ctx->last_l1 = layer_end;
    ctx->last_stream = stream;
    for (int l = 0; l < c->n_layers; ++l) a.scale_log2[l] = scale[l] * 1.4426950408889634f;

    const bool paged = c->layout == LETHE_PAGED;
    const bool mma_ok = c->dtype == LETHE_BF16 && (!paged || c->page_tokens == kGroupTokens);
    const int cap_groups = (a.cap_tokens + kGroupTokens - 1) / kGroupTokens;
    int variant = ctx->variant;

    if (c->dtype == LETHE_FP8_E4M3 || c->dtype == LETHE_FP8_E5M2) {
        // quantised cache: its own clustered tensor-core kernel; variants 2..7 pick its shape, the rest mean "default"
        if (paged && c->page_tokens != kGroupTokens) return fail(ctx, LETHE_ERR_UNSUPPORTED, "quantised caches need 16-token pages");
        if (c->n_layers > kMaxLayers) return fail(ctx, LETHE_ERR_UNSUPPORTED, "more than 128 layers");
        for (int l = 0; l < c->n_layers; ++l) {
            a.k_scale[l] = c->k_scale ? c->k_scale[l] : 1.f;
            a.v_scale[l] = c->v_scale ? c->v_scale[l] : 1.f;
            a.scale_log2[l] = scale[l] * a.k_scale[l] * 1.4426950408889634f;
        }
        // The clustered kernel (variants 2..7 pick its shape) is the default at every size: with two CTAs per SM
        // covering each other's epilogues it beats the persistent one (variants 8..13) on this conversion-bound
        // path (Llama-8B shape: 0.124 ms against 0.153 to 0.161 ms; a version of the asynchronous-epilogue kernel for
        // byte caches was measured too: 0.156 to 0.178 ms with two epilogue warps, 0.131 ms at best with four and the
        // batched relevance update (8 streaming warps x 2 stages), worse again with six; not kept).
        // Tensor-memory kernel (variant 14, and the automatic choice for launches with many items): tcgen05 f8f6f4 MMAs
        // on the cache's bytes, tiles by TMA, head_dim 128, the item's logits parked on chip; 0.097 ms on the same
        // shape (paged 0.121 against the clustered kernel's 0.146).  Falls back to the kernels below when the cache
        // does not fit it.
        const bool want_tc = variant == 14 || (variant == 0 && a.n_items >= 2 * ctx->sm_count && ctx->splits <= 1);
        if (want_tc && c->head_dim == 128 && resolve_tma_encode(ctx) && sizeof(ctx->kv8_maps) >= kv8_tc_maps_bytes()) {
            const int cap_full = ((a.cap_tokens + 127) / 128) * 128;
            const int ng = 2;  // softmax groups
            // The deepest rings (K and V: half each) that fit beside the groups' logit buffers.  A wide group (more than
            // five heads) at a capacity that does not fit even beside four slots keeps the first `park` tokens of an
            // item on chip and lets the rest overflow into a per-CTA slice of scratch (caches are sized well above the
            // lengths items reach between rounds), provided at least 0.4 of the capacity stays on chip.
            int nslot = 8, park = cap_full;
            while (nslot > 4 && kv8_tc_smem_bytes(nslot, G, park, ng) > ctx->max_smem) --nslot;
            if (kv8_tc_smem_bytes(nslot, G, park, ng) > ctx->max_smem && 3 * G > 16) {
                const size_t fixed = kv8_tc_smem_bytes(nslot, G, 0, ng);
                park = fixed < ctx->max_smem ? (int)((ctx->max_smem - fixed) / ((size_t)ng * G * 4) / 128) * 128 : 0;
                if (park * 5 < cap_full * 2) park = 0;
            }
            const int per_sm = 1;
            const int grid = a.n_items < per_sm * ctx->sm_count ? a.n_items : per_sm * ctx->sm_count;
            const unsigned long long rows = paged ? (unsigned long long)c->n_pages * c->page_tokens
                                                  : (unsigned long long)c->n_layers * c->batch * c->n_kv_heads * c->capacity;
            if (park >= 128 && kv8_tc_smem_bytes(nslot, G, park, ng) <= ctx->max_smem && rows <= 0x7fffffffULL) {
                if (park < cap_full) {
                    a.spill_tokens = cap_full - park;
                    const size_t need = (size_t)grid * ng * G * a.spill_tokens * sizeof(float);
                    st = ensure(ctx, &ctx->scratch, &ctx->scratch_bytes, need, "logit overflow scratch", stream);
                    if (st != LETHE_OK) return st;
                    a.spill = (float*)ctx->scratch;
                }
                if (ctx->kv8_k != c->k || ctx->kv8_v != c->v || ctx->kv8_rows != rows || ctx->kv8_paged != (int)paged) {
                    if (!build_kv8_tc_maps(ctx->tma_encode, c->k, c->v, rows, paged, ctx->kv8_maps))
                        return fail(ctx, LETHE_ERR_CUDA, "cuTensorMapEncodeTiled failed");
                    ctx->kv8_k = c->k; ctx->kv8_v = c->v; ctx->kv8_rows = rows; ctx->kv8_paged = (int)paged;
                }
                a.splits = 1;
                const cudaError_t et = launch_attend_kv8_tc(a, ctx->kv8_maps, paged, c->dtype == LETHE_FP8_E5M2, ng, nslot, park, grid,
                                                            (cudaStream_t)stream);
                if (et != cudaSuccess) return cuda_fail(ctx, et, "decode_attend launch (quantised cache, tensor memory)");
                return LETHE_OK;
            }
            if (variant == 14) return fail(ctx, LETHE_ERR_UNSUPPORTED, "capacity too large for the tensor-memory kernel's on-chip logit buffer");
        } else if (variant == 14) {
            return fail(ctx, LETHE_ERR_UNSUPPORTED, "the tensor-memory kernel for quantised caches needs head_dim 128");
        }
        // Many items whose logits do not fit the tensor-memory kernel's on-chip buffers (wide groups at large
        // capacities): the persistent kernel, which lets the tail of long items overflow to scratch (Qwen-7B shape,
        // G = 7 at capacity 5312: 0.46 ms against the clustered kernel's 0.77 ms).
        bool auto_persistent = variant == 0 && a.n_items >= 2 * ctx->sm_count && ctx->splits <= 1 && c->dtype == LETHE_FP8_E4M3 &&
                               c->head_dim == 128;
        if (auto_persistent && kv8_stream_smem_bytes(c->head_dim, 0, kGroupTokens, a.GP) > ctx->max_smem) auto_persistent = false;
        const bool want_persistent = (variant >= 8 && variant <= 13) || auto_persistent;
        const bool want_clustered = variant >= 2 && variant <= 7;
        if (want_persistent && ctx->splits <= 1 && c->dtype == LETHE_FP8_E4M3) {
            const int pshape = auto_persistent ? 0 : variant - 8;
            const size_t fixed = kv8_stream_smem_bytes(c->head_dim, pshape, 0, a.GP);
            int fit = 0;
            if (fixed < ctx->max_smem) fit = (int)((ctx->max_smem - fixed) / ((size_t)a.GP * 4) / kGroupTokens) * kGroupTokens;
            a.splits = 1;
            a.chunk_tokens = fit < cap_groups * kGroupTokens ? fit : cap_groups * kGroupTokens;
            if (a.chunk_tokens < kGroupTokens)
                return fail(ctx, LETHE_ERR_UNSUPPORTED, "no shared memory left for the logit buffer of this persistent shape");
            const int grid = a.n_items < ctx->sm_count ? a.n_items : ctx->sm_count;
            if (a.chunk_tokens < cap_groups * kGroupTokens) {  // overflow of the logit buffer: one slice per CTA
                a.spill_tokens = cap_groups * kGroupTokens - a.chunk_tokens;
                const size_t need = (size_t)grid * a.spill_tokens * a.GP * sizeof(float);
                st = ensure(ctx, &ctx->scratch, &ctx->scratch_bytes, need, "logit overflow scratch", stream);
                if (st != LETHE_OK) return st;
                a.spill = (float*)ctx->scratch;
            }
            const cudaError_t ep = launch_attend_kv8_stream(a, c->head_dim, pshape, paged, grid, (cudaStream_t)stream);
            if (ep != cudaSuccess) return cuda_fail(ctx, ep, "decode_attend launch (quantised cache, persistent)");
            return LETHE_OK;
        }
        const int shape = want_clustered ? variant - 2 : 0;
        // Few items per launch (one layer at a time): the layer kernel's byte-cache instance (one-sided merge, tiles
        // fetched before the previous launch completes; variant 44 forces it), head_dim 128; else the clustered kernel.
        const bool layer8 = (variant == 0 || variant == 44) && c->head_dim == 128;
        auto smem_for = [&](int S) -> size_t {
            const int chunk = ((cap_groups + S - 1) / S) * kGroupTokens;
            return layer8 ? kv8_layer_smem_bytes(chunk, a.GP) : kv8_smem_bytes(c->head_dim, shape, chunk, a.GP);
        };
        int S = ctx->splits;
        if (S == 0) {
            S = 1;
            while (S < 16 && smem_for(S) > ctx->max_smem) S *= 2;
            while (S < 8 && ((long long)a.n_items * S < ctx->sm_count || (layer8 && a.n_items <= ctx->sm_count && S < 4)) &&
                   cap_groups / (2 * S) >= 4)
                S *= 2;
        }
        if (smem_for(S) > ctx->max_smem)
            return fail(ctx, LETHE_ERR_UNSUPPORTED, "capacity too large for the on-chip logit buffer at this split count");
        a.splits = S;
        a.chunk_tokens = ((cap_groups + S - 1) / S) * kGroupTokens;
        const cudaError_t e8 = layer8 ? launch_attend_kv8_layer(a, paged, c->dtype == LETHE_FP8_E5M2, (cudaStream_t)stream)
                                      : launch_attend_kv8(a, c->head_dim, shape, paged, c->dtype == LETHE_FP8_E5M2, (cudaStream_t)stream);
        if (e8 != cudaSuccess) return cuda_fail(ctx, e8, "decode_attend launch (quantised cache)");
        return LETHE_OK;
    }
    // persistent kernel: logit-buffer tokens that fit beside a shape's stages (the rest overflows to scratch)
    auto stream_chunk = [&](int shape) -> int {
        const size_t fixed = stream_smem_bytes(c->head_dim, shape, 0, a.GP);
        if (fixed >= ctx->max_smem) return 0;
        const size_t tokens = (ctx->max_smem - fixed) / ((size_t)a.GP * 4);
        const int fit = (int)(tokens / kGroupTokens) * kGroupTokens;
        return fit < cap_groups * kGroupTokens ? fit : cap_groups * kGroupTokens;
    };
    if (variant == 0) {
        // enough items to give every SM several: the persistent kernel; few long items: the clustered one
        if (!mma_ok) variant = 1;
        else if (a.n_items >= 2 * ctx->sm_count && ctx->splits <= 1) {
            // Persistent kernels.  The asynchronous-epilogue kernel (best measured first: (8,2) with four epilogue
            // warps, then (5,3) (6,3) (4,4) with two) when both of its logit buffers cover the capacity on chip.
            // Otherwise the tail of long items overflows to scratch, and what matters is how much of a typical item
            // still fits on chip: the asynchronous (8,2), else (5,3), while each of its two buffers holds at least
            // 0.4 of the capacity (caches are sized well above the lengths they reach between prune rounds), else
            // the synchronous (8,2), whose single buffer gets the most room.  Measured, of the copy peak: Llama
            // shape at capacities 1600 / 2048 / 2560 / 3584 / 4608 / 6144 asynchronous (8,2) 1.02 / 1.00 / 0.95 /
            // 1.00 / 0.99 / 0.99, asynchronous (5,3) 1.00 / 1.00 / 0.93 / 0.96 / 0.95 / 0.95, synchronous 0.97 /
            // 0.96 / 0.93 / 0.97 / 0.96 / 0.92; long-reasoning shape 1.06 / 1.05 / 1.02; Qwen shape (8 logit columns
            // per token, capacity 5312) 0.99 with the synchronous kernel against 0.84 to 0.93.
            const int cap_pad = cap_groups * kGroupTokens;
            auto async_fits = [&](int shape) { return async_smem_bytes(c->head_dim, shape, cap_pad, a.GP) <= ctx->max_smem; };
            auto async_chunk = [&](int shape) -> size_t {
                const size_t fixed = async_smem_bytes(c->head_dim, shape, 0, a.GP);
                return fixed < ctx->max_smem ? (ctx->max_smem - fixed) / ((size_t)2 * a.GP * 4) : 0;
            };
            variant = 0;
            for (int shape : {0, 3, 2, 5})
                if (variant == 0 && async_fits(shape)) variant = 16 + shape;
            for (int shape : {0, 3})
                if (variant == 0 && async_chunk(shape) * 5 >= (size_t)cap_pad * 2) variant = 16 + shape;
            if (variant == 0) variant = 8 + 0;
        } else variant = 44;  // few items per launch (one layer at a time): clustered kernel with the one-sided merge, 4 warps x 3 stages
    }
    if (variant >= 2 && !mma_ok) return fail(ctx, LETHE_ERR_UNSUPPORTED, "tensor-core variants need bf16 and 16-token pages");

    cudaError_t e;
    if (variant >= 32 && variant <= 37) {  // clustered kernel's arithmetic, CTAs of an item merged through scratch instead of a cluster
        const int shape = variant - 32;
        int S = ctx->splits;
        if (S == 0) {  // chunks of about 256 tokens, at most 16 per item
            S = (a.cap_tokens + 255) / 256;
            if (S > 16) S = 16;
            if (S < 1) S = 1;
        }
        const int chunk = ((cap_groups + S - 1) / S) * kGroupTokens;
        if (mma_smem_bytes(c->head_dim, shape, chunk, a.GP) > ctx->max_smem)
            return fail(ctx, LETHE_ERR_UNSUPPORTED, "capacity too large for the on-chip logit buffer at this split count");
        a.splits = S;
        a.chunk_tokens = chunk;
        a.flat_pitch = cap_groups * kGroupTokens;
        auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
        const size_t cnt_bytes = up((size_t)a.n_items * sizeof(int));
        const size_t part_bytes = up((size_t)a.n_items * S * (16 + (size_t)G * c->head_dim) * sizeof(float));
        const size_t lg_bytes = up((size_t)a.n_items * a.flat_pitch * a.GP * sizeof(float));
        const size_t need = cnt_bytes + part_bytes + lg_bytes;
        if (need > ctx->flat_bytes) {
            st = ensure(ctx, &ctx->flat, &ctx->flat_bytes, need, "scratch-merge buffers", stream);
            if (st != LETHE_OK) return st;
            if (cudaMemsetAsync(ctx->flat, 0, ctx->flat_bytes, (cudaStream_t)stream) != cudaSuccess)
                return fail(ctx, LETHE_ERR_CUDA, "clearing the scratch-merge buffers failed");
        }
        // counters sit at the front: they stay zero between launches whatever n_items later calls use
        a.flat_cnt = (int*)ctx->flat;
        a.flat_part = (float*)((char*)ctx->flat + cnt_bytes);
        a.flat_lg = (float*)((char*)ctx->flat + cnt_bytes + part_bytes);
        e = launch_attend_mma(a, c->head_dim, shape, paged, (cudaStream_t)stream);
    } else if (variant >= 16 && variant < 32) {  // persistent, asynchronous epilogue: both logit buffers (item parity) share what is left
        if (ctx->splits > 1) return fail(ctx, LETHE_ERR_INVALID_ARG, "the persistent variants do not split items");
        const bool tma = variant >= 24;
        const int shape = tma ? variant - 24 : variant - 16;
        if (tma) {  // tensor maps over K and V as [rows][D]
            const unsigned long long rows = paged ? (unsigned long long)c->n_pages * c->page_tokens
                                                  : (unsigned long long)c->n_layers * c->batch * c->n_kv_heads * c->capacity;
            if (rows > 0x7fffffffULL) return fail(ctx, LETHE_ERR_UNSUPPORTED, "cache too large for the TMA variant");
            if (sizeof(ctx->tma_maps) < tma_maps_bytes()) return fail(ctx, LETHE_ERR_CUDA, "tensor map storage");
            if (!resolve_tma_encode(ctx)) return fail(ctx, LETHE_ERR_CUDA, "cuTensorMapEncodeTiled is not available");
            if (ctx->tma_k != c->k || ctx->tma_v != c->v || ctx->tma_rows != rows || ctx->tma_d != c->head_dim) {
                if (!build_tma_maps(ctx->tma_encode, c->k, c->v, rows, c->head_dim, ctx->tma_maps))
                    return fail(ctx, LETHE_ERR_CUDA, "cuTensorMapEncodeTiled failed");
                ctx->tma_k = c->k; ctx->tma_v = c->v; ctx->tma_rows = rows; ctx->tma_d = c->head_dim;
            }
        }
        a.splits = 1;
        const size_t fixed = async_smem_bytes(c->head_dim, shape, 0, a.GP);
        int fit = 0;
        if (fixed < ctx->max_smem) fit = (int)((ctx->max_smem - fixed) / ((size_t)2 * a.GP * 4) / kGroupTokens) * kGroupTokens;
        a.chunk_tokens = fit < cap_groups * kGroupTokens ? fit : cap_groups * kGroupTokens;
        if (a.chunk_tokens < kGroupTokens)
            return fail(ctx, LETHE_ERR_UNSUPPORTED, "no shared memory left for the logit buffers of this persistent shape");
        const int grid = a.n_items < ctx->sm_count ? a.n_items : ctx->sm_count;
        if (a.chunk_tokens < cap_groups * kGroupTokens) {
            a.spill_tokens = cap_groups * kGroupTokens - a.chunk_tokens;
            const size_t need = (size_t)grid * 2 * a.spill_tokens * a.GP * sizeof(float);
            st = ensure(ctx, &ctx->scratch, &ctx->scratch_bytes, need, "logit overflow scratch", stream);
            if (st != LETHE_OK) return st;
            a.spill = (float*)ctx->scratch;
        }
        e = launch_attend_async(a, c->head_dim, shape, paged, grid, (cudaStream_t)stream, tma, ctx->tma_maps);
    } else if (variant >= 8 && variant < 16) {  // persistent: one CTA per SM walks all items
        if (ctx->splits > 1) return fail(ctx, LETHE_ERR_INVALID_ARG, "the persistent variant does not split items");
        a.splits = 1;
        a.chunk_tokens = stream_chunk(variant - 8);
        if (a.chunk_tokens < kGroupTokens)
            return fail(ctx, LETHE_ERR_UNSUPPORTED, "no shared memory left for the logit buffer of this persistent shape");
        const int grid = a.n_items < ctx->sm_count ? a.n_items : ctx->sm_count;
        if (a.chunk_tokens < cap_groups * kGroupTokens) {  // overflow of the logit buffer: one slice per CTA
            a.spill_tokens = cap_groups * kGroupTokens - a.chunk_tokens;
            const size_t need = (size_t)grid * a.spill_tokens * a.GP * sizeof(float);
            st = ensure(ctx, &ctx->scratch, &ctx->scratch_bytes, need, "logit overflow scratch", stream);
            if (st != LETHE_OK) return st;
            a.spill = (float*)ctx->scratch;
        }
        e = launch_attend_stream(a, c->head_dim, variant - 8, paged, grid, (cudaStream_t)stream);
    } else {
        // CTAs per item: the smallest cluster whose logit buffer fits, grown until the grid covers the SMs twice.
        const bool layer_kernel = variant >= 44;
        auto smem_for = [&](int S) -> size_t {
            const int chunk = ((cap_groups + S - 1) / S) * kGroupTokens;
            return variant == 1 ? simt_smem_bytes(c->head_dim, chunk, a.GP)
                                : (layer_kernel ? layer_smem_bytes(c->head_dim, variant - 44, chunk, a.GP)
                                                : mma_smem_bytes(c->head_dim, variant - 2, chunk, a.GP));
        };
        int S = ctx->splits;
        if (S == 0) {
            S = 1;
            while (S < 16 && smem_for(S) > ctx->max_smem) S *= 2;
            // enough CTAs to cover the SMs once, and 4-CTA clusters while the items are fewer than the SMs; larger
            // clusters cost more in scheduling and merging than they gain (measured on ~1100-token items, per 32-layer
            // step: 64 items per launch 0.317 ms with 4 CTAs per item against 0.394 with 2; 128 items 0.317 against
            // 0.398; 256 items 0.310 with 1 against 0.318 with 4)
            while (S < 8 && ((long long)a.n_items * S < ctx->sm_count || (a.n_items <= ctx->sm_count && S < 4)) &&
                   cap_groups / (2 * S) >= 4)
                S *= 2;
        }
        if (ctx->variant == 0 && variant == 44) {
            // automatic choice of the layer kernel's shape: two CTAs per SM matter more than a third pipeline stage
            // (wide groups with long chunks, e.g. G = 7 at capacity 5312: 36 us per 128-item launch with two stages
            // against 47 us with three, where only one CTA fits)
            const int chunk = ((cap_groups + S - 1) / S) * kGroupTokens;
            auto two_fit = [&](int shape) { return 2 * (layer_smem_bytes(c->head_dim, shape, chunk, a.GP) + 1024) <= 228 * 1024; };
            if (!two_fit(0) && two_fit(2)) variant = 46;
        }
        if (smem_for(S) > ctx->max_smem)
            return fail(ctx, LETHE_ERR_UNSUPPORTED, "capacity too large for the on-chip logit buffer at this split count");
        a.splits = S;
        a.chunk_tokens = ((cap_groups + S - 1) / S) * kGroupTokens;
        e = variant == 1 ? launch_attend_simt(a, c->dtype, c->head_dim, paged, (cudaStream_t)stream)
                         : (layer_kernel ? launch_attend_layer(a, c->head_dim, variant - 44, paged, (cudaStream_t)stream)
                                         : launch_attend_mma(a, c->head_dim, variant - 2, paged, (cudaStream_t)stream));
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e, "decode_attend launch");
    return LETHE_OK;
}

lethe_status lethe_decode_attend_host(lethe_ctx* ctx, const lethe_cache* c, int layer_begin, int layer_end,
                                      const void* q_host, const void* k_new_host, const void* v_new_host,
                                      const int32_t* token_pos_host, const float* scale, float gamma, void* out_host,
                                      float* lse_host, void* stream) {
    // every host-detectable error is found here, before staging is sized or a copy is enqueued
    lethe_status st = check_attend_args(ctx, c, layer_begin, layer_end, q_host, k_new_host, v_new_host, token_pos_host,
                                        scale, gamma, out_host, false);
    if (st != LETHE_OK) return st;
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, LETHE_ERR_CUDA, "cannot select the context's device");
    const size_t nl = (size_t)(layer_end - layer_begin);
    const size_t eb = c->dtype == LETHE_F32 ? 4 : 2;  // activations: fp32 with an fp32 cache, bf16 otherwise
    auto up = [](size_t x) { return (x + 255) & ~(size_t)255; };
    const size_t q_bytes = nl * c->batch * c->n_q_heads * c->head_dim * eb;
    const size_t kv_bytes = nl * c->batch * c->n_kv_heads * c->head_dim * eb;
    const size_t pos_bytes = (size_t)c->batch * 4;
    const size_t lse_bytes = nl * c->batch * c->n_q_heads * 4;
    cudaStream_t s = (cudaStream_t)stream;
    cudaError_t e;
    // Results that live in page-locked host memory are written there by the kernel itself (the device-side alias of
    // the buffer): the stores cross the bus while the kernel runs and no download follows.  Pageable buffers are
    // staged in device memory and copied; so is a page-locked buffer whose alias is not 16-byte aligned (a pointer
    // into the middle of a larger allocation), which the kernels' vector accesses could not use.
    auto device_alias = [](void* host, size_t bytes, bool need16) -> void* {
        cudaPointerAttributes lo, hi;
        if (cudaPointerGetAttributes(&lo, host) != cudaSuccess ||
            cudaPointerGetAttributes(&hi, (char*)host + bytes - 1) != cudaSuccess) {
            cudaGetLastError();
            return nullptr;
        }
        if (lo.type != cudaMemoryTypeHost || hi.type != cudaMemoryTypeHost || !lo.devicePointer || !hi.devicePointer) return nullptr;
        if ((char*)hi.devicePointer - (char*)lo.devicePointer != (ptrdiff_t)(bytes - 1)) return nullptr;
        if (need16 && ((uintptr_t)lo.devicePointer & 15)) return nullptr;
        return lo.devicePointer;
    };
    void* out_alias = device_alias(out_host, q_bytes, true);
    float* lse_alias = (lse_host && out_alias) ? (float*)device_alias(lse_host, lse_bytes, false) : nullptr;
    if (lse_host && !lse_alias) out_alias = nullptr;  // one path for both results
    // Inputs in page-locked memory as well: the kernels read them over the bus themselves and no upload precedes the
    // launch.  The persistent kernels fetch them an item ahead of their use, under the streaming of the previous
    // item; the asynchronous-epilogue kernel reads every input byte once (an epilogue warp stages an item's query
    // rows and appended row in shared memory), the synchronous one fetches them per warp into registers.  Measured
    // per step, results written by the kernel in both cases: Llama-8B shape 0.22 ms against 0.29 ms with the upload,
    // long-reasoning shape 2.81 against 3.20, Qwen shape 0.67 against 0.80.  The kernels with one CTA or cluster per
    // item need the query rows at once, so each CTA starts with a round trip over the bus, and still come out ahead
    // of the upload (quantised Llama-8B shape 0.20 against 0.23, clustered bf16 kernel 0.35 against 0.37).
    if (out_alias) {
        void* qa = device_alias((void*)q_host, q_bytes, true);
        void* ka = k_new_host ? device_alias((void*)k_new_host, kv_bytes, true) : nullptr;
        void* va = v_new_host ? device_alias((void*)v_new_host, kv_bytes, true) : nullptr;
        void* pa = k_new_host ? device_alias((void*)token_pos_host, pos_bytes, false) : nullptr;
        if (qa && (!k_new_host || (ka && va && pa)))   // nothing is staged: the staging area is not touched
            return lethe_decode_attend(ctx, c, layer_begin, layer_end, qa, ka, va, (const int32_t*)pa, scale, gamma, out_alias,
                                       lse_host ? lse_alias : nullptr, stream);
    }
    // staging: the inputs always, the results only when the kernel cannot write the caller's buffers
    const size_t in_bytes = up(q_bytes) + (k_new_host ? 2 * up(kv_bytes) + up(pos_bytes) : 0);
    const size_t res_bytes = out_alias ? 0 : up(q_bytes) + (lse_host ? up(lse_bytes) : 0);
    st = ensure(ctx, &ctx->staging, &ctx->staging_bytes, in_bytes + res_bytes, "staging", stream);
    if (st != LETHE_OK) return st;
    char* p = (char*)ctx->staging;
    void* dq = p; p += up(q_bytes);
    void* dk = nullptr; void* dv = nullptr; int32_t* dpos = nullptr;
    if (k_new_host) {
        dk = p; p += up(kv_bytes);
        dv = p; p += up(kv_bytes);
        dpos = (int32_t*)p; p += up(pos_bytes);
    }
    void* dout = out_alias;
    float* dlse = lse_alias;
    if (!out_alias) {
        dout = p; p += up(q_bytes);
        dlse = lse_host ? (float*)p : nullptr;
    }
    // Staged path.  Layers are independent, so a call that covers many of them is cut into two chunks of layers: the
    // upload of the second and the download of the first run on their own streams (separate copy engines) under the
    // other chunk's kernel.  (Measured on the Llama-8B shape with staged results: 0.344 ms per step as one chunk,
    // 0.318 as two, 0.326 as three, 0.351 as four: smaller launches lose more than the shorter exposed copies gain.)
    // When the kernel writes the results itself there is no download to hide and one chunk is best (0.288 against
    // 0.305 as two).  Small calls take the plain path: upload, one launch, download, all on the caller's stream.
    const long long items_per_layer = (long long)c->batch * c->n_kv_heads;
    int chunks = 1;
    if (!out_alias && nl >= 4 && items_per_layer * (long long)(nl / 2) >= 4LL * ctx->sm_count) chunks = 2;
    if (chunks > 1 && !ctx->host_pipeline_ready) {
        bool ok = cudaStreamCreateWithFlags(&ctx->up_stream, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaStreamCreateWithFlags(&ctx->down_stream, cudaStreamNonBlocking) == cudaSuccess &&
                  cudaEventCreateWithFlags(&ctx->ev_start, cudaEventDisableTiming) == cudaSuccess &&
                  cudaEventCreateWithFlags(&ctx->ev_down, cudaEventDisableTiming) == cudaSuccess;
        for (int i = 0; i < 8 && ok; ++i)
            ok = cudaEventCreateWithFlags(&ctx->ev_up[i], cudaEventDisableTiming) == cudaSuccess &&
                 cudaEventCreateWithFlags(&ctx->ev_done[i], cudaEventDisableTiming) == cudaSuccess;
        if (!ok) return cuda_fail(ctx, cudaGetLastError(), "decode_attend_host: creating copy streams");
        ctx->host_pipeline_ready = true;
    }
    if (chunks == 1) {
        e = cudaMemcpyAsync(dq, q_host, q_bytes, cudaMemcpyHostToDevice, s);
        if (e == cudaSuccess && k_new_host) {
            e = cudaMemcpyAsync(dk, k_new_host, kv_bytes, cudaMemcpyHostToDevice, s);
            if (e == cudaSuccess) e = cudaMemcpyAsync(dv, v_new_host, kv_bytes, cudaMemcpyHostToDevice, s);
            if (e == cudaSuccess) e = cudaMemcpyAsync(dpos, token_pos_host, pos_bytes, cudaMemcpyHostToDevice, s);
        }
        if (e != cudaSuccess) return cuda_fail(ctx, e, "decode_attend_host: upload");
        st = lethe_decode_attend(ctx, c, layer_begin, layer_end, dq, k_new_host ? dk : nullptr, k_new_host ? dv : nullptr,
                                 k_new_host ? dpos : nullptr, scale, gamma, dout, lse_host ? dlse : nullptr, stream);
        if (st != LETHE_OK) return st;
        if (out_alias) return LETHE_OK;
        e = cudaMemcpyAsync(out_host, dout, q_bytes, cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess && lse_host) e = cudaMemcpyAsync(lse_host, dlse, lse_bytes, cudaMemcpyDeviceToHost, s);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "decode_attend_host: download");
        return LETHE_OK;
    }

    // the copy streams start after whatever the caller's stream holds (the previous call's kernels read the staging)
    e = cudaEventRecord(ctx->ev_start, s);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->up_stream, ctx->ev_start, 0);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->down_stream, ctx->ev_start, 0);
    if (e == cudaSuccess && k_new_host) e = cudaMemcpyAsync(dpos, token_pos_host, pos_bytes, cudaMemcpyHostToDevice, ctx->up_stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "decode_attend_host: pipeline start");
    const size_t q_layer = q_bytes / nl, kv_layer = kv_bytes / nl, lse_layer = lse_bytes / nl;
    size_t l0 = 0;
    for (int ci = 0; ci < chunks; ++ci) {
        const size_t l1 = nl * (size_t)(ci + 1) / chunks;
        const size_t nq = (l1 - l0) * q_layer, nkv = (l1 - l0) * kv_layer;
        e = cudaMemcpyAsync((char*)dq + l0 * q_layer, (const char*)q_host + l0 * q_layer, nq, cudaMemcpyHostToDevice, ctx->up_stream);
        if (e == cudaSuccess && k_new_host) {
            e = cudaMemcpyAsync((char*)dk + l0 * kv_layer, (const char*)k_new_host + l0 * kv_layer, nkv, cudaMemcpyHostToDevice, ctx->up_stream);
            if (e == cudaSuccess)
                e = cudaMemcpyAsync((char*)dv + l0 * kv_layer, (const char*)v_new_host + l0 * kv_layer, nkv, cudaMemcpyHostToDevice, ctx->up_stream);
        }
        if (e == cudaSuccess) e = cudaEventRecord(ctx->ev_up[ci], ctx->up_stream);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(s, ctx->ev_up[ci], 0);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "decode_attend_host: upload");
        st = lethe_decode_attend(ctx, c, layer_begin + (int)l0, layer_begin + (int)l1, (char*)dq + l0 * q_layer,
                                 k_new_host ? (char*)dk + l0 * kv_layer : nullptr, k_new_host ? (char*)dv + l0 * kv_layer : nullptr,
                                 k_new_host ? dpos : nullptr, scale, gamma, (char*)dout + l0 * q_layer,
                                 lse_host ? dlse + l0 * (lse_layer / 4) : nullptr, stream);
        if (st != LETHE_OK) return st;
        if (out_alias) {
            l0 = l1;
            continue;
        }
        e = cudaEventRecord(ctx->ev_done[ci], s);
        if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->down_stream, ctx->ev_done[ci], 0);
        if (e == cudaSuccess)
            e = cudaMemcpyAsync((char*)out_host + l0 * q_layer, (char*)dout + l0 * q_layer, nq, cudaMemcpyDeviceToHost, ctx->down_stream);
        if (e == cudaSuccess && lse_host)
            e = cudaMemcpyAsync((char*)lse_host + l0 * lse_layer, (char*)dlse + l0 * lse_layer, (l1 - l0) * lse_layer,
                                cudaMemcpyDeviceToHost, ctx->down_stream);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "decode_attend_host: download");
        l0 = l1;
    }
    if (out_alias) return LETHE_OK;
    // the caller's stream ends after the last download: synchronising it is enough to read the results
    e = cudaEventRecord(ctx->ev_down, ctx->down_stream);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(s, ctx->ev_down, 0);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "decode_attend_host: pipeline end");
    return LETHE_OK;
}

lethe_status lethe_estimate_sparsity(lethe_ctx* ctx, const lethe_cache* c, float* sparsity, void* stream) {
    lethe_status st = check_cache(ctx, c);
    if (st != LETHE_OK) return st;
    ctx->last_len = nullptr;  // the next decode call does not follow a decode call
    if (!sparsity) return fail(ctx, LETHE_ERR_INVALID_ARG, "sparsity is NULL");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, LETHE_ERR_CUDA, "cannot select the context's device");
    cudaError_t e = launch_sparsity(view_of(c), sparsity, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "estimate_sparsity launch");
    return LETHE_OK;
}

lethe_status lethe_alloc_budgets(lethe_ctx* ctx, int n_layers, int batch, const float* sparsity,
                                 const int64_t* total_budget, int32_t k_min, int32_t* budgets, void* stream) {
    if (!ctx) return LETHE_ERR_INVALID_ARG;
    if (!sparsity || !total_budget || !budgets) return fail(ctx, LETHE_ERR_INVALID_ARG, "NULL argument");
    if (n_layers < 1 || batch < 1 || k_min < 0) return fail(ctx, LETHE_ERR_INVALID_ARG, "bad sizes");
    if (n_layers > 1024) return fail(ctx, LETHE_ERR_UNSUPPORTED, "more than 1024 layers");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, LETHE_ERR_CUDA, "cannot select the context's device");
    cudaError_t e = launch_budgets(n_layers, batch, sparsity, (const long long*)total_budget, k_min, budgets,
                                   ctx->status, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "alloc_budgets launch");
    return LETHE_OK;
}

// Shared by the two retention entry points: where the survivor lists live, then the longest-first item order.
static lethe_status prune_scratch(lethe_ctx* ctx, const CacheView& v, int* smem_tokens, int32_t** list_scratch, void* stream) {
    // keys / source list live in shared memory when an item fits; otherwise the list goes to global scratch
    const size_t budget_smem = ctx->max_smem - 8 * 1024;
    *smem_tokens = v.cap_tokens;
    *list_scratch = nullptr;
    if ((size_t)*smem_tokens * 4 > budget_smem) {
        *smem_tokens = (int)(budget_smem / 4);
        const size_t need = (size_t)v.L * v.B * v.Hkv * v.cap_tokens * sizeof(int32_t);
        lethe_status st = ensure(ctx, &ctx->scratch, &ctx->scratch_bytes, need, "prune scratch", stream);
        if (st != LETHE_OK) return st;
        *list_scratch = (int32_t*)ctx->scratch;
    }
    return LETHE_OK;
}

static lethe_status refresh_order(lethe_ctx* ctx, const lethe_cache* c, const CacheView& v, void* stream) {
    // longest-first order of the items for the persistent attend kernels' work queue
    const long long items = (long long)v.L * v.B * v.Hkv;
    ctx->order_len = nullptr;
    if (items >= 2LL * ctx->sm_count && items <= (1 << 20)) {
        void* buf = ctx->order;
        lethe_status st = ensure(ctx, &buf, &ctx->order_bytes, (size_t)items * sizeof(int32_t), "item order", stream);
        ctx->order = (int32_t*)buf;
        if (st != LETHE_OK) return st;
        cudaError_t e = launch_order(c->len, (int)items, v.cap_tokens, ctx->order, (cudaStream_t)stream);
        if (e != cudaSuccess) return cuda_fail(ctx, e, "item order launch");
        ctx->order_len = c->len;
        ctx->order_items = (int)items;
    }
    return LETHE_OK;
}

lethe_status lethe_rasr_prune(lethe_ctx* ctx, const lethe_cache* c, const int32_t* budgets, int32_t recent,
                              int32_t sink, int32_t* keep_idx, int32_t max_k, void* stream) {
    lethe_status st = check_cache(ctx, c);
    if (st != LETHE_OK) return st;
    ctx->last_len = nullptr;  // the next decode call does not follow a decode call
    if (!budgets) return fail(ctx, LETHE_ERR_INVALID_ARG, "budgets is NULL");
    if (recent < 0 || sink < 0) return fail(ctx, LETHE_ERR_INVALID_ARG, "recent and sink must be >= 0");
    if (keep_idx && max_k < 1) return fail(ctx, LETHE_ERR_INVALID_ARG, "max_k must be positive with keep_idx");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, LETHE_ERR_CUDA, "cannot select the context's device");
    const CacheView v = view_of(c);
    int smem_tokens;
    int32_t* list_scratch;
    st = prune_scratch(ctx, v, &smem_tokens, &list_scratch, stream);
    if (st != LETHE_OK) return st;
    cudaError_t e = launch_rasr_prune(v, budgets, recent, sink, keep_idx, keep_idx ? max_k : 0, smem_tokens,
                                      list_scratch, ctx->status, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "rasr_prune launch");
    return refresh_order(ctx, c, v, stream);
}

lethe_status lethe_segment_prune(lethe_ctx* ctx, const lethe_cache* c, int32_t n_segments, float tau, int32_t recent,
                                 int32_t sink, int32_t* l_evict, int32_t* keep_idx, int32_t max_k, void* stream) {
    lethe_status st = check_cache(ctx, c);
    if (st != LETHE_OK) return st;
    ctx->last_len = nullptr;  // the next decode call does not follow a decode call
    if (!l_evict) return fail(ctx, LETHE_ERR_INVALID_ARG, "l_evict is NULL");
    if (n_segments < 2) return fail(ctx, LETHE_ERR_INVALID_ARG, "n_segments must be at least 2");
    if (!(tau >= 1.0f)) return fail(ctx, LETHE_ERR_INVALID_ARG, "tau must be >= 1");
    if (recent < 0 || sink < 0) return fail(ctx, LETHE_ERR_INVALID_ARG, "recent and sink must be >= 0");
    if (keep_idx && max_k < 1) return fail(ctx, LETHE_ERR_INVALID_ARG, "max_k must be positive with keep_idx");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, LETHE_ERR_CUDA, "cannot select the context's device");
    const CacheView v = view_of(c);
    int smem_tokens;
    int32_t* list_scratch;
    st = prune_scratch(ctx, v, &smem_tokens, &list_scratch, stream);
    if (st != LETHE_OK) return st;
    cudaError_t e = launch_segment_prune(v, n_segments, tau, recent, sink, l_evict, keep_idx, keep_idx ? max_k : 0,
                                         smem_tokens, list_scratch, ctx->status, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "segment_prune launch");
    return refresh_order(ctx, c, v, stream);
}

lethe_status lethe_collapsed_prune(lethe_ctx* ctx, const lethe_cache* c, const int32_t* budgets, int32_t recent,
                                   int32_t sink, int32_t scope, int32_t* keep_idx, int32_t max_k, void* stream) {
    lethe_status st = check_cache(ctx, c);
    if (st != LETHE_OK) return st;
    ctx->last_len = nullptr;  // the next decode call does not follow a decode call
    if (!budgets) return fail(ctx, LETHE_ERR_INVALID_ARG, "budgets is NULL");
    if (recent < 0 || sink < 0) return fail(ctx, LETHE_ERR_INVALID_ARG, "recent and sink must be >= 0");
    if (scope != LETHE_COLLAPSE_HEADS && scope != LETHE_COLLAPSE_HEADS_BATCH)
        return fail(ctx, LETHE_ERR_INVALID_ARG, "scope must be LETHE_COLLAPSE_HEADS or LETHE_COLLAPSE_HEADS_BATCH");
    if (keep_idx && max_k < 1) return fail(ctx, LETHE_ERR_INVALID_ARG, "max_k must be positive with keep_idx");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, LETHE_ERR_CUDA, "cannot select the context's device");
    const CacheView v = view_of(c);
    const int per_group = scope == LETHE_COLLAPSE_HEADS ? v.Hkv : v.B * v.Hkv;
    const size_t groups = (size_t)v.L * v.B * v.Hkv / per_group;
    // scratch: plan [groups] (padded to 256 bytes) | lists [groups][cap_tokens] | keys [groups][cap_tokens] if a
    // group's keys do not fit in shared memory
    const size_t budget_smem = ctx->max_smem - 8 * 1024;
    int smem_tokens = v.cap_tokens;
    const bool spill_keys = (size_t)smem_tokens * 4 > budget_smem;
    if (spill_keys) smem_tokens = (int)(budget_smem / 4);
    const size_t plan_bytes = (groups * sizeof(int32_t) + 255) / 256 * 256;
    const size_t list_bytes = groups * v.cap_tokens * sizeof(int32_t);
    st = ensure(ctx, &ctx->scratch, &ctx->scratch_bytes, plan_bytes + list_bytes * (spill_keys ? 2 : 1), "collapsed prune scratch", stream);
    if (st != LETHE_OK) return st;
    int32_t* plan = (int32_t*)ctx->scratch;
    int32_t* lists = (int32_t*)((char*)ctx->scratch + plan_bytes);
    uint32_t* keys = spill_keys ? (uint32_t*)((char*)ctx->scratch + plan_bytes + list_bytes) : nullptr;
    cudaError_t e = launch_collapsed_prune(v, budgets, recent, sink, per_group, keep_idx, keep_idx ? max_k : 0, smem_tokens,
                                           keys, lists, plan, ctx->status, (cudaStream_t)stream);
    if (e != cudaSuccess) return cuda_fail(ctx, e, "collapsed_prune launch");
    return refresh_order(ctx, c, v, stream);
}

lethe_status lethe_prefill_seed(lethe_ctx* ctx, const lethe_cache* c, const void* q_prompt, int32_t prompt_len,
                                const float* scale, float gamma, void* stream) {
    lethe_status st = check_cache(ctx, c);
    if (st != LETHE_OK) return st;
    ctx->last_len = nullptr;  // the next decode call does not follow a decode call
    if (!q_prompt || !scale) return fail(ctx, LETHE_ERR_INVALID_ARG, "q_prompt and scale are required");
    if (prompt_len < 1 || prompt_len > cap_tokens_of(c)) return fail(ctx, LETHE_ERR_INVALID_ARG, "prompt_len out of range");
    if (!(gamma > 0.f && gamma <= 1.f)) return fail(ctx, LETHE_ERR_INVALID_ARG, "gamma must be in (0, 1]");
    if (c->dtype != LETHE_BF16) return fail(ctx, LETHE_ERR_UNSUPPORTED, "prefill seeding needs a bf16 cache");
    if (c->n_layers > kMaxLayers) return fail(ctx, LETHE_ERR_UNSUPPORTED, "more than 128 layers");
    const int G = c->n_q_heads / c->n_kv_heads;
    if (G > kMaxGroup) return fail(ctx, LETHE_ERR_UNSUPPORTED, "more than 8 query heads per KV head");
    if ((uintptr_t)q_prompt & 15) return fail(ctx, LETHE_ERR_INVALID_ARG, "q_prompt must be 16-byte aligned");
    DeviceGuard guard(ctx->device);
    if (!guard.ok) return fail(ctx, LETHE_ERR_CUDA, "cannot select the context's device");
    PrefillArgs a;
    memset(&a, 0, sizeof(a));
    a.k = c->k; a.page_table = c->page_table; a.len = c->len; a.rel = c->rel; a.q = q_prompt;
    a.status = ctx->status;
    a.n_pages = c->n_pages;
    a.B = c->batch; a.Hq = c->n_q_heads; a.Hkv = c->n_kv_heads; a.G = G; a.P = prompt_len;
    a.HP = G <= 1 ? 1 : (G <= 2 ? 2 : (G <= 4 ? 4 : 8));
    a.capacity = c->capacity; a.cap_tokens = cap_tokens_of(c);
    a.paged = c->layout == LETHE_PAGED;
    a.page_tokens = a.paged ? c->page_tokens : 1;
    a.gamma_log2 = log2f(gamma);
    a.wait_limit = ctx->wait_limit;
    for (int l = 0; l < c->n_layers; ++l) {
        if (!(scale[l] == scale[l]) || fabsf(scale[l]) > 1e30f) return fail(ctx, LETHE_ERR_INVALID_ARG, "scale must be finite");
        a.scale_log2[l] = scale[l] * 1.4426950408889634f;
    }
    const int items = c->n_layers * c->batch * c->n_kv_heads;
    const size_t stats_bytes = ctx->prefill_engine == 1 ? prefill_stats_bytes(items, prompt_len, a.HP)
                                                        : prefill_tc_stats_bytes(items, prompt_len, a.HP);
    st = ensure(ctx, &ctx->scratch, &ctx->scratch_bytes, stats_bytes, "prefill statistics", stream);
    if (st != LETHE_OK) return st;
    a.stats = (float2*)ctx->scratch;
    cudaError_t e;
    if (ctx->prefill_engine == 1) {
        e = launch_prefill(a, items, c->head_dim, (cudaStream_t)stream);
    } else {
        const bool allow_tma = ctx->prefill_engine == 0 && resolve_tma_encode(ctx);
        e = launch_prefill_tc(a, items, c->n_layers, c->head_dim, ctx->tma_encode, allow_tma, (cudaStream_t)stream);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e, "prefill_seed launch");
    return LETHE_OK;
}

}  // extern "C"
