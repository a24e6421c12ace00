// Shared device-side definitions of the Lethe kernels (sm_100a).
#pragma once

#include <cooperative_groups.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "../../include/lethe.h"

namespace cg = cooperative_groups;

namespace lethe {

constexpr int kMaxLayers = 128;  // layers addressable by one decode call (scale table travels by value)
constexpr int kMaxGroup = 8;     // query heads per KV head the attend kernels hold at once
constexpr int kGroupTokens = 16; // tokens per streaming group (= one page in the paged layout)

// Arguments of one lethe_decode_attend launch.
struct AttendArgs {
    const void* k;
    const void* v;
    float* rel;
    int32_t* pos;
    int32_t* len;
    const int32_t* page_table;
    const void* q;
    const void* k_new;
    const void* v_new;
    const int32_t* token_pos;
    void* out;
    float* lse;
    int32_t* status;      // device status word: {code, item}
    unsigned int* sched;  // persistent kernel only: {next ticket, CTAs finished}, zero between launches
    // scratch-merged split ("flat") mode of the clustered kernel: the CTAs of an item do not form a cluster; each
    // publishes its partial result and logits, the last one to arrive finishes the item
    int* flat_cnt;        // [n_items] arrival counters, zero between launches
    float* flat_part;     // [n_items][splits][16 + G * D]: 8 x (max, sum), then O
    float* flat_lg;       // [n_items][flat_pitch][GP] scaled logits
    int flat_pitch;       // tokens per item in flat_lg
    const int32_t* order; // persistent kernels: ticket -> item of the call, longest items first (NULL = identity)
    float* spill;         // persistent kernel only: global overflow of the logit buffer, [grid][spill_tokens][GP]
    int spill_tokens;     // tokens per CTA the overflow can hold (0 = the shared-memory buffer covers cap_tokens)
    long long n_pages;
    int B, Hq, Hkv, G, GP;  // GP = G rounded up to even: row pitch of the logit buffer
    int capacity, cap_tokens, page_tokens;
    int layer_begin, n_items;  // items of this call: nl * B * Hkv
    int splits;                // CTAs per item (cluster size)
    int chunk_tokens;          // logit-buffer capacity of one CTA, in tokens
    float gamma;
    int wait_limit;            // poll limit of the bounded mbarrier waits (0 = the kernel's default)
    int early_prefetch;        // layer-pipelined clustered kernel: cached K / V tiles may be fetched before the previous
                               // kernel of the stream has completed (it does not write this call's items)
    float scale_log2[kMaxLayers];  // scale[l] * log2(e) (times the key scale for a quantised cache), by absolute layer
    float k_scale[kMaxLayers];     // quantised caches: a stored key byte x means k_scale[l] * x (else unused)
    float v_scale[kMaxLayers];     // the same for values
};


// Cache state as the prune-round kernels see it.
struct CacheView {
    void* k;
    void* v;
    float* rel;
    int32_t* pos;
    int32_t* len;
    const int32_t* page_table;
    long long n_pages;
    int L, B, Hkv, D, elt_bytes, capacity, cap_tokens, page_tokens, paged;
};

// Host: opt a kernel into the largest dynamic shared memory and non-portable cluster sizes, once per
// (function, device); implemented in api.cu.
cudaError_t prepare_kernel(const void* func, size_t smem_needed);

__device__ __forceinline__ void record_error(int32_t* status, int code, int item) {
    if (atomicCAS(status, 0, code) == 0) status[1] = item;
}

__device__ __forceinline__ float fast_exp2(float x) {
    float y;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(y) : "f"(x));
    return y;
}

// exp2(a - b) that reads (-inf) - (-inf) as 0 rather than NaN
__device__ __forceinline__ float exp2_diff(float a, float b) { return (a == -INFINITY) ? 0.f : fast_exp2(a - b); }

template <typename T>
__device__ __forceinline__ float to_float(T x);
template <>
__device__ __forceinline__ float to_float<float>(float x) {
    return x;
}
template <>
__device__ __forceinline__ float to_float<__nv_bfloat16>(__nv_bfloat16 x) {
    return __bfloat162float(x);
}
template <typename T>
__device__ __forceinline__ T from_float(float x);
template <>
__device__ __forceinline__ float from_float<float>(float x) {
    return x;
}
template <>
__device__ __forceinline__ __nv_bfloat16 from_float<__nv_bfloat16>(float x) {
    return __float2bfloat16_rn(x);
}

// Decoded position of a CTA inside the launch.
struct ItemCoord {
    int item_call;  // item index within the call
    int item;       // absolute flat item (l * B + b) * Hkv + hkv
    int li, l, b, hkv;
    int rank;  // CTA rank among the item's splits
};

__device__ __forceinline__ ItemCoord decode_item(const AttendArgs& a) {
    ItemCoord c;
    c.item_call = blockIdx.x / a.splits;
    c.rank = blockIdx.x % a.splits;
    c.hkv = c.item_call % a.Hkv;
    c.b = (c.item_call / a.Hkv) % a.B;
    c.li = c.item_call / (a.Hkv * a.B);
    c.l = a.layer_begin + c.li;
    c.item = (c.l * a.B + c.b) * a.Hkv + c.hkv;
    return c;
}

// Token range of this CTA: whole 16-token groups [g_begin, g_end) of the item's ceil(n/16) groups.
__device__ __forceinline__ void split_range(int n, int splits, int rank, int& g_begin, int& g_end) {
    const int ng = (n + kGroupTokens - 1) / kGroupTokens;
    const int per = (ng + splits - 1) / splits;
    g_begin = min(ng, rank * per);
    g_end = min(ng, g_begin + per);
}

// Byte address of row `slot` of an item in K or V.  PAGED returns nullptr for a page id outside the pool.
template <bool PAGED>
__device__ __forceinline__ const char* row_ptr(const AttendArgs& a, const void* base, int item, int slot, int row_bytes,
                                               bool* bad_page) {
    if (!PAGED) return (const char*)base + ((size_t)item * a.capacity + slot) * row_bytes;
    const int page = a.page_table[(size_t)item * a.capacity + slot / a.page_tokens];
    if (page < 0 || page >= a.n_pages) {
        *bad_page = true;
        return nullptr;
    }
    return (const char*)base + ((size_t)page * a.page_tokens + slot % a.page_tokens) * row_bytes;
}

// Shared-memory bookkeeping used by the common epilogue.
struct EpilogueSmem {
    float2 wstat[16][kMaxGroup];  // per warp, per head: (running max in log2 units, partial sum)
    float wscale[16][kMaxGroup];  // per warp rescale factor to the CTA max
    float2 cta_stat[kMaxGroup];   // per head: (CTA max, CTA sum)
    float2 fin[kMaxGroup];        // per head: (global max, 1 / global sum)
    float rscale[16][kMaxGroup];  // per cluster rank: exp2(m_r - m) / l
    int flags[4];
};

// Old relevance values a thread will update: loaded early so that their latency hides behind the merge.
constexpr int kRelPrefetch = 8;
constexpr int kRelBatch = 4;  // tokens per thread per batch in the tail of a long item's relevance update

template <int NT>
__device__ __forceinline__ void prefetch_rel(const AttendArgs& a, const ItemCoord& ic, int t0, int hi_tok,
                                             int append_slot, float (&old)[kRelPrefetch]) {
    const float* rel = a.rel + (size_t)ic.item * a.cap_tokens;
#pragma unroll
    for (int i = 0; i < kRelPrefetch; ++i) {
        const int j = t0 + (int)threadIdx.x + i * NT;
        old[i] = (j < hi_tok && j != append_slot) ? rel[j] : 0.f;
    }
}

// Eq. 5 for the tokens [t0, hi_tok) of an item whose scaled logits (log2 units) are parked in `lg`:
// rel[j] = gamma * rel[j] + sum over the group's heads of exp2(s_hj - m_h) / l_h, with fin[h] = (m_h, 1 / l_h) the
// exact global statistics.  rel_old holds the values prefetch_rel loaded for the thread's first kRelPrefetch tokens;
// with first_batch = kRelPrefetch those tokens are skipped and [t0, hi_tok) is a range that starts after them.
template <int NT, int GT = 0>  // GT: the group size when it is a compile-time constant of the caller, else 0
__device__ __forceinline__ void relevance_update(const AttendArgs& a, const ItemCoord& ic, const float2* fin, const float* lg,
                                                 int t0, int hi_tok, int append_slot, const float (&rel_old)[kRelPrefetch],
                                                 int first_batch = 0) {
    const int tid = threadIdx.x;
    const int G = GT ? GT : a.G;
    float* rel = a.rel + (size_t)ic.item * a.cap_tokens;
    const int GP = GT ? ((GT + 1) & ~1) : a.GP;
    float fm[kMaxGroup], fi[kMaxGroup];
#pragma unroll
    for (int h = 0; h < kMaxGroup; ++h) {
        fm[h] = fin[h].x;
        fi[h] = fin[h].y;
    }
    // Rows are loaded a batch ahead of the stores to rel: the compiler cannot tell that rel and the logit buffer
    // never alias, and would otherwise keep every token's loads behind the previous token's store.
    auto load_row = [&](int j, float (&s)[kMaxGroup]) {
        const float* row = lg + (size_t)(j - t0) * GP;
#pragma unroll
        for (int h = 0; h < kMaxGroup; ++h)
            if (h < G) s[h] = row[h];
    };
    auto mass_from = [&](const float (&s)[kMaxGroup]) {
        float mass = 0.f;
#pragma unroll
        for (int h = 0; h < kMaxGroup; ++h)
            if (h < G) mass += fast_exp2(s[h] - fm[h]) * fi[h];
        return mass;
    };
#pragma unroll
    for (int i0 = 0; i0 < kRelPrefetch; i0 += kRelBatch) {
        if (i0 < first_batch) continue;  // the caller has already updated the tokens rel_old was fetched for
        float s[kRelBatch][kMaxGroup];
#pragma unroll
        for (int u = 0; u < kRelBatch; ++u) {
            const int j = t0 + tid + (i0 + u) * NT;
            if (j < hi_tok) load_row(j, s[u]);
        }
#pragma unroll
        for (int u = 0; u < kRelBatch; ++u) {
            const int j = t0 + tid + (i0 + u) * NT;
            if (j < hi_tok) rel[j] = fmaf(a.gamma, rel_old[i0 + u], mass_from(s[u]));
        }
    }
    for (int j0 = t0 + tid + (first_batch ? 0 : kRelPrefetch * NT); j0 < hi_tok; j0 += kRelBatch * NT) {
        float old[kRelBatch];
        float s[kRelBatch][kMaxGroup];
#pragma unroll
        for (int u = 0; u < kRelBatch; ++u) {
            const int j = j0 + u * NT;
            if (j < hi_tok) {
                old[u] = (j == append_slot) ? 0.f : rel[j];
                load_row(j, s[u]);
            }
        }
#pragma unroll
        for (int u = 0; u < kRelBatch; ++u) {
            const int j = j0 + u * NT;
            if (j < hi_tok) rel[j] = fmaf(a.gamma, old[u], mass_from(s[u]));
        }
    }
}

/*
 * Common tail of both attend kernels.  On entry every warp has written, for the tokens it streamed,
 *   es.wstat[w][h]   = (m, l): running max (log2 units) and sum of exp2(s - m) of head h
 *   wo[w*wo_stride + h*D + d] = sum_j exp2(s_hj - m) V_j[d]
 *   lg[(j - t0)*GP + h] = s_hj in log2 units for every token j of the CTA's range [t0, t1)
 * The function merges warps, then the CTAs of the cluster (distributed shared memory), writes out / lse, and
 * applies Eq. 5 to rel[t0..t1) with the exact global normaliser.
 */
template <typename T, int D, int NW>
__device__ void combine_and_finish(const AttendArgs& a, const ItemCoord& ic, EpilogueSmem& es, float* wo, int wo_stride,
                                   float* cta_o /*[kMaxGroup][D]*/, const float* lg, int t0, int t1, int append_slot,
                                   int n, const float (&rel_old)[kRelPrefetch]) {
    const int tid = threadIdx.x;
    const int G = a.G;
    constexpr int NT = NW * 32;
    __syncthreads();
    if (tid < kMaxGroup) {
        const int h = tid;
        float m = -INFINITY;
        for (int w = 0; w < NW; ++w) m = fmaxf(m, es.wstat[w][h].x);
        float l = 0.f;
        for (int w = 0; w < NW; ++w) {
            const float sc = exp2_diff(es.wstat[w][h].x, m);
            es.wscale[w][h] = sc;
            l += es.wstat[w][h].y * sc;
        }
        es.cta_stat[h] = make_float2(m, l);
    }
    __syncthreads();
    for (int idx = tid; idx < G * D; idx += NT) {
        const int h = idx / D;
        float acc = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) acc += wo[w * wo_stride + idx] * es.wscale[w][h];
        cta_o[idx] = acc;
    }

    const int S = a.splits;
    T* out = (T*)a.out + ((size_t)(ic.li * a.B + ic.b) * a.Hq + ic.hkv * G) * D;
    float* lse = a.lse ? a.lse + (size_t)(ic.li * a.B + ic.b) * a.Hq + ic.hkv * G : nullptr;
    if (S == 1) {
        __syncthreads();
        if (tid < kMaxGroup) {
            const float2 st = es.cta_stat[tid];
            es.fin[tid] = make_float2(st.x, st.y > 0.f ? 1.f / st.y : 0.f);
            if (lse && tid < G) lse[tid] = st.y > 0.f ? (st.x + log2f(st.y)) * 0.6931471805599453f : -INFINITY;
        }
        __syncthreads();
        for (int idx = tid; idx < G * D; idx += NT) out[idx] = from_float<T>(cta_o[idx] * es.fin[idx / D].y);
    } else {
        cg::cluster_group cluster = cg::this_cluster();
        cluster.sync();  // every CTA's cta_o / cta_stat is complete and visible cluster-wide
        // all ranks' (max, sum) pairs into local shared memory with one remote round trip (wstat is free by now)
        if (tid < S * kMaxGroup) {
            const int r = tid / kMaxGroup, h = tid % kMaxGroup;
            es.wstat[r][h] = cluster.map_shared_rank(&es.cta_stat[0], r)[h];
        }
        __syncthreads();
        if (tid < kMaxGroup) {
            const int h = tid;
            float m = -INFINITY;
            for (int r = 0; r < S; ++r) m = fmaxf(m, es.wstat[r][h].x);
            float l = 0.f;
            for (int r = 0; r < S; ++r) l += es.wstat[r][h].y * exp2_diff(es.wstat[r][h].x, m);
            const float inv = l > 0.f ? 1.f / l : 0.f;
            for (int r = 0; r < S; ++r) es.rscale[r][h] = exp2_diff(es.wstat[r][h].x, m) * inv;
            es.fin[h] = make_float2(m, inv);
            if (lse && ic.rank == 0 && h < G) lse[h] = l > 0.f ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
        }
        __syncthreads();
        // each rank finishes an equal slice of the G*D outputs
        const int total = G * D;
        const int per = (total + S - 1) / S;
        const int lo = ic.rank * per, hi = min(total, lo + per);
        for (int idx = lo + tid; idx < hi; idx += NT) {
            const int h = idx / D;
            float acc = 0.f;
            for (int r = 0; r < S; ++r) acc += cluster.map_shared_rank(cta_o, r)[idx] * es.rscale[r][h];
            out[idx] = from_float<T>(acc);
        }
    }

    relevance_update<NT>(a, ic, es.fin, lg, t0, min(t1, n), append_slot, rel_old);
    if (S > 1) cg::this_cluster().sync();  // peers may still be reading this CTA's shared memory
    if (append_slot >= 0 && ic.rank == 0 && tid == 0) a.len[ic.item] = n;
}

/*
 * Tail of the clustered kernel in scratch-merged mode.  Same inputs as combine_and_finish.  Every CTA merges its
 * warps, publishes (max, sum, O) and its logits to global scratch and bumps the item's arrival counter; the CTA
 * that arrives last merges all partials, writes out / lse, applies Eq. 5 to the whole item, resets the counter
 * and stores len.  Nobody waits for anybody, so the CTAs need not be co-scheduled.
 */
template <typename T, int D, int NW>
__device__ void flat_finish(const AttendArgs& a, const ItemCoord& ic, EpilogueSmem& es, float* wo, int wo_stride,
                            float* cta_o /*[kMaxGroup][D]*/, const float* lg, int t0, int t1, int append_slot, int n) {
    const int tid = threadIdx.x;
    const int G = a.G, GP = a.GP, S = a.splits;
    constexpr int NT = NW * 32;
    __syncthreads();
    if (tid < kMaxGroup) {
        const int h = tid;
        float m = -INFINITY;
        for (int w = 0; w < NW; ++w) m = fmaxf(m, es.wstat[w][h].x);
        float l = 0.f;
        for (int w = 0; w < NW; ++w) {
            const float sc = exp2_diff(es.wstat[w][h].x, m);
            es.wscale[w][h] = sc;
            l += es.wstat[w][h].y * sc;
        }
        es.cta_stat[h] = make_float2(m, l);
    }
    __syncthreads();
    const int part_floats = 16 + G * D;
    float* part = a.flat_part + ((size_t)ic.item_call * S + ic.rank) * part_floats;
    if (tid < kMaxGroup) reinterpret_cast<float2*>(part)[tid] = es.cta_stat[tid];
    for (int idx = tid; idx < G * D; idx += NT) {
        const int h = idx / D;
        float acc = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) acc += wo[w * wo_stride + idx] * es.wscale[w][h];
        part[16 + idx] = acc;
    }
    float* glg = a.flat_lg + ((size_t)ic.item_call * a.flat_pitch + t0) * GP;
    const int n_lg = (min(t1, n) - t0) * GP;
    for (int i = tid; 2 * i < n_lg; i += NT)  // GP is even and t0 a multiple of 16: 8-byte pieces are aligned
        reinterpret_cast<float2*>(glg)[i] = reinterpret_cast<const float2*>(lg)[i];
    __threadfence();
    __syncthreads();
    if (tid == 0) es.flags[0] = (atomicAdd(&a.flat_cnt[ic.item_call], 1) == S - 1) ? 1 : 0;
    __syncthreads();
    if (!es.flags[0]) return;
    __threadfence();  // the other CTAs' partials and logits were published before their arrivals

    const float* parts = a.flat_part + (size_t)ic.item_call * S * part_floats;
    // all (max, sum) pairs into shared memory with one round trip, then eight threads merge them
    if (tid < S * kMaxGroup) {
        const int r = tid / kMaxGroup, h = tid % kMaxGroup;
        es.wstat[r][h] = __ldcg(reinterpret_cast<const float2*>(parts + (size_t)r * part_floats) + h);
    }
    __syncthreads();
    if (tid < kMaxGroup) {
        const int h = tid;
        float m = -INFINITY;
        for (int r = 0; r < S; ++r) m = fmaxf(m, es.wstat[r][h].x);
        float l = 0.f;
        for (int r = 0; r < S; ++r) l += es.wstat[r][h].y * exp2_diff(es.wstat[r][h].x, m);
        const float inv = l > 0.f ? 1.f / l : 0.f;
        for (int r = 0; r < S; ++r) es.rscale[r][h] = exp2_diff(es.wstat[r][h].x, m) * inv;
        es.fin[h] = make_float2(m, inv);
        if (a.lse && h < G)
            a.lse[(size_t)(ic.li * a.B + ic.b) * a.Hq + ic.hkv * G + h] = l > 0.f ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
    }
    __syncthreads();
    T* out = (T*)a.out + ((size_t)(ic.li * a.B + ic.b) * a.Hq + ic.hkv * G) * D;
    for (int idx = tid; idx < G * D; idx += NT) {
        const int h = idx / D;
        float acc = 0.f;
#pragma unroll 4
        for (int r = 0; r < S; ++r) acc += __ldcg(parts + (size_t)r * part_floats + 16 + idx) * es.rscale[r][h];
        out[idx] = from_float<T>(acc);
    }
    float fm[kMaxGroup], fi[kMaxGroup];
#pragma unroll
    for (int h = 0; h < kMaxGroup; ++h) {
        fm[h] = es.fin[h].x;
        fi[h] = es.fin[h].y;
    }
    // Eq. 5 over the whole item: logits (L2-resident, written by the item's CTAs) and old scores are fetched for
    // a batch of tokens before any of them is used
    float* rel = a.rel + (size_t)ic.item * a.cap_tokens;
    const float2* item_lg = reinterpret_cast<const float2*>(a.flat_lg + (size_t)ic.item_call * a.flat_pitch * GP);
    const int GP2 = GP / 2;
    constexpr int RB = 4;
    for (int base = 0; base < n; base += RB * NT) {
        float2 lgv[RB][kMaxGroup / 2];
        float oldv[RB];
#pragma unroll
        for (int i = 0; i < RB; ++i) {
            const int j = base + tid + i * NT;
#pragma unroll
            for (int h2 = 0; h2 < kMaxGroup / 2; ++h2)
                lgv[i][h2] = (j < n && h2 < GP2) ? __ldcg(item_lg + (size_t)j * GP2 + h2) : make_float2(0.f, 0.f);
            oldv[i] = (j < n && j != append_slot) ? rel[j] : 0.f;
        }
#pragma unroll
        for (int i = 0; i < RB; ++i) {
            const int j = base + tid + i * NT;
            if (j < n) {
                float mass = 0.f;
#pragma unroll
                for (int h2 = 0; h2 < kMaxGroup / 2; ++h2) {
                    if (2 * h2 < G) mass += fast_exp2(lgv[i][h2].x - fm[2 * h2]) * fi[2 * h2];
                    if (2 * h2 + 1 < G) mass += fast_exp2(lgv[i][h2].y - fm[2 * h2 + 1]) * fi[2 * h2 + 1];
                }
                rel[j] = fmaf(a.gamma, oldv[i], mass);
            }
        }
    }
    if (tid == 0) {
        a.flat_cnt[ic.item_call] = 0;
        if (append_slot >= 0) a.len[ic.item] = n;
    }
}

}  // namespace lethe
