// Arguments shared by the prompt-relevance (prefill seeding) kernels and their launchers.
#pragma once
#include "common.cuh"

namespace lethe {

struct PrefillArgs {
    const void* k;
    const int32_t* page_table;
    const int32_t* len;
    float* rel;
    const void* q;   // [L][B][P][Hq][D]
    float2* stats;   // [items][P][HP]: (max in log2 units, sum)
    int32_t* status;
    long long n_pages;
    int B, Hq, Hkv, G, HP, P;
    int capacity, cap_tokens, page_tokens, paged;
    float gamma_log2;
    int wait_limit;  // poll limit of the bounded mbarrier waits of the tensor-memory kernels (0 = their default)
    float scale_log2[kMaxLayers];
};

size_t prefill_stats_bytes(int items, int P, int HP);
// mma.sync kernels (any bf16 cache)
cudaError_t launch_prefill(const PrefillArgs& a, int items, int D, cudaStream_t stream);
// tcgen05 kernels (accumulators in tensor memory); their statistics scratch holds two partials per column
size_t prefill_tc_stats_bytes(int items, int P, int HP);
cudaError_t launch_prefill_tc(const PrefillArgs& a, int items, int L, int D, void* encode, bool allow_tma, cudaStream_t stream);

__device__ __forceinline__ const char* prefill_row(const PrefillArgs& a, int item, int slot, int row_bytes) {
    if (!a.paged) return (const char*)a.k + ((size_t)item * a.capacity + slot) * row_bytes;
    int page = a.page_table[(size_t)item * a.capacity + slot / a.page_tokens];
    if (page < 0 || page >= a.n_pages) page = 0;  // never read outside the pool (the decode and prune calls report bad ids)
    return (const char*)a.k + ((size_t)page * a.page_tokens + slot % a.page_tokens) * row_bytes;
}

}  // namespace lethe
