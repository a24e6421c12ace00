// Prune-round kernels: Hoyer sparsity per (layer, sequence), integer budget allocation, and the RASR
// retention step (protected top-k by radix select on the fp32 bit pattern + in-place stable compaction).
#include "common.cuh"

namespace lethe {


// ------------------------------------------------------------------------------------------------ Eq. 1
// One CTA per (layer, sequence); loops over the KV heads; deterministic tree reductions in double.
__global__ void __launch_bounds__(256) sparsity_kernel(CacheView c, float* __restrict__ sparsity) {
    __shared__ double s1[256], s2[256];
    const int lb = blockIdx.x;
    const int tid = threadIdx.x;
    double acc = 0.0;
    for (int h = 0; h < c.Hkv; ++h) {
        const size_t item = (size_t)lb * c.Hkv + h;
        const int n = c.len[item];
        const float* r = c.rel + item * c.cap_tokens;
        double a1 = 0.0, a2 = 0.0;
        for (int j = tid; j < n; j += 256) {
            const double x = (double)r[j];
            a1 += fabs(x);
            a2 += x * x;
        }
        s1[tid] = a1;
        s2[tid] = a2;
        __syncthreads();
        for (int off = 128; off > 0; off >>= 1) {
            if (tid < off) {
                s1[tid] += s1[tid + off];
                s2[tid] += s2[tid + off];
            }
            __syncthreads();
        }
        if (tid == 0) {
            double s = 0.0;
            if (n > 1 && s2[0] > 0.0) {
                const double rn = sqrt((double)n);
                s = (rn - s1[0] / sqrt(s2[0])) / (rn - 1.0);
                s = fmin(fmax(s, 0.0), 1.0);
            }
            acc += s;
        }
        __syncthreads();
    }
    if (tid == 0) sparsity[lb] = (float)(acc / (double)c.Hkv);
}

cudaError_t launch_sparsity(const CacheView& c, float* sparsity, cudaStream_t stream) {
    sparsity_kernel<<<c.L * c.B, 256, 0, stream>>>(c, sparsity);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------------------- budget allocation
// One CTA per sequence.  w_l from one fp32 subtraction and an exact power-of-two scaling; everything after
// is 64-bit integer arithmetic (largest-remainder apportionment, ties to the lower layer).
constexpr int kBudgetMaxLayers = 1024;

__global__ void __launch_bounds__(128) budgets_kernel(int L, int B, const float* __restrict__ sparsity,
                                                      const long long* __restrict__ total, int k_min,
                                                      int32_t* __restrict__ budgets, int32_t* status) {
    __shared__ long long w[kBudgetMaxLayers], rem[kBudgetMaxLayers];
    __shared__ long long red[128];
    __shared__ long long W_sh, R_sh;
    const int b = blockIdx.x, tid = threadIdx.x;
    long long part = 0;
    for (int l = tid; l < L; l += 128) {
        float s = sparsity[(size_t)l * B + b];
        if (!(s >= 0.0f)) s = 0.0f;
        if (s > 1.0f) s = 1.0f;
        const float d = __fsub_rn(1.0f, s);
        long long wl = (long long)rintf(__fmul_rn(d, 1048576.0f));
        if (wl < 1) wl = 1;
        w[l] = wl;
        part += wl;
    }
    red[tid] = part;
    __syncthreads();
    for (int off = 64; off > 0; off >>= 1) {
        if (tid < off) red[tid] += red[tid + off];
        __syncthreads();
    }
    if (tid == 0) W_sh = red[0];
    __syncthreads();
    const long long W = W_sh;
    long long F = total[b] - (long long)L * k_min;
    if (F < 0) {
        for (int l = tid; l < L; l += 128) budgets[(size_t)l * B + b] = k_min;
        if (tid == 0) record_error(status, LETHE_ERR_BUDGET, b);
        return;
    }
    part = 0;
    for (int l = tid; l < L; l += 128) {
        const long long prod = w[l] * F;
        const long long base = prod / W;
        rem[l] = prod - base * W;
        w[l] = base;  // reuse: floor share
        part += base;
    }
    __syncthreads();
    red[tid] = part;
    __syncthreads();
    for (int off = 64; off > 0; off >>= 1) {
        if (tid < off) red[tid] += red[tid + off];
        __syncthreads();
    }
    if (tid == 0) R_sh = F - red[0];
    __syncthreads();
    const long long R = R_sh;  // 0 <= R < L
    for (int l = tid; l < L; l += 128) {
        // rank of layer l by (remainder desc, layer asc)
        long long rank = 0;
        const long long rl = rem[l];
        for (int o = 0; o < L; ++o) rank += (rem[o] > rl) || (rem[o] == rl && o < l);
        budgets[(size_t)l * B + b] = (int32_t)((long long)k_min + w[l] + (rank < R ? 1 : 0));
    }
}

cudaError_t launch_budgets(int L, int B, const float* sparsity, const long long* total, int k_min, int32_t* budgets,
                           int32_t* status, cudaStream_t stream) {
    budgets_kernel<<<B, 128, 0, stream>>>(L, B, sparsity, total, k_min, budgets, status);
    return cudaGetLastError();
}

// ------------------------------------------------------------------------- RASR retention + compaction
// Order-preserving map from fp32 to uint32 (zero of either sign maps to the same key).
__device__ __forceinline__ uint32_t score_key(float x) {
    uint32_t u = __float_as_uint(x);
    if ((u << 1) == 0u) u = 0u;
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

constexpr int kPruneThreads = 512;

// Row index (in rows of the K / V arrays, which share it) of logical slot `slot` of an item, or -1 for a page id
// outside the pool.  Pages of 16 tokens, the only size the tensor-core kernels take, are split with a shift.
__device__ __forceinline__ long long prune_row_index(const CacheView& c, size_t item, int slot, bool* bad) {
    if (!c.paged) return (long long)(item * c.capacity + slot);
    int pg, within;
    if (c.page_tokens == 16) {
        pg = slot >> 4;
        within = slot & 15;
    } else {
        pg = slot / c.page_tokens;
        within = slot % c.page_tokens;
    }
    const int page = c.page_table[item * c.capacity + pg];
    if (page < 0 || page >= c.n_pages) {
        *bad = true;
        return -1;
    }
    return (long long)page * c.page_tokens + within;
}

// Block-wide exclusive scan of one counter per thread (kPruneThreads threads): returns this thread's
// exclusive prefix and the block total.  Ends with a barrier, so warp_buf may be reused at once.
__device__ __forceinline__ void block_scan(int v, int* warp_buf, int& ex, int& tot) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int inc = v;
#pragma unroll
    for (int off = 1; off < 32; off <<= 1) {
        const int t = __shfl_up_sync(0xffffffffu, inc, off);
        if (lane >= off) inc += t;
    }
    if (lane == 31) warp_buf[warp] = inc;
    __syncthreads();
    int base = 0;
    tot = 0;
#pragma unroll
    for (int w = 0; w < kPruneThreads / 32; ++w) {
        const int x = warp_buf[w];
        if (w < warp) base += x;
        tot += x;
    }
    ex = base + inc - v;
    __syncthreads();
}

struct PruneShared {
    int hist[256];
    int warp_buf[kPruneThreads / 32];
    uint32_t sel_prefix;
    int sel_remaining;
    float bcast;
    int ibcast;
};

// take-th largest key (take >= 1) among slots [lo, hi): 4 passes of an 8-bit radix select.  T receives that key
// and need_eq how many of the slots equal to T belong to the top `take` (the oldest ones are meant).
template <class KeyAt>
__device__ __forceinline__ void radix_select(PruneShared& sh, KeyAt key_at, int lo, int hi, int take, uint32_t& T,
                                             int& need_eq) {
    const int tid = threadIdx.x;
    if (tid == 0) {
        sh.sel_prefix = 0u;
        sh.sel_remaining = take;
    }
    for (int pass = 0; pass < 4; ++pass) {
        const int shift = 24 - 8 * pass;
        const uint32_t mask_hi = pass == 0 ? 0u : (0xffffffffu << (shift + 8));
        if (tid < 256) sh.hist[tid] = 0;
        __syncthreads();
        const uint32_t prefix = sh.sel_prefix;
        for (int j = lo + tid; j < hi; j += kPruneThreads) {
            const uint32_t key = key_at(j);
            if ((key & mask_hi) == prefix) atomicAdd(&sh.hist[(key >> shift) & 0xffu], 1);
        }
        __syncthreads();
        // bin holding the remaining-th largest key: suffix sums over the 256 bins by one block scan
        const int remaining = sh.sel_remaining;
        const int h = tid < 256 ? sh.hist[255 - tid] : 0;  // thread t looks at bin 255 - t
        int ex, tot;
        block_scan(h, sh.warp_buf, ex, tot);               // ex = keys in bins above this thread's bin
        if (tid < 256 && ex < remaining && ex + h >= remaining) {
            sh.sel_prefix = prefix | ((uint32_t)(255 - tid) << shift);
            sh.sel_remaining = remaining - ex;
        }
        __syncthreads();
    }
    T = sh.sel_prefix;
    need_eq = sh.sel_remaining;
    __syncthreads();
}

// Ascending sweep over slots [0, n): a slot survives if it is protected (j < prot_lo or j >= prot_hi) or if it
// lies in [sel_lo, sel_hi) and is selected (key > T, or key == T among the first need_eq such slots).  Block
// scans turn the flags into destination slots; the source slot of every destination goes to src_list (which
// may alias the key array: a destination never exceeds its source, and a chunk's keys are read before its
// scans' barriers) and to kout.  Returns the number of survivors.
template <class KeyAt>
__device__ __forceinline__ int sweep_keep(PruneShared& sh, KeyAt key_at, int n, int prot_lo, int prot_hi, int sel_lo,
                                          int sel_hi, bool any_selected, uint32_t T, int need_eq, int32_t* src_list,
                                          int32_t* kout, int max_k) {
    const int tid = threadIdx.x;
    int run_keep = 0, run_eq = 0;
    for (int base = 0; base < n; base += kPruneThreads) {
        const int j = base + tid;
        int is_keep = 0, is_eq = 0;
        if (j < n) {
            if (j < prot_lo || j >= prot_hi) is_keep = 1;
            if (any_selected && j >= sel_lo && j < sel_hi) {
                const uint32_t key = key_at(j);
                if (key > T) is_keep = 1;
                else if (key == T) is_eq = 1;
            }
        }
        int ex_keep, ex_eq, tot_keep, tot_eq;
        // first the rank among slots equal to the threshold (slot order), then the keep scan that depends on it
        block_scan(is_eq, sh.warp_buf, ex_eq, tot_eq);
        if (is_eq && run_eq + ex_eq < need_eq) is_keep = 1;
        block_scan(is_keep, sh.warp_buf, ex_keep, tot_keep);
        if (is_keep) {
            const int dst = run_keep + ex_keep;
            src_list[dst] = j;
            if (kout && dst < max_k) kout[dst] = j;
        }
        run_keep += tot_keep;
        run_eq += tot_eq;
    }
    __syncthreads();
    if (kout)
        for (int i = run_keep + tid; i < max_k; i += kPruneThreads) kout[i] = -1;
    return run_keep;
}

// Rows of K, V, rel, pos move to their destinations in ascending waves: load wave -> barrier -> store wave.
// Because a survivor's destination never exceeds its source and waves ascend, no unread source is overwritten.
// A wave carries RPT rows per thread slot in registers: 4 where two CTAs share an SM, 8 in the instance whose CTA has
// the SM (and its registers) to itself; deeper waves beat overlapping a wave's stores with the next wave's loads at
// the same register budget (ragged round: 3.97 ms against 4.52 ms).
template <int RPT_>
struct MoveWave {
    static constexpr int RPT = RPT_;  // rows each thread slot carries per wave
    uint4 kv[RPT], vv[RPT];
    float rv[RPT];
    int pv[RPT], srcs[RPT];
};
template <int RPT>
__device__ __forceinline__ void move_wave_load(const CacheView& c, size_t item, int keep_n, const int32_t* src_list, int w0, int slots,
                                               int rslot, int piece, int row_bytes, const float* rel, const int32_t* pos,
                                               MoveWave<RPT>& w, bool& bad) {
#pragma unroll
    for (int r = 0; r < RPT; ++r) {
        const int dst = w0 + r * slots + rslot;
        int src = -1;
        if (dst < keep_n) src = src_list[dst];
        // destinations whose source is themselves (the unmoved prefix, and any later fixed point) are skipped
        w.srcs[r] = (src >= 0 && src != dst) ? src : -1;
        w.kv[r] = make_uint4(0, 0, 0, 0);
        w.vv[r] = make_uint4(0, 0, 0, 0);
        w.rv[r] = 0.f;
        w.pv[r] = 0;
        if (w.srcs[r] >= 0) {
            const long long row = prune_row_index(c, item, w.srcs[r], &bad);  // K and V rows share the index
            const char* ks = row < 0 ? nullptr : (const char*)c.k + (size_t)row * row_bytes;
            const char* vs = row < 0 ? nullptr : (const char*)c.v + (size_t)row * row_bytes;
            if (ks && vs) {
                w.kv[r] = *reinterpret_cast<const uint4*>(ks + piece * 16);
                w.vv[r] = *reinterpret_cast<const uint4*>(vs + piece * 16);
            }
            if (piece == 0) {
                w.rv[r] = rel[w.srcs[r]];
                w.pv[r] = pos[w.srcs[r]];
            }
        }
    }
}
template <int RPT>
__device__ __forceinline__ void move_wave_store(const CacheView& c, size_t item, int w0, int slots, int rslot, int piece, int row_bytes,
                                                float* rel, int32_t* pos, const MoveWave<RPT>& w, bool& bad) {
#pragma unroll
    for (int r = 0; r < RPT; ++r) {
        if (w.srcs[r] >= 0) {
            const int dst = w0 + r * slots + rslot;
            const long long row = prune_row_index(c, item, dst, &bad);
            char* kd = row < 0 ? nullptr : (char*)c.k + (size_t)row * row_bytes;
            char* vd = row < 0 ? nullptr : (char*)c.v + (size_t)row * row_bytes;
            if (kd && vd) {
                *reinterpret_cast<uint4*>(kd + piece * 16) = w.kv[r];
                *reinterpret_cast<uint4*>(vd + piece * 16) = w.vv[r];
            }
            if (piece == 0) {
                rel[dst] = w.rv[r];
                pos[dst] = w.pv[r];
            }
        }
    }
}
template <int RPT>
__device__ __forceinline__ void move_rows(const CacheView& c, size_t item, int keep_n, const int32_t* src_list, bool& bad) {
    const int tid = threadIdx.x;
    float* rel = c.rel + item * c.cap_tokens;
    int32_t* pos = c.pos + item * c.cap_tokens;
    const int row_bytes = c.D * c.elt_bytes;
    const int lanes_per_row = row_bytes / 16;            // 16-byte pieces per row (8, 16 or 32)
    const int slots = kPruneThreads / lanes_per_row;     // row slots per pass
    const int rows_per_wave = slots * RPT;
    const int piece = tid % lanes_per_row, rslot = tid / lanes_per_row;
    for (int w0 = 0; w0 < keep_n; w0 += rows_per_wave) {
        MoveWave<RPT> cur;
        move_wave_load(c, item, keep_n, src_list, w0, slots, rslot, piece, row_bytes, rel, pos, cur, bad);
        __syncthreads();  // every source row of this wave has been read
        move_wave_store(c, item, w0, slots, rslot, piece, row_bytes, rel, pos, cur, bad);
        // no barrier needed here: the next wave's sources lie above every destination written so far
    }
}

/*
 * RASR retention, one CTA per item.
 *  1. keys: score_key(rel[j]) into shared memory (or re-read from global when the item is too long).
 *  2. radix select of the `take`-th largest candidate key -> threshold T.
 *  3. ascending sweep -> destination of every survivor (source list in shared memory, in place over the keys;
 *     global scratch for items longer than smem_tokens).
 *  4. rows move in ascending waves.
 */
// DEEP: the item's keys take more shared memory than half an SM has, so one CTA has the SM (and its registers) to
// itself and carries twice the rows per wave.
template <bool DEEP>
__global__ void __launch_bounds__(kPruneThreads, DEEP ? 1 : 2) rasr_prune_kernel(CacheView c, const int32_t* __restrict__ budgets,
                                                                   int recent, int sink, int32_t* keep_idx, int max_k,
                                                                   int smem_tokens, int32_t* list_scratch,
                                                                   int32_t* status) {
    extern __shared__ __align__(16) uint32_t dyn[];  // keys, later the source list  [smem_tokens]
    __shared__ PruneShared sh;

    const size_t item = blockIdx.x;
    const int tid = threadIdx.x;
    const int l = (int)(item / ((size_t)c.B * c.Hkv));
    const int b = (int)((item / c.Hkv) % c.B);
    const int n = c.len[item];
    long long k = budgets[(size_t)l * c.B + b];
    if (k < 0) k = 0;
    int32_t* kout = keep_idx ? keep_idx + item * max_k : nullptr;
    if (k >= n) {  // identity
        if (kout)
            for (int i = tid; i < max_k; i += kPruneThreads) kout[i] = (i < n) ? i : -1;
        return;
    }
    const int n_sink = min(sink, n), n_recent = min(recent, n);
    const int cand_lo = n_sink;
    const int cand_hi = max(n - n_recent, cand_lo);
    const int n_prot = n - (cand_hi - cand_lo);
    if (n_prot > k) {
        k = n_prot;
        if (tid == 0) record_error(status, LETHE_ERR_BUDGET, (int)item);
    }
    const int take = (int)k - n_prot;
    const float* rel = c.rel + item * c.cap_tokens;
    const bool in_smem = n <= smem_tokens;

    if (in_smem)
        for (int j = tid; j < n; j += kPruneThreads) dyn[j] = score_key(rel[j]);
    __syncthreads();
    auto key_at = [&](int j) -> uint32_t { return in_smem ? dyn[j] : score_key(rel[j]); };

    uint32_t T = 0xffffffffu;
    int need_eq = 0;
    if (take > 0) radix_select(sh, key_at, cand_lo, cand_hi, take, T, need_eq);

    int32_t* src_list = in_smem ? reinterpret_cast<int32_t*>(dyn) : list_scratch + item * c.cap_tokens;
    const int keep_n = sweep_keep(sh, key_at, n, cand_lo, cand_hi, cand_lo, cand_hi, take > 0, T, need_eq, src_list, kout, max_k);
    bool bad = false;
    move_rows<DEEP ? 8 : 4>(c, item, keep_n, src_list, bad);
    // any thread may have met the bad page id (each carries its own row slots): reduce over the CTA
    if (__syncthreads_or(bad) && tid == 0) record_error(status, LETHE_ERR_PAGE, (int)item);
    if (tid == 0) c.len[item] = keep_n;
}

/*
 * Algorithm 1 (segmented attention-based token shrinking), one CTA per item, with the size trigger of Sec. 4.1.
 *  n <= l_evict: untouched.  Otherwise the value at every cut point floor(n d / D) of the descending order is
 *  found with a radix select (no full sort), the first cut with v_head >= tau * v_cut is the breakpoint, the
 *  breakpoint highest scores plus sinks plus the recent window survive (same sweep and row moves as the RASR
 *  kernel), and l_evict grows to max(l_evict, breakpoint + recent); without a breakpoint nothing is pruned and
 *  l_evict doubles.
 */
__global__ void __launch_bounds__(kPruneThreads, 2) segment_prune_kernel(CacheView c, int n_segments, float tau, int recent,
                                                                      int sink, int32_t* __restrict__ l_evict,
                                                                      int32_t* keep_idx, int max_k, int smem_tokens,
                                                                      int32_t* list_scratch, int32_t* status) {
    extern __shared__ __align__(16) uint32_t dyn[];
    __shared__ PruneShared sh;

    const size_t item = blockIdx.x;
    const int tid = threadIdx.x;
    const int n = c.len[item];
    const int le = l_evict[item];
    int32_t* kout = keep_idx ? keep_idx + item * max_k : nullptr;
    auto identity = [&]() {
        if (kout)
            for (int i = tid; i < max_k; i += kPruneThreads) kout[i] = (i < n) ? i : -1;
    };
    if (n <= le) {  // not triggered
        identity();
        return;
    }
    const float* rel = c.rel + item * c.cap_tokens;
    const bool in_smem = n <= smem_tokens;
    if (in_smem)
        for (int j = tid; j < n; j += kPruneThreads) dyn[j] = score_key(rel[j]);
    __syncthreads();
    auto key_at = [&](int j) -> uint32_t { return in_smem ? dyn[j] : score_key(rel[j]); };
    auto key_value = [](uint32_t key) -> float {  // inverse of score_key
        return __uint_as_float((key & 0x80000000u) ? (key & 0x7fffffffu) : ~key);
    };

    // v at a rank of the descending order = (rank + 1)-th largest key
    uint32_t T;
    int need_eq;
    radix_select(sh, key_at, 0, n, 1, T, need_eq);
    const float v_head = key_value(T);
    int breakpoint = -1;
    for (int d = 1; d < n_segments; ++d) {
        const int cut = (int)(((long long)n * d) / n_segments);
        if (cut >= n) break;
        float v_cut = v_head;
        if (cut > 0) {
            radix_select(sh, key_at, 0, n, cut + 1, T, need_eq);
            v_cut = key_value(T);
        }
        if (v_head >= __fmul_rn(tau, v_cut)) {
            breakpoint = cut;
            break;
        }
    }
    if (breakpoint < 0) {  // no sharp drop: delay pruning, double the threshold
        identity();
        if (tid == 0) l_evict[item] = (int32_t)min(2LL * le, (long long)(1 << 30));
        return;
    }
    T = 0xffffffffu;
    need_eq = 0;
    if (breakpoint > 0) radix_select(sh, key_at, 0, n, breakpoint, T, need_eq);
    int32_t* src_list = in_smem ? reinterpret_cast<int32_t*>(dyn) : list_scratch + item * c.cap_tokens;
    const int keep_n = sweep_keep(sh, key_at, n, min(sink, n), max(n - recent, 0), 0, n, breakpoint > 0, T, need_eq, src_list,
                                  kout, max_k);
    bool bad = false;
    move_rows<4>(c, item, keep_n, src_list, bad);
    if (__syncthreads_or(bad) && tid == 0) record_error(status, LETHE_ERR_PAGE, (int)item);
    if (tid == 0) {
        c.len[item] = keep_n;
        l_evict[item] = max(le, breakpoint + recent);
    }
}

cudaError_t launch_segment_prune(const CacheView& c, int n_segments, float tau, int recent, int sink, int32_t* l_evict,
                                 int32_t* keep_idx, int max_k, int smem_tokens, int32_t* list_scratch, int32_t* status,
                                 cudaStream_t stream) {
    const size_t smem = (size_t)smem_tokens * 4;
    cudaError_t e = prepare_kernel((const void*)segment_prune_kernel, smem);
    if (e != cudaSuccess) return e;
    segment_prune_kernel<<<c.L * c.B * c.Hkv, kPruneThreads, smem, stream>>>(c, n_segments, tau, recent, sink, l_evict,
                                                                            keep_idx, max_k, smem_tokens, list_scratch,
                                                                            status);
    return cudaGetLastError();
}

cudaError_t launch_rasr_prune(const CacheView& c, const int32_t* budgets, int recent, int sink, int32_t* keep_idx,
                              int max_k, int smem_tokens, int32_t* list_scratch, int32_t* status,
                              cudaStream_t stream) {
    const size_t smem = (size_t)smem_tokens * 4;
    const bool deep = smem > 100 * 1024;  // two CTAs of that size do not fit an SM
    cudaError_t e = prepare_kernel(deep ? (const void*)rasr_prune_kernel<true> : (const void*)rasr_prune_kernel<false>, smem);
    if (e != cudaSuccess) return e;
    if (deep)
        rasr_prune_kernel<true><<<c.L * c.B * c.Hkv, kPruneThreads, smem, stream>>>(c, budgets, recent, sink, keep_idx, max_k,
                                                                                   smem_tokens, list_scratch, status);
    else
        rasr_prune_kernel<false><<<c.L * c.B * c.Hkv, kPruneThreads, smem, stream>>>(c, budgets, recent, sink, keep_idx, max_k,
                                                                                    smem_tokens, list_scratch, status);
    return cudaGetLastError();
}

// ------------------------------------------------------------------ collapsed score (Eq. 2 as printed)
/*
 * One score per token per group (scope 0: the Hkv items of a (layer, sequence); scope 1: the B * Hkv items of a
 * layer) and one retention set shared by the group.  Two launches:
 *   collapsed_select_kernel  one CTA per group: checks that the group's items have one length, sums rel over the
 *                            items in ascending item order (fp32, one rounded add each: the sum decides who is
 *                            kept, so its precision and order are part of the result), radix-selects the
 *                            threshold, sweeps the survivors' source slots into lists[group] and writes
 *                            plan[group] = survivors, or -1 when nothing moves;
 *   collapsed_move_kernel    one CTA per item: compacts the item by its group's list.
 * Items of a group are consecutive in the [L][B][Hkv] order, so group g owns items [g * per_group, (g+1) * per_group).
 */
__global__ void __launch_bounds__(kPruneThreads, 2) collapsed_select_kernel(CacheView c, const int32_t* __restrict__ budgets,
                                                                         int recent, int sink, int per_group,
                                                                         int32_t* keep_idx, int max_k, int smem_tokens,
                                                                         uint32_t* key_scratch, int32_t* lists,
                                                                         int32_t* plan, int32_t* status) {
    extern __shared__ __align__(16) uint32_t dyn[];  // keys [smem_tokens]
    __shared__ PruneShared sh;

    const size_t group = blockIdx.x;
    const size_t first = group * per_group;
    const int tid = threadIdx.x;
    const int n = c.len[first];
    int32_t* kout = keep_idx ? keep_idx + group * max_k : nullptr;

    int differs = 0;
    for (int t = 1 + tid; t < per_group; t += kPruneThreads) differs |= (c.len[first + t] != n);
    if (__syncthreads_or(differs)) {  // slots do not mean the same token in every item: refuse the group
        if (tid == 0) {
            record_error(status, LETHE_ERR_INVALID_ARG, (int)first);
            plan[group] = -1;
        }
        if (kout)
            for (int i = tid; i < max_k; i += kPruneThreads) kout[i] = -1;
        return;
    }
    long long k = budgets[group];
    if (k < 0) k = 0;
    if (k >= n) {  // identity
        if (tid == 0) plan[group] = -1;
        if (kout)
            for (int i = tid; i < max_k; i += kPruneThreads) kout[i] = (i < n) ? i : -1;
        return;
    }
    const int n_sink = min(sink, n), n_recent = min(recent, n);
    const int cand_lo = n_sink;
    const int cand_hi = max(n - n_recent, cand_lo);
    const int n_prot = n - (cand_hi - cand_lo);
    if (n_prot > k) {
        k = n_prot;
        if (tid == 0) record_error(status, LETHE_ERR_BUDGET, (int)first);
    }
    const int take = (int)k - n_prot;

    const bool in_smem = n <= smem_tokens;
    uint32_t* keys = in_smem ? dyn : key_scratch + group * c.cap_tokens;
    const float* rel0 = c.rel + first * c.cap_tokens;
    for (int j = tid; j < n; j += kPruneThreads) {
        float s = 0.f;
        for (int t = 0; t < per_group; ++t) s = __fadd_rn(s, rel0[(size_t)t * c.cap_tokens + j]);
        keys[j] = score_key(s);
    }
    __syncthreads();
    auto key_at = [&](int j) -> uint32_t { return keys[j]; };

    uint32_t T = 0xffffffffu;
    int need_eq = 0;
    if (take > 0) radix_select(sh, key_at, cand_lo, cand_hi, take, T, need_eq);
    const int keep_n = sweep_keep(sh, key_at, n, cand_lo, cand_hi, cand_lo, cand_hi, take > 0, T, need_eq,
                                  lists + group * c.cap_tokens, kout, max_k);
    if (tid == 0) plan[group] = keep_n;
}

__global__ void __launch_bounds__(kPruneThreads, 2) collapsed_move_kernel(CacheView c, int per_group,
                                                                       const int32_t* __restrict__ lists,
                                                                       const int32_t* __restrict__ plan,
                                                                       int32_t* status) {
    const size_t item = blockIdx.x;
    const size_t group = item / per_group;
    const int keep_n = plan[group];
    if (keep_n < 0) return;
    bool bad = false;
    move_rows<4>(c, item, keep_n, lists + group * c.cap_tokens, bad);
    if (__syncthreads_or(bad) && threadIdx.x == 0) record_error(status, LETHE_ERR_PAGE, (int)item);
    if (threadIdx.x == 0) c.len[item] = keep_n;
}

cudaError_t launch_collapsed_prune(const CacheView& c, const int32_t* budgets, int recent, int sink, int per_group,
                                   int32_t* keep_idx, int max_k, int smem_tokens, uint32_t* key_scratch,
                                   int32_t* lists, int32_t* plan, int32_t* status, cudaStream_t stream) {
    const size_t smem = (size_t)smem_tokens * 4;
    cudaError_t e = prepare_kernel((const void*)collapsed_select_kernel, smem);
    if (e != cudaSuccess) return e;
    const int items = c.L * c.B * c.Hkv;
    collapsed_select_kernel<<<items / per_group, kPruneThreads, smem, stream>>>(
        c, budgets, recent, sink, per_group, keep_idx, max_k, smem_tokens, key_scratch, lists, plan, status);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    collapsed_move_kernel<<<items, kPruneThreads, 0, stream>>>(c, per_group, lists, plan, status);
    return cudaGetLastError();
}

// ------------------------------------------------------------ longest-first item order for the attend queue
// One CTA: counting sort of the items by len (1024 buckets over [0, cap_tokens]), longest bucket first.  The
// order only steers the persistent attend kernels' work queue (longest items first shortens the tail of a
// launch); any permutation gives the same results, so ties inside a bucket may land in any order.
__global__ void __launch_bounds__(1024) order_kernel(const int32_t* __restrict__ len, int n_items, int cap_tokens,
                                                     int32_t* __restrict__ order) {
    __shared__ int cnt[1024];
    __shared__ int base[1024];
    const int tid = threadIdx.x;
    cnt[tid] = 0;
    __syncthreads();
    auto bucket = [&](int n) {
        long long bkt = (long long)n * 1023 / (cap_tokens > 0 ? cap_tokens : 1);
        bkt = bkt < 0 ? 0 : (bkt > 1023 ? 1023 : bkt);
        return 1023 - (int)bkt;  // bucket 0 = longest
    };
    for (int i = tid; i < n_items; i += 1024) atomicAdd(&cnt[bucket(len[i])], 1);
    __syncthreads();
    {   // exclusive prefix over the 1024 buckets (Hillis-Steele in shared memory)
        base[tid] = cnt[tid];
        __syncthreads();
        for (int off = 1; off < 1024; off <<= 1) {
            const int add = tid >= off ? base[tid - off] : 0;
            __syncthreads();
            base[tid] += add;
            __syncthreads();
        }
        const int incl = base[tid];
        __syncthreads();
        base[tid] = incl - cnt[tid];
        __syncthreads();
    }
    for (int i = tid; i < n_items; i += 1024) order[atomicAdd(&base[bucket(len[i])], 1)] = i;
}

cudaError_t launch_order(const int32_t* len, int n_items, int cap_tokens, int32_t* order, cudaStream_t stream) {
    order_kernel<<<1, 1024, 0, stream>>>(len, n_items, cap_tokens, order);
    return cudaGetLastError();
}

}  // namespace lethe

// ------------------------------------------------------------------ retention with no allocation at all
// Scratch of lethe_rasr_prune_static: a status word (first 256 bytes) followed by the survivors' source-slot
// lists of every item.  It lives in the library image, so each GPU that loads the library holds these
// 16 MiB + 256 B until the process exits; every call reuses it and finds the previous call's contents.
static __device__ __align__(256) int32_t g_static_prune_scratch[64 + LETHE_STATIC_PRUNE_MAX_ENTRIES];

#include <mutex>

namespace {
// Device address of the scratch on the current device.  In host code the array's name is only a handle, not a
// device address, so the address is asked for once per device (with that device current) and remembered.
cudaError_t static_prune_scratch(int32_t** out) {
    constexpr int kMaxDevices = 64;
    static std::mutex mu;
    static int32_t* addr[kMaxDevices] = {};
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(mu);
    if (!addr[dev]) {
        void* p = nullptr;
        e = cudaGetSymbolAddress(&p, g_static_prune_scratch);
        if (e != cudaSuccess) return e;
        addr[dev] = static_cast<int32_t*>(p);
    }
    *out = addr[dev];
    return cudaSuccess;
}
}  // namespace

extern "C" lethe_status lethe_rasr_prune_static(const lethe_cache* c, const int32_t* budgets, int32_t recent,
                                                int32_t sink, int32_t* keep_idx, int32_t max_k, int32_t* status_out,
                                                void* stream) {
    using namespace lethe;
    if (!c || !budgets || !c->k || !c->v || !c->rel || !c->pos || !c->len) return LETHE_ERR_INVALID_ARG;
    if (c->n_layers < 1 || c->batch < 1 || c->n_kv_heads < 1 || c->capacity < 1) return LETHE_ERR_INVALID_ARG;
    if (c->head_dim != 64 && c->head_dim != 128) return LETHE_ERR_UNSUPPORTED;
    if (c->dtype != LETHE_F32 && c->dtype != LETHE_BF16 && c->dtype != LETHE_FP8_E4M3 && c->dtype != LETHE_FP8_E5M2)
        return LETHE_ERR_INVALID_ARG;
    if (c->layout != LETHE_CONTIG && c->layout != LETHE_PAGED) return LETHE_ERR_INVALID_ARG;
    if (c->layout == LETHE_PAGED && (!c->page_table || c->page_tokens < 1 || c->n_pages < 1)) return LETHE_ERR_INVALID_ARG;
    if (recent < 0 || sink < 0 || (keep_idx && max_k < 1)) return LETHE_ERR_INVALID_ARG;
    if ((((uintptr_t)c->k) | ((uintptr_t)c->v)) & 15) return LETHE_ERR_INVALID_ARG;

    CacheView v;
    v.k = c->k; v.v = c->v; v.rel = c->rel; v.pos = c->pos; v.len = c->len; v.page_table = c->page_table;
    v.n_pages = c->n_pages;
    v.L = c->n_layers; v.B = c->batch; v.Hkv = c->n_kv_heads; v.D = c->head_dim;
    v.elt_bytes = c->dtype == LETHE_BF16 ? 2 : (c->dtype == LETHE_F32 ? 4 : 1);
    v.capacity = c->capacity;
    v.page_tokens = c->layout == LETHE_PAGED ? c->page_tokens : 1;
    v.paged = c->layout == LETHE_PAGED;
    const long long cap_tokens = (long long)c->capacity * v.page_tokens;
    const long long items = (long long)v.L * v.B * v.Hkv;
    if (cap_tokens > 0x7fffffffLL || items > 0x7fffffffLL) return LETHE_ERR_TOO_LARGE;
    v.cap_tokens = (int)cap_tokens;
    // one list entry per (item, slot): refuse what the fixed scratch cannot hold
    if (items * cap_tokens > (long long)LETHE_STATIC_PRUNE_MAX_ENTRIES) return LETHE_ERR_TOO_LARGE;

    int32_t* scratch = nullptr;
    if (static_prune_scratch(&scratch) != cudaSuccess) return LETHE_ERR_CUDA;
    int32_t* status = scratch;        // {code, item}: must start at zero for this call
    int32_t* lists = scratch + 64;    // fully written before it is read: no clearing needed
    cudaStream_t s = (cudaStream_t)stream;
    if (cudaMemsetAsync(status, 0, 2 * sizeof(int32_t), s) != cudaSuccess) return LETHE_ERR_CUDA;
    // smem_tokens = 0: every item keeps its source list in the global scratch and re-reads its keys from rel
    rasr_prune_kernel<false><<<(unsigned)items, kPruneThreads, 0, s>>>(v, budgets, recent, sink, keep_idx, keep_idx ? max_k : 0,
                                                               0, lists, status);
    if (cudaGetLastError() != cudaSuccess) return LETHE_ERR_CUDA;
    if (status_out &&
        cudaMemcpyAsync(status_out, status, 2 * sizeof(int32_t), cudaMemcpyDeviceToDevice, s) != cudaSuccess)
        return LETHE_ERR_CUDA;
    return LETHE_OK;
}
