// Persistent tensor-core decode-attend kernel with an asynchronous epilogue (bf16, D in {64, 128}, G <= 8).
//
// Same per-group arithmetic and the same work queue as attend_stream.cu, but the CTA is warp-specialised:
//   * NWS streaming warps never stop at a CTA-wide barrier.  When a warp has consumed its groups of item i it
//     parks its partial (max, sum, O) in the item's parity buffer, signals an mbarrier and goes straight on to
//     item i+1, whose first groups its pipeline has already prefetched;
//   * 2 or 4 epilogue warps (epilogue_warps()) wait for that mbarrier, merge the partials, write out / lse, apply Eq. 5 to rel with the
//     exact normaliser, store len, draw the ticket of the item after next (and read its len), copy that item's
//     query rows and appended k / v row from the call's inputs into a staging area in shared memory, and hand
//     the parity buffer back through a second mbarrier.  The streaming warps take their query fragments and the
//     appended row from the staging area, so each input byte is read once per launch (the inputs may therefore
//     sit in page-locked host memory and be read over the bus, an item ahead of their use).
// The logit buffer, the partial-output buffer and the item descriptor are double-buffered by item parity, so the
// epilogue of item i runs entirely under the HBM stream of item i+1.  Every mbarrier wait is bounded: if it
// runs out, the CTA records LETHE_ERR_TIMEOUT, drains its copies and returns.
#include "common.cuh"
#include "mma_utils.cuh"

#include <string.h>

#include <cuda.h>  // CUtensorMap (type only: the encoder is resolved at run time by the host code)

namespace lethe {

// Epilogue warps per CTA.  Measured on the Llama-8B shape, of the copy peak: (8,2) with 2 / 3 / 4 epilogue warps
// 0.98 / 1.015 / 1.03, (5,3) with 2 / 4: 1.01 / 0.79, (7,2) with 4 / 6: 1.005 / 0.83.
__host__ __device__ constexpr int epilogue_warps(int nws) { return nws >= 8 ? 4 : 2; }
constexpr int kWaitLimit = 200000;  // default poll limit of a bounded wait (AttendArgs::wait_limit overrides it when > 0)

// Tensor maps of K and V for the TMA variant (rows x D, box 16 rows x 64 elements, 128-byte swizzle).
struct alignas(64) TmaMaps {
    CUtensorMap k, v;
};

struct AsyncHeader {
    unsigned long long tma_full[16][6];  // TMA variant: per warp, per stage slot: the tile has landed
    unsigned long long full[2];   // streaming warps -> epilogue: item's partials are complete
    unsigned long long empty[2];  // epilogue -> streaming warps: parity buffers are free, next descriptor is published
    int desc_ticket[4];           // ring by item sequence number: ticket (>= n_items: no more work)
    int desc_n_old[4];            //                              len of that item before this call
    int abort;
    int new_pos[2];               // by item parity: position of the appended token
    int pad;
    float2 wstat[2][16][kMaxGroup];
    // The call's inputs of an item, staged once per item by an epilogue warp (by item parity): the G query rows and
    // the appended k / v row.  Every byte of q, k_new, v_new is therefore read once per launch, which is what lets
    // these buffers sit in page-locked host memory.
    uint4 q_stage[2][kMaxGroup * 128 * 2 / 16];
    uint4 new_stage[2][2][16];
};

__device__ __forceinline__ void mbar_init(unsigned long long* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive(unsigned long long* bar) {
    asm volatile("{ .reg .b64 st; mbarrier.arrive.shared::cta.b64 st, [%0]; }" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(unsigned long long* bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// The same test without any waiting inside the instruction.
__device__ __forceinline__ bool mbar_test_wait(unsigned long long* bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void mbar_arrive_expect_tx(unsigned long long* bar, unsigned bytes) {
    asm volatile("{ .reg .b64 st; mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1; }" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
// One box (64 elements x 16 rows) of a 2-D tensor map into shared memory; completion is counted on `bar`.
// x is always 0 or 64 elements (a multiple of 16 bytes), y is a row index.
__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, int x, int y, unsigned long long* bar,
                                            uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }

// Bounded wait for a tile: polls without backing off for a long while (the data is usually microseconds away).
__device__ __forceinline__ bool mbar_wait_tile(unsigned long long* bar, unsigned parity, volatile int* abort_flag, int limit) {
    if (mbar_test_wait(bar, parity)) return true;  // poll 0 does not block, so a limit of one poll is exactly one look
    for (long long it = 1; it < (long long)limit * 8; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((it & 1023) == 1023) {
            if (*abort_flag) return false;
            __nanosleep(200);
        }
    }
    *abort_flag = 1;
    return false;
}

// Bounded wait; false = gave up (or another warp already did).
__device__ __forceinline__ bool mbar_wait(unsigned long long* bar, unsigned parity, volatile int* abort_flag, int limit) {
    if (mbar_test_wait(bar, parity)) return true;
    for (int it = 1; it < limit; ++it) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (it > 16) __nanosleep(100);
    }
    *abort_flag = 1;
    return false;
}

struct AsyncItem {
    int valid;
    int item, li, l, b, hkv;
    int n_old, n, full;
    int count, app_idx, par;  // streaming warps only (par: parity of the item's sequence number in this CTA)
};

// Registers that carry one item's inputs from global (or mapped host) memory to the staging area: loaded early,
// stored once the staging slot is free.
template <int D>
struct StagedInputs {
    uint4 q[D / 32];  // 16-byte chunks lane, lane + 32, ... of the item's G query rows
    uint4 row;        // lanes 0..15: chunk of the appended k row; lanes 16..31: of the v row
    int pos;
};

__device__ __forceinline__ void async_decode(const AttendArgs& a, int ticket, int n_old, AsyncItem& it) {
    it.valid = ticket < a.n_items;
    const int t = it.valid ? ticket : 0;
    it.hkv = t % a.Hkv;
    it.b = (t / a.Hkv) % a.B;
    it.li = t / (a.Hkv * a.B);
    it.l = a.layer_begin + it.li;
    it.item = (it.l * a.B + it.b) * a.Hkv + it.hkv;
    const bool append = a.k_new != nullptr;
    it.n_old = n_old;
    it.full = append && n_old >= a.cap_tokens;
    it.n = it.full ? 0 : n_old + (append ? 1 : 0);
    it.count = 0;
    it.app_idx = -1;
}

template <int D>
__device__ __forceinline__ void load_inputs(const AttendArgs& a, const AsyncItem& it, int lane, StagedInputs<D>& r) {
    using T = __nv_bfloat16;
    constexpr int ROW_CHUNKS = D * 2 / 16;
    const int q_chunks = a.G * D * 2 / 16;
    const uint4* qsrc = reinterpret_cast<const uint4*>((const T*)a.q + ((size_t)(it.li * a.B + it.b) * a.Hq + it.hkv * a.G) * D);
#pragma unroll
    for (int i = 0; i < D / 32; ++i) {
        const int c = i * 32 + lane;
        r.q[i] = (it.valid && c < q_chunks) ? qsrc[c] : make_uint4(0u, 0u, 0u, 0u);
    }
    r.row = make_uint4(0u, 0u, 0u, 0u);
    r.pos = 0;
    if (a.k_new && it.valid) {
        const size_t src = ((size_t)(it.li * a.B + it.b) * a.Hkv + it.hkv) * ROW_CHUNKS;
        const int c = lane & 15;
        if (c < ROW_CHUNKS) r.row = reinterpret_cast<const uint4*>(lane < 16 ? a.k_new : a.v_new)[src + c];
        if (lane == 0) r.pos = a.token_pos[it.b];
    }
}
template <int D>
__device__ __forceinline__ void store_inputs(AsyncHeader& hd, int par, int lane, const StagedInputs<D>& r) {
#pragma unroll
    for (int i = 0; i < D / 32; ++i) hd.q_stage[par][i * 32 + lane] = r.q[i];
    hd.new_stage[par][lane >> 4][lane & 15] = r.row;
    if (lane == 0) hd.new_pos[par] = r.pos;
}

// Sec. 4.1: the generated token's k / v row enters the cache, from the staging area (kept out of line: once per item).
template <bool PAGED>
__device__ __noinline__ void append_row(const AttendArgs& a, int item, int n_old, int row_bytes, const uint4* staged_k,
                                        const uint4* staged_v, int token_pos, int lane) {
    bool bad = false;
    char* kd = const_cast<char*>(row_ptr<PAGED>(a, a.k, item, n_old, row_bytes, &bad));
    char* vd = const_cast<char*>(row_ptr<PAGED>(a, a.v, item, n_old, row_bytes, &bad));
    if (kd && vd && lane * 16 < row_bytes) {
        *reinterpret_cast<uint4*>(kd + lane * 16) = staged_k[lane];
        *reinterpret_cast<uint4*>(vd + lane * 16) = staged_v[lane];
    }
    if (lane == 0) a.pos[(size_t)item * a.cap_tokens + n_old] = token_pos;
    __syncwarp();
}

// GT: query heads per KV head when known at compile time (0 = from the arguments): strides and head loops of the
// streaming and epilogue warps become constants (worth 2 % on the Llama-8B shape).
template <int D, int NWS, int NS, bool PAGED, bool SPILL, bool TMA, int GT = 0>
__global__ void __launch_bounds__((NWS + epilogue_warps(NWS)) * 32, 1)
    attend_async_kernel(const __grid_constant__ AttendArgs a, const __grid_constant__ TmaMaps maps) {
    using T = __nv_bfloat16;
    constexpr int ROW_BYTES = D * 2;
    constexpr int CHUNKS = ROW_BYTES / 16;
    constexpr int TILE_BYTES = kGroupTokens * ROW_BYTES;
    constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    constexpr int WARP_BYTES = NS * STAGE_BYTES;
    constexpr int KS = D / 16;
    constexpr int kEpilogueWarps = epilogue_warps(NWS);
    constexpr int ET = kEpilogueWarps * 32;
    static_assert(NS >= 2 && NS <= 6 && NWS <= 16, "shape");
    extern __shared__ __align__(1024) unsigned char smem_raw[];  // TMA tiles with a 128-byte swizzle need 1 KB alignment
    // layout: stages [NWS][NS][K tile | V tile] | AsyncHeader | wo [2][NWS][GP][D] fp32 | lg [2][chunk][GP] fp32
    // Tile layout.  cp.async: rows of ROW_BYTES with the 16-byte chunk index XORed by (row & 7).  TMA: one 2 KB box
    // per 64 elements of D (16 rows x 128 B, chunk index XORed by (row & 7) by the hardware swizzle).
    const int G = GT ? GT : a.G, GP = GT ? ((GT + 1) & ~1) : a.GP;
    const int wo_stride = GP * D;  // floats per warp
    AsyncHeader& hd = *reinterpret_cast<AsyncHeader*>(smem_raw + (size_t)NWS * WARP_BYTES);
    float* wo_all = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(&hd) + sizeof(AsyncHeader));
    float* lg_all = wo_all + (size_t)2 * NWS * wo_stride;
    const int chunk = a.chunk_tokens;
    float* spill_all = SPILL ? a.spill + (size_t)blockIdx.x * 2 * a.spill_tokens * GP : nullptr;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const bool append = a.k_new != nullptr;
    unsigned int* sched = a.sched;
    volatile int* abort_flag = &hd.abort;
    const int wait_limit = a.wait_limit > 0 ? a.wait_limit : kWaitLimit;

    // ---- set-up: barriers, first two descriptors
    bool drew_fail = false;  // meaningful in the ticket-drawing lane only
    if (tid == 0) {
        mbar_init(&hd.full[0], NWS);
        mbar_init(&hd.full[1], NWS);
        mbar_init(&hd.empty[0], kEpilogueWarps);
        mbar_init(&hd.empty[1], kEpilogueWarps);
        if (TMA)
            for (int w = 0; w < NWS; ++w)
                for (int sl = 0; sl < NS; ++sl) mbar_init(&hd.tma_full[w][sl], 1);
        hd.abort = 0;
    }
    if (TMA && (smem_u32(smem_raw) & 1023u)) {  // would break the hardware swizzle: refuse rather than compute garbage
        if (tid == 0) record_error(a.status, LETHE_ERR_UNSUPPORTED, (int)blockIdx.x);
        // still take part in the queue protocol so that the launch ends cleanly
        if (tid == 0) {
            (void)atomicAdd(&sched[0], 1u);
            __threadfence();
            const unsigned int done = atomicAdd(&sched[1], 1u);
            if (done == gridDim.x - 1) {
                sched[0] = 0u;
                sched[1] = 0u;
            }
        }
        return;
    }
    if (warp == NWS) {  // the first two tickets, and what their items need from the call's inputs
        int t0 = a.n_items, t1 = a.n_items;
        if (lane == 0) {
            t0 = (int)atomicAdd(&sched[0], 1u);
            if (t0 >= a.n_items) drew_fail = true;
            else {
                t1 = (int)atomicAdd(&sched[0], 1u);
                if (t1 >= a.n_items) drew_fail = true;
            }
            if (a.order) {  // longest-first order of the items (valid tickets only)
                if (t0 < a.n_items) t0 = a.order[t0];
                if (t1 < a.n_items) t1 = a.order[t1];
            }
        }
        t0 = __shfl_sync(0xffffffffu, t0, 0);
        t1 = __shfl_sync(0xffffffffu, t1, 0);
        AsyncItem i0, i1;
        async_decode(a, t0, 0, i0);
        async_decode(a, t1, 0, i1);
        StagedInputs<D> r0, r1;
        load_inputs<D>(a, i0, lane, r0);
        load_inputs<D>(a, i1, lane, r1);
        if (lane == 0) {
            hd.desc_ticket[0] = t0;
            hd.desc_n_old[0] = i0.valid ? a.len[i0.item] : 0;
            hd.desc_ticket[1] = t1;
            hd.desc_n_old[1] = i1.valid ? a.len[i1.item] : 0;
        }
        store_inputs<D>(hd, 0, lane, r0);
        store_inputs<D>(hd, 1, lane, r1);
    }
    __syncthreads();

    if (warp < NWS) {
        // =================================================================== streaming warps
        const int gq = lane >> 2, tq = lane & 3;
        auto load_q = [&](const AsyncItem& it, uint32_t (&bq)[KS][2]) {
            const uint32_t* qrow = reinterpret_cast<const uint32_t*>(hd.q_stage[it.par]) + gq * (D / 2);
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                bq[ks][0] = (it.valid && gq < G) ? qrow[8 * ks + tq] : 0u;
                bq[ks][1] = (it.valid && gq < G) ? qrow[8 * ks + 4 + tq] : 0u;
            }
        };
        auto set_counts = [&](AsyncItem& it) {
            const int ng = (it.n + kGroupTokens - 1) / kGroupTokens;
            it.count = ng > warp ? (ng - warp + NWS - 1) / NWS : 0;
            it.app_idx = -1;
            if (append && !it.full && it.valid) {
                const int g = it.n_old / kGroupTokens;
                if (g % NWS == warp) it.app_idx = g / NWS;
            }
        };
        unsigned char* my_stage = smem_raw + (size_t)warp * WARP_BYTES;
        const uint32_t my_stage_u32 = smem_u32(my_stage);
        bool bad_page = false;
        const uint64_t stream_policy = l2_evict_first_policy();  // K / V tiles are read once: evict-first in L2
        unsigned slot_bad = 0;    // TMA: slots whose tile must be ignored (page id outside the pool)
        unsigned slot_phase = 0;  // TMA: parity of the next completion of each slot's mbarrier
        unsigned slot_busy = 0;   // TMA: slots with a load in flight or landed but not yet consumed

        // PAGED: page ids of this warp's local groups are fetched 32 at a time, one lane each, a block ahead of
        // their use, so that staging a group never waits on a page-table load.
        int pg_lo = 0, pg_hi = 0, pg_nxt = 0;  // current item: blocks pg_blk and pg_blk + 1; next item: block 0
        int pg_blk = 0;
        auto load_pages = [&](const AsyncItem& it, int blk) -> int {
            const int g = blk * 32 + lane;
            return (PAGED && it.valid && g < it.count) ? a.page_table[(size_t)it.item * a.capacity + warp + g * NWS] : 0;
        };
        auto issue = [&](const AsyncItem& it, int idx, int slot, bool is_cur) {
            const int grp = warp + idx * NWS;
            const int tok0 = grp * kGroupTokens;
            if (idx == it.app_idx) {
                append_row<PAGED>(a, it.item, it.n_old, ROW_BYTES, hd.new_stage[it.par][0], hd.new_stage[it.par][1],
                                  hd.new_pos[it.par], lane);
                if (TMA) {  // the row was written through the generic proxy; the TMA load reads through the async proxy
                    fence_proxy_async();
                    __syncwarp();
                }
            }
            const char* kb;
            const char* vb;
            bool ok = true;
            if (PAGED) {
                int page;
                if (!is_cur) page = __shfl_sync(0xffffffffu, pg_nxt, idx & 31);  // only the first NS-1 groups
                else {
                    if ((idx >> 5) > pg_blk) {  // first group of the next block: rotate and fetch one more ahead
                        pg_lo = pg_hi;
                        ++pg_blk;
                        pg_hi = load_pages(it, pg_blk + 1);
                    }
                    page = __shfl_sync(0xffffffffu, pg_lo, idx & 31);
                }
                ok = page >= 0 && page < a.n_pages;
                if (!ok) bad_page = true;
                const size_t off = (size_t)(ok ? page : 0) * TILE_BYTES;
                kb = (const char*)a.k + off;
                vb = (const char*)a.v + off;
            } else {
                const size_t off = ((size_t)it.item * a.capacity + tok0) * ROW_BYTES;
                kb = (const char*)a.k + off;
                vb = (const char*)a.v + off;
            }
            const uint32_t ks_u32 = my_stage_u32 + slot * STAGE_BYTES;
            const uint32_t vs_u32 = ks_u32 + TILE_BYTES;
            if constexpr (TMA) {
                // row index of the group's first token in the 2-D view of the cache (rows x D)
                const long long row0 = (long long)((kb - (const char*)a.k) / ROW_BYTES);
                if (!ok) slot_bad |= 1u << slot;
                else slot_bad &= ~(1u << slot);
                slot_busy |= 1u << slot;
                if (lane == 0) {
                    unsigned long long* bar = &hd.tma_full[warp][slot];
                    mbar_arrive_expect_tx(bar, STAGE_BYTES);
#pragma unroll
                    for (int hx = 0; hx < D / 64; ++hx) {
                        tma_load_2d(ks_u32 + hx * 2048, &maps.k, hx * 64, (int)row0, bar, stream_policy);
                        tma_load_2d(vs_u32 + hx * 2048, &maps.v, hx * 64, (int)row0, bar, stream_policy);
                    }
                }
                return;
            }
#pragma unroll
            for (int i = 0; i < kGroupTokens * CHUNKS / 32; ++i) {
                const int c_idx = i * 32 + lane;
                const int r = c_idx / CHUNKS, c = c_idx % CHUNKS;
                const bool valid = ok && (tok0 + r < it.n);
                const int soff = valid ? r * ROW_BYTES + c * 16 : 0;
                const uint32_t doff = r * ROW_BYTES + ((c ^ (r & 7)) << 4);
                cp_async16_hint(ks_u32 + doff, kb + soff, valid ? 16 : 0, stream_policy);
                cp_async16_hint(vs_u32 + doff, vb + soff, valid ? 16 : 0, stream_policy);
            }
        };

        const int k_row = (lane & 7) + ((lane >> 3) & 1) * 8, k_chunk = lane >> 4;
        const int v_row = (lane & 7) + ((lane >> 4) & 1) * 8, v_chunk = (lane >> 3) & 1;

        AsyncItem cur, nxt;
        async_decode(a, hd.desc_ticket[0], hd.desc_n_old[0], cur);
        cur.par = 0;
        set_counts(cur);
        uint32_t bq[KS][2], bqn[KS][2];
        load_q(cur, bq);
        pg_lo = load_pages(cur, 0);
        pg_hi = load_pages(cur, 1);
        nxt.valid = 0;
        int seq = 0;          // sequence number of the current item within this CTA
        int vp = 0;           // stage slot of the current item's local group 0
        unsigned issued = 0;  // bit j: local group j (< NS-1) of the current item was prefetched by the previous tail
        bool alive = true;

        while (cur.valid && alive) {
            const int p = seq & 1;
            const float sl2 = a.scale_log2[cur.l];
            const uint32_t lg_u32 = smem_u32(lg_all + (size_t)p * chunk * GP);
            float* spill = SPILL ? spill_all + (size_t)p * a.spill_tokens * GP : nullptr;
            bool nxt_ready = false;
            // descriptor of the next item: wait until the epilogue of item seq-1 (same parity as seq+1) has
            // handed its buffers back, which also publishes that descriptor
            auto acquire_next = [&]() {
                const int sn = seq + 1;
                if (sn >= 2 && !mbar_wait(&hd.empty[sn & 1], (unsigned)(((sn >> 1) - 1) & 1), abort_flag, wait_limit)) {
                    alive = false;
                    nxt.valid = 0;
                } else {
                    async_decode(a, hd.desc_ticket[sn & 3], hd.desc_n_old[sn & 3], nxt);
                    nxt.par = sn & 1;
                    set_counts(nxt);
                    load_q(nxt, bqn);
                    pg_nxt = load_pages(nxt, 0);
                }
                nxt_ready = true;
            };

            bool topped = false;
#pragma unroll
            for (int j = 0; j < NS - 1; ++j) {
                if (!((issued >> j) & 1u) && j < cur.count) {
                    issue(cur, j, (vp + j) % NS, true);
                    topped = true;
                }
            }
            if (topped) cp_async_commit();
            unsigned issued_next = 0;

            float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
            float o[KS][4];
#pragma unroll
            for (int mt = 0; mt < KS; ++mt)
#pragma unroll
                for (int i = 0; i < 4; ++i) o[mt][i] = 0.f;

            constexpr bool OVF = SPILL;
            for (int it = 0; it < cur.count; ++it) {
                const int cslot = (vp + it) % NS;
                // Refill first, wait second: the slot of group it-1 is free as soon as every lane has left the
                // previous iteration, so the copy of the group NS-1 ahead (possibly of the next item) is already
                // in flight while this warp waits for group `it`.
                __syncwarp();
                const bool strict = !TMA && topped && it < NS - 1;  // after a top-up the group order is not the commit order
                if (strict) cp_async_wait<0>();
                {
                    const int idx = it + NS - 1;
                    const int slot = (vp + idx) % NS;
                    if (idx < cur.count) issue(cur, idx, slot, true);
                    else {
                        if (!nxt_ready) acquire_next();
                        const int j = idx - cur.count;
                        if (nxt.valid && j < nxt.count) {
                            issue(nxt, j, slot, false);
                            issued_next |= 1u << j;
                        }
                    }
                    cp_async_commit();
                }
                if constexpr (TMA) {
                    if (!mbar_wait_tile(&hd.tma_full[warp][cslot], (slot_phase >> cslot) & 1u, abort_flag, wait_limit)) {
                        alive = false;
                        break;
                    }
                    slot_phase ^= 1u << cslot;
                    slot_busy &= ~(1u << cslot);
                    // rows past the item's end (and tiles of a bad page) hold whatever memory held: V rows must be
                    // zero so that a zero probability times them stays zero; K rows are masked by the logit test
                    const int grp_w = warp + it * NWS;
                    int valid_rows = cur.n - grp_w * kGroupTokens;
                    if ((slot_bad >> cslot) & 1u) valid_rows = 0;
                    if (valid_rows < kGroupTokens) {
                        const uint32_t vt = my_stage_u32 + cslot * STAGE_BYTES + TILE_BYTES;
                        for (int e = lane; e < (kGroupTokens - valid_rows) * CHUNKS; e += 32) {
                            const int r = valid_rows + e / CHUNKS, cch = e % CHUNKS;
                            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(vt + (cch >> 3) * 2048 + r * 128 + ((cch & 7) << 4)), "r"(0) : "memory");
                        }
                    }
                } else {
                    if (!strict) cp_async_wait<NS - 1>();  // everything but the NS-1 newest groups, i.e. group `it`, has landed
                }
                __syncwarp();
                const int grp = warp + it * NWS;
                const uint32_t ks_u32 = my_stage_u32 + ((vp + it) % NS) * STAGE_BYTES;
                const uint32_t vs_u32 = ks_u32 + TILE_BYTES;

                float ca[4] = {0.f, 0.f, 0.f, 0.f}, cb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    uint32_t af[4];
                    const int kc = 2 * ks + k_chunk;
                    if constexpr (TMA) ldmatrix_x4(ks_u32 + (kc >> 3) * 2048 + k_row * 128 + (((kc & 7) ^ (k_row & 7)) << 4), af);
                    else ldmatrix_x4(ks_u32 + k_row * ROW_BYTES + ((kc ^ (k_row & 7)) << 4), af);
                    if (ks & 1) mma_bf16(cb, af, bq[ks][0], bq[ks][1]);
                    else mma_bf16(ca, af, bq[ks][0], bq[ks][1]);
                }
                const int tokA = grp * kGroupTokens + gq, tokB = tokA + 8;
                const float s00 = (tokA < cur.n) ? (ca[0] + cb[0]) * sl2 : -INFINITY;
                const float s01 = (tokA < cur.n) ? (ca[1] + cb[1]) * sl2 : -INFINITY;
                const float s10 = (tokB < cur.n) ? (ca[2] + cb[2]) * sl2 : -INFINITY;
                const float s11 = (tokB < cur.n) ? (ca[3] + cb[3]) * sl2 : -INFINITY;
                if (2 * tq < GP) {
                    if (!OVF || tokA < chunk) st_shared_f2(lg_u32 + (tokA * GP + 2 * tq) * 4, s00, s01);
                    else *reinterpret_cast<float2*>(spill + (size_t)(tokA - chunk) * GP + 2 * tq) = make_float2(s00, s01);
                    if (!OVF || tokB < chunk) st_shared_f2(lg_u32 + (tokB * GP + 2 * tq) * 4, s10, s11);
                    else *reinterpret_cast<float2*>(spill + (size_t)(tokB - chunk) * GP + 2 * tq) = make_float2(s10, s11);
                }
                float mx0 = fmaxf(s00, s10), mx1 = fmaxf(s01, s11);
#pragma unroll
                for (int off = 4; off < 32; off <<= 1) {
                    mx0 = fmaxf(mx0, __shfl_xor_sync(0xffffffffu, mx0, off));
                    mx1 = fmaxf(mx1, __shfl_xor_sync(0xffffffffu, mx1, off));
                }
                const float mn0 = fmaxf(m0, mx0), mn1 = fmaxf(m1, mx1);
                if (__any_sync(0xffffffffu, (mn0 > m0) || (mn1 > m1))) {
                    const float c0 = exp2_diff(m0, mn0), c1 = exp2_diff(m1, mn1);
                    l0 *= c0;
                    l1 *= c1;
#pragma unroll
                    for (int mt = 0; mt < KS; ++mt) {
                        o[mt][0] *= c0; o[mt][2] *= c0;
                        o[mt][1] *= c1; o[mt][3] *= c1;
                    }
                    m0 = mn0;
                    m1 = mn1;
                }
                const float p00 = fast_exp2(s00 - m0), p01 = fast_exp2(s01 - m1);
                const float p10 = fast_exp2(s10 - m0), p11 = fast_exp2(s11 - m1);
                l0 += p00 + p10;
                l1 += p01 + p11;
                const uint32_t pb0 = movmatrix_trans(pack_bf16(p00, p01));
                const uint32_t pb1 = movmatrix_trans(pack_bf16(p10, p11));
#pragma unroll
                for (int mt = 0; mt < KS; ++mt) {
                    uint32_t af[4];
                    const int vc = 2 * mt + v_chunk;
                    if constexpr (TMA) ldmatrix_x4_trans(vs_u32 + (vc >> 3) * 2048 + v_row * 128 + (((vc & 7) ^ (v_row & 7)) << 4), af);
                    else ldmatrix_x4_trans(vs_u32 + v_row * ROW_BYTES + ((vc ^ (v_row & 7)) << 4), af);
                    mma_bf16(o[mt], af, pb0, pb1);
                }
            }
            vp = (vp + cur.count) % NS;

            // ---- park this warp's partials in the parity buffer and signal the epilogue warps
#pragma unroll
            for (int off = 4; off < 32; off <<= 1) {
                l0 += __shfl_xor_sync(0xffffffffu, l0, off);
                l1 += __shfl_xor_sync(0xffffffffu, l1, off);
            }
            if (gq == 0) {
                hd.wstat[p][warp][2 * tq] = make_float2(m0, l0);
                hd.wstat[p][warp][2 * tq + 1] = make_float2(m1, l1);
            }
            if (2 * tq < GP) {
                float* wo = wo_all + ((size_t)p * NWS + warp) * wo_stride;
#pragma unroll
                for (int mt = 0; mt < KS; ++mt) {
                    wo[(2 * tq) * D + 16 * mt + gq] = o[mt][0];
                    wo[(2 * tq + 1) * D + 16 * mt + gq] = o[mt][1];
                    wo[(2 * tq) * D + 16 * mt + gq + 8] = o[mt][2];
                    wo[(2 * tq + 1) * D + 16 * mt + gq + 8] = o[mt][3];
                }
            }
            // (overflowed logits written to global memory are released to the epilogue warps by the mbarrier
            // arrive below, which has release semantics at CTA scope, like the shared-memory writes)
            __syncwarp();
            if (lane == 0) mbar_arrive(&hd.full[p]);

            // ---- rotate
            if (!nxt_ready) acquire_next();
            cur = nxt;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                bq[ks][0] = bqn[ks][0];
                bq[ks][1] = bqn[ks][1];
            }
            pg_lo = pg_nxt;
            pg_blk = 0;
            pg_hi = load_pages(cur, 1);
            issued = issued_next;
            ++seq;
        }
        cp_async_wait<0>();
        if (TMA) {  // only after a timeout can loads still be in flight: wait for them (bounded) before leaving
            for (int sl = 0; sl < NS; ++sl)
                if ((slot_busy >> sl) & 1u) {
                    for (int spin = 0; spin < kWaitLimit; ++spin)
                        if (mbar_try_wait(&hd.tma_full[warp][sl], (slot_phase >> sl) & 1u)) break;
                }
        }
        if (bad_page && lane == 0) record_error(a.status, LETHE_ERR_PAGE, 0);
    } else {
        // =================================================================== epilogue warps
        const int ew = warp - NWS;
        const int et = ew * 32 + lane;
        bool alive = true;
        for (int seq = 0; alive; ++seq) {
            const int p = seq & 1;
            // the descriptor of item seq was published by epilogue warp 0 while finishing item seq-2; waiting
            // for that hand-back (both epilogue warps arrive on it) makes the write visible to this warp too
            if (seq >= 2 && !mbar_wait(&hd.empty[p], (unsigned)(((seq >> 1) - 1) & 1), abort_flag, wait_limit)) {
                alive = false;
                break;
            }
            AsyncItem it;
            async_decode(a, hd.desc_ticket[seq & 3], hd.desc_n_old[seq & 3], it);
            if (!it.valid) break;
            if (!mbar_wait(&hd.full[p], (unsigned)((seq >> 1) & 1), abort_flag, wait_limit)) {
                alive = false;
                break;
            }
            // ticket of the item after next: its round trips hide behind the merge below
            int t_new = a.n_items;
            if (ew == 0 && lane == 0 && !drew_fail) t_new = (int)atomicAdd(&sched[0], 1u);

            const uint32_t lg_u32 = smem_u32(lg_all + (size_t)p * chunk * GP);
            const float* spill = SPILL ? spill_all + (size_t)p * a.spill_tokens * GP : nullptr;
            float* relp = a.rel + (size_t)it.item * a.cap_tokens;
            const int app = (append && !it.full) ? it.n_old : -1;

            // merged statistics of every head (each thread computes them all: off the critical path)
            float fm[kMaxGroup], fi[kMaxGroup];
#pragma unroll
            for (int h = 0; h < kMaxGroup; ++h) {
                fm[h] = -INFINITY;
                fi[h] = 0.f;
                if (h < G) {
                    float m = -INFINITY;
#pragma unroll
                    for (int w = 0; w < NWS; ++w) m = fmaxf(m, hd.wstat[p][w][h].x);
                    float l = 0.f;
#pragma unroll
                    for (int w = 0; w < NWS; ++w) l += hd.wstat[p][w][h].y * exp2_diff(hd.wstat[p][w][h].x, m);
                    fm[h] = m;
                    fi[h] = l > 0.f ? 1.f / l : 0.f;
                    if (a.lse && et == h)
                        a.lse[(size_t)(it.li * a.B + it.b) * a.Hq + it.hkv * G + h] =
                            l > 0.f ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
                }
            }
            // Epilogue warp 0 fetches what the item after next needs from the call's inputs; the loads complete
            // behind the output and relevance work below.
            AsyncItem nx;
            StagedInputs<D> staged;
            int nx_n_old = 0;
            if (ew == 0) {
                if (lane == 0) {
                    if (t_new >= a.n_items) drew_fail = true;
                    else if (a.order) t_new = a.order[t_new];
                }
                t_new = __shfl_sync(0xffffffffu, t_new, 0);
                async_decode(a, t_new, 0, nx);
                load_inputs<D>(a, nx, lane, staged);
                if (lane == 0 && nx.valid) nx_n_old = a.len[nx.item];
            }
            const bool item_overflows = SPILL && it.n > chunk;
            // One token's G logits (from shared memory, or from the overflow area), then its attention mass.
            auto load_row = [&](int j, float2 (&s)[kMaxGroup / 2]) {
                const bool in_smem = !item_overflows || j < chunk;
#pragma unroll
                for (int h = 0; h < kMaxGroup; h += 2)
                    if (h < GP)
                        s[h / 2] = in_smem ? ld_shared_f2(lg_u32 + (j * GP + h) * 4)
                                           : *reinterpret_cast<const float2*>(spill + (size_t)(j - chunk) * GP + h);
            };
            auto mass_from = [&](const float2 (&s)[kMaxGroup / 2]) {
                float mass = 0.f;
#pragma unroll
                for (int h = 0; h < kMaxGroup; h += 2) {
                    if (h < GP) {
                        mass += fast_exp2(s[h / 2].x - fm[h]) * fi[h];
                        if (h + 1 < G) mass += fast_exp2(s[h / 2].y - fm[h + 1]) * fi[h + 1];
                    }
                }
                return mass;
            };
            // Eq. 5 on rel[0..n): old values are fetched a batch ahead of their use
            constexpr int RB = 8;
            float oldv[RB];
            auto fetch = [&](int base) {
#pragma unroll
                for (int i = 0; i < RB; ++i) {
                    const int j = base + et + i * ET;
                    oldv[i] = (j < it.n && j != app) ? relp[j] : 0.f;
                }
            };
            fetch(0);
            {
                T* out = (T*)a.out + ((size_t)(it.li * a.B + it.b) * a.Hq + it.hkv * G) * D;
                for (int idx = et; idx < G * D; idx += ET) {
                    const int h = idx / D;
                    float mh = -INFINITY, ih = 0.f;
#pragma unroll
                    for (int hh = 0; hh < kMaxGroup; ++hh)
                        if (hh == h) {
                            mh = fm[hh];
                            ih = fi[hh];
                        }
                    float acc = 0.f;
#pragma unroll
                    for (int w = 0; w < NWS; ++w)
                        acc += wo_all[((size_t)p * NWS + w) * wo_stride + idx] * exp2_diff(hd.wstat[p][w][h].x, mh);
                    out[idx] = __float2bfloat16_rn(acc * ih);
                }
            }
            for (int base = 0; base < it.n; base += RB * ET) {
                float cur_old[RB];
#pragma unroll
                for (int i = 0; i < RB; ++i) cur_old[i] = oldv[i];
                if (base + RB * ET < it.n) fetch(base + RB * ET);
                // kRelBatch rows are loaded before the first of them is used: the stores to rel would otherwise
                // order the overflow area's loads one token at a time.
#pragma unroll
                for (int i0 = 0; i0 < RB; i0 += kRelBatch) {
                    float2 s[kRelBatch][kMaxGroup / 2];
#pragma unroll
                    for (int u = 0; u < kRelBatch; ++u) {
                        const int j = base + et + (i0 + u) * ET;
                        load_row(j < it.n ? j : it.n - 1, s[u]);
                    }
#pragma unroll
                    for (int u = 0; u < kRelBatch; ++u) {
                        const int j = base + et + (i0 + u) * ET;
                        if (j < it.n) relp[j] = fmaf(a.gamma, cur_old[i0 + u], mass_from(s[u]));
                    }
                }
            }
            if (ew == 0) {
                store_inputs<D>(hd, p, lane, staged);  // item seq + 2 has the parity of this one, whose slot is free
                if (lane == 0) {
                    if (it.full) record_error(a.status, LETHE_ERR_CAPACITY, it.item);
                    else if (append) a.len[it.item] = it.n;
                    hd.desc_n_old[(seq + 2) & 3] = nx_n_old;
                    hd.desc_ticket[(seq + 2) & 3] = t_new;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(&hd.empty[p]);
        }
        if (!alive && lane == 0) record_error(a.status, LETHE_ERR_TIMEOUT, (int)blockIdx.x);
        // ---- the last CTA out re-arms the queue for the next launch
        if (ew == 0 && lane == 0) {
            __threadfence();
            const unsigned int done = atomicAdd(&sched[1], 1u);
            if (done == gridDim.x - 1) {
                sched[0] = 0u;
                sched[1] = 0u;
                __threadfence();
            }
        }
    }
}

template <int D, int NWS, int NS>
static size_t async_smem(int chunk_tokens, int GP) {
    return (size_t)NWS * NS * 2 * kGroupTokens * D * 2 + sizeof(AsyncHeader) + (size_t)2 * NWS * GP * D * 4 +
           (size_t)2 * chunk_tokens * GP * 4;
}

template <int D, int NWS, int NS, bool PAGED, bool SPILL, bool TMA, int GT = 0>
static cudaError_t launch_async_t(const AttendArgs& a, const TmaMaps& maps, int grid, cudaStream_t stream) {
    auto kern = attend_async_kernel<D, NWS, NS, PAGED, SPILL, TMA, GT>;
    const size_t smem = async_smem<D, NWS, NS>(a.chunk_tokens, a.GP);
    cudaError_t e = prepare_kernel((const void*)kern, smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, (NWS + epilogue_warps(NWS)) * 32, smem, stream>>>(a, maps);
    return cudaGetLastError();
}

template <int D, int NWS, int NS, bool TMA, int GT = 0>
static cudaError_t dispatch_async(const AttendArgs& a, const TmaMaps& maps, bool paged, int grid, cudaStream_t stream) {
    const bool spill = a.spill != nullptr;
    if (paged)
        return spill ? launch_async_t<D, NWS, NS, true, true, TMA, GT>(a, maps, grid, stream)
                     : launch_async_t<D, NWS, NS, true, false, TMA, GT>(a, maps, grid, stream);
    return spill ? launch_async_t<D, NWS, NS, false, true, TMA, GT>(a, maps, grid, stream)
                 : launch_async_t<D, NWS, NS, false, false, TMA, GT>(a, maps, grid, stream);
}

// Shapes: (streaming warps per CTA, stages per warp); epilogue_warps() more warps run the epilogue.
#define LETHE_ASYNC_SHAPES(X, D) X(0, D, 8, 2) X(1, D, 7, 2) X(2, D, 6, 3) X(3, D, 5, 3) X(4, D, 6, 2) X(5, D, 4, 4)

size_t async_smem_bytes(int D, int shape, int chunk_tokens, int GP) {
#define X(id, DD, NW, NS) \
    if (shape == id && D == DD) return async_smem<DD, NW, NS>(chunk_tokens, GP);
    LETHE_ASYNC_SHAPES(X, 128)
    LETHE_ASYNC_SHAPES(X, 64)
#undef X
    return (size_t)-1;
}

// tma: stage K / V tiles with cp.async.bulk.tensor through `maps` (a TmaMaps built by the caller) instead of
// 16-byte cp.async; maps may be NULL when tma is false.
cudaError_t launch_attend_async(const AttendArgs& a, int D, int shape, bool paged, int grid, cudaStream_t stream, bool tma,
                                const void* maps) {
    TmaMaps none;
    memset(&none, 0, sizeof(none));
    const TmaMaps& m = (tma && maps) ? *reinterpret_cast<const TmaMaps*>(maps) : none;
    // the default shape on the common geometries (four, five or eight query heads per KV head), group size compiled in
    if (D == 128 && shape == 0 && !tma) {
        if (a.G == 4) return dispatch_async<128, 8, 2, false, 4>(a, m, paged, grid, stream);
        if (a.G == 5) return dispatch_async<128, 8, 2, false, 5>(a, m, paged, grid, stream);
        if (a.G == 8) return dispatch_async<128, 8, 2, false, 8>(a, m, paged, grid, stream);
    }
#define X(id, DD, NW, NS)                                                                            \
    if (shape == id && D == DD)                                                                      \
        return tma ? dispatch_async<DD, NW, NS, true>(a, m, paged, grid, stream) : dispatch_async<DD, NW, NS, false>(a, m, paged, grid, stream);
    LETHE_ASYNC_SHAPES(X, 128)
    LETHE_ASYNC_SHAPES(X, 64)
#undef X
    return cudaErrorInvalidValue;
}

// Host: fill a TmaMaps for K and V seen as 2-D bf16 tensors [rows][D] with a (16 rows x 64 elements) box and the
// 128-byte swizzle.  `encode` is cuTensorMapEncodeTiled, resolved by the caller.  Returns false on failure.
bool build_tma_maps(void* encode, void* k, void* v, unsigned long long rows, int D, void* out_maps) {
    typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    encode_fn fn = reinterpret_cast<encode_fn>(encode);
    TmaMaps* m = reinterpret_cast<TmaMaps*>(out_maps);
    const cuuint64_t dims[2] = {(cuuint64_t)D, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {(cuuint64_t)D * 2};
    const cuuint32_t box[2] = {64, (cuuint32_t)kGroupTokens};
    const cuuint32_t estr[2] = {1, 1};
    for (int which = 0; which < 2; ++which) {
        CUresult r = fn(which ? &m->v : &m->k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, which ? v : k, dims, strides, box, estr,
                        CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                        CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        if (r != CUDA_SUCCESS) return false;
    }
    return true;
}

size_t tma_maps_bytes() { return sizeof(TmaMaps); }

}  // namespace lethe
