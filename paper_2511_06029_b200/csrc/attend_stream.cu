// Persistent tensor-core decode-attend kernel (bf16, D in {64, 128}, G <= 8): one CTA per SM walks a
// dynamic queue of items and never lets the HBM stream drain between them.
//
// Arithmetic and data movement per 16-token group are those of attend_mma.cu (tokens on the M axis of
// mma.m16n8k16, heads on N, per-warp private cp.async pipelines, XOR-swizzled staging, scaled logits parked
// in shared memory for the exact Eq. 5 update).  What differs is the schedule:
//   * work queue: items are handed out through one atomic ticket counter in global scratch, one item ahead
//     of need, so that SMs finish within about one item of each other whatever the length mix;
//   * cross-item prefetch: a warp's pipeline refills run past the end of the current item into the first
//     groups of the next one, so the merge / output / relevance epilogue of item i overlaps the loads of
//     item i+1 instead of exposing a prologue (len -> first tile round trips) and an epilogue per CTA.
// The whole item is handled by one CTA (no cluster), so the kernel is used when there are at least as many
// items as SMs; the clustered kernel covers launches with few, long items.
#include "common.cuh"
#include "mma_utils.cuh"

namespace lethe {

struct StreamItem {
    int valid;       // ticket < n_items
    int item, li, l, b, hkv;
    int n_old, n;    // tokens before / after the append (a full item keeps n = 0: it is skipped)
    int full;        // append requested on a full item
    int count;       // 16-token groups this warp streams: global groups warp, warp + NW, ...
    int app_idx;     // this warp's local group index that holds the appended slot, or -1
};

template <int NW>
__device__ __forceinline__ void fill_counts(const AttendArgs& a, StreamItem& it, int n_old, int warp) {
    const bool append = a.k_new != nullptr;
    it.n_old = n_old;
    it.full = append && n_old >= a.cap_tokens;
    it.n = it.full ? 0 : n_old + (append ? 1 : 0);
    const int ng = (it.n + kGroupTokens - 1) / kGroupTokens;
    it.count = ng > warp ? (ng - warp + NW - 1) / NW : 0;
    it.app_idx = -1;
    if (append && !it.full) {
        const int g = n_old / kGroupTokens;
        if (g % NW == warp) it.app_idx = g / NW;
    }
}

__device__ __forceinline__ void decode_ticket(const AttendArgs& a, int ticket, StreamItem& it) {
    it.valid = ticket < a.n_items;
    const int t = it.valid ? ticket : 0;
    it.hkv = t % a.Hkv;
    it.b = (t / a.Hkv) % a.B;
    it.li = t / (a.Hkv * a.B);
    it.l = a.layer_begin + it.li;
    it.item = (it.l * a.B + it.b) * a.Hkv + it.hkv;
}

__device__ __forceinline__ int opaque(int x) {
    asm volatile("" : "+r"(x));
    return x;
}

// GT: query heads per KV head when known at compile time (0 = from the arguments).
template <int D, int NW, int NS, bool PAGED, bool SPILL, int GT = 0>
__global__ void __launch_bounds__(NW * 32, 1) attend_stream_kernel(const __grid_constant__ AttendArgs a) {
    using T = __nv_bfloat16;
    constexpr int NT = NW * 32;
    constexpr int ROW_BYTES = D * 2;
    constexpr int CHUNKS = ROW_BYTES / 16;
    constexpr int TILE_BYTES = kGroupTokens * ROW_BYTES;
    constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    constexpr int WARP_BYTES = NS * STAGE_BYTES;
    constexpr int KS = D / 16;
    static_assert(NS >= 2 && NS <= 5, "pipeline depth");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    // layout: stages [NW][NS][K tile | V tile] | wo [NW][GP][D] fp32 | EpilogueSmem | lg [chunk_tokens][GP]
    const int G = GT ? GT : a.G, GP = GT ? ((GT + 1) & ~1) : a.GP;
    const int wo_stride = GP * D;
    float* wo_all = reinterpret_cast<float*>(smem_raw + (size_t)NW * WARP_BYTES);
    EpilogueSmem& es = *reinterpret_cast<EpilogueSmem*>(wo_all + (size_t)NW * wo_stride);
    float* lg = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(&es) + sizeof(EpilogueSmem));
    // Logits of tokens beyond the shared-memory buffer overflow to this CTA's slice of global scratch.
    // (SPILL is a compile-time switch so that launches whose buffer covers the capacity pay nothing for it.)
    const int chunk = SPILL ? a.chunk_tokens : 0x7fffffff;
    float* spill = SPILL ? a.spill + (size_t)blockIdx.x * a.spill_tokens * GP : nullptr;
    const uint32_t lg_u32 = smem_u32(lg);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int gq = lane >> 2, tq = lane & 3;
    const bool append = a.k_new != nullptr;
    unsigned int* sched = a.sched;  // [0] next ticket, [1] CTAs that have finished

    // ---- first two tickets
    bool drew_fail = false;  // meaningful in thread 0 only
    if (tid == 0) {
        int t0 = (int)atomicAdd(&sched[0], 1u);
        int t1 = a.n_items;
        if (t0 >= a.n_items) drew_fail = true;
        else {
            t1 = (int)atomicAdd(&sched[0], 1u);
            if (t1 >= a.n_items) drew_fail = true;
        }
        es.flags[0] = t0;
        es.flags[1] = t1;
    }
    __syncthreads();
    StreamItem cur, nxt;
    decode_ticket(a, es.flags[0], cur);
    decode_ticket(a, es.flags[1], nxt);
    fill_counts<NW>(a, cur, cur.valid ? a.len[cur.item] : 0, warp);
    int nxt_n_raw = nxt.valid ? a.len[nxt.item] : 0;  // consumed lazily (see opaque) so the load stays in flight

    auto load_q = [&](const StreamItem& it, uint32_t (&bq)[KS][2]) {
        const uint32_t* qrow = reinterpret_cast<const uint32_t*>(
            (const T*)a.q + ((size_t)(it.li * a.B + it.b) * a.Hq + it.hkv * G + gq) * D);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            bq[ks][0] = (it.valid && gq < G) ? qrow[8 * ks + tq] : 0u;
            bq[ks][1] = (it.valid && gq < G) ? qrow[8 * ks + 4 + tq] : 0u;
        }
    };
    // The appended row of an item (lanes 0..15: 16-byte chunks of the k row, lanes 16..31: of the v row) and its
    // position are fetched together with the query rows, an item ahead: the append itself then never waits on them.
    auto load_new = [&](const StreamItem& it, uint4& row, int& pos) {
        row = make_uint4(0u, 0u, 0u, 0u);
        pos = 0;
        if (append && it.valid) {
            const size_t src = ((size_t)(it.li * a.B + it.b) * a.Hkv + it.hkv) * CHUNKS;
            if ((lane & 15) < CHUNKS) row = reinterpret_cast<const uint4*>(lane < 16 ? a.k_new : a.v_new)[src + (lane & 15)];
            pos = a.token_pos[it.b];
        }
    };
    uint32_t bq[KS][2], bqn[KS][2];
    uint4 new_row, new_row_n;
    int new_pos, new_pos_n;
    load_q(cur, bq);
    load_q(nxt, bqn);
    load_new(cur, new_row, new_pos);
    load_new(nxt, new_row_n, new_pos_n);

    unsigned char* my_stage = smem_raw + (size_t)warp * WARP_BYTES;
    const uint32_t my_stage_u32 = smem_u32(my_stage);
    bool bad_page = false;
    const uint64_t stream_policy = l2_evict_first_policy();
    const uint64_t spill_policy = l2_evict_last_policy();

    // issue the copies of this warp's local group `idx` of item `it` into stage slot `slot`
    // PAGED: page ids of this warp's local groups are fetched 32 at a time, one lane each, a block ahead of their
    // use, so that staging a group never waits on a page-table load.
    int pg_lo = 0, pg_hi = 0, pg_nxt = 0;  // current item: blocks pg_blk and pg_blk + 1; next item: block 0
    int pg_blk = 0;
    auto load_pages = [&](const StreamItem& it, int count, int blk) -> int {
        const int g = blk * 32 + lane;
        return (PAGED && it.valid && g < count) ? a.page_table[(size_t)it.item * a.capacity + warp + g * NW] : 0;
    };
    auto issue = [&](const StreamItem& it, int idx, int slot, bool is_cur) {
        const int grp = warp + idx * NW;
        const int tok0 = grp * kGroupTokens;
        if (idx == it.app_idx) {  // Sec. 4.1: the generated token's k / v row enters the cache first
            bool bad = false;
            char* kd = const_cast<char*>(row_ptr<PAGED>(a, a.k, it.item, it.n_old, ROW_BYTES, &bad));
            char* vd = const_cast<char*>(row_ptr<PAGED>(a, a.v, it.item, it.n_old, ROW_BYTES, &bad));
            if (kd && vd && (lane & 15) < CHUNKS)
                *reinterpret_cast<uint4*>((lane < 16 ? kd : vd) + (lane & 15) * 16) = is_cur ? new_row : new_row_n;
            if (lane == 0) a.pos[(size_t)it.item * a.cap_tokens + it.n_old] = is_cur ? new_pos : new_pos_n;
            __syncwarp();
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
                    pg_hi = load_pages(it, it.count, pg_blk + 1);
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
#pragma unroll
        for (int i = 0; i < kGroupTokens * CHUNKS / 32; ++i) {
            const int c_idx = i * 32 + lane;
            const int r = c_idx / CHUNKS, c = c_idx % CHUNKS;
            const bool valid = ok && (tok0 + r < it.n);
            const int soff = valid ? r * ROW_BYTES + c * 16 : 0;  // rows past n are zero-filled, never read
            const uint32_t doff = r * ROW_BYTES + ((c ^ (r & 7)) << 4);
            cp_async16_hint(ks_u32 + doff, kb + soff, valid ? 16 : 0, stream_policy);
            cp_async16_hint(vs_u32 + doff, vb + soff, valid ? 16 : 0, stream_policy);
        }
    };

    const int k_row = (lane & 7) + ((lane >> 3) & 1) * 8, k_chunk = lane >> 4;
    const int v_row = (lane & 7) + ((lane >> 4) & 1) * 8, v_chunk = (lane >> 3) & 1;

    pg_lo = load_pages(cur, cur.count, 0);
    pg_hi = load_pages(cur, cur.count, 1);

    int vp = 0;              // stage slot of the current item's local group 0
    unsigned issued = 0;     // bit j: local group j (< NS-1) of the current item was prefetched by the previous tail

    while (cur.valid) {
        const float sl2 = a.scale_log2[cur.l];
        // ---- top-up: whatever of the first NS-1 groups the previous tail did not prefetch
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
        bool nxt_ready = false;  // nxt's counts derived from its len

        float m0 = -INFINITY, m1 = -INFINITY, l0 = 0.f, l1 = 0.f;
        float o[KS][4];
#pragma unroll
        for (int mt = 0; mt < KS; ++mt)
#pragma unroll
            for (int i = 0; i < 4; ++i) o[mt][i] = 0.f;

        for (int it = 0; it < cur.count; ++it) {
            // Refill first, wait second: the slot of group it-1 is free once every lane has left the previous
            // iteration, so the copy of the group NS-1 ahead (possibly of the next item) is already in flight
            // while this warp waits for group `it`.
            __syncwarp();
            const bool strict = topped && it < NS - 1;  // after a top-up the group order is not the commit order
            if (strict) cp_async_wait<0>();
            {
                const int idx = it + NS - 1;
                const int slot = (vp + idx) % NS;
                if (idx < cur.count) issue(cur, idx, slot, true);
                else if (nxt.valid) {
                    if (!nxt_ready) {
                        fill_counts<NW>(a, nxt, opaque(nxt_n_raw), warp);
                        pg_nxt = load_pages(nxt, nxt.count, 0);
                        nxt_ready = true;
                    }
                    const int j = idx - cur.count;
                    if (j < nxt.count) {
                        issue(nxt, j, slot, false);
                        issued_next |= 1u << j;
                    }
                }
                cp_async_commit();
            }
            if (!strict) cp_async_wait<NS - 1>();  // everything but the NS-1 newest groups, i.e. group `it`, has landed
            __syncwarp();
            const int grp = warp + it * NW;
            const uint32_t ks_u32 = my_stage_u32 + ((vp + it) % NS) * STAGE_BYTES;
            const uint32_t vs_u32 = ks_u32 + TILE_BYTES;

            float ca[4] = {0.f, 0.f, 0.f, 0.f}, cb[4] = {0.f, 0.f, 0.f, 0.f};
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                uint32_t af[4];
                ldmatrix_x4(ks_u32 + k_row * ROW_BYTES + (((2 * ks + k_chunk) ^ (k_row & 7)) << 4), af);
                if (ks & 1) mma_bf16(cb, af, bq[ks][0], bq[ks][1]);
                else mma_bf16(ca, af, bq[ks][0], bq[ks][1]);
            }
            const int tokA = grp * kGroupTokens + gq, tokB = tokA + 8;
            const float s00 = (tokA < cur.n) ? (ca[0] + cb[0]) * sl2 : -INFINITY;
            const float s01 = (tokA < cur.n) ? (ca[1] + cb[1]) * sl2 : -INFINITY;
            const float s10 = (tokB < cur.n) ? (ca[2] + cb[2]) * sl2 : -INFINITY;
            const float s11 = (tokB < cur.n) ? (ca[3] + cb[3]) * sl2 : -INFINITY;
            if (2 * tq < GP) {
                if (!SPILL || tokA < chunk) st_shared_f2(lg_u32 + (tokA * GP + 2 * tq) * 4, s00, s01);
                else st_global_f2_hint(spill + (size_t)(tokA - chunk) * GP + 2 * tq, s00, s01, spill_policy);
                if (!SPILL || tokB < chunk) st_shared_f2(lg_u32 + (tokB * GP + 2 * tq) * 4, s10, s11);
                else st_global_f2_hint(spill + (size_t)(tokB - chunk) * GP + 2 * tq, s10, s11, spill_policy);
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
                ldmatrix_x4_trans(vs_u32 + v_row * ROW_BYTES + (((2 * mt + v_chunk) ^ (v_row & 7)) << 4), af);
                mma_bf16(o[mt], af, pb0, pb1);
            }
        }
        vp = (vp + cur.count) % NS;

        // ---- epilogue of the item: merge warps, write out / lse, Eq. 5 on rel[0..n)
        float rel_old[kRelPrefetch];
        {
            const float* relp = a.rel + (size_t)cur.item * a.cap_tokens;
            const int app = (append && !cur.full) ? cur.n_old : -1;
#pragma unroll
            for (int i = 0; i < kRelPrefetch; ++i) {
                const int j = tid + i * NT;
                rel_old[i] = (j < cur.n && j != app) ? relp[j] : 0.f;
            }
        }
#pragma unroll
        for (int off = 4; off < 32; off <<= 1) {
            l0 += __shfl_xor_sync(0xffffffffu, l0, off);
            l1 += __shfl_xor_sync(0xffffffffu, l1, off);
        }
        if (gq == 0) {
            es.wstat[warp][2 * tq] = make_float2(m0, l0);
            es.wstat[warp][2 * tq + 1] = make_float2(m1, l1);
        }
        if (2 * tq < GP) {
            float* wo = wo_all + (size_t)warp * wo_stride;
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) {
                wo[(2 * tq) * D + 16 * mt + gq] = o[mt][0];
                wo[(2 * tq + 1) * D + 16 * mt + gq] = o[mt][1];
                wo[(2 * tq) * D + 16 * mt + gq + 8] = o[mt][2];
                wo[(2 * tq + 1) * D + 16 * mt + gq + 8] = o[mt][3];
            }
        }
        int t_new = a.n_items;
        if (tid == 0 && !drew_fail)  // ticket of the item after next; its latency hides behind the barrier wait
            t_new = (int)atomicAdd(&sched[0], 1u);
        __syncthreads();  // B1: every warp's partials are in shared memory
        if (tid < kMaxGroup) {
            const int h = tid;
            float m = -INFINITY;
#pragma unroll
            for (int w = 0; w < NW; ++w) m = fmaxf(m, es.wstat[w][h].x);
            float l = 0.f;
#pragma unroll
            for (int w = 0; w < NW; ++w) {
                const float sc = exp2_diff(es.wstat[w][h].x, m);
                es.wscale[w][h] = sc;
                l += es.wstat[w][h].y * sc;
            }
            es.fin[h] = make_float2(m, l > 0.f ? 1.f / l : 0.f);
            if (a.lse && h < G)
                a.lse[(size_t)(cur.li * a.B + cur.b) * a.Hq + cur.hkv * G + h] =
                    l > 0.f ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
        }
        __syncthreads();  // B2
        {
            T* out = (T*)a.out + ((size_t)(cur.li * a.B + cur.b) * a.Hq + cur.hkv * G) * D;
            for (int idx = tid; idx < G * D; idx += NT) {
                const int h = idx / D;
                float acc = 0.f;
#pragma unroll
                for (int w = 0; w < NW; ++w) acc += wo_all[(size_t)w * wo_stride + idx] * es.wscale[w][h];
                out[idx] = __float2bfloat16_rn(acc * es.fin[h].y);
            }
            float fm[kMaxGroup], fi[kMaxGroup];
#pragma unroll
            for (int h = 0; h < kMaxGroup; ++h) {
                fm[h] = es.fin[h].x;
                fi[h] = es.fin[h].y;
            }
            float* relp = a.rel + (size_t)cur.item * a.cap_tokens;
            // One token's G logits (from shared memory, or from the overflow area), then its attention mass.
            auto load_row = [&](int j, float2 (&s)[kMaxGroup / 2]) {
                const bool in_smem = !SPILL || j < chunk;
#pragma unroll
                for (int h = 0; h < kMaxGroup; h += 2)
                    if (h < GP)
                        s[h / 2] = in_smem ? ld_shared_f2(lg_u32 + (j * GP + h) * 4)
                                           : ld_global_f2_hint(spill + (size_t)(j - chunk) * GP + h, spill_policy);
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
#pragma unroll
            for (int i = 0; i < kRelPrefetch; ++i) {
                const int j = tid + i * NT;
                if (j < cur.n) {
                    float2 s[kMaxGroup / 2];
                    load_row(j, s);
                    relp[j] = fmaf(a.gamma, rel_old[i], mass_from(s));
                }
            }
            // The tail of a long item: kRelBatch tokens per thread at a time, every load of the batch issued
            // before the first use, so that the global-memory latency is paid once per batch.
            for (int j0 = tid + kRelPrefetch * NT; j0 < cur.n; j0 += kRelBatch * NT) {
                float old[kRelBatch];
                float2 s[kRelBatch][kMaxGroup / 2];
#pragma unroll
                for (int u = 0; u < kRelBatch; ++u) {
                    const int j = j0 + u * NT;
                    const bool ok = j < cur.n;
                    old[u] = (ok && !(append && j == cur.n_old)) ? relp[j] : 0.f;
                    load_row(ok ? j : j0, s[u]);
                }
#pragma unroll
                for (int u = 0; u < kRelBatch; ++u) {
                    const int j = j0 + u * NT;
                    if (j < cur.n) relp[j] = fmaf(a.gamma, old[u], mass_from(s[u]));
                }
            }
        }
        if (tid == 0) {
            if (cur.full) record_error(a.status, LETHE_ERR_CAPACITY, cur.item);
            else if (append) a.len[cur.item] = cur.n;
            if (t_new >= a.n_items) drew_fail = true;
            es.flags[2] = t_new;
        }
        __syncthreads();  // B3: lg / wo / wstat may be reused; the next ticket is visible

        // ---- rotate: next becomes current
        if (nxt.valid && !nxt_ready) {
            fill_counts<NW>(a, nxt, nxt_n_raw, warp);
            pg_nxt = load_pages(nxt, nxt.count, 0);
        }
        cur = nxt;
        pg_lo = pg_nxt;
        pg_blk = 0;
        pg_hi = load_pages(cur, cur.valid ? cur.count : 0, 1);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            bq[ks][0] = bqn[ks][0];
            bq[ks][1] = bqn[ks][1];
        }
        new_row = new_row_n;
        new_pos = new_pos_n;
        issued = issued_next;
        decode_ticket(a, es.flags[2], nxt);
        nxt_n_raw = nxt.valid ? a.len[nxt.item] : 0;
        load_q(nxt, bqn);
        load_new(nxt, new_row_n, new_pos_n);
    }
    cp_async_wait<0>();
    if (bad_page) record_error(a.status, LETHE_ERR_PAGE, 0);

    // ---- the last CTA out re-arms the queue for the next launch
    if (tid == 0) {
        __threadfence();
        const unsigned int done = atomicAdd(&sched[1], 1u);
        if (done == gridDim.x - 1) {
            sched[0] = 0u;
            sched[1] = 0u;
            __threadfence();
        }
    }
}

template <int D, int NW, int NS>
static size_t stream_smem(int chunk_tokens, int GP) {
    return (size_t)NW * NS * 2 * kGroupTokens * D * 2 + (size_t)NW * GP * D * 4 + sizeof(EpilogueSmem) +
           (size_t)chunk_tokens * GP * 4;
}

template <int D, int NW, int NS, bool PAGED, bool SPILL, int GT = 0>
static cudaError_t launch_stream_t(const AttendArgs& a, int grid, cudaStream_t stream) {
    auto kern = attend_stream_kernel<D, NW, NS, PAGED, SPILL, GT>;
    const size_t smem = stream_smem<D, NW, NS>(a.chunk_tokens, a.GP);
    cudaError_t e = prepare_kernel((const void*)kern, smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, NW * 32, smem, stream>>>(a);
    return cudaGetLastError();
}

template <int D, int NW, int NS, int GT = 0>
static cudaError_t dispatch_stream(const AttendArgs& a, bool paged, int grid, cudaStream_t stream) {
    const bool spill = a.spill != nullptr;
    if (paged) return spill ? launch_stream_t<D, NW, NS, true, true, GT>(a, grid, stream) : launch_stream_t<D, NW, NS, true, false, GT>(a, grid, stream);
    return spill ? launch_stream_t<D, NW, NS, false, true, GT>(a, grid, stream) : launch_stream_t<D, NW, NS, false, false, GT>(a, grid, stream);
}

// Shapes of the persistent kernel: (warps per CTA, stages per warp).
#define LETHE_STREAM_SHAPES(X, D) X(0, D, 8, 2) X(1, D, 6, 3) X(2, D, 10, 2) X(3, D, 8, 3) X(4, D, 7, 3) X(5, D, 5, 4) X(6, D, 6, 2) \
        X(7, D, 5, 3)

size_t stream_smem_bytes(int D, int shape, int chunk_tokens, int GP) {
#define X(id, DD, NW, NS) \
    if (shape == id && D == DD) return stream_smem<DD, NW, NS>(chunk_tokens, GP);
    LETHE_STREAM_SHAPES(X, 128)
    LETHE_STREAM_SHAPES(X, 64)
#undef X
    return (size_t)-1;
}

cudaError_t launch_attend_stream(const AttendArgs& a, int D, int shape, bool paged, int grid, cudaStream_t stream) {
    // the automatic choice for wide groups (seven query heads per KV head: the Qwen geometry), group size compiled in
    if (D == 128 && shape == 0 && a.G == 7) return dispatch_stream<128, 8, 2, 7>(a, paged, grid, stream);
#define X(id, DD, NW, NS)                                                                                   \
    if (shape == id && D == DD)                                                                             \
        return dispatch_stream<DD, NW, NS>(a, paged, grid, stream);
    LETHE_STREAM_SHAPES(X, 128)
    LETHE_STREAM_SHAPES(X, 64)
#undef X
    return cudaErrorInvalidValue;
}

}  // namespace lethe
