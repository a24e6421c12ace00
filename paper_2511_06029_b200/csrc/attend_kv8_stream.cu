// Persistent decode-attend kernel for quantised caches (K / V as e4m3 bytes with one scale per layer, bf16
// activations; D in {64, 128}, G <= 8): the schedule of the persistent bf16 kernel — one CTA per SM walking a
// dynamic, longest-first queue of items, per-warp cp.async pipelines whose refills run on into the next item, a
// CTA-wide epilogue per item — around the byte-to-fragment arithmetic of the clustered quantised kernel
// (attend_kv8.cu): f16 MMAs on fragments converted in registers, the key bytes' permuted contraction order
// matched by the Q^T fragments, even / odd output dimensions separated by a byte permute on the V side, the key
// scale folded into the softmax scale, the value scale applied to each warp's partial output, and an append path
// that quantises (fp32 division by the scale, round to nearest even, saturate at +-448).
#include <cuda_fp16.h>

#include "common.cuh"
#include "mma_utils.cuh"

namespace lethe {
namespace {

__device__ __forceinline__ void mma_f16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile(
        "mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
        : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
        : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
// two e4m3 bytes (low 16 bits of x) -> f16x2, byte 0 in the low half
__device__ __forceinline__ uint32_t e4m3x2_to_f16x2(uint32_t x) {
    uint32_t y;
    asm("{ .reg .b16 lo; cvt.u16.u32 lo, %1; cvt.rn.f16x2.e4m3x2 %0, lo; }" : "=r"(y) : "r"(x));
    return y;
}
__device__ __forceinline__ uint32_t pack_f16(float lo, float hi) {
    __half2 v = __floats2half2_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}
// two fp32 -> two e4m3 bytes (round to nearest even, saturating), `lo` in the low byte
__device__ __forceinline__ uint32_t f32x2_to_e4m3x2(float lo, float hi) {
    uint32_t y;
    asm("{ .reg .b16 r; cvt.rn.satfinite.e4m3x2.f32 r, %2, %1; cvt.u32.u16 %0, r; }" : "=r"(y) : "f"(lo), "f"(hi));
    return y;
}
// two bf16 values times a power of two -> two f16 values (exact while the products are within f16's range)
__device__ __forceinline__ uint32_t bf16x2_to_f16x2_scaled(uint32_t x, float mul) {
    return pack_f16(__uint_as_float(x << 16) * mul, __uint_as_float(x & 0xffff0000u) * mul);
}
// The divisor (a power of two, returned in `div`) that brings the largest magnitude of a query row into [128, 256), and
// its inverse (the return value): f16 holds 6e-8 .. 65504, bf16 queries can be anything.  The row is spread over the
// four lanes that share gq = lane >> 2; w holds this lane's bf16 pairs.
template <int KS>
__device__ __forceinline__ float query_row_scale(const uint2 (&w)[KS], float& div) {
    float big = 0.f;
#pragma unroll
    for (int ks = 0; ks < KS; ++ks) {
        big = fmaxf(big, fmaxf(fabsf(__uint_as_float(w[ks].x << 16)), fabsf(__uint_as_float(w[ks].x & 0xffff0000u))));
        big = fmaxf(big, fmaxf(fabsf(__uint_as_float(w[ks].y << 16)), fabsf(__uint_as_float(w[ks].y & 0xffff0000u))));
    }
    big = fmaxf(big, __shfl_xor_sync(0xffffffffu, big, 1));
    big = fmaxf(big, __shfl_xor_sync(0xffffffffu, big, 2));
    int ex = (int)((__float_as_uint(big) >> 23) & 0xffu) - 7;  // biased exponent of the divisor
    ex = big > 0.f && big < INFINITY ? min(max(ex, 2), 252) : 127;
    div = __uint_as_float((uint32_t)ex << 23);
    return __uint_as_float((uint32_t)(254 - ex) << 23);
}

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

}  // namespace

// GT: query heads per KV head when known at compile time (0 = from the arguments).
template <int D, int NW, int NS, bool PAGED, bool SPILL, int GT = 0>
__global__ void __launch_bounds__(NW * 32, 1) attend_kv8_stream_kernel(const __grid_constant__ AttendArgs a) {
    using T = __nv_bfloat16;
    constexpr int NT = NW * 32;
    constexpr int ROW_BYTES = D;                    // one byte per element
    constexpr int CHUNKS = ROW_BYTES / 16;
    constexpr int ROWS_PER_LINE = 128 / ROW_BYTES;  // rows sharing a 128-byte line of shared memory
    constexpr int MT = D / 32;                      // 32-wide blocks of the output dimension
    constexpr int TILE_BYTES = kGroupTokens * ROW_BYTES;
    constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    constexpr int WARP_BYTES = NS * STAGE_BYTES;
    constexpr int KS = D / 16;
    static_assert(NS >= 2 && NS <= 5, "pipeline depth");
    // bank-conflict-free placement of 16-byte chunk c of row r (the eight rows an ldmatrix touches land in eight
    // different chunk positions of their 128-byte lines)
    auto swz = [](int r, int c) -> uint32_t {
        return (uint32_t)(r * ROW_BYTES + ((c ^ ((r / ROWS_PER_LINE) & (CHUNKS - 1))) << 4));
    };
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

    auto load_q = [&](const StreamItem& it, uint32_t (&bq)[KS][2], float& qdiv) {
        // f16, in the permuted order of the key bytes: b0 = Q[head gq][16 ks + 4 tq + {0, 1}], b1 = ... + {2, 3}; the row is
        // divided by the power of two qdiv first (see query_row_scale), the head's logits are multiplied back
        const uint2* qrow = reinterpret_cast<const uint2*>(
            (const T*)a.q + ((size_t)(it.li * a.B + it.b) * a.Hq + it.hkv * G + gq) * D);
        uint2 w[KS];
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) w[ks] = (it.valid && gq < G) ? qrow[4 * ks + tq] : make_uint2(0u, 0u);
        const float inv = query_row_scale(w, qdiv);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            bq[ks][0] = bf16x2_to_f16x2_scaled(w[ks].x, inv);
            bq[ks][1] = bf16x2_to_f16x2_scaled(w[ks].y, inv);
        }
    };
    uint32_t bq[KS][2], bqn[KS][2];
    float qdiv = 1.f, qdivn = 1.f;
    load_q(cur, bq, qdiv);
    load_q(nxt, bqn, qdivn);

    unsigned char* my_stage = smem_raw + (size_t)warp * WARP_BYTES;
    const uint32_t my_stage_u32 = smem_u32(my_stage);
    bool bad_page = false;
    const uint64_t stream_policy = l2_evict_first_policy();

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
            const size_t src = ((size_t)(it.li * a.B + it.b) * a.Hkv + it.hkv) * D;  // elements
            bool bad = false;
            char* kd = const_cast<char*>(row_ptr<PAGED>(a, a.k, it.item, it.n_old, ROW_BYTES, &bad));
            char* vd = const_cast<char*>(row_ptr<PAGED>(a, a.v, it.item, it.n_old, ROW_BYTES, &bad));
            if (kd && vd && lane * 4 < D) {  // four elements per lane, quantised
                const float ks_l = a.k_scale[it.l], vs_l = a.v_scale[it.l];
                const uint2 kw = *reinterpret_cast<const uint2*>((const T*)a.k_new + src + lane * 4);
                const uint2 vw = *reinterpret_cast<const uint2*>((const T*)a.v_new + src + lane * 4);
                auto quant4 = [](uint2 w, float sc) -> uint32_t {
                    const float x0 = __uint_as_float(w.x << 16), x1 = __uint_as_float(w.x & 0xffff0000u);
                    const float x2 = __uint_as_float(w.y << 16), x3 = __uint_as_float(w.y & 0xffff0000u);
                    return f32x2_to_e4m3x2(__fdiv_rn(x0, sc), __fdiv_rn(x1, sc)) |
                           (f32x2_to_e4m3x2(__fdiv_rn(x2, sc), __fdiv_rn(x3, sc)) << 16);
                };
                *reinterpret_cast<uint32_t*>(kd + lane * 4) = quant4(kw, ks_l);
                *reinterpret_cast<uint32_t*>(vd + lane * 4) = quant4(vw, vs_l);
            }
            if (lane == 0) a.pos[(size_t)it.item * a.cap_tokens + it.n_old] = a.token_pos[it.b];
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
            const uint32_t doff = swz(r, c);
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
        // this thread's two logit columns are heads 2 tq and 2 tq + 1: their divisors sit in the lanes with gq = head
        const float sl2_0 = sl2 * __shfl_sync(0xffffffffu, qdiv, (2 * tq) * 4), sl2_1 = sl2 * __shfl_sync(0xffffffffu, qdiv, (2 * tq + 1) * 4);
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
            for (int pr = 0; pr < KS / 2; ++pr) {  // 32 bytes of every key row: two k-steps
                uint32_t r[4];  // rows gq | gq + 8 of bytes [32 pr, +16) | rows gq | gq + 8 of bytes [32 pr + 16, +16)
                ldmatrix_x4(ks_u32 + swz(k_row, 2 * pr + k_chunk), r);
                const uint32_t a0[4] = {e4m3x2_to_f16x2(r[0]), e4m3x2_to_f16x2(r[1]), e4m3x2_to_f16x2(r[0] >> 16), e4m3x2_to_f16x2(r[1] >> 16)};
                const uint32_t a1[4] = {e4m3x2_to_f16x2(r[2]), e4m3x2_to_f16x2(r[3]), e4m3x2_to_f16x2(r[2] >> 16), e4m3x2_to_f16x2(r[3] >> 16)};
                mma_f16(ca, a0, bq[2 * pr][0], bq[2 * pr][1]);
                mma_f16(cb, a1, bq[2 * pr + 1][0], bq[2 * pr + 1][1]);
            }
            const int tokA = grp * kGroupTokens + gq, tokB = tokA + 8;
            const float s00 = (tokA < cur.n) ? (ca[0] + cb[0]) * sl2_0 : -INFINITY;
            const float s01 = (tokA < cur.n) ? (ca[1] + cb[1]) * sl2_1 : -INFINITY;
            const float s10 = (tokB < cur.n) ? (ca[2] + cb[2]) * sl2_0 : -INFINITY;
            const float s11 = (tokB < cur.n) ? (ca[3] + cb[3]) * sl2_1 : -INFINITY;
            if (2 * tq < GP) {
                if (!SPILL || tokA < chunk) st_shared_f2(lg_u32 + (tokA * GP + 2 * tq) * 4, s00, s01);
                else *reinterpret_cast<float2*>(spill + (size_t)(tokA - chunk) * GP + 2 * tq) = make_float2(s00, s01);
                if (!SPILL || tokB < chunk) st_shared_f2(lg_u32 + (tokB * GP + 2 * tq) * 4, s10, s11);
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
            const uint32_t pb0 = movmatrix_trans(pack_f16(p00, p01));
            const uint32_t pb1 = movmatrix_trans(pack_f16(p10, p11));
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                // per register: {tok: d, d+1}, {tok+1: d, d+1}; tokens 2tq, 2tq+1 (r[0], r[1]) and +8 (r[2], r[3]);
                // d = 32 mt + 2 gq (r[0], r[2]) and d + 16 (r[1], r[3])
                uint32_t r[4];
                ldmatrix_x4_trans(vs_u32 + swz(v_row, 2 * mt + v_chunk), r);
                uint32_t ae[4], ao[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    ae[i] = e4m3x2_to_f16x2(__byte_perm(r[i], 0u, 0x4420));  // even d: bytes 0 and 2
                    ao[i] = e4m3x2_to_f16x2(__byte_perm(r[i], 0u, 0x4431));  // odd d:  bytes 1 and 3
                }
                mma_f16(o[2 * mt], ae, pb0, pb1);
                mma_f16(o[2 * mt + 1], ao, pb0, pb1);
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
            // accumulator o[2 mt + par]: rows gq / gq + 8 are d = 32 mt + 2 gq + par and d + 16; a value byte x means
            // v_scale * x
            const float vs_l = a.v_scale[cur.l];
            float* wo = wo_all + (size_t)warp * wo_stride;
#pragma unroll
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int par = 0; par < 2; ++par) {
                    const int d = 32 * mt + 2 * gq + par;
                    wo[(2 * tq) * D + d] = o[2 * mt + par][0] * vs_l;
                    wo[(2 * tq + 1) * D + d] = o[2 * mt + par][1] * vs_l;
                    wo[(2 * tq) * D + d + 16] = o[2 * mt + par][2] * vs_l;
                    wo[(2 * tq + 1) * D + d + 16] = o[2 * mt + par][3] * vs_l;
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
            auto mass_of = [&](int j) {
                const bool in_smem = !SPILL || j < chunk;
                float mass = 0.f;
#pragma unroll
                for (int h = 0; h < kMaxGroup; h += 2) {
                    if (h < GP) {
                        const float2 s2 = in_smem ? ld_shared_f2(lg_u32 + (j * GP + h) * 4)
                                                  : *reinterpret_cast<const float2*>(spill + (size_t)(j - chunk) * GP + h);
                        mass += fast_exp2(s2.x - fm[h]) * fi[h];
                        if (h + 1 < G) mass += fast_exp2(s2.y - fm[h + 1]) * fi[h + 1];
                    }
                }
                return mass;
            };
#pragma unroll
            for (int i = 0; i < kRelPrefetch; ++i) {
                const int j = tid + i * NT;
                if (j < cur.n) relp[j] = fmaf(a.gamma, rel_old[i], mass_of(j));
            }
            for (int j = tid + kRelPrefetch * NT; j < cur.n; j += NT) {
                const float old = (append && j == cur.n_old) ? 0.f : relp[j];
                relp[j] = fmaf(a.gamma, old, mass_of(j));
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
        qdiv = qdivn;
        issued = issued_next;
        decode_ticket(a, es.flags[2], nxt);
        nxt_n_raw = nxt.valid ? a.len[nxt.item] : 0;
        load_q(nxt, bqn, qdivn);
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
static size_t kv8s_smem(int chunk_tokens, int GP) {
    return (size_t)NW * NS * 2 * kGroupTokens * D + (size_t)NW * GP * D * 4 + sizeof(EpilogueSmem) +
           (size_t)chunk_tokens * GP * 4;
}

template <int D, int NW, int NS, bool PAGED, bool SPILL, int GT = 0>
static cudaError_t launch_kv8s_t(const AttendArgs& a, int grid, cudaStream_t stream) {
    auto kern = attend_kv8_stream_kernel<D, NW, NS, PAGED, SPILL, GT>;
    const size_t smem = kv8s_smem<D, NW, NS>(a.chunk_tokens, a.GP);
    cudaError_t e = prepare_kernel((const void*)kern, smem);
    if (e != cudaSuccess) return e;
    kern<<<grid, NW * 32, smem, stream>>>(a);
    return cudaGetLastError();
}

template <int D, int NW, int NS, int GT = 0>
static cudaError_t dispatch_kv8s(const AttendArgs& a, bool paged, int grid, cudaStream_t stream) {
    const bool spill = a.spill != nullptr;
    if (paged) return spill ? launch_kv8s_t<D, NW, NS, true, true, GT>(a, grid, stream) : launch_kv8s_t<D, NW, NS, true, false, GT>(a, grid, stream);
    return spill ? launch_kv8s_t<D, NW, NS, false, true, GT>(a, grid, stream) : launch_kv8s_t<D, NW, NS, false, false, GT>(a, grid, stream);
}

// Shapes of the persistent kernel: (warps per CTA, stages per warp); tiles are half the size of the bf16 kernel's
// and the arithmetic per byte is heavier, so the shapes have more warps and deeper pipelines.
#define LETHE_KV8S_SHAPES(X, D) X(0, D, 8, 4) X(1, D, 12, 3) X(2, D, 10, 4) X(3, D, 8, 5) X(4, D, 16, 2) X(5, D, 12, 2)

size_t kv8_stream_smem_bytes(int D, int shape, int chunk_tokens, int GP) {
#define X(id, DD, NW, NS) \
    if (shape == id && D == DD) return kv8s_smem<DD, NW, NS>(chunk_tokens, GP);
    LETHE_KV8S_SHAPES(X, 128)
    LETHE_KV8S_SHAPES(X, 64)
#undef X
    return (size_t)-1;
}

cudaError_t launch_attend_kv8_stream(const AttendArgs& a, int D, int shape, bool paged, int grid, cudaStream_t stream) {
    // the automatic fallback for wide groups at large capacities (seven query heads per KV head), group size compiled in
    if (D == 128 && shape == 0 && a.G == 7) return dispatch_kv8s<128, 8, 4, 7>(a, paged, grid, stream);
#define X(id, DD, NW, NS)                                                                                   \
    if (shape == id && D == DD)                                                                             \
        return dispatch_kv8s<DD, NW, NS>(a, paged, grid, stream);
    LETHE_KV8S_SHAPES(X, 128)
    LETHE_KV8S_SHAPES(X, 64)
#undef X
    return cudaErrorInvalidValue;
}

}  // namespace lethe
