// Clustered tensor-core decode-attend kernel for launches of one layer (few items per launch): bf16 caches,
// D in {64, 128}, G <= 8, contiguous or 16-token pages.
//
// Same per-group arithmetic as attend_mma.cu (tokens on M, the group's heads on N, one private cp.async pipeline
// per warp, parked logits).  What differs is everything around the streaming loop, because a launch of one layer
// (64 items of ~1100 tokens on the Llama-8B shape: 37 MB, 6 us of HBM time) is bound by its fixed costs:
//
//   * Layer pipelining.  A served model issues one launch per layer, and layer l+1's query does not exist before
//     layer l is done; but the K / V rows layer l+1 will read were written long before.  Launched with programmatic
//     stream serialisation, a CTA of this kernel fills its pipeline stages with cached K / V tiles *before*
//     griddepcontrol.wait, i.e. while the previous layer's CTAs are still merging, updating relevance and exiting;
//     only then does it wait for that kernel, read its query rows, append the new row and start consuming.  It
//     releases the next launch (griddepcontrol.launch_dependents) right after its own wait, so at most two
//     generations are ever in flight.  The early fetch is taken only when the host code knows that the previous
//     kernel of the stream cannot have written this call's items (AttendArgs::early_prefetch).
//   * One-sided merge.  The CTAs of an item (a thread-block cluster) do not meet at cluster barriers.  Each CTA
//     pushes its per-head (max, sum) to every peer and slice r of its partial output to rank r through distributed
//     shared memory, then arrives (release) on the peers' mbarriers; a CTA waits only on its own mbarrier, after
//     which everything it needs is in its own shared memory.  Nobody reads a peer's memory, so a CTA may exit as
//     soon as it has finished — no closing barrier.  The wait is bounded (LETHE_ERR_TIMEOUT).
#include "common.cuh"
#include "kv8_utils.cuh"
#include "mma_utils.cuh"

namespace lethe {

constexpr int kLayerWaitLimit = 4000000;  // polls of the merge barrier before giving up (seconds)

struct LayerSmem {
    unsigned long long bar;             // one arrival per rank of the cluster, after that rank's pushes
    int abort;
    int pad;
    float2 wstat[8][kMaxGroup];         // per warp (at most 8 per CTA), per head: (running max in log2 units, partial sum)
    float2 peer_stat[16][kMaxGroup];    // pushed by rank r: its per-head (max, sum) over its whole token range
    alignas(16) float peer_o[kMaxGroup * 128 + 16]; // pushed by rank r: this CTA's slice of rank r's partial output, [S][per]
};

__device__ __forceinline__ uint32_t cluster_map(uint32_t local_addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(local_addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_f32(uint32_t addr, float v) {
    asm volatile("st.shared::cluster.f32 [%0], %1;" ::"r"(addr), "f"(v) : "memory");
}
__device__ __forceinline__ void st_cluster_f2(uint32_t addr, float2 v) {
    asm volatile("st.shared::cluster.v2.f32 [%0], {%1, %2};" ::"r"(addr), "f"(v.x), "f"(v.y) : "memory");
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
__device__ __forceinline__ void mbar_remote_arrive(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait_cluster(unsigned long long* bar, unsigned parity) {
    unsigned ok;
    asm volatile(
        "{ .reg .pred p; mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}

// GT: query heads per KV head when known at compile time (0 = from the arguments): the merge, output and relevance
// loops over heads then carry no run-time bounds.
// KV: 0 = bf16 cache; 1 / 2 = quantised cache (e4m3 / e5m2 bytes, one scale per layer): the same kernel around the
// byte-cache group arithmetic (bytes -> f16 fragments, f16 MMAs; see attend_kv8.cu for the fragment layouts).
template <int D, int NW, int NSTAGE, bool PAGED, int GT, int KV = 0>
__global__ void __launch_bounds__(NW * 32) attend_layer_kernel(const __grid_constant__ AttendArgs a) {
    using T = __nv_bfloat16;  // type of q, k_new, v_new, out (and of a bf16 cache)
    constexpr bool BYTES = KV != 0, E5M2 = KV == 2;
    constexpr int NT = NW * 32;
    constexpr int ROW_BYTES = BYTES ? D : D * 2;
    constexpr int CHUNKS = ROW_BYTES / 16;
    constexpr int ROWS_PER_LINE = ROW_BYTES >= 128 ? 1 : 128 / ROW_BYTES;  // rows sharing a 128-byte line of shared memory
    constexpr int TILE_BYTES = kGroupTokens * ROW_BYTES;
    constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    constexpr int WARP_BYTES = NSTAGE * STAGE_BYTES;
    constexpr int KS = D / 16;
    constexpr int MT = D / 32;  // byte caches: 32-wide blocks of the output dimension
    static_assert(WARP_BYTES >= kMaxGroup * D * 4, "per-warp stage area doubles as the partial-output buffer");
    static_assert(NW <= 8, "LayerSmem::wstat holds eight warps");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    // layout: stages [NW][NSTAGE][K tile | V tile] | LayerSmem | lg [chunk_tokens][GP]
    unsigned char* stage_base = smem_raw;
    LayerSmem& ls = *reinterpret_cast<LayerSmem*>(smem_raw + (size_t)NW * WARP_BYTES);
    float* lg = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(&ls) + sizeof(LayerSmem));

    // placement of 16-byte chunk c of row r in a tile: the eight rows an ldmatrix touches land in eight different chunk
    // positions of their 128-byte lines
    auto swz = [](int r, int c) -> uint32_t {
        return (uint32_t)(r * ROW_BYTES + ((c ^ ((r / ROWS_PER_LINE) & (CHUNKS < 8 ? CHUNKS - 1 : 7))) << 4));
    };

    const bool early = a.early_prefetch != 0;
    if (!early) asm volatile("griddepcontrol.wait;" ::: "memory");  // nothing is read before the previous kernel is done
    const ItemCoord ic = decode_item(a);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int gq = lane >> 2, tq = lane & 3;
    const int G = GT ? GT : a.G, GP = GT ? ((GT + 1) & ~1) : a.GP, S = a.splits;
    const bool append = a.k_new != nullptr;

    if (tid == 0) {
        asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(&ls.bar)), "r"(S) : "memory");
        ls.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    __syncwarp();
    cluster_arrive();  // peers may touch this CTA's barrier only after cluster_wait(), long after this point

    const int n_old = a.len[ic.item];
    const bool full = append && n_old >= a.cap_tokens;
    const int n = n_old + (append ? 1 : 0);
    const int append_slot = append ? n_old : -1;
    int g_begin, g_end;
    split_range(full ? 0 : n, S, ic.rank, g_begin, g_end);
    const int t0 = g_begin * kGroupTokens, t1 = g_end * kGroupTokens;

    bool bad_page = false;
    const uint64_t stream_policy = l2_evict_first_policy();
    unsigned char* my_stage = stage_base + (size_t)warp * WARP_BYTES;
    const uint32_t my_stage_u32 = smem_u32(my_stage);

    auto issue = [&](int grp, int s) {
        const int tok0 = grp * kGroupTokens;
        const char* kb;
        const char* vb;
        bool ok = true;
        if (PAGED) {
            const int page = a.page_table[(size_t)ic.item * a.capacity + grp];
            ok = page >= 0 && page < a.n_pages;
            if (!ok) bad_page = true;
            const size_t off = (size_t)(ok ? page : 0) * TILE_BYTES;
            kb = (const char*)a.k + off;
            vb = (const char*)a.v + off;
        } else {
            const size_t off = ((size_t)ic.item * a.capacity + tok0) * ROW_BYTES;
            kb = (const char*)a.k + off;
            vb = (const char*)a.v + off;
        }
        const uint32_t ks_u32 = my_stage_u32 + s * STAGE_BYTES;
        const uint32_t vs_u32 = ks_u32 + TILE_BYTES;
#pragma unroll
        for (int i = 0; i < kGroupTokens * CHUNKS / 32; ++i) {
            const int idx = i * 32 + lane;
            const int r = idx / CHUNKS, c = idx % CHUNKS;
            const bool valid = ok && (tok0 + r < n);
            const int soff = valid ? r * ROW_BYTES + c * 16 : 0;
            const uint32_t doff = swz(r, c);
            cp_async16_hint(ks_u32 + doff, kb + soff, valid ? 16 : 0, stream_policy);
            cp_async16_hint(vs_u32 + doff, vb + soff, valid ? 16 : 0, stream_policy);
        }
    };

    const int my_first = g_begin + warp;
    const int my_count = (g_end > my_first) ? (g_end - my_first + NW - 1) / NW : 0;

    // ---- before the previous kernel is known to be done: groups that hold cached rows only
    int pre = 0;
    if (early) {
#pragma unroll
        for (int s = 0; s < NSTAGE - 1; ++s) {
            const int grp = my_first + s * NW;
            if (pre == s && s < my_count && (grp + 1) * kGroupTokens <= n_old) {
                issue(grp, s);
                cp_async_commit();
                pre = s + 1;
            }
        }
        asm volatile("griddepcontrol.wait;" ::: "memory");
    }
    // this kernel's own inputs are complete from here on; the next launch of the stream may be scheduled (it will
    // itself wait for this kernel before touching anything this kernel writes)
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    T* out_rows = (T*)a.out + ((size_t)(ic.li * a.B + ic.b) * a.Hq + ic.hkv * G) * D;
    if (full) {  // leave the item untouched (every CTA of the cluster takes this path)
        cp_async_wait<0>();
        if (ic.rank == 0) {
            for (int i = tid; i < G * D; i += NT) out_rows[i] = __float2bfloat16_rn(0.f);
            if (a.lse && tid < G) a.lse[(size_t)(ic.li * a.B + ic.b) * a.Hq + ic.hkv * G + tid] = -INFINITY;
            if (tid == 0) record_error(a.status, LETHE_ERR_CAPACITY, ic.item);
        }
        return;
    }

    // Q^T fragments (B operand).  bf16 cache: b0 = Q[head gq][16 ks + 2 tq, +1], b1 = Q[head gq][16 ks + 8 + 2 tq, +1].
    // Byte cache: f16, in the permuted order of the key bytes (b0 = Q[head gq][16 ks + 4 tq + {0, 1}], b1 = ... + {2, 3}),
    // the row divided by the power of two qdiv first so that it fits f16 (the head's logits are multiplied back).
    uint32_t bq[KS][2];
    float qdiv = 1.f;
    if constexpr (!BYTES) {
        const uint32_t* qrow =
            reinterpret_cast<const uint32_t*>((const T*)a.q + ((size_t)(ic.li * a.B + ic.b) * a.Hq + ic.hkv * G + gq) * D);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            bq[ks][0] = (gq < G) ? qrow[8 * ks + tq] : 0u;
            bq[ks][1] = (gq < G) ? qrow[8 * ks + 4 + tq] : 0u;
        }
    } else {
        const uint2* qrow =
            reinterpret_cast<const uint2*>((const T*)a.q + ((size_t)(ic.li * a.B + ic.b) * a.Hq + ic.hkv * G + gq) * D);
        uint2 w[KS];
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) w[ks] = gq < G ? qrow[4 * ks + tq] : make_uint2(0u, 0u);
        const float inv = query_row_scale(w, qdiv);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            bq[ks][0] = bf16x2_to_f16x2_scaled(w[ks].x, inv);
            bq[ks][1] = bf16x2_to_f16x2_scaled(w[ks].y, inv);
        }
    }
    // Sec. 4.1: append the generated token's key / value; the CTA whose range holds slot n_old stores it.
    const bool i_append = append && n_old >= t0 && n_old < t1;
    if (i_append && warp == 0) {
        const size_t src = ((size_t)(ic.li * a.B + ic.b) * a.Hkv + ic.hkv) * ROW_BYTES;
        char* kd = const_cast<char*>(row_ptr<PAGED>(a, a.k, ic.item, n_old, ROW_BYTES, &bad_page));
        char* vd = const_cast<char*>(row_ptr<PAGED>(a, a.v, ic.item, n_old, ROW_BYTES, &bad_page));
        if constexpr (!BYTES) {
            if (kd && vd && lane * 16 < ROW_BYTES) {
                *reinterpret_cast<uint4*>(kd + lane * 16) = *reinterpret_cast<const uint4*>((const char*)a.k_new + src + lane * 16);
                *reinterpret_cast<uint4*>(vd + lane * 16) = *reinterpret_cast<const uint4*>((const char*)a.v_new + src + lane * 16);
            }
        } else if (kd && vd && lane * 4 < D) {  // quantised: x / scale in fp32, round to nearest even, saturate; four elements per lane
            const float ks_l = a.k_scale[ic.l], vs_l = a.v_scale[ic.l];
            const uint2 kw = *reinterpret_cast<const uint2*>((const T*)a.k_new + src + lane * 4);
            const uint2 vw = *reinterpret_cast<const uint2*>((const T*)a.v_new + src + lane * 4);
            auto quant4 = [](uint2 w, float sc) -> uint32_t {
                const float x0 = __uint_as_float(w.x << 16), x1 = __uint_as_float(w.x & 0xffff0000u);
                const float x2 = __uint_as_float(w.y << 16), x3 = __uint_as_float(w.y & 0xffff0000u);
                return f32x2_to_fp8x2<E5M2>(__fdiv_rn(x0, sc), __fdiv_rn(x1, sc)) | (f32x2_to_fp8x2<E5M2>(__fdiv_rn(x2, sc), __fdiv_rn(x3, sc)) << 16);
            };
            *reinterpret_cast<uint32_t*>(kd + lane * 4) = quant4(kw, ks_l);
            *reinterpret_cast<uint32_t*>(vd + lane * 4) = quant4(vw, vs_l);
        }
        if (lane == 0) a.pos[(size_t)ic.item * a.cap_tokens + n_old] = a.token_pos[ic.b];
    }
    if (i_append) __syncthreads();  // (uniform for the CTA) the appended row is in global memory before any warp streams it

    const float sl2 = a.scale_log2[ic.l];  // (byte caches: the key scale is folded in by the host)
    // byte caches: this thread's two logit columns are heads 2 tq and 2 tq + 1, whose query divisors sit in the lanes with gq = head
    const float sl2_0 = BYTES ? sl2 * __shfl_sync(0xffffffffu, qdiv, (2 * tq) * 4) : sl2;
    const float sl2_1 = BYTES ? sl2 * __shfl_sync(0xffffffffu, qdiv, (2 * tq + 1) * 4) : sl2;
#pragma unroll
    for (int s = 0; s < NSTAGE - 1; ++s) {
        if (s >= pre) {
            if (s < my_count) issue(my_first + s * NW, s);
            cp_async_commit();
        }
    }

    // The old relevance values this thread will update are fetched now, long before they are needed: asked for at
    // the end of the streaming loop they queue behind the other CTAs' K / V requests and arrive after the merge.
    constexpr int PF = 4;  // tokens per thread updated from prefetched values (a CTA's range is rarely longer than PF * NT)
    float rel_old[PF];
    {
        const float* relp = a.rel + (size_t)ic.item * a.cap_tokens;
#pragma unroll
        for (int i = 0; i < PF; ++i) {
            const int j = t0 + tid + i * NT;
            rel_old[i] = (j < min(t1, n) && j != append_slot) ? relp[j] : 0.f;
        }
    }

    float m0 = -INFINITY, m1 = -INFINITY;
    float l0 = 0.f, l1 = 0.f;
    // O^T fragments.  bf16: block mt covers d = 16 mt .. + 15 (rows gq, gq + 8).  Bytes: block mt / parity par covers
    // d = 32 mt + 2 gq + par and d + 16; o8 aliases the same registers as [MT][2][4].
    float o[KS][4];
#pragma unroll
    for (int mt = 0; mt < KS; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) o[mt][i] = 0.f;
    float (&o8)[MT][2][4] = reinterpret_cast<float (&)[MT][2][4]>(o);

    const int k_row = (lane & 7) + ((lane >> 3) & 1) * 8, k_chunk = lane >> 4;
    const int v_row = (lane & 7) + ((lane >> 4) & 1) * 8, v_chunk = (lane >> 3) & 1;

    for (int it = 0; it < my_count; ++it) {
        cp_async_wait<NSTAGE - 2>();
        __syncwarp();
        const int s = it % NSTAGE;
        const int grp = my_first + it * NW;
        const uint32_t ks_u32 = my_stage_u32 + s * STAGE_BYTES;
        const uint32_t vs_u32 = ks_u32 + TILE_BYTES;

        float ca[4] = {0.f, 0.f, 0.f, 0.f}, cb[4] = {0.f, 0.f, 0.f, 0.f};
        if constexpr (!BYTES) {
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                uint32_t af[4];
                ldmatrix_x4(ks_u32 + k_row * ROW_BYTES + (((2 * ks + k_chunk) ^ (k_row & 7)) << 4), af);
                if (ks & 1) mma_bf16(cb, af, bq[ks][0], bq[ks][1]);
                else mma_bf16(ca, af, bq[ks][0], bq[ks][1]);
            }
        } else {
#pragma unroll
            for (int pr = 0; pr < KS / 2; ++pr) {  // 32 bytes of every key row: two k-steps
                uint32_t r[4];                     // rows gq | gq + 8 of bytes [32 pr, +16) | rows gq | gq + 8 of [32 pr + 16, +16)
                ldmatrix_x4(ks_u32 + swz(k_row, 2 * pr + k_chunk), r);
                const uint32_t a0[4] = {bytes_to_f16x2<E5M2, 0, 1>(r[0]), bytes_to_f16x2<E5M2, 0, 1>(r[1]),
                                        bytes_to_f16x2<E5M2, 2, 3>(r[0]), bytes_to_f16x2<E5M2, 2, 3>(r[1])};
                const uint32_t a1[4] = {bytes_to_f16x2<E5M2, 0, 1>(r[2]), bytes_to_f16x2<E5M2, 0, 1>(r[3]),
                                        bytes_to_f16x2<E5M2, 2, 3>(r[2]), bytes_to_f16x2<E5M2, 2, 3>(r[3])};
                mma_f16(ca, a0, bq[2 * pr][0], bq[2 * pr][1]);
                mma_f16(cb, a1, bq[2 * pr + 1][0], bq[2 * pr + 1][1]);
            }
        }
        const int tokA = grp * kGroupTokens + gq, tokB = tokA + 8;
        float s00 = (tokA < n) ? (ca[0] + cb[0]) * sl2_0 : -INFINITY;
        float s01 = (tokA < n) ? (ca[1] + cb[1]) * sl2_1 : -INFINITY;
        float s10 = (tokB < n) ? (ca[2] + cb[2]) * sl2_0 : -INFINITY;
        float s11 = (tokB < n) ? (ca[3] + cb[3]) * sl2_1 : -INFINITY;
        if (2 * tq < GP) {
            *reinterpret_cast<float2*>(lg + (size_t)(tokA - t0) * GP + 2 * tq) = make_float2(s00, s01);
            *reinterpret_cast<float2*>(lg + (size_t)(tokB - t0) * GP + 2 * tq) = make_float2(s10, s11);
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
        if constexpr (!BYTES) {
            const uint32_t pb0 = movmatrix_trans(pack_bf16(p00, p01));
            const uint32_t pb1 = movmatrix_trans(pack_bf16(p10, p11));
#pragma unroll
            for (int mt = 0; mt < KS; ++mt) {
                uint32_t af[4];
                ldmatrix_x4_trans(vs_u32 + v_row * ROW_BYTES + (((2 * mt + v_chunk) ^ (v_row & 7)) << 4), af);
                mma_bf16(o[mt], af, pb0, pb1);
            }
        } else {
            const uint32_t pb0 = movmatrix_trans(pack_f16(p00, p01));
            const uint32_t pb1 = movmatrix_trans(pack_f16(p10, p11));
#pragma unroll
            for (int mt = 0; mt < MT; ++mt) {
                // per register: the byte pairs (d, d + 1) of two consecutive tokens; a byte permute separates even and odd d
                uint32_t r[4];
                ldmatrix_x4_trans(vs_u32 + swz(v_row, 2 * mt + v_chunk), r);
                uint32_t ae[4], ao[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    ae[i] = bytes_to_f16x2<E5M2, 0, 2>(r[i]);
                    ao[i] = bytes_to_f16x2<E5M2, 1, 3>(r[i]);
                }
                mma_f16(o8[mt][0], ae, pb0, pb1);
                mma_f16(o8[mt][1], ao, pb0, pb1);
            }
        }
        __syncwarp();
        const int nxt = it + NSTAGE - 1;
        if (nxt < my_count) issue(my_first + nxt * NW, nxt % NSTAGE);
        cp_async_commit();
    }
    cp_async_wait<0>();
    __syncwarp();
    if (bad_page) record_error(a.status, LETHE_ERR_PAGE, ic.item);

    // ---- this warp's partial result into shared memory (its own stage area doubles as the buffer)
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
        l0 += __shfl_xor_sync(0xffffffffu, l0, off);
        l1 += __shfl_xor_sync(0xffffffffu, l1, off);
    }
    if (gq == 0) {
        ls.wstat[warp][2 * tq] = make_float2(m0, l0);
        ls.wstat[warp][2 * tq + 1] = make_float2(m1, l1);
    }
    float* wo = reinterpret_cast<float*>(my_stage);
    if constexpr (!BYTES) {
#pragma unroll
        for (int mt = 0; mt < KS; ++mt) {
            wo[(2 * tq) * D + 16 * mt + gq] = o[mt][0];
            wo[(2 * tq + 1) * D + 16 * mt + gq] = o[mt][1];
            wo[(2 * tq) * D + 16 * mt + gq + 8] = o[mt][2];
            wo[(2 * tq + 1) * D + 16 * mt + gq + 8] = o[mt][3];
        }
    } else {
        const float vs_l = a.v_scale[ic.l];  // a stored value byte x means v_scale * x
#pragma unroll
        for (int mt = 0; mt < MT; ++mt)
#pragma unroll
            for (int par = 0; par < 2; ++par) {
                const int d = 32 * mt + 2 * gq + par;
                wo[(2 * tq) * D + d] = o8[mt][par][0] * vs_l;
                wo[(2 * tq + 1) * D + d] = o8[mt][par][1] * vs_l;
                wo[(2 * tq) * D + d + 16] = o8[mt][par][2] * vs_l;
                wo[(2 * tq + 1) * D + d + 16] = o8[mt][par][3] * vs_l;
            }
    }
    __syncthreads();   // every warp's (max, sum) and partial output are in shared memory
    cluster_wait();    // every peer has initialised its barrier (they arrived at the top of the kernel)

    // ---- push: this CTA's (max, sum) of every head to every rank; slice r of its partial output to rank r.
    // Each thread derives the CTA-level statistics it needs from the warps' pairs itself (NW shared-memory reads),
    // so nothing but the barrier above precedes the pushes.
    const int total = G * D;
    const int per = (total + S - 1) / S;
    const float* wo_all = reinterpret_cast<const float*>(stage_base);
    constexpr int WO_STRIDE = WARP_BYTES / 4;
    auto cta_max = [&](int h) {
        float m = -INFINITY;
#pragma unroll
        for (int w = 0; w < NW; ++w) m = fmaxf(m, ls.wstat[w][h].x);
        return m;
    };
    for (int i = tid; i < S * kMaxGroup; i += NT) {
        const int r = i / kMaxGroup, h = i % kMaxGroup;
        const float m = cta_max(h);
        float l = 0.f;
#pragma unroll
        for (int w = 0; w < NW; ++w) l += ls.wstat[w][h].y * exp2_diff(ls.wstat[w][h].x, m);
        st_cluster_f2(cluster_map(smem_u32(&ls.peer_stat[ic.rank][h]), (uint32_t)r), make_float2(m, l));
    }
    // four consecutive outputs per thread (one head, one destination rank: D and the slice length are multiples
    // of four): the warps' scales are worked out once, the partial outputs are read and pushed as 16-byte vectors
    for (int idx = 4 * tid; idx < total; idx += 4 * NT) {
        const int h = idx / D;
        const float m = cta_max(h);
        float4 acc = make_float4(0.f, 0.f, 0.f, 0.f);
#pragma unroll
        for (int w = 0; w < NW; ++w) {
            const float sc = exp2_diff(ls.wstat[w][h].x, m);
            const float4 x = *reinterpret_cast<const float4*>(wo_all + w * WO_STRIDE + idx);
            acc.x += x.x * sc; acc.y += x.y * sc; acc.z += x.z * sc; acc.w += x.w * sc;
        }
        const int r = idx / per;
        const uint32_t dst = cluster_map(smem_u32(&ls.peer_o[ic.rank * per + (idx - r * per)]), (uint32_t)r);
        asm volatile("st.shared::cluster.v4.f32 [%0], {%1, %2, %3, %4};" ::"r"(dst), "f"(acc.x), "f"(acc.y), "f"(acc.z), "f"(acc.w) : "memory");
    }
    __syncthreads();  // every thread's pushes are issued; the arrivals below release them cluster-wide
    if (tid < S) {
        asm volatile("fence.acq_rel.cluster;" ::: "memory");
        mbar_remote_arrive(cluster_map(smem_u32(&ls.bar), (uint32_t)tid));
    }
    const int hi_tok = min(t1, n);
    // ---- wait for the peers' pushes (bounded)
    {
        // (always the built-in limit: a CTA that gave up early would exit while its peers may still push to it)
        bool ok = false;
        for (int it = 0; it < kLayerWaitLimit; ++it) {
            if (mbar_try_wait_cluster(&ls.bar, 0u)) {
                ok = true;
                break;
            }
            if (*(volatile int*)&ls.abort) break;
        }
        if (!ok) {
            ls.abort = 1;
            if (tid == 0) record_error(a.status, LETHE_ERR_TIMEOUT, ic.item);
            return;
        }
    }
    // ---- global statistics: every warp works them out for itself (lane = rank * 8 + head covers four ranks per
    // round), so no block-wide barrier follows the wait.  Lane h < 8 ends up with (global max, 1 / global sum) of head h.
    float2 fin[kMaxGroup];
    {
        const int h = lane & 7;
        float m = -INFINITY;
        for (int r = lane >> 3; r < S; r += 4) m = fmaxf(m, ls.peer_stat[r][h].x);
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 8));
        m = fmaxf(m, __shfl_xor_sync(0xffffffffu, m, 16));
        float l = 0.f;
        for (int r = lane >> 3; r < S; r += 4) l += ls.peer_stat[r][h].y * exp2_diff(ls.peer_stat[r][h].x, m);
        l += __shfl_xor_sync(0xffffffffu, l, 8);
        l += __shfl_xor_sync(0xffffffffu, l, 16);
        const float inv = l > 0.f ? 1.f / l : 0.f;
        if (a.lse && warp == 0 && lane < G && ic.rank == 0)
            a.lse[(size_t)(ic.li * a.B + ic.b) * a.Hq + ic.hkv * G + h] = l > 0.f ? (m + log2f(l)) * 0.6931471805599453f : -INFINITY;
#pragma unroll
        for (int hh = 0; hh < kMaxGroup; ++hh) {
            fin[hh].x = __shfl_sync(0xffffffffu, m, hh);
            fin[hh].y = __shfl_sync(0xffffffffu, inv, hh);
        }
    }
    {   // this rank's slice of the outputs
        const int lo = ic.rank * per, hi = min(total, lo + per);
        for (int idx = lo + tid; idx < hi; idx += NT) {
            const int h = idx / D;
            float fm = 0.f, fi = 0.f;
#pragma unroll
            for (int hh = 0; hh < kMaxGroup; ++hh)
                if (hh == h) {
                    fm = fin[hh].x;
                    fi = fin[hh].y;
                }
            float acc = 0.f;
            for (int r = 0; r < S; ++r) acc += ls.peer_o[r * per + (idx - lo)] * exp2_diff(ls.peer_stat[r][h].x, fm);
            out_rows[idx] = __float2bfloat16_rn(acc * fi);
        }
    }
    {   // Eq. 5 for this thread's first tokens, from the logits fetched above; longer ranges take the general loop
        float* rel = a.rel + (size_t)ic.item * a.cap_tokens;
#pragma unroll
        for (int i = 0; i < PF; ++i) {
            const int j = t0 + tid + i * NT;
            if (j < hi_tok) {
                const float* row = lg + (size_t)(j - t0) * GP;
                float mass = 0.f;
#pragma unroll
                for (int h = 0; h < kMaxGroup; ++h)
                    if (h < G) mass += fast_exp2(row[h] - fin[h].x) * fin[h].y;
                rel[j] = fmaf(a.gamma, rel_old[i], mass);
            }
        }
    }
    if (t0 + PF * NT < hi_tok) {  // the rest of a long range: the general batched loop, starting after the tokens done above
        float none[kRelPrefetch];
#pragma unroll
        for (int i = 0; i < kRelPrefetch; ++i) none[i] = 0.f;
        relevance_update<NT, GT>(a, ic, fin, lg + (size_t)PF * NT * GP, t0 + PF * NT, hi_tok, append_slot, none, kRelPrefetch);
    }
    if (append_slot >= 0 && ic.rank == 0 && tid == 0) a.len[ic.item] = n;
}

template <int D, int NW, int NSTAGE, int KV = 0>
static size_t layer_smem(int chunk_tokens, int GP) {
    return (size_t)NW * NSTAGE * 2 * kGroupTokens * D * (KV ? 1 : 2) + sizeof(LayerSmem) + (size_t)chunk_tokens * GP * 4;
}

template <int D, int NW, int NSTAGE, bool PAGED, int GT, int KV = 0>
static cudaError_t launch_layer_t(const AttendArgs& a, cudaStream_t stream) {
    auto kern = attend_layer_kernel<D, NW, NSTAGE, PAGED, GT, KV>;
    const size_t smem = layer_smem<D, NW, NSTAGE, KV>(a.chunk_tokens, a.GP);
    cudaError_t e = prepare_kernel((const void*)kern, smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(a.n_items * a.splits), 1, 1);
    cfg.blockDim = dim3(NW * 32, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)a.splits;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, a);
}

// Kernel shapes (warps per CTA, pipeline stages per warp), selected by `shape`.
#define LETHE_LAYER_SHAPES(X, D) \
    X(0, D, 4, 3) X(1, D, 8, 3) X(2, D, 4, 2) X(3, D, 8, 2) X(4, D, 4, 4) X(5, D, 2, 4)

size_t layer_smem_bytes(int D, int shape, int chunk_tokens, int GP) {
#define X(id, DD, NW, NS) \
    if (shape == id && D == DD) return layer_smem<DD, NW, NS>(chunk_tokens, GP);
    LETHE_LAYER_SHAPES(X, 128)
    LETHE_LAYER_SHAPES(X, 64)
#undef X
    return (size_t)-1;
}

cudaError_t launch_attend_layer(const AttendArgs& a, int D, int shape, bool paged, cudaStream_t stream) {
    // the automatic choices for the two common geometries with their group size compiled in
    if (D == 128 && shape == 0 && a.G == 4)
        return paged ? launch_layer_t<128, 4, 3, true, 4>(a, stream) : launch_layer_t<128, 4, 3, false, 4>(a, stream);
    if (D == 128 && shape == 2 && a.G == 7)
        return paged ? launch_layer_t<128, 4, 2, true, 7>(a, stream) : launch_layer_t<128, 4, 2, false, 7>(a, stream);
#define X(id, DD, NW, NS)                                                                    \
    if (shape == id && D == DD)                                                              \
        return paged ? launch_layer_t<DD, NW, NS, true, 0>(a, stream) : launch_layer_t<DD, NW, NS, false, 0>(a, stream);
    LETHE_LAYER_SHAPES(X, 128)
    LETHE_LAYER_SHAPES(X, 64)
#undef X
    return cudaErrorInvalidValue;
}

// Quantised caches: 4 warps x 4 stages (a stage is half the bytes of a bf16 one), head_dim 128.
size_t kv8_layer_smem_bytes(int chunk_tokens, int GP) { return layer_smem<128, 4, 4, 1>(chunk_tokens, GP); }

cudaError_t launch_attend_kv8_layer(const AttendArgs& a, bool paged, bool e5m2, cudaStream_t stream) {
#define LETHE_L8(GT)                                                                                                   \
    (paged ? (e5m2 ? launch_layer_t<128, 4, 4, true, GT, 2>(a, stream) : launch_layer_t<128, 4, 4, true, GT, 1>(a, stream))   \
           : (e5m2 ? launch_layer_t<128, 4, 4, false, GT, 2>(a, stream) : launch_layer_t<128, 4, 4, false, GT, 1>(a, stream)))
    if (a.G == 4) return LETHE_L8(4);
    return LETHE_L8(0);
#undef LETHE_L8
}

}  // namespace lethe
