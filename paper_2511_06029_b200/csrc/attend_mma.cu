// Tensor-core decode-attend kernel for bf16 caches (D in {64, 128}, G <= 8), contiguous or 16-token pages.
//
// The work is an HBM stream, not a dense contraction: per token one K row and one V row are read once and
// used by the G query heads of the group.  Tensor cores are used only to take the per-token arithmetic off
// the issue slots: tokens sit on the M axis of mma.m16n8k16 and the (at most 8) heads of the group on N, so
//     S^T[16 tok x 8 heads] = K[16 tok x D] . Q^T[D x 8 heads]          (D/16 mma)
//     O^T[D x 8 heads]     += V^T[D x 16 tok] . P^T[16 tok x 8 heads]   (D/16 mma)
// i.e. one mma per token.  Each warp owns a private multi-stage cp.async pipeline over its own 16-token
// groups (group i of the CTA's range goes to warp i mod NW), so the main loop has no block-level barrier.
// Rows are staged with a 16-byte-chunk XOR swizzle so that both ldmatrix (K) and ldmatrix.trans (V) are
// bank-conflict free.  Scaled logits of every token are parked in shared memory (G floats per token); once
// the exact softmax normaliser of each head is known (after merging warps and, through distributed shared
// memory, the CTAs of the item's cluster) the common epilogue turns them into the Eq. 5 relevance update —
// no second pass over K and no scratch in global memory.
#include "common.cuh"
#include "mma_utils.cuh"

namespace lethe {

template <int D, int NW, int NSTAGE, bool PAGED, bool FLAT>
__global__ void __launch_bounds__(NW * 32) attend_mma_kernel(const __grid_constant__ AttendArgs a) {
    using T = __nv_bfloat16;
    constexpr int ROW_BYTES = D * 2;
    constexpr int CHUNKS = ROW_BYTES / 16;           // 16-byte chunks per row
    constexpr int TILE_BYTES = kGroupTokens * ROW_BYTES;  // one group of K (or V)
    constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    constexpr int WARP_BYTES = NSTAGE * STAGE_BYTES;
    constexpr int KS = D / 16;
    static_assert(WARP_BYTES >= kMaxGroup * D * 4, "per-warp stage area doubles as the partial-output buffer");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    // layout: stages [NW][NSTAGE][K tile | V tile] | cta_o [kMaxGroup][D] | EpilogueSmem | lg [chunk_tokens][GP]
    unsigned char* stage_base = smem_raw;
    float* cta_o = reinterpret_cast<float*>(smem_raw + (size_t)NW * WARP_BYTES);
    EpilogueSmem& es = *reinterpret_cast<EpilogueSmem*>(cta_o + kMaxGroup * D);
    float* lg = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(&es) + sizeof(EpilogueSmem));

    // Programmatic dependent launch: when the launch carries the attribute this CTA may have been scheduled while
    // the previous kernel of the stream was still draining; everything it reads may come from that kernel, so it
    // waits here for it to complete (a no-op for ordinary launches).
    asm volatile("griddepcontrol.wait;" ::: "memory");
    const ItemCoord ic = decode_item(a);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int gq = lane >> 2, tq = lane & 3;  // fragment coordinates: row group, column pair
    const int G = a.G, GP = a.GP;
    const bool append = a.k_new != nullptr;
    const int n_old = a.len[ic.item];
    // Q^T fragments (B operand): b0 = Q[head gq][16 ks + 2 tq, +1], b1 = Q[head gq][16 ks + 8 + 2 tq, +1]
    uint32_t bq[KS][2];
    {
        const uint32_t* qrow =
            reinterpret_cast<const uint32_t*>((const T*)a.q + ((size_t)(ic.li * a.B + ic.b) * a.Hq + ic.hkv * G + gq) * D);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            bq[ks][0] = (gq < G) ? qrow[8 * ks + tq] : 0u;
            bq[ks][1] = (gq < G) ? qrow[8 * ks + 4 + tq] : 0u;
        }
    }
    T* out_rows = (T*)a.out + ((size_t)(ic.li * a.B + ic.b) * a.Hq + ic.hkv * G) * D;
    if (append && n_old >= a.cap_tokens) {  // full: leave the item untouched (every CTA of the cluster returns)
        if (ic.rank == 0) {
            for (int i = tid; i < G * D; i += NW * 32) out_rows[i] = __float2bfloat16_rn(0.f);
            if (a.lse && tid < G) a.lse[(size_t)(ic.li * a.B + ic.b) * a.Hq + ic.hkv * G + tid] = -INFINITY;
            if (tid == 0) record_error(a.status, LETHE_ERR_CAPACITY, ic.item);
        }
        return;
    }
    const int n = n_old + (append ? 1 : 0);
    const int append_slot = append ? n_old : -1;
    int g_begin, g_end;
    split_range(n, a.splits, ic.rank, g_begin, g_end);
    const int t0 = g_begin * kGroupTokens, t1 = g_end * kGroupTokens;

    bool bad_page = false;
    const uint64_t stream_policy = l2_evict_first_policy();  // K / V tiles are read once: evict-first in L2
    // Sec. 4.1: append the generated token's key / value; the CTA whose range holds slot n_old stores it.
    if (append && n_old >= t0 && n_old < t1 && warp == 0) {
        const size_t src = ((size_t)(ic.li * a.B + ic.b) * a.Hkv + ic.hkv) * ROW_BYTES;
        char* kd = const_cast<char*>(row_ptr<PAGED>(a, a.k, ic.item, n_old, ROW_BYTES, &bad_page));
        char* vd = const_cast<char*>(row_ptr<PAGED>(a, a.v, ic.item, n_old, ROW_BYTES, &bad_page));
        if (kd && vd && lane * 16 < ROW_BYTES) {
            *reinterpret_cast<uint4*>(kd + lane * 16) = *reinterpret_cast<const uint4*>((const char*)a.k_new + src + lane * 16);
            *reinterpret_cast<uint4*>(vd + lane * 16) = *reinterpret_cast<const uint4*>((const char*)a.v_new + src + lane * 16);
        }
        if (lane == 0) a.pos[(size_t)ic.item * a.cap_tokens + n_old] = a.token_pos[ic.b];
    }
    __syncthreads();  // the appended row is in global memory before any warp streams it

    const float sl2 = a.scale_log2[ic.l];

    unsigned char* my_stage = stage_base + (size_t)warp * WARP_BYTES;
    const uint32_t my_stage_u32 = smem_u32(my_stage);

    // issue the copies of group `grp` into stage slot `s`
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
            const int soff = valid ? r * ROW_BYTES + c * 16 : 0;  // rows past n are zero-filled, never read
            const uint32_t doff = r * ROW_BYTES + ((c ^ (r & 7)) << 4);
            cp_async16_hint(ks_u32 + doff, kb + soff, valid ? 16 : 0, stream_policy);
            cp_async16_hint(vs_u32 + doff, vb + soff, valid ? 16 : 0, stream_policy);
        }
    };

    float m0 = -INFINITY, m1 = -INFINITY;  // running max of heads 2tq, 2tq+1 (log2 units)
    float l0 = 0.f, l1 = 0.f;              // this thread's share of the running sums
    float o[KS][4];                        // O^T fragments: d = 16 mt + gq (+8), heads 2tq, 2tq+1
#pragma unroll
    for (int mt = 0; mt < KS; ++mt)
#pragma unroll
        for (int i = 0; i < 4; ++i) o[mt][i] = 0.f;

    const int my_first = g_begin + warp;
    const int my_count = (g_end > my_first) ? (g_end - my_first + NW - 1) / NW : 0;
#pragma unroll
    for (int s = 0; s < NSTAGE - 1; ++s) {
        if (s < my_count) issue(my_first + s * NW, s);
        cp_async_commit();
    }

    // ldmatrix lane addressing (row within the 16-token group, chunk offset inside a 32-byte k-step)
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
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            uint32_t af[4];
            ldmatrix_x4(ks_u32 + k_row * ROW_BYTES + (((2 * ks + k_chunk) ^ (k_row & 7)) << 4), af);
            if (ks & 1) mma_bf16(cb, af, bq[ks][0], bq[ks][1]);
            else mma_bf16(ca, af, bq[ks][0], bq[ks][1]);
        }
        const int tokA = grp * kGroupTokens + gq, tokB = tokA + 8;
        float s00 = (tokA < n) ? (ca[0] + cb[0]) * sl2 : -INFINITY;  // token A, head 2tq
        float s01 = (tokA < n) ? (ca[1] + cb[1]) * sl2 : -INFINITY;  // token A, head 2tq+1
        float s10 = (tokB < n) ? (ca[2] + cb[2]) * sl2 : -INFINITY;
        float s11 = (tokB < n) ? (ca[3] + cb[3]) * sl2 : -INFINITY;
        if (2 * tq < GP) {
            float2* row = reinterpret_cast<float2*>(lg + (size_t)(tokA - t0) * GP + 2 * tq);
            row[0] = make_float2(s00, s01);
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
        // P^T as B operand: transpose the two 8x8 (token x head) blocks across the warp
        const uint32_t pb0 = movmatrix_trans(pack_bf16(p00, p01));
        const uint32_t pb1 = movmatrix_trans(pack_bf16(p10, p11));
#pragma unroll
        for (int mt = 0; mt < KS; ++mt) {
            uint32_t af[4];
            ldmatrix_x4_trans(vs_u32 + v_row * ROW_BYTES + (((2 * mt + v_chunk) ^ (v_row & 7)) << 4), af);
            mma_bf16(o[mt], af, pb0, pb1);
        }
        __syncwarp();  // every lane is done reading slot s before it is refilled
        const int nxt = it + NSTAGE - 1;
        if (nxt < my_count) issue(my_first + nxt * NW, nxt % NSTAGE);
        cp_async_commit();
    }
    // the streaming part is over: let the next kernel of the stream be scheduled onto the SMs as they free up
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    float rel_old[kRelPrefetch];
    if constexpr (!FLAT) prefetch_rel<NW * 32>(a, ic, t0, min(t1, n), append_slot, rel_old);
    cp_async_wait<0>();
    __syncwarp();
    if (bad_page) record_error(a.status, LETHE_ERR_PAGE, ic.item);

    // hand the warp's partial result to the common epilogue (its own stage area doubles as the buffer)
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
        l0 += __shfl_xor_sync(0xffffffffu, l0, off);
        l1 += __shfl_xor_sync(0xffffffffu, l1, off);
    }
    if (gq == 0) {
        es.wstat[warp][2 * tq] = make_float2(m0, l0);
        es.wstat[warp][2 * tq + 1] = make_float2(m1, l1);
    }
    float* wo = reinterpret_cast<float*>(my_stage);
#pragma unroll
    for (int mt = 0; mt < KS; ++mt) {
        wo[(2 * tq) * D + 16 * mt + gq] = o[mt][0];
        wo[(2 * tq + 1) * D + 16 * mt + gq] = o[mt][1];
        wo[(2 * tq) * D + 16 * mt + gq + 8] = o[mt][2];
        wo[(2 * tq + 1) * D + 16 * mt + gq + 8] = o[mt][3];
    }
    if constexpr (FLAT)
        flat_finish<T, D, NW>(a, ic, es, reinterpret_cast<float*>(stage_base), WARP_BYTES / 4, cta_o, lg, t0, t1, append_slot, n);
    else
        combine_and_finish<T, D, NW>(a, ic, es, reinterpret_cast<float*>(stage_base), WARP_BYTES / 4, cta_o, lg, t0, t1,
                                     append_slot, n, rel_old);
}

template <int D, int NW, int NSTAGE>
static size_t mma_smem(int chunk_tokens, int GP) {
    return (size_t)NW * NSTAGE * 2 * kGroupTokens * D * 2 + (size_t)kMaxGroup * D * 4 + sizeof(EpilogueSmem) +
           (size_t)chunk_tokens * GP * 4;
}

template <int D, int NW, int NSTAGE, bool PAGED, bool FLAT>
static cudaError_t launch_mma_t(const AttendArgs& a, cudaStream_t stream) {
    auto kern = attend_mma_kernel<D, NW, NSTAGE, PAGED, FLAT>;
    const size_t smem = mma_smem<D, NW, NSTAGE>(a.chunk_tokens, a.GP);
    cudaError_t e = prepare_kernel((const void*)kern, smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(a.n_items * a.splits), 1, 1);
    cfg.blockDim = dim3(NW * 32, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = FLAT ? 1u : (unsigned)a.splits;  // scratch-merged mode needs no co-scheduling
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // launches of this kernel may overlap their scheduling with the tail of the previous kernel in the stream
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 2;
    return cudaLaunchKernelEx(&cfg, kern, a);
}

template <int D, int NW, int NS>
static cudaError_t dispatch_mma(const AttendArgs& a, bool paged, cudaStream_t stream) {
    const bool flat = a.flat_cnt != nullptr;
    if (paged) return flat ? launch_mma_t<D, NW, NS, true, true>(a, stream) : launch_mma_t<D, NW, NS, true, false>(a, stream);
    return flat ? launch_mma_t<D, NW, NS, false, true>(a, stream) : launch_mma_t<D, NW, NS, false, false>(a, stream);
}

// Kernel shapes (warps per CTA, pipeline stages per warp), selected by `shape`.
#define LETHE_MMA_SHAPES(X, D) \
    X(0, D, 4, 3) X(1, D, 8, 3) X(2, D, 4, 2) X(3, D, 8, 2) X(4, D, 4, 4) X(5, D, 2, 4)

size_t mma_smem_bytes(int D, int shape, int chunk_tokens, int GP) {
#define X(id, DD, NW, NS) \
    if (shape == id && D == DD) return mma_smem<DD, NW, NS>(chunk_tokens, GP);
    LETHE_MMA_SHAPES(X, 128)
    LETHE_MMA_SHAPES(X, 64)
#undef X
    return (size_t)-1;
}

cudaError_t launch_attend_mma(const AttendArgs& a, int D, int shape, bool paged, cudaStream_t stream) {
#define X(id, DD, NW, NS)                                                                           \
    if (shape == id && D == DD)                                                                     \
        return dispatch_mma<DD, NW, NS>(a, paged, stream);
    LETHE_MMA_SHAPES(X, 128)
    LETHE_MMA_SHAPES(X, 64)
#undef X
    return cudaErrorInvalidValue;
}

}  // namespace lethe
