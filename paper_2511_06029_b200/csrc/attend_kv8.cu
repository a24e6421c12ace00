// Decode-attend kernel for quantised caches: K and V stored as e4m3 or e5m2 bytes with one scale per layer (a
// stored byte x means scale * x), q / k_new / v_new / out in bf16.  D in {64, 128}, G <= 8, contiguous or 16-token pages.
//
// Same structure as the clustered bf16 kernel (tokens on the M axis of mma.m16n8k16, the group's heads on N, one
// private cp.async pipeline per warp, logits parked in shared memory, CTAs of an item merged through distributed
// shared memory, common relevance epilogue); what differs is how fragments are made from bytes:
//   S^T = K . Q^T   ldmatrix (b16 view) hands each thread four consecutive bytes of a key row per register; they
//                   become two f16x2 A registers.  The contraction index is therefore permuted inside each 32-byte
//                   step (thread t holds d = 4 t .. 4 t + 3 of both 16-byte halves); the Q^T fragments, converted
//                   once per item from bf16 to f16, are loaded with the same permutation, so the sum is unchanged.
//   O^T += V^T P^T  ldmatrix.trans (b16 view) hands each thread, per register, the byte pairs (d, d + 1) of two
//                   consecutive tokens; a byte permute separates even and odd d, giving the A fragments of two
//                   MMAs whose rows are the even and the odd dimensions of a 32-wide block.  Only the bookkeeping
//                   of which accumulator row is which dimension changes.
// Byte -> f16 is exact (a conversion instruction per pair for e4m3, for e5m2 the byte permute alone: an e5m2 byte is
// the upper byte of the half of the same value); the MMAs run in f16 with fp32 accumulation; P is rounded to f16.  The layer's key scale is
// folded into the softmax scale on the host, the value scale multiplies the warp's partial output once.
// Appending quantises: x / scale in fp32 (IEEE division), round to nearest even, saturate at +-448.
#include <cuda_fp16.h>

#include "common.cuh"
#include "kv8_utils.cuh"
#include "mma_utils.cuh"

namespace lethe {

template <int D, int NW, int NSTAGE, bool PAGED, bool E5M2>
__global__ void __launch_bounds__(NW * 32) attend_kv8_kernel(const __grid_constant__ AttendArgs a) {
    using T = __nv_bfloat16;                               // type of q, k_new, v_new, out
    constexpr int ROW_BYTES = D;                           // one byte per element
    constexpr int CHUNKS = ROW_BYTES / 16;                 // 16-byte chunks per row: 8 or 4
    constexpr int ROWS_PER_LINE = 128 / ROW_BYTES;         // rows sharing a 128-byte line of shared memory
    constexpr int TILE_BYTES = kGroupTokens * ROW_BYTES;   // one group of K (or V)
    constexpr int STAGE_BYTES = 2 * TILE_BYTES;
    constexpr int WARP_BYTES = NSTAGE * STAGE_BYTES;
    constexpr int KS = D / 16;                             // k-steps of the logit MMAs
    constexpr int MT = D / 32;                             // 32-wide blocks of the output dimension
    static_assert(WARP_BYTES >= kMaxGroup * D * 4, "per-warp stage area doubles as the partial-output buffer");
    extern __shared__ __align__(128) unsigned char smem_raw[];
    // layout: stages [NW][NSTAGE][K tile | V tile] | cta_o [kMaxGroup][D] | EpilogueSmem | lg [chunk_tokens][GP]
    unsigned char* stage_base = smem_raw;
    float* cta_o = reinterpret_cast<float*>(smem_raw + (size_t)NW * WARP_BYTES);
    EpilogueSmem& es = *reinterpret_cast<EpilogueSmem*>(cta_o + kMaxGroup * D);
    float* lg = reinterpret_cast<float*>(reinterpret_cast<unsigned char*>(&es) + sizeof(EpilogueSmem));

    // bank-conflict-free placement of 16-byte chunk c of row r: the eight rows an ldmatrix touches land in eight
    // different chunk positions of their 128-byte lines
    auto swz = [](int r, int c) -> uint32_t {
        return (uint32_t)(r * ROW_BYTES + ((c ^ ((r / ROWS_PER_LINE) & (CHUNKS - 1))) << 4));
    };

    const ItemCoord ic = decode_item(a);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int gq = lane >> 2, tq = lane & 3;  // fragment coordinates: row group, column pair
    const int G = a.G, GP = a.GP;
    const bool append = a.k_new != nullptr;
    const int n_old = a.len[ic.item];
    // Q^T fragments (B operand) in f16, in the permuted order of the key bytes: step ks covers d = 16 ks .. + 15,
    // b0 = Q[head gq][16 ks + 4 tq + {0, 1}], b1 = Q[head gq][16 ks + 4 tq + {2, 3}]
    // f16 holds 6e-8 .. 65504, so the row of head gq is first divided by the power of two that brings its largest
    // magnitude into [128, 256) (exact); qdiv is that divisor, and the head's logits are multiplied back below.
    uint32_t bq[KS][2];
    float qdiv = 1.f;
    {
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
    // Sec. 4.1: append the generated token's key / value, quantised; the CTA whose range holds slot n_old stores it.
    if (append && n_old >= t0 && n_old < t1 && warp == 0) {
        const size_t src = ((size_t)(ic.li * a.B + ic.b) * a.Hkv + ic.hkv) * D;  // elements
        char* kd = const_cast<char*>(row_ptr<PAGED>(a, a.k, ic.item, n_old, ROW_BYTES, &bad_page));
        char* vd = const_cast<char*>(row_ptr<PAGED>(a, a.v, ic.item, n_old, ROW_BYTES, &bad_page));
        if (kd && vd && lane * 4 < D) {  // four elements per lane
            const float ks_l = a.k_scale[ic.l], vs_l = a.v_scale[ic.l];
            const uint2 kw = *reinterpret_cast<const uint2*>((const T*)a.k_new + src + lane * 4);
            const uint2 vw = *reinterpret_cast<const uint2*>((const T*)a.v_new + src + lane * 4);
            auto quant4 = [](uint2 w, float s) -> uint32_t {
                const float x0 = __uint_as_float(w.x << 16), x1 = __uint_as_float(w.x & 0xffff0000u);
                const float x2 = __uint_as_float(w.y << 16), x3 = __uint_as_float(w.y & 0xffff0000u);
                return f32x2_to_fp8x2<E5M2>(__fdiv_rn(x0, s), __fdiv_rn(x1, s)) | (f32x2_to_fp8x2<E5M2>(__fdiv_rn(x2, s), __fdiv_rn(x3, s)) << 16);
            };
            *reinterpret_cast<uint32_t*>(kd + lane * 4) = quant4(kw, ks_l);
            *reinterpret_cast<uint32_t*>(vd + lane * 4) = quant4(vw, vs_l);
        }
        if (lane == 0) a.pos[(size_t)ic.item * a.cap_tokens + n_old] = a.token_pos[ic.b];
    }
    __syncthreads();  // the appended row is in global memory before any warp streams it

    const float sl2 = a.scale_log2[ic.l];  // softmax scale x key scale x log2(e)
    // this thread's two logit columns are heads 2 tq and 2 tq + 1: their divisors sit in the lanes with gq = head
    const float sl2_0 = sl2 * __shfl_sync(0xffffffffu, qdiv, (2 * tq) * 4), sl2_1 = sl2 * __shfl_sync(0xffffffffu, qdiv, (2 * tq + 1) * 4);

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
            const uint32_t doff = swz(r, c);
            cp_async16_hint(ks_u32 + doff, kb + soff, valid ? 16 : 0, stream_policy);
            cp_async16_hint(vs_u32 + doff, vb + soff, valid ? 16 : 0, stream_policy);
        }
    };

    float m0 = -INFINITY, m1 = -INFINITY;  // running max of heads 2tq, 2tq+1 (log2 units)
    float l0 = 0.f, l1 = 0.f;              // this thread's share of the running sums
    // O^T fragments: block mt, parity par: rows gq / gq + 8 are d = 32 mt + 2 gq + par and d + 16; heads 2tq, 2tq+1
    float o[MT][2][4];
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int par = 0; par < 2; ++par)
#pragma unroll
            for (int i = 0; i < 4; ++i) o[mt][par][i] = 0.f;

    const int my_first = g_begin + warp;
    const int my_count = (g_end > my_first) ? (g_end - my_first + NW - 1) / NW : 0;
#pragma unroll
    for (int s = 0; s < NSTAGE - 1; ++s) {
        if (s < my_count) issue(my_first + s * NW, s);
        cp_async_commit();
    }

    // ldmatrix lane addressing (row within the 16-token group, 16-byte chunk inside a 32-byte step)
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
        const int tokA = grp * kGroupTokens + gq, tokB = tokA + 8;
        float s00 = (tokA < n) ? (ca[0] + cb[0]) * sl2_0 : -INFINITY;  // token A, head 2tq
        float s01 = (tokA < n) ? (ca[1] + cb[1]) * sl2_1 : -INFINITY;  // token A, head 2tq+1
        float s10 = (tokB < n) ? (ca[2] + cb[2]) * sl2_0 : -INFINITY;
        float s11 = (tokB < n) ? (ca[3] + cb[3]) * sl2_1 : -INFINITY;
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
            for (int mt = 0; mt < MT; ++mt)
#pragma unroll
                for (int par = 0; par < 2; ++par) {
                    o[mt][par][0] *= c0; o[mt][par][2] *= c0;
                    o[mt][par][1] *= c1; o[mt][par][3] *= c1;
                }
            m0 = mn0;
            m1 = mn1;
        }
        const float p00 = fast_exp2(s00 - m0), p01 = fast_exp2(s01 - m1);
        const float p10 = fast_exp2(s10 - m0), p11 = fast_exp2(s11 - m1);
        l0 += p00 + p10;
        l1 += p01 + p11;
        // P^T as B operand (f16): transpose the two 8x8 (token x head) blocks across the warp
        const uint32_t pb0 = movmatrix_trans(pack_f16(p00, p01));
        const uint32_t pb1 = movmatrix_trans(pack_f16(p10, p11));
#pragma unroll
        for (int mt = 0; mt < MT; ++mt) {
            // registers: tokens 2tq, 2tq+1 (r[0], r[1]) and 2tq+8, 2tq+9 (r[2], r[3]); bytes (d, d+1) with
            // d = 32 mt + 2 gq (r[0], r[2]) and d + 16 (r[1], r[3]); per register: {tok: d, d+1}, {tok+1: d, d+1}
            uint32_t r[4];
            ldmatrix_x4_trans(vs_u32 + swz(v_row, 2 * mt + v_chunk), r);
            uint32_t ae[4], ao[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                ae[i] = bytes_to_f16x2<E5M2, 0, 2>(r[i]);  // even d: bytes 0 and 2 (tokens t, t+1)
                ao[i] = bytes_to_f16x2<E5M2, 1, 3>(r[i]);  // odd d:  bytes 1 and 3
            }
            mma_f16(o[mt][0], ae, pb0, pb1);
            mma_f16(o[mt][1], ao, pb0, pb1);
        }
        __syncwarp();  // every lane is done reading slot s before it is refilled
        const int nxt = it + NSTAGE - 1;
        if (nxt < my_count) issue(my_first + nxt * NW, nxt % NSTAGE);
        cp_async_commit();
    }
    float rel_old[kRelPrefetch];
    prefetch_rel<NW * 32>(a, ic, t0, min(t1, n), append_slot, rel_old);
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
    const float vs_l = a.v_scale[ic.l];  // a stored value byte x means v_scale * x
    float* wo = reinterpret_cast<float*>(my_stage);
#pragma unroll
    for (int mt = 0; mt < MT; ++mt)
#pragma unroll
        for (int par = 0; par < 2; ++par) {
            const int d = 32 * mt + 2 * gq + par;
            wo[(2 * tq) * D + d] = o[mt][par][0] * vs_l;
            wo[(2 * tq + 1) * D + d] = o[mt][par][1] * vs_l;
            wo[(2 * tq) * D + d + 16] = o[mt][par][2] * vs_l;
            wo[(2 * tq + 1) * D + d + 16] = o[mt][par][3] * vs_l;
        }
    combine_and_finish<T, D, NW>(a, ic, es, reinterpret_cast<float*>(stage_base), WARP_BYTES / 4, cta_o, lg, t0, t1,
                                 append_slot, n, rel_old);
}

template <int D, int NW, int NSTAGE>
static size_t kv8_smem(int chunk_tokens, int GP) {
    return (size_t)NW * NSTAGE * 2 * kGroupTokens * D + (size_t)kMaxGroup * D * 4 + sizeof(EpilogueSmem) +
           (size_t)chunk_tokens * GP * 4;
}

template <int D, int NW, int NSTAGE, bool PAGED, bool E5M2>
static cudaError_t launch_kv8_t(const AttendArgs& a, cudaStream_t stream) {
    auto kern = attend_kv8_kernel<D, NW, NSTAGE, PAGED, E5M2>;
    const size_t smem = kv8_smem<D, NW, NSTAGE>(a.chunk_tokens, a.GP);
    cudaError_t e = prepare_kernel((const void*)kern, smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)(a.n_items * a.splits), 1, 1);
    cfg.blockDim = dim3(NW * 32, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = (unsigned)a.splits;
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, a);
}

// Kernel shapes (warps per CTA, pipeline stages per warp), selected by `shape`: tiles are half the size of the bf16
// kernel's, so the pipelines are deeper.
#define LETHE_KV8_SHAPES(X, D) X(0, D, 4, 4) X(1, D, 8, 4) X(2, D, 4, 2) X(3, D, 4, 3) X(4, D, 2, 4) X(5, D, 8, 2)

size_t kv8_smem_bytes(int D, int shape, int chunk_tokens, int GP) {
#define X(id, DD, NW, NS) \
    if (shape == id && D == DD) return kv8_smem<DD, NW, NS>(chunk_tokens, GP);
    LETHE_KV8_SHAPES(X, 128)
    LETHE_KV8_SHAPES(X, 64)
#undef X
    return (size_t)-1;
}

cudaError_t launch_attend_kv8(const AttendArgs& a, int D, int shape, bool paged, bool e5m2, cudaStream_t stream) {
#define X(id, DD, NW, NS)                                                                                           \
    if (shape == id && D == DD) {                                                                                   \
        if (e5m2) return paged ? launch_kv8_t<DD, NW, NS, true, true>(a, stream) : launch_kv8_t<DD, NW, NS, false, true>(a, stream); \
        return paged ? launch_kv8_t<DD, NW, NS, true, false>(a, stream) : launch_kv8_t<DD, NW, NS, false, false>(a, stream);         \
    }
    LETHE_KV8_SHAPES(X, 128)
    LETHE_KV8_SHAPES(X, 64)
#undef X
    return cudaErrorInvalidValue;
}

}  // namespace lethe
