// Relevance of the prompt tokens from the prefill attention (Eq. 2 with Q > 1, folded through Eq. 5):
//   rel[j] = sum_{i >= j} gamma^(P-1-i) sum_{h in group} softmax_{j' <= i}(scale q_{i,h} . K_{j'})[j]      (j < P)
// Unlike the decode path this is a dense contraction (every prompt query against every earlier key), done on the
// tensor cores with the same operand orientation as the decode kernels: keys on the M axis of mma.m16n8k16, eight
// (query, head) columns on N.  Two kernels, both deterministic (no floating-point atomics):
//   prefill_stats_kernel   each warp owns eight columns, walks the keys 0..i and keeps the online (max, sum) of
//                          every column; result to scratch [item][P][HP]
//   prefill_colsum_kernel  each warp owns sixteen keys (A fragments stay in registers), walks the columns with
//                          query >= key, turns logits into probabilities with the stored statistics and the decay
//                          weight, and accumulates the column sums of its keys; result to rel
// Columns are laid out query-major with the G heads of the group padded to HP = 1, 2, 4 or 8.
#include "common.cuh"
#include "mma_utils.cuh"
#include "prefill.cuh"

namespace lethe {

constexpr int kPrefillWarps = 8;
constexpr int kPrefillKeyTile = 64;  // keys per staged tile in the statistics kernel

// Stage `rows` key rows starting at slot j0 into a swizzled tile (16-byte chunk index XOR (row & 7)); rows at or
// beyond `limit` are zero-filled.  All threads of the CTA take part.
template <int D>
__device__ __forceinline__ void stage_keys(const PrefillArgs& a, int item, int j0, int rows, int limit, uint32_t tile_u32) {
    constexpr int ROW_BYTES = D * 2, CHUNKS = ROW_BYTES / 16;
    for (int idx = threadIdx.x; idx < rows * CHUNKS; idx += kPrefillWarps * 32) {
        const int r = idx / CHUNKS, c = idx % CHUNKS;
        const int j = j0 + r;
        const bool valid = j < limit;
        const char* src = prefill_row(a, item, valid ? j : 0, ROW_BYTES) + c * 16;
        cp_async16(tile_u32 + r * ROW_BYTES + ((c ^ (r & 7)) << 4), src, valid ? 16 : 0);
    }
}

template <int D>
__global__ void __launch_bounds__(kPrefillWarps * 32) prefill_stats_kernel(const __grid_constant__ PrefillArgs a) {
    using T = __nv_bfloat16;
    constexpr int ROW_BYTES = D * 2, KS = D / 16;
    __shared__ __align__(128) unsigned char tiles[2][kPrefillKeyTile * ROW_BYTES];
    const int item = blockIdx.y;
    const int hkv = item % a.Hkv, b = (item / a.Hkv) % a.B, l = item / (a.Hkv * a.B);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31, gq = lane >> 2, tq = lane & 3;
    const int P = a.P, HP = a.HP, QW = 8 / HP;
    if (a.len[item] < P) {
        if (threadIdx.x == 0 && blockIdx.x == 0) record_error(a.status, LETHE_ERR_CAPACITY, item);
        return;
    }
    const int q0w = (blockIdx.x * kPrefillWarps + warp) * QW;  // first query of this warp's eight columns
    // B operand: column gq of the block = (query q0w + gq / HP, head gq % HP)
    uint32_t bq[KS][2];
    {
        const int qi = q0w + gq / HP, h = gq % HP;
        const bool ok = qi < P && h < a.G;
        const uint32_t* qrow = reinterpret_cast<const uint32_t*>(
            (const T*)a.q + ((((size_t)l * a.B + b) * P + (ok ? qi : 0)) * a.Hq + hkv * a.G + (ok ? h : 0)) * D);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
            bq[ks][0] = ok ? qrow[8 * ks + tq] : 0u;
            bq[ks][1] = ok ? qrow[8 * ks + 4 + tq] : 0u;
        }
    }
    const float sl2 = a.scale_log2[l];
    const int qA = q0w + (2 * tq) / HP, qB = q0w + (2 * tq + 1) / HP;  // queries of this thread's two columns
    const int q_hi_warp = min(P - 1, q0w + QW - 1);
    const int q_hi_cta = min(P - 1, (int)(blockIdx.x + 1) * kPrefillWarps * QW - 1);
    const int n_tiles = q_hi_cta / kPrefillKeyTile + 1;
    float mA = -INFINITY, lA = 0.f, mB = -INFINITY, lB = 0.f;
    const int k_row = (lane & 7) + ((lane >> 3) & 1) * 8, k_chunk = lane >> 4;

    stage_keys<D>(a, item, 0, kPrefillKeyTile, P, smem_u32(tiles[0]));
    cp_async_commit();
    for (int t = 0; t < n_tiles; ++t) {
        if (t + 1 < n_tiles) stage_keys<D>(a, item, (t + 1) * kPrefillKeyTile, kPrefillKeyTile, P, smem_u32(tiles[(t + 1) & 1]));
        cp_async_commit();
        cp_async_wait<1>();
        __syncthreads();
        const uint32_t tile = smem_u32(tiles[t & 1]);
        if (t * kPrefillKeyTile <= q_hi_warp && q0w < P) {  // causal: later tiles hold no key this warp's queries see
#pragma unroll
            for (int mt = 0; mt < kPrefillKeyTile / 16; ++mt) {
                float c[4] = {0.f, 0.f, 0.f, 0.f};
                const int r = 16 * mt + k_row;
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    uint32_t af[4];
                    ldmatrix_x4(tile + r * ROW_BYTES + (((2 * ks + k_chunk) ^ (r & 7)) << 4), af);
                    mma_bf16(c, af, bq[ks][0], bq[ks][1]);
                }
                const int j0 = t * kPrefillKeyTile + 16 * mt + gq, j1 = j0 + 8;
                auto upd = [&](float s, int j, int qi, float& m, float& lsum) {
                    if (j <= qi && qi < P) {
                        const float v = s * sl2;
                        const float mn = fmaxf(m, v);
                        lsum = lsum * exp2_diff(m, mn) + fast_exp2(v - mn);
                        m = mn;
                    }
                };
                upd(c[0], j0, qA, mA, lA);
                upd(c[1], j0, qB, mB, lB);
                upd(c[2], j1, qA, mA, lA);
                upd(c[3], j1, qB, mB, lB);
            }
        }
        __syncthreads();  // the tile may be refilled
    }
    // merge the eight row groups of the warp (lanes with the same tq)
#pragma unroll
    for (int off = 4; off < 32; off <<= 1) {
        const float m2 = __shfl_xor_sync(0xffffffffu, mA, off), l2 = __shfl_xor_sync(0xffffffffu, lA, off);
        const float mn = fmaxf(mA, m2);
        lA = lA * exp2_diff(mA, mn) + l2 * exp2_diff(m2, mn);
        mA = mn;
        const float m3 = __shfl_xor_sync(0xffffffffu, mB, off), l3 = __shfl_xor_sync(0xffffffffu, lB, off);
        const float mo = fmaxf(mB, m3);
        lB = lB * exp2_diff(mB, mo) + l3 * exp2_diff(m3, mo);
        mB = mo;
    }
    if (gq == 0) {
        float2* st = a.stats + (size_t)item * P * HP;
        if (qA < P) st[(size_t)qA * HP + (2 * tq) % HP] = make_float2(mA, lA);
        if (qB < P) st[(size_t)qB * HP + (2 * tq + 1) % HP] = make_float2(mB, lB);
    }
}

constexpr int kColsumKeys = kPrefillWarps * 16;  // keys per CTA of the column-sum kernel
constexpr int kColsumCols = 64;                  // columns per staged block of queries

template <int D>
__global__ void __launch_bounds__(kPrefillWarps * 32) prefill_colsum_kernel(const __grid_constant__ PrefillArgs a) {
    using T = __nv_bfloat16;
    constexpr int ROW_BYTES = D * 2, KS = D / 16, CHUNKS = ROW_BYTES / 16;
    extern __shared__ __align__(128) unsigned char dyn[];
    // layout: key tile [128][ROW] | query blocks [2][64][ROW] | column factors [2][64] float2 (max, weight / sum)
    unsigned char* ktile = dyn;
    unsigned char* qtile = dyn + kColsumKeys * ROW_BYTES;
    float2* cfac = reinterpret_cast<float2*>(qtile + 2 * kColsumCols * ROW_BYTES);
    const int item = blockIdx.y;
    const int hkv = item % a.Hkv, b = (item / a.Hkv) % a.B, l = item / (a.Hkv * a.B);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31, gq = lane >> 2, tq = lane & 3;
    const int P = a.P, HP = a.HP;
    if (a.len[item] < P) return;  // reported by the statistics kernel
    const int j_cta = blockIdx.x * kColsumKeys;
    const int j_warp = j_cta + warp * 16;
    const int qpb = kColsumCols / HP;                // queries per staged block
    const float sl2 = a.scale_log2[l];

    // stage the CTA's keys, and the first query block
    stage_keys<D>(a, item, j_cta, kColsumKeys, P, smem_u32(ktile));
    auto stage_queries = [&](int q_first, int buf) {
        const uint32_t base = smem_u32(qtile + (size_t)buf * kColsumCols * ROW_BYTES);
        for (int idx = tid; idx < kColsumCols * CHUNKS; idx += kPrefillWarps * 32) {
            const int col = idx / CHUNKS, c = idx % CHUNKS;
            const int qi = q_first + col / HP, h = col % HP;
            const bool ok = qi < P && h < a.G;
            const char* src = (const char*)a.q +
                              ((((size_t)l * a.B + b) * P + (ok ? qi : 0)) * a.Hq + hkv * a.G + (ok ? h : 0)) * ROW_BYTES + c * 16;
            cp_async16(base + col * ROW_BYTES + ((c ^ (col & 7)) << 4), src, ok ? 16 : 0);
        }
        if (tid < kColsumCols) {
            const int qi = q_first + tid / HP, h = tid % HP;
            float2 f = make_float2(0.f, 0.f);
            if (qi < P && h < a.G) {
                const float2 st = a.stats[((size_t)item * P + qi) * HP + h];
                const float wgt = fast_exp2((float)(P - 1 - qi) * a.gamma_log2);
                f = make_float2(st.x, st.y > 0.f ? wgt / st.y : 0.f);
            }
            cfac[buf * kColsumCols + tid] = f;
        }
    };
    const int q_start = (j_cta / qpb) * qpb;  // earlier queries see none of this CTA's keys
    stage_queries(q_start, 0);
    cp_async_commit();
    cp_async_wait<0>();
    __syncthreads();

    // this warp's sixteen keys as A fragments, kept for the whole kernel
    uint32_t af[KS][4];
    {
        const int k_row = warp * 16 + (lane & 7) + ((lane >> 3) & 1) * 8, k_chunk = lane >> 4;
        const uint32_t kt = smem_u32(ktile);
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) ldmatrix_x4(kt + k_row * ROW_BYTES + (((2 * ks + k_chunk) ^ (k_row & 7)) << 4), af[ks]);
    }
    const int jA = j_warp + gq, jB = jA + 8;
    float accA = 0.f, accB = 0.f;
    int buf = 0;
    for (int q_first = q_start; q_first < P; q_first += qpb, buf ^= 1) {
        if (q_first + qpb < P) stage_queries(q_first + qpb, buf ^ 1);
        cp_async_commit();
        const uint32_t qt = smem_u32(qtile + (size_t)buf * kColsumCols * ROW_BYTES);
        const float2* cf = cfac + buf * kColsumCols;
        if (q_first + qpb - 1 >= j_warp && j_warp < P) {  // causal: some query of the block sees some key of this warp
#pragma unroll
            for (int cb = 0; cb < kColsumCols / 8; ++cb) {
                float c[4] = {0.f, 0.f, 0.f, 0.f};
                const int col = 8 * cb + gq;  // B operand: this thread supplies column gq of the block
#pragma unroll
                for (int ks = 0; ks < KS; ++ks) {
                    uint32_t b0, b1;
                    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(b0) : "r"(qt + col * ROW_BYTES + (((2 * ks) ^ (col & 7)) << 4) + 4 * tq) : "memory");
                    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(b1) : "r"(qt + col * ROW_BYTES + (((2 * ks + 1) ^ (col & 7)) << 4) + 4 * tq) : "memory");
                    mma_bf16(c, af[ks], b0, b1);
                }
                const int c0 = 8 * cb + 2 * tq, c1 = c0 + 1;  // accumulator columns of this thread
                const int qi0 = q_first + c0 / HP, qi1 = q_first + c1 / HP;
                const float2 f0 = cf[c0], f1 = cf[c1];
                if (jA <= qi0) accA += fast_exp2(c[0] * sl2 - f0.x) * f0.y;
                if (jA <= qi1) accA += fast_exp2(c[1] * sl2 - f1.x) * f1.y;
                if (jB <= qi0) accB += fast_exp2(c[2] * sl2 - f0.x) * f0.y;
                if (jB <= qi1) accB += fast_exp2(c[3] * sl2 - f1.x) * f1.y;
            }
        }
        cp_async_wait<0>();
        __syncthreads();  // the next block has landed and everyone is done with this one
    }
    accA += __shfl_xor_sync(0xffffffffu, accA, 1);
    accA += __shfl_xor_sync(0xffffffffu, accA, 2);
    accB += __shfl_xor_sync(0xffffffffu, accB, 1);
    accB += __shfl_xor_sync(0xffffffffu, accB, 2);
    if (tq == 0) {
        float* rel = a.rel + (size_t)item * a.cap_tokens;
        if (jA < P) rel[jA] = accA;
        if (jB < P) rel[jB] = accB;
    }
}

size_t prefill_stats_bytes(int items, int P, int HP) { return (size_t)items * P * HP * sizeof(float2); }

cudaError_t launch_prefill(const PrefillArgs& a, int items, int D, cudaStream_t stream) {
    const int QW = 8 / a.HP;
    const dim3 g1((a.P + kPrefillWarps * QW - 1) / (kPrefillWarps * QW), items);
    const dim3 g2((a.P + kColsumKeys - 1) / kColsumKeys, items);
    const size_t smem2 = (size_t)(kColsumKeys + 2 * kColsumCols) * D * 2 + 2 * kColsumCols * sizeof(float2);
    cudaError_t e;
    if (D == 128) {
        e = prepare_kernel((const void*)prefill_colsum_kernel<128>, smem2);
        if (e != cudaSuccess) return e;
        prefill_stats_kernel<128><<<g1, kPrefillWarps * 32, 0, stream>>>(a);
        prefill_colsum_kernel<128><<<g2, kPrefillWarps * 32, smem2, stream>>>(a);
    } else {
        e = prepare_kernel((const void*)prefill_colsum_kernel<64>, smem2);
        if (e != cudaSuccess) return e;
        prefill_stats_kernel<64><<<g1, kPrefillWarps * 32, 0, stream>>>(a);
        prefill_colsum_kernel<64><<<g2, kPrefillWarps * 32, smem2, stream>>>(a);
    }
    return cudaGetLastError();
}

}  // namespace lethe
