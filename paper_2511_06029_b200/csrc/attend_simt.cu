// CUDA-core decode-attend kernel: fp32 or bf16 cache, D in {64, 128}, contiguous or paged.
//
// One CTA (NW warps) streams a contiguous range of 16-token groups of one item; warp w takes groups
// g_begin + w, g_begin + w + NW, ...  Each lane owns D/32 consecutive elements of a row, so a warp reads one
// K row (and one V row) with a single fully-coalesced request; the G logits of a token are finished with a
// butterfly reduction.  The kernel keeps an online softmax per head (log2 units) and hands the per-warp
// partial results to the common epilogue (common.cuh), which also applies the Eq. 5 relevance update.
#include "common.cuh"

namespace lethe {

template <typename T, int E>
struct RowSlice;  // E consecutive elements of a row, loaded with one vector instruction

template <>
struct RowSlice<float, 4> {
    float4 raw;
    __device__ __forceinline__ void load(const char* p) { raw = *reinterpret_cast<const float4*>(p); }
    __device__ __forceinline__ void zero() { raw = make_float4(0.f, 0.f, 0.f, 0.f); }
    __device__ __forceinline__ void unpack(float* f) const { f[0] = raw.x; f[1] = raw.y; f[2] = raw.z; f[3] = raw.w; }
};
template <>
struct RowSlice<float, 2> {
    float2 raw;
    __device__ __forceinline__ void load(const char* p) { raw = *reinterpret_cast<const float2*>(p); }
    __device__ __forceinline__ void zero() { raw = make_float2(0.f, 0.f); }
    __device__ __forceinline__ void unpack(float* f) const { f[0] = raw.x; f[1] = raw.y; }
};
template <>
struct RowSlice<__nv_bfloat16, 4> {
    uint2 raw;
    __device__ __forceinline__ void load(const char* p) { raw = *reinterpret_cast<const uint2*>(p); }
    __device__ __forceinline__ void zero() { raw = make_uint2(0u, 0u); }
    __device__ __forceinline__ void unpack(float* f) const {
        f[0] = __uint_as_float(raw.x << 16); f[1] = __uint_as_float(raw.x & 0xffff0000u);
        f[2] = __uint_as_float(raw.y << 16); f[3] = __uint_as_float(raw.y & 0xffff0000u);
    }
};
template <>
struct RowSlice<__nv_bfloat16, 2> {
    uint32_t raw;
    __device__ __forceinline__ void load(const char* p) { raw = *reinterpret_cast<const uint32_t*>(p); }
    __device__ __forceinline__ void zero() { raw = 0u; }
    __device__ __forceinline__ void unpack(float* f) const {
        f[0] = __uint_as_float(raw << 16); f[1] = __uint_as_float(raw & 0xffff0000u);
    }
};

template <typename T, int D, int NW, bool PAGED>
__global__ void __launch_bounds__(NW * 32) attend_simt_kernel(const __grid_constant__ AttendArgs a) {
    constexpr int E = D / 32;
    constexpr int ROW_BYTES = D * (int)sizeof(T);
    constexpr int TB = 4;  // tokens whose loads are issued together
    extern __shared__ __align__(16) unsigned char smem_raw[];
    // layout: EpilogueSmem | wo [NW][kMaxGroup][D] | cta_o [kMaxGroup][D] | lg [chunk_tokens][GP]
    EpilogueSmem& es = *reinterpret_cast<EpilogueSmem*>(smem_raw);
    float* wo = reinterpret_cast<float*>(smem_raw + sizeof(EpilogueSmem));
    float* cta_o = wo + NW * kMaxGroup * D;
    float* lg = cta_o + kMaxGroup * D;

    const ItemCoord ic = decode_item(a);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = a.G, GP = a.GP;
    const bool append = a.k_new != nullptr;
    const int n_old = a.len[ic.item];
    T* out_rows = (T*)a.out + ((size_t)(ic.li * a.B + ic.b) * a.Hq + ic.hkv * G) * D;
    if (append && n_old >= a.cap_tokens) {  // full: leave the item untouched (every CTA of the cluster returns)
        if (ic.rank == 0) {
            for (int i = tid; i < G * D; i += NW * 32) out_rows[i] = from_float<T>(0.f);
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
    // Sec. 4.1: the cache grows by the token just generated; the CTA whose range holds slot n_old stores it.
    if (append && n_old >= t0 && n_old < t1 && warp == 0) {
        const size_t src = ((size_t)(ic.li * a.B + ic.b) * a.Hkv + ic.hkv) * ROW_BYTES;
        char* kd = const_cast<char*>(row_ptr<PAGED>(a, a.k, ic.item, n_old, ROW_BYTES, &bad_page));
        char* vd = const_cast<char*>(row_ptr<PAGED>(a, a.v, ic.item, n_old, ROW_BYTES, &bad_page));
        if (kd && vd) {
            for (int i = lane * 4; i < ROW_BYTES; i += 128) {
                *reinterpret_cast<uint32_t*>(kd + i) = *reinterpret_cast<const uint32_t*>((const char*)a.k_new + src + i);
                *reinterpret_cast<uint32_t*>(vd + i) = *reinterpret_cast<const uint32_t*>((const char*)a.v_new + src + i);
            }
        }
        if (lane == 0) a.pos[(size_t)ic.item * a.cap_tokens + n_old] = a.token_pos[ic.b];
    }
    __syncthreads();  // the appended row is visible to every warp of this CTA

    const float sl2 = a.scale_log2[ic.l];
    float qf[kMaxGroup][E];
#pragma unroll
    for (int h = 0; h < kMaxGroup; ++h) {
#pragma unroll
        for (int e = 0; e < E; ++e)
            qf[h][e] = (h < G) ? to_float<T>(((const T*)a.q)[((size_t)(ic.li * a.B + ic.b) * a.Hq + ic.hkv * G + h) * D + lane * E + e]) * sl2
                               : 0.f;
    }
    float m[kMaxGroup], l[kMaxGroup], o[kMaxGroup][E];
#pragma unroll
    for (int h = 0; h < kMaxGroup; ++h) {
        m[h] = -INFINITY;
        l[h] = 0.f;
#pragma unroll
        for (int e = 0; e < E; ++e) o[h][e] = 0.f;
    }

    for (int grp = g_begin + warp; grp < g_end; grp += NW) {
        const int tok0 = grp * kGroupTokens;
        for (int tb = 0; tb < kGroupTokens; tb += TB) {
            RowSlice<T, E> kr[TB], vr[TB];
#pragma unroll
            for (int i = 0; i < TB; ++i) {
                const int j = tok0 + tb + i;
                const char* kp = (j < n) ? row_ptr<PAGED>(a, a.k, ic.item, j, ROW_BYTES, &bad_page) : nullptr;
                const char* vp = (j < n) ? row_ptr<PAGED>(a, a.v, ic.item, j, ROW_BYTES, &bad_page) : nullptr;
                if (kp && vp) {
                    kr[i].load(kp + lane * E * sizeof(T));
                    vr[i].load(vp + lane * E * sizeof(T));
                } else {
                    kr[i].zero();
                    vr[i].zero();
                }
            }
#pragma unroll
            for (int i = 0; i < TB; ++i) {
                const int j = tok0 + tb + i;
                if (j >= n) break;  // warp-uniform
                float kf[E], vf[E];
                kr[i].unpack(kf);
                vr[i].unpack(vf);
                float s[kMaxGroup];
#pragma unroll
                for (int h = 0; h < kMaxGroup; ++h) {
                    float acc = 0.f;
#pragma unroll
                    for (int e = 0; e < E; ++e) acc = fmaf(qf[h][e], kf[e], acc);
                    s[h] = acc;
                }
#pragma unroll
                for (int h = 0; h < kMaxGroup; ++h) {
                    if (h < G) {
#pragma unroll
                        for (int off = 16; off > 0; off >>= 1) s[h] += __shfl_xor_sync(0xffffffffu, s[h], off);
                    }
                }
#pragma unroll
                for (int h = 0; h < kMaxGroup; ++h) {
                    if (h < G) {
                        if (lane == 0) lg[(size_t)(j - t0) * GP + h] = s[h];
                        const float mn = fmaxf(m[h], s[h]);
                        const float corr = exp2_diff(m[h], mn);
                        const float p = fast_exp2(s[h] - mn);
                        m[h] = mn;
                        l[h] = fmaf(l[h], corr, p);
#pragma unroll
                        for (int e = 0; e < E; ++e) o[h][e] = fmaf(o[h][e], corr, p * vf[e]);
                    }
                }
            }
        }
    }
    if (bad_page) record_error(a.status, LETHE_ERR_PAGE, ic.item);

#pragma unroll
    for (int h = 0; h < kMaxGroup; ++h) {
        if (lane == 0) es.wstat[warp][h] = make_float2(m[h], l[h]);
#pragma unroll
        for (int e = 0; e < E; ++e) wo[(warp * kMaxGroup + h) * D + lane * E + e] = o[h][e];
    }
    float rel_old[kRelPrefetch];
    prefetch_rel<NW * 32>(a, ic, t0, min(t1, n), append_slot, rel_old);
    combine_and_finish<T, D, NW>(a, ic, es, wo, kMaxGroup * D, cta_o, lg, t0, t1, append_slot, n, rel_old);
}

template <typename T, int D, int NW, bool PAGED>
static cudaError_t launch_simt_t(const AttendArgs& a, cudaStream_t stream) {
    auto kern = attend_simt_kernel<T, D, NW, PAGED>;
    const size_t smem = sizeof(EpilogueSmem) + (size_t)(NW + 1) * kMaxGroup * D * sizeof(float) +
                        (size_t)a.chunk_tokens * a.GP * sizeof(float);
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

size_t simt_smem_bytes(int D, int chunk_tokens, int GP) {
    return sizeof(EpilogueSmem) + (size_t)(4 + 1) * kMaxGroup * D * sizeof(float) + (size_t)chunk_tokens * GP * sizeof(float);
}

// dtype: LETHE_F32 / LETHE_BF16; D: 64 / 128
cudaError_t launch_attend_simt(const AttendArgs& a, int dtype, int D, bool paged, cudaStream_t stream) {
    constexpr int NW = 4;
    if (dtype == LETHE_F32) {
        if (D == 64) return paged ? launch_simt_t<float, 64, NW, true>(a, stream) : launch_simt_t<float, 64, NW, false>(a, stream);
        return paged ? launch_simt_t<float, 128, NW, true>(a, stream) : launch_simt_t<float, 128, NW, false>(a, stream);
    }
    if (D == 64)
        return paged ? launch_simt_t<__nv_bfloat16, 64, NW, true>(a, stream) : launch_simt_t<__nv_bfloat16, 64, NW, false>(a, stream);
    return paged ? launch_simt_t<__nv_bfloat16, 128, NW, true>(a, stream) : launch_simt_t<__nv_bfloat16, 128, NW, false>(a, stream);
}

}  // namespace lethe
