// Relevance of the prompt tokens from the prefill attention (Eq. 2 with Q > 1, folded through Eq. 5) on the
// fifth-generation tensor cores: tcgen05.mma with both operands in shared memory and the 128 x 128 fp32 logit
// tile in tensor memory (TMEM), read back by the softmax warps with tcgen05.ld.
//
// Same two deterministic passes as the mma.sync kernels (prefill.cu), one CTA per item in each:
//   STATS   the rows of a tile are 128 (query, head) columns of the attention matrix, its columns 128 keys; the
//           thread that owns a row keeps that column's online (max, sum) over the keys j <= i in registers;
//   COLSUM  the rows are 128 keys, the columns 128 (query, head) pairs; the thread that owns a key adds up
//           exp2(logit - max) * weight / sum over the columns with i >= j.
// In both, the reduction runs along the TMEM row a thread owns, so no value crosses threads.
//
// Roles (288 threads): warps 0-3 read TMEM and do the arithmetic (warp w owns TMEM lanes 32 w .. 32 w + 31),
// warp 4 allocates TMEM and one of its lanes issues the MMAs, warps 5-8 copy operand tiles with cp.async into the
// 128-byte-swizzled K-major layout the MMA's shared-memory descriptors name.  Hand-offs are mbarriers: loaders ->
// MMA (a_full, b_full), MMA -> loaders (a_empty, b_empty, by tcgen05.commit), MMA -> softmax (t_full, by
// tcgen05.commit), softmax -> MMA (t_empty).  Every wait is bounded: when one runs out the CTA sets an abort
// flag, every role leaves its loop, LETHE_ERR_TIMEOUT is recorded, TMEM is freed and the CTA returns.
#include "common.cuh"
#include "mma_utils.cuh"
#include "prefill.cuh"

namespace lethe {
namespace {

constexpr int kTcSoftmaxWarps = 4;
constexpr int kTcLoaderWarps = 4;
constexpr int kTcMmaWarp = kTcSoftmaxWarps;                                   // warp index of the MMA warp
constexpr int kTcThreads = (kTcSoftmaxWarps + 1 + kTcLoaderWarps) * 32;       // 288
constexpr int kTcLoaderThreads = kTcLoaderWarps * 32;
constexpr int kTcTile = 128;                                                  // rows of either operand: M = N = 128
constexpr int kTcStages = 3;                                                  // stages of the streamed operand
constexpr int kTcTmemCols = 2 * kTcTile;                                      // two accumulator buffers
constexpr int kTcWaitLimit = 400000;

enum { kModeStats = 0, kModeColsum = 1 };

struct TcShared {
    unsigned long long a_full[2], a_empty[2];
    unsigned long long b_full[kTcStages], b_empty[kTcStages];
    unsigned long long t_full[2], t_empty[2];
    uint32_t tmem_base;
    int abort;
    float2 cf[kTcSoftmaxWarps][2][kTcTile];  // COLSUM: (max, weight / sum) of the columns of the tiles in flight, one copy per warp
};

__device__ __forceinline__ void tc_mbar_init(unsigned long long* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void tc_mbar_arrive(unsigned long long* bar) {
    asm volatile("{ .reg .b64 st; mbarrier.arrive.shared::cta.b64 st, [%0]; }" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool tc_mbar_try_wait(unsigned long long* bar, unsigned parity) {
    unsigned ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok)
                 : "r"(smem_u32(bar)), "r"(parity)
                 : "memory");
    return ok != 0;
}
// Bounded wait; false = gave up (or another thread already did).
__device__ __forceinline__ bool tc_wait(unsigned long long* bar, unsigned parity, volatile int* abort_flag) {
    for (int it = 0; it < kTcWaitLimit; ++it) {
        if (tc_mbar_try_wait(bar, parity)) return true;
        if (*abort_flag) return false;
        if (it > 64) __nanosleep(64);
    }
    *abort_flag = 1;
    return false;
}

__device__ __forceinline__ void tc_fence_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_fence_proxy_async() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// Shared-memory matrix descriptor of a K-major bf16 operand tile stored as rows of 128 bytes (64 elements) with the
// 128-byte swizzle (16-byte chunk index XOR (row & 7)); groups of eight rows are 1024 bytes apart.
__device__ __forceinline__ uint64_t tc_smem_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);  // start address, 16-byte units
    d |= (uint64_t)1 << 16;                    // leading-dimension byte offset: unused by swizzled K-major layouts
    d |= (uint64_t)(1024 >> 4) << 32;          // stride between 8-row groups
    d |= (uint64_t)1 << 46;                    // descriptor version of this architecture
    d |= (uint64_t)2 << 61;                    // 128-byte swizzle
    return d;
}

// Instruction descriptor of tcgen05.mma.kind::f16: bf16 x bf16 -> fp32, both operands K-major, M x N tile.
__device__ __forceinline__ uint32_t tc_instr_desc(int M, int N) {
    uint32_t d = 0;
    d |= 1u << 4;                    // accumulator format: fp32
    d |= 1u << 7;                    // A format: bf16
    d |= 1u << 10;                   // B format: bf16
    d |= (uint32_t)(N >> 3) << 17;   // N / 8
    d |= (uint32_t)(M >> 4) << 24;   // M / 16
    return d;
}

__device__ __forceinline__ void tc_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n"
        ".reg .pred p;\n"
        "setp.ne.b32 p, %4, 0;\n"
        "tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n"
        "}\n" ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
// The barrier receives one arrival once every MMA this thread issued before has finished (reads of shared memory
// included).
__device__ __forceinline__ void tc_commit(unsigned long long* bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(bar)) : "memory");
}

// 32 consecutive columns of this thread's TMEM lane.
__device__ __forceinline__ void tc_ld32(uint32_t taddr, uint32_t (&v)[32]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x32.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15, "
        "%16, %17, %18, %19, %20, %21, %22, %23, %24, %25, %26, %27, %28, %29, %30, %31}, [%32];"
        : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
          "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15]), "=r"(v[16]),
          "=r"(v[17]), "=r"(v[18]), "=r"(v[19]), "=r"(v[20]), "=r"(v[21]), "=r"(v[22]), "=r"(v[23]), "=r"(v[24]),
          "=r"(v[25]), "=r"(v[26]), "=r"(v[27]), "=r"(v[28]), "=r"(v[29]), "=r"(v[30]), "=r"(v[31])
        : "r"(taddr)
        : "memory");
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// Which tiles of the streamed operand meet A block `a`.
//   STATS : A = query block a (qpb queries x HP heads = 128 rows); streamed = key tiles 0 .. (last query of a) / 128
//   COLSUM: A = key tile a; streamed = query blocks from the one holding key 128 a to the last
template <int MODE>
__device__ __forceinline__ void tc_range(int a, int P, int qpb, int& begin, int& end) {
    if (MODE == kModeStats) {
        begin = 0;
        end = min(P - 1, (a + 1) * qpb - 1) / kTcTile + 1;
    } else {
        begin = (a * kTcTile) / qpb;
        end = (P + qpb - 1) / qpb;
    }
}

template <int D>
__device__ __forceinline__ uint32_t tc_chunk_addr(uint32_t tile, int r, int c) {
    // 16-byte chunk c of row r: halves of 64 elements are separate 128-row regions
    return tile + (c >> 3) * (kTcTile * 128) + r * 128 + (((c & 7) ^ (r & 7)) << 4);
}

// 128 (query, head) columns starting at query qf, as K-major rows; columns of missing queries / padded heads are zero.
template <int D>
__device__ __forceinline__ void tc_load_queries(const PrefillArgs& a, int l, int b, int hkv, int qf, uint32_t tile, int ltid) {
    constexpr int CH = D * 2 / 16;
#pragma unroll 4
    for (int idx = ltid; idx < kTcTile * CH; idx += kTcLoaderThreads) {
        const int r = idx / CH, c = idx % CH;
        const int qi = qf + r / a.HP, h = r % a.HP;
        const bool ok = qi < a.P && h < a.G;
        const char* src = (const char*)a.q +
                          ((((size_t)l * a.B + b) * a.P + (ok ? qi : 0)) * a.Hq + hkv * a.G + (ok ? h : 0)) * (D * 2) + c * 16;
        cp_async16(tc_chunk_addr<D>(tile, r, c), src, ok ? 16 : 0);
    }
}

// 128 keys starting at slot j0; rows at or beyond the prompt are zero.
template <int D>
__device__ __forceinline__ void tc_load_keys(const PrefillArgs& a, int item, int j0, uint32_t tile, int ltid) {
    constexpr int CH = D * 2 / 16;
#pragma unroll 4
    for (int idx = ltid; idx < kTcTile * CH; idx += kTcLoaderThreads) {
        const int r = idx / CH, c = idx % CH;
        const int j = j0 + r;
        const bool ok = j < a.P;
        const char* src = prefill_row(a, item, ok ? j : 0, D * 2) + c * 16;
        cp_async16(tc_chunk_addr<D>(tile, r, c), src, ok ? 16 : 0);
    }
}

template <int D, int MODE>
__global__ void __launch_bounds__(kTcThreads, 1) prefill_tc_kernel(const __grid_constant__ PrefillArgs a) {
    constexpr int TILE_BYTES = kTcTile * D * 2;
    constexpr int KS = D / 16;
    extern __shared__ unsigned char dyn_raw[];
    __shared__ TcShared sh;

    const int item = blockIdx.x;
    const int hkv = item % a.Hkv, b = (item / a.Hkv) % a.B, l = item / (a.Hkv * a.B);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int P = a.P, HP = a.HP, qpb = kTcTile / HP;
    if (a.len[item] < P) {  // the prompt's keys are not all there: skip the item (uniform for the CTA)
        if (MODE == kModeStats && tid == 0) record_error(a.status, LETHE_ERR_CAPACITY, item);
        return;
    }
    // operand tiles: 1024-byte aligned (the swizzle pattern is anchored at 1024-byte boundaries)
    const uint32_t dyn = (smem_u32(dyn_raw) + 1023u) & ~1023u;
    const uint32_t a_tile[2] = {dyn, dyn + TILE_BYTES};
    const uint32_t b_tile0 = dyn + 2 * TILE_BYTES;
    volatile int* abort_flag = &sh.abort;

    if (tid == 0) {
        for (int i = 0; i < 2; ++i) {
            tc_mbar_init(&sh.a_full[i], kTcLoaderThreads);
            tc_mbar_init(&sh.a_empty[i], 1);
            tc_mbar_init(&sh.t_full[i], 1);
            tc_mbar_init(&sh.t_empty[i], kTcSoftmaxWarps * 32);
        }
        for (int i = 0; i < kTcStages; ++i) {
            tc_mbar_init(&sh.b_full[i], kTcLoaderThreads);
            tc_mbar_init(&sh.b_empty[i], 1);
        }
        sh.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == kTcMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&sh.tmem_base)),
                     "r"(kTcTmemCols)
                     : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = sh.tmem_base;

    const int nA = MODE == kModeStats ? (P + qpb - 1) / qpb : (P + kTcTile - 1) / kTcTile;

    if (warp > kTcMmaWarp) {
        // ------------------------------------------------------------------ loaders
        const int ltid = tid - (kTcMmaWarp + 1) * 32;
        int step = 0, prev_stage = -1, prev_a = -1;
        bool prev_first = false, alive = true;
        for (int ab = 0; ab < nA && alive; ++ab) {
            int t0, t1;
            tc_range<MODE>(ab, P, qpb, t0, t1);
            for (int t = t0; t < t1; ++t, ++step) {
                const int s = step % kTcStages;
                const bool first = t == t0;
                if (first) {
                    if (ab >= 2 && !tc_wait(&sh.a_empty[ab & 1], (unsigned)(((ab >> 1) - 1) & 1), abort_flag)) { alive = false; break; }
                    if (MODE == kModeStats) tc_load_queries<D>(a, l, b, hkv, ab * qpb, a_tile[ab & 1], ltid);
                    else tc_load_keys<D>(a, item, ab * kTcTile, a_tile[ab & 1], ltid);
                }
                if (step >= kTcStages && !tc_wait(&sh.b_empty[s], (unsigned)(((step / kTcStages) - 1) & 1), abort_flag)) { alive = false; break; }
                if (MODE == kModeStats) tc_load_keys<D>(a, item, t * kTcTile, b_tile0 + s * TILE_BYTES, ltid);
                else tc_load_queries<D>(a, l, b, hkv, t * qpb, b_tile0 + s * TILE_BYTES, ltid);
                cp_async_commit();
                if (prev_stage >= 0) {  // the previous step's copies have landed: publish them to the MMA's proxy
                    cp_async_wait<1>();
                    tc_fence_proxy_async();
                    if (prev_first) tc_mbar_arrive(&sh.a_full[prev_a & 1]);
                    tc_mbar_arrive(&sh.b_full[prev_stage]);
                }
                prev_stage = s; prev_a = ab; prev_first = first;
            }
        }
        cp_async_wait<0>();
        if (alive && prev_stage >= 0) {
            tc_fence_proxy_async();
            if (prev_first) tc_mbar_arrive(&sh.a_full[prev_a & 1]);
            tc_mbar_arrive(&sh.b_full[prev_stage]);
        }
    } else if (warp == kTcMmaWarp) {
        // ------------------------------------------------------------------ MMA issue (one lane)
        if (lane == 0) {
            const uint32_t idesc = tc_instr_desc(kTcTile, kTcTile);
            int step = 0;
            bool alive = true;
            for (int ab = 0; ab < nA && alive; ++ab) {
                int t0, t1;
                tc_range<MODE>(ab, P, qpb, t0, t1);
                for (int t = t0; t < t1; ++t, ++step) {
                    const int s = step % kTcStages, buf = step & 1;
                    if (t == t0 && !tc_wait(&sh.a_full[ab & 1], (unsigned)((ab >> 1) & 1), abort_flag)) { alive = false; break; }
                    if (!tc_wait(&sh.b_full[s], (unsigned)((step / kTcStages) & 1), abort_flag)) { alive = false; break; }
                    if (step >= 2 && !tc_wait(&sh.t_empty[buf], (unsigned)(((step >> 1) - 1) & 1), abort_flag)) { alive = false; break; }
                    tc_fence_after();
                    const uint32_t at = a_tile[ab & 1], bt = b_tile0 + s * TILE_BYTES;
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        // 16 elements of K per MMA: 32 bytes along the swizzled row; the second 64 elements are the next region
                        const uint32_t off = (ks >> 2) * (kTcTile * 128) + (ks & 3) * 32;
                        tc_mma(tmem + buf * kTcTile, tc_smem_desc(at + off), tc_smem_desc(bt + off), idesc, ks > 0 ? 1u : 0u);
                    }
                    tc_commit(&sh.b_empty[s]);
                    if (t == t1 - 1) tc_commit(&sh.a_empty[ab & 1]);
                    tc_commit(&sh.t_full[buf]);
                }
            }
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ softmax warps
        const int r = tid;  // TMEM lane = tile row
        const float sl2 = a.scale_log2[l];
        const uint32_t t_lane = tmem + ((uint32_t)(warp * 32) << 16);
        int step = 0;
        bool alive = true;
        // COLSUM: every warp keeps its own copy of the tile's 128 column factors (lane x fetches columns x, x + 32,
        // x + 64, x + 96 one step ahead), so the softmax warps never wait for one another
        auto column_factor = [&](int u, int col) -> float2 {
            const int qc = u * qpb + col / HP, h = col % HP;
            float2 f = make_float2(0.f, 0.f);
            if (qc < P && h < a.G) {
                const float2 st = a.stats[((size_t)item * P + qc) * HP + h];
                const float wgt = fast_exp2((float)(P - 1 - qc) * a.gamma_log2);
                f = make_float2(st.x, st.y > 0.f ? wgt / st.y : 0.f);
            }
            return f;
        };
        for (int ab = 0; ab < nA && alive; ++ab) {
            int t0, t1;
            tc_range<MODE>(ab, P, qpb, t0, t1);
            // STATS state of this thread's column; COLSUM accumulators of this thread's key
            const int qi = ab * qpb + r / HP;
            const bool row_ok = MODE == kModeStats ? (qi < P && (r % HP) < a.G) : (ab * kTcTile + r < P);
            float m = -INFINITY, lsum = 0.f;
            float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
            float2 f_next[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) f_next[k] = MODE == kModeColsum ? column_factor(t0, lane + 32 * k) : make_float2(0.f, 0.f);
            for (int t = t0; t < t1; ++t, ++step) {
                const int buf = step & 1;
                if (MODE == kModeColsum) {
                    __syncwarp();
#pragma unroll
                    for (int k = 0; k < 4; ++k) {
                        sh.cf[warp][buf][lane + 32 * k] = f_next[k];
                        if (t + 1 < t1) f_next[k] = column_factor(t + 1, lane + 32 * k);
                    }
                    __syncwarp();
                }
                if (!tc_wait(&sh.t_full[buf], (unsigned)((step >> 1) & 1), abort_flag)) { alive = false; break; }
                tc_fence_after();
#pragma unroll 1
                for (int ch = 0; ch < kTcTile / 32; ++ch) {
                    uint32_t v[32];
                    tc_ld32(t_lane + buf * kTcTile + ch * 32, v);
                    if (MODE == kModeStats) {
                        const int nv = qi - (t * kTcTile + ch * 32) + 1;  // keys of this chunk that query qi sees
                        if (row_ok && nv > 0) {
                            float mx = m;
#pragma unroll
                            for (int c = 0; c < 32; ++c) {
                                const float x = __uint_as_float(v[c]) * sl2;
                                v[c] = __float_as_uint(x);
                                if (c < nv) mx = fmaxf(mx, x);
                            }
                            float l0 = lsum * exp2_diff(m, mx), l1 = 0.f, l2 = 0.f, l3 = 0.f;
#pragma unroll
                            for (int c = 0; c < 32; c += 4) {
                                if (c < nv) l0 += fast_exp2(__uint_as_float(v[c]) - mx);
                                if (c + 1 < nv) l1 += fast_exp2(__uint_as_float(v[c + 1]) - mx);
                                if (c + 2 < nv) l2 += fast_exp2(__uint_as_float(v[c + 2]) - mx);
                                if (c + 3 < nv) l3 += fast_exp2(__uint_as_float(v[c + 3]) - mx);
                            }
                            lsum = (l0 + l1) + (l2 + l3);
                            m = mx;
                        }
                    } else {
                        // column cc = (query t * qpb + cc / HP, head cc % HP) counts for key j when query >= j
                        const int c_start = (ab * kTcTile + r - t * qpb) * HP - ch * 32;  // first counted column of this chunk
                        if (row_ok && c_start < 32) {
                            const float2* cf = sh.cf[warp][buf] + ch * 32;
#pragma unroll
                            for (int c = 0; c < 32; c += 4) {
                                const float2 f0 = cf[c], f1 = cf[c + 1], f2 = cf[c + 2], f3 = cf[c + 3];
                                if (c >= c_start) acc0 += fast_exp2(__uint_as_float(v[c]) * sl2 - f0.x) * f0.y;
                                if (c + 1 >= c_start) acc1 += fast_exp2(__uint_as_float(v[c + 1]) * sl2 - f1.x) * f1.y;
                                if (c + 2 >= c_start) acc2 += fast_exp2(__uint_as_float(v[c + 2]) * sl2 - f2.x) * f2.y;
                                if (c + 3 >= c_start) acc3 += fast_exp2(__uint_as_float(v[c + 3]) * sl2 - f3.x) * f3.y;
                            }
                        }
                    }
                }
                tc_fence_before();
                tc_mbar_arrive(&sh.t_empty[buf]);
            }
            if (alive && row_ok) {
                if (MODE == kModeStats) a.stats[((size_t)item * P + qi) * HP + r % HP] = make_float2(m, lsum);
                else a.rel[(size_t)item * a.cap_tokens + ab * kTcTile + r] = (acc0 + acc1) + (acc2 + acc3);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (sh.abort && tid == 0) record_error(a.status, LETHE_ERR_TIMEOUT, item);
    if (warp == kTcMmaWarp)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTcTmemCols) : "memory");
}

template <int D>
cudaError_t launch_tc(const PrefillArgs& a, int items, cudaStream_t stream) {
    const size_t smem = 1024 + (size_t)(2 + kTcStages) * kTcTile * D * 2;
    cudaError_t e = prepare_kernel((const void*)prefill_tc_kernel<D, kModeStats>, smem);
    if (e != cudaSuccess) return e;
    e = prepare_kernel((const void*)prefill_tc_kernel<D, kModeColsum>, smem);
    if (e != cudaSuccess) return e;
    prefill_tc_kernel<D, kModeStats><<<items, kTcThreads, smem, stream>>>(a);
    prefill_tc_kernel<D, kModeColsum><<<items, kTcThreads, smem, stream>>>(a);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_prefill_tc(const PrefillArgs& a, int items, int D, cudaStream_t stream) {
    return D == 128 ? launch_tc<128>(a, items, stream) : launch_tc<64>(a, items, stream);
}

}  // namespace lethe
