// Relevance of the prompt tokens from the prefill attention (Eq. 2 with Q > 1, folded through Eq. 5) on the
// fifth-generation tensor cores: tcgen05.mma with both operands in shared memory and the 128 x 128 fp32 logit
// tile in tensor memory (TMEM), read back by the softmax warps with tcgen05.ld.
//
// Same two deterministic passes as the mma.sync kernels (prefill.cu), one CTA per item in each:
//   STATS   the rows of a tile are 128 (query, head) columns of the attention matrix, its columns 128 keys; the
//           thread that owns a row keeps that column's online (max, sum) over the keys j <= i in registers;
//   COLSUM  the rows are 128 keys, the columns 128 (query, head) pairs; the thread that owns a key adds up
//           exp2(logit + bias) over the columns with i >= j, the bias of a column being log2(weight / sum) - max.
// In both, the reduction runs along the TMEM row a thread owns.  Two warps share a row (TMEM lanes are reachable
// only from the warps whose index has the same low two bits): each takes 64 of the 128 columns.  STATS writes the
// two partial (max, sum) pairs side by side; the prologue of COLSUM merges them into the item's column biases
// (in place); COLSUM's two partial sums of a key meet in rel[j], zeroed by STATS, through two atomic adds (two
// addends commute, so the result does not depend on their order).  Two CTAs share an SM (one block buffer, two
// streamed stages and 256 TMEM columns each) and cover each other's hand-off latencies.
//
// (query, head) columns are numbered query-major over the G heads of the group: column c of a block that starts
// at query q0 is (q0 + c / G, c % G); a block holds qpb = 128 / G queries and its last 128 - qpb G columns are
// unused (zero operand rows, never counted).
//
// Roles: warps 0-7 read TMEM and do the arithmetic (warp w owns TMEM lanes 32 (w % 4) .. + 31 and columns
// 64 (w / 4) .. + 63), warp 8 allocates TMEM and one of its lanes issues the MMAs, and the operand tiles arrive in
// the 128-byte-swizzled K-major layout the MMA's shared-memory descriptors name either by TMA (one lane of warp 9
// issues cp.async.bulk.tensor boxes: one per 128-row tile of a contiguous cache, one per page of a paged one) or
// by 16-byte cp.async from warps 9-12 (selectable; also the fallback when no tensor map can be made).
// Hand-offs are mbarriers: producer -> MMA (a_full, b_full), MMA -> producer (a_empty, b_empty, by
// tcgen05.commit), MMA -> softmax (t_full, by tcgen05.commit), softmax -> MMA (t_empty).  Every wait is bounded:
// when one runs out the CTA sets an abort flag, every role leaves its loop, LETHE_ERR_TIMEOUT is recorded, TMEM is
// freed and the CTA returns.
#include <cuda.h>

#include "common.cuh"
#include "mma_utils.cuh"
#include "prefill.cuh"

namespace lethe {
namespace {

constexpr int kTcSoftmaxWarps = 8;
constexpr int kTcSoftmaxThreads = kTcSoftmaxWarps * 32;
constexpr int kTcMmaWarp = kTcSoftmaxWarps;                                   // warp index of the MMA warp
constexpr int kTcLoaderWarps = 4;                                             // cp.async path only
constexpr int kTcLoaderThreads = kTcLoaderWarps * 32;
constexpr int kTcTile = 128;                                                  // rows of either operand: M = N = 128
constexpr int kTcStages = 2;                                                  // stages of the streamed operand
constexpr int kTcABuffers = 1;                                                // buffers of the block operand
constexpr int kTcCtasPerSm = 2;                                               // co-resident CTAs hide each other's waits
constexpr int kTcTmemCols = 2 * kTcTile;                                      // two accumulator buffers
constexpr int kTcWaitLimit = 400000;

template <bool TMA>
__host__ __device__ constexpr int tc_threads() { return (kTcSoftmaxWarps + 1 + (TMA ? 1 : kTcLoaderWarps)) * 32; }

enum { kModeStats = 0, kModeColsum = 1 };


// Tensor maps of the TMA path: K as [items][capacity][D] with a 128-row box, the prompt's queries as
// [L B][P][Hq][D] with a (qpb queries x G heads) box; 64-element (128-byte) inner boxes, 128-byte swizzle.
struct alignas(64) TcMaps {
    CUtensorMap k, q;
};

struct TcShared {
    unsigned long long a_full[kTcABuffers], a_empty[kTcABuffers];
    unsigned long long b_full[kTcStages], b_empty[kTcStages];
    unsigned long long t_full[2], t_empty[2];
    unsigned long long mma_drained;  // used only after a timeout: every MMA issued so far has finished
    int armed_a, armed_steps, mma_steps;  // TMA boxes and MMA steps issued when the roles left their loops
    uint32_t tmem_base;
    int abort;
    // COLSUM: bias (log2(weight / sum) - max) of the 64 columns a warp reads, of the tiles in flight; one copy per warp
    alignas(16) float cf[kTcSoftmaxWarps][2][kTcTile / 2];
};

__device__ __forceinline__ void tc_mbar_init(unsigned long long* bar, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void tc_mbar_arrive(unsigned long long* bar) {
    asm volatile("{ .reg .b64 st; mbarrier.arrive.shared::cta.b64 st, [%0]; }" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ void tc_mbar_expect_tx(unsigned long long* bar, unsigned bytes) {
    asm volatile("{ .reg .b64 st; mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1; }" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool tc_mbar_try_wait(unsigned long long* bar, unsigned parity) {
    unsigned ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok)
                 : "r"(smem_u32(bar)), "r"(parity)
                 : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool tc_mbar_test_wait(unsigned long long* bar, unsigned parity) {  // never waits inside
    unsigned ok;
    asm volatile("{ .reg .pred p; mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok)
                 : "r"(smem_u32(bar)), "r"(parity)
                 : "memory");
    return ok != 0;
}
// Bounded wait; false = gave up (or another thread already did).  Poll 0 does not block, so a limit of one poll
// is exactly one look at the barrier.
__device__ __forceinline__ bool tc_wait(unsigned long long* bar, unsigned parity, volatile int* abort_flag, int limit) {
    if (tc_mbar_test_wait(bar, parity)) return true;
    for (int it = 1; it < limit; ++it) {
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

// One box of a tensor map into shared memory; completion is counted in bytes on `bar`.  x is 0 or 64 elements (a
// multiple of 16 bytes); the other coordinates have no alignment rule.
__device__ __forceinline__ void tc_tma_3d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, unsigned long long* bar) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4}], [%5];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(smem_u32(bar))
        : "memory");
}
__device__ __forceinline__ void tc_tma_4d(uint32_t dst, const CUtensorMap* map, int x, int y, int z, int w, unsigned long long* bar) {
    asm volatile(
        "cp.async.bulk.tensor.4d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3, %4, %5}], [%6];"
        ::"r"(dst), "l"(map), "r"(x), "r"(y), "r"(z), "r"(w), "r"(smem_u32(bar))
        : "memory");
}

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

// 32 consecutive columns of this thread's TMEM lane (asynchronous: tc_ld_wait before the registers are used).
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
}
__device__ __forceinline__ void tc_ld_wait() { asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory"); }

// Which tiles of the streamed operand meet A block `a`.
//   STATS : A = query block a (qpb queries x G heads); streamed = key tiles 0 .. (last query of a) / 128
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

__device__ __forceinline__ uint32_t tc_chunk_addr(uint32_t tile, int r, int c) {
    // 16-byte chunk c of row r: halves of 64 elements are separate 128-row regions
    return tile + (c >> 3) * (kTcTile * 128) + r * 128 + (((c & 7) ^ (r & 7)) << 4);
}

// cp.async path: the (query, head) columns of the block starting at query qf, as K-major rows; rows of missing
// queries and the unused tail are zero.
template <int D>
__device__ __forceinline__ void tc_load_queries(const PrefillArgs& a, int l, int b, int hkv, int qf, int used, uint32_t tile, int ltid) {
    constexpr int CH = D * 2 / 16;
#pragma unroll 4
    for (int idx = ltid; idx < kTcTile * CH; idx += kTcLoaderThreads) {
        const int r = idx / CH, c = idx % CH;
        const int qi = qf + r / a.G, h = r % a.G;
        const bool ok = r < used && qi < a.P;
        const char* src = (const char*)a.q +
                          ((((size_t)l * a.B + b) * a.P + (ok ? qi : 0)) * a.Hq + hkv * a.G + (ok ? h : 0)) * (D * 2) + c * 16;
        cp_async16(tc_chunk_addr(tile, r, c), src, ok ? 16 : 0);
    }
}

// cp.async path: 128 keys starting at slot j0; rows at or beyond the prompt are zero.
template <int D>
__device__ __forceinline__ void tc_load_keys(const PrefillArgs& a, int item, int j0, uint32_t tile, int ltid) {
    constexpr int CH = D * 2 / 16;
#pragma unroll 4
    for (int idx = ltid; idx < kTcTile * CH; idx += kTcLoaderThreads) {
        const int r = idx / CH, c = idx % CH;
        const int j = j0 + r;
        const bool ok = j < a.P;
        const char* src = prefill_row(a, item, ok ? j : 0, D * 2) + c * 16;
        cp_async16(tc_chunk_addr(tile, r, c), src, ok ? 16 : 0);
    }
}

template <int D, int MODE, bool TMA>
__global__ void __launch_bounds__(tc_threads<TMA>(), kTcCtasPerSm)
    prefill_tc_kernel(const __grid_constant__ PrefillArgs a, const __grid_constant__ TcMaps maps) {
    constexpr int TILE_BYTES = kTcTile * D * 2;
    constexpr int HALF_BYTES = kTcTile * 128;  // one 64-element half of a tile
    constexpr int KS = D / 16;
    extern __shared__ unsigned char dyn_raw[];
    __shared__ TcShared sh;

    const int item = blockIdx.x;
    const int hkv = item % a.Hkv, b = (item / a.Hkv) % a.B, l = item / (a.Hkv * a.B);
    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int P = a.P, G = a.G, HP = a.HP, qpb = kTcTile / G, used = qpb * G;
    if (a.len[item] < P) {  // the prompt's keys are not all there: skip the item (uniform for the CTA)
        if (MODE == kModeStats && tid == 0) record_error(a.status, LETHE_ERR_CAPACITY, item);
        return;
    }
    // operand tiles: 1024-byte aligned (the swizzle pattern is anchored at 1024-byte boundaries)
    const uint32_t dyn = (smem_u32(dyn_raw) + 1023u) & ~1023u;
    const uint32_t a_tile0 = dyn;
    const uint32_t b_tile0 = dyn + kTcABuffers * TILE_BYTES;
    volatile int* abort_flag = &sh.abort;
    const int wait_limit = a.wait_limit > 0 ? a.wait_limit : kTcWaitLimit;
    // After a wait has run out, copies and MMAs this CTA started may still be in flight; the thread that started them
    // waits for them (with the fixed limit, whatever wait_limit says) before the CTA gives its shared and tensor
    // memory back.
    auto drain = [&](unsigned long long* bar, unsigned parity) {
        for (int it = 0; it < kTcWaitLimit; ++it) {
            if (tc_mbar_try_wait(bar, parity)) return;
            if (it > 64) __nanosleep(64);
        }
    };

    if (tid == 0) {
        const int producers = TMA ? 1 : kTcLoaderThreads;
        for (int i = 0; i < kTcABuffers; ++i) {
            tc_mbar_init(&sh.a_full[i], producers);
            tc_mbar_init(&sh.a_empty[i], 1);
        }
        for (int i = 0; i < 2; ++i) {
            tc_mbar_init(&sh.t_full[i], 1);
            tc_mbar_init(&sh.t_empty[i], kTcSoftmaxThreads);
        }
        for (int i = 0; i < kTcStages; ++i) {
            tc_mbar_init(&sh.b_full[i], producers);
            tc_mbar_init(&sh.b_empty[i], 1);
        }
        tc_mbar_init(&sh.mma_drained, 1);
        sh.armed_a = -1;
        sh.armed_steps = 0;
        sh.mma_steps = 0;
        sh.abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (TMA && used < kTcTile) {
        // rows the query boxes never write: zero them once (in every buffer that will hold queries)
        const uint32_t first = MODE == kModeStats ? a_tile0 : b_tile0;
        const int n_buf = MODE == kModeStats ? kTcABuffers : kTcStages;
        const int tail_chunks = (kTcTile - used) * 8;  // 16-byte chunks per 64-element half
        for (int idx = tid; idx < n_buf * (D / 64) * tail_chunks; idx += tc_threads<TMA>()) {
            const int c = idx % tail_chunks, hb = idx / tail_chunks;  // hb = buffer * halves + half
            const uint32_t addr = first + (hb / (D / 64)) * TILE_BYTES + (hb % (D / 64)) * HALF_BYTES + used * 128 + c * 16;
            asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(addr), "r"(0) : "memory");
        }
        tc_fence_proxy_async();
    }
    if (MODE == kModeStats && warp < kTcSoftmaxWarps) {
        // COLSUM adds its two partial sums of every key into rel: start them at zero
        float* rel = a.rel + (size_t)item * a.cap_tokens;
        for (int j = tid; j < P; j += kTcSoftmaxThreads) rel[j] = 0.f;
    }
    if (MODE == kModeColsum) {
        // turn the item's two partial (max, sum) pairs of every (query, head) column into the column's bias
        // log2(decay weight / sum) - max, in place over the first partial; the softmax warps then only copy biases
        const size_t part = (size_t)gridDim.x * P * HP;
        for (int idx = tid; idx < P * G; idx += tc_threads<TMA>()) {
            const int qc = idx / G, h = idx - qc * G;
            const size_t at = ((size_t)item * P + qc) * HP + h;
            const float2 s0 = a.stats[at], s1 = a.stats[part + at];
            const float mx = fmaxf(s0.x, s1.x);
            const float sum = s0.y * exp2_diff(s0.x, mx) + s1.y * exp2_diff(s1.x, mx);
            // exp2(logit - max) * weight / sum = exp2(logit + bias) with one bias per column
            const float bias = sum > 0.f ? (float)(P - 1 - qc) * a.gamma_log2 - mx - __log2f(sum) : -INFINITY;
            a.stats[at] = make_float2(bias, 0.f);
        }
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
        // ------------------------------------------------------------------ producers
        if (TMA) {
            if (warp == kTcMmaWarp + 1 && lane == 0) {
                const unsigned q_bytes = (unsigned)used * D * 2, k_bytes = TILE_BYTES;
                auto load_queries = [&](int q0, uint32_t tile, unsigned long long* bar) {
#pragma unroll
                    for (int hf = 0; hf < D / 64; ++hf) tc_tma_4d(tile + hf * HALF_BYTES, &maps.q, 64 * hf, hkv * G, q0, l * a.B + b, bar);
                };
                auto load_keys = [&](int j0, uint32_t tile, unsigned long long* bar) {
                    if (!a.paged) {
#pragma unroll
                        for (int hf = 0; hf < D / 64; ++hf) tc_tma_3d(tile + hf * HALF_BYTES, &maps.k, 64 * hf, j0, item, bar);
                        return;
                    }
                    // paged: one box per page (the map sees the pool as [pages][page_tokens][D]); slots beyond the
                    // item's table and bad ids read page 0 — rows that no query sees
                    const int pt = a.page_tokens, per_tile = kTcTile / pt;
                    int pages[8];
#pragma unroll
                    for (int pg = 0; pg < 8; ++pg) {
                        const int slot = j0 / pt + pg;
                        int page = (pg < per_tile && slot < a.capacity) ? a.page_table[(size_t)item * a.capacity + slot] : 0;
                        pages[pg] = (page < 0 || page >= a.n_pages) ? 0 : page;
                    }
#pragma unroll
                    for (int pg = 0; pg < 8; ++pg)
                        if (pg < per_tile)
#pragma unroll
                            for (int hf = 0; hf < D / 64; ++hf)
                                tc_tma_3d(tile + hf * HALF_BYTES + pg * pt * 128, &maps.k, 64 * hf, 0, pages[pg], bar);
                };
                int step = 0;
                bool alive = true;
                int a_armed = -1;  // last block operand whose box was issued
                for (int ab = 0; ab < nA && alive; ++ab) {
                    int t0, t1;
                    tc_range<MODE>(ab, P, qpb, t0, t1);
                    for (int t = t0; t < t1; ++t, ++step) {
                        const int s = step % kTcStages;
                        if (t == t0) {
                            if (ab >= kTcABuffers && !tc_wait(&sh.a_empty[ab % kTcABuffers], (unsigned)(((ab / kTcABuffers) - 1) & 1), abort_flag, wait_limit)) { alive = false; break; }
                            const uint32_t at = a_tile0 + (ab % kTcABuffers) * TILE_BYTES;
                            a_armed = ab;
                            tc_mbar_expect_tx(&sh.a_full[ab % kTcABuffers], MODE == kModeStats ? q_bytes : k_bytes);
                            if (MODE == kModeStats) load_queries(ab * qpb, at, &sh.a_full[ab % kTcABuffers]);
                            else load_keys(ab * kTcTile, at, &sh.a_full[ab % kTcABuffers]);
                        }
                        if (step >= kTcStages && !tc_wait(&sh.b_empty[s], (unsigned)(((step / kTcStages) - 1) & 1), abort_flag, wait_limit)) { alive = false; break; }
                        const uint32_t bt = b_tile0 + s * TILE_BYTES;
                        tc_mbar_expect_tx(&sh.b_full[s], MODE == kModeStats ? k_bytes : q_bytes);
                        if (MODE == kModeStats) load_keys(t * kTcTile, bt, &sh.b_full[s]);
                        else load_queries(t * qpb, bt, &sh.b_full[s]);
                    }
                }
                sh.armed_a = a_armed;  // what was issued, for the drain after a timeout
                sh.armed_steps = step;
            }
            __syncwarp();
        } else {
            const int ltid = tid - (kTcMmaWarp + 1) * 32;
            int step = 0;
            bool alive = true;
            for (int ab = 0; ab < nA && alive; ++ab) {
                int t0, t1;
                tc_range<MODE>(ab, P, qpb, t0, t1);
                for (int t = t0; t < t1; ++t, ++step) {
                    const int s = step % kTcStages;
                    const bool first = t == t0;
                    if (first) {
                        if (ab >= kTcABuffers && !tc_wait(&sh.a_empty[ab % kTcABuffers], (unsigned)(((ab / kTcABuffers) - 1) & 1), abort_flag, wait_limit)) { alive = false; break; }
                        const uint32_t at = a_tile0 + (ab % kTcABuffers) * TILE_BYTES;
                        if (MODE == kModeStats) tc_load_queries<D>(a, l, b, hkv, ab * qpb, used, at, ltid);
                        else tc_load_keys<D>(a, item, ab * kTcTile, at, ltid);
                    }
                    if (step >= kTcStages && !tc_wait(&sh.b_empty[s], (unsigned)(((step / kTcStages) - 1) & 1), abort_flag, wait_limit)) { alive = false; break; }
                    if (MODE == kModeStats) tc_load_keys<D>(a, item, t * kTcTile, b_tile0 + s * TILE_BYTES, ltid);
                    else tc_load_queries<D>(a, l, b, hkv, t * qpb, used, b_tile0 + s * TILE_BYTES, ltid);
                    // the step's copies must have landed and be visible to the MMA's proxy before it is told; nothing
                    // is held back (a later wait of this loop may depend on the MMA of this very step)
                    cp_async_commit();
                    cp_async_wait<0>();
                    tc_fence_proxy_async();
                    if (first) tc_mbar_arrive(&sh.a_full[ab % kTcABuffers]);
                    tc_mbar_arrive(&sh.b_full[s]);
                }
            }
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
                    if (t == t0 && !tc_wait(&sh.a_full[ab % kTcABuffers], (unsigned)((ab / kTcABuffers) & 1), abort_flag, wait_limit)) { alive = false; break; }
                    if (!tc_wait(&sh.b_full[s], (unsigned)((step / kTcStages) & 1), abort_flag, wait_limit)) { alive = false; break; }
                    if (step >= 2 && !tc_wait(&sh.t_empty[buf], (unsigned)(((step >> 1) - 1) & 1), abort_flag, wait_limit)) { alive = false; break; }
                    tc_fence_after();
                    const uint32_t at = a_tile0 + (ab % kTcABuffers) * TILE_BYTES, bt = b_tile0 + s * TILE_BYTES;
#pragma unroll
                    for (int ks = 0; ks < KS; ++ks) {
                        // 16 elements of K per MMA: 32 bytes along the swizzled row; the second 64 elements are the next region
                        const uint32_t off = (ks >> 2) * HALF_BYTES + (ks & 3) * 32;
                        tc_mma(tmem + buf * kTcTile, tc_smem_desc(at + off), tc_smem_desc(bt + off), idesc, ks > 0 ? 1u : 0u);
                    }
                    tc_commit(&sh.b_empty[s]);
                    if (t == t1 - 1) tc_commit(&sh.a_empty[ab % kTcABuffers]);
                    tc_commit(&sh.t_full[buf]);
                }
            }
            sh.mma_steps = step;
        }
        __syncwarp();
    } else {
        // ------------------------------------------------------------------ softmax warps
        const int quarter = warp & 3, half = warp >> 2;
        const int r = quarter * 32 + lane;  // TMEM lane = tile row
        const float sl2 = a.scale_log2[l];
        const uint32_t t_lane = tmem + ((uint32_t)(quarter * 32) << 16) + half * 64;
        const size_t half_stride = (size_t)gridDim.x * P * HP;  // STATS partials of the upper 64 key columns come second
        int step = 0;
        bool alive = true;
        // COLSUM: every warp keeps its own copy of the factors of the 64 columns it reads (lane x owns columns x and
        // x + 32 of its half, fetched one step ahead), so the softmax warps never wait for one another
        int col_q[2], col_h[2];
#pragma unroll
        for (int k = 0; k < 2; ++k) {
            const int col = half * 64 + lane + 32 * k;
            col_q[k] = col < used ? col / G : -1;
            col_h[k] = col % G;
        }
        auto fetch_factor = [&](int u, int k) -> float {
            const int qc = u * qpb + col_q[k];
            if (col_q[k] < 0 || qc >= P) return -INFINITY;
            return a.stats[((size_t)item * P + qc) * HP + col_h[k]].x;
        };
        for (int ab = 0; ab < nA && alive; ++ab) {
            int t0, t1;
            tc_range<MODE>(ab, P, qpb, t0, t1);
            // STATS: state of this thread's column over its half of every key tile; COLSUM: partial sum of its key
            const int qi = ab * qpb + r / G;
            const bool row_ok = MODE == kModeStats ? (r < used && qi < P) : (ab * kTcTile + r < P);
            float m = -INFINITY, lsum = 0.f;
            float acc0 = 0.f, acc1 = 0.f, acc2 = 0.f, acc3 = 0.f;
            float f_next[2];
#pragma unroll
            for (int k = 0; k < 2; ++k) f_next[k] = MODE == kModeColsum ? fetch_factor(t0, k) : 0.f;
            for (int t = t0; t < t1; ++t, ++step) {
                const int buf = step & 1;
                if (MODE == kModeColsum) {
                    __syncwarp();
#pragma unroll
                    for (int k = 0; k < 2; ++k) {
                        sh.cf[warp][buf][lane + 32 * k] = f_next[k];
                        if (t + 1 < t1) f_next[k] = fetch_factor(t + 1, k);
                    }
                    __syncwarp();
                }
                if (!tc_wait(&sh.t_full[buf], (unsigned)((step >> 1) & 1), abort_flag, wait_limit)) { alive = false; break; }
                tc_fence_after();
#pragma unroll
                for (int ch = 0; ch < 2; ++ch) {
                    uint32_t v[32];
                    tc_ld32(t_lane + buf * kTcTile + ch * 32, v);
                    tc_ld_wait();
                    if (ch == 1) {  // the tile is in registers: the MMA may overwrite this buffer
                        tc_fence_before();
                        tc_mbar_arrive(&sh.t_empty[buf]);
                    }
                    const int cbase = half * 64 + ch * 32;  // first tile column of this chunk
                    if (MODE == kModeStats) {
                        const int nv = qi - (t * kTcTile + cbase) + 1;  // keys of this chunk that query qi sees
                        if (row_ok && nv >= 32 && sl2 >= 0.f) {
                            float r0 = __uint_as_float(v[0]), r1 = __uint_as_float(v[1]), r2 = __uint_as_float(v[2]), r3 = __uint_as_float(v[3]);
#pragma unroll
                            for (int c = 4; c < 32; c += 4) {
                                r0 = fmaxf(r0, __uint_as_float(v[c]));
                                r1 = fmaxf(r1, __uint_as_float(v[c + 1]));
                                r2 = fmaxf(r2, __uint_as_float(v[c + 2]));
                                r3 = fmaxf(r3, __uint_as_float(v[c + 3]));
                            }
                            const float rm = fmaxf(fmaxf(r0, r1), fmaxf(r2, r3));
                            const float mx = fmaxf(m, rm * sl2), nmx = -mx;
                            float l0 = lsum * exp2_diff(m, mx), l1 = 0.f, l2 = 0.f, l3 = 0.f;
#pragma unroll
                            for (int c = 0; c < 32; c += 4) {
                                l0 += fast_exp2(fmaf(__uint_as_float(v[c]), sl2, nmx));
                                l1 += fast_exp2(fmaf(__uint_as_float(v[c + 1]), sl2, nmx));
                                l2 += fast_exp2(fmaf(__uint_as_float(v[c + 2]), sl2, nmx));
                                l3 += fast_exp2(fmaf(__uint_as_float(v[c + 3]), sl2, nmx));
                            }
                            lsum = (l0 + l1) + (l2 + l3);
                            m = mx;
                        } else if (row_ok && nv > 0) {
                            float mx = m;
#pragma unroll
                            for (int c = 0; c < 32; ++c) {
                                const float x = __uint_as_float(v[c]) * sl2;
                                v[c] = __float_as_uint(x);
                                if (c < nv) mx = fmaxf(mx, x);
                            }
                            float l0 = lsum * exp2_diff(m, mx), l1 = 0.f;
#pragma unroll
                            for (int c = 0; c < 32; c += 2) {
                                if (c < nv) l0 += fast_exp2(__uint_as_float(v[c]) - mx);
                                if (c + 1 < nv) l1 += fast_exp2(__uint_as_float(v[c + 1]) - mx);
                            }
                            lsum = l0 + l1;
                            m = mx;
                        }
                    } else {
                        // tile column cc = (query t qpb + cc / G, head cc % G) counts for key j when its query >= j
                        const int c_lo = (ab * kTcTile + r - t * qpb) * G - cbase;  // first counted column of this chunk
                        const int c_hi = used - cbase;                             // columns beyond are unused
                        const float4* cf4 = reinterpret_cast<const float4*>(sh.cf[warp][buf] + ch * 32);
                        if (row_ok && c_lo <= 0 && c_hi >= 32) {
#pragma unroll
                            for (int c = 0; c < 32; c += 4) {
                                const float4 fb = cf4[c / 4];  // biases of columns c .. c + 3
                                acc0 += fast_exp2(fmaf(__uint_as_float(v[c]), sl2, fb.x));
                                acc1 += fast_exp2(fmaf(__uint_as_float(v[c + 1]), sl2, fb.y));
                                acc2 += fast_exp2(fmaf(__uint_as_float(v[c + 2]), sl2, fb.z));
                                acc3 += fast_exp2(fmaf(__uint_as_float(v[c + 3]), sl2, fb.w));
                            }
                        } else if (row_ok && c_lo < 32 && c_hi > 0) {
#pragma unroll
                            for (int c = 0; c < 32; c += 4) {
                                const float4 fb = cf4[c / 4];
                                if (c >= c_lo && c < c_hi) acc0 += fast_exp2(fmaf(__uint_as_float(v[c]), sl2, fb.x));
                                if (c + 1 >= c_lo && c + 1 < c_hi) acc1 += fast_exp2(fmaf(__uint_as_float(v[c + 1]), sl2, fb.y));
                                if (c + 2 >= c_lo && c + 2 < c_hi) acc2 += fast_exp2(fmaf(__uint_as_float(v[c + 2]), sl2, fb.z));
                                if (c + 3 >= c_lo && c + 3 < c_hi) acc3 += fast_exp2(fmaf(__uint_as_float(v[c + 3]), sl2, fb.w));
                            }
                        }
                    }
                }
            }
            if (alive && row_ok) {
                if (MODE == kModeStats) a.stats[half * half_stride + ((size_t)item * P + qi) * HP + r % G] = make_float2(m, lsum);
                else atomicAdd(a.rel + (size_t)item * a.cap_tokens + ab * kTcTile + r, (acc0 + acc1) + (acc2 + acc3));
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    if (sh.abort) {  // uniform for the CTA
        if (tid == 0) record_error(a.status, LETHE_ERR_TIMEOUT, item);
        if (warp == kTcMmaWarp && lane == 0 && sh.mma_steps > 0) {
            tc_commit(&sh.mma_drained);  // arrives once every MMA issued so far has finished
            drain(&sh.mma_drained, 0u);
        }
        if (TMA && warp == kTcMmaWarp + 1 && lane == 0) {  // boxes issued but perhaps not landed yet
            const int aa = sh.armed_a, steps = sh.armed_steps;
            if (aa >= 0) drain(&sh.a_full[aa % kTcABuffers], (unsigned)((aa / kTcABuffers) & 1));
            for (int st = max(0, steps - kTcStages); st < steps; ++st)
                drain(&sh.b_full[st % kTcStages], (unsigned)((st / kTcStages) & 1));
        }
        tc_fence_before();
        __syncthreads();
        tc_fence_after();
    }
    if (warp == kTcMmaWarp)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTcTmemCols) : "memory");
}

template <int D, bool TMA>
cudaError_t launch_tc(const PrefillArgs& a, const TcMaps& maps, int items, cudaStream_t stream) {
    const size_t smem = 1024 + (size_t)(kTcABuffers + kTcStages) * kTcTile * D * 2;
    cudaError_t e = prepare_kernel((const void*)prefill_tc_kernel<D, kModeStats, TMA>, smem);
    if (e != cudaSuccess) return e;
    e = prepare_kernel((const void*)prefill_tc_kernel<D, kModeColsum, TMA>, smem);
    if (e != cudaSuccess) return e;
    prefill_tc_kernel<D, kModeStats, TMA><<<items, tc_threads<TMA>(), smem, stream>>>(a, maps);
    prefill_tc_kernel<D, kModeColsum, TMA><<<items, tc_threads<TMA>(), smem, stream>>>(a, maps);
    return cudaGetLastError();
}

}  // namespace

// Two (max, sum) partials per (query, head) column.
size_t prefill_tc_stats_bytes(int items, int P, int HP) { return 2 * (size_t)items * P * HP * sizeof(float2); }

// encode: cuTensorMapEncodeTiled resolved by the caller, or NULL; the TMA path is taken when it is there, `allow_tma`
// is set and the maps can be made, the cp.async path otherwise.
cudaError_t launch_prefill_tc(const PrefillArgs& a, int items, int L, int D, void* encode, bool allow_tma, cudaStream_t stream) {
    TcMaps maps;
    memset(&maps, 0, sizeof(maps));
    bool tma = false;
    // paged pools take one box per page: pages of 16 to 128 tokens that divide the 128-row tile
    const bool pages_ok = !a.paged || (a.page_tokens >= 16 && a.page_tokens <= kTcTile && kTcTile % a.page_tokens == 0 &&
                                       a.n_pages <= 0x7fffffffLL);
    if (encode && allow_tma && pages_ok) {
        typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                      const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                      CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
        encode_fn fn = reinterpret_cast<encode_fn>(encode);
        const cuuint32_t qpb = (cuuint32_t)(kTcTile / a.G);
        const cuuint64_t rows = a.paged ? (cuuint64_t)a.page_tokens : (cuuint64_t)a.capacity;   // rows of one item / page
        const cuuint64_t kd[3] = {(cuuint64_t)D, rows, a.paged ? (cuuint64_t)a.n_pages : (cuuint64_t)items};
        const cuuint64_t ks[2] = {(cuuint64_t)D * 2, rows * D * 2};
        const cuuint32_t kb[3] = {64, a.paged ? (cuuint32_t)a.page_tokens : (cuuint32_t)kTcTile, 1};
        const cuuint64_t qd[4] = {(cuuint64_t)D, (cuuint64_t)a.Hq, (cuuint64_t)a.P, (cuuint64_t)L * a.B};
        const cuuint64_t qs[3] = {(cuuint64_t)D * 2, (cuuint64_t)a.Hq * D * 2, (cuuint64_t)a.P * a.Hq * D * 2};
        const cuuint32_t qb[4] = {64, (cuuint32_t)a.G, qpb, 1};
        const cuuint32_t es[4] = {1, 1, 1, 1};
        const CUresult r1 = fn(&maps.k, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(a.k), kd, ks, kb, es,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        const CUresult r2 = fn(&maps.q, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 4, const_cast<void*>(a.q), qd, qs, qb, es,
                               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
        tma = r1 == CUDA_SUCCESS && r2 == CUDA_SUCCESS;
    }
    if (tma) return D == 128 ? launch_tc<128, true>(a, maps, items, stream) : launch_tc<64, true>(a, maps, items, stream);
    return D == 128 ? launch_tc<128, false>(a, maps, items, stream) : launch_tc<64, false>(a, maps, items, stream);
}

}  // namespace lethe

