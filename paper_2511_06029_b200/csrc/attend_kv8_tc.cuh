// Persistent decode-attend kernel for quantised caches on the fifth-generation tensor cores (D = 128, G <= 8,
// e4m3 or e5m2 bytes with one scale per layer, contiguous or 16-token pages).
//
// The mma.sync kernels for byte caches spend their issue slots turning bytes into f16 (about 400 instructions per
// 16-token group) and stop at three quarters of the copy bandwidth.  tcgen05.mma.kind::f8f6f4 reads e4m3 / e5m2
// operands straight from shared memory, so here no cache byte is ever converted:
//
//   logits   S[128 tokens x N] = K tile [128 x 128 B, as TMA left it]  .  Qs^T      (4 MMAs of K = 32 per tile)
//   output   O^T[128 dims x N] += V tile^T (the same memory image, read MN-major) . Ps^T
//
// The other operand has to be an 8-bit float as well.  A bf16 query value is split exactly into three e4m3 terms,
// q = t1 + t2 / 16 + t3 / 256 (after its row has been divided by a power of two that puts the row's largest magnitude
// into e4m3's range; the head's logits are multiplied back), and the probabilities likewise, p * 256 = u1 + u2 / 16 + u3 / 256 (12 bits, one more
// than the f16 the mma.sync kernels round them to); the terms sit on the N axis (N = 3 G padded to 16 or 32) and
// are recombined from the fp32 accumulators, once per token for the logits and once per item for the output.
//
// An item is processed in two streaming phases, K tiles then V tiles, so every cache byte still crosses HBM once:
//   phase 1  logits of all tiles -> parked in shared memory (head-major; in the instances for wide groups and large
//            capacities the tail of an item longer than that buffer goes to a per-CTA slice of global scratch, which
//            stays in L2), running maximum per thread;
//   phase 2  with the exact maximum known: p = exp2(s - m) from the parked logits, row sums, the three terms of p
//            written as bytes in the MMA's operand layout, output accumulated in tensor memory — no online
//            rescaling and no correction step;
//   tail     1 / l, output rows from tensor memory, Eq. 5 from the parked logits (the same exact normaliser).
//
// One CTA per SM walks the launch's items (atomic ticket queue, longest first when an order is known).  Roles:
//   warp 11    set-up, one item ahead: draws the ticket, appends the new row (quantised), splits the item's query
//              rows into the B operand, publishes the item's descriptor;
//   warp 8     one lane streams the K tiles by TMA into a ring of 16 KB slots, running ahead of its consumer by the
//              depth of the ring, across item boundaries;
//   warp 12    the same for the V tiles, into a ring of their own;
//   warp 9     one lane issues the logit MMAs (K tiles); the warp owns the tensor-memory allocation;
//   warp 10    one lane issues the output MMAs (V tiles);
//   warps 0-7  NG = 2 softmax groups of four (with three, the role warps follow at 12: measured, no gain, not instantiated);
//              group g owns items g, g + NG, ... of the CTA's sequence, start to finish (thread =
//              token in phase 1, thread = (head, four tokens) in phase 2, thread = dimension for the output rows).
// The K stream runs about an item ahead of the V stream, so the groups are in different phases: while one
// computes probabilities and finishes its item, the other parks the next item's logits, and the streams from HBM
// do not pause for a phase change or a tail.  The two streams are independent (a ring, a producer and a consumer
// each): issued in one fixed interleaved order, the stream whose consumer is momentarily behind would hold the
// other one's copies back and leave its slots empty.
// All hand-offs are mbarriers (tcgen05.commit on the MMA side); every wait is bounded and a timeout ends the CTA
// with LETHE_ERR_TIMEOUT after it has waited for its own copies and MMAs and freed its tensor memory.
#pragma once
#include <cuda.h>
#include <cuda_fp16.h>
#include <string.h>

#include "common.cuh"
#include "mma_utils.cuh"

namespace lethe {

size_t kv8_tc_smem_bytes(int nslot, int G, int cap_pad, int ng);

namespace {

constexpr int kTile = 128;                  // tokens per tile
constexpr int kRowB = 128;                  // bytes per cache row (D = 128, one byte per element)
constexpr int kTileBytes = kTile * kRowB;   // 16 KB: one K tile or one V tile
constexpr int kMaxSlots = 8;                // ring slots
constexpr int kMaxNG = 3;                   // softmax groups of four warps the header has room for (the kernel is instantiated with two)
constexpr int kGroupThreads = 128;          // threads of one softmax group = tokens of a tile = lanes of tensor memory
constexpr int kRoleWarps = 5;               // after the softmax warps: K producer, K MMA, V MMA, set-up, V producer
constexpr int kGB = 4;                      // per group: logit tiles in tensor memory, and probability tiles in shared memory, in flight
constexpr int kMaxBufs = kMaxNG * kGB;
static_assert(kGB == 4, "buffer numbers are taken as (tile count) & 3");
constexpr int kTmemCols = 512;              // logit buffers at columns 32 i (i < 4 NG); the groups' output accumulators behind them, 32 columns each
constexpr int kTc8WaitLimit = 400000;
constexpr int kRelPf = 6;                   // tokens per thread whose old relevance is fetched before the tail

struct alignas(64) Kv8Maps {
    CUtensorMap k, v;      // box = a whole tile (128 rows) of a contiguous cache, one page (16 rows) of a paged one
    CUtensorMap k16, v16;  // box = 16 rows: the partly filled last tile of an item is fetched in 16-row pieces
};

struct Kv8Desc {
    int valid, item, li, l, b, hkv, n_old, n, full, T;
    float qmul[kMaxGroup];  // per head: the power of two its query row was divided by before the split (see the set-up warp)
};

struct Kv8Header {
    unsigned long long full[kMaxSlots], empty[kMaxSlots];
    unsigned long long s_full[kMaxBufs], s_empty[kMaxBufs], p_full[kMaxBufs], p_empty[kMaxBufs];   // buffers kGB g .. kGB g + kGB - 1 belong to group g
    unsigned long long q_full[kMaxNG], q_empty[kMaxNG], o_full[kMaxNG], o_empty[kMaxNG];         // by group = item number modulo NG
    unsigned long long sync[kMaxNG][3];  // the three meeting points of a group's 128 threads in an item (bounded, unlike bar.sync)
    unsigned long long drained[2];
    Kv8Desc desc[8];
    uint32_t tmem_base;
    int abort;
    int issued_tiles[2];  // producer: K / V tiles issued when it left its loop (for the drain after a timeout)
    int mma_steps[2];
    float red_m[4 * kMaxNG][kMaxGroup];
    float red_l[4 * kMaxNG][2];
};

__device__ __forceinline__ void bar_init(unsigned long long* b, int count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(b)), "r"(count) : "memory");
}
__device__ __forceinline__ void bar_arrive(unsigned long long* b) {
    asm volatile("{ .reg .b64 st; mbarrier.arrive.shared::cta.b64 st, [%0]; }" ::"r"(smem_u32(b)) : "memory");
}
__device__ __forceinline__ void bar_expect_tx(unsigned long long* b, unsigned bytes) {
    asm volatile("{ .reg .b64 st; mbarrier.arrive.expect_tx.shared::cta.b64 st, [%0], %1; }" ::"r"(smem_u32(b)), "r"(bytes) : "memory");
}
__device__ __forceinline__ bool bar_try(unsigned long long* b, unsigned parity) {
    unsigned ok;
    asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok)
                 : "r"(smem_u32(b)), "r"(parity)
                 : "memory");
    return ok != 0;
}
__device__ __forceinline__ bool bar_test(unsigned long long* b, unsigned parity) {
    unsigned ok;
    asm volatile("{ .reg .pred p; mbarrier.test_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                 : "=r"(ok)
                 : "r"(smem_u32(b)), "r"(parity)
                 : "memory");
    return ok != 0;
}
// Bounded wait; false = gave up (or another thread already did).  The first look never blocks.
__device__ __forceinline__ bool bar_wait(unsigned long long* b, unsigned parity, volatile int* abort_flag, int limit) {
    if (bar_test(b, parity)) return true;
    for (int it = 1; it < limit; ++it) {
        if (bar_try(b, parity)) return true;
        if (*abort_flag) return false;
        if (it > 64) __nanosleep(64);
    }
    *abort_flag = 1;
    return false;
}
// One lane of a converged warp (the compiler can then keep what that lane issues on the uniform datapath, which the
// descriptor operands of tcgen05.mma and of the bulk copies want).
__device__ __forceinline__ bool elect_one() {
    unsigned ok;
    asm volatile("{ .reg .pred p; elect.sync _|p, 0xffffffff; selp.u32 %0, 1, 0, p; }" : "=r"(ok));
    return ok != 0;
}
__device__ __forceinline__ void tc_before() { asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void tc_after() { asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory"); }
__device__ __forceinline__ void proxy_fence_shared() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }
__device__ __forceinline__ void proxy_fence_all() { asm volatile("fence.proxy.async;" ::: "memory"); }
__device__ __forceinline__ void commit_to(unsigned long long* b) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(smem_u32(b)) : "memory");
}
// One box of a 2-D byte tensor map (128 bytes x `rows of the map's box`) into shared memory.
__device__ __forceinline__ void tma_rows(uint32_t dst, const CUtensorMap* map, int row, unsigned long long* bar, uint64_t policy) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.L2::cache_hint [%0], [%1, {%2, %3}], [%4], %5;"
        ::"r"(dst), "l"(map), "r"(0), "r"(row), "r"(smem_u32(bar)), "l"(policy)
        : "memory");
}
// Shared-memory matrix descriptor: rows of 128 bytes, 128-byte swizzle, 8-row groups 1024 bytes apart.  The same
// form serves a K-major operand (the row is the contraction axis) and an MN-major one (the row is the M axis).
__device__ __forceinline__ uint64_t sw128_desc(uint32_t saddr) {
    uint64_t d = 0;
    d |= (uint64_t)((saddr & 0x3FFFFu) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor of tcgen05.mma.kind::f8f6f4: fp32 accumulate, A format 0 = e4m3 / 1 = e5m2, B = e4m3,
// A read K-major (0) or MN-major (1), B K-major, M = 128, N columns.
__device__ __forceinline__ uint32_t f8_idesc(int a_fmt, int a_mn_major, int N) {
    uint32_t d = 0;
    d |= 1u << 4;
    d |= (uint32_t)a_fmt << 7;
    d |= (uint32_t)a_mn_major << 15;
    d |= (uint32_t)(N >> 3) << 17;
    d |= (uint32_t)(128 >> 4) << 24;
    return d;
}
__device__ __forceinline__ void f8_mma(uint32_t d_tmem, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{ .reg .pred p; setp.ne.b32 p, %4, 0; tcgen05.mma.cta_group::1.kind::f8f6f4 [%0], %1, %2, %3, p; }"
        ::"r"(d_tmem), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate)
        : "memory");
}
template <int NP>
__device__ __forceinline__ void tmem_ld(uint32_t taddr, uint32_t (&v)[NP]) {
    if constexpr (NP == 16) {
        asm volatile(
            "tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
            : "=r"(v[0]), "=r"(v[1]), "=r"(v[2]), "=r"(v[3]), "=r"(v[4]), "=r"(v[5]), "=r"(v[6]), "=r"(v[7]), "=r"(v[8]),
              "=r"(v[9]), "=r"(v[10]), "=r"(v[11]), "=r"(v[12]), "=r"(v[13]), "=r"(v[14]), "=r"(v[15])
            : "r"(taddr)
            : "memory");
    } else {
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
    asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
}

// two fp32 -> two fp8 bytes (round to nearest even, saturating), `lo` in the low byte
template <bool E5M2>
__device__ __forceinline__ uint32_t to_fp8x2(float lo, float hi) {
    uint32_t y;
    if (E5M2) asm("{ .reg .b16 r; cvt.rn.satfinite.e5m2x2.f32 r, %2, %1; cvt.u32.u16 %0, r; }" : "=r"(y) : "f"(lo), "f"(hi));
    else asm("{ .reg .b16 r; cvt.rn.satfinite.e4m3x2.f32 r, %2, %1; cvt.u32.u16 %0, r; }" : "=r"(y) : "f"(lo), "f"(hi));
    return y;
}
__device__ __forceinline__ float2 e4m3x2_to_f32x2(uint32_t x) {
    uint32_t y;
    asm("{ .reg .b16 lo; cvt.u16.u32 lo, %1; cvt.rn.f16x2.e4m3x2 %0, lo; }" : "=r"(y) : "r"(x));
    return __half22float2(*reinterpret_cast<__half2*>(&y));
}
// Four values -> their three e4m3 terms, four bytes per term (value i in byte i): x = t1 + t2 / 16 + t3 / 256.
__device__ __forceinline__ void split3(float x0, float x1, float x2, float x3, uint32_t (&w)[3]) {
#pragma unroll
    for (int t = 0; t < 3; ++t) {
        const uint32_t lo = to_fp8x2<false>(x0, x1), hi = to_fp8x2<false>(x2, x3);
        w[t] = lo | (hi << 16);
        if (t < 2) {
            const float2 a = e4m3x2_to_f32x2(lo), b = e4m3x2_to_f32x2(hi);
            x0 = (x0 - a.x) * 16.f;
            x1 = (x1 - a.y) * 16.f;
            x2 = (x2 - b.x) * 16.f;
            x3 = (x3 - b.y) * 16.f;
        }
    }
}
// byte offset `col` (a multiple of 4) of row `row` in a 128-byte-swizzled operand tile
__device__ __forceinline__ uint32_t sw128_at(uint32_t base, int row, int col) {
    return base + row * 128 + ((((col >> 4) ^ (row & 7)) << 4) | (col & 15));
}

// GT: the number of query heads per KV head when it is known at compile time (the loops over heads then carry no
// run-time bounds), 0 = read it from the arguments.
// SPILL: items may be longer than the on-chip logit buffer (cap_pad tokens per head); the logits of the tokens beyond
// it are parked in this CTA's slice of global scratch.  A separate instance, so that caches that fit pay nothing.
template <int NP, bool PAGED, bool E5M2, int NG, int GT, bool SPILL>
__global__ void __launch_bounds__((4 * NG + kRoleWarps) * 32, 1)
    attend_kv8_tc_kernel(const __grid_constant__ AttendArgs a, const __grid_constant__ Kv8Maps maps, int nslot, int cap_pad) {
    using T = __nv_bfloat16;
    extern __shared__ unsigned char dyn_raw[];
    // layout from a 1024-byte boundary: ring [nslot][16 KB] | query operand [NG][NP x 128 B] | probability operand
    // [NG groups][kGB][NP x 128 B] | parked logits [NG groups][G][cap_pad] fp32 | header
    const uint32_t base_u32 = (smem_u32(dyn_raw) + 1023u) & ~1023u;
    unsigned char* base = dyn_raw + (base_u32 - smem_u32(dyn_raw));
    const uint32_t ring_u32 = base_u32;
    const uint32_t qs_u32 = ring_u32 + (uint32_t)nslot * kTileBytes;
    constexpr int kBufs = NG * kGB, kOutCol = kBufs * 32;
    constexpr int kProducerWarp = 4 * NG, kMmaWarp = 4 * NG + 1, kPvWarp = 4 * NG + 2, kSetupWarp = 4 * NG + 3, kVProducerWarp = 4 * NG + 4;
    constexpr int kTcThreads = (4 * NG + kRoleWarps) * 32;
    static_assert(kOutCol + NG * 32 <= kTmemCols, "tensor memory columns");
    const uint32_t ps_u32 = qs_u32 + NG * NP * 128;
    float* park_all = reinterpret_cast<float*>(base + (size_t)nslot * kTileBytes + (NG + kBufs) * NP * 128);
    Kv8Header& hd = *reinterpret_cast<Kv8Header*>(reinterpret_cast<unsigned char*>(park_all) + (size_t)NG * a.G * cap_pad * 4);

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    const int G = GT ? GT : a.G;
    const bool append = a.k_new != nullptr;
    volatile int* abort_flag = &hd.abort;
    const int wait_limit = a.wait_limit > 0 ? a.wait_limit : kTc8WaitLimit;
    unsigned int* sched = a.sched;

    if (tid == 0) {
        for (int i = 0; i < kMaxSlots; ++i) {
            bar_init(&hd.full[i], 1);
            bar_init(&hd.empty[i], 1);
        }
        for (int i = 0; i < kBufs; ++i) {
            bar_init(&hd.s_full[i], 1);
            bar_init(&hd.s_empty[i], 4);  // one arrival per warp of the group (128 arrivals on one barrier serialise)
            bar_init(&hd.p_full[i], 4);
            bar_init(&hd.p_empty[i], 1);
        }
        for (int i = 0; i < NG; ++i) {
            bar_init(&hd.q_full[i], 1);
            bar_init(&hd.q_empty[i], 1 + 4 + 3);  // K thread's commit, the group's four warps, the V thread and the two TMA lanes
            bar_init(&hd.o_full[i], 1);
            bar_init(&hd.o_empty[i], 4);
            for (int j = 0; j < 3; ++j) bar_init(&hd.sync[i][j], 4);
        }
        bar_init(&hd.drained[0], 1);
        bar_init(&hd.drained[1], 1);
        hd.abort = 0;
        hd.issued_tiles[0] = hd.issued_tiles[1] = 0;
        hd.mma_steps[0] = hd.mma_steps[1] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    // the operand rows the splits never write (N is 3 G padded to NP) stay zero for the whole launch
    for (int i = tid; i < (NG + kBufs) * NP * 128 / 16; i += kTcThreads)
        asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(qs_u32 + i * 16), "r"(0) : "memory");
    proxy_fence_shared();
    if (warp == kMmaWarp) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&hd.tmem_base)), "r"(kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    // Everything above touches only this CTA's shared and tensor memory, so under a programmatic dependent launch it
    // runs while the previous kernel of the stream is still finishing; nothing global is read before this point.
    asm volatile("griddepcontrol.wait;" ::: "memory");
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");
    tc_before();
    __syncthreads();
    tc_after();
    const uint32_t tmem = hd.tmem_base;
    const int nk = (nslot + 1) >> 1, nv = nslot - nk;  // slots of the K ring and of the V ring

    // Item e of this CTA's sequence belongs to softmax group e & 1: while one group turns logits into probabilities and
    // finishes its item, the other is already parking the next item's logits.
    if (warp == kSetupWarp) {
        // ============================================================ setup: queue, append, query split — one item ahead of
        // the stream (one query operand buffer and one set of item barriers per group), so that the global
        // round trips of an item's set-up (ticket, length, new row, query rows) never hold the tile stream up
        int ended = 0;  // end-of-work descriptors published so far: each group needs one
        bool bad_page = false;
        for (int e = 0; ended < NG; ++e) {
            Kv8Desc d;
            d.valid = 0;
            d.T = 0;
            const int par = e % NG;  // the item's group; the query operand and the barriers of an item go by it
            int ticket = a.n_items;
            if (ended == 0) {
                if (lane == 0) ticket = (int)atomicAdd(&sched[0], 1u);
                ticket = __shfl_sync(0xffffffffu, ticket, 0);
            }
            d.valid = ticket < a.n_items;
            if (e >= NG && !bar_wait(&hd.q_empty[par], (unsigned)(((e / NG) - 1) & 1), abort_flag, wait_limit)) break;
            if (d.valid) {
                const int t = a.order ? a.order[ticket] : ticket;
                d.hkv = t % a.Hkv;
                d.b = (t / a.Hkv) % a.B;
                d.li = t / (a.Hkv * a.B);
                d.l = a.layer_begin + d.li;
                d.item = (d.l * a.B + d.b) * a.Hkv + d.hkv;
                // the query rows are requested first: with the step's inputs in host memory they, the length and the
                // appended row then share one trip over the bus instead of queueing behind each other
                const T* q = (const T*)a.q + ((size_t)(d.li * a.B + d.b) * a.Hq + d.hkv * G) * 128;
                uint2 qw[kMaxGroup];  // lane holds dims 4 lane .. 4 lane + 3 of every head
#pragma unroll
                for (int h = 0; h < kMaxGroup; ++h)
                    qw[h] = h < G ? *reinterpret_cast<const uint2*>(q + h * 128 + lane * 4) : make_uint2(0u, 0u);
                d.n_old = a.len[d.item];
                d.full = append && d.n_old >= a.cap_tokens;
                d.n = d.full ? 0 : d.n_old + (append ? 1 : 0);
                d.T = max(1, (d.n + kTile - 1) / kTile);
                __syncwarp();  // every lane has read len before lane 0 stores the new length
                if (append && !d.full) {  // Sec. 4.1: the generated token's key / value, quantised, into slot n_old
                    const size_t src = ((size_t)(d.li * a.B + d.b) * a.Hkv + d.hkv) * 128;
                    bool bad = false;
                    char* kd = const_cast<char*>(row_ptr<PAGED>(a, a.k, d.item, d.n_old, kRowB, &bad));
                    char* vd = const_cast<char*>(row_ptr<PAGED>(a, a.v, d.item, d.n_old, kRowB, &bad));
                    if (bad) bad_page = true;
                    if (kd && vd) {
                        const float ks_l = a.k_scale[d.l], vs_l = a.v_scale[d.l];
                        const uint2 kw = *reinterpret_cast<const uint2*>((const T*)a.k_new + src + lane * 4);
                        const uint2 vw = *reinterpret_cast<const uint2*>((const T*)a.v_new + src + lane * 4);
                        auto quant4 = [](uint2 w, float s) -> uint32_t {
                            const float x0 = __uint_as_float(w.x << 16), x1 = __uint_as_float(w.x & 0xffff0000u);
                            const float x2 = __uint_as_float(w.y << 16), x3 = __uint_as_float(w.y & 0xffff0000u);
                            return to_fp8x2<E5M2>(__fdiv_rn(x0, s), __fdiv_rn(x1, s)) | (to_fp8x2<E5M2>(__fdiv_rn(x2, s), __fdiv_rn(x3, s)) << 16);
                        };
                        *reinterpret_cast<uint32_t*>(kd + lane * 4) = quant4(kw, ks_l);
                        *reinterpret_cast<uint32_t*>(vd + lane * 4) = quant4(vw, vs_l);
                    }
                    if (lane == 0) {
                        a.pos[(size_t)d.item * a.cap_tokens + d.n_old] = a.token_pos[d.b];
                        a.len[d.item] = d.n;
                    }
                    proxy_fence_all();  // the new rows are read back by TMA (the async proxy) below
                }
                // the item's query rows as the B operand of the logit MMAs: row (term * G + h), 128 bytes of d
                // e4m3 covers 2^-9 .. 448, so each row is first divided by a power of two that brings its largest
                // magnitude into [128, 256) (exact; the three terms then hold every bf16 value of the row down to 2^-25
                // of that maximum); the logits of the head are multiplied back when they are read out of tensor memory
                const uint32_t qb = qs_u32 + par * NP * 128;
#pragma unroll
                for (int h = 0; h < kMaxGroup; ++h) {
                    d.qmul[h] = 1.f;
                    if (h < G) {
                        float x0 = __uint_as_float(qw[h].x << 16), x1 = __uint_as_float(qw[h].x & 0xffff0000u);
                        float x2 = __uint_as_float(qw[h].y << 16), x3 = __uint_as_float(qw[h].y & 0xffff0000u);
                        float big = fmaxf(fmaxf(fabsf(x0), fabsf(x1)), fmaxf(fabsf(x2), fabsf(x3)));
#pragma unroll
                        for (int off = 16; off > 0; off >>= 1) big = fmaxf(big, __shfl_xor_sync(0xffffffffu, big, off));
                        // exponent field of the maximum -> 2^(e - 7), clamped so that both it and its inverse are normal
                        int ex = (int)((__float_as_uint(big) >> 23) & 0xffu) - 7;   // biased exponent of the divisor
                        ex = big > 0.f && big < INFINITY ? min(max(ex, 2), 252) : 127;
                        const float div = __uint_as_float((uint32_t)ex << 23), inv = __uint_as_float((uint32_t)(254 - ex) << 23);
                        d.qmul[h] = div;
                        x0 *= inv; x1 *= inv; x2 *= inv; x3 *= inv;
                        uint32_t terms[3];
                        split3(x0, x1, x2, x3, terms);
#pragma unroll
                        for (int t3 = 0; t3 < 3; ++t3)
                            asm volatile("st.shared.b32 [%0], %1;" ::"r"(sw128_at(qb, t3 * G + h, lane * 4)), "r"(terms[t3]) : "memory");
                    }
                }
                proxy_fence_shared();
            }
            __syncwarp();
            if (lane == 0) {
                hd.desc[e & 7] = d;
                bar_arrive(&hd.q_full[par]);
            }
            if (!d.valid) ++ended;
        }
        if (lane == 0 && bad_page) record_error(a.status, LETHE_ERR_PAGE, 0);
    } else if (warp == kProducerWarp || warp == kVProducerWarp) {
        // ============================================================ producers: one lane streams K tiles, one V tiles
        // Two rings, K slots [0, nk) and V slots [nk, nslot): every slot's barriers have exactly one consumer, which
        // sees each of the slot's phases in turn.  (With one shared ring the thread that skips the other's tiles can get
        // two phases ahead of a slot, or behind it, and a parity wait cannot tell those apart.)
        {
            const bool is_k = warp == kProducerWarp;
            const uint64_t policy = l2_evict_first_policy();
            const CUtensorMap* map = is_k ? &maps.k : &maps.v;
            const CUtensorMap* map16 = is_k ? &maps.k16 : &maps.v16;
            const int slot0 = is_k ? 0 : nk, nring = is_k ? nk : nv;
            int issued = 0;      // tiles issued so far
            int slot = 0;        // next slot of the ring (no division on this warp's path)
            int lap = 0;         // how often the ring has wrapped
            bool alive = true;
            bool bad_page = false;
            // Paged caches: lane pg < 8 owns page pg of every tile (one 16-row box each); it fetches the id of its page
            // of the next tile before the current tile is issued, so the table's latency is off the stream's path.
            auto page_of = [&](const Kv8Desc& d, int t) -> int {
                const int en = t * 8 + lane;
                int page = -1;
                if (lane < 8 && t < d.T && en < a.capacity && en * kGroupTokens < d.n) {
                    page = a.page_table[(size_t)d.item * a.capacity + en];
                    if (page < 0 || page >= a.n_pages) {
                        page = -1;
                        bad_page = true;
                    }
                }
                return page;
            };
            for (int e = 0; alive; ++e) {
                if (!bar_wait(&hd.q_full[e % NG], (unsigned)((e / NG) & 1), abort_flag, wait_limit)) break;
                const Kv8Desc d = hd.desc[e & 7];
                __syncwarp();
                if (lane == 0) bar_arrive(&hd.q_empty[e % NG]);
                if (!d.valid) break;
                int page_next = PAGED ? page_of(d, 0) : -1;
                for (int t = 0; t < d.T; ++t) {
                    const int ps = slot0 + slot;
                    if (lap >= 1 && !bar_wait(&hd.empty[ps], (unsigned)((lap - 1) & 1), abort_flag, wait_limit)) { alive = false; break; }
                    const uint32_t dst = ring_u32 + ps * kTileBytes;
                    if (!PAGED) {
                        if (lane == 0) {
                            const int row0 = d.item * a.capacity + t * kTile, rows_valid = d.n - t * kTile;
                            if (rows_valid > kTile - kGroupTokens) {
                                bar_expect_tx(&hd.full[ps], kTileBytes);
                                tma_rows(dst, map, row0, &hd.full[ps], policy);
                            } else {
                                // the item's last tile: only the 16-row pieces that hold tokens cross HBM; the rows
                                // behind them keep what the slot held (masked on the K side, zeroed on the V side)
                                const int pieces = (max(rows_valid, 0) + kGroupTokens - 1) / kGroupTokens;
                                bar_expect_tx(&hd.full[ps], (unsigned)(pieces * kGroupTokens * kRowB));
                                for (int pc = 0; pc < pieces; ++pc)
                                    tma_rows(dst + pc * kGroupTokens * kRowB, map16, row0 + pc * kGroupTokens, &hd.full[ps], policy);
                            }
                        }
                    } else {
                        // one box per 16-token page; pages past the item's end and bad ids are skipped
                        const int page = page_next;
                        page_next = page_of(d, t + 1);
                        const unsigned have = __ballot_sync(0xffffffffu, page >= 0);
                        if (lane == 0) bar_expect_tx(&hd.full[ps], (unsigned)(__popc(have) * kGroupTokens * kRowB));  // (zero bytes: the arrival alone completes the phase)
                        __syncwarp();
                        if (page >= 0) tma_rows(dst + lane * kGroupTokens * kRowB, map, page * kGroupTokens, &hd.full[ps], policy);
                    }
                    __syncwarp();
                    ++issued;
                    if (++slot == nring) {
                        slot = 0;
                        ++lap;
                    }
                }
            }
            if (lane == 0) hd.issued_tiles[is_k ? 0 : 1] = issued;
            if (__any_sync(0xffffffffu, bad_page) && lane == 0 && is_k) record_error(a.status, LETHE_ERR_PAGE, 0);
        }
        __syncwarp();
    } else if (warp == kMmaWarp || warp == kPvWarp) {
        // ============================================================ MMA issue: one lane of warp 9 issues the logit MMAs
        // (K tiles), one lane of warp 10 the output MMAs (V tiles), each walking its own ring in the producer's order.
        // A single thread taking both could not keep up, and even so the loop below is what the kernel's rate hangs
        // on: a 16 KB tile is four small MMAs, and every instruction around them (waits, descriptors, commits, ring
        // arithmetic) sits on one thread's dependent chain.  So nothing in it divides, indexes local memory or
        // rebuilds a descriptor: slots, phase bits and buffer numbers are carried along, descriptors are a base plus
        // an offset.  All lanes walk (the output warp's lanes share the zeroing of an item's last V tile); lane 0 issues.
        const bool do_k = warp == kMmaWarp;
        const uint32_t idesc = f8_idesc(E5M2 ? 1 : 0, do_k ? 0 : 1, NP);
        const uint64_t d_ring = sw128_desc(ring_u32), d_qs = sw128_desc(qs_u32), d_ps = sw128_desc(ps_u32);
        const int slot0 = do_k ? 0 : nk, nring = do_k ? nk : nv;
        int slot = 0, steps = 0;       // next slot of this thread's ring, MMAs batches issued
        unsigned lap = 0;              // phase bit of that slot's next tile
        unsigned c_grp[3] = {0u, 0u, 0u};  // tiles taken so far for each softmax group: buffer c & 3, phase c >> 2
        bool alive = true;
        for (int e = 0; alive; ++e) {
            const int par = e % NG;
            if (!bar_wait(&hd.q_full[par], (unsigned)((e / NG) & 1), abort_flag, wait_limit)) break;
            const Kv8Desc d = hd.desc[e & 7];
            __syncwarp();
            if (!do_k && lane == 0) bar_arrive(&hd.q_empty[par]);  // (the K thread's arrival is its commit after the item's last logit MMA)
            if (!d.valid) break;
            // item e belongs to softmax group par: the K thread takes its K tiles, the V thread (later) its V tiles
            const int grp = par;
            const int T = d.T;
            const int n_item = d.n;
            unsigned c = grp == 0 ? c_grp[0] : (grp == 1 ? c_grp[1] : c_grp[2]);
            const uint64_t d_q = d_qs + (uint64_t)(par * (NP * 128 >> 4));
            const uint32_t t_acc = do_k ? tmem + grp * kGB * 32 : tmem + kOutCol + grp * 32;
            if (!do_k && e >= NG) {  // the group has read its previous item's output out of tensor memory
                if (!bar_wait(&hd.o_empty[grp], (unsigned)(((e / NG) - 1) & 1), abort_flag, wait_limit)) break;
            }
            for (int t = 0; t < T; ++t) {
                const int ps = slot0 + slot, bi = (int)(c & 3u), bf = grp * kGB + bi;
                if (!bar_wait(&hd.full[ps], lap, abort_flag, wait_limit)) { alive = false; break; }
                const uint64_t d_tile = d_ring + (uint64_t)(ps * (kTileBytes >> 4));
                if (do_k) {  // ---- logits of K tile t of item e
                    if (c >= 4u && !bar_wait(&hd.s_empty[bf], ((c >> 2) - 1u) & 1u, abort_flag, wait_limit)) { alive = false; break; }
                    tc_after();
                    if (elect_one()) {
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)  // 32 bytes of the row (32 dims) per MMA
                            f8_mma(t_acc + bi * 32, d_tile + (uint64_t)(2 * ks), d_q + (uint64_t)(2 * ks), idesc, ks > 0 ? 1u : 0u);
                        commit_to(&hd.empty[ps]);
                        commit_to(&hd.s_full[bf]);
                        if (t == T - 1) commit_to(&hd.q_empty[par]);  // the query operand is free once its last logit MMA has read it
                    }
                } else {  // ---- output from V tile t of item e
                    if (!bar_wait(&hd.p_full[bf], (c >> 2) & 1u, abort_flag, wait_limit)) { alive = false; break; }
                    tc_after();
                    const int valid_rows = n_item - t * kTile;  // rows of this tile that hold tokens of the item
                    if (valid_rows < kTile) {
                        // the rows past the item's end hold whatever memory held (possibly NaN bytes): zero them, so
                        // that a zero probability times them stays zero
                        const uint32_t at = ring_u32 + ps * kTileBytes;
                        for (int r = max(valid_rows, 0) + lane; r < kTile; r += 32) {
#pragma unroll
                            for (int c16 = 0; c16 < 8; ++c16)
                                asm volatile("st.shared.v4.b32 [%0], {%1, %1, %1, %1};" ::"r"(at + r * kRowB + c16 * 16), "r"(0) : "memory");
                        }
                        proxy_fence_shared();
                        __syncwarp();
                    }
                    if (elect_one()) {
                        const uint64_t d_p = d_ps + (uint64_t)(bf * (NP * 128 >> 4));
#pragma unroll
                        for (int ks = 0; ks < 4; ++ks)  // 32 tokens per MMA: 32 rows of the V tile, 32 bytes of each probability row
                            f8_mma(t_acc, d_tile + (uint64_t)(ks * (32 * kRowB >> 4)), d_p + (uint64_t)(2 * ks), idesc, (t > 0 || ks > 0) ? 1u : 0u);
                        commit_to(&hd.empty[ps]);
                        commit_to(&hd.p_empty[bf]);
                        if (t == T - 1) commit_to(&hd.o_full[grp]);
                    }
                }
                __syncwarp();
                ++c;
                ++steps;
                if (++slot == nring) {
                    slot = 0;
                    lap ^= 1u;
                }
            }
            if (grp == 0) c_grp[0] = c;
            else if (grp == 1) c_grp[1] = c;
            else c_grp[2] = c;
        }
        if (lane == 0) hd.mma_steps[do_k ? 0 : 1] = steps;
        __syncwarp();
    } else {
        // ============================================================ softmax warps: group g owns items g, g + 2, ...
        const int g = warp >> 2, w4 = warp & 3;
        const int tg = w4 * 32 + lane;                             // thread within its group = TMEM lane
        const uint32_t t_lane = tmem + ((uint32_t)(w4 * 32) << 16);
        float* park = park_all + (size_t)g * G * cap_pad;
        // [CTA][group][head][a.spill_tokens]; a tile lies wholly on one side (cap_pad is a multiple of the tile)
        float* spill = SPILL ? a.spill + ((size_t)blockIdx.x * NG + g) * G * a.spill_tokens : nullptr;
        unsigned cs = 0, cw = 0;  // logit tiles read / probability tiles written by this group so far: buffer c & 3, phase c >> 2
        for (int seq = g, k = 0;; seq += NG, ++k) {
            if (!bar_wait(&hd.q_full[g], (unsigned)(k & 1), abort_flag, wait_limit)) break;
            const Kv8Desc d = hd.desc[seq & 7];
            __syncwarp();
            if (lane == 0) bar_arrive(&hd.q_empty[g]);
            if (!d.valid) break;
            float sl2h[kMaxGroup];  // softmax scale (log2 units) times the head's query divisor
#pragma unroll
            for (int h = 0; h < kMaxGroup; ++h) sl2h[h] = a.scale_log2[d.l] * d.qmul[h];
            const int n = d.n;
            bool alive = true;
            // ---- phase 1: logits of the item's K tiles, one token per thread
            float mx[kMaxGroup];
#pragma unroll
            for (int h = 0; h < kMaxGroup; ++h) mx[h] = -INFINITY;
            for (int t = 0; t < d.T; ++t) {
                const int bf = g * kGB + (int)(cs & 3u);
                const unsigned used = cs >> 2;
                ++cs;
                if (!bar_wait(&hd.s_full[bf], used & 1u, abort_flag, wait_limit)) { alive = false; break; }
                tc_after();
                uint32_t c[NP];
                tmem_ld<NP>(t_lane + bf * 32, c);
                tc_before();
                __syncwarp();
                if (lane == 0) bar_arrive(&hd.s_empty[bf]);
                const int tok = t * kTile + tg;
#pragma unroll
                for (int h = 0; h < kMaxGroup; ++h) {
                    if (h < G) {
                        float s = fmaf(__uint_as_float(c[2 * G + h]), 0.00390625f, fmaf(__uint_as_float(c[G + h]), 0.0625f, __uint_as_float(c[h])));
                        s = tok < n ? s * sl2h[h] : -INFINITY;
                        if (!SPILL || tok < cap_pad) park[(size_t)h * cap_pad + tok] = s;
                        else spill[(size_t)h * a.spill_tokens + (tok - cap_pad)] = s;
                        mx[h] = fmaxf(mx[h], s);
                    }
                }
            }
            if (!alive) break;
#pragma unroll
            for (int h = 0; h < kMaxGroup; ++h) {
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], off));
            }
            if (lane < kMaxGroup) {
                float v = -INFINITY;
#pragma unroll
                for (int h = 0; h < kMaxGroup; ++h)
                    if (h == lane) v = mx[h];
                hd.red_m[warp][lane] = v;
            }
            // the group's logits are parked and its maxima posted (a bounded meeting point: after a timeout nobody is left waiting)
            __syncwarp();
            if (lane == 0) bar_arrive(&hd.sync[g][0]);
            if (!bar_wait(&hd.sync[g][0], (unsigned)(k & 1), abort_flag, wait_limit)) break;
            float fm[kMaxGroup];
#pragma unroll
            for (int h = 0; h < kMaxGroup; ++h) {
                float v = -INFINITY;
#pragma unroll
                for (int w = 0; w < 4; ++w) v = fmaxf(v, hd.red_m[g * 4 + w][h]);
                fm[h] = v;
            }
            // ---- phase 2: probabilities of the item's V tiles: (head, four tokens) per thread and step
            float lacc[2] = {0.f, 0.f};
            for (int t = 0; t < d.T; ++t) {
                const int bf = g * kGB + (int)(cw & 3u);
                const unsigned used = cw >> 2;
                ++cw;
                if (used >= 1u && !bar_wait(&hd.p_empty[bf], (used - 1u) & 1u, abort_flag, wait_limit)) { alive = false; break; }
                const uint32_t pb = ps_u32 + bf * NP * 128;
#pragma unroll
                for (int i = 0; i < 2; ++i) {
                    const int h = w4 + 4 * i;
                    if (h < G) {
                        const float4 s4 = (!SPILL || t * kTile < cap_pad)
                                              ? *reinterpret_cast<const float4*>(park + (size_t)h * cap_pad + t * kTile + 4 * lane)
                                              : *reinterpret_cast<const float4*>(spill + (size_t)h * a.spill_tokens + (t * kTile - cap_pad) + 4 * lane);
                        const float off = 8.f - fm[h];  // probabilities are carried times 256: e4m3 keeps them normal down to 2^-14
                        const float p0 = s4.x == -INFINITY ? 0.f : fast_exp2(s4.x + off);
                        const float p1 = s4.y == -INFINITY ? 0.f : fast_exp2(s4.y + off);
                        const float p2 = s4.z == -INFINITY ? 0.f : fast_exp2(s4.z + off);
                        const float p3 = s4.w == -INFINITY ? 0.f : fast_exp2(s4.w + off);
                        lacc[i] += (p0 + p1) + (p2 + p3);
                        uint32_t terms[3];
                        split3(p0, p1, p2, p3, terms);
#pragma unroll
                        for (int t3 = 0; t3 < 3; ++t3)
                            asm volatile("st.shared.b32 [%0], %1;" ::"r"(sw128_at(pb, t3 * G + h, 4 * lane)), "r"(terms[t3]) : "memory");
                    }
                }
                proxy_fence_shared();  // every lane publishes its own bytes to the MMA's proxy, then one arrival per warp
                __syncwarp();
                if (lane == 0) bar_arrive(&hd.p_full[bf]);
            }
            if (!alive) break;
            // ---- tail: normalisers, outputs, Eq. 5
            float* rel = a.rel + (size_t)d.item * a.cap_tokens;
            const int app = (append && !d.full) ? d.n_old : -1;
            float rel_old[kRelPf];
#pragma unroll
            for (int i = 0; i < kRelPf; ++i) {
                const int j = tg + i * kGroupThreads;
                rel_old[i] = (j < n && j != app) ? rel[j] : 0.f;
            }
#pragma unroll
            for (int i = 0; i < 2; ++i) {
#pragma unroll
                for (int off = 16; off > 0; off >>= 1) lacc[i] += __shfl_xor_sync(0xffffffffu, lacc[i], off);
            }
            if (lane == 0) {
                hd.red_l[warp][0] = lacc[0];
                hd.red_l[warp][1] = lacc[1];
            }
            __syncwarp();
            if (lane == 0) bar_arrive(&hd.sync[g][1]);
            if (!bar_wait(&hd.sync[g][1], (unsigned)(k & 1), abort_flag, wait_limit)) break;
            float inv[kMaxGroup];
#pragma unroll
            for (int h = 0; h < kMaxGroup; ++h) {
                const float l = hd.red_l[g * 4 + (h & 3)][h >> 2] * 0.00390625f;  // sum of p
                inv[h] = l > 0.f ? 1.f / l : 0.f;
                if (a.lse && tg == h && h < G)
                    a.lse[(size_t)(d.li * a.B + d.b) * a.Hq + d.hkv * G + h] = l > 0.f ? (fm[h] + log2f(l)) * 0.6931471805599453f : -INFINITY;
            }
            if (d.full && tg == 0) record_error(a.status, LETHE_ERR_CAPACITY, d.item);
            if (!bar_wait(&hd.o_full[g], (unsigned)(k & 1), abort_flag, wait_limit)) break;
            {   // output rows: thread = dimension d, columns = (term, head)
                tc_after();
                uint32_t c[NP];
                tmem_ld<NP>(t_lane + kOutCol + g * 32, c);
                tc_before();
                __syncwarp();
                if (lane == 0) bar_arrive(&hd.o_empty[g]);
                T* out = (T*)a.out + ((size_t)(d.li * a.B + d.b) * a.Hq + d.hkv * G) * 128;
                const float vs = a.v_scale[d.l] * 0.00390625f;
#pragma unroll
                for (int h = 0; h < kMaxGroup; ++h) {
                    if (h < G) {
                        const float o = fmaf(__uint_as_float(c[2 * G + h]), 0.00390625f, fmaf(__uint_as_float(c[G + h]), 0.0625f, __uint_as_float(c[h])));
                        out[h * 128 + tg] = __float2bfloat16_rn(o * vs * inv[h]);
                    }
                }
            }
            // Eq. 5 from the parked logits with the exact (maximum, 1 / sum) of every head
            {
                auto mass_of = [&](int j) {
                    float mass = 0.f;
#pragma unroll
                    for (int h = 0; h < kMaxGroup; ++h)
                        if (h < G) {
                            const float sj = (!SPILL || j < cap_pad) ? park[(size_t)h * cap_pad + j] : spill[(size_t)h * a.spill_tokens + (j - cap_pad)];
                            mass += fast_exp2(sj - fm[h]) * inv[h];
                        }
                    return mass;
                };
#pragma unroll
                for (int i = 0; i < kRelPf; ++i) {
                    const int j = tg + i * kGroupThreads;
                    if (j < n) rel[j] = fmaf(a.gamma, rel_old[i], mass_of(j));
                }
                for (int j = tg + kRelPf * kGroupThreads; j < n; j += kGroupThreads) {
                    const float old = j == app ? 0.f : rel[j];
                    rel[j] = fmaf(a.gamma, old, mass_of(j));
                }
            }
            __syncwarp();
            if (lane == 0) bar_arrive(&hd.sync[g][2]);  // the group's parked logits are free for its next item once all of it is here
            if (!bar_wait(&hd.sync[g][2], (unsigned)(k & 1), abort_flag, wait_limit)) break;
        }
    }

    // ---- the way out: after a timeout, wait (bounded, built-in limit) for what this CTA started
    tc_before();
    __syncthreads();
    tc_after();
    if (hd.abort) {
        auto drain = [&](unsigned long long* b, unsigned parity) {
            for (int i = 0; i < kTc8WaitLimit; ++i) {
                if (bar_try(b, parity)) return;
                if (i > 64) __nanosleep(64);
            }
        };
        if (tid == 0) record_error(a.status, LETHE_ERR_TIMEOUT, (int)blockIdx.x);
        if ((warp == kMmaWarp || warp == kPvWarp) && lane == 0 && hd.mma_steps[warp - kMmaWarp] > 0) {
            commit_to(&hd.drained[warp - kMmaWarp]);
            drain(&hd.drained[warp - kMmaWarp], 0u);
        }
        if (warp == kProducerWarp && lane == 0) {
            const int ik = hd.issued_tiles[0];
            for (int i = max(0, ik - nk); i < ik; ++i) drain(&hd.full[i % nk], (unsigned)((i / nk) & 1));
        }
        if (warp == kVProducerWarp && lane == 0) {
            const int iv = hd.issued_tiles[1];
            for (int i = max(0, iv - nv); i < iv; ++i) drain(&hd.full[nk + i % nv], (unsigned)((i / nv) & 1));
        }
        tc_before();
        __syncthreads();
        tc_after();
    }
    if (warp == kProducerWarp && lane == 0) {  // the last CTA out re-arms the queue for the next launch
        __threadfence();
        const unsigned int done = atomicAdd(&sched[1], 1u);
        if (done == gridDim.x - 1) {
            sched[0] = 0u;
            sched[1] = 0u;
            __threadfence();
        }
    }
    if (warp == kMmaWarp)
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(kTmemCols) : "memory");
}

}  // namespace
}  // namespace lethe

namespace lethe {
namespace {

template <int NP, bool PAGED, bool E5M2, int NG, int GT, bool SPILL>
static cudaError_t launch_kv8_tc_t(const AttendArgs& a, const Kv8Maps& maps, int nslot, int cap_pad, int grid, cudaStream_t stream) {
    auto kern = attend_kv8_tc_kernel<NP, PAGED, E5M2, NG, GT, SPILL>;
    const size_t smem = kv8_tc_smem_bytes(nslot, a.G, cap_pad, NG);
    cudaError_t e = prepare_kernel((const void*)kern, smem);
    if (e != cudaSuccess) return e;
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3((unsigned)grid, 1, 1);
    cfg.blockDim = dim3((4 * NG + kRoleWarps) * 32, 1, 1);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;  // the prologue may overlap the previous kernel's tail
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kern, a, maps, nslot, cap_pad);
}

// The four instances (contiguous / paged x e4m3 / e5m2) of one (operand width, group size) pair; one translation unit
// per pair, so that they compile side by side.
template <int NP, int GT, bool WITH_SPILL>
cudaError_t launch_kv8_tc_pair(const AttendArgs& a, const void* maps_raw, bool paged, bool e5m2, int nslot, int cap_pad, int grid,
                               cudaStream_t stream) {
    Kv8Maps maps;
    memcpy(&maps, maps_raw, sizeof(maps));
    if (a.spill) {  // the instances with logit overflow exist for the wide groups only
        if constexpr (WITH_SPILL)
            return paged ? (e5m2 ? launch_kv8_tc_t<NP, true, true, 2, GT, true>(a, maps, nslot, cap_pad, grid, stream)
                                 : launch_kv8_tc_t<NP, true, false, 2, GT, true>(a, maps, nslot, cap_pad, grid, stream))
                         : (e5m2 ? launch_kv8_tc_t<NP, false, true, 2, GT, true>(a, maps, nslot, cap_pad, grid, stream)
                                 : launch_kv8_tc_t<NP, false, false, 2, GT, true>(a, maps, nslot, cap_pad, grid, stream));
        else
            return cudaErrorInvalidValue;
    }
    return paged ? (e5m2 ? launch_kv8_tc_t<NP, true, true, 2, GT, false>(a, maps, nslot, cap_pad, grid, stream)
                         : launch_kv8_tc_t<NP, true, false, 2, GT, false>(a, maps, nslot, cap_pad, grid, stream))
                 : (e5m2 ? launch_kv8_tc_t<NP, false, true, 2, GT, false>(a, maps, nslot, cap_pad, grid, stream)
                         : launch_kv8_tc_t<NP, false, false, 2, GT, false>(a, maps, nslot, cap_pad, grid, stream));
}

}  // namespace
}  // namespace lethe
