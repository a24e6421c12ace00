// Host side of the tensor-memory kernel for quantised caches (attend_kv8_tc.cuh): shared-memory size, tensor maps,
// and the choice of the instance: the group sizes of the common model geometries (4, 5, 7 and 8 query heads per KV
// head) are compiled in, every other one runs the instances that read it from the arguments.
#include "attend_kv8_tc.cuh"

namespace lethe {

// Shared memory of one CTA: alignment slack, ring, the two operand buffers of queries and of probabilities, the
// parked logits, the header.
size_t kv8_tc_smem_bytes(int nslot, int G, int cap_pad, int ng) {
    const int NP = 3 * G <= 16 ? 16 : 32;
    return 1024 + (size_t)nslot * kTileBytes + (size_t)(ng + ng * kGB) * NP * 128 + (size_t)ng * G * cap_pad * 4 + sizeof(Kv8Header) + 64;
}

size_t kv8_tc_maps_bytes() { return sizeof(Kv8Maps); }

// Tensor maps over K and V seen as [rows][128 bytes]: boxes of 128 rows (contiguous cache) or 16 rows (one page).
bool build_kv8_tc_maps(void* encode, void* k, void* v, unsigned long long rows, bool paged, void* out_maps) {
    typedef CUresult (*encode_fn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
    encode_fn fn = reinterpret_cast<encode_fn>(encode);
    Kv8Maps* m = reinterpret_cast<Kv8Maps*>(out_maps);
    const cuuint64_t dims[2] = {128, (cuuint64_t)rows};
    const cuuint64_t strides[1] = {128};
    const cuuint32_t box[2] = {128, paged ? (cuuint32_t)kGroupTokens : (cuuint32_t)kTile};
    const cuuint32_t es[2] = {1, 1};
    const CUresult r1 = fn(&m->k, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, k, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    const CUresult r2 = fn(&m->v, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, v, dims, strides, box, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    const cuuint32_t box16[2] = {128, (cuuint32_t)kGroupTokens};
    const CUresult r3 = fn(&m->k16, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, k, dims, strides, box16, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    const CUresult r4 = fn(&m->v16, CU_TENSOR_MAP_DATA_TYPE_UINT8, 2, v, dims, strides, box16, es, CU_TENSOR_MAP_INTERLEAVE_NONE,
                           CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r1 == CUDA_SUCCESS && r2 == CUDA_SUCCESS && r3 == CUDA_SUCCESS && r4 == CUDA_SUCCESS;
}


#define LETHE_KV8TC_DECL(name) \
    cudaError_t name(const AttendArgs& a, const void* maps, bool paged, bool e5m2, int nslot, int cap_pad, int grid, cudaStream_t stream)
LETHE_KV8TC_DECL(launch_kv8_tc_g4);
LETHE_KV8TC_DECL(launch_kv8_tc_g5);
LETHE_KV8TC_DECL(launch_kv8_tc_g7);
LETHE_KV8TC_DECL(launch_kv8_tc_g8);
LETHE_KV8TC_DECL(launch_kv8_tc_n16);
LETHE_KV8TC_DECL(launch_kv8_tc_n32);
#undef LETHE_KV8TC_DECL

// (three softmax groups: built and measured, 0.1137 ms against 0.1130 ms with two on the Llama-8B shape; not instantiated)
cudaError_t launch_attend_kv8_tc(const AttendArgs& a, const void* maps, bool paged, bool e5m2, int ng, int nslot, int cap_pad, int grid,
                                 cudaStream_t stream) {
    if (ng != 2) return cudaErrorInvalidValue;
    switch (a.G) {
        case 4: return launch_kv8_tc_g4(a, maps, paged, e5m2, nslot, cap_pad, grid, stream);
        case 5: return launch_kv8_tc_g5(a, maps, paged, e5m2, nslot, cap_pad, grid, stream);
        case 7: return launch_kv8_tc_g7(a, maps, paged, e5m2, nslot, cap_pad, grid, stream);
        case 8: return launch_kv8_tc_g8(a, maps, paged, e5m2, nslot, cap_pad, grid, stream);
        default: break;
    }
    return 3 * a.G > 16 ? launch_kv8_tc_n32(a, maps, paged, e5m2, nslot, cap_pad, grid, stream)
                        : launch_kv8_tc_n16(a, maps, paged, e5m2, nslot, cap_pad, grid, stream);
}

}  // namespace lethe
