// Instances of the tensor-memory kernel for quantised caches: 5 query heads per KV head, compiled in.
#include "attend_kv8_tc.cuh"

namespace lethe {

cudaError_t launch_kv8_tc_g5(const AttendArgs& a, const void* maps, bool paged, bool e5m2, int nslot, int cap_pad, int grid,
                            cudaStream_t stream) {
    return launch_kv8_tc_pair<16, 5, false>(a, maps, paged, e5m2, nslot, cap_pad, grid, stream);
}

}  // namespace lethe
