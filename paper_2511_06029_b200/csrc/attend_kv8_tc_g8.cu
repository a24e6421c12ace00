// Instances of the tensor-memory kernel for quantised caches: 8 query heads per KV head, compiled in, with and without logit overflow.
#include "attend_kv8_tc.cuh"

namespace lethe {

cudaError_t launch_kv8_tc_g8(const AttendArgs& a, const void* maps, bool paged, bool e5m2, int nslot, int cap_pad, int grid,
                            cudaStream_t stream) {
    return launch_kv8_tc_pair<32, 8, true>(a, maps, paged, e5m2, nslot, cap_pad, grid, stream);
}

}  // namespace lethe
