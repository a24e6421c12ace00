// Instances of the tensor-memory kernel for quantised caches: any group size up to 8, read from the arguments, with and without logit overflow.
#include "attend_kv8_tc.cuh"

namespace lethe {

cudaError_t launch_kv8_tc_n32(const AttendArgs& a, const void* maps, bool paged, bool e5m2, int nslot, int cap_pad, int grid,
                            cudaStream_t stream) {
    return launch_kv8_tc_pair<32, 0, true>(a, maps, paged, e5m2, nslot, cap_pad, grid, stream);
}

}  // namespace lethe
