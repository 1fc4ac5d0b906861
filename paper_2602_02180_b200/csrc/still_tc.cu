// Tensor-core (tcgen05) prefill path -- placeholder until the kernel lands.
#include "still_tc.h"

namespace still {

bool tc_supported(const still_params_t *) { return false; }
long long tc_sel_rows(const still_params_t *, long long) { return 0; }
int tc_sa_merge(const still_params_t *, long long, const void *, const void *, const void *,
                const int32_t *, const float *, const float *, void *, void *, void *, long long, int *,
                cudaStream_t, int *) {
    return STILL_ERR_UNSUPPORTED;
}

}  // namespace still
