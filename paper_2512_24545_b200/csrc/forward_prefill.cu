// Large-T ("prefill") path — placeholder until the tcgen05 kernel lands.
#include "common.cuh"

namespace mdbf {

mdbf_status_t launch_forward_prefill(Layer &, const void *, void *, int, cudaStream_t, int *) {
    set_error("mdbf_linear_forward: the large-T kernel is not built yet");
    return MDBF_ERR_SHAPE;
}

}  // namespace mdbf
