// Placeholder until the tcgen05 kernel lands: reports "not supported" so that
// the step uses the mma.sync kernel.
#include "xsv_kernels.h"

cudaError_t xsv_launch_attn_tc5(const LayerView&, int, const void*, const void*, const void*, void*, int, int, int,
                                int*, cudaStream_t) {
    return cudaErrorNotSupported;
}
