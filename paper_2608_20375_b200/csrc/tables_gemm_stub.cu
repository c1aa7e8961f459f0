// Stand-in for tables_gemm.cu in a build without a CUTLASS tree: the tensor-core table precompute reports that it
// cannot take any problem (scratch size 0), and graft_tdes_precompute then runs the fp32 FMA kernel of tdes.cu for
// every input.  Everything else in the library is unaffected.
#include <cuda_runtime.h>

#include "internal.h"

namespace graft {

size_t tables_tc_scratch_bytes(int, int, int) { return 0; }

cudaError_t tables_tc_launch(const void*, int, int, int, const float*, const float*, float*, void*, int*,
                             cudaStream_t) {
    return cudaErrorNotSupported;
}

}  // namespace graft
