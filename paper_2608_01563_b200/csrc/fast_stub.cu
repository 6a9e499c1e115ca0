// Placeholder for the tensor-core backward while it is being brought up.
#include "kernels.h"
namespace mgn {
cudaError_t launch_fast_bwd(const Problem&, const void*, const void*, const void*, const void*, const float*,
                            const float*, float*, void*, void*, void*, unsigned*, cudaStream_t)
{ return cudaErrorNotSupported; }
}
