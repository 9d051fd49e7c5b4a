// Ahead-of-time instantiations of the fused kernel for one aggregation path (AGG_SCALAR); one translation unit per
// path so that the four compile in parallel.
#include "sjq_fused_device.cuh"

namespace sjq {

fused_fn fused_variant_scalar(bool mul, bool hash)
{
    if (mul) return hash ? fused_kernel<AGG_SCALAR, true, true> : fused_kernel<AGG_SCALAR, true, false>;
    return hash ? fused_kernel<AGG_SCALAR, false, true> : fused_kernel<AGG_SCALAR, false, false>;
}

} // namespace sjq
