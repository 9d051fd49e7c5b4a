// Ahead-of-time instantiations of the fused kernel for one aggregation path (AGG_GLOBAL); one translation unit per
// path so that the four compile in parallel.
#include "sjq_fused_device.cuh"

namespace sjq {

fused_fn fused_variant_global(bool mul, bool hash)
{
    if (mul) return hash ? fused_kernel<AGG_GLOBAL, true, true> : fused_kernel<AGG_GLOBAL, true, false>;
    return hash ? fused_kernel<AGG_GLOBAL, false, true> : fused_kernel<AGG_GLOBAL, false, false>;
}

} // namespace sjq
