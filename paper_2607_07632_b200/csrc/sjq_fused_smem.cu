// Ahead-of-time instantiations of the fused kernel for one aggregation path (AGG_SMEM); one translation unit per
// path so that the four compile in parallel.
#include "sjq_fused_device.cuh"

namespace sjq {

fused_fn fused_variant_smem(bool mul, bool hash)
{
    if (mul) return hash ? fused_kernel<AGG_SMEM, true, true> : fused_kernel<AGG_SMEM, true, false>;
    return hash ? fused_kernel<AGG_SMEM, false, true> : fused_kernel<AGG_SMEM, false, false>;
}

} // namespace sjq
