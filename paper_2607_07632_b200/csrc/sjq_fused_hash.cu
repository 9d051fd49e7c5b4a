// Ahead-of-time instantiations of the fused kernel for one aggregation path (AGG_HASH); one translation unit per
// path so that the four compile in parallel.
#include "sjq_fused_device.cuh"

namespace sjq {

fused_fn fused_variant_hash(bool mul, bool hash)
{
    if (mul) return hash ? fused_kernel<AGG_HASH, true, true> : fused_kernel<AGG_HASH, true, false>;
    return hash ? fused_kernel<AGG_HASH, false, true> : fused_kernel<AGG_HASH, false, false>;
}

} // namespace sjq
