// Forward kernels with the MODE_ROW2 cell update (see spdy_device.cuh), compiled on their own so that the
// modes build in parallel.  This is the default cell update of its table format: it is also built with
// the row buffers in global memory and as one warp per candidate, and it is kept in the debug build.
#include "spdy_device.cuh"

namespace spdy {

namespace {
const FwdVariant kForward[] = {SPDY_FULL_VARIANTS(MODE_ROW2)};
const ClusterVariant kCluster[] = {SPDY_CLUSTER_VARIANTS(MODE_ROW2)};
}  // namespace

VariantList variants_row2()
{
    return VariantList{kForward, static_cast<int>(sizeof(kForward) / sizeof(kForward[0])), kCluster,
                       static_cast<int>(sizeof(kCluster) / sizeof(kCluster[0]))};
}

}  // namespace spdy
