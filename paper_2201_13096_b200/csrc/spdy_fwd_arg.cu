// Forward kernels with the MODE_ARG cell update (see spdy_device.cuh), compiled on their own so that the
// modes build in parallel.  A measured baseline and cross-check of the default cell update; left out of the debug build.
#include "spdy_device.cuh"

namespace spdy {

#ifndef SPDY_DEBUG_CHECKS
namespace {
const FwdVariant kForward[] = {SPDY_CTA_VARIANTS(MODE_ARG)};
const ClusterVariant kCluster[] = {SPDY_CLUSTER_VARIANTS(MODE_ARG)};
}  // namespace

VariantList variants_arg()
{
    return VariantList{kForward, static_cast<int>(sizeof(kForward) / sizeof(kForward[0])), kCluster,
                       static_cast<int>(sizeof(kCluster) / sizeof(kCluster[0]))};
}
#else
VariantList variants_arg() { return VariantList{nullptr, 0, nullptr, 0}; }
#endif

}  // namespace spdy
