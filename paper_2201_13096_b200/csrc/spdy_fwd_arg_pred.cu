// Forward kernels with the MODE_ARG_PRED cell update (see spdy_device.cuh), compiled on their own so that the
// modes build in parallel.  A measured baseline and cross-check of the default cell update; left out of the debug build.
#include "spdy_device.cuh"

namespace spdy {

#ifndef SPDY_DEBUG_CHECKS
namespace {
const FwdVariant kForward[] = {SPDY_CTA_VARIANTS(MODE_ARG_PRED)};
}  // namespace

// No cluster build: with a cluster's masked stores on top of its float-coded indices this update does not
// fit the 128 registers a 512-thread CTA leaves.
VariantList variants_arg_pred()
{
    return VariantList{kForward, static_cast<int>(sizeof(kForward) / sizeof(kForward[0])), nullptr, 0};
}
#else
VariantList variants_arg_pred() { return VariantList{nullptr, 0, nullptr, 0}; }
#endif

}  // namespace spdy
