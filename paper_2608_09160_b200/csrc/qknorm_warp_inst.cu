// Instantiations of the warp-per-row kernel for ONE value of L (16-byte chunk
// slots per lane), chosen with -DQKNORM_L=<l>; one translation unit per L.
#include "qknorm_warp.cuh"

#ifndef QKNORM_L
#error "compile with -DQKNORM_L=<chunk slots per lane>"
#endif
#define QKNORM_CAT_(a, b) a##b
#define QKNORM_CAT(a, b) QKNORM_CAT_(a, b)

namespace qknorm {

WarpKernel QKNORM_CAT(warp_kernel_l, QKNORM_L)(bool exact) {
  return exact ? warp_kernel<QKNORM_L, true> : warp_kernel<QKNORM_L, false>;
}

}  // namespace qknorm
