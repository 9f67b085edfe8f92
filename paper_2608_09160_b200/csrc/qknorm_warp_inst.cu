// Instantiations of the warp-per-token kernel for ONE value of L (16-byte chunk
// slots per lane) and ONE storage format, chosen with -DQKNORM_L=<l>
// -DQKNORM_IO=<IoBf16|IoE4m3> -DQKNORM_IO_TAG=<bf16|e4m3>; one translation unit each.
#include "qknorm_warp.cuh"

#if !defined(QKNORM_L) || !defined(QKNORM_IO) || !defined(QKNORM_IO_TAG)
#error "compile with -DQKNORM_L=<chunk slots per lane> -DQKNORM_IO=<format> -DQKNORM_IO_TAG=<tag>"
#endif
#define QKNORM_CAT3_(a, b, c, d) a##b##c##d
#define QKNORM_CAT3(a, b, c, d) QKNORM_CAT3_(a, b, c, d)

namespace qknorm {

WarpKernel QKNORM_CAT3(warp_kernel_, QKNORM_IO_TAG, _l, QKNORM_L)(bool exact) {
  return exact ? warp_kernel<QKNORM_L, true, QKNORM_IO> : warp_kernel<QKNORM_L, false, QKNORM_IO>;
}

}  // namespace qknorm
