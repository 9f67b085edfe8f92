// Instantiation of the tensor-parallel kernel for ONE value of L (16-byte chunk slots
// per lane) and ONE storage format, chosen with -DQKNORM_L=<l> -DQKNORM_IO=<IoBf16|IoE4m3>
// -DQKNORM_IO_TAG=<bf16|e4m3>; one translation unit each.
#include "qknorm_tp.cuh"

#if !defined(QKNORM_L) || !defined(QKNORM_IO) || !defined(QKNORM_IO_TAG)
#error "compile with -DQKNORM_L=<chunk slots per lane> -DQKNORM_IO=<format> -DQKNORM_IO_TAG=<tag>"
#endif
#define QKNORM_CAT3_(a, b, c, d) a##b##c##d
#define QKNORM_CAT3(a, b, c, d) QKNORM_CAT3_(a, b, c, d)

namespace qknorm {

TpKernel QKNORM_CAT3(tp_kernel_, QKNORM_IO_TAG, _l, QKNORM_L)() { return tp_kernel<QKNORM_L, QKNORM_IO>; }

}  // namespace qknorm
