// Instantiations of the register-resident row kernel (both storage formats) and
// of the TMA ring kernel for ONE value of N (16-byte chunks per thread), chosen
// with -DQKNORM_N=<n>.  One translation unit per N keeps the build parallel.
#include "qknorm_ring.cuh"
#include "qknorm_rows.cuh"

#ifndef QKNORM_N
#error "compile with -DQKNORM_N=<chunks per thread>"
#endif
#define QKNORM_CAT_(a, b) a##b
#define QKNORM_CAT(a, b) QKNORM_CAT_(a, b)

namespace qknorm {

RowsKernel QKNORM_CAT(rows_kernel_n, QKNORM_N)(int elem_bytes) {
  return elem_bytes == 1 ? rows_kernel<QKNORM_N, IoE4m3> : rows_kernel<QKNORM_N, IoBf16>;
}
RingKernel QKNORM_CAT(ring_kernel_n, QKNORM_N)() { return ring_kernel<QKNORM_N>; }

}  // namespace qknorm
