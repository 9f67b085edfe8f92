// Instantiations of the register-resident row kernel for ONE value of NQ
// (chunks of the Q row per thread), chosen with -DQKNORM_NQ=<n>, and every NK.
// One translation unit per NQ keeps the build parallel.
#include "qknorm_rows.cuh"

#ifndef QKNORM_NQ
#error "compile with -DQKNORM_NQ=<chunks of Q per thread>"
#endif
#define QKNORM_CAT_(a, b) a##b
#define QKNORM_CAT(a, b) QKNORM_CAT_(a, b)

namespace qknorm {

RowsKernel QKNORM_CAT(rows_throughput_nq, QKNORM_NQ)(int nk) {
  switch (nk) {
    case 0: return rows_kernel<QKNORM_NQ, 0, 256>;
    case 1: return rows_kernel<QKNORM_NQ, 1, 256>;
    case 2: return rows_kernel<QKNORM_NQ, 2, 256>;
    case 3: return rows_kernel<QKNORM_NQ, 3, 256>;
    case 4: return rows_kernel<QKNORM_NQ, 4, 256>;
    case 5: return rows_kernel<QKNORM_NQ, 5, 256>;
    case 6: return rows_kernel<QKNORM_NQ, 6, 256>;
    case 8: return rows_kernel<QKNORM_NQ, 8, 256>;
    default: return nullptr;
  }
}

#if QKNORM_NQ == 0 || QKNORM_NQ == 1 || QKNORM_NQ == 2 || QKNORM_NQ == 4
RowsKernel QKNORM_CAT(rows_latency_nq, QKNORM_NQ)(int nk) {
  switch (nk) {
    case 0: return rows_kernel<QKNORM_NQ, 0, 512>;
    case 1: return rows_kernel<QKNORM_NQ, 1, 512>;
    case 2: return rows_kernel<QKNORM_NQ, 2, 512>;
    case 4: return rows_kernel<QKNORM_NQ, 4, 512>;
    default: return nullptr;
  }
}
#endif

}  // namespace qknorm
