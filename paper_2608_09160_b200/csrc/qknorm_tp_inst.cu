// The tensor-parallel kernel, one instantiation per tile shape and storage format, in a translation
// unit of its own so that it compiles in parallel with the others.
#include "qknorm_tp.cuh"

namespace qknorm {

TpKernel tp_kernel_for(int log_g, int elem_bytes) {
  const bool f8 = elem_bytes == 1;
  switch (log_g) {
    case 2: return f8 ? tp_kernel<2, IoE4m3> : tp_kernel<2, IoBf16>;
    case 3: return f8 ? tp_kernel<3, IoE4m3> : tp_kernel<3, IoBf16>;
    case 4: return f8 ? tp_kernel<4, IoE4m3> : tp_kernel<4, IoBf16>;
    case 5: return f8 ? tp_kernel<5, IoE4m3> : tp_kernel<5, IoBf16>;
    default: return nullptr;
  }
}

}  // namespace qknorm
