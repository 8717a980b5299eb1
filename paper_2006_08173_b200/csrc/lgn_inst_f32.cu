// Instances of the grouped kernel for fp32 tensors.
#include "lgn_kernels.cuh"

namespace lgn {
const void *const kCompressTableF32[kVariants] = LGN_CK_ROW(LGN_F32, kTileElems);
}  // namespace lgn
