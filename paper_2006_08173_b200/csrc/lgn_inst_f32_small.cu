// Instances of the grouped kernel for fp32 tensors, tiles of a quarter of the elements (small calls).
#include "lgn_kernels.cuh"

namespace lgn {
const void *const kCompressTableF32Small[kVariants] = LGN_CK_ROW(LGN_F32, kSmallTileElemsF32);
}  // namespace lgn
