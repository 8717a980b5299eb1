// Instances of the grouped kernel for bf16 tensors, tiles of twice the elements (large calls).
#include "lgn_kernels.cuh"

namespace lgn {
const void *const kCompressTableBf16Big[kVariants] = LGN_CK_ROW(LGN_BF16, kBigTileElems);
}  // namespace lgn
