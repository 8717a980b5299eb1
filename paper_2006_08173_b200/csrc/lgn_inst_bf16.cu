// Instances of the grouped kernel for bf16 tensors, tiles of kTileElems elements.
#include "lgn_kernels.cuh"

namespace lgn {
const void *const kCompressTableBf16[kVariants] = LGN_CK_ROW(LGN_BF16, kTileElems);
}  // namespace lgn
