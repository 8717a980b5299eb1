// Instances of the grouped kernel for bf16 tensors, tiles of half the elements (small calls).
#include "lgn_kernels.cuh"

namespace lgn {
const void *const kCompressTableBf16Small[kVariants] = LGN_CK_ROW(LGN_BF16, kSmallTileElemsBf16);
}  // namespace lgn
