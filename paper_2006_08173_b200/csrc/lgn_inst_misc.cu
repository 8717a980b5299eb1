// The general kernel for mixed groups and the stand-alone apply kernels.
#include "lgn_kernels.cuh"

namespace lgn {
const void *const kCompressGeneral = LGN_CK(kAny, kAny, kAny, kAny, false, kTileElems);

#define LGN_QK(DT, NB, SR) reinterpret_cast<const void *>(&quantize_kernel<DT, NB, SR>)
#define LGN_QK_ROW(DT) { LGN_QK(DT, 4, 0), LGN_QK(DT, 4, 1), LGN_QK(DT, 5, 0), LGN_QK(DT, 5, 1), LGN_QK(DT, 6, 0), \
    LGN_QK(DT, 6, 1), LGN_QK(DT, 7, 0), LGN_QK(DT, 7, 1), LGN_QK(DT, 8, 0), LGN_QK(DT, 8, 1) }
const void *const kQuantizeTable[2][10] = { LGN_QK_ROW(LGN_F32), LGN_QK_ROW(LGN_BF16) };
const void *const kPruneTable[2] = { reinterpret_cast<const void *>(&prune_kernel<LGN_F32>),
                                     reinterpret_cast<const void *>(&prune_kernel<LGN_BF16>) };
}  // namespace lgn
