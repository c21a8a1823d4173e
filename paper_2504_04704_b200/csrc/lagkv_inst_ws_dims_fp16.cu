// Instantiations of the warp-specialised prefill kernel for fp16 caches: head_dim 64, 96 and 256.
#include "lagkv_tables.h"

namespace lagkv {
namespace {
const KernelEntry kTable[] = {
    LAGKV_WS_ENTRY_DT(64, 1, 8, 32, 1), LAGKV_WS_ENTRY_DT(64, 1, 8, 16, 1), LAGKV_WS_ENTRY_DT(256, 2, 8, 16, 1),
    LAGKV_WS_ENTRY_DT(96, 3, 8, 32, 1), LAGKV_WS_ENTRY_DT(96, 3, 8, 16, 1),
};
}  // namespace

int ws_dims_fp16_kernels(const KernelEntry** table) {
    *table = kTable;
    return int(sizeof(kTable) / sizeof(kTable[0]));
}
}  // namespace lagkv
