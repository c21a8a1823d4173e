// Instantiations of the warp-specialised prefill kernel, one per geometry and scoring variant: head_dim 128.
#include "lagkv_tables.h"

namespace lagkv {
namespace {
const KernelEntry kTable[] = {
    LAGKV_WS_ENTRY(128, 2, 8, 32), LAGKV_WS_ENTRY(128, 2, 8, 16), LAGKV_WS_ENTRY_DT(128, 2, 8, 32, 1),
    LAGKV_WS_ENTRY_DT(128, 2, 8, 16, 1),
};
}  // namespace

int ws_kernels(const KernelEntry** table) {
    *table = kTable;
    return int(sizeof(kTable) / sizeof(kTable[0]));
}
}  // namespace lagkv
