// Instantiations of the warp-specialised prefill kernel: head_dim 64, 96 and 256.
#include "lagkv_tables.h"

namespace lagkv {
namespace {
const KernelEntry kTable[] = {
    LAGKV_WS_ENTRY(64, 1, 8, 32), LAGKV_WS_ENTRY(64, 1, 8, 16), LAGKV_WS_ENTRY(256, 2, 8, 16), LAGKV_WS_ENTRY(96, 3, 8, 32),
    LAGKV_WS_ENTRY(96, 3, 8, 16),
};
}  // namespace

int ws_dims_kernels(const KernelEntry** table) {
    *table = kTable;
    return int(sizeof(kTable) / sizeof(kTable[0]));
}
}  // namespace lagkv
