// Instantiations of the warp-specialised prefill kernel for paged caches (LagKV scoring): head_dim 128.
#include "lagkv_tables.h"

namespace lagkv {
namespace {
const KernelEntry kTable[] = {
    LAGKV_WS_PAGED_ENTRY(128, 2, 8, 32, 0), LAGKV_WS_PAGED_ENTRY(128, 2, 8, 16, 0),
    LAGKV_WS_PAGED_ENTRY(128, 2, 8, 32, 1), LAGKV_WS_PAGED_ENTRY(128, 2, 8, 16, 1),
};
}  // namespace

int ws_paged_kernels(const KernelEntry** table) {
    *table = kTable;
    return int(sizeof(kTable) / sizeof(kTable[0]));
}
}  // namespace lagkv
