// Instantiations of the uniform kernel: head_dim 64, 96 and 256.
#include "lagkv_tables.h"

namespace lagkv {
namespace {
const KernelEntry kTable[] = {
    LAGKV_SHAPE_ENTRIES(64, 1),  LAGKV_VARIANT_ENTRIES(64, 1),  LAGKV_SHAPE_ENTRIES(96, 3), LAGKV_VARIANT_ENTRIES(96, 3),
    LAGKV_SHAPE_ENTRIES(256, 2), LAGKV_VARIANT_ENTRIES(256, 2),
};
}  // namespace

int uniform_dims_kernels(const KernelEntry** table) {
    *table = kTable;
    return int(sizeof(kTable) / sizeof(kTable[0]));
}
}  // namespace lagkv
