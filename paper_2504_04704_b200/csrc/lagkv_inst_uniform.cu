// Instantiations of the uniform kernel (prefill for short partitions, every append): head_dim 128.
#include "lagkv_tables.h"

namespace lagkv {
namespace {
const KernelEntry kTable[] = {
    LAGKV_SHAPE_ENTRIES(128, 2), LAGKV_VARIANT_ENTRIES(128, 2), LAGKV_FP16_ENTRIES(128, 2),
};
}  // namespace

int uniform_kernels(const KernelEntry** table) {
    *table = kTable;
    return int(sizeof(kTable) / sizeof(kTable[0]));
}
}  // namespace lagkv
