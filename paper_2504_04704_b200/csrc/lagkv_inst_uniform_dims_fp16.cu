// Instantiations of the uniform kernel for fp16 caches: head_dim 64, 96 and 256.
#include "lagkv_tables.h"

namespace lagkv {
namespace {
const KernelEntry kTable[] = {
    LAGKV_FP16_ENTRIES(64, 1), LAGKV_FP16_ENTRIES(96, 3), LAGKV_FP16_ENTRIES(256, 2),
};
}  // namespace

int uniform_dims_fp16_kernels(const KernelEntry** table) {
    *table = kTable;
    return int(sizeof(kTable) / sizeof(kTable[0]));
}
}  // namespace lagkv
