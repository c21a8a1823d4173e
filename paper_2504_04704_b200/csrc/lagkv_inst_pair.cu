// Instantiations of the pair kernel for short partitions (LagKV).
#include "lagkv_tables.h"

namespace lagkv {
namespace {
#define LAGKV_PAIR_ENTRY_DT(D, V, TR, DT) \
    { D, LAGKV_TUNE_PAIRS, TR, 0, DT, true, (2 * kPairs + kPairs) * 32, \
      &lagkv_pair_kernel<Geo<D, V, 2 * kPairs, TR, DT>>, &pair_smem_total_bytes<Geo<D, V, 2 * kPairs, TR, DT>> }
#define LAGKV_PAIR_ENTRY(D, V, TR) LAGKV_PAIR_ENTRY_DT(D, V, TR, 0)

const KernelEntry kTable[] = {
    LAGKV_PAIR_ENTRY(128, 2, 32), LAGKV_PAIR_ENTRY(128, 2, 16), LAGKV_PAIR_ENTRY(64, 1, 32), LAGKV_PAIR_ENTRY(256, 2, 16),
    LAGKV_PAIR_ENTRY(96, 3, 32), LAGKV_PAIR_ENTRY_DT(128, 2, 32, 1),
    LAGKV_PAIR_ENTRY_DT(64, 1, 32, 1), LAGKV_PAIR_ENTRY_DT(256, 2, 16, 1), LAGKV_PAIR_ENTRY_DT(96, 3, 32, 1),
};
}  // namespace

int pair_kernels(const KernelEntry** table) {
    *table = kTable;
    return int(sizeof(kTable) / sizeof(kTable[0]));
}
}  // namespace lagkv
