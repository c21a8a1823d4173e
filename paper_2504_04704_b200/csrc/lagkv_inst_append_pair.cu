// Instantiations of the one-partition append kernel (a cluster of CTAs per unit): every
// head_dim and storage format, LagKV scoring.
#include "lagkv_tables.h"

namespace lagkv {
namespace {
#define LAGKV_APPEND_PAIR_ENTRY(D, V, NW, CODE, DT) \
    { D, CODE, kAppendPairTileRows, 0, DT, true, NW * 32, \
      &lagkv_append_pair_kernel<Geo<D, V, NW, kAppendPairTileRows, DT>>, \
      &append_pair_smem_fixed<Geo<D, V, NW, kAppendPairTileRows, DT>> }
#define LAGKV_APPEND4(D, V, DT) LAGKV_APPEND_PAIR_ENTRY(D, V, 4, LAGKV_TUNE_APPEND_CLUSTER, DT)
#define LAGKV_APPEND8(D, V, DT) LAGKV_APPEND_PAIR_ENTRY(D, V, 8, LAGKV_TUNE_APPEND_CLUSTER8, DT)

const KernelEntry kTable[] = {
    LAGKV_APPEND4(128, 2, 0), LAGKV_APPEND4(128, 2, 1), LAGKV_APPEND4(64, 1, 0),  LAGKV_APPEND4(64, 1, 1),
    LAGKV_APPEND4(96, 3, 0),  LAGKV_APPEND4(96, 3, 1),  LAGKV_APPEND4(256, 2, 0), LAGKV_APPEND4(256, 2, 1),
    LAGKV_APPEND8(128, 2, 0), LAGKV_APPEND8(128, 2, 1),
};
}  // namespace

int append_pair_kernels(const KernelEntry** table) {
    *table = kTable;
    return int(sizeof(kTable) / sizeof(kTable[0]));
}
}  // namespace lagkv
