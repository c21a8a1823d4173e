// Instantiations for fp8 (e4m3) caches, head_dim 128: a row is 128 bytes, eight 16-byte vectors,
// one per lane of an eight-lane row group.  The planner's default shapes of every kernel family.
#include "lagkv_tables.h"

namespace lagkv {
namespace {
#define LAGKV_FP8_PAIR_ENTRY(TR) \
    { 128, LAGKV_TUNE_PAIRS, TR, 0, 2, true, (2 * kPairs + kPairs) * 32, \
      &lagkv_pair_kernel<Geo<128, 1, 2 * kPairs, TR, 2>>, &pair_smem_total_bytes<Geo<128, 1, 2 * kPairs, TR, 2>> }
#define LAGKV_FP8_APPEND_ENTRY \
    { 128, LAGKV_TUNE_APPEND_CLUSTER, kAppendPairTileRows, 0, 2, true, 4 * 32, \
      &lagkv_append_pair_kernel<Geo<128, 1, 4, kAppendPairTileRows, 2>>, \
      &append_pair_smem_fixed<Geo<128, 1, 4, kAppendPairTileRows, 2>> }

const KernelEntry kTable[] = {
    LAGKV_FP16_ENTRIES_DT(128, 1, 2),
    LAGKV_WS_ENTRY_DT(128, 1, 8, 32, 2), LAGKV_WS_ENTRY_DT(128, 1, 8, 16, 2),
    LAGKV_FP8_PAIR_ENTRY(32), LAGKV_FP8_PAIR_ENTRY(16), LAGKV_FP8_APPEND_ENTRY,
};
}  // namespace

int fp8_kernels(const KernelEntry** table) {
    *table = kTable;
    return int(sizeof(kTable) / sizeof(kTable[0]));
}
}  // namespace lagkv
