// Instantiations for fp8 (e4m3) caches: head_dim 64, 96 and 256 (rows of 64, 96 and 256 bytes).
#include "lagkv_tables.h"

namespace lagkv {
namespace {
#define LAGKV_FP8_PAIR_ENTRY(D, V, TR) \
    { D, LAGKV_TUNE_PAIRS, TR, 0, 2, true, (2 * kPairs + kPairs) * 32, \
      &lagkv_pair_kernel<Geo<D, V, 2 * kPairs, TR, 2>>, &pair_smem_total_bytes<Geo<D, V, 2 * kPairs, TR, 2>> }
#define LAGKV_FP8_APPEND_ENTRY(D, V) \
    { D, LAGKV_TUNE_APPEND_CLUSTER, kAppendPairTileRows, 0, 2, true, 4 * 32, \
      &lagkv_append_pair_kernel<Geo<D, V, 4, kAppendPairTileRows, 2>>, \
      &append_pair_smem_fixed<Geo<D, V, 4, kAppendPairTileRows, 2>> }

const KernelEntry kTable[] = {
    LAGKV_FP16_ENTRIES_DT(64, 1, 2),  LAGKV_WS_ENTRY_DT(64, 1, 8, 32, 2),  LAGKV_FP8_PAIR_ENTRY(64, 1, 32),
    LAGKV_FP8_APPEND_ENTRY(64, 1),
    /* 96-byte rows: no warp-specialised kernel (its final gather wants row groups that fill a warp) */
    LAGKV_FP16_ENTRIES_DT(96, 3, 2),  LAGKV_FP8_PAIR_ENTRY(96, 3, 32),
    LAGKV_FP8_APPEND_ENTRY(96, 3),
    LAGKV_FP16_ENTRIES_DT(256, 2, 2), LAGKV_WS_ENTRY_DT(256, 2, 8, 32, 2), LAGKV_FP8_PAIR_ENTRY(256, 2, 32),
    LAGKV_FP8_APPEND_ENTRY(256, 2),
};
}  // namespace

int fp8_dims_kernels(const KernelEntry** table) {
    *table = kTable;
    return int(sizeof(kTable) / sizeof(kTable[0]));
}
}  // namespace lagkv
