// Instantiations of the uniform kernel (prefill for short partitions, every append).
#include "lagkv_tables.h"

namespace lagkv {
namespace {
#define LAGKV_ENTRY2(D, V, NW, TR, VAR, DT) \
    { D, NW, TR, VAR, DT, false, NW * 32, &lagkv_stream_kernel<Geo<D, V, NW, TR, DT>, VAR>, \
      &smem_total_bytes<Geo<D, V, NW, TR, DT>> }
#define LAGKV_ENTRY1(D, V, NW, TR, VAR) LAGKV_ENTRY2(D, V, NW, TR, VAR, 0)
#define LAGKV_ENTRY(D, V, NW, TR) LAGKV_ENTRY1(D, V, NW, TR, 0)
/* the two shapes the planner uses for appends, also for the LocalKV and L2-norm variants */
#define LAGKV_VARIANT_ENTRIES(D, V) \
    LAGKV_ENTRY1(D, V, 4, 32, 1), LAGKV_ENTRY1(D, V, 4, 32, 2), LAGKV_ENTRY1(D, V, 2, 16, 1), LAGKV_ENTRY1(D, V, 2, 16, 2)
/* fp16 caches: the planner's default shapes, every variant */
#define LAGKV_FP16_ENTRIES(D, V) \
    LAGKV_ENTRY2(D, V, 8, 32, 0, 1), LAGKV_ENTRY2(D, V, 4, 32, 0, 1), LAGKV_ENTRY2(D, V, 2, 16, 0, 1), \
    LAGKV_ENTRY2(D, V, 4, 32, 1, 1), LAGKV_ENTRY2(D, V, 4, 32, 2, 1), LAGKV_ENTRY2(D, V, 2, 16, 1, 1), \
    LAGKV_ENTRY2(D, V, 2, 16, 2, 1)

const KernelEntry kTable[] = {
    LAGKV_ENTRY(128, 2, 8, 32), LAGKV_ENTRY(128, 2, 4, 32), LAGKV_ENTRY(128, 2, 2, 32),
    LAGKV_ENTRY(128, 2, 8, 16), LAGKV_ENTRY(128, 2, 4, 16), LAGKV_ENTRY(128, 2, 2, 16),
    LAGKV_ENTRY(64, 1, 8, 32),  LAGKV_ENTRY(64, 1, 4, 32),  LAGKV_ENTRY(64, 1, 2, 32),
    LAGKV_ENTRY(64, 1, 8, 16),  LAGKV_ENTRY(64, 1, 4, 16),  LAGKV_ENTRY(64, 1, 2, 16),
    LAGKV_ENTRY(256, 2, 8, 32), LAGKV_ENTRY(256, 2, 4, 32), LAGKV_ENTRY(256, 2, 2, 32),
    LAGKV_ENTRY(256, 2, 8, 16), LAGKV_ENTRY(256, 2, 4, 16), LAGKV_ENTRY(256, 2, 2, 16),
    LAGKV_ENTRY(96, 3, 8, 32),  LAGKV_ENTRY(96, 3, 4, 32),  LAGKV_ENTRY(96, 3, 2, 32),
    LAGKV_ENTRY(96, 3, 8, 16),  LAGKV_ENTRY(96, 3, 4, 16),  LAGKV_ENTRY(96, 3, 2, 16),
    LAGKV_VARIANT_ENTRIES(128, 2), LAGKV_VARIANT_ENTRIES(64, 1), LAGKV_VARIANT_ENTRIES(256, 2),
    LAGKV_VARIANT_ENTRIES(96, 3),
    LAGKV_FP16_ENTRIES(128, 2),
};
}  // namespace

int uniform_kernels(const KernelEntry** table) {
    *table = kTable;
    return int(sizeof(kTable) / sizeof(kTable[0]));
}
}  // namespace lagkv
