// Instantiations of the warp-specialised prefill kernel, one per geometry and scoring variant.
#include "lagkv_tables.h"

namespace lagkv {
namespace {
#define LAGKV_WS_ENTRY1(D, V, NWS, TR, VAR) \
    { D, NWS + kWsEpiWarps, TR, VAR, true, (NWS + kWsEpiWarps) * 32, &lagkv_ws_kernel<Geo<D, V, NWS, TR>, VAR>, \
      &ws_smem_total_bytes<Geo<D, V, NWS, TR>> }
#define LAGKV_WS_ENTRY(D, V, NWS, TR) \
    LAGKV_WS_ENTRY1(D, V, NWS, TR, 0), LAGKV_WS_ENTRY1(D, V, NWS, TR, 1), LAGKV_WS_ENTRY1(D, V, NWS, TR, 2)

const KernelEntry kTable[] = {
    LAGKV_WS_ENTRY(128, 2, 8, 32), LAGKV_WS_ENTRY(128, 2, 8, 16), LAGKV_WS_ENTRY(64, 1, 8, 32),
    LAGKV_WS_ENTRY(64, 1, 8, 16), LAGKV_WS_ENTRY(256, 2, 8, 16), LAGKV_WS_ENTRY(96, 3, 8, 32),
    LAGKV_WS_ENTRY(96, 3, 8, 16),
};
}  // namespace

int ws_kernels(const KernelEntry** table) {
    *table = kTable;
    return int(sizeof(kTable) / sizeof(kTable[0]));
}
}  // namespace lagkv
