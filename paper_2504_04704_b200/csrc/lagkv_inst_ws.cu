// Instantiations of the warp-specialised prefill kernel, one per geometry and scoring variant.
#include "lagkv_tables.h"

namespace lagkv {
namespace {
#define LAGKV_WS_ENTRY2(D, V, NWS, TR, VAR, DT) \
    { D, NWS + kWsEpiWarps, TR, VAR, DT, true, (NWS + kWsEpiWarps) * 32, \
      &lagkv_ws_kernel<Geo<D, V, NWS, TR, DT>, VAR>, &ws_smem_total_bytes<Geo<D, V, NWS, TR, DT>> }
#define LAGKV_WS_ENTRY_DT(D, V, NWS, TR, DT) \
    LAGKV_WS_ENTRY2(D, V, NWS, TR, 0, DT), LAGKV_WS_ENTRY2(D, V, NWS, TR, 1, DT), LAGKV_WS_ENTRY2(D, V, NWS, TR, 2, DT)
#define LAGKV_WS_ENTRY(D, V, NWS, TR) LAGKV_WS_ENTRY_DT(D, V, NWS, TR, 0)

const KernelEntry kTable[] = {
    LAGKV_WS_ENTRY(128, 2, 8, 32), LAGKV_WS_ENTRY(128, 2, 8, 16), LAGKV_WS_ENTRY(64, 1, 8, 32),
    LAGKV_WS_ENTRY(64, 1, 8, 16), LAGKV_WS_ENTRY(256, 2, 8, 16), LAGKV_WS_ENTRY(96, 3, 8, 32),
    LAGKV_WS_ENTRY(96, 3, 8, 16), LAGKV_WS_ENTRY_DT(128, 2, 8, 32, 1), LAGKV_WS_ENTRY_DT(128, 2, 8, 16, 1),
};
}  // namespace

int ws_kernels(const KernelEntry** table) {
    *table = kTable;
    return int(sizeof(kTable) / sizeof(kTable[0]));
}
}  // namespace lagkv
