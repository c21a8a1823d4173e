// Tables of the compiled kernel instantiations.  Each kernel family is instantiated in a
// translation unit of its own (they compile in parallel); the host code sees them through
// these tables only.
#pragma once
#include "lagkv.h"
#include "lagkv_kernels.cuh"
#include "lagkv_ws_kernel.cuh"
#include "lagkv_pair_kernel.cuh"
#include "lagkv_append_pair_kernel.cuh"

namespace lagkv {

typedef void (*stream_kernel_t)(const Params);
typedef size_t (*smem_fn_t)(int, int);

struct KernelEntry {
    int D, NW, TR;  // NW: warps per CTA as named in lagkv_plan_tune() (LAGKV_TUNE_PAIRS for the pair kernel)
    int variant;    // enum lagkv_variant the kernel was compiled for
    int dtype;      // enum lagkv_dtype of the cache elements
    bool ws;        // a persistent prefill-only kernel (warp-specialised or pair), one CTA per SM
    int threads;    // CTA size
    stream_kernel_t fn;
    smem_fn_t smem;
    bool paged = false;  // reads its caches through a block table (the uniform kernel does both)
};

// each returns the number of entries and sets *table; the "_dims" tables hold the head
// dimensions other than 128 (separate translation units, so that they compile side by side)
int uniform_kernels(const KernelEntry** table);       // lagkv_stream_kernel: prefill and append
int uniform_dims_kernels(const KernelEntry** table);
int uniform_dims_fp16_kernels(const KernelEntry** table);
int ws_kernels(const KernelEntry** table);            // lagkv_ws_kernel: warp-specialised prefill
int ws_dims_kernels(const KernelEntry** table);
int ws_dims_fp16_kernels(const KernelEntry** table);
int pair_kernels(const KernelEntry** table);          // lagkv_pair_kernel: prefill, short partitions
// lagkv_append_pair_kernel: one-partition appends on a cluster of 2, 4 or 8 CTAs per unit.  NW
// holds LAGKV_TUNE_APPEND_CLUSTER (4 warps per CTA) or LAGKV_TUNE_APPEND_CLUSTER8 (8 warps);
// smem() gives the size without resident tiles (TILE_BYTES + 8 each).
int append_pair_kernels(const KernelEntry** table);
constexpr int kAppendPairTileRows = 16;

// ---- table entries: (head_dim, vectors per lane, warps, tile rows, variant, element format)
#define LAGKV_ENTRY2(D, V, NW, TR, VAR, DT) \
    { D, NW, TR, VAR, DT, false, NW * 32, &lagkv_stream_kernel<Geo<D, V, NW, TR, DT>, VAR>, \
      &smem_total_bytes<Geo<D, V, NW, TR, DT>> }
#define LAGKV_ENTRY1(D, V, NW, TR, VAR) LAGKV_ENTRY2(D, V, NW, TR, VAR, 0)
#define LAGKV_ENTRY(D, V, NW, TR) LAGKV_ENTRY1(D, V, NW, TR, 0)
/* every uniform shape for LagKV */
#define LAGKV_SHAPE_ENTRIES(D, V) \
    LAGKV_ENTRY(D, V, 8, 32), LAGKV_ENTRY(D, V, 4, 32), LAGKV_ENTRY(D, V, 2, 32), LAGKV_ENTRY(D, V, 8, 16), \
    LAGKV_ENTRY(D, V, 4, 16), LAGKV_ENTRY(D, V, 2, 16)
/* the two shapes the planner uses for appends, also for the LocalKV and L2-norm variants */
#define LAGKV_VARIANT_ENTRIES(D, V) \
    LAGKV_ENTRY1(D, V, 4, 32, 1), LAGKV_ENTRY1(D, V, 4, 32, 2), LAGKV_ENTRY1(D, V, 2, 16, 1), LAGKV_ENTRY1(D, V, 2, 16, 2)
/* fp16 (or another format's) caches: the planner's default shapes, every variant */
#define LAGKV_FP16_ENTRIES_DT(D, V, DT) \
    LAGKV_ENTRY2(D, V, 8, 32, 0, DT), LAGKV_ENTRY2(D, V, 4, 32, 0, DT), LAGKV_ENTRY2(D, V, 2, 16, 0, DT), \
    LAGKV_ENTRY2(D, V, 4, 32, 1, DT), LAGKV_ENTRY2(D, V, 4, 32, 2, DT), LAGKV_ENTRY2(D, V, 2, 16, 1, DT), \
    LAGKV_ENTRY2(D, V, 2, 16, 2, DT)
#define LAGKV_FP16_ENTRIES(D, V) LAGKV_FP16_ENTRIES_DT(D, V, 1)
#define LAGKV_WS_ENTRY2(D, V, NWS, TR, VAR, DT) \
    { D, NWS + kWsEpiWarps, TR, VAR, DT, true, (NWS + kWsEpiWarps) * 32, \
      &lagkv_ws_kernel<Geo<D, V, NWS, TR, DT>, VAR>, &ws_smem_total_bytes<Geo<D, V, NWS, TR, DT>> }
#define LAGKV_WS_ENTRY_DT(D, V, NWS, TR, DT) \
    LAGKV_WS_ENTRY2(D, V, NWS, TR, 0, DT), LAGKV_WS_ENTRY2(D, V, NWS, TR, 1, DT), LAGKV_WS_ENTRY2(D, V, NWS, TR, 2, DT)
#define LAGKV_WS_ENTRY(D, V, NWS, TR) LAGKV_WS_ENTRY_DT(D, V, NWS, TR, 0)
/* the same kernel for paged caches (LagKV scoring) */
#define LAGKV_WS_PAGED_ENTRY(D, V, NWS, TR, DT) \
    { D, NWS + kWsEpiWarps, TR, 0, DT, true, (NWS + kWsEpiWarps) * 32, \
      &lagkv_ws_kernel<Geo<D, V, NWS, TR, DT>, 0, true>, &ws_smem_total_bytes<Geo<D, V, NWS, TR, DT>>, true }
int ws_paged_kernels(const KernelEntry** table);      // lagkv_ws_kernel reading paged caches
int fp8_kernels(const KernelEntry** table);           // every family for fp8 (e4m3) caches, head_dim 128
int fp8_dims_kernels(const KernelEntry** table);      // ... head_dim 64, 96, 256

}  // namespace lagkv
