// Tables of the compiled kernel instantiations.  Each kernel family is instantiated in a
// translation unit of its own (they compile in parallel); the host code sees them through
// these tables only.
#pragma once
#include "lagkv.h"
#include "lagkv_kernels.cuh"
#include "lagkv_ws_kernel.cuh"
#include "lagkv_pair_kernel.cuh"

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
};

// each returns the number of entries and sets *table
int uniform_kernels(const KernelEntry** table);  // lagkv_stream_kernel: prefill and append
int ws_kernels(const KernelEntry** table);       // lagkv_ws_kernel: warp-specialised prefill
int pair_kernels(const KernelEntry** table);     // lagkv_pair_kernel: prefill, short partitions

}  // namespace lagkv
