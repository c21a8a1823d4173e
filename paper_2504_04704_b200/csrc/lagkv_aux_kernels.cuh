// Small non-template kernels of the library: the bounded-wait self-test, the identity pass
// and the row gather.  Included by the host translation unit only.
#pragma once
#include "lagkv_kernels.cuh"

namespace lagkv {

// Self-test of the bounded wait: one warp waits on an mbarrier phase that nothing will ever
// complete; the wait must give up after limit_ns and the status block must say so.
__global__ void lagkv_selftest_wait_kernel(int32_t* status, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    const uint32_t b = smem_u32(&bar);
    if (threadIdx.x == 0) mbar_init(b, 1);
    fence_mbar_init();
    __syncthreads();
    if (!mbar_wait_bounded(b, 0u, limit_ns) && threadIdx.x == 0) record_status(status, ST_ETIMEOUT, -1);
}

// Where the caches of a call live (contiguous with strides, or a pool of pages with a block table):
// the fields of Params that make_rowmap() reads.
struct CacheLayout {
    long long sb, sh, ss, page_stride;
    const int32_t* block_table;
    int H, max_blocks, page_shift;
};
__device__ __forceinline__ RowMap layout_rowmap(const CacheLayout& c, long long u) {
    Params P;
    P.sb = c.sb;
    P.sh = c.sh;
    P.ss = c.ss;
    P.H = c.H;
    P.block_table = c.block_table;
    P.page_stride = c.page_stride;
    P.max_blocks = c.max_blocks;
    P.page_shift = c.page_shift;
    return make_rowmap(P, int(u));
}

// identity pass (S_in < S + 2L) and plain strided / paged -> contiguous copy
__global__ void lagkv_copy_kernel(const uint16_t* __restrict__ K, const uint16_t* __restrict__ V, const CacheLayout lay,
                                  int rows, int vpr, uint16_t* __restrict__ K_out,
                                  uint16_t* __restrict__ V_out, int32_t* __restrict__ idx_out, long long units) {
    const long long per_unit = (long long)rows * vpr;
    const long long total = units * per_unit;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const long long u = i / per_unit, r = (i % per_unit) / vpr;
        const int vec = int(i % vpr);
        const long long src = layout_rowmap(lay, u).off(int(r));
        if (K_out) reinterpret_cast<uint4*>(K_out + (u * rows + r) * vpr * 8)[vec] = __ldg(reinterpret_cast<const uint4*>(K + src) + vec);
        if (V_out) reinterpret_cast<uint4*>(V_out + (u * rows + r) * vpr * 8)[vec] = __ldg(reinterpret_cast<const uint4*>(V + src) + vec);
        if (idx_out && vec == 0) idx_out[u * rows + r] = int(r);
    }
}

// gather: out[u, j, :] = in[u, idx[u, j], :]
__global__ void lagkv_gather_kernel(const uint16_t* __restrict__ K, const uint16_t* __restrict__ V,
                                    const CacheLayout lay, int S_in, int vpr,
                                    const int32_t* __restrict__ idx, long long n_idx, uint16_t* __restrict__ K_out,
                                    uint16_t* __restrict__ V_out, long long units, int32_t* status) {
    const long long per_unit = n_idx * vpr;
    const long long total = units * per_unit;
    for (long long i = blockIdx.x * (long long)blockDim.x + threadIdx.x; i < total;
         i += (long long)gridDim.x * blockDim.x) {
        const long long u = i / per_unit, j = (i % per_unit) / vpr;
        const int vec = int(i % vpr);
        const int r = idx[u * n_idx + j];
        if (r < 0 || r >= S_in) {
            if (vec == 0) record_status(status, ST_EINVAL, int(u));
            continue;
        }
        const long long src = layout_rowmap(lay, u).off(r);
        reinterpret_cast<uint4*>(K_out + (u * n_idx + j) * vpr * 8)[vec] = __ldg(reinterpret_cast<const uint4*>(K + src) + vec);
        if (V_out) reinterpret_cast<uint4*>(V_out + (u * n_idx + j) * vpr * 8)[vec] = __ldg(reinterpret_cast<const uint4*>(V + src) + vec);
    }
}

}  // namespace lagkv
