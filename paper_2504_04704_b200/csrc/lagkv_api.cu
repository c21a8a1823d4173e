// LagKV compress pass -- host side of the C ABI declared in include/lagkv.h:
// argument checks, the planner (integers of Section 2.2 / Eq. 12, launch shapes) and the
// kernel launches.  No device memory is allocated here.
#include "lagkv.h"

#include <cmath>
#include <cstdio>
#include <cstring>
#include <mutex>
#include <new>

#include "lagkv_aux_kernels.cuh"
#include "lagkv_tables.h"

using namespace lagkv;

namespace {

// every compiled kernel: the three tables live in translation units of their own
struct KernelTable {
    static constexpr int kMaxEntries = 384;
    const KernelEntry* e[kMaxEntries];
    int n = 0;
    KernelTable() {
        const KernelEntry* t;
        int c = uniform_kernels(&t);
        for (int i = 0; i < c && n < kMaxEntries; ++i) e[n++] = t + i;
        c = uniform_dims_kernels(&t);
        for (int i = 0; i < c && n < kMaxEntries; ++i) e[n++] = t + i;
        c = uniform_dims_fp16_kernels(&t);
        for (int i = 0; i < c && n < kMaxEntries; ++i) e[n++] = t + i;
        c = ws_dims_fp16_kernels(&t);
        for (int i = 0; i < c && n < kMaxEntries; ++i) e[n++] = t + i;
        c = ws_kernels(&t);
        for (int i = 0; i < c && n < kMaxEntries; ++i) e[n++] = t + i;
        c = ws_dims_kernels(&t);
        for (int i = 0; i < c && n < kMaxEntries; ++i) e[n++] = t + i;
        c = pair_kernels(&t);
        for (int i = 0; i < c && n < kMaxEntries; ++i) e[n++] = t + i;
        c = append_pair_kernels(&t);
        for (int i = 0; i < c && n < kMaxEntries; ++i) e[n++] = t + i;
        c = ws_paged_kernels(&t);
        for (int i = 0; i < c && n < kMaxEntries; ++i) e[n++] = t + i;
        c = fp8_kernels(&t);
        for (int i = 0; i < c && n < kMaxEntries; ++i) e[n++] = t + i;
        c = fp8_dims_kernels(&t);
        for (int i = 0; i < c && n < kMaxEntries; ++i) e[n++] = t + i;
    }
};
const KernelTable& table() {
    static const KernelTable t;
    return t;
}
struct KernelRef {  // kKernels[i] reads like an array
    const KernelEntry& operator[](int i) const { return *table().e[i]; }
};
const KernelRef kKernels;
#define kNumKernels (table().n)

int find_kernel(int D, int NW, int TR, int variant, int dtype, bool paged = false) {
    for (int i = 0; i < kNumKernels; ++i)
        if (kKernels[i].D == D && kKernels[i].NW == NW && kKernels[i].TR == TR && kKernels[i].variant == variant &&
            kKernels[i].dtype == dtype && kKernels[i].paged == paged)
            return i;
    return -1;
}

constexpr int kSmemPerSm = 233472;  // 228 KiB per SM, 1 KiB reserved per resident CTA

// bytes per cache element of a storage format (enum lagkv_dtype)
int elem_bytes(int dtype) { return dtype == LAGKV_DTYPE_FP8_E4M3 ? 1 : 2; }
size_t row_bytes(const lagkv_config& c) { return size_t(c.D) * elem_bytes(c.dtype); }

}  // namespace

struct Shape {
    int kidx;         // index into kKernels
    int stages;       // ring depth per streaming warp
    int ctas_per_sm;  // grid sizing for prefill
    size_t smem;      // dynamic shared memory
};

struct lagkv_plan_s {
    lagkv_config cfg;
    int k;
    int sm_count;
    int max_smem_optin;
    Shape pre;        // kernel used by lagkv_compress_prefill
    Shape pair;       // pair kernel, preferred for short partitions with enough of them (kidx < 0: none)
    bool tuned;       // lagkv_plan_tune() fixed the prefill kernel: no switching by size
    Shape app;        // uniform kernel of lagkv_compress_append (any number of partitions per call)
    Shape app_pair;   // one-partition appends: a cluster of two CTAs per unit (kidx < 0: none)
    int app_pair_res_tiles;  // tiles of the window a CTA keeps in shared memory
    int app_pair_splits;     // row splits per tensor: the cluster has twice as many CTAs
    bool app_tuned;   // lagkv_plan_tune() fixed the uniform append shape: no pair kernel
    // lagkv_compress_prefill_host(): three streams and the events between them, made on first use
    std::mutex host_mu;
    bool host_ready = false;
    cudaStream_t host_stream[3] = {nullptr, nullptr, nullptr};  // copy in, compute, copy out
    cudaEvent_t host_start = nullptr, host_in[2] = {nullptr, nullptr}, host_comp[2] = {nullptr, nullptr},
                host_out[2] = {nullptr, nullptr};
    ~lagkv_plan_s() {
        if (!host_stream[0] && !host_start) return;
        int prev = -1;
        const bool sw = cfg.device >= 0 && cudaGetDevice(&prev) == cudaSuccess && prev != cfg.device &&
                        cudaSetDevice(cfg.device) == cudaSuccess;
        for (int i = 0; i < 3; ++i)
            if (host_stream[i]) cudaStreamDestroy(host_stream[i]);
        if (host_start) cudaEventDestroy(host_start);
        for (int i = 0; i < 2; ++i) {
            if (host_in[i]) cudaEventDestroy(host_in[i]);
            if (host_comp[i]) cudaEventDestroy(host_comp[i]);
            if (host_out[i]) cudaEventDestroy(host_out[i]);
        }
        if (sw) cudaSetDevice(prev);
    }
};

namespace {

struct DeviceGuard {
    int prev = -1;
    bool switched = false;
    explicit DeviceGuard(int dev) {
        if (dev >= 0 && cudaGetDevice(&prev) == cudaSuccess && prev != dev)
            switched = (cudaSetDevice(dev) == cudaSuccess);
    }
    ~DeviceGuard() {
        if (switched) cudaSetDevice(prev);
    }
};

int keep_count(double r, int L) {
    long long k = (long long)std::ceil(r * (double)L - 1e-9);
    if (k < 1) k = 1;
    if (k > L) k = L;
    return int(k);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

// The dynamic shared memory limit belongs to the function, not to the plan: only ever raise it, so
// that shapes of the same kernel with larger needs (this plan's or another's) keep launching.
bool raise_smem_limit(const void* fn, size_t smem) {
    static std::mutex limit_mu;  // read-then-raise must not interleave between threads
    std::lock_guard<std::mutex> lock(limit_mu);
    cudaFuncAttributes attr;
    if (cudaFuncGetAttributes(&attr, fn) != cudaSuccess) return false;
    return size_t(attr.maxDynamicSharedSizeBytes) >= smem ||
           cudaFuncSetAttribute(fn, cudaFuncAttributeMaxDynamicSharedMemorySize, int(smem)) == cudaSuccess;
}

// Try one launch shape (NW = warps per CTA, 12 = the warp-specialised kernel).
int make_shape(const lagkv_plan_s* pl, int NW, int TR, int stages, int ctas, Shape* out) {
    const int kidx = find_kernel(pl->cfg.D, NW, TR, pl->cfg.variant, pl->cfg.dtype);
    if (kidx < 0 || stages < 2 || stages > 8 || ctas < 1) return LAGKV_EUNSUPPORTED;
    if (kKernels[kidx].ws && ctas != 1) return LAGKV_EUNSUPPORTED;
    if (NW == LAGKV_TUNE_PAIRS && pl->cfg.lag > 512) return LAGKV_EUNSUPPORTED;  // one warp selects: L <= 512
    const size_t smem = kKernels[kidx].smem(stages, pl->cfg.lag);
    if (smem > size_t(pl->max_smem_optin)) return LAGKV_EUNSUPPORTED;
    if ((smem + 1024) * size_t(ctas) > size_t(kSmemPerSm)) return LAGKV_EUNSUPPORTED;
    if (pl->cfg.device >= 0 && !raise_smem_limit(reinterpret_cast<const void*>(kKernels[kidx].fn), smem))
        return LAGKV_ECUDA;
    out->kidx = kidx;
    out->stages = stages;
    out->ctas_per_sm = ctas;
    out->smem = smem;
    return LAGKV_OK;
}

// Shape of the one-partition append kernel: `code` = LAGKV_TUNE_APPEND_CLUSTER / _CLUSTER8, `splits`
// row splits per tensor, room for `ctas` CTAs per SM.  `full` demands that the whole window stays
// resident (mandatory with more than one split).
int make_append_cluster(lagkv_plan_s* pl, int code, int splits, int stages, int ctas, bool full) {
    if (splits != 1 && splits != 2 && splits != 4) return LAGKV_EUNSUPPORTED;
    if (stages < 2 || stages > 4 || ctas < 1 || ctas > 4) return LAGKV_EUNSUPPORTED;
    const int kidx = find_kernel(pl->cfg.D, code, kAppendPairTileRows, LAGKV_VARIANT_LAGKV, pl->cfg.dtype);
    if (kidx < 0 || pl->cfg.variant != LAGKV_VARIANT_LAGKV) return LAGKV_EUNSUPPORTED;
    const int L = pl->cfg.lag;
    const size_t rowb = row_bytes(pl->cfg), per_tile = size_t(kAppendPairTileRows) * rowb + 8;
    const size_t fixed = kKernels[kidx].smem(stages, L);
    size_t budget = size_t(kSmemPerSm) / size_t(ctas) - 1024;
    if (budget > size_t(pl->max_smem_optin)) budget = size_t(pl->max_smem_optin);
    if (fixed > budget) return LAGKV_EUNSUPPORTED;
    const int ntiles = (L + kAppendPairTileRows - 1) / kAppendPairTileRows;
    const int nloc = (ntiles + splits - 1) / splits;  // tiles of the largest share
    long long fit = (long long)((budget - fixed) / per_tile);
    const int res_tiles = int(fit < nloc ? fit : nloc);
    if ((full || splits > 1) && res_tiles < nloc) return LAGKV_EUNSUPPORTED;
    // with row splits a CTA gathers its share of the kept rows into the rings in one go
    const size_t ring = size_t(kKernels[kidx].threads / 32) * stages * kAppendPairTileRows * rowb;
    if (splits > 1 && size_t((pl->k + splits - 1) / splits) * rowb > ring) return LAGKV_EUNSUPPORTED;
    const size_t smem = fixed + size_t(res_tiles) * per_tile;
    if (pl->cfg.device >= 0 && !raise_smem_limit(reinterpret_cast<const void*>(kKernels[kidx].fn), smem))
        return LAGKV_ECUDA;
    pl->app_pair = Shape{kidx, stages, ctas, smem};
    pl->app_pair_res_tiles = res_tiles;
    pl->app_pair_splits = splits;
    return LAGKV_OK;
}

struct Cand {
    int NW, TR, stages, ctas;
};
int first_fit(const lagkv_plan_s* pl, const Cand* cands, int nc, Shape* out) {
    int rc = LAGKV_EUNSUPPORTED;
    for (int i = 0; i < nc; ++i) {
        rc = make_shape(pl, cands[i].NW, cands[i].TR, cands[i].stages, cands[i].ctas, out);
        if (rc == LAGKV_OK || rc == LAGKV_ECUDA) return rc;
    }
    return rc;
}

// Planner defaults.  Prefill: the warp-specialised kernel when partitions are long enough
// to keep eight streaming warps busy, else many small uniform CTAs (the per-partition
// select phase is a fixed cost that other CTAs must hide).  Append: uniform kernel, one
// CTA per (b, h).
int choose_shape(lagkv_plan_s* pl) {
    const int L = pl->cfg.lag;
    Cand uni[8];
    int nu = 0;
    if (L >= 1024 && pl->cfg.variant == LAGKV_VARIANT_LAGKV) {  // eight-warp CTAs are compiled for LagKV only
        uni[nu++] = {8, 32, 3, 1};
        uni[nu++] = {8, 32, 2, 1};
    }
    if (L >= 256) {
        uni[nu++] = {4, 32, 3, 2};
        uni[nu++] = {4, 32, 2, 2};
    }
    const int two_warp = nu;
    uni[nu++] = {2, 16, 3, 6};
    uni[nu++] = {2, 16, 3, 4};
    uni[nu++] = {2, 16, 2, 2};
    uni[nu++] = {2, 16, 2, 1};
    int rc = first_fit(pl, uni, nu, &pl->app);  // appends: deeper rings also mean larger chunks for the in-place move
    if (rc != LAGKV_OK) return rc;
    pl->pre = pl->app;
    if (two_warp == 0) {  // short partitions, prefill: two stages are 3-4 % ahead of three on the sweep cells
        Shape sh;
        if (make_shape(pl, 2, 16, 2, 6, &sh) == LAGKV_OK) pl->pre = sh;
    }
    pl->pair.kidx = -1;
    pl->tuned = false;
    pl->app_tuned = false;
    pl->app_pair.kidx = -1;
    // One-partition appends (decode).  Measured on the decode workload (L = 512, k = 128): a CTA's
    // chain of dependent steps (loads, two exchanges, selection, gather, stores) takes 15-20 us
    // whatever its share, so clusters only pay while the GPU is not full: with 64 units a cluster
    // of four per unit takes 32 us against 50 us for one CTA per unit, with 128 units a pair
    // 38 us against 42-50 us; from 256 units on the uniform kernel (two large CTAs per SM) wins.
    if (pl->cfg.variant == LAGKV_VARIANT_LAGKV) {
        const long long U = (long long)pl->cfg.B * pl->cfg.H_kv;
        int rc2 = LAGKV_EUNSUPPORTED;
        if (2 * U <= pl->sm_count) rc2 = make_append_cluster(pl, LAGKV_TUNE_APPEND_CLUSTER, 2, 2, 2, true);
        if (rc2 == LAGKV_EUNSUPPORTED && U <= pl->sm_count)
            rc2 = make_append_cluster(pl, LAGKV_TUNE_APPEND_CLUSTER, 1, 2, 2, false);
        if (rc2 == LAGKV_ECUDA) return rc2;
    }
    if (L >= 256) {
        const Cand ws[] = {{12, 32, 2, 1}, {12, 16, 3, 1}, {12, 16, 2, 1}};
        Shape sh;
        rc = first_fit(pl, ws, 3, &sh);
        if (rc == LAGKV_ECUDA) return rc;
        if (rc == LAGKV_OK) pl->pre = sh;
    }
    // Short partitions, few rows kept: four independent streams per CTA beat one partition at a
    // time (measured on the Ls = 65536 sweep).  Whether there are enough partitions to feed
    // them is known only at the call.
    if (pl->cfg.variant == LAGKV_VARIANT_LAGKV && ((L <= 128 && 4 * pl->k <= L) || (L <= 256 && 8 * pl->k <= L))) {
        // 16-row tiles when many rows are kept (2-5 % on those sweep cells), 32-row tiles otherwise
        const bool small_tiles = 4 * pl->k >= L || (L >= 128 && 8 * pl->k >= L);
        const Cand pr[] = {{LAGKV_TUNE_PAIRS, small_tiles ? 16 : 32, 2, 1}, {LAGKV_TUNE_PAIRS, small_tiles ? 32 : 16, 2, 1}};
        Shape sh;
        rc = first_fit(pl, pr, 2, &sh);
        if (rc == LAGKV_ECUDA) return rc;
        if (rc == LAGKV_OK) pl->pair = sh;
    }
    return LAGKV_OK;
}

// The prefill kernel for a call with `slots` (unit, partition) slots.
const Shape& prefill_shape(const lagkv_plan_s* pl, long long slots) {
    if (!pl->tuned && pl->pair.kidx >= 0 && slots >= 6ll * kPairs * pl->sm_count) return pl->pair;
    return pl->pre;
}

struct Strides {
    long long sb, sh, ss;
    // paged caches: block table and page geometry (block_table == nullptr: not paged)
    const int32_t* block_table = nullptr;
    long long page_stride = 0;
    int max_blocks = 0, page_shift = 0;
};
// Checks a paged layout and turns it into strides; S is the number of rows the call addresses.
int resolve_paged(const lagkv_config& c, const lagkv_paged_layout* lay, int64_t S, Strides* out) {
    if (lay == nullptr || lay->block_table == nullptr || (reinterpret_cast<uintptr_t>(lay->block_table) & 3u))
        return LAGKV_EINVAL;
    if (c.stride_b != 0 || c.stride_h != 0 || c.stride_s != 0) return LAGKV_EINVAL;  // the layout carries the strides
    const int ps = lay->page_size;
    if (ps < 16 || ps > (1 << 20) || (ps & (ps - 1)) != 0 || lay->max_blocks < 1) return LAGKV_EINVAL;
    if ((long long)lay->max_blocks * ps < S) return LAGKV_EINVAL;
    long long ss = lay->stride_s ? lay->stride_s : c.D;
    long long sh = lay->stride_h ? lay->stride_h : (long long)ps * ss;
    long long sp = lay->stride_page ? lay->stride_page : (long long)c.H_kv * sh;
    const int eb = elem_bytes(c.dtype), q = 16 / eb;  // strides are given in elements: multiples of 16 bytes
    if (ss < c.D || (ss % q) || (sh % q) || (sp % q) || sh < 0 || sp <= 0) return LAGKV_EINVAL;
    out->sb = 0;  // the kernels count in 16-bit units
    out->sh = sh * eb / 2;
    out->ss = ss * eb / 2;
    out->block_table = lay->block_table;
    out->page_stride = sp * eb / 2;
    out->max_blocks = lay->max_blocks;
    out->page_shift = 0;
    while ((1 << out->page_shift) < ps) ++out->page_shift;
    return LAGKV_OK;
}
CacheLayout cache_layout(const Strides& st, int H) {
    CacheLayout l;
    l.sb = st.sb;
    l.sh = st.sh;
    l.ss = st.ss;
    l.page_stride = st.page_stride;
    l.block_table = st.block_table;
    l.H = H;
    l.max_blocks = st.max_blocks;
    l.page_shift = st.page_shift;
    return l;
}
void set_layout(Params& P, const Strides& st) {
    P.sb = st.sb;
    P.sh = st.sh;
    P.ss = st.ss;
    P.block_table = st.block_table;
    P.page_stride = st.page_stride;
    P.max_blocks = st.max_blocks;
    P.page_shift = st.page_shift;
}
int resolve_strides(const lagkv_config& c, int64_t S, Strides* out) {
    long long ss = c.stride_s ? c.stride_s : c.D;
    long long sh = c.stride_h ? c.stride_h : (long long)S * ss;
    long long sb = c.stride_b ? c.stride_b : (long long)c.H_kv * sh;
    const int eb = elem_bytes(c.dtype), q = 16 / eb;  // strides are given in elements: multiples of 16 bytes
    if (ss < c.D || (ss % q) || (sh % q) || (sb % q) || sh < 0 || sb < 0) return LAGKV_EINVAL;
    out->sb = sb * eb / 2;  // the kernels count in 16-bit units
    out->sh = sh * eb / 2;
    out->ss = ss * eb / 2;
    return LAGKV_OK;
}

int check_launch() {
    return cudaPeekAtLastError() == cudaSuccess ? LAGKV_OK : LAGKV_ECUDA;
}

}  // namespace

// ------------------------------------------------------------------ append without a workspace
// Scratch that lagkv_compress_append_noalloc() hands to the append kernel in place of a
// caller-supplied workspace: the 256-byte status block followed by the kept-position list.
// It lives in the library image, one copy per GPU that loads the library, until the process
// exits.  In host code the symbol below is only a handle: the address a kernel can use comes
// from cudaGetSymbolAddress(), asked once per device with that device current.
static __device__ __align__(256) unsigned char g_noalloc_scratch[LAGKV_NOALLOC_SCRATCH_BYTES];

namespace {
constexpr int kMaxDevices = 64;
std::mutex g_noalloc_mutex;
void* g_noalloc_ptr[kMaxDevices] = {};

// Device address of the scratch array on `device` (which must be current); nullptr on error.
void* noalloc_scratch_for(int device) {
    if (device < 0 || device >= kMaxDevices) return nullptr;
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (g_noalloc_ptr[device] == nullptr) {
        int current = -1;  // the lookup answers for the CURRENT device: never cache it under another ordinal
        if (cudaGetDevice(&current) != cudaSuccess || current != device) return nullptr;
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_noalloc_scratch) != cudaSuccess) return nullptr;
        g_noalloc_ptr[device] = ptr;
    }
    return g_noalloc_ptr[device];
}
}  // namespace

extern "C" {

int lagkv_plan(const lagkv_config* cfg, lagkv_plan_t* out) {
    if (cfg == nullptr || out == nullptr) return LAGKV_EINVAL;
    *out = nullptr;
    if (cfg->B < 1 || cfg->H_kv < 1 || cfg->sink < 0 || cfg->lag < 2 || cfg->lag > 8192) return LAGKV_EINVAL;
    if (cfg->std_ddof != 0 && cfg->std_ddof != 1) return LAGKV_EINVAL;
    if (cfg->keep_k < 0 || cfg->keep_k > cfg->lag) return LAGKV_EINVAL;
    if (cfg->keep_k == 0 && !(cfg->keep_ratio > 0.0 && cfg->keep_ratio <= 1.0)) return LAGKV_EINVAL;
    if (cfg->stride_b < 0 || cfg->stride_h < 0 || cfg->stride_s < 0) return LAGKV_EINVAL;
    if (cfg->dtype != LAGKV_DTYPE_BF16 && cfg->dtype != LAGKV_DTYPE_FP16 && cfg->dtype != LAGKV_DTYPE_FP8_E4M3)
        return LAGKV_EINVAL;
    if (cfg->D <= 0 || (cfg->D * elem_bytes(cfg->dtype)) % 16 != 0) return LAGKV_EINVAL;
    if (cfg->variant < LAGKV_VARIANT_LAGKV || cfg->variant > LAGKV_VARIANT_L2NORM) return LAGKV_EINVAL;
    if (cfg->D != 64 && cfg->D != 96 && cfg->D != 128 && cfg->D != 256) return LAGKV_EUNSUPPORTED;
    if ((long long)cfg->B * cfg->H_kv > (1ll << 30) || 8 * (long long)cfg->H_kv >= kSeqFailed) return LAGKV_EINVAL;

    lagkv_plan_s* pl = new (std::nothrow) lagkv_plan_s();
    if (pl == nullptr) return LAGKV_EINVAL;
    pl->cfg = *cfg;
    pl->k = cfg->keep_k > 0 ? cfg->keep_k : keep_count(cfg->keep_ratio, cfg->lag);
    DeviceGuard guard(cfg->device);
    if (cfg->device < 0) {  // host-only plan: nominal B200 figures, launches are refused
        pl->sm_count = 148;
        pl->max_smem_optin = 232448;
    } else if (cudaDeviceGetAttribute(&pl->sm_count, cudaDevAttrMultiProcessorCount, cfg->device) != cudaSuccess ||
               cudaDeviceGetAttribute(&pl->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, cfg->device) !=
                   cudaSuccess) {
        delete pl;
        return LAGKV_ECUDA;
    }
    const int rc = choose_shape(pl);
    if (rc != LAGKV_OK) {
        delete pl;
        return rc;
    }
    *out = pl;
    return LAGKV_OK;
}

void lagkv_plan_destroy(lagkv_plan_t plan) { delete plan; }

int32_t lagkv_keep_count(lagkv_plan_t plan) { return plan ? plan->k : 0; }

int64_t lagkv_compressed_len(lagkv_plan_t plan, int64_t seq_len, int64_t static_len) {
    if (plan == nullptr) return -1;
    const int64_t L = plan->cfg.lag, st = static_len < 0 ? plan->cfg.sink : static_len;
    const int64_t rest = seq_len - st;
    if (rest < 2 * L) return seq_len;
    return st + int64_t(plan->k) * (rest / L - 1) + L + rest % L;
}

int lagkv_lengths_after(lagkv_plan_t plan, int64_t seq_len, int64_t static_len, int64_t* new_seq_len,
                        int64_t* new_static_len) {
    if (plan == nullptr || new_seq_len == nullptr || new_static_len == nullptr) return LAGKV_EINVAL;
    const int64_t L = plan->cfg.lag, st = static_len < 0 ? plan->cfg.sink : static_len;
    const int64_t rest = seq_len - st;
    if (rest < 0) return LAGKV_EINVAL;
    if (rest < 2 * L) {  // third bullet of Section 2.2: nothing happens
        *new_seq_len = seq_len;
        *new_static_len = st;
        return LAGKV_OK;
    }
    *new_static_len = st + int64_t(plan->k) * (rest / L - 1);
    *new_seq_len = *new_static_len + L + rest % L;
    return LAGKV_OK;
}

int32_t lagkv_keep_for_target(int64_t Ls, int32_t sink, int32_t lag, double target_C) {
    if (lag < 1 || Ls < sink + 2ll * lag) return lag;
    const int64_t n = (Ls - sink) / lag, rem = (Ls - sink) % lag;
    for (int32_t k = 1; k <= lag; ++k) {
        const int64_t L_R = sink + int64_t(k) * (n - 1) + lag + rem;
        const double C = 1.0 - double(L_R) / double(Ls);
        if (C <= target_C + 1e-12) return k;
    }
    return lag;
}

// Workspace layout: [status block | per-sequence head counters (append) | kept positions (append)]
static size_t counter_words(const lagkv_plan_s* plan) { return (size_t(plan->cfg.B) + 63) / 64 * 64; }

size_t lagkv_workspace_bytes(lagkv_plan_t plan, int32_t max_new_chunks) {
    if (plan == nullptr || max_new_chunks < 0) return 0;
    size_t bytes = kStatusWords * sizeof(int32_t);
    if (max_new_chunks > 0) bytes += counter_words(plan) * sizeof(int32_t);
    bytes += size_t(plan->cfg.B) * plan->cfg.H_kv * size_t(max_new_chunks) * plan->k * sizeof(int32_t);
    return (bytes + 255) & ~size_t(255);
}

int lagkv_workspace_init(lagkv_plan_t plan, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (plan == nullptr || plan->cfg.device < 0) return LAGKV_EINVAL;
    if (workspace == nullptr || workspace_bytes < kStatusWords * sizeof(int32_t)) return LAGKV_EWORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return LAGKV_EINVAL;
    DeviceGuard guard(plan->cfg.device);
    size_t clear = (kStatusWords + counter_words(plan)) * sizeof(int32_t);  // status block and head counters
    if (clear > workspace_bytes) clear = kStatusWords * sizeof(int32_t);    // a prefill-only workspace
    if (cudaMemsetAsync(workspace, 0, clear, static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return LAGKV_ECUDA;
    return LAGKV_OK;
}

// lagkv_compress_prefill() for the first B sequences of the plan (the host pipeline runs it chunk by chunk)
static int prefill_impl(lagkv_plan_t plan, int B, const void* K, const void* V, int64_t S_in, void* K_out,
                        void* V_out, int32_t* idx_out, float* scores_out, void* workspace,
                        size_t workspace_bytes, void* cuda_stream, const lagkv_paged_layout* paged = nullptr) {
    if (plan == nullptr || K == nullptr || V == nullptr || plan->cfg.device < 0) return LAGKV_EINVAL;
    if ((K_out == nullptr) != (V_out == nullptr)) return LAGKV_EINVAL;
    if (S_in < 0 || S_in > 0x7fffffffll - 65536) return LAGKV_EINVAL;
    if (!aligned16(K) || !aligned16(V) || !aligned16(K_out) || !aligned16(V_out)) return LAGKV_EINVAL;
    if ((reinterpret_cast<uintptr_t>(idx_out) & 3u) || (reinterpret_cast<uintptr_t>(scores_out) & 3u))
        return LAGKV_EINVAL;
    if (K_out != nullptr && (K_out == K || V_out == V || K_out == V || V_out == K)) return LAGKV_EINVAL;
    if (workspace == nullptr || workspace_bytes < kStatusWords * sizeof(int32_t)) return LAGKV_EWORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return LAGKV_EINVAL;
    const lagkv_config& c = plan->cfg;
    Strides st;
    if (paged != nullptr) {
        if (resolve_paged(c, paged, S_in, &st) != LAGKV_OK) return LAGKV_EINVAL;
    } else if (resolve_strides(c, S_in, &st) != LAGKV_OK) {
        return LAGKV_EINVAL;
    }
    if (S_in == 0) return LAGKV_OK;

    DeviceGuard guard(c.device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const long long U = (long long)B * c.H_kv;
    const int64_t rest = S_in - c.sink;

    if (rest < 2ll * c.lag) {  // pass skipped: identity
        if (K_out == nullptr && idx_out == nullptr) return LAGKV_OK;
        const int vpr = int(row_bytes(c) / 16);
        const long long total = U * S_in * vpr;
        const int block = 256;
        const long long want = (total + block - 1) / block;
        const int grid = int(want < (long long)plan->sm_count * 16 ? want : (long long)plan->sm_count * 16);
        lagkv_copy_kernel<<<grid, block, 0, stream>>>(
            static_cast<const uint16_t*>(K), static_cast<const uint16_t*>(V), cache_layout(st, c.H_kv),
            int(S_in), vpr, static_cast<uint16_t*>(K_out), static_cast<uint16_t*>(V_out), idx_out, U);
        return check_launch();
    }

    Params P;
    std::memset(&P, 0, sizeof P);
    P.K = static_cast<const uint16_t*>(K);
    P.V = static_cast<const uint16_t*>(V);
    P.K_out = static_cast<uint16_t*>(K_out);
    P.V_out = static_cast<uint16_t*>(V_out);
    P.idx_out = idx_out;
    P.scores_out = scores_out;
    P.status = static_cast<int32_t*>(workspace);
    set_layout(P, st);
    P.B = B;
    P.H = c.H_kv;
    P.L = c.lag;
    P.k = plan->k;
    P.ddof = c.std_ddof;
    P.variant = c.variant;
    P.mode = MODE_PREFILL;
    P.S_in = int(S_in);
    P.sink = c.sink;
    P.n = int(rest / c.lag);
    P.rem = int(rest % c.lag);
    P.L_R = int(lagkv_compressed_len(plan, S_in, -1));
    P.spu = c.variant == LAGKV_VARIANT_LOCALKV ? 2 * (P.n - 1) : (c.variant == LAGKV_VARIANT_L2NORM ? P.n - 1 : P.n);
    P.total_slots = U * P.spu;
    // Paged caches: the warp-specialised kernel's paged twin where the plan would use that kernel and
    // the twin is compiled (same shared memory, so the limit is raised the same way); else the
    // uniform kernel, which looks rows up page by page in every instantiation.
    Shape paged_shape;
    if (paged != nullptr) {
        paged_shape = kKernels[plan->pre.kidx].ws ? plan->app : plan->pre;
        const KernelEntry& pre = kKernels[plan->pre.kidx];
        if (pre.ws && pre.NW != LAGKV_TUNE_PAIRS) {
            const int twin = find_kernel(pre.D, pre.NW, pre.TR, pre.variant, pre.dtype, true);
            if (twin >= 0 && raise_smem_limit(reinterpret_cast<const void*>(kKernels[twin].fn), plan->pre.smem)) {
                paged_shape = plan->pre;
                paged_shape.kidx = twin;
            }
        }
    }
    const Shape& shape = paged != nullptr ? paged_shape : prefill_shape(plan, P.total_slots);
    P.stages = shape.stages;
    // Measured on the Ls = 65536 sweep and the 32K / 128K configurations: with L >= 1024 and
    // 1/8 <= k/L <= 1/4 the select warps gain 2-7 % by moving every second partition's kept rows;
    // with shorter partitions (or more rows to move) they fall behind the streamers (-4 to -25 %).
    P.sel_emit = (c.lag >= 1024 && 4 * plan->k <= c.lag && 8 * plan->k >= c.lag) ? 1 : 0;

    const KernelEntry& ke = kKernels[shape.kidx];
    long long grid = (long long)plan->sm_count * shape.ctas_per_sm;
    if (grid > P.total_slots) grid = P.total_slots;
    void* args[] = {&P};
    if (cudaLaunchKernel(reinterpret_cast<const void*>(ke.fn), dim3((unsigned)grid), dim3(ke.threads), args,
                         shape.smem, stream) != cudaSuccess)
        return LAGKV_ECUDA;
    return check_launch();
}

int lagkv_compress_prefill(lagkv_plan_t plan, const void* K, const void* V, int64_t S_in, void* K_out,
                           void* V_out, int32_t* idx_out, float* scores_out, void* workspace,
                           size_t workspace_bytes, void* cuda_stream) {
    if (plan == nullptr) return LAGKV_EINVAL;
    return prefill_impl(plan, plan->cfg.B, K, V, S_in, K_out, V_out, idx_out, scores_out, workspace, workspace_bytes,
                        cuda_stream);
}

// ---- host-resident caches ------------------------------------------------------------------
namespace {
size_t round256(size_t v) { return (v + 255) & ~size_t(255); }
struct HostSlot {  // byte offsets of one staging slot
    size_t K, V, K_out, V_out, idx, total;
};
HostSlot host_slot_layout(const lagkv_plan_s* plan, int64_t S_in, int chunk_B, int64_t L_R) {
    const size_t units = size_t(chunk_B) * plan->cfg.H_kv, row = row_bytes(plan->cfg);
    HostSlot h;
    h.K = 0;
    h.V = h.K + round256(units * S_in * row);
    h.K_out = h.V + round256(units * S_in * row);
    h.V_out = h.K_out + round256(units * L_R * row);
    h.idx = h.V_out + round256(units * L_R * row);
    h.total = h.idx + round256(units * L_R * sizeof(int32_t));
    return h;
}
int host_pipe_make(lagkv_plan_s* plan) {  // caller holds host_mu and has set the device
    if (plan->host_ready) return LAGKV_OK;
    bool ok = true;
    for (int i = 0; i < 3; ++i)
        ok = ok && cudaStreamCreateWithFlags(&plan->host_stream[i], cudaStreamNonBlocking) == cudaSuccess;
    ok = ok && cudaEventCreateWithFlags(&plan->host_start, cudaEventDisableTiming) == cudaSuccess;
    for (int i = 0; i < 2; ++i) {
        ok = ok && cudaEventCreateWithFlags(&plan->host_in[i], cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&plan->host_comp[i], cudaEventDisableTiming) == cudaSuccess;
        ok = ok && cudaEventCreateWithFlags(&plan->host_out[i], cudaEventDisableTiming) == cudaSuccess;
    }
    plan->host_ready = ok;
    return ok ? LAGKV_OK : LAGKV_ECUDA;
}
}  // namespace

size_t lagkv_host_staging_bytes(lagkv_plan_t plan, int64_t S_in, int32_t chunk_B) {
    if (plan == nullptr || S_in < 1 || S_in > 0x7fffffffll - 65536 || chunk_B < 1 || chunk_B > plan->cfg.B) return 0;
    return 2 * host_slot_layout(plan, S_in, chunk_B, lagkv_compressed_len(plan, S_in, -1)).total;
}

int lagkv_compress_prefill_host(lagkv_plan_t plan, const void* K_host, const void* V_host, int64_t S_in,
                                void* K_out_host, void* V_out_host, int32_t* idx_out_host, int32_t chunk_B,
                                void* staging, size_t staging_bytes, void* workspace, size_t workspace_bytes,
                                void* cuda_stream) {
    if (plan == nullptr || K_host == nullptr || V_host == nullptr || K_out_host == nullptr || V_out_host == nullptr ||
        idx_out_host == nullptr || plan->cfg.device < 0)
        return LAGKV_EINVAL;
    const lagkv_config& c = plan->cfg;
    if (S_in < 1 || S_in > 0x7fffffffll - 65536 || chunk_B < 1 || (c.B % chunk_B) != 0) return LAGKV_EINVAL;
    if (c.stride_b != 0 || c.stride_h != 0 || c.stride_s != 0) return LAGKV_EINVAL;  // host caches are contiguous
    if (staging == nullptr || (reinterpret_cast<uintptr_t>(staging) & 255u)) return LAGKV_EINVAL;
    if (workspace == nullptr || workspace_bytes < kStatusWords * sizeof(int32_t)) return LAGKV_EWORKSPACE;
    const int64_t L_R = lagkv_compressed_len(plan, S_in, -1);
    const HostSlot lay = host_slot_layout(plan, S_in, chunk_B, L_R);
    if (staging_bytes < 2 * lay.total) return LAGKV_EWORKSPACE;

    DeviceGuard guard(c.device);
    std::lock_guard<std::mutex> lock(plan->host_mu);  // one pipeline per plan: calls enqueue one after another
    if (host_pipe_make(plan) != LAGKV_OK) return LAGKV_ECUDA;
    cudaStream_t user = static_cast<cudaStream_t>(cuda_stream);
    cudaStream_t s_in = plan->host_stream[0], s_comp = plan->host_stream[1], s_out = plan->host_stream[2];
    bool ok = cudaEventRecord(plan->host_start, user) == cudaSuccess;
    for (int i = 0; i < 3; ++i) ok = ok && cudaStreamWaitEvent(plan->host_stream[i], plan->host_start, 0) == cudaSuccess;

    const size_t units = size_t(chunk_B) * c.H_kv, row = row_bytes(c);
    const size_t in_bytes = units * S_in * row, out_bytes = units * L_R * row, idx_bytes = units * L_R * sizeof(int32_t);
    const int chunks = c.B / chunk_B;
    int rc = LAGKV_OK;
    for (int ch = 0; ch < chunks && ok && rc == LAGKV_OK; ++ch) {
        const int sl = ch & 1;
        unsigned char* base = static_cast<unsigned char*>(staging) + size_t(sl) * lay.total;
        const unsigned char* kh = static_cast<const unsigned char*>(K_host) + size_t(ch) * in_bytes;
        const unsigned char* vh = static_cast<const unsigned char*>(V_host) + size_t(ch) * in_bytes;
        // copy in: the slot's inputs are free once the kernel of chunk ch-2 is done
        if (ch >= 2) ok = ok && cudaStreamWaitEvent(s_in, plan->host_comp[sl], 0) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(base + lay.K, kh, in_bytes, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(base + lay.V, vh, in_bytes, cudaMemcpyHostToDevice, s_in) == cudaSuccess;
        ok = ok && cudaEventRecord(plan->host_in[sl], s_in) == cudaSuccess;
        // compute: the slot's outputs are free once chunk ch-2 has been copied out
        ok = ok && cudaStreamWaitEvent(s_comp, plan->host_in[sl], 0) == cudaSuccess;
        if (ch >= 2) ok = ok && cudaStreamWaitEvent(s_comp, plan->host_out[sl], 0) == cudaSuccess;
        if (ok)
            rc = prefill_impl(plan, chunk_B, base + lay.K, base + lay.V, S_in, base + lay.K_out, base + lay.V_out,
                              reinterpret_cast<int32_t*>(base + lay.idx), nullptr, workspace, workspace_bytes, s_comp);
        ok = ok && cudaEventRecord(plan->host_comp[sl], s_comp) == cudaSuccess;
        // copy out
        ok = ok && cudaStreamWaitEvent(s_out, plan->host_comp[sl], 0) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(static_cast<unsigned char*>(K_out_host) + size_t(ch) * out_bytes, base + lay.K_out,
                                   out_bytes, cudaMemcpyDeviceToHost, s_out) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(static_cast<unsigned char*>(V_out_host) + size_t(ch) * out_bytes, base + lay.V_out,
                                   out_bytes, cudaMemcpyDeviceToHost, s_out) == cudaSuccess;
        ok = ok && cudaMemcpyAsync(reinterpret_cast<unsigned char*>(idx_out_host) + size_t(ch) * idx_bytes,
                                   base + lay.idx, idx_bytes, cudaMemcpyDeviceToHost, s_out) == cudaSuccess;
        ok = ok && cudaEventRecord(plan->host_out[sl], s_out) == cudaSuccess;
    }
    // the caller's stream continues when everything enqueued above is done (also after an error,
    // so that the staging buffers are never reused under a copy still in flight)
    for (int sl = 0; sl < 2 && sl < chunks; ++sl) {
        cudaStreamWaitEvent(user, plan->host_out[sl], 0);
        cudaStreamWaitEvent(user, plan->host_comp[sl], 0);
        cudaStreamWaitEvent(user, plan->host_in[sl], 0);
    }
    if (rc != LAGKV_OK) return rc;
    return ok ? LAGKV_OK : LAGKV_ECUDA;
}

// Host-side checks of an append call (everything that can be refused before any stream work).
static int append_check(lagkv_plan_t plan, const void* K_cache, const void* V_cache, int64_t S_cap,
                        const int32_t* seq_len, const int32_t* static_len, int32_t max_new_chunks,
                        const int32_t* idx_out, const float* scores_out, const void* workspace,
                        size_t workspace_bytes, Strides* st) {
    if (plan == nullptr || K_cache == nullptr || V_cache == nullptr || seq_len == nullptr || static_len == nullptr ||
        plan->cfg.device < 0)
        return LAGKV_EINVAL;
    if (S_cap < 1 || S_cap > 0x7fffffffll - 65536 || max_new_chunks < 1) return LAGKV_EINVAL;
    if (!aligned16(K_cache) || !aligned16(V_cache) || K_cache == V_cache) return LAGKV_EINVAL;
    if ((reinterpret_cast<uintptr_t>(idx_out) & 3u) || (reinterpret_cast<uintptr_t>(scores_out) & 3u) ||
        (reinterpret_cast<uintptr_t>(seq_len) & 3u) || (reinterpret_cast<uintptr_t>(static_len) & 3u))
        return LAGKV_EINVAL;
    if (workspace == nullptr) return LAGKV_EWORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return LAGKV_EINVAL;
    const size_t head = (kStatusWords + counter_words(plan)) * sizeof(int32_t);
    const size_t need = idx_out ? head : lagkv_workspace_bytes(plan, max_new_chunks);
    if (workspace_bytes < need) return LAGKV_EWORKSPACE;
    if (resolve_strides(plan->cfg, S_cap, st) != LAGKV_OK) return LAGKV_EINVAL;
    return LAGKV_OK;
}

static int append_impl(lagkv_plan_t plan, void* K_cache, void* V_cache, int64_t S_cap, int32_t* seq_len,
                       int32_t* static_len, int32_t max_new_chunks, int32_t* idx_out, float* scores_out,
                       void* workspace, size_t workspace_bytes, void* cuda_stream, const lagkv_paged_layout* paged) {
    Strides st;
    const int chk = append_check(plan, K_cache, V_cache, S_cap, seq_len, static_len, max_new_chunks, idx_out,
                                 scores_out, workspace, workspace_bytes, &st);
    if (chk != LAGKV_OK) return chk;
    const lagkv_config& c = plan->cfg;
    if (paged != nullptr && resolve_paged(c, paged, S_cap, &st) != LAGKV_OK) return LAGKV_EINVAL;

    DeviceGuard guard(c.device);
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    Params P;
    std::memset(&P, 0, sizeof P);
    P.K = static_cast<const uint16_t*>(K_cache);
    P.V = static_cast<const uint16_t*>(V_cache);
    P.K_out = static_cast<uint16_t*>(K_cache);
    P.V_out = static_cast<uint16_t*>(V_cache);
    P.scores_out = scores_out;
    P.seq_len = seq_len;
    P.static_len = static_len;
    P.status = static_cast<int32_t*>(workspace);
    P.seq_done = static_cast<int32_t*>(workspace) + kStatusWords;
    P.kept_pos = idx_out ? idx_out : P.seq_done + counter_words(plan);
    set_layout(P, st);
    P.B = c.B;
    P.H = c.H_kv;
    P.L = c.lag;
    P.k = plan->k;
    P.ddof = c.std_ddof;
    P.variant = c.variant;
    P.mode = MODE_APPEND;
    P.S_in = int(S_cap);
    P.sink = c.sink;
    P.max_chunks = max_new_chunks;
    P.stages = plan->app.stages;

    const long long U = (long long)c.B * c.H_kv;
    void* args[] = {&P};
    if (max_new_chunks == 1 && plan->app_pair.kidx >= 0 && !plan->app_tuned && paged == nullptr) {
        // decode: at most one partition per sequence and call -> a cluster of CTAs per unit
        const KernelEntry& kp = kKernels[plan->app_pair.kidx];
        P.idx_out = idx_out;
        P.stages = plan->app_pair.stages;
        P.res_tiles = plan->app_pair_res_tiles;
        cudaLaunchConfig_t cfg;
        std::memset(&cfg, 0, sizeof cfg);
        const unsigned cs = 2u * unsigned(plan->app_pair_splits);
        cfg.gridDim = dim3((unsigned)(cs * U));
        cfg.blockDim = dim3(kp.threads);
        cfg.dynamicSmemBytes = plan->app_pair.smem;
        cfg.stream = stream;
        cudaLaunchAttribute attr;
        attr.id = cudaLaunchAttributeClusterDimension;
        attr.val.clusterDim.x = cs;
        attr.val.clusterDim.y = 1;
        attr.val.clusterDim.z = 1;
        cfg.attrs = &attr;
        cfg.numAttrs = 1;
        if (cudaLaunchKernelExC(&cfg, reinterpret_cast<const void*>(kp.fn), args) != cudaSuccess) return LAGKV_ECUDA;
        return check_launch();
    }
    const KernelEntry& ke = kKernels[plan->app.kidx];
    if (cudaLaunchKernel(reinterpret_cast<const void*>(ke.fn), dim3((unsigned)U), dim3(ke.NW * 32), args,
                         plan->app.smem, stream) != cudaSuccess)
        return LAGKV_ECUDA;
    return check_launch();
}

int lagkv_compress_append(lagkv_plan_t plan, void* K_cache, void* V_cache, int64_t S_cap, int32_t* seq_len,
                          int32_t* static_len, int32_t max_new_chunks, int32_t* idx_out, float* scores_out,
                          void* workspace, size_t workspace_bytes, void* cuda_stream) {
    return append_impl(plan, K_cache, V_cache, S_cap, seq_len, static_len, max_new_chunks, idx_out, scores_out,
                       workspace, workspace_bytes, cuda_stream, nullptr);
}

int lagkv_compress_prefill_paged(lagkv_plan_t plan, const void* K_pool, const void* V_pool,
                                 const lagkv_paged_layout* layout, int64_t S_in, void* K_out, void* V_out,
                                 int32_t* idx_out, float* scores_out, void* workspace, size_t workspace_bytes,
                                 void* cuda_stream) {
    if (plan == nullptr || layout == nullptr) return LAGKV_EINVAL;
    return prefill_impl(plan, plan->cfg.B, K_pool, V_pool, S_in, K_out, V_out, idx_out, scores_out, workspace,
                        workspace_bytes, cuda_stream, layout);
}

int lagkv_compress_append_paged(lagkv_plan_t plan, void* K_pool, void* V_pool, const lagkv_paged_layout* layout,
                                int32_t* seq_len, int32_t* static_len, int32_t max_new_chunks, int32_t* idx_out,
                                float* scores_out, void* workspace, size_t workspace_bytes, void* cuda_stream) {
    if (plan == nullptr || layout == nullptr || layout->page_size < 1 || layout->max_blocks < 1) return LAGKV_EINVAL;
    const int64_t S_cap = (int64_t)layout->max_blocks * layout->page_size;  // rows a sequence's table can address
    return append_impl(plan, K_pool, V_pool, S_cap, seq_len, static_len, max_new_chunks, idx_out, scores_out,
                       workspace, workspace_bytes, cuda_stream, layout);
}

static int gather_impl(lagkv_plan_t plan, const void* K, const void* V, int64_t S_in, const int32_t* idx,
                       int64_t n_idx, void* K_out, void* V_out, void* workspace, void* cuda_stream,
                       const lagkv_paged_layout* paged) {
    if (plan == nullptr || K == nullptr || K_out == nullptr || idx == nullptr || plan->cfg.device < 0)
        return LAGKV_EINVAL;
    if ((V == nullptr) != (V_out == nullptr)) return LAGKV_EINVAL;
    if (S_in < 1 || S_in > 0x7fffffffll - 65536 || n_idx < 0) return LAGKV_EINVAL;
    if (!aligned16(K) || !aligned16(V) || !aligned16(K_out) || !aligned16(V_out)) return LAGKV_EINVAL;
    if ((reinterpret_cast<uintptr_t>(idx) & 3u) || (reinterpret_cast<uintptr_t>(workspace) & 255u))
        return LAGKV_EINVAL;
    const lagkv_config& c = plan->cfg;
    Strides st;
    if (paged != nullptr) {
        if (resolve_paged(c, paged, S_in, &st) != LAGKV_OK) return LAGKV_EINVAL;
    } else if (resolve_strides(c, S_in, &st) != LAGKV_OK) {
        return LAGKV_EINVAL;
    }
    if (n_idx == 0) return LAGKV_OK;
    DeviceGuard guard(c.device);
    const long long U = (long long)c.B * c.H_kv;
    const int vpr = int(row_bytes(c) / 16);
    const long long total = U * n_idx * vpr;
    const int block = 256;
    const long long want = (total + block - 1) / block;
    const int grid = int(want < (long long)plan->sm_count * 16 ? want : (long long)plan->sm_count * 16);
    lagkv_gather_kernel<<<grid, block, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        static_cast<const uint16_t*>(K), static_cast<const uint16_t*>(V), cache_layout(st, c.H_kv), int(S_in),
        vpr, idx, n_idx, static_cast<uint16_t*>(K_out), static_cast<uint16_t*>(V_out), U,
        static_cast<int32_t*>(workspace));
    return check_launch();
}

int lagkv_gather(lagkv_plan_t plan, const void* K, const void* V, int64_t S_in, const int32_t* idx, int64_t n_idx,
                 void* K_out, void* V_out, void* workspace, void* cuda_stream) {
    return gather_impl(plan, K, V, S_in, idx, n_idx, K_out, V_out, workspace, cuda_stream, nullptr);
}

int lagkv_gather_paged(lagkv_plan_t plan, const void* K_pool, const void* V_pool, const lagkv_paged_layout* layout,
                       int64_t S_in, const int32_t* idx, int64_t n_idx, void* K_out, void* V_out, void* workspace,
                       void* cuda_stream) {
    if (layout == nullptr) return LAGKV_EINVAL;
    return gather_impl(plan, K_pool, V_pool, S_in, idx, n_idx, K_out, V_out, workspace, cuda_stream, layout);
}

int lagkv_read_status(lagkv_plan_t plan, void* workspace, void* cuda_stream, int32_t host_status[4]) {
    if (plan == nullptr || host_status == nullptr || plan->cfg.device < 0) return LAGKV_EINVAL;
    DeviceGuard guard(plan->cfg.device);
    if (workspace == nullptr) {  // the status block of the library's built-in scratch on the plan's device
        workspace = noalloc_scratch_for(plan->cfg.device);
        if (workspace == nullptr) return LAGKV_ECUDA;
    }
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    if (cudaMemcpyAsync(host_status, workspace, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost, stream) != cudaSuccess)
        return LAGKV_ECUDA;
    if (cudaMemsetAsync(workspace, 0, kStatusWords * sizeof(int32_t), stream) != cudaSuccess) return LAGKV_ECUDA;
    if (cudaStreamSynchronize(stream) != cudaSuccess) return LAGKV_ECUDA;
    return host_status[0];
}

int lagkv_launch_info(lagkv_plan_t plan, int64_t S_in, int32_t info[6]) {
    if (plan == nullptr || info == nullptr || S_in < 0) return LAGKV_EINVAL;
    const lagkv_config& c = plan->cfg;
    const long long U = (long long)c.B * c.H_kv;
    const int64_t rest = S_in - c.sink;
    if (rest < 2ll * c.lag) {
        const long long total = U * S_in * (long long)(row_bytes(c) / 16);
        const long long want = (total + 255) / 256;
        info[0] = int(want < (long long)plan->sm_count * 16 ? want : (long long)plan->sm_count * 16);
        info[1] = 256;
        info[2] = 0;
        info[3] = S_in > 0 ? 1 : 0;
        info[4] = info[5] = 0;
        return LAGKV_OK;
    }
    const long long nparts = rest / c.lag;
    const long long slots = U * (c.variant == LAGKV_VARIANT_LOCALKV ? 2 * (nparts - 1)
                                 : c.variant == LAGKV_VARIANT_L2NORM ? nparts - 1 : nparts);
    const Shape& shape = prefill_shape(plan, slots);
    const long long grid = (long long)plan->sm_count * shape.ctas_per_sm;
    info[0] = int(grid < slots ? grid : slots);
    info[1] = kKernels[shape.kidx].threads;
    info[2] = int(shape.smem);
    info[3] = 1;
    const KernelEntry& ke = kKernels[shape.kidx];
    info[4] = !ke.ws ? 1 : (ke.NW == LAGKV_TUNE_PAIRS ? 3 : 2);
    // family of the same call on a paged cache: the warp-specialised kernel where its paged twin is
    // compiled and the plan would use that family, else the uniform kernel
    const KernelEntry& pre = kKernels[plan->pre.kidx];
    info[5] = (pre.ws && pre.NW != LAGKV_TUNE_PAIRS && find_kernel(pre.D, pre.NW, pre.TR, pre.variant, pre.dtype, true) >= 0) ? 2 : 1;
    return LAGKV_OK;
}

int lagkv_plan_tune(lagkv_plan_t plan, int32_t warps, int32_t tile_rows, int32_t stages, int32_t ctas_per_sm) {
    if (plan == nullptr) return LAGKV_EINVAL;
    DeviceGuard guard(plan->cfg.device);
    if (warps == LAGKV_TUNE_APPEND_CLUSTER || warps == LAGKV_TUNE_APPEND_CLUSTER8) {
        const int splits = tile_rows ? tile_rows : (plan->app_pair.kidx >= 0 ? plan->app_pair_splits : 1);
        const int st = stages ? stages : 2, ct = ctas_per_sm ? ctas_per_sm : 1;
        const int rc = make_append_cluster(plan, warps, splits, st, ct, false);
        if (rc == LAGKV_OK) plan->app_tuned = false;
        return rc;
    }
    const KernelEntry& cur = kKernels[plan->pre.kidx];
    Shape sh;
    const int rc = make_shape(plan, warps ? warps : cur.NW, tile_rows ? tile_rows : cur.TR,
                              stages ? stages : plan->pre.stages, ctas_per_sm ? ctas_per_sm : plan->pre.ctas_per_sm,
                              &sh);
    if (rc != LAGKV_OK) return rc;
    plan->pre = sh;
    plan->tuned = true;
    if (!kKernels[sh.kidx].ws) {
        plan->app = sh;
        plan->app_tuned = true;
    }
    return LAGKV_OK;
}

int lagkv_selftest_bounded_wait(lagkv_plan_t plan, void* workspace, int32_t limit_ms, void* cuda_stream) {
    if (plan == nullptr || workspace == nullptr || plan->cfg.device < 0 || limit_ms < 1 || limit_ms > 2000)
        return LAGKV_EINVAL;
    if (reinterpret_cast<uintptr_t>(workspace) & 255u) return LAGKV_EINVAL;
    DeviceGuard guard(plan->cfg.device);
    lagkv_selftest_wait_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        static_cast<int32_t*>(workspace), 1000000ull * (unsigned long long)limit_ms);
    return check_launch();
}

const char* lagkv_status_string(int status) {
    switch (status) {
        case LAGKV_OK: return "ok";
        case LAGKV_EINVAL: return "invalid argument";
        case LAGKV_EUNSUPPORTED: return "unsupported configuration";
        case LAGKV_EWORKSPACE: return "workspace missing or too small";
        case LAGKV_ECUDA: return "CUDA error";
        case LAGKV_ETIMEOUT: return "device wait timed out";
        case LAGKV_ECAPACITY: return "append needs more chunks than max_new_chunks";
        case LAGKV_ENOALLOC_LIMIT: return "request exceeds the library's built-in scratch (LAGKV_NOALLOC_SCRATCH_BYTES)";
        default: return "unknown status";
    }
}

const char* lagkv_version(void) { return "lagkv-b200 0.1 (sm_100a)"; }

}  // extern "C"

extern "C" int lagkv_compress_append_noalloc(lagkv_plan_t plan, void* K_cache, void* V_cache, int64_t S_cap,
                                             int32_t* seq_len, int32_t* static_len, int32_t max_new_chunks,
                                             int32_t* idx_out, float* scores_out, int32_t* status_out,
                                             void* cuda_stream) {
    if (plan == nullptr || plan->cfg.device < 0 || max_new_chunks < 1) return LAGKV_EINVAL;
    if (reinterpret_cast<uintptr_t>(status_out) & 3u) return LAGKV_EINVAL;
    // without idx_out the kernel parks the kept positions in the scratch: that list must fit
    const size_t head = (kStatusWords + counter_words(plan)) * sizeof(int32_t);
    const size_t need = idx_out ? head : lagkv_workspace_bytes(plan, max_new_chunks);
    if (need == 0 || need > size_t(LAGKV_NOALLOC_SCRATCH_BYTES)) return LAGKV_ENOALLOC_LIMIT;
    DeviceGuard guard(plan->cfg.device);
    void* scratch = noalloc_scratch_for(plan->cfg.device);
    if (scratch == nullptr) return LAGKV_ECUDA;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    {  // refuse bad arguments before anything is enqueued: a refused call leaves the scratch as it was
        Strides st;
        const int chk = append_check(plan, K_cache, V_cache, S_cap, seq_len, static_len, max_new_chunks, idx_out,
                                     scores_out, scratch, size_t(LAGKV_NOALLOC_SCRATCH_BYTES), &st);
        if (chk != LAGKV_OK) return chk;
    }
    // the array keeps what the previous call left: the status block and the per-sequence head
    // counters have to start at zero
    if (cudaMemsetAsync(scratch, 0, head, stream) != cudaSuccess) return LAGKV_ECUDA;
    const int rc = lagkv_compress_append(plan, K_cache, V_cache, S_cap, seq_len, static_len, max_new_chunks, idx_out,
                                         scores_out, scratch, size_t(LAGKV_NOALLOC_SCRATCH_BYTES), stream);
    if (rc != LAGKV_OK) return rc;
    if (status_out != nullptr &&
        cudaMemcpyAsync(status_out, scratch, 4 * sizeof(int32_t), cudaMemcpyDeviceToDevice, stream) != cudaSuccess)
        return LAGKV_ECUDA;
    return LAGKV_OK;
}
