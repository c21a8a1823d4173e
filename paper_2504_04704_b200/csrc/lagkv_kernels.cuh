// LagKV compress pass -- sm_100a device code.
//
// One kernel family does the whole pass of Section 2.2 (arXiv 2504.04704) with a single
// read of the cache from HBM:
//
//   * Work is a list of "slots" (unit u = (b, h), partition p), ordered so that inside a
//     unit the partitions come in DESCENDING p.  A CTA walks a contiguous range of that
//     list.  When it streams partition p it already holds the per-channel min/max of
//     partition p+1 (Eq. 7, Eq. 8) from the previous step, so in one pass over the rows it
//     (a) normalises and accumulates the per-token sum and sum of squares over head_dim
//     (Eq. 9, Eq. 10) and (b) collects p's own min/max for use by p-1.
//   * Each warp owns a private ring of shared-memory tiles filled by bulk async copies
//     (cp.async.bulk + mbarrier complete_tx); lane 0 of the warp is its own producer, so
//     the streaming loop has no block-level synchronisation.  Even warps stream K, odd
//     warps stream V.
//   * At the end of a partition the CTA runs softmax over the L tokens for K and V, adds
//     them (Eq. 11), selects the k best with a radix select on the fp32 bit pattern
//     (ties to the lower index) and copies the kept rows straight to the output layout
//     (a second read: by then the rows have left L2 again and come from DRAM).
//
// No tensor cores: the pass is a streaming reduction / selection / gather.
#pragma once
#include <cuda_runtime.h>
#include <stdint.h>

namespace lagkv {

constexpr int kStatusWords = 64;  // 256-byte status block at the start of the workspace
constexpr int kMaxWarps = 16;
constexpr int kSeqFailed = 1 << 24;  // added to a sequence's head counter by a head that gave up (H_kv < 2^24)

enum { MODE_PREFILL = 0, MODE_APPEND = 1 };
enum { ST_OK = 0, ST_EINVAL = 1, ST_ETIMEOUT = 5, ST_ECAPACITY = 6 };

struct Params {
    const uint16_t* K;  // input cache (prefill) / cache updated in place (append)
    const uint16_t* V;
    uint16_t* K_out;  // prefill: contiguous [U, L_R, D]; append: same memory as K / V
    uint16_t* V_out;
    int32_t* idx_out;
    float* scores_out;
    const int32_t* seq_len;     // append: device [B]
    const int32_t* static_len;  // append: device [B]
    int32_t* kept_pos;          // append: [U, max_chunks * k] pre-call positions of kept rows
    int32_t* seq_done;          // append: [B] heads of a sequence that have finished (workspace, zero between calls)
    int32_t* status;            // status block
    long long sb, sh, ss;       // cache strides in elements
    long long total_slots;      // prefill: U * n
    int B, H, L, k, ddof, variant, mode;
    int S_in, sink, n, rem, L_R;  // prefill
    int spu;                      // prefill, warp-specialised kernel: slots per (b, h) unit
    int max_chunks;               // append
    int stages;                   // ring depth per warp
    int sel_emit;                 // warp-specialised kernel: select warps move the kept rows of odd slots
    int res_tiles;                // append pair kernel: tiles of the window that stay in shared memory
    // paged caches (uniform kernel, gather): K / V point at a pool of pages, a sequence's rows
    // [j * page, (j + 1) * page) live in page block_table[b * max_blocks + j]; sh and ss are the
    // head and row strides inside a page, sb is unused
    const int32_t* block_table;   // device [B, max_blocks]; nullptr = not paged
    long long page_stride;        // elements between pages
    int max_blocks;
    int page_shift;               // rows per page = 1 << page_shift
};

// Where the rows of one (b, h) unit live: element offset of row r from the tensor's base pointer.
// Contiguous caches: base + r * ss.  Paged caches: page lookup, then head and row inside the page.
struct RowMap {
    long long base;        // offset of the unit (contiguous) or of the head inside a page (paged)
    long long ss;          // row stride
    const int32_t* pages;  // this sequence's row of the block table; nullptr = not paged
    long long page_stride;
    int page_shift;
    __device__ __forceinline__ long long off(int row) const {
        if (pages == nullptr) return base + (long long)row * ss;
        return (long long)__ldg(pages + (row >> page_shift)) * page_stride + base +
               (long long)(row & ((1 << page_shift) - 1)) * ss;
    }
    // how many rows starting at `row` are laid out one after another (up to the end of its page)
    __device__ __forceinline__ int run(int row) const {
        return pages == nullptr ? 0x40000000 : (1 << page_shift) - (row & ((1 << page_shift) - 1));
    }
};
__device__ __forceinline__ RowMap make_rowmap(const Params& P, int u) {
    RowMap m;
    const int b = u / P.H, h = u % P.H;
    m.ss = P.ss;
    m.page_stride = P.page_stride;
    m.page_shift = P.page_shift;
    if (P.block_table == nullptr) {
        m.pages = nullptr;
        m.base = (long long)b * P.sb + (long long)h * P.sh;
    } else {
        m.pages = P.block_table + (long long)b * P.max_blocks;
        m.base = (long long)h * P.sh;
    }
    return m;
}
// rows [row0, row0 + rows) of a unit -> shared memory at dst, completing on bar, as few bulk
// copies as the layout allows (lane 0 alone when rows are dense, else one row per lane).
// The expect_tx for all of it must already be posted.  Warp-collective.
__device__ __forceinline__ void fetch_rows(const uint16_t* X, const RowMap& m, int row0, int rows, uint32_t dst,
                                           uint32_t bar, uint32_t rowb, bool dense, int lane);


// ------------------------------------------------------------------------------ PTX helpers
__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}
__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_arrive_expect_tx(uint32_t bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(bar), "r"(parity)
        : "memory");
    return ok != 0;
}
__device__ __forceinline__ void bulk_g2s(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
        "l"(src), "r"(bytes), "r"(bar)
        : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint32_t bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void bulk_s2g(void* dst, uint32_t src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst), "r"(src), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
// every bulk store committed by this thread has finished reading shared memory
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }
// barrier over `nthreads` threads (a multiple of 32) that all name the same id (1..15)
__device__ __forceinline__ void named_bar_sync(int id, int nthreads) {
    asm volatile("bar.sync %0, %1;" ::"r"(id), "r"(nthreads) : "memory");
}
// same barrier, returning the OR of `pred` over all participants
__device__ __forceinline__ bool named_bar_or(int id, int nthreads, bool pred) {
    uint32_t r;
    asm volatile(
        "{\n\t.reg .pred p, q;\n\t"
        "setp.ne.u32 q, %3, 0;\n\t"
        "bar.red.or.pred p, %1, %2, q;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(r)
        : "r"(id), "r"(nthreads), "r"(uint32_t(pred))
        : "memory");
    return r != 0;
}
// ask L2 to fetch `bytes` (a multiple of 16, 16-byte aligned address) of global memory
__device__ __forceinline__ void prefetch_l2(const void* p, uint32_t bytes) {
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(p), "r"(bytes) : "memory");
}
__device__ __forceinline__ void fence_proxy_async() {
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
}
__device__ __forceinline__ void fence_mbar_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ unsigned long long global_timer_ns() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %globaltimer;" : "=l"(t));
    return t;
}
// Warp-collective bounded wait on an mbarrier phase: every lane polls, the warp leaves
// together, and lane 0's clock decides when to give up (about one second).  Returns false
// when the wait ran out.
__device__ __forceinline__ bool mbar_wait_bounded(uint32_t bar, uint32_t parity,
                                                  unsigned long long limit_ns = 1000000000ull) {
    if (__all_sync(0xffffffffu, mbar_try_wait(bar, parity))) return true;
    const unsigned long long t0 = global_timer_ns();
    for (int it = 0; it < (1 << 24); ++it) {
        if (__all_sync(0xffffffffu, mbar_try_wait(bar, parity))) return true;
        if ((it & 255) == 255) {
            const int late = global_timer_ns() - t0 > limit_ns;
            if (__shfl_sync(0xffffffffu, late, 0)) break;
        }
    }
    return false;
}
// packed pair of fp32 in one 64-bit register (Blackwell f32x2 arithmetic)
typedef unsigned long long f32x2;
__device__ __forceinline__ f32x2 pack2(float lo, float hi) {
    f32x2 r;
    asm("mov.b64 %0, {%1, %2};" : "=l"(r) : "f"(lo), "f"(hi));
    return r;
}
__device__ __forceinline__ void unpack2(f32x2 v, float& lo, float& hi) {
    asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(v));
}
__device__ __forceinline__ f32x2 fma2(f32x2 a, f32x2 b, f32x2 c) {
    f32x2 r;
    asm("fma.rn.f32x2 %0, %1, %2, %3;" : "=l"(r) : "l"(a), "l"(b), "l"(c));
    return r;
}
__device__ __forceinline__ f32x2 add2(f32x2 a, f32x2 b) {
    f32x2 r;
    asm("add.rn.f32x2 %0, %1, %2;" : "=l"(r) : "l"(a), "l"(b));
    return r;
}
// Storage format of the cache elements (enum lagkv_dtype): how two packed 16-bit values
// are compared and widened to fp32.  Both widenings are exact; everything after them is
// the same fp32 arithmetic.
template <int DT>
struct Elem;
template <>
struct Elem<0> {  // bf16: the upper half of an IEEE binary32
    static constexpr int EB = 2;  // bytes per element
    static constexpr int PW = 1;  // packed pairs per 32-bit word of cache data
    static __device__ __forceinline__ void expand(uint32_t w, uint32_t (&p)[1]) { p[0] = w; }
    static constexpr uint32_t kPosInf2 = 0x7f807f80u, kNegInf2 = 0xff80ff80u;
    static __device__ __forceinline__ uint32_t min2(uint32_t a, uint32_t b) {
        uint32_t r;
        asm("min.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
        return r;
    }
    static __device__ __forceinline__ uint32_t max2(uint32_t a, uint32_t b) {
        uint32_t r;
        asm("max.bf16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
        return r;
    }
    static __device__ __forceinline__ float lo(uint32_t w) { return __uint_as_float(w << 16); }
    static __device__ __forceinline__ float hi(uint32_t w) { return __uint_as_float(w & 0xffff0000u); }
};
template <>
struct Elem<1> {  // fp16: IEEE binary16
    static constexpr int EB = 2;
    static constexpr int PW = 1;
    static __device__ __forceinline__ void expand(uint32_t w, uint32_t (&p)[1]) { p[0] = w; }
    static constexpr uint32_t kPosInf2 = 0x7c007c00u, kNegInf2 = 0xfc00fc00u;
    static __device__ __forceinline__ uint32_t min2(uint32_t a, uint32_t b) {
        uint32_t r;
        asm("min.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
        return r;
    }
    static __device__ __forceinline__ uint32_t max2(uint32_t a, uint32_t b) {
        uint32_t r;
        asm("max.f16x2 %0, %1, %2;" : "=r"(r) : "r"(a), "r"(b));
        return r;
    }
    static __device__ __forceinline__ float lo(uint32_t w) {
        float f;
        asm("{ .reg .b16 l, h; mov.b32 {l, h}, %1; cvt.f32.f16 %0, l; }" : "=f"(f) : "r"(w));
        return f;
    }
    static __device__ __forceinline__ float hi(uint32_t w) {
        float f;
        asm("{ .reg .b16 l, h; mov.b32 {l, h}, %1; cvt.f32.f16 %0, h; }" : "=f"(f) : "r"(w));
        return f;
    }
};
// fp8 (e4m3, finite-only: the "fn" flavour, no infinities, 0x7f / 0xff are NaN): four values per
// word.  Every e4m3 value is a binary16 value, so a word is first expanded exactly into two packed
// fp16 pairs (one conversion instruction each) and from there on treated like fp16 data: packed
// min / max, exact widening to fp32.
template <>
struct Elem<2> : Elem<1> {
    static constexpr int EB = 1;
    static constexpr int PW = 2;
    static __device__ __forceinline__ void expand(uint32_t w, uint32_t (&p)[2]) {
        asm("{ .reg .b16 l, h; mov.b32 {l, h}, %2; cvt.rn.f16x2.e4m3x2 %0, l; cvt.rn.f16x2.e4m3x2 %1, h; }"
            : "=r"(p[0]), "=r"(p[1])
            : "r"(w));
    }
};
// two packed 16-bit values in one word -> two fp32 (exact)
template <class E>
__device__ __forceinline__ f32x2 widen2(uint32_t w) {
    return pack2(E::lo(w), E::hi(w));
}

__device__ __forceinline__ uint4 ld_nc(const uint4* p) { return __ldg(p); }
__device__ __forceinline__ void st_stream(uint4* p, uint4 v) { __stcs(p, v); }

__device__ __forceinline__ void fetch_rows(const uint16_t* X, const RowMap& m, int row0, int rows, uint32_t dst,
                                           uint32_t bar, uint32_t rowb, bool dense, int lane) {
    if (dense) {
        if (lane == 0) {
            for (int r = 0; r < rows;) {
                const int seg = min(rows - r, m.run(row0 + r));
                bulk_g2s(dst + uint32_t(r) * rowb, X + m.off(row0 + r), uint32_t(seg) * rowb, bar);
                r += seg;
            }
        }
    } else {
        __syncwarp();
        for (int r = lane; r < rows; r += 32) bulk_g2s(dst + uint32_t(r) * rowb, X + m.off(row0 + r), rowb, bar);
    }
}
// the reverse: shared memory -> rows [row0, row0 + rows) of a unit (bulk-group stores; the caller commits)
__device__ __forceinline__ void store_rows(uint16_t* X, const RowMap& m, int row0, int rows, uint32_t src, uint32_t rowb,
                                           bool dense, int lane) {
    if (dense) {
        if (lane == 0) {
            for (int r = 0; r < rows;) {
                const int seg = min(rows - r, m.run(row0 + r));
                bulk_s2g(X + m.off(row0 + r), src + uint32_t(r) * rowb, uint32_t(seg) * rowb);
                r += seg;
            }
        }
    } else {
        for (int r = lane; r < rows; r += 32) bulk_s2g(X + m.off(row0 + r), src + uint32_t(r) * rowb, rowb);
    }
}

__device__ __forceinline__ void record_status(int32_t* status, int code, int detail) {
    if (status != nullptr && atomicCAS(status, 0, code) == 0) status[1] = detail;
}

// order-preserving map fp32 -> uint32 (larger float <=> larger key)
__device__ __forceinline__ uint32_t float_key(float f) {
    uint32_t u = __float_as_uint(f);
    return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
}

// ------------------------------------------------------------------------- geometry / smem
template <int D_, int V_, int NW_, int TR_, int DT_ = 0>
struct Geo {
    using E = Elem<DT_>;                   // storage format of the cache elements
    static constexpr int DT = DT_;
    static constexpr int D = D_;           // head_dim (channels per row)
    static constexpr int V = V_;           // 16-byte vectors per thread per row
    static constexpr int NW = NW_;         // warps per CTA (even: K warps, odd: V warps)
    static constexpr int TR = TR_;         // rows per staged tile
    static constexpr int NT = NW * 32;
    static constexpr int WT = NW / 2;      // warps per tensor
    static constexpr int ROWB = D * E::EB; // bytes per row
    static constexpr int ROW16 = ROWB / 2; // row length in the 16-bit units the cache pointers count in
    static constexpr int VPR = ROWB / 16;  // 16-byte vectors per row
    static constexpr int LPR = VPR / V;    // lanes per row
    static constexpr int RPL = 32 / LPR;   // rows per warp-wide load
    static constexpr int NV = TR / RPL;    // row partials per thread per tile
    static constexpr int NWORD = 4 * V;    // 32-bit words of cache data per thread per row
    static constexpr int PW = E::PW;       // packed pairs of channels per such word (2 for fp8)
    static constexpr int NPW = NWORD * PW; // packed pairs per thread per row: min / max / coefficient registers
    static constexpr int STAT = D / 2;     // packed pairs per min (or max) row of a tensor
    static constexpr int TILE_BYTES = TR * ROWB;
    static_assert(LPR * V == VPR && RPL * LPR == 32 && NV * RPL == TR, "bad geometry");
    static_assert(NV >= 1 && NV <= LPR, "tile too tall for the transposed reduction");
    static_assert(NW >= 2 && NW <= kMaxWarps && (NW % 2) == 0, "bad warp count");
};

struct SelScratch {
    unsigned long long redq[2][kMaxWarps];
    float red[2][kMaxWarps];
    int cnt[2][kMaxWarps];
    int hist[256];
    int wsum[kMaxWarps];
    int bin;
    int krem;
    int sel_done;  // warp-specialised kernel: slots whose kept positions are published
    int claimed;   // warp-specialised kernel: leading slots whose kept rows the copy warp moves
    int abort;  // set by a warp whose bounded wait ran out; the CTA stops at the next barrier
};

template <class G>
__host__ __device__ constexpr size_t smem_ring_bytes(int stages) {
    return size_t(G::NW) * stages * G::TILE_BYTES;
}
template <class G>
__host__ __device__ inline size_t smem_total_bytes(int stages, int L) {
    size_t s = smem_ring_bytes<G>(stages);         // tile rings
    s += size_t(G::NW) * stages * 8 + 16;          // mbarriers: the rings', and two for the append move
    s += size_t(2) * G::WT * 2 * G::STAT * 4;   // per-warp min/max partials
    s += sizeof(SelScratch);
    s = (s + 15) & ~size_t(15);
    s += size_t(2) * ((L + 3) & ~3) * 4;           // sigma / score / kept arrays
    return s + 128;                                // alignment slack
}

// -------------------------------------------------------------- cross-lane row reduction
// v[i] holds this lane's partial for row-slot i; LPR consecutive lanes share the rows.
// After the call lane cg holds the full sum of slot (cg >> log2(LPR/NV)) in v[0].
template <int NV, int LPR>
__device__ __forceinline__ void transposed_reduce(float (&v)[NV], int cg) {
    int o = LPR / 2;
#pragma unroll
    for (int n = NV; n > 1; n >>= 1, o >>= 1) {
        const bool up = (cg & o) != 0;
        const int h = n / 2;
#pragma unroll
        for (int i = 0; i < h; ++i) {
            const float send = up ? v[i] : v[i + h];
            const float keep = up ? v[i + h] : v[i];
            v[i] = keep + __shfl_xor_sync(0xffffffffu, send, o);
        }
    }
#pragma unroll
    for (; o >= 1; o >>= 1) v[0] += __shfl_xor_sync(0xffffffffu, v[0], o);
}

// ---------------------------------------------------------------------------- tile math
// One staged tile of one tensor: rows [0, nrows) valid.  Updates the packed per-channel
// min / max (unless STATS is off: a partition nobody takes statistics from); when SCORE, also
// writes sigma (Std. of Eq. 10) for every valid row.
template <class G, bool SCORE, bool FULL, bool STATS = true>
__device__ __forceinline__ void process_tile(const uint4* __restrict__ tile, int nrows,
                                             const f32x2 (&a2)[G::NPW], const f32x2 (&b2)[G::NPW],
                                             uint32_t (&mn)[G::NPW], uint32_t (&mx)[G::NPW],
                                             float* __restrict__ sig_out, float inv_D, float inv_Dm,
                                             int lane) {
    const int cg = lane % G::LPR, rl = lane / G::LPR;
    float p1[G::NV], p2[G::NV];
#pragma unroll
    for (int i = 0; i < G::NV; ++i) {
        const int row = i * G::RPL + rl;
        const bool valid = FULL || row < nrows;
        f32x2 s1 = 0ull, s2 = 0ull;
#pragma unroll
        for (int v = 0; v < G::V; ++v) {
            const uint4 q = tile[row * G::VPR + v * G::LPR + cg];
            const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t pw[G::PW];
                G::E::expand(w[c], pw);
#pragma unroll
                for (int q = 0; q < G::PW; ++q) {
                    const int j = (v * 4 + c) * G::PW + q;
                    if (STATS && valid) {
                        mn[j] = G::E::min2(mn[j], pw[q]);
                        mx[j] = G::E::max2(mx[j], pw[q]);
                    }
                    if (SCORE) {
                        const f32x2 y = fma2(widen2<typename G::E>(pw[q]), a2[j], b2[j]);  // Eq. 9 (centred)
                        s1 = add2(s1, y);
                        s2 = fma2(y, y, s2);
                    }
                }
            }
        }
        if (SCORE) {
            float lo, hi;
            unpack2(s1, lo, hi);
            p1[i] = lo + hi;
            unpack2(s2, lo, hi);
            p2[i] = lo + hi;
        }
    }
    if (SCORE) {
        transposed_reduce<G::NV, G::LPR>(p1, cg);
        transposed_reduce<G::NV, G::LPR>(p2, cg);
        constexpr int DUP = G::LPR / G::NV;
        const int row = (cg / DUP) * G::RPL + rl;
        if ((cg % DUP) == 0 && (FULL || row < nrows)) {
            const float mean = p1[0] * inv_D;
            float var = (p2[0] - p1[0] * mean) * inv_Dm;
            var = fmaxf(var, 0.0f);
            sig_out[row] = sqrtf(var);
        }
    }
}

// L2-norm variant (Eq. 16): the Euclidean norm of every valid row of a staged K tile.
template <class G, bool FULL>
__device__ __forceinline__ void process_tile_l2(const uint4* __restrict__ tile, int nrows,
                                                float* __restrict__ norm_out, int lane) {
    const int cg = lane % G::LPR, rl = lane / G::LPR;
    float p2[G::NV];
#pragma unroll
    for (int i = 0; i < G::NV; ++i) {
        const int row = i * G::RPL + rl;
        f32x2 s2 = 0ull;
#pragma unroll
        for (int v = 0; v < G::V; ++v) {
            const uint4 q = tile[row * G::VPR + v * G::LPR + cg];
            const uint32_t w[4] = {q.x, q.y, q.z, q.w};
#pragma unroll
            for (int c = 0; c < 4; ++c) {
                uint32_t pw[G::PW];
                G::E::expand(w[c], pw);
#pragma unroll
                for (int q = 0; q < G::PW; ++q) {
                    const f32x2 z = widen2<typename G::E>(pw[q]);
                    s2 = fma2(z, z, s2);
                }
            }
        }
        float lo, hi;
        unpack2(s2, lo, hi);
        p2[i] = lo + hi;
    }
    transposed_reduce<G::NV, G::LPR>(p2, cg);
    constexpr int DUP = G::LPR / G::NV;
    const int row = (cg / DUP) * G::RPL + rl;
    if ((cg % DUP) == 0 && (FULL || row < nrows)) norm_out[row] = sqrtf(p2[0]);
}

// This lane's packed min / max pairs -> its places in a [mn | mx] row of shared memory (STAT words
// each; the lane owns 4 * PW consecutive words per 16-byte vector of cache data it reads).
template <class G>
__device__ __forceinline__ void store_stats_row(uint32_t* st, const uint32_t (&mn)[G::NPW], const uint32_t (&mx)[G::NPW],
                                                int cg) {
#pragma unroll
    for (int v = 0; v < G::V; ++v)
#pragma unroll
        for (int c = 0; c < 4 * G::PW; ++c) {
            st[(v * G::LPR + cg) * 4 * G::PW + c] = mn[v * 4 * G::PW + c];
            st[G::STAT + (v * G::LPR + cg) * 4 * G::PW + c] = mx[v * 4 * G::PW + c];
        }
}

// ------------------------------------------------------------------ coefficients of Eq. 9
// Combine the per-warp min / max partials of one tensor (nw rows of [mn | mx], STAT words
// each, packed bf16x2) and turn them into y = a * z + b for this lane's channels:
// y = (z - mid) / range, a shift of Eq. 9 by -1/2 that leaves the std unchanged.  A channel
// whose range is zero gets a = 0 (y constant).  Returns how many of this lane's channels
// had zero range.  The reciprocal is the hardware approximation (1 ulp), the same in every
// kernel, so scores do not depend on which kernel ran.
template <class G>
__device__ __forceinline__ int make_coefficients(const uint32_t* stats_t, int nw, int cg, f32x2 (&a2)[G::NPW],
                                                 f32x2 (&b2)[G::NPW]) {
    constexpr int STAT = G::STAT;
    uint32_t fmn[G::NPW], fmx[G::NPW];
#pragma unroll
    for (int j = 0; j < G::NPW; ++j) {
        fmn[j] = G::E::kPosInf2;
        fmx[j] = G::E::kNegInf2;
    }
    for (int w = 0; w < nw; ++w) {
        const uint4* st = reinterpret_cast<const uint4*>(stats_t + w * 2 * STAT);
#pragma unroll
        for (int v = 0; v < G::V * G::PW; ++v) {  // this lane's pairs: 4 * PW per vector, four to a 16-byte load
            const int i = (v / G::PW * G::LPR + cg) * G::PW + v % G::PW;
            const uint4 lo = st[i], hi = st[STAT / 4 + i];
            fmn[v * 4 + 0] = G::E::min2(fmn[v * 4 + 0], lo.x);
            fmn[v * 4 + 1] = G::E::min2(fmn[v * 4 + 1], lo.y);
            fmn[v * 4 + 2] = G::E::min2(fmn[v * 4 + 2], lo.z);
            fmn[v * 4 + 3] = G::E::min2(fmn[v * 4 + 3], lo.w);
            fmx[v * 4 + 0] = G::E::max2(fmx[v * 4 + 0], hi.x);
            fmx[v * 4 + 1] = G::E::max2(fmx[v * 4 + 1], hi.y);
            fmx[v * 4 + 2] = G::E::max2(fmx[v * 4 + 2], hi.z);
            fmx[v * 4 + 3] = G::E::max2(fmx[v * 4 + 3], hi.w);
        }
    }
    int zero_range = 0;
#pragma unroll
    for (int j = 0; j < G::NPW; ++j) {
        const float lo0 = G::E::lo(fmn[j]), lo1 = G::E::hi(fmn[j]);
        const float hi0 = G::E::lo(fmx[j]), hi1 = G::E::hi(fmx[j]);
        const float r0 = hi0 - lo0, r1 = hi1 - lo1;
        float i0, i1;
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(i0) : "f"(r0));
        asm("rcp.approx.ftz.f32 %0, %1;" : "=f"(i1) : "f"(r1));
        const float a0 = r0 > 0.f ? i0 : 0.f, a1 = r1 > 0.f ? i1 : 0.f;
        const float c0 = r0 > 0.f ? -(0.5f * (lo0 + hi0)) * a0 : -0.5f;
        const float c1 = r1 > 0.f ? -(0.5f * (lo1 + hi1)) * a1 : -0.5f;
        zero_range += !(r0 > 0.f);
        zero_range += !(r1 > 0.f);
        a2[j] = pack2(a0, a1);
        b2[j] = pack2(c0, c1);
    }
    return zero_range;
}

// -------------------------------------------------------------- softmax + top-k (block)
// The softmax denominators are accumulated as integers (exp value times 2^30, rounded), so
// they do not depend on which thread adds what: the scores, and with them the selection,
// are a function of the sigma values alone, bit-identical for every launch shape and for
// both implementations below.  exp is the hardware exponential of base 2 (relative error
// about 2^-22) and the division by the denominator a multiplication by its reciprocal:
// both far inside the score tolerance, and the same in every kernel.
__device__ __forceinline__ float softmax_exp(float x, float m) {
    float r;
    asm("ex2.approx.ftz.f32 %0, %1;" : "=f"(r) : "f"((x - m) * 1.4426950408889634f));
    return r;
}
__device__ __forceinline__ unsigned long long fx30(float e) { return __float2uint_rn(e * 1073741824.0f); }
__device__ __forceinline__ float fx30_to_recip(unsigned long long q) {
    return __frcp_rn(__ull2float_rn(q) * (1.0f / 1073741824.0f));
}
// Eq. 11 from the two exponentials and the reciprocals of the two softmax denominators
__device__ __forceinline__ float combine_scores(float e0, float r0, float e1, float r1) {
    return __fmaf_rn(e0, r0, __fmul_rn(e1, r1));
}
__device__ __forceinline__ unsigned long long warp_sum_u64(unsigned long long v) {
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) v += __shfl_xor_sync(0xffffffffu, v, o);
    return v;
}

// Both selectors: in sg0 = sigma(K), sg1 = sigma(V), L entries each (shared memory); out
// kept[0..k) = the selected indices ascending (kept may alias sg1), scores_g (global, may
// be null) = final scores.  All NT threads of the group call with group-local tid; sync()
// is a barrier over exactly those NT threads; release() is called by every thread once no
// thread of the group reads sg0 / sg1 any more (it may hand the buffers to a producer).

// Selector for L <= NT * E: every thread keeps E consecutive tokens in registers; the key of
// the k-th largest score is built bit by bit from block-wide counts.
template <int NT, int E, bool SOFTMAX, class Sync, class Release>
__device__ void select_in_registers(const float* sg0, const float* sg1, int L, int k,
                                    float* __restrict__ scores_g, int* kept, SelScratch& sc, int tid, Sync sync,
                                    Release release) {
    constexpr int NWARP = NT / 32;
    const int lane = tid & 31, warp = tid >> 5;
    const int t_lo = tid * E;
    float x0[E], x1[E];
    float m0 = -INFINITY, m1 = -INFINITY;
#pragma unroll
    for (int j = 0; j < E; ++j) {
        const int t = t_lo + j;
        x0[j] = t < L ? sg0[t] : -INFINITY;
        x1[j] = t < L ? sg1[t] : -INFINITY;
        m0 = fmaxf(m0, x0[j]);
        m1 = fmaxf(m1, x1[j]);
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, o));
        m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, o));
    }
    if (lane == 0) {
        sc.red[0][warp] = m0;
        sc.red[1][warp] = m1;
    }
    sync();
    release();
    m0 = sc.red[0][0];
    m1 = sc.red[1][0];
#pragma unroll
    for (int w = 1; w < NWARP; ++w) {
        m0 = fmaxf(m0, sc.red[0][w]);
        m1 = fmaxf(m1, sc.red[1][w]);
    }
    // ---- softmax over the partition's tokens, K and V side by side (Eq. 10)
    float r0 = 0.f, r1 = 0.f;
    if (SOFTMAX) {
        unsigned long long q0 = 0, q1 = 0;
#pragma unroll
        for (int j = 0; j < E; ++j) {
            x0[j] = softmax_exp(x0[j], m0);  // exp(-inf) = 0 for the padding
            x1[j] = softmax_exp(x1[j], m1);
            q0 += fx30(x0[j]);
            q1 += fx30(x1[j]);
        }
        q0 = warp_sum_u64(q0);
        q1 = warp_sum_u64(q1);
        if (lane == 0) {
            sc.redq[0][warp] = q0;
            sc.redq[1][warp] = q1;
        }
        sync();
        q0 = q1 = 0;
#pragma unroll
        for (int w = 0; w < NWARP; ++w) {
            q0 += sc.redq[0][w];
            q1 += sc.redq[1][w];
        }
        r0 = fx30_to_recip(q0);
        r1 = fx30_to_recip(q1);
    }
    // ---- Eq. 11, then the order-preserving integer image; padding gets the smallest key
    uint32_t key[E];
    uint32_t kor = 0u, kand = 0xffffffffu;
#pragma unroll
    for (int j = 0; j < E; ++j) {
        const int t = t_lo + j;
        // without the softmax (Eq. 16) sg0 holds the key norms and the score is minus the norm
        const float sco = SOFTMAX ? combine_scores(x0[j], r0, x1[j], r1) : -x0[j];
        key[j] = t < L ? float_key(sco) : 0u;
        if (t < L) {
            kor |= key[j];
            kand &= key[j];
        }
        if (scores_g != nullptr && t < L) scores_g[t] = sco;
    }
    // bits on which all keys agree need no search: find the highest bit where two keys differ
    kor = __reduce_or_sync(0xffffffffu, kor);
    kand = __reduce_and_sync(0xffffffffu, kand);
    if (lane == 0) {
        sc.cnt[0][warp] = int(kor);
        sc.cnt[1][warp] = int(kand);
    }
    sync();
#pragma unroll
    for (int w = 0; w < NWARP; ++w) {
        kor |= uint32_t(sc.cnt[0][w]);
        kand &= uint32_t(sc.cnt[1][w]);
    }
    sync();  // sc.cnt is reused by the counting rounds
    const uint32_t diff = kor ^ kand;
    const int top = 31 - __clz(diff);  // -1 when every key is the same
    // ---- T = key of the k-th largest score: the largest T with count(key >= T) >= k
    uint32_t T = top >= 0 ? (kand & ~((2u << top) - 1u)) : kand;
    for (int bit = top; bit >= 0; --bit) {
        const uint32_t cand = T | (1u << bit);
        int c = 0;
#pragma unroll
        for (int j = 0; j < E; ++j) c += key[j] >= cand;
        c = __reduce_add_sync(0xffffffffu, c);
        const int par = bit & 1;
        if (lane == 0) sc.cnt[par][warp] = c;
        sync();
        int tot = 0;
#pragma unroll
        for (int w = 0; w < NWARP; ++w) tot += sc.cnt[par][w];
        if (tot >= k) T = cand;
        if (tot == k) break;  // exactly the k largest lie at or above T: the low bits are free
    }
    // ---- positions: tokens above T all stay; of those equal to T the first krem
    int cgt = 0, ceq = 0;
#pragma unroll
    for (int j = 0; j < E; ++j) {
        cgt += key[j] > T;
        ceq += key[j] == T;
    }
    const int packed = cgt | (ceq << 16);
    int incl = packed;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) sc.wsum[warp] = incl;
    sync();
    int off = 0, total = 0;
#pragma unroll
    for (int w = 0; w < NWARP; ++w) {
        const int ws = sc.wsum[w];
        if (w < warp) off += ws;
        total += ws;
    }
    const int krem = k - (total & 0xffff);
    const int excl = off + incl - packed;
    int pgt = excl & 0xffff, peq = excl >> 16;
#pragma unroll
    for (int j = 0; j < E; ++j) {
        if (key[j] > T) {
            kept[pgt + min(peq, krem)] = t_lo + j;
            ++pgt;
        } else if (key[j] == T) {
            if (peq < krem) kept[pgt + peq] = t_lo + j;
            ++peq;
        }
    }
    sync();
}

// Selector for any L: scores stay in shared memory (sg0 is overwritten with them), radix
// select with 8 bits per pass.
template <int NT, class Sync, class Release>
__device__ void select_in_shared(float* sg0, float* sg1, int L, int k, bool softmax, float* __restrict__ scores_g,
                                 int* kept, SelScratch& sc, int tid, Sync sync, Release release) {
    constexpr int NWARP = NT / 32;
    const int lane = tid & 31, warp = tid >> 5;
    if (!softmax) {  // Eq. 16: sg0 holds the key norms, the score is minus the norm
        for (int t = tid; t < L; t += NT) {
            const float sco = -sg0[t];
            sg0[t] = sco;
            if (scores_g != nullptr) scores_g[t] = sco;
        }
        sync();
    } else {

    // ---- softmax over the partition's tokens, K and V side by side (Eq. 10)
    float m0 = -INFINITY, m1 = -INFINITY;
    for (int t = tid; t < L; t += NT) {
        m0 = fmaxf(m0, sg0[t]);
        m1 = fmaxf(m1, sg1[t]);
    }
#pragma unroll
    for (int o = 16; o >= 1; o >>= 1) {
        m0 = fmaxf(m0, __shfl_xor_sync(0xffffffffu, m0, o));
        m1 = fmaxf(m1, __shfl_xor_sync(0xffffffffu, m1, o));
    }
    if (lane == 0) {
        sc.red[0][warp] = m0;
        sc.red[1][warp] = m1;
    }
    sync();
    m0 = sc.red[0][0];
    m1 = sc.red[1][0];
#pragma unroll
    for (int w = 1; w < NWARP; ++w) {
        m0 = fmaxf(m0, sc.red[0][w]);
        m1 = fmaxf(m1, sc.red[1][w]);
    }
    unsigned long long q0 = 0, q1 = 0;
    for (int t = tid; t < L; t += NT) {
        const float e0 = softmax_exp(sg0[t], m0), e1 = softmax_exp(sg1[t], m1);
        sg0[t] = e0;
        sg1[t] = e1;
        q0 += fx30(e0);
        q1 += fx30(e1);
    }
    q0 = warp_sum_u64(q0);
    q1 = warp_sum_u64(q1);
    if (lane == 0) {
        sc.redq[0][warp] = q0;
        sc.redq[1][warp] = q1;
    }
    sync();
    q0 = q1 = 0;
#pragma unroll
    for (int w = 0; w < NWARP; ++w) {
        q0 += sc.redq[0][w];
        q1 += sc.redq[1][w];
    }
    const float r0 = fx30_to_recip(q0), r1 = fx30_to_recip(q1);
    // ---- Eq. 11
    for (int t = tid; t < L; t += NT) {
        const float sco = combine_scores(sg0[t], r0, sg1[t], r1);
        sg0[t] = sco;
        if (scores_g != nullptr) scores_g[t] = sco;
    }
    sync();
    }

    // ---- radix select: key of the k-th largest score, 8 bits per pass
    uint32_t prefix = 0, mask = 0;
    int krem = k;
    for (int shift = 24; shift >= 0; shift -= 8) {
        for (int i = tid; i < 256; i += NT) sc.hist[i] = 0;
        sync();
        for (int t0 = 0; t0 < L; t0 += NT) {
            const int t = t0 + tid;
            const bool in = t < L;
            const uint32_t key = in ? float_key(sg0[t]) : 0u;
            const bool act = in && ((key & mask) == prefix);
            const int bin = act ? int((key >> shift) & 255u) : -1 - lane;
            // warp-aggregated histogram update
            const uint32_t peers = __match_any_sync(0xffffffffu, bin);
            if (act && lane == (__ffs(peers) - 1)) atomicAdd(&sc.hist[bin], __popc(peers));
        }
        sync();
        if (warp == 0) {
            // lane owns bins [8*lane, 8*lane+8); walk from the top bin down
            int c[8], tot = 0;
#pragma unroll
            for (int i = 0; i < 8; ++i) {
                c[i] = sc.hist[lane * 8 + i];
                tot += c[i];
            }
            int above = tot;  // inclusive suffix sum over lanes >= this one
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int v = __shfl_down_sync(0xffffffffu, above, o);
                if (lane + o < 32) above += v;
            }
            const int excl = above - tot;  // count in bins of higher lanes
            if (excl < krem && krem <= above) {
                int acc = excl;
#pragma unroll
                for (int i = 7; i >= 0; --i) {
                    if (acc < krem && krem <= acc + c[i]) {
                        sc.bin = lane * 8 + i;
                        sc.krem = krem - acc;
                    }
                    acc += c[i];
                }
            }
        }
        sync();
        prefix |= uint32_t(sc.bin) << shift;
        mask |= 255u << shift;
        krem = sc.krem;
    }
    // prefix = key of the k-th largest; krem = how many tokens with exactly that key are kept

    // ---- positions: each thread owns a contiguous index range, block scan over counts
    const int E = (L + NT - 1) / NT;
    const int t_lo = min(tid * E, L), t_hi = min(t_lo + E, L);
    int cgt = 0, ceq = 0;
    for (int t = t_lo; t < t_hi; ++t) {
        const uint32_t key = float_key(sg0[t]);
        cgt += key > prefix;
        ceq += key == prefix;
    }
    int packed = cgt | (ceq << 16), incl = packed;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int v = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += v;
    }
    if (lane == 31) sc.wsum[warp] = incl;
    sync();  // also: every thread is done reading sg1, so kept[] may overwrite it
    int off = 0;
#pragma unroll
    for (int w = 0; w < NWARP; ++w)
        if (w < warp) off += sc.wsum[w];
    const int excl = off + incl - packed;
    int pgt = excl & 0xffff, peq = excl >> 16;
    for (int t = t_lo; t < t_hi; ++t) {
        const uint32_t key = float_key(sg0[t]);
        if (key > prefix) {
            kept[pgt + min(peq, krem)] = t;
            ++pgt;
        } else if (key == prefix) {
            if (peq < krem) kept[pgt + peq] = t;
            ++peq;
        }
    }
    sync();
    release();
}

// Dispatch: registers when the partition fits E tokens per thread, else shared memory.
// softmax = false: the L2-norm variant (sg0 = key norms, sg1 unused).
template <int NT, class Sync, class Release>
__device__ __forceinline__ void score_and_select(float* sg0, float* sg1, int L, int k, bool softmax,
                                                 float* __restrict__ scores_g, int* kept, SelScratch& sc, int tid,
                                                 Sync sync, Release release) {
    if (!softmax) {
        if (L <= NT * 22) select_in_registers<NT, 22, false>(sg0, sg0, L, k, scores_g, kept, sc, tid, sync, release);
        else select_in_shared<NT>(sg0, sg1, L, k, false, scores_g, kept, sc, tid, sync, release);
    } else if (L <= NT * 6) {
        select_in_registers<NT, 6, true>(sg0, sg1, L, k, scores_g, kept, sc, tid, sync, release);
    } else if (L <= NT * 11) {
        select_in_registers<NT, 11, true>(sg0, sg1, L, k, scores_g, kept, sc, tid, sync, release);
    } else if (L <= NT * 22) {
        select_in_registers<NT, 22, true>(sg0, sg1, L, k, scores_g, kept, sc, tid, sync, release);
    } else {
        select_in_shared<NT>(sg0, sg1, L, k, true, scores_g, kept, sc, tid, sync, release);
    }
}

// --------------------------------------------------------------------------- row copies
// dst rows [dst_row0, +nrows) <- src rows [src_row0, +nrows), both tensors, disjoint buffers.
template <int NT, int VPR>
__device__ void copy_rows(const uint16_t* __restrict__ srcK, const uint16_t* __restrict__ srcV,
                          const RowMap& m, uint16_t* __restrict__ dstK, uint16_t* __restrict__ dstV,
                          int src_row0, int dst_row0, int nrows, int32_t* __restrict__ idx_dst, int tid) {
    if (dstK != nullptr) {
        const long long items = (long long)nrows * 2 * VPR;
        constexpr int U = 4;
        for (long long base = 0; base < items; base += NT * U) {
            uint4 buf[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const long long i = base + u * NT + tid;
                if (i < items) {
                    const int vec = int(i % VPR);
                    const long long r2 = i / VPR;
                    const int row = int(r2 >> 1);
                    const uint16_t* s = (r2 & 1) ? srcV : srcK;
                    buf[u] = ld_nc(reinterpret_cast<const uint4*>(s + m.off(src_row0 + row)) + vec);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const long long i = base + u * NT + tid;
                if (i < items) {
                    const int vec = int(i % VPR);
                    const long long r2 = i / VPR;
                    const int row = int(r2 >> 1);
                    uint16_t* d = (r2 & 1) ? dstV : dstK;
                    st_stream(reinterpret_cast<uint4*>(d + (long long)(dst_row0 + row) * (VPR * 8)) + vec, buf[u]);
                }
            }
        }
    }
    if (idx_dst != nullptr)
        for (int r = tid; r < nrows; r += NT) idx_dst[dst_row0 + r] = src_row0 + r;
}

// kept rows of one partition -> output (prefill, out of place)
template <int NT, int VPR, int U = 4, bool PREFETCH = false>
__device__ void emit_kept(const uint16_t* __restrict__ srcK, const uint16_t* __restrict__ srcV,
                          const RowMap& m, uint16_t* __restrict__ dstK, uint16_t* __restrict__ dstV,
                          int src_row0, int dst_row0, const int* __restrict__ kept, int k,
                          int32_t* __restrict__ idx_dst, int tid) {
    if (dstK != nullptr) {
        if (PREFETCH) {  // put every kept row in flight towards L2 before the first load waits
            for (int j = tid; j < 2 * k; j += NT) {
                const uint16_t* s = (j & 1) ? srcV : srcK;
                prefetch_l2(s + m.off(src_row0 + kept[j >> 1]), VPR * 16);
            }
        }
        const int items = k * 2 * VPR;
        for (int base = 0; base < items; base += NT * U) {
            uint4 buf[U];
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int i = base + u * NT + tid;
                if (i < items) {
                    const int vec = i % VPR, r2 = i / VPR, j = r2 >> 1;
                    const uint16_t* s = (r2 & 1) ? srcV : srcK;
                    buf[u] = ld_nc(reinterpret_cast<const uint4*>(s + m.off(src_row0 + kept[j])) + vec);
                }
            }
#pragma unroll
            for (int u = 0; u < U; ++u) {
                const int i = base + u * NT + tid;
                if (i < items) {
                    const int vec = i % VPR, r2 = i / VPR, j = r2 >> 1;
                    uint16_t* d = (r2 & 1) ? dstV : dstK;
                    st_stream(reinterpret_cast<uint4*>(d + (long long)(dst_row0 + j) * (VPR * 8)) + vec, buf[u]);
                }
            }
        }
    }
    if (idx_dst != nullptr)
        for (int j = tid; j < k; j += NT) idx_dst[dst_row0 + j] = src_row0 + kept[j];
}

// In-place move inside one cache (append), by one warp through the bulk-copy engine.  Row j of
// the moved sequence (j < total) goes to row dst_row0 + j and comes from kept_pos[j] for
// j < n_kept (the picks, ascending) and from win_src0 + j after that (the window).  Sources
// and destinations both ascend and src >= dst for every j, so when chunks of R rows are taken
// in order, what a chunk overwrites lies below everything a later chunk reads: the load of
// chunk c+1 may be in flight while chunk c is stored.  Two stages of R rows of K and R rows of
// V in shared memory (the tile rings, idle by now), one mbarrier each.  K and V are the
// tensors' base pointers, m says where the unit's rows are (contiguous or paged).  Returns
// false when a bounded wait ran out.
template <class G>
__device__ bool move_rows_bulk(uint16_t* K, uint16_t* V, const RowMap& m, int dst_row0, int total, int n_kept,
                               const int32_t* kept_pos, int win_src0, uint32_t stage0, int R,
                               uint32_t bar0, int lane) {
    constexpr uint32_t ROWB = G::ROWB;
    const uint32_t stage_bytes = 2u * uint32_t(R) * ROWB;
    const bool dense = m.ss == G::ROW16;
    const int nchunks = (total + R - 1) / R;
    auto load = [&](int c) {
        const int j0 = c * R, nr = min(R, total - j0);
        const uint32_t dK = stage0 + uint32_t(c & 1) * stage_bytes, dV = dK + uint32_t(R) * ROWB;
        const uint32_t bar = bar0 + 8 * (c & 1);
        if (lane == 0) {
            fence_proxy_async();
            mbar_arrive_expect_tx(bar, 2u * uint32_t(nr) * ROWB);
        }
        __syncwarp();
        if (dense && j0 >= n_kept) {  // window rows: as few copies per tensor as the layout allows
            fetch_rows(K, m, win_src0 + j0, nr, dK, bar, ROWB, true, lane);
            fetch_rows(V, m, win_src0 + j0, nr, dV, bar, ROWB, true, lane);
        } else {
            for (int r = lane; r < nr; r += 32) {
                const int j = j0 + r;
                const long long src = m.off(j < n_kept ? kept_pos[j] : win_src0 + j);
                bulk_g2s(dK + uint32_t(r) * ROWB, K + src, ROWB, bar);
                bulk_g2s(dV + uint32_t(r) * ROWB, V + src, ROWB, bar);
            }
        }
    };
    auto store = [&](int c) -> bool {
        const int j0 = c * R, nr = min(R, total - j0);
        const uint32_t sK = stage0 + uint32_t(c & 1) * stage_bytes, sV = sK + uint32_t(R) * ROWB;
        if (!mbar_wait_bounded(bar0 + 8 * (c & 1), uint32_t(c >> 1) & 1u)) return false;
        store_rows(K, m, dst_row0 + j0, nr, sK, ROWB, dense, lane);
        store_rows(V, m, dst_row0 + j0, nr, sV, ROWB, dense, lane);
        bulk_commit();  // every lane closes a group (empty for the lanes that stored nothing)
        return true;
    };
    bool ok = true;
    for (int c = 0; c < nchunks && ok; ++c) {
        if (c >= 2) {  // this stage was last read by the store of chunk c-2
            bulk_wait_read_all();
            __syncwarp();
        }
        load(c);
        if (c >= 1) ok = store(c - 1);
    }
    if (ok && nchunks > 0) ok = store(nchunks - 1);
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // stores performed before the lengths change
    __syncwarp();
    return ok;
}

// ------------------------------------------------------------------------------- kernel
// VAR: 0 = LagKV, 1 = LocalKV, 2 = L2 norm (enum lagkv_variant), a template parameter so that the
// LagKV kernel carries none of the other variants' code.
// Two-warp CTAs are meant to run six to an SM (short partitions): their registers are capped for that.
template <class G, int VAR>
__global__ void __launch_bounds__(G::NT, (G::NW == 2 ? 6 : 1)) lagkv_stream_kernel(const Params P) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    const int NS = P.stages;
    unsigned char* ring = sm;
    uint64_t* bars = reinterpret_cast<uint64_t*>(ring + smem_ring_bytes<G>(NS));
    uint64_t* move_bars = bars + G::NW * NS;  // two more for the in-place move of the append pass
    uint32_t* stats = reinterpret_cast<uint32_t*>(move_bars + 2);  // [2][WT][2][D/2]
    SelScratch& sc = *reinterpret_cast<SelScratch*>(stats + 2 * G::WT * 2 * G::STAT);
    float* sg = reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(&sc + 1) + 15) & ~uintptr_t(15));
    const int Lp = (P.L + 3) & ~3;
    float* sg0 = sg;
    float* sg1 = sg + Lp;

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int tensor = warp & 1, wj = warp >> 1;
    const int cg = lane % G::LPR, rl = lane / G::LPR;
    const int L = P.L, k = P.k;
    const int ntiles = (L + G::TR - 1) / G::TR;
    const bool contiguous = (P.ss == G::ROW16);

    // Slot j of a unit.  LagKV (Eq. 7-9): partitions n-1 ... 0, each scored with the statistics
    // of the slot before it.  LocalKV (Eq. 14, Eq. 15): partitions n-2 ... 0, each visited twice
    // in a row, once for its own statistics and once to be scored with them.  L2 norm (Eq. 16):
    // partitions n-2 ... 0, each scored on its own from K alone.
    constexpr bool local_stats = VAR == 1, l2norm = VAR == 2;

    // ---- which slots does this CTA walk?
    long long s_first, s_hi;  // owned slots [s_first, s_hi)
    int n, spu, stat_rows, unit_fixed = 0, rem = 0;
    if (P.mode == MODE_PREFILL) {
        n = P.n;
        spu = P.spu;
        stat_rows = P.sink;
        s_first = P.total_slots * blockIdx.x / gridDim.x;
        s_hi = P.total_slots * (blockIdx.x + 1) / gridDim.x;
    } else {
        unit_fixed = blockIdx.x;
        const int b = unit_fixed / P.H;
        const int seq = P.seq_len[b];
        stat_rows = P.static_len[b];
        const int rest = seq - stat_rows;
        if (seq > P.S_in || stat_rows < 0 || rest < 0) {  // lengths that do not describe this cache
            if (tid == 0) record_status(P.status, ST_EINVAL, b);
            return;
        }
        if (rest < 2 * L) return;  // third bullet of Section 2.2: skip
        n = rest / L;
        rem = rest % L;
        if (n - 1 > P.max_chunks) {
            if (tid == 0) record_status(P.status, ST_ECAPACITY, b);
            return;
        }
        spu = local_stats ? 2 * (n - 1) : (l2norm ? n - 1 : n);
        s_first = 0;
        s_hi = spu;
    }
    if (s_first >= s_hi) return;
    auto part_of = [&](int j) -> int { return local_stats ? n - 2 - (j >> 1) : (l2norm ? n - 2 - j : n - 1 - j); };
    auto scored = [&](int j) -> bool { return local_stats ? (j & 1) != 0 : (l2norm || j != 0); };
    auto needs_prev = [&](int j) -> bool { return !l2norm && scored(j); };
    // a range that starts at a slot that needs the one before it first re-reads that one
    const bool extra = (P.mode == MODE_PREFILL) && needs_prev(int(s_first % spu));
    const long long s_lo = extra ? s_first - 1 : s_first;

    auto slot_unit = [&](long long s) -> int { return P.mode == MODE_PREFILL ? int(s / spu) : unit_fixed; };
    auto slot_part = [&](long long s) -> int { return part_of(int(s % spu)); };
    const uint16_t* tbase = tensor ? P.V : P.K;

    // ---- per-warp ring
    const uint32_t ring_w = smem_u32(ring) + uint32_t(warp) * NS * G::TILE_BYTES;
    const uint32_t bar_w = smem_u32(bars) + uint32_t(warp) * NS * 8;
    if (lane == 0)
        for (int i = 0; i < NS; ++i) mbar_init(bar_w + 8 * i, 1);
    if (tid == 0) {
        sc.abort = 0;
        mbar_init(smem_u32(move_bars), 1);
        mbar_init(smem_u32(move_bars) + 8, 1);
    }
    fence_mbar_init();
    fence_proxy_async();
    __syncthreads();

    const bool has_tiles = wj < ntiles && !(l2norm && tensor == 1);  // Eq. 16 reads K only
    long long ps = s_lo;  // producer cursor: next tile to request
    int pt = wj;
    int pslot = 0;
    int pmap_u = -1;      // unit the producer's row map is for
    RowMap pmap;
    auto issue_next = [&]() {  // warp-collective
        if (!has_tiles || ps >= s_hi) return;
        const int u = slot_unit(ps), p = slot_part(ps);
        if (u != pmap_u) {
            pmap = make_rowmap(P, u);
            pmap_u = u;
        }
        const int row0 = stat_rows + p * L + pt * G::TR;
        const int rows = min(G::TR, L - pt * G::TR);
        const uint32_t dst = ring_w + uint32_t(pslot) * G::TILE_BYTES;
        const uint32_t bar = bar_w + 8 * pslot;
        if (lane == 0) {
            fence_proxy_async();
            mbar_arrive_expect_tx(bar, uint32_t(rows) * G::ROWB);
        }
        fetch_rows(tbase, pmap, row0, rows, dst, bar, G::ROWB, contiguous, lane);
        pt += G::WT;
        if (pt >= ntiles) {
            pt = wj;
            ++ps;
        }
        if (++pslot == NS) pslot = 0;
    };
    for (int i = 0; i < NS; ++i) issue_next();

    int cslot = 0;
    uint32_t cparity = 0;
    bool timed_out = false, aborted = false;
    const float inv_D = 1.0f / float(G::D), inv_Dm = 1.0f / float(G::D - P.ddof);

    f32x2 a2[G::NPW], b2[G::NPW];
#pragma unroll
    for (int j = 0; j < G::NPW; ++j) a2[j] = b2[j] = 0ull;
    bool have_ref = false;

    for (long long s = s_lo; s < s_hi; ++s) {
        const int u = slot_unit(s), sj = int(s % spu), p = part_of(sj);
        const bool first_of_unit = sj == 0, last_of_unit = sj == spu - 1;
        const bool score = scored(sj) && s >= s_first && (have_ref || !needs_prev(sj));

        uint32_t mn[G::NPW], mx[G::NPW];
#pragma unroll
        for (int j = 0; j < G::NPW; ++j) {
            mn[j] = G::E::kPosInf2;  // +inf, +inf
            mx[j] = G::E::kNegInf2;  // -inf, -inf
        }
        float* sig = tensor ? sg1 : sg0;

        for (int t = wj; has_tiles && t < ntiles; t += G::WT) {
            if (timed_out) break;  // nothing more is consumed once a wait has run out
            const uint32_t bar = bar_w + 8 * cslot;
            if (!mbar_wait_bounded(bar, cparity)) {
                timed_out = true;
                if (lane == 0) {
                    record_status(P.status, ST_ETIMEOUT, blockIdx.x);
                    *reinterpret_cast<volatile int*>(&sc.abort) = 1;
                }
                break;
            }
            const uint4* tile = reinterpret_cast<const uint4*>(ring + size_t(warp) * NS * G::TILE_BYTES +
                                                               size_t(cslot) * G::TILE_BYTES);
            const int nrows = min(G::TR, L - t * G::TR);
            float* so = sig + t * G::TR;
            if (l2norm) {
                if (nrows == G::TR) process_tile_l2<G, true>(tile, nrows, so, lane);
                else process_tile_l2<G, false>(tile, nrows, so, lane);
            } else if (nrows == G::TR) {
                if (score) process_tile<G, true, true>(tile, nrows, a2, b2, mn, mx, so, inv_D, inv_Dm, lane);
                else process_tile<G, false, true>(tile, nrows, a2, b2, mn, mx, so, inv_D, inv_Dm, lane);
            } else {
                if (score) process_tile<G, true, false>(tile, nrows, a2, b2, mn, mx, so, inv_D, inv_Dm, lane);
                else process_tile<G, false, false>(tile, nrows, a2, b2, mn, mx, so, inv_D, inv_Dm, lane);
            }
            __syncwarp();
            issue_next();  // refill the slot just drained
            if (++cslot == NS) {
                cslot = 0;
                cparity ^= 1u;
            }
        }

        // ---- this partition's min / max (Eq. 7, Eq. 8): lanes sharing channels, then warps
#pragma unroll
        for (int j = 0; j < G::NPW; ++j) {
#pragma unroll
            for (int o = G::LPR; o < 32; o <<= 1) {
                mn[j] = G::E::min2(mn[j], __shfl_xor_sync(0xffffffffu, mn[j], o));
                mx[j] = G::E::max2(mx[j], __shfl_xor_sync(0xffffffffu, mx[j], o));
            }
        }
        if (rl == 0) {
            store_stats_row<G>(stats + ((tensor * G::WT + wj) * 2) * G::STAT, mn, mx, cg);
        }
        __syncthreads();
        aborted = *reinterpret_cast<volatile int*>(&sc.abort) != 0;
        if (aborted) break;  // uniform: every thread reads the flag after the same barrier

        // ---- select and emit partition p
        if (score) {
            const int n_c = n - 1;
            float* scores_g = nullptr;
            if (P.scores_out != nullptr)
                scores_g = (P.mode == MODE_PREFILL)
                               ? P.scores_out + ((long long)u * n_c + p) * L
                               : P.scores_out + ((long long)u * P.max_chunks + p) * L;
            score_and_select<G::NT>(sg0, sg1, L, k, !l2norm, scores_g, reinterpret_cast<int*>(sg1), sc, tid,
                                     [] { __syncthreads(); }, [] {});
            const int* kept = reinterpret_cast<const int*>(sg1);
            if (P.mode == MODE_PREFILL) {
                emit_kept<G::NT, G::VPR>(P.K, P.V, make_rowmap(P, u),
                                         P.K_out ? P.K_out + (long long)u * P.L_R * G::ROW16 : nullptr,
                                         P.V_out ? P.V_out + (long long)u * P.L_R * G::ROW16 : nullptr,
                                         stat_rows + p * L, stat_rows + p * k, kept, k,
                                         P.idx_out ? P.idx_out + (long long)u * P.L_R : nullptr, tid);
            } else {
                int32_t* kp = P.kept_pos + ((long long)u * P.max_chunks + p) * k;
                for (int j = tid; j < k; j += G::NT) kp[j] = stat_rows + p * L + kept[j];
            }
        }

        // ---- coefficients for the next (lower) partition from this one's statistics
        {
            const int zero_range = make_coefficients<G>(stats + (tensor * G::WT) * 2 * G::STAT, G::WT, cg, a2, b2);
            if (zero_range != 0 && wj == 0 && rl == 0 && !l2norm && P.status != nullptr)
                atomicAdd(P.status + 2, zero_range);
            have_ref = true;
        }

        // ---- rows copied verbatim (prefill): window with a unit's first slot, sink with its last
        if (P.mode == MODE_PREFILL && s >= s_first) {
            const RowMap um = make_rowmap(P, u);
            uint16_t* ok = P.K_out ? P.K_out + (long long)u * P.L_R * G::ROW16 : nullptr;
            uint16_t* ov = P.V_out ? P.V_out + (long long)u * P.L_R * G::ROW16 : nullptr;
            int32_t* oi = P.idx_out ? P.idx_out + (long long)u * P.L_R : nullptr;
            if (first_of_unit)
                copy_rows<G::NT, G::VPR>(P.K, P.V, um, ok, ov, stat_rows + (n - 1) * L, stat_rows + (n - 1) * k,
                                         L + P.rem, oi, tid);
            if (last_of_unit) copy_rows<G::NT, G::VPR>(P.K, P.V, um, ok, ov, 0, 0, stat_rows, oi, tid);
        }
        if (last_of_unit) have_ref = false;  // next slot belongs to another unit
        __syncthreads();
    }

    // ---- append: pack kept rows behind the static part, then slide the window down
    if (P.mode == MODE_APPEND) {
        const int u = unit_fixed;
        uint16_t* ck = const_cast<uint16_t*>(P.K);
        uint16_t* cv = const_cast<uint16_t*>(P.V);
        const int n_c = n - 1;
        const int32_t* kp = P.kept_pos + (long long)u * P.max_chunks * k;
        if (!aborted && k < L && warp == 0) {  // kept rows, then the window, as one ascending sequence of rows
            const int R = int(smem_ring_bytes<G>(NS) / (4 * G::ROWB));
            if (!move_rows_bulk<G>(ck, cv, make_rowmap(P, u), stat_rows, n_c * k + L + rem, n_c * k, kp,
                                   stat_rows + n_c * L - n_c * k, smem_u32(ring), R, smem_u32(move_bars), lane)) {
                timed_out = true;
                if (lane == 0) record_status(P.status, ST_ETIMEOUT, blockIdx.x);
            }
        }
        // The lengths of a sequence change once all of its heads are done: every head's CTA has
        // read the old values by then.  The last one to finish writes the new ones and clears
        // the counter for the next call.  A head whose wait ran out still counts (so that the
        // counter returns to zero) and marks the sequence as failed: its lengths stay as they
        // were, and its rows after the static part are undefined.
        if (tid == 0) {
            const int b = u / P.H;
            const bool failed = aborted || timed_out;  // tid 0 sits in warp 0, which did the move
            const int old = atomicAdd(P.seq_done + b, failed ? 1 + kSeqFailed : 1);
            if ((old & (kSeqFailed - 1)) == P.H - 1) {
                P.seq_done[b] = 0;
                if (!failed && old < kSeqFailed) {
                    const int ns = stat_rows + n_c * k;
                    const_cast<int32_t*>(P.static_len)[b] = ns;
                    const_cast<int32_t*>(P.seq_len)[b] = ns + L + rem;
                }
            }
        }
    }

    // a wait that ran out may have left copies in flight: give them one more bounded chance
    if (timed_out) {
        const unsigned long long t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000000ull) { /* bounded drain delay */ }
    }
}

}  // namespace lagkv
