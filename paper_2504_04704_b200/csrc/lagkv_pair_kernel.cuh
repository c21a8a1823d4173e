// LagKV prefill compress pass for SHORT partitions -- persistent "pair" kernel for sm_100a.
//
// With short partitions (L <= 512) a CTA that works on one partition at a time is bound by
// the serial chain per partition (wait for the tiles, reduce, exchange statistics, select),
// not by memory.  Here a CTA runs four independent streams instead.  A stream is a pair of
// streaming warps (one for K, one for V) plus one epilogue warp, and owns its own contiguous
// range of slots (LagKV, Eq. 7-11: partitions of a unit in descending order, so the
// statistics of partition p+1 are in registers when p streams through):
//
//   * the K warp and the V warp each stream all tiles of a partition through a private ring
//     of bulk async copies, compute sigma (Eq. 9, Eq. 10) and the partition's own min / max
//     and derive the next coefficients themselves: no barrier between streaming warps at all;
//   * the epilogue warp takes the two sigma vectors (double buffered, mbarrier hand-off), runs
//     softmax, K + V (Eq. 11) and the top-k entirely with warp shuffles, writes the positions
//     and copies the kept rows right away, as well as the unit's window and sink rows.
//
// Scores are bit-identical to the other kernels' (same row sums, same integer softmax
// denominators, same exp and reciprocal), so the selection is too.
// Every wait on an mbarrier is bounded; a warp whose wait ran out records LAGKV_ETIMEOUT and
// keeps only the arrivals alive so that its partners do not block.
#pragma once
#include "lagkv_kernels.cuh"

namespace lagkv {

constexpr int kPairs = 4;  // streams per CTA: 8 streaming warps + 4 epilogue warps

template <class G>
__host__ __device__ inline size_t pair_smem_total_bytes(int stages, int L) {
    const size_t Lp = (L + 3) & ~3;
    size_t s = smem_ring_bytes<G>(stages);             // tile rings
    s += (size_t(G::NW) * stages + 4 * kPairs) * 8;    // mbarriers: rings, full[2] / empty[2] per pair
    s += size_t(G::NW) * 2 * G::STAT * 4;           // own min / max row of every streaming warp
    s += size_t(kPairs) * 2 * 2 * Lp * 4;              // sigma [pair][2 buffers][K, V]
    s += size_t(kPairs) * Lp * 4;                      // kept indices [pair]
    s += size_t(kPairs) * 4;                           // give-up flag [pair]
    return s + 128;                                    // alignment slack
}

// Selection by one warp: lane l holds tokens [l*E, l*E + E).  Same arithmetic as
// select_in_registers, with shuffles in place of shared memory and barriers.
template <int E, class Release>
__device__ void select_in_warp(const float* sg0, const float* sg1, int L, int k, float* __restrict__ scores_g,
                               int* kept, int lane, Release release) {
    const int t_lo = lane * E;
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
    __syncwarp();
    release();  // every lane has its sigma values in registers
    // ---- softmax over the partition's tokens, K and V side by side (Eq. 10)
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
    const float r0 = fx30_to_recip(q0), r1 = fx30_to_recip(q1);
    // ---- Eq. 11, then the order-preserving integer image; padding gets the smallest key
    uint32_t key[E];
    uint32_t kor = 0u, kand = 0xffffffffu;
#pragma unroll
    for (int j = 0; j < E; ++j) {
        const int t = t_lo + j;
        const float sco = combine_scores(x0[j], r0, x1[j], r1);
        key[j] = t < L ? float_key(sco) : 0u;
        if (t < L) {
            kor |= key[j];
            kand &= key[j];
        }
        if (scores_g != nullptr && t < L) scores_g[t] = sco;
    }
    kor = __reduce_or_sync(0xffffffffu, kor);
    kand = __reduce_and_sync(0xffffffffu, kand);
    const uint32_t diff = kor ^ kand;
    const int top = 31 - __clz(diff);  // -1 when every key is the same
    // ---- T = key of the k-th largest score: the largest T with count(key >= T) >= k
    uint32_t T = top >= 0 ? (kand & ~((2u << top) - 1u)) : kand;
    for (int bit = top; bit >= 0; --bit) {
        const uint32_t cand = T | (1u << bit);
        int c = 0;
#pragma unroll
        for (int j = 0; j < E; ++j) c += key[j] >= cand;
        const int tot = __reduce_add_sync(0xffffffffu, c);
        if (tot >= k) T = cand;
        if (tot == k) break;  // exactly the k largest lie at or above T
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
    const int total = __shfl_sync(0xffffffffu, incl, 31);
    const int krem = k - (total & 0xffff);
    const int excl = incl - packed;
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
    __syncwarp();
}

template <class Release>
__device__ __forceinline__ void select_in_warp_dispatch(const float* sg0, const float* sg1, int L, int k,
                                                        float* __restrict__ scores_g, int* kept, int lane,
                                                        Release release) {
    if (L <= 64) select_in_warp<2>(sg0, sg1, L, k, scores_g, kept, lane, release);
    else if (L <= 128) select_in_warp<4>(sg0, sg1, L, k, scores_g, kept, lane, release);
    else if (L <= 256) select_in_warp<8>(sg0, sg1, L, k, scores_g, kept, lane, release);
    else select_in_warp<16>(sg0, sg1, L, k, scores_g, kept, lane, release);  // L <= 512
}

template <class G>
__global__ void __launch_bounds__(G::NT + kPairs * 32, 1) lagkv_pair_kernel(const Params P) {
    static_assert(G::NW == 2 * kPairs, "one K warp and one V warp per pair");
    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    const int NS = P.stages;
    constexpr int STAT_WORDS = G::STAT;  // packed bf16x2 words per min (or max) row
    unsigned char* ring = sm;
    uint64_t* bars = reinterpret_cast<uint64_t*>(ring + smem_ring_bytes<G>(NS));
    uint64_t* xbars = bars + G::NW * NS;  // per pair: full[2], empty[2]
    uint32_t* stats = reinterpret_cast<uint32_t*>(xbars + 4 * kPairs);
    float* sgbase = reinterpret_cast<float*>(stats + G::NW * 2 * STAT_WORDS);
    const int Lp = (P.L + 3) & ~3;
    int* keptbase = reinterpret_cast<int*>(sgbase + kPairs * 4 * Lp);
    volatile int* gave_up = reinterpret_cast<volatile int*>(keptbase + kPairs * Lp);  // [pair]

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int L = P.L, k = P.k, n = P.n, sink = P.sink;
    const int ntiles = (L + G::TR - 1) / G::TR;
    const bool contiguous = (P.ss == G::ROW16);
    const bool streamer = warp < G::NW;
    const int pair = streamer ? (warp >> 1) : (warp - G::NW);

    // Slots [s_first, s_hi) of the global list belong to this pair; a range that starts inside
    // a unit first re-reads the partition above it (statistics only).  Slot s is partition
    // n - 1 - s % n of unit s / n.
    const long long rid = (long long)blockIdx.x * kPairs + pair, nranges = (long long)gridDim.x * kPairs;
    const long long s_first = P.total_slots * rid / nranges;
    const long long s_hi = P.total_slots * (rid + 1) / nranges;
    const bool extra = s_first < s_hi && (s_first % n) != 0;
    const long long s_lo = extra ? s_first - 1 : s_first;

    const uint32_t full_bar = smem_u32(xbars + 4 * pair), empty_bar = full_bar + 16;
    if (streamer && lane == 0)
        for (int i = 0; i < NS; ++i) mbar_init(smem_u32(bars) + uint32_t(warp * NS + i) * 8, 1);
    if (!streamer && lane == 0) {
        for (int b = 0; b < 2; ++b) {
            mbar_init(full_bar + 8 * b, 2);   // the K warp and the V warp
            mbar_init(empty_bar + 8 * b, 1);  // the epilogue warp
        }
        gave_up[pair] = 0;
    }
    fence_mbar_init();
    fence_proxy_async();
    __syncthreads();

    auto unit_base = [&](const uint16_t* base, int u) -> const uint16_t* {
        return base + (long long)(u / P.H) * P.sb + (long long)(u % P.H) * P.sh;
    };
    float* sg_pair = sgbase + pair * 4 * Lp;  // [2 buffers][K, V][Lp]
    bool dead = false;
    // A warp whose wait ran out stops working, raises its pair's flag (the sigma values it owes
    // are incomplete, so the pair's epilogue warp must not select or emit from them any more)
    // and keeps only its arrivals alive.
    auto give_up = [&]() {  // warp-collective
        dead = true;
        if (lane == 0) {
            record_status(P.status, ST_ETIMEOUT, blockIdx.x);
            gave_up[pair] = 1;
        }
    };

    if (streamer) {
        // =============================================================== streaming warps
        const int tensor = warp & 1;
        const int cg = lane % G::LPR, rl = lane / G::LPR;
        const uint16_t* tbase = tensor ? P.V : P.K;
        const uint32_t ring_w = smem_u32(ring) + uint32_t(warp) * NS * G::TILE_BYTES;
        const uint32_t bar_w = smem_u32(bars) + uint32_t(warp) * NS * 8;
        uint32_t* stats_w = stats + warp * 2 * STAT_WORDS;

        // producer cursor: next tile to request, advanced without divisions
        long long pleft = s_hi - s_lo;
        int pu = int(s_lo / n), pp = n - 1 - int(s_lo % n);
        const uint16_t* pbase = unit_base(tbase, pu);
        int pt = 0, pslot = 0;
        auto issue_next = [&]() {  // warp-collective
            if (dead || pleft <= 0) return;
            const int row0 = sink + pp * L + pt * G::TR;
            const int rows = min(G::TR, L - pt * G::TR);
            const uint16_t* src = pbase + (long long)row0 * P.ss;
            const uint32_t dst = ring_w + uint32_t(pslot) * G::TILE_BYTES;
            const uint32_t bar = bar_w + 8 * pslot;
            const uint32_t bytes = uint32_t(rows) * G::ROWB;
            if (lane == 0) {
                fence_proxy_async();
                mbar_arrive_expect_tx(bar, bytes);
            }
            if (contiguous) {
                if (lane == 0) bulk_g2s(dst, src, bytes, bar);
            } else {
                __syncwarp();
                for (int r = lane; r < rows; r += 32)
                    bulk_g2s(dst + uint32_t(r) * G::ROWB, src + (long long)r * P.ss, G::ROWB, bar);
            }
            if (++pt == ntiles) {  // next slot: the partition below, or the top of the next unit
                pt = 0;
                --pleft;
                if (--pp < 0) {
                    pp = n - 1;
                    ++pu;
                    pbase = unit_base(tbase, pu);
                }
            }
            if (++pslot == NS) pslot = 0;
        };
        for (int i = 0; i < NS; ++i) issue_next();

        int cslot = 0;
        uint32_t cparity = 0;
        const float inv_D = 1.0f / float(G::D), inv_Dm = 1.0f / float(G::D - P.ddof);
        f32x2 a2[G::NPW], b2[G::NPW];
#pragma unroll
        for (int j = 0; j < G::NPW; ++j) a2[j] = b2[j] = 0ull;

        int p = n - 1 - int(s_lo % n);
        for (long long s = s_lo; s < s_hi; ++s, p = (p == 0 ? n - 1 : p - 1)) {
            const int i = int(s - s_lo), buf = i & 1;
            const bool score = (p != n - 1) && s >= s_first;
            // the epilogue warp must have released this sigma buffer (slot i - 2)
            if (i >= 2 && !dead && !mbar_wait_bounded(empty_bar + 8 * buf, uint32_t((i >> 1) - 1) & 1u)) give_up();

            uint32_t mn[G::NPW], mx[G::NPW];
#pragma unroll
            for (int j = 0; j < G::NPW; ++j) {
                mn[j] = G::E::kPosInf2;  // +inf, +inf
                mx[j] = G::E::kNegInf2;  // -inf, -inf
            }
            float* sig = sg_pair + (buf * 2 + tensor) * Lp;

            for (int t = 0; t < ntiles; ++t) {
                if (dead) break;
                if (!mbar_wait_bounded(bar_w + 8 * cslot, cparity)) {
                    give_up();
                    break;
                }
                const uint4* tile = reinterpret_cast<const uint4*>(ring + size_t(warp) * NS * G::TILE_BYTES +
                                                                   size_t(cslot) * G::TILE_BYTES);
                const int nrows = min(G::TR, L - t * G::TR);
                float* so = sig + t * G::TR;
                if (nrows == G::TR) {
                    if (score) process_tile<G, true, true>(tile, nrows, a2, b2, mn, mx, so, inv_D, inv_Dm, lane);
                    else process_tile<G, false, true>(tile, nrows, a2, b2, mn, mx, so, inv_D, inv_Dm, lane);
                } else {
                    if (score) process_tile<G, true, false>(tile, nrows, a2, b2, mn, mx, so, inv_D, inv_Dm, lane);
                    else process_tile<G, false, false>(tile, nrows, a2, b2, mn, mx, so, inv_D, inv_Dm, lane);
                }
                __syncwarp();
                issue_next();  // refill the stage just drained
                if (++cslot == NS) {
                    cslot = 0;
                    cparity ^= 1u;
                }
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(full_bar + 8 * buf);  // this tensor's sigma is complete

            // ---- this partition's min / max (Eq. 7, Eq. 8) across the lanes sharing channels,
            //      then the coefficients for the next (lower) partition
#pragma unroll
            for (int j = 0; j < G::NPW; ++j) {
#pragma unroll
                for (int o = G::LPR; o < 32; o <<= 1) {
                    mn[j] = G::E::min2(mn[j], __shfl_xor_sync(0xffffffffu, mn[j], o));
                    mx[j] = G::E::max2(mx[j], __shfl_xor_sync(0xffffffffu, mx[j], o));
                }
            }
            if (rl == 0) {
                store_stats_row<G>(stats_w, mn, mx, cg);
            }
            __syncwarp();
            const int zero_range = make_coefficients<G>(stats_w, 1, cg, a2, b2);
            if (zero_range != 0 && rl == 0 && !dead && P.status != nullptr) atomicAdd(P.status + 2, zero_range);
            __syncwarp();  // the row is rewritten at the end of the next slot
        }
        if (dead) {  // copies may still be in flight towards this CTA's shared memory
            const unsigned long long t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000000ull) { /* bounded drain delay */ }
        }
    } else {
        // ================================================================= epilogue warp
        int* kept = keptbase + pair * Lp;
        for (long long s = s_lo; s < s_hi; ++s) {
            const int i = int(s - s_lo), buf = i & 1;
            const int u = int(s / n), p = n - 1 - int(s % n);
            const bool top = p == n - 1;
            const bool score = !top && s >= s_first;
            if (!dead && !mbar_wait_bounded(full_bar + 8 * buf, uint32_t(i >> 1) & 1u)) give_up();
            // the flag is raised before the arrival that completes the phase waited for above
            if (!dead && __shfl_sync(0xffffffffu, gave_up[pair], 0) != 0) dead = true;
            const uint32_t ebar = empty_bar + 8 * buf;
            const RowMap um = make_rowmap(P, u);
            uint16_t* ok = P.K_out ? P.K_out + (long long)u * P.L_R * G::ROW16 : nullptr;
            uint16_t* ov = P.V_out ? P.V_out + (long long)u * P.L_R * G::ROW16 : nullptr;
            int32_t* oi = P.idx_out ? P.idx_out + (long long)u * P.L_R : nullptr;
            if (score && !dead) {
                const float* sg0 = sg_pair + (buf * 2) * Lp;
                float* scores_g = P.scores_out ? P.scores_out + ((long long)u * (n - 1) + p) * L : nullptr;
                select_in_warp_dispatch(sg0, sg0 + Lp, L, k, scores_g, kept, lane, [&] {
                    if (lane == 0) mbar_arrive(ebar);  // the sigma buffer goes back to the streamers
                });
                emit_kept<32, G::VPR, 8>(P.K, P.V, um, ok, ov, sink + p * L, sink + p * k, kept, k, oi, lane);
                __syncwarp();  // kept[] is rewritten by the next selection
            } else if (lane == 0) {
                mbar_arrive(ebar);
            }
            // rows copied verbatim: the window with the unit's top slot, the sink with slot p = 0
            if (s >= s_first && !dead) {
                if (top) copy_rows<32, G::VPR>(P.K, P.V, um, ok, ov, sink + (n - 1) * L, sink + (n - 1) * k, L + P.rem, oi, lane);
                if (p == 0) copy_rows<32, G::VPR>(P.K, P.V, um, ok, ov, 0, 0, sink, oi, lane);
            }
        }
    }
}

}  // namespace lagkv
