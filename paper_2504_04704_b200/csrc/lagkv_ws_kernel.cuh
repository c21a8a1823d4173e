// LagKV prefill compress pass -- warp-specialised persistent kernel for sm_100a.
//
// Same slot walk as lagkv_stream_kernel (for LagKV: partitions of a unit in DESCENDING p, so
// the statistics of partition p+1, Eq. 7 / Eq. 8, are at hand when p streams through; the
// LocalKV and L2-norm variants of Section 4.3 have their own slot lists, see below), but the
// CTA is split into three roles so that the streaming never stops:
//
//   * NW streaming warps (even: K, odd: V).  Each owns a ring of shared-memory tiles
//     filled by bulk async copies, normalises and accumulates the per-token moments
//     (Eq. 9, Eq. 10) and the partition's own min / max, writes sigma into one of two
//     sigma buffers and hands the slot over through an mbarrier.  The warps of one
//     tensor meet once per partition on a named barrier to combine their min / max.
//   * 3 select warps: softmax over the partition, K + V (Eq. 11) and top-k with ties to
//     the lower index -- one partition behind the streamers, overlapped with them.  They
//     publish where the kept rows come from and move the rows of every second partition
//     themselves; the others are moved by the copy warp or, what it has not claimed by the
//     end, in the gather phase.
//   * 1 copy warp: moves rows global -> shared -> global with bulk async copies: the kept
//     rows of partitions whose positions are published (bandwidth the streamers leave
//     unused), and the rows that are kept verbatim (sink and sliding window) of ALL units,
//     cut into chunks dealt round-robin to the CTAs.
//
// When a CTA has walked all its slots, all of its warps together copy the kept rows the
// copy warp has not claimed (gather phase).
//
// Every wait on an mbarrier is bounded; a warp whose wait ran out raises the CTA's abort
// flag, records LAGKV_ETIMEOUT and from then on only keeps the barrier protocol alive so
// that no other warp blocks.
#pragma once
#include "lagkv_kernels.cuh"

namespace lagkv {

constexpr int kWsEpiWarps = 4;      // 3 select warps + 1 copy warp
constexpr int kWsSelThreads = 96;
constexpr int kWsCopyRows = 32;     // rows per staged chunk of the copy warp
constexpr int kBarTensor = 1;       // named barriers 1, 2: streaming warps of K, of V
constexpr int kBarSelect = 3;       // named barrier 3: the select warps

template <class G>
__host__ __device__ inline size_t ws_smem_total_bytes(int stages, int L) {
    size_t s = smem_ring_bytes<G>(stages);                  // tile rings
    s += size_t(2) * 2 * kWsCopyRows * G::ROWB;            // copy staging [2 stages][K, V]
    s += (size_t(G::NW) * stages + 6) * 8;                  // mbarriers
    s += size_t(2) * 2 * G::WT * 2 * G::STAT * 4;        // min/max partials [2][K,V][WT][mn,mx]
    s += sizeof(SelScratch);
    s = (s + 15) & ~size_t(15);
    s += size_t(2) * 2 * ((L + 3) & ~3) * 4;                // sigma [2 buffers][K, V]
    s += size_t((L + 3) & ~3) * 4;                          // kept indices of one partition
    return s + 128;                                         // alignment slack
}

// VAR: 0 = LagKV, 1 = LocalKV, 2 = L2 norm (enum lagkv_variant), compiled apart so that the
// LagKV kernel carries none of the other variants' code.  PAGED: the caches are pools of pages
// behind a block table (every row address goes through RowMap; a tile that straddles a page
// boundary takes two copies); compiled apart too, so that the kernel for contiguous caches keeps
// its plain pointer arithmetic and its registers.
template <class G, int VAR, bool PAGED = false>
__global__ void __launch_bounds__(G::NT + kWsEpiWarps * 32, 1) lagkv_ws_kernel(const Params P) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    const int NS = P.stages;
    constexpr int CHUNK_BYTES = kWsCopyRows * G::ROWB;     // one tensor, one staged chunk
    unsigned char* ring = sm;
    unsigned char* stage = ring + smem_ring_bytes<G>(NS);
    uint64_t* bars = reinterpret_cast<uint64_t*>(stage + 4 * CHUNK_BYTES);
    uint64_t* xbars = bars + G::NW * NS;                    // full[2], empty[2], copy[2]
    uint32_t* stats = reinterpret_cast<uint32_t*>(xbars + 6);
    constexpr int STAT_WORDS = G::STAT;                    // packed bf16x2 words per min (or max) row
    SelScratch& sc = *reinterpret_cast<SelScratch*>(stats + 2 * 2 * G::WT * 2 * STAT_WORDS);
    float* sgbase = reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(&sc + 1) + 15) & ~uintptr_t(15));
    const int Lp = (P.L + 3) & ~3;
    int* kept = reinterpret_cast<int*>(sgbase + 4 * Lp);

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int L = P.L, k = P.k, n = P.n, sink = P.sink;
    const int ntiles = (L + G::TR - 1) / G::TR;
    const bool contiguous = (P.ss == G::ROW16);

    // slots [s_first, s_hi) belong to this CTA; a range that starts inside a unit first
    // re-reads the partition above it (statistics only)
    const long long s_first = P.total_slots * blockIdx.x / gridDim.x;
    const long long s_hi = P.total_slots * (blockIdx.x + 1) / gridDim.x;
    // Slot j of a unit.  LagKV (Eq. 7-9): partitions n-1 ... 0, each scored with the statistics
    // of the slot before it.  LocalKV (Eq. 14, Eq. 15): partitions n-2 ... 0, each visited
    // twice in a row, once for its own statistics and once to be scored with them.
    // L2 norm (Eq. 16): partitions n-2 ... 0, each scored on its own from K alone.
    const int spu = P.spu;
    constexpr bool local_stats = VAR == 1, l2norm = VAR == 2;
    auto slot_part = [&](int j) -> int { return local_stats ? n - 2 - (j >> 1) : (l2norm ? n - 2 - j : n - 1 - j); };
    auto slot_scored = [&](int j) -> bool { return local_stats ? (j & 1) != 0 : (l2norm || j != 0); };
    auto slot_needs_prev = [&](int j) -> bool { return !l2norm && slot_scored(j); };
    // Slots (counted from the first one this CTA streams) whose kept rows the select warps move
    // themselves: every second one where the host found that they have the time (P.sel_emit).
    const bool sel_emit = P.sel_emit != 0;
    auto sel_moves = [&](long long i) -> bool { return sel_emit && (i & 1) != 0; };
    const bool extra = s_first < s_hi && slot_needs_prev(int(s_first % spu));
    const long long s_lo = extra ? s_first - 1 : s_first;

    const uint32_t full_bar = smem_u32(xbars), empty_bar = smem_u32(xbars + 2), copy_bar = smem_u32(xbars + 4);
    if (warp < G::NW && lane == 0)
        for (int i = 0; i < NS; ++i) mbar_init(smem_u32(bars) + uint32_t(warp * NS + i) * 8, 1);
    if (tid == 0) {
        for (int b = 0; b < 2; ++b) {
            mbar_init(full_bar + 8 * b, G::NW);
            mbar_init(empty_bar + 8 * b, 1);
            mbar_init(copy_bar + 8 * b, 1);
        }
        sc.abort = 0;
        sc.sel_done = 0;
        sc.claimed = 0;
    }
    fence_mbar_init();
    fence_proxy_async();
    __syncthreads();

    volatile int* abort_flag = reinterpret_cast<volatile int*>(&sc.abort);
    auto raise_abort = [&]() {  // warp-collective
        if (lane == 0) {
            record_status(P.status, ST_ETIMEOUT, blockIdx.x);
            *abort_flag = 1;
        }
    };
    auto unit_base = [&](const uint16_t* base, int u) -> const uint16_t* {
        return base + (long long)(u / P.H) * P.sb + (long long)(u % P.H) * P.sh;
    };

    if (warp < G::NW) {
        // =============================================================== streaming warps
        // even warps stream K, odd warps V; the L2-norm variant reads K only and puts every warp on it
        constexpr int WTE = l2norm ? G::NW : G::WT;  // warps that share a tensor's tiles
        const int tensor = l2norm ? 0 : (warp & 1), wj = l2norm ? warp : (warp >> 1);
        const int cg = lane % G::LPR, rl = lane / G::LPR;
        const uint16_t* tbase = tensor ? P.V : P.K;
        const uint32_t ring_w = smem_u32(ring) + uint32_t(warp) * NS * G::TILE_BYTES;
        const uint32_t bar_w = smem_u32(bars) + uint32_t(warp) * NS * 8;
        bool dead = false;

        const bool has_tiles = wj < ntiles;
        // producer cursor: next tile to request, kept as (slots left, unit, partition, tile)
        // and advanced without divisions
        long long pleft = s_hi - s_lo;
        int pu = int(s_lo / spu), pj = int(s_lo % spu);
        const uint16_t* pbase = unit_base(tbase, pu);
        RowMap pmap;  // PAGED only
        if (PAGED) pmap = make_rowmap(P, pu);
        int pt = wj, pslot = 0;
        auto issue_next = [&]() {  // warp-collective
            if (dead || !has_tiles || pleft <= 0) return;
            const int row0 = sink + slot_part(pj) * L + pt * G::TR;
            const int rows = min(G::TR, L - pt * G::TR);
            const uint32_t dst = ring_w + uint32_t(pslot) * G::TILE_BYTES;
            const uint32_t bar = bar_w + 8 * pslot;
            const uint32_t bytes = uint32_t(rows) * G::ROWB;
            if (lane == 0) {
                fence_proxy_async();
                mbar_arrive_expect_tx(bar, bytes);
            }
            if (PAGED) {
                fetch_rows(tbase, pmap, row0, rows, dst, bar, G::ROWB, contiguous, lane);
            } else {
                const uint16_t* src = pbase + (long long)row0 * P.ss;
                if (contiguous) {
                    if (lane == 0) bulk_g2s(dst, src, bytes, bar);
                } else {
                    __syncwarp();
                    for (int r = lane; r < rows; r += 32)
                        bulk_g2s(dst + uint32_t(r) * G::ROWB, src + (long long)r * P.ss, G::ROWB, bar);
                }
            }
            pt += WTE;
            if (pt >= ntiles) {  // next slot of this unit, or the first slot of the next unit
                pt = wj;
                --pleft;
                if (++pj == spu) {
                    pj = 0;
                    ++pu;
                    if (PAGED) pmap = make_rowmap(P, pu);
                    else pbase = unit_base(tbase, pu);
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

        int cj = int(s_lo % spu);
        for (long long s = s_lo; s < s_hi; ++s, cj = (cj + 1 == spu ? 0 : cj + 1)) {
            const int i = int(s - s_lo), buf = i & 1;
            const bool score = slot_scored(cj) && s >= s_first;
            dead = __any_sync(0xffffffffu, dead || *abort_flag != 0);
            // the select warps must have released this sigma buffer (slot i - 2)
            if (i >= 2 && !dead && !mbar_wait_bounded(empty_bar + 8 * buf, uint32_t((i >> 1) - 1) & 1u)) {
                dead = true;
                raise_abort();
            }

            uint32_t mn[G::NPW], mx[G::NPW];
#pragma unroll
            for (int j = 0; j < G::NPW; ++j) {
                mn[j] = G::E::kPosInf2;  // +inf, +inf
                mx[j] = G::E::kNegInf2;  // -inf, -inf
            }
            float* sig = sgbase + (buf * 2 + tensor) * Lp;

            for (int t = wj; has_tiles && t < ntiles; t += WTE) {
                if (dead) break;
                if (!mbar_wait_bounded(bar_w + 8 * cslot, cparity)) {
                    dead = true;
                    raise_abort();
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
            uint32_t* stats_t = stats + ((buf * 2 + tensor) * G::WT) * 2 * STAT_WORDS;
            if (rl == 0) {
                store_stats_row<G>(stats_t + wj * 2 * STAT_WORDS, mn, mx, cg);
            }
            named_bar_sync(kBarTensor + tensor, WTE * 32);
            // sigma of this tensor is complete: hand the slot to the select warps
            if (lane == 0) mbar_arrive(full_bar + 8 * buf);

            // ---- coefficients for the next (lower) partition from this one's statistics
            {
                const int zero_range = make_coefficients<G>(stats_t, G::WT, cg, a2, b2);
                if (zero_range != 0 && wj == 0 && rl == 0 && !dead && !l2norm && P.status != nullptr)
                    atomicAdd(P.status + 2, zero_range);
            }
        }
        if (dead) {  // copies may still be in flight towards this CTA's shared memory
            const unsigned long long t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000000ull) { /* bounded drain delay */ }
        }
    } else if (warp < G::NW + 3) {
        // ================================================================== select warps
        const int etid = tid - G::NT;
        bool dead = false;
        auto sync_sel = [] { named_bar_sync(kBarSelect, kWsSelThreads); };
        for (long long s = s_lo; s < s_hi; ++s) {
            const int i = int(s - s_lo), buf = i & 1;
            const int u = int(s / spu), sj = int(s % spu), p = slot_part(sj);
            const bool score = slot_scored(sj) && s >= s_first;
            bool bad = __any_sync(0xffffffffu, dead || *abort_flag != 0);
            if (!bad && !mbar_wait_bounded(full_bar + 8 * buf, uint32_t(i >> 1) & 1u)) {
                bad = true;
                raise_abort();
            }
            dead = named_bar_or(kBarSelect, kWsSelThreads, bad);  // one decision for the group
            if (score && !dead) {
                float* sg0 = sgbase + (buf * 2) * Lp;
                float* sg1 = sg0 + Lp;
                float* scores_g = P.scores_out ? P.scores_out + ((long long)u * (n - 1) + p) * L : nullptr;
                const uint32_t ebar = empty_bar + 8 * buf;
                // the sigma buffer goes back to the streamers as soon as the selector has
                // taken its values (called after a group barrier; one arrival is expected)
                score_and_select<kWsSelThreads>(sg0, sg1, L, k, !l2norm, scores_g, kept, sc, etid, sync_sel, [&] {
                    if (etid == 0) mbar_arrive(ebar);
                });
                // where the kept rows come from: in idx_out when the caller wants it, else (even
                // slots only, whose rows the copy warp or the gather phase move later) in the
                // first word of each destination row of K_out
                {
                    const long long o = (long long)u * P.L_R + sink + p * k;
                    const int row0 = sink + p * L;
                    if (P.idx_out != nullptr) {
                        for (int j = etid; j < k; j += kWsSelThreads) P.idx_out[o + j] = row0 + kept[j];
                    } else if (P.K_out != nullptr && !sel_moves(i)) {
                        for (int j = etid; j < k; j += kWsSelThreads)
                            *reinterpret_cast<int32_t*>(P.K_out + (o + j) * G::ROW16) = row0 + kept[j];
                    }
                }
                // Long partitions: the select warps, idle most of the time, move the kept rows of
                // odd slots themselves while kept[] is at hand (the others are left to the copy
                // warp and the gather phase).  Every second slot is what they can carry without
                // holding up the streamers; with short partitions they have no time to spare.
                if (sel_moves(i) && P.K_out != nullptr)
                    emit_kept<kWsSelThreads, G::VPR, 16>(P.K, P.V, make_rowmap(P, u),
                                                         P.K_out + (long long)u * P.L_R * G::ROW16,
                                                         P.V_out + (long long)u * P.L_R * G::ROW16, sink + p * L,
                                                         sink + p * k, kept, k, nullptr, etid);
                __threadfence_block();  // the positions above are visible before the count below
                sync_sel();             // every thread is done with kept[] and has written its share
            } else if (etid == 0) {
                mbar_arrive(empty_bar + 8 * buf);
            }
            if (etid == 0) *reinterpret_cast<volatile int*>(&sc.sel_done) = i + 1;  // slot i is published
        }
    } else {
        // ===================================================================== copy warp
        // Two kinds of 32-row chunks go through the same two-stage pipeline (bulk loads into
        // shared memory, one bulk store per tensor out of it):
        //   * gather chunks: kept rows of this CTA's partitions, as soon as the select warps
        //     have published their positions (row by row loads, contiguous store).  While
        //     the streamers leave bandwidth unused this moves most kept rows for free;
        //     what is not claimed when the last slot is published is left to the gather
        //     phase of the whole CTA;
        //   * verbatim chunks: sink and window rows of ALL units, dealt round-robin over the
        //     CTAs (chunk g belongs to CTA g mod gridDim.x): per unit first the window
        //     chunks, then the sink chunks.
        const int win_rows = L + P.rem;
        const int cw = (win_rows + kWsCopyRows - 1) / kWsCopyRows, cs = (sink + kWsCopyRows - 1) / kWsCopyRows;
        const long long U = (long long)P.B * P.H;
        const long long total_chunks = U * (cw + cs);
        const bool rows_wanted = P.K_out != nullptr;
        const uint32_t stage_u32 = smem_u32(stage);
        const int nslots = int(s_hi - s_lo);
        volatile int* sel_done = reinterpret_cast<volatile int*>(&sc.sel_done);
        long long vg = blockIdx.x;          // next verbatim chunk of this CTA
        int gslot = 0, gbatch = 0;          // gather cursor: slot index, batch inside it
        bool gclaimed = false;
        int nload = 0;                      // chunks loaded so far (stage = nload & 1)
        bool pending = false, dead = false;
        long long po = 0;                   // pending chunk: first destination row (global row index)
        int pnr = 0;
        for (;;) {
            if (__any_sync(0xffffffffu, *abort_flag != 0)) dead = true;
            // ---- pick the next chunk: a gather chunk if one is ready, else a verbatim chunk
            int kind = 0;  // 0 none, 1 verbatim, 2 gather
            int u = 0, src = 0, nr = 0;
            long long o = 0;  // first destination row: u * L_R + row
            const int done = *sel_done;
            if (rows_wanted && !dead) {
                if (!gclaimed) {
                    // skip slots without kept rows (top partitions, the statistics-only extra slot)
                    // and the odd slots, whose rows the select warps move
                    while (gslot < nslots) {
                        const long long sl = s_lo + gslot;
                        if (slot_scored(int(sl % spu)) && sl >= s_first && !sel_moves(gslot)) break;
                        ++gslot;
                    }
                    if (gslot < done && done < nslots) {
                        gclaimed = true;
                        gbatch = 0;
                        if (lane == 0) *reinterpret_cast<volatile int*>(&sc.claimed) = gslot + 1;
                    }
                }
                if (gclaimed) {
                    const long long sl = s_lo + gslot;
                    const int p = slot_part(int(sl % spu));
                    u = int(sl / spu);
                    nr = min(kWsCopyRows, k - gbatch * kWsCopyRows);
                    o = (long long)u * P.L_R + sink + p * k + gbatch * kWsCopyRows;
                    kind = 2;
                    if ((++gbatch) * kWsCopyRows >= k) {
                        gclaimed = false;
                        ++gslot;
                    }
                }
            }
            if (kind == 0 && vg < total_chunks && !dead) {
                u = int(vg / (cw + cs));
                const int j = int(vg % (cw + cs));
                int dst;
                if (j < cw) {
                    src = sink + (n - 1) * L + j * kWsCopyRows;
                    dst = sink + (n - 1) * k + j * kWsCopyRows;
                    nr = min(kWsCopyRows, win_rows - j * kWsCopyRows);
                } else {
                    src = dst = (j - cw) * kWsCopyRows;
                    nr = min(kWsCopyRows, sink - (j - cw) * kWsCopyRows);
                }
                o = (long long)u * P.L_R + dst;
                if (P.idx_out != nullptr)
                    for (int r = lane; r < nr; r += 32) P.idx_out[o + r] = src + r;
                kind = 1;
                vg += gridDim.x;
            }
            const bool more = !dead && (vg < total_chunks || (rows_wanted && done < nslots));
            if (kind == 0 && !pending) {
                if (!more) break;
                __nanosleep(500);  // nothing to do right now: the select warps are still at work
                continue;
            }
            const bool load = kind != 0 && rows_wanted;
            if (load) {
                const int st = nload & 1;
                // this stage was last read by the store committed two loads ago
                if (lane == 0) {
                    bulk_wait_read_all();
                    fence_proxy_async();
                    mbar_arrive_expect_tx(copy_bar + 8 * st, uint32_t(2 * nr) * G::ROWB);
                }
                __syncwarp();
                const uint32_t dK = stage_u32 + uint32_t(2 * st) * CHUNK_BYTES, dV = dK + CHUNK_BYTES;
                // where the unit's rows are: an offset from the tensor's base pointer
                RowMap um;
                if (PAGED) {
                    um = make_rowmap(P, u);
                } else {
                    um.pages = nullptr;
                    um.ss = P.ss;
                    um.base = (long long)(u / P.H) * P.sb + (long long)(u % P.H) * P.sh;
                }
                if (kind == 1 && contiguous) {
                    if (PAGED) {
                        fetch_rows(P.K, um, src, nr, dK, copy_bar + 8 * st, G::ROWB, true, lane);
                        fetch_rows(P.V, um, src, nr, dV, copy_bar + 8 * st, G::ROWB, true, lane);
                    } else if (lane == 0) {
                        bulk_g2s(dK, P.K + um.base + (long long)src * P.ss, uint32_t(nr) * G::ROWB, copy_bar + 8 * st);
                        bulk_g2s(dV, P.V + um.base + (long long)src * P.ss, uint32_t(nr) * G::ROWB, copy_bar + 8 * st);
                    }
                } else if (lane < nr) {  // one row of K and of V per lane
                    int row = src + lane;
                    if (kind == 2) {
                        __threadfence_block();
                        row = P.idx_out != nullptr ? __ldcg(P.idx_out + o + lane)
                                                   : __ldcg(reinterpret_cast<const int32_t*>(P.K_out + (o + lane) * G::ROW16));
                    }
                    const long long ro = um.off(row);
                    bulk_g2s(dK + uint32_t(lane) * G::ROWB, P.K + ro, G::ROWB, copy_bar + 8 * st);
                    bulk_g2s(dV + uint32_t(lane) * G::ROWB, P.V + ro, G::ROWB, copy_bar + 8 * st);
                }
            }
            if (pending) {  // the chunk loaded before this one goes out
                const int pl = nload - 1;  // nload still names the chunk loaded above, if any
                const int pst = pl & 1;
                if (!mbar_wait_bounded(copy_bar + 8 * pst, uint32_t(pl >> 1) & 1u)) {
                    dead = true;
                    raise_abort();
                } else if (lane == 0) {
                    fence_proxy_async();
                    const uint32_t sK = stage_u32 + uint32_t(2 * pst) * CHUNK_BYTES, sV = sK + CHUNK_BYTES;
                    bulk_s2g(P.K_out + po * G::ROW16, sK, uint32_t(pnr) * G::ROWB);
                    bulk_s2g(P.V_out + po * G::ROW16, sV, uint32_t(pnr) * G::ROWB);
                    bulk_commit();
                }
            }
            pending = load;
            po = o;
            pnr = nr;
            if (load) ++nload;
        }
        if (lane == 0) bulk_wait_read_all();
        if (dead) {
            const unsigned long long t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000000ull) { /* bounded drain delay */ }
        }
    }

    // ================================================================== gather phase
    // Every warp of the CTA now moves the kept rows of the CTA's own partitions.  Doing it
    // here, with the whole CTA and many loads in flight per thread, instead of partition
    // by partition beside the streamers, keeps the gather off the latency of a saturated
    // memory system.
    __syncthreads();
    if (P.K_out != nullptr && *abort_flag == 0) {
        constexpr int NWALL = G::NW + kWsEpiWarps;
        // A kept row is 2 * VPR 16-byte vectors (K, then V).  A warp always moves WHOLE rows, GR at
        // a time (the smallest count whose vectors fill the 32 lanes evenly, IPL per lane), UG
        // such groups per pass so that 6-8 loads are in flight per lane.  Without idx_out the
        // position of a kept row is parked in the first word of its K_out row: because the warp
        // that reads that word is the only one that ever writes the row, reading all positions
        // of a pass before its first store (warp barrier below) is enough for every head_dim.
        constexpr int RV = 2 * G::VPR;
        constexpr int GR = (RV % 32 == 0) ? 1 : ((RV % 16 == 0) ? 2 : 4);
        constexpr int IPL = GR * RV / 32;
        constexpr int UG = IPL == 1 ? 8 : (IPL == 2 ? 4 : 2);
        static_assert((GR * RV) % 32 == 0 && IPL * 32 == GR * RV, "a row group must fill the warp evenly");
        const int ngroups = (k + GR - 1) / GR;
        // slots the copy warp claimed are done; the rest (at least the last one) is moved here
        const long long s_from = s_lo + *reinterpret_cast<volatile int*>(&sc.claimed);
        for (long long s = (s_from > s_first ? s_from : s_first); s < s_hi; ++s) {
            const int u = int(s / spu), sj = int(s % spu), p = slot_part(sj);
            if (!slot_scored(sj) || sel_moves(s - s_lo)) continue;  // done by the select warps
            const uint16_t* srcK = PAGED ? P.K : unit_base(P.K, u);
            const uint16_t* srcV = PAGED ? P.V : unit_base(P.V, u);
            RowMap um;  // PAGED only
            if (PAGED) um = make_rowmap(P, u);
            const long long o = (long long)u * P.L_R + sink + p * k;
            uint16_t* dstK = P.K_out + o * G::ROW16;
            uint16_t* dstV = P.V_out + o * G::ROW16;
            for (int g0 = warp; g0 < ngroups; g0 += NWALL * UG) {
                int src[UG][IPL];
                uint4 buf[UG][IPL];
#pragma unroll
                for (int q = 0; q < UG; ++q)
#pragma unroll
                    for (int e = 0; e < IPL; ++e) {
                        const int j = (g0 + q * NWALL) * GR + (e * 32 + lane) / RV;
                        src[q][e] = -1;
                        if (g0 + q * NWALL < ngroups && j < k)
                            src[q][e] = P.idx_out != nullptr
                                            ? __ldcg(P.idx_out + o + j)
                                            : __ldcg(reinterpret_cast<const int32_t*>(dstK + (long long)j * G::ROW16));
                    }
                __syncwarp();  // every parked position of this pass is read before a row is overwritten
#pragma unroll
                for (int q = 0; q < UG; ++q)
#pragma unroll
                    for (int e = 0; e < IPL; ++e)
                        if (src[q][e] >= 0) {
                            const int va = (e * 32 + lane) % RV;
                            const uint16_t* sp = va >= G::VPR ? srcV : srcK;
                            const long long ro = PAGED ? um.off(src[q][e]) : (long long)src[q][e] * P.ss;
                            buf[q][e] = ld_nc(reinterpret_cast<const uint4*>(sp + ro) + (va % G::VPR));
                        }
#pragma unroll
                for (int q = 0; q < UG; ++q)
#pragma unroll
                    for (int e = 0; e < IPL; ++e)
                        if (src[q][e] >= 0) {
                            const int va = (e * 32 + lane) % RV;
                            const int j = (g0 + q * NWALL) * GR + (e * 32 + lane) / RV;
                            uint16_t* dp = va >= G::VPR ? dstV : dstK;
                            st_stream(reinterpret_cast<uint4*>(dp + (long long)j * G::ROW16) + (va % G::VPR), buf[q][e]);
                        }
            }
        }
    }
}

}  // namespace lagkv
