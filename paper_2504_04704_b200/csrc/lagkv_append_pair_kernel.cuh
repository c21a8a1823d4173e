// LagKV incremental pass for decode (Section 2.2, bullets 2-4; Fig. 1) -- one partition per call,
// a thread-block cluster per (sequence, KV head) unit, for sm_100a.
//
// When a sequence triggers during decode exactly 2L rows (plus a remainder) lie behind its
// static part: partition P0, which is scored and cut down to k rows, and partition P1, whose
// per-channel min / max (Eq. 7, Eq. 8) normalise P0 (Eq. 9) and which then becomes the sliding
// window.  P1 is therefore needed twice: for its statistics, and to be moved down by L - k rows.
// The uniform kernel reads it from DRAM both times.  Here a cluster of 2 * RS CTAs shares the
// unit -- by TENSOR (even ranks: K, odd ranks: V) and, within a tensor, by tiles dealt round
// robin over RS row splits -- so that every CTA is small enough to keep its share of P1 in
// shared memory between the two uses while two or more CTAs of different units still fit an SM
// (their latency-bound phases then overlap each other's copies):
//
//   1. every tile of the CTA's share of P1 is fetched by a bulk async copy straight into a
//      resident buffer, all copies in flight from the first instruction; the warps fold
//      min / max as tiles land; the row splits of a tensor exchange their min / max rows
//      through distributed shared memory;
//   2. the CTA's tiles of P0 stream through the per-warp rings: sigma of Eq. 10 per token;
//   3. every CTA sends its sigma values to all others (plain remote stores, one cluster
//      barrier) and all run the same softmax, K + V sum (Eq. 11) and top-k: bit-identical, so
//      nobody has to send anybody the picks;
//   4. the kept rows of a tensor are split over its row splits: each gathers its share from
//      global memory into the (now idle) rings; after a cluster barrier -- every source row
//      has been read -- the shares are stored behind the static part and every CTA writes its
//      resident tiles of the window to their new place; the rows behind the window (the
//      remainder) are moved by split 0 with staged copies.
//
// With RS = 1 (a pair of CTAs) the resident buffer may hold only a part of P1; the rest then
// goes through the rings and is read a second time for the move.
// No multicast of any kind.  Every mbarrier wait is bounded; the cluster barriers are reached by
// all CTAs on every path once the (identical) decision to work has been taken.
#pragma once
#include "lagkv_kernels.cuh"

namespace lagkv {

__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t cluster_nctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_nctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ void cluster_arrive() { asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory"); }
__device__ __forceinline__ void cluster_wait() { asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory"); }
// address of the same shared-memory location in another CTA of the cluster
__device__ __forceinline__ uint32_t map_to_cta(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void st_cluster_u32(uint32_t addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(addr), "r"(v) : "memory");
}

constexpr int kAppendMaxSplits = 4;  // row splits per tensor: clusters of 2, 4 or 8 CTAs

// Shared memory without the resident buffer; every resident tile adds TILE_BYTES + 8.
template <class G>
__host__ __device__ inline size_t append_pair_smem_fixed(int stages, int L) {
    size_t s = smem_ring_bytes<G>(stages);              // tile rings (also the staging of the moves)
    s += (size_t(G::NW) * stages + 3) * 8 + 16;         // mbarriers: rings, two for the staged moves, one for the
                                                        // gather (+ those of the resident tiles), padded to 16 bytes
    s += size_t(G::NW) * 2 * G::STAT * 4;            // min / max partials, one row per warp
    s += size_t(kAppendMaxSplits) * 2 * G::STAT * 4; // min / max rows of the row splits
    s += sizeof(SelScratch);
    s = (s + 15) & ~size_t(15);
    s += size_t(2) * ((L + 3) & ~3) * 4;                // sigma of K and of V
    return s + 160;                                     // alignment slack (base to 128, two paddings to 16)
}

// Rows [dst_row0, dst_row0 + total) of one tensor <- rows src(j), j ascending, through two
// stages of R rows each in shared memory (the load of chunk c + 1 is in flight while chunk c is
// stored).  The caller guarantees src(j) >= dst_row0 + j and ascending sources, so that a chunk
// never overwrites what a later chunk still has to read.  `chunk0` continues the stage / parity
// sequence of the two barriers across calls and is advanced.  Returns false on a timed-out wait.
template <class G, class Src>
__device__ bool move_rows_staged(uint16_t* X, long long ss, int dst_row0, int total, Src src, bool src_contiguous,
                                 uint32_t stage0, int R, uint32_t bar0, int& chunk0, int lane) {
    constexpr uint32_t ROWB = G::ROWB;
    const bool contiguous = ss == G::ROW16;
    const int nchunks = (total + R - 1) / R;
    auto load = [&](int c) {
        const int j0 = c * R, nr = min(R, total - j0), g = chunk0 + c;
        const uint32_t dX = stage0 + uint32_t(g & 1) * uint32_t(R) * ROWB, bar = bar0 + 8 * (g & 1);
        if (lane == 0) {
            fence_proxy_async();
            mbar_arrive_expect_tx(bar, uint32_t(nr) * ROWB);
        }
        __syncwarp();
        if (contiguous && src_contiguous) {
            if (lane == 0) bulk_g2s(dX, X + (long long)src(j0) * ss, uint32_t(nr) * ROWB, bar);
        } else {
            for (int r = lane; r < nr; r += 32) bulk_g2s(dX + uint32_t(r) * ROWB, X + (long long)src(j0 + r) * ss, ROWB, bar);
        }
    };
    auto store = [&](int c) -> bool {
        const int j0 = c * R, nr = min(R, total - j0), g = chunk0 + c;
        const uint32_t sX = stage0 + uint32_t(g & 1) * uint32_t(R) * ROWB;
        if (!mbar_wait_bounded(bar0 + 8 * (g & 1), uint32_t(g >> 1) & 1u)) return false;
        if (contiguous) {
            if (lane == 0) bulk_s2g(X + (long long)(dst_row0 + j0) * ss, sX, uint32_t(nr) * ROWB);
        } else {
            for (int r = lane; r < nr; r += 32)
                bulk_s2g(X + (long long)(dst_row0 + j0 + r) * ss, sX + uint32_t(r) * ROWB, ROWB);
        }
        bulk_commit();  // every lane closes a group (empty for the lanes that stored nothing)
        return true;
    };
    bool ok = true;
    for (int c = 0; c < nchunks && ok; ++c) {
        if (c >= 2) {  // this stage was last read by the store of chunk c - 2
            bulk_wait_read_all();
            __syncwarp();
        }
        load(c);
        if (c >= 1) ok = store(c - 1);
    }
    if (ok && nchunks > 0) ok = store(nchunks - 1);
    bulk_wait_read_all();  // the stages are free again for the next call
    __syncwarp();
    if (ok) chunk0 += nchunks;
    return ok;
}

// Two resident CTAs per SM are the point of the row splits: registers capped for that.
template <class G>
__global__ void __launch_bounds__(G::NT, (G::NW <= 4 ? 2 : 1)) lagkv_append_pair_kernel(const Params P) {
    extern __shared__ unsigned char smem_raw[];
    unsigned char* sm = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~uintptr_t(127));
    constexpr uint32_t ROWB = G::ROWB;
    constexpr int STAT = G::STAT;      // packed words per min (or max) row
    const int NS = P.stages;
    const int res_tiles = P.res_tiles;  // room for that many resident tiles (the same in every CTA)
    unsigned char* ring = sm;
    unsigned char* res = ring + smem_ring_bytes<G>(NS);
    uint64_t* bars = reinterpret_cast<uint64_t*>(res + size_t(res_tiles) * G::TILE_BYTES);
    uint64_t* move_bars = bars + G::NW * NS;
    uint64_t* tile_bars = move_bars + 3;
    // [NW][mn | mx][D/2], read with 16-byte loads: the barrier count before it may be odd
    uint32_t* stats = reinterpret_cast<uint32_t*>((reinterpret_cast<uintptr_t>(tile_bars + res_tiles) + 15) & ~uintptr_t(15));
    uint32_t* xstats = stats + G::NW * 2 * STAT;                           // [splits][mn | mx][D/2]
    SelScratch& sc = *reinterpret_cast<SelScratch*>(xstats + kAppendMaxSplits * 2 * STAT);
    float* sg = reinterpret_cast<float*>((reinterpret_cast<uintptr_t>(&sc + 1) + 15) & ~uintptr_t(15));
    const int Lp = (P.L + 3) & ~3;
    float* sg0 = sg;       // sigma of K
    float* sg1 = sg + Lp;  // sigma of V

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int cg = lane % G::LPR, rl = lane / G::LPR;
    const int L = P.L, k = P.k;
    const int ntiles = (L + G::TR - 1) / G::TR;
    const bool contiguous = (P.ss == G::ROW16);
    const uint32_t rank = cluster_ctarank(), CS = cluster_nctarank();
    const int tensor = int(rank & 1u);           // 0: this CTA handles K, 1: V
    const int RS = int(CS >> 1), h = int(rank >> 1);  // row splits per tensor, this CTA's split
    const int u = int(blockIdx.x / CS), b = u / P.H;

    // ---- what is there to do?  All CTAs of the cluster read the same two integers and decide alike.
    const int seq = P.seq_len[b], stat = P.static_len[b], rest = seq - stat;
    if (seq > P.S_in || stat < 0 || rest < 0) {  // lengths that do not describe this cache
        if (tid == 0 && rank == 0) record_status(P.status, ST_EINVAL, b);
        return;
    }
    if (rest < 2 * L) return;  // third bullet of Section 2.2: skip
    const int rem = rest % L;
    if (rest / L - 1 > 1) {    // this kernel compresses one partition per call
        if (tid == 0 && rank == 0) record_status(P.status, ST_ECAPACITY, b);
        return;
    }
    cluster_arrive();  // "started": matched by the wait before the first remote store

    uint16_t* X = const_cast<uint16_t*>(tensor ? P.V : P.K) + (long long)b * P.sb + (long long)(u % P.H) * P.sh;
    const int p0_row = stat, p1_row = stat + L;
    // this CTA's tiles of a partition: global tile t = tau * RS + h for tau = 0 .. nloc - 1
    const int nloc = (ntiles - h + RS - 1) / RS;
    const int nres = min(res_tiles, nloc);  // tiles of this CTA's share of P1 that stay in shared memory

    const uint32_t ring_w = smem_u32(ring) + uint32_t(warp) * NS * G::TILE_BYTES;
    const uint32_t bar_w = smem_u32(bars) + uint32_t(warp) * NS * 8;
    if (lane == 0)
        for (int i = 0; i < NS; ++i) mbar_init(bar_w + 8 * i, 1);
    for (int t = tid; t < nres; t += G::NT) mbar_init(smem_u32(tile_bars + t), 1);
    if (tid == 0) {
        sc.abort = 0;
        for (int i = 0; i < 3; ++i) mbar_init(smem_u32(move_bars + i), 1);
    }
    fence_mbar_init();
    fence_proxy_async();
    __syncthreads();

    // rows [row0, row0 + rows) of this tensor -> shared memory at dst, completing on bar (warp-collective)
    auto fetch_tile = [&](int row0, int rows, uint32_t dst, uint32_t bar) {
        const uint16_t* src = X + (long long)row0 * P.ss;
        if (lane == 0) {
            fence_proxy_async();
            mbar_arrive_expect_tx(bar, uint32_t(rows) * ROWB);
        }
        if (contiguous) {
            if (lane == 0) bulk_g2s(dst, src, uint32_t(rows) * ROWB, bar);
        } else {
            __syncwarp();
            for (int r = lane; r < rows; r += 32) bulk_g2s(dst + uint32_t(r) * ROWB, src + (long long)r * P.ss, ROWB, bar);
        }
    };
    auto tile_row = [&](int tau) { return (tau * RS + h) * G::TR; };           // first row of local tile tau
    auto tile_rows = [&](int tau) { return min(G::TR, L - tile_row(tau)); };   // its valid rows
    // ---- 1. all resident tiles of P1 in flight at once (local tile tau belongs to warp tau mod NW)
    for (int tau = warp; tau < nres; tau += G::NW)
        fetch_tile(p1_row + tile_row(tau), tile_rows(tau), smem_u32(res) + uint32_t(tau) * G::TILE_BYTES,
                   smem_u32(tile_bars + tau));
    // Through this warp's ring go, in this order: its tiles of P1 that are not resident, then its
    // tiles of P0.  Producer cursor (phase 0: P1, 1: P0, 2: done).
    const int t1 = nres + ((warp - nres) % G::NW + G::NW) % G::NW;  // first streamed P1 tile of this warp
    int pphase = 0, pt = t1, pslot = 0;
    auto settle = [&]() {  // skip exhausted phases
        if (pphase == 0 && pt >= nloc) {
            pphase = 1;
            pt = warp;
        }
        if (pphase == 1 && pt >= nloc) pphase = 2;
    };
    settle();
    bool dead = false;
    auto issue_next = [&]() {  // warp-collective
        if (pphase > 1 || dead) return;
        fetch_tile((pphase == 0 ? p1_row : p0_row) + tile_row(pt), tile_rows(pt), ring_w + uint32_t(pslot) * G::TILE_BYTES,
                   bar_w + 8 * pslot);
        pt += G::NW;
        settle();
        if (++pslot == NS) pslot = 0;
    };
    for (int i = 0; i < NS; ++i) issue_next();

    int cslot = 0;
    uint32_t cparity = 0;
    const float inv_D = 1.0f / float(G::D), inv_Dm = 1.0f / float(G::D - P.ddof);
    f32x2 a2[G::NPW], b2[G::NPW];
    uint32_t mn[G::NPW], mx[G::NPW];
#pragma unroll
    for (int j = 0; j < G::NPW; ++j) {
        a2[j] = b2[j] = 0ull;
        mn[j] = G::E::kPosInf2;
        mx[j] = G::E::kNegInf2;
    }
    auto give_up = [&]() {  // warp-collective
        dead = true;
        if (lane == 0) {
            record_status(P.status, ST_ETIMEOUT, blockIdx.x);
            *reinterpret_cast<volatile int*>(&sc.abort) = 1;
        }
    };
    auto ring_tile = [&]() -> const uint4* {
        return reinterpret_cast<const uint4*>(ring + size_t(warp) * NS * G::TILE_BYTES + size_t(cslot) * G::TILE_BYTES);
    };
    auto ring_advance = [&]() {
        __syncwarp();
        issue_next();  // refill the stage just drained
        if (++cslot == NS) {
            cslot = 0;
            cparity ^= 1u;
        }
    };
    float* sig = tensor ? sg1 : sg0;

    // ---- statistics of P1 (Eq. 7, Eq. 8): resident tiles, then streamed ones
    for (int tau = warp; tau < nres && !dead; tau += G::NW) {
        if (!mbar_wait_bounded(smem_u32(tile_bars + tau), 0u)) {
            give_up();
            break;
        }
        const uint4* tile = reinterpret_cast<const uint4*>(res + size_t(tau) * G::TILE_BYTES);
        const int nrows = tile_rows(tau);
        if (nrows == G::TR) process_tile<G, false, true>(tile, nrows, a2, b2, mn, mx, sig, inv_D, inv_Dm, lane);
        else process_tile<G, false, false>(tile, nrows, a2, b2, mn, mx, sig, inv_D, inv_Dm, lane);
    }
    for (int tau = t1; tau < nloc && !dead; tau += G::NW) {
        if (!mbar_wait_bounded(bar_w + 8 * cslot, cparity)) {
            give_up();
            break;
        }
        const int nrows = tile_rows(tau);
        if (nrows == G::TR) process_tile<G, false, true>(ring_tile(), nrows, a2, b2, mn, mx, sig, inv_D, inv_Dm, lane);
        else process_tile<G, false, false>(ring_tile(), nrows, a2, b2, mn, mx, sig, inv_D, inv_Dm, lane);
        ring_advance();
    }
#pragma unroll
    for (int j = 0; j < G::NPW; ++j) {
#pragma unroll
        for (int o = G::LPR; o < 32; o <<= 1) {
            mn[j] = G::E::min2(mn[j], __shfl_xor_sync(0xffffffffu, mn[j], o));
            mx[j] = G::E::max2(mx[j], __shfl_xor_sync(0xffffffffu, mx[j], o));
        }
    }
    if (rl == 0) {
        store_stats_row<G>(stats + warp * 2 * STAT, mn, mx, cg);
    }
    __syncthreads();
    cluster_wait();  // every CTA of the cluster is running: its shared memory may be written
    // this CTA's min / max row goes to slot h of every row split of the same tensor (itself included)
    for (int w = tid; w < 2 * STAT; w += G::NT) {
        uint32_t v = stats[w];
        for (int q = 1; q < G::NW; ++q)
            v = (w < STAT) ? G::E::min2(v, stats[q * 2 * STAT + w]) : G::E::max2(v, stats[q * 2 * STAT + w]);
        const uint32_t slot = smem_u32(xstats + h * 2 * STAT + w);
        for (int s = 0; s < RS; ++s) st_cluster_u32(map_to_cta(slot, uint32_t(2 * s + tensor)), v);
    }
    cluster_arrive();
    cluster_wait();  // A: the rows of all splits are here
    {
        const int zero_range = make_coefficients<G>(xstats, RS, cg, a2, b2);
        if (zero_range != 0 && h == 0 && warp == 0 && rl == 0 && P.status != nullptr) atomicAdd(P.status + 2, zero_range);
    }

    // ---- 2. sigma of this CTA's tokens of P0 (Eq. 9, Eq. 10), sent to every CTA of the cluster
    for (int tau = warp; tau < nloc && !dead; tau += G::NW) {
        if (!mbar_wait_bounded(bar_w + 8 * cslot, cparity)) {
            give_up();
            break;
        }
        const int nrows = tile_rows(tau);
        float* so = sig + tile_row(tau);
        if (nrows == G::TR) process_tile<G, true, true, false>(ring_tile(), nrows, a2, b2, mn, mx, so, inv_D, inv_Dm, lane);
        else process_tile<G, true, false, false>(ring_tile(), nrows, a2, b2, mn, mx, so, inv_D, inv_Dm, lane);
        ring_advance();
    }
    __syncthreads();  // this CTA's sigma values are complete
    for (int i = tid; i < nloc * G::TR; i += G::NT) {
        const int token = tile_row(i / G::TR) + i % G::TR;
        if (token < L) {
            const uint32_t v = __float_as_uint(sig[token]), a = smem_u32(sig + token);
            for (uint32_t r = 0; r < CS; ++r)
                if (r != rank) st_cluster_u32(map_to_cta(a, r), v);
        }
    }
    cluster_arrive();
    cluster_wait();  // B: both sigma vectors are complete everywhere
    const bool aborted = *reinterpret_cast<volatile int*>(&sc.abort) != 0;
    bool failed = aborted;

    // ---- 3. the same selection in every CTA
    const int* kept = reinterpret_cast<const int*>(sg1);
    const int kk = (k + RS - 1) / RS;                       // kept rows per row split
    const int j_lo = min(k, h * kk), j_n = min(k, j_lo + kk) - j_lo;  // this CTA's share of them
    const bool moving = k < L && warp == 0 && !aborted;
    const uint32_t stage0 = smem_u32(ring), mbar0 = smem_u32(move_bars), gather_bar = smem_u32(move_bars + 2);
    const int R = int(smem_ring_bytes<G>(NS) / (2 * ROWB));  // rows per stage of a staged move
    int chunk = 0;                                           // stage / parity sequence of the staged moves
    if (!aborted) {
        float* scores_g = (P.scores_out != nullptr && rank == 0) ? P.scores_out + (long long)u * P.max_chunks * L : nullptr;
        score_and_select<G::NT>(sg0, sg1, L, k, true, scores_g, reinterpret_cast<int*>(sg1), sc, tid,
                                [] { __syncthreads(); }, [] {});
        if (P.idx_out != nullptr && rank == 0) {
            int32_t* kp = P.idx_out + (long long)u * P.max_chunks * k;
            for (int j = tid; j < k; j += G::NT) kp[j] = p0_row + kept[j];
        }
        // ---- 4a. the kept rows of this tensor (one warp: the copy engine does the work).  A pair
        //          owns its tensor alone and packs them with staged copies, any number of them.
        //          With row splits each CTA gathers its share into the idle rings in one go (the
        //          host made sure that a share fits) and stores it after the barrier below.
        if (moving && RS == 1) {
            if (!move_rows_staged<G>(X, P.ss, stat, k, [&](int j) { return p0_row + kept[j]; }, false, stage0, R,
                                     mbar0, chunk, lane))
                failed = true;
        } else if (moving && j_n > 0) {
            if (lane == 0) {
                fence_proxy_async();
                mbar_arrive_expect_tx(gather_bar, uint32_t(j_n) * ROWB);
            }
            __syncwarp();
            for (int r = lane; r < j_n; r += 32)
                bulk_g2s(stage0 + uint32_t(r) * ROWB, X + (long long)(p0_row + kept[j_lo + r]) * P.ss, ROWB, gather_bar);
            if (!mbar_wait_bounded(gather_bar, 0u)) failed = true;
        }
    }
    cluster_arrive();
    cluster_wait();  // C: every kept row of the unit has been read: P0's rows may be overwritten
    if (moving && !failed) {
        // ---- 4b. kept rows to their place, the window out of the resident buffer, the rest staged
        if (RS > 1 && j_n > 0) {
            if (contiguous) {
                if (lane == 0) bulk_s2g(X + (long long)(stat + j_lo) * P.ss, stage0, uint32_t(j_n) * ROWB);
            } else {
                for (int r = lane; r < j_n; r += 32)
                    bulk_s2g(X + (long long)(stat + j_lo + r) * P.ss, stage0 + uint32_t(r) * ROWB, ROWB);
            }
        }
        for (int tau = lane; tau < nres; tau += 32) {
            const int r0 = tile_row(tau), nr = tile_rows(tau);
            const uint32_t src = smem_u32(res) + uint32_t(tau) * G::TILE_BYTES;
            if (contiguous) {
                bulk_s2g(X + (long long)(stat + k + r0) * P.ss, src, uint32_t(nr) * ROWB);
            } else {
                for (int r = 0; r < nr; ++r) bulk_s2g(X + (long long)(stat + k + r0 + r) * P.ss, src + uint32_t(r) * ROWB, ROWB);
            }
        }
        bulk_commit();
        bulk_wait_read_all();  // the rings are free again
        __syncwarp();
        if (h == 0) {
            // rows of P1 that were not resident (pairs only: with row splits the host keeps all of P1
            // resident) and the remainder behind the window: ascending, sources above destinations
            const int res_rows = RS == 1 ? min(L, nres * G::TR) : L;
            if (!move_rows_staged<G>(X, P.ss, stat + k + res_rows, (L - res_rows) + rem,
                                     [&](int j) { return p1_row + res_rows + j; }, true, stage0, R, mbar0, chunk, lane))
                failed = true;
        }
        asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");  // stores performed before the lengths change
        __syncwarp();
    }
    if (failed && !aborted && warp == 0 && lane == 0) record_status(P.status, ST_ETIMEOUT, blockIdx.x);
    // The lengths of a sequence change once all CTAs of all of its heads are done: each has read
    // the old values by then.  The last one writes the new ones and clears the counter.  A CTA
    // that gave up still counts and marks the sequence: its lengths stay as they were.
    if (tid == 0) {
        const int old = atomicAdd(P.seq_done + b, failed ? 1 + kSeqFailed : 1);
        if ((old & (kSeqFailed - 1)) == int(CS) * P.H - 1) {
            P.seq_done[b] = 0;
            if (!failed && old < kSeqFailed) {
                const_cast<int32_t*>(P.static_len)[b] = stat + k;
                const_cast<int32_t*>(P.seq_len)[b] = stat + k + L + rem;
            }
        }
    }
    if (failed) {  // copies may still be in flight towards this CTA's shared memory
        const unsigned long long t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 200000000ull) { /* bounded drain delay */ }
    }
}

}  // namespace lagkv
