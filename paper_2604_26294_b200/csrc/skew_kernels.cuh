// CTA-pair kernel whose tile holds the SAME 256 token rows of TWO neighbouring ranks, for the GEMMs that walk all D
// weight shards in ring order (down projection, dX) when a rank owns few token tiles.
//
// Ranks 2q+1 and 2q meet the shards in the orders (2q+1, 2q, 2q-1, ...) and (2q, 2q-1, ..., 2q+1): the second order is
// the first one shifted by one step.  A "tall" tile runs D + 1 slots; in slot s it loads the weight panel of shard
// (2q+1 - s) mod D ONCE and uses it for the odd rank (slots 0 .. D-1, accumulator 0) and for the even rank (slots
// 1 .. D, accumulator 1).  Each rank still adds its D partial products in its own ring order (Algorithm 2: the shard
// held at step t is (r - t) mod D), so the sums are the same bits as in a one-rank tile; only the number of times a
// weight panel crosses L2 -> shared memory halves, and with it the DRAM re-reads when panels fall out of L2.
// The two accumulators finish one slot apart: accumulator 0 is drained by the epilogue warps while the MMAs of the
// last slot still run on accumulator 1, and accumulator 1 while the next tile starts on accumulator 0.
//
// Tile list: `skew_tiles` tall tiles (whole rounds of the CTA pairs, as many as fit without adding a time unit),
// then one-rank 256 x 256 tiles for the rest, handed out dynamically (see dyn_kernels.cuh for the queue).
// Positions: rank pair (last pair first) -> hidden block -> token tile of the rank; a tall tile is a position, the
// one-rank tiles are the remaining positions split in two.  The token tiles of a rank pair that share a weight panel
// are neighbours in the list, so they run at the same time wherever a round of the CTA pairs begins (with the token
// tile as the slow index, the 74 pairs cut the 64 tiles of a rank pair at a different place every round and most
// panels were fetched twice: measured 2.72 GB of DRAM reads for dX at S = 8192, D = 8, against 1.5 GB of operands).
//
// Policy (besides Params::sched / num_tiles / stages / status / timeout_ns):
//   Params::D, S_loc, tiles_per_rank, n_blocks, skew_tiles;  inner(p) = k-blocks per shard;
//   load_a(p, first token row, shard, i, cta, smem, bar), load_b(p, hidden block, shard, i, cta, smem, bar);
//   epilogue(p, Tile, cta, row, tmem row address) with Tile = {mt, nb, r, halves, row0, valid}.
#pragma once
#include "dyn_kernels.cuh"

namespace tsp {

struct SkewTile {
    int tall;   // 1: both ranks of the pair, 0: the rank `r` alone
    int r;      // rank of accumulator 0 (tall: the odd rank 2q+1; accumulator 1 then belongs to rank r - 1)
    int m, nb;  // token tile within the rank, hidden block
};

template <class Params>
__device__ __forceinline__ SkewTile skew_decode(const Params& p, int t) {
    SkewTile o;
    o.tall = t < p.skew_tiles;
    const int u = t - p.skew_tiles;
    const int pos = o.tall ? t : p.skew_tiles + (u >> 1);
    const int per_pair = p.tiles_per_rank * p.n_blocks;
    const int qi = pos / per_pair;
    const int rem = pos - qi * per_pair;
    o.nb = rem / p.tiles_per_rank;
    o.m = rem - o.nb * p.tiles_per_rank;
    o.r = 2 * (p.D / 2 - 1 - qi) + 1;
    if (!o.tall && (u & 1)) --o.r;
    return o;
}

template <class Policy>
__device__ __forceinline__ typename Policy::Tile skew_rank_tile(const typename Policy::Params& p, const SkewTile& st,
                                                                int r) {
    typename Policy::Tile tl;
    tl.r = r;
    tl.mt = r * p.tiles_per_rank + st.m;
    tl.nb = st.nb;
    tl.halves = 1;
    tl.row0 = r * p.S_loc + st.m * 256;
    tl.valid = min(256, p.S_loc - st.m * 256);
    return tl;
}

// Stage layout per CTA: [A rows of accumulator 0: 16 KB][A rows of accumulator 1: 16 KB][B: 16 KB] = kWideStageBytes.
template <class Policy>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kNumThreads, 1)
pair_skew_kernel(const __grid_constant__ typename Policy::Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_1024(smem_raw);
    SharedCtl* ctl = reinterpret_cast<SharedCtl*>(smem + p.stages * kWideStageBytes);
    DynCtl* q = reinterpret_cast<DynCtl*>(reinterpret_cast<uint8_t*>(ctl) + sizeof(SharedCtl));
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta = cluster_ctarank();
    const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kQueueSlots; ++s) {
            mbar_init(smem_u32(&q->q_full[s]), 1);
            mbar_init(smem_u32(&q->q_empty[s]), 10);
        }
    }
    pair_setup(ctl, p.stages, 2);   // tmem_full[a] / tmem_empty[a]: accumulator a complete / drained
    const uint32_t tmem_base = ctl->tmem_base;
    WaitCtx w{&ctl->abort, p.status, p.timeout_ns};
    const int n_inner = Policy::inner(p);
    const int D = p.D;

    if (warp == 0) {
        if (lane == 0) {
            Policy::prefetch(p);
            PipeState ps;
            bool ok = true;
            QueueReader qr;
            int seq = 0;
            int next = pair_id - n_pairs;   // first tile = own index; later ones n_pairs + the counter's hand-out
            while (ok) {
                int tile;
                if (cta == 0) {
                    tile = next + n_pairs < p.num_tiles ? next + n_pairs : -1;
                    if (!(ok = queue_push(q, w, seq++, tile))) break;
                } else {
                    if (!(ok = qr.pop(q, w, false, tile))) break;
                }
                if (tile < 0) break;
                const SkewTile st = skew_decode(p, tile);
                const int row_a = st.r * p.S_loc + st.m * 256 + static_cast<int>(cta) * 128;
                const int row_b = row_a - p.S_loc;   // the even rank's rows (tall tiles only)
                const int n_slots = st.tall ? D + 1 : D;
                draw_async(p.sched, cta == 0, next);
                for (int s = 0; s < n_slots && ok; ++s) {
                    int k = st.r - s;
                    if (k < 0) k += D;
                    const bool on0 = s < D, on1 = st.tall && s >= 1;
                    const uint32_t bytes = 2u * 16384u * (1u + static_cast<uint32_t>(on0) + static_cast<uint32_t>(on1));
                    for (int i = 0; i < n_inner; ++i) {
                        if (!(ok = wait_bar(smem_u32(&ctl->empty[ps.stage]), ps.phase ^ 1u, w, kErrWaitEmpty))) break;
                        const uint32_t bar = map_to_cta(smem_u32(&ctl->full[ps.stage]), 0);
                        const uint32_t sa = smem_base + ps.stage * kWideStageBytes;
                        if (cta == 0) mbar_arrive_expect_tx(smem_u32(&ctl->full[ps.stage]), bytes);
                        if (on0) Policy::load_a(p, row_a, k, i, cta, sa, bar);
                        if (on1) Policy::load_a(p, row_b, k, i, cta, sa + 16384u, bar);
                        Policy::load_b(p, st.nb, k, i, cta, sa + 32768u, bar);
                        ps.advance(p.stages);
                    }
                }
            }
            if (cta == 0) scheduler_done(p.sched, n_pairs);
        }
    } else if (warp == 1) {
        if (lane == 0 && cta == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(256, 256, Policy::kAMn, Policy::kBMn);
            PipeState ps;
            bool ok = true;
            QueueReader qr;
            uint32_t uses[2] = {0u, 0u};   // how often each accumulator has been started so far
            int singles = 0;               // one-rank tiles since the last tall one: they alternate between the accumulators
            while (ok) {
                int tile;
                if (!(ok = qr.peek(q, w, false, tile)) || tile < 0) break;
                const bool tall = tile < p.skew_tiles;
                const int lone = tall ? -1 : (singles & 1);   // accumulator of a one-rank tile
                singles = tall ? 0 : singles + 1;
                const int n_slots = tall ? D + 1 : D;
                for (int s = 0; s < n_slots && ok; ++s) {
                    // accumulator a is live in slots first[a] .. last[a]
                    const bool live0 = tall ? s < D : lone == 0;
                    const bool live1 = tall ? s >= 1 : lone == 1;
                    const int first0 = 0, first1 = tall ? 1 : 0;
                    for (int i = 0; i < n_inner && ok; ++i) {
                        if (!(ok = wait_bar(smem_u32(&ctl->full[ps.stage]), ps.phase, w, kErrWaitFull))) break;
                        tc_fence_after_sync();
                        const uint32_t sa = smem_base + ps.stage * kWideStageBytes, sb = sa + 32768u;
                        if (live0) {
                            const bool start = s == first0 && i == 0;
                            if (start) {   // the previous user's epilogue must have drained the accumulator
                                if (!(ok = wait_bar(smem_u32(&ctl->tmem_empty[0]), (uses[0] & 1u) ^ 1u, w, kErrWaitTmemEmpty))) break;
                                tc_fence_after_sync();
                                ++uses[0];
                            }
                            pair_issue_kblock<Policy::kAMn, Policy::kBMn>(tmem_base, sa, sb, idesc, !start);
                        }
                        if (live1) {
                            const bool start = s == first1 && i == 0;
                            if (start) {
                                if (!(ok = wait_bar(smem_u32(&ctl->tmem_empty[1]), (uses[1] & 1u) ^ 1u, w, kErrWaitTmemEmpty))) break;
                                tc_fence_after_sync();
                                ++uses[1];
                            }
                            pair_issue_kblock<Policy::kAMn, Policy::kBMn>(tmem_base + 256, tall ? sa + 16384u : sa, sb, idesc, !start);
                        }
                        const uint32_t e = smem_u32(&ctl->empty[ps.stage]);
                        umma_commit_pair(e);
                        umma_commit_pair(map_to_cta(e, 1));
                        ps.advance(p.stages);
                    }
                    if (!ok) break;
                    if (live0 && s == D - 1) {
                        const uint32_t f = smem_u32(&ctl->tmem_full[0]);
                        umma_commit_pair(f);
                        umma_commit_pair(map_to_cta(f, 1));
                    }
                    if (live1 && s == n_slots - 1) {
                        const uint32_t f = smem_u32(&ctl->tmem_full[1]);
                        umma_commit_pair(f);
                        umma_commit_pair(map_to_cta(f, 1));
                    }
                }
                qr.release(q, false);
            }
        }
    } else {
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        bool ok = true;
        QueueReader qr;
        uint32_t uses0 = 0u, uses1 = 0u;
        int singles = 0;
        while (ok) {
            int tile;
            if (!(ok = qr.pop(q, w, true, tile)) || tile < 0) break;
            const SkewTile st = skew_decode(p, tile);
            const int lone = st.tall ? -1 : (singles & 1);
            singles = st.tall ? 0 : singles + 1;
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
#pragma unroll 1
            for (int a = 0; a < 2 && ok; ++a) {
                if (!st.tall && a != lone) continue;
                if (!(ok = wait_bar(smem_u32(&ctl->tmem_full[a]), (a ? uses1 : uses0) & 1u, w, kErrWaitTmemFull))) break;
                if (a) ++uses1; else ++uses0;
                tc_fence_after_sync();
                const typename Policy::Tile tl = skew_rank_tile<Policy>(p, st, st.tall ? st.r - a : st.r);
                Policy::epilogue(p, tl, cta, row, t_row + a * 256);
                tc_fence_before_sync();
                mbar_arrive_cluster(map_to_cta(smem_u32(&ctl->tmem_empty[a]), 0));
            }
        }
    }
    pair_teardown(ctl, w);
}

}  // namespace tsp
