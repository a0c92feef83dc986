// CTA-pair GEMM kernel with a dynamic tile hand-out, and the fused ring step that needs it.
//
// pair_dyn_kernel is pair_gemm_kernel (256 x 256 tiles, cta_group::2, two accumulator buffers) except that the CTA
// pairs do not take tiles round-robin: the leader CTA's producer lane draws the next list index from a counter in
// global memory and hands it to every role of both CTAs through a small queue in shared memory.  Which pair runs a
// tile never changes what the tile computes, so outputs are bit-identical to the static kernels.  Two properties
// follow from drawing the list in order:
//   * the tiles that run at the same time are neighbours in the list, however far the pairs drift apart in time, so a
//     tile order laid out for sharing operand blocks through L2 keeps working over thousands of tiles;
//   * a tile may wait for the results of tiles EARLIER in the list (they have been drawn, hence are running on a
//     resident CTA pair or are finished), without any assumption about how many CTAs are resident.  The fused ring
//     step below relies on this: gate|up tiles first, then down-projection tiles that wait for their token rows of A.
//
// Queue protocol (kQueueSlots entries, one writer = leader producer lane):
//   q_empty[s] (leader's): 10 arrivals = leader MMA lane + 4 leader epilogue warps + peer producer lane + 4 peer
//              epilogue warps, each after it has read slot s;
//   q_full[s]  (one per CTA): one arrival by the writer after it has stored the tile index into both CTAs' slot s.
//   A tile index of -1 ends every role's loop.
// Scheduler words in global memory: sched[0] = list indices handed out beyond the first one of every pair (pair i
// starts with index i), sched[1] = leaders that have stopped drawing; the last leader to stop resets both, so the words
// are zero again when the kernel ends.
#pragma once
#include "pair_kernels.cuh"

namespace tsp {

constexpr int kQueueSlots = 4;
constexpr int kErrWaitQueue = 7, kErrWaitReady = 8;

struct __align__(16) DynCtl {
    uint64_t q_full[kQueueSlots];
    uint64_t q_empty[kQueueSlots];
    volatile int q_tile[kQueueSlots];
};

__device__ __forceinline__ void st_shared_cluster_u32(uint32_t cluster_addr, uint32_t v) {
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(cluster_addr), "r"(v) : "memory");
}
__device__ __forceinline__ int ld_acquire_gpu(const int* p) {
    int v;
    asm volatile("ld.acquire.gpu.global.s32 %0, [%1];" : "=r"(v) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ void red_release_gpu_add(int* p, int v) {
    asm volatile("red.release.gpu.global.add.s32 [%0], %1;" ::"l"(p), "r"(v) : "memory");
}
// Draw the next list index if `take` is set: the atomic is issued here, its result lands in `next` whenever it arrives;
// the thread only waits for it where it first reads `next` (a plain C++ atomicAdd inside a branch makes the compiler
// merge the old and the new value right after the branch, which stalls the producer lane for the atomic's round trip).
__device__ __forceinline__ void draw_async(int* counter, bool take, int& next) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.u32 p, %2, 0;\n\t"
        "@p atom.global.add.u32 %0, [%1], 1;\n\t}"
        : "+r"(next)
        : "l"(counter), "r"(static_cast<uint32_t>(take))
        : "memory");
}
// Orders this thread's accesses through the generic proxy against accesses through the async proxy (TMA).
__device__ __forceinline__ void fence_proxy_async_all() { asm volatile("fence.proxy.async;" ::: "memory"); }

// One reader of the tile queue: a single lane, or a whole epilogue warp (`warp_wide`: every lane reads the slot, lane 0
// releases it once the warp has converged).
struct QueueReader {
    int n = 0;
    // wait for the next entry and read it; the slot stays reserved until release()
    __device__ __forceinline__ bool peek(DynCtl* q, const WaitCtx& w, bool warp_wide, int& tile) {
        const int slot = n % kQueueSlots;
        const uint32_t parity = (n / kQueueSlots) & 1;
        bool ok = wait_bar(smem_u32(&q->q_full[slot]), parity, w, kErrWaitQueue);
        if (warp_wide) ok = __all_sync(0xffffffffu, ok);   // the warp leaves together
        if (!ok) return false;
        tile = q->q_tile[slot];
        return true;
    }
    __device__ __forceinline__ void release(DynCtl* q, bool warp_wide) {
        const int slot = n % kQueueSlots;
        ++n;
        if (warp_wide) __syncwarp();
        if (!warp_wide || (threadIdx.x & 31) == 0) mbar_arrive_cluster(map_to_cta(smem_u32(&q->q_empty[slot]), 0));
    }
    __device__ __forceinline__ bool pop(DynCtl* q, const WaitCtx& w, bool warp_wide, int& tile) {
        if (!peek(q, w, warp_wide, tile)) return false;
        release(q, warp_wide);
        return true;
    }
};

// The writer (leader producer lane) stores entry number `seq` into both CTAs' queues.
__device__ __forceinline__ bool queue_push(DynCtl* q, const WaitCtx& w, int seq, int tile) {
    const int slot = seq % kQueueSlots;
    const uint32_t parity = (seq / kQueueSlots) & 1;
    if (!wait_bar(smem_u32(&q->q_empty[slot]), parity ^ 1u, w, kErrWaitQueue)) return false;
    q->q_tile[slot] = tile;
    st_shared_cluster_u32(map_to_cta(smem_u32(const_cast<int*>(&q->q_tile[slot])), 1), static_cast<uint32_t>(tile));
    mbar_arrive(smem_u32(&q->q_full[slot]));
    mbar_arrive_cluster(map_to_cta(smem_u32(&q->q_full[slot]), 1));
    return true;
}
// A leader that draws no more says so; the last one zeroes the scheduler words for the next launch.
__device__ __forceinline__ void scheduler_done(int* sched, int n_pairs) {
    __threadfence();
    if (atomicAdd(sched + 1, 1) == n_pairs - 1) {
        atomicExch(sched, 0);
        atomicExch(sched + 1, 0);
    }
}

// Adapter: the static policies of pair_kernels.cuh have one K-loop shape per launch and no dependencies.
template <class P>
struct DynOf : P {
    using Params = typename P::Params;
    using Tile = typename P::Tile;
    static constexpr bool kOrderedDraws = false;   // no tile waits for another
    __device__ static __forceinline__ int outer_t(const Params& p, const Tile&) { return P::outer(p); }
    __device__ static __forceinline__ int inner_t(const Params& p, const Tile&) { return P::inner(p); }
    __device__ static __forceinline__ int k_blocks_of(const Params& p, int) { return P::outer(p) * P::inner(p); }
    __device__ static __forceinline__ bool wait_ready(const Params&, const Tile&, const WaitCtx&, bool&) { return true; }
    __device__ static __forceinline__ void publish(const Params&, const Tile&) {}
    __device__ static __forceinline__ void prologue(const Params&, int) {}
};

// Policy (in addition to what pair_gemm_kernel asks for): Params::sched; outer_t / inner_t(p, tile) = K-loop shape of
// that tile, k_blocks_of(p, list index) their product without decoding the tile (the MMA lane's only question);
// wait_ready(p, tile, w, state) called by each CTA's producer lane before the tile's first load (`state` is a flag the
// lane keeps for the policy across its tiles);
// publish(p, tile) called by the 128 epilogue threads of a CTA after the tile's stores;
// prologue(p, pair_id) called once by the epilogue threads of CTA 0.
template <class Policy>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kNumThreads, 1)
pair_dyn_kernel(const __grid_constant__ typename Policy::Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_1024(smem_raw);
    SharedCtl* ctl = reinterpret_cast<SharedCtl*>(smem + p.stages * kPairStageBytes);
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
    pair_setup(ctl, p.stages, 2);   // initialises the pipeline barriers, fences all initialisations, cluster-wide sync
    const uint32_t tmem_base = ctl->tmem_base;
    WaitCtx w{&ctl->abort, p.status, p.timeout_ns};

    if (warp == 0) {
        if (lane == 0) {
            Policy::prefetch(p);
            PipeState ps;
            bool ok = true;
            QueueReader qr;
            int seq = 0;
            // Without dependencies between tiles the first tile of a pair is its own index and later ones are n_pairs +
            // what the counter hands out.  With dependencies every index comes from the counter, the first one too: a
            // tile then only ever waits for tiles drawn by CTA pairs that are running.  Later indices are drawn when
            // the previous tile's loads begin, so that the atomic's latency never shows.
            bool ready_state = false;
            const int base = Policy::kOrderedDraws ? 0 : n_pairs;
            int next = Policy::kOrderedDraws ? (cta == 0 ? atomicAdd(p.sched, 1) : 0) : pair_id - n_pairs;
            while (ok) {
                int tile;
                if (cta == 0) {   // scheduler: hand the drawn index to both CTAs
                    tile = next + base < p.num_tiles ? next + base : -1;
                    if (!(ok = queue_push(q, w, seq++, tile))) break;
                } else {
                    if (!(ok = qr.pop(q, w, false, tile))) break;
                }
                if (tile < 0) break;
                const typename Policy::Tile tl = Policy::decode(p, tile);
                const int n_outer = Policy::outer_t(p, tl), n_inner = Policy::inner_t(p, tl);
                if (!(ok = Policy::wait_ready(p, tl, w, ready_state))) break;
                draw_async(p.sched, cta == 0, next);
                for (int o = 0; o < n_outer && ok; ++o) {
                    const int sel = Policy::select(p, tl, o);
                    for (int i = 0; i < n_inner; ++i) {
                        if (!(ok = wait_bar(smem_u32(&ctl->empty[ps.stage]), ps.phase ^ 1u, w, kErrWaitEmpty))) break;
                        const uint32_t bar = map_to_cta(smem_u32(&ctl->full[ps.stage]), 0);
                        const uint32_t sa = smem_base + ps.stage * kPairStageBytes, sb = sa + kPairABytes;
                        if (cta == 0) mbar_arrive_expect_tx(smem_u32(&ctl->full[ps.stage]), 2 * kPairStageBytes);
                        Policy::load(p, tl, sel, i, cta, sa, sb, bar);
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
            for (int it = 0; ok; ++it) {
                int tile;
                if (!(ok = qr.peek(q, w, false, tile)) || tile < 0) break;
                const int k_blocks = Policy::k_blocks_of(p, tile);   // no tile decoding on the MMA lane: it is the critical path
                const int buf = it & 1;
                if (!(ok = wait_bar(smem_u32(&ctl->tmem_empty[buf]), ((it >> 1) & 1) ^ 1u, w, kErrWaitTmemEmpty))) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * 256;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!(ok = wait_bar(smem_u32(&ctl->full[ps.stage]), ps.phase, w, kErrWaitFull))) break;
                    tc_fence_after_sync();
                    const uint32_t sa = smem_base + ps.stage * kPairStageBytes, sb = sa + kPairABytes;
                    pair_issue_kblock<Policy::kAMn, Policy::kBMn>(d_tmem, sa, sb, idesc, kb > 0);
                    const uint32_t e = smem_u32(&ctl->empty[ps.stage]);
                    umma_commit_pair(e);
                    umma_commit_pair(map_to_cta(e, 1));
                    ps.advance(p.stages);
                }
                if (ok) {
                    const uint32_t f = smem_u32(&ctl->tmem_full[buf]);
                    umma_commit_pair(f);
                    umma_commit_pair(map_to_cta(f, 1));
                }
                qr.release(q, false);   // after the tile's MMAs are issued: the queue slot is not the bottleneck
            }
        }
    } else {
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        if (cta == 0) Policy::prologue(p, pair_id);
        bool ok = true;
        QueueReader qr;
        for (int it = 0; ok; ++it) {
            int tile;
            if (!(ok = qr.pop(q, w, true, tile)) || tile < 0) break;
            const typename Policy::Tile tl = Policy::decode(p, tile);
            const int buf = it & 1;
            if (!(ok = wait_bar(smem_u32(&ctl->tmem_full[buf]), (it >> 1) & 1, w, kErrWaitTmemFull))) break;
            tc_fence_after_sync();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * 256;
            Policy::epilogue(p, tl, cta, row, t_row);
            tc_fence_before_sync();
            mbar_arrive_cluster(map_to_cta(smem_u32(&ctl->tmem_empty[buf]), 0));
            Policy::publish(p, tl);
        }
    }
    pair_teardown(ctl, w);
}

// Mixed-width kernel (pair_wide_kernel: 256 x 512 and 256 x 256 tiles, one accumulator set) with the same dynamic
// hand-out.  Policies are those of pair_wide_kernel (decode_mixed / load_wide / epilogue_half) plus Params::sched.
template <class Policy>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kNumThreads, 1)
pair_wide_dyn_kernel(const __grid_constant__ typename Policy::Params p) {
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
    pair_setup(ctl, p.stages, 2);   // tmem_empty[h]: column half h drained; tmem_full[0]: whole tile accumulated
    const uint32_t tmem_base = ctl->tmem_base;
    WaitCtx w{&ctl->abort, p.status, p.timeout_ns};
    const int n_outer = Policy::outer(p), n_inner = Policy::inner(p);
    const int k_blocks = n_outer * n_inner;

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
                const typename Policy::Tile tl = Policy::decode_mixed(p, tile);
                const uint32_t bytes = 2u * (kPairABytes + static_cast<uint32_t>(tl.halves) * 16384u);
                draw_async(p.sched, cta == 0, next);
                for (int o = 0; o < n_outer && ok; ++o) {
                    const int sel = Policy::select(p, tl, o);
                    for (int i = 0; i < n_inner; ++i) {
                        if (!(ok = wait_bar(smem_u32(&ctl->empty[ps.stage]), ps.phase ^ 1u, w, kErrWaitEmpty))) break;
                        const uint32_t bar = map_to_cta(smem_u32(&ctl->full[ps.stage]), 0);
                        const uint32_t sa = smem_base + ps.stage * kWideStageBytes, sb = sa + kPairABytes;
                        if (cta == 0) mbar_arrive_expect_tx(smem_u32(&ctl->full[ps.stage]), bytes);
                        Policy::load_wide(p, tl, sel, i, cta, sa, sb, bar);
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
            uint32_t uses[2] = {0u, 0u};   // how often each column half has been filled so far
            while (ok) {
                int tile;
                if (!(ok = qr.peek(q, w, false, tile)) || tile < 0) break;
                const int halves = Policy::halves_of(p, tile);
                for (int kb = 0; kb < k_blocks && ok; ++kb) {
                    if (!(ok = wait_bar(smem_u32(&ctl->full[ps.stage]), ps.phase, w, kErrWaitFull))) break;
                    tc_fence_after_sync();
                    const uint32_t sa = smem_base + ps.stage * kWideStageBytes, sb = sa + kPairABytes;
                    for (int h = 0; h < halves; ++h) {
                        if (kb == 0) {  // the previous user's epilogue must have drained this half
                            if (!(ok = wait_bar(smem_u32(&ctl->tmem_empty[h]), (uses[h] & 1u) ^ 1u, w, kErrWaitTmemEmpty))) break;
                            tc_fence_after_sync();
                            ++uses[h];
                        }
                        pair_issue_kblock<Policy::kAMn, Policy::kBMn>(tmem_base + h * 256, sa, sb + h * 16384, idesc, kb > 0);
                    }
                    if (!ok) break;
                    const uint32_t e = smem_u32(&ctl->empty[ps.stage]);
                    umma_commit_pair(e);
                    umma_commit_pair(map_to_cta(e, 1));
                    ps.advance(p.stages);
                }
                if (ok) {
                    const uint32_t f = smem_u32(&ctl->tmem_full[0]);
                    umma_commit_pair(f);
                    umma_commit_pair(map_to_cta(f, 1));
                }
                qr.release(q, false);
            }
        }
    } else {
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        bool ok = true;
        QueueReader qr;
        for (int it = 0; ok; ++it) {
            int tile;
            if (!(ok = qr.pop(q, w, true, tile)) || tile < 0) break;
            const typename Policy::Tile tl = Policy::decode_mixed(p, tile);
            if (!(ok = wait_bar(smem_u32(&ctl->tmem_full[0]), it & 1, w, kErrWaitTmemFull))) break;
            tc_fence_after_sync();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
#pragma unroll 1
            for (int h = 0; h < tl.halves; ++h) {
                Policy::epilogue_half(p, tl, cta, row, t_row + h * 256, h);
                tc_fence_before_sync();
                mbar_arrive_cluster(map_to_cta(smem_u32(&ctl->tmem_empty[h]), 0));
            }
        }
    }
    pair_teardown(ctl, w);
}

// ------------------------------------------------------------------------------------------------
// Fused ring step(s) of ONE rank (Algorithm 2, loop body, as one launch): for the n shards the rank holds,
//   phase 0 tiles: A[:, s] = act(X_p Wg_s) * (X_p Wu_s)        256 tokens x 128 intermediate columns, K = H
//   phase 1 tiles: Yacc (+)= sum_s A[:, s] Wd_s                256 tokens x 256 hidden, K = n * F/D, shards in order
// The list holds all phase-0 tiles, then the phase-1 tiles.  A phase-1 tile waits until every phase-0 tile of its
// 256 token rows has published (ready[mt] reaches ready_target: eight epilogue warps per tile, jl_blocks * n tiles
// per token tile).  A goes through global memory, but a rank's A is a few MB, written and read back within microseconds: it
// lives in L2.  `ready_clear` is the counter set of the NEXT launch (two sets alternate), zeroed here.
// ------------------------------------------------------------------------------------------------
struct PairFusedStepPolicy {
    static constexpr bool kAMn = false, kBMn = true;
    static constexpr bool kOrderedDraws = true;    // phase-1 tiles wait for phase-0 tiles earlier in the list
    struct Params {
        CUtensorMap map_x, map_wg, map_wu;  // X (H, S_loc, 1) box (64,128); Wg, Wu (F/D, H, n) box (64,64)
        CUtensorMap map_a, map_wd;          // A (n F/D, S_loc, 1) box (64,128); Wd (H, F/D, n) box (64,64)
        __nv_bfloat16* A;                   // [S_loc, n * F/D]
        float* Yacc;                        // [S_loc, H] fp32 partial sums carried from call to call
        CarryTma carry_tma;                 // Yacc through the TMA unit (epi_off = 0: element-wise accesses instead)
        __nv_bfloat16* Y;                   // [S_loc, H]
        int* ready;                         // [m_tiles] counters of this launch (zero on entry)
        int* ready_clear;                   // counters of the next launch
        int ready_clear_count;
        int ready_target;
        int* ready_all;                     // one more counter of the same set: publishing warps of ALL gate|up tiles
        int ready_all_target;
        int S_loc, H, F_d, n_shards, mode, act;   // mode: 0 first, 1 middle, 2 last (bf16 Y), 3 only call
        int m_tiles, jl_blocks, n_blocks, gate_tiles;
        int band, group;                    // token tiles per band of phase 0 / per group of phase 1
        int* sched;
        int num_tiles, stages;
        int* status;
        unsigned long long timeout_ns;
    };
    struct Tile {
        int phase, mt, s, jl, nb, row0, valid;
    };
    __device__ static __forceinline__ void prefetch(const Params& p) {
        tma_prefetch_desc(&p.map_x);
        tma_prefetch_desc(&p.map_wg);
        tma_prefetch_desc(&p.map_wu);
        tma_prefetch_desc(&p.map_a);
        tma_prefetch_desc(&p.map_wd);
    }
    // phase 0: band of token tiles -> shard -> column block -> token tile (the band's rows of X stay in L2 while the
    // shards' weights stream past once per band); phase 1: group of token tiles -> hidden block -> token tile
    __device__ static __forceinline__ Tile decode(const Params& p, int tile) {
        Tile o;
        o.s = o.jl = o.nb = 0;
        if (tile < p.gate_tiles) {
            o.phase = 0;
            const int per_band = p.band * p.n_shards * p.jl_blocks;
            const int b = tile / per_band;
            const int b_start = b * p.band;
            const int b_sz = min(p.band, p.m_tiles - b_start);
            int rem = tile - b * per_band;
            const int col = rem / b_sz;          // (shard, column block)
            o.mt = b_start + rem - col * b_sz;
            o.s = col / p.jl_blocks;
            o.jl = col - o.s * p.jl_blocks;
        } else {
            const int t = tile - p.gate_tiles;
            o.phase = 1;
            const int per_group = p.group * p.n_blocks;
            const int g = t / per_group;
            const int g_start = g * p.group;
            const int g_sz = min(p.group, p.m_tiles - g_start);
            const int rem = t - g * per_group;
            o.nb = rem / g_sz;
            o.mt = g_start + rem - o.nb * g_sz;
        }
        o.row0 = o.mt * 256;
        o.valid = min(256, p.S_loc - o.row0);
        return o;
    }
    __device__ static __forceinline__ int outer_t(const Params& p, const Tile& tl) { return tl.phase ? p.n_shards : 1; }
    __device__ static __forceinline__ int inner_t(const Params& p, const Tile& tl) {
        return (tl.phase ? p.F_d : p.H) / kBK;
    }
    __device__ static __forceinline__ int k_blocks_of(const Params& p, int tile) {
        return tile < p.gate_tiles ? p.H / kBK : p.n_shards * (p.F_d / kBK);
    }
    __device__ static __forceinline__ int select(const Params&, const Tile& tl, int o) { return tl.phase ? o : tl.s; }
    __device__ static __forceinline__ void load(const Params& p, const Tile& tl, int s, int i, uint32_t cta, uint32_t sa,
                                                uint32_t sb, uint32_t bar) {
        if (tl.phase == 0) {
            pair_load_kmajor(sa, &p.map_x, bar, i * kBK, tl.row0 + cta * 128, 0);
            pair_load_mnmajor(sb, cta == 0 ? &p.map_wg : &p.map_wu, bar, tl.jl * 128, i * kBK, s, 2);
        } else {
            pair_load_kmajor(sa, &p.map_a, bar, s * p.F_d + i * kBK, tl.row0 + cta * 128, 0);
            pair_load_mnmajor(sb, &p.map_wd, bar, tl.nb * 256 + cta * 128, i * kBK, s, 2);
        }
    }
    // `all_ready` is the calling producer lane's memory of having seen every gate|up tile published (ready_all reached
    // ready_all_target): from then on no phase-1 tile has anything to wait for, and nothing is read.
    __device__ static __forceinline__ bool wait_ready(const Params& p, const Tile& tl, const WaitCtx& w, bool& all_ready) {
        if (tl.phase == 0 || all_ready) return true;
        if (ld_acquire_gpu(p.ready_all) >= p.ready_all_target) {
            all_ready = true;
            fence_proxy_async_all();
            return true;
        }
        const int* flag = p.ready + tl.mt;
        if (ld_acquire_gpu(flag) < p.ready_target) {
            const uint64_t t0 = global_timer_ns();
            while (ld_acquire_gpu(flag) < p.ready_target) {
                if (*w.abort) return false;
                if (global_timer_ns() - t0 > w.limit_ns) {
                    *w.abort = 1u;
                    atomicCAS(w.status, 0, kErrWaitReady);
                    return false;
                }
                __nanosleep(64);
            }
        }
        fence_proxy_async_all();   // the rows were written with ordinary stores; the loads that follow are TMA loads
        return true;
    }
    __device__ static __forceinline__ void epilogue(const Params& p, const Tile& tl, uint32_t cta, int row, uint32_t t_row) {
        const bool live = static_cast<int>(cta) * 128 + row < tl.valid;
        const size_t r = static_cast<size_t>(tl.row0 + cta * 128 + row);
        if (tl.phase == 0) {
            gated_row128(p.A + r * (static_cast<size_t>(p.n_shards) * p.F_d) + static_cast<size_t>(tl.s) * p.F_d + tl.jl * 128,
                         t_row, live, p.act);
        } else {
            const size_t off = r * p.H + tl.nb * 256;
            if (p.carry_tma.epi_off && p.mode != 3) {
                WaitCtx w{&reinterpret_cast<SharedCtl*>(align_1024(dyn_smem()) + p.carry_tma.epi_off)->abort, p.status,
                          p.timeout_ns};
                carry_block_tma(p.carry_tma, w, p.mode, tl.nb * 256, tl.row0 + cta * 128, 0, p.Y + off, t_row, row, live);
            } else {
                carry_row256(p.Yacc + off, p.Y + off, t_row, live, p.mode == 1 || p.mode == 2, p.mode <= 1);
            }
        }
    }
    // After a gate|up tile: every epilogue thread orders its stores of A before later TMA reads, the warp converges,
    // and lane 0 bumps the token tile's counter with release semantics at GPU scope (cumulative over what the warp's
    // lanes stored: they synchronised with lane 0 at the warp barrier).  Four warps per CTA, two CTAs per tile.
    __device__ static __forceinline__ void publish(const Params& p, const Tile& tl) {
        if (tl.phase != 0) return;
        fence_proxy_async_all();
        __syncwarp();
        if ((threadIdx.x & 31) == 0) {
            red_release_gpu_add(p.ready + tl.mt, 1);
            red_release_gpu_add(p.ready_all, 1);
        }
    }
    __device__ static __forceinline__ void prologue(const Params& p, int pair_id) {
        if (pair_id != 0) return;
        for (int i = threadIdx.x - 64; i < p.ready_clear_count; i += kEpilogueThreads) p.ready_clear[i] = 0;
    }
};

}  // namespace tsp
