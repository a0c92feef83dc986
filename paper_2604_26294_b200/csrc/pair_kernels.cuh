// CTA-pair (tcgen05 cta_group::2) versions of the kernels: two CTAs of a 2-CTA cluster, on the two SMs of a TPC,
// work on one 256-row tile.  Each CTA loads its own 128 rows of the A operand and its own half of the B operand
// (half of N), the leader CTA issues one M=256 MMA per k-step that reads both CTAs' shared memory and writes
// 128 accumulator rows into each CTA's tensor memory.  Per SM this moves 32 KB per k-block instead of 48 KB.
//
// Synchronisation (all mbarriers are bounded-wait):
//   full[s]       leader's only: the leader's producer arrives with the byte count of BOTH CTAs; both CTAs' TMA
//                 loads complete on it (peer loads signal the leader's barrier through the cta_group::2 form).
//   empty[s]      one per CTA: the leader's MMA thread commits to its own and to the peer's (two plain commits).
//   tmem_full[b]  one per CTA, committed by the leader to both.
//   tmem_empty[b] leader's only: 256 arrivals = the epilogue threads of both CTAs (the peer arrives remotely).
// No load in this file names more than one destination CTA.
#pragma once
#include "bwd_kernels.cuh"
#include "fwd_kernels.cuh"

namespace tsp {

// ------------------------------------------------------------------ cluster / pair PTX
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
__device__ __forceinline__ uint32_t map_to_cta(uint32_t smem_addr, uint32_t cta_rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(smem_addr), "r"(cta_rank));
    return r;
}
__device__ __forceinline__ void cluster_sync_all() {
    asm volatile("barrier.cluster.arrive.release.aligned;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire.aligned;" ::: "memory");
}
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// TMA load into this CTA's shared memory; the completion may signal a barrier of the peer CTA.
__device__ __forceinline__ void tma_load_3d_pair(uint32_t smem_dst, const CUtensorMap* map, uint32_t bar_cluster_addr,
                                                 int c0, int c1, int c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.shared::cluster.global.tile.mbarrier::complete_tx::bytes.cta_group::2 "
        "[%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(smem_dst), "l"(map), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2)
        : "memory");
}
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols)
                 : "memory");
}
__device__ __forceinline__ void tmem_relinquish_pair() {
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc,
                                               uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate)
        : "memory");
}
__device__ __forceinline__ void umma_commit_pair(uint32_t bar_cluster_addr) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar_cluster_addr)
                 : "memory");
}

// Timeline probes for development builds (-DTSP_TRACE=2): eight time stamps per CTA pair of the last launch;
// -DTSP_TRACE=1 keeps only kernel entry, last epilogue end and exit (slots 0, 6, 7), which do not touch the MMA lane's loop.
#ifdef TSP_TRACE
__device__ unsigned long long* g_trace = nullptr;
__device__ __forceinline__ void trace_mark(int pair_id, int slot) {
    if (TSP_TRACE < 2 && slot != 0 && slot != 6 && slot != 7) return;
    if (g_trace) g_trace[pair_id * 8 + slot] = global_timer_ns();
}
__device__ __forceinline__ void trace_tile(int pair_id, int it, int k) {
    if (TSP_TRACE < 2) return;
    if (g_trace && it < 16) g_trace[74 * 8 + pair_id * 64 + it * 4 + k] = global_timer_ns();
}
#else
__device__ __forceinline__ void trace_mark(int, int) {}
__device__ __forceinline__ void trace_tile(int, int, int) {}
#endif

// The dynamic shared memory of the running kernel (the kernels declare the same array).
__device__ __forceinline__ uint8_t* dyn_smem() {
    extern __shared__ uint8_t smem_raw[];
    return smem_raw;
}

constexpr uint32_t kPairStageBytes = 32 * 1024;  // per CTA: 128 rows of A (16 KB) + half of B (<= 16 KB)
constexpr uint32_t kPairABytes = 16 * 1024;

__device__ __forceinline__ void pair_load_kmajor(uint32_t smem, const CUtensorMap* map, uint32_t bar, int k0, int row0,
                                                 int z) {
    tma_load_3d_pair(smem, map, bar, k0, row0, z);
}
__device__ __forceinline__ void pair_load_mnmajor(uint32_t smem, const CUtensorMap* map, uint32_t bar, int mn0, int k0,
                                                  int z, int chunks) {
    for (int c = 0; c < chunks; ++c) tma_load_3d_pair(smem + c * 8192, map, bar, mn0 + c * 64, k0, z);
}

template <bool kAMn, bool kBMn>
__device__ __forceinline__ void pair_issue_kblock(uint32_t d_tmem, uint32_t a_smem, uint32_t b_smem, uint32_t idesc,
                                                  bool accumulate_first) {
    const uint64_t a_desc = make_smem_desc_sw128(a_smem, kAMn ? 8192u : 0u, 1024u);
    const uint64_t b_desc = make_smem_desc_sw128(b_smem, kBMn ? 8192u : 0u, 1024u);
    constexpr uint64_t a_step = (kAMn ? 2048u : 32u) >> 4;
    constexpr uint64_t b_step = (kBMn ? 2048u : 32u) >> 4;
#pragma unroll
    for (int kk = 0; kk < kBK / kUmmaK; ++kk)
        umma_bf16_pair(d_tmem, a_desc + kk * a_step, b_desc + kk * b_step, idesc, (accumulate_first || kk > 0) ? 1u : 0u);
}

// All threads of both CTAs call.  n_acc accumulator barrier pairs.
__device__ __forceinline__ void pair_setup(SharedCtl* ctl, int stages, int n_acc) {
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), 1);
            mbar_init(smem_u32(&ctl->empty[s]), 1);
            ctl->issued[s] = 0;
        }
        for (int b = 0; b < n_acc; ++b) {
            mbar_init(smem_u32(&ctl->tmem_full[b]), 1);
            mbar_init(smem_u32(&ctl->tmem_empty[b]), 2 * kEpilogueThreads);
        }
        mbar_init(smem_u32(&ctl->teardown), 1);
        mbar_init(smem_u32(&ctl->epi[0]), 1);
        mbar_init(smem_u32(&ctl->epi[1]), 1);
        ctl->abort = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc_pair(smem_u32(&ctl->tmem_base), kTmemCols);
        tmem_relinquish_pair();
    }
    tc_fence_before_sync();
    cluster_sync_all();
    tc_fence_after_sync();
    // Everything above touched only this CTA's shared and tensor memory, so it may run while the previous kernel of the
    // stream is still finishing (the host launches the pair kernels with programmatic serialisation).  From here on
    // the kernel reads and writes global memory: wait for the previous grid, then let the next one start its own set-up
    // under this kernel's tail.  The trigger comes after the wait, so at most two kernels overlap.
    griddep_wait();
    griddep_launch_dependents();
}

__device__ __forceinline__ void pair_teardown(SharedCtl* ctl, const WaitCtx& w) {
    const int warp = threadIdx.x >> 5;
    tc_fence_before_sync();
    __syncthreads();
    if (*w.abort) {
        // error path: give copies and MMAs still in flight time to land before shared / tensor memory is released
        const uint64_t t0 = global_timer_ns();
        while (global_timer_ns() - t0 < 2000000ull) __nanosleep(1000);
    }
    cluster_sync_all();
    tc_fence_after_sync();
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc_pair(ctl->tmem_base, kTmemCols);
    }
}

// ------------------------------------------------------------------------------------------------
// Generic pair kernel: tile = 256 rows (128 per CTA) x 256 columns, one K loop, two accumulator buffers.
// Policy: Params{num_tiles, stages, status, timeout_ns}; Tile decode(p, tile); the K loop is outer(p) x inner(p)
//         k-blocks with sel = select(p, tile, o) chosen once per outer step (the shard or rank met at that ring step);
//         load(p, tile, sel, i, cta, sa, sb, bar) issues this CTA's TMA loads of one k-block; kAMn / kBMn give the
//         operand majors; epilogue(p, tile, cta, row, t_row) drains one accumulator row.
// ------------------------------------------------------------------------------------------------
template <class Policy>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kNumThreads, 1)
pair_gemm_kernel(const __grid_constant__ typename Policy::Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_1024(smem_raw);
    SharedCtl* ctl = reinterpret_cast<SharedCtl*>(smem + p.stages * kPairStageBytes);
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta = cluster_ctarank();
    const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

    if (threadIdx.x == 0 && cta == 0) trace_mark(pair_id, 0);
    pair_setup(ctl, p.stages, 2);
    if (threadIdx.x == 0 && cta == 0) trace_mark(pair_id, 1);
    const uint32_t tmem_base = ctl->tmem_base;
    WaitCtx w{&ctl->abort, p.status, p.timeout_ns};
    // The K loop is outer() x inner() k-blocks; the policy maps (outer, inner) to coordinates without divisions.
    const int n_outer = Policy::outer(p), n_inner = Policy::inner(p);
    const int k_blocks = n_outer * n_inner;

    if (warp == 0) {
        if (lane == 0) {
            Policy::prefetch(p);
            PipeState ps;
            bool ok = true;
            for (int tile = pair_id; tile < p.num_tiles && ok; tile += n_pairs) {
                const typename Policy::Tile tl = Policy::decode(p, tile);
                for (int o = 0; o < n_outer && ok; ++o) {
                    const int sel = Policy::select(p, tl, o);  // shard (or rank) met at outer step o
                    for (int i = 0; i < n_inner; ++i) {
                        if (!(ok = wait_bar(smem_u32(&ctl->empty[ps.stage]), ps.phase ^ 1u, w, kErrWaitEmpty))) break;
                        const uint32_t bar = map_to_cta(smem_u32(&ctl->full[ps.stage]), 0);
                        const uint32_t sa = smem_base + ps.stage * kPairStageBytes, sb = sa + kPairABytes;
                        if (cta == 0) mbar_arrive_expect_tx(smem_u32(&ctl->full[ps.stage]), 2 * kPairStageBytes);
                        Policy::load(p, tl, sel, i, cta, sa, sb, bar);
                        if (cta == 0 && tile == pair_id && o == 0 && i == 0) trace_mark(pair_id, 2);
                        ps.advance(p.stages);
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && cta == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(256, 256, Policy::kAMn, Policy::kBMn);
            PipeState ps;
            bool ok = true;
            int it = 0;
            for (int tile = pair_id; tile < p.num_tiles && ok; tile += n_pairs, ++it) {
                const int buf = it & 1;
                if (!(ok = wait_bar(smem_u32(&ctl->tmem_empty[buf]), ((it >> 1) & 1) ^ 1u, w, kErrWaitTmemEmpty))) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * 256;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!(ok = wait_bar(smem_u32(&ctl->full[ps.stage]), ps.phase, w, kErrWaitFull))) break;
                    if (it == 0 && kb == 0) trace_mark(pair_id, 3);
                    if (kb == 0) trace_tile(pair_id, it, 0);
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
                    trace_mark(pair_id, 4);
                    trace_tile(pair_id, it, 1);
                }
            }
        }
    } else {
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        bool ok = true;
        int it = 0;
        for (int tile = pair_id; tile < p.num_tiles && ok; tile += n_pairs, ++it) {
            const typename Policy::Tile tl = Policy::decode(p, tile);
            const int buf = it & 1;
            if (!(ok = wait_bar(smem_u32(&ctl->tmem_full[buf]), (it >> 1) & 1, w, kErrWaitTmemFull))) break;
            if (threadIdx.x == 64 && cta == 0) { trace_mark(pair_id, 5); trace_tile(pair_id, it, 2); }
            tc_fence_after_sync();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * 256;
            Policy::epilogue(p, tl, cta, row, t_row);
            tc_fence_before_sync();
            mbar_arrive_cluster(map_to_cta(smem_u32(&ctl->tmem_empty[buf]), 0));
            if (threadIdx.x == 64 && cta == 0) { trace_mark(pair_id, 6); trace_tile(pair_id, it, 3); }
        }
    }
    pair_teardown(ctl, w);
    if (threadIdx.x == 0 && cta == 0) trace_mark(pair_id, 7);
}

// ------------------------------------------------------------------------------------------------
// Mixed-width pair kernel for the long-K GEMMs.  A tile is 256 rows x 512 columns ("wide": ONE accumulator set that
// fills all 512 tensor-memory columns) or 256 x 256 ("narrow": the first 256 columns only).  Per k-block each CTA
// loads 128 rows of A once (16 KB) and one 16 KB half-B block per 256 columns; the leader issues one N = 256 MMA per
// column half, sharing the A descriptor.  A wide tile moves 48 KB instead of 64 KB per CTA pair and 256x256-tile-
// k-block from L2, and a round of 74 wide tiles spans twice the columns, which halves the DRAM re-reads of the row
// operand.  The price: the epilogue no longer overlaps the next main loop (the two column halves are released
// separately, so the first half of the next tile starts early); worth it when K is long.
// The tile list holds `wide_tiles` wide tiles first, then narrow ones that fill the last round, so the 74 pairs
// finish together (e.g. 512 narrow tiles = 3 rounds of wide tiles + 68 narrow tiles).  Tiles are numbered row-major
// over (row tile, 256-column block); a wide tile covers two neighbouring column blocks.
// Policy provides Tile decode_mixed(p, list_index) with Tile::halves and Tile::nb in 256-column units,
// load_wide(p, tile, sel, i, cta, sa, sb, bar) and epilogue_half(p, tile, cta, row, t_row, h).
// ------------------------------------------------------------------------------------------------
constexpr uint32_t kWideStageBytes = 48 * 1024;

// list index -> (row tile, first 256-column block, halves); rows are taken from the last to the first when `reverse`
__device__ __forceinline__ void mixed_tile(int t, int wide_tiles, int n_blocks, int rows, bool reverse, int& row, int& nb,
                                           int& halves) {
    const bool wide = t < wide_tiles;
    const int flat = wide ? 2 * t : 2 * wide_tiles + (t - wide_tiles);
    row = flat / n_blocks;
    nb = flat - row * n_blocks;
    if (reverse) row = rows - 1 - row;
    halves = wide ? 2 : 1;
}

template <class Policy>
__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kNumThreads, 1)
pair_wide_kernel(const __grid_constant__ typename Policy::Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_1024(smem_raw);
    SharedCtl* ctl = reinterpret_cast<SharedCtl*>(smem + p.stages * kWideStageBytes);
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t cta = cluster_ctarank();
    const int pair_id = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

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
            for (int tile = pair_id; tile < p.num_tiles && ok; tile += n_pairs) {
                const typename Policy::Tile tl = Policy::decode_mixed(p, tile);
                const uint32_t bytes = 2u * (kPairABytes + static_cast<uint32_t>(tl.halves) * 16384u);
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
        }
    } else if (warp == 1) {
        if (lane == 0 && cta == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(256, 256, Policy::kAMn, Policy::kBMn);
            PipeState ps;
            bool ok = true;
            uint32_t uses[2] = {0u, 0u};   // how often each column half has been filled so far
            for (int tile = pair_id; tile < p.num_tiles && ok; tile += n_pairs) {
                // the policy decides (its list index may be offset when a long list is cut into several launches)
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
            }
        }
    } else {
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        bool ok = true;
        int it = 0;
        for (int tile = pair_id; tile < p.num_tiles && ok; tile += n_pairs, ++it) {
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

// ---- store helpers ---------------------------------------------------------------------------------
__device__ __forceinline__ void store_bf16_row256(__nv_bfloat16* out, uint32_t t_row, bool live) {
#pragma unroll 1
    for (int c = 0; c < 8; ++c) {
        uint32_t v[32];
        tmem_ld32(t_row + c * 32, v);
        tmem_ld_wait();
        uint32_t pk[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) pk[i] = pack_bf16x2(__uint_as_float(v[2 * i]), __uint_as_float(v[2 * i + 1]));
        if (live) {
            st_global_256(out + c * 32, pk[0], pk[1], pk[2], pk[3], pk[4], pk[5], pk[6], pk[7]);
            st_global_256(out + c * 32 + 16, pk[8], pk[9], pk[10], pk[11], pk[12], pk[13], pk[14], pk[15]);
        }
    }
}

// One accumulator row of 256 columns whose sum is carried from launch to launch in an fp32 buffer (one ring step per
// launch): add_prev reads the carried value and adds it, to_fp32 writes the new partial sum back, otherwise the row is
// rounded once to bf16 into `out`.  Rows that are not live only drain tensor memory.
__device__ __forceinline__ void carry_row256(float* acc_row, __nv_bfloat16* out, uint32_t t_row, bool live, bool add_prev,
                                             bool to_fp32) {
    // Every lane owns one row, so a warp's accesses are 32 separate segments however they are issued; 256-bit accesses
    // halve the number of requests (measured on a one-tile-per-pair step: the fp32 carry took 11 us with 128-bit
    // accesses, longer than the tile's MMAs).  The carried values of chunk c + 1 are requested while chunk c is
    // processed: they do not depend on the accumulator.
    uint32_t nxt[4][8] = {};
    if (live && add_prev) {
#pragma unroll
        for (int q = 0; q < 4; ++q) ld_global_256(acc_row + q * 8, nxt[q]);
    }
#pragma unroll 1
    for (int c = 0; c < 8; ++c) {
        uint32_t prev[4][8];
#pragma unroll
        for (int q = 0; q < 4; ++q)
#pragma unroll
            for (int i = 0; i < 8; ++i) prev[q][i] = nxt[q][i];
        if (live && add_prev && c < 7) {
#pragma unroll
            for (int q = 0; q < 4; ++q) ld_global_256(acc_row + (c + 1) * 32 + q * 8, nxt[q]);
        }
        uint32_t v[32];
        tmem_ld32(t_row + c * 32, v);
        tmem_ld_wait();
        float f[32];
#pragma unroll
        for (int i = 0; i < 32; ++i) f[i] = __uint_as_float(v[i]);
        if (add_prev) {
#pragma unroll
            for (int i = 0; i < 32; ++i) f[i] += __uint_as_float(prev[i >> 3][i & 7]);
        }
        if (!live) continue;
        if (to_fp32) {
#pragma unroll
            for (int q = 0; q < 4; ++q)
                st_global_256(acc_row + c * 32 + q * 8, __float_as_uint(f[8 * q]), __float_as_uint(f[8 * q + 1]),
                              __float_as_uint(f[8 * q + 2]), __float_as_uint(f[8 * q + 3]), __float_as_uint(f[8 * q + 4]),
                              __float_as_uint(f[8 * q + 5]), __float_as_uint(f[8 * q + 6]), __float_as_uint(f[8 * q + 7]));
        } else {
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 16; ++i) pk[i] = pack_bf16x2(f[2 * i], f[2 * i + 1]);
            st_global_256(out + c * 32, pk[0], pk[1], pk[2], pk[3], pk[4], pk[5], pk[6], pk[7]);
            st_global_256(out + c * 32 + 16, pk[8], pk[9], pk[10], pk[11], pk[12], pk[13], pk[14], pk[15]);
        }
    }
}

// The same carried sum with the fp32 traffic done by the TMA unit (one 128-row x 256-column block per CTA).
// A lane owns one accumulator row, so element-wise accesses from registers are 32 scattered segments per warp
// instruction; the carried sums are 1 KB per row in, 1 KB out, and on a step with one tile per CTA pair that epilogue
// took longer than the tile's MMAs.  Here the rows go through two 16 KB staging buffers (128 rows x 32 columns,
// 128-byte swizzle, conflict-free for row-per-lane accesses) after the pipeline stages:
//   kind 0  store:     staging -> global (TMA store)
//   kind 1  add:       staging -> global with an fp32 add performed by the memory system (TMA reduce-add)
//   kind 2  add+round: global -> staging (TMA loads running ahead of their use), accumulator + carried value
//                      rounded once to bf16 and stored from registers
// The tensor map is (H, tokens of one rank, ranks): rows past a rank's end are clipped by the TMA unit on the way out
// and zero-filled on the way in.  `epi_off` is the byte offset of the control block after the pipeline stages; the
// staging buffers follow it at +1024.  Called by the 128 epilogue threads of a CTA together (hardware barrier 1).
struct CarryTma {
    CUtensorMap map;      // fp32 (H, S_loc, ranks), box (32, 128)
    uint32_t epi_off;     // 0: not used (element-wise path)
};

__device__ __forceinline__ void carry_block_tma(const CarryTma& ct, const WaitCtx& w, int kind, int x0, int y0, int z,
                                                __nv_bfloat16* out_row, uint32_t t_row, int row, bool live) {
    uint8_t* base = align_1024(dyn_smem()) + ct.epi_off;
    SharedCtl* ctl = reinterpret_cast<SharedCtl*>(base);
    const uint32_t stage = smem_u32(base + 1024);
    const bool elected = threadIdx.x == 64;
    const uint32_t my_row = static_cast<uint32_t>(row) * 128u, sw = static_cast<uint32_t>(row) & 7u;
    if (kind == 2 && elected) {
#pragma unroll
        for (int b = 0; b < 2; ++b) {
            mbar_arrive_expect_tx(smem_u32(&ctl->epi[b]), 16384u);
            tma_load_3d(stage + b * 16384u, &ct.map, smem_u32(&ctl->epi[b]), x0 + b * 32, y0, z);
        }
    }
#pragma unroll 1
    for (int c = 0; c < 8; ++c) {
        const uint32_t sbuf = stage + static_cast<uint32_t>(c & 1) * 16384u + my_row;
        uint32_t v[32];
        if (kind == 2) {
            // a failed wait has set the status word; control flow stays uniform so that nobody is left at a barrier
            (void)wait_bar(smem_u32(&ctl->epi[c & 1]), static_cast<uint32_t>(c >> 1) & 1u, w, kErrWaitFull);
            uint32_t prev[32];
#pragma unroll
            for (int j = 0; j < 8; ++j)
                ld_shared_v4(sbuf + ((static_cast<uint32_t>(j) ^ sw) << 4), prev[4 * j], prev[4 * j + 1], prev[4 * j + 2],
                             prev[4 * j + 3]);
            named_bar_sync(1, kEpilogueThreads);      // everybody has read this buffer
            if (elected && c + 2 < 8) {
                mbar_arrive_expect_tx(smem_u32(&ctl->epi[c & 1]), 16384u);
                tma_load_3d(stage + static_cast<uint32_t>(c & 1) * 16384u, &ct.map, smem_u32(&ctl->epi[c & 1]),
                            x0 + (c + 2) * 32, y0, z);
            }
            tmem_ld32(t_row + c * 32, v);
            tmem_ld_wait();
            uint32_t pk[16];
#pragma unroll
            for (int i = 0; i < 16; ++i)
                pk[i] = pack_bf16x2(__uint_as_float(v[2 * i]) + __uint_as_float(prev[2 * i]),
                                    __uint_as_float(v[2 * i + 1]) + __uint_as_float(prev[2 * i + 1]));
            if (live) {
                st_global_256(out_row + c * 32, pk[0], pk[1], pk[2], pk[3], pk[4], pk[5], pk[6], pk[7]);
                st_global_256(out_row + c * 32 + 16, pk[8], pk[9], pk[10], pk[11], pk[12], pk[13], pk[14], pk[15]);
            }
        } else {
            if (c >= 2) {   // the transfer that read this buffer two chunks ago has finished reading it
                if (elected) bulk_wait_group_read<1>();
                named_bar_sync(1, kEpilogueThreads);
            }
            tmem_ld32(t_row + c * 32, v);
            tmem_ld_wait();
#pragma unroll
            for (int j = 0; j < 8; ++j)
                st_shared_v4(sbuf + ((static_cast<uint32_t>(j) ^ sw) << 4), v[4 * j], v[4 * j + 1], v[4 * j + 2], v[4 * j + 3]);
            fence_proxy_async_smem();
            named_bar_sync(1, kEpilogueThreads);      // the buffer is complete
            if (elected) {
                const uint32_t src = stage + static_cast<uint32_t>(c & 1) * 16384u;
                if (kind == 0) tma_store_3d(&ct.map, src, x0 + c * 32, y0, z);
                else tma_reduce_add_3d(&ct.map, src, x0 + c * 32, y0, z);
                bulk_commit_group();
            }
        }
    }
    if (kind != 2) {   // both buffers free again before the next block (or the end of the kernel)
        if (elected) bulk_wait_group_read<0>();
        named_bar_sync(1, kEpilogueThreads);
    }
}

// A 128-row x 256-column block of the accumulator written TRANSPOSED (global element [column][row]) by the TMA unit:
// two staging buffers of 32 columns x 128 rows (512-byte lines, no swizzle: for a fixed column the 32 lanes of a warp
// write consecutive words).  kind 0 stores, kind 1 adds.  The tensor map is (rows, columns, shards) with boxes (128, 32).
__device__ __forceinline__ void store_block_tma_transposed(const CUtensorMap* map, uint32_t epi_off, int kind, int x0, int y0,
                                                           int z, uint32_t t_row, int row) {
    const uint32_t stage = smem_u32(align_1024(dyn_smem()) + epi_off + 1024);
    const bool elected = threadIdx.x == 64;
#pragma unroll 1
    for (int c = 0; c < 8; ++c) {
        const uint32_t sbuf = stage + static_cast<uint32_t>(c & 1) * 16384u;
        if (c >= 2) {
            if (elected) bulk_wait_group_read<1>();
            named_bar_sync(1, kEpilogueThreads);
        }
        uint32_t v[32];
        tmem_ld32(t_row + c * 32, v);
        tmem_ld_wait();
#pragma unroll
        for (int i = 0; i < 32; ++i)
            asm volatile("st.shared.b32 [%0], %1;" ::"r"(sbuf + static_cast<uint32_t>(i) * 512u + static_cast<uint32_t>(row) * 4u),
                         "r"(v[i])
                         : "memory");
        fence_proxy_async_smem();
        named_bar_sync(1, kEpilogueThreads);
        if (elected) {
            if (kind == 0) tma_store_3d(map, sbuf, x0, y0 + c * 32, z);
            else tma_reduce_add_3d(map, sbuf, x0, y0 + c * 32, z);
            bulk_commit_group();
        }
    }
    if (elected) bulk_wait_group_read<0>();
    named_bar_sync(1, kEpilogueThreads);
}

// One accumulator row of a gate|up tile: tensor-memory columns 0..127 hold G, 128..255 hold U; writes
// A = act(G) * U for the 128 intermediate columns, rounded once to bf16.  Rows that are not live only drain.
__device__ __forceinline__ void gated_row128(__nv_bfloat16* out, uint32_t t_row, bool live, int act) {
#pragma unroll 1
    for (int c = 0; c < 4; ++c) {
        uint32_t g[32], u[32];
        tmem_ld32(t_row + c * 32, g);
        tmem_ld32(t_row + 128 + c * 32, u);
        tmem_ld_wait();
        uint32_t packed[16];
#pragma unroll
        for (int i = 0; i < 16; ++i) {
            const float g0 = __uint_as_float(g[2 * i]), g1 = __uint_as_float(g[2 * i + 1]);
            packed[i] = pack_bf16x2(gate_act(g0, act) * __uint_as_float(u[2 * i]),
                                    gate_act(g1, act) * __uint_as_float(u[2 * i + 1]));
        }
        if (live) {
            st_global_256(out + c * 32, packed[0], packed[1], packed[2], packed[3], packed[4], packed[5], packed[6],
                          packed[7]);
            st_global_256(out + c * 32 + 16, packed[8], packed[9], packed[10], packed[11], packed[12], packed[13],
                          packed[14], packed[15]);
        }
    }
}

// ---- gate | up + SwiGLU: tile = 256 tokens x 128 intermediate columns; CTA 0 loads the Wg half of B, CTA 1 the Wu half.
// kMode 0 (forward)            : epilogue writes A = sigma(G) * U.
// kMode 1 (backward, recompute): epilogue also reads dA (fp32, from the dA GEMM) and writes A, dG = dA*U*sigma'(G),
//                                dU = dA*sigma(G).
// kMode 2 (forward, storing)   : epilogue writes A and the two factors the backward pass needs, P = U*sigma'(G) and
//                                Q = sigma(G), in bf16 (into p.dG and p.dU), so that no recomputation is needed later.
template <int kMode>
struct PairGateUpPolicyT {
    static constexpr bool kAMn = false, kBMn = true;
    struct Params {
        CUtensorMap map_x, map_wg, map_wu;  // boxes (64,128), (64,64), (64,64)
        __nv_bfloat16* A;
        const float* dA;      // [S, F] fp32 (backward only)
        __nv_bfloat16* dG;    // [S, F] (backward only)
        __nv_bfloat16* dU;    // [S, F] (backward only)
        int S, H, F, D, F_d, S_loc;
        int m_tiles, tiles_per_rank, jl_blocks, band, shared_order;
        int mt_base;          // first token tile of this launch (a long problem is cut into several launches)
        int act;              // gate activation
        int rank_indexed;     // staged mode: one ring step per launch; the weight tensors hold, at index r, the
                              // shard rank r currently has in its receive buffer, and A is [S, F/D]
        int* sched;   // dynamic tile hand-out: {next list index, leaders done} in global memory (unused by the static kernels)
        int num_tiles, stages;
        int* status;
        unsigned long long timeout_ns;
    };
    struct Tile {
        int mt, k, jl, row0, valid;
    };
    __device__ static __forceinline__ int outer(const Params&) { return 1; }
    __device__ static __forceinline__ int inner(const Params& p) { return p.H / kBK; }
    __device__ static __forceinline__ int select(const Params&, const Tile& tl, int) { return tl.k; }
    __device__ static __forceinline__ void prefetch(const Params& p) {
        tma_prefetch_desc(&p.map_x);
        tma_prefetch_desc(&p.map_wg);
        tma_prefetch_desc(&p.map_wu);
    }
    // band of token tiles -> step t -> column block of the shard -> token tile
    __device__ static __forceinline__ Tile decode(const Params& p, int tile) {
        const int steps = p.rank_indexed ? 1 : p.D;
        const int per_band = p.band * steps * p.jl_blocks;
        const int band_idx = tile / per_band;
        const int band_start = band_idx * p.band;
        const int band_sz = min(p.band, p.m_tiles - band_start);
        int rem = tile - band_idx * per_band;
        const int t = rem / (p.jl_blocks * band_sz);
        rem -= t * p.jl_blocks * band_sz;
        Tile o;
        o.jl = rem / band_sz;
        o.mt = p.mt_base + band_start + rem % band_sz;
        int r;
        token_tile(o.mt, p.tiles_per_rank, p.S_loc, 256, r, o.row0, o.valid);
        o.k = p.rank_indexed ? r : (p.shared_order ? t : (r - t + p.D) % p.D);
        return o;
    }
    __device__ static __forceinline__ void load(const Params& p, const Tile& tl, int k, int kb, uint32_t cta,
                                                uint32_t sa, uint32_t sb, uint32_t bar) {
        pair_load_kmajor(sa, &p.map_x, bar, kb * kBK, tl.row0 + cta * 128, 0);
        pair_load_mnmajor(sb, cta == 0 ? &p.map_wg : &p.map_wu, bar, tl.jl * 128, kb * kBK, k, 2);
    }
    __device__ static __forceinline__ void epilogue(const Params& p, const Tile& tl, uint32_t cta, int row, uint32_t t_row) {
        // p.F is the row pitch of A: F in direct mode, F/D in staged mode (where the shard offset is dropped)
        const bool live = static_cast<int>(cta) * 128 + row < tl.valid;   // rows past the rank's end are not stored
        const size_t off = static_cast<size_t>(tl.row0 + cta * 128 + row) * p.F +
                           (p.rank_indexed ? 0 : static_cast<size_t>(tl.k) * p.F_d) + tl.jl * 128;
        if constexpr (kMode == 0) {
            gated_row128(p.A + off, t_row, live, p.act);
        } else if constexpr (kMode == 2) {
#pragma unroll 1
            for (int c = 0; c < 8; ++c) {
                uint32_t g[16], u[16];
                tmem_ld16(t_row + c * 16, g);
                tmem_ld16(t_row + 128 + c * 16, u);
                tmem_ld_wait();
                uint32_t pa[8], pp[8], pq[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    float va[2], vp[2], vq[2];
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const float gg = __uint_as_float(g[2 * i + e]);
                        const float uu = __uint_as_float(u[2 * i + e]);
                        float sg, ds;
                        gate_act_grad(gg, p.act, sg, ds);
                        va[e] = sg * uu;   // A
                        vp[e] = uu * ds;   // P = U * sigma'(G)
                        vq[e] = sg;        // Q = sigma(G)
                    }
                    pa[i] = pack_bf16x2(va[0], va[1]);
                    pp[i] = pack_bf16x2(vp[0], vp[1]);
                    pq[i] = pack_bf16x2(vq[0], vq[1]);
                }
                if (live) {
                    st_global_256(p.A + off + c * 16, pa[0], pa[1], pa[2], pa[3], pa[4], pa[5], pa[6], pa[7]);
                    st_global_256(p.dG + off + c * 16, pp[0], pp[1], pp[2], pp[3], pp[4], pp[5], pp[6], pp[7]);
                    st_global_256(p.dU + off + c * 16, pq[0], pq[1], pq[2], pq[3], pq[4], pq[5], pq[6], pq[7]);
                }
            }
        } else {
            const float* da_row = p.dA + off;
#pragma unroll 1
            for (int c = 0; c < 8; ++c) {
                uint32_t da4[2][8] = {};
                if (live) {
                    ld_global_nc_256(da_row + c * 16, da4[0]);       // issued before the tensor-memory loads
                    ld_global_nc_256(da_row + c * 16 + 8, da4[1]);
                }
                uint32_t g[16], u[16];
                tmem_ld16(t_row + c * 16, g);
                tmem_ld16(t_row + 128 + c * 16, u);
                tmem_ld_wait();
                uint32_t pa[8], pg[8], pu[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    float va[2], vg[2], vu[2];
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const float gg = __uint_as_float(g[2 * i + e]);
                        const float uu = __uint_as_float(u[2 * i + e]);
                        const float dd = __uint_as_float(da4[(2 * i + e) >> 3][(2 * i + e) & 7]);
                        float sg, ds;
                        gate_act_grad(gg, p.act, sg, ds);                   // sigma(G), sigma'(G)
                        va[e] = sg * uu;                                    // A
                        vu[e] = dd * sg;                                    // dU = dA * sigma(G)
                        vg[e] = dd * uu * ds;                               // dG = dA * U * sigma'(G)
                    }
                    pa[i] = pack_bf16x2(va[0], va[1]);
                    pg[i] = pack_bf16x2(vg[0], vg[1]);
                    pu[i] = pack_bf16x2(vu[0], vu[1]);
                }
                if (live) {
                    st_global_256(p.A + off + c * 16, pa[0], pa[1], pa[2], pa[3], pa[4], pa[5], pa[6], pa[7]);
                    st_global_256(p.dG + off + c * 16, pg[0], pg[1], pg[2], pg[3], pg[4], pg[5], pg[6], pg[7]);
                    st_global_256(p.dU + off + c * 16, pu[0], pu[1], pu[2], pu[3], pu[4], pu[5], pu[6], pu[7]);
                }
            }
        }
    }
};
using PairGateUpPolicy = PairGateUpPolicyT<0>;
using PairGateBwdPolicy = PairGateUpPolicyT<1>;
using PairGateSavePolicy = PairGateUpPolicyT<2>;

// ---- dA = dY Wd^T: tile = 256 tokens x 256 intermediate columns; K = H ------------------------------------
// kSaved = false: dA is written in fp32 (the gate|up GEMM of the recomputing backward consumes it).
// kSaved = true : the forward pass stored P = U*sigma'(G) and Q = sigma(G); the epilogue forms dG = dA*P and
//                 dU = dA*Q in fp32 and writes them in bf16, so dA never leaves tensor memory.
template <bool kSaved>
struct PairDaPolicyT {
    static constexpr bool kAMn = false, kBMn = false;
    struct Params {
        CUtensorMap map_dy, map_wd;  // (H, S, 1) box (64,128); (H, F, 1) box (64,128)
        float* dA;                   // [S, F] fp32 (kSaved = false)
        const __nv_bfloat16* P;      // [S, F] (kSaved = true)
        const __nv_bfloat16* Q;      // [S, F]
        __nv_bfloat16* dG;           // [S, F]
        __nv_bfloat16* dU;           // [S, F]
        int S, H, F, D, S_loc;
        int m_tiles, tiles_per_rank, j_tiles, band;
        int j_tiles_per_shard;       // 0: Wd is one [F, H] matrix; n > 0: the map's third coordinate is the shard, each
                                     // shard holding n tiles of 256 rows (packed shard buffers of a ring-step group)
        int mt_base;                 // first token tile of this launch
        int* sched;   // dynamic tile hand-out: {next list index, leaders done} in global memory (unused by the static kernels)
        int num_tiles, stages;
        int* status;
        unsigned long long timeout_ns;
    };
    struct Tile {
        int mt, jt, row0, valid, wz, wrow;   // wz, wrow: shard and first row inside it of the tile's 256 rows of Wd
    };
    __device__ static __forceinline__ int outer(const Params&) { return 1; }
    __device__ static __forceinline__ int inner(const Params& p) { return p.H / kBK; }
    __device__ static __forceinline__ int select(const Params&, const Tile&, int) { return 0; }
    __device__ static __forceinline__ void prefetch(const Params& p) {
        tma_prefetch_desc(&p.map_dy);
        tma_prefetch_desc(&p.map_wd);
    }
    // band of token tiles -> intermediate tile -> token tile (the dY rows of a band stay in L2 while Wd streams)
    __device__ static __forceinline__ Tile decode(const Params& p, int tile) {
        const int per_band = p.band * p.j_tiles;
        const int band_idx = tile / per_band;
        const int band_start = band_idx * p.band;
        const int band_sz = min(p.band, p.m_tiles - band_start);
        const int rem = tile - band_idx * per_band;
        Tile o;
        o.jt = rem / band_sz;
        o.mt = p.mt_base + band_start + rem % band_sz;
        int r;
        token_tile(o.mt, p.tiles_per_rank, p.S_loc, 256, r, o.row0, o.valid);
        o.wz = p.j_tiles_per_shard ? o.jt / p.j_tiles_per_shard : 0;
        o.wrow = (o.jt - o.wz * p.j_tiles_per_shard) * 256;
        return o;
    }
    __device__ static __forceinline__ void load(const Params& p, const Tile& tl, int, int kb, uint32_t cta, uint32_t sa,
                                                uint32_t sb, uint32_t bar) {
        pair_load_kmajor(sa, &p.map_dy, bar, kb * kBK, tl.row0 + cta * 128, 0);
        pair_load_kmajor(sb, &p.map_wd, bar, kb * kBK, tl.wrow + cta * 128, tl.wz);
    }
    __device__ static __forceinline__ void epilogue(const Params& p, const Tile& tl, uint32_t cta, int row, uint32_t t_row) {
        const bool live = static_cast<int>(cta) * 128 + row < tl.valid;
        const size_t off = static_cast<size_t>(tl.row0 + cta * 128 + row) * p.F + tl.jt * 256;
        if constexpr (!kSaved) {
            float* dst = p.dA + off;
#pragma unroll 1
            for (int c = 0; c < 8; ++c) {
                uint32_t v[32];
                tmem_ld32(t_row + c * 32, v);
                tmem_ld_wait();
                if (live) {
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        st_global_256(dst + c * 32 + q * 8, v[8 * q], v[8 * q + 1], v[8 * q + 2], v[8 * q + 3], v[8 * q + 4],
                                      v[8 * q + 5], v[8 * q + 6], v[8 * q + 7]);
                }
            }
        } else {
#pragma unroll 1
            for (int c = 0; c < 16; ++c) {
                uint32_t pr[8] = {}, qr[8] = {}, v[16];
                if (live) {
                    ld_global_nc_256(p.P + off + c * 16, pr);   // 16 bf16 each, issued before the tensor-memory load
                    ld_global_nc_256(p.Q + off + c * 16, qr);
                }
                tmem_ld16(t_row + c * 16, v);
                tmem_ld_wait();
                uint32_t og[8], ou[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    // a bf16 pair widens to fp32 by shifting: low half is element 2i, high half element 2i+1
                    const float p0 = __uint_as_float(pr[i] << 16), p1 = __uint_as_float(pr[i] & 0xFFFF0000u);
                    const float q0 = __uint_as_float(qr[i] << 16), q1 = __uint_as_float(qr[i] & 0xFFFF0000u);
                    const float d0 = __uint_as_float(v[2 * i]), d1 = __uint_as_float(v[2 * i + 1]);
                    og[i] = pack_bf16x2(d0 * p0, d1 * p1);   // dG = dA * U * sigma'(G)
                    ou[i] = pack_bf16x2(d0 * q0, d1 * q1);   // dU = dA * sigma(G)
                }
                if (live) {
                    st_global_256(p.dG + off + c * 16, og[0], og[1], og[2], og[3], og[4], og[5], og[6], og[7]);
                    st_global_256(p.dU + off + c * 16, ou[0], ou[1], ou[2], ou[3], ou[4], ou[5], ou[6], ou[7]);
                }
            }
        }
    }
};
using PairDaPolicy = PairDaPolicyT<false>;
using PairDaSavedPolicy = PairDaPolicyT<true>;

// ---- down projection: tile = 256 tokens x 256 hidden; K = F in ring order --------------------------
struct PairDownPolicy {
    static constexpr bool kAMn = false, kBMn = true;
    struct Params {
        CUtensorMap map_a, map_wd;  // boxes (64,128), (64,64)
        __nv_bfloat16* Y;
        int S, H, F, D, F_d, S_loc;
        int m_tiles, n_blocks, tiles_per_rank, group;
        int wide_tiles;   // mixed-width kernel: number of 256 x 512 tiles at the head of the tile list
        int skew_tiles;   // two-rank kernel: number of tall tiles (both ranks of a pair) at the head of the tile list
        int mt_base;  // first token tile of this launch (a long problem is cut into several launches)
        int* sched;   // dynamic tile hand-out: {next list index, leaders done} in global memory (unused by the static kernels)
        int num_tiles, stages;
        int* status;
        unsigned long long timeout_ns;
    };
    struct Tile {
        int mt, nb, r, halves, row0, valid;
    };
    __device__ static __forceinline__ int outer(const Params& p) { return p.D; }
    __device__ static __forceinline__ int inner(const Params& p) { return p.F_d / kBK; }
    // shard held at ring step t: k = (r - t) mod D
    __device__ static __forceinline__ int select(const Params& p, const Tile& tl, int t) {
        const int k = tl.r - t;
        return k < 0 ? k + p.D : k;
    }
    __device__ static __forceinline__ void prefetch(const Params& p) {
        tma_prefetch_desc(&p.map_a);
        tma_prefetch_desc(&p.map_wd);
    }
    __device__ static __forceinline__ Tile decode(const Params& p, int tile) {
        const int per_group = p.group * p.n_blocks;
        const int g = tile / per_group;
        const int g_start = g * p.group;
        const int g_sz = min(p.group, p.m_tiles - g_start);
        const int rem = tile - g * per_group;
        Tile o;
        o.nb = rem / g_sz;
        // token tiles are taken from the last to the first: the producer kernel wrote the last rows most recently,
        // so they are the ones still in L2
        o.mt = p.mt_base + p.m_tiles - 1 - (g_start + rem % g_sz);
        token_tile(o.mt, p.tiles_per_rank, p.S_loc, 256, o.r, o.row0, o.valid);
        return o;
    }
    __device__ static __forceinline__ void load(const Params& p, const Tile& tl, int k, int i, uint32_t cta,
                                                uint32_t sa, uint32_t sb, uint32_t bar) {
        const int f0 = k * p.F_d + i * kBK;
        pair_load_kmajor(sa, &p.map_a, bar, f0, tl.row0 + cta * 128, 0);
        pair_load_mnmajor(sb, &p.map_wd, bar, tl.nb * 256 + cta * 128, f0, 0, 2);
    }
    // the two operands separately (two-rank kernel): `row` is this CTA's first token row
    __device__ static __forceinline__ void load_a(const Params& p, int row, int k, int i, uint32_t, uint32_t sa, uint32_t bar) {
        pair_load_kmajor(sa, &p.map_a, bar, k * p.F_d + i * kBK, row, 0);
    }
    __device__ static __forceinline__ void load_b(const Params& p, int nb, int k, int i, uint32_t cta, uint32_t sb, uint32_t bar) {
        pair_load_mnmajor(sb, &p.map_wd, bar, nb * 256 + cta * 128, k * p.F_d + i * kBK, 0, 2);
    }
    __device__ static __forceinline__ void epilogue(const Params& p, const Tile& tl, uint32_t cta, int row, uint32_t t_row) {
        store_bf16_row256(p.Y + static_cast<size_t>(tl.row0 + cta * 128 + row) * p.H + tl.nb * 256, t_row,
                          static_cast<int>(cta) * 128 + row < tl.valid);
    }
    // mixed-width kernel: tl.nb is the first 256-column block, tl.halves the number of column blocks
    __device__ static __forceinline__ int halves_of(const Params& p, int t) { return t < p.wide_tiles ? 2 : 1; }
    __device__ static __forceinline__ Tile decode_mixed(const Params& p, int t) {
        Tile o;
        mixed_tile(t, p.wide_tiles, p.n_blocks, p.m_tiles, true, o.mt, o.nb, o.halves);
        o.mt += p.mt_base;
        token_tile(o.mt, p.tiles_per_rank, p.S_loc, 256, o.r, o.row0, o.valid);
        return o;
    }
    __device__ static __forceinline__ void load_wide(const Params& p, const Tile& tl, int k, int i, uint32_t cta,
                                                     uint32_t sa, uint32_t sb, uint32_t bar) {
        const int f0 = k * p.F_d + i * kBK;
        pair_load_kmajor(sa, &p.map_a, bar, f0, tl.row0 + cta * 128, 0);
        for (int h = 0; h < tl.halves; ++h)
            pair_load_mnmajor(sb + h * 16384, &p.map_wd, bar, (tl.nb + h) * 256 + cta * 128, f0, 0, 2);
    }
    __device__ static __forceinline__ void epilogue_half(const Params& p, const Tile& tl, uint32_t cta, int row,
                                                         uint32_t t_row, int h) {
        store_bf16_row256(p.Y + static_cast<size_t>(tl.row0 + cta * 128 + row) * p.H + (tl.nb + h) * 256, t_row,
                          static_cast<int>(cta) * 128 + row < tl.valid);
    }
};

// ---- staged mode, one ring step: Y_acc (fp32) += A_step Wd_cur, K = F/D.  The weights of rank r are read from
// index r of the receive buffer.  mode 0: first step (store), 1: middle (add), 2: last (add, round to bf16 Y),
// 3: only step (D = 1: round to bf16 Y directly).
struct PairDownStagedPolicy {
    static constexpr bool kAMn = false, kBMn = true;
    struct Params {
        CUtensorMap map_a, map_wd;  // A_step (F/D, S, 1) box (64,128); Wd buffers (H, F/D, D) box (64,64)
        float* Yacc;                // [S, H] fp32
        __nv_bfloat16* Y;           // [S, H]
        CarryTma carry_tma;         // Yacc through the TMA unit (epi_off = 0: element-wise accesses instead)
        int S, H, F_d, D, mode, S_loc;
        int n_shards;               // 0: one ring step of every rank (buffer slot = rank).  n > 0: ONE rank, n consecutive
                                    // ring steps in one launch: A is [S, n * F/D], the weight map holds the n shards in
                                    // the order they are met
        int m_tiles, n_blocks, tiles_per_rank, group;
        int* sched;   // dynamic tile hand-out: {next list index, leaders done} in global memory (unused by the static kernels)
        int num_tiles, stages;
        int* status;
        unsigned long long timeout_ns;
    };
    using Tile = PairDownPolicy::Tile;
    __device__ static __forceinline__ int outer(const Params& p) { return p.n_shards > 0 ? p.n_shards : 1; }
    __device__ static __forceinline__ int inner(const Params& p) { return p.F_d / kBK; }
    __device__ static __forceinline__ int select(const Params& p, const Tile& tl, int t) {
        return p.n_shards > 0 ? t : tl.r;
    }
    __device__ static __forceinline__ void prefetch(const Params& p) {
        tma_prefetch_desc(&p.map_a);
        tma_prefetch_desc(&p.map_wd);
    }
    __device__ static __forceinline__ Tile decode(const Params& p, int tile) {
        const int per_group = p.group * p.n_blocks;
        const int g = tile / per_group;
        const int g_start = g * p.group;
        const int g_sz = min(p.group, p.m_tiles - g_start);
        const int rem = tile - g * per_group;
        Tile o;
        o.nb = rem / g_sz;
        // token tiles are taken from the last to the first: the producer kernel wrote the last rows most recently,
        // so they are the ones still in L2
        o.mt = p.m_tiles - 1 - (g_start + rem % g_sz);
        token_tile(o.mt, p.tiles_per_rank, p.S_loc, 256, o.r, o.row0, o.valid);
        return o;
    }
    __device__ static __forceinline__ void load(const Params& p, const Tile& tl, int r, int i, uint32_t cta, uint32_t sa,
                                                uint32_t sb, uint32_t bar) {
        pair_load_kmajor(sa, &p.map_a, bar, (p.n_shards > 0 ? r * p.F_d : 0) + i * kBK, tl.row0 + cta * 128, 0);
        pair_load_mnmajor(sb, &p.map_wd, bar, tl.nb * 256 + cta * 128, i * kBK, r, 2);
    }
    __device__ static __forceinline__ void epilogue(const Params& p, const Tile& tl, uint32_t cta, int row, uint32_t t_row) {
        const bool live = static_cast<int>(cta) * 128 + row < tl.valid;
        const size_t off = static_cast<size_t>(tl.row0 + cta * 128 + row) * p.H + tl.nb * 256;
        if (p.carry_tma.epi_off && p.mode != 3) {
            WaitCtx w{&reinterpret_cast<SharedCtl*>(align_1024(dyn_smem()) + p.carry_tma.epi_off)->abort, p.status, p.timeout_ns};
            carry_block_tma(p.carry_tma, w, p.mode, tl.nb * 256, tl.row0 - tl.r * p.S_loc + cta * 128, tl.r, p.Y + off, t_row,
                            row, live);
        } else {
            carry_row256(p.Yacc + off, p.Y + off, t_row, live, p.mode == 1 || p.mode == 2, p.mode <= 1);
        }
    }
};

// ---- dX: tile = 256 tokens x 256 hidden; K = 2F (dG Wg^T then dU Wu^T per 64-slice), ring order ------
struct PairDxPolicy {
    static constexpr bool kAMn = false, kBMn = false;
    struct Params {
        CUtensorMap map_dg, map_du, map_wg, map_wu;  // boxes (64,128) all
        __nv_bfloat16* dX;
        float* dXacc;  // [S, H] fp32 partial sums carried between launches (one ring step per launch), or null
        CarryTma carry_tma;  // dXacc through the TMA unit (epi_off = 0: element-wise accesses instead)
        int carry;     // 0: the launch covers all shards, dX stored directly; 1 first, 2 middle, 3 last step of a carried sum
        int linear_shards;  // 1: ONE rank, the D shards of the maps are the ones it meets, in that order (ring-step group)
        int S, H, F, D, F_d, S_loc;
        int m_tiles, n_blocks, tiles_per_rank, group;
        int wide_tiles;
        int skew_tiles;   // two-rank kernel: number of tall tiles at the head of the tile list
        int mt_base;   // first token tile of this launch
        int* sched;   // dynamic tile hand-out: {next list index, leaders done} in global memory (unused by the static kernels)
        int num_tiles, stages;
        int* status;
        unsigned long long timeout_ns;
    };
    using Tile = PairDownPolicy::Tile;
    __device__ static __forceinline__ int outer(const Params& p) { return p.D; }
    __device__ static __forceinline__ int inner(const Params& p) { return 2 * (p.F_d / kBK); }
    __device__ static __forceinline__ int select(const Params& p, const Tile& tl, int t) {
        if (p.linear_shards) return t;
        const int k = tl.r - t;
        return k < 0 ? k + p.D : k;
    }
    __device__ static __forceinline__ void prefetch(const Params& p) {
        tma_prefetch_desc(&p.map_dg);
        tma_prefetch_desc(&p.map_du);
        tma_prefetch_desc(&p.map_wg);
        tma_prefetch_desc(&p.map_wu);
    }
    __device__ static __forceinline__ Tile decode(const Params& p, int tile) {
        const int per_group = p.group * p.n_blocks;
        const int g = tile / per_group;
        const int g_start = g * p.group;
        const int g_sz = min(p.group, p.m_tiles - g_start);
        const int rem = tile - g * per_group;
        Tile o;
        o.nb = rem / g_sz;
        // token tiles are taken from the last to the first: the producer kernel wrote the last rows most recently,
        // so they are the ones still in L2
        o.mt = p.mt_base + p.m_tiles - 1 - (g_start + rem % g_sz);
        token_tile(o.mt, p.tiles_per_rank, p.S_loc, 256, o.r, o.row0, o.valid);
        return o;
    }
    __device__ static __forceinline__ void load(const Params& p, const Tile& tl, int k, int i, uint32_t cta,
                                                uint32_t sa, uint32_t sb, uint32_t bar) {
        const int j0 = (i >> 1) * kBK;
        const bool up = i & 1;
        pair_load_kmajor(sa, up ? &p.map_du : &p.map_dg, bar, k * p.F_d + j0, tl.row0 + cta * 128, 0);
        pair_load_kmajor(sb, up ? &p.map_wu : &p.map_wg, bar, j0, tl.nb * 256 + cta * 128, k);
    }
    // the two operands separately (two-rank kernel): `row` is this CTA's first token row
    __device__ static __forceinline__ void load_a(const Params& p, int row, int k, int i, uint32_t, uint32_t sa, uint32_t bar) {
        pair_load_kmajor(sa, (i & 1) ? &p.map_du : &p.map_dg, bar, k * p.F_d + (i >> 1) * kBK, row, 0);
    }
    __device__ static __forceinline__ void load_b(const Params& p, int nb, int k, int i, uint32_t cta, uint32_t sb, uint32_t bar) {
        pair_load_kmajor(sb, (i & 1) ? &p.map_wu : &p.map_wg, bar, (i >> 1) * kBK, nb * 256 + cta * 128, k);
    }
    __device__ static __forceinline__ void store_block(const Params& p, const Tile& tl, uint32_t cta, int row,
                                                       uint32_t t_row, int nb) {
        const size_t off = static_cast<size_t>(tl.row0 + cta * 128 + row) * p.H + nb * 256;
        const bool live = static_cast<int>(cta) * 128 + row < tl.valid;
        if (p.carry == 0) {
            store_bf16_row256(p.dX + off, t_row, live);
        } else if (p.carry_tma.epi_off) {
            WaitCtx w{&reinterpret_cast<SharedCtl*>(align_1024(dyn_smem()) + p.carry_tma.epi_off)->abort, p.status, p.timeout_ns};
            carry_block_tma(p.carry_tma, w, p.carry - 1, nb * 256, tl.row0 - tl.r * p.S_loc + cta * 128, tl.r, p.dX + off, t_row,
                            row, live);
        } else {
            carry_row256(p.dXacc + off, p.dX + off, t_row, live, p.carry >= 2, p.carry <= 2);
        }
    }
    __device__ static __forceinline__ void epilogue(const Params& p, const Tile& tl, uint32_t cta, int row, uint32_t t_row) {
        store_block(p, tl, cta, row, t_row, tl.nb);
    }
    __device__ static __forceinline__ int halves_of(const Params& p, int t) { return t < p.wide_tiles ? 2 : 1; }
    __device__ static __forceinline__ Tile decode_mixed(const Params& p, int t) {
        Tile o;
        mixed_tile(t, p.wide_tiles, p.n_blocks, p.m_tiles, true, o.mt, o.nb, o.halves);
        o.mt += p.mt_base;
        token_tile(o.mt, p.tiles_per_rank, p.S_loc, 256, o.r, o.row0, o.valid);
        return o;
    }
    __device__ static __forceinline__ void load_wide(const Params& p, const Tile& tl, int k, int i, uint32_t cta,
                                                     uint32_t sa, uint32_t sb, uint32_t bar) {
        const int j0 = (i >> 1) * kBK;
        const bool up = i & 1;
        const CUtensorMap* mw = up ? &p.map_wu : &p.map_wg;
        pair_load_kmajor(sa, up ? &p.map_du : &p.map_dg, bar, k * p.F_d + j0, tl.row0 + cta * 128, 0);
        for (int h = 0; h < tl.halves; ++h) pair_load_kmajor(sb + h * 16384, mw, bar, j0, (tl.nb + h) * 256 + cta * 128, k);
    }
    __device__ static __forceinline__ void epilogue_half(const Params& p, const Tile& tl, uint32_t cta, int row,
                                                         uint32_t t_row, int h) {
        store_block(p, tl, cta, row, t_row, tl.nb + h);
    }
};

// ---- weight gradients: tile = 256 intermediate columns x 256 hidden; K = all S tokens ------------------
struct PairDwPolicy {
    static constexpr bool kAMn = true, kBMn = true;
    struct Params {
        CUtensorMap map_a, map_dg, map_du, map_dy, map_x;  // boxes (64,64) all
        float* dWd;
        float* dWg;
        float* dWu;
        int S, H, F, D, F_d, S_loc;
        int j_tiles, n_blocks, j_tiles_per_shard;
        int n_group;   // hidden blocks per group: their columns of X / dY stay in L2 while the [S,F] operand streams
        int k_linear;  // 0, or ceil(S / 64) when the token contraction runs in ascending order (ragged ranks)
        int accumulate;  // 0: dW overwritten; 1: the tile's sum is added to what dW holds (partial sums of other ranks)
        long long out_shard_stride;  // elements between consecutive shards' matrices in each of dWd, dWg, dWu (H * F/D when
                                     // the outputs are the contiguous [D][..][..] arrays)
        CarryTma carry_tma;          // dWd (H, F/D, D) through the TMA unit (epi_off = 0: element-wise accesses instead)
        CUtensorMap map_owg, map_owu;  // dWg, dWu (F/D, H, D), boxes (128, 32), written transposed through the TMA unit
        int wide_tiles;
        int tile_base;   // first entry of the tile list this launch covers (a long list is cut into several launches)
        int* sched;   // dynamic tile hand-out: {next list index, leaders done} in global memory (unused by the static kernels)
        int num_tiles, stages;
        int* status;
        unsigned long long timeout_ns;
    };
    struct Tile {
        int which, jt, nb, k, halves;
    };
    // Tokens are contracted rank by rank in the order shard k meets the ranks, r = (k + t) mod D.  When the tokens per
    // rank are not a multiple of the k-block (64) a k-block would straddle two ranks, so the tokens are then taken in
    // plain ascending order, the tail k-block being zero-filled by the TMA unit (p.k_linear = number of k-blocks).
    __device__ static __forceinline__ int outer(const Params& p) { return p.k_linear ? 1 : p.D; }
    __device__ static __forceinline__ int inner(const Params& p) { return p.k_linear ? p.k_linear : p.S_loc / kBK; }
    __device__ static __forceinline__ int select(const Params& p, const Tile& tl, int t) {
        if (p.k_linear) return 0;
        const int r = tl.k + t;
        return r >= p.D ? r - p.D : r;
    }
    __device__ static __forceinline__ void prefetch(const Params& p) {
        tma_prefetch_desc(&p.map_a);
        tma_prefetch_desc(&p.map_dg);
        tma_prefetch_desc(&p.map_du);
        tma_prefetch_desc(&p.map_dy);
        tma_prefetch_desc(&p.map_x);
    }
    __device__ static __forceinline__ Tile decode(const Params& p, int tile) {
        // family (dWd, dWg, dWu) -> group of hidden blocks -> intermediate tile -> hidden block of the group
        tile += p.tile_base;
        Tile o;
        const int per_which = p.j_tiles * p.n_blocks;
        o.which = tile / per_which;
        int rem = tile - o.which * per_which;
        const int per_group = p.j_tiles * p.n_group;
        const int g = rem / per_group;
        const int g_start = g * p.n_group;
        const int g_sz = min(p.n_group, p.n_blocks - g_start);
        rem -= g * per_group;
        o.jt = rem / g_sz;
        o.nb = g_start + rem - o.jt * g_sz;
        o.k = o.jt / p.j_tiles_per_shard;
        return o;
    }
    __device__ static __forceinline__ void load(const Params& p, const Tile& tl, int r, int i, uint32_t cta,
                                                uint32_t sa, uint32_t sb, uint32_t bar) {
        const int s0 = r * p.S_loc + i * kBK;
        const CUtensorMap* ma = tl.which == 0 ? &p.map_a : (tl.which == 1 ? &p.map_dg : &p.map_du);
        const CUtensorMap* mb = tl.which == 0 ? &p.map_dy : &p.map_x;
        pair_load_mnmajor(sa, ma, bar, tl.jt * 256 + cta * 128, s0, 0, 2);
        pair_load_mnmajor(sb, mb, bar, tl.nb * 256 + cta * 128, s0, 0, 2);
    }
    // writes the 256 hidden columns starting at h_base for this lane's intermediate index
    __device__ static __forceinline__ void store_cols(const Params& p, const Tile& tl, uint32_t cta, int row,
                                                      uint32_t t_row, int h_base) {
        const int j = tl.jt * 256 + cta * 128 + row;  // global intermediate index of this lane
        const int F_d = p.F_d;
        if (p.carry_tma.epi_off) {
            const int jl0 = tl.jt * 256 + static_cast<int>(cta) * 128 - tl.k * F_d;   // first row of this CTA inside shard k
            if (tl.which == 0) {
                WaitCtx w{&reinterpret_cast<SharedCtl*>(align_1024(dyn_smem()) + p.carry_tma.epi_off)->abort, p.status,
                          p.timeout_ns};
                carry_block_tma(p.carry_tma, w, p.accumulate ? 1 : 0, h_base, jl0, tl.k, nullptr, t_row, row, true);
            } else {
                store_block_tma_transposed(tl.which == 1 ? &p.map_owg : &p.map_owu, p.carry_tma.epi_off, p.accumulate ? 1 : 0,
                                           jl0, h_base, tl.k, t_row, row);
            }
            return;
        }
#pragma unroll 1
        for (int c = 0; c < 8; ++c) {
            uint32_t v[32];
            tmem_ld32(t_row + c * 32, v);
            tmem_ld_wait();
            const int h0 = h_base + c * 32;
            if (tl.which == 0) {
                float* dst = p.dWd + static_cast<size_t>(tl.k) * p.out_shard_stride + static_cast<size_t>(j - tl.k * F_d) * p.H + h0;
                if (p.accumulate) {
#pragma unroll
                    for (int q = 0; q < 8; ++q) {
                        const float4 prev = *reinterpret_cast<const float4*>(dst + q * 4);
                        v[4 * q] = __float_as_uint(__uint_as_float(v[4 * q]) + prev.x);
                        v[4 * q + 1] = __float_as_uint(__uint_as_float(v[4 * q + 1]) + prev.y);
                        v[4 * q + 2] = __float_as_uint(__uint_as_float(v[4 * q + 2]) + prev.z);
                        v[4 * q + 3] = __float_as_uint(__uint_as_float(v[4 * q + 3]) + prev.w);
                    }
                }
#pragma unroll
                for (int q = 0; q < 4; ++q)
                    st_global_256(dst + q * 8, v[8 * q], v[8 * q + 1], v[8 * q + 2], v[8 * q + 3], v[8 * q + 4], v[8 * q + 5],
                                  v[8 * q + 6], v[8 * q + 7]);
            } else {
                float* base = (tl.which == 1 ? p.dWg : p.dWu) + static_cast<size_t>(tl.k) * p.out_shard_stride + (j - tl.k * F_d);
#pragma unroll
                for (int i = 0; i < 32; ++i) {
                    float* dst = base + static_cast<size_t>(h0 + i) * F_d;
                    *dst = p.accumulate ? __uint_as_float(v[i]) + *dst : __uint_as_float(v[i]);
                }
            }
        }
    }
    __device__ static __forceinline__ void epilogue(const Params& p, const Tile& tl, uint32_t cta, int row, uint32_t t_row) {
        store_cols(p, tl, cta, row, t_row, tl.nb * 256);
    }
    // mixed-width kernel: rows of the tile grid are (family, intermediate tile); the list index is offset by tile_base
    // when a long list is cut into several launches
    __device__ static __forceinline__ int halves_of(const Params& p, int t) { return t + p.tile_base < p.wide_tiles ? 2 : 1; }
    __device__ static __forceinline__ Tile decode_mixed(const Params& p, int t) {
        Tile o;
        int row;
        mixed_tile(t + p.tile_base, p.wide_tiles, p.n_blocks, 3 * p.j_tiles, false, row, o.nb, o.halves);
        o.which = row / p.j_tiles;
        o.jt = row - o.which * p.j_tiles;
        o.k = o.jt / p.j_tiles_per_shard;
        return o;
    }
    __device__ static __forceinline__ void load_wide(const Params& p, const Tile& tl, int r, int i, uint32_t cta,
                                                     uint32_t sa, uint32_t sb, uint32_t bar) {
        const int s0 = r * p.S_loc + i * kBK;
        const CUtensorMap* ma = tl.which == 0 ? &p.map_a : (tl.which == 1 ? &p.map_dg : &p.map_du);
        const CUtensorMap* mb = tl.which == 0 ? &p.map_dy : &p.map_x;
        pair_load_mnmajor(sa, ma, bar, tl.jt * 256 + cta * 128, s0, 0, 2);
        for (int h = 0; h < tl.halves; ++h) pair_load_mnmajor(sb + h * 16384, mb, bar, (tl.nb + h) * 256 + cta * 128, s0, 0, 2);
    }
    __device__ static __forceinline__ void epilogue_half(const Params& p, const Tile& tl, uint32_t cta, int row,
                                                         uint32_t t_row, int h) {
        store_cols(p, tl, cta, row, t_row, (tl.nb + h) * 256);
    }
};

}  // namespace tsp
