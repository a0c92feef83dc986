// Forward kernels of the TSP gated ring MLP (Algorithm 2, loop body):
//   gate_up_swiglu_kernel : A = silu(X Wg_k) * (X Wu_k)  for every (rank r, shard k) pair   [lines "G <- ", "H <- "]
//   down_accumulate_kernel: Y_r = sum over ring steps t of A_{r,k(t)} Wd_{k(t)}, k(t) = (r - t) mod D  ["Y <- Y + ..."]
// Both are persistent, warp-specialised tcgen05 GEMMs: warp 0 issues TMA loads into a ring of
// 128B-swizzled stages, warp 1 issues the MMAs into tensor memory (two accumulator buffers), warps 2-5
// drain the finished accumulator (tcgen05.ld), apply the epilogue and store bf16.
#pragma once
#include "gemm_core.cuh"

namespace tsp {

constexpr int kBM = 128;  // token rows per tile

// ------------------------------------------------------------------------------------------------
// Kernel 1: gate | up GEMM + SwiGLU epilogue.
// Tile = 128 tokens x 128 intermediate columns; one N=256 MMA per k-step over [Wg tile | Wu tile] so
// tensor-memory columns 0..127 hold G and 128..255 hold U.  K = H.
// ------------------------------------------------------------------------------------------------
struct GateUpParams {
    CUtensorMap map_x;   // X  as (H, S, 1),    box (64, 128, 1)   K-major A operand
    CUtensorMap map_wg;  // Wg as (F/D, H, D),  box (64, 64, 1)    MN-major B operand
    CUtensorMap map_wu;  // Wu likewise
    __nv_bfloat16* A;    // [S, F] bf16 intermediate
    int S, H, F, D, S_loc;
    int m_blocks;        // D * blocks_per_rank
    int blocks_per_rank; // ceil((S/D) / 128): the last block of a rank may be partial
    int jl_blocks;       // (F/D) / 128
    int band;            // token blocks per band (their X rows stay L2-resident while the shards stream)
    int shared_order;    // 0: ranks of a band follow the ring (different shards at a time); 1: same column block for all
    int act;             // gate activation (kActSilu / kActGelu / kActRelu)
    int num_tiles;
    int stages;
    int* status;
    unsigned long long timeout_ns;
};

struct GateUpTile {
    int mb, r, k, jl, row0, valid;
};

// Tile order: band of token blocks -> ring step t -> column block jl of the shard -> token block.
// Within a band, every rank is at the same ring step and therefore on a different shard, as in the ring.
__device__ __forceinline__ GateUpTile gate_up_tile(const GateUpParams& p, int tile) {
    const int per_band = p.band * p.D * p.jl_blocks;
    const int band_idx = tile / per_band;
    const int band_start = band_idx * p.band;
    const int band_sz = min(p.band, p.m_blocks - band_start);
    int rem = tile - band_idx * per_band;
    const int t = rem / (p.jl_blocks * band_sz);
    rem -= t * p.jl_blocks * band_sz;
    GateUpTile o;
    o.jl = rem / band_sz;
    o.mb = band_start + rem % band_sz;
    token_tile(o.mb, p.blocks_per_rank, p.S_loc, kBM, o.r, o.row0, o.valid);
    o.k = p.shared_order ? t : (o.r - t + p.D) % p.D;
    return o;
}

__global__ void __launch_bounds__(kNumThreads, 1) gate_up_swiglu_kernel(const __grid_constant__ GateUpParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_1024(smem_raw);
    constexpr uint32_t kABytes = kBM * 128, kBBytes = 256 * 128, kStageBytes = kABytes + kBBytes;
    SharedCtl* ctl = reinterpret_cast<SharedCtl*>(smem + p.stages * kStageBytes);
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    cta_setup(ctl, p.stages, 2, kEpilogueThreads);
    const uint32_t tmem_base = ctl->tmem_base;
    WaitCtx w{&ctl->abort, p.status, p.timeout_ns};
    const int k_blocks = p.H / kBK;

    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&p.map_x);
            tma_prefetch_desc(&p.map_wg);
            tma_prefetch_desc(&p.map_wu);
            PipeState ps;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x) {
                const GateUpTile tl = gate_up_tile(p, tile);
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!(ok = wait_bar(smem_u32(&ctl->empty[ps.stage]), ps.phase ^ 1u, w, kErrWaitEmpty))) break;
                    const uint32_t bar = smem_u32(&ctl->full[ps.stage]);
                    const uint32_t sa = smem_base + ps.stage * kStageBytes, sb = sa + kABytes;
                    ctl->issued[ps.stage] = 1u + ps.phase;
                    mbar_arrive_expect_tx(bar, kStageBytes);
                    load_kmajor(sa, &p.map_x, bar, kb * kBK, tl.row0, 0);
                    load_mnmajor(sb, &p.map_wg, bar, tl.jl * 128, kb * kBK, tl.k, 2);
                    load_mnmajor(sb + 2 * 8192, &p.map_wu, bar, tl.jl * 128, kb * kBK, tl.k, 2);
                    ps.advance(p.stages);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(128, 256, false, true);
            PipeState ps;
            bool ok = true;
            int it = 0;
            for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++it) {
                const int buf = it & 1;
                const uint32_t acc_phase = (it >> 1) & 1;
                if (!(ok = wait_bar(smem_u32(&ctl->tmem_empty[buf]), acc_phase ^ 1u, w, kErrWaitTmemEmpty))) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * 256;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!(ok = wait_bar(smem_u32(&ctl->full[ps.stage]), ps.phase, w, kErrWaitFull))) break;
                    tc_fence_after_sync();
                    const uint32_t sa = smem_base + ps.stage * kStageBytes, sb = sa + kABytes;
                    issue_kblock<false, true>(d_tmem, sa, sb, idesc, kb > 0);
                    umma_commit(smem_u32(&ctl->empty[ps.stage]));
                    ps.advance(p.stages);
                }
                if (ok) umma_commit(smem_u32(&ctl->tmem_full[buf]));
            }
        }
    } else {
        const int quarter = warp & 3;  // tensor-memory lanes this warp may read
        const int row = quarter * 32 + lane;
        bool ok = true;
        int it = 0;
        for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++it) {
            const GateUpTile tl = gate_up_tile(p, tile);
            const int buf = it & 1;
            const uint32_t acc_phase = (it >> 1) & 1;
            if (!(ok = wait_bar(smem_u32(&ctl->tmem_full[buf]), acc_phase, w, kErrWaitTmemFull))) break;
            tc_fence_after_sync();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * 256;
            const bool live = row < tl.valid;   // rows past the rank's end are not stored
            __nv_bfloat16* out = p.A + static_cast<size_t>(tl.row0 + row) * p.F +
                                 static_cast<size_t>(tl.k) * (p.F / p.D) + tl.jl * 128;
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
                    const float a0 = gate_act(g0, p.act) * __uint_as_float(u[2 * i]);
                    const float a1 = gate_act(g1, p.act) * __uint_as_float(u[2 * i + 1]);
                    packed[i] = pack_bf16x2(a0, a1);
                }
                uint4* dst = reinterpret_cast<uint4*>(out + c * 32);
                if (live) {
#pragma unroll
                    for (int q = 0; q < 4; ++q)
                        dst[q] = make_uint4(packed[4 * q], packed[4 * q + 1], packed[4 * q + 2], packed[4 * q + 3]);
                }
            }
            tc_fence_before_sync();
            mbar_arrive(smem_u32(&ctl->tmem_empty[buf]));
        }
    }
    cta_teardown(ctl, p.stages, w);
}

// ------------------------------------------------------------------------------------------------
// Kernel 2: down projection, accumulated in tensor memory over all D shards in ring order.
// Tile = 128 tokens x 256 hidden columns; K = F, walked shard by shard: k = (r - t) mod D, t = 0..D-1.
// ------------------------------------------------------------------------------------------------
struct DownParams {
    CUtensorMap map_a;   // A  as (F, S, 1), box (64, 128, 1)   K-major A operand
    CUtensorMap map_wd;  // Wd as (H, F, 1), box (64, 64, 1)    MN-major B operand ([D][F/D][H] is [F][H])
    __nv_bfloat16* Y;    // [S, H]
    int S, H, F, D, S_loc;
    int m_blocks, n_blocks;  // D * blocks_per_rank, H/256
    int blocks_per_rank;
    int group;               // token blocks per tile group (share Wd column blocks in L2)
    int num_tiles;
    int stages;
    int* status;
    unsigned long long timeout_ns;
};

struct DownTile {
    int mb, nb, r, row0, valid;
};

__device__ __forceinline__ DownTile down_tile(const DownParams& p, int tile) {
    const int per_group = p.group * p.n_blocks;
    const int g = tile / per_group;
    const int g_start = g * p.group;
    const int g_sz = min(p.group, p.m_blocks - g_start);
    const int rem = tile - g * per_group;
    DownTile o;
    o.nb = rem / g_sz;
    o.mb = g_start + rem % g_sz;
    token_tile(o.mb, p.blocks_per_rank, p.S_loc, kBM, o.r, o.row0, o.valid);
    return o;
}

__global__ void __launch_bounds__(kNumThreads, 1) down_accumulate_kernel(const __grid_constant__ DownParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_1024(smem_raw);
    constexpr uint32_t kABytes = kBM * 128, kBBytes = 256 * 128, kStageBytes = kABytes + kBBytes;
    SharedCtl* ctl = reinterpret_cast<SharedCtl*>(smem + p.stages * kStageBytes);
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    cta_setup(ctl, p.stages, 2, kEpilogueThreads);
    const uint32_t tmem_base = ctl->tmem_base;
    WaitCtx w{&ctl->abort, p.status, p.timeout_ns};
    const int F_d = p.F / p.D;
    const int kb_per_shard = F_d / kBK;

    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&p.map_a);
            tma_prefetch_desc(&p.map_wd);
            PipeState ps;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x) {
                const DownTile tl = down_tile(p, tile);
                for (int t = 0; t < p.D && ok; ++t) {
                    const int k = (tl.r - t + p.D) % p.D;  // shard held at ring step t
                    for (int kb = 0; kb < kb_per_shard; ++kb) {
                        if (!(ok = wait_bar(smem_u32(&ctl->empty[ps.stage]), ps.phase ^ 1u, w, kErrWaitEmpty))) break;
                        const uint32_t bar = smem_u32(&ctl->full[ps.stage]);
                        const uint32_t sa = smem_base + ps.stage * kStageBytes, sb = sa + kABytes;
                        const int f0 = k * F_d + kb * kBK;
                        ctl->issued[ps.stage] = 1u + ps.phase;
                        mbar_arrive_expect_tx(bar, kStageBytes);
                        load_kmajor(sa, &p.map_a, bar, f0, tl.row0, 0);
                        load_mnmajor(sb, &p.map_wd, bar, tl.nb * 256, f0, 0, 4);
                        ps.advance(p.stages);
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(128, 256, false, true);
            PipeState ps;
            bool ok = true;
            int it = 0;
            const int k_blocks = p.D * kb_per_shard;
            for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++it) {
                const int buf = it & 1;
                const uint32_t acc_phase = (it >> 1) & 1;
                if (!(ok = wait_bar(smem_u32(&ctl->tmem_empty[buf]), acc_phase ^ 1u, w, kErrWaitTmemEmpty))) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * 256;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!(ok = wait_bar(smem_u32(&ctl->full[ps.stage]), ps.phase, w, kErrWaitFull))) break;
                    tc_fence_after_sync();
                    const uint32_t sa = smem_base + ps.stage * kStageBytes, sb = sa + kABytes;
                    issue_kblock<false, true>(d_tmem, sa, sb, idesc, kb > 0);
                    umma_commit(smem_u32(&ctl->empty[ps.stage]));
                    ps.advance(p.stages);
                }
                if (ok) umma_commit(smem_u32(&ctl->tmem_full[buf]));
            }
        }
    } else {
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        bool ok = true;
        int it = 0;
        for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++it) {
            const DownTile tl = down_tile(p, tile);
            const int buf = it & 1;
            const uint32_t acc_phase = (it >> 1) & 1;
            if (!(ok = wait_bar(smem_u32(&ctl->tmem_full[buf]), acc_phase, w, kErrWaitTmemFull))) break;
            tc_fence_after_sync();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * 256;
            const bool live = row < tl.valid;
            __nv_bfloat16* out = p.Y + static_cast<size_t>(tl.row0 + row) * p.H + tl.nb * 256;
#pragma unroll 1
            for (int c = 0; c < 8; ++c) {
                uint32_t v[32];
                tmem_ld32(t_row + c * 32, v);
                tmem_ld_wait();
                uint4* dst = reinterpret_cast<uint4*>(out + c * 32);
                if (live) {
#pragma unroll
                    for (int q = 0; q < 4; ++q) {
                        dst[q] = make_uint4(
                            pack_bf16x2(__uint_as_float(v[8 * q + 0]), __uint_as_float(v[8 * q + 1])),
                            pack_bf16x2(__uint_as_float(v[8 * q + 2]), __uint_as_float(v[8 * q + 3])),
                            pack_bf16x2(__uint_as_float(v[8 * q + 4]), __uint_as_float(v[8 * q + 5])),
                            pack_bf16x2(__uint_as_float(v[8 * q + 6]), __uint_as_float(v[8 * q + 7])));
                    }
                }
            }
            tc_fence_before_sync();
            mbar_arrive(smem_u32(&ctl->tmem_empty[buf]));
        }
    }
    cta_teardown(ctl, p.stages, w);
}

}  // namespace tsp
