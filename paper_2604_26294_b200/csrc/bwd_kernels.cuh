// Backward kernels of the TSP gated ring MLP.  The backward pass mirrors the forward weight
// movement; every rank produces partial gradients for each shard it meets and they are summed to
// the shard's owner (Sections 4.3.4, 4.7).  With all ranks on one GPU that sum is the contraction
// over all S tokens.
//
//   bwd_gate_kernel : per (rank r, shard k) tile: recompute G = X Wg_k, U = X Wu_k, dA = dY Wd_k^T;
//                     emit A = silu(G)*U, dG = dA*U*silu'(G), dU = dA*silu(G) as bf16
//   bwd_dx_kernel   : dX_r = sum over ring steps of dG_{r,k} Wg_k^T + dU_{r,k} Wu_k^T   (bf16 out)
//   bwd_dw_kernel   : dWd_k = sum_r A_{r,k}^T dY_r, dWg_k = sum_r X_r^T dG_{r,k}, dWu_k likewise (fp32 out)
#pragma once
#include "gemm_core.cuh"

namespace tsp {

__device__ __forceinline__ void tmem_ld16(uint32_t taddr, uint32_t (&r)[16]) {
    asm volatile(
        "tcgen05.ld.sync.aligned.32x32b.x16.b32 "
        "{%0, %1, %2, %3, %4, %5, %6, %7, %8, %9, %10, %11, %12, %13, %14, %15}, [%16];"
        : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
          "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
        : "r"(taddr)
        : "memory");
}

// ------------------------------------------------------------------------------------------------
// bwd_gate_kernel.  Tile = 128 tokens x 128 intermediate columns of one (r, k) pair.
// Tensor memory: columns 0..255 hold G | U (one slot), columns 256..383 / 384..511 hold dA (two slots,
// alternating per tile), so the dA loop of the next tile runs while the epilogue drains this one.
// ------------------------------------------------------------------------------------------------
struct BwdGateParams {
    CUtensorMap map_x;    // X  (H, S, 1)     box (64, 128)  K-major A operand
    CUtensorMap map_dy;   // dY (H, S, 1)     box (64, 128)  K-major A operand
    CUtensorMap map_wg;   // Wg (F/D, H, D)   box (64, 64)   MN-major B operand
    CUtensorMap map_wu;   // Wu likewise
    CUtensorMap map_wd;   // Wd (H, F, 1)     box (64, 128)  K-major B operand (rows = intermediate index)
    __nv_bfloat16* A;     // [S, F]
    __nv_bfloat16* dG;    // [S, F]
    __nv_bfloat16* dU;    // [S, F]
    int S, H, F, D, S_loc;
    int m_blocks, blocks_per_rank, jl_blocks, band, num_tiles, stages;
    int act;              // gate activation
    int* status;
    unsigned long long timeout_ns;
};

struct BwdGateTile {
    int mb, r, k, jl, row0, valid;
};

__device__ __forceinline__ BwdGateTile bwd_gate_tile(const BwdGateParams& p, int tile) {
    const int per_band = p.band * p.D * p.jl_blocks;
    const int band_idx = tile / per_band;
    const int band_start = band_idx * p.band;
    const int band_sz = min(p.band, p.m_blocks - band_start);
    int rem = tile - band_idx * per_band;
    const int t = rem / (p.jl_blocks * band_sz);
    rem -= t * p.jl_blocks * band_sz;
    BwdGateTile o;
    o.jl = rem / band_sz;
    o.mb = band_start + rem % band_sz;
    token_tile(o.mb, p.blocks_per_rank, p.S_loc, 128, o.r, o.row0, o.valid);
    o.k = (o.r - t + p.D) % p.D;
    return o;
}

__global__ void __launch_bounds__(kNumThreads, 1) bwd_gate_kernel(const __grid_constant__ BwdGateParams p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_1024(smem_raw);
    constexpr uint32_t kABytes = 128 * 128, kStageBytes = 48 * 1024;
    constexpr uint32_t kBytesDA = kABytes + 128 * 128, kBytesGU = kABytes + 256 * 128;
    SharedCtl* ctl = reinterpret_cast<SharedCtl*>(smem + p.stages * kStageBytes);
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    cta_setup(ctl, p.stages, 3, kEpilogueThreads);
    const uint32_t tmem_base = ctl->tmem_base;
    WaitCtx w{&ctl->abort, p.status, p.timeout_ns};
    const int k_blocks = p.H / kBK;
    const int F_d = p.F / p.D;

    if (warp == 0) {
        if (lane == 0) {
            tma_prefetch_desc(&p.map_x);
            tma_prefetch_desc(&p.map_dy);
            tma_prefetch_desc(&p.map_wg);
            tma_prefetch_desc(&p.map_wu);
            tma_prefetch_desc(&p.map_wd);
            PipeState ps;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x) {
                const BwdGateTile tl = bwd_gate_tile(p, tile);
                for (int kb = 0; kb < 2 * k_blocks; ++kb) {
                    if (!(ok = wait_bar(smem_u32(&ctl->empty[ps.stage]), ps.phase ^ 1u, w, kErrWaitEmpty))) break;
                    const uint32_t bar = smem_u32(&ctl->full[ps.stage]);
                    const uint32_t sa = smem_base + ps.stage * kStageBytes, sb = sa + kABytes;
                    ctl->issued[ps.stage] = 1u + ps.phase;
                    if (kb < k_blocks) {  // dA = dY Wd_k^T
                        mbar_arrive_expect_tx(bar, kBytesDA);
                        load_kmajor(sa, &p.map_dy, bar, kb * kBK, tl.row0, 0);
                        load_kmajor(sb, &p.map_wd, bar, kb * kBK, tl.k * F_d + tl.jl * 128, 0);
                    } else {              // G | U = X [Wg_k | Wu_k]
                        const int h0 = (kb - k_blocks) * kBK;
                        mbar_arrive_expect_tx(bar, kBytesGU);
                        load_kmajor(sa, &p.map_x, bar, h0, tl.row0, 0);
                        load_mnmajor(sb, &p.map_wg, bar, tl.jl * 128, h0, tl.k, 2);
                        load_mnmajor(sb + 2 * 8192, &p.map_wu, bar, tl.jl * 128, h0, tl.k, 2);
                    }
                    ps.advance(p.stages);
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc_da = make_idesc_bf16(128, 128, false, false);
            constexpr uint32_t idesc_gu = make_idesc_bf16(128, 256, false, true);
            PipeState ps;
            bool ok = true;
            int it = 0;
            for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++it) {
                const int slot = it & 1;
                if (!(ok = wait_bar(smem_u32(&ctl->tmem_empty[slot]), ((it >> 1) & 1) ^ 1u, w, kErrWaitTmemEmpty))) break;
                tc_fence_after_sync();
                const uint32_t d_da = tmem_base + 256 + slot * 128;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!(ok = wait_bar(smem_u32(&ctl->full[ps.stage]), ps.phase, w, kErrWaitFull))) break;
                    tc_fence_after_sync();
                    const uint32_t sa = smem_base + ps.stage * kStageBytes, sb = sa + kABytes;
                    issue_kblock<false, false>(d_da, sa, sb, idesc_da, kb > 0);
                    umma_commit(smem_u32(&ctl->empty[ps.stage]));
                    ps.advance(p.stages);
                }
                if (!ok) break;
                if (!(ok = wait_bar(smem_u32(&ctl->tmem_empty[2]), (it & 1) ^ 1u, w, kErrWaitTmemEmpty))) break;
                tc_fence_after_sync();
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!(ok = wait_bar(smem_u32(&ctl->full[ps.stage]), ps.phase, w, kErrWaitFull))) break;
                    tc_fence_after_sync();
                    const uint32_t sa = smem_base + ps.stage * kStageBytes, sb = sa + kABytes;
                    issue_kblock<false, true>(tmem_base, sa, sb, idesc_gu, kb > 0);
                    umma_commit(smem_u32(&ctl->empty[ps.stage]));
                    ps.advance(p.stages);
                }
                if (ok) umma_commit(smem_u32(&ctl->tmem_full[slot]));
            }
        }
    } else {
        const int quarter = warp & 3;
        const int row = quarter * 32 + lane;
        bool ok = true;
        int it = 0;
        for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++it) {
            const BwdGateTile tl = bwd_gate_tile(p, tile);
            const int slot = it & 1;
            if (!(ok = wait_bar(smem_u32(&ctl->tmem_full[slot]), (it >> 1) & 1, w, kErrWaitTmemFull))) break;
            tc_fence_after_sync();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16);
            const bool live = row < tl.valid;
            const size_t off = static_cast<size_t>(tl.row0 + row) * p.F + static_cast<size_t>(tl.k) * F_d + tl.jl * 128;
#pragma unroll 1
            for (int c = 0; c < 8; ++c) {
                uint32_t g[16], u[16], da[16];
                tmem_ld16(t_row + c * 16, g);
                tmem_ld16(t_row + 128 + c * 16, u);
                tmem_ld16(t_row + 256 + slot * 128 + c * 16, da);
                tmem_ld_wait();
                uint32_t pa[8], pg[8], pu[8];
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    float va[2], vg[2], vu[2];
#pragma unroll
                    for (int e = 0; e < 2; ++e) {
                        const float gg = __uint_as_float(g[2 * i + e]);
                        const float uu = __uint_as_float(u[2 * i + e]);
                        const float dd = __uint_as_float(da[2 * i + e]);
                        float sg, ds;
                        gate_act_grad(gg, p.act, sg, ds);              // sigma(G), sigma'(G)
                        va[e] = sg * uu;                               // A
                        vu[e] = dd * sg;                               // dU = dA * sigma(G)
                        vg[e] = dd * uu * ds;                          // dG = dA * U * sigma'(G)
                    }
                    pa[i] = pack_bf16x2(va[0], va[1]);
                    pg[i] = pack_bf16x2(vg[0], vg[1]);
                    pu[i] = pack_bf16x2(vu[0], vu[1]);
                }
                uint4* oa = reinterpret_cast<uint4*>(p.A + off + c * 16);
                uint4* og = reinterpret_cast<uint4*>(p.dG + off + c * 16);
                uint4* ou = reinterpret_cast<uint4*>(p.dU + off + c * 16);
                if (live) {
                    oa[0] = make_uint4(pa[0], pa[1], pa[2], pa[3]);
                    oa[1] = make_uint4(pa[4], pa[5], pa[6], pa[7]);
                    og[0] = make_uint4(pg[0], pg[1], pg[2], pg[3]);
                    og[1] = make_uint4(pg[4], pg[5], pg[6], pg[7]);
                    ou[0] = make_uint4(pu[0], pu[1], pu[2], pu[3]);
                    ou[1] = make_uint4(pu[4], pu[5], pu[6], pu[7]);
                }
            }
            tc_fence_before_sync();
            mbar_arrive(smem_u32(&ctl->tmem_empty[2]));
            mbar_arrive(smem_u32(&ctl->tmem_empty[slot]));
        }
    }
    cta_teardown(ctl, p.stages, w);
}

// ------------------------------------------------------------------------------------------------
// Generic 128 x 256 tile GEMM with one K loop and two accumulator buffers; the policy supplies
// the tile decode, the operand loads of k-block `kb` and the store of one 32-column chunk.
// ------------------------------------------------------------------------------------------------
template <class Policy>
__global__ void __launch_bounds__(kNumThreads, 1) tile_gemm_kernel(const __grid_constant__ typename Policy::Params p) {
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = align_1024(smem_raw);
    constexpr uint32_t kABytes = 128 * 128, kBBytes = 256 * 128, kStageBytes = kABytes + kBBytes;
    SharedCtl* ctl = reinterpret_cast<SharedCtl*>(smem + p.stages * kStageBytes);
    const uint32_t smem_base = smem_u32(smem);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    cta_setup(ctl, p.stages, 2, kEpilogueThreads);
    const uint32_t tmem_base = ctl->tmem_base;
    WaitCtx w{&ctl->abort, p.status, p.timeout_ns};
    // The K loop is outer() x inner() k-blocks; the shard (or rank) of an outer step is chosen once, so the producer's
    // per-k-block path has no integer division.
    const int n_outer = Policy::outer(p), n_inner = Policy::inner(p);
    const int k_blocks = n_outer * n_inner;

    if (warp == 0) {
        if (lane == 0) {
            Policy::prefetch(p);
            PipeState ps;
            bool ok = true;
            for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x) {
                const typename Policy::Tile tl = Policy::decode(p, tile);
                for (int o = 0; o < n_outer && ok; ++o) {
                    const int sel = Policy::select(p, tl, o);
                    for (int i = 0; i < n_inner; ++i) {
                        if (!(ok = wait_bar(smem_u32(&ctl->empty[ps.stage]), ps.phase ^ 1u, w, kErrWaitEmpty))) break;
                        const uint32_t bar = smem_u32(&ctl->full[ps.stage]);
                        const uint32_t sa = smem_base + ps.stage * kStageBytes, sb = sa + kABytes;
                        ctl->issued[ps.stage] = 1u + ps.phase;
                        mbar_arrive_expect_tx(bar, kStageBytes);
                        Policy::load(p, tl, sel, i, sa, sb, bar);
                        ps.advance(p.stages);
                    }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            constexpr uint32_t idesc = make_idesc_bf16(128, 256, Policy::kAMn, Policy::kBMn);
            PipeState ps;
            bool ok = true;
            int it = 0;
            for (int tile = blockIdx.x; tile < p.num_tiles && ok; tile += gridDim.x, ++it) {
                const int buf = it & 1;
                if (!(ok = wait_bar(smem_u32(&ctl->tmem_empty[buf]), ((it >> 1) & 1) ^ 1u, w, kErrWaitTmemEmpty))) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + buf * 256;
                for (int kb = 0; kb < k_blocks; ++kb) {
                    if (!(ok = wait_bar(smem_u32(&ctl->full[ps.stage]), ps.phase, w, kErrWaitFull))) break;
                    tc_fence_after_sync();
                    const uint32_t sa = smem_base + ps.stage * kStageBytes, sb = sa + kABytes;
                    issue_kblock<Policy::kAMn, Policy::kBMn>(d_tmem, sa, sb, idesc, kb > 0);
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
            const typename Policy::Tile tl = Policy::decode(p, tile);
            const int buf = it & 1;
            if (!(ok = wait_bar(smem_u32(&ctl->tmem_full[buf]), (it >> 1) & 1, w, kErrWaitTmemFull))) break;
            tc_fence_after_sync();
            const uint32_t t_row = tmem_base + (static_cast<uint32_t>(quarter * 32) << 16) + buf * 256;
#pragma unroll 1
            for (int c = 0; c < 8; ++c) {
                uint32_t v[32];
                tmem_ld32(t_row + c * 32, v);
                tmem_ld_wait();
                Policy::store(p, tl, row, c, v);
            }
            tc_fence_before_sync();
            mbar_arrive(smem_u32(&ctl->tmem_empty[buf]));
        }
    }
    cta_teardown(ctl, p.stages, w);
}

// ---- dX = sum_k dG_k Wg_k^T + dU_k Wu_k^T ---------------------------------------------------------
struct BwdDxPolicy {
    static constexpr bool kAMn = false, kBMn = false;
    struct Params {
        CUtensorMap map_dg;  // dG (F, S, 1)     box (64, 128)   K-major A operand
        CUtensorMap map_du;  // dU likewise
        CUtensorMap map_wg;  // Wg (F/D, H, D)   box (64, 256)   K-major B operand (rows = hidden index)
        CUtensorMap map_wu;  // Wu likewise
        __nv_bfloat16* dX;   // [S, H]
        int S, H, F, D, S_loc, F_d;
        int m_blocks, n_blocks, blocks_per_rank, group, num_tiles, stages;
        int* status;
        unsigned long long timeout_ns;
    };
    struct Tile {
        int mb, nb, r, row0, valid;
    };
    __device__ static __forceinline__ int outer(const Params& p) { return p.D; }
    __device__ static __forceinline__ int inner(const Params& p) { return 2 * (p.F_d / kBK); }
    // shard held at ring step t: k = (r - t) mod D
    __device__ static __forceinline__ int select(const Params& p, const Tile& tl, int t) {
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
        const int g_sz = min(p.group, p.m_blocks - g_start);
        const int rem = tile - g * per_group;
        Tile o;
        o.nb = rem / g_sz;
        o.mb = g_start + rem % g_sz;
        token_tile(o.mb, p.blocks_per_rank, p.S_loc, 128, o.r, o.row0, o.valid);
        return o;
    }
    // k-block order: ring step t -> shard k = (r - t) mod D -> 64-wide slice of the shard -> (dG Wg^T, dU Wu^T)
    __device__ static __forceinline__ void load(const Params& p, const Tile& tl, int k, int i, uint32_t sa, uint32_t sb,
                                                uint32_t bar) {
        const int j0 = (i >> 1) * kBK;
        const bool up = i & 1;
        load_kmajor(sa, up ? &p.map_du : &p.map_dg, bar, k * p.F_d + j0, tl.row0, 0);
        load_kmajor(sb, up ? &p.map_wu : &p.map_wg, bar, j0, tl.nb * 256, k);
    }
    __device__ static __forceinline__ void store(const Params& p, const Tile& tl, int row, int c, const uint32_t (&v)[32]) {
        if (row >= tl.valid) return;
        __nv_bfloat16* out = p.dX + static_cast<size_t>(tl.row0 + row) * p.H + tl.nb * 256 + c * 32;
        uint4* dst = reinterpret_cast<uint4*>(out);
#pragma unroll
        for (int q = 0; q < 4; ++q) {
            dst[q] = make_uint4(pack_bf16x2(__uint_as_float(v[8 * q + 0]), __uint_as_float(v[8 * q + 1])),
                                pack_bf16x2(__uint_as_float(v[8 * q + 2]), __uint_as_float(v[8 * q + 3])),
                                pack_bf16x2(__uint_as_float(v[8 * q + 4]), __uint_as_float(v[8 * q + 5])),
                                pack_bf16x2(__uint_as_float(v[8 * q + 6]), __uint_as_float(v[8 * q + 7])));
        }
    }
};

// ---- weight gradients, contraction over all S tokens ------------------------------------------------
// Tile = 128 intermediate columns (tensor-memory lanes) x 256 hidden columns; which = 0: dWd, 1: dWg, 2: dWu.
// dWd[j][h] is stored as is; dWg / dWu tiles are the transpose of the [H][F/D] layout, so each lane writes one
// float per hidden row and a warp covers 32 consecutive floats.
struct BwdDwPolicy {
    static constexpr bool kAMn = true, kBMn = true;
    struct Params {
        CUtensorMap map_a;   // A  (F, S, 1)  box (64, 64)  MN-major A operand
        CUtensorMap map_dg;  // dG likewise
        CUtensorMap map_du;  // dU likewise
        CUtensorMap map_dy;  // dY (H, S, 1)  box (64, 64)  MN-major B operand
        CUtensorMap map_x;   // X  likewise
        float* dWd;          // [D][F/D][H] = [F][H]
        float* dWg;          // [D][H][F/D]
        float* dWu;          // [D][H][F/D]
        int S, H, F, D, S_loc;
        int k_linear;        // 0, or ceil(S / 64) when the tokens are contracted in ascending order (ragged ranks)
        int accumulate;      // 0: dW overwritten; 1: the tile's sum is added to what dW holds
        int j_blocks, n_blocks, num_tiles, stages;
        int* status;
        unsigned long long timeout_ns;
    };
    struct Tile {
        int which, jb, nb, k;
    };
    // rank order r = (k + t) mod D; ascending token order when a 64-token k-block would straddle two ranks
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
        Tile o;
        const int per_which = p.j_blocks * p.n_blocks;
        o.which = tile / per_which;
        const int rem = tile - o.which * per_which;
        o.jb = rem / p.n_blocks;
        o.nb = rem - o.jb * p.n_blocks;
        o.k = o.jb / ((p.F / p.D) / 128);
        return o;
    }
    __device__ static __forceinline__ void load(const Params& p, const Tile& tl, int r, int i, uint32_t sa, uint32_t sb,
                                                uint32_t bar) {
        const int s0 = r * p.S_loc + i * kBK;
        const CUtensorMap* ma = tl.which == 0 ? &p.map_a : (tl.which == 1 ? &p.map_dg : &p.map_du);
        const CUtensorMap* mb = tl.which == 0 ? &p.map_dy : &p.map_x;
        load_mnmajor(sa, ma, bar, tl.jb * 128, s0, 0, 2);
        load_mnmajor(sb, mb, bar, tl.nb * 256, s0, 0, 4);
    }
    __device__ static __forceinline__ void store(const Params& p, const Tile& tl, int row, int c, const uint32_t (&v)[32]) {
        if (tl.which == 0) {
            float4* dst = reinterpret_cast<float4*>(p.dWd + static_cast<size_t>(tl.jb * 128 + row) * p.H + tl.nb * 256 + c * 32);
#pragma unroll
            for (int q = 0; q < 8; ++q) {
                float4 o = make_float4(__uint_as_float(v[4 * q]), __uint_as_float(v[4 * q + 1]),
                                       __uint_as_float(v[4 * q + 2]), __uint_as_float(v[4 * q + 3]));
                if (p.accumulate) {
                    const float4 prev = dst[q];
                    o.x += prev.x; o.y += prev.y; o.z += prev.z; o.w += prev.w;
                }
                dst[q] = o;
            }
        } else {
            const int F_d = p.F / p.D;
            float* base = (tl.which == 1 ? p.dWg : p.dWu) + static_cast<size_t>(tl.k) * p.H * F_d +
                          (tl.jb * 128 - tl.k * F_d) + row;
            const int h0 = tl.nb * 256 + c * 32;
#pragma unroll
            for (int i = 0; i < 32; ++i) {
                float* dst = base + static_cast<size_t>(h0 + i) * F_d;
                *dst = p.accumulate ? __uint_as_float(v[i]) + *dst : __uint_as_float(v[i]);
            }
        }
    }
};

}  // namespace tsp
