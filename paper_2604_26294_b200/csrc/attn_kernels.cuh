// Projection GEMMs of TSP attention (Algorithm 1) as policies of the CTA-pair GEMM kernel.
//
//   PairQkvPolicy : [Q | K | V] = X [Wq | Wk | Wv]^T.  One launch covers the three projections of all D shards: shard r
//                   owns heads r*H_s .. (r+1)*H_s - 1, i.e. rows r*Hq/D .. of Wq, so the shards' rows stacked are the
//                   ordinary [Hq, H] matrix and the heads of shard r land in the columns r*Hq/D .. of Q.
//   PairOutPolicy : Y = sum_r A_r Wo^(r)T, accumulated in tensor memory over the D shards in the order of the
//                   algorithm's loop (r = 0..D-1, the same on every rank), one bf16 store of Y.
// Both operands are K-major (the weights are stored with the contraction index contiguous).
// Backward: PairAttnDxPolicy (dX = dQ Wq + dK Wk + dV Wv), PairAttnDaPolicy (dA = dY Wo) and PairAttnDwPolicy (all
// weight gradients, contracted over the tokens of all ranks: the sum-to-owner of the partial gradients).
#pragma once
#include "pair_kernels.cuh"

namespace tsp {

// ---- Q, K, V projections: tile = 256 tokens x 256 output features of one of the three matrices -----------------
struct PairQkvPolicy {
    static constexpr bool kAMn = false, kBMn = false;
    struct Params {
        CUtensorMap map_x, map_wq, map_wk, map_wv;  // (H, S, 1) box (64,128); (H, rows, 1) box (64,128) each
        __nv_bfloat16* Q;   // [S, Hq]
        __nv_bfloat16* K;   // [S, Hkv]
        __nv_bfloat16* V;   // [S, Hkv]
        int S, H, Hq, Hkv;
        int m_tiles, q_blocks, kv_blocks, n_blocks, band;
        int mt_base;        // first token tile of this launch (long problems are cut into several launches)
        int* sched;   // dynamic tile hand-out: {next list index, leaders done} in global memory (unused by the static kernels)
        int num_tiles, stages;
        int* status;
        unsigned long long timeout_ns;
    };
    struct Tile {
        int row0, valid, which, cb;
    };
    __device__ static __forceinline__ int outer(const Params&) { return 1; }
    __device__ static __forceinline__ int inner(const Params& p) { return p.H / kBK; }
    __device__ static __forceinline__ int select(const Params&, const Tile&, int) { return 0; }
    __device__ static __forceinline__ void prefetch(const Params& p) {
        tma_prefetch_desc(&p.map_x);
        tma_prefetch_desc(&p.map_wq);
        tma_prefetch_desc(&p.map_wk);
        tma_prefetch_desc(&p.map_wv);
    }
    // Bands of token tiles whose rows of X stay in L2; inside a band the weight block is the slow index, so that a
    // 256-row block of a weight matrix is read once per band.
    __device__ static __forceinline__ Tile decode(const Params& p, int tile) {
        const int per_band = p.band * p.n_blocks;
        const int b = tile / per_band;
        const int b_start = b * p.band;
        const int b_sz = min(p.band, p.m_tiles - b_start);
        const int rem = tile - b * per_band;
        const int nb = rem / b_sz;
        const int mt = p.mt_base + b_start + rem - nb * b_sz;
        Tile o;
        o.row0 = mt * 256;
        o.valid = min(256, p.S - o.row0);
        if (nb < p.q_blocks) {
            o.which = 0;
            o.cb = nb;
        } else if (nb < p.q_blocks + p.kv_blocks) {
            o.which = 1;
            o.cb = nb - p.q_blocks;
        } else {
            o.which = 2;
            o.cb = nb - p.q_blocks - p.kv_blocks;
        }
        return o;
    }
    __device__ static __forceinline__ void load(const Params& p, const Tile& tl, int, int i, uint32_t cta, uint32_t sa,
                                                uint32_t sb, uint32_t bar) {
        const CUtensorMap* mw = tl.which == 0 ? &p.map_wq : (tl.which == 1 ? &p.map_wk : &p.map_wv);
        pair_load_kmajor(sa, &p.map_x, bar, i * kBK, tl.row0 + cta * 128, 0);
        pair_load_kmajor(sb, mw, bar, i * kBK, tl.cb * 256 + cta * 128, 0);
    }
    __device__ static __forceinline__ void epilogue(const Params& p, const Tile& tl, uint32_t cta, int row, uint32_t t_row) {
        __nv_bfloat16* out = tl.which == 0 ? p.Q : (tl.which == 1 ? p.K : p.V);
        const int width = tl.which == 0 ? p.Hq : p.Hkv;
        store_bf16_row256(out + static_cast<size_t>(tl.row0 + cta * 128 + row) * width + tl.cb * 256, t_row,
                          static_cast<int>(cta) * 128 + row < tl.valid);
    }
};

// ---- output projection: tile = 256 tokens x 256 hidden; K = Hq, taken shard by shard -----------------------------
struct PairOutPolicy {
    static constexpr bool kAMn = false, kBMn = false;
    struct Params {
        CUtensorMap map_a, map_wo;  // A (Hq, S, 1) box (64,128); Wo (Hq/D, H, D) box (64,128)
        __nv_bfloat16* Y;           // [S, H]
        int S, H, Hq, D, Hq_d;
        int m_tiles, n_blocks, group;
        int mt_base;
        int* sched;   // dynamic tile hand-out: {next list index, leaders done} in global memory (unused by the static kernels)
        int num_tiles, stages;
        int* status;
        unsigned long long timeout_ns;
    };
    struct Tile {
        int row0, valid, nb;
    };
    __device__ static __forceinline__ int outer(const Params& p) { return p.D; }
    __device__ static __forceinline__ int inner(const Params& p) { return p.Hq_d / kBK; }
    __device__ static __forceinline__ int select(const Params&, const Tile&, int t) { return t; }  // r = 0..D-1
    __device__ static __forceinline__ void prefetch(const Params& p) {
        tma_prefetch_desc(&p.map_a);
        tma_prefetch_desc(&p.map_wo);
    }
    // groups of token tiles share the pass over the hidden blocks, as in the down projection
    __device__ static __forceinline__ Tile decode(const Params& p, int tile) {
        const int per_group = p.group * p.n_blocks;
        const int g = tile / per_group;
        const int g_start = g * p.group;
        const int g_sz = min(p.group, p.m_tiles - g_start);
        const int rem = tile - g * per_group;
        Tile o;
        o.nb = rem / g_sz;
        const int mt = p.mt_base + g_start + rem - o.nb * g_sz;
        o.row0 = mt * 256;
        o.valid = min(256, p.S - o.row0);
        return o;
    }
    __device__ static __forceinline__ void load(const Params& p, const Tile& tl, int r, int i, uint32_t cta, uint32_t sa,
                                                uint32_t sb, uint32_t bar) {
        pair_load_kmajor(sa, &p.map_a, bar, r * p.Hq_d + i * kBK, tl.row0 + cta * 128, 0);
        pair_load_kmajor(sb, &p.map_wo, bar, i * kBK, tl.nb * 256 + cta * 128, r);
    }
    __device__ static __forceinline__ void epilogue(const Params& p, const Tile& tl, uint32_t cta, int row, uint32_t t_row) {
        store_bf16_row256(p.Y + static_cast<size_t>(tl.row0 + cta * 128 + row) * p.H + tl.nb * 256, t_row,
                          static_cast<int>(cta) * 128 + row < tl.valid);
    }
};

// ---- backward of the Q/K/V projections: dX = dQ Wq + dK Wk + dV Wv; tile = 256 tokens x 256 hidden ----------------
// One K loop over the concatenated features [Hq | Hkv | Hkv]; the weights are read as they are stored ([features][H],
// i.e. MN-major for this product).
struct PairAttnDxPolicy {
    static constexpr bool kAMn = false, kBMn = true;
    struct Params {
        CUtensorMap map_dq, map_dk, map_dv;  // (width, S, 1) box (64,128)
        CUtensorMap map_wq, map_wk, map_wv;  // (H, width, 1) box (64,64)
        __nv_bfloat16* dX;                   // [S, H]
        int S, H, q_kb, kv_kb;               // k-blocks of 64 features per matrix
        int m_tiles, n_blocks, group;
        int mt_base;
        int* sched;   // dynamic tile hand-out: {next list index, leaders done} in global memory (unused by the static kernels)
        int num_tiles, stages;
        int* status;
        unsigned long long timeout_ns;
    };
    using Tile = PairOutPolicy::Tile;
    __device__ static __forceinline__ int outer(const Params&) { return 1; }
    __device__ static __forceinline__ int inner(const Params& p) { return p.q_kb + 2 * p.kv_kb; }
    __device__ static __forceinline__ int select(const Params&, const Tile&, int) { return 0; }
    __device__ static __forceinline__ void prefetch(const Params& p) {
        tma_prefetch_desc(&p.map_dq);
        tma_prefetch_desc(&p.map_dk);
        tma_prefetch_desc(&p.map_dv);
        tma_prefetch_desc(&p.map_wq);
        tma_prefetch_desc(&p.map_wk);
        tma_prefetch_desc(&p.map_wv);
    }
    __device__ static __forceinline__ Tile decode(const Params& p, int tile) {
        const int per_group = p.group * p.n_blocks;
        const int g = tile / per_group;
        const int g_start = g * p.group;
        const int g_sz = min(p.group, p.m_tiles - g_start);
        const int rem = tile - g * per_group;
        Tile o;
        o.nb = rem / g_sz;
        const int mt = p.mt_base + g_start + rem - o.nb * g_sz;
        o.row0 = mt * 256;
        o.valid = min(256, p.S - o.row0);
        return o;
    }
    __device__ static __forceinline__ void load(const Params& p, const Tile& tl, int, int i, uint32_t cta, uint32_t sa,
                                                uint32_t sb, uint32_t bar) {
        const CUtensorMap* ma;
        const CUtensorMap* mw;
        int kk = i;
        if (kk < p.q_kb) {
            ma = &p.map_dq; mw = &p.map_wq;
        } else if ((kk -= p.q_kb) < p.kv_kb) {
            ma = &p.map_dk; mw = &p.map_wk;
        } else {
            kk -= p.kv_kb;
            ma = &p.map_dv; mw = &p.map_wv;
        }
        pair_load_kmajor(sa, ma, bar, kk * kBK, tl.row0 + cta * 128, 0);
        pair_load_mnmajor(sb, mw, bar, tl.nb * 256 + cta * 128, kk * kBK, 0, 2);
    }
    __device__ static __forceinline__ void epilogue(const Params& p, const Tile& tl, uint32_t cta, int row, uint32_t t_row) {
        store_bf16_row256(p.dX + static_cast<size_t>(tl.row0 + cta * 128 + row) * p.H + tl.nb * 256, t_row,
                          static_cast<int>(cta) * 128 + row < tl.valid);
    }
};

// ---- backward of the output projection, activations: dA = dY Wo; tile = 256 tokens x 256 head columns ------------
// Column c of dA belongs to shard c / (Hq/D); a 64-column chunk never straddles two shards ((Hq/D) % 64 == 0).
struct PairAttnDaPolicy {
    static constexpr bool kAMn = false, kBMn = true;
    struct Params {
        CUtensorMap map_dy, map_wo;  // dY (H, S, 1) box (64,128); Wo (Hq/D, H, D) box (64,64)
        __nv_bfloat16* dA;           // [S, Hq]
        int S, H, Hq, Hq_d;
        int m_tiles, n_blocks, band;
        int mt_base;
        int* sched;   // dynamic tile hand-out: {next list index, leaders done} in global memory (unused by the static kernels)
        int num_tiles, stages;
        int* status;
        unsigned long long timeout_ns;
    };
    struct Tile {
        int row0, valid, nb;
        int r0, j0, r1, j1, r2, j2, r3, j3;  // shard and column inside the shard of the tile's four 64-column chunks
    };
    __device__ static __forceinline__ int outer(const Params&) { return 1; }
    __device__ static __forceinline__ int inner(const Params& p) { return p.H / kBK; }
    __device__ static __forceinline__ int select(const Params&, const Tile&, int) { return 0; }
    __device__ static __forceinline__ void prefetch(const Params& p) {
        tma_prefetch_desc(&p.map_dy);
        tma_prefetch_desc(&p.map_wo);
    }
    __device__ static __forceinline__ Tile decode(const Params& p, int tile) {
        const int per_band = p.band * p.n_blocks;
        const int b = tile / per_band;
        const int b_start = b * p.band;
        const int b_sz = min(p.band, p.m_tiles - b_start);
        const int rem = tile - b * per_band;
        Tile o;
        o.nb = rem / b_sz;
        const int mt = p.mt_base + b_start + rem - o.nb * b_sz;
        o.row0 = mt * 256;
        o.valid = min(256, p.S - o.row0);
        const int c = o.nb * 256;
        o.r0 = c / p.Hq_d;          o.j0 = c - o.r0 * p.Hq_d;
        o.r1 = (c + 64) / p.Hq_d;   o.j1 = c + 64 - o.r1 * p.Hq_d;
        o.r2 = (c + 128) / p.Hq_d;  o.j2 = c + 128 - o.r2 * p.Hq_d;
        o.r3 = (c + 192) / p.Hq_d;  o.j3 = c + 192 - o.r3 * p.Hq_d;
        return o;
    }
    __device__ static __forceinline__ void load(const Params& p, const Tile& tl, int, int i, uint32_t cta, uint32_t sa,
                                                uint32_t sb, uint32_t bar) {
        pair_load_kmajor(sa, &p.map_dy, bar, i * kBK, tl.row0 + cta * 128, 0);
        tma_load_3d_pair(sb, &p.map_wo, bar, cta ? tl.j2 : tl.j0, i * kBK, cta ? tl.r2 : tl.r0);
        tma_load_3d_pair(sb + 8192, &p.map_wo, bar, cta ? tl.j3 : tl.j1, i * kBK, cta ? tl.r3 : tl.r1);
    }
    __device__ static __forceinline__ void epilogue(const Params& p, const Tile& tl, uint32_t cta, int row, uint32_t t_row) {
        store_bf16_row256(p.dA + static_cast<size_t>(tl.row0 + cta * 128 + row) * p.Hq + tl.nb * 256, t_row,
                          static_cast<int>(cta) * 128 + row < tl.valid);
    }
};

// ---- weight gradients of both projections: C_f = M_f^T N over ALL tokens (the sum-to-owner), fp32 -----------------
// Up to three families f share the N operand.  qkv: M_f = dQ, dK, dV, N = X, C_f = dWq, dWk, dWv [features][H].
// output projection: M = dY, N = A, C = dWo stored shard by shard, [D][H][Hq/D].  Tile = 256 rows of C x 256 columns;
// the K loop runs over the tokens in ascending order, the tail k-block zero-filled by the TMA unit.
struct PairAttnDwPolicy {
    static constexpr bool kAMn = true, kBMn = true;
    struct Params {
        CUtensorMap map_m0, map_m1, map_m2, map_n;  // (rows of C, S, 1) and (columns of C, S, 1), boxes (64,64)
        float* out0;
        float* out1;
        float* out2;
        int m_tiles0, m_tiles1, m_tiles2;  // 256-row tiles of C per family (0 = family absent)
        int rows0;                         // rows of C of family 0 (needed for the sharded layout)
        int N;                             // columns of C
        int shard_w;                       // 0: C row-major [rows][N]; else C stored as [N / shard_w][rows][shard_w]
        int accumulate;                    // 0: C overwritten; 1: the tile's sum is added to what C holds
        int S, k_blocks;
        int n_blocks, n_group;
        int* sched;   // dynamic tile hand-out: {next list index, leaders done} in global memory (unused by the static kernels)
        int num_tiles, stages;
        int* status;
        unsigned long long timeout_ns;
    };
    struct Tile {
        int which, jt, nb;
    };
    __device__ static __forceinline__ int outer(const Params&) { return 1; }
    __device__ static __forceinline__ int inner(const Params& p) { return p.k_blocks; }
    __device__ static __forceinline__ int select(const Params&, const Tile&, int) { return 0; }
    __device__ static __forceinline__ void prefetch(const Params& p) {
        tma_prefetch_desc(&p.map_m0);
        tma_prefetch_desc(&p.map_n);
    }
    // group of column blocks (their columns of N stay in L2) -> row tile over all families -> column block of the group
    __device__ static __forceinline__ Tile decode(const Params& p, int tile) {
        const int rows_all = p.m_tiles0 + p.m_tiles1 + p.m_tiles2;
        const int per_group = rows_all * p.n_group;
        const int g = tile / per_group;
        const int g_start = g * p.n_group;
        const int g_sz = min(p.n_group, p.n_blocks - g_start);
        const int rem = tile - g * per_group;
        int rt = rem / g_sz;
        Tile o;
        o.nb = g_start + rem - rt * g_sz;
        if (rt < p.m_tiles0) {
            o.which = 0;
        } else if ((rt -= p.m_tiles0) < p.m_tiles1) {
            o.which = 1;
        } else {
            rt -= p.m_tiles1;
            o.which = 2;
        }
        o.jt = rt;
        return o;
    }
    __device__ static __forceinline__ void load(const Params& p, const Tile& tl, int, int i, uint32_t cta, uint32_t sa,
                                                uint32_t sb, uint32_t bar) {
        const CUtensorMap* mm = tl.which == 0 ? &p.map_m0 : (tl.which == 1 ? &p.map_m1 : &p.map_m2);
        pair_load_mnmajor(sa, mm, bar, tl.jt * 256 + cta * 128, i * kBK, 0, 2);
        pair_load_mnmajor(sb, &p.map_n, bar, tl.nb * 256 + cta * 128, i * kBK, 0, 2);
    }
    __device__ static __forceinline__ void epilogue(const Params& p, const Tile& tl, uint32_t cta, int row, uint32_t t_row) {
        float* out = tl.which == 0 ? p.out0 : (tl.which == 1 ? p.out1 : p.out2);
        const int j = tl.jt * 256 + cta * 128 + row;  // row of C
#pragma unroll 1
        for (int c = 0; c < 8; ++c) {
            uint32_t v[32];
            tmem_ld32(t_row + c * 32, v);
            tmem_ld_wait();
            const int col = tl.nb * 256 + c * 32;
            float* dst;
            if (p.shard_w == 0) {
                dst = out + static_cast<size_t>(j) * p.N + col;
            } else {
                const int r = col / p.shard_w;
                dst = out + (static_cast<size_t>(r) * p.rows0 + j) * p.shard_w + (col - r * p.shard_w);
            }
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
        }
    }
};

}  // namespace tsp
