// Projection GEMMs of TSP attention (Algorithm 1) as policies of the CTA-pair GEMM kernel.
//
//   PairQkvPolicy : [Q | K | V] = X [Wq | Wk | Wv]^T.  One launch covers the three projections of all D shards: shard r
//                   owns heads r*H_s .. (r+1)*H_s - 1, i.e. rows r*Hq/D .. of Wq, so the shards' rows stacked are the
//                   ordinary [Hq, H] matrix and the heads of shard r land in the columns r*Hq/D .. of Q.
//   PairOutPolicy : Y = sum_r A_r Wo^(r)T, accumulated in tensor memory over the D shards in the order of the
//                   algorithm's loop (r = 0..D-1, the same on every rank), one bf16 store of Y.
// Both operands are K-major (the weights are stored with the contraction index contiguous).
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
        const int mt = b_start + rem - nb * b_sz;
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
        const int mt = g_start + rem - o.nb * g_sz;
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

}  // namespace tsp
