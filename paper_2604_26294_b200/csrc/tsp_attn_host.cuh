// C-ABI of the attention projection GEMMs (include/tsp_attn.h).  Included once, at the end of tsp_mlp.cu, because
// it reuses that file's host helpers (tensor-map encoding, pair launch, status word, profiling events).
#pragma once
#include "../../include/tsp_attn.h"
#include "attn_kernels.cuh"

struct tsp_attn_plan {
    tsp_mlp_plan_t* base;  // device-side part shared with the MLP plan: device properties, tensor-map encoder,
                           // status word, profiling events
    int H, Hq, Hkv, D;
};

extern "C" {

tsp_status_t tsp_attn_plan(int H, int Hq, int Hkv, int D, tsp_attn_plan_t** out) {
    if (!out) return TSP_ERR_INVALID_ARG;
    *out = nullptr;
    if (H <= 0 || Hq <= 0 || Hkv <= 0 || D <= 0 || D > 64) return TSP_ERR_INVALID_ARG;
    if (H % 256 != 0 || Hq % 256 != 0 || Hkv % 256 != 0) return TSP_ERR_UNSUPPORTED_SHAPE;
    if (Hq % D != 0 || Hkv % D != 0 || (Hq / D) % 64 != 0) return TSP_ERR_UNSUPPORTED_SHAPE;
    if (H > (1 << 20) || Hq > (1 << 20) || Hkv > (1 << 20)) return TSP_ERR_UNSUPPORTED_SHAPE;
    tsp_mlp_plan_t* base = nullptr;
    tsp_status_t st = make_plan(H, 0, 1, nullptr, &base);  // device-side part only; the MLP fields stay unused
    if (st != TSP_OK) return st;
    tsp_attn_plan_t* plan = new (std::nothrow) tsp_attn_plan_t();
    if (!plan) {
        tsp_mlp_plan_destroy(base);
        return TSP_ERR_INVALID_ARG;
    }
    plan->base = base;
    plan->H = H; plan->Hq = Hq; plan->Hkv = Hkv; plan->D = D;
    *out = plan;
    return TSP_OK;
}

tsp_status_t tsp_attn_plan_destroy(tsp_attn_plan_t* plan) {
    if (!plan) return TSP_ERR_INVALID_ARG;
    tsp_mlp_plan_destroy(plan->base);
    delete plan;
    return TSP_OK;
}

tsp_status_t tsp_attn_qkv_forward(tsp_attn_plan_t* plan, const void* X, const void* Wq, const void* Wk, const void* Wv,
                                  void* Q, void* K, void* V, int64_t S, int D, void* cuda_stream) {
    if (!plan || D != plan->D || S < 1) return TSP_ERR_INVALID_ARG;
    if (S > (1ll << 24)) return TSP_ERR_UNSUPPORTED_SHAPE;
    if (!X || !Wq || !Wk || !Wv || !Q || !K || !V) return TSP_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(Wq) || !aligned16(Wk) || !aligned16(Wv) || !aligned32(Q) || !aligned32(K) || !aligned32(V))
        return TSP_ERR_INVALID_ARG;
    tsp_mlp_plan_t* base = plan->base;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int H = plan->H, Hq = plan->Hq, Hkv = plan->Hkv;
    tsp::PairQkvPolicy::Params p;
    std::memset(&p, 0, sizeof(p));
    if (!encode_matrix(base, &p.map_x, X, S, H, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_matrix(base, &p.map_wq, Wq, Hq, H, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_matrix(base, &p.map_wk, Wk, Hkv, H, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_matrix(base, &p.map_wv, Wv, Hkv, H, 64, 128)) return TSP_ERR_CUDA;
    p.Q = static_cast<__nv_bfloat16*>(Q);
    p.K = static_cast<__nv_bfloat16*>(K);
    p.V = static_cast<__nv_bfloat16*>(V);
    p.S = static_cast<int>(S); p.H = H; p.Hq = Hq; p.Hkv = Hkv;
    p.m_tiles = static_cast<int>((S + 255) / 256);
    p.q_blocks = Hq / 256;
    p.kv_blocks = Hkv / 256;
    p.n_blocks = p.q_blocks + 2 * p.kv_blocks;
    p.band = gate_band(base, p.m_tiles);   // the band's rows of X take about 32 MB of L2
    Profiler prof(base, stream);
    tsp_status_t st = for_tile_chunks(p.m_tiles, base->chunk_bands * p.band, false, [&](int first, int count) {
        p.mt_base = first;
        p.m_tiles = count;
        fill_common(base, p, count * p.n_blocks);
        return launch_pair<tsp::PairQkvPolicy>(base, p, stream);
    });
    prof.mark();
    return st;
}

tsp_status_t tsp_attn_out_forward(tsp_attn_plan_t* plan, const void* A, const void* Wo, void* Y, int64_t S, int D,
                                  void* cuda_stream) {
    if (!plan || D != plan->D || S < 1) return TSP_ERR_INVALID_ARG;
    if (S > (1ll << 24)) return TSP_ERR_UNSUPPORTED_SHAPE;
    if (!A || !Wo || !Y) return TSP_ERR_INVALID_ARG;
    if (!aligned16(A) || !aligned16(Wo) || !aligned32(Y)) return TSP_ERR_INVALID_ARG;
    tsp_mlp_plan_t* base = plan->base;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int H = plan->H, Hq = plan->Hq, Hq_d = plan->Hq / plan->D;
    tsp::PairOutPolicy::Params p;
    std::memset(&p, 0, sizeof(p));
    if (!encode_matrix(base, &p.map_a, A, S, Hq, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_sharded(base, &p.map_wo, Wo, D, H, Hq_d, 64, 128)) return TSP_ERR_CUDA;
    p.Y = static_cast<__nv_bfloat16*>(Y);
    p.S = static_cast<int>(S); p.H = H; p.Hq = Hq; p.D = D; p.Hq_d = Hq_d;
    p.m_tiles = static_cast<int>((S + 255) / 256);
    p.n_blocks = H / 256;
    const int group = base->group > 0 ? base->group : 8;
    p.group = p.m_tiles < group ? p.m_tiles : group;
    Profiler prof(base, stream);
    tsp_status_t st = for_tile_chunks(p.m_tiles, base->chunk_tiles, false, [&](int first, int count) {
        p.mt_base = first;
        p.m_tiles = count;
        p.group = count < group ? count : group;
        fill_common(base, p, count * p.n_blocks);
        return launch_pair<tsp::PairOutPolicy>(base, p, stream, kDynDown);
    });
    prof.mark();
    return st;
}

tsp_status_t tsp_attn_qkv_backward(tsp_attn_plan_t* plan, const void* X, const void* Wq, const void* Wk, const void* Wv,
                                   const void* dQ, const void* dK, const void* dV, void* dX, float* dWq, float* dWk,
                                   float* dWv, int64_t S, int D, void* cuda_stream) {
    if (!plan || D != plan->D || S < 1) return TSP_ERR_INVALID_ARG;
    if (S > (1ll << 24)) return TSP_ERR_UNSUPPORTED_SHAPE;
    if (!X || !Wq || !Wk || !Wv || !dQ || !dK || !dV || !dX || !dWq || !dWk || !dWv) return TSP_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(Wq) || !aligned16(Wk) || !aligned16(Wv) || !aligned16(dQ) || !aligned16(dK) ||
        !aligned16(dV) || !aligned32(dX) || !aligned32(dWq) || !aligned32(dWk) || !aligned32(dWv))
        return TSP_ERR_INVALID_ARG;
    tsp_mlp_plan_t* base = plan->base;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int H = plan->H, Hq = plan->Hq, Hkv = plan->Hkv;
    Profiler prof(base, stream);
    {
        tsp::PairAttnDxPolicy::Params p;
        std::memset(&p, 0, sizeof(p));
        if (!encode_matrix(base, &p.map_dq, dQ, S, Hq, 64, 128)) return TSP_ERR_CUDA;
        if (!encode_matrix(base, &p.map_dk, dK, S, Hkv, 64, 128)) return TSP_ERR_CUDA;
        if (!encode_matrix(base, &p.map_dv, dV, S, Hkv, 64, 128)) return TSP_ERR_CUDA;
        if (!encode_matrix(base, &p.map_wq, Wq, Hq, H, 64, 64)) return TSP_ERR_CUDA;
        if (!encode_matrix(base, &p.map_wk, Wk, Hkv, H, 64, 64)) return TSP_ERR_CUDA;
        if (!encode_matrix(base, &p.map_wv, Wv, Hkv, H, 64, 64)) return TSP_ERR_CUDA;
        p.dX = static_cast<__nv_bfloat16*>(dX);
        p.S = static_cast<int>(S); p.H = H;
        p.q_kb = Hq / 64; p.kv_kb = Hkv / 64;
        p.m_tiles = static_cast<int>((S + 255) / 256);
        p.n_blocks = H / 256;
        const int group = base->dx_group > 0 ? base->dx_group : 8;
        p.group = p.m_tiles < group ? p.m_tiles : group;
        tsp_status_t st = for_tile_chunks(p.m_tiles, base->chunk_tiles, false, [&](int first, int count) {
            p.mt_base = first;
            p.m_tiles = count;
            p.group = count < group ? count : group;
            fill_common(base, p, count * p.n_blocks);
            return launch_pair<tsp::PairAttnDxPolicy>(base, p, stream, kDynDx);
        });
        if (st != TSP_OK) return st;
        prof.mark();
    }
    // weight gradients: token chunks, see for_token_chunks
    tsp_status_t st = for_token_chunks(S, [&](int64_t c0, int64_t len, bool) {
        tsp::PairAttnDwPolicy::Params p;
        std::memset(&p, 0, sizeof(p));
        if (!encode_matrix(base, &p.map_m0, row_offset(dQ, c0, Hq), len, Hq, 64, 64)) return TSP_ERR_CUDA;
        if (!encode_matrix(base, &p.map_m1, row_offset(dK, c0, Hkv), len, Hkv, 64, 64)) return TSP_ERR_CUDA;
        if (!encode_matrix(base, &p.map_m2, row_offset(dV, c0, Hkv), len, Hkv, 64, 64)) return TSP_ERR_CUDA;
        if (!encode_matrix(base, &p.map_n, row_offset(X, c0, H), len, H, 64, 64)) return TSP_ERR_CUDA;
        p.out0 = dWq; p.out1 = dWk; p.out2 = dWv;
        p.m_tiles0 = Hq / 256; p.m_tiles1 = Hkv / 256; p.m_tiles2 = Hkv / 256;
        p.rows0 = Hq; p.N = H; p.shard_w = 0;
        p.accumulate = c0 > 0;
        p.S = static_cast<int>(len);
        p.k_blocks = static_cast<int>((len + 63) / 64);
        p.n_blocks = H / 256;
        int n_group = base->dw_group > 0 ? base->dw_group : static_cast<int>((64ull << 20) / (512ull * static_cast<size_t>(len)));
        if (n_group < 1) n_group = 1;
        p.n_group = n_group > p.n_blocks ? p.n_blocks : n_group;
        fill_common(base, p, (p.m_tiles0 + p.m_tiles1 + p.m_tiles2) * p.n_blocks);
        return launch_pair<tsp::PairAttnDwPolicy>(base, p, stream, kDynDw);
    });
    if (st != TSP_OK) return st;
    prof.mark();
    return TSP_OK;
}

tsp_status_t tsp_attn_out_backward(tsp_attn_plan_t* plan, const void* A, const void* Wo, const void* dY, void* dA,
                                   float* dWo, int64_t S, int D, void* cuda_stream) {
    if (!plan || D != plan->D || S < 1) return TSP_ERR_INVALID_ARG;
    if (S > (1ll << 24)) return TSP_ERR_UNSUPPORTED_SHAPE;
    if (!A || !Wo || !dY || !dA || !dWo) return TSP_ERR_INVALID_ARG;
    if (!aligned16(A) || !aligned16(Wo) || !aligned16(dY) || !aligned32(dA) || !aligned32(dWo)) return TSP_ERR_INVALID_ARG;
    tsp_mlp_plan_t* base = plan->base;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int H = plan->H, Hq = plan->Hq, Hq_d = plan->Hq / plan->D;
    Profiler prof(base, stream);
    {
        tsp::PairAttnDaPolicy::Params p;
        std::memset(&p, 0, sizeof(p));
        if (!encode_matrix(base, &p.map_dy, dY, S, H, 64, 128)) return TSP_ERR_CUDA;
        if (!encode_sharded(base, &p.map_wo, Wo, D, H, Hq_d, 64, 64)) return TSP_ERR_CUDA;
        p.dA = static_cast<__nv_bfloat16*>(dA);
        p.S = static_cast<int>(S); p.H = H; p.Hq = Hq; p.Hq_d = Hq_d;
        p.m_tiles = static_cast<int>((S + 255) / 256);
        p.n_blocks = Hq / 256;
        p.band = gate_band(base, p.m_tiles);
        tsp_status_t st = for_tile_chunks(p.m_tiles, base->chunk_bands * p.band, false, [&](int first, int count) {
            p.mt_base = first;
            p.m_tiles = count;
            fill_common(base, p, count * p.n_blocks);
            return launch_pair<tsp::PairAttnDaPolicy>(base, p, stream);
        });
        if (st != TSP_OK) return st;
        prof.mark();
    }
    tsp_status_t st = for_token_chunks(S, [&](int64_t c0, int64_t len, bool) {
        tsp::PairAttnDwPolicy::Params p;
        std::memset(&p, 0, sizeof(p));
        if (!encode_matrix(base, &p.map_m0, row_offset(dY, c0, H), len, H, 64, 64)) return TSP_ERR_CUDA;
        p.map_m1 = p.map_m0;
        p.map_m2 = p.map_m0;
        if (!encode_matrix(base, &p.map_n, row_offset(A, c0, Hq), len, Hq, 64, 64)) return TSP_ERR_CUDA;
        p.out0 = dWo; p.out1 = dWo; p.out2 = dWo;
        p.m_tiles0 = H / 256; p.m_tiles1 = 0; p.m_tiles2 = 0;
        p.rows0 = H; p.N = Hq; p.shard_w = Hq_d;
        p.accumulate = c0 > 0;
        p.S = static_cast<int>(len);
        p.k_blocks = static_cast<int>((len + 63) / 64);
        p.n_blocks = Hq / 256;
        int n_group = base->dw_group > 0 ? base->dw_group : static_cast<int>((64ull << 20) / (512ull * static_cast<size_t>(len)));
        if (n_group < 1) n_group = 1;
        p.n_group = n_group > p.n_blocks ? p.n_blocks : n_group;
        fill_common(base, p, p.m_tiles0 * p.n_blocks);
        return launch_pair<tsp::PairAttnDwPolicy>(base, p, stream, kDynDw);
    });
    if (st != TSP_OK) return st;
    prof.mark();
    return TSP_OK;
}

tsp_status_t tsp_attn_status(tsp_attn_plan_t* plan) { return plan ? tsp_mlp_status(plan->base) : TSP_ERR_INVALID_ARG; }

tsp_status_t tsp_attn_profile_begin(tsp_attn_plan_t* plan, int max_calls) {
    return plan ? tsp_mlp_profile_begin(plan->base, max_calls) : TSP_ERR_INVALID_ARG;
}
tsp_status_t tsp_attn_profile_read(tsp_attn_plan_t* plan, int call_index, int* n_kernels_out, float* ms_out) {
    if (!plan) return TSP_ERR_INVALID_ARG;
    return tsp_mlp_profile_read(plan->base, call_index, n_kernels_out, ms_out);
}
tsp_status_t tsp_attn_profile_end(tsp_attn_plan_t* plan) {
    return plan ? tsp_mlp_profile_end(plan->base) : TSP_ERR_INVALID_ARG;
}

}  // extern "C"
