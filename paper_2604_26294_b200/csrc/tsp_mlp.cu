// C-ABI of the TSP gated ring MLP library: plan, shape checks, tensor-map encoding, launches.
// Every step of the path runs in the kernels of fwd_kernels.cuh / bwd_kernels.cuh; this file only
// validates, encodes TMA descriptors and enqueues.
#include <cuda.h>
#include <cuda_runtime.h>

#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <new>
#include <vector>

#include "../../include/tsp_mlp.h"
#include "bwd_kernels.cuh"
#include "fwd_kernels.cuh"
#include "pair_kernels.cuh"
#include "dyn_kernels.cuh"
#include "skew_kernels.cuh"

namespace {

using tsp::GateUpParams;
using tsp::DownParams;

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

constexpr int kMaxKernelsPerCall = 8;

// Device control block of a plan (ints): [0] status word; [16 + 2 i] scheduler words of slot i (dynamic tile
// hand-out: next list index, leaders done); [64 ...] two sets of per-token-tile "rows of A are ready" counters
// of the fused ring step, which alternate from launch to launch.
constexpr int kCtlSchedBase = 16, kCtlSchedSlots = 8;
constexpr int kCtlReadyBase = 64, kCtlReadyCount = 1024;
constexpr size_t kCtlBytes = (kCtlReadyBase + 2 * kCtlReadyCount) * sizeof(int);
static_assert(kCtlSchedBase + 2 * kCtlSchedSlots <= kCtlReadyBase, "scheduler words overlap the ready counters");

struct ProfileCall {
    cudaEvent_t ev[kMaxKernelsPerCall + 1];
    int n_kernels;
};

}  // namespace

struct tsp_mlp_plan {
    int H, F, D;
    int device;
    int sm_count;
    int max_smem;
    int* status_dev;
    void* workspace;
    size_t workspace_bytes;
    int last_cuda_error;
    unsigned long long timeout_ns;
    EncodeTiledFn encode;
    std::vector<ProfileCall> profile;
    int profile_next;
    // tunables (environment overrides read at plan creation; 0 = default)
    int use_pairs;      // CTA-pair (cta_group::2) kernels where the shape allows
    int band;           // token tiles per band in the gate|up tile order
    int shared_order;   // gate|up tile order: 1 = all ranks of a band on the same shard column block
    int group;          // token tiles per group in the down / dX tile order
    int pair_stages;
    int last_backward_kernels;  // kernels launched by the most recent backward call
    int last_forward_kernels;   // kernels launched by the most recent forward call
    int launch_count;           // kernels launched since the current call began
    int dw_group;               // hidden blocks per group in the dW tile order
    int dx_group;               // token tiles per group in the dX tile order
    int act;                    // gate activation (TSP_ACT_*)
    int wide_mask;              // 256 x 512 tiles for: bit 0 down, bit 1 dX, bit 2 dW (env TSP_MLP_WIDE)
    int chunk_bands;            // token bands per launch of the band-ordered kernels (gate|up, dA); 0 = one launch
    int dw_chunk_rounds;        // rounds of the CTA pairs per launch of the weight-gradient kernel; 0 = about 3 ms of
                                // work per launch, negative = one launch
    int chunk_tiles;            // token tiles per launch of the group-ordered kernels (down, dX); 0 = one launch
    int phase_mask;             // profiling aid (env TSP_MLP_PHASES): bit 0 = gate|up, bit 1 = down; default both
    int dynamic_tiles;          // CTA pairs draw their tiles from a device counter instead of a fixed round-robin
    int fuse_steps;             // per-rank ring steps: gate|up and down projection in one launch
    int ready_parity;           // which of the two ready-counter sets the next fused launch uses
    int tma_carry;              // carried fp32 sums (Yacc, dXacc) move through the TMA unit
    int rank_pair_tiles;        // bit 0 down, bit 1 dX: tiles of two neighbouring ranks share their weight panels
    int overlap_launches;       // pair kernels are launched with programmatic serialisation
    int64_t tma_dw_max_tokens;  // weight gradients also go out through the TMA unit up to this many tokens per launch
    std::vector<cudaEvent_t> staged_events;  // 2 per ring step: "shards received", "step computed"
    cudaStream_t host_copy_stream;           // tsp_mlp_forward_host: uploads (X, then the shards, then Wd by column blocks)
    cudaStream_t host_down_stream;           // tsp_mlp_forward_host: downloads of Y
    cudaEvent_t host_events[8];
    std::vector<cudaEvent_t> host_shard_events;   // "shard k has arrived"
    bool host_ready;
};

namespace {

inline size_t align_up(size_t v, size_t a) { return (v + a - 1) / a * a; }

tsp_status_t cuda_fail(tsp_mlp_plan_t* plan, int err) {
    if (plan) plan->last_cuda_error = err;
    return TSP_ERR_CUDA;
}

// 3-D bf16 tensor map with 128-byte swizzle: dims (d0 innermost, d1, d2), byte strides of d1 and d2.
bool encode_map(tsp_mlp_plan_t* plan, CUtensorMap* map, const void* base, CUtensorMapDataType dtype, size_t elem,
                uint64_t d0, uint64_t d1, uint64_t d2, uint64_t stride1, uint64_t stride2, uint32_t box0,
                uint32_t box1, CUtensorMapSwizzle swizzle = CU_TENSOR_MAP_SWIZZLE_128B) {
    cuuint64_t dims[3] = {d0, d1, d2};
    cuuint64_t strides[2] = {stride1, stride2};
    cuuint32_t box[3] = {box0, box1, 1};
    cuuint32_t estr[3] = {1, 1, 1};
    (void)elem;
    CUresult r = plan->encode(map, dtype, 3, const_cast<void*>(base), dims, strides, box, estr,
                              CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle,
                              CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        plan->last_cuda_error = static_cast<int>(r);
        return false;
    }
    return true;
}

// [rows, cols] row-major bf16 matrix viewed as (cols, rows, 1).
bool encode_matrix(tsp_mlp_plan_t* plan, CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint32_t box0,
                   uint32_t box1) {
    return encode_map(plan, map, base, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, cols, rows, 1, cols * 2, rows * cols * 2,
                      box0, box1);
}
// [D][rows][cols] row-major bf16 viewed as (cols, rows, D).
bool encode_sharded(tsp_mlp_plan_t* plan, CUtensorMap* map, const void* base, uint64_t D, uint64_t rows, uint64_t cols,
                    uint32_t box0, uint32_t box1) {
    return encode_map(plan, map, base, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, cols, rows, D, cols * 2, rows * cols * 2,
                      box0, box1);
}

// [n][rows][cols] bf16 with an arbitrary distance between consecutive matrices (packed shard buffers in a row).
bool encode_strided(tsp_mlp_plan_t* plan, CUtensorMap* map, const void* base, uint64_t n, uint64_t rows, uint64_t cols,
                    uint64_t stride_bytes, uint32_t box0, uint32_t box1) {
    return encode_map(plan, map, base, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, cols, rows, n, cols * 2, stride_bytes, box0, box1);
}

// [rows, cols] bf16 block of a wider row-major matrix (`pitch` elements per row), viewed as (cols, rows, 1).
bool encode_block(tsp_mlp_plan_t* plan, CUtensorMap* map, const void* base, uint64_t rows, uint64_t cols, uint64_t pitch,
                  uint32_t box0, uint32_t box1) {
    return encode_map(plan, map, base, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, cols, rows, 1, pitch * 2, rows * pitch * 2, box0,
                      box1);
}

bool aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }
bool aligned32(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 31u) == 0; }  // outputs: 256-bit stores

tsp_status_t check_call(const tsp_mlp_plan_t* plan, int64_t S, int D) {
    if (!plan) return TSP_ERR_INVALID_ARG;
    if (D != plan->D || S <= 0) return TSP_ERR_INVALID_ARG;
    if (S % D != 0) return TSP_ERR_UNSUPPORTED_SHAPE;   // equal token shards; any number of tokens per rank
    if (S > (1ll << 24)) return TSP_ERR_UNSUPPORTED_SHAPE;
    return TSP_OK;
}

// Shared-memory layout of the pair kernels: [stages][1 KB control area: SharedCtl, DynCtl][optional 32 KB of epilogue
// staging (carried fp32 sums through the TMA unit)], plus 1 KB of slack for the 1024-byte alignment of the base.
constexpr size_t kCtlAreaBytes = 1024, kEpiStagingBytes = 32 * 1024;
static_assert(sizeof(tsp::SharedCtl) + sizeof(tsp::DynCtl) <= kCtlAreaBytes, "control area too small");

int pick_stages(const tsp_mlp_plan_t* plan, size_t stage_bytes, int want, size_t extra_fixed = 0) {
    const size_t fixed = kCtlAreaBytes + 1024 + extra_fixed;
    int s = want;
    while (s > 2 && s * stage_bytes + fixed > static_cast<size_t>(plan->max_smem)) --s;
    return s;
}

struct Profiler {
    tsp_mlp_plan_t* plan;
    cudaStream_t stream;
    ProfileCall* call;
    int n;
    Profiler(tsp_mlp_plan_t* p, cudaStream_t s) : plan(p), stream(s), call(nullptr), n(0) {
        if (p->profile_next < static_cast<int>(p->profile.size())) {
            call = &p->profile[p->profile_next++];
            call->n_kernels = 0;
            cudaEventRecord(call->ev[0], stream);
        }
    }
    void mark() {
        if (call && n < kMaxKernelsPerCall) {
            ++n;
            cudaEventRecord(call->ev[n], stream);
            call->n_kernels = n;
        }
    }
};

// Token tiles (of 256 rows) per band of the gate|up tile order.
int gate_band(const tsp_mlp_plan_t* plan, int m_tiles) {
    // default: the band's rows of X (256 * band * H * 2 bytes) take about 32 MB, a quarter of L2, so they stay
    // resident while the weights stream past once per band (16 tiles at H = 4096)
    int band = plan->band > 0 ? plan->band : static_cast<int>((32ull << 20) / (512ull * plan->H));
    if (band < 1) band = 1;
    return band > m_tiles ? m_tiles : band;
}

// ---------------------------------------------------------------------------------------------
// launches
// ---------------------------------------------------------------------------------------------
tsp_status_t launch_gate_up(tsp_mlp_plan_t* plan, const void* X, const void* Wg, const void* Wu, void* A, int64_t S,
                            cudaStream_t stream) {
    const int H = plan->H, F = plan->F, D = plan->D, F_d = F / D;
    GateUpParams p;
    std::memset(&p, 0, sizeof(p));
    if (!encode_matrix(plan, &p.map_x, X, S, H, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_sharded(plan, &p.map_wg, Wg, D, H, F_d, 64, 64)) return TSP_ERR_CUDA;
    if (!encode_sharded(plan, &p.map_wu, Wu, D, H, F_d, 64, 64)) return TSP_ERR_CUDA;
    p.A = static_cast<__nv_bfloat16*>(A);
    p.S = static_cast<int>(S); p.H = H; p.F = F; p.D = D;
    p.S_loc = static_cast<int>(S / D);
    p.blocks_per_rank = (p.S_loc + 127) / 128;
    p.m_blocks = D * p.blocks_per_rank;
    p.jl_blocks = F_d / 128;
    p.band = 2 * gate_band(plan, (p.m_blocks + 1) / 2);   // same band, counted in 128-token blocks
    if (p.band > p.m_blocks) p.band = p.m_blocks;
    p.shared_order = plan->shared_order;
    p.act = plan->act;
    p.num_tiles = p.m_blocks * D * p.jl_blocks;
    p.stages = pick_stages(plan, 48 * 1024, 4);
    p.status = plan->status_dev;
    p.timeout_ns = plan->timeout_ns;
    const size_t smem = p.stages * 48 * 1024 + sizeof(tsp::SharedCtl) + 1024;
    cudaError_t e = cudaFuncSetAttribute(tsp::gate_up_swiglu_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem));
    if (e != cudaSuccess) return cuda_fail(plan, e);
    const int grid = p.num_tiles < plan->sm_count ? p.num_tiles : plan->sm_count;
    tsp::gate_up_swiglu_kernel<<<grid, tsp::kNumThreads, smem, stream>>>(p);
    ++plan->launch_count;
    e = cudaGetLastError();
    return e == cudaSuccess ? TSP_OK : cuda_fail(plan, e);
}

tsp_status_t launch_down(tsp_mlp_plan_t* plan, const void* A, const void* Wd, void* Y, int64_t S, cudaStream_t stream) {
    const int H = plan->H, F = plan->F, D = plan->D;
    DownParams p;
    std::memset(&p, 0, sizeof(p));
    if (!encode_matrix(plan, &p.map_a, A, S, F, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_matrix(plan, &p.map_wd, Wd, F, H, 64, 64)) return TSP_ERR_CUDA;
    p.Y = static_cast<__nv_bfloat16*>(Y);
    p.S = static_cast<int>(S); p.H = H; p.F = F; p.D = D;
    p.S_loc = static_cast<int>(S / D);
    p.blocks_per_rank = (p.S_loc + 127) / 128;
    p.m_blocks = D * p.blocks_per_rank;
    p.n_blocks = H / 256;
    p.group = p.m_blocks < 16 ? p.m_blocks : 16;
    p.num_tiles = p.m_blocks * p.n_blocks;
    p.stages = pick_stages(plan, 48 * 1024, 4);
    p.status = plan->status_dev;
    p.timeout_ns = plan->timeout_ns;
    const size_t smem = p.stages * 48 * 1024 + sizeof(tsp::SharedCtl) + 1024;
    cudaError_t e = cudaFuncSetAttribute(tsp::down_accumulate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem));
    if (e != cudaSuccess) return cuda_fail(plan, e);
    const int grid = p.num_tiles < plan->sm_count ? p.num_tiles : plan->sm_count;
    tsp::down_accumulate_kernel<<<grid, tsp::kNumThreads, smem, stream>>>(p);
    ++plan->launch_count;
    e = cudaGetLastError();
    return e == cudaSuccess ? TSP_OK : cuda_fail(plan, e);
}

tsp_status_t launch_bwd_gate(tsp_mlp_plan_t* plan, const void* X, const void* Wg, const void* Wu, const void* Wd,
                             const void* dY, void* A, void* dG, void* dU, int64_t S, cudaStream_t stream) {
    const int H = plan->H, F = plan->F, D = plan->D, F_d = F / D;
    tsp::BwdGateParams p;
    std::memset(&p, 0, sizeof(p));
    if (!encode_matrix(plan, &p.map_x, X, S, H, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_matrix(plan, &p.map_dy, dY, S, H, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_sharded(plan, &p.map_wg, Wg, D, H, F_d, 64, 64)) return TSP_ERR_CUDA;
    if (!encode_sharded(plan, &p.map_wu, Wu, D, H, F_d, 64, 64)) return TSP_ERR_CUDA;
    if (!encode_matrix(plan, &p.map_wd, Wd, F, H, 64, 128)) return TSP_ERR_CUDA;
    p.A = static_cast<__nv_bfloat16*>(A);
    p.dG = static_cast<__nv_bfloat16*>(dG);
    p.dU = static_cast<__nv_bfloat16*>(dU);
    p.S = static_cast<int>(S); p.H = H; p.F = F; p.D = D;
    p.S_loc = static_cast<int>(S / D);
    p.blocks_per_rank = (p.S_loc + 127) / 128;
    p.m_blocks = D * p.blocks_per_rank;
    p.jl_blocks = F_d / 128;
    p.band = 2 * gate_band(plan, (p.m_blocks + 1) / 2);
    if (p.band > p.m_blocks) p.band = p.m_blocks;
    p.act = plan->act;
    p.num_tiles = p.m_blocks * D * p.jl_blocks;
    p.stages = pick_stages(plan, 48 * 1024, 4);
    p.status = plan->status_dev;
    p.timeout_ns = plan->timeout_ns;
    const size_t smem = p.stages * 48 * 1024 + sizeof(tsp::SharedCtl) + 1024;
    cudaError_t e = cudaFuncSetAttribute(tsp::bwd_gate_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         static_cast<int>(smem));
    if (e != cudaSuccess) return cuda_fail(plan, e);
    const int grid = p.num_tiles < plan->sm_count ? p.num_tiles : plan->sm_count;
    tsp::bwd_gate_kernel<<<grid, tsp::kNumThreads, smem, stream>>>(p);
    ++plan->launch_count;
    e = cudaGetLastError();
    return e == cudaSuccess ? TSP_OK : cuda_fail(plan, e);
}

tsp_status_t launch_bwd_dx(tsp_mlp_plan_t* plan, const void* dG, const void* dU, const void* Wg, const void* Wu, void* dX,
                           int64_t S, cudaStream_t stream) {
    const int H = plan->H, F = plan->F, D = plan->D, F_d = F / D;
    tsp::BwdDxPolicy::Params p;
    std::memset(&p, 0, sizeof(p));
    if (!encode_matrix(plan, &p.map_dg, dG, S, F, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_matrix(plan, &p.map_du, dU, S, F, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_sharded(plan, &p.map_wg, Wg, D, H, F_d, 64, 256)) return TSP_ERR_CUDA;
    if (!encode_sharded(plan, &p.map_wu, Wu, D, H, F_d, 64, 256)) return TSP_ERR_CUDA;
    p.dX = static_cast<__nv_bfloat16*>(dX);
    p.S = static_cast<int>(S); p.H = H; p.F = F; p.D = D; p.F_d = F_d;
    p.S_loc = static_cast<int>(S / D);
    p.blocks_per_rank = (p.S_loc + 127) / 128;
    p.m_blocks = D * p.blocks_per_rank;
    p.n_blocks = H / 256;
    p.group = p.m_blocks < 16 ? p.m_blocks : 16;
    p.num_tiles = p.m_blocks * p.n_blocks;
    p.stages = pick_stages(plan, 48 * 1024, 4);
    p.status = plan->status_dev;
    p.timeout_ns = plan->timeout_ns;
    const size_t smem = p.stages * 48 * 1024 + sizeof(tsp::SharedCtl) + 1024;
    auto kernel = tsp::tile_gemm_kernel<tsp::BwdDxPolicy>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return cuda_fail(plan, e);
    const int grid = p.num_tiles < plan->sm_count ? p.num_tiles : plan->sm_count;
    kernel<<<grid, tsp::kNumThreads, smem, stream>>>(p);
    ++plan->launch_count;
    e = cudaGetLastError();
    return e == cudaSuccess ? TSP_OK : cuda_fail(plan, e);
}

tsp_status_t launch_bwd_dw(tsp_mlp_plan_t* plan, const void* X, const void* dY, const void* A, const void* dG,
                           const void* dU, float* dWg, float* dWu, float* dWd, int64_t S, cudaStream_t stream,
                           int accumulate = 0, bool linear = false) {
    const int H = plan->H, F = plan->F, D = plan->D;
    tsp::BwdDwPolicy::Params p;
    std::memset(&p, 0, sizeof(p));
    if (!encode_matrix(plan, &p.map_a, A, S, F, 64, 64)) return TSP_ERR_CUDA;
    if (!encode_matrix(plan, &p.map_dg, dG, S, F, 64, 64)) return TSP_ERR_CUDA;
    if (!encode_matrix(plan, &p.map_du, dU, S, F, 64, 64)) return TSP_ERR_CUDA;
    if (!encode_matrix(plan, &p.map_dy, dY, S, H, 64, 64)) return TSP_ERR_CUDA;
    if (!encode_matrix(plan, &p.map_x, X, S, H, 64, 64)) return TSP_ERR_CUDA;
    p.dWd = dWd; p.dWg = dWg; p.dWu = dWu;
    p.S = static_cast<int>(S); p.H = H; p.F = F; p.D = D;
    p.S_loc = static_cast<int>(S / D);
    p.k_linear = (linear || p.S_loc % 64 != 0) ? static_cast<int>((S + 63) / 64) : 0;
    p.accumulate = accumulate;
    p.j_blocks = F / 128;
    p.n_blocks = H / 256;
    p.num_tiles = 3 * p.j_blocks * p.n_blocks;
    p.stages = pick_stages(plan, 48 * 1024, 4);
    p.status = plan->status_dev;
    p.timeout_ns = plan->timeout_ns;
    const size_t smem = p.stages * 48 * 1024 + sizeof(tsp::SharedCtl) + 1024;
    auto kernel = tsp::tile_gemm_kernel<tsp::BwdDwPolicy>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return cuda_fail(plan, e);
    const int grid = p.num_tiles < plan->sm_count ? p.num_tiles : plan->sm_count;
    kernel<<<grid, tsp::kNumThreads, smem, stream>>>(p);
    ++plan->launch_count;
    e = cudaGetLastError();
    return e == cudaSuccess ? TSP_OK : cuda_fail(plan, e);
}


// ---------------------------------------------------------------------------------------------
// CTA-pair launches (tile = 256 rows per pair).  Chosen when (S/D) % 256 == 0 (and (F/D) % 256 == 0 for dW).
// ---------------------------------------------------------------------------------------------
// Mixed-width tile list for the long-K GEMMs: how many 256 x 512 tiles to put in front of the 256 x 256 ones.
// Wide tiles move a quarter less data per FLOP and halve DRAM re-reads, but take two time units each and do not
// overlap their epilogue; they are used for whole rounds of the CTA pairs as long as the total number of time units
// does not grow, and only when the K loop is long enough to amortise the epilogue.  Returns 0 for "narrow kernel".
int mixed_wide_tiles(const tsp_mlp_plan_t* plan, int bit, int n_blocks, int narrow_tiles, int k_blocks) {
    if (n_blocks % 2 != 0) return 0;
    const int pairs = plan->sm_count / 2;
    const int all_wide = narrow_tiles / 2;
    if (plan->wide_mask >= 0) return (plan->wide_mask & bit) ? all_wide : 0;
    if (k_blocks < 200) return 0;
    const int rounds_narrow = (narrow_tiles + pairs - 1) / pairs;
    if (2 * ((all_wide + pairs - 1) / pairs) <= rounds_narrow) return all_wide;
    for (int k = all_wide / pairs; k >= 1; --k) {
        const int wide = k * pairs;
        const int rest = narrow_tiles - 2 * wide;
        if (2 * k + (rest + pairs - 1) / pairs <= rounds_narrow) return wide;
    }
    return 0;
}

// The CTA pairs of a launch take their tiles in a fixed round-robin order.  Over hundreds of tiles they drift apart in
// time, and the tiles that were laid out to share an operand block through L2 no longer run together (measured at
// S = 65536: 2.4 x the DRAM reads of the same tile order at S = 8192, 4-5 % of the time).  A long problem is therefore
// cut into several launches of `chunk` token tiles each; every launch boundary realigns the pairs.  fn(first token
// tile, token tiles) launches one chunk; `reverse` walks the chunks from the last to the first.
template <class Fn>
tsp_status_t for_tile_chunks(int m_tiles, int chunk, bool reverse, Fn fn) {
    if (chunk <= 0 || m_tiles <= chunk + chunk / 2) return fn(0, m_tiles);
    int n = m_tiles / chunk;                       // the remainder joins the last chunk if it is less than half a chunk
    if (m_tiles - n * chunk >= chunk / 2 && m_tiles - n * chunk > 0) ++n;
    for (int i = 0; i < n; ++i) {
        const int c = reverse ? n - 1 - i : i;
        const int first = c * chunk;
        const int count = c == n - 1 ? m_tiles - first : chunk;
        tsp_status_t st = fn(first, count);
        if (st != TSP_OK) return st;
    }
    return TSP_OK;
}

template <class Params>
void fill_common(tsp_mlp_plan_t* plan, Params& p, int num_tiles, int sched_slot = 0) {
    p.num_tiles = num_tiles;
    p.sched = plan->status_dev + kCtlSchedBase + 2 * sched_slot;
    p.stages = pick_stages(plan, tsp::kPairStageBytes, plan->pair_stages > 0 ? plan->pair_stages : 6);
    p.status = plan->status_dev;
    p.timeout_ns = plan->timeout_ns;
}

// Params with a `carry_tma` member may route their carried fp32 sums through the TMA unit: the launch then reserves the
// staging buffers and tells the kernel where the control block sits (which depends on the stage count chosen here).
template <class P>
auto carry_wanted(const P& p, int) -> decltype(p.carry_tma.epi_off, bool()) { return p.carry_tma.epi_off != 0; }
template <class P>
bool carry_wanted(const P&, long) { return false; }
template <class P>
auto carry_place(P& p, uint32_t off, int) -> decltype(p.carry_tma.epi_off, void()) { p.carry_tma.epi_off = off; }
template <class P>
void carry_place(P&, uint32_t, long) {}

// fp32 [ranks][rows][H] accumulator viewed as (H, rows, ranks) with boxes of 32 columns x 128 rows, 128-byte swizzle
bool encode_carry(tsp_mlp_plan_t* plan, tsp::CarryTma* ct, const float* acc, uint64_t rows_per_rank, uint64_t ranks) {
    const uint64_t H = plan->H;
    ct->epi_off = 0;
    if (!plan->tma_carry || !acc) return true;
    if (!encode_map(plan, &ct->map, acc, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, H, rows_per_rank, ranks, H * 4,
                    rows_per_rank * H * 4, 32, 128))
        return false;
    ct->epi_off = 1;   // "wanted"; the launch replaces it by the real offset
    return true;
}

// Launch of a CTA-pair kernel.  With `overlap_launches` the launch carries the programmatic-serialisation attribute:
// its CTAs may become resident while the previous kernel of the stream is finishing, run their set-up (barriers,
// tensor-memory allocation, cluster sync) and then wait, on the device, for the previous grid to complete before they
// touch global memory (pair_setup).  After anything that is not such a kernel the launch is ordered as usual.
template <class Kernel, class Params>
cudaError_t launch_pairs(const tsp_mlp_plan_t* plan, Kernel kernel, int pairs, size_t smem, cudaStream_t stream,
                         const Params& p) {
    cudaLaunchConfig_t cfg = {};
    cfg.gridDim = dim3(2 * pairs);
    cfg.blockDim = dim3(tsp::kNumThreads);
    cfg.dynamicSmemBytes = smem;
    cfg.stream = stream;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = plan->overlap_launches ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, p);
}

// Which kernels draw their tiles dynamically (bits of the plan's dynamic_tiles mask).
constexpr int kDynGate = 1, kDynDown = 2, kDynDx = 4, kDynDw = 8;

template <class Policy>
tsp_status_t launch_pair_wide(tsp_mlp_plan_t* plan, typename Policy::Params& p, cudaStream_t stream, int kind) {
    const bool staging = carry_wanted(p, 0);
    p.stages = pick_stages(plan, tsp::kWideStageBytes, 4, staging ? kEpiStagingBytes : 0);
    const bool dynamic = (plan->dynamic_tiles & kind) != 0;
    if (staging) carry_place(p, static_cast<uint32_t>(p.stages * tsp::kWideStageBytes), 0);
    const size_t smem = p.stages * tsp::kWideStageBytes + kCtlAreaBytes + (staging ? kEpiStagingBytes : 0) + 1024;
    auto kernel = dynamic ? tsp::pair_wide_dyn_kernel<Policy> : tsp::pair_wide_kernel<Policy>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return cuda_fail(plan, e);
    const int pairs_avail = plan->sm_count / 2;
    const int pairs = p.num_tiles < pairs_avail ? p.num_tiles : pairs_avail;
    e = launch_pairs(plan, kernel, pairs, smem, stream, p);
    ++plan->launch_count;
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? TSP_OK : cuda_fail(plan, e);
}

// Two-rank tiles (pair_skew_kernel): how many of the `positions` (rank pair, token tile, hidden block) run as tall tiles.
// A tall tile is two time units of MMA work, like two one-rank tiles; whole rounds of the CTA pairs are made tall as long
// as the number of time units does not grow, the remaining positions are split into one-rank tiles.
int skew_tile_count(const tsp_mlp_plan_t* plan, int positions) {
    if (plan->rank_pair_tiles & 4) return positions;
    const int pairs = plan->sm_count / 2;
    const int rounds_narrow = (2 * positions + pairs - 1) / pairs;
    if (2 * ((positions + pairs - 1) / pairs) <= rounds_narrow) return positions;
    for (int k = positions / pairs; k >= 1; --k) {
        const int rest = 2 * (positions - k * pairs);
        if (2 * k + (rest + pairs - 1) / pairs <= rounds_narrow) return k * pairs;
    }
    return 0;
}

// Whether a launch over all D ranks' token tiles may use two-rank tiles: the ranks must pair up, a rank must own few
// token tiles (with many, consecutive one-rank tiles already share their weight panels), and the launch must be whole.
bool skew_possible(const tsp_mlp_plan_t* plan, int bit, int dyn_kind, int tiles_per_rank, int m_tiles) {
    if (!(plan->rank_pair_tiles & bit) || !(plan->dynamic_tiles & dyn_kind)) return false;
    if (plan->D < 2 || plan->D % 2 != 0 || tiles_per_rank > 8) return false;
    return plan->chunk_tiles <= 0 || m_tiles <= plan->chunk_tiles + plan->chunk_tiles / 2;
}

template <class Policy>
tsp_status_t launch_pair_skew(tsp_mlp_plan_t* plan, typename Policy::Params& p, cudaStream_t stream) {
    p.stages = pick_stages(plan, tsp::kWideStageBytes, 4, 0);
    const size_t smem = p.stages * tsp::kWideStageBytes + kCtlAreaBytes + 1024;
    auto kernel = tsp::pair_skew_kernel<Policy>;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return cuda_fail(plan, e);
    const int pairs_avail = plan->sm_count / 2;
    const int pairs = p.num_tiles < pairs_avail ? p.num_tiles : pairs_avail;
    e = launch_pairs(plan, kernel, pairs, smem, stream, p);
    ++plan->launch_count;
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? TSP_OK : cuda_fail(plan, e);
}

template <class Kernel, class Params>
tsp_status_t launch_pair_kernel(tsp_mlp_plan_t* plan, Kernel kernel, Params p, cudaStream_t stream) {
    const bool staging = carry_wanted(p, 0);
    if (staging) {
        p.stages = pick_stages(plan, tsp::kPairStageBytes, p.stages, kEpiStagingBytes);
        carry_place(p, static_cast<uint32_t>(p.stages * tsp::kPairStageBytes), 0);
    }
    const size_t smem = p.stages * tsp::kPairStageBytes + kCtlAreaBytes + (staging ? kEpiStagingBytes : 0) + 1024;
    cudaError_t e = cudaFuncSetAttribute(kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, static_cast<int>(smem));
    if (e != cudaSuccess) return cuda_fail(plan, e);
    const int pairs_avail = plan->sm_count / 2;
    const int pairs = p.num_tiles < pairs_avail ? p.num_tiles : pairs_avail;
    e = launch_pairs(plan, kernel, pairs, smem, stream, p);
    ++plan->launch_count;
    if (e == cudaSuccess) e = cudaGetLastError();
    return e == cudaSuccess ? TSP_OK : cuda_fail(plan, e);
}

// 256 x 256 tiles of `Policy`: CTA pairs take them round-robin, or draw them from the plan's scheduler words
template <class Policy>
tsp_status_t launch_pair(tsp_mlp_plan_t* plan, const typename Policy::Params& p, cudaStream_t stream, int kind = kDynGate) {
    if (plan->dynamic_tiles & kind)
        return launch_pair_kernel(plan, tsp::pair_dyn_kernel<tsp::DynOf<Policy>>, p, stream);
    return launch_pair_kernel(plan, tsp::pair_gemm_kernel<Policy>, p, stream);
}

template <int kMode>
tsp_status_t launch_gate_pair(tsp_mlp_plan_t* plan, const void* X, const void* Wg, const void* Wu, void* A,
                              const float* dA, void* dG, void* dU, int64_t S, cudaStream_t stream) {
    using Policy = tsp::PairGateUpPolicyT<kMode>;
    const int H = plan->H, F = plan->F, D = plan->D, F_d = F / D;
    typename Policy::Params p;
    std::memset(&p, 0, sizeof(p));
    if (!encode_matrix(plan, &p.map_x, X, S, H, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_sharded(plan, &p.map_wg, Wg, D, H, F_d, 64, 64)) return TSP_ERR_CUDA;
    if (!encode_sharded(plan, &p.map_wu, Wu, D, H, F_d, 64, 64)) return TSP_ERR_CUDA;
    p.A = static_cast<__nv_bfloat16*>(A);
    p.dA = dA;
    p.dG = static_cast<__nv_bfloat16*>(dG);
    p.dU = static_cast<__nv_bfloat16*>(dU);
    p.S = static_cast<int>(S); p.H = H; p.F = F; p.D = D;
    p.F_d = F_d;
    p.S_loc = static_cast<int>(S / D);
    p.tiles_per_rank = (p.S_loc + 255) / 256;
    p.m_tiles = D * p.tiles_per_rank;
    p.jl_blocks = F_d / 128;
    p.band = gate_band(plan, p.m_tiles);
    p.shared_order = plan->shared_order;
    p.act = plan->act;
    return for_tile_chunks(p.m_tiles, plan->chunk_bands * p.band, false, [&](int first, int count) {
        p.mt_base = first;
        p.m_tiles = count;
        fill_common(plan, p, count * D * p.jl_blocks);
        return launch_pair<Policy>(plan, p, stream);
    });
}

tsp_status_t launch_gate_up_pair(tsp_mlp_plan_t* plan, const void* X, const void* Wg, const void* Wu, void* A, int64_t S,
                                 cudaStream_t stream) {
    return launch_gate_pair<0>(plan, X, Wg, Wu, A, nullptr, nullptr, nullptr, S, stream);
}

// The gate|up tiles of ONE shard k for all tokens (the host-buffer forward launches shard by shard, each as soon as its
// weights have arrived): the same tiles as in the full launch, writing columns k F/D .. of A.
tsp_status_t launch_gate_up_shard(tsp_mlp_plan_t* plan, const void* X, const void* Wg, const void* Wu, void* A, int k,
                                  int64_t S, cudaStream_t stream) {
    using Policy = tsp::PairGateUpPolicyT<0>;
    const int H = plan->H, F = plan->F, D = plan->D, F_d = F / D;
    const size_t shard = static_cast<size_t>(H) * F_d * 2;
    Policy::Params p;
    std::memset(&p, 0, sizeof(p));
    if (!encode_matrix(plan, &p.map_x, X, S, H, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_sharded(plan, &p.map_wg, static_cast<const uint8_t*>(Wg) + k * shard, 1, H, F_d, 64, 64)) return TSP_ERR_CUDA;
    if (!encode_sharded(plan, &p.map_wu, static_cast<const uint8_t*>(Wu) + k * shard, 1, H, F_d, 64, 64)) return TSP_ERR_CUDA;
    p.A = static_cast<__nv_bfloat16*>(A) + static_cast<size_t>(k) * F_d;
    p.S = static_cast<int>(S); p.H = H; p.F = F; p.D = 1; p.F_d = F_d;
    p.S_loc = static_cast<int>(S / D);
    p.tiles_per_rank = (p.S_loc + 255) / 256;
    p.m_tiles = D * p.tiles_per_rank;
    p.jl_blocks = F_d / 128;
    p.band = gate_band(plan, p.m_tiles);
    p.shared_order = 1;
    p.act = plan->act;
    return for_tile_chunks(p.m_tiles, plan->chunk_bands * p.band, false, [&](int first, int count) {
        p.mt_base = first;
        p.m_tiles = count;
        fill_common(plan, p, count * p.jl_blocks);
        return launch_pair<Policy>(plan, p, stream);
    });
}

// dA = dY Wd^T (needs F % 256 == 0).  kSaved = false: fp32 dA out; kSaved = true: dG = dA*P, dU = dA*Q out.
template <bool kSaved>
tsp_status_t launch_da_pair_t(tsp_mlp_plan_t* plan, const void* dY, const void* Wd, float* dA, const void* P, const void* Q,
                              void* dG, void* dU, int64_t S, cudaStream_t stream) {
    using Policy = tsp::PairDaPolicyT<kSaved>;
    const int H = plan->H, F = plan->F, D = plan->D;
    typename Policy::Params p;
    std::memset(&p, 0, sizeof(p));
    if (!encode_matrix(plan, &p.map_dy, dY, S, H, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_matrix(plan, &p.map_wd, Wd, F, H, 64, 128)) return TSP_ERR_CUDA;
    p.dA = dA;
    p.P = static_cast<const __nv_bfloat16*>(P);
    p.Q = static_cast<const __nv_bfloat16*>(Q);
    p.dG = static_cast<__nv_bfloat16*>(dG);
    p.dU = static_cast<__nv_bfloat16*>(dU);
    p.S = static_cast<int>(S); p.H = H; p.F = F; p.D = D;
    p.S_loc = static_cast<int>(S / D);
    p.tiles_per_rank = (p.S_loc + 255) / 256;
    p.m_tiles = D * p.tiles_per_rank;
    p.j_tiles = F / 256;
    p.band = gate_band(plan, p.m_tiles);
    return for_tile_chunks(p.m_tiles, plan->chunk_bands * p.band, false, [&](int first, int count) {
        p.mt_base = first;
        p.m_tiles = count;
        fill_common(plan, p, count * p.j_tiles);
        return launch_pair<Policy>(plan, p, stream);
    });
}

tsp_status_t launch_da_pair(tsp_mlp_plan_t* plan, const void* dY, const void* Wd, float* dA, int64_t S, cudaStream_t stream) {
    return launch_da_pair_t<false>(plan, dY, Wd, dA, nullptr, nullptr, nullptr, nullptr, S, stream);
}

// tile_first / tile_count: restrict the launch to a range of token tiles (default: all of them)
// tile_first / tile_count restrict the launch to a range of token tiles, nb_first / nb_count to a range of 256-column
// hidden blocks (default: everything); the tiles and their K loops are the same whichever way the work is cut
tsp_status_t launch_down_pair(tsp_mlp_plan_t* plan, const void* A, const void* Wd, void* Y, int64_t S, cudaStream_t stream,
                              int tile_first = 0, int tile_count = -1, int nb_first = 0, int nb_count = -1) {
    const int H = plan->H, F = plan->F, D = plan->D;
    if (nb_count < 0) nb_count = H / 256 - nb_first;
    tsp::PairDownPolicy::Params p;
    std::memset(&p, 0, sizeof(p));
    if (!encode_matrix(plan, &p.map_a, A, S, F, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_block(plan, &p.map_wd, static_cast<const uint8_t*>(Wd) + static_cast<size_t>(nb_first) * 512, F,
                      static_cast<uint64_t>(nb_count) * 256, H, 64, 64))
        return TSP_ERR_CUDA;
    p.Y = static_cast<__nv_bfloat16*>(Y) + static_cast<size_t>(nb_first) * 256;
    p.S = static_cast<int>(S); p.H = H; p.F = F; p.D = D; p.F_d = F / D;
    p.S_loc = static_cast<int>(S / D);
    p.tiles_per_rank = (p.S_loc + 255) / 256;
    p.m_tiles = D * p.tiles_per_rank;
    p.n_blocks = nb_count;
    const int group = plan->group > 0 ? plan->group : 8;
    if (tile_count < 0) tile_count = p.m_tiles - tile_first;
    if (tile_first == 0 && tile_count == p.m_tiles && skew_possible(plan, 1, kDynDown, p.tiles_per_rank, p.m_tiles)) {
        const int positions = (D / 2) * p.tiles_per_rank * p.n_blocks;
        p.skew_tiles = skew_tile_count(plan, positions);
        if (p.skew_tiles > 0) {
            fill_common(plan, p, 2 * positions - p.skew_tiles);   // a tall tile is one list entry
            return launch_pair_skew<tsp::PairDownPolicy>(plan, p, stream);
        }
    }
    // chunks from the last token tiles to the first: the rows the gate|up kernel wrote last are still in L2
    return for_tile_chunks(tile_count, plan->chunk_tiles, true, [&](int first, int count) {
        p.mt_base = tile_first + first;
        p.m_tiles = count;
        p.group = count < group ? count : group;
        p.wide_tiles = mixed_wide_tiles(plan, 1, p.n_blocks, count * p.n_blocks, F / 64);
        if (p.wide_tiles > 0) {
            fill_common(plan, p, count * p.n_blocks - p.wide_tiles);   // wide tiles count once in the list
            return launch_pair_wide<tsp::PairDownPolicy>(plan, p, stream, kDynDown);
        }
        fill_common(plan, p, count * p.n_blocks);
        return launch_pair<tsp::PairDownPolicy>(plan, p, stream, kDynDown);
    });
}

tsp_status_t launch_bwd_dx_pair(tsp_mlp_plan_t* plan, const void* dG, const void* dU, const void* Wg, const void* Wu,
                                void* dX, int64_t S, cudaStream_t stream, float* dXacc = nullptr, int carry = 0) {
    const int H = plan->H, F = plan->F, D = plan->D, F_d = F / D;
    tsp::PairDxPolicy::Params p;
    std::memset(&p, 0, sizeof(p));
    if (!encode_matrix(plan, &p.map_dg, dG, S, F, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_matrix(plan, &p.map_du, dU, S, F, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_sharded(plan, &p.map_wg, Wg, D, H, F_d, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_sharded(plan, &p.map_wu, Wu, D, H, F_d, 64, 128)) return TSP_ERR_CUDA;
    p.dX = static_cast<__nv_bfloat16*>(dX);
    p.dXacc = dXacc;
    p.carry = carry;
    if (carry != 0 && !encode_carry(plan, &p.carry_tma, dXacc, static_cast<uint64_t>(S / D), D)) return TSP_ERR_CUDA;
    p.S = static_cast<int>(S); p.H = H; p.F = F; p.D = D; p.F_d = F_d;
    p.S_loc = static_cast<int>(S / D);
    p.tiles_per_rank = (p.S_loc + 255) / 256;
    p.m_tiles = D * p.tiles_per_rank;
    p.n_blocks = H / 256;
    const int group = plan->dx_group > 0 ? plan->dx_group : 8;
    if (carry == 0 && skew_possible(plan, 2, kDynDx, p.tiles_per_rank, p.m_tiles)) {
        const int positions = (D / 2) * p.tiles_per_rank * p.n_blocks;
        p.skew_tiles = skew_tile_count(plan, positions);
        if (p.skew_tiles > 0) {
            fill_common(plan, p, 2 * positions - p.skew_tiles);
            return launch_pair_skew<tsp::PairDxPolicy>(plan, p, stream);
        }
    }
    return for_tile_chunks(p.m_tiles, plan->chunk_tiles, true, [&](int first, int count) {
        p.mt_base = first;
        p.m_tiles = count;
        p.group = count < group ? count : group;
        p.wide_tiles = mixed_wide_tiles(plan, 2, p.n_blocks, count * p.n_blocks, 2 * F / 64);
        if (p.wide_tiles > 0) {
            fill_common(plan, p, count * p.n_blocks - p.wide_tiles);
            return launch_pair_wide<tsp::PairDxPolicy>(plan, p, stream, kDynDx);
        }
        fill_common(plan, p, count * p.n_blocks);
        return launch_pair<tsp::PairDxPolicy>(plan, p, stream, kDynDx);
    });
}

tsp_status_t launch_bwd_dw_pair(tsp_mlp_plan_t* plan, const void* X, const void* dY, const void* A, const void* dG,
                                const void* dU, float* dWg, float* dWu, float* dWd, int64_t S, cudaStream_t stream,
                                int accumulate = 0, bool linear = false, int64_t pitch = 0) {
    const int H = plan->H, F = plan->F, D = plan->D;
    if (pitch <= 0) pitch = F;   // A, dG, dU may be column blocks of wider matrices (the scratch of a ring-step group)
    tsp::PairDwPolicy::Params p;
    std::memset(&p, 0, sizeof(p));
    if (!encode_block(plan, &p.map_a, A, S, F, pitch, 64, 64)) return TSP_ERR_CUDA;
    if (!encode_block(plan, &p.map_dg, dG, S, F, pitch, 64, 64)) return TSP_ERR_CUDA;
    if (!encode_block(plan, &p.map_du, dU, S, F, pitch, 64, 64)) return TSP_ERR_CUDA;
    if (!encode_matrix(plan, &p.map_dy, dY, S, H, 64, 64)) return TSP_ERR_CUDA;
    if (!encode_matrix(plan, &p.map_x, X, S, H, 64, 64)) return TSP_ERR_CUDA;
    p.dWd = dWd; p.dWg = dWg; p.dWu = dWu;
    p.accumulate = accumulate;
    p.S = static_cast<int>(S); p.H = H; p.F = F; p.D = D;
    p.F_d = F / D;
    p.out_shard_stride = static_cast<long long>(H) * p.F_d;
    // With few tokens the K loop of a tile is shorter than its epilogue (256 KB of fp32 per tile, read and written when
    // accumulating): the outputs then go through the TMA unit (stores, or adds performed by the memory system).
    if (plan->tma_carry && S <= plan->tma_dw_max_tokens) {
        const uint64_t st = static_cast<uint64_t>(p.out_shard_stride) * 4;
        if (!encode_map(plan, &p.carry_tma.map, dWd, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, H, p.F_d, D, static_cast<uint64_t>(H) * 4,
                        st, 32, 128))
            return TSP_ERR_CUDA;
        if (!encode_map(plan, &p.map_owg, dWg, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, p.F_d, H, D,
                        static_cast<uint64_t>(p.F_d) * 4, st, 128, 32, CU_TENSOR_MAP_SWIZZLE_NONE))
            return TSP_ERR_CUDA;
        if (!encode_map(plan, &p.map_owu, dWu, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 4, p.F_d, H, D,
                        static_cast<uint64_t>(p.F_d) * 4, st, 128, 32, CU_TENSOR_MAP_SWIZZLE_NONE))
            return TSP_ERR_CUDA;
        p.carry_tma.epi_off = 1;
    }
    p.S_loc = static_cast<int>(S / D);
    p.k_linear = (linear || p.S_loc % 64 != 0) ? static_cast<int>((S + 63) / 64) : 0;
    p.j_tiles = F / 256;
    p.j_tiles_per_shard = p.F_d / 256;
    p.n_blocks = H / 256;
    // hidden blocks are taken in groups whose columns of X / dY (S * 512 bytes per block) take about 64 MB (measured:
    // DRAM reads of the dW kernel at S = 8192 are 8.9 / 7.2 / 4.4 / 4.1 GB for groups of 2 / 4 / 8 / 16 blocks)
    int n_group = plan->dw_group > 0 ? plan->dw_group : static_cast<int>((64ull << 20) / (512ull * static_cast<size_t>(S)));
    if (n_group < 1) n_group = 1;
    p.wide_tiles = mixed_wide_tiles(plan, 4, p.n_blocks, 3 * p.j_tiles * p.n_blocks, static_cast<int>(S / 64));
    p.n_group = n_group > p.n_blocks ? p.n_blocks : n_group;
    // the tile list is cut into launches of `dw_chunk_rounds` rounds of the CTA pairs (see for_tile_chunks)
    const int list = 3 * p.j_tiles * p.n_blocks - p.wide_tiles;
    // about 3 ms of work per launch: a tile takes about 0.44 us per 64-token k-block (twice that for a wide tile)
    int rounds = plan->dw_chunk_rounds;
    if (rounds == 0) {
        const double tile_us = 0.44 * static_cast<double>((S + 63) / 64) * (p.wide_tiles > 0 ? 2.0 : 1.0);
        rounds = static_cast<int>(3000.0 / tile_us + 0.5);
        if (rounds < 1) rounds = 1;
    }
    const int chunk = rounds > 0 ? rounds * (plan->sm_count / 2) : 0;
    return for_tile_chunks(list, chunk, false, [&](int first, int count) {
        p.tile_base = first;
        fill_common(plan, p, count);
        return p.wide_tiles > 0 ? launch_pair_wide<tsp::PairDwPolicy>(plan, p, stream, kDynDw)
                                : launch_pair<tsp::PairDwPolicy>(plan, p, stream, kDynDw);
    });
}

// CTA pairs work on 256-row token tiles, single CTAs on 128-row tiles; a rank's last tile is padded.  Pairs are the
// faster kernels, so they are taken unless their padding costs clearly more rows than the single-CTA tiling.
bool pairs_for_tokens(const tsp_mlp_plan_t* plan, int64_t S) {
    if (!plan->use_pairs) return false;
    const int64_t s_loc = S / plan->D;
    const int64_t padded_pair = (s_loc + 255) / 256 * 256, padded_single = (s_loc + 127) / 128 * 128;
    return padded_pair * 100 <= padded_single * 106;
}
bool pairs_for_dw(const tsp_mlp_plan_t* plan) { return plan->use_pairs && (plan->F / plan->D) % 256 == 0; }

// The tensor cores add into their fp32 accumulators with truncation, so a contraction over very many tokens drifts
// towards zero (measured: 1.9 % after 2^24 tokens, 0.4 % after 2^22).  The weight-gradient contractions are therefore
// cut into chunks of at most kDwChunkTokens tokens, one launch per chunk in ascending token order; every launch after
// the first adds its fp32 result to what the output holds (round to nearest), which bounds the drift at about 3e-4.
// Up to kDwChunkTokens tokens (all the 7B-shaped workloads) there is one launch and the rank order of the sum is kept.
constexpr int64_t kDwChunkTokens = 1 << 18;

template <class Fn>
tsp_status_t for_token_chunks(int64_t S, Fn fn) {
    if (S <= kDwChunkTokens) return fn(static_cast<int64_t>(0), S, false);
    for (int64_t c0 = 0; c0 < S; c0 += kDwChunkTokens) {
        const int64_t len = S - c0 < kDwChunkTokens ? S - c0 : kDwChunkTokens;
        tsp_status_t st = fn(c0, len, true);
        if (st != TSP_OK) return st;
    }
    return TSP_OK;
}

inline const void* row_offset(const void* base, int64_t row, int64_t cols) {
    return static_cast<const uint8_t*>(base) + static_cast<size_t>(row) * static_cast<size_t>(cols) * 2;
}

// All weight gradients of the MLP for S tokens; `accumulate`: add to what dW* hold instead of overwriting.
tsp_status_t launch_dw_all(tsp_mlp_plan_t* plan, const void* X, const void* dY, const void* A, const void* dG,
                           const void* dU, float* dWg, float* dWu, float* dWd, int64_t S, cudaStream_t stream,
                           int accumulate, int64_t pitch = 0) {
    const int H = plan->H, F = plan->F;
    const bool pairs = pairs_for_dw(plan);
    if (pitch <= 0) pitch = F;
    if (pitch != F && !pairs) return TSP_ERR_UNSUPPORTED_SHAPE;
    return for_token_chunks(S, [&](int64_t c0, int64_t len, bool chunked) {
        const int acc = (accumulate || c0 > 0) ? 1 : 0;
        const void* x = row_offset(X, c0, H);
        const void* dy = row_offset(dY, c0, H);
        const void* a = row_offset(A, c0, pitch);
        const void* dg = row_offset(dG, c0, pitch);
        const void* du = row_offset(dU, c0, pitch);
        return pairs ? launch_bwd_dw_pair(plan, x, dy, a, dg, du, dWg, dWu, dWd, len, stream, acc, chunked, pitch)
                     : launch_bwd_dw(plan, x, dy, a, dg, du, dWg, dWu, dWd, len, stream, acc, chunked);
    });
}

// While alive, the plan describes ONE rank's problem: a single shard of width F/D applied to that rank's tokens
// (the launch helpers read H, F, D from the plan).  Used by the per-rank ring-step entry points.
struct OneShardView {
    tsp_mlp_plan_t* plan;
    int F, D;
    explicit OneShardView(tsp_mlp_plan_t* p) : plan(p), F(p->F), D(p->D) {
        plan->F = F / D;
        plan->D = 1;
    }
    ~OneShardView() {
        plan->F = F;
        plan->D = D;
    }
};

// One ring step for `n_ranks` ranks at once (S tokens in all): gate|up GEMM of every rank's tokens against the shard
// in that rank's buffer slot into the [S, F/D] scratch, then the down projection of that shard added to the fp32
// accumulator.  mode: 0 first step, 1 middle, 2 last (rounds to bf16 Y), 3 only step.
tsp_status_t launch_step_gate(tsp_mlp_plan_t* plan, const void* X, const void* cur_g, const void* cur_u, void* A_step,
                              int64_t S, int n_ranks, cudaStream_t cs) {
    const int H = plan->H, F_d = plan->F / plan->D, D = n_ranks;
    tsp_status_t st;
    {
        using Policy = tsp::PairGateUpPolicyT<0>;
        Policy::Params p;
        std::memset(&p, 0, sizeof(p));
        if (!encode_matrix(plan, &p.map_x, X, S, H, 64, 128)) return TSP_ERR_CUDA;
        if (!encode_sharded(plan, &p.map_wg, cur_g, D, H, F_d, 64, 64)) return TSP_ERR_CUDA;
        if (!encode_sharded(plan, &p.map_wu, cur_u, D, H, F_d, 64, 64)) return TSP_ERR_CUDA;
        p.A = static_cast<__nv_bfloat16*>(A_step);
        p.S = static_cast<int>(S); p.H = H; p.F = F_d; p.D = D; p.F_d = F_d;
        p.S_loc = static_cast<int>(S / D);
        p.tiles_per_rank = (p.S_loc + 255) / 256;
        p.m_tiles = D * p.tiles_per_rank;
        p.jl_blocks = F_d / 128;
        p.band = gate_band(plan, p.m_tiles);
        p.rank_indexed = 1;
        p.act = plan->act;
        fill_common(plan, p, p.m_tiles * p.jl_blocks);
        st = launch_pair<Policy>(plan, p, cs);
        if (st != TSP_OK) return st;
    }
    return TSP_OK;
}

tsp_status_t launch_step_down(tsp_mlp_plan_t* plan, const void* cur_d, const void* A_step, float* Yacc, void* Y, int64_t S,
                              int n_ranks, int mode, cudaStream_t cs) {
    const int H = plan->H, F_d = plan->F / plan->D, D = n_ranks;
    tsp_status_t st;
    {
        tsp::PairDownStagedPolicy::Params p;
        std::memset(&p, 0, sizeof(p));
        if (!encode_matrix(plan, &p.map_a, A_step, S, F_d, 64, 128)) return TSP_ERR_CUDA;
        if (!encode_sharded(plan, &p.map_wd, cur_d, D, F_d, H, 64, 64)) return TSP_ERR_CUDA;
        p.Yacc = Yacc;
        p.Y = static_cast<__nv_bfloat16*>(Y);
        if (!encode_carry(plan, &p.carry_tma, Yacc, static_cast<uint64_t>(S / D), D)) return TSP_ERR_CUDA;
        p.S = static_cast<int>(S); p.H = H; p.F_d = F_d; p.D = D;
        p.mode = mode;
        p.S_loc = static_cast<int>(S / D);
        p.tiles_per_rank = (p.S_loc + 255) / 256;
        p.m_tiles = D * p.tiles_per_rank;
        p.n_blocks = H / 256;
        const int group = plan->group > 0 ? plan->group : 8;
        p.group = p.m_tiles < group ? p.m_tiles : group;
        fill_common(plan, p, p.m_tiles * p.n_blocks, 1);   // own scheduler words: may run beside the next step's gate|up GEMM
        st = launch_pair<tsp::PairDownStagedPolicy>(plan, p, cs, kDynDown);
        if (st != TSP_OK) return st;
    }
    return TSP_OK;
}

tsp_status_t launch_forward_step(tsp_mlp_plan_t* plan, const void* X, const void* cur_g, const void* cur_u,
                                 const void* cur_d, void* A_step, float* Yacc, void* Y, int64_t S, int n_ranks, int mode,
                                 cudaStream_t cs) {
    tsp_status_t st = launch_step_gate(plan, X, cur_g, cur_u, A_step, S, n_ranks, cs);
    if (st != TSP_OK) return st;
    return launch_step_down(plan, cur_d, A_step, Yacc, Y, S, n_ranks, mode, cs);
}

// n consecutive ring steps of ONE rank in two launches: gate|up of the rank's tokens against the n shards (A becomes
// [S, n * F/D]), then one down projection whose K loop runs over the n shards in the order given.
tsp_status_t launch_steps_group(tsp_mlp_plan_t* plan, const void* X, const void* Wg0, const void* Wu0, const void* Wd0,
                                size_t stride_bytes, int n, void* A, float* Yacc, void* Y, int64_t S, int mode,
                                cudaStream_t cs) {
    const int H = plan->H, F_d = plan->F / plan->D;
    {
        using Policy = tsp::PairGateUpPolicyT<0>;
        Policy::Params p;
        std::memset(&p, 0, sizeof(p));
        if (!encode_matrix(plan, &p.map_x, X, S, H, 64, 128)) return TSP_ERR_CUDA;
        if (!encode_strided(plan, &p.map_wg, Wg0, n, H, F_d, stride_bytes, 64, 64)) return TSP_ERR_CUDA;
        if (!encode_strided(plan, &p.map_wu, Wu0, n, H, F_d, stride_bytes, 64, 64)) return TSP_ERR_CUDA;
        p.A = static_cast<__nv_bfloat16*>(A);
        p.S = static_cast<int>(S); p.H = H; p.F = n * F_d; p.D = n; p.F_d = F_d;
        p.S_loc = static_cast<int>(S);          // one rank: every token tile belongs to it
        p.tiles_per_rank = (p.S_loc + 255) / 256;
        p.m_tiles = p.tiles_per_rank;
        p.jl_blocks = F_d / 128;
        p.band = gate_band(plan, p.m_tiles);
        p.shared_order = 1;                     // tile order: band -> shard -> column block -> token tile
        p.act = plan->act;
        tsp_status_t st = for_tile_chunks(p.m_tiles, plan->chunk_bands * p.band, false, [&](int first, int count) {
            p.mt_base = first;
            p.m_tiles = count;
            fill_common(plan, p, count * n * p.jl_blocks);
            return launch_pair<Policy>(plan, p, cs);
        });
        if (st != TSP_OK) return st;
    }
    {
        tsp::PairDownStagedPolicy::Params p;
        std::memset(&p, 0, sizeof(p));
        if (!encode_matrix(plan, &p.map_a, A, S, static_cast<uint64_t>(n) * F_d, 64, 128)) return TSP_ERR_CUDA;
        if (!encode_strided(plan, &p.map_wd, Wd0, n, F_d, H, stride_bytes, 64, 64)) return TSP_ERR_CUDA;
        p.Yacc = Yacc;
        p.Y = static_cast<__nv_bfloat16*>(Y);
        if (!encode_carry(plan, &p.carry_tma, Yacc, static_cast<uint64_t>(S), 1)) return TSP_ERR_CUDA;
        p.S = static_cast<int>(S); p.H = H; p.F_d = F_d; p.D = 1;
        p.mode = mode;
        p.n_shards = n;
        p.S_loc = static_cast<int>(S);
        p.tiles_per_rank = (p.S_loc + 255) / 256;
        p.m_tiles = p.tiles_per_rank;
        p.n_blocks = H / 256;
        const int group = plan->group > 0 ? plan->group : 8;
        p.group = p.m_tiles < group ? p.m_tiles : group;
        fill_common(plan, p, p.m_tiles * p.n_blocks);
        return launch_pair<tsp::PairDownStagedPolicy>(plan, p, cs, kDynDown);
    }
}

// Backward of n consecutive ring steps of ONE rank, everything except the weight gradients: dA = dY_p [Wd_0 .. Wd_n-1]^T
// (fp32, [S, n F/D]); the gate|up GEMM over the n shards with the backward epilogue (A, dG, dU, each [S, n F/D]); the
// dX GEMM whose K loop walks the n shards in the order given and carries the fp32 sum from call to call.
tsp_status_t launch_steps_group_backward(tsp_mlp_plan_t* plan, const void* X, const void* Wg0, const void* Wu0,
                                         const void* Wd0, size_t stride_bytes, int n, const void* dY, void* A, void* dG,
                                         void* dU, float* dA, float* dXacc, void* dX, int64_t S, int carry,
                                         Profiler& prof, cudaStream_t cs) {
    const int H = plan->H, F_d = plan->F / plan->D;
    const int m_tiles = static_cast<int>((S + 255) / 256);
    {
        using Policy = tsp::PairDaPolicyT<false>;
        Policy::Params p;
        std::memset(&p, 0, sizeof(p));
        if (!encode_matrix(plan, &p.map_dy, dY, S, H, 64, 128)) return TSP_ERR_CUDA;
        if (!encode_strided(plan, &p.map_wd, Wd0, n, F_d, H, stride_bytes, 64, 128)) return TSP_ERR_CUDA;
        p.dA = dA;
        p.S = static_cast<int>(S); p.H = H; p.F = n * F_d; p.D = 1;
        p.S_loc = static_cast<int>(S);
        p.tiles_per_rank = m_tiles;
        p.m_tiles = m_tiles;
        p.j_tiles = n * F_d / 256;
        p.j_tiles_per_shard = F_d / 256;
        p.band = gate_band(plan, m_tiles);
        tsp_status_t st = for_tile_chunks(m_tiles, plan->chunk_bands * p.band, false, [&](int first, int count) {
            p.mt_base = first;
            p.m_tiles = count;
            fill_common(plan, p, count * p.j_tiles);
            return launch_pair<Policy>(plan, p, cs);
        });
        if (st != TSP_OK) return st;
        prof.mark();
    }
    {
        using Policy = tsp::PairGateUpPolicyT<1>;
        Policy::Params p;
        std::memset(&p, 0, sizeof(p));
        if (!encode_matrix(plan, &p.map_x, X, S, H, 64, 128)) return TSP_ERR_CUDA;
        if (!encode_strided(plan, &p.map_wg, Wg0, n, H, F_d, stride_bytes, 64, 64)) return TSP_ERR_CUDA;
        if (!encode_strided(plan, &p.map_wu, Wu0, n, H, F_d, stride_bytes, 64, 64)) return TSP_ERR_CUDA;
        p.A = static_cast<__nv_bfloat16*>(A);
        p.dA = dA;
        p.dG = static_cast<__nv_bfloat16*>(dG);
        p.dU = static_cast<__nv_bfloat16*>(dU);
        p.S = static_cast<int>(S); p.H = H; p.F = n * F_d; p.D = n; p.F_d = F_d;
        p.S_loc = static_cast<int>(S);
        p.tiles_per_rank = m_tiles;
        p.m_tiles = m_tiles;
        p.jl_blocks = F_d / 128;
        p.band = gate_band(plan, m_tiles);
        p.shared_order = 1;
        p.act = plan->act;
        tsp_status_t st = for_tile_chunks(m_tiles, plan->chunk_bands * p.band, false, [&](int first, int count) {
            p.mt_base = first;
            p.m_tiles = count;
            fill_common(plan, p, count * n * p.jl_blocks);
            return launch_pair<Policy>(plan, p, cs);
        });
        if (st != TSP_OK) return st;
        prof.mark();
    }
    {
        tsp::PairDxPolicy::Params p;
        std::memset(&p, 0, sizeof(p));
        const uint64_t width = static_cast<uint64_t>(n) * F_d;
        if (!encode_matrix(plan, &p.map_dg, dG, S, width, 64, 128)) return TSP_ERR_CUDA;
        if (!encode_matrix(plan, &p.map_du, dU, S, width, 64, 128)) return TSP_ERR_CUDA;
        if (!encode_strided(plan, &p.map_wg, Wg0, n, H, F_d, stride_bytes, 64, 128)) return TSP_ERR_CUDA;
        if (!encode_strided(plan, &p.map_wu, Wu0, n, H, F_d, stride_bytes, 64, 128)) return TSP_ERR_CUDA;
        p.dX = static_cast<__nv_bfloat16*>(dX);
        p.dXacc = dXacc;
        p.carry = carry;
        if (carry != 0 && !encode_carry(plan, &p.carry_tma, dXacc, static_cast<uint64_t>(S), 1)) return TSP_ERR_CUDA;
        p.linear_shards = 1;
        p.S = static_cast<int>(S); p.H = H; p.F = n * F_d; p.D = n; p.F_d = F_d;
        p.S_loc = static_cast<int>(S);
        p.tiles_per_rank = m_tiles;
        p.n_blocks = H / 256;
        const int group = plan->dx_group > 0 ? plan->dx_group : 8;
        tsp_status_t st = for_tile_chunks(m_tiles, plan->chunk_tiles, true, [&](int first, int count) {
            p.mt_base = first;
            p.m_tiles = count;
            p.group = count < group ? count : group;
            p.wide_tiles = mixed_wide_tiles(plan, 2, p.n_blocks, count * p.n_blocks, 2 * n * F_d / 64);
            if (p.wide_tiles > 0) {
                p.carry_tma.epi_off = 0;   // long K loop: the epilogue is a small part, element-wise accesses do (measured)
                fill_common(plan, p, count * p.n_blocks - p.wide_tiles);
                return launch_pair_wide<tsp::PairDxPolicy>(plan, p, cs, kDynDx);
            }
            fill_common(plan, p, count * p.n_blocks);
            return launch_pair<tsp::PairDxPolicy>(plan, p, cs, kDynDx);
        });
        if (st != TSP_OK) return st;
        prof.mark();
    }
    return TSP_OK;
}

// The same n ring steps of one rank as ONE launch (PairFusedStepPolicy): gate|up tiles, then down-projection tiles
// that wait for their token rows of A.  Same tiles, same K order, same epilogues as launch_steps_group: same bits.
bool fused_steps_possible(const tsp_mlp_plan_t* plan, int64_t S) {
    return plan->fuse_steps && (S + 255) / 256 < kCtlReadyCount;   // one counter per token tile + one for all of them
}

tsp_status_t launch_steps_fused(tsp_mlp_plan_t* plan, const void* X, const void* Wg0, const void* Wu0, const void* Wd0,
                                size_t stride_bytes, int n, void* A, float* Yacc, void* Y, int64_t S, int mode,
                                cudaStream_t cs) {
    using Policy = tsp::PairFusedStepPolicy;
    const int H = plan->H, F_d = plan->F / plan->D;
    Policy::Params p;
    std::memset(&p, 0, sizeof(p));
    if (!encode_matrix(plan, &p.map_x, X, S, H, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_strided(plan, &p.map_wg, Wg0, n, H, F_d, stride_bytes, 64, 64)) return TSP_ERR_CUDA;
    if (!encode_strided(plan, &p.map_wu, Wu0, n, H, F_d, stride_bytes, 64, 64)) return TSP_ERR_CUDA;
    if (!encode_matrix(plan, &p.map_a, A, S, static_cast<uint64_t>(n) * F_d, 64, 128)) return TSP_ERR_CUDA;
    if (!encode_strided(plan, &p.map_wd, Wd0, n, F_d, H, stride_bytes, 64, 64)) return TSP_ERR_CUDA;
    p.A = static_cast<__nv_bfloat16*>(A);
    p.Yacc = Yacc;
    p.Y = static_cast<__nv_bfloat16*>(Y);
    if (!encode_carry(plan, &p.carry_tma, Yacc, static_cast<uint64_t>(S), 1)) return TSP_ERR_CUDA;
    p.S_loc = static_cast<int>(S); p.H = H; p.F_d = F_d; p.n_shards = n;
    p.mode = mode;
    p.act = plan->act;
    p.m_tiles = static_cast<int>((S + 255) / 256);
    p.jl_blocks = F_d / 128;
    p.n_blocks = H / 256;
    p.gate_tiles = p.m_tiles * p.jl_blocks * n;
    p.band = gate_band(plan, p.m_tiles);
    const int group = plan->group > 0 ? plan->group : 8;
    p.group = p.m_tiles < group ? p.m_tiles : group;
    int* ready = plan->status_dev + kCtlReadyBase;
    p.ready = ready + plan->ready_parity * kCtlReadyCount;
    p.ready_clear = ready + (plan->ready_parity ^ 1) * kCtlReadyCount;
    p.ready_clear_count = kCtlReadyCount;
    p.ready_target = 8 * p.jl_blocks * n;   // the eight epilogue warps of every gate|up tile of a token tile
    p.ready_all = p.ready + kCtlReadyCount - 1;   // last counter of the set: all token tiles together
    p.ready_all_target = p.ready_target * p.m_tiles;
    plan->ready_parity ^= 1;
    fill_common(plan, p, p.gate_tiles + p.m_tiles * p.n_blocks);
    return launch_pair_kernel(plan, tsp::pair_dyn_kernel<Policy>, p, cs);
}

// ---------------------------------------------------------------------------------------------
// Fixed scratch for tsp_mlp_forward_static: part of the library image, so every GPU that loads the
// library holds these bytes until the process exits.  First 256 bytes: device status word; the rest:
// the bf16 intermediate A = silu(G)*U [S, F].  In host code the array's name is only a stand-in for
// the symbol, not a device address: the address is fetched once per device with cudaGetSymbolAddress.
// ---------------------------------------------------------------------------------------------
constexpr size_t kStaticHeaderBytes = 256;
constexpr size_t kStaticScratchBytes = TSP_MLP_STATIC_SCRATCH_BYTES;
static __device__ __align__(256) unsigned char g_static_scratch[kStaticHeaderBytes + kStaticScratchBytes];

struct StaticDeviceState {
    bool ready;
    unsigned char* scratch;  // device address of g_static_scratch on this device
    int sm_count;
    int max_smem;
    unsigned long long timeout_ns;  // limit of the device-side waits (TSP_MLP_TIMEOUT_MS, read at set-up; default 2 s)
    EncodeTiledFn encode;
};
int g_static_last_cuda_error = 0;   // cudaError_t of the last failed CUDA call inside tsp_mlp_forward_static
constexpr int kMaxStaticDevices = 64;
StaticDeviceState g_static_state[kMaxStaticDevices];
std::mutex g_static_mutex;

// Once per device, with that device current.  Allocates nothing.
tsp_status_t static_device_setup(int dev, StaticDeviceState** out) {
    if (dev < 0 || dev >= kMaxStaticDevices) return TSP_ERR_UNSUPPORTED_DEVICE;
    std::lock_guard<std::mutex> lock(g_static_mutex);
    StaticDeviceState& st = g_static_state[dev];
    if (!st.ready) {
        int major = 0, sms = 0, smem = 0;
        if (cudaDeviceGetAttribute(&major, cudaDevAttrComputeCapabilityMajor, dev) != cudaSuccess) return TSP_ERR_CUDA;
        if (major != 10) return TSP_ERR_UNSUPPORTED_DEVICE;
        if (cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess) return TSP_ERR_CUDA;
        if (cudaDeviceGetAttribute(&smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) != cudaSuccess) return TSP_ERR_CUDA;
        void* fn = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess || !fn)
            return TSP_ERR_CUDA;
        unsigned char* ptr = nullptr;
        if (cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_static_scratch) != cudaSuccess || !ptr)
            return TSP_ERR_CUDA;
        st.scratch = ptr;
        st.timeout_ns = 2000ull * 1000 * 1000;
        if (const char* t = std::getenv("TSP_MLP_TIMEOUT_MS")) {
            const long ms = std::atol(t);
            if (ms > 0) st.timeout_ns = static_cast<unsigned long long>(ms) * 1000 * 1000;
        }
        st.sm_count = sms;
        st.max_smem = smem;
        st.encode = reinterpret_cast<EncodeTiledFn>(fn);
        st.ready = true;
    }
    *out = &st;
    return TSP_OK;
}

}  // namespace

// ---------------------------------------------------------------------------------------------
// C ABI
// ---------------------------------------------------------------------------------------------
extern "C" {

// Device-side part of a plan, common to the MLP and the attention-projection entry points: device properties, the
// tensor-map encoder, the status word, tunables.  The caller has validated the shape arguments it passes.
static tsp_status_t make_plan(int H, int F, int D, const tsp_mlp_options_t* opt, tsp_mlp_plan_t** out);

void tsp_mlp_options_default(tsp_mlp_options_t* o) {
    if (!o) return;
    o->struct_bytes = static_cast<uint32_t>(sizeof(tsp_mlp_options_t));
    o->use_pairs = o->gate_band = o->gate_order = o->down_group = o->dx_group = o->dw_group = TSP_OPT_AUTO;
    o->wide_mask = o->pair_stages = o->chunk_bands = o->chunk_tiles = o->dw_chunk_rounds = TSP_OPT_AUTO;
    o->phase_mask = o->timeout_ms = o->dynamic_tiles = o->fuse_ring_steps = o->tma_carry = TSP_OPT_AUTO;
    o->rank_pair_tiles = o->overlap_launches = TSP_OPT_AUTO;
}

static bool options_valid(const tsp_mlp_options_t* o) {
    if (o->struct_bytes != sizeof(tsp_mlp_options_t)) return false;
    auto in = [](int v, int lo, int hi) { return v == TSP_OPT_AUTO || (v >= lo && v <= hi); };
    return in(o->use_pairs, 0, 1) && in(o->gate_band, 1, 1 << 16) && in(o->gate_order, 0, 1) &&
           in(o->down_group, 1, 1 << 16) && in(o->dx_group, 1, 1 << 16) && in(o->dw_group, 1, 1 << 16) &&
           in(o->wide_mask, 0, 7) && in(o->pair_stages, 2, tsp::kMaxStages) && in(o->chunk_bands, 0, 1 << 16) &&
           in(o->chunk_tiles, 0, 1 << 20) && in(o->dw_chunk_rounds, 0, 1 << 20) && in(o->phase_mask, 0, 3) &&
           in(o->timeout_ms, 1, 60000) && in(o->dynamic_tiles, 0, 15) && in(o->fuse_ring_steps, 0, 1) &&
           in(o->tma_carry, 0, 1) && in(o->rank_pair_tiles, 0, 7) && in(o->overlap_launches, 0, 1);
}

tsp_status_t tsp_mlp_plan_ex(int H, int F, int D, const tsp_mlp_options_t* options, tsp_mlp_plan_t** out) {
    if (!out) return TSP_ERR_INVALID_ARG;
    *out = nullptr;
    if (H <= 0 || F <= 0 || D <= 0 || D > 64) return TSP_ERR_INVALID_ARG;
    if (options && !options_valid(options)) return TSP_ERR_INVALID_ARG;
    if (F % D != 0 || (F / D) % 128 != 0 || H % 256 != 0) return TSP_ERR_UNSUPPORTED_SHAPE;
    if (H > (1 << 20) || F > (1 << 24)) return TSP_ERR_UNSUPPORTED_SHAPE;
    return make_plan(H, F, D, options, out);
}

tsp_status_t tsp_mlp_plan(int H, int F, int D, tsp_mlp_plan_t** out) { return tsp_mlp_plan_ex(H, F, D, nullptr, out); }

static tsp_status_t make_plan(int H, int F, int D, const tsp_mlp_options_t* opt, tsp_mlp_plan_t** out) {
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return TSP_ERR_CUDA;
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, dev);
    if (e != cudaSuccess) return TSP_ERR_CUDA;
    if (prop.major != 10) return TSP_ERR_UNSUPPORTED_DEVICE;

    tsp_mlp_plan_t* plan = new (std::nothrow) tsp_mlp_plan_t();
    if (!plan) return TSP_ERR_INVALID_ARG;
    plan->H = H; plan->F = F; plan->D = D;
    plan->device = dev;
    plan->sm_count = prop.multiProcessorCount;
    plan->max_smem = static_cast<int>(prop.sharedMemPerBlockOptin);
    plan->status_dev = nullptr;
    plan->workspace = nullptr;
    plan->workspace_bytes = 0;
    plan->last_cuda_error = 0;
    plan->profile_next = 0;
    tsp_mlp_options_t o;
    if (opt) o = *opt; else tsp_mlp_options_default(&o);
    // an explicit option wins; a field left at "auto" takes the environment variable, if set, else the default
    auto pick = [](int option, const char* env, int dflt) {
        if (option != TSP_OPT_AUTO) return option;
        const char* v = std::getenv(env);
        return v ? std::atoi(v) : dflt;
    };
    const int timeout_ms = pick(o.timeout_ms, "TSP_MLP_TIMEOUT_MS", 2000);
    plan->timeout_ns = static_cast<unsigned long long>(timeout_ms > 0 ? timeout_ms : 2000) * 1000 * 1000;
    plan->use_pairs = pick(o.use_pairs, "TSP_MLP_PAIR", 1);
    plan->band = pick(o.gate_band, "TSP_MLP_BAND", 0);
    plan->shared_order = pick(o.gate_order, "TSP_MLP_GATE_ORDER", 1);
    plan->group = pick(o.down_group, "TSP_MLP_GROUP", 0);
    plan->pair_stages = pick(o.pair_stages, "TSP_MLP_PAIR_STAGES", 0);
    plan->last_backward_kernels = 3;
    plan->last_forward_kernels = 2;
    plan->launch_count = 0;
    plan->host_ready = false;
    plan->phase_mask = pick(o.phase_mask, "TSP_MLP_PHASES", 3);
    plan->act = TSP_ACT_SILU;
    plan->wide_mask = pick(o.wide_mask, "TSP_MLP_WIDE", -1);   // -1: decide per launch from the tile counts
    plan->dw_group = pick(o.dw_group, "TSP_MLP_DW_GROUP", 0);
    plan->chunk_bands = pick(o.chunk_bands, "TSP_MLP_CHUNK_BANDS", 3);
    plan->chunk_tiles = pick(o.chunk_tiles, "TSP_MLP_CHUNK_TILES", 96);
    // option: 0 = one launch, n > 0 = n rounds; plan / environment: negative = one launch, 0 = about 3 ms per launch
    plan->dw_chunk_rounds = o.dw_chunk_rounds == TSP_OPT_AUTO ? pick(TSP_OPT_AUTO, "TSP_MLP_DW_CHUNK_ROUNDS", 0)
                                                              : (o.dw_chunk_rounds == 0 ? -1 : o.dw_chunk_rounds);
    plan->dx_group = pick(o.dx_group, "TSP_MLP_DX_GROUP", 0);
    // measured (ncu, S = 8192 training shapes): drawing tiles dynamically cuts the DRAM reads of dX from 3.4 to 2.7 GB, of
    // dW from 4.2 to 3.1 GB and of the down projection from 0.91 to 0.85 GB at equal or slightly better speed; the
    // short-K kernels (gate|up, dA) lose 1-2 % to it, so they keep the round-robin
    plan->dynamic_tiles = pick(o.dynamic_tiles, "TSP_MLP_DYNAMIC", kDynDown | kDynDx | kDynDw);
    // measured: one fused launch is on a par with two launches at best (it saves a kernel boundary, but its phase
    // change costs as much), so two launches stay the default
    plan->fuse_steps = pick(o.fuse_ring_steps, "TSP_MLP_FUSE_STEPS", 0);
    plan->ready_parity = 0;
    plan->tma_carry = pick(o.tma_carry, "TSP_MLP_TMA_CARRY", 1);
    plan->tma_dw_max_tokens = pick(TSP_OPT_AUTO, "TSP_MLP_TMA_DW_TOKENS", 4096);
    // measured (S = 8192, D = 8, 7B shapes): two-rank tiles cut the DRAM reads of dX from 2.7 to 2.0 GB and gain 0.7-0.9 %
    // on a training step; for the down projection they lose 1.3 % against the mixed-width list, so only dX takes them.
    // A caller who forces a tile width gets it.
    plan->overlap_launches = pick(o.overlap_launches, "TSP_MLP_OVERLAP_LAUNCHES", 1);
    plan->rank_pair_tiles = pick(o.rank_pair_tiles, "TSP_MLP_RANK_PAIRS", plan->wide_mask >= 0 ? 0 : 2);
    void* fn = nullptr;
    cudaDriverEntryPointQueryResult q;
    e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &q);
    if (e != cudaSuccess || q != cudaDriverEntryPointSuccess || !fn) {
        delete plan;
        return TSP_ERR_CUDA;
    }
    plan->encode = reinterpret_cast<EncodeTiledFn>(fn);
    e = cudaMalloc(reinterpret_cast<void**>(&plan->status_dev), kCtlBytes);
    if (e == cudaSuccess) e = cudaMemset(plan->status_dev, 0, kCtlBytes);
    if (e != cudaSuccess) {
        if (plan->status_dev) cudaFree(plan->status_dev);
        delete plan;
        return TSP_ERR_CUDA;
    }
    *out = plan;
    return TSP_OK;
}

tsp_status_t tsp_mlp_plan_destroy(tsp_mlp_plan_t* plan) {
    if (!plan) return TSP_ERR_INVALID_ARG;
    tsp_mlp_profile_end(plan);
    for (auto& ev : plan->staged_events) cudaEventDestroy(ev);
    if (plan->host_ready) {
        for (auto& ev : plan->host_events) cudaEventDestroy(ev);
        for (auto& ev : plan->host_shard_events) cudaEventDestroy(ev);
        cudaStreamDestroy(plan->host_copy_stream);
        cudaStreamDestroy(plan->host_down_stream);
    }
    if (plan->status_dev) cudaFree(plan->status_dev);
    delete plan;
    return TSP_OK;
}

size_t tsp_mlp_workspace_bytes(const tsp_mlp_plan_t* plan, int64_t S, int pass) {
    if (!plan || S <= 0 || (pass != TSP_WS_FORWARD && pass != TSP_WS_BACKWARD)) return 0;
    const size_t one = align_up(static_cast<size_t>(S) * plan->F * 2, 256);
    return pass == TSP_WS_BACKWARD ? 5 * one : one;   // A, dG, dU in bf16 and dA in fp32
}

size_t tsp_mlp_workspace_bytes_host(const tsp_mlp_plan_t* plan, int64_t S) {
    if (!plan || S <= 0) return 0;
    const size_t a = align_up(static_cast<size_t>(S) * plan->F * 2, 256);
    const size_t x = align_up(static_cast<size_t>(S) * plan->H * 2, 256);
    const size_t w = align_up(static_cast<size_t>(plan->H) * plan->F * 2, 256);
    return a + 2 * x + 3 * w;
}

tsp_status_t tsp_mlp_set_workspace(tsp_mlp_plan_t* plan, void* dev_ptr, size_t bytes) {
    if (!plan) return TSP_ERR_INVALID_ARG;
    if (dev_ptr && (reinterpret_cast<uintptr_t>(dev_ptr) & 255u)) return TSP_ERR_INVALID_ARG;
    plan->workspace = dev_ptr;
    plan->workspace_bytes = dev_ptr ? bytes : 0;
    return TSP_OK;
}

tsp_status_t tsp_mlp_set_activation(tsp_mlp_plan_t* plan, int activation) {
    if (!plan) return TSP_ERR_INVALID_ARG;
    if (activation != TSP_ACT_SILU && activation != TSP_ACT_GELU && activation != TSP_ACT_RELU) return TSP_ERR_INVALID_ARG;
    plan->act = activation;
    return TSP_OK;
}

static tsp_status_t forward_impl(tsp_mlp_plan_t* plan, const void* X, const void* Wg, const void* Wu, const void* Wd,
                                 void* Y, int64_t S, int D, void* cuda_stream, cudaEvent_t wait_before_down);

tsp_status_t tsp_mlp_forward(tsp_mlp_plan_t* plan, const void* X, const void* Wg, const void* Wu, const void* Wd,
                             void* Y, int64_t S, int D, void* cuda_stream) {
    return forward_impl(plan, X, Wg, Wu, Wd, Y, S, D, cuda_stream, nullptr);
}

// `wait_before_down`: if set, the down-projection kernel additionally waits for this event (Wd still arriving).
static tsp_status_t forward_impl(tsp_mlp_plan_t* plan, const void* X, const void* Wg, const void* Wu, const void* Wd,
                                 void* Y, int64_t S, int D, void* cuda_stream, cudaEvent_t wait_before_down) {
    tsp_status_t st = check_call(plan, S, D);
    if (st != TSP_OK) return st;
    if (!X || !Wg || !Wu || !Wd || !Y) return TSP_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(Wg) || !aligned16(Wu) || !aligned16(Wd) || !aligned32(Y)) return TSP_ERR_INVALID_ARG;
    if (!plan->workspace || plan->workspace_bytes < tsp_mlp_workspace_bytes(plan, S, TSP_WS_FORWARD))
        return TSP_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    plan->launch_count = 0;
    Profiler prof(plan, stream);
    const bool pairs = pairs_for_tokens(plan, S);
    if (plan->phase_mask & 1) {
        st = pairs ? launch_gate_up_pair(plan, X, Wg, Wu, plan->workspace, S, stream)
                   : launch_gate_up(plan, X, Wg, Wu, plan->workspace, S, stream);
        if (st != TSP_OK) return st;
    }
    prof.mark();
    if (wait_before_down) {
        cudaError_t e = cudaStreamWaitEvent(stream, wait_before_down, 0);
        if (e != cudaSuccess) return cuda_fail(plan, e);
    }
    if (plan->phase_mask & 2) {
        st = pairs ? launch_down_pair(plan, plan->workspace, Wd, Y, S, stream)
                   : launch_down(plan, plan->workspace, Wd, Y, S, stream);
        if (st != TSP_OK) return st;
    }
    prof.mark();
    plan->last_forward_kernels = plan->launch_count;
    return TSP_OK;
}

tsp_status_t tsp_mlp_forward_host(tsp_mlp_plan_t* plan, const void* X_host, const void* Wg_host, const void* Wu_host,
                                  const void* Wd_host, void* Y_host, int64_t S, int D, void* cuda_stream) {
    tsp_status_t st = check_call(plan, S, D);
    if (st != TSP_OK) return st;
    if (!X_host || !Wg_host || !Wu_host || !Wd_host || !Y_host) return TSP_ERR_INVALID_ARG;
    if (!plan->workspace || plan->workspace_bytes < tsp_mlp_workspace_bytes_host(plan, S)) return TSP_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const int H = plan->H, F = plan->F, F_d = F / D;
    const size_t a = align_up(static_cast<size_t>(S) * F * 2, 256);
    const size_t xb = static_cast<size_t>(S) * H * 2, x = align_up(xb, 256);
    const size_t wb = static_cast<size_t>(H) * F * 2, w = align_up(wb, 256);
    uint8_t* base = static_cast<uint8_t*>(plan->workspace);
    uint8_t* dX = base + a;
    uint8_t* dY = dX + x;
    uint8_t* dWg = dY + x;
    uint8_t* dWu = dWg + w;
    uint8_t* dWd = dWu + w;
    cudaError_t e;
    if (!plan->host_ready) {   // created on first use: two side streams and a few events (no device memory)
        if ((e = cudaStreamCreateWithFlags(&plan->host_copy_stream, cudaStreamNonBlocking)) != cudaSuccess)
            return cuda_fail(plan, e);
        if ((e = cudaStreamCreateWithFlags(&plan->host_down_stream, cudaStreamNonBlocking)) != cudaSuccess)
            return cuda_fail(plan, e);
        for (auto& ev : plan->host_events)
            if ((e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(plan, e);
        plan->host_ready = true;
    }
    while (plan->host_shard_events.size() < static_cast<size_t>(D)) {
        cudaEvent_t ev;
        if ((e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming)) != cudaSuccess) return cuda_fail(plan, e);
        plan->host_shard_events.push_back(ev);
    }
    cudaStream_t up = plan->host_copy_stream, down = plan->host_down_stream;
    // the staging buffers may still be in use by whatever precedes this call on `stream`
    if ((e = cudaEventRecord(plan->host_events[0], stream)) != cudaSuccess) return cuda_fail(plan, e);
    if ((e = cudaStreamWaitEvent(up, plan->host_events[0], 0)) != cudaSuccess) return cuda_fail(plan, e);
    if ((e = cudaStreamWaitEvent(down, plan->host_events[0], 0)) != cudaSuccess) return cuda_fail(plan, e);

    const int tiles_per_rank = static_cast<int>((S / D + 255) / 256), m_tiles = D * tiles_per_rank;
    const int n_blocks = H / 256;
    constexpr int kParts = 4;
    const bool pipelined = pairs_for_tokens(plan, S) && plan->phase_mask == 3 && n_blocks % (2 * kParts) == 0 && m_tiles >= 4;
    if (!pipelined) {
        // small or unusual shapes: upload everything, run the two kernels, download Y
        if ((e = cudaMemcpyAsync(dX, X_host, xb, cudaMemcpyHostToDevice, up)) != cudaSuccess) return cuda_fail(plan, e);
        if ((e = cudaMemcpyAsync(dWg, Wg_host, wb, cudaMemcpyHostToDevice, up)) != cudaSuccess) return cuda_fail(plan, e);
        if ((e = cudaMemcpyAsync(dWu, Wu_host, wb, cudaMemcpyHostToDevice, up)) != cudaSuccess) return cuda_fail(plan, e);
        if ((e = cudaEventRecord(plan->host_events[1], up)) != cudaSuccess) return cuda_fail(plan, e);
        if ((e = cudaMemcpyAsync(dWd, Wd_host, wb, cudaMemcpyHostToDevice, up)) != cudaSuccess) return cuda_fail(plan, e);
        if ((e = cudaEventRecord(plan->host_events[2], up)) != cudaSuccess) return cuda_fail(plan, e);
        if ((e = cudaStreamWaitEvent(stream, plan->host_events[1], 0)) != cudaSuccess) return cuda_fail(plan, e);
        st = forward_impl(plan, dX, dWg, dWu, dWd, dY, S, D, cuda_stream, plan->host_events[2]);
        if (st != TSP_OK) return st;
        if ((e = cudaMemcpyAsync(Y_host, dY, xb, cudaMemcpyDeviceToHost, stream)) != cudaSuccess) return cuda_fail(plan, e);
        return TSP_OK;
    }
    // Uploads in the order they are needed, all on one stream (the link is the bottleneck): X, then shard by shard
    // Wg_k and Wu_k, then Wd in kParts blocks of hidden columns.  The gate|up tiles of shard k are launched as soon as
    // shard k is on the device, the down projection of a column block as soon as its part of Wd is, and every block of
    // Y goes back on a third stream while later uploads are still running (the link is full duplex).
    const size_t shard_bytes = static_cast<size_t>(H) * F_d * 2;
    if ((e = cudaMemcpyAsync(dX, X_host, xb, cudaMemcpyHostToDevice, up)) != cudaSuccess) return cuda_fail(plan, e);
    for (int k = 0; k < D; ++k) {
        if ((e = cudaMemcpyAsync(dWg + k * shard_bytes, static_cast<const uint8_t*>(Wg_host) + k * shard_bytes, shard_bytes,
                                 cudaMemcpyHostToDevice, up)) != cudaSuccess)
            return cuda_fail(plan, e);
        if ((e = cudaMemcpyAsync(dWu + k * shard_bytes, static_cast<const uint8_t*>(Wu_host) + k * shard_bytes, shard_bytes,
                                 cudaMemcpyHostToDevice, up)) != cudaSuccess)
            return cuda_fail(plan, e);
        if ((e = cudaEventRecord(plan->host_shard_events[k], up)) != cudaSuccess) return cuda_fail(plan, e);
    }
    const int nb_per = n_blocks / kParts;
    const size_t col_bytes = static_cast<size_t>(nb_per) * 256 * 2, pitch = static_cast<size_t>(H) * 2;
    for (int q = 0; q < kParts; ++q) {
        if ((e = cudaMemcpy2DAsync(dWd + q * col_bytes, pitch, static_cast<const uint8_t*>(Wd_host) + q * col_bytes, pitch,
                                   col_bytes, static_cast<size_t>(F), cudaMemcpyHostToDevice, up)) != cudaSuccess)
            return cuda_fail(plan, e);
        if ((e = cudaEventRecord(plan->host_events[1 + q], up)) != cudaSuccess) return cuda_fail(plan, e);
    }
    plan->launch_count = 0;
    Profiler prof(plan, stream);
    for (int k = 0; k < D; ++k) {
        if ((e = cudaStreamWaitEvent(stream, plan->host_shard_events[k], 0)) != cudaSuccess) return cuda_fail(plan, e);
        st = launch_gate_up_shard(plan, dX, dWg, dWu, plan->workspace, k, S, stream);
        if (st != TSP_OK) return st;
    }
    prof.mark();
    for (int q = 0; q < kParts; ++q) {
        if ((e = cudaStreamWaitEvent(stream, plan->host_events[1 + q], 0)) != cudaSuccess) return cuda_fail(plan, e);
        st = launch_down_pair(plan, plan->workspace, dWd, dY, S, stream, 0, -1, q * nb_per, nb_per);
        if (st != TSP_OK) return st;
        cudaEvent_t ev = plan->host_events[5];          // reused: the download stream has waited for it before the next record
        if ((e = cudaEventRecord(ev, stream)) != cudaSuccess) return cuda_fail(plan, e);
        if ((e = cudaStreamWaitEvent(down, ev, 0)) != cudaSuccess) return cuda_fail(plan, e);
        if ((e = cudaMemcpy2DAsync(static_cast<uint8_t*>(Y_host) + q * col_bytes, pitch, dY + q * col_bytes, pitch, col_bytes,
                                   static_cast<size_t>(S), cudaMemcpyDeviceToHost, down)) != cudaSuccess)
            return cuda_fail(plan, e);
    }
    prof.mark();
    plan->last_forward_kernels = plan->launch_count;
    // the caller synchronizes `stream`: make it wait for the downloads
    if ((e = cudaEventRecord(plan->host_events[6], down)) != cudaSuccess) return cuda_fail(plan, e);
    if ((e = cudaStreamWaitEvent(stream, plan->host_events[6], 0)) != cudaSuccess) return cuda_fail(plan, e);
    return TSP_OK;
}

// ---------------------------------------------------------------------------------------------
// STAGED mode: Algorithm 2 step by step.  Every ring step is its own pair of launches on the compute
// stream; meanwhile the copy stream moves each rank's current shard buffers into the next rank's
// receive buffers (the stand-in for AsyncRingSendRecv); events implement Wait() and the buffer swap.
// ---------------------------------------------------------------------------------------------
size_t tsp_mlp_workspace_bytes_staged(const tsp_mlp_plan_t* plan, int64_t S) {
    if (!plan || S <= 0) return 0;
    const size_t a_step = align_up(static_cast<size_t>(S) * (plan->F / plan->D) * 2, 256);
    const size_t y_acc = align_up(static_cast<size_t>(S) * plan->H * 4, 256);
    const size_t w = align_up(static_cast<size_t>(plan->H) * plan->F * 2, 256);  // one matrix, all D receive buffers
    return a_step + y_acc + 2 * 3 * w;
}

tsp_status_t tsp_mlp_forward_staged(tsp_mlp_plan_t* plan, const void* X, const void* Wg, const void* Wu,
                                    const void* Wd, void* Y, int64_t S, int D, void* compute_stream,
                                    void* copy_stream) {
    tsp_status_t st = check_call(plan, S, D);
    if (st != TSP_OK) return st;
    if (!X || !Wg || !Wu || !Wd || !Y) return TSP_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(Wg) || !aligned16(Wu) || !aligned16(Wd) || !aligned32(Y)) return TSP_ERR_INVALID_ARG;
    if (compute_stream == copy_stream) return TSP_ERR_INVALID_ARG;
    if (!pairs_for_tokens(plan, S)) return TSP_ERR_UNSUPPORTED_SHAPE;
    if (!plan->workspace || plan->workspace_bytes < tsp_mlp_workspace_bytes_staged(plan, S)) return TSP_ERR_WORKSPACE;
    cudaStream_t cs = static_cast<cudaStream_t>(compute_stream), xs = static_cast<cudaStream_t>(copy_stream);
    const int H = plan->H, F = plan->F, F_d = F / D;
    const size_t a_step_bytes = align_up(static_cast<size_t>(S) * F_d * 2, 256);
    const size_t y_acc_bytes = align_up(static_cast<size_t>(S) * H * 4, 256);
    const size_t w = align_up(static_cast<size_t>(H) * F * 2, 256);
    const size_t shard_bytes = static_cast<size_t>(H) * F_d * 2;
    uint8_t* base = static_cast<uint8_t*>(plan->workspace);
    void* A_step = base;
    float* Yacc = reinterpret_cast<float*>(base + a_step_bytes);
    uint8_t* rb = base + a_step_bytes + y_acc_bytes;  // receive buffers [parity][matrix][rank]
    auto recv = [&](int parity, int m) { return rb + (static_cast<size_t>(parity) * 3 + m) * w; };
    const void* own[3] = {Wg, Wu, Wd};

    const size_t need_events = 2 * static_cast<size_t>(D) + 2;
    while (plan->staged_events.size() < need_events) {
        cudaEvent_t ev;
        cudaError_t e = cudaEventCreateWithFlags(&ev, cudaEventDisableTiming);
        if (e != cudaSuccess) return cuda_fail(plan, e);
        plan->staged_events.push_back(ev);
    }
    auto ev_recv = [&](int t) { return plan->staged_events[2 * t]; };
    auto ev_done = [&](int t) { return plan->staged_events[2 * t + 1]; };
    cudaError_t e;
    // the copy stream starts after whatever precedes this call on the compute stream
    cudaEvent_t ev_start = plan->staged_events[2 * D];
    if ((e = cudaEventRecord(ev_start, cs)) != cudaSuccess) return cuda_fail(plan, e);
    if ((e = cudaStreamWaitEvent(xs, ev_start, 0)) != cudaSuccess) return cuda_fail(plan, e);

    Profiler prof(plan, cs);
    for (int t = 0; t < D; ++t) {
        // ---- AsyncRingSendRecv for step t + 1: rank r's primed buffers <- rank (r-1)'s current buffers
        if (t < D - 1) {
            // the primed buffers (parity (t+1)&1) were last read by the compute of step t-1
            if (t >= 1 && (e = cudaStreamWaitEvent(xs, ev_done(t - 1), 0)) != cudaSuccess) return cuda_fail(plan, e);
            for (int m = 0; m < 3; ++m) {
                const uint8_t* cur = t == 0 ? static_cast<const uint8_t*>(own[m]) : recv(t & 1, m);
                uint8_t* dst = recv((t + 1) & 1, m);
                // ranks 1..D-1 receive from ranks 0..D-2 (one contiguous block), rank 0 from rank D-1
                if (D > 1) {
                    if ((e = cudaMemcpyAsync(dst + shard_bytes, cur, shard_bytes * (D - 1), cudaMemcpyDeviceToDevice, xs)) !=
                        cudaSuccess)
                        return cuda_fail(plan, e);
                }
                if ((e = cudaMemcpyAsync(dst, cur + shard_bytes * (D - 1), shard_bytes, cudaMemcpyDeviceToDevice, xs)) !=
                    cudaSuccess)
                    return cuda_fail(plan, e);
            }
            if ((e = cudaEventRecord(ev_recv(t + 1), xs)) != cudaSuccess) return cuda_fail(plan, e);
        }
        // ---- compute of step t with the current buffers
        if (t >= 1 && (e = cudaStreamWaitEvent(cs, ev_recv(t), 0)) != cudaSuccess) return cuda_fail(plan, e);  // Wait()
        const void* cur_g = t == 0 ? Wg : recv(t & 1, 0);
        const void* cur_u = t == 0 ? Wu : recv(t & 1, 1);
        const void* cur_d = t == 0 ? Wd : recv(t & 1, 2);
        st = launch_forward_step(plan, X, cur_g, cur_u, cur_d, A_step, Yacc, Y, S, D,
                                 D == 1 ? 3 : (t == 0 ? 0 : (t == D - 1 ? 2 : 1)), cs);
        if (st != TSP_OK) return st;
        if ((e = cudaEventRecord(ev_done(t), cs)) != cudaSuccess) return cuda_fail(plan, e);
    }
    prof.mark();
    // later work on the copy stream must not overtake this call: join it back
    cudaEvent_t ev_end = plan->staged_events[2 * D + 1];
    if ((e = cudaEventRecord(ev_end, xs)) != cudaSuccess) return cuda_fail(plan, e);
    if ((e = cudaStreamWaitEvent(cs, ev_end, 0)) != cudaSuccess) return cuda_fail(plan, e);
    return TSP_OK;
}

// ---------------------------------------------------------------------------------------------
// One ring step on one rank's data (every rank on a GPU of its own; the caller moves the shards).
// ---------------------------------------------------------------------------------------------
size_t tsp_mlp_workspace_bytes_ring(const tsp_mlp_plan_t* plan, int64_t S_loc, int pass) {
    if (!plan || S_loc <= 0) return 0;
    const size_t one = align_up(static_cast<size_t>(S_loc) * (plan->F / plan->D) * 2, 256);
    const size_t acc = align_up(static_cast<size_t>(S_loc) * plan->H * 4, 256);
    if (pass == TSP_WS_FORWARD) return 2 * one + acc;                   // A of even steps | A of odd steps | Yacc
    if (pass == TSP_WS_BACKWARD) return 3 * one + 2 * one + acc;        // A, dG, dU | dA (fp32) | dXacc
    return 0;
}

namespace {
// argument checks shared by the forward ring-step entry points; on success the scratch of step t and the accumulator
tsp_status_t ring_step_setup(tsp_mlp_plan_t* plan, int64_t S_loc, int t, int D, void** A_step, float** Yacc) {
    if (!plan || D != plan->D || t < 0 || t >= D) return TSP_ERR_INVALID_ARG;
    if (S_loc < 1 || S_loc > (1ll << 24)) return TSP_ERR_UNSUPPORTED_SHAPE;
    if (!plan->workspace || plan->workspace_bytes < tsp_mlp_workspace_bytes_ring(plan, S_loc, TSP_WS_FORWARD))
        return TSP_ERR_WORKSPACE;
    const size_t one = align_up(static_cast<size_t>(S_loc) * (plan->F / plan->D) * 2, 256);
    uint8_t* base = static_cast<uint8_t*>(plan->workspace);
    *A_step = base + static_cast<size_t>(t & 1) * one;   // two scratch buffers alternate, so that the down projection
    *Yacc = reinterpret_cast<float*>(base + 2 * one);    // of step t may overlap the gate|up GEMM of step t + 1
    return TSP_OK;
}
}  // namespace

tsp_status_t tsp_mlp_ring_step_gate(tsp_mlp_plan_t* plan, const void* X_p, const void* Wg_k, const void* Wu_k,
                                    int64_t S_loc, int t, int D, void* cuda_stream) {
    void* A_step = nullptr;
    float* Yacc = nullptr;
    tsp_status_t st = ring_step_setup(plan, S_loc, t, D, &A_step, &Yacc);
    if (st != TSP_OK) return st;
    if (!X_p || !Wg_k || !Wu_k) return TSP_ERR_INVALID_ARG;
    if (!aligned16(X_p) || !aligned16(Wg_k) || !aligned16(Wu_k)) return TSP_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(cuda_stream);
    Profiler prof(plan, cs);
    st = launch_step_gate(plan, X_p, Wg_k, Wu_k, A_step, S_loc, 1, cs);
    prof.mark();
    return st;
}

tsp_status_t tsp_mlp_ring_step_down(tsp_mlp_plan_t* plan, const void* Wd_k, void* Y_p, int64_t S_loc, int t, int D,
                                    void* cuda_stream) {
    void* A_step = nullptr;
    float* Yacc = nullptr;
    tsp_status_t st = ring_step_setup(plan, S_loc, t, D, &A_step, &Yacc);
    if (st != TSP_OK) return st;
    if (!Wd_k || !Y_p) return TSP_ERR_INVALID_ARG;
    if (!aligned16(Wd_k) || !aligned32(Y_p)) return TSP_ERR_INVALID_ARG;
    cudaStream_t cs = static_cast<cudaStream_t>(cuda_stream);
    Profiler prof(plan, cs);
    st = launch_step_down(plan, Wd_k, A_step, Yacc, Y_p, S_loc, 1, D == 1 ? 3 : (t == 0 ? 0 : (t == D - 1 ? 2 : 1)), cs);
    prof.mark();
    return st;
}

tsp_status_t tsp_mlp_ring_step(tsp_mlp_plan_t* plan, const void* X_p, const void* Wg_k, const void* Wu_k,
                               const void* Wd_k, void* Y_p, int64_t S_loc, int t, int D, void* cuda_stream) {
    if (!Wd_k || !Y_p || !aligned16(Wd_k) || !aligned32(Y_p)) return TSP_ERR_INVALID_ARG;   // before anything is launched
    if (plan && fused_steps_possible(plan, S_loc)) {
        void* A_step = nullptr;
        float* Yacc = nullptr;
        tsp_status_t fs = ring_step_setup(plan, S_loc, t, D, &A_step, &Yacc);
        if (fs != TSP_OK) return fs;
        if (!X_p || !Wg_k || !Wu_k || !aligned16(X_p) || !aligned16(Wg_k) || !aligned16(Wu_k)) return TSP_ERR_INVALID_ARG;
        cudaStream_t cs = static_cast<cudaStream_t>(cuda_stream);
        plan->launch_count = 0;
        Profiler prof(plan, cs);
        fs = launch_steps_fused(plan, X_p, Wg_k, Wu_k, Wd_k, static_cast<size_t>(plan->H) * (plan->F / plan->D) * 2, 1,
                                A_step, Yacc, Y_p, S_loc, D == 1 ? 3 : (t == 0 ? 0 : (t == D - 1 ? 2 : 1)), cs);
        prof.mark();
        plan->last_forward_kernels = plan->launch_count;
        return fs;
    }
    tsp_status_t st = tsp_mlp_ring_step_gate(plan, X_p, Wg_k, Wu_k, S_loc, t, D, cuda_stream);
    if (st != TSP_OK) return st;
    return tsp_mlp_ring_step_down(plan, Wd_k, Y_p, S_loc, t, D, cuda_stream);
}

size_t tsp_mlp_workspace_bytes_ring_group(const tsp_mlp_plan_t* plan, int64_t S_loc, int n_shards) {
    if (!plan || S_loc <= 0 || n_shards < 1 || n_shards > plan->D) return 0;
    return align_up(static_cast<size_t>(S_loc) * (plan->F / plan->D) * 2 * n_shards, 256) +
           align_up(static_cast<size_t>(S_loc) * plan->H * 4, 256);            // Yacc | A of the group
}

tsp_status_t tsp_mlp_ring_steps(tsp_mlp_plan_t* plan, const void* X_p, const void* Wg_first, const void* Wu_first,
                                const void* Wd_first, int64_t shard_stride, int n_shards, void* Y_p, int64_t S_loc,
                                int t_first, int D, void* cuda_stream) {
    if (!plan || D != plan->D || n_shards < 1 || t_first < 0 || t_first + n_shards > D) return TSP_ERR_INVALID_ARG;
    if (S_loc < 1 || S_loc > (1ll << 24)) return TSP_ERR_UNSUPPORTED_SHAPE;
    if (!X_p || !Wg_first || !Wu_first || !Wd_first || !Y_p) return TSP_ERR_INVALID_ARG;
    if (!aligned16(X_p) || !aligned16(Wg_first) || !aligned16(Wu_first) || !aligned16(Wd_first) || !aligned32(Y_p))
        return TSP_ERR_INVALID_ARG;
    const int64_t shard_elems = static_cast<int64_t>(plan->H) * (plan->F / plan->D);
    if (n_shards > 1 && (shard_stride < shard_elems || shard_stride % 8 != 0)) return TSP_ERR_INVALID_ARG;
    if (!plan->workspace || plan->workspace_bytes < tsp_mlp_workspace_bytes_ring_group(plan, S_loc, n_shards))
        return TSP_ERR_WORKSPACE;
    cudaStream_t cs = static_cast<cudaStream_t>(cuda_stream);
    // the accumulator comes first, so that its place does not depend on the size of the group
    float* Yacc = static_cast<float*>(plan->workspace);
    uint8_t* base = static_cast<uint8_t*>(plan->workspace) + align_up(static_cast<size_t>(S_loc) * plan->H * 4, 256);
    const bool first = t_first == 0, last = t_first + n_shards == D;
    const int mode = first && last ? 3 : (first ? 0 : (last ? 2 : 1));
    const size_t stride_bytes = n_shards > 1 ? static_cast<size_t>(shard_stride) * 2 : static_cast<size_t>(shard_elems) * 2;
    plan->launch_count = 0;
    Profiler prof(plan, cs);
    tsp_status_t st = fused_steps_possible(plan, S_loc)
                          ? launch_steps_fused(plan, X_p, Wg_first, Wu_first, Wd_first, stride_bytes, n_shards, base, Yacc,
                                               Y_p, S_loc, mode, cs)
                          : launch_steps_group(plan, X_p, Wg_first, Wu_first, Wd_first, stride_bytes, n_shards, base, Yacc,
                                               Y_p, S_loc, mode, cs);
    prof.mark();
    plan->last_forward_kernels = plan->launch_count;
    return st;
}

tsp_status_t tsp_mlp_ring_step_backward_dx(tsp_mlp_plan_t* plan, const void* X_p, const void* Wg_k, const void* Wu_k,
                                           const void* Wd_k, const void* dY_p, void* dX_p, int64_t S_loc, int t, int D,
                                           void* cuda_stream) {
    if (!plan || D != plan->D || t < 0 || t >= D) return TSP_ERR_INVALID_ARG;
    if (S_loc < 1 || S_loc > (1ll << 24) || (plan->F / plan->D) % 256 != 0) return TSP_ERR_UNSUPPORTED_SHAPE;
    if (!X_p || !Wg_k || !Wu_k || !Wd_k || !dY_p || !dX_p) return TSP_ERR_INVALID_ARG;
    if (!aligned16(X_p) || !aligned16(Wg_k) || !aligned16(Wu_k) || !aligned16(Wd_k) || !aligned16(dY_p) || !aligned32(dX_p))
        return TSP_ERR_INVALID_ARG;
    if (!plan->workspace || plan->workspace_bytes < tsp_mlp_workspace_bytes_ring(plan, S_loc, TSP_WS_BACKWARD))
        return TSP_ERR_WORKSPACE;
    cudaStream_t cs = static_cast<cudaStream_t>(cuda_stream);
    const size_t one = align_up(static_cast<size_t>(S_loc) * (plan->F / plan->D) * 2, 256);
    uint8_t* base = static_cast<uint8_t*>(plan->workspace);
    void* A = base;
    void* dG = base + one;
    void* dU = base + 2 * one;
    float* dA = reinterpret_cast<float*>(base + 3 * one);
    float* dXacc = reinterpret_cast<float*>(base + 5 * one);
    Profiler prof(plan, cs);
    OneShardView view(plan);
    tsp_status_t st = launch_da_pair(plan, dY_p, Wd_k, dA, S_loc, cs);
    if (st != TSP_OK) return st;
    prof.mark();
    st = launch_gate_pair<1>(plan, X_p, Wg_k, Wu_k, A, dA, dG, dU, S_loc, cs);
    if (st != TSP_OK) return st;
    prof.mark();
    const int carry = D == 1 ? 0 : (t == 0 ? 1 : (t == D - 1 ? 3 : 2));
    st = launch_bwd_dx_pair(plan, dG, dU, Wg_k, Wu_k, dX_p, S_loc, cs, dXacc, carry);
    prof.mark();
    return st;
}

tsp_status_t tsp_mlp_ring_step_backward_dw(tsp_mlp_plan_t* plan, const void* X_p, const void* dY_p, float* dWg_k,
                                           float* dWu_k, float* dWd_k, int64_t S_loc, int accumulate, int D,
                                           void* cuda_stream) {
    if (!plan || D != plan->D || (accumulate != 0 && accumulate != 1)) return TSP_ERR_INVALID_ARG;
    if (S_loc < 1 || S_loc > (1ll << 24) || (plan->F / plan->D) % 256 != 0) return TSP_ERR_UNSUPPORTED_SHAPE;
    if (!X_p || !dY_p || !dWg_k || !dWu_k || !dWd_k) return TSP_ERR_INVALID_ARG;
    if (!aligned16(X_p) || !aligned16(dY_p) || !aligned32(dWg_k) || !aligned32(dWu_k) || !aligned32(dWd_k))
        return TSP_ERR_INVALID_ARG;
    if (!plan->workspace || plan->workspace_bytes < tsp_mlp_workspace_bytes_ring(plan, S_loc, TSP_WS_BACKWARD))
        return TSP_ERR_WORKSPACE;
    cudaStream_t cs = static_cast<cudaStream_t>(cuda_stream);
    const size_t one = align_up(static_cast<size_t>(S_loc) * (plan->F / plan->D) * 2, 256);
    uint8_t* base = static_cast<uint8_t*>(plan->workspace);
    Profiler prof(plan, cs);
    OneShardView view(plan);
    tsp_status_t st = launch_dw_all(plan, X_p, dY_p, base, base + one, base + 2 * one, dWg_k, dWu_k, dWd_k, S_loc, cs,
                                    accumulate);
    prof.mark();
    return st;
}

size_t tsp_mlp_workspace_bytes_ring_group_backward(const tsp_mlp_plan_t* plan, int64_t S_loc, int n_shards) {
    if (!plan || S_loc <= 0 || n_shards < 1 || n_shards > plan->D) return 0;
    const size_t one = align_up(static_cast<size_t>(S_loc) * (plan->F / plan->D) * 2 * n_shards, 256);
    return align_up(static_cast<size_t>(S_loc) * plan->H * 4, 256) + 5 * one;   // dXacc | A | dG | dU | dA (fp32)
}

namespace {
// layout of the grouped backward workspace; the accumulator comes first so that its place does not depend on n
struct GroupBackwardWs {
    float* dXacc;
    uint8_t *A, *dG, *dU;
    float* dA;
};
GroupBackwardWs group_backward_ws(const tsp_mlp_plan_t* plan, int64_t S_loc, int n) {
    const size_t one = align_up(static_cast<size_t>(S_loc) * (plan->F / plan->D) * 2 * n, 256);
    uint8_t* base = static_cast<uint8_t*>(plan->workspace);
    GroupBackwardWs w;
    w.dXacc = reinterpret_cast<float*>(base);
    base += align_up(static_cast<size_t>(S_loc) * plan->H * 4, 256);
    w.A = base;
    w.dG = base + one;
    w.dU = base + 2 * one;
    w.dA = reinterpret_cast<float*>(base + 3 * one);
    return w;
}
}  // namespace

tsp_status_t tsp_mlp_ring_steps_backward_dx(tsp_mlp_plan_t* plan, const void* X_p, const void* Wg_first,
                                            const void* Wu_first, const void* Wd_first, int64_t shard_stride,
                                            int n_shards, const void* dY_p, void* dX_p, int64_t S_loc, int t_first, int D,
                                            void* cuda_stream) {
    if (!plan || D != plan->D || n_shards < 1 || t_first < 0 || t_first + n_shards > D) return TSP_ERR_INVALID_ARG;
    if (S_loc < 1 || S_loc > (1ll << 24) || (plan->F / plan->D) % 256 != 0) return TSP_ERR_UNSUPPORTED_SHAPE;
    if (!X_p || !Wg_first || !Wu_first || !Wd_first || !dY_p || !dX_p) return TSP_ERR_INVALID_ARG;
    if (!aligned16(X_p) || !aligned16(Wg_first) || !aligned16(Wu_first) || !aligned16(Wd_first) || !aligned16(dY_p) ||
        !aligned32(dX_p))
        return TSP_ERR_INVALID_ARG;
    const int64_t shard_elems = static_cast<int64_t>(plan->H) * (plan->F / plan->D);
    if (n_shards > 1 && (shard_stride < shard_elems || shard_stride % 8 != 0)) return TSP_ERR_INVALID_ARG;
    if (!plan->workspace || plan->workspace_bytes < tsp_mlp_workspace_bytes_ring_group_backward(plan, S_loc, n_shards))
        return TSP_ERR_WORKSPACE;
    cudaStream_t cs = static_cast<cudaStream_t>(cuda_stream);
    const GroupBackwardWs w = group_backward_ws(plan, S_loc, n_shards);
    const bool first = t_first == 0, last = t_first + n_shards == D;
    const int carry = first && last ? 0 : (first ? 1 : (last ? 3 : 2));
    const size_t stride_bytes = n_shards > 1 ? static_cast<size_t>(shard_stride) * 2 : static_cast<size_t>(shard_elems) * 2;
    plan->launch_count = 0;
    Profiler prof(plan, cs);
    tsp_status_t st = launch_steps_group_backward(plan, X_p, Wg_first, Wu_first, Wd_first, stride_bytes, n_shards, dY_p,
                                                  w.A, w.dG, w.dU, w.dA, w.dXacc, dX_p, S_loc, carry, prof, cs);
    plan->last_backward_kernels = plan->launch_count;
    return st;
}

tsp_status_t tsp_mlp_ring_steps_backward_dw(tsp_mlp_plan_t* plan, const void* X_p, const void* dY_p, float* dWg_k,
                                            float* dWu_k, float* dWd_k, int64_t S_loc, int shard_in_group, int n_shards,
                                            int accumulate, int D, void* cuda_stream) {
    if (!plan || D != plan->D || (accumulate != 0 && accumulate != 1)) return TSP_ERR_INVALID_ARG;
    if (n_shards < 1 || n_shards > D || shard_in_group < 0 || shard_in_group >= n_shards) return TSP_ERR_INVALID_ARG;
    if (S_loc < 1 || S_loc > (1ll << 24) || (plan->F / plan->D) % 256 != 0) return TSP_ERR_UNSUPPORTED_SHAPE;
    if (!X_p || !dY_p || !dWg_k || !dWu_k || !dWd_k) return TSP_ERR_INVALID_ARG;
    if (!aligned16(X_p) || !aligned16(dY_p) || !aligned32(dWg_k) || !aligned32(dWu_k) || !aligned32(dWd_k))
        return TSP_ERR_INVALID_ARG;
    if (!plan->workspace || plan->workspace_bytes < tsp_mlp_workspace_bytes_ring_group_backward(plan, S_loc, n_shards))
        return TSP_ERR_WORKSPACE;
    cudaStream_t cs = static_cast<cudaStream_t>(cuda_stream);
    const GroupBackwardWs w = group_backward_ws(plan, S_loc, n_shards);
    const int F_d = plan->F / plan->D;
    const size_t col = static_cast<size_t>(shard_in_group) * F_d * 2;   // this shard's column block of A, dG, dU
    Profiler prof(plan, cs);
    OneShardView view(plan);
    tsp_status_t st = launch_dw_all(plan, X_p, dY_p, w.A + col, w.dG + col, w.dU + col, dWg_k, dWu_k, dWd_k, S_loc, cs,
                                    accumulate, static_cast<int64_t>(n_shards) * F_d);
    prof.mark();
    return st;
}

// ---------------------------------------------------------------------------------------------
// Stored-activation training path (the "no recomputation" regime of the activation-memory analysis): the forward
// pass keeps A, P = U*sigma'(G) and Q = sigma(G) in a caller-owned buffer; the backward pass then needs no gate|up GEMM.
// ---------------------------------------------------------------------------------------------
size_t tsp_mlp_saved_bytes(const tsp_mlp_plan_t* plan, int64_t S) {
    if (!plan || S <= 0) return 0;
    return 3 * align_up(static_cast<size_t>(S) * plan->F * 2, 256);
}

static tsp_status_t check_saved_shapes(const tsp_mlp_plan_t* plan, int64_t S) {
    if (!pairs_for_tokens(plan, S) || plan->F % 256 != 0) return TSP_ERR_UNSUPPORTED_SHAPE;
    return TSP_OK;
}

tsp_status_t tsp_mlp_forward_save(tsp_mlp_plan_t* plan, const void* X, const void* Wg, const void* Wu, const void* Wd,
                                  void* Y, void* saved, int64_t S, int D, void* cuda_stream) {
    tsp_status_t st = check_call(plan, S, D);
    if (st != TSP_OK) return st;
    if (!X || !Wg || !Wu || !Wd || !Y || !saved) return TSP_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(Wg) || !aligned16(Wu) || !aligned16(Wd) || !aligned32(Y) ||
        (reinterpret_cast<uintptr_t>(saved) & 255u))
        return TSP_ERR_INVALID_ARG;
    if ((st = check_saved_shapes(plan, S)) != TSP_OK) return st;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t one = align_up(static_cast<size_t>(S) * plan->F * 2, 256);
    uint8_t* base = static_cast<uint8_t*>(saved);
    Profiler prof(plan, stream);
    st = launch_gate_pair<2>(plan, X, Wg, Wu, base, nullptr, base + one, base + 2 * one, S, stream);
    if (st != TSP_OK) return st;
    prof.mark();
    st = launch_down_pair(plan, base, Wd, Y, S, stream);
    if (st != TSP_OK) return st;
    prof.mark();
    return TSP_OK;
}

tsp_status_t tsp_mlp_backward_saved(tsp_mlp_plan_t* plan, const void* X, const void* Wg, const void* Wu, const void* Wd,
                                    const void* dY, const void* saved, void* dX, float* dWg, float* dWu, float* dWd,
                                    int64_t S, int D, void* cuda_stream) {
    tsp_status_t st = check_call(plan, S, D);
    if (st != TSP_OK) return st;
    if (!X || !Wg || !Wu || !Wd || !dY || !saved || !dX || !dWg || !dWu || !dWd) return TSP_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(Wg) || !aligned16(Wu) || !aligned16(Wd) || !aligned16(dY) || !aligned32(dX) ||
        !aligned32(dWg) || !aligned32(dWu) || !aligned32(dWd) || (reinterpret_cast<uintptr_t>(saved) & 255u))
        return TSP_ERR_INVALID_ARG;
    if ((st = check_saved_shapes(plan, S)) != TSP_OK) return st;
    const size_t one = align_up(static_cast<size_t>(S) * plan->F * 2, 256);
    if (!plan->workspace || plan->workspace_bytes < 2 * one) return TSP_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const uint8_t* sv = static_cast<const uint8_t*>(saved);
    uint8_t* ws = static_cast<uint8_t*>(plan->workspace);
    void* dG = ws;
    void* dU = ws + one;
    Profiler prof(plan, stream);
    st = launch_da_pair_t<true>(plan, dY, Wd, nullptr, sv + one, sv + 2 * one, dG, dU, S, stream);
    if (st != TSP_OK) return st;
    prof.mark();
    st = launch_bwd_dx_pair(plan, dG, dU, Wg, Wu, dX, S, stream);
    if (st != TSP_OK) return st;
    prof.mark();
    st = launch_dw_all(plan, X, dY, sv, dG, dU, dWg, dWu, dWd, S, stream, 0);
    if (st != TSP_OK) return st;
    prof.mark();
    return TSP_OK;
}

tsp_status_t tsp_mlp_backward(tsp_mlp_plan_t* plan, const void* X, const void* Wg, const void* Wu, const void* Wd,
                              const void* dY, void* dX, float* dWg, float* dWu, float* dWd, int64_t S, int D,
                              void* cuda_stream) {
    tsp_status_t st = check_call(plan, S, D);
    if (st != TSP_OK) return st;
    if (!X || !Wg || !Wu || !Wd || !dY || !dX || !dWg || !dWu || !dWd) return TSP_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(Wg) || !aligned16(Wu) || !aligned16(Wd) || !aligned16(dY) || !aligned32(dX) ||
        !aligned32(dWg) || !aligned32(dWu) || !aligned32(dWd))
        return TSP_ERR_INVALID_ARG;
    if (!plan->workspace || plan->workspace_bytes < tsp_mlp_workspace_bytes(plan, S, TSP_WS_BACKWARD))
        return TSP_ERR_WORKSPACE;
    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    const size_t one = align_up(static_cast<size_t>(S) * plan->F * 2, 256);
    uint8_t* base = static_cast<uint8_t*>(plan->workspace);
    void* A = base;
    void* dG = base + one;
    void* dU = base + 2 * one;
    plan->launch_count = 0;
    Profiler prof(plan, stream);
    const bool pairs = pairs_for_tokens(plan, S);
    if (pairs && plan->F % 256 == 0) {
        // dA in fp32 by a full-rate GEMM, then the gate|up GEMM whose epilogue consumes it
        float* dA = reinterpret_cast<float*>(base + 3 * one);
        st = launch_da_pair(plan, dY, Wd, dA, S, stream);
        if (st != TSP_OK) return st;
        prof.mark();
        st = launch_gate_pair<1>(plan, X, Wg, Wu, A, dA, dG, dU, S, stream);
    } else {
        st = launch_bwd_gate(plan, X, Wg, Wu, Wd, dY, A, dG, dU, S, stream);
    }
    if (st != TSP_OK) return st;
    prof.mark();
    st = pairs ? launch_bwd_dx_pair(plan, dG, dU, Wg, Wu, dX, S, stream)
               : launch_bwd_dx(plan, dG, dU, Wg, Wu, dX, S, stream);
    if (st != TSP_OK) return st;
    prof.mark();
    st = launch_dw_all(plan, X, dY, A, dG, dU, dWg, dWu, dWd, S, stream, 0);
    if (st != TSP_OK) return st;
    prof.mark();
    plan->last_backward_kernels = plan->launch_count;
    return TSP_OK;
}

tsp_status_t tsp_mlp_forward_static(int H, int F, int D, const void* X, const void* Wg, const void* Wu,
                                    const void* Wd, void* Y, int64_t S, int* timed_out_host, void* cuda_stream) {
    if (H <= 0 || F <= 0 || D <= 0 || D > 64 || S <= 0) return TSP_ERR_INVALID_ARG;
    if (F % D != 0 || (F / D) % 128 != 0 || H % 256 != 0) return TSP_ERR_UNSUPPORTED_SHAPE;
    if (S % D != 0) return TSP_ERR_UNSUPPORTED_SHAPE;
    if (!X || !Wg || !Wu || !Wd || !Y) return TSP_ERR_INVALID_ARG;
    if (!aligned16(X) || !aligned16(Wg) || !aligned16(Wu) || !aligned16(Wd) || !aligned16(Y)) return TSP_ERR_INVALID_ARG;
    // the intermediate must fit the fixed scratch: S * F bf16 elements
    if (static_cast<unsigned long long>(S) * static_cast<unsigned long long>(F) * 2ull > kStaticScratchBytes)
        return TSP_ERR_STATIC_LIMIT;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return TSP_ERR_CUDA;
    StaticDeviceState* sd = nullptr;
    tsp_status_t st = static_device_setup(dev, &sd);
    if (st != TSP_OK) return st;

    // A plan-shaped bundle on the host stack (no device memory behind it) so the ordinary launch code is reused.
    tsp_mlp_plan_t tmp{};
    tmp.H = H; tmp.F = F; tmp.D = D;
    tmp.device = dev;
    tmp.sm_count = sd->sm_count;
    tmp.max_smem = sd->max_smem;
    tmp.status_dev = reinterpret_cast<int*>(sd->scratch);
    tmp.workspace = sd->scratch + kStaticHeaderBytes;
    tmp.workspace_bytes = kStaticScratchBytes;
    tmp.last_cuda_error = 0;
    tmp.timeout_ns = sd->timeout_ns;
    tmp.encode = sd->encode;
    tmp.profile_next = 0;

    cudaStream_t stream = static_cast<cudaStream_t>(cuda_stream);
    // The array keeps what the previous call left: the status word has to start at zero.
    {
        cudaError_t e = cudaMemsetAsync(sd->scratch, 0, kStaticHeaderBytes, stream);
        if (e != cudaSuccess) {
            g_static_last_cuda_error = static_cast<int>(e);
            return TSP_ERR_CUDA;
        }
    }
    st = launch_gate_up(&tmp, X, Wg, Wu, tmp.workspace, S, stream);
    if (st == TSP_OK) st = launch_down(&tmp, tmp.workspace, Wd, Y, S, stream);
    if (st != TSP_OK) {
        g_static_last_cuda_error = tmp.last_cuda_error;   // the stack plan is gone after this call
        return st;
    }
    if (timed_out_host) {
        cudaError_t e = cudaMemcpyAsync(timed_out_host, sd->scratch, sizeof(int), cudaMemcpyDeviceToHost, stream);
        if (e != cudaSuccess) {
            g_static_last_cuda_error = static_cast<int>(e);
            return TSP_ERR_CUDA;
        }
    }
    return TSP_OK;
}

tsp_status_t tsp_mlp_status(tsp_mlp_plan_t* plan) {
    if (!plan) return TSP_ERR_INVALID_ARG;
    int v = 0;
    cudaError_t e = cudaMemcpy(&v, plan->status_dev, sizeof(int), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(plan, e);
    if (v != 0) {
        plan->last_cuda_error = v;
        // kernels that gave up may have left scheduler words and ready counters half-way: start from zero again
        e = cudaMemset(plan->status_dev, 0, kCtlBytes);
        plan->ready_parity = 0;
        if (e != cudaSuccess) return cuda_fail(plan, e);
        return TSP_ERR_DEVICE_TIMEOUT;
    }
    return TSP_OK;
}

tsp_status_t tsp_mlp_selftest_wait_expiry(tsp_mlp_plan_t* plan, int limit_ms, void* cuda_stream) {
    if (!plan || limit_ms <= 0 || limit_ms > 1000) return TSP_ERR_INVALID_ARG;
    tsp::wait_expiry_selftest_kernel<<<1, 32, 0, static_cast<cudaStream_t>(cuda_stream)>>>(
        plan->status_dev, static_cast<unsigned long long>(limit_ms) * 1000 * 1000);
    cudaError_t e = cudaGetLastError();
    return e == cudaSuccess ? TSP_OK : cuda_fail(plan, e);
}

const char* tsp_mlp_error_string(tsp_status_t s) {
    switch (s) {
        case TSP_OK: return "ok";
        case TSP_ERR_INVALID_ARG: return "invalid argument";
        case TSP_ERR_UNSUPPORTED_SHAPE: return "unsupported shape";
        case TSP_ERR_UNSUPPORTED_DEVICE: return "unsupported device (needs compute capability 10.x)";
        case TSP_ERR_CUDA: return "CUDA call failed";
        case TSP_ERR_WORKSPACE: return "workspace missing or too small";
        case TSP_ERR_DEVICE_TIMEOUT: return "device-side wait timed out";
        case TSP_ERR_STATIC_LIMIT: return "problem too large for the fixed scratch of tsp_mlp_forward_static (S*F*2 bytes > TSP_MLP_STATIC_SCRATCH_BYTES)";
    }
    return "unknown status";
}

int tsp_mlp_last_cuda_error(const tsp_mlp_plan_t* plan) { return plan ? plan->last_cuda_error : g_static_last_cuda_error; }

tsp_status_t tsp_mlp_ring_order(const tsp_mlp_plan_t* plan, int* table_host) {
    if (!plan || !table_host) return TSP_ERR_INVALID_ARG;
    const int D = plan->D;
    for (int r = 0; r < D; ++r)
        for (int t = 0; t < D; ++t) table_host[r * D + t] = (r - t + D) % D;
    return TSP_OK;
}

tsp_status_t tsp_mlp_profile_begin(tsp_mlp_plan_t* plan, int max_calls) {
    if (!plan || max_calls <= 0 || max_calls > 4096) return TSP_ERR_INVALID_ARG;
    tsp_mlp_profile_end(plan);
    plan->profile.resize(max_calls);
    for (auto& c : plan->profile) {
        c.n_kernels = 0;
        for (auto& ev : c.ev) {
            cudaError_t e = cudaEventCreate(&ev);
            if (e != cudaSuccess) return cuda_fail(plan, e);
        }
    }
    plan->profile_next = 0;
    return TSP_OK;
}

tsp_status_t tsp_mlp_profile_read(tsp_mlp_plan_t* plan, int call_index, int* n_kernels_out, float* ms_out) {
    if (!plan || !n_kernels_out || !ms_out) return TSP_ERR_INVALID_ARG;
    if (call_index < 0 || call_index >= plan->profile_next) return TSP_ERR_INVALID_ARG;
    ProfileCall& c = plan->profile[call_index];
    *n_kernels_out = c.n_kernels;
    for (int i = 0; i < c.n_kernels; ++i) {
        cudaError_t e = cudaEventElapsedTime(&ms_out[i], c.ev[i], c.ev[i + 1]);
        if (e != cudaSuccess) return cuda_fail(plan, e);
    }
    return TSP_OK;
}

tsp_status_t tsp_mlp_profile_end(tsp_mlp_plan_t* plan) {
    if (!plan) return TSP_ERR_INVALID_ARG;
    for (auto& c : plan->profile)
        for (auto& ev : c.ev) cudaEventDestroy(ev);
    plan->profile.clear();
    plan->profile_next = 0;
    return TSP_OK;
}

int tsp_mlp_kernels_per_call(const tsp_mlp_plan_t* plan, int pass) {
    if (!plan) return 0;
    return pass == TSP_WS_BACKWARD ? plan->last_backward_kernels : plan->last_forward_kernels;
}

}  // extern "C"

#ifdef TSP_TRACE
// development builds only: where the kernels of pair_kernels.cuh write their time stamps (8 per CTA pair), or null
extern "C" int tsp_mlp_debug_set_trace(unsigned long long* dev_buffer) {
    return cudaMemcpyToSymbol(tsp::g_trace, &dev_buffer, sizeof(dev_buffer)) == cudaSuccess ? 0 : -1;
}
#endif

// Projection GEMMs of TSP attention (Algorithm 1): same library, own header and entry points.
#include "tsp_attn_host.cuh"
