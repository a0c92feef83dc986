// Building blocks shared by all kernels of the path: the shared-memory control block,
// bounded mbarrier waits, operand loaders (TMA into 128B-swizzled tiles) and the UMMA issue
// of one 64-deep k-block for K-major and MN-major operands.
//
// Operand tiles in shared memory (bf16, BK = 64):
//   K-major  operand with R rows : [R][64] elements, one TMA box {64, R}; 8-row groups are 1024 B apart.
//   MN-major operand with R rows : R/64 chunks of [64 k][64 mn] (8 KB each), one TMA box {64, 64} per chunk;
//                                  8-k groups are 1024 B apart, chunks 8192 B apart.
// Both take R * 128 bytes and must start on a 1024-byte boundary.
#pragma once
#include "ptx.cuh"

namespace tsp {

constexpr int kBK = 64;              // k-block depth in elements (128 bytes of bf16 = one swizzle row)
constexpr int kUmmaK = 16;           // K of one bf16 tcgen05.mma
constexpr int kMaxStages = 8;
constexpr int kNumThreads = 192;     // warp 0: TMA producer, warp 1: MMA issuer, warps 2-5: epilogue
constexpr int kEpilogueThreads = 128;
constexpr uint32_t kTmemCols = 512;

// Error codes written to the device status word (first one wins).
constexpr int kErrWaitEmpty = 1, kErrWaitFull = 2, kErrWaitTmemEmpty = 3, kErrWaitTmemFull = 4, kErrTeardown = 5,
              kErrSelfTest = 6;

struct __align__(16) SharedCtl {
    uint64_t full[kMaxStages];
    uint64_t empty[kMaxStages];
    uint64_t tmem_full[4];
    uint64_t tmem_empty[4];
    uint64_t teardown;
    uint64_t epi[2];              // epilogue staging buffers filled by TMA loads (carried fp32 sums)
    uint32_t issued[kMaxStages];  // 1 + parity of the last TMA phase issued into the stage (0 = none)
    uint32_t tmem_base;
    uint32_t abort;
};

struct WaitCtx {
    volatile uint32_t* abort;  // shared memory
    int* status;               // global status word
    uint64_t limit_ns;
};

// Wait for the phase with `parity` of `bar` to complete, for at most limit_ns.  On expiry the CTA-wide
// abort flag and the global status word are set and false is returned; callers leave their role loop.
__device__ __forceinline__ bool wait_bar(uint32_t bar, uint32_t parity, const WaitCtx& w, int code) {
    if (mbar_try_wait(bar, parity)) return true;
    const uint64_t t0 = global_timer_ns();
    uint32_t spins = 0;
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if ((++spins & 31u) == 0u) {
            if (*w.abort) return false;
            if (global_timer_ns() - t0 > w.limit_ns) {
                *w.abort = 1u;
                atomicCAS(w.status, 0, code);
                return false;
            }
        }
    }
}

struct PipeState {
    int stage = 0;
    uint32_t phase = 0;
    __device__ __forceinline__ void advance(int stages) {
        if (++stage == stages) { stage = 0; phase ^= 1u; }
    }
};

// ---- operand loaders (one thread) -------------------------------------------------------------
// K-major operand: rows [row0, row0+R) x k [k0, k0+64) of a [.., rows, K] tensor (inner dim = K).
__device__ __forceinline__ void load_kmajor(uint32_t smem, const CUtensorMap* map, uint32_t bar, int k0, int row0, int z) {
    tma_load_3d(smem, map, bar, k0, row0, z);
}
// MN-major operand: k rows [k0, k0+64) x mn [mn0, mn0 + 64*chunks) of a [.., K, MN] tensor (inner dim = MN).
__device__ __forceinline__ void load_mnmajor(uint32_t smem, const CUtensorMap* map, uint32_t bar, int mn0, int k0, int z,
                                             int chunks) {
    for (int c = 0; c < chunks; ++c) tma_load_3d(smem + c * 8192, map, bar, mn0 + c * 64, k0, z);
}

// ---- UMMA issue of one k-block (one thread) ----------------------------------------------------
template <bool kAMn, bool kBMn>
__device__ __forceinline__ void issue_kblock(uint32_t d_tmem, uint32_t a_smem, uint32_t b_smem, uint32_t idesc,
                                             bool accumulate_first) {
    // K-major: 8-row groups 1024 B apart, LBO unused; advance 32 B per UMMA_K inside the swizzle row.
    // MN-major: 64-wide chunks 8192 B apart (LBO), 8-k groups 1024 B apart (SBO); advance 2 groups per UMMA_K.
    const uint64_t a_desc = make_smem_desc_sw128(a_smem, kAMn ? 8192u : 0u, 1024u);
    const uint64_t b_desc = make_smem_desc_sw128(b_smem, kBMn ? 8192u : 0u, 1024u);
    constexpr uint64_t a_step = (kAMn ? 2048u : 32u) >> 4;
    constexpr uint64_t b_step = (kBMn ? 2048u : 32u) >> 4;
#pragma unroll
    for (int kk = 0; kk < kBK / kUmmaK; ++kk) {
        umma_bf16(d_tmem, a_desc + kk * a_step, b_desc + kk * b_step, idesc, (accumulate_first || kk > 0) ? 1u : 0u);
    }
}

// ---- CTA set-up / tear-down ---------------------------------------------------------------------
__device__ __forceinline__ uint8_t* align_1024(uint8_t* p) {
    return reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(p) + 1023) & ~static_cast<uintptr_t>(1023));
}

// All threads call.  `n_acc` accumulator barriers pairs are initialised.
__device__ __forceinline__ void cta_setup(SharedCtl* ctl, int stages, int n_acc, uint32_t epilogue_arrivals) {
    const int warp = threadIdx.x >> 5;
    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            mbar_init(smem_u32(&ctl->full[s]), 1);
            mbar_init(smem_u32(&ctl->empty[s]), 1);
            ctl->issued[s] = 0;
        }
        for (int b = 0; b < n_acc; ++b) {
            mbar_init(smem_u32(&ctl->tmem_full[b]), 1);
            mbar_init(smem_u32(&ctl->tmem_empty[b]), epilogue_arrivals);
        }
        mbar_init(smem_u32(&ctl->teardown), 1);
        ctl->abort = 0;
        fence_mbar_init();
    }
    if (warp == 1) {
        tmem_alloc(smem_u32(&ctl->tmem_base), kTmemCols);
        tmem_relinquish();
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
}

// All threads call after their role loops.  On the error path the copies and MMAs still in flight are
// waited for (bounded) before tensor memory is released.
__device__ __forceinline__ void cta_teardown(SharedCtl* ctl, int stages, const WaitCtx& w) {
    const int warp = threadIdx.x >> 5;
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (*w.abort) {
        WaitCtx quiet = w;
        uint32_t dummy = 0;
        quiet.abort = &dummy;  // keep waiting even though the abort flag is up
        quiet.limit_ns = 20ull * 1000 * 1000;
        if (threadIdx.x == 0) {
            for (int s = 0; s < stages; ++s)
                if (ctl->issued[s]) wait_bar(smem_u32(&ctl->full[s]), ctl->issued[s] - 1u, quiet, kErrTeardown);
        }
        if (threadIdx.x == 32) {
            umma_commit(smem_u32(&ctl->teardown));
            wait_bar(smem_u32(&ctl->teardown), 0, quiet, kErrTeardown);
        }
        __syncthreads();
    }
    if (warp == 1) {
        __syncwarp();
        tmem_dealloc(ctl->tmem_base, kTmemCols);
    }
}

// One warp waits, with the usual bound, on a barrier that nothing ever arrives on: the wait expires, the status
// word is set and the kernel returns normally.  Proves the error path without faulting or hanging anything.
__global__ void wait_expiry_selftest_kernel(int* status, unsigned long long limit_ns) {
    __shared__ uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        mbar_init(smem_u32(&bar), 1);
        abort_flag = 0;
        fence_mbar_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) {
        WaitCtx w{&abort_flag, status, limit_ns};
        wait_bar(smem_u32(&bar), 0, w, kErrSelfTest);
    }
    __syncthreads();
}

// Token tile `mt` when every rank owns S_loc consecutive rows cut into tiles of TM rows; the last tile of a rank may be
// partial (its remaining rows belong to the next rank, or lie beyond the tensor, and are loaded but never stored).
__device__ __forceinline__ void token_tile(int mt, int tiles_per_rank, int S_loc, int TM, int& r, int& row0, int& valid) {
    r = mt / tiles_per_rank;
    const int lt = mt - r * tiles_per_rank;
    row0 = r * S_loc + lt * TM;
    valid = min(TM, S_loc - lt * TM);
}

// ---- epilogue helpers ---------------------------------------------------------------------------
__device__ __forceinline__ uint32_t pack_bf16x2(float lo, float hi) {
    __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<uint32_t*>(&v);
}

// 1 / (1 + e^-z); the exponent is clamped so the denominator stays finite (below 2^126).
__device__ __forceinline__ float sigmoid_fast(float z) {
    return __fdividef(1.0f, 1.0f + __expf(fminf(-z, 80.0f)));
}

// Gate activations sigma of Algorithm 2 ("Activation sigma"): 0 = SiLU (SwiGLU), 1 = GELU, exact erf form (GeGLU),
// 2 = ReLU (ReGLU).  `act` is uniform over the launch, so the branch does not diverge.
constexpr int kActSilu = 0, kActGelu = 1, kActRelu = 2;

__device__ __forceinline__ float gate_act(float z, int act) {
    if (act == kActSilu) return z * sigmoid_fast(z);
    if (act == kActGelu) return 0.5f * z * (1.0f + erff(z * 0.70710678118654752f));
    return fmaxf(z, 0.0f);
}
// value and derivative of the activation
__device__ __forceinline__ void gate_act_grad(float z, int act, float& val, float& der) {
    if (act == kActSilu) {
        const float s = sigmoid_fast(z);
        val = z * s;
        der = s * (1.0f + z * (1.0f - s));
    } else if (act == kActGelu) {
        const float cdf = 0.5f * (1.0f + erff(z * 0.70710678118654752f));
        val = z * cdf;
        der = cdf + z * 0.3989422804014327f * __expf(-0.5f * z * z);
    } else {
        val = fmaxf(z, 0.0f);
        der = z > 0.0f ? 1.0f : 0.0f;
    }
}

}  // namespace tsp
