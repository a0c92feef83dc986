/*
 * tsp_mlp.h - C ABI of the B200 (sm_100a) TSP gated ring MLP library.
 *
 * The library computes the per-rank work of the TSP gated ring MLP (Algorithm 2 of
 * "Folding Tensor and Sequence Parallelism ...") for all D ranks on ONE GPU: rank r
 * owns token rows [r*S/D, (r+1)*S/D) of X and, at ring step t, applies weight shard
 * k = (r - t) mod D:   Y_r += (silu(X_r Wg_k) * (X_r Wu_k)) Wd_k,   t = 0..D-1.
 * The ring transfer itself is absent (all shards are resident); the ring only fixes
 * the order in which each rank's fp32 accumulator meets the shards.
 *
 * Conventions for every entry point
 *   - All matrix arguments are DEVICE pointers unless the name ends in _host.
 *     Row-major, bf16 (2 bytes) unless stated; inputs 16-byte aligned, outputs (Y, dX, dW*) 32-byte aligned.
 *       X, Y, dY, dX : [S, H]            rank r = rows [r*S/D, (r+1)*S/D)
 *       Wg, Wu       : [D][H][F/D]       shard k = gate/up columns k*F/D .. (k+1)*F/D
 *       Wd           : [D][F/D][H]       shard k = down rows       k*F/D .. (k+1)*F/D
 *       dWg, dWu, dWd: same shapes as the weights, FP32, overwritten (not accumulated)
 *   - The caller owns every buffer, including the workspace.  The library owns only
 *     the plan (host tables, tensor maps, an 8.5 KB device control block: status word, tile-scheduler words and
 *     ready counters; profiling events).
 *     tsp_mlp_forward / tsp_mlp_backward allocate nothing.
 *   - Calls are asynchronous on `cuda_stream` (a cudaStream_t passed as void*; NULL is
 *     the default stream).  Argument and launch errors are returned at once; a device
 *     wait that ran out of time is reported by tsp_mlp_status after a synchronize.
 *   - No exceptions, no abort, no CPU fallback.  Unsupported shapes are refused before
 *     any launch.  Supported: H % 256 == 0, (F/D) % 128 == 0, F % D == 0, S % D == 0 (any number
 *     of tokens per rank >= 1), 1 <= D <= 64, S <= 2^24.  The model dimensions must fit the tile
 *     sizes; the token count need not: the last token tile of a rank is loaded whole and only its
 *     valid rows are stored.  When S/D is not a multiple of 64 the weight gradients contract the
 *     tokens in ascending order instead of rank order (a k-block would otherwise straddle two ranks).
 *   - A plan must not be used from two host threads at once, nor on two streams at
 *     once (the workspace and status word are shared).
 *   - Results are deterministic: no atomics, fixed accumulation order.
 *   - "One kernel" / "two kernels" below name the distinct kernels of a call.  A long problem runs each of them
 *     as several launches over consecutive token ranges (beyond about 18 000 tokens; the launch boundaries keep
 *     the thread blocks aligned in time so that they keep sharing operand blocks through L2); outputs do not
 *     depend on where the cuts fall.  tsp_mlp_kernels_per_call reports the launches actually made.
 */
#ifndef TSP_MLP_H
#define TSP_MLP_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct tsp_mlp_plan tsp_mlp_plan_t; /* opaque; created by tsp_mlp_plan, owned by the library */

typedef enum {
    TSP_OK = 0,
    TSP_ERR_INVALID_ARG = -1,        /* null pointer, misaligned pointer, D differs from the plan, S <= 0 */
    TSP_ERR_UNSUPPORTED_SHAPE = -2,  /* divisibility rules above not met (or a path-specific rule, see each call) */
    TSP_ERR_UNSUPPORTED_DEVICE = -3, /* current device is not compute capability 10.x */
    TSP_ERR_CUDA = -4,               /* a CUDA runtime / driver call failed (see tsp_mlp_last_cuda_error) */
    TSP_ERR_WORKSPACE = -5,          /* workspace missing or smaller than tsp_mlp_workspace_bytes */
    TSP_ERR_DEVICE_TIMEOUT = -6,     /* a bounded device-side wait expired; outputs are invalid */
    TSP_ERR_STATIC_LIMIT = -7        /* tsp_mlp_forward_static: S*F*2 bytes exceed TSP_MLP_STATIC_SCRATCH_BYTES */
} tsp_status_t;

/* Which passes a workspace must serve. */
#define TSP_WS_FORWARD 0
#define TSP_WS_BACKWARD 1

/*
 * tsp_mlp_plan - validate (H, F, D) for the current device and build a plan.
 * Follows the inputs of Algorithm 2: hidden size H, intermediate width F (the paper's
 * F*h), world size D.  *out receives the plan; release it with tsp_mlp_plan_destroy.
 * Allocates the plan's device control block (8.5 KB).  Errors: INVALID_ARG, UNSUPPORTED_SHAPE,
 * UNSUPPORTED_DEVICE, CUDA.
 */
tsp_status_t tsp_mlp_plan(int H, int F, int D, tsp_mlp_plan_t** out);
tsp_status_t tsp_mlp_plan_destroy(tsp_mlp_plan_t* plan);

/*
 * Plan options: how the kernels of a plan walk their tiles.  None of them changes WHAT is computed (Algorithm 2
 * and its gradients, ring accumulation order k = (r - t) mod D included); they select kernel families, tile
 * orders and launch cuts, i.e. speed and, for a few of them, the grouping of fp32 partial sums.  The paper has no
 * counterpart (it runs library GEMMs); the fields exist so that every path can be selected per plan, from tests
 * and sweeps, without touching the process environment.
 * Fill the struct with tsp_mlp_options_default, change what is wanted, pass it to tsp_mlp_plan_ex.
 * In every field TSP_OPT_AUTO (-1) means "the library decides from the shape".
 *   use_pairs        1: CTA-pair (cta_group::2) kernels where the token count allows (auto); 0: single-CTA kernels only
 *   gate_band        token tiles (256 rows) per band of the gate|up and dA tile order (auto: rows worth 32 MB of L2)
 *   gate_order       1 (auto): all ranks of a band work on the same column block of the same shard;
 *                    0: ring-faithful, every rank of a band on the shard it holds at that step (same results: the
 *                    gate|up tiles are independent; 8x the weight traffic)
 *   down_group       token tiles per group of the narrow down-projection tile order (auto: 8)
 *   dx_group         the same for the dX kernel (auto: 8)
 *   dw_group         hidden blocks (256 columns) per group of the weight-gradient tile order (auto: from S)
 *   wide_mask        bit 0 down, bit 1 dX, bit 2 dW: force 256 x 512 tiles for that kernel; 0 forces 256 x 256
 *                    everywhere; auto: a mixed list chosen per launch from the tile counts
 *   pair_stages      shared-memory stages of the 256 x 256 pair kernels (auto: 6)
 *   chunk_bands      token bands per launch of gate|up / dA (auto: 3; 0 = one launch however long)
 *   chunk_tiles      token tiles per launch of down / dX (auto: 96; 0 = one launch)
 *   dw_chunk_rounds  rounds of the CTA pairs per launch of the weight-gradient kernel (auto: about 3 ms of tiles;
 *                    n > 0: n rounds; 0 = one launch)
 *   phase_mask       profiling aid: bit 0 run gate|up, bit 1 run down in tsp_mlp_forward (auto: both)
 *   timeout_ms       limit of every device-side wait (auto: 2000)
 *   dynamic_tiles    bit mask of the kernels whose CTA pairs draw tiles from a device counter instead of taking them
 *                    round-robin: bit 0 the short-K kernels (gate|up, dA, Q/K/V), bit 1 down projection (and the
 *                    attention output projection), bit 2 dX, bit 3 weight gradients (auto: 14 = all but the short-K
 *                    kernels).  Same tiles, same bits: the tile -> accumulator order does not depend on which pair
 *                    runs a tile.
 *   fuse_ring_steps  1: tsp_mlp_ring_step / tsp_mlp_ring_steps run the gate|up GEMM and the down projection of their
 *                    shard(s) as ONE launch (up to 261888 tokens per rank): gate|up tiles first, then down-projection
 *                    tiles that wait, per 256 token rows, for the rows of A they read; 0 (auto): two launches.  Same
 *                    bits either way.  (Measured on B200: on a par at best, so not the default.)
 *   tma_carry        1 (auto): the fp32 partial sums that the per-step calls carry from launch to launch (Yacc, dXacc)
 *                    are stored, added and read back by the TMA unit through shared-memory staging; 0: element-wise
 *                    accesses from registers.  Same arithmetic (one fp32 round-to-nearest add per step).
 *   rank_pair_tiles  bit 0 down projection, bit 1 dX: when a rank owns at most 8 token tiles (S/D <= 2048), D is even
 *                    and the whole problem is one launch, tiles hold the same 256 token rows of TWO neighbouring
 *                    ranks.  Rank 2q meets the shards in the order of rank 2q+1 shifted by one ring step, so one
 *                    loaded weight panel serves both ranks (each in its own step), which halves the weight traffic
 *                    into shared memory.  Every rank still adds its D partial products in ring order: same bits.
 *                    As many whole rounds of the CTA pairs as fit without adding a time unit run as two-rank tiles,
 *                    the rest as one-rank tiles; bit 2 makes every position a two-rank tile (tests, sweeps).
 *                    0: one-rank tiles only.  Needs the dynamic hand-out of the kernel (dynamic_tiles).
 *                    Auto: 2 (dX only; measured slower for the down projection), 0 when wide_mask is given.
 *   overlap_launches 1 (auto): the CTA-pair kernels are launched with programmatic stream serialisation: a kernel's
 *                    CTAs may start while the previous kernel of the stream is finishing, set up their barriers and
 *                    tensor memory, and wait on the device for the previous grid to complete (and its writes to be
 *                    visible) before their first access to global memory.  Hides the launch gap and the set-up at
 *                    every kernel boundary; results are the same.  0: ordinary launches.
 * Environment variables of the same meaning (TSP_MLP_PAIR, TSP_MLP_BAND, TSP_MLP_GATE_ORDER, TSP_MLP_GROUP,
 * TSP_MLP_DX_GROUP, TSP_MLP_DW_GROUP, TSP_MLP_WIDE, TSP_MLP_PAIR_STAGES, TSP_MLP_CHUNK_BANDS, TSP_MLP_CHUNK_TILES,
 * TSP_MLP_DW_CHUNK_ROUNDS (negative = one launch), TSP_MLP_PHASES, TSP_MLP_TIMEOUT_MS, TSP_MLP_DYNAMIC,
 * TSP_MLP_FUSE_STEPS, TSP_MLP_TMA_CARRY, TSP_MLP_RANK_PAIRS, TSP_MLP_OVERLAP_LAUNCHES) are read
 * when a plan is created and fill only the fields the caller left at TSP_OPT_AUTO: an explicit option wins.
 * struct_bytes must be sizeof(tsp_mlp_options_t) as the caller was compiled (tsp_mlp_options_default sets it);
 * a different size is refused with INVALID_ARG, as is a field outside its range.
 */
#define TSP_OPT_AUTO (-1)
typedef struct {
    uint32_t struct_bytes;
    int use_pairs;
    int gate_band;
    int gate_order;
    int down_group;
    int dx_group;
    int dw_group;
    int wide_mask;
    int pair_stages;
    int chunk_bands;
    int chunk_tiles;
    int dw_chunk_rounds;
    int phase_mask;
    int timeout_ms;
    int dynamic_tiles;
    int fuse_ring_steps;
    int tma_carry;
    int rank_pair_tiles;
    int overlap_launches;
} tsp_mlp_options_t;
void tsp_mlp_options_default(tsp_mlp_options_t* options);
/* tsp_mlp_plan with options (NULL options = tsp_mlp_plan).  Errors as tsp_mlp_plan. */
tsp_status_t tsp_mlp_plan_ex(int H, int F, int D, const tsp_mlp_options_t* options, tsp_mlp_plan_t** out);

/*
 * tsp_mlp_set_activation - choose the gate activation sigma of Algorithm 2 ("Activation sigma"; the paper
 * names SwiGLU as the example of a gated MLP).  TSP_ACT_SILU (default): sigma(z) = z / (1 + e^-z);
 * TSP_ACT_GELU: sigma(z) = z * Phi(z), Phi the standard normal CDF (erf form, not the tanh approximation);
 * TSP_ACT_RELU: sigma(z) = max(z, 0), with sigma'(0) = 0 in the backward pass.  Applies to every later
 * forward / backward / staged call on the plan.  Error: INVALID_ARG for any other value.
 */
#define TSP_ACT_SILU 0
#define TSP_ACT_GELU 1
#define TSP_ACT_RELU 2
tsp_status_t tsp_mlp_set_activation(tsp_mlp_plan_t* plan, int activation);

/*
 * Workspace: scratch for the bf16 intermediate A = silu(G)*U [S,F] (forward) and for
 * A, dG, dU [S,F] in bf16 plus dA [S,F] in fp32 (backward).  tsp_mlp_workspace_bytes returns the size needed
 * for S tokens (`pass` = TSP_WS_FORWARD or TSP_WS_BACKWARD; backward covers forward);
 * 0 on bad arguments.  tsp_mlp_set_workspace hands a caller-owned device buffer
 * (256-byte aligned) to the plan; it must stay valid while calls using it are in flight.
 */
size_t tsp_mlp_workspace_bytes(const tsp_mlp_plan_t* plan, int64_t S, int pass);
tsp_status_t tsp_mlp_set_workspace(tsp_mlp_plan_t* plan, void* dev_ptr, size_t bytes);

/*
 * tsp_mlp_forward - Algorithm 2 for all D ranks: Y = (silu(X Wg) * (X Wu)) Wd with
 * each rank's fp32 accumulator visiting the shards in ring order k = (r - t) mod D.
 * Two kernels: gate|up GEMM with the SwiGLU epilogue (G, U live only in tensor memory,
 * A is rounded once to bf16), then the down projection accumulated in tensor memory
 * over all D shards with one bf16 store of Y.  `D` must equal the plan's.
 */
tsp_status_t tsp_mlp_forward(tsp_mlp_plan_t* plan, const void* X, const void* Wg, const void* Wu,
                             const void* Wd, void* Y, int64_t S, int D, void* cuda_stream);

/*
 * tsp_mlp_backward - gradients of the forward above for upstream dY (the backward
 * pass mirrors the forward weight movement; the partial weight gradients every rank
 * produces for shard k are summed to the owner, Sections 4.3.4 and 4.7).  G and U are
 * recomputed from X; dA = dY Wd^T (kept in fp32); dU = dA*silu(G); dG = dA*U*silu'(G);
 * A, dG, dU are rounded once to bf16 into the workspace.  dX [S,H] bf16 accumulates over shards in
 * ring order; dWg, dWu [D][H][F/D] and dWd [D][F/D][H] are fp32 and contract over all S
 * tokens, rank order r = (k + t) mod D.  Beyond 2^18 tokens the token contraction of the weight
 * gradients is cut into chunks of 2^18 tokens (ascending order, one launch per chunk, partial sums added
 * in fp32 round-to-nearest): the tensor cores add into their accumulators with truncation, and an
 * unbroken sum over millions of tokens would drift towards zero (about 2 % at 2^24 tokens).
 */
tsp_status_t tsp_mlp_backward(tsp_mlp_plan_t* plan, const void* X, const void* Wg, const void* Wu,
                              const void* Wd, const void* dY, void* dX, float* dWg, float* dWu,
                              float* dWd, int64_t S, int D, void* cuda_stream);

/*
 * Stored-activation training path.  The activation-memory analysis (Section 4.2) distinguishes full
 * recomputation (only the layer input is kept: what tsp_mlp_backward does, recomputing G and U from X)
 * from keeping the MLP activations.  This pair of calls is the second regime: tsp_mlp_forward_save computes
 * the same Y as tsp_mlp_forward and additionally keeps, in the caller-owned device buffer `saved`
 * (tsp_mlp_saved_bytes(plan, S) bytes, 256-byte aligned), A = sigma(G)*U, P = U*sigma'(G) and Q = sigma(G),
 * each [S,F] in bf16.  tsp_mlp_backward_saved then needs no gate|up GEMM: dA = dY Wd^T stays in tensor memory
 * and its epilogue writes dG = dA*P and dU = dA*Q (bf16, workspace); dX and the fp32 weight gradients follow
 * as in tsp_mlp_backward (A is read from `saved`).  Hardware FLOPs equal model FLOPs (18 S H F per training
 * step instead of 22 S H F); the cost is 3 S F bf16 elements of memory and one more bf16 rounding in dG, dU.
 * Workspace for tsp_mlp_backward_saved: 2 * S * F * 2 bytes (tsp_mlp_workspace_bytes(.., TSP_WS_BACKWARD) is
 * enough).  Shapes: F % 256 == 0 and a token count per rank that the CTA-pair kernels take (S/D a multiple of
 * 256, or large enough that padding the last 256-row tile costs little), otherwise TSP_ERR_UNSUPPORTED_SHAPE.
 * tsp_mlp_forward_save
 * does not use the plan's workspace.
 */
size_t tsp_mlp_saved_bytes(const tsp_mlp_plan_t* plan, int64_t S);
tsp_status_t tsp_mlp_forward_save(tsp_mlp_plan_t* plan, const void* X, const void* Wg, const void* Wu,
                                  const void* Wd, void* Y, void* saved, int64_t S, int D, void* cuda_stream);
tsp_status_t tsp_mlp_backward_saved(tsp_mlp_plan_t* plan, const void* X, const void* Wg, const void* Wu,
                                    const void* Wd, const void* dY, const void* saved, void* dX, float* dWg,
                                    float* dWu, float* dWd, int64_t S, int D, void* cuda_stream);

/*
 * tsp_mlp_forward_host - the same forward for callers whose tensors live in HOST
 * memory (pinned memory gives asynchronous copies).  Everything is uploaded on one plan-owned side stream in the
 * order it is needed - X, then shard by shard Wg_k and Wu_k, then Wd in four blocks of hidden columns - into staging
 * inside the workspace; the gate|up tiles of shard k are launched on `cuda_stream` as soon as shard k has arrived, the
 * down projection of a column block as soon as its part of Wd has, and every column block of Y goes back to Y_host on
 * a second side stream while later uploads are still running.  Same tiles, same K order: Y has the bits of
 * tsp_mlp_forward.  Ordered with respect to `cuda_stream` (synchronizing it is enough to read Y_host).  Small shapes
 * (single-CTA path, or H / 256 not a multiple of 8) upload everything first and run the two kernels unsplit.  The side
 * streams and events are created on first use.  Needs a workspace of tsp_mlp_workspace_bytes_host(plan, S) bytes.
 */
size_t tsp_mlp_workspace_bytes_host(const tsp_mlp_plan_t* plan, int64_t S);
tsp_status_t tsp_mlp_forward_host(tsp_mlp_plan_t* plan, const void* X_host, const void* Wg_host,
                                  const void* Wu_host, const void* Wd_host, void* Y_host,
                                  int64_t S, int D, void* cuda_stream);

/*
 * tsp_mlp_forward_staged - Algorithm 2 executed step by step, with the ring transfer stood in for by
 * device-to-device copies on a second stream (Section 4.9: send/receive on a dedicated communication
 * stream while the default stream computes; wait only when the next shard is needed).
 * For t = 0..D-1: the copy stream moves every rank's current (Wg, Wu, Wd) buffers into the next rank's
 * receive buffers (send to (p+1) mod D, receive from (p-1) mod D; two buffer sets alternate), while the
 * compute stream runs step t for all ranks: the gate|up GEMM with the SwiGLU epilogue into a [S, F/D]
 * scratch, then the down projection of that shard added into an fp32 [S, H] accumulator; the last step
 * rounds the accumulator to bf16 Y.  Events order "received" before "compute t+1" and "computed t-1"
 * before the buffers are overwritten.  Same result as tsp_mlp_forward up to fp32 summation order
 * (per-shard partial sums are formed first).  Needs a token count per rank that the CTA-pair kernels
 * take (S/D a multiple of 256, or large enough that padding the last 256-row tile costs little: the same
 * rule tsp_mlp_forward applies internally), two distinct streams, and a
 * workspace of tsp_mlp_workspace_bytes_staged(plan, S) bytes (scratch, accumulator, 2 x 3 receive buffers
 * of the size of one weight matrix).  2*D kernels and at most 6*(D-1) copies per call.
 */
size_t tsp_mlp_workspace_bytes_staged(const tsp_mlp_plan_t* plan, int64_t S);
tsp_status_t tsp_mlp_forward_staged(tsp_mlp_plan_t* plan, const void* X, const void* Wg, const void* Wu,
                                    const void* Wd, void* Y, int64_t S, int D, void* compute_stream,
                                    void* copy_stream);

/*
 * tsp_mlp_ring_step - ONE step of Algorithm 2 on ONE rank's data: what rank p runs between the
 * AsyncRingSendRecv and the Wait of ring step t, when every rank has a GPU of its own and the weight shards
 * really travel (the caller moves them: NCCL send / receive or peer copies on a communication stream).
 *   t = 0:        Yacc  = (act(X_p Wg_k) * (X_p Wu_k)) Wd_k         (the "Y <- 0" of the algorithm is folded in)
 *   0 < t < D-1:  Yacc += ...
 *   t = D-1:      Y_p   = bf16(Yacc + ...)                          (D = 1: Y_p = bf16(...) directly)
 * X_p, Y_p: [S_loc, H] bf16 (this rank's tokens only); Wg_k, Wu_k: [H, F/D] bf16 and Wd_k: [F/D, H] bf16, the
 * shard the rank holds at this step (k = (p - t) mod D when the caller follows the ring; the kernels do not
 * care which).  The fp32 accumulator Yacc [S_loc, H] and two bf16 scratch buffers A [S_loc, F/D] (even / odd
 * steps) live in the plan's
 * workspace (tsp_mlp_workspace_bytes_ring(plan, S_loc, TSP_WS_FORWARD) bytes) and carry the state from step to
 * step, so the D calls of one forward pass must use the same plan, workspace and S_loc, in the order t = 0..D-1 on
 * one stream (or otherwise ordered).  Two kernels per call (gate|up with the activation epilogue; down projection
 * of the shard added to the accumulator).  Any S_loc >= 1.  The result equals tsp_mlp_forward_staged's
 * rows of rank p bit for bit (same kernels, same summation order).
 * Errors: INVALID_ARG (null / misaligned pointer, t outside [0, D), D not the plan's), UNSUPPORTED_SHAPE
 * (S_loc < 1 or > 2^24), WORKSPACE.
 */
size_t tsp_mlp_workspace_bytes_ring(const tsp_mlp_plan_t* plan, int64_t S_loc, int pass);
tsp_status_t tsp_mlp_ring_step(tsp_mlp_plan_t* plan, const void* X_p, const void* Wg_k, const void* Wu_k,
                               const void* Wd_k, void* Y_p, int64_t S_loc, int t, int D, void* cuda_stream);

/*
 * The two halves of tsp_mlp_ring_step as calls of their own: _gate writes A = act(X_p Wg_k) * (X_p Wu_k) into the
 * scratch buffer of step t (buffer t & 1), _down adds A Wd_k to the accumulator (or stores Y_p at t = D-1).  With
 * few tokens per rank one step is less than a full round of tiles, so a caller can fill the GPU by running the
 * down projection of step t on a second stream while the gate|up GEMM of step t+1 runs on the first.  Ordering
 * the caller must provide: _down(t) after _gate(t); _gate(t+2) after _down(t) (it reuses the scratch buffer);
 * _down(t+1) after _down(t) (the accumulator).  Same bits as tsp_mlp_ring_step.  (These two calls are the one
 * exception to the rule that a plan is used on one stream at a time; the host thread is still one.)
 */
tsp_status_t tsp_mlp_ring_step_gate(tsp_mlp_plan_t* plan, const void* X_p, const void* Wg_k, const void* Wu_k,
                                    int64_t S_loc, int t, int D, void* cuda_stream);
tsp_status_t tsp_mlp_ring_step_down(tsp_mlp_plan_t* plan, const void* Wd_k, void* Y_p, int64_t S_loc, int t, int D,
                                    void* cuda_stream);

/*
 * tsp_mlp_ring_steps - n consecutive ring steps t_first .. t_first + n - 1 of ONE rank in one call (two kernels
 * instead of 2 n): with few tokens per rank a single step is less than one round of tiles and its launches cost as
 * much as its math, so a rank that has already received the next n shards applies them together.  The n shards
 * are n packed buffers at a constant distance: shard i has its gate / up / down matrices at Wg_first, Wu_first,
 * Wd_first + i * shard_stride ELEMENTS (bf16; shard_stride a multiple of 8 and at least H * F/D; ignored for n = 1),
 * in the order the rank meets them.  The fp32 sum is carried across calls exactly as by tsp_mlp_ring_step (first call
 * t_first = 0, last call ends at D), and the shards of a call are accumulated in tensor memory in the order given,
 * so the result differs from the step-by-step one only in fp32 summation grouping.  Workspace:
 * tsp_mlp_workspace_bytes_ring_group(plan, S_loc, n) bytes for the largest n used (the accumulator, then
 * A [S_loc, n * F/D]); the calls of a pass may use different n, but not be mixed with tsp_mlp_ring_step calls (which
 * lay the workspace out differently).  Errors as tsp_mlp_ring_step; INVALID_ARG also for a bad stride
 * or t_first + n > D.
 */
size_t tsp_mlp_workspace_bytes_ring_group(const tsp_mlp_plan_t* plan, int64_t S_loc, int n_shards);
tsp_status_t tsp_mlp_ring_steps(tsp_mlp_plan_t* plan, const void* X_p, const void* Wg_first, const void* Wu_first,
                                const void* Wd_first, int64_t shard_stride, int n_shards, void* Y_p, int64_t S_loc,
                                int t_first, int D, void* cuda_stream);

/*
 * Backward pass of one ring step on one rank's data (the backward mirrors the forward weight movement, and the
 * partial weight gradients the ranks produce for a shard are summed to its owner: Sections 4.3.4 and 4.7).  Split
 * in two calls so that the caller can let a travelling dW accumulator arrive while the first call computes:
 *
 * tsp_mlp_ring_step_backward_dx: with the shard (Wg_k, Wu_k, Wd_k) held at step t and this rank's X_p, dY_p
 *   [S_loc, H] bf16: recomputes G, U; dA = dY_p Wd_k^T (fp32); A, dG, dU (bf16, left in the workspace for the dW
 *   call); dXacc (+)= dG Wg_k^T + dU Wu_k^T, with the fp32 partial sum carried in the workspace from t = 0 to
 *   t = D-1, where dX_p [S_loc, H] is stored in bf16 (D = 1: stored directly).  Three kernels.
 * tsp_mlp_ring_step_backward_dw: from the A, dG, dU the preceding _dx call left: this rank's contribution to the
 *   shard's weight gradients, dWd_k (+)= A^T dY_p [F/D, H], dWg_k (+)= X_p^T dG, dWu_k (+)= X_p^T dU [H, F/D], fp32.
 *   accumulate = 0 overwrites (the owner's own contribution, or a partial to be reduced by the caller),
 *   accumulate = 1 adds to what the buffers hold (an accumulator that travels with the shard: the sum then runs
 *   over the ranks in the order the shard meets them, r = (k + t) mod D).  One kernel.
 * Both need (F/D) % 256 == 0 and the workspace of tsp_mlp_workspace_bytes_ring(plan, S_loc, TSP_WS_BACKWARD);
 * calls of one backward pass go t = 0..D-1, _dx before _dw within a step, ordered on the GPU.
 * Errors as for tsp_mlp_ring_step; UNSUPPORTED_SHAPE also when (F/D) % 256 != 0.
 */
tsp_status_t tsp_mlp_ring_step_backward_dx(tsp_mlp_plan_t* plan, const void* X_p, const void* Wg_k, const void* Wu_k,
                                           const void* Wd_k, const void* dY_p, void* dX_p, int64_t S_loc, int t, int D,
                                           void* cuda_stream);
tsp_status_t tsp_mlp_ring_step_backward_dw(tsp_mlp_plan_t* plan, const void* X_p, const void* dY_p, float* dWg_k,
                                           float* dWu_k, float* dWd_k, int64_t S_loc, int accumulate, int D,
                                           void* cuda_stream);

/*
 * Backward pass of n consecutive ring steps t_first .. t_first + n - 1 of ONE rank per call (the counterpart of
 * tsp_mlp_ring_steps; Sections 4.3.4 and 4.7 as for the single-step calls).  With few tokens per rank the GEMMs of one
 * step leave most of the GPU idle, so a rank that already holds the next n shards (same packed layout and
 * shard_stride as for tsp_mlp_ring_steps, in the order it meets them) runs
 *   tsp_mlp_ring_steps_backward_dx: dA = dY_p [Wd_0 .. Wd_n-1]^T (fp32), the gate|up GEMM over the n shards with the
 *     backward epilogue (A, dG, dU for all n shards, bf16, left in the workspace), and ONE dX GEMM whose K loop walks
 *     the n shards in the order given; the fp32 sum of dX_p is carried across calls as by the single-step call (first
 *     call t_first = 0, the call ending at D stores bf16 dX_p).  Three kernels.  dX_p differs from the step-by-step
 *     result only in the grouping of fp32 partial sums.
 *   tsp_mlp_ring_steps_backward_dw: the weight gradients of ONE shard of the group (shard_in_group = 0 .. n-1), from
 *     the A, dG, dU columns the _dx call left: exactly tsp_mlp_ring_step_backward_dw's arithmetic (accumulate = 1 adds
 *     to a travelling accumulator in the kernel's epilogue), so the weight gradients keep every bit of the
 *     step-by-step result and the order of the sum over ranks, r = (k + t) mod D.  It is a call of its own because a
 *     shard's accumulator arrives from the left neighbour only after that rank has added its share: the caller issues
 *     the n calls one by one as the accumulators arrive, while nothing else of the group has to wait.  One kernel.
 * Workspace: tsp_mlp_workspace_bytes_ring_group_backward(plan, S_loc, n) for the largest n used (dXacc, then A, dG,
 * dU [S_loc, n F/D] bf16 and dA fp32); not to be mixed with the single-step backward calls within one pass.
 * Needs (F/D) % 256 == 0.  Errors as for tsp_mlp_ring_steps / tsp_mlp_ring_step_backward_dw.
 */
size_t tsp_mlp_workspace_bytes_ring_group_backward(const tsp_mlp_plan_t* plan, int64_t S_loc, int n_shards);
tsp_status_t tsp_mlp_ring_steps_backward_dx(tsp_mlp_plan_t* plan, const void* X_p, const void* Wg_first,
                                            const void* Wu_first, const void* Wd_first, int64_t shard_stride,
                                            int n_shards, const void* dY_p, void* dX_p, int64_t S_loc, int t_first, int D,
                                            void* cuda_stream);
tsp_status_t tsp_mlp_ring_steps_backward_dw(tsp_mlp_plan_t* plan, const void* X_p, const void* dY_p, float* dWg_k,
                                            float* dWu_k, float* dWd_k, int64_t S_loc, int shard_in_group, int n_shards,
                                            int accumulate, int D, void* cuda_stream);

/*
 * tsp_mlp_forward_static - the forward pass for callers that cannot obtain device memory at call time.
 * (The paper has no counterpart of this entry point; it exists for integration reasons only.)
 *
 * Who needs it: a plug-in living inside a host framework that has already claimed the whole GPU for its
 * own pool, so that cudaMalloc fails; code on a latency-critical path that cannot accept the device-wide
 * synchronisation an allocation implies; deployments whose rules forbid allocating after start-up.  Such
 * a caller cannot create a plan (the plan allocates its control block) nor hand over a workspace.
 *
 * What it does: the same two kernels as tsp_mlp_forward, but the bf16 intermediate A = silu(G)*U [S,F]
 * and the device status word live in a fixed array compiled into the library
 * (TSP_MLP_STATIC_SCRATCH_BYTES + 256 bytes of device memory on every GPU that loads the library, held
 * until the process exits).  The call performs no cudaMalloc / cudaFree and calls no allocating routine.
 * The caller passes only inputs and outputs, all DEVICE pointers with the layouts given at the top of this
 * file, plus optionally `timed_out_host`: a HOST int that, after `cuda_stream` has been synchronized,
 * is 0 if the kernels completed and non-zero if a bounded device-side wait expired (Y is then invalid).
 * The int is filled by a 4-byte asynchronous copy at the end of the call: give it PINNED host memory
 * (cudaHostAlloc / cudaHostRegister).  With ordinary pageable memory the copy makes the calling thread wait
 * until both kernels have finished, which a latency-critical caller does not want.  Pass NULL to skip the copy.
 *
 * Limits and rules:
 *   - S * F * 2 bytes must not exceed TSP_MLP_STATIC_SCRATCH_BYTES (8 MiB: e.g. S=1024, F=4096), otherwise
 *     TSP_ERR_STATIC_LIMIT is returned and nothing is launched.  Shape rules as for tsp_mlp_plan / forward.
 *   - The first call on each device looks up the array's device address and the device's properties (host
 *     work only, with that device current).  Make that first call outside any stream capture.
 *   - All calls on a device share the one array, and it keeps whatever the previous call left in it.  The
 *     entry point clears the status word on `cuda_stream` before launching; the intermediate is fully
 *     rewritten before it is read.  Two calls that overlap on the GPU (different streams, or different
 *     host threads) race on the array: serialize them on one stream.
 *   - The limit of the device-side waits is 2 s, or TSP_MLP_TIMEOUT_MS milliseconds if that environment
 *     variable is set when the first call on the device is made.
 *   - Errors: INVALID_ARG, UNSUPPORTED_SHAPE, UNSUPPORTED_DEVICE, STATIC_LIMIT, CUDA (there is no plan to ask:
 *     tsp_mlp_last_cuda_error(NULL) returns the cudaError_t of the last CUDA call that failed in this entry point).
 */
#define TSP_MLP_STATIC_SCRATCH_BYTES (8u << 20)
tsp_status_t tsp_mlp_forward_static(int H, int F, int D, const void* X, const void* Wg, const void* Wu,
                                    const void* Wd, void* Y, int64_t S, int* timed_out_host, void* cuda_stream);

/*
 * tsp_mlp_status - synchronizes nothing; reads (and clears) the plan's device status
 * word with a blocking 4-byte copy.  Call after synchronizing the stream.  Returns
 * TSP_OK or TSP_ERR_DEVICE_TIMEOUT (or TSP_ERR_CUDA if the copy failed).
 */
tsp_status_t tsp_mlp_status(tsp_mlp_plan_t* plan);

/*
 * tsp_mlp_selftest_wait_expiry - exercise the bounded-wait error path (no counterpart in the paper).
 * Launches one warp that waits, for at most `limit_ms` (1..1000), on a barrier nothing arrives on.  The
 * wait expires, the kernel sets the plan's status word and returns normally; after a synchronize,
 * tsp_mlp_status reports TSP_ERR_DEVICE_TIMEOUT (and clears the word) and the plan stays usable.
 * Nothing faults, traps or hangs.
 */
tsp_status_t tsp_mlp_selftest_wait_expiry(tsp_mlp_plan_t* plan, int limit_ms, void* cuda_stream);

/* Static, never-null description of a status code. */
const char* tsp_mlp_error_string(tsp_status_t status);
/* The cudaError_t / CUresult value of the last failed CUDA call on this plan (0 if none); with plan == NULL, of the
 * last failed CUDA call inside tsp_mlp_forward_static. */
int tsp_mlp_last_cuda_error(const tsp_mlp_plan_t* plan);

/*
 * tsp_mlp_ring_order - fill table[r*D + t] with the shard rank r uses at ring step t
 * (Algorithm 2: send to (p+1) mod D, receive from (p-1) mod D).  Host pointer, D*D ints.
 */
tsp_status_t tsp_mlp_ring_order(const tsp_mlp_plan_t* plan, int* table_host);

/*
 * Per-kernel timing.  tsp_mlp_profile_begin makes the plan record CUDA events on the
 * caller's stream around each kernel of the next `max_calls` forward/backward calls
 * (creates events; no device memory).  After synchronizing, tsp_mlp_profile_read
 * returns for call `call_index` the number of kernels and their durations in ms
 * (`ms_out` holds up to 8 floats; order: launch order).  tsp_mlp_profile_end frees the events.
 */
tsp_status_t tsp_mlp_profile_begin(tsp_mlp_plan_t* plan, int max_calls);
tsp_status_t tsp_mlp_profile_read(tsp_mlp_plan_t* plan, int call_index, int* n_kernels_out, float* ms_out);
tsp_status_t tsp_mlp_profile_end(tsp_mlp_plan_t* plan);

/* Number of kernels the most recent tsp_mlp_forward (pass=TSP_WS_FORWARD) or tsp_mlp_backward (pass=TSP_WS_BACKWARD)
 * on this plan launched.  Up to 12288 tokens per phase a forward call is 2 kernels and a backward call 4 (CTA-pair
 * path with F % 256 == 0, else 3); longer problems are cut into several launches per phase (token chunks), and the
 * weight-gradient contraction into one launch per 2^18 tokens.  Before the first call: 2 and 3. */
int tsp_mlp_kernels_per_call(const tsp_mlp_plan_t* plan, int pass);

#ifdef __cplusplus
}
#endif
#endif /* TSP_MLP_H */
