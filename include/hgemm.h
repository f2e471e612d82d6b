/*
 * hgemm.h -- C ABI of the B200 (sm_100a) half-precision GEMM library.
 *
 * Operation (paper section 2.1 "HGEMM": C = alpha*A*B + beta*C with alpha = 1,
 * beta = 0; operand layout of the "TN" baseline, appendix Listing 6):
 *
 *     C[i][j] = fp16_rn( sum_{k<K} A[i][k] * B[j][k] ),   i < M, j < N
 *
 *   A : M x K fp16, row-major, dense (row stride K)           -- device memory
 *   B : N x K fp16, K-contiguous (the K x N operand stored     -- device memory
 *       column-major), dense (row stride K)
 *   C : M x N fp16, row-major, dense (row stride N)            -- device memory
 *
 * Products are exact, sums are accumulated in fp32 on the tensor cores
 * (the paper allows fp16 or fp32 accumulators, section 1), and each result is
 * rounded once to fp16, round-to-nearest-even.  C is overwritten, never read.
 *
 * Conventions
 *   - All functions return a status; nothing throws across the boundary; out
 *     parameters are written only on HGEMM_OK.
 *   - Pointers passed to hgemm_run are DEVICE pointers on the context's device,
 *     16-byte aligned; the caller owns A, B, C; A and B must not overlap C.
 *   - Shapes: any M, N, K >= 1 (each at most 2^22).  The kernels address rows of
 *     16-byte multiples; when K % 8 != 0 the plan owns zero-padded copies of A and B
 *     that hgemm_run refreshes with a small copy kernel before the GEMM, and when
 *     N % 8 != 0 the rows of C are stored with 2-byte stores, 32 consecutive elements of
 *     a row per instruction (both slower than the
 *     aligned case, same results).  There is no CPU or library fallback path.
 *   - hgemm_run is asynchronous on the given stream.  It creates no stream,
 *     allocates nothing and never synchronises (the timing rules of paper
 *     section 2.4 "Avoiding Timing Measurement Hacking" forbid side streams);
 *     its return value is the launch status only.  The context's device must be
 *     the calling thread's current device.
 *   - A plan owns its split-K workspace: one plan must not run on two streams at
 *     the same time.  Plans are not thread-safe; use one per thread.
 */
#ifndef HGEMM_H_
#define HGEMM_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct hgemm_ctx_s hgemm_ctx_t;   /* opaque; one per device; owns its plans */
typedef struct hgemm_plan_s hgemm_plan_t; /* opaque; owned by its context */

typedef enum {
    HGEMM_OK = 0,
    HGEMM_ERR_INVALID_ARG = 1, /* null pointer, misaligned pointer, non-positive size */
    HGEMM_ERR_UNSUPPORTED = 2, /* shape or configuration the kernels cannot run */
    HGEMM_ERR_ALLOC = 3,       /* host or device allocation failed */
    HGEMM_ERR_CUDA = 4,        /* a CUDA runtime/driver call failed (see hgemm_last_cuda_error) */
    HGEMM_ERR_ARCH = 5,        /* the device is not compute capability 10.0 */
    HGEMM_ERR_TIMEOUT = 6,     /* a bounded device-side wait ran out (see hgemm_last_device_status) */
    HGEMM_ERR_SCRATCH_LIMIT = 7, /* hgemm_run_splitk_static: the call needs more scratch than the built-in buffer holds */
    HGEMM_ERR_CHECK = 8         /* the checked build (see hgemm_build_is_checked) found one of its invariants violated */
} hgemm_status_t;

/* Kernel families (section 5.1 of the paper picks a different kernel structure
 * for small and for large shapes; the families here are this library's own). */
enum {
    HGEMM_FAMILY_UMMA_1CTA = 0, /* persistent, warp-specialised, 128 x block_n tiles, one CTA per tile */
    HGEMM_FAMILY_UMMA_2CTA = 1, /* the same with CTA pairs: 256 x block_n tiles, B split across the pair */
    HGEMM_FAMILY_LIGHT = 2,     /* the small-problem kernel: one 128 x block_n tile per CTA, no persistent loop, one
                                   accumulator, no CTA-wide barrier at the end, only the shared memory it uses; its first
                                   loads leave before the CTA's set-up has finished.  Needs K % 8 == 0 and N % 8 == 0, split_k == 1, no
                                   tail_split, no swap_ab, fp32 accumulators, the TN layout, HGEMM_EPILOGUE_DIRECT or HGEMM_EPILOGUE_TMA */
    HGEMM_FAMILY_SMALL = 3      /* the register-accumulator kernel for the smallest problems: 64 x 64 or 32 x 32 tiles, cp.async +
                                   ldmatrix + mma.sync with fp32 accumulators in registers -- no tensor memory to allocate
                                   (0.7 us on B200), no tensor maps, no mbarriers.  Two tiles: block_m = block_n = 64 or 32,
                                   with block_k = 64, stages = 3, HGEMM_EPILOGUE_DIRECT; split_k in 1..16 (at most one slice per
                                   64-wide k-block), and with split_k > 1 split_mode = HGEMM_SPLIT_CLUSTER: the slices of a tile are
                                   the CTAs of one cluster and sum their partial tiles through its shared memory in slice order.
                                   Needs K % 8 == 0 and N % 8 == 0, no tail_split, no swap_ab, fp32 accumulators, the TN layout */
};

/* Where the fp32 partial sums of a split-K tile meet.  Both sum the slices in slice
 * order 0..S-1, so a configuration reproduces its own bits run after run. */
enum {
    HGEMM_SPLIT_WORKSPACE = 0, /* partials parked in a global workspace; any family; split_k <= 64.  The slices of a
                                  tile wait for one another on the GPU, which is safe because the grid never exceeds
                                  the SM count and holds one CTA per SM: all of them are resident at once WHEN THE
                                  GPU IS THEIRS.  If another long-running kernel holds SMs at the same time, slices
                                  may wait for CTAs that cannot start; the wait is bounded (hgemm_set_wait_budget),
                                  the launch then gives up and hgemm_last_device_status reports HGEMM_ERR_TIMEOUT */
    HGEMM_SPLIT_CLUSTER = 1    /* the slices of a tile form one thread-block cluster and are summed through
                                  distributed shared memory; split_k CTAs (1-CTA family) or CTA pairs (2-CTA family)
                                  per cluster, at most 16 CTAs: split_k in [2, 16] or [2, 8]; the tile's
                                  fp32 partial (512 * block_n bytes) plus split_k - 1 received shares of
                                  ceil(1/split_k) of it must fit in the stage ring and store staging
                                  (hgemm_validate_config answers) */
};

enum {
    HGEMM_ACC_F32 = 0,
    HGEMM_ACC_F16 = 1
};

enum {
    HGEMM_TAIL_K = 0,
    HGEMM_TAIL_N = 1,
    HGEMM_TAIL_STREAM = 2
};

enum {
    HGEMM_RASTER_SWEEP = 0,     /* every group of raster_group m-tiles sweeps the n-tiles from first to last */
    HGEMM_RASTER_SERPENTINE = 1 /* odd groups sweep from last to first (boustrophedon), so a group starts on the B
                                   tiles the group before it used last and finds them in L2 */
};

enum {
    HGEMM_EPILOGUE_DIRECT = 0,  /* registers -> 16-byte global stores */
    HGEMM_EPILOGUE_TMA = 1,     /* registers -> swizzled shared memory -> TMA store, 32 x 32 boxes */
    HGEMM_EPILOGUE_TMA_WIDE = 2 /* the same with 32-row x 64-column boxes: half as many fences, stores and
                                   commits per tile, for 32 KB more shared memory (fewer stages fit).  Needs
                                   split_k == 1 and block_n -- and the column pieces of HGEMM_TAIL_N -- a
                                   multiple of 64; with tail_split cutting along K, or a C whose rows are not
                                   multiples of 16 bytes, the cut tiles / the whole problem finish as with
                                   HGEMM_EPILOGUE_TMA resp. with element stores */
};

/* One point of the per-shape configuration space (the paper's BM/BN/BK, stage
 * count and block-swizzle stride of sections 5.2 and 6, plus split-K). */
typedef struct {
    int32_t family;       /* HGEMM_FAMILY_* */
    int32_t block_m;      /* 128 (1-CTA and light families), 256 (2-CTA pair), or block_n (small family) */
    int32_t block_n;      /* multiple of 32 in [32, 256]; or 512 (CTA-pair family only): a 256 x 512 tile held in both
                             tensor-memory accumulators at once, two MMAs per K step sharing the A tile -- a quarter less
                             shared-memory fill per flop than 256 x 256, no overlap of a tile's epilogue with the next
                             tile's MMAs.  Needs N % 512 == 0, split_k == 1, no tail_split, no swap_ab, the TN layout */
    int32_t block_k;      /* K extent of a pipeline stage: 64 or 128 (one or two 128-byte swizzle spans) */
    int32_t stages;       /* shared-memory ring depth, 2..12, bounded by shared memory */
    int32_t split_k;      /* >= 1; K slices reduced in slice order (deterministic) */
    int32_t raster_group; /* m-tiles per raster group (>= 1): tile order for L2 reuse */
    int32_t epilogue;     /* HGEMM_EPILOGUE_* (split_k > 1 always finishes with direct stores) */
    int32_t split_mode;   /* HGEMM_SPLIT_* : how the K slices of a tile are summed (ignored when split_k == 1) */
    int32_t tail_split;   /* 0 or 1: off.  >= 2 (needs split_k == 1): when the tiles do not fill a whole number of
                             waves of the persistent grid and the last wave is at most 1/tail_split full, its tiles
                             are cut into tail_split K slices (summed in slice order through the workspace) so that
                             every SM works until the end; otherwise ignored */
    int32_t tail_mode;    /* how tail_split cuts those tiles: HGEMM_TAIL_K (0) as above; HGEMM_TAIL_N (1): into
                             tail_split (2 or 4) column pieces of block_n / tail_split columns (a multiple of 32),
                             each an independent narrower tile -- no partial sums, no workspace;
                             HGEMM_TAIL_STREAM (2): stream-K.  The tiles beyond the last full wave (all tiles when there are
                             fewer tiles than SMs) are taken as one sequence of k-blocks in tile order and dealt out in equal
                             contiguous shares to min(SMs, tiles_left * tail_split) CTAs, so a CTA works on the end of one
                             tile and the start of the next; the pieces of a tile are summed in K order through the workspace
                             (deterministic).  Unlike the two other modes it applies whenever such tiles exist and K has at
                             least twice as many k-blocks as a share; needs block_n <= 256, no swap_ab, fp32 accumulators, not the wide epilogue */
    int32_t accumulate;   /* HGEMM_ACC_F32 (0): fp32 accumulators, the paper's main setting and this library's default;
                             HGEMM_ACC_F16 (1): fp16 accumulators in tensor memory (the paper's other valid setting for
                             fp16 inputs, section 1): every 16-wide K step rounds the running sums to fp16, so
                             results carry the larger error of that arithmetic.  Needs split_k == 1 and no K tail
                             split; never chosen by the planner or the tuned table */
    int32_t swap_ab;      /* 0: the tile's 128 (256 for a pair) accumulator rows are rows of C, block_n its columns.
                             1: the operands trade places inside the kernel -- the rows of B (N of them) go to the
                             accumulator rows, block_n covers rows of A, and the epilogue stores the tile transposed,
                             so C is the same row-major M x N matrix with the same values.  For few rows and many
                             columns (M <= 256, a projection of a few tokens through a wide weight matrix: the
                             paper's "BM ~ M" cases, section 5.2) this fills the 128-row side of the MMA with weight rows instead of zero
                             padding, and a CTA pair splits the small operand instead of re-reading all of it.
                             Needs N % 8 == 0, fp32 accumulators, the TN layout, no tail_split and not the wide epilogue */
    int32_t raster_mode;  /* HGEMM_RASTER_* : the order in which raster groups sweep the n-tiles */
    int32_t wave_pace;    /* 0 or 1.  1: the CTAs of the persistent grid start their r-th tile together -- a producer holds its
                             first load of a tile until every CTA has issued the last load of its previous tile (a counter in
                             device memory; the wait gives up after 50 us, nothing depends on it).  With many equal tiles per
                             CTA the CTAs otherwise drift apart and stop finding each other's operand panels in L2.  Same
                             arithmetic, same bits.  Needs the 1-CTA or CTA-pair family, split_k == 1 and no tail_split */
    int32_t reserved[1];  /* must be zero */
} hgemm_config_t;

/* Create a context on CUDA device `device` (>= 0).  HGEMM_ERR_ARCH unless the
 * device has compute capability 10.0.  Allocates 32 KB of device memory: status words
 * (one for the context, one per live plan: at most 4095 plans at a time) and, behind
 * them, one wave-pacing counter per plan (see hgemm_config_t::wave_pace). */
hgemm_status_t hgemm_create(hgemm_ctx_t **out, int device);

/* Free the context, every plan it still owns and their workspaces. */
hgemm_status_t hgemm_destroy(hgemm_ctx_t *ctx);

/* Plan one (M, N, K): picks a configuration (tuned table, else heuristic; rows of a table file named
 * by the environment variable HGEMM_TABLE, in the syntax the tuner writes, override the built-in table) and
 * allocates the split-K workspace if the configuration needs one.  May call
 * cudaMalloc/cudaMemset (synchronising); call it outside timed regions and
 * outside stream capture. */
hgemm_status_t hgemm_plan(hgemm_ctx_t *ctx, int64_t M, int64_t N, int64_t K, hgemm_plan_t **out);

/* How B is stored (paper section 2.2 evaluates both): HGEMM_LAYOUT_TN is the default of
 * hgemm_plan (B is N x K, K-contiguous: the K x N operand column-major); HGEMM_LAYOUT_NN
 * takes B as the K x N operand ROW-major (N-contiguous, row stride N), so that
 * C[i][j] = sum_k A[i][k] * B[k][j] with all three matrices row-major.  The NN layout
 * needs K % 8 == 0 and N % 8 == 0 (HGEMM_ERR_UNSUPPORTED otherwise) and tile widths that
 * are multiples of 64 (128 for the CTA-pair family); the planner rounds its choice up. */
typedef enum { HGEMM_LAYOUT_TN = 0, HGEMM_LAYOUT_NN = 1 } hgemm_layout_t;

hgemm_status_t hgemm_plan_layout(hgemm_ctx_t *ctx, int64_t M, int64_t N, int64_t K, hgemm_layout_t layout,
                                 hgemm_plan_t **out);

/* Launch C = A * B^T for the plan's shape on `stream` (a cudaStream_t, may be
 * NULL for the default stream).  A, B, C: device pointers as described above. */
hgemm_status_t hgemm_run(hgemm_plan_t *plan, const void *A, const void *B, void *C, void *stream);

/* The general form of the operation (paper section 2.1, "HGEMM"): C = alpha * A * B^T + beta * C,
 * in place in C (DEVICE pointers and layouts as for hgemm_run; alpha and beta are fp32
 * values passed by value).  The accumulator is fp32; each element is computed as
 * fma(beta, C_old, alpha * acc) in fp32 and rounded to fp16 once.  With beta == 0 the old
 * contents of C are never read (they may be uninitialised or NaN).  Every configuration the
 * plan can hold supports it, split-K included (the scaling is applied where the slices are
 * summed).  hgemm_run is the case alpha = 1, beta = 0, which the paper's experiments use.
 * HGEMM_ERR_INVALID_ARG for a NaN factor. */
hgemm_status_t hgemm_run_scaled(hgemm_plan_t *plan, float alpha, float beta, const void *A, const void *B, void *C,
                                void *stream);

/* The same operation on HOST buffers (paper section 2.3 builds its inputs on the
 * CPU): copies A and B to device staging owned by the plan, runs, copies C back.
 * A_host, B_host, C_host are HOST pointers with the layouts above; with page-locked
 * memory the call is asynchronous and the result is in C_host once `stream` has been
 * synchronised (work enqueued on `stream` after the call is ordered after the result
 * copy); with pageable memory the copies block.
 * The product runs on `stream`; the two operand copies and the result copy run on two
 * streams owned by the context, tied to it by events, so that over a sequence of calls
 * the inbound copies of one call overlap the product and the outbound copy of the calls
 * before it (PCIe carries both directions at once).  Consequence for the caller: A_host
 * and B_host are read from the moment of the call on -- NOT after the work queued on
 * `stream` before it -- so they must be complete when the call is made and stay
 * untouched until the call's work has finished.  Calls on one plan are ordered among
 * themselves (its staging is reused).
 * The first call on a context creates the two streams, the first call on a plan
 * allocates the staging and three events (cudaMalloc, synchronising): make it outside
 * timed regions.  HGEMM_ERR_ALLOC if the allocation fails. */
hgemm_status_t hgemm_run_host(hgemm_plan_t *plan, const void *A_host, const void *B_host, void *C_host, void *stream);

/* Split-K GEMM for callers that must not allocate.  (The paper has no counterpart:
 * this entry point exists for deployment, not for the method.)
 *
 * Who needs it: code that runs where device allocation is off limits -- a serving
 * process whose memory was frozen at start-up, a callback inside another library, a
 * job under a fixed-footprint policy.  hgemm_create and hgemm_plan call cudaMalloc,
 * so such callers cannot use them; this function needs neither a context nor a plan
 * and calls no cudaMalloc, cudaFree or any other allocating routine.  The split-K
 * partial sums, the arrival counters and the status word live in one static device
 * array inside the library: 8 MiB of partial sums plus a 4 KiB control page, held by
 * every GPU that loads the library until the process exits.  That array receives its
 * memory when the CUDA runtime loads the library's module on the device: under
 * CUDA's default lazy loading that is this function's FIRST call on the device,
 * under CUDA_MODULE_LOADING=EAGER it is context creation.  Make that first call (or
 * load eagerly) before memory is frozen; every later call leaves the amount of free
 * device memory as it found it.
 *
 * Same operation and layouts as hgemm_run (A: M x K, B: N x K, C: M x N, fp16, DEVICE
 * pointers, 16-byte aligned, caller-owned) on the calling thread's CURRENT device,
 * with the 1-CTA kernel family, tile width `block_n` (multiple of 32 in [32, 256]),
 * 64-wide K stages and `split_k` K slices summed in slice order through that array
 * (split_k == 1 is allowed; it neither reads nor writes the array).  Asynchronous on
 * `stream`.
 *
 * Limits and errors, checked before anything is launched:
 *   - ceil(M/128) * ceil(N/block_n) * split_k * 128 * block_n * 4 bytes of partial sums
 *     must fit in 8 MiB and the tile count in the control page (at most 480 tiles),
 *     else HGEMM_ERR_SCRATCH_LIMIT;
 *   - split_k <= min(64, ceil(K/64), SM count); K % 8 == 0 and N % 8 == 0 (no padded
 *     copies can be made here); otherwise as for hgemm_plan: HGEMM_ERR_UNSUPPORTED /
 *     HGEMM_ERR_INVALID_ARG; HGEMM_ERR_ARCH off sm_100.
 *
 * The first call on each device also looks up the array's device address
 * (cudaGetSymbolAddress) and sets the kernel's shared-memory limit; make it before any
 * stream capture begins.  That set-up is serialised inside the library, so first calls
 * from several threads are safe as far as the set-up goes.  Every call with
 * split_k > 1 shares the one array, which keeps the previous call's contents: the
 * function clears the control page on `stream` before each such launch (the partial
 * sums need no clearing), and two such calls that overlap on the GPU -- different
 * streams, or different threads -- race on it.  Serialise them.  A bounded wait that
 * runs out leaves C undefined; this variant has no status read-back. */
hgemm_status_t hgemm_run_splitk_static(int64_t M, int64_t N, int64_t K, int32_t block_n, int32_t split_k,
                                       const void *A, const void *B, void *C, void *stream);

/* Operands that no kernel ahead of the call in its stream writes.  hgemm_run launches with
 * programmatic stream serialisation (see hgemm_set_dependent_launch): the kernel may become
 * resident while the kernel ahead of it is still running, but it must not read A or B before that
 * kernel has completed, because it may be the one that produces them.  A caller who knows better
 * -- a projection whose weight matrix was written long ago -- can say so: with HGEMM_STATIC_B
 * (HGEMM_STATIC_A) the first pipeline stages' loads of B (A) are issued before the stream
 * dependency is resolved, so they are in flight while the previous kernel drains; the other
 * operand's loads and every store still wait.  `which` is a bit mask; 0 (the default) withdraws
 * the promise.  A wrong promise is a data race on that operand.  Applies to the two persistent
 * families with K-contiguous operands and K % 8 == 0; ignored elsewhere. */
enum { HGEMM_STATIC_A = 1, HGEMM_STATIC_B = 2 };
hgemm_status_t hgemm_plan_set_static_operands(hgemm_plan_t *plan, uint32_t which);

/* Free one plan early (hgemm_destroy frees the rest). */
hgemm_status_t hgemm_plan_destroy(hgemm_plan_t *plan);

/* Read / override the plan's configuration (tuner, tests).  set_config returns
 * HGEMM_ERR_UNSUPPORTED, leaving the plan unchanged, if the configuration is
 * illegal for the shape or does not fit shared/tensor memory; it may reallocate
 * the workspace (synchronising).  If that allocation fails it returns
 * HGEMM_ERR_ALLOC and the plan keeps its configuration and buffers and still runs. */
hgemm_status_t hgemm_plan_get_config(const hgemm_plan_t *plan, hgemm_config_t *out);
hgemm_status_t hgemm_plan_set_config(hgemm_plan_t *plan, const hgemm_config_t *cfg);

/* Run-time tuning of one plan (the library auto-tuning baseline of the paper's
 * section 6.1, for shapes the tuned table does not hold): times the plan's current
 * configuration and up to `max_candidates` others -- the legal configurations of
 * the shape, ranked by the planner's cost model -- with the caller's buffers on
 * `stream` (two untimed calls, then 3-64 back-to-back calls between CUDA events,
 * each candidate), installs the fastest, and runs it once more, so that on return
 * C (DEVICE, M x N) holds A B^T computed by the installed configuration.  A, B:
 * DEVICE pointers laid out as for hgemm_run; C is overwritten (no alpha / beta).
 * *best_us (HOST, may be NULL) receives the installed configuration's time per
 * call in microseconds.  Synchronous: it waits for the stream, many times, and may
 * reallocate the workspace.  It reads and clears the plan's device status; if a
 * bounded wait ran out during the search the plan keeps the configuration it had
 * and HGEMM_ERR_TIMEOUT is returned.  Candidates the plan's layout does not
 * support are skipped.  Costs about (max_candidates + 1) x 0.3-1 ms. */
hgemm_status_t hgemm_plan_autotune(hgemm_plan_t *plan, const void *A, const void *B, void *C, void *stream,
                                   int32_t max_candidates, float *best_us);

/* The candidates hgemm_plan_autotune draws from, as a pure host function: the legal
 * configurations of (M, N, K) on a device with `num_sms` SMs, ranked by the cost
 * model, best first; writes at most `max` of them to `out` (HOST array) and returns
 * how many (0 for an illegal shape or arguments). */
int32_t hgemm_candidate_configs(int64_t M, int64_t N, int64_t K, int32_t num_sms, hgemm_config_t *out, int32_t max);

/* The heuristic the planner falls back to, as a pure host function (no GPU
 * needed): configuration for (M, N, K) on a device with `num_sms` SMs. */
hgemm_status_t hgemm_heuristic_config(int64_t M, int64_t N, int64_t K, int32_t num_sms, hgemm_config_t *out);

/* The configuration hgemm_plan starts from, as a pure host function: the tuned table's
 * entry for a tabulated shape; for any other shape the best, by the cost model calibrated
 * on the measured times of the tabulated shapes around it, of the heuristic's choice and
 * those neighbours' configurations re-fitted to the shape. */
hgemm_status_t hgemm_planned_config(int64_t M, int64_t N, int64_t K, int32_t num_sms, hgemm_config_t *out);

/* Check a configuration against a shape without a GPU: HGEMM_OK if legal. */
hgemm_status_t hgemm_validate_config(int64_t M, int64_t N, int64_t K, const hgemm_config_t *cfg);

/* The planner's cost model: estimated SM clock cycles of one run (a ranking aid for
 * the tuner, not a prediction); negative if the configuration is illegal. */
double hgemm_estimate_config(int64_t M, int64_t N, int64_t K, int32_t num_sms, const hgemm_config_t *cfg);

/* Dynamic shared memory (bytes) and split-K workspace (bytes) a configuration needs. */
int64_t hgemm_config_smem_bytes(const hgemm_config_t *cfg);
int64_t hgemm_config_workspace_bytes(int64_t M, int64_t N, int64_t K, const hgemm_config_t *cfg);

/* Number of kernels the last hgemm_run of this plan launched (1). */
int32_t hgemm_plan_launches_per_run(const hgemm_plan_t *plan);

/* Every device-side wait is bounded (the timing rules of paper section 2.4 presuppose calls that
 * return); when one runs out the kernel records (role << 24 | barrier index << 8 | stage) in the
 * status word of the plan whose launch it was, drains and returns.  Each plan has its own word, so
 * two plans running on two streams can tell whose wait ran out.
 *
 * hgemm_last_device_status(plan, code): synchronises the device, reads the plan's word into *code
 * (HOST pointer; 0 = no event), clears it, and returns HGEMM_ERR_TIMEOUT if it was non-zero; in that
 * case the plan's split-K arrival counters (no other plan's) are started again from zero, so the
 * plan is usable afterwards.
 *
 * hgemm_ctx_last_device_status(ctx, code): the same over the whole context -- its own word (written
 * by hgemm_debug_timeout_probe) and the word of every live plan; *code receives the first non-zero
 * one (the context's, then plans in creation order), all are cleared, and every plan whose word was
 * set has its counters restarted. */
hgemm_status_t hgemm_last_device_status(hgemm_plan_t *plan, uint32_t *code);
hgemm_status_t hgemm_ctx_last_device_status(hgemm_ctx_t *ctx, uint32_t *code);

/* Wait budget of the bounded waits, in SM clock cycles (default 2e9, about a
 * second).  Affects plans created afterwards and later hgemm_run calls. */
hgemm_status_t hgemm_set_wait_budget(hgemm_ctx_t *ctx, int64_t cycles);

/* 1 when this library was compiled as the checked build (-DHGEMM_CHECKED=1, `python -m paper_2512_02551_b200.build
 * --checked` writes it beside the ordinary one as libhgemm_checked.so), else 0.  The checked build tests, where they are
 * used, the invariants the kernels otherwise rely on: a work item inside the tile grid and the K range, TMA coordinates on
 * 16-byte boundaries, reduced units and the small family's stores inside C, parked partial sums inside the workspace and
 * their arrival counters inside their array, accumulator columns inside the tensor-memory allocation.  A violation is
 * recorded in the plan's status word -- code (7 << 24) | (site << 8) -- the access is skipped, and
 * hgemm_last_device_status / hgemm_ctx_last_device_status return HGEMM_ERR_CHECK.  Same ABI, same results, a few
 * per cent slower; meant for the test suite and for chasing a suspected library bug, not for production. */
int32_t hgemm_build_is_checked(void);

/* Test hook: a one-thread kernel that evaluates an invariant that is false by construction, so that the reporting path
 * can be exercised without any bad access.  In the checked build the context's status word then reads HGEMM_ERR_CHECK with
 * code (7 << 24) | (99 << 8); in the ordinary build nothing is recorded. */
hgemm_status_t hgemm_debug_check_probe(hgemm_ctx_t *ctx, void *stream);

/* Test hook for the stream-K tail (HGEMM_TAIL_STREAM): work item `h` (0 or 1) of CTA position `position` under
 * configuration `cfg` on a device with `num_sms` SMs, as the kernel decodes it.  out[0..5] = tile index, first
 * k-block, number of k-blocks (0: no such item), slice (the item's place among the pieces of its tile, in K
 * order), slices (pieces of that tile), positions in use.  HGEMM_ERR_UNSUPPORTED when the configuration has no
 * stream-K tail on this shape.  Host arithmetic only; no device is touched. */
hgemm_status_t hgemm_debug_stream_item(int64_t M, int64_t N, int64_t K, const hgemm_config_t *cfg, int32_t num_sms,
                                       int32_t position, int32_t h, int32_t out[6]);

/* hgemm_run launches with programmatic stream serialisation (on by default): the
 * kernel may become resident, and run the set-up that touches no global memory,
 * while the kernel ahead of it in the stream is still finishing; it waits for that
 * kernel's completion before its first global-memory access, so stream order is
 * kept for every buffer.  Back-to-back calls then overlap launch latency and set-up
 * with the previous call's tail.  enabled = 0 restores plain stream-ordered launches. */
hgemm_status_t hgemm_set_dependent_launch(hgemm_ctx_t *ctx, int32_t enabled);

/* Test hook for the timeout path: launches one small kernel on `stream` whose
 * only wait is on a barrier that nothing signals, with the context's wait
 * budget.  The kernel returns by itself; hgemm_ctx_last_device_status then reports
 * HGEMM_ERR_TIMEOUT.  Nothing faults or hangs. */
hgemm_status_t hgemm_debug_timeout_probe(hgemm_ctx_t *ctx, void *stream);

/* Instrumentation: when `device_buf` (DEVICE pointer to 24 uint64, or NULL to switch
 * it off) is set, CTA 0 of every later launch of this plan writes nanosecond
 * %globaltimer stamps of its pipeline events: 0 and 1 the producer's dependency wait
 * has returned (set-up done, first work item decoded, first stage claimed),
 * 2 first TMA load issued, 3 first k-block landed, 4 last MMA issued, 5 first
 * accumulator ready, 6 epilogue done, 7 tensor memory freed; and SM-clock totals:
 * 8/9/10 MMA thread waiting for data / issuing MMAs / committing, 11/12 producer
 * waiting for a free stage / issuing loads, 13 MMA thread waiting for a free
 * accumulator, 15 k-blocks processed; and for split-K stamps 16 partial parked,
 * 17 all slices arrived, 18 share reduced; for cluster split-K 16 arrived at the
 * cluster's first barrier, 17 partial staged, 19 cluster gathered, 18 shares sent,
 * 20 shares received, 22 share reduced, 21 cluster released.  The caller owns the
 * buffer.  While a trace buffer or a skip mask (below) is set, launches run the
 * instrumented instantiation of the kernel, which is 10-15 % slower on small and
 * mid-size shapes than the one that runs otherwise: the stamps describe the
 * pipeline's structure and proportions, not the production kernel's absolute times.
 * The instrumented kernels do not exist for swapped-operand configurations (swap_ab = 1),
 * for the 512-wide tile or for the small family: hgemm_run returns HGEMM_ERR_UNSUPPORTED for such a plan while a
 * trace buffer or a skip mask is set.  The light family writes its own stamps, SM-clock
 * values (clock64) of CTA 0 in slots 0..12: 0 entry, 1 first barriers initialised, 2 first
 * loads issued, 3 tensor memory allocated, 4 set-up barrier passed, 5 first k-block landed,
 * 6 last MMA issued, 7 accumulator ready, 8 first chunk converted, 9 last store issued,
 * 10 epilogue warp done, 11 tensor memory read by every epilogue warp, 12 tensor memory
 * freed; it has no skip mask. */
hgemm_status_t hgemm_debug_set_trace(hgemm_plan_t *plan, void *device_buf);

/* Instrumentation for bottleneck analysis: bit 0 makes later launches of this plan
 * issue no TMA loads, bit 1 no MMAs, bit 2 no TMA stores (the pipeline still runs;
 * C is garbage).  Bit 3 changes no arithmetic: with a trace buffer set, EVERY CTA
 * also writes the stamps 0 (started) and 7 (finished) behind CTA 0's 24 slots, at
 * entries 24 + 2 * blockIdx and 25 + 2 * blockIdx -- the buffer must then hold
 * 24 + 2 * 148 uint64.
 * 0 restores normal operation. */
hgemm_status_t hgemm_debug_set_skip(hgemm_plan_t *plan, uint32_t mask);

/* Test hook for the allocation-failure paths (an injected error code, no memory pressure on the
 * GPU): of the device allocations the library makes through this context from now on -- split-K
 * workspace and counters, padded operand copies, host-call staging -- the first `after` go
 * through, the next `count` report failure without calling cudaMalloc, so the caller sees
 * HGEMM_ERR_ALLOC.  count = 0 switches it off. */
hgemm_status_t hgemm_debug_fail_allocs(hgemm_ctx_t *ctx, int32_t after, int32_t count);

/* cudaError_t (as int) of the last failing CUDA call made through this context. */
int32_t hgemm_last_cuda_error(const hgemm_ctx_t *ctx);

const char *hgemm_status_string(hgemm_status_t s);

#ifdef __cplusplus
}
#endif
#endif /* HGEMM_H_ */
