// C ABI of the HGEMM library (see include/hgemm.h): contexts, plans, tensor maps, launches.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstdio>
#include <cstring>
#include <new>
#include <vector>

#include "../../include/hgemm.h"
#include "hgemm_kernel.cuh"
#include "hgemm_light_kernel.cuh"
#include "hgemm_small_kernel.cuh"
#include "hgemm_planner.h"

using hgemm_dev::KernelParams;

typedef CUresult (*encode_tiled_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *,
                                    const cuuint64_t *, const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave,
                                    CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

// Device status words: one array per context.  Slot 0 belongs to the context itself (the timeout probe), every
// plan owns one of the others, so that a wait that ran out names the plan whose launch it was.
constexpr int kStatusSlots = 4096;

struct hgemm_ctx_s {
    int device = 0;
    int num_sms = 0;
    uint32_t *d_status = nullptr;          // kStatusSlots words
    std::vector<int> free_status_slots;    // slots no plan owns (never holds 0)
    int pass_allocs = 0, fail_allocs = 0;  // test hook: after pass_allocs more device allocations, fail_allocs of them report failure
    long long wait_budget = 2000000000LL;
    encode_tiled_fn encode = nullptr;
    int last_cuda_error = 0;
    bool dependent_launch = true;
    bool tma_3d = true;
    std::vector<hgemm_plan_s *> plans;
    // hgemm_run_host: the operand copies and the result copy run on streams of their own (created by its first call), so that
    // one call's copies overlap the compute and the opposite-direction copy of the calls around it
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
};

struct hgemm_plan_s {
    hgemm_ctx_s *ctx = nullptr;
    int64_t M = 0, N = 0, K = 0;   // K is the padded K (multiple of 8) every kernel parameter is derived from
    int64_t K_user = 0;            // the caller's K
    int layout = HGEMM_LAYOUT_TN;  // how B is stored
    void *pad_a = nullptr, *pad_b = nullptr;   // K-padded copies of A and B when K_user % 8 != 0
    hgemm_config_t cfg;
    KernelParams params;
    int grid = 0;
    int cluster_dim = 1;
    int smem = 0;
    unsigned long long *trace = nullptr;
    uint32_t debug_skip = 0;
    uint32_t static_operands = 0;  // HGEMM_STATIC_A | HGEMM_STATIC_B as the caller declared them
    void *workspace = nullptr;
    int64_t workspace_bytes = 0;
    uint32_t *counters = nullptr;
    int64_t counter_bytes = 0;
    uint32_t epoch = 0;            // launches that have used `counters` since they were last cleared
    uint32_t wave_total = 0;       // arrivals that earlier launches have added to this plan's pacing counter (modulo 2^32)
    int status_slot = 0;           // this plan's word in the context's status array
    // tensor maps depend on the pointers: a small cache keyed by (A, B, C), round-robin replacement
    struct MapEntry {
        const void *a = nullptr, *b = nullptr;
        void *c = nullptr;
        CUtensorMap tmap_a, tmap_b, tmap_c;
        CUtensorMap tmap_bt;   // B for the column pieces of tail tiles (fewer rows per box)
    };
    static constexpr int kMapCache = 64;
    MapEntry maps[kMapCache];
    int maps_used = 0, maps_next = 0;
    // device staging of hgemm_run_host (allocated by its first call)
    void *stage_a = nullptr, *stage_b = nullptr, *stage_c = nullptr;
    // ... and its hand-offs: operands on the device / product computed / result on the host (of the plan's latest call)
    cudaEvent_t ev_in = nullptr, ev_gemm = nullptr, ev_out = nullptr;
    bool host_call_in_flight = false;   // the events above have been recorded at least once
};

namespace {

hgemm_status_t cuda_fail(hgemm_ctx_s *ctx, cudaError_t e)
{
    if (ctx) ctx->last_cuda_error = int(e);
    (void)cudaGetLastError();
    return HGEMM_ERR_CUDA;
}

// Every device allocation of the library goes through here (hgemm_debug_fail_allocs can make it fail).
cudaError_t ctx_malloc(hgemm_ctx_s *ctx, void **out, size_t bytes)
{
    if (ctx && ctx->fail_allocs > 0) {
        if (ctx->pass_allocs > 0) {
            --ctx->pass_allocs;
        } else {
            --ctx->fail_allocs;
            *out = nullptr;
            return cudaErrorMemoryAllocation;
        }
    }
    return cudaMalloc(out, bytes);
}

int32_t pow2_at_least(int32_t x)
{
    int32_t p = 32;
    while (p < x) p <<= 1;
    return p;
}

uint32_t make_idesc(int m, int n, bool b_mn_major = false, bool d_f16 = false)
{
    // tcgen05 instruction descriptor, kind::f16: D = fp32 (or fp16), A = B = fp16, both K-major, dense
    uint32_t d = 0;
    d |= (d_f16 ? 0u : 1u) << 4;       // [4,6)   D format: 0 = fp16, 1 = fp32
    d |= 0u << 7;                      // [7,10)  A format: 0 = fp16
    d |= 0u << 10;                     // [10,13) B format: 0 = fp16
    d |= 0u << 15;                     // [15]    A major: 0 = K
    d |= (b_mn_major ? 1u : 0u) << 16; // [16]    B major: 0 = K, 1 = N (B stored K x N row-major)
    d |= uint32_t(n >> 3) << 17;       // [17,23) N >> 3
    d |= uint32_t(m >> 4) << 24;       // [24,29) M >> 4
    return d;
}

// Applies a validated configuration to a plan: derived kernel parameters, workspace.
hgemm_status_t apply_config(hgemm_plan_s *pl, const hgemm_config_t &cfg)
{
    hgemm_ctx_s *ctx = pl->ctx;
    const int cg = hgemm_host::cta_group_of(cfg);
    // the slices of a tile wait for each other: each needs its own SM (or SM pair)
    if (cfg.split_k > 1 && cfg.split_k > ctx->num_sms / cg) return HGEMM_ERR_UNSUPPORTED;
    if (pl->layout == HGEMM_LAYOUT_NN && (cfg.block_n % (64 * cg)) != 0) return HGEMM_ERR_UNSUPPORTED;
    if (pl->layout == HGEMM_LAYOUT_NN && cfg.swap_ab) return HGEMM_ERR_UNSUPPORTED;   // the swapped form is built for K-contiguous operands
    if (pl->layout == HGEMM_LAYOUT_NN && cfg.block_n == 512) return HGEMM_ERR_UNSUPPORTED;   // so is the double-accumulator tile
    if (pl->layout == HGEMM_LAYOUT_NN && (cfg.family == HGEMM_FAMILY_LIGHT || cfg.family == HGEMM_FAMILY_SMALL)) return HGEMM_ERR_UNSUPPORTED;   // and the two small-problem kernels
    // row-major B is staged in blocks of 64 columns: column pieces of tail tiles must be whole blocks per CTA
    if (pl->layout == HGEMM_LAYOUT_NN && cfg.tail_mode == HGEMM_TAIL_N && cfg.tail_split >= 2 &&
        ((cfg.block_n / cfg.tail_split) % (64 * cg)) != 0)
        return HGEMM_ERR_UNSUPPORTED;
    // (the small family's K slices are a cluster of its own kernel: at most 16 CTAs of 128 threads and 48 KB, placed anywhere)
    const bool cluster_split = cfg.split_k > 1 && cfg.split_mode == HGEMM_SPLIT_CLUSTER && cfg.family != HGEMM_FAMILY_SMALL;
    if (cluster_split) {
        // can the device place a cluster of split_k CTAs of this kernel at all?
        cudaLaunchConfig_t lc;
        std::memset(&lc, 0, sizeof(lc));
        lc.gridDim = dim3(unsigned(cfg.split_k * cg), 1, 1);
        lc.blockDim = dim3(hgemm_dev::kThreads, 1, 1);
        lc.dynamicSmemBytes = size_t(hgemm_host::kSmemOptInBytes);
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = unsigned(cfg.split_k * cg);      // the slices' CTAs (CTA pairs) form one cluster
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        lc.attrs = attr;
        lc.numAttrs = 1;
        int clusters = 0;
        cudaError_t e = cg == 2 ? cudaOccupancyMaxActiveClusters(&clusters, hgemm_dev::hgemm_umma_kernel<2, false, 2, true, false, 1>, &lc)
                                : cudaOccupancyMaxActiveClusters(&clusters, hgemm_dev::hgemm_umma_kernel<1, false, 2, true, false, 1>, &lc);
        if (e != cudaSuccess) {
            (void)cudaGetLastError();
            return HGEMM_ERR_UNSUPPORTED;
        }
        if (clusters < 1) return HGEMM_ERR_UNSUPPORTED;
    }
    const hgemm_host::SplitLayout layout = hgemm_host::split_layout(pl->M, pl->N, pl->K, ctx->num_sms, cfg);
    const int64_t ws = hgemm_host::workspace_bytes(pl->M, pl->N, pl->K, cfg, ctx->num_sms);
    const int64_t cb = hgemm_host::counter_bytes(pl->M, pl->N, cfg, ctx->num_sms, pl->K);
    // Nothing of the plan changes until every step that can fail has succeeded: larger buffers are allocated
    // beside the old ones and swapped in only then, so a failed call leaves a plan that still runs as before.
    void *new_ws = nullptr;
    uint32_t *new_ctr = nullptr;
    if (ws > pl->workspace_bytes) {
        cudaError_t e = ctx_malloc(ctx, &new_ws, size_t(ws));
        if (e != cudaSuccess) {
            cuda_fail(ctx, e);
            return HGEMM_ERR_ALLOC;
        }
    }
    if (cb > pl->counter_bytes) {
        cudaError_t e = ctx_malloc(ctx, reinterpret_cast<void **>(&new_ctr), size_t(cb));
        if (e != cudaSuccess) {
            if (new_ws) cudaFree(new_ws);
            cuda_fail(ctx, e);
            return HGEMM_ERR_ALLOC;
        }
    }
    {
        // arrival counters start from zero under a new configuration (harmless for the old one, whose next
        // launch then counts from epoch 1 again)
        uint32_t *ctr = new_ctr ? new_ctr : pl->counters;
        const int64_t ctr_bytes = new_ctr ? cb : pl->counter_bytes;
        if (ctr) {
            cudaError_t e = cudaMemset(ctr, 0, size_t(ctr_bytes));
            if (e != cudaSuccess) {
                if (new_ws) cudaFree(new_ws);
                if (new_ctr) cudaFree(new_ctr);
                return cuda_fail(ctx, e);
            }
            pl->epoch = 0;
        }
    }
    if (new_ws) {
        if (pl->workspace) cudaFree(pl->workspace);
        pl->workspace = new_ws;
        pl->workspace_bytes = ws;
    }
    if (new_ctr) {
        if (pl->counters) cudaFree(pl->counters);
        pl->counters = new_ctr;
        pl->counter_bytes = cb;
    }

    pl->cfg = cfg;
    KernelParams &p = pl->params;
    std::memset(&p, 0, sizeof(p));
    // a swapped configuration runs the kernel on the transposed problem: its rows are the caller's columns
    const int64_t kM = cfg.swap_ab ? pl->N : pl->M, kN = cfg.swap_ab ? pl->M : pl->N;
    p.M = int32_t(kM);
    p.N = int32_t(kN);
    p.K = int32_t(pl->K);
    p.transposed = cfg.swap_ab ? 1 : 0;
    p.raster_serpentine = cfg.raster_mode == HGEMM_RASTER_SERPENTINE ? 1 : 0;
    p.tiles_m = int32_t((kM + 128 * cg - 1) / (128 * cg));
    p.tiles_n = int32_t((kN + cfg.block_n - 1) / cfg.block_n);
    p.split_k = int32_t(layout.slices);
    p.first_split_tile = int32_t(layout.first_split_tile);
    p.total_work = int32_t(layout.work_items);
    p.tail_pieces = int32_t(layout.pieces);
    p.block_k = cfg.block_k;
    p.kblocks = int32_t((pl->K + cfg.block_k - 1) / cfg.block_k);
    p.block_n = cfg.block_n;
    p.stages = cfg.stages;
    p.raster_group = std::min(cfg.raster_group, p.tiles_m);
    {
        // divisors of the work decode as multiply-and-shift constants
        const int32_t rg = std::max(1, std::min(p.raster_group, p.tiles_m));
        const int32_t last = p.tiles_m - ((p.tiles_m - 1) / rg) * rg;       // m-tiles of the last raster group
        p.fd_per_group = hgemm_dev::make_fast_div(uint32_t(rg) * uint32_t(p.tiles_n));
        p.fd_raster = hgemm_dev::make_fast_div(uint32_t(rg));
        p.fd_last_group = hgemm_dev::make_fast_div(uint32_t(last));
        p.fd_split = hgemm_dev::make_fast_div(uint32_t(std::max(1, p.split_k)));
        p.fd_pieces = hgemm_dev::make_fast_div(uint32_t(std::max(1, p.tail_pieces)));
        // stream-K tail: positions, k-blocks of the tail, k-blocks of a tile
        p.stream_units = int32_t(layout.stream_units);
        p.stream_q = int32_t((layout.tiles - layout.first_split_tile) * p.kblocks);
        p.grid_units = std::max(1, ctx->num_sms / cg);
        p.fd_stream_units = hgemm_dev::make_fast_div(uint32_t(std::max(1, p.stream_units)));
        p.fd_stream_q = hgemm_dev::make_fast_div(uint32_t(std::max(1, p.stream_q)));
        p.fd_kblocks = hgemm_dev::make_fast_div(uint32_t(std::max(1, p.kblocks)));
    }
    p.tmem_cols = cfg.block_n == 512 ? 512 : pow2_at_least(2 * cfg.block_n);   // two accumulators either way
    if (cfg.family == HGEMM_FAMILY_LIGHT) p.tmem_cols = pow2_at_least(cfg.block_n);   // ... except in the light kernel: one
    p.ragged_n = (!cfg.swap_ab && (pl->N % 8) != 0) ? 1 : 0;   // (a swapped configuration needs N % 8 == 0 and stores by its own rule)
    p.epilogue_tma = (cfg.epilogue != HGEMM_EPILOGUE_DIRECT && cfg.split_k == 1 && !p.ragged_n)             // whole tiles only
                         ? (cfg.epilogue == HGEMM_EPILOGUE_TMA_WIDE ? 2 : 1) : 0;
    // (the 512-wide double tile issues two MMAs of N = 256 per K step)
    p.idesc = make_idesc(128 * cg, cfg.block_n == 512 ? 256 : cfg.block_n, pl->layout == HGEMM_LAYOUT_NN, cfg.accumulate == HGEMM_ACC_F16);
    p.acc_f16 = cfg.accumulate == HGEMM_ACC_F16 ? 1 : 0;
    p.idesc_tail = make_idesc(128 * cg, cfg.block_n / int(std::max<int64_t>(1, layout.pieces)), pl->layout == HGEMM_LAYOUT_NN,
                              cfg.accumulate == HGEMM_ACC_F16);
    p.b_row_major = pl->layout == HGEMM_LAYOUT_NN ? 1 : 0;
    p.workspace = static_cast<float *>(pl->workspace);
    p.workspace_floats = static_cast<unsigned long long>(pl->workspace_bytes / 4);
    p.counter_words = static_cast<unsigned long long>(pl->counter_bytes / 4);
    p.counters = pl->counters;
    p.status = ctx->d_status + pl->status_slot;
    p.cluster_split = cluster_split ? 1 : 0;
    p.tma_3d = (cfg.block_k == 128 && (pl->K % 64) == 0 && ctx->tma_3d && pl->layout == HGEMM_LAYOUT_TN && cfg.family != HGEMM_FAMILY_LIGHT) ? 1 : 0;
    p.C = nullptr;
    p.wait_budget = ctx->wait_budget;
    {
        // wave pacing needs at least two tiles per CTA (pair) to have anything to pace
        const int pace_units = std::max(1, ctx->num_sms / cg);
        p.wave_rounds = (p.total_work + pace_units - 1) / pace_units;
        p.wave_pace = (cfg.wave_pace && p.wave_rounds >= 2) ? 1 : 0;
        p.wave_counter = ctx->d_status + kStatusSlots + pl->status_slot;
    }
    const int units = std::max(1, ctx->num_sms / cg);
    // cluster split-K is not persistent: one CTA per (tile, slice), the hardware schedules the clusters
    pl->grid = cluster_split ? cg * p.total_work : cg * std::min(p.total_work, units);
    pl->cluster_dim = cluster_split ? cg * cfg.split_k : cg;
    // Always ask for the whole opt-in shared memory: it keeps a second CTA off the SM, so two
    // CTAs can never wait on each other's tensor-memory allocation.  (Letting small configurations ask for what
    // they use, so that the next call's CTAs become resident beside this call's, made those calls slower.)
    pl->smem = int(hgemm_host::kSmemOptInBytes);
    if (cfg.family == HGEMM_FAMILY_SMALL) {
        // 64 x 64 or 32 x 32 tiles, one CTA each, static shared memory, no tensor maps
        p.tiles_m = int32_t((pl->M + cfg.block_n - 1) / cfg.block_n);
        p.tiles_n = int32_t((pl->N + cfg.block_n - 1) / cfg.block_n);
        pl->grid = p.tiles_m * p.tiles_n * std::max(1, cfg.split_k);
        pl->cluster_dim = std::max(1, cfg.split_k);
        pl->smem = 0;
    }
    if (cfg.family == HGEMM_FAMILY_LIGHT) {
        // one CTA per tile, and only the shared memory the configuration uses
        pl->grid = p.tiles_m * p.tiles_n;
        pl->cluster_dim = 1;
        pl->smem = int(hgemm_host::smem_bytes(cfg));
    }
    pl->maps_used = pl->maps_next = 0;   // the B box depends on the configuration
    return HGEMM_OK;
}

// The kernel instantiation for a CTA group size, store-box width and kind of split-K reduction
// (0: no K slices, 1: through the workspace -- also a tail cut along K --, 2: inside a cluster); `plain` selects
// the instantiation without the optional features, `trace` the one with the instrumentation (never plain).
template <bool PLAIN, bool TRACE, int SUBS, bool XPOSE>
const void *kernel_of(int cg, bool wide, int split)
{
    using namespace hgemm_dev;
#define HGEMM_K(CG, W, S) reinterpret_cast<const void *>(hgemm_umma_kernel<CG, W, S, PLAIN, TRACE, SUBS, XPOSE>)
    if constexpr (XPOSE) {                   // transposed stores: no wide boxes
        if (cg == 1) return split == 0 ? HGEMM_K(1, false, 0) : split == 1 ? HGEMM_K(1, false, 1) : HGEMM_K(1, false, 2);
        return split == 0 ? HGEMM_K(2, false, 0) : split == 1 ? HGEMM_K(2, false, 1) : HGEMM_K(2, false, 2);
    } else {
        if (cg == 1) {
            if (wide) return split == 0 ? HGEMM_K(1, true, 0) : HGEMM_K(1, true, 1);      // no split_k > 1 with wide boxes
            return split == 0 ? HGEMM_K(1, false, 0) : split == 1 ? HGEMM_K(1, false, 1) : HGEMM_K(1, false, 2);
        }
        if (wide) return split == 0 ? HGEMM_K(2, true, 0) : HGEMM_K(2, true, 1);
        return split == 0 ? HGEMM_K(2, false, 0) : split == 1 ? HGEMM_K(2, false, 1) : HGEMM_K(2, false, 2);
    }
#undef HGEMM_K
}

// The double-accumulator pair tile (block_n == 512): CTA pairs, no K slices, no transposed stores, no instrumentation.
template <bool PLAIN, int SUBS>
const void *dual_kernel_of(bool wide)
{
    using namespace hgemm_dev;
    return wide ? reinterpret_cast<const void *>(hgemm_umma_kernel<2, true, 0, PLAIN, false, SUBS, false, true>)
                : reinterpret_cast<const void *>(hgemm_umma_kernel<2, false, 0, PLAIN, false, SUBS, false, true>);
}

// The stream-K tail (HGEMM_TAIL_STREAM): 32-column store boxes or direct stores, no transposed stores, no instrumentation.
template <bool PLAIN, int SUBS>
const void *stream_kernel_of(int cg)
{
    using namespace hgemm_dev;
    return cg == 1 ? reinterpret_cast<const void *>(hgemm_umma_kernel<1, false, 3, PLAIN, false, SUBS, false, false>)
                   : reinterpret_cast<const void *>(hgemm_umma_kernel<2, false, 3, PLAIN, false, SUBS, false, false>);
}

// `subs`: 64-wide sub-tiles per stage (block_k / 64); the plain instantiations are compiled for each value.
// `xpose`: the instantiations that store the tile transposed (swapped operands); they exist without instrumentation.
// `dual`: the instantiations for block_n == 512.
const void *kernel_for(int cg, bool wide, int split, bool plain, bool trace, int subs, bool xpose = false, bool dual = false)
{
    if (dual) {
        if (!plain) return dual_kernel_of<false, 0>(wide);
        return subs == 2 ? dual_kernel_of<true, 2>(wide) : dual_kernel_of<true, 1>(wide);
    }
    if (split == 3) {
        if (!plain) return stream_kernel_of<false, 0>(cg);
        return subs == 2 ? stream_kernel_of<true, 2>(cg) : stream_kernel_of<true, 1>(cg);
    }
    if (xpose) {
        if (!plain) return kernel_of<false, false, 0, true>(cg, false, split);
        return subs == 2 ? kernel_of<true, false, 2, true>(cg, false, split) : kernel_of<true, false, 1, true>(cg, false, split);
    }
    if (trace) return kernel_of<false, true, 0, false>(cg, wide, split);
    if (!plain) return kernel_of<false, false, 0, false>(cg, wide, split);
    return subs == 2 ? kernel_of<true, false, 2, false>(cg, wide, split) : kernel_of<true, false, 1, false>(cg, wide, split);
}

bool encode_2d(hgemm_ctx_s *ctx, CUtensorMap *map, const void *base, uint64_t inner, uint64_t outer, uint32_t box_inner,
               uint32_t box_outer, CUtensorMapSwizzle swizzle)
{
    cuuint64_t dims[2] = {inner, outer};
    cuuint64_t strides[1] = {inner * 2};   // bytes between rows
    cuuint32_t box[2] = {box_inner, box_outer};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = ctx->encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, swizzle, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        ctx->last_cuda_error = int(r);
        return false;
    }
    return true;
}

// A and B as 3-D tensors {64, rows, K / 64}: element (x, y, z) = row y, column 64 z + x.  A box
// {64, rows, 2} then lands as two consecutive 64-wide sub-tiles, which is the layout of a 128-wide stage.
// Only valid when K is a multiple of 64 (dimension 0 must not run past the end of a row).
bool encode_3d_ksub(hgemm_ctx_s *ctx, CUtensorMap *map, const void *base, uint64_t K, uint64_t rows, uint32_t box_rows)
{
    cuuint64_t dims[3] = {64, rows, K / 64};
    cuuint64_t strides[2] = {K * 2, 128};   // bytes: next row, next 64-wide sub-tile
    cuuint32_t box[3] = {64, box_rows, 2};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = ctx->encode(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 3, const_cast<void *>(base), dims, strides, box, estr,
                             CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                             CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        ctx->last_cuda_error = int(r);
        return false;
    }
    return true;
}

} // namespace

extern "C" {

const char *hgemm_status_string(hgemm_status_t s)
{
    switch (s) {
    case HGEMM_OK: return "ok";
    case HGEMM_ERR_INVALID_ARG: return "invalid argument";
    case HGEMM_ERR_UNSUPPORTED: return "unsupported shape or configuration";
    case HGEMM_ERR_ALLOC: return "allocation failed";
    case HGEMM_ERR_CUDA: return "CUDA call failed";
    case HGEMM_ERR_ARCH: return "device is not compute capability 10.0";
    case HGEMM_ERR_TIMEOUT: return "a bounded device-side wait ran out";
    case HGEMM_ERR_SCRATCH_LIMIT: return "the call needs more scratch memory than the library's built-in buffer holds";
    case HGEMM_ERR_CHECK: return "the checked build found an invariant violated";
    }
    return "unknown status";
}

hgemm_status_t hgemm_create(hgemm_ctx_t **out, int device)
{
    if (!out || device < 0) return HGEMM_ERR_INVALID_ARG;
    int count = 0;
    cudaError_t e = cudaGetDeviceCount(&count);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    if (device >= count) return HGEMM_ERR_INVALID_ARG;
    cudaDeviceProp prop;
    e = cudaGetDeviceProperties(&prop, device);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);
    if (prop.major != 10 || prop.minor != 0) return HGEMM_ERR_ARCH;
    int prev = 0;
    cudaGetDevice(&prev);
    e = cudaSetDevice(device);
    if (e != cudaSuccess) return cuda_fail(nullptr, e);

    hgemm_ctx_s *ctx = new (std::nothrow) hgemm_ctx_s;
    if (!ctx) return HGEMM_ERR_ALLOC;
    ctx->device = device;
    ctx->num_sms = prop.multiProcessorCount;
    hgemm_status_t st = HGEMM_OK;
    do {
        void *fn = nullptr;
        cudaDriverEntryPointQueryResult qres;
        e = cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &fn, cudaEnableDefault, &qres);
        if (e != cudaSuccess || qres != cudaDriverEntryPointSuccess || !fn) {
            st = cuda_fail(ctx, e);
            break;
        }
        ctx->encode = reinterpret_cast<encode_tiled_fn>(fn);
        e = cudaMalloc(reinterpret_cast<void **>(&ctx->d_status), 2 * kStatusSlots * sizeof(uint32_t));   // status words, then the plans' pacing counters
        if (e != cudaSuccess) {
            cuda_fail(ctx, e);
            st = HGEMM_ERR_ALLOC;
            break;
        }
        e = cudaMemset(ctx->d_status, 0, 2 * kStatusSlots * sizeof(uint32_t));
        if (e != cudaSuccess) {
            st = cuda_fail(ctx, e);
            break;
        }
        ctx->free_status_slots.reserve(kStatusSlots);
        for (int slot = kStatusSlots - 1; slot >= 1; --slot) ctx->free_status_slots.push_back(slot);
        // every instantiation: 1-CTA / CTA-pair, narrow / wide store boxes, no K slices / workspace / cluster reduction
        for (int k = 0; k < 72 && e == cudaSuccess; ++k) {
            // k / 12: 0 full-featured, 1 instrumented, 2 and 3 plain with 64- and 128-wide stages; 4 and 5: transposed stores
            // (full-featured, then plain with either stage width)
            const bool xp = k >= 48;
            const void *fn_k = xp ? kernel_for(1 + (k & 1), false, (k >> 2) % 3, k >= 60, false, (k & 2) ? 2 : 1, true)
                                  : kernel_for(1 + (k & 1), (k & 2) != 0, (k >> 2) % 3, k / 12 >= 2, k / 12 == 1, k / 12 == 3 ? 2 : 1);
            e = cudaFuncSetAttribute(fn_k, cudaFuncAttributeMaxDynamicSharedMemorySize, int(hgemm_host::kSmemOptInBytes));
            if (e == cudaSuccess) e = cudaFuncSetAttribute(fn_k, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        }
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(hgemm_dev::hgemm_light_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(hgemm_host::kSmemOptInBytes));
        if (e == cudaSuccess)
            e = cudaFuncSetAttribute(hgemm_dev::hgemm_light_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, int(hgemm_host::kSmemOptInBytes));
        if (e == cudaSuccess) e = cudaFuncSetAttribute(hgemm_dev::hgemm_small_kernel<32>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        if (e == cudaSuccess) e = cudaFuncSetAttribute(hgemm_dev::hgemm_small_kernel<64>, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        for (int k = 0; k < 6 && e == cudaSuccess; ++k) {           // the stream-K instantiations
            const void *fn_k = kernel_for(1 + (k & 1), false, 3, k >= 2, false, k >= 4 ? 2 : 1);
            e = cudaFuncSetAttribute(fn_k, cudaFuncAttributeMaxDynamicSharedMemorySize, int(hgemm_host::kSmemOptInBytes));
            if (e == cudaSuccess) e = cudaFuncSetAttribute(fn_k, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        }
        for (int k = 0; k < 6 && e == cudaSuccess; ++k) {           // the double-accumulator instantiations
            const void *fn_k = kernel_for(2, (k & 1) != 0, 0, k >= 2, false, k >= 4 ? 2 : 1, false, true);
            e = cudaFuncSetAttribute(fn_k, cudaFuncAttributeMaxDynamicSharedMemorySize, int(hgemm_host::kSmemOptInBytes));
            if (e == cudaSuccess) e = cudaFuncSetAttribute(fn_k, cudaFuncAttributeNonPortableClusterSizeAllowed, 1);
        }
        if (e != cudaSuccess) {
            st = cuda_fail(ctx, e);
            break;
        }
    } while (false);
    cudaSetDevice(prev);
    if (st != HGEMM_OK) {
        if (ctx->d_status) cudaFree(ctx->d_status);
        delete ctx;
        return st;
    }
    *out = ctx;
    return HGEMM_OK;
}

hgemm_status_t hgemm_plan_destroy(hgemm_plan_t *plan)
{
    if (!plan) return HGEMM_ERR_INVALID_ARG;
    hgemm_ctx_s *ctx = plan->ctx;
    if (ctx) {
        auto it = std::find(ctx->plans.begin(), ctx->plans.end(), plan);
        if (it != ctx->plans.end()) ctx->plans.erase(it);
        if (plan->status_slot > 0) ctx->free_status_slots.push_back(plan->status_slot);
    }
    if (plan->workspace) cudaFree(plan->workspace);
    if (plan->counters) cudaFree(plan->counters);
    if (plan->pad_a) cudaFree(plan->pad_a);
    if (plan->pad_b) cudaFree(plan->pad_b);
    if (plan->stage_a) cudaFree(plan->stage_a);
    if (plan->stage_b) cudaFree(plan->stage_b);
    if (plan->stage_c) cudaFree(plan->stage_c);
    if (plan->ev_in) cudaEventDestroy(plan->ev_in);
    if (plan->ev_gemm) cudaEventDestroy(plan->ev_gemm);
    if (plan->ev_out) cudaEventDestroy(plan->ev_out);
    delete plan;
    return HGEMM_OK;
}

hgemm_status_t hgemm_destroy(hgemm_ctx_t *ctx)
{
    if (!ctx) return HGEMM_ERR_INVALID_ARG;
    while (!ctx->plans.empty()) hgemm_plan_destroy(ctx->plans.back());
    if (ctx->d_status) cudaFree(ctx->d_status);
    if (ctx->copy_in) cudaStreamDestroy(ctx->copy_in);
    if (ctx->copy_out) cudaStreamDestroy(ctx->copy_out);
    delete ctx;
    return HGEMM_OK;
}

hgemm_status_t hgemm_planned_config(int64_t M, int64_t N, int64_t K, int32_t num_sms, hgemm_config_t *out)
{
    if (!out) return HGEMM_ERR_INVALID_ARG;
    hgemm_status_t s = hgemm_host::validate_shape(M, N, K);
    if (s != HGEMM_OK) return s;
    hgemm_config_t c;
    s = hgemm_host::plan_config(M, N, hgemm_host::padded_k(K), num_sms, &c);
    if (s == HGEMM_OK) *out = c;
    return s;
}

hgemm_status_t hgemm_heuristic_config(int64_t M, int64_t N, int64_t K, int32_t num_sms, hgemm_config_t *out)
{
    if (!out) return HGEMM_ERR_INVALID_ARG;
    hgemm_config_t c;
    const hgemm_status_t s = hgemm_host::heuristic(M, N, K, num_sms, &c);
    if (s == HGEMM_OK) *out = c;
    return s;
}

hgemm_status_t hgemm_validate_config(int64_t M, int64_t N, int64_t K, const hgemm_config_t *cfg)
{
    if (!cfg) return HGEMM_ERR_INVALID_ARG;
    return hgemm_host::validate(M, N, K, *cfg);
}

double hgemm_estimate_config(int64_t M, int64_t N, int64_t K, int32_t num_sms, const hgemm_config_t *cfg)
{
    if (!cfg || hgemm_host::validate(M, N, K, *cfg) != HGEMM_OK) return -1.0;
    return hgemm_host::estimate_cycles(M, N, K, num_sms, *cfg);
}

int64_t hgemm_config_smem_bytes(const hgemm_config_t *cfg)
{
    return cfg ? hgemm_host::smem_bytes(*cfg) : -1;
}

int64_t hgemm_config_workspace_bytes(int64_t M, int64_t N, int64_t K, const hgemm_config_t *cfg)
{
    return cfg ? hgemm_host::workspace_bytes(M, N, K, *cfg) + hgemm_host::counter_bytes(M, N, *cfg, 148, K) : -1;
}

hgemm_status_t hgemm_plan(hgemm_ctx_t *ctx, int64_t M, int64_t N, int64_t K, hgemm_plan_t **out)
{
    return hgemm_plan_layout(ctx, M, N, K, HGEMM_LAYOUT_TN, out);
}

hgemm_status_t hgemm_plan_layout(hgemm_ctx_t *ctx, int64_t M, int64_t N, int64_t K, hgemm_layout_t layout, hgemm_plan_t **out)
{
    if (!ctx || !out) return HGEMM_ERR_INVALID_ARG;
    if (layout != HGEMM_LAYOUT_TN && layout != HGEMM_LAYOUT_NN) return HGEMM_ERR_INVALID_ARG;
    hgemm_status_t s = layout == HGEMM_LAYOUT_NN ? hgemm_host::validate_shape_aligned(M, N, K) : hgemm_host::validate_shape(M, N, K);
    if (s != HGEMM_OK) return s;
    const int64_t Kp = hgemm_host::padded_k(K);
    hgemm_config_t cfg;
    s = hgemm_host::plan_config(M, N, Kp, ctx->num_sms, &cfg);   // the table, else the neighbours' configurations re-fitted
    if (s != HGEMM_OK) return s;
    if (layout == HGEMM_LAYOUT_NN &&
        (cfg.swap_ab || cfg.block_n == 512 || cfg.family == HGEMM_FAMILY_LIGHT || cfg.family == HGEMM_FAMILY_SMALL)) {
        // forms that exist only for K-contiguous operands: plan a row-major B from the cost model's own choice instead
        s = hgemm_host::heuristic(M, N, Kp, ctx->num_sms, &cfg);
        if (s != HGEMM_OK) return s;
    }
    if (layout == HGEMM_LAYOUT_NN) {
        // row-major B is staged in blocks of 64 columns: widen the tile to the next legal width and
        // give back stages until it fits
        const int unit = 64 * hgemm_host::cta_group_of(cfg);
        cfg.block_n = std::min(256, (cfg.block_n + unit - 1) / unit * unit);
        cfg.stages = std::min(cfg.stages, hgemm_host::max_stages_of(cfg));       // with this epilogue's store staging
        if (cfg.stages < 1) {
            cfg.block_k = 64;
            cfg.stages = std::min(4, hgemm_host::max_stages_of(cfg));
        }
        if (cfg.stages < 1) {                                                     // the wide epilogue's staging is what does not fit
            cfg.epilogue = HGEMM_EPILOGUE_TMA;
            cfg.stages = std::min(4, hgemm_host::max_stages_of(cfg));
        }
        if (cfg.tail_mode == HGEMM_TAIL_N && cfg.tail_split >= 2 && ((cfg.block_n / cfg.tail_split) % unit) != 0) {
            cfg.tail_split = 0;
            cfg.tail_mode = HGEMM_TAIL_K;
        }
        if (cfg.split_k > 1 && cfg.split_mode == HGEMM_SPLIT_CLUSTER && hgemm_host::validate(M, N, Kp, cfg) != HGEMM_OK)
            cfg.split_mode = HGEMM_SPLIT_WORKSPACE;   // the wider tile's partial sums no longer fit in shared memory
        if (hgemm_host::validate(M, N, Kp, cfg) != HGEMM_OK) return HGEMM_ERR_UNSUPPORTED;
    }
    if (ctx->free_status_slots.empty()) return HGEMM_ERR_ALLOC;   // more live plans than status words
    hgemm_plan_s *pl = new (std::nothrow) hgemm_plan_s;
    if (!pl) return HGEMM_ERR_ALLOC;
    pl->layout = layout;
    pl->ctx = ctx;
    pl->status_slot = ctx->free_status_slots.back();             // taken for good only when the plan is handed out
    pl->M = M;
    pl->N = N;
    pl->K = Kp;
    pl->K_user = K;
    if (Kp != K) {
        // rows of A and B are not multiples of 16 bytes: the kernels read zero-padded copies instead
        cudaError_t e = ctx_malloc(ctx, &pl->pad_a, size_t(M) * size_t(Kp) * 2);
        if (e == cudaSuccess) e = ctx_malloc(ctx, &pl->pad_b, size_t(N) * size_t(Kp) * 2);
        if (e != cudaSuccess) {
            if (pl->pad_a) cudaFree(pl->pad_a);
            cuda_fail(ctx, e);
            delete pl;
            return HGEMM_ERR_ALLOC;
        }
    }
    s = apply_config(pl, cfg);
    if (s != HGEMM_OK) {
        if (pl->workspace) cudaFree(pl->workspace);
        if (pl->counters) cudaFree(pl->counters);
        if (pl->pad_a) cudaFree(pl->pad_a);
        if (pl->pad_b) cudaFree(pl->pad_b);
        delete pl;
        return s;
    }
    ctx->free_status_slots.pop_back();
    ctx->plans.push_back(pl);
    *out = pl;
    return HGEMM_OK;
}

hgemm_status_t hgemm_plan_get_config(const hgemm_plan_t *plan, hgemm_config_t *out)
{
    if (!plan || !out) return HGEMM_ERR_INVALID_ARG;
    *out = plan->cfg;
    return HGEMM_OK;
}

hgemm_status_t hgemm_plan_set_config(hgemm_plan_t *plan, const hgemm_config_t *cfg)
{
    if (!plan || !cfg) return HGEMM_ERR_INVALID_ARG;
    const hgemm_status_t s = hgemm_host::validate(plan->M, plan->N, plan->K, *cfg);
    if (s != HGEMM_OK) return s;
    cudaError_t e = cudaDeviceSynchronize();   // the old workspace may still be in use
    if (e != cudaSuccess) return cuda_fail(plan->ctx, e);
    return apply_config(plan, *cfg);
}

int32_t hgemm_candidate_configs(int64_t M, int64_t N, int64_t K, int32_t num_sms, hgemm_config_t *out, int32_t max)
{
    if (!out || max < 1) return 0;
    if (hgemm_host::validate_shape(M, N, K) != HGEMM_OK) return 0;
    return hgemm_host::ranked_candidates(M, N, hgemm_host::padded_k(K), num_sms, out, max);
}

hgemm_status_t hgemm_plan_autotune(hgemm_plan_t *plan, const void *A, const void *B, void *C, void *stream, int32_t max_candidates,
                                   float *best_us)
{
    if (!plan || !A || !B || !C || max_candidates < 1) return HGEMM_ERR_INVALID_ARG;
    hgemm_ctx_s *ctx = plan->ctx;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const hgemm_config_t start = plan->cfg;
    std::vector<hgemm_config_t> cands(size_t(std::min<int32_t>(max_candidates, 256)) + 1);
    cands[0] = start;                                            // the planner's own choice is always timed
    const int32_t n = 1 + hgemm_host::ranked_candidates(plan->M, plan->N, plan->K, ctx->num_sms, cands.data() + 1,
                                                        int32_t(cands.size()) - 1);
    cudaEvent_t e0 = nullptr, e1 = nullptr;
    cudaError_t e = cudaEventCreate(&e0);
    if (e == cudaSuccess) e = cudaEventCreate(&e1);
    if (e != cudaSuccess) {
        if (e0) cudaEventDestroy(e0);
        return cuda_fail(ctx, e);
    }
    hgemm_status_t result = HGEMM_OK;
    hgemm_config_t best = start;
    float best_ms = -1.0f;
    for (int32_t i = 0; i < n && result == HGEMM_OK; ++i) {
        if (i > 0 && std::memcmp(&cands[size_t(i)], &start, sizeof(start)) == 0) continue;
        if (hgemm_plan_set_config(plan, &cands[size_t(i)]) != HGEMM_OK) continue;      // e.g. a layout's extra rules
        // two untimed calls, then enough back-to-back calls to fill about a quarter of a millisecond
        hgemm_status_t s = hgemm_run(plan, A, B, C, stream);
        if (s == HGEMM_OK) s = hgemm_run(plan, A, B, C, stream);
        float probe_ms = 0.0f;
        if (s == HGEMM_OK) {
            cudaEventRecord(e0, st);
            s = hgemm_run(plan, A, B, C, stream);
            cudaEventRecord(e1, st);
            e = cudaEventSynchronize(e1);
            if (e == cudaSuccess) e = cudaEventElapsedTime(&probe_ms, e0, e1);
            if (e != cudaSuccess) result = cuda_fail(ctx, e);
        }
        if (s != HGEMM_OK || result != HGEMM_OK) continue;
        const int reps = std::max(3, std::min(64, int(0.25f / std::max(probe_ms, 1e-3f))));
        cudaEventRecord(e0, st);
        for (int r = 0; r < reps && s == HGEMM_OK; ++r) s = hgemm_run(plan, A, B, C, stream);
        cudaEventRecord(e1, st);
        float ms = 0.0f;
        e = cudaEventSynchronize(e1);
        if (e == cudaSuccess) e = cudaEventElapsedTime(&ms, e0, e1);
        if (e != cudaSuccess) {
            result = cuda_fail(ctx, e);
            break;
        }
        if (s != HGEMM_OK) continue;
        ms /= float(reps);
        if (best_ms < 0.0f || ms < best_ms) {
            best_ms = ms;
            best = cands[size_t(i)];
        }
    }
    cudaEventDestroy(e0);
    cudaEventDestroy(e1);
    // a wait that ran out during the search disqualifies the search, not the plan: back to where it started
    uint32_t code = 0;
    if (result == HGEMM_OK && hgemm_last_device_status(plan, &code) != HGEMM_OK) {
        const hgemm_status_t back = hgemm_plan_set_config(plan, &start);
        return back != HGEMM_OK ? back : HGEMM_ERR_TIMEOUT;
    }
    hgemm_status_t s = hgemm_plan_set_config(plan, result == HGEMM_OK ? &best : &start);
    if (s != HGEMM_OK && result == HGEMM_OK) s = hgemm_plan_set_config(plan, &start);   // the plan never shrinks its buffers: this fits
    if (result != HGEMM_OK) return result;
    if (s != HGEMM_OK) return s;
    if (best_us) *best_us = best_ms * 1e3f;
    return hgemm_run(plan, A, B, C, stream);                     // C holds the product computed by the installed configuration
}

int32_t hgemm_plan_launches_per_run(const hgemm_plan_t *plan)
{
    return plan ? 1 : 0;
}

static hgemm_status_t run_impl(hgemm_plan_t *plan, float alpha, float beta, bool scaled, const void *A, const void *B, void *C,
                               void *stream);

hgemm_status_t hgemm_run(hgemm_plan_t *plan, const void *A, const void *B, void *C, void *stream)
{
    return run_impl(plan, 1.0f, 0.0f, false, A, B, C, stream);
}

hgemm_status_t hgemm_run_scaled(hgemm_plan_t *plan, float alpha, float beta, const void *A, const void *B, void *C, void *stream)
{
    if (!(alpha == alpha) || !(beta == beta)) return HGEMM_ERR_INVALID_ARG;   // NaN factors
    return run_impl(plan, alpha, beta, true, A, B, C, stream);
}

static hgemm_status_t run_impl(hgemm_plan_t *plan, float alpha, float beta, bool scaled, const void *A, const void *B, void *C,
                               void *stream)
{
    if (!plan || !A || !B || !C) return HGEMM_ERR_INVALID_ARG;
    if ((reinterpret_cast<uintptr_t>(A) | reinterpret_cast<uintptr_t>(B) | reinterpret_cast<uintptr_t>(C)) & 15u)
        return HGEMM_ERR_INVALID_ARG;
    hgemm_ctx_s *ctx = plan->ctx;
    const hgemm_config_t &cfg = plan->cfg;
    const int cg = hgemm_host::cta_group_of(cfg);

    if (plan->pad_a) {
        // K is not a multiple of 8: copy A and B into the plan's zero-padded buffers first (same stream)
        cudaStream_t st = static_cast<cudaStream_t>(stream);
        const int64_t ga = (plan->M * (plan->K / 8) + 255) / 256, gb = (plan->N * (plan->K / 8) + 255) / 256;
        hgemm_dev::hgemm_pad_k_kernel<<<unsigned(std::min<int64_t>(ga, 65535)), 256, 0, st>>>(
            static_cast<const __half *>(A), static_cast<__half *>(plan->pad_a), plan->M, plan->K_user, plan->K);
        hgemm_dev::hgemm_pad_k_kernel<<<unsigned(std::min<int64_t>(gb, 65535)), 256, 0, st>>>(
            static_cast<const __half *>(B), static_cast<__half *>(plan->pad_b), plan->N, plan->K_user, plan->K);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        A = plan->pad_a;
        B = plan->pad_b;
    }

    if (cfg.family == HGEMM_FAMILY_SMALL) {
        // the register-accumulator kernel: plain pointers, no tensor maps, no cluster
        if (plan->trace != nullptr || plan->debug_skip != 0) return HGEMM_ERR_UNSUPPORTED;       // it has no instrumentation
        hgemm_dev::SmallParams sp;
        sp.A = static_cast<const __half *>(A);
        sp.B = static_cast<const __half *>(B);
        sp.C = static_cast<__half *>(C);
        sp.M = int32_t(plan->M);
        sp.N = int32_t(plan->N);
        sp.K = int32_t(plan->K);
        sp.tiles_m = plan->params.tiles_m;
        sp.scaled = scaled ? 1u : 0u;
        sp.alpha = alpha;
        sp.beta = beta;
        sp.split_k = plan->cluster_dim;
        sp.status = ctx->d_status + plan->status_slot;
        cudaLaunchConfig_t lc;
        std::memset(&lc, 0, sizeof(lc));
        lc.gridDim = dim3(unsigned(plan->grid), 1, 1);
        lc.blockDim = dim3(hgemm_dev::kSmallThreads, 1, 1);
        lc.stream = static_cast<cudaStream_t>(stream);
        cudaLaunchAttribute attr[2];
        int na = 0;
        if (plan->cluster_dim > 1) {                     // the K slices of a tile are one cluster
            attr[na].id = cudaLaunchAttributeClusterDimension;
            attr[na].val.clusterDim.x = unsigned(plan->cluster_dim);
            attr[na].val.clusterDim.y = 1;
            attr[na].val.clusterDim.z = 1;
            ++na;
        }
        if (ctx->dependent_launch) {
            attr[na].id = cudaLaunchAttributeProgrammaticStreamSerialization;
            attr[na].val.programmaticStreamSerializationAllowed = 1;
            ++na;
        }
        lc.attrs = attr;
        lc.numAttrs = unsigned(na);
        void *sargs[1] = {&sp};
        cudaError_t e = cudaLaunchKernelExC(&lc, cfg.block_n == 32 ? reinterpret_cast<const void *>(hgemm_dev::hgemm_small_kernel<32>)
                                                                   : reinterpret_cast<const void *>(hgemm_dev::hgemm_small_kernel<64>), sargs);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        return HGEMM_OK;
    }

    if (cfg.swap_ab) std::swap(A, B);       // the kernel's A operand (its 128-row side) is the caller's B

    hgemm_plan_s::MapEntry *me = nullptr;
    for (int i = 0; i < plan->maps_used; ++i) {
        hgemm_plan_s::MapEntry &e = plan->maps[i];
        if (e.a == A && e.b == B && e.c == C) {
            me = &e;
            break;
        }
    }
    if (!me) {
        hgemm_plan_s::MapEntry &e = plan->maps[plan->maps_next];
        e.a = e.b = nullptr;
        e.c = nullptr;
        const uint64_t M = uint64_t(plan->params.M), N = uint64_t(plan->params.N), K = uint64_t(plan->K);   // as the kernel sees them
        if (plan->params.tma_3d) {
            if (!encode_3d_ksub(ctx, &e.tmap_a, A, K, M, 128)) return HGEMM_ERR_CUDA;
            if (!encode_3d_ksub(ctx, &e.tmap_b, B, K, N, uint32_t(cfg.block_n / cg))) return HGEMM_ERR_CUDA;
        } else if (plan->layout == HGEMM_LAYOUT_NN) {
            if (!encode_2d(ctx, &e.tmap_a, A, K, M, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B)) return HGEMM_ERR_CUDA;
            // B is K rows of N: boxes of 64 columns x 64 k-rows
            if (!encode_2d(ctx, &e.tmap_b, B, N, K, 64, 64, CU_TENSOR_MAP_SWIZZLE_128B)) return HGEMM_ERR_CUDA;
        } else {
            if (!encode_2d(ctx, &e.tmap_a, A, K, M, 64, 128, CU_TENSOR_MAP_SWIZZLE_128B)) return HGEMM_ERR_CUDA;
            if (!encode_2d(ctx, &e.tmap_b, B, K, N, 64, uint32_t(cfg.block_n / cg), CU_TENSOR_MAP_SWIZZLE_128B))
                return HGEMM_ERR_CUDA;
        }
        e.tmap_bt = e.tmap_b;      // unused unless tail tiles are cut into column pieces
        if (plan->params.tail_pieces > 1 && plan->layout != HGEMM_LAYOUT_NN &&
            !encode_2d(ctx, &e.tmap_bt, B, K, N, 64, uint32_t(cfg.block_n / plan->params.tail_pieces / cg), CU_TENSOR_MAP_SWIZZLE_128B))
            return HGEMM_ERR_CUDA;
        if (plan->params.ragged_n) {
            e.tmap_c = e.tmap_a;   // never used: a C with ragged rows is stored element by element
        } else if (plan->params.epilogue_tma == 2) {
            // wide epilogue: 32-row x 64-column store boxes (128-byte rows)
            if (!encode_2d(ctx, &e.tmap_c, C, N, M, 64, 32, CU_TENSOR_MAP_SWIZZLE_128B)) return HGEMM_ERR_CUDA;
        } else if (plan->params.transposed) {
            // the caller's C: rows of the kernel's M elements, the kernel's N of them; boxes are stored transposed
            if (!encode_2d(ctx, &e.tmap_c, C, M, N, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B)) return HGEMM_ERR_CUDA;
        } else if (!encode_2d(ctx, &e.tmap_c, C, N, M, 32, 32, CU_TENSOR_MAP_SWIZZLE_64B)) {
            return HGEMM_ERR_CUDA;
        }
        e.a = A;
        e.b = B;
        e.c = C;
        me = &e;
        plan->maps_next = (plan->maps_next + 1) % hgemm_plan_s::kMapCache;
        plan->maps_used = std::min(plan->maps_used + 1, int(hgemm_plan_s::kMapCache));
    }
    plan->params.C = static_cast<__half *>(C);
    plan->params.wait_budget = ctx->wait_budget;
    plan->params.trace = plan->trace;
    plan->params.debug_skip = plan->debug_skip;
    // a static operand in the caller's terms is the kernel's other operand when the configuration swaps them
    plan->params.early_ops = cfg.swap_ab ? (((plan->static_operands & 1u) << 1) | ((plan->static_operands >> 1) & 1u)) : plan->static_operands;
    if (plan->pad_a) plan->params.early_ops = 0u;     // the kernel reads padded copies that this very call has just written
    plan->params.scaled = scaled ? 1u : 0u;
    plan->params.alpha = alpha;
    plan->params.beta = beta;
    if (plan->counters) plan->params.epoch = ++plan->epoch;   // the arrival counters count on from launch to launch
    if (plan->params.wave_pace) {
        // wave pacing: this launch's arrivals count on from where the plan's earlier launches left the counter
        plan->params.wave_base = plan->wave_total;
        plan->wave_total += uint32_t(plan->params.wave_rounds) * uint32_t(plan->grid / cg);
    }

    cudaLaunchConfig_t lc;
    std::memset(&lc, 0, sizeof(lc));
    lc.gridDim = dim3(unsigned(plan->grid), 1, 1);
    lc.blockDim = dim3(hgemm_dev::kThreads, 1, 1);
    lc.dynamicSmemBytes = size_t(plan->smem);
    lc.stream = static_cast<cudaStream_t>(stream);
    cudaLaunchAttribute attr[2];
    attr[0].id = cudaLaunchAttributeClusterDimension;
    attr[0].val.clusterDim.x = unsigned(plan->cluster_dim);
    attr[0].val.clusterDim.y = 1;
    attr[0].val.clusterDim.z = 1;
    // programmatic stream serialisation: this launch may become resident before the kernel ahead of
    // it in the stream has finished; the kernel itself waits for that kernel before it touches memory
    attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[1].val.programmaticStreamSerializationAllowed = 1;
    lc.attrs = attr;
    lc.numAttrs = ctx->dependent_launch ? 2 : 1;
    cudaError_t e;
    // The wide instantiation lays its store staging out differently, so it runs whenever the configuration asks for
    // it, also when a C with ragged rows makes it fall back to element stores; the instantiation without the
    // split-K reductions runs whenever no work item is a K slice.
    const KernelParams &kp = plan->params;
    const bool trace = kp.trace != nullptr || kp.debug_skip != 0;
    const bool plain = !kp.scaled && !kp.acc_f16 && !kp.ragged_n && !kp.b_row_major && kp.tail_pieces <= 1;
    const bool light = plan->cfg.family == HGEMM_FAMILY_LIGHT;
    if (trace && (kp.transposed || kp.block_n == 512)) return HGEMM_ERR_UNSUPPORTED;   // no instrumented kernels for these
    if (light && kp.debug_skip != 0) return HGEMM_ERR_UNSUPPORTED;                       // the light kernel has stamps, no skip mask
    if (trace && kp.stream_units > 0) return HGEMM_ERR_UNSUPPORTED;                      // ... nor for the stream-K tail
    const void *fn = kernel_for(cg, plan->cfg.epilogue == HGEMM_EPILOGUE_TMA_WIDE, kp.stream_units > 0 ? 3 : kp.split_k > 1 ? (kp.cluster_split ? 2 : 1) : 0, plain,
                                trace, kp.block_k / 64, kp.transposed != 0, kp.block_n == 512);
    void *args[5] = {&me->tmap_a, &me->tmap_b, &me->tmap_c, &me->tmap_bt, &plan->params};
    if (light) {
        void *largs[4] = {&me->tmap_a, &me->tmap_b, &me->tmap_c, &plan->params};
        lc.blockDim = dim3(hgemm_dev::kLightThreads, 1, 1);
        lc.attrs = attr + 1;                         // no cluster attribute: a plain grid, with or without the dependent-launch one
        lc.numAttrs = ctx->dependent_launch ? 1 : 0;
        e = cudaLaunchKernelExC(&lc, kp.trace != nullptr ? reinterpret_cast<const void *>(hgemm_dev::hgemm_light_kernel<true>)
                                                         : reinterpret_cast<const void *>(hgemm_dev::hgemm_light_kernel<false>), largs);
    } else {
        e = cudaLaunchKernelExC(&lc, fn, args);
    }
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return HGEMM_OK;
}

hgemm_status_t hgemm_run_host(hgemm_plan_t *plan, const void *A_host, const void *B_host, void *C_host, void *stream)
{
    if (!plan || !A_host || !B_host || !C_host) return HGEMM_ERR_INVALID_ARG;
    hgemm_ctx_s *ctx = plan->ctx;
    const size_t a_bytes = size_t(plan->M) * size_t(plan->K_user) * 2, b_bytes = size_t(plan->N) * size_t(plan->K_user) * 2,
                 c_bytes = size_t(plan->M) * size_t(plan->N) * 2;
    cudaError_t e = cudaSuccess;
    if (!ctx->copy_in) {
        e = cudaStreamCreateWithFlags(&ctx->copy_in, cudaStreamNonBlocking);
        if (e == cudaSuccess) e = cudaStreamCreateWithFlags(&ctx->copy_out, cudaStreamNonBlocking);
        if (e != cudaSuccess) {
            if (ctx->copy_in) cudaStreamDestroy(ctx->copy_in);
            ctx->copy_in = ctx->copy_out = nullptr;
            return cuda_fail(ctx, e);
        }
    }
    if (!plan->stage_a) {
        e = ctx_malloc(ctx, &plan->stage_a, a_bytes);
        if (e == cudaSuccess) e = ctx_malloc(ctx, &plan->stage_b, b_bytes);
        if (e == cudaSuccess) e = ctx_malloc(ctx, &plan->stage_c, c_bytes);
        if (e != cudaSuccess) {
            if (plan->stage_a) cudaFree(plan->stage_a);
            if (plan->stage_b) cudaFree(plan->stage_b);
            plan->stage_a = plan->stage_b = plan->stage_c = nullptr;
            cuda_fail(ctx, e);
            return HGEMM_ERR_ALLOC;
        }
    }
    if (!plan->ev_in) {
        e = cudaEventCreateWithFlags(&plan->ev_in, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&plan->ev_gemm, cudaEventDisableTiming);
        if (e == cudaSuccess) e = cudaEventCreateWithFlags(&plan->ev_out, cudaEventDisableTiming);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
    }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    // operands: host -> staging on the inbound copy stream, as soon as the staging is free (the plan's previous product has
    // been computed from it); they do not queue behind the caller's stream
    if (plan->host_call_in_flight) {
        e = cudaStreamWaitEvent(ctx->copy_in, plan->ev_gemm, 0);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
    }
    e = cudaMemcpyAsync(plan->stage_a, A_host, a_bytes, cudaMemcpyHostToDevice, ctx->copy_in);
    if (e == cudaSuccess) e = cudaMemcpyAsync(plan->stage_b, B_host, b_bytes, cudaMemcpyHostToDevice, ctx->copy_in);
    if (e == cudaSuccess) e = cudaEventRecord(plan->ev_in, ctx->copy_in);
    // the product: on the caller's stream, once the operands are there and the staging of C is free (the plan's previous
    // result has left it)
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st, plan->ev_in, 0);
    if (e == cudaSuccess && plan->host_call_in_flight) e = cudaStreamWaitEvent(st, plan->ev_out, 0);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    const hgemm_status_t s = hgemm_run(plan, plan->stage_a, plan->stage_b, plan->stage_c, stream);
    if (s != HGEMM_OK) return s;
    e = cudaEventRecord(plan->ev_gemm, st);
    // the result: staging -> host on the outbound copy stream; the caller's stream then waits for it, so whatever the caller
    // enqueues next -- and a synchronisation of the stream -- comes after C_host is complete
    if (e == cudaSuccess) e = cudaStreamWaitEvent(ctx->copy_out, plan->ev_gemm, 0);
    if (e == cudaSuccess) e = cudaMemcpyAsync(C_host, plan->stage_c, c_bytes, cudaMemcpyDeviceToHost, ctx->copy_out);
    if (e == cudaSuccess) e = cudaEventRecord(plan->ev_out, ctx->copy_out);
    if (e == cudaSuccess) e = cudaStreamWaitEvent(st, plan->ev_out, 0);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    plan->host_call_in_flight = true;
    return HGEMM_OK;
}

hgemm_status_t hgemm_plan_set_static_operands(hgemm_plan_t *plan, uint32_t which)
{
    if (!plan || which > 3u) return HGEMM_ERR_INVALID_ARG;
    plan->static_operands = which;
    return HGEMM_OK;
}

hgemm_status_t hgemm_debug_set_trace(hgemm_plan_t *plan, void *device_buf)
{
    if (!plan) return HGEMM_ERR_INVALID_ARG;
    plan->trace = static_cast<unsigned long long *>(device_buf);
    return HGEMM_OK;
}

hgemm_status_t hgemm_debug_set_skip(hgemm_plan_t *plan, uint32_t mask)
{
    if (!plan || mask > 15u) return HGEMM_ERR_INVALID_ARG;
    plan->debug_skip = mask;
    return HGEMM_OK;
}

// A launch that gave up may have left the plan's split-K arrival counters part-way: start them again from zero.
static hgemm_status_t reset_counters(hgemm_plan_s *pl)
{
    if (!pl->counters) return HGEMM_OK;
    cudaError_t e = cudaMemset(pl->counters, 0, size_t(pl->counter_bytes));
    if (e != cudaSuccess) return cuda_fail(pl->ctx, e);
    pl->epoch = 0;
    return HGEMM_OK;
}

hgemm_status_t hgemm_last_device_status(hgemm_plan_t *plan, uint32_t *code)
{
    if (!plan || !code) return HGEMM_ERR_INVALID_ARG;
    hgemm_ctx_s *ctx = plan->ctx;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    uint32_t v = 0;
    uint32_t *word = ctx->d_status + plan->status_slot;
    e = cudaMemcpy(&v, word, 4, cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    if (v != 0) {
        e = cudaMemset(word, 0, 4);
        if (e != cudaSuccess) return cuda_fail(ctx, e);
        const hgemm_status_t s = reset_counters(plan);
        if (s != HGEMM_OK) return s;
    }
    *code = v;
    return v == 0 ? HGEMM_OK : (v >> 24) == hgemm_dev::kRoleCheck ? HGEMM_ERR_CHECK : HGEMM_ERR_TIMEOUT;
}

hgemm_status_t hgemm_ctx_last_device_status(hgemm_ctx_t *ctx, uint32_t *code)
{
    if (!ctx || !code) return HGEMM_ERR_INVALID_ARG;
    cudaError_t e = cudaDeviceSynchronize();
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    std::vector<uint32_t> words(size_t(kStatusSlots), 0u);
    e = cudaMemcpy(words.data(), ctx->d_status, words.size() * sizeof(uint32_t), cudaMemcpyDeviceToHost);
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    uint32_t v = words[0];                                   // the context's own word first, then the plans' in creation order
    bool any = v != 0;
    for (hgemm_plan_s *pl : ctx->plans) {
        const uint32_t w = words[size_t(pl->status_slot)];
        if (w == 0) continue;
        any = true;
        if (v == 0) v = w;
        const hgemm_status_t s = reset_counters(pl);
        if (s != HGEMM_OK) return s;
    }
    if (any) {
        e = cudaMemset(ctx->d_status, 0, words.size() * sizeof(uint32_t));
        if (e != cudaSuccess) return cuda_fail(ctx, e);
    }
    *code = v;
    return v == 0 ? HGEMM_OK : (v >> 24) == hgemm_dev::kRoleCheck ? HGEMM_ERR_CHECK : HGEMM_ERR_TIMEOUT;
}

hgemm_status_t hgemm_debug_fail_allocs(hgemm_ctx_t *ctx, int32_t after, int32_t count)
{
    if (!ctx || after < 0 || count < 0) return HGEMM_ERR_INVALID_ARG;
    ctx->pass_allocs = after;
    ctx->fail_allocs = count;
    return HGEMM_OK;
}

hgemm_status_t hgemm_set_wait_budget(hgemm_ctx_t *ctx, int64_t cycles)
{
    if (!ctx || cycles < 1) return HGEMM_ERR_INVALID_ARG;
    ctx->wait_budget = cycles;
    return HGEMM_OK;
}

hgemm_status_t hgemm_debug_stream_item(int64_t M, int64_t N, int64_t K, const hgemm_config_t *cfg, int32_t num_sms,
                                       int32_t position, int32_t h, int32_t out[6])
{
    if (!cfg || !out || position < 0 || (h != 0 && h != 1)) return HGEMM_ERR_INVALID_ARG;
    if (hgemm_host::validate(M, N, K, *cfg) != HGEMM_OK) return HGEMM_ERR_UNSUPPORTED;
    const hgemm_host::SplitLayout L = hgemm_host::split_layout(M, N, K, num_sms, *cfg);
    if (L.stream_units <= 0) return HGEMM_ERR_UNSUPPORTED;
    const int32_t kb = int32_t((K + cfg->block_k - 1) / cfg->block_k);
    const int32_t q = int32_t((L.tiles - L.first_split_tile) * kb);
    const hgemm_dev::StreamItem si = hgemm_dev::stream_item(position, h, int32_t(L.stream_units), q, kb, hgemm_dev::make_fast_div(uint32_t(L.stream_units)),
                                                            hgemm_dev::make_fast_div(uint32_t(q)), hgemm_dev::make_fast_div(uint32_t(kb)));
    out[0] = int32_t(L.first_split_tile) + si.tile_rel;
    out[1] = si.kb_begin;
    out[2] = si.kb_count;
    out[3] = si.slice;
    out[4] = si.slices;
    out[5] = int32_t(L.stream_units);
    return HGEMM_OK;
}

hgemm_status_t hgemm_set_dependent_launch(hgemm_ctx_t *ctx, int32_t enabled)
{
    if (!ctx) return HGEMM_ERR_INVALID_ARG;
    ctx->dependent_launch = enabled != 0;
    return HGEMM_OK;
}

hgemm_status_t hgemm_debug_timeout_probe(hgemm_ctx_t *ctx, void *stream)
{
    if (!ctx) return HGEMM_ERR_INVALID_ARG;
    hgemm_dev::hgemm_timeout_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(ctx->d_status, ctx->wait_budget);   // slot 0
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return HGEMM_OK;
}

int32_t hgemm_build_is_checked(void)
{
    return HGEMM_CHECKED;
}

hgemm_status_t hgemm_debug_check_probe(hgemm_ctx_t *ctx, void *stream)
{
    if (!ctx) return HGEMM_ERR_INVALID_ARG;
    hgemm_dev::hgemm_check_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(ctx->d_status);   // slot 0
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return cuda_fail(ctx, e);
    return HGEMM_OK;
}

int32_t hgemm_last_cuda_error(const hgemm_ctx_t *ctx)
{
    return ctx ? ctx->last_cuda_error : 0;
}

} // extern "C"
