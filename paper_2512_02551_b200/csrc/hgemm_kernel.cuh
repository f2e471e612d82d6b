// The persistent, warp-specialised tcgen05 HGEMM kernel (all kernel families are
// instances of this one template).
//
// Structure per CTA (192 threads):
//   warp 0      TMA producer: fills a ring of shared-memory stages with 64-wide
//               k-blocks of A (128 rows) and B (block_n rows, or block_n/2 in a pair)
//   warp 1      allocates tensor memory; one thread issues tcgen05.mma into one of two
//               fp32 accumulators (double-buffered so the epilogue of tile t overlaps
//               the main loop of tile t+1)
//   warps 2..5  epilogue: tensor memory -> registers -> fp16 -> global (direct 16-byte
//               stores, or swizzled shared memory + TMA store); with split-K the fp32
//               partial goes to a workspace and the last slice to finish sums all
//               slices of its tile in slice order.
// This is the tiled structure of the paper's section 2.1 (global -> shared -> tensor
// core main loop over K, then an epilogue) mapped onto Blackwell: TMA in place of
// cp.async, tensor memory in place of register accumulators, a persistent tile loop in
// place of one CTA per tile.  The tile order follows the paper's "block swizzle"
// (section 5.2): m-tiles are visited in groups of raster_group so that concurrently
// running CTAs share A and B tiles in L2.
//
// Every wait on an mbarrier is bounded by a clock budget.  When a wait runs out the
// thread records where, raises a CTA-wide abort flag that all other waits poll, and
// every role falls through to the common teardown, which frees tensor memory.
#pragma once

#include <cuda.h>
#include <cuda_fp16.h>
#include <stdint.h>

#include "ptx_sm100.cuh"

namespace hgemm_dev {

using namespace hgemm_ptx;

constexpr int kBlockM = 128;          // rows of one CTA's accumulator (UMMA M per CTA)
constexpr int kBlockK = 64;           // fp16 elements per k-block = one 128-byte swizzle span
constexpr int kUmmaK = 16;            // K of one tcgen05.mma.kind::f16
constexpr int kMaxStages = 12;
constexpr int kThreads = 192;
constexpr int kATileBytes = kBlockM * kBlockK * 2;           // 16 KB
constexpr int kStoreBoxRows = 32, kStoreBoxCols = 32;        // TMA-store box: one warp's 32 x 32 chunk
constexpr int kStagingBytesPerWarp = 2 * kStoreBoxRows * kStoreBoxCols * 2;  // two 2 KB buffers
constexpr int kStagingBytes = 4 * kStagingBytesPerWarp;      // 16 KB
constexpr int kCtrlBytes = 512;       // barriers, tensor-memory base, abort flag

// Status-word roles
constexpr uint32_t kRoleProducer = 1, kRoleMma = 2, kRoleEpilogue = 3, kRoleProbe = 4;

struct KernelParams {
    int32_t M, N, K;
    int32_t tiles_m, tiles_n;     // tiles_m counts block_m-row tiles (256 rows for a pair)
    int32_t total_work;           // tiles_m * tiles_n * split_k
    int32_t split_k;
    int32_t kblocks;              // ceil(K / 64)
    int32_t block_n;
    int32_t stages;
    int32_t raster_group;
    int32_t tmem_cols;            // power of two >= 2 * block_n
    int32_t epilogue_tma;         // 1: TMA-store epilogue (only when split_k == 1)
    uint32_t idesc;               // tcgen05 instruction descriptor
    float *workspace;             // split-K partials: [work item][chunk][col][128 rows]
    uint32_t *counters;           // split-K arrival counters: [tile][cta of pair][row quarter]
    uint32_t *status;             // device status word (0 = fine)
    __half *C;
    long long wait_budget;        // clock cycles a wait may take before the kernel gives up
    unsigned long long *trace;    // optional: CTA 0 writes %globaltimer stamps of its pipeline events (8 slots)
};

__device__ __forceinline__ void trace_stamp(const KernelParams &p, int slot)
{
    if (p.trace != nullptr && blockIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        p.trace[slot] = t;
    }
}

// -------------------------------------------------------------------------------------
// bounded wait

struct WaitCtl {
    volatile uint32_t *abort_flag;  // shared memory
    uint32_t *status;               // global memory
    long long budget;
};

__device__ __noinline__ bool mbar_wait_slow(uint32_t bar, uint32_t parity, const WaitCtl &ctl, uint32_t code)
{
    const long long t0 = clock64();
#pragma unroll 1
    while (true) {
        if (mbar_try_wait(bar, parity)) return true;
        if (*ctl.abort_flag) return false;
        if (clock64() - t0 > ctl.budget) {
            *ctl.abort_flag = 1u;
            atomicCAS(ctl.status, 0u, code);
            return false;
        }
    }
}

__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity, const WaitCtl &ctl, uint32_t code)
{
#pragma unroll 1
    for (int i = 0; i < 16; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, ctl, code);
}

__device__ __forceinline__ uint32_t status_code(uint32_t role, uint32_t barrier_index, uint32_t stage)
{
    return (role << 24) | ((barrier_index & 0xffffu) << 8) | (stage & 0xffu);
}

// -------------------------------------------------------------------------------------
// descriptors

// Shared-memory matrix descriptor of a K-major tile whose rows are 64 fp16 = 128 bytes,
// laid out by TMA with the 128-byte swizzle: 8-row groups are 1024 bytes apart.
__device__ __forceinline__ uint64_t make_smem_desc_sw128(uint32_t smem_byte_addr)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_byte_addr & 0x3ffffu) >> 4);        // [0,14)  start address >> 4
    d |= static_cast<uint64_t>(1) << 16;                                 // [16,30) leading byte offset (unused here)
    d |= static_cast<uint64_t>(1024 >> 4) << 32;                         // [32,46) stride byte offset: 8 rows * 128 B
    d |= static_cast<uint64_t>(1) << 46;                                 // [46,48) descriptor version (sm_100)
    d |= static_cast<uint64_t>(2) << 61;                                 // [61,64) 128-byte swizzle
    return d;
}

// -------------------------------------------------------------------------------------
// tile schedule

struct WorkItem {
    int32_t tile;       // linear tile index (tm, tn recovered by raster())
    int32_t m0, n0;     // first row / column of the (pair) tile
    int32_t slice;      // split-K slice
    int32_t kb_begin, kb_count;
};

__device__ __forceinline__ WorkItem decode_work(int32_t w, const KernelParams &p, int32_t block_m_total)
{
    WorkItem it;
    it.tile = w / p.split_k;
    it.slice = w - it.tile * p.split_k;
    // grouped raster: groups of raster_group m-tiles, swept along n inside a group
    const int32_t per_group = p.raster_group * p.tiles_n;
    const int32_t g = it.tile / per_group;
    const int32_t first_m = g * p.raster_group;
    const int32_t gsize = min(p.raster_group, p.tiles_m - first_m);
    const int32_t r = it.tile - g * per_group;
    const int32_t tn = r / gsize;
    const int32_t tm = first_m + (r - tn * gsize);
    it.m0 = tm * block_m_total;
    it.n0 = tn * p.block_n;
    const int32_t base = p.kblocks / p.split_k, rem = p.kblocks - base * p.split_k;
    it.kb_begin = it.slice * base + min(it.slice, rem);
    it.kb_count = base + (it.slice < rem ? 1 : 0);
    return it;
}

// -------------------------------------------------------------------------------------
// the kernel

template <int CTA_GROUP>
__global__ void __launch_bounds__(kThreads, 1)
hgemm_umma_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                  const __grid_constant__ CUtensorMap tmap_c, const KernelParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_addr(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - smem_addr(smem_raw));

    const int32_t b_rows = p.block_n / CTA_GROUP;            // B rows this CTA stages per k-block
    const uint32_t b_tile_bytes = static_cast<uint32_t>(b_rows) * kBlockK * 2;
    const uint32_t stage_bytes = kATileBytes + b_tile_bytes;
    const uint32_t staging_base = smem_base + static_cast<uint32_t>(p.stages) * stage_bytes;
    const uint32_t ctrl_base = staging_base + kStagingBytes;
    uint8_t *ctrl_gen = smem_gen + (ctrl_base - smem_base);

    // control block: full[12] | empty[12] | tmem_full[2] | tmem_empty[2] | tmem base | abort
    const uint32_t bar_full = ctrl_base;
    const uint32_t bar_empty = ctrl_base + 8 * kMaxStages;
    const uint32_t bar_tmem_full = ctrl_base + 16 * kMaxStages;
    const uint32_t bar_tmem_empty = bar_tmem_full + 16;
    volatile uint32_t *tmem_base_slot = reinterpret_cast<volatile uint32_t *>(ctrl_gen + 16 * kMaxStages + 32);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(ctrl_gen + 16 * kMaxStages + 36);

    const uint32_t warp = threadIdx.x >> 5;
    const uint32_t lane = threadIdx.x & 31;
    const uint32_t cta_rank = (CTA_GROUP == 2) ? cluster_ctarank() : 0u;
    const bool is_leader = (cta_rank == 0);
    const int32_t unit = (CTA_GROUP == 2) ? static_cast<int32_t>(blockIdx.x >> 1) : static_cast<int32_t>(blockIdx.x);
    const int32_t num_units = (CTA_GROUP == 2) ? static_cast<int32_t>(gridDim.x >> 1) : static_cast<int32_t>(gridDim.x);
    constexpr int32_t kBlockMTotal = kBlockM * CTA_GROUP;

    WaitCtl ctl{abort_flag, p.status, p.wait_budget};

    // ---- set-up -----------------------------------------------------------------------
    if (threadIdx.x == 0) {
        trace_stamp(p, 0);
        *abort_flag = 0u;
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(bar_full + 8 * s, CTA_GROUP);   // one arrive.expect_tx per CTA of the pair
            mbar_init(bar_empty + 8 * s, 1);          // one tcgen05.commit
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tmem_full + 8 * a, 1);              // one tcgen05.commit
            mbar_init(bar_tmem_empty + 8 * a, 4 * CTA_GROUP); // one arrive per epilogue warp (of both CTAs)
        }
        fence_mbar_init();
        prefetch_tensormap(&tmap_a);
        prefetch_tensormap(&tmap_b);
        prefetch_tensormap(&tmap_c);
    }
    if (warp == 1) {
        tmem_alloc<CTA_GROUP>(smem_addr(const_cast<uint32_t *>(tmem_base_slot)), static_cast<uint32_t>(p.tmem_cols));
        tmem_relinquish<CTA_GROUP>();
    }
    tc_fence_before_sync();
    __syncthreads();
    if constexpr (CTA_GROUP == 2) {   // the peer's barriers must exist before anything signals them
        cluster_arrive();
        cluster_wait();
    }
    tc_fence_after_sync();
    const uint32_t tmem_base = *tmem_base_slot;
    if (threadIdx.x == 0) trace_stamp(p, 1);

    // ---- roles ------------------------------------------------------------------------
    if (warp == 0) {
        if (lane == 0) {
            // ===== TMA producer =====
            int s = 0;
            uint32_t ph = 0;
            const uint32_t full_leader = (CTA_GROUP == 2) ? mapa(bar_full, 0) : bar_full;
            bool ok = true;
            for (int32_t w = unit; ok && w < p.total_work; w += num_units) {
                const WorkItem it = decode_work(w, p, kBlockMTotal);
                const int32_t a_row = it.m0 + static_cast<int32_t>(cta_rank) * kBlockM;
                const int32_t b_row = it.n0 + static_cast<int32_t>(cta_rank) * b_rows;
                for (int32_t kb = 0; kb < it.kb_count; ++kb) {
                    ok = mbar_wait(bar_empty + 8 * s, ph ^ 1u, ctl, status_code(kRoleProducer, 0, s));
                    if (!ok) break;
                    const uint32_t a_dst = smem_base + static_cast<uint32_t>(s) * stage_bytes;
                    const uint32_t b_dst = a_dst + kATileBytes;
                    const int32_t k0 = (it.kb_begin + kb) * kBlockK;
                    if constexpr (CTA_GROUP == 1) {
                        mbar_arrive_expect_tx(bar_full + 8 * s, stage_bytes);
                        tma_load_2d(a_dst, &tmap_a, k0, a_row, bar_full + 8 * s);
                        tma_load_2d(b_dst, &tmap_b, k0, b_row, bar_full + 8 * s);
                    } else {
                        // both CTAs of the pair announce their bytes on the leader's barrier; the peer's
                        // remote arrive is relaxed (it orders nothing: the data arrives through TMA)
                        const uint32_t fb = full_leader + 8 * s;
                        if (is_leader) mbar_arrive_expect_tx(bar_full + 8 * s, stage_bytes);
                        else mbar_arrive_expect_tx_cluster_relaxed(fb, stage_bytes);
                        tma_load_2d_pair(a_dst, &tmap_a, k0, a_row, fb);
                        tma_load_2d_pair(b_dst, &tmap_b, k0, b_row, fb);
                    }
                    if (w == unit && kb == 0) trace_stamp(p, 2);
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                }
            }
        }
    } else if (warp == 1) {
        if (lane == 0 && is_leader) {
            // ===== MMA issuer =====
            int s = 0;
            uint32_t ph = 0;
            uint32_t local_tile = 0;
            bool ok = true;
            for (int32_t w = unit; ok && w < p.total_work; w += num_units, ++local_tile) {
                const WorkItem it = decode_work(w, p, kBlockMTotal);
                const uint32_t acc = local_tile & 1u;
                const uint32_t acc_ph = (local_tile >> 1) & 1u;
                ok = mbar_wait(bar_tmem_empty + 8 * acc, acc_ph ^ 1u, ctl, status_code(kRoleMma, 1, acc));
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * static_cast<uint32_t>(p.block_n);
                for (int32_t kb = 0; kb < it.kb_count; ++kb) {
                    ok = mbar_wait(bar_full + 8 * s, ph, ctl, status_code(kRoleMma, 0, s));
                    if (!ok) break;
                    if (w == unit && kb == 0) trace_stamp(p, 3);
                    tc_fence_after_sync();
                    const uint32_t a_addr = smem_base + static_cast<uint32_t>(s) * stage_bytes;
                    const uint64_t a_desc = make_smem_desc_sw128(a_addr);
                    const uint64_t b_desc = make_smem_desc_sw128(a_addr + kATileBytes);
#pragma unroll
                    for (int k = 0; k < kBlockK / kUmmaK; ++k) {
                        // advancing K by 16 fp16 inside the swizzle span = +32 bytes = +2 in the address field
                        umma_f16<CTA_GROUP>(d_tmem, a_desc + 2u * k, b_desc + 2u * k, p.idesc,
                                            (kb | k) != 0 ? 1u : 0u);
                    }
                    // free the stage (in both CTAs of a pair) once these MMAs have read it
                    if constexpr (CTA_GROUP == 1) {
                        umma_commit<1>(bar_empty + 8 * s);
                    } else {
                        umma_commit<2>(mapa(bar_empty + 8 * s, 0));
                        umma_commit<2>(mapa(bar_empty + 8 * s, 1));
                    }
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                }
                if (!ok) break;
                if (w == unit) trace_stamp(p, 4);
                if constexpr (CTA_GROUP == 1) {
                    umma_commit<1>(bar_tmem_full + 8 * acc);
                } else {
                    umma_commit<2>(mapa(bar_tmem_full + 8 * acc, 0));
                    umma_commit<2>(mapa(bar_tmem_full + 8 * acc, 1));
                }
            }
        }
    } else {
        // ===== epilogue (warps 2..5) =====
        const uint32_t q = warp & 3u;                               // tensor-memory lane quarter of this warp
        const uint32_t row_in_tile = q * 32u + lane;                // accumulator row = tensor-memory lane
        const uint32_t staging = staging_base + (warp - 2u) * kStagingBytesPerWarp;
        const uint32_t tmem_empty_leader = (CTA_GROUP == 2) ? mapa(bar_tmem_empty, 0) : bar_tmem_empty;
        const int32_t chunks = p.block_n / 32;
        uint32_t local_tile = 0;
        uint32_t store_count = 0;
        bool ok = true;
        for (int32_t w = unit; ok && w < p.total_work; w += num_units, ++local_tile) {
            const WorkItem it = decode_work(w, p, kBlockMTotal);
            const uint32_t acc = local_tile & 1u;
            const uint32_t acc_ph = (local_tile >> 1) & 1u;
            ok = mbar_wait(bar_tmem_full + 8 * acc, acc_ph, ctl, status_code(kRoleEpilogue, 2, acc));
            ok = __all_sync(0xffffffffu, ok);   // the warp-wide tensor-memory loads below need the whole warp
            if (!ok) break;
            if (w == unit && threadIdx.x == 64) trace_stamp(p, 5);
            tc_fence_after_sync();
            const int32_t row0 = it.m0 + static_cast<int32_t>(cta_rank) * kBlockM;  // first row of this CTA's 128
            const int32_t grow = row0 + static_cast<int32_t>(row_in_tile);          // this thread's global row
            const uint32_t t_addr = tmem_base + ((q * 32u) << 16) + acc * static_cast<uint32_t>(p.block_n);

            if (p.split_k == 1) {
                for (int32_t c = 0; c < chunks; ++c) {
                    uint32_t v[32];
                    const int32_t col0 = it.n0 + c * 32;
                    if (p.epilogue_tma) {
                        const uint32_t buf = staging + (store_count & 1u) * (kStagingBytesPerWarp / 2);
                        // the buffer written two stores ago must have been read by its TMA store
                        if (lane == 0) bulk_wait_group_read<1>();
                        __syncwarp();
                        tmem_ld_32x32b_x32(t_addr + static_cast<uint32_t>(c) * 32u, v);
                        tmem_ld_wait();
                        // row `lane` of the 32 x 32 box is 64 bytes; 64-byte swizzle: 16-byte chunk j of
                        // row r lives at chunk j ^ ((r >> 1) & 3)
                        const uint32_t row_addr = buf + lane * 64u;
                        const uint32_t sw = (lane >> 1) & 3u;
#pragma unroll
                        for (uint32_t j = 0; j < 4; ++j) {
                            st_shared_v4(row_addr + ((j ^ sw) << 4),
                                         pack_half2_rn(v[8 * j + 0], v[8 * j + 1]), pack_half2_rn(v[8 * j + 2], v[8 * j + 3]),
                                         pack_half2_rn(v[8 * j + 4], v[8 * j + 5]), pack_half2_rn(v[8 * j + 6], v[8 * j + 7]));
                        }
                        fence_proxy_async_smem();
                        __syncwarp();
                        if (lane == 0) {
                            const int32_t box_row = row0 + static_cast<int32_t>(q) * 32;
                            if (box_row < p.M && col0 < p.N) {
                                tma_store_2d(&tmap_c, col0, box_row, buf);
                            }
                            bulk_commit_group();
                        }
                        ++store_count;
                    } else {
                        tmem_ld_32x32b_x32(t_addr + static_cast<uint32_t>(c) * 32u, v);
                        tmem_ld_wait();
                        if (grow < p.M) {
                            __half *dst = p.C + static_cast<size_t>(grow) * p.N + col0;
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                if (col0 + 8 * j + 8 <= p.N) {
                                    uint4 o;
                                    o.x = pack_half2_rn(v[8 * j + 0], v[8 * j + 1]);
                                    o.y = pack_half2_rn(v[8 * j + 2], v[8 * j + 3]);
                                    o.z = pack_half2_rn(v[8 * j + 4], v[8 * j + 5]);
                                    o.w = pack_half2_rn(v[8 * j + 6], v[8 * j + 7]);
                                    *reinterpret_cast<uint4 *>(dst + 8 * j) = o;
                                }
                            }
                        }
                    }
                }
                // accumulator drained: hand it back to the MMA issuer
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) {
                    if constexpr (CTA_GROUP == 1) mbar_arrive(bar_tmem_empty + 8 * acc);
                    else mbar_arrive_cluster(tmem_empty_leader + 8 * acc);
                }
            } else {
                // ---- split-K: park the fp32 partial, the last slice to arrive reduces in slice order ----
                const size_t slot_floats = static_cast<size_t>(kBlockM) * p.block_n;
                // one slot per (work item, CTA of the pair); layout [chunk][col][128 rows] so a warp's
                // 32 rows of one column are one 128-byte line
                float *slot = p.workspace + (static_cast<size_t>(w) * CTA_GROUP + cta_rank) * slot_floats;
                for (int32_t c = 0; c < chunks; ++c) {
                    uint32_t v[32];
                    tmem_ld_32x32b_x32(t_addr + static_cast<uint32_t>(c) * 32u, v);
                    tmem_ld_wait();
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        __stcg(slot + (static_cast<size_t>(c) * 32 + j) * kBlockM + row_in_tile, __uint_as_float(v[j]));
                }
                tc_fence_before_sync();
                __threadfence();
                __syncwarp();
                uint32_t prev = 0;
                uint32_t *counter = p.counters + (static_cast<size_t>(it.tile) * CTA_GROUP + cta_rank) * 4 + q;
                if (lane == 0) {
                    if constexpr (CTA_GROUP == 1) mbar_arrive(bar_tmem_empty + 8 * acc);
                    else mbar_arrive_cluster(tmem_empty_leader + 8 * acc);
                    prev = atomicAdd(counter, 1u);
                    __threadfence();
                }
                prev = __shfl_sync(0xffffffffu, prev, 0);
                if (prev == static_cast<uint32_t>(p.split_k) - 1u) {
                    __threadfence();
                    // all slices of this tile quarter are in the workspace: sum them in slice order
                    const size_t first_slot = static_cast<size_t>(it.tile) * p.split_k;
                    for (int32_t c = 0; c < chunks; ++c) {
                        float accv[32];
#pragma unroll
                        for (int j = 0; j < 32; ++j) accv[j] = 0.0f;
                        for (int32_t sl = 0; sl < p.split_k; ++sl) {
                            const float *src = p.workspace + ((first_slot + sl) * CTA_GROUP + cta_rank) * slot_floats;
#pragma unroll
                            for (int j = 0; j < 32; ++j)
                                accv[j] += __ldcg(src + (static_cast<size_t>(c) * 32 + j) * kBlockM + row_in_tile);
                        }
                        const int32_t col0 = it.n0 + c * 32;
                        if (grow < p.M) {
                            __half *dst = p.C + static_cast<size_t>(grow) * p.N + col0;
#pragma unroll
                            for (int j = 0; j < 4; ++j) {
                                if (col0 + 8 * j + 8 <= p.N) {
                                    uint4 o;
                                    o.x = pack_half2_rn(__float_as_uint(accv[8 * j + 0]), __float_as_uint(accv[8 * j + 1]));
                                    o.y = pack_half2_rn(__float_as_uint(accv[8 * j + 2]), __float_as_uint(accv[8 * j + 3]));
                                    o.z = pack_half2_rn(__float_as_uint(accv[8 * j + 4]), __float_as_uint(accv[8 * j + 5]));
                                    o.w = pack_half2_rn(__float_as_uint(accv[8 * j + 6]), __float_as_uint(accv[8 * j + 7]));
                                    *reinterpret_cast<uint4 *>(dst + 8 * j) = o;
                                }
                            }
                        }
                    }
                    if (lane == 0) *counter = 0u;   // ready for the next run of this plan
                }
            }
        }
        // shared memory must stay valid until the last TMA stores have read it
        if (lane == 0) bulk_wait_group<0>();
        if (threadIdx.x == 64) trace_stamp(p, 6);
    }

    // ---- teardown (every thread, also after an abort) ----------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if constexpr (CTA_GROUP == 2) {   // no CTA of the pair leaves while the other may still signal it
        cluster_arrive();
        cluster_wait();
    }
    if (warp == 1) {
        if (*abort_flag) {
            // give loads and MMAs that were in flight when a wait ran out time to land
            for (int i = 0; i < 200; ++i) __nanosleep(1000);
        }
        tc_fence_after_sync();
        tmem_dealloc<CTA_GROUP>(tmem_base, static_cast<uint32_t>(p.tmem_cols));
        if (lane == 0) trace_stamp(p, 7);
    }
}

// A kernel whose only wait is on a barrier nothing ever signals: exercises the bounded
// wait and the status word without any fault.
__global__ void hgemm_timeout_probe_kernel(uint32_t *status, long long budget)
{
    __shared__ __align__(8) uint64_t bar;
    __shared__ uint32_t abort_flag;
    if (threadIdx.x == 0) {
        abort_flag = 0u;
        mbar_init(smem_addr(&bar), 1);
        fence_mbar_init();
        WaitCtl ctl{&abort_flag, status, budget};
        (void)mbar_wait(smem_addr(&bar), 0u, ctl, status_code(kRoleProbe, 0xffff, 0xff));
    }
}

} // namespace hgemm_dev
