// The persistent, warp-specialised tcgen05 HGEMM kernel (the 1-CTA and CTA-pair families are
// instances of this one template; the light and the small family have files of their own).
//
// Structure per CTA (320 threads):
//   warp 0      TMA producer: fills a ring of shared-memory stages with 64-wide
//               k-blocks of A (128 rows) and B (block_n rows, or block_n/2 in a pair)
//   warp 1      allocates tensor memory; one thread issues tcgen05.mma into one of two
//               fp32 accumulators (double-buffered so the epilogue of tile t overlaps
//               the main loop of tile t+1)
//   warps 2..9  epilogue: tensor memory -> registers -> fp16 -> global (direct 16-byte
//               stores, or swizzled shared memory + TMA store); with split-K each slice
//               parks its fp32 partial in a workspace, waits (bounded) for the other
//               slices of its tile, and sums its share of the tile over all slices in
//               slice order.
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

#include <type_traits>

#include "ptx_sm100.cuh"

namespace hgemm_dev {

using namespace hgemm_ptx;

constexpr int kBlockM = 128;          // rows of one CTA's accumulator (UMMA M per CTA)
constexpr int kSubK = 64;             // fp16 elements of one sub-tile row = one 128-byte swizzle span
constexpr int kUmmaK = 16;            // K of one tcgen05.mma.kind::f16
constexpr int kMaxStages = 12;
constexpr int kThreads = 320;          // producer warp + MMA warp + 8 epilogue warps
constexpr int kATileBytes = kBlockM * kSubK * 2;             // 16 KB: one 128 x 64 sub-tile of A
constexpr int kStoreBoxRows = 32, kStoreBoxCols = 32;        // TMA-store box: one warp's 32 x 32 chunk
constexpr int kStagingBytesPerWarp = 2 * kStoreBoxRows * kStoreBoxCols * 2;  // two 2 KB buffers
constexpr int kStagingBytes = 8 * kStagingBytesPerWarp;      // 32 KB
constexpr int kWideBoxBytes = kStoreBoxRows * 64 * 2;        // wide TMA epilogue: 32 rows x 64 columns, two per warp (64 KB in all)
constexpr int kCtrlBytes = 512;       // barriers, tensor-memory base, abort flag

// Status-word roles
constexpr uint32_t kRoleProducer = 1, kRoleMma = 2, kRoleEpilogue = 3, kRoleProbe = 4;
// The checked build (-DHGEMM_CHECKED=1, a second library beside the ordinary one): invariants that the ordinary build relies
// on without testing them -- a work item inside the tile grid and the K range, TMA coordinates on 16-byte boundaries, stores
// of reduced units inside C, parked pieces inside the workspace, arrival counters inside their array, accumulator columns
// inside the allocation -- are tested where they are used.  A violation records (kRoleCheck, site) in the plan's status
// word and the access is skipped; hgemm_last_device_status then reports HGEMM_ERR_CHECK.
#ifndef HGEMM_CHECKED
#define HGEMM_CHECKED 0
#endif
constexpr uint32_t kRoleCheck = 7;
constexpr uint32_t kCheckWorkItem = 1, kCheckLoadCoord = 2, kCheckUnitStore = 3, kCheckSlot = 4, kCheckCounter = 5, kCheckStoreCoord = 6,
                   kCheckTmemColumn = 7, kCheckSmallStore = 8, kCheckProbe = 99;

// x / d for x < 2^31 without a division instruction: q = umulhi(x, mul) >> shr (d == 1: q = x).
// mul = ceil(2^(31 + ceil(log2 d)) / d), shr = ceil(log2 d) - 1.
struct FastDiv {
    uint32_t mul, shr, d;
};

__host__ __device__ inline FastDiv make_fast_div(uint32_t d)
{
    FastDiv f;
    f.d = d < 1u ? 1u : d;
    f.mul = 0u;
    f.shr = 0u;
    if (f.d > 1u) {
        uint32_t lg = 0;
        while ((1ull << lg) < f.d) ++lg;                                 // ceil(log2 d) >= 1
        const unsigned long long pw = 1ull << (31u + lg);
        f.mul = static_cast<uint32_t>((pw + f.d - 1u) / f.d);
        f.shr = lg - 1u;
    }
    return f;
}

__host__ __device__ __forceinline__ int32_t fast_div(int32_t x, const FastDiv &f)
{
#ifdef __CUDA_ARCH__
    return f.d == 1u ? x : static_cast<int32_t>(__umulhi(static_cast<uint32_t>(x), f.mul) >> f.shr);
#else
    return static_cast<int32_t>(static_cast<uint32_t>(x) / f.d);      // the host's copy (layout computations, tests)
#endif
}

// Stream-K tail (paper section 5.2 picks a tile shape per problem; a tile count that does not fill the last wave of
// SMs is what this evens out): the `rem` tiles that remain after the full waves are `q = rem * kblocks` k-blocks in
// tile-major order, dealt out as `gs` contiguous ranges [floor(j q / gs), floor((j + 1) q / gs)), one per CTA
// position j.  rem <= gs, so a range is at most one tile long and crosses at most one tile boundary: position j has
// up to two work items, h = 0 (the part in the tile where its range starts) and h = 1 (the part in the next tile).
// The positions that share a tile are consecutive; the item's slice is its place among them, and the tile's
// partial sums are added in that order.
struct StreamItem {
    int32_t tile_rel;    // tile, counted from the first tile of the tail
    int32_t kb_begin, kb_count;
    int32_t slice, slices;
};

__host__ __device__ __forceinline__ StreamItem stream_item(int32_t j, int32_t h, int32_t gs, int32_t q, int32_t kblocks,
                                                           const FastDiv &fd_gs, const FastDiv &fd_q, const FastDiv &fd_kblocks)
{
    StreamItem s;
    s.tile_rel = 0; s.kb_begin = 0; s.kb_count = 0; s.slice = 0; s.slices = 1;
    if (j >= gs) return s;                                            // a position without a share of the tail
    const int32_t b0 = fast_div(j * q, fd_gs), b1 = fast_div((j + 1) * q, fd_gs);
    const int32_t t0 = fast_div(b0, fd_kblocks);
    const int32_t edge = (t0 + 1) * kblocks;                          // first k-block of the next tile
    if (h == 0) {
        s.tile_rel = t0;
        s.kb_begin = b0 - t0 * kblocks;
        s.kb_count = (b1 < edge ? b1 : edge) - b0;
    } else {
        s.tile_rel = t0 + 1;
        s.kb_count = b1 - edge;
    }
    if (s.kb_count <= 0) {
        s.tile_rel = 0;
        s.kb_count = 0;
        return s;
    }
    // positions whose ranges meet this tile: the largest j' with floor(j' q / gs) <= x is floor(((x + 1) gs - 1) / q)
    const int32_t x = s.tile_rel * kblocks;
    const int32_t j_lo = fast_div((x + 1) * gs - 1, fd_q), j_hi = fast_div((x + kblocks) * gs - 1, fd_q);
    s.slice = j - j_lo;
    s.slices = j_hi - j_lo + 1;
    return s;
}

struct KernelParams {
    int32_t M, N, K;
    int32_t tiles_m, tiles_n;     // tiles_m counts block_m-row tiles (256 rows for a pair)
    int32_t total_work;           // first_split_tile + (tiles - first_split_tile) * split_k
    int32_t split_k;              // K slices per split tile
    int32_t first_split_tile;     // tiles below this index are whole work items; tiles from it on are split into
                                  // split_k slices (0: every tile is split; tiles_m * tiles_n with split_k == 1: none)
    int32_t kblocks;              // ceil(K / block_k)
    int32_t block_k;              // K extent of one pipeline stage: 64 or 128 (one or two 64-wide sub-tiles)
    int32_t block_n;
    int32_t stages;
    int32_t raster_group;
    int32_t tmem_cols;            // power of two >= 2 * block_n
    int32_t epilogue_tma;         // 1: TMA-store epilogue, 32 x 32 boxes; 2: 32 x 64 boxes (only when split_k == 1)
    int32_t b_row_major;          // 1: B is the K x N row-major operand ("NN" layout): B tiles are N-major in shared memory
    int32_t ragged_n;             // 1: N % 8 != 0: rows of C are not 16-byte multiples, store element by element
    int32_t tma_3d;               // 1: the A and B maps are 3-D {64, rows, K / 64}: one load per operand per stage
    int32_t cluster_split;        // 1: the split_k slices of a tile are one cluster and reduce through shared memory
    uint32_t idesc;               // tcgen05 instruction descriptor
    uint32_t idesc_tail;          // the same with N = block_n / tail_pieces (column pieces of tail tiles)
    float *workspace;             // split-K partials: [work item][cta of pair][chunk][128 rows][32 cols]
    uint32_t *counters;           // split-K counters: [tile][cta of pair][arrived, finished]
    uint32_t *status;             // device status word (0 = fine)
    __half *C;
    long long wait_budget;        // clock cycles a wait may take before the kernel gives up
    unsigned long long *trace;    // optional: CTA 0 writes %globaltimer stamps of its pipeline events (8 slots)
    uint32_t debug_skip;          // instrumentation: bit 0 = no TMA loads, bit 1 = no MMAs, bit 2 = no TMA stores (results are garbage)
    uint32_t epoch;               // workspace split-K: number of this launch among the launches that used `counters` (from 1)
    // division by run-time constants of the work decode as multiply-high and shift (set by the host)
    FastDiv fd_per_group, fd_raster, fd_last_group, fd_split, fd_pieces;
    int32_t acc_f16;              // 1: fp16 accumulators (one result in the low half of each 32-bit tensor-memory column)
    int32_t tail_pieces;          // > 1: work items from first_split_tile on are tiles cut into this many column pieces (no K split)
    uint32_t scaled;              // 0: C = A B^T; 1: C = alpha A B^T + beta C (paper section 2.1)
    float alpha, beta;
    int32_t transposed;           // 1: the kernel computes the transposed problem (the caller's B is its A, M and N are
                                  // traded) and stores element (row, col) of its tile at C[col * M + row]: the
                                  // caller's row-major C (whose rows are this kernel's M long)
    int32_t raster_serpentine;    // 1: odd raster groups sweep the n-tiles from last to first
    uint32_t early_ops;           // bit 0 / bit 1: the kernel's A / B operand is static (no kernel ahead in the stream writes
                                  // it): its first loads may leave before the stream dependency is resolved
    // stream-K tail (see stream_item): 0 positions = none.  Then split_k is the largest number of slices of a tile
    // (the stride of a tile's workspace slots) and the work items from first_split_tile on are numbered
    // first_split_tile + h * grid_units + j.
    unsigned long long workspace_floats;   // capacity of `workspace` and of `counters` (32-bit words): what the checked build
    unsigned long long counter_words;      // tests parked pieces and arrivals against
    // wave pacing (0: off): no producer starts the loads of its tile number r before every CTA (pair) of the grid has issued
    // the last load of its tile number r - 1.  Pacing only -- a wait gives up after 50 us and nothing depends on it.
    int32_t wave_pace, wave_rounds;        // rounds = tiles per CTA (pair), rounded up
    uint32_t *wave_counter;                // arrivals, never reset: this launch counts on from wave_base
    uint32_t wave_base;
    int32_t stream_units;         // positions that share the tail's k-blocks
    int32_t stream_q;             // k-blocks of the tail: (tiles - first_split_tile) * kblocks
    int32_t grid_units;           // CTAs (pairs) of the grid
    FastDiv fd_stream_units, fd_stream_q, fd_kblocks;
};

template <bool OFF = false>
__device__ __forceinline__ void trace_stamp(const KernelParams &p, int slot)
{
    if constexpr (OFF) return;
    if (p.trace != nullptr && blockIdx.x == 0) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        p.trace[slot] = t;
    }
    // debug bit 3: every CTA also records when it started working (slot 0) and when it finished (slot 7)
    // behind the 24 slots of CTA 0: entries 24 + 2 * blockIdx.x and + 1
    if (p.trace != nullptr && (p.debug_skip & 8u) && (slot == 0 || slot == 7)) {
        unsigned long long t;
        asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
        p.trace[24 + 2 * blockIdx.x + (slot == 7 ? 1 : 0)] = t;
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
    if (mbar_test_wait(bar, parity)) return true;      // already complete: the cheap query answers
#pragma unroll 1
    for (int i = 0; i < 16; ++i)
        if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, ctl, code);
}

__device__ __forceinline__ uint32_t status_code(uint32_t role, uint32_t barrier_index, uint32_t stage)
{
    return (role << 24) | ((barrier_index & 0xffffu) << 8) | (stage & 0xffu);
}

// Checked build: `holds` is an invariant of site `site`; false records it and tells the caller to skip the access.
// Ordinary build: always true, and the test of `holds` is compiled out with it.
__device__ __forceinline__ bool checked(uint32_t *status, bool holds, uint32_t site)
{
#if HGEMM_CHECKED
    if (!holds) {
        atomicCAS(status, 0u, status_code(kRoleCheck, site, 0));
        return false;
    }
#endif
    return true;
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
// stores for a C whose rows are not multiples of 16 bytes (N % 8 != 0)

__device__ __forceinline__ void store_ragged(__half *C, int64_t N, int32_t row, int32_t col, const float *vals, int count)
{
    for (int j = 0; j < count; ++j)
        if (col + j < N) C[static_cast<size_t>(row) * N + col + j] = __float2half_rn(vals[j]);
}

// Transposed result (see KernelParams::transposed): `count` consecutive columns of one row of the kernel's tile are
// `count` elements of one COLUMN of the caller's C, p.M apart.
__device__ __forceinline__ void store_transposed(__half *C, int64_t ldc, int32_t n_cols, int32_t row, int32_t col, const float *vals, int count)
{
    for (int j = 0; j < count; ++j)
        if (col + j < n_cols) C[static_cast<size_t>(col + j) * ldc + row] = __float2half_rn(vals[j]);
}

// Four consecutive columns of one row of the kernel's tile, for the two layouts of C that rule out 8-byte stores
// (rows that are not multiples of 16 bytes; the transposed result).  Out of line on purpose: the split-K reductions
// call it from loops that keep dozens of partial sums in registers, and inlined there it made them spill.
__device__ __noinline__ void store_unit4_slow(__half *C, int32_t M, int32_t N, int32_t transposed, int32_t row, int32_t col,
                                              float x, float y, float z, float w)
{
    const float f[4] = {x, y, z, w};
    if (transposed) store_transposed(C, M, N, row, col, f, 4);
    else store_ragged(C, N, row, col, f, 4);
}

// The same for a tile that is contiguous along its M/N dimension (a row-major K x N operand): the tile
// is stored as blocks of 64 columns, each block 64 k-rows of 128 bytes under the 128-byte swizzle.
// Leading byte offset = distance between 64-column blocks, stride byte offset = distance between
// groups of 8 k-rows (1024 bytes); one UMMA (K = 16) spans two such groups.
__device__ __forceinline__ uint64_t make_smem_desc_sw128_mn_major(uint32_t smem_byte_addr, uint32_t block_bytes)
{
    uint64_t d = 0;
    d |= static_cast<uint64_t>((smem_byte_addr & 0x3ffffu) >> 4);
    d |= static_cast<uint64_t>((block_bytes >> 4) & 0x3fffu) << 16;
    d |= static_cast<uint64_t>(1024 >> 4) << 32;
    d |= static_cast<uint64_t>(1) << 46;
    d |= static_cast<uint64_t>(2) << 61;
    return d;
}

// -------------------------------------------------------------------------------------
// tile schedule

// -------------------------------------------------------------------------------------
// C = alpha A B^T + beta C (paper section 2.1, the general form of the operation): the scaling step of every
// store path.  All in fp32 -- alpha * acc rounded once, then one fused multiply-add with the old element --
// and the result is rounded to fp16 once by the caller.  With beta == 0 the old C is never read.

__device__ __forceinline__ float scaled_value(float acc, float alpha, float beta, float old)
{
    return fmaf(beta, old, alpha * acc);
}

// v[0..7]: fp32 bit patterns of eight consecutive columns col .. col + 7 of row `row`.
template <bool XPOSE = false>
__device__ __forceinline__ void scale_group8(uint32_t *v, const KernelParams &p, int32_t row, int32_t col)
{
    float old[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) old[i] = 0.0f;
    if (XPOSE && p.beta != 0.0f) {
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (col + i < p.N) old[i] = __half2float(p.C[static_cast<size_t>(col + i) * p.M + row]);
    } else if (p.beta != 0.0f) {
        const __half *src = p.C + static_cast<size_t>(row) * p.N + col;
        if (!p.ragged_n && col + 8 <= p.N) {
            const uint4 o = *reinterpret_cast<const uint4 *>(src);   // N % 8 == 0: 16-byte aligned
            const __half2 *h = reinterpret_cast<const __half2 *>(&o);
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const float2 f = __half22float2(h[i]);
                old[2 * i] = f.x;
                old[2 * i + 1] = f.y;
            }
        } else {
#pragma unroll
            for (int i = 0; i < 8; ++i)
                if (col + i < p.N) old[i] = __half2float(src[i]);
        }
    }
#pragma unroll
    for (int i = 0; i < 8; ++i) v[i] = __float_as_uint(scaled_value(__uint_as_float(v[i]), p.alpha, p.beta, old[i]));
}

// s: four consecutive columns col .. col + 3 of row `row`.
template <bool XPOSE = false>
__device__ __forceinline__ void scale_unit4(float4 &s, const KernelParams &p, int32_t row, int32_t col)
{
    float old[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    if (XPOSE && p.beta != 0.0f) {
#pragma unroll
        for (int i = 0; i < 4; ++i)
            if (col + i < p.N) old[i] = __half2float(p.C[static_cast<size_t>(col + i) * p.M + row]);
    } else if (p.beta != 0.0f) {
        const __half *src = p.C + static_cast<size_t>(row) * p.N + col;
        if (!p.ragged_n) {                                            // N % 8 == 0 and col % 4 == 0: 8-byte aligned, in bounds
            const uint2 o = *reinterpret_cast<const uint2 *>(src);
            const __half2 *h = reinterpret_cast<const __half2 *>(&o);
            const float2 f0 = __half22float2(h[0]), f1 = __half22float2(h[1]);
            old[0] = f0.x; old[1] = f0.y; old[2] = f1.x; old[3] = f1.y;
        } else {
#pragma unroll
            for (int i = 0; i < 4; ++i)
                if (col + i < p.N) old[i] = __half2float(src[i]);
        }
    }
    s.x = scaled_value(s.x, p.alpha, p.beta, old[0]);
    s.y = scaled_value(s.y, p.alpha, p.beta, old[1]);
    s.z = scaled_value(s.z, p.alpha, p.beta, old[2]);
    s.w = scaled_value(s.w, p.alpha, p.beta, old[3]);
}

struct WorkItem {
    int32_t tile;       // linear tile index (tm, tn recovered by raster())
    int32_t m0, n0;     // first row / column of the (pair) tile
    int32_t slice;      // split-K slice
    int32_t slices;     // number of slices of this tile (1: the tile is one work item)
    int32_t split_index;   // index of this (tile, slice) among the split work items; split tiles are numbered from 0
    int32_t kb_begin, kb_count;
    int32_t bn;         // columns of this work item: block_n, or block_n / tail_pieces for a piece of a tail tile
};

// SPLIT = false: the caller knows that no work item is a K slice (split_k == 1 and no tail cut along K).
template <bool SPLIT = true, bool PLAIN = false>
__device__ __forceinline__ WorkItem decode_work(int32_t w, const KernelParams &p, int32_t block_m_total)
{
    WorkItem it;
    // Whole tiles first, then the cut ones: with a persistent grid the cut tiles form the last,
    // partly filled wave, whose tiles are cut along K (slices, summed afterwards) or into column
    // pieces (independent narrower tiles) so that every SM has work until the end.
    int32_t n_off = 0;
    bool own_k_range = false;
    it.bn = p.block_n;
    if (w < p.first_split_tile) {
        it.tile = w;
        it.slice = 0;
        it.slices = 1;
        it.split_index = 0;
    } else if (!PLAIN && p.tail_pieces > 1) {
        const int32_t idx = w - p.first_split_tile;
        const int32_t t = fast_div(idx, p.fd_pieces);
        it.tile = p.first_split_tile + t;
        it.slice = 0;
        it.slices = 1;
        it.split_index = 0;
        it.bn = p.block_n / p.tail_pieces;
        n_off = (idx - t * p.tail_pieces) * it.bn;
    } else if (!SPLIT) {
        it.tile = w;                     // not reached: without K slices every item is a whole tile or a column piece
        it.slice = 0;
        it.slices = 1;
        it.split_index = 0;
    } else if (p.stream_units > 0) {
        const int32_t idx = w - p.first_split_tile;
        const int32_t h = idx >= p.grid_units ? 1 : 0;
        const StreamItem si = stream_item(idx - h * p.grid_units, h, p.stream_units, p.stream_q, p.kblocks, p.fd_stream_units,
                                          p.fd_stream_q, p.fd_kblocks);
        it.tile = p.first_split_tile + si.tile_rel;
        it.slice = si.slice;
        it.slices = si.slices;
        it.split_index = si.tile_rel * p.split_k + si.slice;
        it.kb_begin = si.kb_begin;
        it.kb_count = si.kb_count;                       // 0: this position has no such item; every role skips it
        own_k_range = true;
    } else {
        it.split_index = w - p.first_split_tile;
        const int32_t t = fast_div(it.split_index, p.fd_split);
        it.tile = p.first_split_tile + t;
        it.slice = it.split_index - t * p.split_k;
        it.slices = p.split_k;
    }
    // grouped raster: groups of raster_group m-tiles, swept along n inside a group
    const int32_t per_group = p.raster_group * p.tiles_n;
    const int32_t g = fast_div(it.tile, p.fd_per_group);
    const int32_t first_m = g * p.raster_group;
    const int32_t gsize = min(p.raster_group, p.tiles_m - first_m);   // the last group may hold fewer m-tiles
    const int32_t r = it.tile - g * per_group;
    const int32_t tn = gsize == p.raster_group ? fast_div(r, p.fd_raster) : fast_div(r, p.fd_last_group);
    const int32_t tm = first_m + (r - tn * gsize);
    // serpentine: an odd group walks the n-tiles backwards, starting on the B tiles the group before it used last
    const int32_t tn_at = (p.raster_serpentine && (g & 1)) ? p.tiles_n - 1 - tn : tn;
    it.m0 = tm * block_m_total;
    it.n0 = tn_at * p.block_n + n_off;
    if (SPLIT && own_k_range) {
        // (a stream-K item brought its own range)
    } else if (!SPLIT || it.slices == 1) {
        it.kb_begin = 0;
        it.kb_count = p.kblocks;
    } else {
        const int32_t base = fast_div(p.kblocks, p.fd_split), rem = p.kblocks - base * it.slices;   // slices == split_k here
        it.kb_begin = it.slice * base + min(it.slice, rem);
        it.kb_count = base + (it.slice < rem ? 1 : 0);
    }
    return it;
}

// The same work item with every field passed through a shuffle from lane 0: all lanes already hold the same
// values, but only after the shuffle does the compiler know it, and TMA and tcgen05 instructions take their
// operands from uniform registers -- values it cannot prove uniform cost a move per instruction.
__device__ __forceinline__ WorkItem warp_uniform(const WorkItem &it)
{
    WorkItem u;
    u.tile = __shfl_sync(0xffffffffu, it.tile, 0);
    u.m0 = __shfl_sync(0xffffffffu, it.m0, 0);
    u.n0 = __shfl_sync(0xffffffffu, it.n0, 0);
    u.slice = __shfl_sync(0xffffffffu, it.slice, 0);
    u.slices = __shfl_sync(0xffffffffu, it.slices, 0);
    u.split_index = __shfl_sync(0xffffffffu, it.split_index, 0);
    u.kb_begin = __shfl_sync(0xffffffffu, it.kb_begin, 0);
    u.kb_count = __shfl_sync(0xffffffffu, it.kb_count, 0);
    u.bn = __shfl_sync(0xffffffffu, it.bn, 0);
    return u;
}

// -------------------------------------------------------------------------------------
// the kernel

// SPLIT: 0 for configurations without K slices (split_k == 1, no tail cut along K), 1 for slices summed through the
// global workspace, 2 for slices summed inside a cluster, 3 for the stream-K tail (pieces of a tile parked in the
// workspace and added by the CTA that finishes the tile); each instantiation carries only its own reduction, which
// saves registers and shortens the start-up of every call.
// PLAIN: the instantiation for the plain call -- C = A B^T with fp32 accumulators, K-contiguous B, rows of C that are
// multiples of 16 bytes, whole-width tail tiles: all of those branches are compiled out.
// SUBS: 1 or 2 fixes the stage width (64 or 128 columns of K) at compile time, so that the producer's and the MMA
// issuer's loops over the 64-wide sub-tiles of a stage unroll (1-4 % on small and mid-size shapes); 0 reads it from the
// parameters.  The plain instantiations exist for both widths, the others use 0.
// TRACE: the instantiation that carries the instrumentation (trace stamps, per-role cycle counters, the skip mask);
// compiled in but switched off it cost 10-15 % on small and mid-size shapes, so it only runs when one of them is set.
// WIDE_STORE: the instantiation for HGEMM_EPILOGUE_TMA_WIDE (whole tiles leave through 32 x 64 store boxes and the
// store staging is 64 KB); the other one is the code for every other configuration, unchanged by the wide path.
// XPOSE: the instantiations that store the tile transposed (KernelParams::transposed, the swapped-operand
// configurations); kept out of all the others, where its store paths cost registers the widest reductions do not have.
// DUAL (CTA pairs only, block_n == 512): one work item is a 256 x 512 tile held in BOTH accumulators at once -- every
// 16-wide K step issues two MMAs (N = 256 each) that read the same A sub-tile -- so each CTA fetches 128 rows of A and
// 256 rows of B per k-block for 128 x 512 results: a quarter less shared-memory fill per flop than the 256 x 256 pair
// tile, which is what bounds the large shapes when L2 cannot feed 64 B/clk to every SM.  There is no spare accumulator;
// the epilogue overlaps the MMAs by staggering the two halves instead (see the MMA issuer).  Each CTA
// loads 256 CONSECUTIVE rows of B (one box); MMA h (h = 0, 1) takes rows 128 h .. 128 h + 127 of both CTAs' boxes, so
// accumulator column t holds column  256 * ((t % 256) / 128) + 128 * (t / 256) + t % 128  of the tile.
template <int CTA_GROUP, bool WIDE_STORE = false, int SPLIT = 1, bool PLAIN = false, bool TRACE = !PLAIN, int SUBS = 0, bool XPOSE = false,
          bool DUAL = false>
__global__ void __launch_bounds__(kThreads, 1)
hgemm_umma_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                  const __grid_constant__ CUtensorMap tmap_c, const __grid_constant__ CUtensorMap tmap_bt, const KernelParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_addr(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - smem_addr(smem_raw));

    const int32_t b_rows = p.block_n / CTA_GROUP;            // B rows this CTA stages per k-block
    const int32_t subs = SUBS != 0 ? SUBS : p.block_k / kSubK;   // 64-wide sub-tiles per stage (1 or 2)
    const uint32_t b_sub_bytes = static_cast<uint32_t>(b_rows) * kSubK * 2;
    const uint32_t a_stage_bytes = static_cast<uint32_t>(subs) * kATileBytes;
    const uint32_t stage_bytes = a_stage_bytes + static_cast<uint32_t>(subs) * b_sub_bytes;   // [A sub-tiles | B sub-tiles]
    const uint32_t staging_base = smem_base + static_cast<uint32_t>(p.stages) * stage_bytes;
    constexpr uint32_t staging_per_warp = WIDE_STORE ? 2u * kWideBoxBytes : static_cast<uint32_t>(kStagingBytesPerWarp);
    const uint32_t ctrl_base = staging_base + 8u * staging_per_warp;
    uint8_t *ctrl_gen = smem_gen + (ctrl_base - smem_base);

    // control block: full[12] | empty[12] | tmem_full[2] | tmem_empty[2] | tmem base | abort | recv
    const uint32_t bar_full = ctrl_base;
    const uint32_t bar_empty = ctrl_base + 8 * kMaxStages;
    const uint32_t bar_tmem_full = ctrl_base + 16 * kMaxStages;
    const uint32_t bar_tmem_empty = bar_tmem_full + 16;
    volatile uint32_t *tmem_base_slot = reinterpret_cast<volatile uint32_t *>(ctrl_gen + 16 * kMaxStages + 32);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(ctrl_gen + 16 * kMaxStages + 36);
    const uint32_t bar_recv = ctrl_base + 16 * kMaxStages + 40;   // cluster split-K: bytes received from the other slices

    // the warp index through a shuffle: a value the compiler knows to be warp-uniform
    const uint32_t warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0);
    const uint32_t lane = lane_id();
    // A pair is two CTAs whose ranks in the cluster differ in the last bit (cluster split-K puts several pairs
    // in one cluster); cta_rank is the CTA's place in its pair, leader_rank the cluster rank of the pair's leader.
    const uint32_t cluster_rank = (CTA_GROUP == 2) ? cluster_ctarank() : 0u;
    const uint32_t cta_rank = cluster_rank & 1u;
    const uint32_t leader_rank = cluster_rank & ~1u;
    const bool is_leader = (cta_rank == 0);
    const int32_t unit = (CTA_GROUP == 2) ? static_cast<int32_t>(blockIdx.x >> 1) : static_cast<int32_t>(blockIdx.x);
    const int32_t num_units = (CTA_GROUP == 2) ? static_cast<int32_t>(gridDim.x >> 1) : static_cast<int32_t>(gridDim.x);
    constexpr int32_t kBlockMTotal = kBlockM * CTA_GROUP;

    WaitCtl ctl{abort_flag, p.status, p.wait_budget};

    // ---- set-up -----------------------------------------------------------------------
    // Programmatic dependent launch: the next kernel in the stream may become resident (on SMs this
    // grid does not occupy, or as its CTAs retire) and run its own set-up while this grid works.
    // No thread touches global memory before its own grid_dependency_wait() has returned, so a dependent
    // launch never sees or disturbs the data of the kernel before it: the producer waits just before its
    // first load (its first work item is decoded and its first stage claimed by then), the epilogue warps
    // before their loop, the MMA warp -- which reads and writes only shared and tensor memory -- only when
    // it has trace stamps to write.
    grid_launch_dependents();
    if (threadIdx.x == 0) {
        *abort_flag = 0u;
        for (int s = 0; s < p.stages; ++s) {
            mbar_init(bar_full + 8 * s, CTA_GROUP);   // one arrive.expect_tx per CTA of the pair
            mbar_init(bar_empty + 8 * s, 1);          // one tcgen05.commit
        }
        for (int a = 0; a < 2; ++a) {
            mbar_init(bar_tmem_full + 8 * a, 1);              // one tcgen05.commit
            mbar_init(bar_tmem_empty + 8 * a, 8 * CTA_GROUP); // one arrive per epilogue warp (of both CTAs)
        }
        mbar_init(bar_recv, 1);                               // one arrive.expect_tx
        fence_mbar_init();
        prefetch_tensormap(&tmap_a);
        prefetch_tensormap(&tmap_b);
        if ((!PLAIN && p.tail_pieces > 1)) prefetch_tensormap(&tmap_bt);
        prefetch_tensormap(&tmap_c);
    }
    if (warp == 1) {
        tmem_alloc<CTA_GROUP>(smem_addr(const_cast<uint32_t *>(tmem_base_slot)), static_cast<uint32_t>(p.tmem_cols));
        // No tcgen05.relinquish_alloc_permit: it exists to let ANOTHER CTA on this SM allocate, and this kernel asks for
        // all of the SM's shared memory, so there is none; the instruction measured 0.3 us in an otherwise empty kernel.
    }
    tc_fence_before_sync();
    __syncthreads();
    if constexpr (CTA_GROUP == 2) {   // the peer's barriers must exist before anything signals them
        cluster_arrive();
        cluster_wait();
    }
    tc_fence_after_sync();
    // broadcast through a shuffle so that the compiler knows the address is warp-uniform
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_base_slot, 0);

    // ---- roles ------------------------------------------------------------------------
    // Producer and MMA loops are executed by their whole warp with warp-uniform control flow (the
    // wait results are voted), and the single-thread instructions elect their lane inside the asm block:
    // TMA and tcgen05 instructions take their operands from uniform registers, so operands the
    // compiler can prove warp-uniform cost nothing to issue, while per-thread ones each need a move.
    bool tmem_freed = false;                       // warp 1: tensor memory was freed before the teardown
    int32_t cs_m0 = 0, cs_n0 = 0, cs_slice = 0;   // cluster split-K: the epilogue warps' one work item, kept for the exchange
    if (warp == 0) {
        // ===== TMA producer =====
        int s = 0;
        uint32_t ph = 0;
        const uint32_t full_leader = (CTA_GROUP == 2) ? mapa(bar_full, leader_rank) : bar_full;
        const bool tr = (TRACE && p.trace != nullptr) && blockIdx.x == 0;
        long long t_wait = 0, t_work = 0;
        bool ok = true;
        bool dependencies_met = false;
        // One stage's loads of the plain K-contiguous path, split by operand (for the early loads below): `expect` arms
        // the stage's barrier with the bytes of BOTH operands, whichever part comes first.
        auto issue_part = [&](int32_t js, int32_t jk0, int32_t a_row, int32_t b_row, bool expect, bool do_a, bool do_b) {
            const uint32_t a_dst = smem_base + static_cast<uint32_t>(js) * stage_bytes;
            const uint32_t b_dst = a_dst + a_stage_bytes;
            const uint32_t fb = full_leader + 8 * js;
            if (expect) {
                if constexpr (CTA_GROUP == 1) mbar_arrive_expect_tx_elect(bar_full + 8 * js, stage_bytes);
                else if (is_leader) mbar_arrive_expect_tx_elect(bar_full + 8 * js, stage_bytes);
                else mbar_arrive_expect_tx_cluster_relaxed_elect(fb, stage_bytes);
            }
            if (p.tma_3d) {
                if constexpr (CTA_GROUP == 1) {
                    if (do_a) tma_load_3d_elect(a_dst, &tmap_a, 0, a_row, jk0 / kSubK, fb);
                    if (do_b) tma_load_3d_elect(b_dst, &tmap_b, 0, b_row, jk0 / kSubK, fb);
                } else {
                    if (do_a) tma_load_3d_pair_elect(a_dst, &tmap_a, 0, a_row, jk0 / kSubK, fb);
                    if (do_b) tma_load_3d_pair_elect(b_dst, &tmap_b, 0, b_row, jk0 / kSubK, fb);
                }
            } else {
                for (int32_t sub = 0; sub < subs; ++sub) {
                    if constexpr (CTA_GROUP == 1) {
                        if (do_a) tma_load_2d_elect(a_dst + sub * kATileBytes, &tmap_a, jk0 + sub * kSubK, a_row, fb);
                        if (do_b) tma_load_2d_elect(b_dst + sub * b_sub_bytes, &tmap_b, jk0 + sub * kSubK, b_row, fb);
                    } else {
                        if (do_a) tma_load_2d_pair_elect(a_dst + sub * kATileBytes, &tmap_a, jk0 + sub * kSubK, a_row, fb);
                        if (do_b) tma_load_2d_pair_elect(b_dst + sub * b_sub_bytes, &tmap_b, jk0 + sub * kSubK, b_row, fb);
                    }
                }
            }
        };
        int32_t round = 0;
        for (int32_t w = unit; ok && w < p.total_work; w += num_units, ++round) {
            const WorkItem it = warp_uniform(decode_work<SPLIT != 0, PLAIN>(w, p, kBlockMTotal));
            if (SPLIT == 0 && p.wave_pace && round > 0) {
                // Wave pacing.  The CTAs that share an operand panel in a wave find each other's lines in L2 only while
                // they walk K in step; over many equal tiles they drift apart (whoever gets its operands late stays
                // late), and the panels are fetched from HBM again and again: 12288^3 read 7.2 GB, twelve times its
                // operands.  Holding every producer at the start of a tile until all have issued the previous tile's
                // loads keeps them in step: 2.8 GB, and the launch 8 % shorter.  Nothing depends on the wait, so it
                // gives up after 50 us instead of raising the abort flag.
                if (lane == 0) {
                    const uint32_t target = p.wave_base + static_cast<uint32_t>(round) * static_cast<uint32_t>(num_units);
                    const long long t0 = clock64();
                    while (true) {
                        uint32_t seen;
                        asm volatile("ld.relaxed.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(p.wave_counter) : "memory");
                        if (static_cast<int32_t>(seen - target) >= 0 || clock64() - t0 > 100000) break;
                        __nanosleep(64);
                    }
                }
                __syncwarp();
            }
            if (HGEMM_CHECKED && !checked(p.status, it.tile >= 0 && it.tile < p.tiles_m * p.tiles_n && it.m0 >= 0 && it.m0 < p.M && it.n0 >= 0 &&
                                                        it.n0 < p.tiles_n * p.block_n && it.kb_begin >= 0 && it.kb_count >= 0 && it.kb_begin + it.kb_count <= p.kblocks &&
                                                        it.slice >= 0 && it.slice < it.slices, kCheckWorkItem))
                break;                                         // (the other roles then run into their bounded waits)
            const int32_t a_row = it.m0 + static_cast<int32_t>(cta_rank) * kBlockM;
            // this CTA's rows of B: its share of the work item's columns
            const int32_t b_row = it.n0 + static_cast<int32_t>(cta_rank) * (it.bn / CTA_GROUP);
            for (int32_t kb = 0; kb < it.kb_count; ++kb) {
                const long long c0 = tr ? clock64() : 0;
                ok = mbar_wait(bar_empty + 8 * s, ph ^ 1u, ctl, status_code(kRoleProducer, 0, s));
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                const long long c1 = tr ? clock64() : 0;
                const uint32_t a_dst = smem_base + static_cast<uint32_t>(s) * stage_bytes;
                const uint32_t b_dst = a_dst + a_stage_bytes;
                const int32_t k0 = (it.kb_begin + kb) * p.block_k;
                if (HGEMM_CHECKED && !checked(p.status, (k0 & 7) == 0 && k0 >= 0 && k0 < p.kblocks * p.block_k && a_row >= 0 && b_row >= 0 && s >= 0 &&
                                                            s < p.stages, kCheckLoadCoord)) {
                    ok = false;
                    break;
                }
                const uint32_t fb = full_leader + 8 * s;      // the (leader's) full barrier of this stage
                if (!dependencies_met) {
                    // Operands the caller declared static (KernelParams::early_ops: no kernel ahead of this call in the
                    // stream writes them) may be fetched BEFORE the stream dependency is resolved: the first pass of the
                    // ring -- every stage is free -- is armed and that operand's loads go out now, the other operand's
                    // after the wait.  A projection's weights then stream in while the previous kernel drains.
                    int32_t pre = 0;
                    if (p.early_ops != 0u && !(TRACE && (p.debug_skip & 1u)) && !(!PLAIN && (p.b_row_major || it.bn != p.block_n))) {
                        pre = min(it.kb_count, p.stages);
                        for (int32_t j = 0; j < pre; ++j)
                            issue_part(j, (it.kb_begin + j) * p.block_k, a_row, b_row, true, (p.early_ops & 1u) != 0u, (p.early_ops & 2u) != 0u);
                    }
                    grid_dependency_wait();                   // the kernels before this one are complete: global memory may be read
                    dependencies_met = true;
                    if (threadIdx.x == 0) {
                        trace_stamp<!TRACE>(p, 0);
                        trace_stamp<!TRACE>(p, 1);
                    }
                    if (pre > 0) {
                        for (int32_t j = 0; j < pre; ++j)
                            issue_part(j, (it.kb_begin + j) * p.block_k, a_row, b_row, false, (p.early_ops & 1u) == 0u, (p.early_ops & 2u) == 0u);
                        if (lane == 0) trace_stamp<!TRACE>(p, 2);
                        if (pre == p.stages) { s = 0; ph ^= 1u; } else { s = pre; }
                        kb = pre - 1;                          // the loop's increment moves on to the first k-block not yet issued
                        continue;
                    }
                }
                if ((TRACE ? p.debug_skip : 0u) & 1u) {
                    if (lane == 0) {
                        if (is_leader) mbar_arrive(bar_full + 8 * s);
                        else mbar_arrive_cluster(fb);
                    }
                } else if ((!PLAIN && p.b_row_major)) {
                    // B is K x N row-major: per 64-wide K sub-tile, one {64 columns, 64 k-rows} box per 64-column block
                    const int32_t b_col = it.n0 + static_cast<int32_t>(cta_rank) * (it.bn / CTA_GROUP);
                    const int32_t blocks = (it.bn / CTA_GROUP) / 64;       // a column piece of a tail tile loads fewer blocks
                    const uint32_t tx = a_stage_bytes + static_cast<uint32_t>(subs * blocks) * (kSubK * 128u);
                    if constexpr (CTA_GROUP == 1) mbar_arrive_expect_tx_elect(bar_full + 8 * s, tx);
                    else if (is_leader) mbar_arrive_expect_tx_elect(bar_full + 8 * s, tx);
                    else mbar_arrive_expect_tx_cluster_relaxed_elect(fb, tx);
                    for (int32_t sub = 0; sub < subs; ++sub) {
                        if constexpr (CTA_GROUP == 1) tma_load_2d_elect(a_dst + sub * kATileBytes, &tmap_a, k0 + sub * kSubK, a_row, fb);
                        else tma_load_2d_pair_elect(a_dst + sub * kATileBytes, &tmap_a, k0 + sub * kSubK, a_row, fb);
                        for (int32_t nb = 0; nb < blocks; ++nb) {
                            const uint32_t dst = b_dst + sub * b_sub_bytes + nb * (kSubK * 128);
                            if constexpr (CTA_GROUP == 1) tma_load_2d_elect(dst, &tmap_b, b_col + nb * 64, k0 + sub * kSubK, fb);
                            else tma_load_2d_pair_elect(dst, &tmap_b, b_col + nb * 64, k0 + sub * kSubK, fb);
                        }
                    }
                } else if ((!PLAIN && it.bn != p.block_n)) {
                    // a column piece of a tail tile: its rows of B come through the narrower map `tmap_bt`, one box per
                    // 64-wide K sub-tile, each placed where the full-height box of that sub-tile would start
                    const uint32_t tx = a_stage_bytes + static_cast<uint32_t>(subs * (it.bn / CTA_GROUP)) * (kSubK * 2u);
                    if constexpr (CTA_GROUP == 1) mbar_arrive_expect_tx_elect(bar_full + 8 * s, tx);
                    else if (is_leader) mbar_arrive_expect_tx_elect(bar_full + 8 * s, tx);
                    else mbar_arrive_expect_tx_cluster_relaxed_elect(fb, tx);
                    if (p.tma_3d) {
                        if constexpr (CTA_GROUP == 1) tma_load_3d_elect(a_dst, &tmap_a, 0, a_row, k0 / kSubK, fb);
                        else tma_load_3d_pair_elect(a_dst, &tmap_a, 0, a_row, k0 / kSubK, fb);
                    }
                    for (int32_t sub = 0; sub < subs; ++sub) {
                        if constexpr (CTA_GROUP == 1) {
                            if (!p.tma_3d) tma_load_2d_elect(a_dst + sub * kATileBytes, &tmap_a, k0 + sub * kSubK, a_row, fb);
                            tma_load_2d_elect(b_dst + sub * b_sub_bytes, &tmap_bt, k0 + sub * kSubK, b_row, fb);
                        } else {
                            if (!p.tma_3d) tma_load_2d_pair_elect(a_dst + sub * kATileBytes, &tmap_a, k0 + sub * kSubK, a_row, fb);
                            tma_load_2d_pair_elect(b_dst + sub * b_sub_bytes, &tmap_bt, k0 + sub * kSubK, b_row, fb);
                        }
                    }
                } else if (p.tma_3d) {
                    // one instruction per operand: dimension 2 of the map counts 64-wide K sub-tiles
                    const int32_t ksub = k0 / kSubK;
                    if constexpr (CTA_GROUP == 1) {
                        mbar_arrive_expect_tx_elect(bar_full + 8 * s, stage_bytes);
                        tma_load_3d_elect(a_dst, &tmap_a, 0, a_row, ksub, bar_full + 8 * s);
                        tma_load_3d_elect(b_dst, &tmap_b, 0, b_row, ksub, bar_full + 8 * s);
                    } else {
                        if (is_leader) mbar_arrive_expect_tx_elect(bar_full + 8 * s, stage_bytes);
                        else mbar_arrive_expect_tx_cluster_relaxed_elect(fb, stage_bytes);
                        tma_load_3d_pair_elect(a_dst, &tmap_a, 0, a_row, ksub, fb);
                        tma_load_3d_pair_elect(b_dst, &tmap_b, 0, b_row, ksub, fb);
                    }
                } else if constexpr (CTA_GROUP == 1) {
                    mbar_arrive_expect_tx_elect(bar_full + 8 * s, stage_bytes);
                    for (int32_t sub = 0; sub < subs; ++sub) {
                        tma_load_2d_elect(a_dst + sub * kATileBytes, &tmap_a, k0 + sub * kSubK, a_row, bar_full + 8 * s);
                        tma_load_2d_elect(b_dst + sub * b_sub_bytes, &tmap_b, k0 + sub * kSubK, b_row, bar_full + 8 * s);
                    }
                } else {
                    // both CTAs of the pair announce their bytes on the leader's barrier; the peer's
                    // remote arrive is relaxed (it orders nothing: the data arrives through TMA)
                    if (is_leader) mbar_arrive_expect_tx_elect(bar_full + 8 * s, stage_bytes);
                    else mbar_arrive_expect_tx_cluster_relaxed_elect(fb, stage_bytes);
                    for (int32_t sub = 0; sub < subs; ++sub) {
                        tma_load_2d_pair_elect(a_dst + sub * kATileBytes, &tmap_a, k0 + sub * kSubK, a_row, fb);
                        tma_load_2d_pair_elect(b_dst + sub * b_sub_bytes, &tmap_b, k0 + sub * kSubK, b_row, fb);
                    }
                }
                if (w == unit && kb == 0 && lane == 0) trace_stamp<!TRACE>(p, 2);
                if (tr) { t_wait += c1 - c0; t_work += clock64() - c1; }
                if (++s == p.stages) { s = 0; ph ^= 1u; }
            }
            // (one arrival per CTA or pair and tile; dependencies_met: the loop above ran, so the stream dependency is resolved)
            if (SPLIT == 0 && p.wave_pace && is_leader && lane == 0 && dependencies_met) atomicAdd(p.wave_counter, 1u);
        }
        if (SPLIT == 0 && p.wave_pace && is_leader && lane == 0 && dependencies_met)
            for (; round < p.wave_rounds; ++round) atomicAdd(p.wave_counter, 1u);       // the rounds this CTA sits out
        if (tr && lane == 0) { p.trace[11] = t_wait; p.trace[12] = t_work; }
    } else if (warp == 1) {
        if ((TRACE && p.trace != nullptr)) grid_dependency_wait();   // this warp's only global accesses are trace stamps
        if (is_leader) {
            // ===== MMA issuer =====
            int s = 0;
            uint32_t ph = 0;
            uint32_t local_tile = 0;
            const bool tr = (TRACE && p.trace != nullptr) && blockIdx.x == 0;
            long long t_wait = 0, t_issue = 0, t_commit = 0, t_acc = 0, n_kb = 0;
            const uint64_t desc_a0 = make_smem_desc_sw128(smem_base);
            // B tile: K-major (B stored N x K) or N-major in 64-column blocks of 64 k-rows (B stored K x N)
            const uint64_t desc_b0 = (!PLAIN && p.b_row_major) ? make_smem_desc_sw128_mn_major(smem_base + a_stage_bytes, kSubK * 128u)
                                                   : make_smem_desc_sw128(smem_base + a_stage_bytes);
            // advancing K by 16: +32 bytes inside a K-major swizzle row, +16 k-rows (2048 bytes) in an N-major tile
            const uint32_t b_kstep = (!PLAIN && p.b_row_major) ? (16u * 128u) >> 4 : 2u;
            const uint32_t desc_stage_step = stage_bytes >> 4;
            const bool issue_mma = !((TRACE ? p.debug_skip : 0u) & 2u);
            bool ok = true;
            for (int32_t w = unit; ok && w < p.total_work; w += num_units, ++local_tile) {
                const WorkItem it = warp_uniform(decode_work<SPLIT != 0, PLAIN>(w, p, kBlockMTotal));
                if (SPLIT == 3 && it.kb_count <= 0) {      // a stream-K position without this item: it takes no accumulator
                    --local_tile;                          // (the loop's increment puts it back)
                    continue;
                }
                const uint32_t acc = DUAL ? 0u : (local_tile & 1u);            // DUAL: one work item fills both accumulators
                const uint32_t acc_ph = DUAL ? (local_tile & 1u) : ((local_tile >> 1) & 1u);
                if constexpr (DUAL) {
                    // ---- the 256 x 512 tile: accumulator h (columns 256 h ..) takes rows 128 h .. of both CTAs' B boxes ----
                    // There is no spare accumulator, so the hand-off to the epilogue is staggered between the halves
                    // instead: at the head of a tile the first `stages` k-blocks go into accumulator 0 as soon as the
                    // epilogue has drained it -- while it still drains accumulator 1 -- and only then into accumulator 1;
                    // at the tail the last `stages` k-blocks finish accumulator 0 first, so that its epilogue runs under
                    // accumulator 1's last MMAs.  A stage is freed by the MMAs of its second half.  In between both
                    // halves take each k-block in turn.  (Tiles with fewer than 2 * stages k-blocks are not staggered.)
                    const int32_t S = p.stages, kbc = it.kb_count;
                    auto acc_free = [&](uint32_t h) {
                        ok = mbar_wait(bar_tmem_empty + 8 * h, acc_ph ^ 1u, ctl, status_code(kRoleMma, 1, h));
                        ok = __all_sync(0xffffffffu, ok);
                        if (ok) tc_fence_after_sync();
                    };
                    auto stage_full = [&](int32_t st, uint32_t par) {
                        ok = mbar_wait(bar_full + 8 * st, par, ctl, status_code(kRoleMma, 0, st));
                        ok = __all_sync(0xffffffffu, ok);
                        if (ok) tc_fence_after_sync();
                    };
                    auto issue_half = [&](int32_t st, uint32_t h, bool overwrite) {
                        const uint64_t a_desc = desc_a0 + static_cast<uint64_t>(static_cast<uint32_t>(st) * desc_stage_step);
                        const uint64_t b_desc = desc_b0 + static_cast<uint64_t>(static_cast<uint32_t>(st) * desc_stage_step) +
                                                static_cast<uint64_t>(h * ((128u * 128u) >> 4));
                        for (int32_t sub = 0; sub < subs; ++sub) {
                            const uint64_t a_sub = a_desc + static_cast<uint64_t>(static_cast<uint32_t>(sub) * (kATileBytes >> 4));
                            const uint64_t b_sub = b_desc + static_cast<uint64_t>(static_cast<uint32_t>(sub) * (b_sub_bytes >> 4));
#pragma unroll
                            for (int k = 0; k < kSubK / kUmmaK; ++k)
                                umma_f16_elect<CTA_GROUP>(tmem_base + h * 256u, a_sub + 2u * k, b_sub + 2u * k, p.idesc,
                                                       (overwrite && (sub | k) == 0) ? 0u : 1u);
                        }
                    };
                    auto advance = [&]() { if (++s == S) { s = 0; ph ^= 1u; } };
                    if (kbc < 2 * S) {
                        acc_free(0);
                        if (ok) acc_free(1);
                        for (int32_t kb = 0; ok && kb < kbc; ++kb) {
                            stage_full(s, ph);
                            if (!ok) break;
                            issue_half(s, 0, kb == 0);
                            issue_half(s, 1, kb == 0);
                            umma_commit_elect<CTA_GROUP>(bar_empty + 8 * s, leader_rank);
                            advance();
                        }
                        if (!ok) break;
                        umma_commit_elect<CTA_GROUP>(bar_tmem_full, leader_rank);
                        umma_commit_elect<CTA_GROUP>(bar_tmem_full + 8, leader_rank);
                    } else {
                        // head
                        acc_free(0);
                        const int s_head = s;
                        const uint32_t ph_head = ph;
                        for (int32_t j = 0; ok && j < S; ++j) {
                            stage_full(s, ph);
                            if (!ok) break;
                            issue_half(s, 0, j == 0);
                            advance();
                        }
                        if (ok) acc_free(1);
                        if (!ok) break;
                        s = s_head;
                        ph = ph_head;
                        for (int32_t j = 0; j < S; ++j) {
                            issue_half(s, 1, j == 0);
                            umma_commit_elect<CTA_GROUP>(bar_empty + 8 * s, leader_rank);
                            advance();
                        }
                        // middle
                        for (int32_t kb = S; ok && kb < kbc - S; ++kb) {
                            stage_full(s, ph);
                            if (!ok) break;
                            issue_half(s, 0, false);
                            issue_half(s, 1, false);
                            umma_commit_elect<CTA_GROUP>(bar_empty + 8 * s, leader_rank);
                            advance();
                        }
                        if (!ok) break;
                        // tail
                        const int s_tail = s;
                        const uint32_t ph_tail = ph;
                        for (int32_t j = 0; ok && j < S; ++j) {
                            stage_full(s, ph);
                            if (!ok) break;
                            issue_half(s, 0, false);
                            advance();
                        }
                        if (!ok) break;
                        umma_commit_elect<CTA_GROUP>(bar_tmem_full, leader_rank);
                        s = s_tail;
                        ph = ph_tail;
                        for (int32_t j = 0; j < S; ++j) {
                            issue_half(s, 1, false);
                            umma_commit_elect<CTA_GROUP>(bar_empty + 8 * s, leader_rank);
                            advance();
                        }
                        umma_commit_elect<CTA_GROUP>(bar_tmem_full + 8, leader_rank);
                    }
                    continue;
                }
                const long long ca = tr ? clock64() : 0;
                ok = mbar_wait(bar_tmem_empty + 8 * acc, acc_ph ^ 1u, ctl, status_code(kRoleMma, 1, acc));
                ok = __all_sync(0xffffffffu, ok);
                if (tr) t_acc += clock64() - ca;
                if (!ok) break;
                tc_fence_after_sync();
                const uint32_t d_tmem = tmem_base + acc * static_cast<uint32_t>(p.block_n);
                // The instruction descriptor's N field follows the work item's width: p.idesc for whole tiles,
                // p.idesc_tail for the column pieces of tail tiles.  Both are kernel parameters on purpose: a
                // descriptor computed at run time cost every MMA about 25 more cycles to issue than one that the
                // instruction takes straight from the parameter bank, so the k-block loop exists once per descriptor.
                auto run_k_blocks = [&](const uint32_t idesc) {
                for (int32_t kb = 0; kb < it.kb_count; ++kb) {
                    const long long c0 = tr ? clock64() : 0;
                    ok = mbar_wait(bar_full + 8 * s, ph, ctl, status_code(kRoleMma, 0, s));
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    const long long c1 = tr ? clock64() : 0;
                    tc_fence_after_sync();
                    const uint64_t a_desc = desc_a0 + static_cast<uint64_t>(static_cast<uint32_t>(s) * desc_stage_step);
                    const uint64_t b_desc = desc_b0 + static_cast<uint64_t>(static_cast<uint32_t>(s) * desc_stage_step);
                    if (w == unit && kb == 0 && lane == 0) trace_stamp<!TRACE>(p, 3);
                    if (issue_mma) {
                        for (int32_t sub = 0; sub < subs; ++sub) {
                            const uint64_t a_sub = a_desc + static_cast<uint64_t>(static_cast<uint32_t>(sub) * (kATileBytes >> 4));
                            const uint64_t b_sub = b_desc + static_cast<uint64_t>(static_cast<uint32_t>(sub) * (b_sub_bytes >> 4));
#pragma unroll
                            for (int k = 0; k < kSubK / kUmmaK; ++k) {
                                // advancing K by 16 fp16 inside the swizzle span = +32 bytes = +2 in the address field
                                umma_f16_elect<CTA_GROUP>(d_tmem, a_sub + 2u * k, b_sub + b_kstep * k, idesc,
                                                       (kb | sub | k) != 0 ? 1u : 0u);
                            }
                        }
                    }
                    const long long c2 = tr ? clock64() : 0;
                    // free the stage (in both CTAs of a pair) once these MMAs have read it
                    umma_commit_elect<CTA_GROUP>(bar_empty + 8 * s, leader_rank);
                    if (tr) { t_wait += c1 - c0; t_issue += c2 - c1; t_commit += clock64() - c2; ++n_kb; }
                    if (++s == p.stages) { s = 0; ph ^= 1u; }
                }
                };
                if (PLAIN || it.bn == p.block_n) run_k_blocks(p.idesc);      // no column pieces in the plain instantiations
                else run_k_blocks(p.idesc_tail);
                if (!ok) break;
                if (w == unit && lane == 0) trace_stamp<!TRACE>(p, 4);
                umma_commit_elect<CTA_GROUP>(bar_tmem_full + 8 * acc, leader_rank);
            }
            if (tr && lane == 0) { p.trace[8] = t_wait; p.trace[9] = t_issue; p.trace[10] = t_commit; p.trace[13] = t_acc; p.trace[15] = n_kb; }
            if constexpr (CTA_GROUP == 1) {
                // Free tensor memory as soon as the epilogue has read the last of it -- each accumulator's last
                // use has been released -- instead of after the CTA-wide barrier of the teardown: the epilogue's
                // final stores then overlap the deallocation.  (Not for cluster split-K, which reads tensor
                // memory after the role loops, and not after an abort.)
                if (ok && SPLIT != 2) {
                    for (uint32_t a = 0; ok && a < 2u; ++a) {
                        const uint32_t uses = (local_tile + 1u - a) / 2u;      // work items that used accumulator a (local_tile items in all)
                        if (local_tile > a && uses > 0u) {
                            ok = mbar_wait(bar_tmem_empty + 8 * a, (uses - 1u) & 1u, ctl, status_code(kRoleMma, 2, a));
                            ok = __all_sync(0xffffffffu, ok);
                        }
                    }
                    if (ok) {
                        tc_fence_after_sync();
                        tmem_dealloc<CTA_GROUP>(tmem_base, static_cast<uint32_t>(p.tmem_cols));
                        tmem_freed = true;
                        if (lane == 0) trace_stamp<!TRACE>(p, 7);
                    }
                }
            }
        }
    } else {
        // ===== epilogue (warps 2..9) =====
        // Two warps share each tensor-memory lane quarter (a warp may only touch lanes
        // 32 * (warp % 4) .. + 31) and take alternate 32-column chunks of the accumulator.
        const uint32_t ew = warp - 2u;                              // 0..7
        const uint32_t q = warp & 3u;                               // tensor-memory lane quarter of this warp
        const uint32_t first_chunk = ew >> 2;                       // chunks first_chunk, first_chunk + 2, ...
        const uint32_t row_in_tile = q * 32u + lane;                // accumulator row = tensor-memory lane
        const uint32_t staging = staging_base + ew * staging_per_warp;
        const uint32_t tmem_empty_leader = (CTA_GROUP == 2) ? mapa(bar_tmem_empty, leader_rank) : bar_tmem_empty;
        const int32_t chunks = p.block_n / 32;
        uint32_t local_tile = 0;
        uint32_t store_count = 0;
        bool ok = true;
        grid_dependency_wait();                            // before the first store to C, workspace or counters
        for (int32_t w = unit; ok && w < p.total_work; w += num_units, ++local_tile) {
            const WorkItem it = decode_work<SPLIT != 0, PLAIN>(w, p, kBlockMTotal);
            if (SPLIT == 3 && it.kb_count <= 0) {          // a stream-K position without this item (see the MMA issuer)
                --local_tile;
                continue;
            }
            const uint32_t acc = DUAL ? 0u : (local_tile & 1u);
            const uint32_t acc_ph = DUAL ? (local_tile & 1u) : ((local_tile >> 1) & 1u);
            // first column, within the tile, of 32-column accumulator chunk c (DUAL: see the template comment)
            auto chunk_col = [](int32_t c) -> int32_t {
                return DUAL ? ((c >> 2) & 1) * 256 + (c >> 3) * 128 + (c & 3) * 32 : c * 32;
            };
            // DUAL: the two halves of the tile become ready one after the other (see the MMA issuer): each is waited
            // for, read and released on its own below
            auto wait_accumulator = [&](uint32_t idx) {
                ok = mbar_wait(bar_tmem_full + 8 * idx, acc_ph, ctl, status_code(kRoleEpilogue, 2, idx));
                ok = __all_sync(0xffffffffu, ok);   // the warp-wide tensor-memory loads below need the whole warp
                if (ok) tc_fence_after_sync();
            };
            if constexpr (!DUAL) {
                wait_accumulator(acc);
                if (!ok) break;
            }
            if (w == unit && threadIdx.x == 64) trace_stamp<!TRACE>(p, 5);
            const int32_t row0 = it.m0 + static_cast<int32_t>(cta_rank) * kBlockM;  // first row of this CTA's 128
            const int32_t grow = row0 + static_cast<int32_t>(row_in_tile);          // this thread's global row
            const uint32_t t_addr = tmem_base + ((q * 32u) << 16) + acc * static_cast<uint32_t>(p.block_n);
            if (HGEMM_CHECKED && !checked(p.status, static_cast<int32_t>(acc) * p.block_n + (DUAL ? 512 : p.block_n) <= p.tmem_cols, kCheckTmemColumn)) {
                ok = false;
                break;
            }

            // One 32-column chunk of this thread's row, converted and sent to C.
            auto emit_chunk = [&](const uint32_t (&v)[32], int32_t c) {
                const int32_t col0 = it.n0 + chunk_col(c);
                if (XPOSE && !WIDE_STORE) {
                    // The caller's C is the transpose of what this kernel computes: this thread's 32 values are 32
                    // elements of one column of C (row col0 + j, column grow).
                    if (p.epilogue_tma) {
                        // stage the chunk transposed -- box row j holds what the 32 lanes computed for column
                        // col0 + j, 64 consecutive bytes per store instruction -- in the 64-byte swizzle the store
                        // box expects (16-byte piece t of row r lives at piece t ^ ((r >> 1) & 3)), then one TMA store
                        const uint32_t buf = staging + (store_count & 1u) * (kStagingBytesPerWarp / 2);
                        bulk_wait_group_read<1>();
                        __syncwarp();
                        const uint32_t piece = lane >> 3, within = (lane & 7u) * 2u;
#pragma unroll
                        for (uint32_t j = 0; j < 32; ++j) {
                            const __half h = __float2half_rn(__uint_as_float(v[j]));
                            st_shared_u16(buf + j * 64u + ((piece ^ ((j >> 1) & 3u)) << 4) + within, __half_as_ushort(h));
                        }
                        fence_proxy_async_smem();
                        __syncwarp();
                        const int32_t box_col = row0 + static_cast<int32_t>(q) * 32;          // first column of C in the box
                        const bool go = lane == 0 && box_col < p.M && col0 < p.N && !((TRACE ? p.debug_skip : 0u) & 4u);
                        tma_store_2d_if(go ? 1u : 0u, &tmap_c, box_col, col0, buf);
                        bulk_commit_group();
                        ++store_count;
                    } else if (grow < p.M) {
                        unsigned short *dst = reinterpret_cast<unsigned short *>(p.C) + static_cast<size_t>(col0) * p.M + grow;
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            if (col0 + j < p.N) dst[static_cast<size_t>(j) * p.M] = __half_as_ushort(__float2half_rn(__uint_as_float(v[j])));
                    }
                } else if (!WIDE_STORE && p.epilogue_tma) {
                    const uint32_t buf = staging + (store_count & 1u) * (kStagingBytesPerWarp / 2);
                    // the buffer written two stores ago must have been read by its TMA store
                    bulk_wait_group_read<1>();                      // lanes other than 0 own no groups
                    __syncwarp();
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
                    {
                        // warp-uniform code: the store is predicated inside its asm block, the commit is executed
                        // by every lane (an empty group for all but lane 0)
                        const int32_t box_row = row0 + static_cast<int32_t>(q) * 32;
                        const bool go = lane == 0 && box_row < p.M && col0 < p.N && !((TRACE ? p.debug_skip : 0u) & 4u) &&
                                        checked(p.status, (col0 & 7) == 0 && col0 >= 0 && box_row >= 0, kCheckStoreCoord);
                        tma_store_2d_if(go ? 1u : 0u, &tmap_c, col0, box_row, buf);
                        bulk_commit_group();
                    }
                    ++store_count;
                } else if ((!PLAIN && p.ragged_n)) {
                    // rows of C are not multiples of 16 bytes: neither TMA nor vector stores apply.  The chunk is
                    // transposed through the warp's staging buffer (same 64-byte swizzle as above) so that each
                    // store instruction writes 32 consecutive elements of one row instead of one element of 32 rows.
                    const uint32_t row_addr = staging + lane * 64u;
                    const uint32_t sw = (lane >> 1) & 3u;
                    __syncwarp();                                   // the previous chunk's reads of the buffer are done
#pragma unroll
                    for (uint32_t j = 0; j < 4; ++j) {
                        st_shared_v4(row_addr + ((j ^ sw) << 4),
                                     pack_half2_rn(v[8 * j + 0], v[8 * j + 1]), pack_half2_rn(v[8 * j + 2], v[8 * j + 3]),
                                     pack_half2_rn(v[8 * j + 4], v[8 * j + 5]), pack_half2_rn(v[8 * j + 6], v[8 * j + 7]));
                    }
                    __syncwarp();
                    const int32_t col = col0 + static_cast<int32_t>(lane);
                    const int32_t first_row = row0 + static_cast<int32_t>(q) * 32;
                    const int32_t rows_here = min(32, p.M - first_row);
                    if (col < p.N) {
                        unsigned short *dst = reinterpret_cast<unsigned short *>(p.C) + static_cast<size_t>(first_row) * p.N + col;
                        for (int32_t r = 0; r < rows_here; ++r) {
                            const uint32_t src = staging + static_cast<uint32_t>(r) * 64u +
                                                 (((lane >> 3) ^ ((static_cast<uint32_t>(r) >> 1) & 3u)) << 4) + (lane & 7u) * 2u;
                            dst[static_cast<size_t>(r) * p.N] = ld_shared_u16(src);
                        }
                    }
                } else if (grow < p.M) {
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
            };
            auto release_accumulator = [&](uint32_t idx) {
                tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) {
                    if constexpr (CTA_GROUP == 1) mbar_arrive(bar_tmem_empty + 8 * idx);
                    else mbar_arrive_cluster(tmem_empty_leader + 8 * idx);
                }
            };
            constexpr uint32_t kHalves = DUAL ? 2u : 1u;        // DUAL: accumulator h = chunks 8 h .. 8 h + 7 = barrier pair h

            // chunks of this tile that hold columns of C, and whether this warp's 32 rows hold rows of C:
            // tiles on the ragged edge (and every tile of a problem with M < 128) skip the dead part
            const int32_t live_chunks = min(it.bn / 32, (p.N - it.n0 + 31) / 32);
            const bool live_rows = row0 + static_cast<int32_t>(q) * 32 < p.M;
            if (WIDE_STORE && (SPLIT == 0 || it.slices == 1) && p.epilogue_tma == 2) {
                // Wide TMA stores: two 32-column chunks are staged side by side as one 32-row x 64-column box
                // (128-byte rows, 128-byte swizzle: 16-byte chunk j of row r lives at chunk j ^ (r & 7)) and leave
                // with one fence, one store and one commit.  The two warps of a lane quarter take alternate boxes.
                // A box whose second half lies beyond N is staged half empty: the store is clipped there.
                uint32_t v[32];
                const int32_t chunks = live_rows ? live_chunks : 0;     // shadows the tile's chunk count
                const int32_t all_boxes = (chunks + 1) >> 1;
                for (uint32_t hf = 0; ok && hf < kHalves; ++hf) {
                const uint32_t rel = DUAL ? hf : acc;
                if constexpr (DUAL) {
                    wait_accumulator(hf);
                    if (!ok) break;
                }
                const int32_t box_lo = DUAL ? 4 * static_cast<int32_t>(hf) : 0;
                const int32_t boxes = DUAL ? min(all_boxes, box_lo + 4) : all_boxes;
                for (int32_t b = box_lo + static_cast<int32_t>(first_chunk); b < boxes; b += 2) {
                    const uint32_t buf = staging + (store_count & 1u) * kWideBoxBytes;
                    bulk_wait_group_read<1>();                      // the box written two stores ago has been read
                    __syncwarp();
                    const uint32_t row_addr = buf + lane * 128u;
                    const uint32_t sw = lane & 7u;
#pragma unroll
                    for (int32_t half = 0; half < 2; ++half) {
                        const int32_t c = 2 * b + half;
                        if (c < chunks) {
                            tmem_ld_32x32b_x32(t_addr + static_cast<uint32_t>(c) * 32u, v);
                            tmem_ld_wait();
                            if ((!PLAIN && p.acc_f16)) {
#pragma unroll
                                for (int j = 0; j < 32; ++j)
                                    v[j] = __float_as_uint(__half2float(__ushort_as_half(static_cast<unsigned short>(v[j] & 0xffffu))));
                            }
                            if (b + 2 >= boxes && c + 1 >= min(chunks, 2 * b + 2)) release_accumulator(rel);   // this warp's last load
                            if ((!PLAIN && p.scaled) && grow < p.M) {
#pragma unroll
                                for (int j = 0; j < 4; ++j)
                                    if (it.n0 + chunk_col(c) + 8 * j < p.N) scale_group8<XPOSE>(v + 8 * j, p, grow, it.n0 + chunk_col(c) + 8 * j);
                            }
#pragma unroll
                            for (uint32_t j = 0; j < 4; ++j) {
                                st_shared_v4(row_addr + (((4u * static_cast<uint32_t>(half) + j) ^ sw) << 4),
                                             pack_half2_rn(v[8 * j + 0], v[8 * j + 1]), pack_half2_rn(v[8 * j + 2], v[8 * j + 3]),
                                             pack_half2_rn(v[8 * j + 4], v[8 * j + 5]), pack_half2_rn(v[8 * j + 6], v[8 * j + 7]));
                            }
                        }
                    }
                    fence_proxy_async_smem();
                    __syncwarp();
                    {
                        const int32_t box_row = row0 + static_cast<int32_t>(q) * 32;
                        const int32_t col0 = it.n0 + chunk_col(2 * b);
                        const bool go = lane == 0 && box_row < p.M && col0 < p.N && !((TRACE ? p.debug_skip : 0u) & 4u);
                        tma_store_2d_if(go ? 1u : 0u, &tmap_c, col0, box_row, buf);
                        bulk_commit_group();
                    }
                    ++store_count;
                }
                if (box_lo + static_cast<int32_t>(first_chunk) >= boxes) release_accumulator(rel);    // nothing to load
                }
                if (!ok) break;
            } else if (SPLIT == 0 || it.slices == 1 || (SPLIT == 3 && it.slice == 0)) {
                // one 32-column chunk at a time: a tensor-memory load takes ~100 cycles, and keeping a second
                // chunk in flight costs more in registers than it hides
                uint32_t v[32];
                const int32_t all_chunks = live_rows ? live_chunks : 0;
                // Stream-K: the piece that holds a tile's first k-block finishes the tile.  The tile's later pieces
                // belong to the positions after this one, which computed them FIRST (a position works through its
                // range in K order, so the end of the tile it starts in comes before the start of the next tile) and
                // parked them in the workspace long ago: wait for their arrivals (8 per piece, one per epilogue warp;
                // the counter is never reset, launch number e sees e times as many), then add them to this piece's
                // accumulator chunk by chunk, in K order, on the way to the ordinary stores.
                const bool add_pieces = SPLIT == 3 && it.slices > 1;
                const size_t slot_floats = static_cast<size_t>(kBlockM) * p.block_n;
                // this CTA's half of the tile's second piece (slice 1)
                const float *piece1 = p.workspace + (static_cast<size_t>(it.split_index + 1) * CTA_GROUP + cta_rank) * slot_floats;
                if (add_pieces) {
                    const uint32_t *ctr = p.counters + (static_cast<size_t>(it.tile - p.first_split_tile) * CTA_GROUP + cta_rank) * 2;
                    const uint32_t target = p.epoch * 8u * static_cast<uint32_t>(it.slices - 1);
                    if (lane == 0) {
                        const long long t0 = clock64();
                        while (true) {
                            uint32_t seen;
                            asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(ctr) : "memory");
                            if (static_cast<int32_t>(seen - target) >= 0) break;
                            if (*abort_flag) { ok = false; break; }
                            if (clock64() - t0 > p.wait_budget) {
                                *abort_flag = 1u;
                                atomicCAS(p.status, 0u, status_code(kRoleEpilogue, 3, it.slice));
                                ok = false;
                                break;
                            }
                            __nanosleep(40);
                        }
                    }
                    ok = __all_sync(0xffffffffu, ok);
                    if (!ok) break;
                    __threadfence();
                }
                for (uint32_t hf = 0; ok && hf < kHalves; ++hf) {
                const uint32_t rel = DUAL ? hf : acc;
                if constexpr (DUAL) {
                    wait_accumulator(hf);
                    if (!ok) break;
                }
                const int32_t chunk_lo = DUAL ? 8 * static_cast<int32_t>(hf) : 0;
                const int32_t chunks = DUAL ? min(all_chunks, chunk_lo + 8) : all_chunks;     // shadows the tile's chunk count
                for (int32_t c = chunk_lo + static_cast<int32_t>(first_chunk); c < chunks; c += 2) {
                    tmem_ld_32x32b_x32(t_addr + static_cast<uint32_t>(c) * 32u, v);
                    tmem_ld_wait();
                    if ((!PLAIN && p.acc_f16)) {
                        // fp16 accumulators (measured layout: one result per 32-bit column, in its low half):
                        // widen them, exactly, so that the store paths below see what they see with fp32 ones
#pragma unroll
                        for (int j = 0; j < 32; ++j)
                            v[j] = __float_as_uint(__half2float(__ushort_as_half(static_cast<unsigned short>(v[j] & 0xffffu))));
                    }
                    if (c + 2 >= chunks) release_accumulator(rel);    // every load of this warp (from this accumulator) has completed
                    if (add_pieces) {
                        // this thread's row of the chunk in every later piece (layout: see the parking below)
                        const float4 *src = reinterpret_cast<const float4 *>(piece1) + static_cast<size_t>(c) * 8 * kBlockM + row_in_tile;
                        for (int32_t sl = 1; sl < it.slices; ++sl, src += static_cast<size_t>(CTA_GROUP) * slot_floats / 4) {
                            float4 x[8];
#pragma unroll
                            for (int g = 0; g < 8; ++g) x[g] = __ldcg(src + g * kBlockM);
#pragma unroll
                            for (int g = 0; g < 8; ++g) {
                                v[4 * g + 0] = __float_as_uint(__uint_as_float(v[4 * g + 0]) + x[g].x);
                                v[4 * g + 1] = __float_as_uint(__uint_as_float(v[4 * g + 1]) + x[g].y);
                                v[4 * g + 2] = __float_as_uint(__uint_as_float(v[4 * g + 2]) + x[g].z);
                                v[4 * g + 3] = __float_as_uint(__uint_as_float(v[4 * g + 3]) + x[g].w);
                            }
                        }
                    }
                    if ((!PLAIN && p.scaled) && grow < p.M) {
#pragma unroll
                        for (int j = 0; j < 4; ++j)
                            if (it.n0 + chunk_col(c) + 8 * j < p.N) scale_group8<XPOSE>(v + 8 * j, p, grow, it.n0 + chunk_col(c) + 8 * j);
                    }
                    emit_chunk(v, c);
                }
                if (chunk_lo + static_cast<int32_t>(first_chunk) >= chunks) release_accumulator(rel);   // nothing to load
                }
                if (!ok) break;
            } else if (SPLIT == 3) {
                // ---- stream-K: a piece that does not hold its tile's first k-block is parked for the one that does ----
                // The slot holds this CTA's 128 rows of the piece as float4 units: columns 4 g .. 4 g + 3 of chunk c, row r,
                // at unit (c * 8 + g) * 128 + r -- rows innermost, so the 32 lanes of a warp (32 consecutive rows, the
                // tensor-memory load's layout) write 512 consecutive bytes per instruction, and the finishing thread,
                // which holds the same rows, reads them back the same way.  (Row-major units -- 32 lanes 128 bytes
                // apart -- measured 15 us for the reads of a 128 x 256 piece.)  Only the part that holds elements of C
                // is written.
                const size_t slot_floats = static_cast<size_t>(kBlockM) * p.block_n;
                float *slot = p.workspace + (static_cast<size_t>(it.split_index) * CTA_GROUP + cta_rank) * slot_floats;
                const bool slot_ok = checked(p.status, (static_cast<size_t>(it.split_index) * CTA_GROUP + cta_rank + 1) * slot_floats <= p.workspace_floats &&
                                                           (static_cast<size_t>(it.tile - p.first_split_tile) * CTA_GROUP + cta_rank) * 2 + 2 <= p.counter_words,
                                             kCheckSlot);
                const int32_t park_chunks = (live_rows && slot_ok) ? live_chunks : 0;
                for (int32_t c = static_cast<int32_t>(first_chunk); c < park_chunks; c += 2) {
                    uint32_t v[32];
                    tmem_ld_32x32b_x32(t_addr + static_cast<uint32_t>(c) * 32u, v);
                    tmem_ld_wait();
                    float4 *dst = reinterpret_cast<float4 *>(slot) + static_cast<size_t>(c) * 8 * kBlockM + row_in_tile;
#pragma unroll
                    for (int g = 0; g < 8; ++g)
                        __stcg(dst + g * kBlockM, make_float4(__uint_as_float(v[4 * g]), __uint_as_float(v[4 * g + 1]), __uint_as_float(v[4 * g + 2]),
                                                    __uint_as_float(v[4 * g + 3])));
                }
                release_accumulator(acc);
                // announce this warp's part: its stores, made visible to the GPU, then one arrival
                __syncwarp();
                if (lane == 0 && slot_ok) {
                    __threadfence();
                    atomicAdd(p.counters + (static_cast<size_t>(it.tile - p.first_split_tile) * CTA_GROUP + cta_rank) * 2, 1u);
                }
            } else if (SPLIT == 2) {
                // split-K inside a cluster: the accumulator is complete; the exchange below needs every
                // thread of the CTA, so it happens after the role branches
                cs_m0 = row0;
                cs_n0 = it.n0;
                cs_slice = it.slice;
            } else {
                // ---- split-K through a global workspace ---------------------------------------------------
                // 1. park this slice's fp32 partial in the workspace.  A slot is a sequence of float4 units: unit
                //    ((chunk * 128 + row) * 8 + g') holds columns 4 g .. 4 g + 3 of the chunk, g = g' ^ (row & 7)
                //    (the swizzle keeps a quarter warp's 16-byte shared-memory stores, 128 bytes apart, on
                //    different banks).  Each warp stages its 32 rows of a chunk (4 KB, contiguous in the slot) in
                //    its store buffer and sends them with one bulk copy.
                const size_t slot_floats = static_cast<size_t>(kBlockM) * p.block_n;
                float *slot = p.workspace + (static_cast<size_t>(it.split_index) * CTA_GROUP + cta_rank) * slot_floats;
                const bool slot_ok = checked(p.status, (static_cast<size_t>(it.split_index) * CTA_GROUP + cta_rank + 1) * slot_floats <= p.workspace_floats &&
                                                           (static_cast<size_t>(it.tile - p.first_split_tile) * CTA_GROUP + cta_rank) * 2 + 2 <= p.counter_words,
                                             kCheckSlot);
                if (HGEMM_CHECKED && !slot_ok) {               // (its tile then never completes: the other slices' waits run out)
                    ok = false;
                    break;
                }
                const int32_t park_chunks = live_rows ? live_chunks : 0;
                for (int32_t c = static_cast<int32_t>(first_chunk); c < park_chunks; c += 2) {
                    uint32_t v[32];
                    tmem_ld_32x32b_x32(t_addr + static_cast<uint32_t>(c) * 32u, v);
                    if (lane == 0) bulk_wait_group_read<0>();      // the buffer's last bulk copy has read it
                    tmem_ld_wait();
                    __syncwarp();
                    const uint32_t row_addr = staging + (lane << 7);
                    const uint32_t sw = lane & 7u;                   // = row & 7: a warp's first row is a multiple of 32
#pragma unroll
                    for (uint32_t g = 0; g < 8; ++g)
                        st_shared_v4(row_addr + ((g ^ sw) << 4), v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
                    fence_proxy_async_smem();
                    __syncwarp();
                    if (lane == 0) {
                        bulk_store_to_global(slot + (static_cast<size_t>(c) * kBlockM + q * 32u) * 32, staging, kStagingBytesPerWarp);
                        bulk_commit_group();
                    }
                }
                release_accumulator(acc);
                if (lane == 0) {
                    bulk_wait_group<0>();                            // this warp's part of the slot is written
                    fence_proxy_async_all();                         // order those writes before the signal below
                }
                if (w == unit && threadIdx.x == 64) trace_stamp<!TRACE>(p, 16);
                // 2. announce it, then wait (bounded) until every slice of this tile has done the same.
                //    All slices of a tile are in flight together: the grid never exceeds the SM count, one
                //    CTA per SM, and work items are handed out in tile order.
                uint32_t *ctr = p.counters + (static_cast<size_t>(it.tile - p.first_split_tile) * CTA_GROUP + cta_rank) * 2;
                //    The counter is never reset: every launch adds 8 S arrivals per tile (one per epilogue warp and
                //    slice), so launch number e waits for e * 8 S, compared modulo 2^32.
                const uint32_t target = p.epoch * 8u * static_cast<uint32_t>(it.slices);
                __syncwarp();
                if (lane == 0) {
                    __threadfence();
                    atomicAdd(ctr, 1u);
                    const long long t0 = clock64();
                    while (true) {
                        uint32_t seen;
                        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(seen) : "l"(ctr) : "memory");
                        if (static_cast<int32_t>(seen - target) >= 0) break;
                        if (*abort_flag) { ok = false; break; }
                        if (clock64() - t0 > p.wait_budget) {
                            *abort_flag = 1u;
                            atomicCAS(p.status, 0u, status_code(kRoleEpilogue, 3, it.slice));
                            ok = false;
                            break;
                        }
                        __nanosleep(40);
                    }
                }
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                if (w == unit && threadIdx.x == 64) trace_stamp<!TRACE>(p, 17);
                __threadfence();
                // 3. every slice reduces its share of the tile: slice s owns the contiguous unit range
                //    [s U / S, (s + 1) U / S), so neighbouring threads read neighbouring addresses.  Each unit is
                //    summed over the slices in slice order 0..S-1; a thread works on eight units at a time and
                //    has the loads of two slices (sixteen float4) in flight.
                const size_t first_slot = static_cast<size_t>(it.tile - p.first_split_tile) * p.split_k;
                const size_t slice_stride = static_cast<size_t>(CTA_GROUP) * slot_floats;
                const float4 *tile_ws = reinterpret_cast<const float4 *>(p.workspace + (first_slot * CTA_GROUP + cta_rank) * slot_floats);
                const int64_t units = static_cast<int64_t>(chunks) * kBlockM * 8;
                const int32_t u_begin = static_cast<int32_t>(units * it.slice / p.split_k);
                const int32_t u_end = static_cast<int32_t>(units * (it.slice + 1) / p.split_k);
                constexpr int kUnitsPerPass = 8;
                for (int32_t u0 = u_begin + static_cast<int32_t>(ew * 32u + lane); u0 < u_end; u0 += kUnitsPerPass * 256) {
                    uint32_t on = 0;                                  // bit j: unit j of this pass holds elements of C
                    float4 sum[kUnitsPerPass];
#pragma unroll
                    for (int j = 0; j < kUnitsPerPass; ++j) {
                        const int32_t u = u0 + j * 256;
                        const int32_t c = u >> 10, r = (u >> 3) & 127, g = (u & 7) ^ (r & 7);   // chunk, row, column group
                        if (u < u_end && row0 + r < p.M && it.n0 + c * 32 + g * 4 < p.N) on |= 1u << j;
                        sum[j] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                    }
                    for (int32_t sl0 = 0; sl0 < p.split_k; sl0 += 2) {
                        float4 x[2][kUnitsPerPass];
#pragma unroll
                        for (int h = 0; h < 2; ++h)
#pragma unroll
                            for (int j = 0; j < kUnitsPerPass; ++j)
                                if (((on >> j) & 1u) && sl0 + h < p.split_k)
                                    x[h][j] = __ldcg(reinterpret_cast<const float4 *>(reinterpret_cast<const float *>(tile_ws + u0 + j * 256) +
                                                                                     static_cast<size_t>(sl0 + h) * slice_stride));
#pragma unroll
                        for (int h = 0; h < 2; ++h)
#pragma unroll
                            for (int j = 0; j < kUnitsPerPass; ++j)
                                if (((on >> j) & 1u) && sl0 + h < p.split_k) {
                                    sum[j].x += x[h][j].x; sum[j].y += x[h][j].y; sum[j].z += x[h][j].z; sum[j].w += x[h][j].w;
                                }
                    }
#pragma unroll
                    for (int j = 0; j < kUnitsPerPass; ++j) {
                        if (!((on >> j) & 1u)) continue;
                        const int32_t u = u0 + j * 256;
                        const int32_t c = u >> 10, r = (u >> 3) & 127, g = (u & 7) ^ (r & 7);
                        const int32_t orow = row0 + r, col = it.n0 + c * 32 + g * 4;
                        if ((!PLAIN && p.scaled)) scale_unit4<XPOSE>(sum[j], p, orow, col);
                        if (XPOSE) {
                            store_unit4_slow(p.C, p.M, p.N, 1, orow, col, sum[j].x, sum[j].y, sum[j].z, sum[j].w);
                            continue;
                        }
                        if ((!PLAIN && p.ragged_n)) {
                            const float f[4] = {sum[j].x, sum[j].y, sum[j].z, sum[j].w};
                            store_ragged(p.C, p.N, orow, col, f, 4);
                            continue;
                        }
                        uint2 o;
                        o.x = pack_half2_rn(__float_as_uint(sum[j].x), __float_as_uint(sum[j].y));
                        o.y = pack_half2_rn(__float_as_uint(sum[j].z), __float_as_uint(sum[j].w));
                        if (checked(p.status, orow >= 0 && orow < p.M && col >= 0 && col + 4 <= p.N && (col & 3) == 0, kCheckUnitStore))
                            *reinterpret_cast<uint2 *>(p.C + static_cast<size_t>(orow) * p.N + col) = o;   // N % 8 == 0: in bounds
                    }
                }
                if (w == unit && threadIdx.x == 64) trace_stamp<!TRACE>(p, 18);
            }
        }
        // shared memory must stay valid until the last TMA stores have read it (their global writes are
        // complete, like every other store of this grid, when the grid completes)
        if (lane == 0) bulk_wait_group_read<0>();
        if (threadIdx.x == 64) trace_stamp<!TRACE>(p, 6);
    }

    // ---- cluster split-K: sum the slices through distributed shared memory -----------------
    // The S slices of a tile are the S CTAs of one cluster.  Every CTA first lays its fp32 partial out in
    // its own shared memory as float4 units: unit ((chunk * rows + row) * 8 + g') holds columns
    // 4 g .. 4 g + 3 of the chunk with g = g' ^ (row & 7) (the swizzle keeps the 16-byte stores of a
    // quarter warp, whose rows are 128 bytes apart, on different banks).  The units are dealt out in
    // contiguous shares of `cap`: CTA o owns [o cap, (o + 1) cap).  One thread per CTA then sends each
    // other owner its share with one bulk copy through the cluster's shared-memory network, completing
    // bytes on the owner's receive barrier; every owner adds, per unit, its own copy and the S - 1
    // received ones in slice order and stores fp16.  Layout: [own tile | S - 1 receive slots of cap units].
    // Both cluster barriers are taken by every thread of every CTA of the cluster, also after an abort.
    if constexpr (SPLIT == 2) {
        if (p.cluster_split) {
            // (warps 0 and 1 only take part in the barriers; what they compute here from zeros is unused)
            const uint32_t S = static_cast<uint32_t>(p.split_k), me = static_cast<uint32_t>(cs_slice);
            // only the part of the tile that holds elements of C is exchanged: `rows` rows (a multiple of 32,
            // the epilogue warps' granule) of `chunks` 32-column chunks
            const int32_t chunks = min(p.block_n / 32, (p.N - cs_n0 + 31) / 32);
            const uint32_t rows = static_cast<uint32_t>(max(0, min(kBlockM, (p.M - cs_m0 + 31) / 32 * 32)));
            const uint32_t units = static_cast<uint32_t>(chunks) * 8u * rows;
            const uint32_t cap = (units + S - 1u) / S;
            const uint32_t own_begin = me * cap;
            const uint32_t own_count = own_begin >= units ? 0u : min(cap, units - own_begin);
            const uint32_t recv_base = smem_base + units * 16u;
            // the bytes this CTA is going to receive: S - 1 copies of its own share
            if (threadIdx.x == 64) mbar_arrive_expect_tx(bar_recv, (S - 1u) * own_count * 16u);
            // barrier 1, arrival: this CTA has finished its main loop (its epilogue warps get here only after the
            // last MMA has completed), so its stage ring is free to be overwritten, and has armed its barrier
            if (threadIdx.x == 64) trace_stamp<!TRACE>(p, 16);
            cluster_arrive();
            if (warp >= 2) {
                // while the other CTAs arrive, stage this CTA's partial in its own ring (after an abort the
                // accumulator holds garbage, which then goes nowhere)
                const uint32_t q = warp & 3u;
                const uint32_t row_in_tile = q * 32u + lane;
                if (row_in_tile < rows) {
                    const uint32_t t_addr = tmem_base + ((q * 32u) << 16);      // the only work item used accumulator 0
                    tc_fence_after_sync();
                    const uint32_t sw = row_in_tile & 7u;
                    for (int32_t c = static_cast<int32_t>((warp - 2u) >> 2); c < chunks; c += 2) {
                        uint32_t v[32];
                        tmem_ld_32x32b_x32(t_addr + static_cast<uint32_t>(c) * 32u, v);
                        tmem_ld_wait();
                        const uint32_t row_addr = smem_base + ((static_cast<uint32_t>(c) * rows + row_in_tile) << 7);
#pragma unroll
                        for (uint32_t g = 0; g < 8; ++g)
                            st_shared_v4(row_addr + ((g ^ sw) << 4), v[4 * g], v[4 * g + 1], v[4 * g + 2], v[4 * g + 3]);
                    }
                    fence_proxy_async_smem();        // the bulk copies below read these writes
                }
            }
            if (threadIdx.x == 64) trace_stamp<!TRACE>(p, 17);
            cluster_wait();                          // barrier 1, wait: every ring of the cluster is free
            const bool live = *abort_flag == 0u;     // stable here: no thread of this CTA is in a wait
            if (threadIdx.x == 64) trace_stamp<!TRACE>(p, 19);
            bool ok = live;
            if (warp >= 2) {
                named_barrier_sync(1, 8 * 32);       // the whole tile is in shared memory
                if (live && threadIdx.x == 64) {
                    for (uint32_t o = 0; o < S; ++o) {
                        const uint32_t o_begin = o * cap;
                        if (o == me || o_begin >= units) continue;
                        const uint32_t slot = me < o ? me : me - 1u;              // receive slots skip the owner's own slice
                        // slice o of this tile is the CTA (of a pair: the CTA with this one's place in its pair) o pairs on
                        const uint32_t o_rank = (CTA_GROUP == 2) ? 2u * o + cta_rank : o;
                        bulk_copy_to_cluster(mapa(recv_base + slot * cap * 16u, o_rank), smem_base + o_begin * 16u,
                                             min(cap, units - o_begin) * 16u, mapa(bar_recv, o_rank));
                    }
                }
                if (threadIdx.x == 64) trace_stamp<!TRACE>(p, 18);
                if (live) ok = mbar_wait(bar_recv, 0u, ctl, status_code(kRoleEpilogue, 4, 0));
                ok = __all_sync(0xffffffffu, ok);
            }
            // barrier 2, arrival: this CTA has received everything (or given up).  Once every CTA of the cluster
            // has arrived, no bulk copy is reading anyone's shared memory any more and all may leave.
            cluster_arrive_relaxed();
            if (threadIdx.x == 64) trace_stamp<!TRACE>(p, 20);
            if (warp >= 2 && ok) {
                const uint32_t ew = warp - 2u;
                const uint32_t own_addr = smem_base + own_begin * 16u;
                // chunk of a unit = (u / 8) / rows without a division: rows = 32 k, k = 1..4, and
                // (t * mul) >> 17 = t / k for the few dozen 32-row groups t of a tile
                const uint32_t kdiv = rows >> 5;
                const uint32_t mul = kdiv == 3u ? 43691u : (1u << 17) >> (kdiv >> 1);
                // four units per thread and pass: four independent chains of loads and adds
                for (uint32_t li0 = ew * 32u + lane; li0 < own_count; li0 += 4u * 256u) {
                    float4 sum[4];
#pragma unroll
                    for (int j = 0; j < 4; ++j) sum[j] = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
                    for (uint32_t sl = 0; sl < S; ++sl) {
                        const uint32_t src = sl == me ? own_addr : recv_base + (sl < me ? sl : sl - 1u) * cap * 16u;
#pragma unroll
                        for (uint32_t j = 0; j < 4; ++j) {
                            const uint32_t li = li0 + j * 256u;
                            if (li < own_count) {
                                const float4 x = ld_shared_v4(src + li * 16u);
                                sum[j].x += x.x; sum[j].y += x.y; sum[j].z += x.z; sum[j].w += x.w;
                            }
                        }
                    }
#pragma unroll
                    for (uint32_t j = 0; j < 4; ++j) {
                        const uint32_t li = li0 + j * 256u;
                        if (li >= own_count) continue;
                        const uint32_t u = own_begin + li;
                        const uint32_t cr = u >> 3, cc = ((cr >> 5) * mul) >> 17, r = cr - cc * rows;
                        const int32_t c = static_cast<int32_t>(cc), g = static_cast<int32_t>((u & 7u) ^ (r & 7u));
                        const int32_t orow = cs_m0 + static_cast<int32_t>(r), col = cs_n0 + c * 32 + g * 4;
                        if (orow >= p.M || col >= p.N) continue;
                        if ((!PLAIN && p.scaled)) scale_unit4<XPOSE>(sum[j], p, orow, col);
                        if (XPOSE) {
                            store_unit4_slow(p.C, p.M, p.N, 1, orow, col, sum[j].x, sum[j].y, sum[j].z, sum[j].w);
                            continue;
                        }
                        if ((!PLAIN && p.ragged_n)) {
                            const float f[4] = {sum[j].x, sum[j].y, sum[j].z, sum[j].w};
                            store_ragged(p.C, p.N, orow, col, f, 4);
                            continue;
                        }
                        uint2 o;
                        o.x = pack_half2_rn(__float_as_uint(sum[j].x), __float_as_uint(sum[j].y));
                        o.y = pack_half2_rn(__float_as_uint(sum[j].z), __float_as_uint(sum[j].w));
                        if (checked(p.status, orow >= 0 && orow < p.M && col >= 0 && col + 4 <= p.N && (col & 3) == 0, kCheckUnitStore))
                            *reinterpret_cast<uint2 *>(p.C + static_cast<size_t>(orow) * p.N + col) = o;   // N % 8 == 0: in bounds
                    }
                }
            }
            if (threadIdx.x == 64) trace_stamp<!TRACE>(p, 22);
            cluster_wait();                          // barrier 2, wait
            if (threadIdx.x == 64) trace_stamp<!TRACE>(p, 21);
        }
    }

    // ---- teardown (every thread, also after an abort) ----------------------------------
    tc_fence_before_sync();
    __syncthreads();
    if constexpr (CTA_GROUP == 2) {   // no CTA of the pair leaves while the other may still signal it
        cluster_arrive_relaxed();
        cluster_wait();
    }
    if (warp == 1 && !tmem_freed) {
        if (*abort_flag) {
            // give loads and MMAs that were in flight when a wait ran out time to land
            for (int i = 0; i < 200; ++i) __nanosleep(1000);
        }
        tc_fence_after_sync();
        tmem_dealloc<CTA_GROUP>(tmem_base, static_cast<uint32_t>(p.tmem_cols));
        if (lane == 0) trace_stamp<!TRACE>(p, 7);
    }
}

// Copies a rows x K fp16 matrix into a rows x K8 one (K8 = K rounded up to 8), zero-filling the new
// columns: gives K-contiguous operands whose rows are multiples of 16 bytes, as TMA needs.  The
// zero columns add nothing to any dot product.  One thread per 8 output columns.
__global__ void hgemm_pad_k_kernel(const __half *src, __half *dst, int64_t rows, int64_t K, int64_t K8)
{
    grid_dependency_wait();
    const int64_t groups = K8 / 8;
    const int64_t total = rows * groups;
    for (int64_t i = blockIdx.x * static_cast<int64_t>(blockDim.x) + threadIdx.x; i < total;
         i += static_cast<int64_t>(gridDim.x) * blockDim.x) {
        const int64_t r = i / groups, c0 = (i - r * groups) * 8;
        __align__(16) __half out[8];
#pragma unroll
        for (int j = 0; j < 8; ++j) out[j] = (c0 + j < K) ? src[r * K + c0 + j] : __float2half_rn(0.0f);
        *reinterpret_cast<uint4 *>(dst + r * K8 + c0) = *reinterpret_cast<const uint4 *>(out);
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

// The reporting path of the checked build without any bad access: an invariant that is false by construction.
__global__ void hgemm_check_probe_kernel(uint32_t *status)
{
    if (threadIdx.x == 0) (void)checked(status, false, kCheckProbe);
}

} // namespace hgemm_dev
