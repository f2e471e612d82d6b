// The register-accumulator kernel for the smallest problems.
//
// A tcgen05 kernel pays fixed costs before and after its MMAs that do not shrink with the problem: allocating
// and freeing tensor memory alone measures about 0.7 us on B200 (an empty kernel: 0.9 us), tensor-map fetches
// and mbarrier round trips add more.  For problems that are a handful of 64 x 64 tiles with a short K loop -- the
// corner of the shape grid where the paper found its largest gains, and where it picks a lighter kernel structure
// (section 5.1) -- those costs are most of the call.  This kernel has none of them: cp.async into swizzled shared
// memory, ldmatrix, mma.sync.m16n8k16 (fp16 x fp16 -> fp32) with the accumulators in registers, 4-byte stores.
// The tensor cores still do the contraction; what is dropped is everything around them.
//
//   CTA: 128 threads = 2 x 2 warps, one T x T tile of C (T = 64 or 32); each warp a quarter of it (T = 64: 2 x 4 MMA tiles
//   of 16 x 8; T = 32: 1 x 2).  The register path issues an MMA every few cycles per SM sub-partition, so a CTA's k-block costs
//   time in proportion to its tile: the 32 x 32 tile spreads a small problem over four times as many SMs and is what the
//   shortest K loops want, the 64 x 64 tile moves half as many bytes per flop.
//   K loop: 64-wide k-blocks through a 3-stage cp.async ring (T x 128 bytes of A and of B per stage)
//   shared memory: rows of 128 bytes; 16-byte piece c of row r lives at piece c ^ (r & 7), so that the eight
//   row addresses of an ldmatrix fall on different banks
//
// Same arithmetic as the tcgen05 kernels: exact fp16 products, fp32 accumulation, one rounding to fp16 (or the
// alpha / beta form before it).  Needs K % 8 == 0 and N % 8 == 0; rows and columns beyond M, N and K are
// zero-filled on the way in and never stored.
//
// Split-K (split_k = S > 1): the S CTAs of a cluster share one tile, each with a contiguous range of the k-blocks;
// the short K loops run side by side instead of one after the other, which is what a problem of a few tiles with
// K in the thousands wants.  Afterwards every CTA lays its fp32 partial tile out in its own shared memory, the
// cluster meets at a barrier, and CTA s adds share s of the tile -- its own copy and the S - 1 others, read through
// the cluster's shared-memory network in slice order 0 .. S - 1, so the result does not depend on who finishes
// first -- and stores it; a second barrier keeps every CTA alive while its memory may still be read.
#pragma once

#include <cuda_fp16.h>
#include <stdint.h>

#include "ptx_sm100.cuh"

namespace hgemm_dev {

constexpr int kSmallBk = 64;          // K extent of a stage
constexpr int kSmallStages = 3;
constexpr int kSmallThreads = 128;

#ifndef HGEMM_CHECKED
#define HGEMM_CHECKED 0        // the checked build: see hgemm_kernel.cuh
#endif

struct SmallParams {
    const __half *A;                  // M x K, K-contiguous
    const __half *B;                  // N x K, K-contiguous
    __half *C;                        // M x N row-major
    int32_t M, N, K;
    int32_t tiles_m;                  // ceil(M / T): cluster b computes tile (b % tiles_m, b / tiles_m)
    uint32_t scaled;                  // 1: C = alpha A B^T + beta C
    float alpha, beta;
    int32_t split_k;                  // CTAs per cluster = K slices per tile (1: none); blockIdx.x = tile * split_k + slice
    uint32_t *status;                 // the plan's status word (written by the checked build only)
};

// Checked build: a store of `width` elements at (row, col) must lie inside C on a 4-byte boundary.
__device__ __forceinline__ bool small_store_ok(const SmallParams &p, int32_t row, int32_t col, int32_t width)
{
#if HGEMM_CHECKED
    if (!(row >= 0 && row < p.M && col >= 0 && col + width <= p.N && (col & 1) == 0)) {
        atomicCAS(p.status, 0u, (7u << 24) | (8u << 8));          // (kRoleCheck, kCheckSmallStore) of the main kernel's encoding
        return false;
    }
#endif
    return true;
}

__device__ __forceinline__ void cp_async_16(uint32_t dst, const void *src, uint32_t src_bytes)
{
    // src_bytes == 0 writes sixteen zero bytes and reads nothing
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}

__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t &r0, uint32_t &r1, uint32_t &r2, uint32_t &r3)
{
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0, %1, %2, %3}, [%4];" : "=r"(r0), "=r"(r1), "=r"(r2), "=r"(r3) : "r"(addr));
}

__device__ __forceinline__ void mma_m16n8k16(float (&d)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1)
{
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.f16.f16.f32 {%0, %1, %2, %3}, {%4, %5, %6, %7}, {%8, %9}, {%0, %1, %2, %3};"
                 : "+f"(d[0]), "+f"(d[1]), "+f"(d[2]), "+f"(d[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}

template <int T>                      // rows and columns of C per CTA: 64 or 32
__global__ void __launch_bounds__(kSmallThreads)
hgemm_small_kernel(const SmallParams p)
{
    static_assert(T == 64 || T == 32, "tile size");
    constexpr int kSmallTile = T;
    constexpr int MI = T / 32;        // 16-row MMA tiles per warp
    constexpr int NI = T / 16;        // 8-column MMA tiles per warp (two per ldmatrix)
    __shared__ __align__(128) uint8_t smem[kSmallStages * 2 * kSmallTile * kSmallBk * 2];     // 48 or 24 KB: [stage][A | B][T rows][128 bytes]
    const uint32_t smem_base = smem_addr(smem);
    const uint32_t tid = threadIdx.x, lane = tid & 31u, warp = tid >> 5;
    const uint32_t wm = warp & 1u, wn = warp >> 1;                      // this warp's quarter of the tile
    const int32_t S = p.split_k;
    const int32_t slice = S > 1 ? static_cast<int32_t>(cluster_ctarank()) : 0;
    const int32_t tile = S > 1 ? static_cast<int32_t>(blockIdx.x) / S : static_cast<int32_t>(blockIdx.x);
    const int32_t tn = tile / p.tiles_m, tm = tile - tn * p.tiles_m;
    const int32_t m0 = tm * kSmallTile, n0 = tn * kSmallTile;
    // this CTA's k-blocks: the first (all mod S) slices take one more
    const int32_t kb_all = (p.K + kSmallBk - 1) / kSmallBk;
    const int32_t kb_base = kb_all / S, kb_rem = kb_all - kb_base * S;
    const int32_t kb_first = slice * kb_base + min(slice, kb_rem);
    const int32_t kblocks = kb_base + (slice < kb_rem ? 1 : 0);
    constexpr uint32_t kTileBytes = kSmallTile * kSmallBk * 2;          // 8 KB

    grid_launch_dependents();          // the next kernel in the stream may start its own set-up
    grid_dependency_wait();            // ... and this one reads nothing before the kernels ahead of it are complete

    // One stage: T rows x eight 16-byte pieces of A and of B, T / 16 pieces of each per thread.
    auto load_stage = [&](int32_t kb, int32_t s) {
        const uint32_t a_dst = smem_base + static_cast<uint32_t>(s) * 2u * kTileBytes;
        const uint32_t b_dst = a_dst + kTileBytes;
        const int32_t k0 = (kb_first + kb) * kSmallBk;
#pragma unroll
        for (int i = 0; i < T / 16; ++i) {
            const uint32_t piece = tid + static_cast<uint32_t>(i) * kSmallThreads;       // 0 .. 8 T - 1
            const uint32_t r = piece >> 3, c = piece & 7u;
            const int32_t k = k0 + static_cast<int32_t>(c) * 8;
            const uint32_t off = r * 128u + ((c ^ (r & 7u)) << 4);
            const bool k_in = k < p.K;                                                     // K % 8 == 0: a piece is inside or outside
            const int32_t ar = m0 + static_cast<int32_t>(r), br = n0 + static_cast<int32_t>(r);
            const bool a_in = k_in && ar < p.M, b_in = k_in && br < p.N;
            // (an address inside the matrix even when nothing is read from it)
            cp_async_16(a_dst + off, p.A + (a_in ? static_cast<size_t>(ar) * p.K + k : 0), a_in ? 16u : 0u);
            cp_async_16(b_dst + off, p.B + (b_in ? static_cast<size_t>(br) * p.K + k : 0), b_in ? 16u : 0u);
        }
        asm volatile("cp.async.commit_group;" ::: "memory");
    };

    float acc[MI][NI][4];
#pragma unroll
    for (int i = 0; i < MI; ++i)
#pragma unroll
        for (int j = 0; j < NI; ++j)
#pragma unroll
            for (int e = 0; e < 4; ++e) acc[i][j][e] = 0.0f;

    // prologue: two stages in flight (an empty group where K is shorter, so that the group count stays uniform)
    for (int32_t s = 0; s < kSmallStages - 1; ++s) {
        if (s < kblocks) load_stage(s, s);
        else asm volatile("cp.async.commit_group;" ::: "memory");
    }

    for (int32_t kb = 0; kb < kblocks; ++kb) {
        asm volatile("cp.async.wait_group %0;" ::"n"(kSmallStages - 2) : "memory");      // k-block kb has landed (this thread's part)
        __syncthreads();                                                                  // ... everyone's; and stage (kb - 1) % 3 is free
        if (kb + kSmallStages - 1 < kblocks) load_stage(kb + kSmallStages - 1, (kb + kSmallStages - 1) % kSmallStages);
        else asm volatile("cp.async.commit_group;" ::: "memory");
        const uint32_t a_tile = smem_base + static_cast<uint32_t>(kb % kSmallStages) * 2u * kTileBytes;
        const uint32_t b_tile = a_tile + kTileBytes;
#pragma unroll
        for (uint32_t kk = 0; kk < kSmallBk / 16; ++kk) {
            // A fragments: rows 16 i .. 16 i + 15 of this warp's T / 2; matrices in the order (rows 0-7, k 0-7),
            // (rows 8-15, k 0-7), (rows 0-7, k 8-15), (rows 8-15, k 8-15) = registers a0..a3 of the MMA
            uint32_t a[MI][4];
#pragma unroll
            for (uint32_t i = 0; i < MI; ++i) {
                const uint32_t row = wm * (T / 2) + i * 16u + (lane & 7u) + ((lane >> 3) & 1u) * 8u;
                const uint32_t piece = kk * 2u + (lane >> 4);
                ldmatrix_x4(a_tile + row * 128u + ((piece ^ (row & 7u)) << 4), a[i][0], a[i][1], a[i][2], a[i][3]);
            }
            // B fragments: two 8-column tiles per ldmatrix; matrices (n 0-7, k 0-7), (n 0-7, k 8-15), (n 8-15, k 0-7),
            // (n 8-15, k 8-15) = b0, b1 of the first tile, b0, b1 of the second
            uint32_t b[NI][2];
#pragma unroll
            for (uint32_t j = 0; j < NI / 2; ++j) {
                const uint32_t row = wn * (T / 2) + j * 16u + (lane & 7u) + (lane >> 4) * 8u;
                const uint32_t piece = kk * 2u + ((lane >> 3) & 1u);
                ldmatrix_x4(b_tile + row * 128u + ((piece ^ (row & 7u)) << 4), b[2 * j][0], b[2 * j][1], b[2 * j + 1][0], b[2 * j + 1][1]);
            }
#pragma unroll
            for (int i = 0; i < MI; ++i)
#pragma unroll
                for (int j = 0; j < NI; ++j) mma_m16n8k16(acc[i][j], a[i], b[j][0], b[j][1]);
        }
    }

    if (S > 1) {
        // ---- split-K: the partial tiles meet in shared memory ------------------------------------------------
        // (every thread of every CTA of the cluster takes both barriers: nothing above or below returns early)
        asm volatile("cp.async.wait_all;" ::: "memory");
        __syncthreads();                                              // the ring is free: it now holds the partial tile,
        const uint32_t part = smem_base;                              // row-major fp32, T floats per row (T * T * 4 <= 16 KB)
#pragma unroll
        for (int i = 0; i < MI; ++i)
#pragma unroll
            for (int h = 0; h < 2; ++h)
#pragma unroll
                for (int j = 0; j < NI; ++j) {
                    const uint32_t r = wm * (T / 2) + i * 16u + h * 8u + (lane >> 2), c = wn * (T / 2) + j * 8u + (lane & 3u) * 2u;
                    asm volatile("st.shared.v2.f32 [%0], {%1, %2};" ::"r"(part + (r * T + c) * 4u), "f"(acc[i][j][2 * h]), "f"(acc[i][j][2 * h + 1]) : "memory");
                }
        cluster_arrive();                                             // release: this CTA's partial is written
        cluster_wait();                                               // acquire: so is everyone's
        // share `slice` of the tile's float4 units (four consecutive columns of one row), one unit per thread and pass
        constexpr int32_t kUnits = T * T / 4;
        const int32_t cap = (kUnits + S - 1) / S;
        const int32_t u_end = min(kUnits, (slice + 1) * cap);
        for (int32_t u = slice * cap + static_cast<int32_t>(tid); u < u_end; u += kSmallThreads) {
            float4 sum = make_float4(0.0f, 0.0f, 0.0f, 0.0f);
            for (int32_t sl = 0; sl < S; ++sl) {                      // slice order: the same sum whoever arrives first
                const float4 x = ld_shared_cluster_v4(mapa(part + static_cast<uint32_t>(u) * 16u, static_cast<uint32_t>(sl)));
                sum.x += x.x; sum.y += x.y; sum.z += x.z; sum.w += x.w;
            }
            const int32_t row = m0 + (u * 4) / T, col = n0 + (u * 4) % T;
            if (row >= p.M || col >= p.N) continue;                   // N % 8 == 0 and col % 4 == 0: the unit is inside or outside
            __half2 *dst = reinterpret_cast<__half2 *>(p.C + static_cast<size_t>(row) * p.N + col);
            if (p.scaled) {
                float2 o0 = make_float2(0.0f, 0.0f), o1 = make_float2(0.0f, 0.0f);
                if (p.beta != 0.0f) {
                    o0 = __half22float2(dst[0]);
                    o1 = __half22float2(dst[1]);
                }
                sum.x = fmaf(p.beta, o0.x, p.alpha * sum.x);
                sum.y = fmaf(p.beta, o0.y, p.alpha * sum.y);
                sum.z = fmaf(p.beta, o1.x, p.alpha * sum.z);
                sum.w = fmaf(p.beta, o1.y, p.alpha * sum.w);
            }
            if (!small_store_ok(p, row, col, 4)) continue;
            dst[0] = __floats2half2_rn(sum.x, sum.y);
            dst[1] = __floats2half2_rn(sum.z, sum.w);
        }
        __syncwarp();                                                 // (the loop above ends at different times within a warp)
        cluster_arrive_relaxed();                                     // no CTA leaves while another may still read its memory
        cluster_wait();
        return;
    }

    // epilogue: accumulator element pairs (row l / 4 [+ 8], columns 2 (l % 4), + 1) -> half2 -> 4-byte stores
#pragma unroll
    for (int i = 0; i < MI; ++i) {
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            const int32_t row = m0 + static_cast<int32_t>(wm * (T / 2) + i * 16u + h * 8u + (lane >> 2));
            if (row >= p.M) continue;
#pragma unroll
            for (int j = 0; j < NI; ++j) {
                const int32_t col = n0 + static_cast<int32_t>(wn * (T / 2) + j * 8u + (lane & 3u) * 2u);
                if (col >= p.N) continue;                                 // N is even: the pair is inside or outside
                float x = acc[i][j][2 * h], y = acc[i][j][2 * h + 1];
                __half2 *dst = reinterpret_cast<__half2 *>(p.C + static_cast<size_t>(row) * p.N + col);
                if (p.scaled) {
                    float ox = 0.0f, oy = 0.0f;
                    if (p.beta != 0.0f) {
                        const float2 o = __half22float2(*dst);
                        ox = o.x;
                        oy = o.y;
                    }
                    x = fmaf(p.beta, ox, p.alpha * x);
                    y = fmaf(p.beta, oy, p.alpha * y);
                }
                if (small_store_ok(p, row, col, 2)) *dst = __floats2half2_rn(x, y);
            }
        }
    }
}

} // namespace hgemm_dev
