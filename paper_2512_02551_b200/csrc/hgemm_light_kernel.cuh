// The light kernel: one 128 x block_n tile per CTA, no persistent loop, one accumulator.
//
// The paper picks a different kernel structure for small problems than for large ones (section 5.1,
// "abstraction selection": few stages and little synchronisation where the whole problem is a handful of
// tiles).  For the shapes of the grid whose run time is a few microseconds the persistent kernel's fixed
// costs -- two accumulators and their hand-off barriers, the work decode, CTA-wide barriers at both ends, a
// CTA that asks for all of shared memory -- are a large part of the call.  This kernel keeps only what one
// tile needs, ordered so that the critical path (load -> MMA -> store) starts as early as it can:
//
//   warp 0      initialises the barriers its first loads need, issues the first `stages` k-blocks' TMA loads, and
//               only then the remaining barriers: the loads' round trip overlaps the rest of the set-up (tensor-memory
//               allocation, the CTA-wide barrier); afterwards it keeps the ring full
//   warp 1      allocates tensor memory (block_n columns rounded up to a power of two), issues the MMAs, frees a
//               stage only if the ring wraps; frees tensor memory as soon as the epilogue warps have read it
//   warps 2..9  epilogue, two warps per tensor-memory lane quarter taking alternate 32-column chunks:
//               tcgen05.ld -> fp16 -> 16-byte stores to C, or -> swizzled shared memory -> TMA store
//
// There is no CTA-wide barrier at the end: a warp leaves when its own work is done.  Same arithmetic as the
// persistent kernel (fp16 products, fp32 accumulation in tensor memory, one rounding), same operand layouts, same
// bounded waits and status word.  K-contiguous A and B whose rows are multiples of 16 bytes, rows of C that are
// multiples of 16 bytes; no K slices.
#pragma once

#include "hgemm_kernel.cuh"

namespace hgemm_dev {

constexpr int kLightThreads = 320;                        // producer + MMA + 8 epilogue warps
constexpr int kLightStagingBytes = 8 * kStagingBytesPerWarp;   // 32 KB: two 32 x 32 fp16 boxes per epilogue warp

// Uses the fields of KernelParams that apply to one tile per CTA: M, N, K, tiles_m, kblocks, block_k, block_n, stages,
// tmem_cols, idesc, epilogue_tma, status, C, wait_budget, scaled, alpha, beta.  Grid: tiles_m * tiles_n CTAs; CTA b
// computes tile (b % tiles_m, b / tiles_m): neighbouring CTAs share their B tile.
// TRACE: the instantiation that also writes SM-clock stamps (clock64) of CTA 0's steps into p.trace[0..12]: 0 entry,
// 1 first barriers initialised, 2 first loads issued, 3 tensor memory allocated, 4 set-up barrier passed, 5 first
// k-block landed, 6 last MMA issued, 7 accumulator ready, 8 first chunk converted, 9 last store issued, 10 epilogue
// warp done, 11 every epilogue warp has read tensor memory, 12 tensor memory freed.
template <bool TRACE = false>
__global__ void __launch_bounds__(kLightThreads, 1)
hgemm_light_kernel(const __grid_constant__ CUtensorMap tmap_a, const __grid_constant__ CUtensorMap tmap_b,
                   const __grid_constant__ CUtensorMap tmap_c, const KernelParams p)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (smem_addr(smem_raw) + 1023u) & ~1023u;
    uint8_t *smem_gen = smem_raw + (smem_base - smem_addr(smem_raw));

    const int32_t subs = p.block_k / kSubK;
    const uint32_t b_sub_bytes = static_cast<uint32_t>(p.block_n) * kSubK * 2;
    const uint32_t a_stage_bytes = static_cast<uint32_t>(subs) * kATileBytes;
    const uint32_t stage_bytes = a_stage_bytes + static_cast<uint32_t>(subs) * b_sub_bytes;
    const uint32_t staging_base = smem_base + static_cast<uint32_t>(p.stages) * stage_bytes;
    const uint32_t ctrl_base = staging_base + (p.epilogue_tma ? kLightStagingBytes : 0u);   // direct stores stage nothing
    uint8_t *ctrl_gen = smem_gen + (ctrl_base - smem_base);

    // control block: full[12] | empty[12] | accumulator ready | accumulator read | tensor-memory base | abort flag
    const uint32_t bar_full = ctrl_base;
    const uint32_t bar_empty = ctrl_base + 8 * kMaxStages;
    const uint32_t bar_acc = ctrl_base + 16 * kMaxStages;
    const uint32_t bar_read = bar_acc + 8;                   // one arrival per epilogue warp: its last tensor-memory load is complete
    volatile uint32_t *tmem_base_slot = reinterpret_cast<volatile uint32_t *>(ctrl_gen + 16 * kMaxStages + 16);
    volatile uint32_t *abort_flag = reinterpret_cast<volatile uint32_t *>(ctrl_gen + 16 * kMaxStages + 20);

    const uint32_t warp = __shfl_sync(0xffffffffu, threadIdx.x >> 5, 0);
    const uint32_t lane = lane_id();
    WaitCtl ctl{abort_flag, p.status, p.wait_budget};
    auto stamp = [&](int slot) {
        if constexpr (TRACE) {
            if (p.trace != nullptr && blockIdx.x == 0 && lane == 0) p.trace[slot] = static_cast<unsigned long long>(clock64());
        }
    };
    if (threadIdx.x == 0) stamp(0);

    const int32_t tile = static_cast<int32_t>(blockIdx.x);
    const int32_t tn = tile / p.tiles_m, tm = tile - tn * p.tiles_m;
    const int32_t m0 = tm * kBlockM, n0 = tn * p.block_n;
    const int32_t first_pass = min(p.kblocks, p.stages);     // k-blocks whose stage is free from the start

    // One stage's loads (whole warp, one elected lane issues).
    auto load_stage = [&](int32_t kb, int32_t s) {
        const uint32_t a_dst = smem_base + static_cast<uint32_t>(s) * stage_bytes;
        const uint32_t b_dst = a_dst + a_stage_bytes;
        const int32_t k0 = kb * p.block_k;
        mbar_arrive_expect_tx_elect(bar_full + 8 * s, stage_bytes);
        for (int32_t sub = 0; sub < subs; ++sub) {
            tma_load_2d_elect(a_dst + sub * kATileBytes, &tmap_a, k0 + sub * kSubK, m0, bar_full + 8 * s);
            tma_load_2d_elect(b_dst + sub * b_sub_bytes, &tmap_b, k0 + sub * kSubK, n0, bar_full + 8 * s);
        }
    };

    // ---- set-up: the first loads go out before anything else ---------------------------------------
    grid_launch_dependents();
    if (warp == 0) {
        if (lane == 0) {
            *abort_flag = 0u;
            for (int s = 0; s < first_pass; ++s) mbar_init(bar_full + 8 * s, 1);
            fence_mbar_init();
        }
        __syncwarp();
        stamp(1);
        grid_dependency_wait();                  // the kernels ahead in the stream are complete: global memory may be read
        for (int32_t kb = 0; kb < first_pass; ++kb) load_stage(kb, kb);
        stamp(2);
        if (lane == 0) {                         // the barriers nothing has needed yet
            for (int s = first_pass; s < p.stages; ++s) mbar_init(bar_full + 8 * s, 1);
            for (int s = 0; s < p.stages; ++s) mbar_init(bar_empty + 8 * s, 1);
            mbar_init(bar_acc, 1);
            mbar_init(bar_read, 8);
            fence_mbar_init();
        }
    } else if (warp == 1) {
        tmem_alloc<1>(smem_addr(const_cast<uint32_t *>(tmem_base_slot)), static_cast<uint32_t>(p.tmem_cols));
        tmem_relinquish<1>();
        stamp(3);
    } else if (warp == 2 && lane == 0) {
        prefetch_tensormap(&tmap_a);
        prefetch_tensormap(&tmap_b);
        if (p.epilogue_tma) prefetch_tensormap(&tmap_c);
    }
    tc_fence_before_sync();
    __syncthreads();
    tc_fence_after_sync();
    if (warp == 1) stamp(4);
    const uint32_t tmem_base = __shfl_sync(0xffffffffu, *tmem_base_slot, 0);

    // ---- roles ---------------------------------------------------------------------------------------
    // bar_read: "tensor memory has been read".  Every epilogue warp arrives exactly once, also when a wait ran out,
    // and warp 1 frees the allocation behind it.
    if (warp == 0) {
        // the ring wraps only when K is longer than the ring: stage s is free again once its MMAs have completed
        bool ok = true;
        for (int32_t kb = first_pass; ok && kb < p.kblocks; ++kb) {
            const int32_t s = kb % p.stages;
            const uint32_t use = static_cast<uint32_t>(kb / p.stages);          // how often the stage has been used before
            ok = mbar_wait(bar_empty + 8 * s, (use - 1u) & 1u, ctl, status_code(kRoleProducer, 0, s));
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            load_stage(kb, s);
        }
    } else if (warp == 1) {
        const uint64_t desc_a0 = make_smem_desc_sw128(smem_base);
        const uint64_t desc_b0 = make_smem_desc_sw128(smem_base + a_stage_bytes);
        const uint32_t desc_stage_step = stage_bytes >> 4;
        bool ok = true;
        for (int32_t kb = 0; ok && kb < p.kblocks; ++kb) {
            const int32_t s = kb % p.stages;
            ok = mbar_wait(bar_full + 8 * s, static_cast<uint32_t>(kb / p.stages) & 1u, ctl, status_code(kRoleMma, 0, s));
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            if (kb == 0) stamp(5);
            tc_fence_after_sync();
            const uint64_t a_desc = desc_a0 + static_cast<uint64_t>(static_cast<uint32_t>(s) * desc_stage_step);
            const uint64_t b_desc = desc_b0 + static_cast<uint64_t>(static_cast<uint32_t>(s) * desc_stage_step);
            for (int32_t sub = 0; sub < subs; ++sub) {
                const uint64_t a_sub = a_desc + static_cast<uint64_t>(static_cast<uint32_t>(sub) * (kATileBytes >> 4));
                const uint64_t b_sub = b_desc + static_cast<uint64_t>(static_cast<uint32_t>(sub) * (b_sub_bytes >> 4));
#pragma unroll
                for (int k = 0; k < kSubK / kUmmaK; ++k)
                    umma_f16_elect<1>(tmem_base, a_sub + 2u * k, b_sub + 2u * k, p.idesc, (kb | sub | k) != 0 ? 1u : 0u);
            }
            if (kb + p.stages < p.kblocks) umma_commit_elect<1>(bar_empty + 8 * s, 0u);   // only a stage that is used again
        }
        if (ok) umma_commit_elect<1>(bar_acc, 0u);
        stamp(6);
        // free tensor memory once the epilogue warps have read it (their stores go on meanwhile)
        (void)mbar_wait(bar_read, 0u, ctl, status_code(kRoleMma, 2, 0));
        __syncwarp();
        stamp(11);
        if (*abort_flag) {
            // Loads and MMAs in flight when a wait ran out may still land: this warp keeps the CTA -- its shared and
            // tensor memory -- alive for a while before it lets go.
            for (int i = 0; i < 200; ++i) __nanosleep(1000);
        }
        tc_fence_after_sync();
        tmem_dealloc<1>(tmem_base, static_cast<uint32_t>(p.tmem_cols));
        stamp(12);
    } else {
        // ===== epilogue: warps 2..9; warp w reads tensor-memory lanes 32 (w % 4) .. + 31, chunks (w - 2) / 4, + 2, ... =====
        const uint32_t q = warp & 3u;
        const uint32_t ew = warp - 2u;
        const uint32_t first_chunk = ew >> 2;
        const uint32_t staging = staging_base + ew * kStagingBytesPerWarp;
        const int32_t row0 = m0 + static_cast<int32_t>(q) * 32;                  // first row of this warp's 32
        const int32_t grow = row0 + static_cast<int32_t>(lane);
        const int32_t chunks = row0 < p.M ? min(p.block_n / 32, (p.N - n0 + 31) / 32) : 0;
        grid_dependency_wait();                                                   // before the first store to C
        bool ok = mbar_wait(bar_acc, 0u, ctl, status_code(kRoleEpilogue, 2, 0));
        ok = __all_sync(0xffffffffu, ok);
        bool arrived = false;
        auto tmem_read_done = [&]() {                                             // this warp's last tensor-memory load has completed
            tc_fence_before_sync();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar_read);
            arrived = true;
        };
        if (ok) {
            if (warp == 2) stamp(7);
            tc_fence_after_sync();
            const uint32_t t_addr = tmem_base + ((q * 32u) << 16);
            uint32_t store_count = 0;
            for (int32_t c = static_cast<int32_t>(first_chunk); c < chunks; c += 2) {
                uint32_t v[32];
                tmem_ld_32x32b_x32(t_addr + static_cast<uint32_t>(c) * 32u, v);
                tmem_ld_wait();
                if (c + 2 >= chunks) tmem_read_done();
                const int32_t col0 = n0 + c * 32;
                if (p.scaled && grow < p.M) {
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (col0 + 8 * j < p.N) scale_group8<false>(v + 8 * j, p, grow, col0 + 8 * j);
                }
                if (warp == 2 && c == 0) stamp(8);
                if (p.epilogue_tma) {
                    const uint32_t buf = staging + (store_count & 1u) * (kStagingBytesPerWarp / 2);
                    bulk_wait_group_read<1>();                   // the box staged two stores ago has been read
                    __syncwarp();
                    // 64-byte rows under the 64-byte swizzle: 16-byte piece j of row r lives at piece j ^ ((r >> 1) & 3)
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
                    tma_store_2d_if(lane == 0 ? 1u : 0u, &tmap_c, col0, row0, buf);
                    bulk_commit_group();
                    ++store_count;
                } else if (grow < p.M) {
                    __half *dst = p.C + static_cast<size_t>(grow) * p.N + col0;
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        if (col0 + 8 * j + 8 <= p.N) {           // N % 8 == 0: a group of eight is inside C or outside it
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
            if (warp == 2) stamp(9);
        }
        if (!arrived) tmem_read_done();                          // nothing to read, or a wait ran out
        if (p.epilogue_tma && lane == 0) bulk_wait_group_read<0>();   // shared memory stays valid until the stores have read it
        if (warp == 2) stamp(10);
    }
}

} // namespace hgemm_dev
