// Host-only planner (see hgemm_planner.h).  No CUDA calls in this file.
#include "hgemm_planner.h"

#include <algorithm>
#include <cmath>
#include <cstring>
#include <utility>
#include <vector>

namespace hgemm_host {

namespace {
constexpr int64_t kATileBytes = 128 * 64 * 2;
constexpr int64_t kStagingBytes = 32768;
constexpr int64_t kCtrlBytes = 512;
constexpr int64_t kAlignSlack = 1024;

inline int64_t ceil_div(int64_t a, int64_t b) { return (a + b - 1) / b; }
} // namespace

int64_t stage_bytes(const hgemm_config_t &c)
{
    const int64_t subs = c.block_k / 64;
    return subs * (kATileBytes + int64_t(c.block_n / cta_group_of(c)) * 64 * 2);
}

// Store staging of the eight epilogue warps: two 2 KB boxes each, or two 4 KB ones for the wide TMA epilogue.
int64_t staging_bytes(const hgemm_config_t &c)
{
    if (c.family == HGEMM_FAMILY_LIGHT) return c.epilogue == HGEMM_EPILOGUE_DIRECT ? 0 : kStagingBytes;   // direct stores stage nothing
    return c.epilogue == HGEMM_EPILOGUE_TMA_WIDE ? 2 * kStagingBytes : kStagingBytes;
}

int64_t smem_bytes(const hgemm_config_t &c)
{
    if (c.family == HGEMM_FAMILY_SMALL) return 3 * 2 * int64_t(c.block_n) * 64 * 2;      // its static ring: three stages of A and B tiles
    return kAlignSlack + int64_t(c.stages) * stage_bytes(c) + staging_bytes(c) + kCtrlBytes;
}

int32_t max_stages(int32_t family, int32_t block_n, int32_t block_k)
{
    hgemm_config_t c;
    std::memset(&c, 0, sizeof(c));
    c.family = family;
    c.block_n = block_n;
    c.block_k = block_k;
    const int64_t room = kSmemOptInBytes - kAlignSlack - kStagingBytes - kCtrlBytes;
    return int32_t(std::min<int64_t>(12, room / stage_bytes(c)));
}

int32_t max_stages_of(const hgemm_config_t &c)
{
    const int64_t room = kSmemOptInBytes - kAlignSlack - staging_bytes(c) - kCtrlBytes;
    return int32_t(std::min<int64_t>(12, room / stage_bytes(c)));
}

SplitLayout split_layout(int64_t M, int64_t N, int64_t K, int32_t num_sms, const hgemm_config_t &c)
{
    if (c.family == HGEMM_FAMILY_SMALL) {
        SplitLayout S;
        S.tiles = ceil_div(M, c.block_n) * ceil_div(N, c.block_n);
        S.first_split_tile = S.tiles;
        S.slices = 1;
        S.pieces = 1;
        S.stream_units = 0;
        S.work_items = S.tiles * std::max(1, c.split_k);          // one CTA per (tile, K slice)
        return S;
    }
    if (c.swap_ab) std::swap(M, N);   // the kernel tiles the transposed problem
    const int cg = cta_group_of(c);
    SplitLayout L;
    L.tiles = ceil_div(M, 128 * cg) * ceil_div(N, c.block_n);
    L.first_split_tile = L.tiles;
    L.slices = 1;
    L.pieces = 1;
    L.stream_units = 0;
    if (c.split_k > 1) {
        L.first_split_tile = 0;
        L.slices = c.split_k;
    } else if (c.tail_split >= 2 && c.tail_mode == HGEMM_TAIL_STREAM) {
        const int64_t units = std::max(1, num_sms / cg);
        const int64_t rem = L.tiles % units;                     // the tiles beyond the full waves
        const int64_t kb = ceil_div(K, c.block_k);
        const int64_t gs = std::min(units, rem * c.tail_split);  // positions that share them
        // worth it only if a share is at least two k-blocks and no tile is cut into more pieces than may wait for each other
        if (rem > 0 && gs > rem && rem * kb >= 2 * gs && rem * kb * gs < (int64_t(1) << 30)) {
            const int64_t q = rem * kb;
            int64_t most = 1;
            for (int64_t t = 0; t < rem; ++t) {
                const int64_t j_lo = ((t * kb + 1) * gs - 1) / q, j_hi = ((t * kb + kb) * gs - 1) / q;
                most = std::max(most, j_hi - j_lo + 1);
            }
            if (most >= 2 && most <= kMaxSplitK && rem * most * cg * 128 * int64_t(c.block_n) * 4 <= kMaxWorkspaceBytes) {
                L.first_split_tile = L.tiles - rem;
                L.slices = most;
                L.stream_units = gs;
                L.work_items = L.first_split_tile + 2 * units;
                return L;
            }
        }
    } else if (c.tail_split >= 2) {
        const int64_t units = std::max(1, num_sms / cg);
        const int64_t tail = L.tiles % units;
        if (L.tiles > units && tail > 0 && tail * c.tail_split <= units) {
            if (c.tail_mode == HGEMM_TAIL_N) {
                L.first_split_tile = L.tiles - tail;
                L.pieces = c.tail_split;
            } else if (c.tail_split <= ceil_div(K, c.block_k)) {
                L.first_split_tile = L.tiles - tail;
                L.slices = c.tail_split;
            }
        }
    }
    L.work_items = L.first_split_tile + (L.tiles - L.first_split_tile) * L.slices * L.pieces;
    return L;
}

int64_t workspace_bytes(int64_t M, int64_t N, int64_t K, const hgemm_config_t &c, int32_t num_sms)
{
    if (c.split_k > 1 && c.split_mode == HGEMM_SPLIT_CLUSTER) return 0;
    const SplitLayout L = split_layout(M, N, K, num_sms, c);
    if (L.slices <= 1) return 0;
    return (L.tiles - L.first_split_tile) * L.slices * cta_group_of(c) * 128 * int64_t(c.block_n) * 4;
}

int64_t counter_bytes(int64_t M, int64_t N, const hgemm_config_t &c, int32_t num_sms, int64_t K)
{
    if (c.split_k > 1 && c.split_mode == HGEMM_SPLIT_CLUSTER) return 0;
    const SplitLayout L = split_layout(M, N, K, num_sms, c);
    if (L.slices <= 1) return 0;
    return (L.tiles - L.first_split_tile) * cta_group_of(c) * 2 * 4;
}

hgemm_status_t validate_shape(int64_t M, int64_t N, int64_t K)
{
    if (M < 1 || N < 1 || K < 1) return HGEMM_ERR_INVALID_ARG;
    if (M > kMaxDim || N > kMaxDim || K > kMaxDim) return HGEMM_ERR_UNSUPPORTED;
    return HGEMM_OK;
}

hgemm_status_t validate_shape_aligned(int64_t M, int64_t N, int64_t K)
{
    const hgemm_status_t s = validate_shape(M, N, K);
    if (s != HGEMM_OK) return s;
    if ((K % 8) != 0 || (N % 8) != 0) return HGEMM_ERR_UNSUPPORTED;   // rows must be multiples of 16 bytes
    return HGEMM_OK;
}

hgemm_status_t validate(int64_t M, int64_t N, int64_t K, const hgemm_config_t &c)
{
    const hgemm_status_t s = validate_shape(M, N, K);
    if (s != HGEMM_OK) return s;
    if (c.swap_ab != 0 && c.swap_ab != 1) return HGEMM_ERR_UNSUPPORTED;
    if (c.raster_mode != HGEMM_RASTER_SWEEP && c.raster_mode != HGEMM_RASTER_SERPENTINE) return HGEMM_ERR_UNSUPPORTED;
    if (c.swap_ab) {
        // the transposed tile is stored through 32 x 32 boxes or 2-byte stores into rows of C that are multiples of
        // 16 bytes; everything below judges the problem the kernel sees: rows and columns traded
        if ((N % 8) != 0 || c.accumulate != HGEMM_ACC_F32 || c.tail_split >= 2 || c.epilogue == HGEMM_EPILOGUE_TMA_WIDE)
            return HGEMM_ERR_UNSUPPORTED;
        std::swap(M, N);
    }
    if (c.family == HGEMM_FAMILY_SMALL) {
        // two fixed configurations: 64 x 64 or 32 x 32 tiles
        if (c.reserved[0] != 0 || c.wave_pace != 0) return HGEMM_ERR_UNSUPPORTED;
        // K slices: the CTAs of one cluster (at most 16), summed through its shared memory
        if (c.split_k < 1 || c.split_k > 16 || c.split_k > ceil_div(K, 64) || (c.split_k > 1 && c.split_mode != HGEMM_SPLIT_CLUSTER)) return HGEMM_ERR_UNSUPPORTED;
        if ((c.block_n != 64 && c.block_n != 32) || c.block_m != c.block_n || c.block_k != 64 || c.stages != 3 || c.tail_split >= 2 || c.swap_ab ||
            c.accumulate != HGEMM_ACC_F32 || c.epilogue != HGEMM_EPILOGUE_DIRECT || c.raster_mode != HGEMM_RASTER_SWEEP || c.raster_group < 1 ||
            (c.split_mode != HGEMM_SPLIT_WORKSPACE && c.split_mode != HGEMM_SPLIT_CLUSTER) || (c.tail_mode != HGEMM_TAIL_K && c.tail_mode != HGEMM_TAIL_N) ||
            (K % 8) != 0 || (N % 8) != 0)
            return HGEMM_ERR_UNSUPPORTED;
        if (ceil_div(M, c.block_n) * ceil_div(N, c.block_n) * c.split_k >= (int64_t(1) << 30)) return HGEMM_ERR_UNSUPPORTED;
        return HGEMM_OK;
    }
    if (c.family != HGEMM_FAMILY_UMMA_1CTA && c.family != HGEMM_FAMILY_UMMA_2CTA && c.family != HGEMM_FAMILY_LIGHT) return HGEMM_ERR_UNSUPPORTED;
    if (c.family == HGEMM_FAMILY_LIGHT) {
        // one plain tile per CTA: nothing that needs the persistent kernel's extra paths
        if (c.split_k != 1 || c.tail_split >= 2 || c.swap_ab || c.accumulate != HGEMM_ACC_F32 || c.epilogue == HGEMM_EPILOGUE_TMA_WIDE ||
            c.raster_mode != HGEMM_RASTER_SWEEP || c.block_n > 256 || (K % 8) != 0 || (N % 8) != 0)
            return HGEMM_ERR_UNSUPPORTED;
    }
    const int cg = cta_group_of(c);
    if (c.block_m != 128 * cg || (c.block_k != 64 && c.block_k != 128)) return HGEMM_ERR_UNSUPPORTED;
    if (c.block_n == 512) {
        // the double-accumulator pair tile (256 x 512): whole tiles only, nothing that needs a spare accumulator or
        // another column order
        if (cg != 2 || c.split_k != 1 || c.tail_split >= 2 || c.swap_ab || (N % 512) != 0) return HGEMM_ERR_UNSUPPORTED;
    } else if (c.block_n < 32 || c.block_n > 256 || (c.block_n % 32) != 0) {
        return HGEMM_ERR_UNSUPPORTED;
    }
    if (c.stages < 1 || c.stages > 12) return HGEMM_ERR_UNSUPPORTED;
    if (smem_bytes(c) > kSmemOptInBytes) return HGEMM_ERR_UNSUPPORTED;
    if (c.split_k < 1 || c.split_k > ceil_div(K, c.block_k)) return HGEMM_ERR_UNSUPPORTED;
    // the slices of one tile wait for each other, so they must all be resident at once
    if (c.split_k > kMaxSplitK) return HGEMM_ERR_UNSUPPORTED;
    if (c.raster_group < 1) return HGEMM_ERR_UNSUPPORTED;
    if (c.epilogue != HGEMM_EPILOGUE_DIRECT && c.epilogue != HGEMM_EPILOGUE_TMA && c.epilogue != HGEMM_EPILOGUE_TMA_WIDE)
        return HGEMM_ERR_UNSUPPORTED;
    if (c.epilogue == HGEMM_EPILOGUE_TMA_WIDE) {
        // 64-column store boxes: whole boxes per tile and per column piece, and no partial sums to exchange
        if (c.split_k != 1 || (c.block_n % 64) != 0) return HGEMM_ERR_UNSUPPORTED;
        if (c.tail_split >= 2 && c.tail_mode == HGEMM_TAIL_N && (c.block_n % (64 * c.tail_split)) != 0) return HGEMM_ERR_UNSUPPORTED;
    }
    if (c.reserved[0] != 0) return HGEMM_ERR_UNSUPPORTED;
    // wave pacing: whole, equal tiles of the persistent kernel
    if (c.wave_pace != 0 && (c.wave_pace != 1 || c.family == HGEMM_FAMILY_LIGHT || c.split_k != 1 || c.tail_split >= 2)) return HGEMM_ERR_UNSUPPORTED;
    if (c.accumulate != HGEMM_ACC_F32 && c.accumulate != HGEMM_ACC_F16) return HGEMM_ERR_UNSUPPORTED;
    // fp16 accumulators: no fp16 partial sums are exchanged, so no split along K
    if (c.accumulate == HGEMM_ACC_F16 && (c.split_k != 1 || (c.tail_split >= 2 && c.tail_mode != HGEMM_TAIL_N))) return HGEMM_ERR_UNSUPPORTED;
    if (c.tail_split < 0 || c.tail_split > 16 || (c.tail_split >= 2 && c.split_k != 1)) return HGEMM_ERR_UNSUPPORTED;
    if (c.tail_mode != HGEMM_TAIL_K && c.tail_mode != HGEMM_TAIL_N && c.tail_mode != HGEMM_TAIL_STREAM) return HGEMM_ERR_UNSUPPORTED;
    // stream-K: partial sums in fp32 through the workspace; the transposed stores and the light kernel have no such path
    if (c.tail_mode == HGEMM_TAIL_STREAM && (c.swap_ab || c.family == HGEMM_FAMILY_LIGHT || c.block_n > 256 || c.epilogue == HGEMM_EPILOGUE_TMA_WIDE))
        return HGEMM_ERR_UNSUPPORTED;
    if (c.tail_mode == HGEMM_TAIL_N && c.tail_split >= 2) {
        // column pieces: whole 32-column chunks, and for a pair a whole number of 8-row groups of B per CTA
        if ((c.tail_split != 2 && c.tail_split != 4) || (c.block_n % (32 * c.tail_split)) != 0) return HGEMM_ERR_UNSUPPORTED;
    }
    if (c.split_mode != HGEMM_SPLIT_WORKSPACE && c.split_mode != HGEMM_SPLIT_CLUSTER) return HGEMM_ERR_UNSUPPORTED;
    if (c.split_k > 1 && c.split_mode == HGEMM_SPLIT_CLUSTER) {
        if (cg * c.split_k > 16) return HGEMM_ERR_UNSUPPORTED;   // the largest cluster holds 16 CTAs
        // once the main loops are done, the stage ring and the store staging behind it hold this CTA's fp32
        // partial (128 x block_n) and the S - 1 copies of its share that the other slices send
        const int64_t units = int64_t(128) * c.block_n / 4;                    // float4 units of a tile
        const int64_t cap = ceil_div(units, c.split_k);
        if (int64_t(c.stages) * stage_bytes(c) + kStagingBytes < (units + (c.split_k - 1) * cap) * 16) return HGEMM_ERR_UNSUPPORTED;
    }
    const int64_t tiles = ceil_div(M, 128 * cg) * ceil_div(N, c.block_n);
    if (tiles * c.split_k >= (int64_t(1) << 30)) return HGEMM_ERR_UNSUPPORTED;
    if (c.split_k > 1 && c.split_mode == HGEMM_SPLIT_WORKSPACE &&
        tiles * c.split_k * cg * 128 * int64_t(c.block_n) * 4 > kMaxWorkspaceBytes)
        return HGEMM_ERR_UNSUPPORTED;
    return HGEMM_OK;
}

double estimate_cycles(int64_t M, int64_t N, int64_t K, int32_t num_sms, const hgemm_config_t &c)
{
    if (c.family == HGEMM_FAMILY_SMALL) {
        // Not fitted: a ranking hint.  Per 64-wide k-block a CTA with 64 x 64 tiles moves 16 KB into shared memory and
        // issues 128 MMAs of 16 x 8 x 16 (a quarter of both with 32 x 32 tiles); a few CTAs share an SM; a short fixed part.
        const double t = c.block_n == 32 ? 0.3 : 1.0;
        const int32_t S = std::max(1, c.split_k);
        const double waves = std::ceil(double(ceil_div(M, c.block_n) * ceil_div(N, c.block_n) * S) / ((c.block_n == 32 ? 8.0 : 4.0) * std::max(1, num_sms)));
        // K slices run side by side; their sum costs a cluster barrier and S reads per element
        return 1400.0 + waves * (double(ceil_div(ceil_div(K, 64), S)) * 600.0 * t + 600.0) + (S > 1 ? 900.0 + 40.0 * S : 0.0);
    }
    // Rough machine model, in SM clock cycles: a ranking aid, not a prediction.  Its form follows the kernel
    // (waves of tiles, k-blocks bounded by the tensor pipe, the stage hand-off, the fill rate of one SM, the
    // aggregate L2 rate or the latency the stage ring can hide; a drain, a reduction for split-K); its constants
    // are a least-squares fit (log error, soft L1) to 32,579 timings of 839 shapes -- the 729 grid shapes and 110
    // others, the tuner's best 24 candidates and 16 random ones each -- on a B200.  Picking by this model among
    // the timed candidates loses 8 % (geometric mean; 26 % at the 90th percentile) against the fastest one.
    const double kMacPerClk = 4096.0;        // fp16 MACs per clock per SM
    const double kSmFillBytesPerClk = 95.0;   // L2 -> one SM's shared memory
    const double kL2BytesPerClk = 7377.1;     // L2 -> all SMs together
    const double kHbmBytesPerClk = 1997.5;    // HBM, all SMs together
    const double kFillLatency = 5079.0;       // first k-block of a work item: TMA round trip
    const double kLaunch = 375.0;
    const double kMmaIssue = 8.75;            // per MMA instruction
    const double kStageFixed = 512.3;         // per stage: barrier hand-off both ways
    const double kLatencyWarm = 1942.8, kLatencyCold = 3130.1;   // what the stage ring has to hide: operands in L2 / in HBM
    const double kPairExtra = 496.8;          // set-up and teardown of a CTA pair
    const double kDirectStores = 1.65;         // drain with direct stores relative to TMA stores
    const double kWideStores = 0.8;            // ... with 64-column boxes (measured on the chunk loop, not fitted)

    const int cg = cta_group_of(c);
    const int64_t units = std::max(1, num_sms / cg);
    const SplitLayout L = split_layout(M, N, K, num_sms, c);   // (trades M and N itself for a swapped configuration)
    if (c.swap_ab) std::swap(M, N);                            // from here on: the problem as the kernel tiles it
    const int64_t work = L.work_items;
    // a cut tail wave costs 1 / slices of a wave (plus the reduction, added below), or a little more than
    // 1 / pieces (narrower tiles run below the wide ones' rate)
    double wave_count;
    if (c.split_k > 1) wave_count = double(ceil_div(work, units));
    else if (L.stream_units > 0) wave_count = double(L.first_split_tile) / double(units) + double(L.tiles - L.first_split_tile) / double(L.stream_units);
    else if (L.slices > 1) wave_count = double(L.first_split_tile) / double(units) + 1.0 / double(L.slices);
    else if (L.pieces > 1) wave_count = double(L.first_split_tile) / double(units) + 1.52 / double(L.pieces);
    else wave_count = double(ceil_div(L.tiles, units));
    const int64_t kb = ceil_div(K, c.block_k);
    const int64_t kb_per = ceil_div(kb, c.split_k);
    const double cta_bytes_kb = double(stage_bytes(c));
    const double subs = c.block_k / 64.0;
    const double mma_kb = std::max(128.0 * c.block_n * c.block_k / kMacPerClk, subs * 4.0 * kMmaIssue + kStageFixed);
    const double fill_kb = cta_bytes_kb / kSmFillBytesPerClk;
    const double concurrent_ctas = double(std::min(work, units)) * cg;
    const double l2_kb = concurrent_ctas * cta_bytes_kb / kL2BytesPerClk;
    const bool cold = 2.0 * (double(M) * K + double(N) * K) > 100e6;          // the operands do not stay in L2
    const double latency_kb = (cold ? kLatencyCold : kLatencyWarm) / double(c.stages);
    const double t_kb = std::max(std::max(mma_kb, fill_kb), std::max(l2_kb, latency_kb));
    const double epilogue = (12.73 * c.block_n + 75.0) *
                            (c.epilogue == HGEMM_EPILOGUE_DIRECT ? kDirectStores : c.epilogue == HGEMM_EPILOGUE_TMA_WIDE ? kWideStores : 1.0);
    double t = wave_count * (double(kb_per) * t_kb + 0.25 * kFillLatency) + 0.75 * kFillLatency + epilogue + (cg - 1) * kPairExtra;
    const double partial = 128.0 * c.block_n * 4.0;
    if (c.split_k == 1 && L.slices > 1) t += (partial / 26.4 + 10069.4) * (L.stream_units > 0 ? 1.5 : 1.0);   // the tail's reduction (stream-K: two items)
    double bytes = 2.0 * (double(M) * K + double(N) * K + double(M) * N);
    if (c.split_k > 1) {
        if (c.split_mode == HGEMM_SPLIT_CLUSTER) {
            // stage in shared memory, send (S - 1) / S of it through the cluster network, ordered sum; only rows
            // that exist in C take part
            const double live = M < 128 ? double((M + 31) / 32 * 32) / 128.0 : 1.0;
            const double p_live = partial * live;
            t += p_live / 560.0 + p_live * double(c.split_k - 1) / double(c.split_k) / 8.72 + p_live / 360.0 + 2177.5;
        } else {
            t += partial / 26.4 + 11110.1;                      // park, signal, wait, pull through L2
            bytes += 2.0 * double(work) * cg * partial;
        }
    }
    t = std::max(t, bytes / kHbmBytesPerClk);
    if (c.family == HGEMM_FAMILY_LIGHT) {
        // not persistent: every wave of CTAs pays its own start, and nothing overlaps a tile's epilogue; in exchange
        // the set-up is shorter (its first loads overlap it).  Not fitted: a ranking hint so that the tuner times it
        const double waves = double(ceil_div(L.tiles, units));
        t = t - 600.0 + (waves - 1.0) * (epilogue + 0.5 * kFillLatency);
    }
    return t + kLaunch;
}

hgemm_status_t heuristic(int64_t M, int64_t N, int64_t K, int32_t num_sms, hgemm_config_t *out)
{
    const hgemm_status_t s = validate_shape(M, N, K);
    if (s != HGEMM_OK) return s;
    if (num_sms < 2) num_sms = 148;
    static const int32_t kSplits[] = {1, 2, 3, 4, 6, 8, 12, 16, 24, 32, 48, 64};
    const int64_t kb = ceil_div(K, 64);
    hgemm_config_t best;
    double best_t = 0.0;
    bool have = false;
    for (int family = 0; family < 2; ++family) {
        const int cg = family == HGEMM_FAMILY_UMMA_2CTA ? 2 : 1;
        for (int32_t bn = 32; bn <= 256; bn += 32) {
            if (bn > 32 && bn - 32 >= N) break;   // a wider tile would only add padding
            for (int32_t split : kSplits) {
                if (split > kb) break;
                for (int mode = 0; mode < 2; ++mode) {
                if (mode == 1 && (split == 1 || split * cg > 16)) continue;
                hgemm_config_t c;
                std::memset(&c, 0, sizeof(c));
                c.split_mode = mode;
                c.family = family;
                c.block_m = 128 * cg;
                c.block_n = bn;
                c.block_k = (K >= 1024 && split == 1) ? 128 : 64;
                c.split_k = split;
                c.epilogue = split == 1 ? HGEMM_EPILOGUE_TMA : HGEMM_EPILOGUE_DIRECT;
                c.stages = std::max(1, std::min<int32_t>(max_stages(family, bn, c.block_k), 8));
                const int64_t units = std::max(1, num_sms / cg);
                const int64_t tiles = ceil_div(M, 128 * cg) * ceil_div(N, bn);
                if (split > 1 && tiles * split > 2 * units) continue;   // split-K only to fill an under-full machine
                const double g = std::sqrt(double(units) * bn / (128.0 * cg));
                c.raster_group = int32_t(std::max<int64_t>(1, std::min<int64_t>(ceil_div(M, 128 * cg), int64_t(g + 0.5))));
                if (validate(M, N, K, c) != HGEMM_OK) continue;
                const double t = estimate_cycles(M, N, K, num_sms, c);
                if (!have || t < best_t) {
                    best = c;
                    best_t = t;
                    have = true;
                }
                }
            }
        }
    }
    if (!have) return HGEMM_ERR_UNSUPPORTED;
    *out = best;
    return HGEMM_OK;
}

namespace {

int32_t raster_group_for(int64_t M, int32_t num_sms, const hgemm_config_t &c)
{
    const int cg = cta_group_of(c);
    const int64_t units = std::max(1, num_sms / cg);
    const double g = std::sqrt(double(units) * c.block_n / (128.0 * cg));
    return int32_t(std::max<int64_t>(1, std::min<int64_t>(ceil_div(M, 128 * cg), int64_t(g + 0.5))));
}

} // namespace

int32_t ranked_candidates(int64_t M, int64_t N, int64_t K, int32_t num_sms, hgemm_config_t *out, int32_t max)
{
    if (!out || max < 1 || validate_shape(M, N, K) != HGEMM_OK) return 0;
    if (num_sms < 2) num_sms = 148;
    static const int32_t kSplits[] = {1, 2, 3, 4, 6, 8, 12, 16, 24, 32, 48, 64};
    std::vector<std::pair<double, hgemm_config_t>> all;
    auto add = [&](const hgemm_config_t &c) {
        if (validate(M, N, K, c) == HGEMM_OK) all.emplace_back(estimate_cycles(M, N, K, num_sms, c), c);
    };
    if (double(M) * double(N) * double(K) <= 2147483648.0) {        // the register-accumulator kernel: small problems only
        hgemm_config_t c;
        std::memset(&c, 0, sizeof(c));
        c.family = HGEMM_FAMILY_SMALL;
        c.block_m = c.block_n = c.block_k = 64;
        c.stages = 3;
        c.split_k = 1;
        c.raster_group = 1;
        add(c);                                                     // (validate() keeps it to K % 8 == 0 and N % 8 == 0)
        c.block_m = c.block_n = 32;
        add(c);
        c.split_mode = HGEMM_SPLIT_CLUSTER;                         // the same with the K loop cut into the CTAs of a cluster
        for (int32_t tile = 64; tile >= 32; tile -= 32)
            for (int32_t split = 2; split <= 16; split *= 2) {
                c.block_m = c.block_n = tile;
                c.split_k = split;
                if (ceil_div(M, tile) * ceil_div(N, tile) * split <= 8 * int64_t(num_sms)) add(c);
            }
    }
    // swap == 1: the operands trade places (few rows, many columns: the rows of B fill the MMA's 128-row side)
    for (int swap = 0; swap < 2; ++swap) {
    if (swap == 1 && !(M <= 256 && N >= 512 && (N % 8) == 0)) continue;
    const int64_t Mk = swap ? N : M, Nk = swap ? M : N;              // the problem as the kernel tiles it
    for (int family = 0; family < 3; ++family) {
        const bool light = family == HGEMM_FAMILY_LIGHT;
        if (light && (swap || (K % 8) != 0 || (N % 8) != 0)) continue;
        const int cg = family == HGEMM_FAMILY_UMMA_2CTA ? 2 : 1;
        const int64_t units = std::max(1, num_sms / cg);
        for (int32_t bn = 32; bn <= 512; bn += (bn == 256 ? 256 : 32)) {      // 32 .. 256, then the 512-wide double tile
            if (bn > 32 && bn - 32 >= Nk) break;                       // a wider tile would only add padding
            if (bn == 512 && (family != HGEMM_FAMILY_UMMA_2CTA || swap || (Nk % 512) != 0)) continue;
            const int64_t tiles = ceil_div(Mk, 128 * cg) * ceil_div(Nk, bn);
            const int64_t tail = tiles % units;
            for (int32_t bk = 64; bk <= 128; bk += 64) {
                if (bn == 512 && bk == 128) continue;                 // two stages only: not worth a candidate
                if (bk == 128 && K < 128) continue;
                const int64_t kb = ceil_div(K, bk);
                for (int32_t split : kSplits) {
                    if (split > kb) break;
                    if (split > 1 && (light || tiles * split > 2 * units)) continue;   // split-K only to fill an under-full machine
                    for (int mode = 0; mode < 2; ++mode) {
                        if (mode == 1 && (split == 1 || split * cg > 16)) continue;
                        for (int epi = 0; epi < 3; ++epi) {
                            if (split > 1 && epi != HGEMM_EPILOGUE_DIRECT) continue;
                            if (light && epi == HGEMM_EPILOGUE_TMA_WIDE) continue;
                            if (epi == HGEMM_EPILOGUE_TMA_WIDE && ((bn % 64) != 0 || swap)) continue;
                            hgemm_config_t c;
                            std::memset(&c, 0, sizeof(c));
                            c.family = family;
                            c.block_m = 128 * cg;
                            c.block_n = bn;
                            c.block_k = bk;
                            c.split_k = split;
                            c.split_mode = mode;
                            c.epilogue = epi;
                            c.swap_ab = swap;
                            c.stages = std::min<int32_t>(max_stages_of(c), 8);
                            if (light) c.stages = int32_t(std::min<int64_t>(std::min<int32_t>(max_stages_of(c), 12), kb));   // no more stages than k-blocks
                            if (c.stages < 1) continue;
                            c.raster_group = light ? 1 : raster_group_for(Mk, num_sms, c);
                            add(c);
                            if (split == 1 && !swap && !light && epi != HGEMM_EPILOGUE_TMA_WIDE && (tiles % units) != 0) {
                                // the tiles beyond the full waves as a stream-K tail (where the layout applies to this shape)
                                hgemm_config_t t = c;
                                t.tail_split = 2;
                                t.tail_mode = HGEMM_TAIL_STREAM;
                                if (split_layout(M, N, K, num_sms, t).stream_units > 0) add(t);
                            }
                            if (split == 1 && !swap && !light && tiles > units && tail > 0 && tail <= units / 2) {
                                const int32_t ts = int32_t(std::min<int64_t>(std::min<int64_t>(units / tail, 8), kb));
                                if (ts >= 2) {
                                    hgemm_config_t t = c;
                                    t.tail_split = ts;
                                    t.tail_mode = HGEMM_TAIL_K;
                                    add(t);
                                }
                                for (int32_t pieces = 2; pieces <= 4; pieces *= 2) {
                                    if (tail * pieces > units || (bn % (32 * pieces)) != 0) continue;
                                    hgemm_config_t t = c;
                                    t.tail_split = pieces;
                                    t.tail_mode = HGEMM_TAIL_N;
                                    add(t);
                                }
                            }
                        }
                    }
                }
            }
        }
    }
    }
    std::stable_sort(all.begin(), all.end(), [](const auto &a, const auto &b) { return a.first < b.first; });
    const int32_t n = int32_t(std::min<size_t>(all.size(), size_t(max)));
    for (int32_t i = 0; i < n; ++i) out[i] = all[size_t(i)].second;
    return n;
}


hgemm_status_t plan_config(int64_t M, int64_t N, int64_t K, int32_t num_sms, hgemm_config_t *out)
{
    if (table_lookup(M, N, K, out)) return HGEMM_OK;
    hgemm_config_t own;
    const hgemm_status_t hs = heuristic(M, N, K, num_sms, &own);
    TableNeighbour nb[8];
    const int count = table_neighbours(M, N, K, nb, 8);
    if (count == 0) {
        if (hs == HGEMM_OK) *out = own;
        return hs;
    }
    if (num_sms < 2) num_sms = 148;
    // measured time per estimated cycle at each neighbour: how far off the cost model is around here
    double calib[8], log_sum = 0.0;
    int calibrated = 0;
    for (int i = 0; i < count; ++i) {
        const double est = estimate_cycles(nb[i].M, nb[i].N, nb[i].K, num_sms, nb[i].cfg);
        calib[i] = (nb[i].us > 0.0 && est > 0.0) ? nb[i].us / est : 0.0;
        if (calib[i] > 0.0) {
            log_sum += std::log(calib[i]);
            ++calibrated;
        }
    }
    const double calib_mean = calibrated ? std::exp(log_sum / calibrated) : 1.0;
    bool have = false;
    double best_score = 0.0;
    hgemm_config_t best;
    auto consider = [&](const hgemm_config_t &c, double scale) {
        if (validate(M, N, K, c) != HGEMM_OK) return;
        const double score = estimate_cycles(M, N, K, num_sms, c) * scale;
        if (!have || score < best_score) {
            have = true;
            best_score = score;
            best = c;
        }
    };
    if (hs == HGEMM_OK) consider(own, calib_mean);
    for (int i = 0; i < count; ++i) {
        const double scale = calib[i] > 0.0 ? calib[i] : calib_mean;
        hgemm_config_t c = nb[i].cfg;
        c.raster_group = raster_group_for(c.swap_ab ? N : M, num_sms, c);
        c.tail_split = 0;
        c.tail_mode = HGEMM_TAIL_K;
        c.stages = std::min(c.stages, max_stages_of(c));
        if (c.stages < 1) continue;
        const int cg = cta_group_of(c);
        const int64_t kb_here = ceil_div(K, c.block_k), kb_there = ceil_div(nb[i].K, c.block_k);
        // the neighbour's split factor, and the one that keeps its k-blocks per slice
        int32_t splits[2] = {c.split_k, c.split_k};
        if (c.split_k > 1) splits[1] = int32_t(std::max<int64_t>(1, (c.split_k * kb_here + kb_there / 2) / kb_there));
        for (int v = 0; v < 2; ++v) {
            if (v == 1 && splits[1] == splits[0]) break;
            hgemm_config_t d = c;
            d.split_k = int32_t(std::min<int64_t>(splits[v], kb_here));
            if (d.split_k > 1 && d.split_mode == HGEMM_SPLIT_CLUSTER && d.split_k * cg > 16) d.split_k = 16 / cg;
            if (d.split_k <= 1) {
                d.split_k = 1;
                d.split_mode = HGEMM_SPLIT_WORKSPACE;
                d.epilogue = nb[i].cfg.split_k > 1 ? HGEMM_EPILOGUE_TMA : d.epilogue;
            }
            consider(d, scale);
            if (d.split_k == 1 && !d.swap_ab) {
                // the last wave's tiles as column pieces, where the wave is at most half full
                const int64_t units = std::max(1, num_sms / cg);
                const int64_t tiles = ceil_div(M, 128 * cg) * ceil_div(N, d.block_n);
                const int64_t tail = tiles % units;
                for (int32_t pieces = 2; pieces <= 4; pieces *= 2) {
                    if (tiles > units && tail > 0 && tail * pieces <= units && d.block_n % (32 * pieces) == 0) {
                        hgemm_config_t t = d;
                        t.tail_split = pieces;
                        t.tail_mode = HGEMM_TAIL_N;
                        consider(t, scale);
                    }
                }
            }
        }
    }
    if (!have) return hs == HGEMM_OK ? HGEMM_ERR_UNSUPPORTED : hs;
    *out = best;
    return HGEMM_OK;
}

} // namespace hgemm_host
