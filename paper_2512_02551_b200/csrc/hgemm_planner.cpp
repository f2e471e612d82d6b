// Host-only planner (see hgemm_planner.h).  No CUDA calls in this file.
#include "hgemm_planner.h"

#include <algorithm>
#include <cmath>
#include <cstring>

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

int64_t smem_bytes(const hgemm_config_t &c)
{
    return kAlignSlack + int64_t(c.stages) * stage_bytes(c) + kStagingBytes + kCtrlBytes;
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

SplitLayout split_layout(int64_t M, int64_t N, int64_t K, int32_t num_sms, const hgemm_config_t &c)
{
    const int cg = cta_group_of(c);
    SplitLayout L;
    L.tiles = ceil_div(M, 128 * cg) * ceil_div(N, c.block_n);
    L.first_split_tile = L.tiles;
    L.slices = 1;
    L.pieces = 1;
    if (c.split_k > 1) {
        L.first_split_tile = 0;
        L.slices = c.split_k;
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
    if (c.family != HGEMM_FAMILY_UMMA_1CTA && c.family != HGEMM_FAMILY_UMMA_2CTA) return HGEMM_ERR_UNSUPPORTED;
    const int cg = cta_group_of(c);
    if (c.block_m != 128 * cg || (c.block_k != 64 && c.block_k != 128)) return HGEMM_ERR_UNSUPPORTED;
    if (c.block_n < 32 || c.block_n > 256 || (c.block_n % 32) != 0) return HGEMM_ERR_UNSUPPORTED;
    if (c.stages < 1 || c.stages > 12) return HGEMM_ERR_UNSUPPORTED;
    if (smem_bytes(c) > kSmemOptInBytes) return HGEMM_ERR_UNSUPPORTED;
    if (c.split_k < 1 || c.split_k > ceil_div(K, c.block_k)) return HGEMM_ERR_UNSUPPORTED;
    // the slices of one tile wait for each other, so they must all be resident at once
    if (c.split_k > kMaxSplitK) return HGEMM_ERR_UNSUPPORTED;
    if (c.raster_group < 1) return HGEMM_ERR_UNSUPPORTED;
    if (c.epilogue != HGEMM_EPILOGUE_DIRECT && c.epilogue != HGEMM_EPILOGUE_TMA) return HGEMM_ERR_UNSUPPORTED;
    for (int i = 0; i < 4; ++i)
        if (c.reserved[i] != 0) return HGEMM_ERR_UNSUPPORTED;
    if (c.accumulate != HGEMM_ACC_F32 && c.accumulate != HGEMM_ACC_F16) return HGEMM_ERR_UNSUPPORTED;
    // fp16 accumulators: no fp16 partial sums are exchanged, so no split along K
    if (c.accumulate == HGEMM_ACC_F16 && (c.split_k != 1 || (c.tail_split >= 2 && c.tail_mode == HGEMM_TAIL_K))) return HGEMM_ERR_UNSUPPORTED;
    if (c.tail_split < 0 || c.tail_split > 16 || (c.tail_split >= 2 && c.split_k != 1)) return HGEMM_ERR_UNSUPPORTED;
    if (c.tail_mode != HGEMM_TAIL_K && c.tail_mode != HGEMM_TAIL_N) return HGEMM_ERR_UNSUPPORTED;
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
    if (workspace_bytes(M, N, K, c) > kMaxWorkspaceBytes) return HGEMM_ERR_UNSUPPORTED;
    return HGEMM_OK;
}

double estimate_cycles(int64_t M, int64_t N, int64_t K, int32_t num_sms, const hgemm_config_t &c)
{
    // Rough machine model, in SM clock cycles.  Constants are fitted by eye to measurements
    // on a B200; the tuned table overrides this wherever it has an entry.
    const double kMacPerClk = 4096.0;        // fp16 MACs per clock per SM
    const double kSmFillBytesPerClk = 90.0;  // L2 -> one SM's shared memory
    const double kL2BytesPerClk = 5500.0;    // L2 -> all SMs together
    const double kHbmBytesPerClk = 3400.0;   // HBM, all SMs together
    const double kFillLatency = 1800.0;      // first k-block of a work item: TMA round trip
    const double kLaunch = 3000.0;

    const int cg = cta_group_of(c);
    const int64_t bm = 128 * cg;
    const int64_t tiles = ceil_div(M, bm) * ceil_div(N, c.block_n);
    const int64_t units = std::max(1, num_sms / cg);
    const SplitLayout L = split_layout(M, N, K, num_sms, c);
    const int64_t work = L.work_items;
    // a split tail wave costs 1 / slices of a wave (plus the reduction, added below)
    double wave_count;
    if (c.split_k > 1) wave_count = double(ceil_div(work, units));
    else if (L.slices > 1) wave_count = double(L.first_split_tile) / double(units) + 1.0 / double(L.slices);
    else if (L.pieces > 1) wave_count = double(L.first_split_tile) / double(units) + 1.1 / double(L.pieces);   // narrower tiles run a little below the wide ones' rate
    else wave_count = double(ceil_div(L.tiles, units));
    const int64_t kb = ceil_div(K, c.block_k);
    const int64_t kb_per = ceil_div(kb, c.split_k);
    const double cta_bytes_kb = double(stage_bytes(c));
    // issuing one MMA costs the issuing thread about 70 cycles whatever its width, plus a fixed
    // wait + commit per stage: narrow tiles are issue-bound
    const double subs = c.block_k / 64.0;
    const double mma_kb = std::max(128.0 * c.block_n * c.block_k / kMacPerClk, subs * 4.0 * 70.0 + 180.0);
    const double fill_kb = cta_bytes_kb / kSmFillBytesPerClk;
    const double concurrent_ctas = double(std::min(work, units)) * cg;
    const double l2_kb = concurrent_ctas * cta_bytes_kb / kL2BytesPerClk;
    const double t_kb = std::max(mma_kb, std::max(fill_kb, l2_kb));
    const double epilogue = 5.0 * c.block_n + 600.0;   // the last tile's drain: 32-column chunks, two warps per row quarter
    double t = wave_count * (double(kb_per) * t_kb + 0.25 * kFillLatency) + 0.75 * kFillLatency + epilogue;
    if (c.split_k == 1 && L.slices > 1) t += 128.0 * c.block_n * 4.0 / 48.0 + 9000.0;   // the tail's reduction
    double bytes = 2.0 * (double(M) * K + double(N) * K + double(M) * N);
    if (c.split_k > 1) {
        const double partial = 128.0 * c.block_n * 4.0;
        if (c.split_mode == HGEMM_SPLIT_CLUSTER) {
            // stage in shared memory, send (S - 1) / S of it through the cluster network (about 18 bytes per
            // clock per SM), ordered sum; only rows that exist in C take part
            const double live = M < 128 ? double((M + 31) / 32 * 32) / 128.0 : 1.0;
            const double p_live = partial * live;
            t += p_live / 70.0 + p_live * double(c.split_k - 1) / double(c.split_k) / 18.0 + p_live / 45.0 + 800.0;
        } else {
            t += partial / 64.0 + partial / 48.0 + 9000.0;                      // park, signal, wait, pull through L2
            bytes += 2.0 * double(work) * cg * partial;
        }
    }
    t = std::max(t, bytes / kHbmBytesPerClk);
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

} // namespace hgemm_host
