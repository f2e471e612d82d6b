// Host-only planner: legality of a configuration, its resource needs, and the heuristic
// choice for a shape.  Pure functions, no CUDA calls, so they can be tested without a GPU.
//
// The configuration space is the paper's per-shape hyper-parameter space (sections 5.2 and
// 6: BM/BN/BK, stage count, block-swizzle stride) restated for tcgen05 tiles, plus split-K
// (which the paper does not use; skinny large-K shapes need it to fill 148 SMs).
#pragma once

#include <stdint.h>

#include "../../include/hgemm.h"

namespace hgemm_host {

constexpr int64_t kSmemOptInBytes = 232448;   // 227 KB per CTA on sm_100
constexpr int64_t kMaxWorkspaceBytes = int64_t(2) << 30;
constexpr int64_t kMaxDim = int64_t(1) << 22;
constexpr int32_t kMaxSplitK = 64;            // at most this many slices per tile (all co-resident)

inline int cta_group_of(const hgemm_config_t &c) { return c.family == HGEMM_FAMILY_UMMA_2CTA ? 2 : 1; }

int64_t stage_bytes(const hgemm_config_t &c);
int64_t smem_bytes(const hgemm_config_t &c);
int64_t staging_bytes(const hgemm_config_t &c);   // store staging of the epilogue warps (32 KB, 64 KB for the wide epilogue)
int32_t max_stages(int32_t family, int32_t block_n, int32_t block_k);   // with 32 KB of store staging
int32_t max_stages_of(const hgemm_config_t &c);                         // with this configuration's staging
// Which tiles are split: tiles [0, first_split_tile) are whole work items, the rest are cut into `slices`
// K slices.  Uniform split-K: first = 0; tail split: first = tiles - (tiles mod units) when it applies.
struct SplitLayout {
    int64_t tiles, first_split_tile, slices, work_items;
    int64_t pieces;   // > 1: the tiles from first_split_tile on are cut into this many column pieces (slices == 1)
    // stream-K tail (HGEMM_TAIL_STREAM): stream_units > 0 CTA positions share the k-blocks of the tiles from
    // first_split_tile on; `slices` is then the largest number of pieces any of those tiles is cut into, and
    // work_items = first_split_tile + 2 * grid units (two items per position, possibly empty).
    int64_t stream_units;
};
SplitLayout split_layout(int64_t M, int64_t N, int64_t K, int32_t num_sms, const hgemm_config_t &c);
int64_t workspace_bytes(int64_t M, int64_t N, int64_t K, const hgemm_config_t &c, int32_t num_sms = 148);
int64_t counter_bytes(int64_t M, int64_t N, const hgemm_config_t &c, int32_t num_sms = 148, int64_t K = 1 << 20);
hgemm_status_t validate_shape(int64_t M, int64_t N, int64_t K);
// The stricter rule of the kernels' own addressing: K % 8 == 0 and N % 8 == 0 (rows of 16-byte multiples).
// hgemm_plan lifts it by padding K in a plan-owned copy and by storing ragged C rows element by element.
hgemm_status_t validate_shape_aligned(int64_t M, int64_t N, int64_t K);
inline int64_t padded_k(int64_t K) { return (K + 7) & ~int64_t(7); }
hgemm_status_t validate(int64_t M, int64_t N, int64_t K, const hgemm_config_t &c);
hgemm_status_t heuristic(int64_t M, int64_t N, int64_t K, int32_t num_sms, hgemm_config_t *out);

// Estimated run time (arbitrary but consistent units: SM clock cycles) of a configuration;
// the heuristic picks the minimum over its candidate set.
double estimate_cycles(int64_t M, int64_t N, int64_t K, int32_t num_sms, const hgemm_config_t &c);

// Tuned table (generated on the box by the tuner; may be empty).  Returns true on a hit.
bool table_lookup(int64_t M, int64_t N, int64_t K, hgemm_config_t *out);

// The tuned shapes around an untabulated one: the (up to 8) tabulated shapes nearest to it in log space,
// nearest first, each with the time the tuner measured.
struct TableNeighbour {
    int64_t M, N, K;
    hgemm_config_t cfg;
    double us;          // measured time of cfg on (M, N, K); 0 if the table does not record it
};
int table_neighbours(int64_t M, int64_t N, int64_t K, TableNeighbour *out, int max_out);

// The configuration hgemm_plan uses: the table's entry for a tabulated shape; otherwise the candidate with
// the lowest calibrated estimate among the cost model's own choice and the neighbouring tuned shapes'
// configurations re-fitted to this shape (split factor clamped and also scaled with K, raster group and tail
// split recomputed), where a neighbour's candidates are scaled by (measured time / estimate) at that neighbour.
// The legal configurations of a shape, ranked by estimate_cycles (best first), at most `max` of them: both
// families, every tile width, both stage widths, the split factors that fill an under-full machine in both
// split modes, the three epilogues, and the tail cuts where the last wave is at most half full.  Returns the count.
int32_t ranked_candidates(int64_t M, int64_t N, int64_t K, int32_t num_sms, hgemm_config_t *out, int32_t max);
hgemm_status_t plan_config(int64_t M, int64_t N, int64_t K, int32_t num_sms, hgemm_config_t *out);

} // namespace hgemm_host
