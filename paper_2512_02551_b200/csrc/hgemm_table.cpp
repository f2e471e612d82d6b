// Tuned-table lookup (see hgemm_planner.h).  The table itself is generated on the GPU machine
// by the tuner and compiled in; an untabulated shape falls back to the heuristic.
#include <cstring>

#include "hgemm_planner.h"

namespace hgemm_host {

namespace {
struct Entry {
    int32_t M, N, K;
    int32_t family, block_n, block_k, stages, split_k, split_mode, tail_split, raster_group, epilogue;
    int32_t tail_mode;   // last, so that rows written before it existed still read as 0
};
const Entry kTable[] = {
#include "hgemm_table.inc"
    {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0}   // sentinel
};
} // namespace

bool table_lookup(int64_t M, int64_t N, int64_t K, hgemm_config_t *out)
{
    const int n = int(sizeof(kTable) / sizeof(kTable[0])) - 1;
    for (int i = 0; i < n; ++i) {
        const Entry &e = kTable[i];
        if (e.M == M && e.N == N && e.K == K) {
            hgemm_config_t c;
            std::memset(&c, 0, sizeof(c));
            c.family = e.family;
            c.block_m = e.family == HGEMM_FAMILY_UMMA_2CTA ? 256 : 128;
            c.block_n = e.block_n;
            c.block_k = e.block_k;
            c.stages = e.stages;
            c.split_k = e.split_k;
            c.split_mode = e.split_mode;
            c.tail_split = e.tail_split;
            c.tail_mode = e.tail_mode;
            c.raster_group = e.raster_group;
            c.epilogue = e.epilogue;
            if (validate(M, N, K, c) != HGEMM_OK) return false;
            *out = c;
            return true;
        }
    }
    return false;
}

} // namespace hgemm_host
