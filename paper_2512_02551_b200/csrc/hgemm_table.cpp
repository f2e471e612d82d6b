// Tuned-table lookup (see hgemm_planner.h).  The table itself is generated on the GPU machine
// by the tuner and compiled in; an untabulated shape falls back to the heuristic.
#include <cmath>
#include <cstring>

#include "hgemm_planner.h"

namespace hgemm_host {

namespace {
struct Entry {
    int32_t M, N, K;
    int32_t family, block_n, block_k, stages, split_k, split_mode, tail_split, raster_group, epilogue;
    int32_t tail_mode;   // after the original columns, so that rows written before it existed still read as 0
    float us;            // time the tuner measured (0 in rows written before the column existed)
    int32_t swap_ab, raster_mode;   // later columns again: absent from older rows, which then read 0
};
const Entry kTable[] = {
#include "hgemm_table.inc"
    {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0.0f, 0, 0}   // sentinel
};
} // namespace

namespace {
hgemm_config_t config_of(const Entry &e)
{
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
    c.swap_ab = e.swap_ab;
    c.raster_mode = e.raster_mode;
    return c;
}

} // namespace

int table_neighbours(int64_t M, int64_t N, int64_t K, TableNeighbour *out, int max_out)
{
    // the max_out tabulated shapes nearest in log space: distance |log M/M'| + |log N/N'| + |log K/K'|
    const int n = int(sizeof(kTable) / sizeof(kTable[0])) - 1;
    if (n <= 0 || max_out <= 0) return 0;
    if (max_out > 8) max_out = 8;
    double dist[8];
    int idx[8];
    int count = 0;
    for (int i = 0; i < n; ++i) {
        const Entry &e = kTable[i];
        const double d = std::fabs(std::log(double(M) / double(e.M))) + std::fabs(std::log(double(N) / double(e.N))) +
                         std::fabs(std::log(double(K) / double(e.K)));
        int pos = count;
        while (pos > 0 && dist[pos - 1] > d) --pos;          // insertion into the sorted short list
        if (pos >= max_out) continue;
        const int last = count < max_out ? count : max_out - 1;
        for (int j = last; j > pos; --j) {
            dist[j] = dist[j - 1];
            idx[j] = idx[j - 1];
        }
        dist[pos] = d;
        idx[pos] = i;
        if (count < max_out) ++count;
    }
    for (int j = 0; j < count; ++j) {
        const Entry &e = kTable[idx[j]];
        out[j].M = e.M;
        out[j].N = e.N;
        out[j].K = e.K;
        out[j].cfg = config_of(e);
        out[j].us = e.us;
    }
    return count;
}

bool table_lookup(int64_t M, int64_t N, int64_t K, hgemm_config_t *out)
{
    const int n = int(sizeof(kTable) / sizeof(kTable[0])) - 1;
    for (int i = 0; i < n; ++i) {
        const Entry &e = kTable[i];
        if (e.M == M && e.N == N && e.K == K) {
            const hgemm_config_t c = config_of(e);
            if (validate(M, N, K, c) != HGEMM_OK) return false;
            *out = c;
            return true;
        }
    }
    return false;
}

} // namespace hgemm_host
