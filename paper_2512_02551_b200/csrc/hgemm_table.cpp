// Tuned-table lookup (see hgemm_planner.h).  The table itself is generated on the GPU machine
// by the tuner and compiled in; an untabulated shape falls back to the heuristic.
#include <cmath>
#include <cstdio>
#include <cstdlib>
#include <cstring>
#include <mutex>
#include <vector>

#include "hgemm_planner.h"

namespace hgemm_host {

namespace {
struct Entry {
    int32_t M, N, K;
    int32_t family, block_n, block_k, stages, split_k, split_mode, tail_split, raster_group, epilogue;
    int32_t tail_mode;   // after the original columns, so that rows written before it existed still read as 0
    float us;            // time the tuner measured (0 in rows written before the column existed)
    int32_t swap_ab, raster_mode;   // later columns again: absent from older rows, which then read 0
    int32_t wave_pace;              // and again
};
const Entry kTable[] = {
#include "hgemm_table.inc"
    {0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0, 0.0f, 0, 0, 0}   // sentinel
};
// Rows read at run time from the file named by the environment variable HGEMM_TABLE (same row syntax as
// hgemm_table.inc, as the tuner writes it; lines that do not start with '{' are skipped): they take precedence over
// the compiled-in rows, so a table re-tuned on another box can be tried without rebuilding the library.
std::vector<Entry> g_file_rows;
std::once_flag g_file_once;

void load_file_rows()
{
    const char *path = std::getenv("HGEMM_TABLE");
    if (!path || !*path) return;
    FILE *f = std::fopen(path, "r");
    if (!f) return;
    char line[512];
    while (std::fgets(line, sizeof(line), f)) {
        const char *p = line;
        while (*p == ' ' || *p == '\t') ++p;
        if (*p != '{') continue;
        Entry e;
        std::memset(&e, 0, sizeof(e));
        const int n = std::sscanf(p, "{%d, %d, %d, %d, %d, %d, %d, %d, %d, %d, %d, %d, %d, %ff, %d, %d, %d", &e.M, &e.N, &e.K, &e.family, &e.block_n,
                                  &e.block_k, &e.stages, &e.split_k, &e.split_mode, &e.tail_split, &e.raster_group, &e.epilogue, &e.tail_mode,
                                  &e.us, &e.swap_ab, &e.raster_mode, &e.wave_pace);
        if (n >= 12 && e.M > 0 && e.N > 0 && e.K > 0) g_file_rows.push_back(e);
    }
    std::fclose(f);
}

const std::vector<Entry> &file_rows()
{
    std::call_once(g_file_once, load_file_rows);
    return g_file_rows;
}
} // namespace

namespace {
hgemm_config_t config_of(const Entry &e)
{
    hgemm_config_t c;
    std::memset(&c, 0, sizeof(c));
    c.family = e.family;
    c.block_m = e.family == HGEMM_FAMILY_UMMA_2CTA ? 256 : e.family == HGEMM_FAMILY_SMALL ? e.block_n : 128;
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
    c.wave_pace = e.wave_pace;
    return c;
}

} // namespace

int table_neighbours(int64_t M, int64_t N, int64_t K, TableNeighbour *out, int max_out)
{
    // the max_out tabulated shapes nearest in log space: distance |log M/M'| + |log N/N'| + |log K/K'|
    const std::vector<Entry> &extra = file_rows();
    const int nt = int(sizeof(kTable) / sizeof(kTable[0])) - 1, n = nt + int(extra.size());
    auto row = [&](int i) -> const Entry & { return i < nt ? kTable[i] : extra[size_t(i - nt)]; };
    if (n <= 0 || max_out <= 0) return 0;
    if (max_out > 8) max_out = 8;
    double dist[8];
    int idx[8];
    int count = 0;
    for (int i = 0; i < n; ++i) {
        const Entry &e = row(i);
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
        const Entry &e = row(idx[j]);
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
    for (const Entry &e : file_rows()) {                     // rows from the HGEMM_TABLE file first
        if (e.M == M && e.N == N && e.K == K) {
            const hgemm_config_t c = config_of(e);
            if (validate(M, N, K, c) != HGEMM_OK) break;     // an illegal row is ignored: the compiled-in table answers
            *out = c;
            return true;
        }
    }
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
