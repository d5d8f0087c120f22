// Host builder of the scheduled backward's processing order (see bwd_schedule.hpp).
#include "bwd_schedule.hpp"

#include <algorithm>
#include <numeric>

namespace e3j {

size_t bwd_schedule_max_words(int T, int n_ranges, int64_t n_nodes, int64_t n_edges) {
    // tiles: every step wastes less than one tile per column set, every receiver row load may cost up to
    // kSchedStages empty tiles, plus one tile of slack per range
    const size_t tiles = (size_t)(n_edges + T - 1) / T + (size_t)(1 + kSchedStages) * (size_t)(n_nodes + n_ranges) + n_ranges;
    return 16 + (size_t)(n_ranges + 1) + (size_t)(n_nodes + 1) + 4 + tiles * (size_t)(T + 1) * 4;
}

int build_bwd_schedule(int T, int n_ranges, int64_t n_nodes, int64_t n_edges, const int32_t* senders,
                       const int32_t* receivers, std::vector<int32_t>& words) {
    const int64_t chunk = std::max<int64_t>(1, (n_edges + n_ranges - 1) / n_ranges);
    struct Run { int32_t sender, start, range, len, row; };
    std::vector<Run> runs;
    std::vector<int32_t> run_of((size_t)n_edges);
    {
        std::vector<int32_t> cur((size_t)n_nodes, -1);
        int32_t prev_r = 0;
        for (int64_t e = 0; e < n_edges; ++e) {
            const int32_t s = senders[e], r = receivers[e];
            if (s < 0 || s >= n_nodes || r < 0 || r >= n_nodes || r < prev_r) return -1;
            prev_r = r;
            const int32_t c = (int32_t)(e / chunk);
            int32_t id = cur[s];
            if (id >= 0 && runs[id].range == c && r - runs[id].start < kSchedWindow) {
                ++runs[id].len;
            } else {
                id = (int32_t)runs.size();
                runs.push_back({s, r, c, 1, -1});
                cur[s] = id;
            }
            run_of[e] = id;
        }
    }
    // rows: a sender's runs in creation order (= processing order), contiguous
    std::vector<int32_t> row_ptr((size_t)n_nodes + 1, 0);
    for (const Run& r : runs) ++row_ptr[r.sender + 1];
    std::partial_sum(row_ptr.begin(), row_ptr.end(), row_ptr.begin());
    {
        std::vector<int32_t> next(row_ptr.begin(), row_ptr.end() - 1);
        for (Run& r : runs) r.row = next[r.sender]++;
    }
    // edges of every run, ascending
    std::vector<int64_t> run_off(runs.size() + 1, 0);
    for (size_t i = 0; i < runs.size(); ++i) run_off[i + 1] = run_off[i] + runs[i].len;
    std::vector<int32_t> run_edges((size_t)n_edges);
    {
        std::vector<int64_t> fill(run_off.begin(), run_off.end() - 1);
        for (int64_t e = 0; e < n_edges; ++e) run_edges[fill[run_of[e]]++] = (int32_t)e;
    }

    const int rec = (T + 1) * 4;
    std::vector<int32_t> tile_ptr((size_t)n_ranges + 1, 0);
    std::vector<int32_t> tiles;   // all ranges, rec words per tile
    size_t run_pos = 0;           // runs are created range by range, step by step
    std::vector<int32_t> base;    // one range: T words per tile (edge or -1)
    std::vector<std::vector<int32_t>> col((size_t)T);
    for (int c = 0; c < n_ranges; ++c) {
        base.clear();
        for (auto& v : col) v.clear();
        // Columns run on from step to step (no padding to the step's fullest column): a tile may hold edges of two
        // neighbouring steps, i.e. of up to kSchedWindow + 1 receivers, which is what the slots hold.  What must
        // not happen is a receiver sharing a tile (or the kSchedStages tiles before it) with the previous occupant
        // of its slot: the rows of a step start no earlier than that.
        std::vector<int64_t> last_row;   // last row (tile of the range) that uses receiver r_first + i
        const int32_t r_first = (run_pos < runs.size() && runs[run_pos].range == c) ? runs[run_pos].start : 0;
        auto last_row_of = [&](int32_t r) -> int64_t {
            const int64_t i = (int64_t)r - r_first;
            return (i >= 0 && i < (int64_t)last_row.size()) ? last_row[i] : -1;
        };
        while (run_pos < runs.size() && runs[run_pos].range == c) {
            size_t end = run_pos;
            const int32_t k = runs[run_pos].start;
            while (end < runs.size() && runs[end].range == c && runs[end].start == k) ++end;
            int64_t guard = 0;
            for (int q = k; q < k + kSchedWindow; ++q) {
                const int64_t lr = last_row_of(q - kSchedSlots);
                if (lr >= 0) guard = std::max(guard, lr + 1 + kSchedStages);
            }
            for (auto& v : col)
                if ((int64_t)v.size() < guard) v.resize((size_t)guard, -1);
            std::vector<int32_t> order(end - run_pos);
            std::iota(order.begin(), order.end(), (int32_t)run_pos);
            std::stable_sort(order.begin(), order.end(), [&](int32_t a, int32_t b) { return runs[a].len > runs[b].len; });
            for (int32_t id : order) {
                int best = 0;
                for (int j = 1; j < T; ++j)
                    if (col[j].size() < col[best].size()) best = j;
                for (int64_t kk = run_off[id]; kk < run_off[id + 1]; ++kk) {
                    const int32_t e = run_edges[kk];
                    const size_t i = (size_t)(receivers[e] - r_first);
                    if (last_row.size() <= i) last_row.resize(i + 1, -1);
                    last_row[i] = std::max<int64_t>(last_row[i], (int64_t)col[best].size());
                    col[best].push_back(e);
                }
            }
            run_pos = end;
        }
        {
            size_t h = 0;
            for (auto& v : col) h = std::max(h, v.size());
            for (size_t i = 0; i < h; ++i)
                for (int j = 0; j < T; ++j) base.push_back(i < col[j].size() ? col[j][i] : -1);
        }
        const int n_base = (int)(base.size() / T);
        // first / last use of every receiver of the range (base tile index), receivers are a contiguous id range
        int32_t r_lo = 0, r_hi = -1;
        {
            const int64_t e0 = std::min<int64_t>(n_edges, (int64_t)c * chunk), e1 = std::min<int64_t>(n_edges, e0 + chunk);
            if (e1 > e0) { r_lo = receivers[e0]; r_hi = receivers[e1 - 1]; }
        }
        const int n_r = r_hi - r_lo + 1;
        std::vector<int32_t> first_use((size_t)std::max(n_r, 0), -1), last_use((size_t)std::max(n_r, 0), -1);
        for (int b = 0; b < n_base; ++b)
            for (int j = 0; j < T; ++j) {
                const int32_t e = base[(size_t)b * T + j];
                if (e < 0) continue;
                const int q = receivers[e] - r_lo;
                if (first_use[q] < 0) first_use[q] = b;
                last_use[q] = b;
            }
        // emit: empty tiles where a row's slot is not free in time; loads attached to the earliest legal tile
        const size_t range_first = tiles.size() / rec;
        tile_ptr[c] = (int32_t)range_first;
        std::vector<int32_t> out_of_base((size_t)n_base, 0);
        int32_t occupant[kSchedSlots];
        for (int u = 0; u < kSchedSlots; ++u) occupant[u] = -1;
        struct Load { int32_t tile, slot, receiver; };
        std::vector<Load> loads;
        std::vector<int> firsts;   // receivers in order of first use
        for (int q = 0; q < n_r; ++q)
            if (first_use[q] >= 0) firsts.push_back(q);
        std::stable_sort(firsts.begin(), firsts.end(), [&](int a, int b) { return first_use[a] < first_use[b]; });
        size_t fpos = 0;
        int32_t n_out = 0;
        auto push_tile = [&]() {
            tiles.resize(tiles.size() + rec, -1);
            int32_t* t = tiles.data() + tiles.size() - rec;
            t[T * 4 + 3] = 0;
            ++n_out;
        };
        for (int b = 0; b < n_base; ++b) {
            while (fpos < firsts.size() && first_use[firsts[fpos]] == b) {
                const int q = firsts[fpos++];
                const int u = (q + r_lo) % kSchedSlots;
                const int32_t p = occupant[u];
                const int32_t earliest = p >= 0 ? out_of_base[last_use[p]] + kSchedStages : 0;
                while (n_out < earliest) push_tile();   // empty tiles: the slot is still in use
                loads.push_back({std::min(earliest, n_out), u, q + r_lo});
                occupant[u] = q;
            }
            out_of_base[b] = n_out;
            push_tile();
            int32_t* t = tiles.data() + tiles.size() - rec;
            for (int j = 0; j < T; ++j) {
                const int32_t e = base[(size_t)b * T + j];
                if (e < 0) continue;
                const Run& r = runs[run_of[e]];
                const bool last_of_run = run_edges[run_off[run_of[e] + 1] - 1] == e;
                t[4 * j + 0] = e;
                t[4 * j + 1] = r.sender;
                t[4 * j + 2] = last_of_run ? r.row : -1;
                t[4 * j + 3] = receivers[e] % kSchedSlots;
            }
        }
        for (const Load& l : loads) tiles[(range_first + l.tile) * rec + T * 4 + l.slot] = l.receiver;
    }
    tile_ptr[n_ranges] = (int32_t)(tiles.size() / rec);

    const int32_t off_tile_ptr = 16;
    const int32_t off_row_ptr = off_tile_ptr + n_ranges + 1;
    int32_t off_tiles = off_row_ptr + (int32_t)n_nodes + 1;
    off_tiles = (off_tiles + 3) / 4 * 4;   // records are read 16 bytes at a time
    words.assign((size_t)off_tiles + tiles.size(), 0);
    const int32_t header[11] = {kSchedMagic, T, kSchedSlots, n_ranges, tile_ptr[n_ranges], (int32_t)runs.size(),
                                (int32_t)n_edges, (int32_t)n_nodes, off_tile_ptr, off_row_ptr, off_tiles};
    std::copy(header, header + 11, words.begin());
    std::copy(tile_ptr.begin(), tile_ptr.end(), words.begin() + off_tile_ptr);
    std::copy(row_ptr.begin(), row_ptr.end(), words.begin() + off_row_ptr);
    std::copy(tiles.begin(), tiles.end(), words.begin() + off_tiles);
    return 0;
}

}  // namespace e3j

extern "C" {

// Host-only entry for tests and tools: builds the schedule into caller memory (host pointers throughout).
// Returns 0, -1 (graph invalid) or -2 (capacity too small; *n_words holds the need).
int e3j_bwd_schedule_build_host(int T, int n_ranges, int64_t n_nodes, int64_t n_edges, const int32_t* senders,
                                const int32_t* receivers, int32_t* out_words, size_t capacity_words, size_t* n_words) {
    if (T < 1 || T > 31 || n_ranges < 1 || n_nodes < 0 || n_edges < 0 || !n_words) return -1;
    std::vector<int32_t> w;
    if (e3j::build_bwd_schedule(T, n_ranges, n_nodes, n_edges, senders, receivers, w)) return -1;
    *n_words = w.size();
    if (w.size() > capacity_words || !out_words) return -2;
    std::copy(w.begin(), w.end(), out_words);
    return 0;
}

}  // extern "C"
