// Internal: processing order of the scheduled edge-wise backward (host side).
//
// The plain backward walks the receiver-sorted edge list and writes one share of grad_x per edge.  The
// scheduled backward walks the same edges of a CTA's range in an order that puts edges with the same sender and
// neighbouring receivers one after the other in the same consumer warp, so that the warp adds their shares in
// registers and writes one row per run.  The order is a property of the graph and of the kernel's tile shape;
// it is built once per neighbour list, like rowptr.
//
// Order of a range: steps k = receivers in ascending order.  Step k holds every edge into k that no earlier step
// took, plus the edges of the same senders into receivers k+1 .. k+window-1 (a run: one sender, consecutive
// processing positions in one column).  The runs of a step are dealt to the T columns (= consumer warps) longest
// first onto the least loaded column; the columns run on from step to step, so a tile (= one row across the
// columns) may hold edges of two neighbouring steps, and slots are empty (-1) only where a step has to wait for a
// grad_out slot and at the end of the range.  The grad_out rows of the receivers in use sit in n_slots
// shared-memory slots (receiver % n_slots);
// a row is loaded with the first tile at which its slot is free again (n_stages tiles after the last use of the
// previous occupant), empty tiles are inserted where that is later than the row's first use.
//
// Words of the schedule (int32): header[16] = {magic, T, n_slots, n_ranges, n_tiles, n_rows, n_edges, n_nodes,
// off_tile_ptr, off_row_ptr, off_tiles, 0...}; tile_ptr[n_ranges + 1] (first tile of every range);
// row_ptr[n_nodes + 1] (the rows of a sender's runs are contiguous, in processing order); tiles: per tile
// (T + 1) records of 4 words: T slots {edge or -1, sender, row to write after this edge or -1, grad_out slot}
// and one record {receiver to load into slot 0, 1, 2 (or -1), 0}.
#pragma once
#include <cstdint>
#include <string>
#include <vector>

namespace e3j {

constexpr int32_t kSchedMagic = 0x53434844;
constexpr int kSchedSlots = 3;     // grad_out rows resident per CTA
constexpr int kSchedWindow = 2;    // receivers a run may span
constexpr int kSchedStages = 2;    // tiles in flight (ring depth of the kernel)

// 0 on success; -1: receivers not sorted or an index out of range.
int build_bwd_schedule(int T, int n_ranges, int64_t n_nodes, int64_t n_edges, const int32_t* senders,
                       const int32_t* receivers, std::vector<int32_t>& words);

// upper bound of the schedule's size in words
size_t bwd_schedule_max_words(int T, int n_ranges, int64_t n_nodes, int64_t n_edges);

}  // namespace e3j
