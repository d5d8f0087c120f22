// Internal: host-side plan (coefficient tables) shared by the C-ABI translation units.
#pragma once
#include <cstdint>
#include <mutex>
#include <string>
#include <vector>

#include "../../include/e3j.h"

namespace e3j {

struct Record {
    int i0, i1, i2, i3;
    double val;
};

// 8-byte packed record (one 64-bit load): three 8-bit indices and the float32 value.
// Which three indices are stored depends on the table (see DeviceTables).
struct PackedRecord {
    uint8_t a, b, c, pad;
    float val;
};
static_assert(sizeof(PackedRecord) == 8, "packed record must be 8 bytes");

// Device-resident tables of one plan on one device (single allocation).
struct DeviceTables {
    int device = -1;
    void* base = nullptr;
    // sorted by i0: (a,b,c) = (i1,i2,path)
    const PackedRecord* by_i0 = nullptr;
    const int32_t* i0_start = nullptr;  // [D+1]
    const int32_t* i0_path = nullptr;   // [D]
    // sorted by i1: (a,b,c) = (i0,i2,path)
    const PackedRecord* by_i1 = nullptr;
    const int32_t* i1_start = nullptr;  // [d+1]
    // sorted by i2: (a,b,c) = (i0,i1,path)
    const PackedRecord* by_i2 = nullptr;
    const int32_t* i2_start = nullptr;  // [d'+1]
    const int32_t* path_out_off = nullptr;  // [P+1] first output row of every path (last entry: D)
    const int32_t* path_rows = nullptr;     // [P] rows of every path, 2L+1
    // the record values in float64, in the order of by_i0 / by_i1 / by_i2 (float64 entry points)
    const double* val64_i0 = nullptr;
    const double* val64_i1 = nullptr;
    const double* val64_i2 = nullptr;
    int32_t* status = nullptr;  // sticky device status word (0 = fine), see e3j_plan_device_status
};

}  // namespace e3j

struct e3j_plan {
    int nq = 0, d = 0, dp = 0, P = 0, D = 0, n_pairs = 0;
    unsigned flags = 0;
    std::vector<e3j_path_info_t> paths;
    std::vector<e3j::Record> rec;  // sorted by (i0,i3,i1,i2)
    std::string signature;         // canonical text of (irreps_in | sh_lmax | output blocks)
    int fast_id = -1;              // index into the specialised-kernel registry, or -1
    mutable std::mutex mu;
    mutable std::vector<e3j::DeviceTables> dev;  // one entry per device that used the plan
};

namespace e3j {
// Builds the host part of a plan; returns an E3J_* status.
int build_plan(e3j_plan& plan, const char* irreps_in, int sh_lmax, const char* irreps_out,
               int out_lmax, unsigned flags);
// Real coupling tensor of one path, [2L+1][2l1+1][2l2+1] row-major, canonical sign.
std::vector<double> real_cg_ladder(int l1, int l2, int L);
}  // namespace e3j
