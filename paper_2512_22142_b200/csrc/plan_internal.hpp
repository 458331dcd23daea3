// Internal host-side representation of a plan.  Not part of the public ABI.
#pragma once

#include <cstdint>
#include <set>
#include <vector>

#include "cleave.h"

namespace cleave {

// Work unit of the exec kernel: one (<=256 row) x (<=256 column) output tile of one task over the
// task's whole K-range.  64 bytes, read by the kernel's scheduler warp with four 16-byte loads.
struct TileDesc {
    uint32_t task;      // owning task (bookkeeping)
    uint32_t gemm;
    uint32_t flags;     // TILE_VALID | TILE_END
    uint32_t n_mma;     // MMA N extent: cols rounded up to 16
    uint32_t m_row;     // first row of the tile in op(A)
    uint32_t n_col;     // first column of the tile in op(B)
    uint32_t k0, k1;
    uint32_t rows;      // valid rows   (1..256)
    uint32_t cols;      // valid columns (1..256)
    uint32_t ld;        // leading dimension of the task's packed block (= beta)
    uint32_t ldc;       // leading dimension of the GEMM's C (= N)
    uint64_t out_off;   // fp32 element offset of the tile's (0,0) in the arena
    uint64_t c_off;     // element offset of the tile's (0,0) in C
};
static_assert(sizeof(TileDesc) == 64, "TileDesc must be 64 bytes");

// A_MN / B_MN: the operand is stored with M (resp. N) contiguous (transA = 1, resp. transB = 0)
// SINGLE: the GEMM has one K-slice, so the tile's block is already the final value of C there;
// DIRECT: (set per launch) write it to C instead of the arena
// A_BIG / B_BIG: the operand has a tensor map with double-size boxes (one TMA operation per 128 rows or columns)
enum : uint32_t { TILE_VALID = 1u, TILE_END = 2u, TILE_A_MN = 4u, TILE_B_MN = 8u, TILE_SINGLE = 16u, TILE_DIRECT = 32u,
                  TILE_A_BIG = 64u, TILE_B_BIG = 128u };

// One unit of assembly work: `nrows` full rows of a rectangle of C in which every K-slice is
// served by one task.  `ref0` indexes `nslices` consecutive AsmRef entries, slice order.
struct AsmItem {
    uint32_t gemm;
    uint32_t i0, nrows;
    uint32_t j0, ncols;
    uint32_t ref0;
    uint32_t nslices;
    uint32_t pad;
};
struct AsmRef {
    uint64_t off;       // arena offset of element (i0, j0) inside the slice's block
    uint32_t ld;        // that block's leading dimension
    uint32_t task;
};

struct DeviceState;     // device mirrors, created on first execution call

}  // namespace cleave

struct cleave_plan_s {
    std::vector<cleave_gemm_t> gemms;
    std::vector<cleave_device_t> devices;
    cleave_plan_opts_t opts;
    std::vector<cleave_task_t> tasks;
    uint32_t n_original = 0;
    uint64_t arena_elems = 0;
    std::vector<uint32_t> ksplit;
    std::vector<uint64_t> makespan, tstar;
    std::vector<std::set<uint32_t>> dead;          // per GEMM: devices lost to churn
    std::vector<uint8_t> dropped;                  // per task: skip on execution

    // exec work list: tiles of the original tasks in raster order, then each reissue's tiles
    std::vector<cleave::TileDesc> tiles;
    std::vector<uint32_t> task_ntiles;             // per task
    uint32_t tiles_original = 0;                   // tiles of the original plan = [0, tiles_original)
    int exec_unsupported = 0;                      // set when a task violates the kernel's alignment rules

    // assembly work list (original tasks only; reissued pieces write into their parents' blocks)
    std::vector<cleave::AsmItem> asm_items;
    std::vector<cleave::AsmRef> asm_refs;
    struct AsmGroup { uint32_t sp, item0, n_items, single; };   // sp: padded slice count, 0 = scalar kernel; single: one-slice GEMMs
    std::vector<AsmGroup> asm_groups;              // one launch each

    bool fused = false;                            // last execution wrote one-slice GEMMs straight to C

    cleave::DeviceState* dev = nullptr;
};

namespace cleave {

int plan_build(cleave_plan_s& p);                                   // planner over p.gemms / p.devices
int plan_build_uniform(cleave_plan_s& p, uint32_t gm, uint32_t gn, uint32_t ks);
int plan_reissue(cleave_plan_s& p, const uint32_t* failed, uint32_t n, uint32_t* first_new);
void build_tiles(cleave_plan_s& p, uint32_t first_task);            // appends tiles of tasks [first_task, end)
int build_assembly(cleave_plan_s& p);
void device_state_free(DeviceState* d);

}  // namespace cleave
