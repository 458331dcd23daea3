// Internal host-side representation of a plan.  Not part of the public ABI.
#pragma once

#include <cstdint>
#include <set>
#include <vector>

#include "cleave.h"

namespace cleave {

// Work unit of the exec kernel: one pair of half-tiles.  A half-tile is <= 128 rows x <= 256 columns
// of a GEMM's output over one K-range; the two halves of a pair are run by the two CTAs of a cluster
// with one M = 256 MMA stream, so they share the GEMM, the K-range and the columns, but each has its
// own rows.  The columns of a half-tile fall into one or two segments (the second starts at column
// `split`), and every (half, segment) quadrant belongs to one task: it is stored into that task's
// packed block and counted in that task's bookkeeping.  Where all block edges of a GEMM lie on
// multiples of 128 the GEMM is tiled on a global grid of 256 x 256 pairs whatever the blocks'
// shapes, each quadrant being the 128 x 128 cell of whichever task owns it there; otherwise every
// task is cut into half-tiles of its own (one segment each) and half-tiles with equal columns share
// a pair.  160 bytes, read by the kernel's scheduler warp with ten 16-byte loads.
struct TileSeg {
    uint32_t task;      // owning task (bookkeeping)
    uint32_t ld;        // leading dimension of the task's packed block (= beta)
    uint64_t out_off;   // fp32 element offset of the quadrant's (0,0) in the arena
    uint32_t fin;       // cell of the in-kernel K-slice sum (kNoFin: none)
    uint32_t live;      // (set per launch) the quadrant runs: its task is neither dropped nor superseded
};
struct TileHalf {
    uint32_t m_row;     // first row of the half-tile in op(A)
    uint32_t rows;      // valid rows (0..128); 0 = the pair has no second half
    TileSeg seg[2];     // columns [0, split) and [split, cols); seg[1] unused when split == cols
};
struct TileDesc {
    uint32_t gemm;
    uint32_t flags;     // TILE_* below
    uint32_t n_col;     // first column in op(B)
    uint32_t n_mma;     // bits 0-15: MMA N extent (columns rounded up to 16); bits 16-31: valid columns (1..256)
    uint32_t k0, k1;
    uint32_t ldc;       // leading dimension of the GEMM's C (= N)
    uint32_t level;     // bits 0-15: DAG level of the GEMM; bits 16-23: its number of K-slices; bits 24-31: this K-slice
    TileHalf h[2];
    uint32_t split;     // first column of the second segment (a multiple of 32), or the number of columns
    uint32_t pad[3];
};
static_assert(sizeof(TileDesc) == 160, "TileDesc must be 160 bytes");
constexpr uint32_t kNoFin = 0xFFFFFFFFu;

// LIVE0 / LIVE1: (set per launch) half 0 / 1 has a quadrant that runs
// A_MN / B_MN: the operand is stored with M (resp. N) contiguous (transA = 1, resp. transB = 0)
// SINGLE: the GEMM has one K-slice, so the half-tile's block is already the final value of C there
// A_BIG / B_BIG: the operand has a tensor map with double-size boxes (one TMA operation per 128 rows or columns)
enum : uint32_t { TILE_LIVE0 = 1u, TILE_LIVE1 = 2u, TILE_END = 4u, TILE_A_MN = 8u, TILE_B_MN = 16u, TILE_SINGLE = 32u,
                  TILE_A_BIG = 64u, TILE_B_BIG = 128u };

// How an execution writes its results (kernel argument, the same for every tile of a launch):
//   DIRECT  blocks of one-slice GEMMs go to their place in C instead of the arena
//   FINISH  in a GEMM with several K-slices the last block of a cell to arrive sums the cell's blocks
//           (all of them are in the arena by then) in the fixed tree order and writes C
//   BF16    C holds bf16 (round to nearest even from the fp32 value) instead of fp32
//   CONSUME (with FINISH) a block that completes its cell when its tile is handed out is summed on arrival and not
//           stored in the arena
enum : uint32_t { MODE_DIRECT = 1u, MODE_FINISH = 2u, MODE_BF16 = 4u, MODE_CONSUME = 8u };

// Partial block of one K-slice inside a cell of the in-kernel sum.
struct FinRef {
    uint64_t off;       // arena offset of the cell's (0,0) inside the slice's block
    uint32_t ld;        // that block's leading dimension
    uint32_t task;
};

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
    std::vector<uint32_t> task_ntiles;             // per task: number of (half-tile, segment) quadrants
    // in-kernel K-slice sum: cell c (one half-tile position of a GEMM with several K-slices) owns the
    // ksplit[gemm] consecutive entries of fin_refs starting at fin_ref0[c], slice order
    std::vector<uint32_t> fin_ref0;
    std::vector<cleave::FinRef> fin_refs;
    std::vector<uint8_t> gemm_finishable;          // per GEMM: every cell has one block per K-slice with equal geometry
    uint32_t n_levels = 1;
    uint32_t tiles_original = 0;                   // tiles of the original plan = [0, tiles_original)
    int exec_unsupported = 0;                      // set when a task violates the kernel's alignment rules

    // assembly work list (original tasks only; reissued pieces write into their parents' blocks)
    std::vector<cleave::AsmItem> asm_items;
    std::vector<cleave::AsmRef> asm_refs;
    // sp: padded slice count, 0 = scalar kernel; single: one-slice GEMMs; finishable: GEMMs the exec kernel can sum itself
    struct AsmGroup { uint32_t sp, item0, n_items, single, finishable; };
    std::vector<AsmGroup> asm_groups;              // one launch each

    uint32_t mode = 0;                             // MODE_* of the last execution
    bool fused = false;                            // last execution wrote one-slice GEMMs straight to C
    bool finished = false;                         // ... and summed every cell of the finishable GEMMs itself, none missing
    bool out_bf16 = false;                         // ... into bf16 outputs
    bool consumed = false;                         // ... without storing the blocks that completed their cells
    uint64_t wait_limit_ns = 2000000000ull;        // bound of every device-side wait

    cleave::DeviceState* dev = nullptr;
};

namespace cleave {

int plan_build(cleave_plan_s& p);                                   // planner over p.gemms / p.devices
int plan_build_uniform(cleave_plan_s& p, uint32_t gm, uint32_t gn, uint32_t ks);
int plan_reissue(cleave_plan_s& p, const uint32_t* failed, uint32_t n, uint32_t* first_new);
void build_tiles(cleave_plan_s& p, uint32_t first_task);            // appends tiles of tasks [first_task, end)
int build_assembly(cleave_plan_s& p);
void device_state_free(DeviceState* d);
int static_assemble_check(const cleave_plan_s* p, float* const* C);   // argument checks shared with cleave_assemble

}  // namespace cleave
