// Shared constants and launcher declarations of the CUDA kernels (internal).
#pragma once

#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "plan_internal.hpp"

namespace cleave {

// exec kernel geometry: a tile of <= 256 rows x <= 256 columns is run by a pair of CTAs
constexpr uint32_t kBlockM = 128;                    // rows of a tile owned by one CTA of the pair
constexpr uint32_t kBlockK = 64;                     // K per pipeline stage: 64 bf16 = one 128-byte swizzle row
constexpr uint32_t kSubRows = 64;                    // rows (or M/N elements) per TMA box
constexpr uint32_t kSubBytes = kSubRows * kBlockK * 2;          // 8192: one 64 x 64 bf16 box
constexpr uint32_t kPairABytes = 2 * kSubBytes;      // per CTA and stage: 128 rows of A ...
constexpr uint32_t kPairBBytes = 2 * kSubBytes;      // ... and half of the (<= 256) columns of B
constexpr uint32_t kPairStageBytes = kPairABytes + kPairBBytes;   // 32768
constexpr int kPairStages = 6;
constexpr int kMapsPerGemm = 4;                      // A, B with 64 x 64 boxes, then A, B with double-size boxes
constexpr int kAccSlots = 2;                         // accumulator slots in tensor memory (double buffer)
constexpr uint32_t kAccCols = 256;
constexpr uint32_t kTmemCols = 512;
constexpr int kSchedSlots = 4;
constexpr int kTileWords16 = sizeof(TileDesc) / 16;   // 16-byte words of a work-list entry
constexpr uint32_t kEpiStageFloats = 32 * 32;        // per epilogue warp: 32 x 32 fp32 staging tile (4 KB, 16-byte chunks XOR-swizzled by row)

constexpr int kTmaWarp = 0, kMmaWarp = 1, kSchedWarp = 2, kEpiWarp0 = 4;
constexpr int kEpiWarpsPerGroup = 4, kEpiWarps = 2 * kEpiWarpsPerGroup;   // group g drains accumulator slot g
constexpr int kExecThreads = 32 * (kEpiWarp0 + kEpiWarps);
constexpr uint32_t kPairDynSmem = kPairStages * kPairStageBytes + 1024 + kEpiWarps * kEpiStageFloats * 4;

// device status word bits
enum : unsigned int { STATUS_TIMEOUT = 1u, STATUS_BOUNDS = 2u, STATUS_INCOMPLETE = 4u };

// Arguments of the exec kernel (passed by value).
struct ExecParams {
    const TileDesc* tiles;          // work list (device)
    uint32_t tile_end;              // the ticket runs up to here
    unsigned int* ticket;
    const CUtensorMap* maps;        // kMapsPerGemm per GEMM
    const CUtensorMap* c_maps;      // per GEMM: C with 32 x 32 boxes as fp32, then as bf16 (bulk stores of blocks that go straight to C)
    float* partials;                // arena
    void* const* c_ptrs;            // per GEMM: C (fp32, or bf16 under MODE_BF16)
    uint32_t* done;                 // per task: finished half-tiles x epilogue warps
    unsigned int* status;
    const uint32_t* fin_ref0;       // per cell: first entry in fin_refs
    const FinRef* fin_refs;
    unsigned int* fin_count;        // per cell and 32-row strip: blocks arrived
    unsigned int* level_left;       // per DAG level: epilogue-warp strips still to finish
    uint32_t mode;                  // MODE_*
    unsigned long long wait_limit_ns;   // bound of every device-side wait
};

// Words of a launch's arming kernel.
struct ArmParams {
    TileDesc* tiles;
    uint32_t tile_begin, tile_end;
    const cleave_task_t* tasks;
    const uint8_t* dropped;
    uint32_t* done;
    unsigned int* ticket;
    unsigned int* status;
    unsigned int* level_left;
    uint32_t mode;
    uint32_t level_begin, level_end;   // only tiles of these DAG levels run
    unsigned long long arena_elems;
};

cudaError_t launch_arm_queue(const ArmParams& a, int clear_status, cudaStream_t st);
cudaError_t exec_pair_kernel_prepare();
cudaError_t launch_exec_pair(uint32_t clusters, const ExecParams& e, cudaStream_t st);
cudaError_t launch_check_done(const cleave_task_t* tasks, const uint32_t* done, const uint32_t* ntiles, uint32_t n_tasks,
                              unsigned int* status, cudaStream_t st);
cudaError_t launch_collect_failed(const cleave_task_t* tasks, const uint32_t* done, const uint32_t* ntiles,
                                  uint32_t n_tasks, uint32_t* out_ids, unsigned int* out_count, cudaStream_t st);
cudaError_t launch_verify(const cleave_task_t* tasks, uint32_t n_tasks, const cleave_gemm_t* gemms, const uint32_t* ksplit,
                          const void* const* ab_ptrs, const float* partials, float* const* c_ptrs, int fused, uint64_t seed,
                          float tol, float4* out, unsigned int* n_bad, uint32_t sign_bytes, cudaStream_t st);
// the sub-GEMMs of tasks [task_begin, task_end) without tensor cores (plans the exec kernel cannot take)
cudaError_t launch_exec_simple(const cleave_task_t* tasks, uint32_t task_begin, uint32_t task_end, const cleave_gemm_t* gemms,
                               const void* const* ab_ptrs, const uint8_t* dropped, const uint32_t* ntiles, float* partials,
                               uint64_t arena_elems, uint32_t* done, unsigned int* status, cudaStream_t st);
// sp = padded slice count of the vectorised kernel (1, 2, 4, 8, 16, 32), 0 = scalar kernel; out_bf16: C holds bf16
cudaError_t launch_assemble(const AsmItem* items, const AsmRef* refs, uint32_t item0, uint32_t n_items, uint32_t sp,
                            const float* partials, void* const* Cptr, const uint32_t* ldcs, int out_bf16, cudaStream_t st);

}  // namespace cleave
