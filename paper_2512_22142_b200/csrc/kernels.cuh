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
constexpr uint32_t kEpiStageFloats = 32 * 33;        // per epilogue warp: padded 32 x 32 transpose tile

constexpr int kTmaWarp = 0, kMmaWarp = 1, kSchedWarp = 2, kEpiWarp0 = 4;
constexpr int kEpiWarpsPerGroup = 4, kEpiWarps = 2 * kEpiWarpsPerGroup;   // group g drains accumulator slot g
constexpr int kExecThreads = 32 * (kEpiWarp0 + kEpiWarps);
constexpr uint32_t kPairDynSmem = kPairStages * kPairStageBytes + 1024 + kEpiWarps * kEpiStageFloats * 4;

constexpr uint64_t kWaitLimitNs = 2000000000ull;     // bound of every device-side wait

// device status word bits
enum : unsigned int { STATUS_TIMEOUT = 1u, STATUS_BOUNDS = 2u, STATUS_INCOMPLETE = 4u };

cudaError_t launch_arm_queue(TileDesc* tiles, uint32_t tile_begin, uint32_t tile_end, const cleave_task_t* tasks,
                             const uint8_t* dropped, uint32_t* done, uint32_t task_begin, uint32_t task_end,
                             unsigned int* ticket, unsigned int* status, int clear_status, int direct, uint64_t arena_elems,
                             cudaStream_t st);
cudaError_t exec_pair_kernel_prepare();
cudaError_t launch_exec_pair(uint32_t clusters, const TileDesc* tiles, uint32_t tile_end, unsigned int* ticket,
                             const CUtensorMap* maps, float* partials, float* const* c_ptrs, uint32_t* done,
                             unsigned int* status, cudaStream_t st);
cudaError_t launch_check_done(const cleave_task_t* tasks, const uint32_t* done, const uint32_t* ntiles, uint32_t n_tasks,
                              unsigned int* status, cudaStream_t st);
cudaError_t launch_collect_failed(const cleave_task_t* tasks, const uint32_t* done, const uint32_t* ntiles,
                                  uint32_t n_tasks, uint32_t* out_ids, unsigned int* out_count, cudaStream_t st);
cudaError_t launch_verify(const cleave_task_t* tasks, uint32_t n_tasks, const cleave_gemm_t* gemms, const uint32_t* ksplit,
                          const void* const* ab_ptrs, const float* partials, float* const* c_ptrs, int fused, uint64_t seed,
                          float tol, float4* out, unsigned int* n_bad, uint32_t sign_bytes, cudaStream_t st);
// sp = padded slice count of the vectorised kernel (1, 2, 4, 8, 16, 32), 0 = scalar kernel
cudaError_t launch_assemble(const AsmItem* items, const AsmRef* refs, uint32_t item0, uint32_t n_items, uint32_t sp,
                            const float* partials, float* const* Cptr, const uint32_t* ldcs, cudaStream_t st);

}  // namespace cleave
