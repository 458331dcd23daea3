// exec_simple_kernel: the sub-GEMM of every task, without tensor cores or TMA, for plans the
// tensor-core kernel cannot take (a K-range that does not start on a multiple of 64, operand rows
// that do not start on 16-byte boundaries, leading dimensions that are no multiples of 8).  Such
// plans only arise from hand-picked granules or ragged uniform grids; the planner's defaults never
// produce them.  Slow but complete: the same blocks, bookkeeping and failure handling as the fast
// path, so every plan cleave_plan hands out can be executed.
//
// One CTA per task.  The block is walked in 64 x 64 sub-tiles; a K-chunk of 32 of the task's rows of A
// and columns of B is staged in shared memory as fp32 (bf16 widens exactly), each thread owns a 4 x 4
// patch and accumulates in fp32 in K order.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cleave.h"
#include "kernels.cuh"

namespace cleave {

namespace {

constexpr int kSimpleTile = 64, kSimpleK = 32, kSimpleThreads = 256;

__device__ __forceinline__ float bf16_at(const uint16_t* p, uint64_t i) { return __uint_as_float((uint32_t)p[i] << 16); }

__global__ void __launch_bounds__(kSimpleThreads)
exec_simple_kernel(const cleave_task_t* __restrict__ tasks, uint32_t task_begin, const cleave_gemm_t* __restrict__ gemms,
                   const void* const* __restrict__ ab_ptrs, const uint8_t* __restrict__ dropped, const uint32_t* __restrict__ ntiles,
                   float* __restrict__ partials, unsigned long long arena_elems, uint32_t* done, unsigned int* status) {
    __shared__ float As[kSimpleTile][kSimpleK + 1];
    __shared__ float Bs[kSimpleK][kSimpleTile + 1];
    const uint32_t id = task_begin + blockIdx.x;
    const cleave_task_t t = tasks[id];
    if (dropped[id] || (t.flags & CLEAVE_TASK_SUPERSEDED)) return;      // left unfinished: the bookkeeping shows it
    const cleave_gemm_t g = gemms[t.gemm];
    const uint32_t alpha = t.m1 - t.m0, beta = t.n1 - t.n0;
    // range check of the block about to be written
    if (t.part_off + (unsigned long long)alpha * beta > arena_elems) {
        if (threadIdx.x == 0) atomicOr(status, STATUS_BOUNDS);
        return;
    }
    const uint16_t* A = static_cast<const uint16_t*>(ab_ptrs[2 * t.gemm]);
    const uint16_t* B = static_cast<const uint16_t*>(ab_ptrs[2 * t.gemm + 1]);
    float* P = partials + t.part_off;
    const uint32_t tx = threadIdx.x % 16, ty = threadIdx.x / 16;          // 16 x 16 threads, 4 x 4 outputs each
    for (uint32_t i0 = 0; i0 < alpha; i0 += kSimpleTile)
        for (uint32_t j0 = 0; j0 < beta; j0 += kSimpleTile) {
            float acc[4][4] = {};
            for (uint32_t k0 = t.k0; k0 < t.k1; k0 += kSimpleK) {
                // stage op(A)[m0 + i0 .. +63, k0 .. +31] and op(B)[k0 .. +31, n0 + j0 .. +63]; outside the task: zero
                for (uint32_t e = threadIdx.x; e < kSimpleTile * kSimpleK; e += kSimpleThreads) {
                    // consecutive threads walk the contiguous direction of the stored operand
                    const uint32_t ai = g.transA ? e % kSimpleTile : e / kSimpleK, ak = g.transA ? e / kSimpleTile : e % kSimpleK;
                    const uint32_t i = t.m0 + i0 + ai, k = k0 + ak;
                    float a = 0.f;
                    if (i < t.m1 && k < t.k1) a = g.transA ? bf16_at(A, (uint64_t)k * g.lda + i) : bf16_at(A, (uint64_t)i * g.lda + k);
                    As[ai][ak] = a;
                    const uint32_t bj = g.transB ? e / kSimpleK : e % kSimpleTile, bk = g.transB ? e % kSimpleK : e / kSimpleTile;
                    const uint32_t j = t.n0 + j0 + bj, kk = k0 + bk;
                    float b = 0.f;
                    if (j < t.n1 && kk < t.k1) b = g.transB ? bf16_at(B, (uint64_t)j * g.ldb + kk) : bf16_at(B, (uint64_t)kk * g.ldb + j);
                    Bs[bk][bj] = b;
                }
                __syncthreads();
#pragma unroll 8
                for (uint32_t k = 0; k < kSimpleK; ++k) {
                    float a[4], b[4];
#pragma unroll
                    for (int x = 0; x < 4; ++x) { a[x] = As[ty * 4 + x][k]; b[x] = Bs[k][tx * 4 + x]; }
#pragma unroll
                    for (int x = 0; x < 4; ++x)
#pragma unroll
                        for (int y = 0; y < 4; ++y) acc[x][y] = fmaf(a[x], b[y], acc[x][y]);
                }
                __syncthreads();
            }
#pragma unroll
            for (int x = 0; x < 4; ++x)
#pragma unroll
                for (int y = 0; y < 4; ++y) {
                    const uint32_t i = i0 + ty * 4 + x, j = j0 + tx * 4 + y;
                    if (i < alpha && j < beta) P[(uint64_t)i * beta + j] = acc[x][y];
                }
        }
    // the whole block is stored: count the task as finished (the fast path counts per quadrant and epilogue warp)
    __threadfence();
    __syncthreads();
    if (threadIdx.x == 0) done[id] = ntiles[id] * (uint32_t)kEpiWarpsPerGroup;
}

}  // namespace

cudaError_t launch_exec_simple(const cleave_task_t* tasks, uint32_t task_begin, uint32_t task_end, const cleave_gemm_t* gemms,
                               const void* const* ab_ptrs, const uint8_t* dropped, const uint32_t* ntiles, float* partials,
                               uint64_t arena_elems, uint32_t* done, unsigned int* status, cudaStream_t st) {
    if (task_end <= task_begin) return cudaSuccess;
    exec_simple_kernel<<<task_end - task_begin, kSimpleThreads, 0, st>>>(tasks, task_begin, gemms, ab_ptrs, dropped, ntiles, partials,
                                                                        (unsigned long long)arena_elems, done, status);
    return cudaGetLastError();
}

}  // namespace cleave
