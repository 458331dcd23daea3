// CUDA kernels of the Cleave hot path for sm_100a.
//
//   arm_queue_kernel    marks each quadrant of every work-list entry runnable or skipped (dropped /
//                       superseded task), clears the bookkeeping of the tasks about to run, counts
//                       the strips each DAG level has to finish, resets the ticket
//   (the grouped GEMM itself, exec_pair_kernel, lives in kernels_pair.cu)
//   check_done_kernel   flags E_INCOMPLETE if a live task has unfinished tiles
//   assemble_kernel     fixed-order sum of the K-slices' partial blocks into C
//   collect_failed_kernel  lists the live tasks whose bookkeeping shows unfinished tiles
//
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cleave.h"
#include "kernels.cuh"
#include "ptx.cuh"

namespace cleave {

__global__ void clear_status_bits_kernel(unsigned int* status, unsigned int mask) { *status &= ~mask; }

// -------------------------------------------------------------------------------------------------
// arm_queue_kernel
// -------------------------------------------------------------------------------------------------
__global__ void arm_queue_kernel(const ArmParams a) {
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) *a.ticket = a.tile_begin;
    const uint32_t t = a.tile_begin + i;
    if (t >= a.tile_end) return;
    TileDesc& d = a.tiles[t];
    uint32_t f = d.flags & ~(uint32_t)(TILE_LIVE0 | TILE_LIVE1);
    const bool direct = (a.mode & MODE_DIRECT) && (f & TILE_SINGLE);
    const uint32_t cols = d.n_mma >> 16, split = d.split;
    const uint32_t level = d.level & 0xFFFFu;
    const bool in_range = level >= a.level_begin && level < a.level_end;
    uint32_t live = 0;
    for (uint32_t r = 0; r < 2; ++r) {
        TileHalf& h = d.h[r];
        for (uint32_t q = 0; q < 2; ++q) {
            TileSeg& sg = h.seg[q];
            sg.live = 0;
            const uint32_t width = q == 0 ? min(split, cols) : (cols > split ? cols - split : 0u);
            if (h.rows == 0 || width == 0 || !in_range) continue;
            a.done[sg.task] = 0;                         // every quadrant of the task writes the same value
            if (a.dropped[sg.task] || (a.tasks[sg.task].flags & CLEAVE_TASK_SUPERSEDED)) continue;
            // range check of what the quadrant will write: one that would leave the arena is not run
            if (!direct && sg.out_off + (unsigned long long)(h.rows - 1) * sg.ld + width > a.arena_elems) {
                atomicOr(a.status, STATUS_BOUNDS);
                continue;
            }
            sg.live = 1;
            f |= TILE_LIVE0 << r;
            ++live;
        }
    }
    d.flags = f;
    if (live) atomicAdd(&a.level_left[level], live * (uint32_t)kEpiWarpsPerGroup);
}

// -------------------------------------------------------------------------------------------------
// bookkeeping kernels
// -------------------------------------------------------------------------------------------------

__global__ void check_done_kernel(const cleave_task_t* tasks, const uint32_t* done, const uint32_t* ntiles,
                                  uint32_t n_tasks, unsigned int* status) {
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_tasks) return;
    if (tasks[i].flags & CLEAVE_TASK_SUPERSEDED) return;
    if (done[i] != ntiles[i] * kEpiWarpsPerGroup) atomicOr(status, STATUS_INCOMPLETE);
}

__global__ void collect_failed_kernel(const cleave_task_t* tasks, const uint32_t* done, const uint32_t* ntiles,
                                      uint32_t n_tasks, uint32_t* out_ids, unsigned int* out_count) {
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_tasks) return;
    if (tasks[i].flags & CLEAVE_TASK_SUPERSEDED) return;
    if (done[i] != ntiles[i] * kEpiWarpsPerGroup) out_ids[atomicAdd(out_count, 1u)] = i;
}

// -------------------------------------------------------------------------------------------------
// assemble_kernel
// -------------------------------------------------------------------------------------------------
// One CTA per item (whole rows of a rectangle of C whose K-slices each come from one block).
// SP = slice count padded to a power of two.  Up to four slices a lane loads all of them for its
// float4 and sums them as a balanced tree in registers (measured 14 % faster than spreading so few
// slices over lanes).  From eight slices on the 32 lanes of a warp form G = 8 groups; group g owns
// the R = SP / 8 adjacent slices g*R .. g*R+R-1 and lane l of a group owns one float4 of the row:
// each lane sums its R slices as a balanced tree in registers, then a butterfly of shfl_xor over the
// group index finishes the balanced tree over all SP slices.  Either way the order is the fixed
// balanced pairwise tree over adjacent slices, so the sum is deterministic; missing slices
// (s >= nslices) contribute +0.0f.  BF16: C holds bf16, each sum is rounded to nearest even.
__device__ __forceinline__ uint32_t pack2_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}
template <int SP, bool BF16>
__global__ void __launch_bounds__(256)
assemble_vec_kernel(const AsmItem* __restrict__ items, const AsmRef* __restrict__ refs, uint32_t item0,
                    const float* __restrict__ partials, void* const* __restrict__ Cptr, const uint32_t* __restrict__ ldcs) {
    constexpr int G = SP <= 4 ? 1 : 8;
    constexpr int R = SP / G;
    constexpr int LG = 32 / G;
    constexpr int U = 4;
    const AsmItem it = items[item0 + blockIdx.x];
    const uint32_t ldc = ldcs[it.gemm];
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5, nwarps = blockDim.x >> 5;
    const uint32_t g = lane / LG, l = lane % LG;
    const uint32_t c4 = it.ncols >> 2;
    const uint32_t units = it.nrows * c4;

    const float* src[R];
    uint32_t ld[R];
#pragma unroll
    for (int r = 0; r < R; ++r) {
        const uint32_t s = g * R + r;
        if (s < it.nslices) { const AsmRef rf = refs[it.ref0 + s]; src[r] = partials + rf.off; ld[r] = rf.ld; }
        else { src[r] = nullptr; ld[r] = 0; }
    }
    const uint64_t c_at = (uint64_t)it.i0 * ldc + it.j0;
    float* crow = static_cast<float*>(Cptr[it.gemm]) + c_at;
    __nv_bfloat16* crow16 = static_cast<__nv_bfloat16*>(Cptr[it.gemm]) + c_at;

    for (uint32_t base = warp * (LG * U); base < units; base += nwarps * (LG * U)) {
        float4 acc[U];
        uint32_t urow[U], ucol[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t unit = base + u * LG + l;
            const bool live = unit < units;
            urow[u] = live ? unit / c4 : 0u;
            ucol[u] = live ? (unit - urow[u] * c4) * 4u : 0u;
            float4 v[R];
#pragma unroll
            for (int r = 0; r < R; ++r) {
                v[r] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (live && src[r]) v[r] = __ldcs(reinterpret_cast<const float4*>(src[r] + (uint64_t)urow[u] * ld[r] + ucol[u]));
            }
#pragma unroll
            for (int w = 1; w < R; w *= 2)
#pragma unroll
                for (int r = 0; r < R; r += 2 * w) {
                    v[r].x += v[r + w].x; v[r].y += v[r + w].y; v[r].z += v[r + w].z; v[r].w += v[r + w].w;
                }
            acc[u] = v[0];
        }
#pragma unroll
        for (int off = LG; off < 32; off *= 2)
#pragma unroll
            for (int u = 0; u < U; ++u) {
                acc[u].x += __shfl_xor_sync(0xFFFFFFFFu, acc[u].x, off);
                acc[u].y += __shfl_xor_sync(0xFFFFFFFFu, acc[u].y, off);
                acc[u].z += __shfl_xor_sync(0xFFFFFFFFu, acc[u].z, off);
                acc[u].w += __shfl_xor_sync(0xFFFFFFFFu, acc[u].w, off);
            }
        if (g == 0) {
#pragma unroll
            for (int u = 0; u < U; ++u)
                if (base + u * LG + l < units) {
                    if (BF16) __stcs(reinterpret_cast<uint2*>(crow16 + (uint64_t)urow[u] * ldc + ucol[u]),
                                     make_uint2(pack2_bf16(acc[u].x, acc[u].y), pack2_bf16(acc[u].z, acc[u].w)));
                    else      __stcs(reinterpret_cast<float4*>(crow + (uint64_t)urow[u] * ldc + ucol[u]), acc[u]);
                }
        }
    }
}

// Any alignment, any slice count up to 32: one thread per output element, the same balanced tree.
__global__ void assemble_scalar_kernel(const AsmItem* __restrict__ items, const AsmRef* __restrict__ refs, uint32_t item0,
                                       const float* __restrict__ partials, void* const* __restrict__ Cptr,
                                       const uint32_t* __restrict__ ldcs, int out_bf16) {
    const AsmItem it = items[item0 + blockIdx.x];
    const uint32_t ldc = ldcs[it.gemm];
    float* C = static_cast<float*>(Cptr[it.gemm]);
    __nv_bfloat16* C16 = static_cast<__nv_bfloat16*>(Cptr[it.gemm]);
    uint32_t sp = 1;
    while (sp < it.nslices) sp *= 2;
    const uint32_t n = it.nrows * it.ncols;
    for (uint32_t e = threadIdx.x; e < n; e += blockDim.x) {
        const uint32_t r = e / it.ncols, c = e - r * it.ncols;
        float v[32];
        for (uint32_t s = 0; s < sp; ++s) {
            v[s] = 0.f;
            if (s < it.nslices) { const AsmRef rf = refs[it.ref0 + s]; v[s] = partials[rf.off + (uint64_t)r * rf.ld + c]; }
        }
        for (uint32_t w = 1; w < sp; w *= 2)
            for (uint32_t s = 0; s < sp; s += 2 * w) v[s] += v[s + w];
        if (out_bf16) C16[(uint64_t)(it.i0 + r) * ldc + it.j0 + c] = __float2bfloat16_rn(v[0]);
        else          C[(uint64_t)(it.i0 + r) * ldc + it.j0 + c] = v[0];
    }
}

// -------------------------------------------------------------------------------------------------
// host-side launchers
// -------------------------------------------------------------------------------------------------
cudaError_t launch_arm_queue(const ArmParams& a, int clear_status, cudaStream_t st) {
    uint32_t n = a.tile_end - a.tile_begin;
    if (n == 0) n = 1;
    // a fresh execution forgets the verdicts of the previous one (before the arming threads may raise new ones)
    if (clear_status) clear_status_bits_kernel<<<1, 1, 0, st>>>(a.status, 0xFFFFFFFFu);
    arm_queue_kernel<<<(n + 255) / 256, 256, 0, st>>>(a);
    return cudaGetLastError();
}

cudaError_t launch_check_done(const cleave_task_t* tasks, const uint32_t* done, const uint32_t* ntiles, uint32_t n_tasks,
                              unsigned int* status, cudaStream_t st) {
    // the verdict belongs to this assembly: forget the one of an earlier call
    clear_status_bits_kernel<<<1, 1, 0, st>>>(status, STATUS_INCOMPLETE);
    if (!n_tasks) return cudaGetLastError();
    check_done_kernel<<<(n_tasks + 255) / 256, 256, 0, st>>>(tasks, done, ntiles, n_tasks, status);
    return cudaGetLastError();
}

cudaError_t launch_collect_failed(const cleave_task_t* tasks, const uint32_t* done, const uint32_t* ntiles,
                                  uint32_t n_tasks, uint32_t* out_ids, unsigned int* out_count, cudaStream_t st) {
    if (!n_tasks) return cudaSuccess;
    collect_failed_kernel<<<(n_tasks + 255) / 256, 256, 0, st>>>(tasks, done, ntiles, n_tasks, out_ids, out_count);
    return cudaGetLastError();
}

template <bool BF16>
static cudaError_t launch_assemble_vec(const AsmItem* items, const AsmRef* refs, uint32_t item0, uint32_t n_items, uint32_t sp,
                                       const float* partials, void* const* Cptr, const uint32_t* ldcs, cudaStream_t st) {
    switch (sp) {
        case 1:  assemble_vec_kernel<1, BF16><<<n_items, 256, 0, st>>>(items, refs, item0, partials, Cptr, ldcs); break;
        case 2:  assemble_vec_kernel<2, BF16><<<n_items, 256, 0, st>>>(items, refs, item0, partials, Cptr, ldcs); break;
        case 4:  assemble_vec_kernel<4, BF16><<<n_items, 256, 0, st>>>(items, refs, item0, partials, Cptr, ldcs); break;
        case 8:  assemble_vec_kernel<8, BF16><<<n_items, 256, 0, st>>>(items, refs, item0, partials, Cptr, ldcs); break;
        case 16: assemble_vec_kernel<16, BF16><<<n_items, 256, 0, st>>>(items, refs, item0, partials, Cptr, ldcs); break;
        case 32: assemble_vec_kernel<32, BF16><<<n_items, 256, 0, st>>>(items, refs, item0, partials, Cptr, ldcs); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
}

cudaError_t launch_assemble(const AsmItem* items, const AsmRef* refs, uint32_t item0, uint32_t n_items, uint32_t sp,
                            const float* partials, void* const* Cptr, const uint32_t* ldcs, int out_bf16, cudaStream_t st) {
    if (!n_items) return cudaSuccess;
    if (sp == 0) {
        assemble_scalar_kernel<<<n_items, 256, 0, st>>>(items, refs, item0, partials, Cptr, ldcs, out_bf16);
        return cudaGetLastError();
    }
    return out_bf16 ? launch_assemble_vec<true>(items, refs, item0, n_items, sp, partials, Cptr, ldcs, st)
                    : launch_assemble_vec<false>(items, refs, item0, n_items, sp, partials, Cptr, ldcs, st);
}

}  // namespace cleave

// -------------------------------------------------------------------------------------------------
// cleave_assemble_static: assembly without any allocation
// -------------------------------------------------------------------------------------------------
// The assembly kernels read three small tables from device memory (work items, block references,
// output pointers and leading dimensions).  cleave_assemble keeps them in buffers it allocates on
// the plan's first use.  This entry point is for callers that must not allocate: it keeps the
// tables in one fixed array that is part of the loaded library image, so no cudaMalloc / cudaFree
// happens here, ever.  Every device that loads the library holds CLEAVE_STATIC_SCRATCH_BYTES for it
// until the process exits.
static __device__ __align__(256) unsigned char g_static_scratch[CLEAVE_STATIC_SCRATCH_BYTES];

namespace {
// In host code `g_static_scratch` is only a handle for the runtime, not a device address: the
// address on the current device has to be asked for, once per device.
unsigned char* static_scratch_on_current_device(int* rc) {
    static unsigned char* cached[64] = {nullptr};
    int dev = -1;
    *rc = CLEAVE_E_CUDA;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) { cudaGetLastError(); return nullptr; }
    if (!cached[dev]) {
        void* ptr = nullptr;
        if (cudaGetSymbolAddress(&ptr, g_static_scratch) != cudaSuccess || !ptr) { cudaGetLastError(); return nullptr; }
        cached[dev] = static_cast<unsigned char*>(ptr);
    }
    *rc = 0;
    return cached[dev];
}
inline size_t round256(size_t x) { return (x + 255) / 256 * 256; }
}  // namespace

extern "C" int cleave_assemble_static(cleave_plan_t* p, const float* partials, float* const* C, void* stream) {
    if (!p || !partials || !C) return CLEAVE_E_INVAL;
    for (uint32_t s : p->ksplit) if (s > 32) return CLEAVE_E_UNSUPPORTED;
    const size_t n = p->gemms.size();
    for (size_t i = 0; i < n; ++i) if (!C[i] || ((uintptr_t)C[i] & 15)) return CLEAVE_E_INVAL;
    const int chk = cleave::static_assemble_check(p, C);
    if (chk) return chk;
    // layout of the fixed array: items | refs | output pointers | leading dimensions
    const size_t items_b = p->asm_items.size() * sizeof(cleave::AsmItem), refs_b = p->asm_refs.size() * sizeof(cleave::AsmRef);
    const size_t off_refs = round256(items_b), off_ptrs = off_refs + round256(refs_b), off_ld = off_ptrs + round256(n * sizeof(float*));
    if (off_ld + n * sizeof(uint32_t) > (size_t)CLEAVE_STATIC_SCRATCH_BYTES) return CLEAVE_E_TOOBIG;
    int rc = 0;
    unsigned char* base = static_scratch_on_current_device(&rc);
    if (!base) return rc;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    uint32_t ldc[1024];
    if (n > 1024) return CLEAVE_E_TOOBIG;
    for (size_t i = 0; i < n; ++i) ldc[i] = p->gemms[i].N;
    // Everything the kernels read is rewritten by these copies, so nothing left by an earlier call is used.
    if (cudaMemcpyAsync(base, p->asm_items.data(), items_b, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(base + off_refs, p->asm_refs.data(), refs_b, cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(base + off_ptrs, C, n * sizeof(float*), cudaMemcpyHostToDevice, st) != cudaSuccess ||
        cudaMemcpyAsync(base + off_ld, ldc, n * sizeof(uint32_t), cudaMemcpyHostToDevice, st) != cudaSuccess) {
        cudaGetLastError();
        return CLEAVE_E_CUDA;
    }
    for (const auto& grp : p->asm_groups) {
        if ((p->fused && grp.single) || (p->finished && grp.finishable)) continue;   // already in C, written by the exec kernel
        if (cleave::launch_assemble(reinterpret_cast<const cleave::AsmItem*>(base), reinterpret_cast<const cleave::AsmRef*>(base + off_refs),
                                    grp.item0, grp.n_items, grp.sp, partials, reinterpret_cast<void* const*>(base + off_ptrs),
                                    reinterpret_cast<const uint32_t*>(base + off_ld), p->out_bf16 ? 1 : 0, st) != cudaSuccess) {
            cudaGetLastError();
            return CLEAVE_E_CUDA;
        }
    }
    return 0;
}

