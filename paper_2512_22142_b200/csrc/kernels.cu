// CUDA kernels of the Cleave hot path for sm_100a.
//
//   arm_queue_kernel    marks each work-list tile runnable or skipped (dropped / superseded task),
//                       clears the bookkeeping of the tasks about to run, resets the ticket
//   exec_kernel         persistent grouped GEMM: one CTA per SM walks the tile list through a
//                       device-side ticket; TMA loads of 64x64 bf16 boxes into 128-byte-swizzled
//                       shared memory, tcgen05 MMA (128 x N x 16, bf16 -> fp32) accumulating in
//                       tensor memory, epilogue warps copy the accumulators to the task's packed
//                       partial block and count each 128-row half-tile in the task's bookkeeping word
//   check_done_kernel   flags E_INCOMPLETE if a live task has unfinished tiles
//   assemble_kernel     fixed-order sum of the K-slices' partial blocks into C
//   collect_failed_kernel  lists the live tasks whose bookkeeping shows unfinished tiles
//
// Every device-side wait is bounded: when a wait expires the CTA records E_TIMEOUT in the status
// word, all its roles leave their loops, outstanding TMA copies and MMAs are drained (again with a
// bound), tensor memory is released and the kernel returns.
#include <cuda.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "cleave.h"
#include "kernels.cuh"
#include "ptx.cuh"

namespace cleave {

// -------------------------------------------------------------------------------------------------
// arm_queue_kernel
// -------------------------------------------------------------------------------------------------
__global__ void arm_queue_kernel(TileDesc* tiles, uint32_t tile_begin, uint32_t tile_end, const cleave_task_t* tasks,
                                 const uint8_t* dropped, uint32_t* done, uint32_t task_begin, uint32_t task_end,
                                 unsigned int* ticket, unsigned int* status, int clear_status) {
    const uint32_t i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i == 0) {
        *ticket = tile_begin;
        if (clear_status) *status = 0;
    }
    const uint32_t t = tile_begin + i;
    if (t < tile_end) {
        const uint32_t task = tiles[t].task;
        const bool skip = dropped[task] || (tasks[task].flags & CLEAVE_TASK_SUPERSEDED);
        const uint32_t f = tiles[t].flags & ~(uint32_t)TILE_VALID;
        tiles[t].flags = skip ? f : (f | TILE_VALID);
    }
    const uint32_t k = task_begin + i;
    if (k < task_end) done[k] = 0;
}

// -------------------------------------------------------------------------------------------------
// exec_kernel
// -------------------------------------------------------------------------------------------------
// Work unit: a tile of up to 256 rows x up to 256 columns of one task over the task's K-range.  The
// rows are two halves of 128 (one MMA each per 16-deep K step) that share the B stage in shared
// memory, so a 256-row tile moves a third fewer operand bytes per FLOP than two 128-row tiles.
// Tensor memory holds two accumulator slots of 256 columns: a tall tile uses both (half h in slot
// h), a tile of at most 128 rows uses one, alternating, so consecutive short tiles double-buffer.
// Epilogue group g (four warps) drains slot g.
struct __align__(16) ExecShared {
    uint64_t full[kStages];        // TMA bytes of a stage have landed
    uint64_t empty[kStages];       // the MMAs reading a stage have completed
    uint64_t acc_full[kAccSlots];  // an accumulator slot holds a finished half-tile
    uint64_t acc_empty[kAccSlots]; // the epilogue has copied an accumulator slot out
    uint64_t sched_full[kSchedSlots];
    uint64_t sched_empty[kSchedSlots];
    uint64_t drain;                // all MMAs completed (teardown)
    uint32_t tmem_base;
    uint32_t abort_flag;
    TileDesc slot[kSchedSlots];
};

__global__ void __launch_bounds__(kExecThreads, 1)
exec_kernel(const TileDesc* __restrict__ tiles, uint32_t tile_end, unsigned int* ticket,
            const CUtensorMap* __restrict__ maps, float* __restrict__ partials, uint32_t* done, unsigned int* status) {
    extern __shared__ uint8_t dyn_smem[];
    __shared__ ExecShared sh;

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    // operand stages, 1024-byte aligned (the swizzle pattern repeats every 1024 bytes)
    const uint32_t stage_base = (smem_u32(dyn_smem) + 1023u) & ~1023u;
    volatile uint32_t* abort_flag = &sh.abort_flag;

    if (threadIdx.x == 0) {
        for (int s = 0; s < kStages; ++s) { mbar_init(smem_u32(&sh.full[s]), 1); mbar_init(smem_u32(&sh.empty[s]), 1); }
        for (int a = 0; a < kAccSlots; ++a) { mbar_init(smem_u32(&sh.acc_full[a]), 1); mbar_init(smem_u32(&sh.acc_empty[a]), kEpiWarpsPerGroup); }
        for (int q = 0; q < kSchedSlots; ++q) { mbar_init(smem_u32(&sh.sched_full[q]), 1); mbar_init(smem_u32(&sh.sched_empty[q]), 2 + kEpiWarps); }
        mbar_init(smem_u32(&sh.drain), 1);
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == kMmaWarp) tmem_alloc(smem_u32(&sh.tmem_base), kTmemCols);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = sh.tmem_base;

    if (warp == kSchedWarp) {
        // ---- scheduler: pulls tickets, skips dropped tiles, feeds the slot ring -----------------
        if (lane == 0) {
            for (uint32_t i = 0;; ++i) {
                const uint32_t q = i % kSchedSlots, par = (i / kSchedSlots) & 1u;
                if (!mbar_wait(smem_u32(&sh.sched_empty[q]), par ^ 1u, abort_flag, status)) break;
                uint4 w0, w1, w2, w3;
                bool end = false;
                for (;;) {
                    const uint32_t t = atomicAdd(ticket, 1u);
                    if (t >= tile_end) { end = true; break; }
                    const uint4* src = reinterpret_cast<const uint4*>(tiles + t);
                    w0 = __ldg(src); w1 = __ldg(src + 1); w2 = __ldg(src + 2); w3 = __ldg(src + 3);
                    if (w0.z & TILE_VALID) break;      // TileDesc::flags
                }
                uint4* dst = reinterpret_cast<uint4*>(&sh.slot[q]);
                if (end) { w0 = make_uint4(0, 0, TILE_END, 0); w1 = w2 = w3 = make_uint4(0, 0, 0, 0); }
                dst[0] = w0; dst[1] = w1; dst[2] = w2; dst[3] = w3;
                mbar_arrive(smem_u32(&sh.sched_full[q]));
                if (end) break;
            }
        }
    } else if (warp == kTmaWarp) {
        // ---- producer: TMA loads of the A and B boxes of every K-block ------------------------------
        // The whole warp walks the loop and lane j issues box j of a stage (up to 4 boxes of A, 4 of
        // B): issued one after the other by a single thread, the boxes of a stage took longer to issue
        // than the MMAs took to consume them.
        uint32_t it = 0, issued = 0, last_gemm = 0xFFFFFFFFu;
        bool ok = true;
        for (uint32_t i = 0; ok; ++i) {
            const uint32_t q = i % kSchedSlots, par = (i / kSchedSlots) & 1u;
            if (!__all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&sh.sched_full[q]), par, abort_flag, status))) break;
            const TileDesc d = sh.slot[q];
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.sched_empty[q]));
            if (d.flags & TILE_END) break;
            const CUtensorMap* map_a = maps + 2 * d.gemm;
            const CUtensorMap* map_b = map_a + 1;
            if (d.gemm != last_gemm) { tensormap_acquire(map_a); tensormap_acquire(map_b); last_gemm = d.gemm; }
            const uint32_t nsub_a = (d.rows + kSubRows - 1) / kSubRows;      // stale rows beyond are never stored
            const uint32_t nsub_b = (d.n_mma + kSubRows - 1) / kSubRows;
            const uint32_t tx = (nsub_a + nsub_b) * kSubBytes;
            const uint32_t nkb = (d.k1 - d.k0 + kBlockK - 1) / kBlockK;
            // this lane's box of a stage: operand, tensor map, offset in the stage, fixed coordinate
            const bool is_a = lane < nsub_a, is_b = !is_a && lane < nsub_a + nsub_b;
            const uint32_t j = is_a ? lane : lane - nsub_a;
            const CUtensorMap* my_map = is_a ? map_a : map_b;
            const bool my_mn = is_a ? (d.flags & TILE_A_MN) : (d.flags & TILE_B_MN);
            const int32_t my_x = (int32_t)((is_a ? d.m_row : d.n_col) + j * kSubRows);
            const uint32_t my_off = (is_a ? 0u : kABytes) + j * kSubBytes;
            for (uint32_t kb = 0; kb < nkb; ++kb, ++it) {
                const uint32_t s = it % kStages, ph = (it / kStages) & 1u;
                if (!__all_sync(0xFFFFFFFFu, mbar_wait(smem_u32(&sh.empty[s]), ph ^ 1u, abort_flag, status))) { ok = false; break; }
                const uint32_t bar = smem_u32(&sh.full[s]);
                if (lane == 0) mbar_arrive_expect_tx(bar, tx);
                __syncwarp();
                const int32_t k = (int32_t)(d.k0 + kb * kBlockK);
                if (is_a || is_b) {
                    const uint32_t dst = stage_base + s * kStageBytes + my_off;
                    if (my_mn) tma_load_2d(dst, my_map, bar, my_x, k);
                    else       tma_load_2d(dst, my_map, bar, k, my_x);
                }
                ++issued;
            }
        }
        // Wait for every copy still in flight before the CTA may exit (bounded).  A stage armed at
        // iteration x completes phase (x / kStages) & 1 of its full barrier.
        if (lane == 0) {
            const uint32_t pending = issued < (uint32_t)kStages ? issued : (uint32_t)kStages;
            for (uint32_t x = it - pending; x < it; ++x) {
                const uint64_t t0 = global_timer_ns();
                while (!mbar_try_wait(smem_u32(&sh.full[x % kStages]), (x / kStages) & 1u))
                    if (global_timer_ns() - t0 > kWaitLimitNs) { atomicOr(status, STATUS_TIMEOUT); break; }
            }
        }
    } else if (warp == kMmaWarp) {
        // ---- MMA issuer ----------------------------------------------------------------------------
        if (lane == 0) {
            uint32_t it = 0, used0 = 0, used1 = 0, toggle = 0;     // used<s>: completed uses of accumulator slot s
            bool ok = true;
            for (uint32_t i = 0; ok; ++i) {
                const uint32_t q = i % kSchedSlots, par = (i / kSchedSlots) & 1u;
                if (!mbar_wait(smem_u32(&sh.sched_full[q]), par, abort_flag, status)) break;
                const TileDesc d = sh.slot[q];
                mbar_arrive(smem_u32(&sh.sched_empty[q]));
                if (d.flags & TILE_END) break;
                const uint32_t a_mn = (d.flags & TILE_A_MN) ? 1u : 0u, b_mn = (d.flags & TILE_B_MN) ? 1u : 0u;
                const uint32_t idesc = instr_desc_bf16(kBlockM, d.n_mma, a_mn, b_mn);
                // K-contiguous tile: rows of 128 bytes, groups of 8 rows 1024 bytes apart; a 16-element K
                // step is 32 bytes inside the swizzled row.  M/N-contiguous tile: 64-element groups along
                // M/N are kSubBytes apart (leading offset), groups of 8 K-rows 1024 bytes apart; a K step
                // of 16 is two such groups.
                const uint32_t a_lbo = a_mn ? kSubBytes : 16u, a_step = a_mn ? 2048u : 32u;
                const uint32_t b_lbo = b_mn ? kSubBytes : 16u, b_step = b_mn ? 2048u : 32u;
                const bool tall = d.rows > kBlockM;
                uint32_t slot0 = 0;
                if (!tall) { slot0 = toggle; toggle ^= 1u; }
                if (!mbar_wait(smem_u32(&sh.acc_empty[slot0]), ((slot0 ? used1 : used0) & 1u) ^ 1u, abort_flag, status)) break;
                if (tall && !mbar_wait(smem_u32(&sh.acc_empty[1]), (used1 & 1u) ^ 1u, abort_flag, status)) break;
                tc_fence_after();
                const uint32_t d0 = tmem_base + slot0 * kAccCols, d1 = tmem_base + kAccCols;
                const uint32_t nkb = (d.k1 - d.k0 + kBlockK - 1) / kBlockK;
                for (uint32_t kb = 0; kb < nkb; ++kb, ++it) {
                    const uint32_t s = it % kStages, ph = (it / kStages) & 1u;
                    if (!mbar_wait(smem_u32(&sh.full[s]), ph, abort_flag, status)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = stage_base + s * kStageBytes, sb = sa + kABytes;
#pragma unroll
                    for (uint32_t k16 = 0; k16 < kBlockK / 16; ++k16) {
                        const uint64_t b_desc = smem_desc_sw128(sb + k16 * b_step, b_lbo, 1024u);
                        umma_bf16(d0, smem_desc_sw128(sa + k16 * a_step, a_lbo, 1024u), b_desc, idesc, (kb | k16) != 0u);
                        if (tall)   // rows 128..255: the second pair of A boxes, same B
                            umma_bf16(d1, smem_desc_sw128(sa + kABytes / 2 + k16 * a_step, a_lbo, 1024u), b_desc, idesc, (kb | k16) != 0u);
                    }
                    umma_commit(smem_u32(&sh.empty[s]));       // stage reusable once these MMAs are done
                }
                if (!ok) break;
                umma_commit(smem_u32(&sh.acc_full[slot0]));    // accumulator(s) complete
                if (slot0) ++used1; else ++used0;
                if (tall) { umma_commit(smem_u32(&sh.acc_full[1])); ++used1; }
            }
            // drain: every MMA issued above has completed before tensor memory is released
            umma_commit(smem_u32(&sh.drain));
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait(smem_u32(&sh.drain), 0u))
                if (global_timer_ns() - t0 > kWaitLimitNs) { atomicOr(status, STATUS_TIMEOUT); break; }
        }
    } else if (warp >= kEpiWarp0) {
        // ---- epilogue: accumulator slot -> registers -> packed partial block --------------------------
        const uint32_t group = (warp - kEpiWarp0) / kEpiWarpsPerGroup;   // the slot this warp drains
        const uint32_t quad = warp & 3u;                     // the 32 TMEM lanes this warp may read
        float* stage_tile = reinterpret_cast<float*>(dyn_smem + (stage_base - smem_u32(dyn_smem)) + kStages * kStageBytes) +
                            (warp - kEpiWarp0) * kEpiStageFloats;
        uint32_t used = 0, toggle = 0;
        for (uint32_t i = 0;; ++i) {
            const uint32_t q = i % kSchedSlots, par = (i / kSchedSlots) & 1u;
            bool ok = mbar_wait(smem_u32(&sh.sched_full[q]), par, abort_flag, status);
            if (!__all_sync(0xFFFFFFFFu, ok)) break;
            const uint32_t flags = sh.slot[q].flags, task = sh.slot[q].task, n_mma = sh.slot[q].n_mma;
            const uint32_t tile_rows = sh.slot[q].rows, cols = sh.slot[q].cols, ld = sh.slot[q].ld;
            uint64_t out_off = sh.slot[q].out_off;
            __syncwarp();
            if (lane == 0) mbar_arrive(smem_u32(&sh.sched_empty[q]));
            if (flags & TILE_END) break;
            // which half-tile, if any, lands in this group's slot (same rule as the MMA issuer)
            uint32_t rows;
            if (tile_rows > kBlockM) {
                rows = group == 0 ? kBlockM : tile_rows - kBlockM;
                out_off += (uint64_t)group * kBlockM * ld;
            } else {
                const bool mine = toggle == group;
                toggle ^= 1u;
                if (!mine) continue;
                rows = tile_rows;
            }
            ok = mbar_wait(smem_u32(&sh.acc_full[group]), used & 1u, abort_flag, status);
            if (!__all_sync(0xFFFFFFFFu, ok)) break;
            ++used;
            tc_fence_after();
            const uint32_t taddr = tmem_base + group * kAccCols + ((quad * 32u) << 16);
            // Thread `lane` holds row quad*32+lane of a 32-column chunk.  Stored from there, a warp store
            // would touch 32 lines with 16 bytes each; the chunk is transposed through a padded 32 x 33
            // staging tile instead, so that every warp store writes 128 contiguous bytes of one row.
            float* out_blk = partials + out_off + (uint64_t)(quad * 32u) * ld;
            const uint32_t rows_here = rows > quad * 32u ? min(32u, rows - quad * 32u) : 0u;
            const bool vec_ok = ((ld & 3u) == 0u) && ((out_off & 3ull) == 0ull);
            const uint32_t nchunk = (n_mma + 31u) / 32u;
            for (uint32_t c = 0; c < nchunk; ++c) {
                uint32_t v[32];
                tmem_ld_32x32(taddr + c * 32u, v);
                tmem_ld_wait();
                if (c + 1 == nchunk) {                       // slot fully read: hand it back
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(smem_u32(&sh.acc_empty[group]));
                }
#pragma unroll
                for (int x = 0; x < 32; ++x) stage_tile[lane * 33 + x] = __uint_as_float(v[x]);
                __syncwarp();
                const uint32_t c0 = c * 32u;
                if (vec_ok && c0 + 32u <= cols) {
                    // lane l: columns 4*(l%8) .. +3 of rows l/8, l/8+4, ...: one instruction writes 4 full rows
                    const uint32_t rr = lane >> 3, cc = (lane & 7u) * 4u;
                    float* dst = out_blk + c0 + cc;
#pragma unroll
                    for (uint32_t r = rr; r < 32u; r += 4u) {
                        if (r < rows_here) {
                            const float* src = stage_tile + r * 33 + cc;
                            *reinterpret_cast<float4*>(dst + (uint64_t)r * ld) = make_float4(src[0], src[1], src[2], src[3]);
                        }
                    }
                } else if (c0 + lane < cols) {
                    float* dst = out_blk + c0 + lane;
#pragma unroll 8
                    for (uint32_t r = 0; r < rows_here; ++r) dst[(uint64_t)r * ld] = stage_tile[r * 33 + lane];
                }
                __syncwarp();
            }
            __threadfence();
            __syncwarp();
            if (lane == 0) atomicAdd(&done[task], 1u);       // bookkeeping: one count per warp and half-tile
        }
    }

    tc_fence_before();
    __syncthreads();
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc(tmem_base, kTmemCols);
    }
}

// -------------------------------------------------------------------------------------------------
// bookkeeping kernels
// -------------------------------------------------------------------------------------------------
__global__ void clear_status_bits_kernel(unsigned int* status, unsigned int mask) { *status &= ~mask; }

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
// SP = slice count padded to a power of two.  The 32 lanes of a warp form G = min(SP, 8) groups;
// group g owns the R = SP / G adjacent slices g*R .. g*R+R-1 and lane l of a group owns one float4
// of the row.  Each lane sums its R slices as a balanced tree in registers, then a butterfly of
// shfl_xor over the group index finishes the balanced tree over all SP slices: the order is fixed,
// so the sum is deterministic.  Missing slices (s >= nslices) contribute +0.0f.
template <int SP>
__global__ void __launch_bounds__(256)
assemble_vec_kernel(const AsmItem* __restrict__ items, const AsmRef* __restrict__ refs, uint32_t item0,
                    const float* __restrict__ partials, float* const* __restrict__ Cptr, const uint32_t* __restrict__ ldcs) {
    constexpr int G = SP < 8 ? SP : 8;
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
    float* crow = Cptr[it.gemm] + (uint64_t)it.i0 * ldc + it.j0;

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
                if (base + u * LG + l < units)
                    __stcs(reinterpret_cast<float4*>(crow + (uint64_t)urow[u] * ldc + ucol[u]), acc[u]);
        }
    }
}

// Any alignment, any slice count up to 32: one thread per output element, the same balanced tree.
__global__ void assemble_scalar_kernel(const AsmItem* __restrict__ items, const AsmRef* __restrict__ refs, uint32_t item0,
                                       const float* __restrict__ partials, float* const* __restrict__ Cptr,
                                       const uint32_t* __restrict__ ldcs) {
    const AsmItem it = items[item0 + blockIdx.x];
    const uint32_t ldc = ldcs[it.gemm];
    float* C = Cptr[it.gemm];
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
        C[(uint64_t)(it.i0 + r) * ldc + it.j0 + c] = v[0];
    }
}

// -------------------------------------------------------------------------------------------------
// host-side launchers
// -------------------------------------------------------------------------------------------------
cudaError_t launch_arm_queue(TileDesc* tiles, uint32_t tile_begin, uint32_t tile_end, const cleave_task_t* tasks,
                             const uint8_t* dropped, uint32_t* done, uint32_t task_begin, uint32_t task_end,
                             unsigned int* ticket, unsigned int* status, int clear_status, cudaStream_t st) {
    uint32_t n = tile_end - tile_begin;
    if (task_end - task_begin > n) n = task_end - task_begin;
    if (n == 0) n = 1;
    arm_queue_kernel<<<(n + 255) / 256, 256, 0, st>>>(tiles, tile_begin, tile_end, tasks, dropped, done, task_begin,
                                                       task_end, ticket, status, clear_status);
    return cudaGetLastError();
}

cudaError_t exec_kernel_prepare() {
    return cudaFuncSetAttribute(exec_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kExecDynSmem);
}

cudaError_t launch_exec(uint32_t grid, const TileDesc* tiles, uint32_t tile_end, unsigned int* ticket,
                        const CUtensorMap* maps, float* partials, uint32_t* done, unsigned int* status,
                        cudaStream_t st) {
    exec_kernel<<<grid, kExecThreads, kExecDynSmem, st>>>(tiles, tile_end, ticket, maps, partials, done, status);
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

cudaError_t launch_assemble(const AsmItem* items, const AsmRef* refs, uint32_t item0, uint32_t n_items, uint32_t sp,
                            const float* partials, float* const* Cptr, const uint32_t* ldcs, cudaStream_t st) {
    if (!n_items) return cudaSuccess;
    switch (sp) {
        case 0:  assemble_scalar_kernel<<<n_items, 256, 0, st>>>(items, refs, item0, partials, Cptr, ldcs); break;
        case 1:  assemble_vec_kernel<1><<<n_items, 256, 0, st>>>(items, refs, item0, partials, Cptr, ldcs); break;
        case 2:  assemble_vec_kernel<2><<<n_items, 256, 0, st>>>(items, refs, item0, partials, Cptr, ldcs); break;
        case 4:  assemble_vec_kernel<4><<<n_items, 256, 0, st>>>(items, refs, item0, partials, Cptr, ldcs); break;
        case 8:  assemble_vec_kernel<8><<<n_items, 256, 0, st>>>(items, refs, item0, partials, Cptr, ldcs); break;
        case 16: assemble_vec_kernel<16><<<n_items, 256, 0, st>>>(items, refs, item0, partials, Cptr, ldcs); break;
        case 32: assemble_vec_kernel<32><<<n_items, 256, 0, st>>>(items, refs, item0, partials, Cptr, ldcs); break;
        default: return cudaErrorInvalidValue;
    }
    return cudaGetLastError();
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
        if (cleave::launch_assemble(reinterpret_cast<const cleave::AsmItem*>(base), reinterpret_cast<const cleave::AsmRef*>(base + off_refs),
                                    grp.item0, grp.n_items, grp.sp, partials, reinterpret_cast<float* const*>(base + off_ptrs),
                                    reinterpret_cast<const uint32_t*>(base + off_ld), st) != cudaSuccess) {
            cudaGetLastError();
            return CLEAVE_E_CUDA;
        }
    }
    return 0;
}

