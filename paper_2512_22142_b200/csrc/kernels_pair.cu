// exec_pair_kernel: the grouped sub-GEMM kernel on pairs of CTAs (thread-block clusters of two,
// tcgen05 cta_group::2).
//
// The unit of work is a pair of half-tiles (up to 128 rows x up to 256 columns each, same GEMM, K-range
// and columns) shared by the two CTAs of a cluster: CTA r loads the rows of half r of A and columns
// r*N/2..(r+1)*N/2-1 of B into its own shared memory, one thread of the leader CTA (rank 0) issues
// M = 256 MMAs that read both CTAs' shared memory, and each CTA receives the 128 accumulator rows of
// its half in its own tensor memory and writes them out.  The halves may lie anywhere in the GEMM and
// belong to different tasks.  Compared with one CTA doing both row halves this halves, per SM, the B
// bytes held, loaded and read by the tensor core and the accumulator columns, so six 32 KB stages
// fit and two accumulator slots double-buffer: the write-out of a tile overlaps the MMAs of the next.
//
// Synchronisation between the two CTAs uses only mbarriers:
//   full[s]      leader's barrier; the leader's producer arms it with the bytes of BOTH CTAs, and
//                the peer's TMA loads complete their bytes on it (cta_group::2 loads)
//   empty[s]     in both CTAs; the leader's MMA thread commits to both at once (one tcgen05.commit
//                with a two-CTA mask)
//   acc_full[a]  in both CTAs, same two-CTA commit;   acc_empty[a]  leader's, both CTAs' epilogue warps
//   sched ring   the leader's scheduler warp pops the ticket, writes the tile descriptor into both
//                CTAs' slot rings and arrives on both CTAs' sched_full; every consumer of either
//                CTA arrives on the leader's sched_empty
// Every TMA load is an ordinary load into the issuing CTA's own shared memory (no load is shared
// between CTAs).
//
// Write-out (epilogue warps, each owning a strip of 32 accumulator rows).  The strip always goes to
// the task's packed block in the arena, or, for a GEMM with one K-slice under MODE_DIRECT, to its
// place in C.  Under MODE_FINISH a strip of a GEMM with several K-slices counts its arrival at its
// cell after its block is stored, and the strip that is last sums the cell's blocks of all K-slices in
// the fixed balanced-tree order -- the order does not depend on which block was last -- and writes C.
// Usually a strip already finds every other slice's block stored when its tile is handed out (a GEMM is
// walked K-range by K-range): it then asks for those blocks to be brought into L2 while its own MMAs
// still run, and adds them to its accumulator values on their way out (no second pass over its own
// block; under MODE_CONSUME it does not even store that block: it is used up on arrival).  A strip that
// only turns out to be last after storing its block reads all blocks back.
// Under MODE_BF16 values written to C are rounded to bf16.
// A whole 32 x 32 chunk that goes straight to an fp32 C leaves as one bulk tensor store from the warp's
// staging tile (the warp issues it and moves on); everything else is written with float4 row stores.
// The bookkeeping counts of a strip (its tasks' done words, its level's counter) must follow a fence
// that waits for the strip's stores; a warp owes them and pays several strips with one fence when it
// would wait anyway.
//
// DAG levels: tiles are ordered by level, and before the scheduler hands out the first tile of a
// level it waits until every strip of the lower levels has been written (a counter per level that
// the epilogue warps count down after their stores), so a GEMM may read what a GEMM of a lower
// level wrote in the same launch.
//
// Every device-side wait is bounded: when a wait expires the CTA records E_TIMEOUT in the status
// word and raises the abort flag of both CTAs, all roles leave their loops, the MMAs in flight are
// drained (again with a bound), both CTAs meet at the cluster barrier, tensor memory is released
// and the kernel returns.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kernels.cuh"
#include "ptx.cuh"

namespace cleave {

// ---- cluster-scope PTX wrappers ---------------------------------------------------------------------
__device__ __forceinline__ uint32_t cluster_ctarank() {
    uint32_t r;
    asm volatile("mov.u32 %0, %%cluster_ctarank;" : "=r"(r));
    return r;
}
// shared::cluster address of the same shared-memory offset in CTA `rank` of this cluster
__device__ __forceinline__ uint32_t mapa_shared(uint32_t addr, uint32_t rank) {
    uint32_t r;
    asm volatile("mapa.shared::cluster.u32 %0, %1, %2;" : "=r"(r) : "r"(addr), "r"(rank));
    return r;
}
__device__ __forceinline__ void cluster_arrive_wait() {
    asm volatile("barrier.cluster.arrive.release;" ::: "memory");
    asm volatile("barrier.cluster.wait.acquire;" ::: "memory");
}
// arrive on a barrier given by its shared::cluster address (own CTA or peer)
__device__ __forceinline__ void mbar_arrive_cluster(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cluster.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
// The same for arrivals that only say "I have read it" (a ring slot, an accumulator slot): nothing this
// thread wrote has to be seen by the waiting side, so the arrival must not wait for the thread's global
// stores in flight, which a cluster-scope release does (about a thousand cycles behind a burst of stores).
__device__ __forceinline__ void mbar_arrive_cluster_read_done(uint32_t cluster_addr) {
    asm volatile("mbarrier.arrive.release.cta.shared::cluster.b64 _, [%0];" ::"r"(cluster_addr) : "memory");
}
__device__ __forceinline__ uint32_t mbar_try_wait_cl(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
// What every wait of this kernel needs to know to give up.
struct WaitCtx {
    volatile uint32_t* abort_flag;
    unsigned int* status;
    uint64_t limit_ns;
};
// Both CTAs of the pair give up: every role leaves at its next check.
__device__ __forceinline__ void raise_abort(const WaitCtx& w) {
    const uint32_t flag = smem_u32(const_cast<uint32_t*>(w.abort_flag));
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(mapa_shared(flag, 0u)), "r"(1u) : "memory");
    asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(mapa_shared(flag, 1u)), "r"(1u) : "memory");
    atomicOr(w.status, STATUS_TIMEOUT);
}
static __device__ __noinline__ bool mbar_wait_cl_slow(uint32_t bar, uint32_t parity, const WaitCtx& w) {
    const uint64_t t0 = global_timer_ns();
    uint32_t spins = 0;
    while (!mbar_try_wait_cl(bar, parity)) {
        if ((spins++ & 255u) == 0) {                     // at the first unsuccessful poll, then every 256
            if (*w.abort_flag) return false;
            if (global_timer_ns() - t0 >= w.limit_ns) { raise_abort(w); return false; }
        }
    }
    return true;
}
__device__ __forceinline__ bool mbar_wait_cl(uint32_t bar, uint32_t parity, const WaitCtx& w) {
    if (mbar_try_wait_cl(bar, parity)) return true;
    return mbar_wait_cl_slow(bar, parity, w);
}
// Bounded wait for a counter in global memory to reach zero (written by other clusters' epilogue warps).
static __device__ __noinline__ bool wait_zero(const unsigned int* ctr, const WaitCtx& w) {
    const uint64_t t0 = global_timer_ns();
    uint32_t spins = 0;
    for (;;) {
        unsigned int v;
        asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(v) : "l"(ctr) : "memory");
        if (v == 0) return true;
        if ((spins++ & 63u) == 0) {
            if (*w.abort_flag) return false;
            if (global_timer_ns() - t0 >= w.limit_ns) { raise_abort(w); return false; }
        }
        __nanosleep(64);
    }
}
__device__ __forceinline__ void st_shared_cluster_v4(uint32_t cluster_addr, uint4 v) {
    asm volatile("st.shared::cluster.v4.u32 [%0], {%1, %2, %3, %4};" ::"r"(cluster_addr), "r"(v.x), "r"(v.y), "r"(v.z), "r"(v.w) : "memory");
}
// TMA load whose bytes are counted on a barrier that may live in the peer CTA of the pair
__device__ __forceinline__ void tma_load_2d_pair(uint32_t dst, const void* tmap, uint32_t bar_cluster_addr, int32_t c0, int32_t c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(tmap), "r"(bar_cluster_addr), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void tma_load_3d_pair(uint32_t dst, const void* tmap, uint32_t bar_cluster_addr, int32_t c0, int32_t c1, int32_t c2) {
    asm volatile(
        "cp.async.bulk.tensor.3d.cta_group::2.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4, %5}], [%2];"
        ::"r"(dst), "l"(tmap), "r"(bar_cluster_addr), "r"(c0), "r"(c1), "r"(c2) : "memory");
}
// Bulk store of a 32 x 32 fp32 box from this CTA's shared memory (rows of 128 bytes, 128-byte swizzle) into a
// matrix in this GPU's memory; completion is tracked by the issuing thread's bulk groups.
__device__ __forceinline__ void tma_store_2d(const void* tmap, uint32_t src, int32_t c0, int32_t c1) {
    asm volatile("cp.async.bulk.tensor.2d.global.shared::cta.bulk_group [%0, {%2, %3}], [%1];" ::"l"(tmap), "r"(src), "r"(c0), "r"(c1) : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() { asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory"); }   // sources may be reused
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }             // the stores are complete
__device__ __forceinline__ void tmem_alloc_pair(uint32_t smem_dst, uint32_t ncols) {
    asm volatile("tcgen05.alloc.cta_group::2.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_dst), "r"(ncols) : "memory");
    asm volatile("tcgen05.relinquish_alloc_permit.cta_group::2.sync.aligned;" ::: "memory");
}
__device__ __forceinline__ void tmem_dealloc_pair(uint32_t taddr, uint32_t ncols) {
    asm volatile("tcgen05.dealloc.cta_group::2.sync.aligned.b32 %0, %1;" ::"r"(taddr), "r"(ncols) : "memory");
}
__device__ __forceinline__ void umma_bf16_pair(uint32_t d_tmem, uint64_t a_desc, uint64_t b_desc, uint32_t idesc, uint32_t accumulate) {
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "setp.ne.b32 p, %4, 0;\n\t"
        "tcgen05.mma.cta_group::2.kind::f16 [%0], %1, %2, %3, p;\n\t}"
        ::"r"(d_tmem), "l"(a_desc), "l"(b_desc), "r"(idesc), "r"(accumulate) : "memory");
}
// arrives, once the MMAs issued so far have completed, on the barrier at this offset in both CTAs
__device__ __forceinline__ void umma_commit_both(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.multicast::cluster.b64 [%0], %1;"
                 ::"r"(bar), "h"((uint16_t)3) : "memory");
}
__device__ __forceinline__ void umma_commit_local_pair(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::2.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
// loads that must see what other SMs wrote a moment ago: from L2, never from this SM's L1
__device__ __forceinline__ float4 ld_cg_f4(const float* p) {
    float4 v;
    asm volatile("ld.global.cg.v4.f32 {%0, %1, %2, %3}, [%4];" : "=f"(v.x), "=f"(v.y), "=f"(v.z), "=f"(v.w) : "l"(p) : "memory");
    return v;
}
__device__ __forceinline__ uint32_t pack_bf16(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);      // round to nearest even; .x = lo is the low half
    return *reinterpret_cast<const uint32_t*>(&v);
}

// Staging tile of an epilogue warp: 32 rows x 32 fp32, row r at r * 128 bytes, its eight 16-byte chunks
// stored at chunk position j ^ (r & 7) (the 128-byte swizzle pattern): a lane writing its own row and
// 8 lanes reading one row both touch all 32 banks once, so neither direction has bank conflicts.
__device__ __forceinline__ void stage_row(float* stage_tile, uint32_t row, const uint32_t (&v)[32]) {
    float4* base = reinterpret_cast<float4*>(stage_tile) + row * 8u;
#pragma unroll
    for (uint32_t j = 0; j < 8; ++j)
        base[j ^ (row & 7u)] = make_float4(__uint_as_float(v[4 * j]), __uint_as_float(v[4 * j + 1]), __uint_as_float(v[4 * j + 2]), __uint_as_float(v[4 * j + 3]));
}
// The same chunk rounded to bf16: 32 rows of 64 bytes, the four 16-byte chunks of row r stored at chunk position
// j ^ ((r >> 1) & 3) (the 64-byte swizzle pattern of the bf16 tensor map of C; a warp's 512 bytes per step
// touch every bank four times, the minimum).
__device__ __forceinline__ void stage_row_bf16(float* stage_tile, uint32_t row, const uint32_t (&v)[32]) {
    uint4* base = reinterpret_cast<uint4*>(stage_tile) + row * 4u;
#pragma unroll
    for (uint32_t j = 0; j < 4; ++j)
        base[j ^ ((row >> 1) & 3u)] = make_uint4(pack_bf16(__uint_as_float(v[8 * j]), __uint_as_float(v[8 * j + 1])),
                                                 pack_bf16(__uint_as_float(v[8 * j + 2]), __uint_as_float(v[8 * j + 3])),
                                                 pack_bf16(__uint_as_float(v[8 * j + 4]), __uint_as_float(v[8 * j + 5])),
                                                 pack_bf16(__uint_as_float(v[8 * j + 6]), __uint_as_float(v[8 * j + 7])));
}
__device__ __forceinline__ float4 staged_f4(const float* stage_tile, uint32_t row, uint32_t col4) {      // columns 4*col4 .. +3
    return reinterpret_cast<const float4*>(stage_tile)[row * 8u + (col4 ^ (row & 7u))];
}
__device__ __forceinline__ float staged_f(const float* stage_tile, uint32_t row, uint32_t col) {
    return stage_tile[row * 32u + (((col >> 2) ^ (row & 7u)) << 2) + (col & 3u)];
}

// bytes CTA with `rows` valid rows loads per K-block of a pair whose MMA is n_mma columns wide
__device__ __forceinline__ uint32_t stage_bytes(uint32_t rows, uint32_t n_mma) {
    const uint32_t nsub_a = (rows + kSubRows - 1) / kSubRows;
    const uint32_t nsub_b = (n_mma / 2 + kSubRows - 1) / kSubRows;
    return (nsub_a + nsub_b) * kSubBytes;
}
struct __align__(16) PairShared {
    uint64_t full[kPairStages];
    uint64_t empty[kPairStages];
    uint64_t acc_full[kAccSlots];
    uint64_t acc_empty[kAccSlots];
    uint64_t sched_full[kSchedSlots];
    uint64_t sched_empty[kSchedSlots];
    uint64_t drain;
    uint32_t tmem_base;
    uint32_t abort_flag;
    TileDesc slot[kSchedSlots];
};

// Sum of the SP (slice count padded to a power of two) blocks of a cell for one 32-row strip, in
// the order of the assembly kernel: balanced pairwise tree over adjacent slices, missing slices
// contribute +0.0f.  One float4 per lane and step, four to eight steps in flight.
template <int SP, bool BF16>
__device__ __forceinline__ void finish_strip(const FinRef* __restrict__ refs, uint32_t nslices, const float* __restrict__ partials,
                                             uint32_t row0, uint32_t nrows, uint32_t cols, void* c_base, uint64_t c_off,
                                             uint32_t ldc, uint32_t lane) {
    constexpr int U = SP <= 2 ? 8 : (SP <= 4 ? 4 : 2);
    const float* src[SP];
    uint32_t ld[SP];
#pragma unroll
    for (int s = 0; s < SP; ++s) {
        if ((uint32_t)s < nslices) { const FinRef rf = refs[s]; src[s] = partials + rf.off + (uint64_t)row0 * rf.ld; ld[s] = rf.ld; }
        else { src[s] = nullptr; ld[s] = 0; }
    }
    const uint32_t c4 = cols >> 2, units = nrows * c4;
    for (uint32_t base = 0; base < units; base += 32 * U) {
        float4 acc[U];
        uint32_t urow[U], ucol[U];
#pragma unroll
        for (int u = 0; u < U; ++u) {
            const uint32_t unit = base + u * 32 + lane;
            const bool live = unit < units;
            urow[u] = live ? unit / c4 : 0u;
            ucol[u] = live ? (unit - urow[u] * c4) * 4u : 0u;
            float4 v[SP];
#pragma unroll
            for (int s = 0; s < SP; ++s) {
                v[s] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (live && src[s]) v[s] = ld_cg_f4(src[s] + (uint64_t)urow[u] * ld[s] + ucol[u]);
            }
#pragma unroll
            for (int w = 1; w < SP; w *= 2)
#pragma unroll
                for (int s = 0; s < SP; s += 2 * w) {
                    v[s].x += v[s + w].x; v[s].y += v[s + w].y; v[s].z += v[s + w].z; v[s].w += v[s + w].w;
                }
            acc[u] = v[0];
        }
#pragma unroll
        for (int u = 0; u < U; ++u) {
            if (base + u * 32 + lane >= units) continue;
            const uint64_t at = c_off + (uint64_t)(row0 + urow[u]) * ldc + ucol[u];
            if (BF16) *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(c_base) + at) =
                          make_uint2(pack_bf16(acc[u].x, acc[u].y), pack_bf16(acc[u].z, acc[u].w));
            else      *reinterpret_cast<float4*>(static_cast<float*>(c_base) + at) = acc[u];
        }
    }
}

// One 32 x 32 chunk of a strip whose cell is complete but for this block: the accumulator values
// (own K-slice `mine`) go to the block in the arena as always, and, added to the other slices' values
// in the fixed tree order, to C.  Lanes: 8 per row segment of 32 columns, 4 rows per step.  The other
// slices' values are asked for before the accumulator chunk is read from tensor memory and staged,
// so their latency (L2: they were prefetched when the tile was handed out) overlaps that work.
struct SummedChunk {
    const FinRef* refs;         // the cell's blocks, slice order
    uint32_t nslices, mine;
    const float* partials;
    float* own_blk;             // the quadrant's (row0, 0) in this task's block
    uint32_t own_ld;
    uint32_t row0, rows_here;
    uint32_t c0, cols;          // first column of the chunk inside the quadrant; the quadrant's columns
    void* c_base;
    uint64_t c_off;             // the quadrant's (0, 0) in C
    uint32_t ldc;
    uint32_t taddr;             // tensor-memory address of the chunk
    bool last_chunk;            // reading it frees the accumulator slot
    bool keep_own;              // the own block is stored in the arena as well
    uint32_t acc_empty_leader;
};
template <int SP, bool BF16>
__device__ __forceinline__ void summed_chunk(const SummedChunk& k, float* stage_tile, uint32_t lane) {
    constexpr int RB = SP <= 2 ? 8 : (SP <= 4 ? 4 : 1);      // rows per lane whose loads are in flight together
    constexpr int NO = SP - 1;                               // other slices (slot j holds slice j, or j + 1 from `mine` on)
    const uint32_t rr = lane >> 3, cc = (lane & 7u) * 4u;
    const uint32_t rows_here = (k.c0 + cc >= k.cols) ? 0u : k.rows_here;   // ragged last chunk (columns come in fours)
    const float* src[NO];
    uint32_t ld[NO];
#pragma unroll
    for (int j = 0; j < NO; ++j) {
        const uint32_t s = (uint32_t)j < k.mine ? (uint32_t)j : (uint32_t)j + 1u;
        if (s < k.nslices) { const FinRef rf = k.refs[s]; src[j] = k.partials + rf.off + (uint64_t)k.row0 * rf.ld + k.c0 + cc; ld[j] = rf.ld; }
        else { src[j] = nullptr; ld[j] = 0; }
    }
    float4 o[RB][NO];
    auto load_batch = [&](int b) {
#pragma unroll
        for (int x = 0; x < RB; ++x) {
            const uint32_t r = rr + 4u * (uint32_t)(b + x);
#pragma unroll
            for (int j = 0; j < NO; ++j) {
                o[x][j] = make_float4(0.f, 0.f, 0.f, 0.f);
                if (r < rows_here && src[j]) o[x][j] = ld_cg_f4(src[j] + (uint64_t)r * ld[j]);
            }
        }
    };
    load_batch(0);
    {
        uint32_t v[32];
        tmem_ld_32x32(k.taddr, v);
        tmem_ld_wait();
        if (k.last_chunk) {                                  // slot fully read: hand it back to the leader
            tc_fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster_read_done(k.acc_empty_leader);
        }
        stage_row(stage_tile, lane, v);
    }
    __syncwarp();
#pragma unroll
    for (int b = 0; b < 8; b += RB) {
        if (b) load_batch(b);
#pragma unroll
        for (int x = 0; x < RB; ++x) {
            const uint32_t r = rr + 4u * (uint32_t)(b + x);
            if (r >= rows_here) continue;
            const float4 own = staged_f4(stage_tile, r, lane & 7u);
            if (k.keep_own) *reinterpret_cast<float4*>(k.own_blk + (uint64_t)r * k.own_ld + k.c0 + cc) = own;
            float4 v[SP];
#pragma unroll
            for (int s = 0; s < SP; ++s) {
                const float4 lo = o[x][s > 0 ? s - 1 : 0], hi = o[x][s < NO ? s : NO - 1];   // slice s sits in slot s - 1 or s
                v[s] = (uint32_t)s == k.mine ? own : ((uint32_t)s > k.mine ? lo : hi);
            }
#pragma unroll
            for (int w = 1; w < SP; w *= 2)
#pragma unroll
                for (int s = 0; s < SP; s += 2 * w) { v[s].x += v[s + w].x; v[s].y += v[s + w].y; v[s].z += v[s + w].z; v[s].w += v[s + w].w; }
            const uint64_t at = k.c_off + (uint64_t)(k.row0 + r) * k.ldc + k.c0 + cc;
            if (BF16) *reinterpret_cast<uint2*>(static_cast<__nv_bfloat16*>(k.c_base) + at) =
                          make_uint2(pack_bf16(v[0].x, v[0].y), pack_bf16(v[0].z, v[0].w));
            else      *reinterpret_cast<float4*>(static_cast<float*>(k.c_base) + at) = v[0];
        }
    }
    __syncwarp();
}

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kExecThreads, 1)
exec_pair_kernel(const __grid_constant__ ExecParams P) {
    extern __shared__ uint8_t dyn_smem[];
    __shared__ PairShared sh;

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();          // 0 = leader (issues the MMAs), 1 = peer
    const uint32_t stage_base = (smem_u32(dyn_smem) + 1023u) & ~1023u;
    const WaitCtx W = {&sh.abort_flag, P.status, P.wait_limit_ns};

    if (threadIdx.x == 0) {
        for (int s = 0; s < kPairStages; ++s) { mbar_init(smem_u32(&sh.full[s]), 1); mbar_init(smem_u32(&sh.empty[s]), 1); }
        for (int a = 0; a < kAccSlots; ++a) { mbar_init(smem_u32(&sh.acc_full[a]), 1); mbar_init(smem_u32(&sh.acc_empty[a]), 2 * kEpiWarpsPerGroup); }
        // consumers of a slot: leader's producer, MMA thread and epilogue warps; peer's producer and epilogue warps
        for (int q = 0; q < kSchedSlots; ++q) { mbar_init(smem_u32(&sh.sched_full[q]), 1); mbar_init(smem_u32(&sh.sched_empty[q]), 3 + 2 * kEpiWarps); }
        mbar_init(smem_u32(&sh.drain), 1);
        sh.abort_flag = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    }
    if (warp == kMmaWarp) tmem_alloc_pair(smem_u32(&sh.tmem_base), kTmemCols);     // one warp of each CTA of the pair
    tc_fence_before();
    cluster_arrive_wait();                            // barriers of both CTAs initialised before any remote arrive
    tc_fence_after();
    const uint32_t tmem_base = sh.tmem_base;

    if (warp == kSchedWarp) {
        // ---- scheduler (leader only): tickets -> descriptors -> both CTAs' slot rings ----------------------------
        // A fetch is two dependent trips to L2 (the ticket, then the descriptor), a few thousand cycles behind a
        // burst of stores: too long for pairs that run a handful of K-blocks.  So after such a pair the next
        // fetch takes four tickets with one atomic and lane b loads descriptor b, all at once; the lanes
        // then publish in ticket order.  Longer pairs are fetched one by one (a cluster that holds several of
        // them would keep the others waiting at the end of the list, or of a small GEMM's share of it).
        if (rank == 0) {
            uint32_t levels_done = 0;                  // every level below this one is known to be complete
            uint32_t i = 0;                            // slots published so far
            uint32_t batch = 1;
            bool stop = false;
            while (!stop) {
                uint32_t t0 = 0;
                if (lane == 0) t0 = atomicAdd(P.ticket, batch);
                t0 = __shfl_sync(0xFFFFFFFFu, t0, 0);
                const uint32_t t = t0 + lane;
                uint4 w[kTileWords16];
                if (lane < batch && t < P.tile_end) {
                    const uint4* src = reinterpret_cast<const uint4*>(P.tiles + t);
#pragma unroll
                    for (int x = 0; x < kTileWords16; ++x) w[x] = __ldg(src + x);
                } else {
#pragma unroll
                    for (int x = 0; x < kTileWords16; ++x) w[x] = make_uint4(0, 0, 0, 0);
                    w[0].y = TILE_END;
                }
                uint32_t next_batch = 1;
                for (uint32_t b = 0; b < batch && !stop; ++b) {
                    uint32_t action = 0;               // 0 nothing to run in this pair, 1 published, 2 end of the list published, 3 gave up
                    if (lane == b && (w[0].y & (TILE_LIVE0 | TILE_LIVE1 | TILE_END))) {      // TileDesc::flags
                        const uint32_t q = i % kSchedSlots, par = (i / kSchedSlots) & 1u;
                        bool ok = mbar_wait_cl(smem_u32(&sh.sched_empty[q]), par ^ 1u, W);
                        if (ok && !(w[0].y & TILE_END)) {
                            // a tile of a higher DAG level runs only after every strip of the lower levels is written
                            const uint32_t level = w[1].w & 0xFFFFu;         // TileDesc::level
                            while (ok && levels_done < level) { ok = wait_zero(P.level_left + levels_done, W); if (ok) ++levels_done; }
                        }
                        if (ok) {
                            uint4* dst = reinterpret_cast<uint4*>(&sh.slot[q]);
                            const uint32_t peer_slot = mapa_shared(smem_u32(&sh.slot[q]), 1u);
#pragma unroll
                            for (int x = 0; x < kTileWords16; ++x) { dst[x] = w[x]; st_shared_cluster_v4(peer_slot + 16 * x, w[x]); }
                            mbar_arrive_cluster(mapa_shared(smem_u32(&sh.sched_full[q]), 0u));
                            mbar_arrive_cluster(mapa_shared(smem_u32(&sh.sched_full[q]), 1u));
                        }
                        action = !ok ? 3u : ((w[0].y & TILE_END) ? 2u : 1u);
                    }
                    action = __shfl_sync(0xFFFFFFFFu, action, b);
                    levels_done = __shfl_sync(0xFFFFFFFFu, levels_done, b);
                    if (action == 1u) {
                        ++i;
                        const uint32_t nkb = __shfl_sync(0xFFFFFFFFu, (w[1].y - w[1].x + kBlockK - 1) / kBlockK, b);   // TileDesc::k1, k0
                        next_batch = nkb <= 4u ? 4u : 1u;
                    }
                    if (action >= 2u) stop = true;
                }
                batch = next_batch;
            }
        }
    } else if (warp == kTmaWarp) {
        // ---- producer (both CTAs): own rows of A, own half of the columns of B ------------------------------
        uint32_t it = 0, last_gemm = 0xFFFFFFFFu, last_level = 0;
        bool ok = true;
        const uint32_t sched_empty_leader0 = mapa_shared(smem_u32(&sh.sched_empty[0]), 0u);
        const uint32_t full_leader0 = mapa_shared(smem_u32(&sh.full[0]), 0u);
        for (uint32_t i = 0; ok; ++i) {
            const uint32_t q = i % kSchedSlots, par = (i / kSchedSlots) & 1u;
            if (!__all_sync(0xFFFFFFFFu, mbar_wait_cl(smem_u32(&sh.sched_full[q]), par, W))) break;
            const TileDesc& sl = sh.slot[q];
            const uint32_t flags = sl.flags, gemm = sl.gemm, level = sl.level & 0xFFFFu, n_mma = sl.n_mma & 0xFFFFu;
            const uint32_t n_col = sl.n_col, k0 = sl.k0, k1 = sl.k1;
            const uint32_t rows0 = (flags & TILE_LIVE0) ? sl.h[0].rows : 0u, rows1 = (flags & TILE_LIVE1) ? sl.h[1].rows : 0u;
            const uint32_t a_x = sl.h[rank].m_row;
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster_read_done(sched_empty_leader0 + q * 8u);
            if (flags & TILE_END) break;
            const CUtensorMap* map_a = P.maps + kMapsPerGemm * gemm;
            const CUtensorMap* map_b = map_a + 1;
            const bool new_gemm = gemm != last_gemm;     // (each issuing lane acquires the one map it uses, below)
            last_gemm = gemm;
            if (level != last_level) {
                // operands of this level may have been written by other SMs a moment ago (ordinary stores, seen
                // through the scheduler's acquire): order them before this thread's asynchronous loads
                asm volatile("fence.proxy.async.global;" ::: "memory");
                last_level = level;
            }
            const uint32_t half_n = n_mma / 2;
            const uint32_t my_rows = rank ? rows1 : rows0;
            const uint32_t b_x = n_col + rank * half_n;
            // More than 64 rows / columns of an operand come with ONE operation where a double-size box
            // exists (fewer, larger TMA operations: +9 % on GEMMs whose operands are K-contiguous); an
            // M/N-contiguous operand also needs its first element on a 64-element group boundary.
            const bool a_big = (flags & TILE_A_BIG) && my_rows > kSubRows && (!(flags & TILE_A_MN) || a_x % kSubRows == 0);
            const bool b_big = (flags & TILE_B_BIG) && half_n > kSubRows && (!(flags & TILE_B_MN) || b_x % kSubRows == 0);
            const uint32_t nsub_a = a_big ? 1u : (my_rows + kSubRows - 1) / kSubRows;
            const uint32_t nsub_b = b_big ? 1u : (half_n + kSubRows - 1) / kSubRows;
            // bytes per stage do not depend on the box size: a double-size box is two 8 KB boxes
            const uint32_t tx_both = stage_bytes(rows0, n_mma) + stage_bytes(rows1, n_mma);
            const uint32_t nkb = (k1 - k0 + kBlockK - 1) / kBlockK;
            const bool is_a = lane < nsub_a, is_b = !is_a && lane < nsub_a + nsub_b;
            const uint32_t j = is_a ? lane : lane - nsub_a;
            const bool my_big = is_a ? a_big : b_big;
            const CUtensorMap* my_map = (is_a ? map_a : map_b) + (my_big ? 2 : 0);
            const bool my_mn = is_a ? (flags & TILE_A_MN) : (flags & TILE_B_MN);
            const int32_t my_x = (int32_t)((is_a ? a_x : b_x) + j * kSubRows);
            const uint32_t my_off = (is_a ? 0u : kPairABytes) + j * kSubBytes;
            if (new_gemm && (is_a || is_b)) tensormap_acquire(my_map);
            for (uint32_t kb = 0; kb < nkb; ++kb, ++it) {
                const uint32_t s = it % kPairStages, ph = (it / kPairStages) & 1u;
                if (!__all_sync(0xFFFFFFFFu, mbar_wait_cl(smem_u32(&sh.empty[s]), ph ^ 1u, W))) { ok = false; break; }
                if (rank == 0 && lane == 0) mbar_arrive_expect_tx(smem_u32(&sh.full[s]), tx_both);
                __syncwarp();
                const int32_t k = (int32_t)(k0 + kb * kBlockK);
                if (is_a || is_b) {
                    const uint32_t dst = stage_base + s * kPairStageBytes + my_off;
                    const uint32_t bar = full_leader0 + s * 8u;
                    if (my_mn && my_big) tma_load_3d_pair(dst, my_map, bar, 0, k, my_x / (int32_t)kSubRows);
                    else if (my_mn)      tma_load_2d_pair(dst, my_map, bar, my_x, k);
                    else                 tma_load_2d_pair(dst, my_map, bar, k, my_x);
                }
            }
        }
        // Every stage armed on the normal path has been waited for by the leader's MMA thread, and a stage
        // only completes once this CTA's own bytes have landed.  When the pair is aborting, copies may
        // still be in flight towards this CTA's shared memory: give them a bounded time to land.
        if (*W.abort_flag && lane == 0) {
            const uint64_t t0 = global_timer_ns();
            while (global_timer_ns() - t0 < 200000ull) { }
        }
    } else if (warp == kMmaWarp) {
        // ---- MMA issuer (leader only) ---------------------------------------------------------------------------
        if (rank == 0 && lane == 0) {
            uint32_t it = 0, tile_no = 0;
            bool ok = true;
            for (uint32_t i = 0; ok; ++i) {
                const uint32_t q = i % kSchedSlots, par = (i / kSchedSlots) & 1u;
                if (!mbar_wait_cl(smem_u32(&sh.sched_full[q]), par, W)) break;
                const uint32_t flags = sh.slot[q].flags, n_mma = sh.slot[q].n_mma & 0xFFFFu;
                const uint32_t k0 = sh.slot[q].k0, k1 = sh.slot[q].k1;
                mbar_arrive(smem_u32(&sh.sched_empty[q]));
                if (flags & TILE_END) break;
                const uint32_t a_mn = (flags & TILE_A_MN) ? 1u : 0u, b_mn = (flags & TILE_B_MN) ? 1u : 0u;
                const uint32_t idesc = instr_desc_bf16(2 * kBlockM, n_mma, a_mn, b_mn);
                const uint32_t a_lbo = a_mn ? kSubBytes : 16u, a_step = a_mn ? 2048u : 32u;
                const uint32_t b_lbo = b_mn ? kSubBytes : 16u, b_step = b_mn ? 2048u : 32u;
                const uint32_t acc = tile_no & 1u, aph = (tile_no >> 1) & 1u;
                if (!mbar_wait_cl(smem_u32(&sh.acc_empty[acc]), aph ^ 1u, W)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * kAccCols;
                const uint32_t nkb = (k1 - k0 + kBlockK - 1) / kBlockK;
                for (uint32_t kb = 0; kb < nkb; ++kb, ++it) {
                    const uint32_t s = it % kPairStages, ph = (it / kPairStages) & 1u;
                    if (!mbar_wait_cl(smem_u32(&sh.full[s]), ph, W)) { ok = false; break; }
                    tc_fence_after();
                    const uint32_t sa = stage_base + s * kPairStageBytes, sb = sa + kPairABytes;
#pragma unroll
                    for (uint32_t k16 = 0; k16 < kBlockK / 16; ++k16)
                        umma_bf16_pair(d_tmem, smem_desc_sw128(sa + k16 * a_step, a_lbo, 1024u),
                                       smem_desc_sw128(sb + k16 * b_step, b_lbo, 1024u), idesc, (kb | k16) != 0u);
                    umma_commit_both(smem_u32(&sh.empty[s]));
                }
                if (!ok) break;
                umma_commit_both(smem_u32(&sh.acc_full[acc]));
                ++tile_no;
            }
            // every MMA issued above has completed before either CTA may release tensor memory or exit
            umma_commit_local_pair(smem_u32(&sh.drain));
            const uint64_t t0 = global_timer_ns();
            while (!mbar_try_wait_cl(smem_u32(&sh.drain), 0u))
                if (global_timer_ns() - t0 > 2000000000ull) { atomicOr(P.status, STATUS_TIMEOUT); break; }
        }
    } else if (warp >= kEpiWarp0) {
        // ---- epilogue (both CTAs): the 128 accumulator rows of this CTA's half -> block / C, bookkeeping --------
        const uint32_t group = (warp - kEpiWarp0) / kEpiWarpsPerGroup;
        const uint32_t quad = warp & 3u;
        float* stage_tile = reinterpret_cast<float*>(dyn_smem + (stage_base - smem_u32(dyn_smem)) + kPairStages * kPairStageBytes) +
                            (warp - kEpiWarp0) * kEpiStageFloats;
        const uint32_t sched_empty_leader0 = mapa_shared(smem_u32(&sh.sched_empty[0]), 0u);
        const uint32_t acc_empty_leader = mapa_shared(smem_u32(&sh.acc_empty[group]), 0u);
        const bool out_bf16 = P.mode & MODE_BF16;
        uint32_t used = 0, tile_no = 0;
        // Bookkeeping owed for strips already stored: lane j keeps entry j (the quadrants' tasks, the level and
        // how many strips to count off it).  The counts may only be made after a fence that waits for the
        // strip's stores, and such a fence costs thousands of cycles behind a burst of stores; so it is paid
        // when the warp would wait anyway (no tile ready), when kMaxOwed entries have gathered, before any
        // bookkeeping that cannot wait (cells of the in-kernel sum), and when the warp leaves.
        constexpr uint32_t kMaxOwed = 8;
        uint32_t owed = 0, owed_task0 = 0xFFFFFFFFu, owed_task1 = 0xFFFFFFFFu, owed_level = 0, owed_strips = 0;
        auto count_owed = [&]() {                         // (the caller has fenced and synchronised the warp)
            if (lane < owed) {
                if (owed_task0 != 0xFFFFFFFFu) atomicAdd(&P.done[owed_task0], 1u);   // one count per warp and quadrant
                if (owed_task1 != 0xFFFFFFFFu) atomicAdd(&P.done[owed_task1], 1u);
                if (owed_strips) atomicSub(&P.level_left[owed_level], owed_strips);
            }
            owed = 0;
            __syncwarp();
        };
        // Blocks that go straight to an fp32 C leave as bulk stores of whole 32 x 32 chunks (issued by lane 0, which
        // then does not wait for them): `bulk_reading` = a store may still be reading the staging tile,
        // `bulk_flying` = stores of this warp may be incomplete (they must be complete before anything is counted).
        bool bulk_reading = false, bulk_flying = false;
        uint32_t c_map_gemm = 0xFFFFFFFFu;
        auto staging_free = [&]() {
            if (bulk_reading) { if (lane == 0) bulk_wait_read_all(); __syncwarp(); bulk_reading = false; }
        };
        auto fence_stores = [&]() {                       // every store of this warp so far, plain or bulk, is visible
            if (bulk_flying) { if (lane == 0) bulk_wait_all(); __syncwarp(); bulk_flying = bulk_reading = false; }
            __threadfence();
            __syncwarp();
        };
        auto settle = [&]() {
            if (owed) { fence_stores(); count_owed(); }
        };
        for (uint32_t i = 0;; ++i) {
            const uint32_t q = i % kSchedSlots, par = (i / kSchedSlots) & 1u;
            bool ok = mbar_try_wait_cl(smem_u32(&sh.sched_full[q]), par);
            if (!__all_sync(0xFFFFFFFFu, ok)) {
                settle();
                ok = mbar_wait_cl(smem_u32(&sh.sched_full[q]), par, W);
                if (!__all_sync(0xFFFFFFFFu, ok)) break;
            }
            const TileDesc& sl = sh.slot[q];
            const uint32_t flags = sl.flags, gemm = sl.gemm, n_mma = sl.n_mma & 0xFFFFu, cols = sl.n_mma >> 16;
            const uint32_t level = sl.level & 0xFFFFu, nslices = (sl.level >> 16) & 0xFFu, kslice = sl.level >> 24;
            const uint32_t ldc = sl.ldc, n_col = sl.n_col, split = sl.split;
            // (the two column segments in variables of their own: an array indexed by the chunk's segment would live
            // in local memory, and a local load queues behind the stores in flight)
            const uint32_t h_m_row = sl.h[rank].m_row, h_rows = sl.h[rank].rows;
            const TileSeg seg0 = sl.h[rank].seg[0], seg1 = sl.h[rank].seg[1];
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster_read_done(sched_empty_leader0 + q * 8u);
            if (flags & TILE_END) break;
            const bool mine = (tile_no & 1u) == group;       // tiles alternate between the two accumulator slots
            ++tile_no;
            if (!mine) continue;
            const uint32_t rows = (flags & (TILE_LIVE0 << rank)) ? h_rows : 0u;
            const uint32_t rows_here = rows > quad * 32u ? min(32u, rows - quad * 32u) : 0u;
            const uint32_t row0 = quad * 32u;
            // a block of a one-slice GEMM is final: it may go straight to its place in C
            const bool direct = (P.mode & MODE_DIRECT) && (flags & TILE_SINGLE);
            const bool to_bf16 = direct && out_bf16;
            const bool bulk_ok = direct && rows_here == 32u && ((ldc | n_col) & (out_bf16 ? 7u : 3u)) == 0u;
            const CUtensorMap* c_map = P.c_maps + 2u * gemm + (out_bf16 ? 1u : 0u);
            if (bulk_ok && gemm != c_map_gemm) {
                if (lane == 0) tensormap_acquire(c_map);
                c_map_gemm = gemm;
            }
            const uint64_t c_off = (uint64_t)h_m_row * ldc + n_col;            // the half-tile's (0, 0) in C
            // the one or two column segments of the half-tile: quadrants of possibly different tasks
            const uint32_t width[2] = {min(split, cols), cols > split ? cols - split : 0u};
            bool cell[2], sum_now[2] = {false, false};
            const FinRef* refs[2] = {nullptr, nullptr};
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const TileSeg& sg = q ? seg1 : seg0;
                cell[q] = rows && sg.live && width[q] && (P.mode & MODE_FINISH) && !direct && sg.fin != kNoFin;
                // Is every other K-slice's block of this strip's cell stored already?  Then this strip is the last
                // one: start bringing those blocks into L2 now, while the MMAs of this tile still run.
                if (cell[q]) {
                    unsigned int arrived;
                    asm volatile("ld.acquire.gpu.global.u32 %0, [%1];" : "=r"(arrived) : "l"(P.fin_count + sg.fin * 4u + quad) : "memory");
                    sum_now[q] = __shfl_sync(0xFFFFFFFFu, arrived, 0) + 1u == nslices;
                    refs[q] = P.fin_refs + __ldg(P.fin_ref0 + sg.fin);
                    if (sum_now[q] && rows_here) {
                        const uint32_t lines_per_row = (width[q] * 4u + 127u) / 128u;
                        for (uint32_t s = 0; s < nslices; ++s) {
                            if (s == kslice) continue;
                            const FinRef rf = refs[q][s];
                            const float* base = P.partials + rf.off + (uint64_t)row0 * rf.ld;
                            for (uint32_t x = lane; x < rows_here * lines_per_row; x += 32u) {
                                const uint32_t r = x / lines_per_row, seg = x - r * lines_per_row;
                                asm volatile("prefetch.global.L2 [%0];" ::"l"(base + (uint64_t)r * rf.ld + seg * 32u));
                            }
                        }
                    }
                }
            }
            ok = mbar_try_wait_cl(smem_u32(&sh.acc_full[group]), used & 1u);
            if (!__all_sync(0xFFFFFFFFu, ok)) {
                settle();
                ok = mbar_wait_cl(smem_u32(&sh.acc_full[group]), used & 1u, W);
                if (!__all_sync(0xFFFFFFFFu, ok)) break;
            }
            ++used;
            tc_fence_after();
            const uint32_t taddr = tmem_base + group * kAccCols + ((quad * 32u) << 16);
            const uint32_t nchunk = (n_mma + 31u) / 32u;
            for (uint32_t c = 0; c < nchunk; ++c) {
                const bool q = c * 32u >= split;             // (split is a multiple of 32 when a second segment exists)
                const uint32_t sg_ld = q ? seg1.ld : seg0.ld, sg_live = q ? seg1.live : seg0.live;
                const uint64_t sg_out_off = q ? seg1.out_off : seg0.out_off;
                const bool live_chunk = rows_here && sg_live && c * 32u < cols;   // warp-uniform
                const uint32_t ct = c * 32u;                 // chunk's first column in the half-tile ...
                const uint32_t c0 = ct - (q ? split : 0u);   // ... and in its quadrant
                if (live_chunk && (q ? sum_now[1] : sum_now[0])) {
                    staging_free();
                    // (cells exist only where float4 accesses are aligned and columns come in fours)
                    SummedChunk k;
                    k.refs = q ? refs[1] : refs[0]; k.nslices = nslices; k.mine = kslice; k.partials = P.partials;
                    k.own_blk = P.partials + sg_out_off + (uint64_t)row0 * sg_ld; k.own_ld = sg_ld;
                    k.row0 = row0; k.rows_here = rows_here; k.c0 = c0; k.cols = q ? width[1] : width[0];
                    k.c_base = P.c_ptrs[gemm]; k.c_off = c_off + (q ? split : 0u); k.ldc = ldc;
                    k.taddr = taddr + ct; k.last_chunk = (c + 1 == nchunk); k.keep_own = !(P.mode & MODE_CONSUME); k.acc_empty_leader = acc_empty_leader;
                    if (nslices <= 2) { if (out_bf16) summed_chunk<2, true>(k, stage_tile, lane); else summed_chunk<2, false>(k, stage_tile, lane); }
                    else if (nslices <= 4) { if (out_bf16) summed_chunk<4, true>(k, stage_tile, lane); else summed_chunk<4, false>(k, stage_tile, lane); }
                    else { if (out_bf16) summed_chunk<8, true>(k, stage_tile, lane); else summed_chunk<8, false>(k, stage_tile, lane); }
                    continue;
                }
                uint32_t v[32];
                tmem_ld_32x32(taddr + ct, v);
                tmem_ld_wait();
                if (c + 1 == nchunk) {                       // slot fully read: hand it back to the leader
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster_read_done(acc_empty_leader);
                }
                if (!live_chunk) continue;
                staging_free();
                if (bulk_ok && ct + 32u <= cols) {
                    if (to_bf16) stage_row_bf16(stage_tile, lane, v); else stage_row(stage_tile, lane, v);
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");      // the staged values, before the bulk store reads them
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(c_map, smem_u32(stage_tile), (int32_t)(n_col + ct), (int32_t)(h_m_row + row0));
                        bulk_commit();
                    }
                    bulk_reading = bulk_flying = true;
                    continue;
                }
                stage_row(stage_tile, lane, v);
                __syncwarp();
                const uint32_t ld = direct ? ldc : sg_ld;
                const uint64_t out_off = direct ? c_off + (uint64_t)row0 * ldc + ct : sg_out_off + (uint64_t)row0 * sg_ld + c0;
                float* out_f32 = (direct ? static_cast<float*>(P.c_ptrs[gemm]) : P.partials) + out_off;
                __nv_bfloat16* out_b16 = static_cast<__nv_bfloat16*>(P.c_ptrs[gemm]) + out_off;
                const bool vec_ok = ((ld & 3u) == 0u) && ((out_off & 3ull) == 0ull);
                if (vec_ok && ct + 32u <= cols) {
                    const uint32_t rr = lane >> 3, cc = (lane & 7u) * 4u;
#pragma unroll
                    for (uint32_t r = rr; r < 32u; r += 4u) {
                        if (r < rows_here) {
                            const float4 x = staged_f4(stage_tile, r, lane & 7u);
                            if (to_bf16) *reinterpret_cast<uint2*>(out_b16 + (uint64_t)r * ld + cc) =
                                             make_uint2(pack_bf16(x.x, x.y), pack_bf16(x.z, x.w));
                            else         *reinterpret_cast<float4*>(out_f32 + (uint64_t)r * ld + cc) = x;
                        }
                    }
                } else if (ct + lane < cols) {
#pragma unroll 8
                    for (uint32_t r = 0; r < rows_here; ++r) {
                        const float x = staged_f(stage_tile, r, lane);
                        if (to_bf16) out_b16[(uint64_t)r * ld + lane] = __float2bfloat16_rn(x);
                        else         out_f32[(uint64_t)r * ld + lane] = x;
                    }
                }
                __syncwarp();
            }
            if (rows) {
                const bool live0 = seg0.live && width[0], live1 = seg1.live && width[1];
                const uint32_t n_live = (live0 ? 1u : 0u) + (live1 ? 1u : 0u);
                if (!cell[0] && !cell[1]) {
                    // nobody waits for these counts right now: owe them (see above)
                    if (lane == owed) {
                        owed_task0 = live0 ? seg0.task : 0xFFFFFFFFu; owed_task1 = live1 ? seg1.task : 0xFFFFFFFFu;
                        owed_level = level; owed_strips = n_live;
                    }
                    if (++owed == kMaxOwed) settle();
                    continue;
                }
                fence_stores();                              // this strip's stores before its arrival is counted
                count_owed();                                // (the fence covered the older strips' stores as well)
#pragma unroll
                for (int q = 0; q < 2; ++q) {
                    const TileSeg& sg = q ? seg1 : seg0;
                    if (!sg.live || !width[q]) continue;
                    if (lane == 0) atomicAdd(&P.done[sg.task], 1u);   // one count per warp and quadrant
                    if (!cell[q]) continue;
                    unsigned int before = 0;
                    if (lane == 0) before = atomicAdd(&P.fin_count[sg.fin * 4u + quad], 1u);
                    before = __shfl_sync(0xFFFFFFFFu, before, 0);
                    // not known to be last when it started, but last all the same: read every block back and sum
                    if (!sum_now[q] && before + 1u == nslices && rows_here) {
                        __threadfence();                     // the other slices' stores are visible after their counts
                        void* cb = P.c_ptrs[gemm];
                        const uint64_t cq = c_off + (q ? split : 0u);
                        if (nslices <= 2) {
                            if (out_bf16) finish_strip<2, true>(refs[q], nslices, P.partials, row0, rows_here, width[q], cb, cq, ldc, lane);
                            else          finish_strip<2, false>(refs[q], nslices, P.partials, row0, rows_here, width[q], cb, cq, ldc, lane);
                        } else if (nslices <= 4) {
                            if (out_bf16) finish_strip<4, true>(refs[q], nslices, P.partials, row0, rows_here, width[q], cb, cq, ldc, lane);
                            else          finish_strip<4, false>(refs[q], nslices, P.partials, row0, rows_here, width[q], cb, cq, ldc, lane);
                        } else {
                            if (out_bf16) finish_strip<8, true>(refs[q], nslices, P.partials, row0, rows_here, width[q], cb, cq, ldc, lane);
                            else          finish_strip<8, false>(refs[q], nslices, P.partials, row0, rows_here, width[q], cb, cq, ldc, lane);
                        }
                    }
                    if (sum_now[q] || before + 1u == nslices) __threadfence();    // the sums, before the level counts this strip
                }
                __syncwarp();
                if (lane == 0 && n_live) atomicSub(&P.level_left[level], n_live);   // after everything this strip had to write
            }
        }
        settle();                                            // whatever is still owed, also when the pair gives up
    }

    __syncwarp();
    tc_fence_before();
    cluster_arrive_wait();                            // both CTAs are done with each other's memory
    if (warp == kMmaWarp) {
        tc_fence_after();
        tmem_dealloc_pair(tmem_base, kTmemCols);
    }
}

cudaError_t exec_pair_kernel_prepare() {
    return cudaFuncSetAttribute(exec_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)kPairDynSmem);
}

cudaError_t launch_exec_pair(uint32_t clusters, const ExecParams& e, cudaStream_t st) {
    exec_pair_kernel<<<2 * clusters, kExecThreads, kPairDynSmem, st>>>(e);
    return cudaGetLastError();
}

}  // namespace cleave
