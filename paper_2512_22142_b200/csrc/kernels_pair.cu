// exec_pair_kernel: the grouped sub-GEMM kernel on pairs of CTAs (thread-block clusters of two,
// tcgen05 cta_group::2).
//
// A tile of up to 256 rows x up to 256 columns is shared by the two CTAs of a cluster: CTA r loads
// rows 128r..128r+127 of A and columns r*N/2..(r+1)*N/2-1 of B into its own shared memory, one
// thread of the leader CTA (rank 0) issues M = 256 MMAs that read both CTAs' shared memory, and each
// CTA receives its 128 rows of the accumulator in its own tensor memory.  Compared with one CTA
// doing both row halves this halves, per SM, the B bytes held, loaded and read by the tensor core
// and the accumulator columns, so six 32 KB stages fit and two accumulator slots double-buffer:
// the write-out of a tile overlaps the MMAs of the next one.
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
// Every device-side wait is bounded: when a wait expires the CTA records E_TIMEOUT in the status
// word and raises its abort flag, all its roles leave their loops, the MMAs in flight are drained
// (again with a bound), both CTAs meet at the cluster barrier, tensor memory is released and the
// kernel returns.
#include <cuda.h>
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
__device__ __forceinline__ uint32_t mbar_try_wait_cl(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.acquire.cluster.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok;
}
static __device__ __noinline__ bool mbar_wait_cl_slow(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                               unsigned int* status) {
    const uint64_t t0 = global_timer_ns();
    uint32_t spins = 0;
    while (!mbar_try_wait_cl(bar, parity)) {
        if ((++spins & 255u) == 0) {
            if (*abort_flag) return false;
            if (global_timer_ns() - t0 > kWaitLimitNs) {
                // give up: raise the abort flag of both CTAs of the pair so that every role leaves at its next check
                const uint32_t flag = smem_u32(const_cast<uint32_t*>(abort_flag));
                asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(mapa_shared(flag, 0u)), "r"(1u) : "memory");
                asm volatile("st.shared::cluster.u32 [%0], %1;" ::"r"(mapa_shared(flag, 1u)), "r"(1u) : "memory");
                atomicOr(status, STATUS_TIMEOUT);
                return false;
            }
        }
    }
    return true;
}
__device__ __forceinline__ bool mbar_wait_cl(uint32_t bar, uint32_t parity, volatile uint32_t* abort_flag,
                                             unsigned int* status) {
    if (mbar_try_wait_cl(bar, parity)) return true;
    return mbar_wait_cl_slow(bar, parity, abort_flag, status);
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

// rows of the tile that belong to CTA `rank` (0..128)
__device__ __forceinline__ uint32_t rows_of_rank(uint32_t tile_rows, uint32_t rank) {
    const uint32_t lo = rank * kBlockM;
    return tile_rows > lo ? min(kBlockM, tile_rows - lo) : 0u;
}
// bytes CTA `rank` loads per K-block of tile d
__device__ __forceinline__ uint32_t stage_bytes_of_rank(uint32_t tile_rows, uint32_t n_mma, uint32_t rank) {
    const uint32_t nsub_a = (rows_of_rank(tile_rows, rank) + kSubRows - 1) / kSubRows;
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

__global__ void __cluster_dims__(2, 1, 1) __launch_bounds__(kExecThreads, 1)
exec_pair_kernel(const TileDesc* __restrict__ tiles, uint32_t tile_end, unsigned int* ticket,
                 const CUtensorMap* __restrict__ maps, float* __restrict__ partials, float* const* __restrict__ c_ptrs,
                 uint32_t* done, unsigned int* status) {
    extern __shared__ uint8_t dyn_smem[];
    __shared__ PairShared sh;

    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t rank = cluster_ctarank();          // 0 = leader (issues the MMAs), 1 = peer
    const uint32_t stage_base = (smem_u32(dyn_smem) + 1023u) & ~1023u;
    volatile uint32_t* abort_flag = &sh.abort_flag;

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
        // ---- scheduler (leader only): ticket -> descriptor -> both CTAs' slot rings -----------------------
        if (rank == 0 && lane == 0) {
            for (uint32_t i = 0;; ++i) {
                const uint32_t q = i % kSchedSlots, par = (i / kSchedSlots) & 1u;
                if (!mbar_wait_cl(smem_u32(&sh.sched_empty[q]), par ^ 1u, abort_flag, status)) break;
                uint4 w0, w1, w2, w3;
                bool end = false;
                for (;;) {
                    const uint32_t t = atomicAdd(ticket, 1u);
                    if (t >= tile_end) { end = true; break; }
                    const uint4* src = reinterpret_cast<const uint4*>(tiles + t);
                    w0 = __ldg(src); w1 = __ldg(src + 1); w2 = __ldg(src + 2); w3 = __ldg(src + 3);
                    if (w0.z & TILE_VALID) break;      // TileDesc::flags
                }
                if (end) { w0 = make_uint4(0, 0, TILE_END, 0); w1 = w2 = w3 = make_uint4(0, 0, 0, 0); }
                uint4* dst = reinterpret_cast<uint4*>(&sh.slot[q]);
                dst[0] = w0; dst[1] = w1; dst[2] = w2; dst[3] = w3;
                const uint32_t peer_slot = mapa_shared(smem_u32(&sh.slot[q]), 1u);
                st_shared_cluster_v4(peer_slot, w0); st_shared_cluster_v4(peer_slot + 16, w1);
                st_shared_cluster_v4(peer_slot + 32, w2); st_shared_cluster_v4(peer_slot + 48, w3);
                mbar_arrive_cluster(mapa_shared(smem_u32(&sh.sched_full[q]), 0u));
                mbar_arrive_cluster(mapa_shared(smem_u32(&sh.sched_full[q]), 1u));
                if (end) break;
            }
        }
    } else if (warp == kTmaWarp) {
        // ---- producer (both CTAs): own rows of A, own half of the columns of B ------------------------------
        uint32_t it = 0, last_gemm = 0xFFFFFFFFu;
        bool ok = true;
        const uint32_t sched_empty_leader0 = mapa_shared(smem_u32(&sh.sched_empty[0]), 0u);
        const uint32_t full_leader0 = mapa_shared(smem_u32(&sh.full[0]), 0u);
        for (uint32_t i = 0; ok; ++i) {
            const uint32_t q = i % kSchedSlots, par = (i / kSchedSlots) & 1u;
            if (!__all_sync(0xFFFFFFFFu, mbar_wait_cl(smem_u32(&sh.sched_full[q]), par, abort_flag, status))) break;
            const TileDesc d = sh.slot[q];
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(sched_empty_leader0 + q * 8u);
            if (d.flags & TILE_END) break;
            const CUtensorMap* map_a = maps + kMapsPerGemm * d.gemm;
            const CUtensorMap* map_b = map_a + 1;
            if (d.gemm != last_gemm) {
                for (int x = 0; x < kMapsPerGemm; ++x) tensormap_acquire(map_a + x);
                last_gemm = d.gemm;
            }
            const uint32_t half_n = d.n_mma / 2;
            const uint32_t my_rows = rows_of_rank(d.rows, rank);
            const uint32_t a_x = d.m_row + rank * kBlockM, b_x = d.n_col + rank * half_n;
            // More than 64 rows / columns of an operand come with ONE operation where a double-size box
            // exists (fewer, larger TMA operations: +9 % on GEMMs whose operands are K-contiguous); an
            // M/N-contiguous operand also needs its first element on a 64-element group boundary.
            const bool a_big = (d.flags & TILE_A_BIG) && my_rows > kSubRows && (!(d.flags & TILE_A_MN) || a_x % kSubRows == 0);
            const bool b_big = (d.flags & TILE_B_BIG) && half_n > kSubRows && (!(d.flags & TILE_B_MN) || b_x % kSubRows == 0);
            const uint32_t nsub_a = a_big ? 1u : (my_rows + kSubRows - 1) / kSubRows;
            const uint32_t nsub_b = b_big ? 1u : (half_n + kSubRows - 1) / kSubRows;
            // bytes per stage do not depend on the box size: a double-size box is two 8 KB boxes
            const uint32_t tx_both = stage_bytes_of_rank(d.rows, d.n_mma, 0u) + stage_bytes_of_rank(d.rows, d.n_mma, 1u);
            const uint32_t nkb = (d.k1 - d.k0 + kBlockK - 1) / kBlockK;
            const bool is_a = lane < nsub_a, is_b = !is_a && lane < nsub_a + nsub_b;
            const uint32_t j = is_a ? lane : lane - nsub_a;
            const bool my_big = is_a ? a_big : b_big;
            const CUtensorMap* my_map = (is_a ? map_a : map_b) + (my_big ? 2 : 0);
            const bool my_mn = is_a ? (d.flags & TILE_A_MN) : (d.flags & TILE_B_MN);
            const int32_t my_x = (int32_t)((is_a ? a_x : b_x) + j * kSubRows);
            const uint32_t my_off = (is_a ? 0u : kPairABytes) + j * kSubBytes;
            for (uint32_t kb = 0; kb < nkb; ++kb, ++it) {
                const uint32_t s = it % kPairStages, ph = (it / kPairStages) & 1u;
                if (!__all_sync(0xFFFFFFFFu, mbar_wait_cl(smem_u32(&sh.empty[s]), ph ^ 1u, abort_flag, status))) { ok = false; break; }
                if (rank == 0 && lane == 0) mbar_arrive_expect_tx(smem_u32(&sh.full[s]), tx_both);
                __syncwarp();
                const int32_t k = (int32_t)(d.k0 + kb * kBlockK);
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
        if (*abort_flag && lane == 0) {
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
                if (!mbar_wait_cl(smem_u32(&sh.sched_full[q]), par, abort_flag, status)) break;
                const TileDesc d = sh.slot[q];
                mbar_arrive(smem_u32(&sh.sched_empty[q]));
                if (d.flags & TILE_END) break;
                const uint32_t a_mn = (d.flags & TILE_A_MN) ? 1u : 0u, b_mn = (d.flags & TILE_B_MN) ? 1u : 0u;
                const uint32_t idesc = instr_desc_bf16(2 * kBlockM, d.n_mma, a_mn, b_mn);
                const uint32_t a_lbo = a_mn ? kSubBytes : 16u, a_step = a_mn ? 2048u : 32u;
                const uint32_t b_lbo = b_mn ? kSubBytes : 16u, b_step = b_mn ? 2048u : 32u;
                const uint32_t acc = tile_no & 1u, aph = (tile_no >> 1) & 1u;
                if (!mbar_wait_cl(smem_u32(&sh.acc_empty[acc]), aph ^ 1u, abort_flag, status)) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + acc * kAccCols;
                const uint32_t nkb = (d.k1 - d.k0 + kBlockK - 1) / kBlockK;
                for (uint32_t kb = 0; kb < nkb; ++kb, ++it) {
                    const uint32_t s = it % kPairStages, ph = (it / kPairStages) & 1u;
                    if (!mbar_wait_cl(smem_u32(&sh.full[s]), ph, abort_flag, status)) { ok = false; break; }
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
                if (global_timer_ns() - t0 > kWaitLimitNs) { atomicOr(status, STATUS_TIMEOUT); break; }
        }
    } else if (warp >= kEpiWarp0) {
        // ---- epilogue (both CTAs): own 128 rows of the accumulator -> packed partial block ---------------------
        const uint32_t group = (warp - kEpiWarp0) / kEpiWarpsPerGroup;
        const uint32_t quad = warp & 3u;
        float* stage_tile = reinterpret_cast<float*>(dyn_smem + (stage_base - smem_u32(dyn_smem)) + kPairStages * kPairStageBytes) +
                            (warp - kEpiWarp0) * kEpiStageFloats;
        const uint32_t sched_empty_leader0 = mapa_shared(smem_u32(&sh.sched_empty[0]), 0u);
        const uint32_t acc_empty_leader = mapa_shared(smem_u32(&sh.acc_empty[group]), 0u);
        uint32_t used = 0, tile_no = 0;
        for (uint32_t i = 0;; ++i) {
            const uint32_t q = i % kSchedSlots, par = (i / kSchedSlots) & 1u;
            bool ok = mbar_wait_cl(smem_u32(&sh.sched_full[q]), par, abort_flag, status);
            if (!__all_sync(0xFFFFFFFFu, ok)) break;
            const uint32_t flags = sh.slot[q].flags, task = sh.slot[q].task, n_mma = sh.slot[q].n_mma;
            const uint32_t tile_rows = sh.slot[q].rows, cols = sh.slot[q].cols, gemm = sh.slot[q].gemm;
            // a block of a one-slice GEMM is final: it may go straight to its place in C
            const bool direct = flags & TILE_DIRECT;
            const uint32_t ld = direct ? sh.slot[q].ldc : sh.slot[q].ld;
            const uint64_t out_off = (direct ? sh.slot[q].c_off : sh.slot[q].out_off) + (uint64_t)rank * kBlockM * ld;
            __syncwarp();
            if (lane == 0) mbar_arrive_cluster(sched_empty_leader0 + q * 8u);
            if (flags & TILE_END) break;
            const bool mine = (tile_no & 1u) == group;       // tiles alternate between the two accumulator slots
            ++tile_no;
            if (!mine) continue;
            const uint32_t rows = rows_of_rank(tile_rows, rank);
            ok = mbar_wait_cl(smem_u32(&sh.acc_full[group]), used & 1u, abort_flag, status);
            if (!__all_sync(0xFFFFFFFFu, ok)) break;
            ++used;
            tc_fence_after();
            const uint32_t taddr = tmem_base + group * kAccCols + ((quad * 32u) << 16);
            float* out_blk = (direct ? c_ptrs[gemm] : partials) + out_off + (uint64_t)(quad * 32u) * ld;
            const uint32_t rows_here = rows > quad * 32u ? min(32u, rows - quad * 32u) : 0u;
            const bool vec_ok = ((ld & 3u) == 0u) && ((out_off & 3ull) == 0ull);
            const uint32_t nchunk = (n_mma + 31u) / 32u;
            for (uint32_t c = 0; c < nchunk; ++c) {
                uint32_t v[32];
                tmem_ld_32x32(taddr + c * 32u, v);
                tmem_ld_wait();
                if (c + 1 == nchunk) {                       // slot fully read: hand it back to the leader
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive_cluster(acc_empty_leader);
                }
                if (rows_here == 0) continue;                // warp-uniform
#pragma unroll
                for (int x = 0; x < 32; ++x) stage_tile[lane * 33 + x] = __uint_as_float(v[x]);
                __syncwarp();
                const uint32_t c0 = c * 32u;
                if (vec_ok && c0 + 32u <= cols) {
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
            if (rows) {
                __threadfence();
                __syncwarp();
                if (lane == 0) atomicAdd(&done[task], 1u);   // one count per warp and 128-row half-tile
            }
        }
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

cudaError_t launch_exec_pair(uint32_t clusters, const TileDesc* tiles, uint32_t tile_end, unsigned int* ticket,
                             const CUtensorMap* maps, float* partials, float* const* c_ptrs, uint32_t* done,
                             unsigned int* status, cudaStream_t st) {
    exec_pair_kernel<<<2 * clusters, kExecThreads, kPairDynSmem, st>>>(tiles, tile_end, ticket, maps, partials, c_ptrs, done, status);
    return cudaGetLastError();
}

}  // namespace cleave
