// C ABI of the library (see include/cleave.h): argument checks, the plan's device mirrors, TMA
// tensor maps, and the launches.  All compute happens in the kernels of kernels.cu.
#include <cuda.h>
#include <cuda_runtime.h>

#include <algorithm>
#include <cstring>
#include <new>
#include <vector>

#include "cleave.h"
#include "kernels.cuh"
#include "plan_internal.hpp"

namespace cleave {

struct DeviceState {
    int device = -1;
    int sm_count = 0;
    cleave_task_t* tasks = nullptr;   uint32_t tasks_cap = 0, tasks_n = 0;
    TileDesc* tiles = nullptr;        uint32_t tiles_cap = 0, tiles_n = 0;
    uint8_t* dropped = nullptr;
    uint32_t* done = nullptr;
    uint32_t* ntiles = nullptr;
    uint32_t* failed_ids = nullptr;
    unsigned int* words = nullptr;    // [0] ticket, [1] status, [2] failed count
    CUtensorMap* maps = nullptr;
    CUtensorMap* c_maps = nullptr;    // per GEMM two maps of C, 32 x 32 boxes (the exec kernel's bulk stores): as fp32, as bf16
    AsmItem* asm_items = nullptr;
    AsmRef* asm_refs = nullptr;
    void** c_ptrs = nullptr;
    uint32_t* ldcs = nullptr;
    uint32_t* fin_ref0 = nullptr;     // cells of the in-kernel K-slice sum
    FinRef* fin_refs = nullptr;
    unsigned int* fin_count = nullptr;    // per cell and 32-row strip: blocks arrived in this execution
    unsigned int* level_left = nullptr;   // per DAG level: strips still to finish in this launch
    std::vector<const void*> last_a, last_b;
    std::vector<void*> last_c;
    bool drops_dirty = true;
    bool tiles_dirty = false;         // the host tile list was re-ordered: send it again in full
    // block verification (created on first cleave_verify)
    cleave_gemm_t* gemm_table = nullptr;
    uint32_t* ksplit_table = nullptr;
    const void** ab_ptrs = nullptr;
    float4* verify_out = nullptr;     uint32_t verify_cap = 0, verify_n = 0;
    cudaEvent_t ev[4] = {nullptr, nullptr, nullptr, nullptr};   // exec begin/end, assemble begin/end
    bool ev_exec = false, ev_asm = false;
};

namespace {

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult qres;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &qres) == cudaSuccess &&
            qres == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
    }
    return fn;
}

// 2-D bf16 tensor map over a row-major [rows x cols] matrix with row stride ld: boxes of
// 64 (contiguous) x box_rows elements, 128-byte swizzle, zero fill outside the matrix.
int encode_map(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return CLEAVE_E_CUDA;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld * 2};
    cuuint32_t box[2] = {kBlockK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : CLEAVE_E_CUDA;
}

// The same matrix, whose cols are a multiple of 64, seen as [cols / 64][rows][64]: one box of
// 64 x 64 x 2 brings two neighbouring 64-column groups (each a 64-row x 128-byte block in shared
// memory, the second 8 KB after the first) with one TMA operation.
int encode_map_groups(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, uint64_t ld) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return CLEAVE_E_CUDA;
    cuuint64_t dims[3] = {kSubRows, rows, cols / kSubRows};
    cuuint64_t strides[2] = {ld * 2, kSubRows * 2};
    cuuint32_t box[3] = {kSubRows, kBlockK, 2};
    cuuint32_t estr[3] = {1, 1, 1};
    CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 3, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : CLEAVE_E_CUDA;
}

// Tensor map over a row-major [rows x cols] matrix C, fp32 or bf16: boxes of 32 x 32 elements (rows of 128
// bytes with the 128-byte swizzle, resp. 64 bytes with the 64-byte swizzle): what an epilogue warp of the exec
// kernel stores with one bulk operation.
int encode_c_map(CUtensorMap* out, const void* base, uint64_t rows, uint64_t cols, bool bf16) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return CLEAVE_E_CUDA;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * (bf16 ? 2u : 4u)};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(out, bf16 ? CU_TENSOR_MAP_DATA_TYPE_BFLOAT16 : CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base),
                    dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
                    bf16 ? CU_TENSOR_MAP_SWIZZLE_64B : CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS ? 0 : CLEAVE_E_CUDA;
}

template <typename T>
int dev_alloc(T** p, size_t n) {
    if (n == 0) n = 1;
    return cudaMalloc(reinterpret_cast<void**>(p), n * sizeof(T)) == cudaSuccess ? 0 : CLEAVE_E_NOMEM;
}

#define CU_TRY(x) do { if ((x) != cudaSuccess) { cudaGetLastError(); return CLEAVE_E_CUDA; } } while (0)
#define RC_TRY(x) do { int rc_ = (x); if (rc_) return rc_; } while (0)

// First use of a plan on a device: the mirrors that never grow.  The state is attached to the plan
// only when every step has succeeded.
int create_device_state(cleave_plan_s* p, cudaStream_t st, DeviceState* d) {
    int ndev = 0;
    if (cudaGetDeviceCount(&ndev) != cudaSuccess || ndev == 0) { cudaGetLastError(); return CLEAVE_E_CUDA; }
    CU_TRY(cudaGetDevice(&d->device));
    CU_TRY(cudaDeviceGetAttribute(&d->sm_count, cudaDevAttrMultiProcessorCount, d->device));
    int cc_major = 0;
    CU_TRY(cudaDeviceGetAttribute(&cc_major, cudaDevAttrComputeCapabilityMajor, d->device));
    if (cc_major != 10) return CLEAVE_E_UNSUPPORTED;
    CU_TRY(exec_pair_kernel_prepare());
    const size_t ng = p->gemms.size();
    RC_TRY(dev_alloc(&d->words, 4));
    CU_TRY(cudaMemsetAsync(d->words, 0, 4 * sizeof(unsigned int), st));
    RC_TRY(dev_alloc(&d->maps, kMapsPerGemm * ng));
    RC_TRY(dev_alloc(&d->c_maps, 2 * ng));
    RC_TRY(dev_alloc(&d->c_ptrs, ng));
    RC_TRY(dev_alloc(&d->ldcs, ng));
    std::vector<uint32_t> ldc;
    for (auto& g : p->gemms) ldc.push_back(g.N);
    CU_TRY(cudaMemcpyAsync(d->ldcs, ldc.data(), ldc.size() * 4, cudaMemcpyHostToDevice, st));
    RC_TRY(dev_alloc(&d->asm_items, p->asm_items.size()));
    RC_TRY(dev_alloc(&d->asm_refs, p->asm_refs.size()));
    CU_TRY(cudaMemcpyAsync(d->asm_items, p->asm_items.data(), p->asm_items.size() * sizeof(AsmItem), cudaMemcpyHostToDevice, st));
    CU_TRY(cudaMemcpyAsync(d->asm_refs, p->asm_refs.data(), p->asm_refs.size() * sizeof(AsmRef), cudaMemcpyHostToDevice, st));
    RC_TRY(dev_alloc(&d->fin_ref0, p->fin_ref0.size()));
    RC_TRY(dev_alloc(&d->fin_refs, p->fin_refs.size()));
    RC_TRY(dev_alloc(&d->fin_count, 4 * p->fin_ref0.size()));
    RC_TRY(dev_alloc(&d->level_left, p->n_levels));
    CU_TRY(cudaMemcpyAsync(d->fin_ref0, p->fin_ref0.data(), p->fin_ref0.size() * 4, cudaMemcpyHostToDevice, st));
    CU_TRY(cudaMemcpyAsync(d->fin_refs, p->fin_refs.data(), p->fin_refs.size() * sizeof(FinRef), cudaMemcpyHostToDevice, st));
    for (auto& e : d->ev) CU_TRY(cudaEventCreate(&e));
    return 0;
}

// Creates the mirrors on first use and brings the growing tables (tasks, tiles) up to date.
int sync_device_state(cleave_plan_s* p, cudaStream_t st) {
    if (!p->dev) {
        DeviceState* d = new (std::nothrow) DeviceState();
        if (!d) return CLEAVE_E_NOMEM;
        const int rc = create_device_state(p, st, d);
        if (rc) { cudaStreamSynchronize(st); device_state_free(d); return rc; }
        p->dev = d;
    }
    DeviceState* d = p->dev;
    const uint32_t nt = (uint32_t)p->tasks.size(), nl = (uint32_t)p->tiles.size();
    if (nt > d->tasks_cap) {
        // grow: the bookkeeping words of finished tasks must survive
        const uint32_t cap = std::max(nt, d->tasks_cap * 2);
        cleave_task_t* tasks; uint8_t* dropped; uint32_t *done, *ntiles, *failed;
        RC_TRY(dev_alloc(&tasks, cap)); RC_TRY(dev_alloc(&dropped, cap)); RC_TRY(dev_alloc(&done, cap));
        RC_TRY(dev_alloc(&ntiles, cap)); RC_TRY(dev_alloc(&failed, cap));
        CU_TRY(cudaMemsetAsync(done, 0, cap * 4, st));
        if (d->tasks_n) CU_TRY(cudaMemcpyAsync(done, d->done, d->tasks_n * 4, cudaMemcpyDeviceToDevice, st));
        CU_TRY(cudaStreamSynchronize(st));
        cudaFree(d->tasks); cudaFree(d->dropped); cudaFree(d->done); cudaFree(d->ntiles); cudaFree(d->failed_ids);
        d->tasks = tasks; d->dropped = dropped; d->done = done; d->ntiles = ntiles; d->failed_ids = failed;
        d->tasks_cap = cap;
        d->drops_dirty = true;
    }
    // task records are re-sent in full: reissue changes the flags of old tasks as well
    if (nt != d->tasks_n || d->drops_dirty) {
        CU_TRY(cudaMemcpyAsync(d->tasks, p->tasks.data(), nt * sizeof(cleave_task_t), cudaMemcpyHostToDevice, st));
        CU_TRY(cudaMemcpyAsync(d->ntiles, p->task_ntiles.data(), nt * 4, cudaMemcpyHostToDevice, st));
        CU_TRY(cudaMemcpyAsync(d->dropped, p->dropped.data(), nt, cudaMemcpyHostToDevice, st));
        d->tasks_n = nt;
        d->drops_dirty = false;
    }
    if (nl > d->tiles_cap) {
        const uint32_t cap = std::max(nl, d->tiles_cap * 2);
        TileDesc* tiles;
        RC_TRY(dev_alloc(&tiles, cap));
        if (d->tiles_n) CU_TRY(cudaMemcpyAsync(tiles, d->tiles, d->tiles_n * sizeof(TileDesc), cudaMemcpyDeviceToDevice, st));
        CU_TRY(cudaStreamSynchronize(st));
        cudaFree(d->tiles);
        d->tiles = tiles; d->tiles_cap = cap;
    }
    if (d->tiles_dirty) { d->tiles_n = 0; d->tiles_dirty = false; }
    if (nl > d->tiles_n) {
        CU_TRY(cudaMemcpyAsync(d->tiles + d->tiles_n, p->tiles.data() + d->tiles_n, (nl - d->tiles_n) * sizeof(TileDesc),
                               cudaMemcpyHostToDevice, st));
        d->tiles_n = nl;
    }
    return 0;
}

int update_maps(cleave_plan_s* p, const void* const* A, const void* const* B, cudaStream_t st) {
    DeviceState* d = p->dev;
    const size_t n = p->gemms.size();
    bool same = d->last_a.size() == n;
    for (size_t i = 0; same && i < n; ++i) same = (d->last_a[i] == A[i] && d->last_b[i] == B[i]);
    if (same) return 0;
    std::vector<CUtensorMap> host(kMapsPerGemm * n);
    for (size_t i = 0; i < n; ++i) {
        const cleave_gemm_t& g = p->gemms[i];
        if (!A[i] || !B[i] || ((uintptr_t)A[i] & 15) || ((uintptr_t)B[i] & 15)) return CLEAVE_E_INVAL;
        // stored shapes: A is [M x K] or, transposed, [K x M]; B is [K x N] or, transposed, [N x K]
        CUtensorMap* m = &host[kMapsPerGemm * i];            // A, B with 64 x 64 boxes; A, B with double-size boxes
        RC_TRY(g.transA ? encode_map(m + 0, A[i], g.K, g.M, g.lda, kSubRows) : encode_map(m + 0, A[i], g.M, g.K, g.lda, kSubRows));
        RC_TRY(g.transB ? encode_map(m + 1, B[i], g.N, g.K, g.ldb, kSubRows) : encode_map(m + 1, B[i], g.K, g.N, g.ldb, kSubRows));
        // double-size boxes: 128 rows of a K-contiguous operand, two 64-wide groups of an M/N-contiguous one
        // (only when M / N is a multiple of 64; otherwise the slot repeats the small map and is never used)
        if (!g.transA) RC_TRY(encode_map(m + 2, A[i], g.M, g.K, g.lda, 2 * kSubRows));
        else if (g.M % kSubRows == 0) RC_TRY(encode_map_groups(m + 2, A[i], g.K, g.M, g.lda));
        else m[2] = m[0];
        if (g.transB) RC_TRY(encode_map(m + 3, B[i], g.N, g.K, g.ldb, 2 * kSubRows));
        else if (g.N % kSubRows == 0) RC_TRY(encode_map_groups(m + 3, B[i], g.K, g.N, g.ldb));
        else m[3] = m[1];
    }
    // pageable source: the copy is staged before the call returns, so `host` may go out of scope
    CU_TRY(cudaMemcpyAsync(d->maps, host.data(), host.size() * sizeof(CUtensorMap), cudaMemcpyHostToDevice, st));
    d->last_a.assign(A, A + n);
    d->last_b.assign(B, B + n);
    return 0;
}

int check_exec_args(cleave_plan_s* p, const void* const* A, const void* const* B, float* partials) {
    if (!p || !A || !B || !partials) return CLEAVE_E_INVAL;
    if ((uintptr_t)partials & 127) return CLEAVE_E_INVAL;
    // plans off the tensor-core kernel's alignment rules run on the plain kernel, one DAG level only
    if (p->exec_unsupported && p->n_levels > 1) return CLEAVE_E_UNSUPPORTED;
    for (const auto& g : p->gemms) {
        const uint32_t need_a = g.transA ? g.M : g.K, need_b = g.transB ? g.K : g.N;
        if (g.lda < need_a || g.ldb < need_b) return CLEAVE_E_INVAL;
    }
    return 0;
}

int upload_c_ptrs(cleave_plan_s* p, void* const* C, cudaStream_t st) {
    DeviceState* d = p->dev;
    const size_t n = p->gemms.size();
    for (size_t i = 0; i < n; ++i) if (!C[i] || ((uintptr_t)C[i] & 15)) return CLEAVE_E_INVAL;
    if (d->last_c.size() != n || !std::equal(C, C + n, d->last_c.begin())) {
        d->last_c.assign(C, C + n);
        CU_TRY(cudaMemcpyAsync(d->c_ptrs, d->last_c.data(), n * sizeof(void*), cudaMemcpyHostToDevice, st));
        // views of the outputs for bulk stores: as fp32 (used when C holds fp32 and N % 4 == 0) and as bf16 (when C
        // holds bf16 and N % 8 == 0); the buffer is whichever the caller made it, the other view is never used
        std::vector<CUtensorMap> host(2 * n);
        for (size_t i = 0; i < n; ++i) {
            const cleave_gemm_t& g = p->gemms[i];
            if (g.N % 4 == 0) RC_TRY(encode_c_map(&host[2 * i], C[i], g.M, g.N, false));
            else std::memset(&host[2 * i], 0, sizeof(CUtensorMap));
            if (g.N % 8 == 0) RC_TRY(encode_c_map(&host[2 * i + 1], C[i], g.M, g.N, true));
            else std::memset(&host[2 * i + 1], 0, sizeof(CUtensorMap));
        }
        CU_TRY(cudaMemcpyAsync(d->c_maps, host.data(), 2 * n * sizeof(CUtensorMap), cudaMemcpyHostToDevice, st));
    }
    return 0;
}

// One launch of the arming kernel and the exec kernel over the work-list range [tile_begin, tile_end).
// `fresh`: a whole execution (the arrival counters of the in-kernel K-slice sums start at zero).
int run_tiles(cleave_plan_s* p, uint32_t tile_begin, uint32_t tile_end, bool fresh, uint32_t level_begin, uint32_t level_end,
              float* partials, cudaStream_t st) {
    DeviceState* d = p->dev;
    CU_TRY(cudaMemsetAsync(d->level_left, 0, p->n_levels * sizeof(unsigned int), st));
    if (fresh && !p->fin_ref0.empty()) CU_TRY(cudaMemsetAsync(d->fin_count, 0, 4 * p->fin_ref0.size() * sizeof(unsigned int), st));
    ArmParams a;
    a.tiles = d->tiles; a.tile_begin = tile_begin; a.tile_end = tile_end;
    a.tasks = d->tasks; a.dropped = d->dropped; a.done = d->done;
    a.ticket = d->words + 0; a.status = d->words + 1; a.level_left = d->level_left;
    a.mode = p->mode; a.level_begin = level_begin; a.level_end = level_end; a.arena_elems = p->arena_elems;
    CU_TRY(launch_arm_queue(a, fresh ? 1 : 0, st));
    if (tile_end > tile_begin) {
        // one cluster of two CTAs per pair of SMs, never more clusters than tiles
        const uint32_t clusters = std::max<uint32_t>(1u, std::min<uint32_t>((uint32_t)d->sm_count / 2, tile_end - tile_begin));
        ExecParams e;
        e.tiles = d->tiles; e.tile_end = tile_end; e.ticket = d->words + 0; e.maps = d->maps; e.c_maps = d->c_maps; e.partials = partials;
        e.c_ptrs = d->c_ptrs; e.done = d->done; e.status = d->words + 1;
        e.fin_ref0 = d->fin_ref0; e.fin_refs = d->fin_refs; e.fin_count = d->fin_count; e.level_left = d->level_left;
        e.mode = p->mode; e.wait_limit_ns = p->wait_limit_ns;
        CU_TRY(cudaEventRecord(d->ev[0], st));
        CU_TRY(launch_exec_pair(clusters, e, st));
        CU_TRY(cudaEventRecord(d->ev[1], st));
        d->ev_exec = true;
    }
    return 0;
}

// Device copies of the GEMM records and of the operand pointers (block verification and the plain exec kernel).
int upload_gemm_tables(cleave_plan_s* p, const void* const* A, const void* const* B, cudaStream_t st) {
    DeviceState* d = p->dev;
    const size_t n = p->gemms.size();
    if (!d->gemm_table) {
        RC_TRY(dev_alloc(&d->gemm_table, n)); RC_TRY(dev_alloc(&d->ksplit_table, n)); RC_TRY(dev_alloc(&d->ab_ptrs, 2 * n));
        CU_TRY(cudaMemcpyAsync(d->gemm_table, p->gemms.data(), n * sizeof(cleave_gemm_t), cudaMemcpyHostToDevice, st));
        CU_TRY(cudaMemcpyAsync(d->ksplit_table, p->ksplit.data(), n * sizeof(uint32_t), cudaMemcpyHostToDevice, st));
    }
    std::vector<const void*> ab(2 * n);
    for (size_t i = 0; i < n; ++i) {
        if (!A[i] || !B[i] || ((uintptr_t)A[i] & 15) || ((uintptr_t)B[i] & 15)) return CLEAVE_E_INVAL;
        ab[2 * i] = A[i]; ab[2 * i + 1] = B[i];
    }
    CU_TRY(cudaMemcpyAsync(d->ab_ptrs, ab.data(), ab.size() * sizeof(void*), cudaMemcpyHostToDevice, st));
    return 0;
}

// The plain kernel over tasks [task_begin, end): every block goes to the arena (cleave_assemble finishes C).
int run_tasks_plain(cleave_plan_s* p, uint32_t task_begin, bool fresh, const void* const* A, const void* const* B,
                    float* partials, cudaStream_t st) {
    DeviceState* d = p->dev;
    RC_TRY(upload_gemm_tables(p, A, B, st));
    if (fresh) {
        CU_TRY(cudaMemsetAsync(d->words + 1, 0, sizeof(unsigned int), st));          // forget earlier verdicts
        CU_TRY(cudaMemsetAsync(d->done, 0, d->tasks_n * sizeof(uint32_t), st));
    }
    CU_TRY(cudaEventRecord(d->ev[0], st));
    CU_TRY(launch_exec_simple(d->tasks, task_begin, d->tasks_n, d->gemm_table, d->ab_ptrs, d->dropped, d->ntiles, partials,
                              p->arena_elems, d->done, d->words + 1, st));
    CU_TRY(cudaEventRecord(d->ev[1], st));
    d->ev_exec = true;
    return 0;
}

int status_to_code(unsigned int s) {
    if (s & STATUS_TIMEOUT) return CLEAVE_E_TIMEOUT;
    if (s & STATUS_BOUNDS) return CLEAVE_E_BOUNDS;
    if (s & STATUS_INCOMPLETE) return CLEAVE_E_INCOMPLETE;
    return 0;
}

}  // namespace

void device_state_free(DeviceState* d) {
    if (!d) return;
    cudaFree(d->tasks); cudaFree(d->tiles); cudaFree(d->dropped); cudaFree(d->done); cudaFree(d->ntiles);
    cudaFree(d->failed_ids); cudaFree(d->words); cudaFree(d->maps); cudaFree(d->c_maps); cudaFree(d->asm_items); cudaFree(d->asm_refs);
    cudaFree(d->c_ptrs); cudaFree(d->ldcs); cudaFree(d->fin_ref0); cudaFree(d->fin_refs); cudaFree(d->fin_count);
    cudaFree(d->level_left); cudaFree(d->gemm_table); cudaFree(d->ksplit_table); cudaFree(d->ab_ptrs);
    cudaFree(d->verify_out);
    for (auto& e : d->ev) if (e) cudaEventDestroy(e);
    cudaGetLastError();
    delete d;
}

}  // namespace cleave

// Checks cleave_assemble_static shares with cleave_assemble (the plan's device state is private to this file).
int cleave::static_assemble_check(const cleave_plan_s* p, float* const* C) {
    if (!p->dev) return 0;
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess) { cudaGetLastError(); return CLEAVE_E_CUDA; }
    if (dev != p->dev->device) return CLEAVE_E_INVAL;          // the plan's blocks live on another device
    const size_t n = p->gemms.size();
    void* const* Cv = reinterpret_cast<void* const*>(C);
    if ((p->fused || p->finished) && (p->dev->last_c.size() != n || !std::equal(Cv, Cv + n, p->dev->last_c.begin())))
        return CLEAVE_E_INVAL;                                   // part of the result sits in the C the execution was given
    return 0;
}

using namespace cleave;

extern "C" {

void cleave_plan_opts_default(cleave_plan_opts_t* o) {
    if (!o) return;
    o->gran_m = o->gran_n = o->gran_k = 128;
    o->kslice_max = 4096;
    o->ksplit = 0;
    o->ksplit_cap = 8;
    o->reissue_fanout = 4;
    o->b_in = 2;
    o->b_out = 4;
    o->tail_alpha_milli = 0;
    o->tail_beta_ppm = 50000;
}

static int new_plan(const cleave_gemm_t* g, uint32_t n_gemms, const cleave_plan_opts_t* o, cleave_plan_s** out) {
    if (!g || !n_gemms || !out) return CLEAVE_E_INVAL;
    *out = nullptr;
    cleave_plan_s* p = new (std::nothrow) cleave_plan_s();
    if (!p) return CLEAVE_E_NOMEM;
    p->gemms.assign(g, g + n_gemms);
    if (o) p->opts = *o; else cleave_plan_opts_default(&p->opts);
    *out = p;
    return 0;
}

int cleave_plan(const cleave_gemm_t* g, uint32_t n_gemms, const cleave_device_t* d, uint32_t n_dev,
                const cleave_plan_opts_t* o, cleave_plan_t** out) {
    cleave_plan_s* p = nullptr;
    int rc = new_plan(g, n_gemms, o, &p);
    if (rc) return rc;
    try {
        if (d && n_dev) p->devices.assign(d, d + n_dev);
        rc = plan_build(*p);
    } catch (const std::bad_alloc&) { rc = CLEAVE_E_NOMEM; }
    if (rc) { delete p; return rc; }
    *out = p;
    return 0;
}

int cleave_plan_uniform(const cleave_gemm_t* g, uint32_t n_gemms, uint32_t grid_m, uint32_t grid_n, uint32_t ksplit,
                        const cleave_plan_opts_t* o, cleave_plan_t** out) {
    cleave_plan_s* p = nullptr;
    int rc = new_plan(g, n_gemms, o, &p);
    if (rc) return rc;
    try { rc = plan_build_uniform(*p, grid_m, grid_n, ksplit); } catch (const std::bad_alloc&) { rc = CLEAVE_E_NOMEM; }
    if (rc) { delete p; return rc; }
    *out = p;
    return 0;
}

uint32_t cleave_plan_num_tasks(const cleave_plan_t* p) { return p ? (uint32_t)p->tasks.size() : 0; }
uint32_t cleave_plan_num_original(const cleave_plan_t* p) { return p ? p->n_original : 0; }
const cleave_task_t* cleave_plan_tasks(const cleave_plan_t* p) { return p ? p->tasks.data() : nullptr; }
uint64_t cleave_plan_arena_elems(const cleave_plan_t* p) { return p ? p->arena_elems : 0; }
uint32_t cleave_plan_ksplit(const cleave_plan_t* p, uint32_t gemm) { return (p && gemm < p->ksplit.size()) ? p->ksplit[gemm] : 0; }
uint64_t cleave_plan_makespan_ns(const cleave_plan_t* p, uint32_t gemm) { return (p && gemm < p->makespan.size()) ? p->makespan[gemm] : 0; }
uint64_t cleave_plan_tstar_ns(const cleave_plan_t* p, uint32_t gemm) { return (p && gemm < p->tstar.size()) ? p->tstar[gemm] : 0; }
uint32_t cleave_plan_num_tiles(const cleave_plan_t* p) { return p ? (uint32_t)p->tiles.size() : 0; }
uint32_t cleave_plan_finishable(const cleave_plan_t* p, uint32_t gemm) { return (p && gemm < p->gemm_finishable.size()) ? p->gemm_finishable[gemm] : 0; }
uint32_t cleave_plan_num_levels(const cleave_plan_t* p) { return p ? p->n_levels : 0; }
uint64_t cleave_plan_level_makespan_ns(const cleave_plan_t* p, uint32_t level) {
    uint64_t worst = 0;
    if (p) for (size_t g = 0; g < p->gemms.size(); ++g) if (p->gemms[g].level == level) worst = std::max(worst, p->makespan[g]);
    return worst;
}
uint64_t cleave_plan_step_makespan_ns(const cleave_plan_t* p) {
    uint64_t sum = 0;
    if (p) for (uint32_t l = 0; l < p->n_levels; ++l) sum += cleave_plan_level_makespan_ns(p, l);
    return sum;
}

uint32_t cleave_plan_num_launches(const cleave_plan_t* p) {
    if (!p) return 0;
    uint32_t n = 5;          // clear + arm + exec, clear verdict + bookkeeping check, then the assembly kernels
    for (const auto& grp : p->asm_groups) if (!((p->fused && grp.single) || (p->finished && grp.finishable))) ++n;
    return n;
}
uint32_t cleave_task_num_tiles(const cleave_plan_t* p, uint32_t task) { return (p && task < p->task_ntiles.size()) ? p->task_ntiles[task] : 0; }

int cleave_set_drops(cleave_plan_t* p, const uint32_t* ids, uint32_t n) {
    if (!p || (n && !ids)) return CLEAVE_E_INVAL;
    for (uint32_t i = 0; i < n; ++i) if (ids[i] >= p->tasks.size()) return CLEAVE_E_RANGE;
    std::fill(p->dropped.begin(), p->dropped.end(), 0);
    for (uint32_t i = 0; i < n; ++i) p->dropped[ids[i]] = 1;
    if (p->dev) p->dev->drops_dirty = true;
    return 0;
}

int cleave_exec_opts(cleave_plan_t* p, const void* const* A, const void* const* B, float* partials, void* const* C,
                     uint32_t flags, uint32_t level_begin, uint32_t level_end, void* stream) {
    int rc = check_exec_args(p, A, B, partials);
    if (rc) return rc;
    if (flags & ~(uint32_t)(CLEAVE_EXEC_DIRECT | CLEAVE_EXEC_FINISH | CLEAVE_EXEC_BF16 | CLEAVE_EXEC_CONSUME)) return CLEAVE_E_INVAL;
    if ((flags & CLEAVE_EXEC_CONSUME) && !(flags & CLEAVE_EXEC_FINISH)) return CLEAVE_E_INVAL;
    if ((flags & (CLEAVE_EXEC_DIRECT | CLEAVE_EXEC_FINISH)) && !C) return CLEAVE_E_INVAL;
    if (level_begin > level_end) return CLEAVE_E_INVAL;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    if (p->exec_unsupported) {
        // every block to the arena with the plain kernel; C is written by the cleave_assemble that follows
        if (level_begin != 0 || level_end < p->n_levels) return CLEAVE_E_UNSUPPORTED;
        try { RC_TRY(sync_device_state(p, st)); } catch (const std::bad_alloc&) { return CLEAVE_E_NOMEM; }
        p->mode = (flags & CLEAVE_EXEC_BF16) ? MODE_BF16 : 0u;
        p->fused = p->finished = p->consumed = false;
        p->out_bf16 = (p->mode & MODE_BF16) != 0;
        try { return run_tasks_plain(p, 0, true, A, B, partials, st); } catch (const std::bad_alloc&) { return CLEAVE_E_NOMEM; }
    }
    try {
        RC_TRY(sync_device_state(p, st));
        RC_TRY(update_maps(p, A, B, st));
        if (C) RC_TRY(upload_c_ptrs(p, C, st));
    } catch (const std::bad_alloc&) { return CLEAVE_E_NOMEM; }
    p->mode = ((flags & CLEAVE_EXEC_DIRECT) ? MODE_DIRECT : 0u) | ((flags & CLEAVE_EXEC_FINISH) ? MODE_FINISH : 0u) |
              ((flags & CLEAVE_EXEC_BF16) ? MODE_BF16 : 0u);
    p->fused = (p->mode & MODE_DIRECT) != 0;
    p->out_bf16 = (p->mode & MODE_BF16) != 0;
    // the exec kernel sums every cell of the finishable GEMMs itself unless a block is going to be missing
    bool whole = level_begin == 0 && level_end >= p->n_levels;
    for (size_t i = 0; whole && i < p->tasks.size(); ++i)
        if (p->dropped[i] || (p->tasks[i].flags & CLEAVE_TASK_SUPERSEDED)) whole = false;   // replacement pieces join no cell
    p->finished = (p->mode & MODE_FINISH) && whole;
    // blocks are only used up on arrival when every cell is going to be summed in this launch: with a task
    // missing, cleave_assemble needs them all
    p->consumed = p->finished && (flags & CLEAVE_EXEC_CONSUME);
    if (p->consumed) p->mode |= MODE_CONSUME;
    return run_tiles(p, 0, (uint32_t)p->tiles.size(), true, level_begin, level_end, partials, st);
}

int cleave_exec(cleave_plan_t* p, const void* const* A, const void* const* B, float* partials, void* stream) {
    return cleave_exec_opts(p, A, B, partials, nullptr, 0u, 0u, 0xFFFFFFFFu, stream);
}

int cleave_exec_fused(cleave_plan_t* p, const void* const* A, const void* const* B, float* partials, float* const* C,
                      void* stream) {
    if (!C) return CLEAVE_E_INVAL;
    return cleave_exec_opts(p, A, B, partials, reinterpret_cast<void* const*>(C), CLEAVE_EXEC_DIRECT | CLEAVE_EXEC_FINISH, 0u,
                            0xFFFFFFFFu, stream);
}

int cleave_set_wait_limit_ns(cleave_plan_t* p, uint64_t ns) {
    if (!p) return CLEAVE_E_INVAL;
    p->wait_limit_ns = ns;
    return 0;
}

int cleave_assemble(cleave_plan_t* p, const float* partials, float* const* C, void* stream) {
    if (!p || !partials || !C) return CLEAVE_E_INVAL;
    for (uint32_t s : p->ksplit) if (s > 32) return CLEAVE_E_UNSUPPORTED;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    try { RC_TRY(sync_device_state(p, st)); } catch (const std::bad_alloc&) { return CLEAVE_E_NOMEM; }
    DeviceState* d = p->dev;
    const size_t n = p->gemms.size();
    void* const* Cv = reinterpret_cast<void* const*>(C);
    // after a fused execution part of the result already sits in the C it was given: it must be the same C
    if ((p->fused || p->finished) && (d->last_c.size() != n || !std::equal(Cv, Cv + n, d->last_c.begin()))) return CLEAVE_E_INVAL;
    try { RC_TRY(upload_c_ptrs(p, Cv, st)); } catch (const std::bad_alloc&) { return CLEAVE_E_NOMEM; }
    CU_TRY(launch_check_done(d->tasks, d->done, d->ntiles, d->tasks_n, d->words + 1, st));
    CU_TRY(cudaEventRecord(d->ev[2], st));
    for (const auto& grp : p->asm_groups) {
        // blocks of one-slice GEMMs were written to C, cells of finishable GEMMs summed, by the exec kernel
        if ((p->fused && grp.single) || (p->finished && grp.finishable)) continue;
        CU_TRY(launch_assemble(d->asm_items, d->asm_refs, grp.item0, grp.n_items, grp.sp, partials, d->c_ptrs, d->ldcs,
                               p->out_bf16 ? 1 : 0, st));
    }
    CU_TRY(cudaEventRecord(d->ev[3], st));
    d->ev_asm = true;
    return 0;
}

int cleave_reissue(cleave_plan_t* p, const uint32_t* failed, uint32_t n, const void* const* A, const void* const* B,
                   float* partials, void* stream) {
    int rc = check_exec_args(p, A, B, partials);
    if (rc) return rc;
    if (n && !failed) return CLEAVE_E_INVAL;
    if (p->consumed) return CLEAVE_E_INVAL;            // the arena lacks the blocks that were used up: execute again first
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    try {
        RC_TRY(sync_device_state(p, st));
        std::vector<uint32_t> ids;
        if (n == 0) {
            // bookkeeping decides: every live task with unfinished tiles
            DeviceState* d = p->dev;
            CU_TRY(cudaMemsetAsync(d->words + 2, 0, sizeof(unsigned int), st));
            CU_TRY(launch_collect_failed(d->tasks, d->done, d->ntiles, d->tasks_n, d->failed_ids, d->words + 2, st));
            unsigned int cnt = 0;
            CU_TRY(cudaMemcpyAsync(&cnt, d->words + 2, sizeof cnt, cudaMemcpyDeviceToHost, st));
            CU_TRY(cudaStreamSynchronize(st));
            ids.resize(cnt);
            if (cnt) CU_TRY(cudaMemcpy(ids.data(), d->failed_ids, cnt * 4, cudaMemcpyDeviceToHost));
            failed = ids.data();
            n = cnt;
            if (n == 0) return 0;
        }
        const uint32_t tiles_before = (uint32_t)p->tiles.size();
        uint32_t first_new = 0;
        const bool was_plain = p->exec_unsupported != 0;
        RC_TRY(plan_reissue(*p, failed, n, &first_new));
        if (p->exec_unsupported) {
            // (a plan that ran on the tensor-core kernel and only now gets a piece off its rules is refused: part
            // of its result may sit in C already)
            if (p->n_levels > 1 || !was_plain) return CLEAVE_E_UNSUPPORTED;
            p->fused = p->finished = false;
            RC_TRY(sync_device_state(p, st));
            return run_tasks_plain(p, first_new, false, A, B, partials, st);
        }
        RC_TRY(sync_device_state(p, st));
        RC_TRY(update_maps(p, A, B, st));
        p->finished = false;                           // cells that lost a block are summed by cleave_assemble
        rc = run_tiles(p, tiles_before, (uint32_t)p->tiles.size(), false, 0u, 0xFFFFFFFFu, partials, st);
        if (p->n_levels > 1) {
            // the scheduler takes levels in list order: keep the whole list sorted by level for later executions
            std::stable_sort(p->tiles.begin(), p->tiles.end(), [](const TileDesc& x, const TileDesc& y) {
                return (x.level & 0xFFFFu) < (y.level & 0xFFFFu);
            });
            p->dev->tiles_dirty = true;
        }
        return rc;
    } catch (const std::bad_alloc&) { return CLEAVE_E_NOMEM; }
}

int cleave_replan(cleave_plan_t* p, const uint32_t* failed, uint32_t n, uint32_t* first_new) {
    if (!p || (n && !failed) || !first_new) return CLEAVE_E_INVAL;
    try { return plan_reissue(*p, failed, n, first_new); } catch (const std::bad_alloc&) { return CLEAVE_E_NOMEM; }
}

int cleave_verify(cleave_plan_t* p, const void* const* A, const void* const* B, const float* partials, uint64_t seed,
                  float tol, uint32_t* n_bad, void* stream) {
    if (!p || !A || !B || !partials || !n_bad || !(tol >= 0.f)) return CLEAVE_E_INVAL;
    for (const auto& g : p->gemms) if ((g.K % 4) || (g.lda % 8) || (g.ldb % 8)) return CLEAVE_E_UNSUPPORTED;
    if (p->fused && p->out_bf16) return CLEAVE_E_UNSUPPORTED;      // blocks written to C as bf16 are not checked
    if (p->consumed) return CLEAVE_E_UNSUPPORTED;                   // blocks used up on arrival are not in the arena
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    try { RC_TRY(sync_device_state(p, st)); } catch (const std::bad_alloc&) { return CLEAVE_E_NOMEM; }
    DeviceState* d = p->dev;
    const size_t n = p->gemms.size();
    RC_TRY(upload_gemm_tables(p, A, B, st));
    if (d->verify_cap < d->tasks_cap) {
        CU_TRY(cudaStreamSynchronize(st));
        cudaFree(d->verify_out);
        d->verify_out = nullptr;
        RC_TRY(dev_alloc(&d->verify_out, d->tasks_cap));
        d->verify_cap = d->tasks_cap;
    }
    uint32_t sign_bytes = 0;
    for (const auto& t : p->tasks) sign_bytes = std::max(sign_bytes, (t.m1 - t.m0) + (t.n1 - t.n0));
    sign_bytes = (sign_bytes + 15) / 16 * 16;
    if (sign_bytes > 200 * 1024) return CLEAVE_E_UNSUPPORTED;
    CU_TRY(cudaMemsetAsync(d->words + 3, 0, sizeof(unsigned int), st));
    CU_TRY(launch_verify(d->tasks, d->tasks_n, d->gemm_table, d->ksplit_table, d->ab_ptrs, partials, reinterpret_cast<float* const*>(d->c_ptrs), p->fused ? 1 : 0,
                         seed, tol, d->verify_out, d->words + 3, sign_bytes, st));
    d->verify_n = d->tasks_n;
    unsigned int bad = 0;
    CU_TRY(cudaMemcpyAsync(&bad, d->words + 3, sizeof bad, cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaStreamSynchronize(st));
    *n_bad = bad;
    return 0;
}

int cleave_verify_values(cleave_plan_t* p, float* out) {
    if (!p || !out || !p->dev || !p->dev->verify_out) return CLEAVE_E_INVAL;
    CU_TRY(cudaMemcpy(out, p->dev->verify_out, (size_t)p->dev->verify_n * sizeof(float4), cudaMemcpyDeviceToHost));
    return 0;
}

int cleave_status(cleave_plan_t* p, void* stream) {
    if (!p) return CLEAVE_E_INVAL;
    if (!p->dev) return 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    unsigned int s = 0;
    CU_TRY(cudaMemcpyAsync(&s, p->dev->words + 1, sizeof s, cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaStreamSynchronize(st));
    return status_to_code(s);
}

int cleave_done_counts(cleave_plan_t* p, uint32_t* done, void* stream) {
    if (!p || !done) return CLEAVE_E_INVAL;
    const size_t n = p->tasks.size();
    if (!p->dev) { std::fill(done, done + n, 0u); return 0; }
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    const size_t have = std::min<size_t>(n, p->dev->tasks_n);
    std::fill(done, done + n, 0u);
    CU_TRY(cudaMemcpyAsync(done, p->dev->done, have * 4, cudaMemcpyDeviceToHost, st));
    CU_TRY(cudaStreamSynchronize(st));
    for (size_t i = 0; i < have; ++i) done[i] /= kEpiWarpsPerGroup;   // the kernel counts once per epilogue warp
    return 0;
}

int cleave_last_kernel_ms(cleave_plan_t* p, float* exec_ms, float* assemble_ms) {
    if (!p || !p->dev) return CLEAVE_E_INVAL;
    DeviceState* d = p->dev;
    if (exec_ms) {
        *exec_ms = 0.f;
        if (d->ev_exec) { CU_TRY(cudaEventSynchronize(d->ev[1])); CU_TRY(cudaEventElapsedTime(exec_ms, d->ev[0], d->ev[1])); }
    }
    if (assemble_ms) {
        *assemble_ms = 0.f;
        if (d->ev_asm) { CU_TRY(cudaEventSynchronize(d->ev[3])); CU_TRY(cudaEventElapsedTime(assemble_ms, d->ev[2], d->ev[3])); }
    }
    return 0;
}

void cleave_destroy(cleave_plan_t* p) {
    if (!p) return;
    device_state_free(p->dev);
    delete p;
}

const char* cleave_strerror(int code) {
    switch (code) {
        case CLEAVE_OK: return "ok";
        case CLEAVE_E_INVAL: return "invalid argument";
        case CLEAVE_E_UNSUPPORTED: return "plan not supported by the kernels (alignment or slice count)";
        case CLEAVE_E_INFEASIBLE: return "no plan satisfies the memory constraint";
        case CLEAVE_E_NO_DEVICES: return "no (surviving) devices";
        case CLEAVE_E_RANGE: return "task id out of range";
        case CLEAVE_E_CUDA: return "CUDA call failed or no CUDA device";
        case CLEAVE_E_TIMEOUT: return "device-side wait expired";
        case CLEAVE_E_BOUNDS: return "device-side range check failed";
        case CLEAVE_E_INCOMPLETE: return "a task feeding the assembly never finished";
        case CLEAVE_E_NOMEM: return "out of memory";
        case CLEAVE_E_TOOBIG: return "plan tables exceed the fixed scratch array (CLEAVE_STATIC_SCRATCH_BYTES)";
        default: return "unknown error";
    }
}

}  // extern "C"
