// verify_kernel: checks every returned block P_t = A_t . B_t with two random +-1 vectors,
//   r^T P_t s  ==  (A_t^T r) . (B_t s),
// three matrix-vector products instead of a GEMM.  One CTA per task; everything is streamed once
// (HBM-bound: (alpha + beta) * kappa * 2 + alpha * beta * 4 bytes per task).
//
// The signs are the top bit of SplitMix64's output function applied to
// seed + (task << 33 | entry << 1 | vector) (vector 0 = r, 1 = s), generated once per task into
// shared memory.  Sums are fp32.
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "kernels.cuh"

namespace cleave {

namespace {

constexpr int kVerifyThreads = 256;
constexpr int kVerifyKChunk = 4 * kVerifyThreads;      // K-range handled per pass: four K per thread

__device__ __forceinline__ uint64_t splitmix64_mix(uint64_t x) {
    uint64_t z = x + 0x9E3779B97F4A7C15ull;
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
__device__ __forceinline__ float sign_of(uint64_t seed, uint32_t task, uint32_t entry, uint32_t which) {
    return (splitmix64_mix(seed + (((uint64_t)task << 33) | ((uint64_t)entry << 1) | which)) >> 63) ? -1.f : 1.f;
}
__device__ __forceinline__ float bf16_lo(uint32_t w) { return __uint_as_float(w << 16); }
__device__ __forceinline__ float bf16_hi(uint32_t w) { return __uint_as_float(w & 0xFFFF0000u); }
__device__ __forceinline__ float bf16_at(const uint16_t* p) { return __uint_as_float((uint32_t)(*p) << 16); }

__device__ __forceinline__ float warp_sum(float v) {
#pragma unroll
    for (int o = 16; o > 0; o >>= 1) v += __shfl_xor_sync(0xFFFFFFFFu, v, o);
    return v;
}

// out[c] = sum over rows of sgn[row] * M[row, c0 + c] for the 4 columns c0..c0+3 owned by this thread,
// M stored with `ld` elements per row, columns contiguous (8-byte loads, coalesced across threads).
__device__ __forceinline__ void column_sums4(const uint16_t* base, uint64_t ld, uint32_t nrows, const int8_t* sgn, float (&acc)[4]) {
    acc[0] = acc[1] = acc[2] = acc[3] = 0.f;
    uint32_t i = 0;
    for (; i + 4 <= nrows; i += 4) {
        uint2 w[4];
#pragma unroll
        for (int x = 0; x < 4; ++x) w[x] = __ldg(reinterpret_cast<const uint2*>(base + (uint64_t)(i + x) * ld));
#pragma unroll
        for (int x = 0; x < 4; ++x) {
            const float s = (float)sgn[i + x];
            acc[0] += s * bf16_lo(w[x].x); acc[1] += s * bf16_hi(w[x].x);
            acc[2] += s * bf16_lo(w[x].y); acc[3] += s * bf16_hi(w[x].y);
        }
    }
    for (; i < nrows; ++i) {
        const uint2 w = __ldg(reinterpret_cast<const uint2*>(base + (uint64_t)i * ld));
        const float s = (float)sgn[i];
        acc[0] += s * bf16_lo(w.x); acc[1] += s * bf16_hi(w.x); acc[2] += s * bf16_lo(w.y); acc[3] += s * bf16_hi(w.y);
    }
}

// sum over c of sgn[c] * row[c], c < n, by one warp (4-byte loads of two elements; `row` is 4-byte aligned)
__device__ __forceinline__ float row_dot(const uint16_t* row, uint32_t n, const int8_t* sgn, uint32_t lane) {
    float acc = 0.f;
    const uint32_t pairs = n >> 1;
    for (uint32_t c = lane; c < pairs; c += 32) {
        const uint32_t w = __ldg(reinterpret_cast<const uint32_t*>(row) + c);
        acc += (float)sgn[2 * c] * bf16_lo(w) + (float)sgn[2 * c + 1] * bf16_hi(w);
    }
    if ((n & 1u) && lane == 0) acc += (float)sgn[n - 1] * bf16_at(row + n - 1);
    return warp_sum(acc);
}

}  // namespace

__global__ void __launch_bounds__(kVerifyThreads)
verify_kernel(const cleave_task_t* __restrict__ tasks, uint32_t n_tasks, const cleave_gemm_t* __restrict__ gemms,
              const uint32_t* __restrict__ ksplit, const void* const* __restrict__ ab_ptrs, const float* __restrict__ partials,
              float* const* __restrict__ c_ptrs, int fused, unsigned long long seed, float tol, float4* __restrict__ out,
              unsigned int* n_bad) {
    extern __shared__ int8_t sgn[];                     // r (alpha entries) then s (beta entries)
    __shared__ float u[kVerifyKChunk], v[kVerifyKChunk];
    __shared__ float red[3][kVerifyThreads / 32];

    const uint32_t tid = blockIdx.x;
    if (tid >= n_tasks) return;
    const cleave_task_t t = tasks[tid];
    if (t.flags & CLEAVE_TASK_SUPERSEDED) {             // replaced: its pieces are checked instead
        if (threadIdx.x == 0) out[tid] = make_float4(0.f, 0.f, 0.f, 0.f);
        return;
    }
    const cleave_gemm_t g = gemms[t.gemm];
    const uint32_t alpha = t.m1 - t.m0, beta = t.n1 - t.n0;
    const uint32_t lane = threadIdx.x & 31u, warp = threadIdx.x >> 5, nwarps = kVerifyThreads / 32;
    int8_t* sr = sgn;
    int8_t* ss = sgn + alpha;
    for (uint32_t e = threadIdx.x; e < alpha; e += kVerifyThreads) sr[e] = (int8_t)sign_of(seed, tid, e, 0u);
    for (uint32_t e = threadIdx.x; e < beta; e += kVerifyThreads) ss[e] = (int8_t)sign_of(seed, tid, e, 1u);
    __syncthreads();

    // ---- lhs = r^T P s: the block sits in the arena, or in C when a one-slice GEMM was written out directly
    const bool in_c = fused && ksplit[t.gemm] == 1;
    const float* P = in_c ? c_ptrs[t.gemm] + (uint64_t)t.m0 * g.N + t.n0 : partials + t.part_off;
    const uint64_t ldp = in_c ? g.N : beta;
    float lhs = 0.f;
    for (uint32_t i = warp; i < alpha; i += nwarps) {
        const float* row = P + (uint64_t)i * ldp;
        float acc = 0.f;
        for (uint32_t j = lane; j < beta; j += 32) acc += __ldcs(row + j) * (float)ss[j];
        lhs += (float)sr[i] * acc;                      // per-lane partial, reduced at the end
    }

    // ---- rhs = (A_t^T r) . (B_t s), K-chunk by K-chunk
    const uint16_t* A = static_cast<const uint16_t*>(ab_ptrs[2 * t.gemm]);
    const uint16_t* B = static_cast<const uint16_t*>(ab_ptrs[2 * t.gemm + 1]);
    float rhs = 0.f, scale = 0.f;
    for (uint32_t kc = t.k0; kc < t.k1; kc += kVerifyKChunk) {
        const uint32_t kn = min((uint32_t)kVerifyKChunk, t.k1 - kc);     // multiple of 8 (K is)
        // u[k] = sum_i r_i A[i, k]
        if (!g.transA) {                                // stored [M x K]: thread owns 4 consecutive k
            const uint32_t k = 4 * threadIdx.x;
            if (k < kn) {
                float a4[4];
                column_sums4(A + (uint64_t)t.m0 * g.lda + kc + k, g.lda, alpha, sr, a4);
                u[k] = a4[0]; u[k + 1] = a4[1]; u[k + 2] = a4[2]; u[k + 3] = a4[3];
            }
        } else {                                        // stored [K x M]: one warp per stored row k
            for (uint32_t k = warp; k < kn; k += nwarps) {
                const float d = row_dot(A + (uint64_t)(kc + k) * g.lda + t.m0, alpha, sr, lane);
                if (lane == 0) u[k] = d;
            }
        }
        // v[k] = sum_j B[k, j] s_j
        if (g.transB) {                                 // stored [N x K]: thread owns 4 consecutive k
            const uint32_t k = 4 * threadIdx.x;
            if (k < kn) {
                float b4[4];
                column_sums4(B + (uint64_t)t.n0 * g.ldb + kc + k, g.ldb, beta, ss, b4);
                v[k] = b4[0]; v[k + 1] = b4[1]; v[k + 2] = b4[2]; v[k + 3] = b4[3];
            }
        } else {                                        // stored [K x N]: one warp per stored row k
            for (uint32_t k = warp; k < kn; k += nwarps) {
                const float d = row_dot(B + (uint64_t)(kc + k) * g.ldb + t.n0, beta, ss, lane);
                if (lane == 0) v[k] = d;
            }
        }
        __syncthreads();
        for (uint32_t k = threadIdx.x; k < kn; k += kVerifyThreads) { rhs += u[k] * v[k]; scale += fabsf(u[k]) * fabsf(v[k]); }
        __syncthreads();
    }

    lhs = warp_sum(lhs); rhs = warp_sum(rhs); scale = warp_sum(scale);
    if (lane == 0) { red[0][warp] = lhs; red[1][warp] = rhs; red[2][warp] = scale; }
    __syncthreads();
    if (threadIdx.x == 0) {
        float l = 0.f, r = 0.f, s = 0.f;
        for (uint32_t w = 0; w < nwarps; ++w) { l += red[0][w]; r += red[1][w]; s += red[2][w]; }
        // NaN (a block never written) must fail: the comparison is written so that NaN is "bad"
        const bool ok = fabsf(l - r) <= tol * s;
        out[tid] = make_float4(l, r, s, ok ? 0.f : 1.f);
        if (!ok) atomicAdd(n_bad, 1u);
    }
}

cudaError_t launch_verify(const cleave_task_t* tasks, uint32_t n_tasks, const cleave_gemm_t* gemms, const uint32_t* ksplit,
                          const void* const* ab_ptrs, const float* partials, float* const* c_ptrs, int fused, uint64_t seed,
                          float tol, float4* out, unsigned int* n_bad, uint32_t sign_bytes, cudaStream_t st) {
    if (!n_tasks) return cudaSuccess;
    if (sign_bytes > 40 * 1024) {
        // the attribute belongs to the current device's copy of the kernel: set it on every such launch
        cudaError_t e = cudaFuncSetAttribute(verify_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sign_bytes);
        if (e != cudaSuccess) return e;
    }
    verify_kernel<<<n_tasks, kVerifyThreads, sign_bytes, st>>>(tasks, n_tasks, gemms, ksplit, ab_ptrs, partials, c_ptrs, fused,
                                                               (unsigned long long)seed, tol, out, n_bad);
    return cudaGetLastError();
}

}  // namespace cleave
