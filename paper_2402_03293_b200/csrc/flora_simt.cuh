// Plain fp32 SIMT kernels for every operation of the path.  They cover what the tensor-core
// kernels do not (fp32 matrices, unaligned pointers) and serve as a second on-device opinion.
// The projection is regenerated per tile in shared memory; nothing of A reaches global memory
// except through materialize_kernel, which exists for bit-exact checks of the generator.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include "flora_rng.cuh"

namespace flora {

__device__ __forceinline__ float to_float(float v) { return v; }
__device__ __forceinline__ float to_float(__nv_bfloat16 v) { return __bfloat162float(v); }
__device__ __forceinline__ void from_float(float& dst, float v) { dst = v; }
__device__ __forceinline__ void from_float(__nv_bfloat16& dst, float v) { dst = __float2bfloat16_rn(v); }

// ------------------------------------------------------------------------------------------------
// A itself (test hook): one thread per Philox block, four columns of one row.
// ------------------------------------------------------------------------------------------------
template <typename TOut>
__global__ void materialize_kernel(TOut* __restrict__ out, int r, int64_t m, int64_t ld, PhiloxKey key, float scale)
{
    const int64_t quads = (m + 3) / 4;
    const int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (t >= quads * r) return;
    const uint32_t j = (uint32_t)(t / quads);
    const uint32_t q = (uint32_t)(t % quads);
    float a[4];
    projection_quad(q, j, key, scale, a);
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int64_t col = 4ll * q + u;
        if (col < m) from_float(out[(int64_t)j * ld + col], a[u]);
    }
}

// ------------------------------------------------------------------------------------------------
// S[i,j] <- b S[i,j] + a sum_k G[i,k] A[j,k]        (Algorithm 1 compression; Algorithm 2 update)
// Block: 32 rows of G, all r columns of S; k advances in chunks of 32.
// ------------------------------------------------------------------------------------------------
constexpr int SIMT_THREADS = 256;

template <typename TG>
__global__ void __launch_bounds__(SIMT_THREADS)
simt_compress_kernel(const TG* __restrict__ G, int64_t n, int64_t m, int64_t ldg,
                     float* __restrict__ S, int64_t lds, int r, PhiloxKey key, float scale, float a, float b)
{
    constexpr bool kBf16A = sizeof(TG) == 2;
    __shared__ float Gs[32][33];
    __shared__ float As[256][33];
    const int tid = threadIdx.x;
    const int ti = tid >> 3, tj = tid & 7;
    const int64_t row0 = (int64_t)blockIdx.x * 32;
    float acc[32];
#pragma unroll
    for (int u = 0; u < 32; ++u) acc[u] = 0.0f;

    for (int64_t k0 = 0; k0 < m; k0 += 32) {
        for (int t = tid; t < r * 8; t += SIMT_THREADS) {
            const int j = t >> 3, qq = t & 7;
            float v[4];
            projection_quad((uint32_t)(k0 / 4 + qq), (uint32_t)j, key, scale, v);
#pragma unroll
            for (int u = 0; u < 4; ++u) As[j][qq * 4 + u] = kBf16A ? bf16_round(v[u]) : v[u];
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int idx = tid + SIMT_THREADS * u;
            const int rr = idx >> 5, cc = idx & 31;
            const int64_t gi = row0 + rr, gk = k0 + cc;
            Gs[rr][cc] = (gi < n && gk < m) ? to_float(G[gi * ldg + gk]) : 0.0f;
        }
        __syncthreads();
#pragma unroll 4
        for (int kk = 0; kk < 32; ++kk) {
            const float g = Gs[ti][kk];
#pragma unroll
            for (int u = 0; u < 32; ++u)
                if (tj + 8 * u < r) acc[u] = fmaf(g, As[tj + 8 * u][kk], acc[u]);
        }
        __syncthreads();
    }
    const int64_t gi = row0 + ti;
    if (gi < n) {
#pragma unroll
        for (int u = 0; u < 32; ++u) {
            const int j = tj + 8 * u;
            if (j < r) {
                float* p = S + gi * lds + j;
                // b == 0 must not propagate whatever the state held before (it may be uninitialised)
                *p = (b == 0.0f) ? a * acc[u] : fmaf(b, *p, a * acc[u]);
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// W[i,k] <- W[i,k] - step * sum_j C[i,j] A[j,k]      (Algorithm 1 decompression as an update)
// Block: 32 rows x 64 columns of W; j advances in chunks of 32.
// ------------------------------------------------------------------------------------------------
template <typename TW>
__global__ void __launch_bounds__(SIMT_THREADS)
simt_decompress_kernel(TW* __restrict__ W, int64_t n, int64_t m, int64_t ldw,
                       const float* __restrict__ C, int64_t ldc, int r, PhiloxKey key, float scale, float step)
{
    constexpr bool kBf16A = sizeof(TW) == 2;
    __shared__ float As[32][65];
    __shared__ float Cs[32][33];
    const int tid = threadIdx.x;
    const int tc = tid & 63, tr = tid >> 6;
    const int64_t row0 = (int64_t)blockIdx.y * 32;
    const int64_t col0 = (int64_t)blockIdx.x * 64;
    float acc[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) acc[u] = 0.0f;

    for (int j0 = 0; j0 < r; j0 += 32) {
        for (int t = tid; t < 32 * 16; t += SIMT_THREADS) {
            const int jj = t >> 4, qq = t & 15;
            float v[4] = {0.0f, 0.0f, 0.0f, 0.0f};
            if (j0 + jj < r) projection_quad((uint32_t)(col0 / 4 + qq), (uint32_t)(j0 + jj), key, scale, v);
#pragma unroll
            for (int u = 0; u < 4; ++u) As[jj][qq * 4 + u] = kBf16A ? bf16_round(v[u]) : v[u];
        }
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            const int idx = tid + SIMT_THREADS * u;
            const int rr = idx >> 5, jj = idx & 31;
            const int64_t gi = row0 + rr;
            Cs[rr][jj] = (gi < n && j0 + jj < r) ? C[gi * ldc + j0 + jj] : 0.0f;
        }
        __syncthreads();
#pragma unroll 4
        for (int jj = 0; jj < 32; ++jj) {
            const float av = As[jj][tc];
#pragma unroll
            for (int u = 0; u < 8; ++u) acc[u] = fmaf(Cs[tr + 4 * u][jj], av, acc[u]);
        }
        __syncthreads();
    }
    const int64_t gk = col0 + tc;
    if (gk < m) {
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int64_t gi = row0 + tr + 4 * u;
            if (gi < n) {
                TW* p = W + gi * ldw + gk;
                from_float(*p, fmaf(-step, acc[u], to_float(*p)));
            }
        }
    }
}

// ------------------------------------------------------------------------------------------------
// T[a,b] += sum_{k in this block's range} A_old[a,k] A_new[b,k]   (r x r; T zeroed beforehand)
// Block: one 32 x 32 tile of T and one slice of k.  k_per_block is a multiple of 32.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(SIMT_THREADS)
simt_gram_kernel(float* __restrict__ T, int r, int64_t m, int64_t k_per_block, bool bf16_a,
                 PhiloxKey key_old, PhiloxKey key_new, float scale)
{
    __shared__ float Ao[32][33];
    __shared__ float An[32][33];
    const int tid = threadIdx.x;
    const int tiles = (r + 31) / 32;
    const int a0 = (blockIdx.x / tiles) * 32, b0 = (blockIdx.x % tiles) * 32;
    const int ta = tid >> 3, tb = tid & 7;      // outputs (ta, tb + 8u), u < 4
    const int64_t kbeg = (int64_t)blockIdx.y * k_per_block;
    const int64_t kend = min(m, kbeg + k_per_block);
    float acc[4] = {0.0f, 0.0f, 0.0f, 0.0f};
    for (int64_t k0 = kbeg; k0 < kend; k0 += 32) {
        {
            const int jj = tid >> 3, qq = tid & 7;      // 32 rows x 8 quads = 256 tasks per matrix
            float v[4] = {0.0f, 0.0f, 0.0f, 0.0f}, w[4] = {0.0f, 0.0f, 0.0f, 0.0f};
            if (a0 + jj < r) projection_quad((uint32_t)(k0 / 4 + qq), (uint32_t)(a0 + jj), key_old, scale, v);
            if (b0 + jj < r) projection_quad((uint32_t)(k0 / 4 + qq), (uint32_t)(b0 + jj), key_new, scale, w);
#pragma unroll
            for (int u = 0; u < 4; ++u) {
                const bool in = k0 + qq * 4 + u < kend;
                Ao[jj][qq * 4 + u] = in ? (bf16_a ? bf16_round(v[u]) : v[u]) : 0.0f;
                An[jj][qq * 4 + u] = in ? (bf16_a ? bf16_round(w[u]) : w[u]) : 0.0f;
            }
        }
        __syncthreads();
#pragma unroll 8
        for (int kk = 0; kk < 32; ++kk) {
            const float av = Ao[ta][kk];
#pragma unroll
            for (int u = 0; u < 4; ++u) acc[u] = fmaf(av, An[tb + 8 * u][kk], acc[u]);
        }
        __syncthreads();
    }
#pragma unroll
    for (int u = 0; u < 4; ++u) {
        const int a = a0 + ta, b = b0 + tb + 8 * u;
        if (a < r && b < r) atomicAdd(T + (int64_t)a * r + b, acc[u]);
    }
}

// ------------------------------------------------------------------------------------------------
// dst[i,:] <- bb dst[i,:] + aa src[i,:] T          (rows are independent; dst may alias src)
// Block: 8 rows; thread b owns column b of the 8 outputs.
// ------------------------------------------------------------------------------------------------
__global__ void __launch_bounds__(SIMT_THREADS)
simt_apply_gram_kernel(float* dst, int64_t ldd, const float* src, int64_t lds,
                       int64_t n, int r, const float* __restrict__ T, float aa, float bb)
{
    __shared__ float Ss[8][256];
    const int tid = threadIdx.x;
    const int64_t row0 = (int64_t)blockIdx.x * 8;
    for (int t = tid; t < 8 * r; t += SIMT_THREADS) {
        const int i = t / r, a = t % r;
        Ss[i][a] = (row0 + i < n) ? src[(row0 + i) * lds + a] : 0.0f;
    }
    __syncthreads();
    if (tid < r) {
        float acc[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) acc[i] = 0.0f;
        for (int a = 0; a < r; ++a) {
            const float t = T[(int64_t)a * r + tid];
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] = fmaf(Ss[i][a], t, acc[i]);
        }
#pragma unroll
        for (int i = 0; i < 8; ++i)
            if (row0 + i < n) {
                float* p = dst + (row0 + i) * ldd + tid;
                *p = (bb == 0.0f) ? aa * acc[i] : fmaf(bb, *p, aa * acc[i]);
            }
    }
}

}  // namespace flora
