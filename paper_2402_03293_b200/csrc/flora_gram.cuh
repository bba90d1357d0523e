// Momentum transfer on tensor cores (Algorithm 2, resampling branch):  dst <- b dst + a src (A_old A_new^T).
//
//   gram_tc_kernel        T += A_old[:, k-range] A_new[:, k-range]^T   (r x r, both operands generated in shared
//                         memory as bf16, tcgen05 MMA into tensor memory, atomic adds of the partial products)
//   apply_gram_jobs_kernel  dst <- b dst + a src T, row block by row block, for a list of matrices
//
// A whole weight set is handled by one launch of each kernel over a job table that is built per call.
#pragma once
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <string.h>

#include <algorithm>
#include <atomic>
#include <vector>

#include "../../include/flora.h"
#include "flora_pool.cuh"
#include "flora_ptx.cuh"
#include "flora_rng.cuh"
#include "flora_tc.cuh"
#include "flora_tc_host.cuh"

namespace flora {

struct GramJob {            // one matrix
    float* T;               // r x r scratch, zeroed before the gram kernel runs
    float* dst;
    const float* src;
    int64_t ldd, lds;
    int32_t n, m;
    uint64_t seed_old, seed_new;
    int32_t mat;            // index of the matrix in the sets' descriptor tables (tensor-core apply kernel)
    int32_t pad;
};

struct GramItem {           // one CTA of the gram kernel
    int32_t job;
    int32_t kstep0;         // first step (a step is kw = 16, 32 or 64 columns, the same for the whole launch)
    int32_t ksteps;
    int32_t pad;
};

constexpr int GRAM_GEN_WARPS = 20;
constexpr int GRAM_THREADS = 32 * (1 + GRAM_GEN_WARPS);   // warp 0: MMA issuer, warps 1..20: generators (1-4 also read back)

struct GramSmem {
    uint64_t full[2], empty[2], acc_full;
    uint32_t tmem_base;
    int abort;
};

// Zeroes the elements of a packed bf16x2 word whose column is >= m.
__device__ __forceinline__ uint32_t mask_pair(uint32_t w, int64_t col, int64_t m)
{
    if (col >= m) return 0u;
    if (col + 1 >= m) return w & 0x0000FFFFu;
    return w;
}

// SINGLE: one matrix, passed by value; CTA b takes the steps [b * per_steps, (b + 1) * per_steps) (no tables in memory).
template <bool SINGLE>
__global__ void __launch_bounds__(GRAM_THREADS, 1)
gram_tc_kernel(const GramJob* __restrict__ jobs, const GramItem* __restrict__ items, const __grid_constant__ GramJob single, int per_steps,
               int r, float scale, int kw)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
    const int r_m = (r + 127) & ~127;                     // rows of the M operand (A_old), whole 128-row MMAs
    const int r_n = (r + 15) & ~15;                       // rows of the N operand (A_new)
    const int halves = r_m >> 7;
    const uint32_t old_bytes = (uint32_t)r_m * 128u, new_bytes = (uint32_t)r_n * 128u;
    const uint32_t stage_bytes = old_bytes + new_bytes;
    GramSmem* ctl = reinterpret_cast<GramSmem*>(smem_raw + (smem_base - ptx::smem_addr(smem_raw)) + 2 * (size_t)stage_bytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    GramItem item;
    if (SINGLE) {
        const int total = (single.m + kw - 1) / kw;
        item.job = 0;
        item.kstep0 = (int)blockIdx.x * per_steps;
        item.ksteps = min(per_steps, total - item.kstep0);
        item.pad = 0;
    } else {
        item = items[blockIdx.x];
    }
    const GramJob job = SINGLE ? single : jobs[item.job];
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < halves * r_n) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->full[s]), GRAM_GEN_WARPS);
            ptx::mbar_init(ptx::smem_addr(&ctl->empty[s]), 1);
        }
        ptx::mbar_init(ptx::smem_addr(&ctl->acc_full), 1);
        ctl->abort = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async_smem();
    }
    if (warp == 0) {
        ptx::tmem_alloc(ptx::smem_addr(&ctl->tmem_base), tmem_cols);
        ptx::tmem_relinquish();
    }
    // rows r .. r_m of the A_old tiles and r .. r_n of the A_new tiles stay zero
    for (int s = 0; s < 2; ++s) {
        const uint32_t st = smem_base + s * stage_bytes;
        for (int t = threadIdx.x; t < (r_m - r) * 8; t += GRAM_THREADS) ptx::st_shared_v4(st + (uint32_t)r * 128u + t * 16u, 0, 0, 0, 0);
        for (int t = threadIdx.x; t < (r_n - r) * 8; t += GRAM_THREADS)
            ptx::st_shared_v4(st + old_bytes + (uint32_t)r * 128u + t * 16u, 0, 0, 0, 0);
    }
    ptx::fence_proxy_async_smem();
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = ctl->tmem_base;
    volatile int* abort = &ctl->abort;

    if (warp == 0) {
        if (lane == 0) {
            const uint32_t idesc = ptx::umma_idesc_bf16((uint32_t)r_n);
            const uint64_t desc_base = ptx::umma_desc_k_sw128(smem_base);
            bool ok = true;
            for (int ks = 0; ks < item.ksteps && ok; ++ks) {
                const int s = ks & 1;
                ok = ptx::mbar_wait(ptx::smem_addr(&ctl->full[s]), (ks >> 1) & 1, abort);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint64_t d_old = desc_base + (uint64_t)((s * stage_bytes) >> 4);
                const uint64_t d_new = d_old + (uint64_t)(old_bytes >> 4);
                for (int h = 0; h < halves; ++h)
                    for (int kk = 0; kk < (kw >> 4); ++kk)
                        ptx::umma_bf16(tmem + h * r_n, d_old + (uint64_t)((h * 128 * 128 + kk * 32) >> 4), d_new + (uint64_t)(kk * 2), idesc,
                                       (ks | kk) != 0);
                ptx::umma_commit(ptx::smem_addr(&ctl->empty[s]));
            }
            if (ok) ptx::umma_commit(ptx::smem_addr(&ctl->acc_full));
        }
    } else {
        const int g = threadIdx.x - 32;
        const PhiloxKey key_old = make_key(job.seed_old), key_new = make_key(job.seed_new);
        const int cpr = kw >> 3;                          // 16-byte chunks (8 columns) per row of a step: 2, 4 or 8
        const int per_mat = r * cpr;                      // (row, 16-byte chunk) tasks of one tile
        bool ok = true;
        for (int ks = 0; ks < item.ksteps && ok; ++ks) {
            const int s = ks & 1;
            ok = ptx::mbar_wait(ptx::smem_addr(&ctl->empty[s]), ((ks >> 1) & 1) ^ 1, abort);
            if (!ok) break;
            const uint32_t st = smem_base + s * stage_bytes;
            const uint32_t q0 = (uint32_t)(item.kstep0 + ks) * (uint32_t)(kw >> 2);
            const int64_t col_base = (int64_t)(item.kstep0 + ks) * kw;
            const bool ragged = col_base + kw > job.m;
            for (int t = g; t < 2 * per_mat; t += 32 * GRAM_GEN_WARPS) {
                const bool is_new = t >= per_mat;
                const int tt = is_new ? t - per_mat : t;
                const int j = tt / cpr, c = tt % cpr;
                const PhiloxKey key = is_new ? key_new : key_old;
                uint2 lo = projection_quad_bf16(q0 + 2 * c, (uint32_t)j, key, scale);
                uint2 hi = projection_quad_bf16(q0 + 2 * c + 1, (uint32_t)j, key, scale);
                if (ragged) {                              // columns >= m contribute nothing
                    const int64_t col = col_base + 8 * c;
                    lo.x = mask_pair(lo.x, col, job.m);
                    lo.y = mask_pair(lo.y, col + 2, job.m);
                    hi.x = mask_pair(hi.x, col + 4, job.m);
                    hi.y = mask_pair(hi.y, col + 6, job.m);
                }
                ptx::st_shared_v4(st + (is_new ? old_bytes : 0u) + j * 128 + ((c ^ (j & 7)) << 4), lo.x, lo.y, hi.x, hi.y);
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->full[s]));
        }
        if (warp <= 4 && ok) {
            // read back: warp w owns tensor-memory lanes 32*(w%4) .. +31 = rows of T within a 128-row half
            const int quarter = warp & 3;
            if (ptx::mbar_wait(ptx::smem_addr(&ctl->acc_full), 0, abort)) {
                ptx::tc_fence_after_sync();
                const bool vec_ok = (r & 3) == 0 && (reinterpret_cast<uintptr_t>(job.T) & 15) == 0;
                for (int h = 0; h < halves; ++h) {
                    const int a = h * 128 + quarter * 32 + lane;
                    float* trow = job.T + (int64_t)a * r;
                    for (int j0 = 0; j0 < r_n; j0 += 16) {
                        uint32_t v[16];
                        ptx::tmem_ld_16(tmem + ((uint32_t)(quarter * 32) << 16) + h * r_n + j0, v);
                        ptx::tmem_ld_wait();
                        if (a < r) {
                            if (vec_ok && j0 + 16 <= r) {
#pragma unroll
                                for (int u = 0; u < 16; u += 4)
                                    ptx::red_add_v4(trow + j0 + u, __uint_as_float(v[u]), __uint_as_float(v[u + 1]), __uint_as_float(v[u + 2]),
                                                    __uint_as_float(v[u + 3]));
                            } else {
#pragma unroll
                                for (int u = 0; u < 16; ++u)
                                    if (j0 + u < r) atomicAdd(trow + j0 + u, __uint_as_float(v[u]));
                            }
                        }
                    }
                }
            }
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 0) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem, tmem_cols);
    }
}

// Fallback of the kernel below for sketches whose rows are not 16-byte aligned or whose rank is no multiple of 4.
// dst[i,:] <- bb dst[i,:] + aa src[i,:] T for every job (or the one passed by value); blockIdx.y = job.  A block
// takes 8 rows and has one thread per column of the sketch (r rounded up to whole warps); the rows are staged in
// shared memory first, so dst may alias src.
constexpr int APPLY_ROWS = 8;
template <bool SINGLE>
__global__ void __launch_bounds__(256)
apply_gram_rows_kernel(const GramJob* __restrict__ jobs, const __grid_constant__ GramJob single, int r, float aa, float bb)
{
    __shared__ float Ss[APPLY_ROWS][256];
    const GramJob job = SINGLE ? single : jobs[blockIdx.y];
    const int tid = threadIdx.x;
    const int64_t row0 = (int64_t)blockIdx.x * APPLY_ROWS;
    if (row0 >= job.n) return;
    for (int t = tid; t < APPLY_ROWS * r; t += (int)blockDim.x) {
        const int i = t / r, a = t % r;
        Ss[i][a] = (row0 + i < job.n) ? job.src[(row0 + i) * job.lds + a] : 0.0f;
    }
    __syncthreads();
    if (tid < r) {
        float acc[APPLY_ROWS];
#pragma unroll
        for (int i = 0; i < APPLY_ROWS; ++i) acc[i] = 0.0f;
        for (int a = 0; a < r; ++a) {
            const float t = job.T[(int64_t)a * r + tid];
#pragma unroll
            for (int i = 0; i < APPLY_ROWS; ++i) acc[i] = fmaf(Ss[i][a], t, acc[i]);
        }
#pragma unroll
        for (int i = 0; i < APPLY_ROWS; ++i)
            if (row0 + i < job.n) {
                float* p = job.dst + (row0 + i) * job.ldd + tid;
                *p = (bb == 0.0f) ? aa * acc[i] : fmaf(bb, *p, aa * acc[i]);
            }
    }
}

// dst[i,:] <- bb dst[i,:] + aa src[i,:] T for every job (or the one passed by value); blockIdx.y = job.
// Register-tiled: a thread owns 8 rows x 4 columns of the output; per four steps of the inner index it reads four
// 16-byte pieces of T and eight of src from shared memory for 128 multiply-adds.  T streams through shared memory in
// tiles of 16 rows, double-buffered with asynchronous copies; the block's rows of src are staged first, so dst may
// alias src.  Needs r % 4 == 0 and 16-byte aligned rows of src, dst and T.
constexpr int APPLY_RT = 8;                 // rows per thread
constexpr int APPLY_AC = 16;                // rows of T per tile
constexpr int APPLY_SRC_FLOATS = 9728;      // >= rows_per_block * (r + 4) for every r <= 256
inline int apply_row_groups(int r) { return std::min(256 / (r >> 2), 32); }
inline size_t apply_smem_bytes(int r) { return sizeof(float) * ((size_t)APPLY_SRC_FLOATS + 2 * (size_t)APPLY_AC * r); }
template <bool SINGLE>
__global__ void __launch_bounds__(256)
apply_gram_jobs_kernel(const GramJob* __restrict__ jobs, const __grid_constant__ GramJob single, int r, int row_groups, float aa, float bb)
{
    extern __shared__ __align__(16) float apply_smem[];
    float* Ss = apply_smem;
    float* Ts = apply_smem + APPLY_SRC_FLOATS;                 // two tiles of APPLY_AC x r
    const GramJob job = SINGLE ? single : jobs[blockIdx.y];
    const int tid = threadIdx.x;
    const int cgs = r >> 2, rs = r + 4;                        // column groups; padded row stride of the src rows
    const int rows = row_groups * APPLY_RT;
    const int64_t row0 = (int64_t)blockIdx.x * rows;
    if (row0 >= job.n) return;
    const int ntiles = (r + APPLY_AC - 1) / APPLY_AC;
    auto load_tile = [&](int k) {
        const int a0 = k * APPLY_AC, na = min(APPLY_AC, r - a0);
        float* dst = Ts + (k & 1) * APPLY_AC * r;
        for (int t = tid; t < na * cgs; t += 256) ptx::cp_async_16(ptx::smem_addr(dst + 4 * t), job.T + (int64_t)a0 * r + 4 * t);
        ptx::cp_async_commit();
    };
    load_tile(0);
    for (int t = tid; t < rows * cgs; t += 256) {
        const int i = t / cgs, c = t % cgs;
        float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
        if (row0 + i < job.n) v = *reinterpret_cast<const float4*>(job.src + (row0 + i) * job.lds + 4 * c);
        *reinterpret_cast<float4*>(&Ss[i * rs + 4 * c]) = v;
    }
    const int rg = tid / cgs, cg = tid % cgs;
    const bool active = rg < row_groups;
    float acc[APPLY_RT][4];
#pragma unroll
    for (int i = 0; i < APPLY_RT; ++i)
#pragma unroll
        for (int j = 0; j < 4; ++j) acc[i][j] = 0.0f;
    const float* srow = &Ss[rg * rs];                          // the thread's rows are rg, rg + row_groups, ...: neighbours in a warp hit different banks
    for (int k = 0; k < ntiles; ++k) {
        if (k + 1 < ntiles) {
            load_tile(k + 1);
            ptx::cp_async_wait<1>();
        } else {
            ptx::cp_async_wait<0>();
        }
        __syncthreads();                                       // tile k (and, the first time, the src rows) visible to all
        if (active) {
            const int a0 = k * APPLY_AC, na = min(APPLY_AC, r - a0);
            const float* tt = Ts + (k & 1) * APPLY_AC * r + 4 * cg;
            for (int al = 0; al < na; al += 4) {
                float4 t[4];
#pragma unroll
                for (int u = 0; u < 4; ++u) t[u] = *reinterpret_cast<const float4*>(tt + (al + u) * r);
#pragma unroll
                for (int i = 0; i < APPLY_RT; ++i) {
                    const float4 sv = *reinterpret_cast<const float4*>(&srow[i * row_groups * rs + a0 + al]);
                    const float sa[4] = {sv.x, sv.y, sv.z, sv.w};
#pragma unroll
                    for (int u = 0; u < 4; ++u) {              // same order of accumulation as one thread per column: a ascending
                        acc[i][0] = fmaf(sa[u], t[u].x, acc[i][0]);
                        acc[i][1] = fmaf(sa[u], t[u].y, acc[i][1]);
                        acc[i][2] = fmaf(sa[u], t[u].z, acc[i][2]);
                        acc[i][3] = fmaf(sa[u], t[u].w, acc[i][3]);
                    }
                }
            }
        }
        __syncthreads();                                       // everyone is done with tile k before it is overwritten
    }
    if (!active) return;
#pragma unroll
    for (int i = 0; i < APPLY_RT; ++i) {
        const int64_t row = row0 + i * row_groups + rg;
        if (row < job.n) {
            float4* p = reinterpret_cast<float4*>(job.dst + row * job.ldd + 4 * cg);
            float4 o = make_float4(aa * acc[i][0], aa * acc[i][1], aa * acc[i][2], aa * acc[i][3]);
            if (bb != 0.0f) {
                const float4 d = *p;
                o = make_float4(fmaf(bb, d.x, o.x), fmaf(bb, d.y, o.y), fmaf(bb, d.z, o.z), fmaf(bb, d.w, o.w));
            }
            *p = o;
        }
    }
}

// ------------------------------------------------------------------------------------------------
// dst <- bb dst + aa src T on tensor cores, for sketches whose rows the TMA can address (16-byte aligned rows).
//
// The product is a dense contraction over the rank (2 n r^2 flops), so it runs as tf32 MMAs that read the fp32 sketch
// as it is stored.  A CTA pair (tcgen05 cta_group::2) multiplies 256 rows at a time: each CTA streams the rows of its
// own 128-row tile of src through a ring of 32-column chunks (TMA), and holds one half of the N x K operand
// T^T (the gram kernel is run with the roles of the two projections exchanged, so that its output is T^T, K-major):
// at r = 256 that half is 128 KB of shared memory, which is why the rows are not split further.  Every row of the
// sketch has one owner, and a tile's rows of src are in shared memory or consumed before any of its rows of dst is
// written: dst may be src.  The accumulators (128 rows x r columns per CTA) are double-buffered in tensor memory, so
// the epilogue of one tile (old values of dst by TMA, dst = bb dst + aa acc, TMA store) overlaps the MMAs of the next.
// Work: per cluster a list of units (matrix, first pair of tiles, number of pairs); persistent.
// ------------------------------------------------------------------------------------------------
struct ApplyUnit {
    int32_t job, tp0, ntp, pad;
};
constexpr int APPLY_TC_THREADS = 32 * 6;    // warp 0: src loads, 1: MMA issue (leader) / relay (follower), 2-5: T^T loads and epilogue
constexpr int APPLY_TC_STAGES = 4;
constexpr int APPLY_TC_CHUNK = 128 * 128;   // 128 rows x 32 fp32
struct ApplyTcSmem {
    uint64_t full_a[APPLY_TC_STAGES], empty_a[APPLY_TC_STAGES], peer_full[APPLY_TC_STAGES], acc_full[2], acc_empty[2], b_full, old_full[2];
    uint32_t tmem_base;
    int abort;
    int epi_go;
};
inline size_t apply_tc_smem_bytes(int r)
{
    const int n_half = ((r + 15) & ~15) / 2, kchunks = (r + 31) / 32;
    return (size_t)kchunks * n_half * 128 + (size_t)(APPLY_TC_STAGES + 2) * APPLY_TC_CHUNK + sizeof(ApplyTcSmem) + 1024;
}

// SINGLE: one matrix; its job and the two tensor maps travel as kernel parameters, and cluster c takes the pairs of
// tiles [c * per_cluster, (c + 1) * per_cluster).
struct ApplySingle {
    CUtensorMap map_dst, map_src;
    GramJob job;
};
template <bool SINGLE>
__global__ void __launch_bounds__(APPLY_TC_THREADS, 1)
apply_tc_kernel(const GramJob* __restrict__ jobs, const TcMatrix* __restrict__ dst_mats, const TcMatrix* __restrict__ src_mats,
                const ApplyUnit* __restrict__ units, const int* __restrict__ slot_begin, const __grid_constant__ ApplySingle single, int per_cluster,
                int r, float aa, float bb)
{
    // A kernel launched behind this one with the programmatic-serialization attribute may start now (the compression of
    // a resampling step does: it streams G, which this kernel does not touch, and waits itself before it reads a sketch).
    ptx::grid_launch_dependents();
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
    const int N = (r + 15) & ~15, n_half = N >> 1, kchunks = (r + 31) >> 5;
    const uint32_t b_block = (uint32_t)n_half * 128u;                    // one 32-column chunk of this CTA's half of T^T
    const uint32_t a_ring = smem_base + (uint32_t)kchunks * b_block;
    const uint32_t staging = a_ring + APPLY_TC_STAGES * APPLY_TC_CHUNK;  // two chunk buffers of the epilogue
    ApplyTcSmem* ctl = reinterpret_cast<ApplyTcSmem*>(smem_raw + (staging - ptx::smem_addr(smem_raw)) + 2 * (size_t)APPLY_TC_CHUNK);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t half = ptx::cluster_ctarank();
    const int slot = (int)(blockIdx.x >> 1);
    int u_begin, u_end;
    if (SINGLE) {
        u_begin = 0;
        u_end = 1;
    } else {
        u_begin = slot_begin[slot];
        u_end = slot_begin[slot + 1];
    }
    auto unit_at = [&](int u) {
        if (SINGLE) {
            const int total = (single.job.n + 255) >> 8;
            ApplyUnit v;
            v.job = 0;
            v.tp0 = slot * per_cluster;
            v.ntp = max(0, min(per_cluster, total - v.tp0));
            v.pad = 0;
            return v;
        }
        return units[u];
    };
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < 2 * N) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < APPLY_TC_STAGES; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->full_a[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->empty_a[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->peer_full[s]), 1);
        }
        for (int k = 0; k < 2; ++k) {
            ptx::mbar_init(ptx::smem_addr(&ctl->acc_full[k]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->acc_empty[k]), 8);      // the four epilogue warps of both CTAs
            ptx::mbar_init(ptx::smem_addr(&ctl->old_full[k]), 1);
        }
        ptx::mbar_init(ptx::smem_addr(&ctl->b_full), 8);                // the four loader warps of both CTAs
        ctl->abort = 0;
        ctl->epi_go = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async_smem();
    }
    if (warp == 1) {
        ptx::tmem_alloc_pair(ptx::smem_addr(&ctl->tmem_base), tmem_cols);
        ptx::tmem_relinquish_pair();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = ctl->tmem_base;
    volatile int* abort = &ctl->abort;

    if (warp == 0) {
        // ------------------------------------------------------------------ src loads: this CTA's tile, chunk by chunk
        if (lane == 0) {
            RingPos pa;
            bool ok = true;
            int issued = 0;
            for (int u = u_begin; u < u_end && ok; ++u) {
                const ApplyUnit un = unit_at(u);
                const GramJob job = SINGLE ? single.job : jobs[un.job];
                const CUtensorMap* map = SINGLE ? &single.map_src : &src_mats[job.mat].map_s;
                ptx::prefetch_tensormap(map);
                for (int tp = un.tp0; tp < un.tp0 + un.ntp && ok; ++tp) {
                    const int row0 = (2 * tp + (int)half) * 128;
                    for (int kc = 0; kc < kchunks; ++kc, pa.advance(APPLY_TC_STAGES)) {
                        ok = ptx::mbar_wait_cluster(ptx::smem_addr(&ctl->empty_a[pa.s]), (pa.wraps & 1u) ^ 1u, abort);
                        if (!ok) break;
                        const uint32_t bar = ptx::smem_addr(&ctl->full_a[pa.s]);
                        if (row0 < job.n) {
                            ptx::mbar_arrive_expect_tx(bar, APPLY_TC_CHUNK);
                            ptx::tma_load_2d(a_ring + pa.s * APPLY_TC_CHUNK, map, kc * 32, row0, bar);
                        } else {
                            ptx::mbar_arrive(bar);                       // the odd CTA of the last pair may have no rows
                        }
                        ++issued;
                    }
                }
            }
            if (*abort)
                for (int k = max(0, issued - APPLY_TC_STAGES); k < issued; ++k)
                    ptx::mbar_wait(ptx::smem_addr(&ctl->full_a[k % APPLY_TC_STAGES]), (uint32_t)(k / APPLY_TC_STAGES) & 1u, abort);
        }
    } else if (warp == 1) {
        if (lane == 0 && half == 0) {
            // -------------------------------------------------------------- MMA issuer (the pair's leader)
            const uint32_t idesc = ptx::umma_idesc_tf32_mn(256u, (uint32_t)N);
            const uint64_t desc_base = ptx::umma_desc_k_sw128(smem_base);
            RingPos pa;
            bool ok = true;
            int gt = 0, nu = 0;
            for (int u = u_begin; u < u_end && ok; ++u, ++nu) {
                const ApplyUnit un = unit_at(u);
                ok = ptx::mbar_wait_cluster(ptx::smem_addr(&ctl->b_full), (uint32_t)nu & 1u, abort);       // both halves of T^T are in place
                for (int tp = 0; tp < un.ntp && ok; ++tp, ++gt) {
                    const uint32_t acc = tmem + (uint32_t)(gt & 1) * N;
                    ok = ptx::mbar_wait_cluster(ptx::smem_addr(&ctl->acc_empty[gt & 1]), (((uint32_t)gt >> 1) & 1u) ^ 1u, abort);
                    for (int kc = 0; kc < kchunks && ok; ++kc, pa.advance(APPLY_TC_STAGES)) {
                        ok = ptx::mbar_wait(ptx::smem_addr(&ctl->full_a[pa.s]), pa.wraps & 1u, abort) &&
                             ptx::mbar_wait_cluster(ptx::smem_addr(&ctl->peer_full[pa.s]), pa.wraps & 1u, abort);
                        if (!ok) break;
                        ptx::tc_fence_after_sync();
                        const int k8s = min(4, (r - kc * 32 + 7) >> 3);      // 8-value slices of this chunk that hold columns below r
#pragma unroll
                        for (int k8 = 0; k8 < 4; ++k8) {
                            if (k8 < k8s) {
                                const uint64_t da = desc_base + (uint64_t)((a_ring - smem_base + pa.s * APPLY_TC_CHUNK + k8 * 32) >> 4);
                                const uint64_t db = desc_base + (uint64_t)((kc * b_block + k8 * 32) >> 4);
                                ptx::umma_tf32_pair(acc, da, db, idesc, (kc | k8) != 0);
                            }
                        }
                        ptx::umma_commit_pair(ptx::smem_addr(&ctl->empty_a[pa.s]), (uint16_t)3u);
                    }
                    if (ok) ptx::umma_commit_pair(ptx::smem_addr(&ctl->acc_full[gt & 1]), (uint16_t)3u);
                }
            }
        } else if (lane == 0) {
            // -------------------------------------------------------------- relay (the follower): its chunk of src has landed
            RingPos pa;
            bool ok = true;
            for (int u = u_begin; u < u_end && ok; ++u) {
                const ApplyUnit un = unit_at(u);
                for (int c = 0; c < un.ntp * kchunks; ++c, pa.advance(APPLY_TC_STAGES)) {
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->full_a[pa.s]), pa.wraps & 1u, abort);
                    if (!ok) break;
                    ptx::mbar_arrive_cluster(ptx::map_to_cta(ptx::smem_addr(&ctl->peer_full[pa.s]), 0u));
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ T^T loads, then the epilogue of every tile
        // Warp w owns tensor-memory lanes 32*(w%4) .. +31, i.e. those rows of the CTA's tile.
        const int quarter = warp & 3;
        const int tid = (int)threadIdx.x - 64;                           // 0 .. 127
        const bool leader = tid == 0;
        const int trow = quarter * 32 + lane;
        const int nchunks = (r + 31) >> 5;
        bool ok = true;
        int gt = 0;                                                      // tiles done
        uint32_t old_use[2] = {0u, 0u};                                  // how often each staging buffer has received an old chunk
        for (int u = u_begin; u < u_end; ++u) {
            const ApplyUnit un = unit_at(u);
            const GramJob job = SINGLE ? single.job : jobs[un.job];
            const CUtensorMap* map_d = SINGLE ? &single.map_dst : &dst_mats[job.mat].map_s;
            // this CTA's half of T^T: rows [half * n_half, +n_half) of the r x r matrix job.T, as the N x K operand
            // (K-major, 128-byte swizzle, chunks of 32 columns); rows and columns beyond r are zero.  The MMAs of the
            // previous unit have completed: this warp has seen the accumulators of its last tile complete.
            {
                const int vec_per_row = kchunks * 8;                     // 16-byte pieces per row
                for (int t = tid; t < n_half * vec_per_row; t += 128) {
                    const int bl = t / vec_per_row, v = t - bl * vec_per_row;
                    const int b = (int)half * n_half + bl, a0 = v * 4;
                    float4 x = make_float4(0.f, 0.f, 0.f, 0.f);
                    if (b < r) {
                        const float* src = job.T + (int64_t)b * r + a0;
                        if (a0 + 3 < r) x = *reinterpret_cast<const float4*>(src);
                        else {
                            if (a0 < r) x.x = src[0];
                            if (a0 + 1 < r) x.y = src[1];
                            if (a0 + 2 < r) x.z = src[2];
                        }
                    }
                    const int kc = v >> 3, c = v & 7;
                    ptx::st_shared_v4(smem_base + kc * b_block + bl * 128 + ((c ^ (bl & 7)) << 4), __float_as_uint(x.x), __float_as_uint(x.y),
                                      __float_as_uint(x.z), __float_as_uint(x.w));
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    if (half == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->b_full));
                    else ptx::mbar_arrive_cluster_release(ptx::map_to_cta(ptx::smem_addr(&ctl->b_full), 0u));
                }
            }
            for (int tp = un.tp0; tp < un.tp0 + un.ntp; ++tp, ++gt) {
                const int row0 = (2 * tp + (int)half) * 128;
                const bool rows = row0 < job.n;
                const bool rmw = bb != 0.0f;
                if (ok) ok = ptx::mbar_wait_cluster(ptx::smem_addr(&ctl->acc_full[gt & 1]), ((uint32_t)gt >> 1) & 1u, abort);
                ptx::tc_fence_after_sync();
                if (rows) {
                    // old values of dst come in by TMA, up to two chunks ahead (one per staging buffer)
                    auto request_old = [&](int c) {
                        const uint32_t bar = ptx::smem_addr(&ctl->old_full[c & 1]);
                        ptx::mbar_arrive_expect_tx(bar, APPLY_TC_CHUNK);
                        ptx::tma_load_2d(staging + (uint32_t)(c & 1) * APPLY_TC_CHUNK, map_d, c * 32, row0, bar);
                    };
                    if (leader && ok && !*abort) {
                        ptx::tma_store_wait_read<0>();                   // both buffers have been read out by the stores of the previous tile
                        if (rmw) {
                            request_old(0);
                            if (nchunks > 1) request_old(1);
                        }
                    }
                    for (int c = 0; c < nchunks; ++c) {
                        const uint32_t buf = staging + (uint32_t)(c & 1) * APPLY_TC_CHUNK;
                        const uint32_t brow = buf + (uint32_t)trow * 128u;
                        if (leader) {
                            const bool go = ok && !*abort;
                            if (go && !rmw) ptx::tma_store_wait_read<1>();   // the store of chunk c - 2 has read this buffer
                            ctl->epi_go = go ? 1 : 0;
                        }
                        ptx::named_barrier_sync(1, 128);
                        if (!*(volatile int*)&ctl->epi_go) break;         // uniform: written before the barrier by one thread
                        uint32_t v[32];
                        const int col0 = c * 32;
                        if (col0 < N) ptx::tmem_ld_16(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(gt & 1) * N + col0, *reinterpret_cast<uint32_t(*)[16]>(&v[0]));
                        if (col0 + 16 < N) ptx::tmem_ld_16(tmem + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(gt & 1) * N + col0 + 16, *reinterpret_cast<uint32_t(*)[16]>(&v[16]));
                        ptx::tmem_ld_wait();
                        if (col0 + 16 >= N) {
#pragma unroll
                            for (int k = 16; k < 32; ++k) v[k] = 0u;
                        }
                        if (rmw) {
                            if (!ptx::mbar_wait(ptx::smem_addr(&ctl->old_full[c & 1]), old_use[c & 1] & 1u, abort)) ok = false;
                            ++old_use[c & 1];
                        }
#pragma unroll
                        for (int q = 0; q < 8; ++q) {
                            const uint32_t addr = brow + (uint32_t)((q ^ (trow & 7)) << 4);
                            float x0 = aa * __uint_as_float(v[4 * q]), x1 = aa * __uint_as_float(v[4 * q + 1]);
                            float x2 = aa * __uint_as_float(v[4 * q + 2]), x3 = aa * __uint_as_float(v[4 * q + 3]);
                            if (rmw) {
                                uint32_t o0, o1, o2, o3;
                                ptx::ld_shared_v4(addr, o0, o1, o2, o3);
                                x0 = fmaf(bb, __uint_as_float(o0), x0);
                                x1 = fmaf(bb, __uint_as_float(o1), x1);
                                x2 = fmaf(bb, __uint_as_float(o2), x2);
                                x3 = fmaf(bb, __uint_as_float(o3), x3);
                            }
                            ptx::st_shared_v4(addr, __float_as_uint(x0), __float_as_uint(x1), __float_as_uint(x2), __float_as_uint(x3));
                        }
                        ptx::fence_proxy_async_smem();
                        ptx::named_barrier_sync(2, 128);
                        if (leader && !*abort) {
                            ptx::tma_store_2d(map_d, c * 32, row0, buf);
                            ptx::tma_store_commit();
                            if (rmw && c + 2 < nchunks) {
                                ptx::tma_store_wait_read<0>();           // this buffer has been read out: the old chunk after next may land in it
                                request_old(c + 2);
                            }
                        }
                    }
                }
                // this warp has read all it needs from the accumulator: the MMAs of the tile after next may overwrite it
                ptx::tc_fence_before_sync();
                __syncwarp();
                if (lane == 0) {
                    const uint32_t ebar = ptx::smem_addr(&ctl->acc_empty[gt & 1]);
                    if (half == 0) ptx::mbar_arrive(ebar);
                    else ptx::mbar_arrive_cluster(ptx::map_to_cta(ebar, 0u));
                }
            }
        }
        if (leader) ptx::tma_store_wait_all<0>();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::cluster_sync();                    // no CTA leaves while its peer may still arrive on its barriers or read its half of T^T
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc_pair(tmem, tmem_cols);
    }
}

// Host side.  A set: scratch (r x r per job, job and item tables) from the stream-ordered allocator, a memset, one
// table upload, the two kernels, the release of the scratch.  A single matrix: only the r x r scratch; the job
// travels as a kernel parameter.  `jobs` come without T; it is assigned here.
inline flora_status transfer_tc(std::vector<GramJob>& jobs, int r, float a, float b, cudaStream_t st, std::atomic<uint64_t>& launches,
                                const TcMatrix* d_dst_mats = nullptr, const TcMatrix* d_src_mats = nullptr, float* static_T = nullptr,
                                void** release_later = nullptr)
{
    // release_later: the caller frees the call's scratch (stream-ordered) itself, after it has put more work behind the
    // last kernel; nothing then stands between that kernel and the caller's next launch
    if (release_later) *release_later = nullptr;
    if (jobs.empty()) return FLORA_OK;
    int sms = 148, dev = 0;
    cudaGetDevice(&dev);
    cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev);
    // step width: 64 columns, or narrower while that leaves fewer than four steps per SM to balance
    int64_t total_cols = 0;
    int max_n = 1;
    for (const auto& j : jobs) {
        total_cols += j.m;
        max_n = std::max(max_n, j.n);
    }
    int kw = 64;
    while (kw > 16 && total_cols / kw < 4 * (int64_t)sms) kw >>= 1;
    int64_t total_steps = 0;
    for (const auto& j : jobs) total_steps += (j.m + kw - 1) / kw;
    const bool single = jobs.size() == 1;
    // a single matrix: one wave of equal chunks; a set: about three items per SM, the largest first
    // (deterministic mode: one CTA per matrix, so that its r x r product is summed in one fixed order)
    const int64_t chunk = deterministic_flag().load() ? std::max<int64_t>(1, total_steps)
                          : std::max<int64_t>(1, single ? (total_steps + sms - 1) / sms : (total_steps + 3 * sms - 1) / (3 * sms));
    const size_t t_bytes = (((size_t)r * r * sizeof(float)) + 255) & ~(size_t)255;
    const int r_m = (r + 127) & ~127, r_n = (r + 15) & ~15;
    const size_t smem = 2 * (size_t)(r_m + r_n) * 128 + sizeof(GramSmem) + 1024;
    const float scale = 1.0f / sqrtf((float)r);
    const unsigned apply_threads = (unsigned)((r + 31) & ~31);        // fallback kernel: one thread per sketch column
    bool tiled = (r & 3) == 0;                                        // register-tiled kernel: 16-byte aligned rows everywhere
    for (const auto& j : jobs)
        tiled = tiled && (j.ldd & 3) == 0 && (j.lds & 3) == 0 && (reinterpret_cast<uintptr_t>(j.dst) & 15) == 0 &&
                (reinterpret_cast<uintptr_t>(j.src) & 15) == 0;
    // the tensor-core apply kernel: rows addressable by TMA, and descriptors at hand (a set's tables, or, for one
    // matrix, two maps encoded here and passed as kernel parameters)
    const bool single_job = jobs.size() == 1;
    bool tc_apply = tiled && encode_tiled_fn() != nullptr && (single_job || (d_dst_mats && d_src_mats));
    ApplySingle single_arg;
    memset(&single_arg, 0, sizeof(single_arg));
    if (tc_apply && single_job) {
        flora_mat md{jobs[0].dst, jobs[0].n, r, jobs[0].ldd, FLORA_F32}, ms{(void*)jobs[0].src, jobs[0].n, r, jobs[0].lds, FLORA_F32};
        tc_apply = make_map_f32(&single_arg.map_dst, md) && make_map_f32(&single_arg.map_src, ms);
    }
    const bool single_maps = tc_apply && single_job;
    if (tc_apply)                            // the kernel wants T^T as its K-major operand: exchange the roles of the two projections
        for (auto& j : jobs) std::swap(j.seed_old, j.seed_new);
    const int row_groups = tiled ? apply_row_groups(r) : 0;
    const unsigned apply_rows = tiled ? (unsigned)(row_groups * APPLY_RT) : (unsigned)APPLY_ROWS;
    std::vector<uint8_t> tables;                 // set: the job table followed by the item table, one upload
    size_t n_items = 0;
    const size_t jobs_bytes = (jobs.size() * sizeof(GramJob) + 255) & ~(size_t)255;
    if (!single) {
        std::vector<GramItem> items;
        for (size_t i = 0; i < jobs.size(); ++i) {
            const int64_t ks = (jobs[i].m + kw - 1) / kw;
            const int64_t nchunks = std::max<int64_t>(1, (ks + chunk - 1) / chunk);
            const int64_t per = (ks + nchunks - 1) / nchunks;
            for (int64_t k0 = 0; k0 < ks; k0 += per) items.push_back({(int)i, (int)k0, (int)std::min(per, ks - k0), 0});
        }
        std::stable_sort(items.begin(), items.end(), [](const GramItem& x, const GramItem& y) { return x.ksteps > y.ksteps; });
        n_items = items.size();
        tables.resize(jobs_bytes + items.size() * sizeof(GramItem));
        memcpy(tables.data() + jobs_bytes, items.data(), items.size() * sizeof(GramItem));
    }
    // work of the tensor-core apply kernel: pairs of 128-row tiles, dealt in equal runs to the clusters of two CTAs
    int64_t total_pairs = 0;
    for (const auto& j : jobs) total_pairs += (j.n + 255) / 256;
    const int apply_clusters = (int)std::max<int64_t>(1, std::min<int64_t>(sms / 2, total_pairs));
    const int64_t pairs_per_cluster = (total_pairs + apply_clusters - 1) / apply_clusters;
    size_t units_off = 0, slots_off = 0;
    if (tc_apply && !single_maps) {
        std::vector<ApplyUnit> units;
        std::vector<int> slot_begin;
        int64_t left = 0;                                        // pairs the current cluster may still take
        for (size_t i = 0; i < jobs.size(); ++i) {
            int64_t tp = 0, ntp = (jobs[i].n + 255) / 256;
            while (tp < ntp) {
                if (left == 0) {
                    slot_begin.push_back((int)units.size());
                    left = pairs_per_cluster;
                }
                const int64_t take = std::min(left, ntp - tp);
                units.push_back({(int)i, (int)tp, (int)take, 0});
                tp += take;
                left -= take;
            }
        }
        while ((int)slot_begin.size() < apply_clusters + 1) slot_begin.push_back((int)units.size());
        units_off = (tables.size() + 255) & ~(size_t)255;
        slots_off = units_off + ((units.size() * sizeof(ApplyUnit) + 255) & ~(size_t)255);
        tables.resize(slots_off + slot_begin.size() * sizeof(int));
        memcpy(tables.data() + units_off, units.data(), units.size() * sizeof(ApplyUnit));
        memcpy(tables.data() + slots_off, slot_begin.data(), slot_begin.size() * sizeof(int));
    }
    const size_t tables_off = t_bytes * jobs.size();
    uint8_t* buf = nullptr;
    if (static_T) {
        if (!single_job || !tables.empty()) return FLORA_ERR_UNSUPPORTED;      // the fixed scratch serves one matrix, without tables
        buf = reinterpret_cast<uint8_t*>(static_T);
    } else if (scratch_alloc((void**)&buf, tables_off + tables.size(), st) != cudaSuccess) {
        cudaGetLastError();
        return FLORA_ERR_ALLOC;
    }
    for (size_t i = 0; i < jobs.size(); ++i) jobs[i].T = reinterpret_cast<float*>(buf + i * t_bytes);
    flora_status rc = FLORA_OK;
    bool ok = cudaMemsetAsync(buf, 0, tables_off, st) == cudaSuccess;
    auto launch_apply_tc = [&](const GramJob* d_jobs, const ApplyUnit* d_units, const int* d_slots) {
        if (!(single_maps ? raise_smem_limit<apply_tc_kernel<true>>() : raise_smem_limit<apply_tc_kernel<false>>())) return false;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(2 * apply_clusters));
        cfg.blockDim = dim3((unsigned)APPLY_TC_THREADS);
        cfg.dynamicSmemBytes = apply_tc_smem_bytes(r);
        cfg.stream = st;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        cudaError_t e;
        if (single_maps) {
            single_arg.job = jobs[0];
            e = cudaLaunchKernelEx(&cfg, apply_tc_kernel<true>, (const GramJob*)nullptr, (const TcMatrix*)nullptr, (const TcMatrix*)nullptr,
                                   (const ApplyUnit*)nullptr, (const int*)nullptr, single_arg, (int)pairs_per_cluster, r, a, b);
        } else {
            e = cudaLaunchKernelEx(&cfg, apply_tc_kernel<false>, d_jobs, d_dst_mats, d_src_mats, d_units, d_slots, single_arg, 0, r, a, b);
        }
        launches.fetch_add(1, std::memory_order_relaxed);
        return e == cudaSuccess;
    };
    if (tiled)
        ok = ok && (single ? raise_smem_limit<apply_gram_jobs_kernel<true>>() : raise_smem_limit<apply_gram_jobs_kernel<false>>());
    if (single) {
        ok = ok && raise_smem_limit<gram_tc_kernel<true>>();
        if (ok) {
            const int ks = (jobs[0].m + kw - 1) / kw;
            if (ks > 0) {
                gram_tc_kernel<true><<<(unsigned)((ks + chunk - 1) / chunk), GRAM_THREADS, smem, st>>>(nullptr, nullptr, jobs[0], (int)chunk, r, scale, kw);
                launches.fetch_add(1, std::memory_order_relaxed);
            }
            const dim3 grid((unsigned)((max_n + apply_rows - 1) / apply_rows), 1);
            if (tc_apply) {
                ok = launch_apply_tc(nullptr, nullptr, nullptr);
            } else {
                if (tiled) apply_gram_jobs_kernel<true><<<grid, 256, apply_smem_bytes(r), st>>>(nullptr, jobs[0], r, row_groups, a, b);
                else apply_gram_rows_kernel<true><<<grid, apply_threads, 0, st>>>(nullptr, jobs[0], r, a, b);
                launches.fetch_add(1, std::memory_order_relaxed);
            }
        }
    } else {
        memcpy(tables.data(), jobs.data(), jobs.size() * sizeof(GramJob));
        // pageable source: staged by the runtime before the call returns
        ok = ok && cudaMemcpyAsync(buf + tables_off, tables.data(), tables.size(), cudaMemcpyHostToDevice, st) == cudaSuccess &&
             raise_smem_limit<gram_tc_kernel<false>>();
        if (ok) {
            const GramJob* d_jobs = reinterpret_cast<const GramJob*>(buf + tables_off);
            const GramItem* d_items = reinterpret_cast<const GramItem*>(buf + tables_off + jobs_bytes);
            if (n_items) {
                gram_tc_kernel<false><<<(unsigned)n_items, GRAM_THREADS, smem, st>>>(d_jobs, d_items, jobs[0], 0, r, scale, kw);
                launches.fetch_add(1, std::memory_order_relaxed);
            }
            if (tc_apply)
                ok = launch_apply_tc(d_jobs, reinterpret_cast<const ApplyUnit*>(buf + tables_off + units_off),
                                     reinterpret_cast<const int*>(buf + tables_off + slots_off));
            for (size_t begin = 0; begin < jobs.size() && !tc_apply; begin += 65535) {
                dim3 grid((unsigned)((max_n + apply_rows - 1) / apply_rows), (unsigned)std::min<size_t>(65535, jobs.size() - begin));
                if (tiled) apply_gram_jobs_kernel<false><<<grid, 256, apply_smem_bytes(r), st>>>(d_jobs + begin, jobs[0], r, row_groups, a, b);
                else apply_gram_rows_kernel<false><<<grid, apply_threads, 0, st>>>(d_jobs + begin, jobs[0], r, a, b);
                launches.fetch_add(1, std::memory_order_relaxed);
            }
        }
    }
    if (!ok || cudaPeekAtLastError() != cudaSuccess) rc = FLORA_ERR_CUDA;
    if (!static_T) {
        if (release_later) *release_later = buf;
        else if (cudaFreeAsync(buf, st) != cudaSuccess && rc == FLORA_OK) rc = FLORA_ERR_CUDA;
    }
    return rc;
}

}  // namespace flora
