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

namespace flora {

struct GramJob {            // one matrix
    float* T;               // r x r scratch, zeroed before the gram kernel runs
    float* dst;
    const float* src;
    int64_t ldd, lds;
    int32_t n, m;
    uint64_t seed_old, seed_new;
};

struct GramItem {           // one CTA of the gram kernel
    int32_t job;
    int32_t kstep0;         // first step (a step is kw = 16, 32 or 64 columns, the same for the whole launch)
    int32_t ksteps;
    int32_t pad;
};

constexpr int GRAM_GEN_WARPS = 12;
constexpr int GRAM_THREADS = 32 * (1 + GRAM_GEN_WARPS);   // warp 0: MMA issuer, warps 1..12: generators (1-4 also read back)

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

// Host side.  A set: scratch (r x r per job, job and item tables) from the stream-ordered allocator, a memset, one
// table upload, the two kernels, the release of the scratch.  A single matrix: only the r x r scratch; the job
// travels as a kernel parameter.  `jobs` come without T; it is assigned here.
inline flora_status transfer_tc(std::vector<GramJob>& jobs, int r, float a, float b, cudaStream_t st, std::atomic<uint64_t>& launches)
{
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
    const int64_t chunk = std::max<int64_t>(1, single ? (total_steps + sms - 1) / sms : (total_steps + 3 * sms - 1) / (3 * sms));
    const size_t t_bytes = (((size_t)r * r * sizeof(float)) + 255) & ~(size_t)255;
    const int r_m = (r + 127) & ~127, r_n = (r + 15) & ~15;
    const size_t smem = 2 * (size_t)(r_m + r_n) * 128 + sizeof(GramSmem) + 1024;
    const float scale = 1.0f / sqrtf((float)r);
    const unsigned apply_threads = (unsigned)((r + 31) & ~31);        // fallback kernel: one thread per sketch column
    bool tiled = (r & 3) == 0;                                        // register-tiled kernel: 16-byte aligned rows everywhere
    for (const auto& j : jobs)
        tiled = tiled && (j.ldd & 3) == 0 && (j.lds & 3) == 0 && (reinterpret_cast<uintptr_t>(j.dst) & 15) == 0 &&
                (reinterpret_cast<uintptr_t>(j.src) & 15) == 0;
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
    const size_t tables_off = t_bytes * jobs.size();
    uint8_t* buf = nullptr;
    if (scratch_alloc((void**)&buf, tables_off + tables.size(), st) != cudaSuccess) {
        cudaGetLastError();
        return FLORA_ERR_ALLOC;
    }
    for (size_t i = 0; i < jobs.size(); ++i) jobs[i].T = reinterpret_cast<float*>(buf + i * t_bytes);
    flora_status rc = FLORA_OK;
    bool ok = cudaMemsetAsync(buf, 0, tables_off, st) == cudaSuccess;
    if (tiled)
        ok = ok && (single ? cudaFuncSetAttribute(apply_gram_jobs_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)apply_smem_bytes(r))
                           : cudaFuncSetAttribute(apply_gram_jobs_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)apply_smem_bytes(r))) ==
                       cudaSuccess;
    if (single) {
        ok = ok && cudaFuncSetAttribute(gram_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) == cudaSuccess;
        if (ok) {
            const int ks = (jobs[0].m + kw - 1) / kw;
            if (ks > 0) {
                gram_tc_kernel<true><<<(unsigned)((ks + chunk - 1) / chunk), GRAM_THREADS, smem, st>>>(nullptr, nullptr, jobs[0], (int)chunk, r, scale, kw);
                launches.fetch_add(1, std::memory_order_relaxed);
            }
            const dim3 grid((unsigned)((max_n + apply_rows - 1) / apply_rows), 1);
            if (tiled) apply_gram_jobs_kernel<true><<<grid, 256, apply_smem_bytes(r), st>>>(nullptr, jobs[0], r, row_groups, a, b);
            else apply_gram_rows_kernel<true><<<grid, apply_threads, 0, st>>>(nullptr, jobs[0], r, a, b);
            launches.fetch_add(1, std::memory_order_relaxed);
        }
    } else {
        memcpy(tables.data(), jobs.data(), jobs.size() * sizeof(GramJob));
        // pageable source: staged by the runtime before the call returns
        ok = ok && cudaMemcpyAsync(buf + tables_off, tables.data(), tables.size(), cudaMemcpyHostToDevice, st) == cudaSuccess &&
             cudaFuncSetAttribute(gram_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem) == cudaSuccess;
        if (ok) {
            const GramJob* d_jobs = reinterpret_cast<const GramJob*>(buf + tables_off);
            const GramItem* d_items = reinterpret_cast<const GramItem*>(buf + tables_off + jobs_bytes);
            if (n_items) {
                gram_tc_kernel<false><<<(unsigned)n_items, GRAM_THREADS, smem, st>>>(d_jobs, d_items, jobs[0], 0, r, scale, kw);
                launches.fetch_add(1, std::memory_order_relaxed);
            }
            for (size_t begin = 0; begin < jobs.size(); begin += 65535) {
                dim3 grid((unsigned)((max_n + apply_rows - 1) / apply_rows), (unsigned)std::min<size_t>(65535, jobs.size() - begin));
                if (tiled) apply_gram_jobs_kernel<false><<<grid, 256, apply_smem_bytes(r), st>>>(d_jobs + begin, jobs[0], r, row_groups, a, b);
                else apply_gram_rows_kernel<false><<<grid, apply_threads, 0, st>>>(d_jobs + begin, jobs[0], r, a, b);
                launches.fetch_add(1, std::memory_order_relaxed);
            }
        }
    }
    if (!ok || cudaPeekAtLastError() != cudaSuccess) rc = FLORA_ERR_CUDA;
    if (cudaFreeAsync(buf, st) != cudaSuccess && rc == FLORA_OK) rc = FLORA_ERR_CUDA;
    return rc;
}

}  // namespace flora
