// Tensor-core kernels of the path for bf16 matrices (sm_100a: TMA, tcgen05.mma, tensor memory).
//
//   compress_tc_kernel     S <- b S + a G A^T     (Algorithm 1 compression; Algorithm 2 update of M)
//   decompress_tc_kernel   W <- W - step * S A    (Algorithm 1 decompression fused with the update)
//
// The projection A is generated inside the kernels, tile by tile, straight into the shared-memory
// layout the tensor core reads (K-major, 128-byte swizzle); it never exists in global memory.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

#include <algorithm>
#include <atomic>
#include <vector>

#include "../../include/flora.h"
#include "flora_ptx.cuh"
#include "flora_rng.cuh"

namespace flora {

// ------------------------------------------------------------------------------------------------
// device-side tables
// ------------------------------------------------------------------------------------------------
struct alignas(128) TcMatrix {
    CUtensorMap map_g;   // gradient G, box 64 columns x 128 rows, 128-byte swizzle
    CUtensorMap map_w;   // weight W, same box (loads and stores)
    CUtensorMap map_s;   // sketch S (fp32), box 32 columns x 128 rows, 128-byte swizzle
    CUtensorMap map_sb;  // bf16 copy of S (scratch, n x k_pad), box 64 columns x 128 rows, 128-byte swizzle
    __nv_bfloat16* Sb;   // the bf16 copy (used by the decompression kernel for ranks above 64)
    float* S;            // sketch, n x r fp32
    int64_t lds;
    int32_t n, m;
    int32_t pad[24];
};
static_assert(sizeof(TcMatrix) % 128 == 0, "matrix records hold TMA descriptors");

struct K1Item {          // one CTA of the compression kernel
    int32_t mat;         // index into the matrix table
    int32_t row0;        // first row of G / S
    int32_t tiles;       // 128-row tiles handled (1..T)
    int32_t kstep0;      // first 64-column step
    int32_t ksteps;      // number of 64-column steps
    int32_t direct;      // 1: the item covers all columns and owns its rows of S (plain read-modify-write)
                         // 0: several items add into the same rows (atomic adds; S pre-scaled by b)
};

struct K2Item {          // one CTA of the decompression kernel
    int32_t mat;
    int32_t col0;        // first column of the slab (multiple of 128)
    int32_t row0;        // first row
    int32_t tiles;       // 128-row tiles handled
};

constexpr int SEEDS_PER_LAUNCH = 448;
struct SeedTable {
    uint64_t s[SEEDS_PER_LAUNCH];
};

// ------------------------------------------------------------------------------------------------
// compression:  S <- b S + a G A^T
//
// One CTA handles `tiles` (<= T) 128-row tiles of one matrix over `ksteps` steps of 64 columns.
// Per step: the producer thread TMA-loads the G tiles; the generator warps write the matching
// r x 64 tile of A (bf16) into shared memory; one thread issues tiles x 4 MMAs (128 x r_pad x 16)
// that accumulate in tensor memory.  At the end four warps read the accumulators back and update S.
// ------------------------------------------------------------------------------------------------
constexpr int K1_MAX_GEN_WARPS = 16;
constexpr int K1_MAX_THREADS = 64 + 32 * K1_MAX_GEN_WARPS + 32;
// threads of a CTA: producer warp, MMA warp, GW generator warps, one warp that forwards slices to cluster peers
inline int k1_threads(int gen_warps) { return 64 + 32 * gen_warps + 32; }
constexpr int G_TILE_BYTES = 128 * 128;   // 128 rows x 64 bf16
constexpr int S_CHUNK_BYTES_K1 = 128 * 128; // 128 rows x 32 fp32

struct K1Smem {                            // barriers and scalars, placed after the tile ring
    uint64_t full_g[8], full_a[8], slice_ready[8], empty[8], acc_full, old_full[16];
    uint32_t tmem_base;
    int abort;
    int epi_go[4];
};

__global__ void __launch_bounds__(K1_MAX_THREADS, 1)
compress_tc_kernel(const TcMatrix* __restrict__ mats, const K1Item* __restrict__ items, const __grid_constant__ SeedTable seeds,
                   int seed_base, int r, float scale, float a, float b, int T, int stages, int S, int GW, int P, int late_wait)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
    const int r_pad = (r + 15) & ~15;
    const uint32_t a_bytes = (uint32_t)r_pad * 128u;
    const uint32_t stage_bytes = (uint32_t)T * G_TILE_BYTES + a_bytes;
    K1Smem* ctl = reinterpret_cast<K1Smem*>(smem_raw + (smem_base - ptx::smem_addr(smem_raw)) + (size_t)stages * stage_bytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    ptx::grid_launch_dependents();
    const K1Item item = items[blockIdx.x];                    // tables and descriptors are written at set creation, not by kernels
    const TcMatrix* mat = mats + item.mat;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < T * r_pad) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < stages; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->full_g[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->full_a[s]), S > 1 ? 1 : GW / P);   // cluster: one arrival + the peers' bytes
            ptx::mbar_init(ptx::smem_addr(&ctl->slice_ready[s]), GW / P);
            ptx::mbar_init(ptx::smem_addr(&ctl->empty[s]), S);                   // every CTA of the cluster has consumed the stage
        }
        ptx::mbar_init(ptx::smem_addr(&ctl->acc_full), 1);
        for (int k = 0; k < 16; ++k) ptx::mbar_init(ptx::smem_addr(&ctl->old_full[k]), 1);
        ctl->abort = 0;
        for (int k = 0; k < 4; ++k) ctl->epi_go[k] = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async_smem();
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_addr(&ctl->tmem_base), tmem_cols);
        ptx::tmem_relinquish();
    }
    // rows r .. r_pad of every A tile stay zero for the whole kernel
    if (r_pad > r) {
        const int pad_chunks = (r_pad - r) * 8;
        for (int s = 0; s < stages; ++s)
            for (int t = threadIdx.x; t < pad_chunks; t += (int)blockDim.x)
                ptx::st_shared_v4(smem_base + s * stage_bytes + T * G_TILE_BYTES + (uint32_t)r * 128u + t * 16u, 0, 0, 0, 0);
        ptx::fence_proxy_async_smem();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (S > 1) ptx::cluster_sync();       // every CTA's barriers exist before anyone arrives on them remotely
    ptx::tc_fence_after_sync();
    // everything above touched only this CTA's shared and tensor memory; G and S may have been written by the
    // previous kernel of the stream.  `late_wait`: that kernel is this library's own pre-scaling of S, which was
    // itself ordered after everything before it and does not touch G, so only the accesses to S need to wait
    if (!late_wait) ptx::grid_dependency_wait();
    const uint32_t tmem = ctl->tmem_base;
    volatile int* abort = &ctl->abort;
    const uint32_t rank = S > 1 ? ptx::cluster_ctarank() : 0u;

    if (warp == 0) {
        // ------------------------------------------------------------------ TMA producer
        if (lane == 0 && item.tiles > 0) {
            ptx::prefetch_tensormap(&mat->map_g);
            int issued = 0;
            for (int ks = 0; ks < item.ksteps; ++ks) {
                const int s = ks % stages, it = ks / stages;
                if (!(S > 1 ? ptx::mbar_wait_cluster(ptx::smem_addr(&ctl->empty[s]), (it & 1) ^ 1, abort)
                            : ptx::mbar_wait(ptx::smem_addr(&ctl->empty[s]), (it & 1) ^ 1, abort)))
                    break;
                const uint32_t bar = ptx::smem_addr(&ctl->full_g[s]);
                ptx::mbar_arrive_expect_tx(bar, (uint32_t)item.tiles * G_TILE_BYTES);
                for (int t = 0; t < item.tiles; ++t)
                    ptx::tma_load_2d(smem_base + s * stage_bytes + t * G_TILE_BYTES, &mat->map_g, (item.kstep0 + ks) * 64,
                                     item.row0 + t * 128, bar);
                issued = ks + 1;
            }
            if (*abort) {
                // nobody consumes any more: wait (bounded) until the copies still in flight have landed
                for (int ks = max(0, issued - stages); ks < issued; ++ks)
                    ptx::mbar_wait(ptx::smem_addr(&ctl->full_g[ks % stages]), (ks / stages) & 1, abort);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = ptx::umma_idesc_bf16((uint32_t)r_pad);
            const uint64_t desc_base = ptx::umma_desc_k_sw128(smem_base);
            bool ok = true;
            for (int ks = 0; ks < item.ksteps && ok; ++ks) {
                const int s = ks % stages, it = ks / stages;
                ok = (item.tiles == 0 || ptx::mbar_wait(ptx::smem_addr(&ctl->full_g[s]), it & 1, abort)) &&
                     (S > 1 ? ptx::mbar_wait_cluster(ptx::smem_addr(&ctl->full_a[s]), it & 1, abort)
                            : ptx::mbar_wait(ptx::smem_addr(&ctl->full_a[s]), it & 1, abort));
                if (!ok) break;
                ptx::tc_fence_after_sync();
                // descriptors differ from the ring base only in the start-address field (16-byte units)
                const uint64_t dstage = desc_base + (uint64_t)((s * stage_bytes) >> 4);
                const uint64_t da_tile = dstage + (uint64_t)((T * G_TILE_BYTES) >> 4);
                for (int t = 0; t < item.tiles; ++t) {
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        ptx::umma_bf16(tmem + t * r_pad, dstage + (uint64_t)((t * G_TILE_BYTES + kk * 32) >> 4), da_tile + (uint64_t)(kk * 2), idesc,
                                       (ks | kk) != 0);
                }
                // the stage is free once every CTA of the cluster has consumed its copy of the A tile
                const uint32_t ebar = ptx::smem_addr(&ctl->empty[s]);
                if (S == 1) ptx::umma_commit(ebar);
                else if (item.tiles > 0) ptx::umma_commit_cluster(ebar, (uint16_t)((1u << S) - 1u));
                else
                    for (int d = 0; d < S; ++d) ptx::mbar_arrive_cluster(ptx::map_to_cta(ebar, d));   // a CTA without rows consumes nothing
            }
            if (ok && item.tiles > 0) ptx::umma_commit(ptx::smem_addr(&ctl->acc_full));
        }
    } else if (warp == 2 + GW) {
        // ------------------------------------------------------------------ forwarder: this CTA's slice of A to the peers
        if (lane == 0 && S > 1) {
            const uint32_t slice_bytes = (uint32_t)(r_pad / S) * 128u;
            for (int ks = 0; ks < item.ksteps; ++ks) {
                const int s = ks % stages, it = ks / stages;
                if (!ptx::mbar_wait(ptx::smem_addr(&ctl->slice_ready[s]), it & 1, abort)) break;
                const uint32_t fbar = ptx::smem_addr(&ctl->full_a[s]);
                const uint32_t src = smem_base + s * stage_bytes + T * G_TILE_BYTES + rank * slice_bytes;
                ptx::mbar_arrive_expect_tx(fbar, (uint32_t)(S - 1) * slice_bytes);   // own slice is in place; peers' bytes to come
                for (int d = 0; d < S; ++d)
                    if (d != (int)rank) ptx::bulk_copy_to_peer(ptx::map_to_cta(src, d), src, slice_bytes, ptx::map_to_cta(fbar, d));
            }
        }
    } else {
        // ------------------------------------------------------------------ generators, then epilogue
        // The generator warps form P teams; team p writes the tiles of the steps p, p + P, ...: a thread's task (eight
        // values) is a long dependent chain, so with few tasks per thread it is latency, not issue rate, that bounds one
        // tile, and teams working on neighbouring steps at the same time hide it.
        const int team_threads = 32 * (GW / P);
        const int team = (threadIdx.x - 64) / team_threads;
        const int g = (threadIdx.x - 64) - team * team_threads;   // 0 .. team_threads-1
        const PhiloxKey key = make_key(seeds.s[item.mat - seed_base]);
        const int tasks = r * 8;                              // (row j, 16-byte chunk c) pairs of one A tile
        bool ok = true;
        for (int ks = team; ks < item.ksteps && ok; ks += P) {
            const int s = ks % stages, it = ks / stages;
            ok = S > 1 ? ptx::mbar_wait_cluster(ptx::smem_addr(&ctl->empty[s]), (it & 1) ^ 1, abort)
                       : ptx::mbar_wait(ptx::smem_addr(&ctl->empty[s]), (it & 1) ^ 1, abort);
            if (!ok) break;
            const uint32_t a_tile = smem_base + s * stage_bytes + T * G_TILE_BYTES;
            const uint32_t q0 = (uint32_t)(item.kstep0 + ks) * 16u;
            if (S == 1) {
                for (int t = g; t < tasks; t += team_threads) {
                    const int j = t >> 3, c = t & 7;
                    const uint2 lo = projection_quad_bf16(q0 + 2 * c, (uint32_t)j, key, scale);
                    const uint2 hi = projection_quad_bf16(q0 + 2 * c + 1, (uint32_t)j, key, scale);
                    ptx::st_shared_v4(a_tile + j * 128 + ((c ^ (j & 7)) << 4), lo.x, lo.y, hi.x, hi.y);
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->full_a[s]));
            } else {
                // the CTAs of a cluster work on the same columns of the same matrix: each generates the rows
                // [rank, rank+1) * r_pad/S of the tile in its own shared memory; the forwarder warp sends them on
                const int rows_per_cta = r_pad / S;
                const int my_tasks = rows_per_cta * 8;
                for (int t = g; t < my_tasks; t += team_threads) {
                    const int j = (int)rank * rows_per_cta + (t >> 3), c = t & 7;
                    if (j < r) {
                        const uint2 lo = projection_quad_bf16(q0 + 2 * c, (uint32_t)j, key, scale);
                        const uint2 hi = projection_quad_bf16(q0 + 2 * c + 1, (uint32_t)j, key, scale);
                        ptx::st_shared_v4(a_tile + j * 128 + ((c ^ (j & 7)) << 4), lo.x, lo.y, hi.x, hi.y);
                    }
                }
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->slice_ready[s]));
            }
        }
        // Epilogue.  The generator warps, now idle, form groups of four; warp w of a group owns tensor-memory lanes
        // 32*(w%4) .. +31, i.e. those rows of every tile.  The accumulators leave in chunks of 32 columns x 128 rows
        // (16 KB), dealt round-robin to the groups: registers -> shared memory in the 128-byte-swizzled layout of the
        // sketch's tensor map -> one bulk tensor operation per chunk, which the hardware clips at the sketch's last row
        // and column:
        //   add   S <- S + a*acc   (b == 1, or several items share the rows and S was scaled by b beforehand):
        //         a bulk reduction, nothing is read back;
        //   store S <- a*acc       (b == 0 and the item owns its rows);
        //   rmw   S <- b*S + a*acc (the item owns its rows): the old chunk comes in by a bulk load, one chunk ahead.
        // The chunk buffers are the tiles of the ring, which nothing uses once the last MMA has completed.
        const int gw = warp - 2;
        const int slots_per_stage = T + (int)(a_bytes / (uint32_t)G_TILE_BYTES);   // 16 KB areas of one stage
        const int areas = stages * slots_per_stage;
        const int EG = min(min(GW >> 2, 4), areas);               // groups at work
        if (gw < 4 * EG && item.tiles > 0) {
            const int grp = gw >> 2;
            const bool leader = (gw & 3) == 0 && lane == 0;
            const int quarter = warp & 3;
            const int trow = quarter * 32 + lane;                 // row inside a tile
            const uint32_t bar_a = 1u + 2u * (uint32_t)grp, bar_b = bar_a + 1u;
            const bool acc_ok = ok && ptx::mbar_wait(ptx::smem_addr(&ctl->acc_full), 0, abort);
            ptx::tc_fence_after_sync();
            if (late_wait) ptx::grid_dependency_wait();
            const bool add = item.direct == 0 || b == 1.0f;
            const bool rmw = !add && b != 0.0f;
            const int nchunks = (r + 31) >> 5;
            const int total = item.tiles * nchunks;               // chunks of this CTA; the group takes grp, grp + EG, ...
            const int NB = min(areas / EG, 4);                    // buffers of this group
            auto buffer = [&](int u) {                            // u: running index of the group's chunks
                const int k = grp * NB + u % NB;
                return smem_base + (uint32_t)(k / slots_per_stage) * stage_bytes + (uint32_t)(k % slots_per_stage) * G_TILE_BYTES;
            };
            auto wait_reads = [&]() {                             // all but the newest NB-2 stores have been read out of shared memory
                if (NB >= 4) ptx::tma_store_wait_read<2>();
                else if (NB == 3) ptx::tma_store_wait_read<1>();
                else ptx::tma_store_wait_read<0>();
            };
            auto load_old = [&](int u) {
                const int i = grp + u * EG;
                const uint32_t bar = ptx::smem_addr(&ctl->old_full[grp * 4 + u % NB]);
                ptx::mbar_arrive_expect_tx(bar, S_CHUNK_BYTES_K1);
                ptx::tma_load_2d(buffer(u), &mat->map_s, (i % nchunks) * 32, item.row0 + (i / nchunks) * 128, bar);
            };
            const int mine = (total - grp + EG - 1) / EG;
            for (int u = 0; u < mine; ++u) {
                const int i = grp + u * EG;
                if (leader) {
                    const bool go = acc_ok && !*abort;
                    if (go) {
                        wait_reads();
                        if (rmw) {
                            if (u == 0) load_old(0);
                            if (NB > 1 && u + 1 < mine) load_old(u + 1);
                            else if (NB == 1 && u > 0) load_old(u);
                        }
                    }
                    ctl->epi_go[grp] = go ? 1 : 0;
                }
                ptx::named_barrier_sync(bar_a, 128);
                if (!*(volatile int*)&ctl->epi_go[grp]) break;    // uniform: written before the barrier by one thread
                const int t = i / nchunks, c = i % nchunks;
                uint32_t v[32];
                ptx::tmem_ld_16(tmem + ((uint32_t)(quarter * 32) << 16) + t * r_pad + c * 32, *reinterpret_cast<uint32_t(*)[16]>(&v[0]));
                if (c * 32 + 16 < r_pad)
                    ptx::tmem_ld_16(tmem + ((uint32_t)(quarter * 32) << 16) + t * r_pad + c * 32 + 16, *reinterpret_cast<uint32_t(*)[16]>(&v[16]));
                else {
#pragma unroll
                    for (int k = 16; k < 32; ++k) v[k] = 0u;
                }
                ptx::tmem_ld_wait();
                const uint32_t brow = buffer(u) + (uint32_t)trow * 128u;
                if (rmw) ptx::mbar_wait(ptx::smem_addr(&ctl->old_full[grp * 4 + u % NB]), (uint32_t)(u / NB) & 1u, abort);
#pragma unroll
                for (int q = 0; q < 8; ++q) {
                    const uint32_t addr = brow + (uint32_t)((q ^ (trow & 7)) << 4);
                    float x0 = a * __uint_as_float(v[4 * q]), x1 = a * __uint_as_float(v[4 * q + 1]);
                    float x2 = a * __uint_as_float(v[4 * q + 2]), x3 = a * __uint_as_float(v[4 * q + 3]);
                    if (rmw) {
                        uint32_t o0, o1, o2, o3;
                        ptx::ld_shared_v4(addr, o0, o1, o2, o3);
                        x0 = fmaf(b, __uint_as_float(o0), x0);
                        x1 = fmaf(b, __uint_as_float(o1), x1);
                        x2 = fmaf(b, __uint_as_float(o2), x2);
                        x3 = fmaf(b, __uint_as_float(o3), x3);
                    }
                    ptx::st_shared_v4(addr, __float_as_uint(x0), __float_as_uint(x1), __float_as_uint(x2), __float_as_uint(x3));
                }
                ptx::fence_proxy_async_smem();
                ptx::named_barrier_sync(bar_b, 128);
                if (leader && !*abort) {
                    if (add) ptx::tma_reduce_add_2d(&mat->map_s, c * 32, item.row0 + t * 128, buffer(u));
                    else ptx::tma_store_2d(&mat->map_s, c * 32, item.row0 + t * 128, buffer(u));
                    ptx::tma_store_commit();
                }
            }
            if (leader) ptx::tma_store_wait_all<0>();             // the sketch is complete in global memory before the CTA ends
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (S > 1) ptx::cluster_sync();       // no CTA leaves while peers may still store into it or arrive on its barriers
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem, tmem_cols);
    }
}

// ------------------------------------------------------------------------------------------------
// decompression fused with the update:  W <- W - step * S A
//
// Persistent kernel: CTA c processes the work items c, c + gridDim.x, ...  An item is a slab of `bn` (128 or 64)
// columns of one matrix and a run of 128-row tiles.  Per item the generator warps write the r x bn slab of A
// (the N x K operand: bf16 values held in 32-bit containers) into one of two slab buffers, so the slab of the
// next item is generated while the current one streams.  Per row tile: TMA brings the fp32 rows of S in
// 32-column chunks and the W tile into shared memory; one thread issues tf32 MMAs (128 x bn x 8) that read S
// as it is stored, into one of two tensor-memory accumulators; four warps combine the accumulator with the W
// tile in shared memory and a TMA store writes the tile back.  W is read once and written once.
// All rings (W slots, S chunks, accumulators, slabs) run across item boundaries.
// ------------------------------------------------------------------------------------------------
constexpr int K2_FIXED_WARPS = 12;  // warp 0: W loads, 1: MMA, 2-5 and 8-11: combine, 6: S loads, 7: W stores, 12..: slab generators
constexpr int K2_MAX_GEN_WARPS = 8;
constexpr int K2_MAX_THREADS = 32 * (K2_FIXED_WARPS + K2_MAX_GEN_WARPS);
constexpr int K2_MAX_SLOTS = 6;
constexpr int K2_MAX_CSTAGES = 8;
constexpr int W_BOX_BYTES = 128 * 128;     // 128 rows x 64 bf16
constexpr int S_CHUNK_BYTES = 128 * 128;   // 128 rows x 32 fp32

struct K2Smem {
    uint64_t w_full[K2_MAX_SLOTS], w_free[K2_MAX_SLOTS], out_ready[K2_MAX_SLOTS];
    uint64_t c_full[K2_MAX_CSTAGES], c_empty[K2_MAX_CSTAGES], acc_full[2], acc_empty[2], slab_full[2], slab_empty[2];
    uint32_t tmem_base;
    int abort;
};

template <bool BF16S>
__global__ void __launch_bounds__(K2_MAX_THREADS, 1)
decompress_tc_kernel(const TcMatrix* __restrict__ mats, const K2Item* __restrict__ items, int n_items,
                     const __grid_constant__ SeedTable seeds, int seed_base, int r, float scale, float step, int bn, int slots,
                     int cstages, int GW)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
    // K chunks: one 128-byte row of S each (32 fp32 values, or 64 bf16 values when the bf16 copy of S is used)
    const int kchunks = BF16S ? (r + 63) >> 6 : (r + 31) >> 5;
    const int boxes = bn >> 6;                                 // 64-column boxes per W tile
    const uint32_t slab_block = (uint32_t)bn * 128u;           // one K chunk of a slab
    const uint32_t slab_bytes = kchunks * slab_block;
    const uint32_t slab0 = smem_base;
    const uint32_t c_ring = slab0 + 2 * slab_bytes;
    const uint32_t w_ring = c_ring + cstages * (uint32_t)S_CHUNK_BYTES;
    const uint32_t slot_bytes = (uint32_t)boxes * W_BOX_BYTES;
    K2Smem* ctl = reinterpret_cast<K2Smem*>(smem_raw + (w_ring - ptx::smem_addr(smem_raw)) + (size_t)slots * slot_bytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t tmem_cols = 2u * (uint32_t)bn;              // 256 or 128: a power of two >= 32

    if (threadIdx.x == 0) {
        for (int s = 0; s < slots; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->w_full[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->w_free[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->out_ready[s]), 8);
        }
        for (int s = 0; s < cstages; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->c_full[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->c_empty[s]), 1);
        }
        for (int s = 0; s < 2; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->acc_full[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->acc_empty[s]), 8);
            ptx::mbar_init(ptx::smem_addr(&ctl->slab_full[s]), GW);
            ptx::mbar_init(ptx::smem_addr(&ctl->slab_empty[s]), 1);
        }
        ctl->abort = 0;
        ptx::fence_barrier_init();
        ptx::fence_proxy_async_smem();
    }
    if (warp == 1) {
        ptx::tmem_alloc(ptx::smem_addr(&ctl->tmem_base), tmem_cols);
        ptx::tmem_relinquish();
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    ptx::tc_fence_after_sync();
    const uint32_t tmem = ctl->tmem_base;
    volatile int* abort = &ctl->abort;

    if (warp == 0) {
        // ------------------------------------------------------------------ W tile loads
        if (lane == 0) {
            int gt = 0, pending_from = 0;                       // tiles issued so far over all items of this CTA
            bool ok = true;
            for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
                const K2Item item = items[it];
                const TcMatrix* mat = mats + item.mat;
                const int live_boxes = min(boxes, (mat->m - item.col0 + 63) >> 6);
                for (int i = 0; i < item.tiles; ++i, ++gt) {
                    const int s = gt % slots;
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->w_free[s]), ((gt / slots) & 1) ^ 1, abort);
                    if (!ok) break;
                    const uint32_t bar = ptx::smem_addr(&ctl->w_full[s]);
                    ptx::mbar_arrive_expect_tx(bar, (uint32_t)live_boxes * W_BOX_BYTES);
                    for (int bx = 0; bx < live_boxes; ++bx)
                        ptx::tma_load_2d(w_ring + s * slot_bytes + bx * W_BOX_BYTES, &mat->map_w, item.col0 + bx * 64, item.row0 + i * 128, bar);
                }
            }
            if (*abort) {   // loads that nobody consumed: wait (bounded) until they have landed
                pending_from = max(0, gt - slots);
                for (int g = pending_from; g < gt; ++g) ptx::mbar_wait(ptx::smem_addr(&ctl->w_full[g % slots]), (g / slots) & 1, abort);
            }
        }
    } else if (warp == 6) {
        // ------------------------------------------------------------------ S chunk loads (fp32 rows, 32 columns each)
        if (lane == 0) {
            int gc = 0;
            bool ok = true;
            for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
                const K2Item item = items[it];
                const TcMatrix* mat = mats + item.mat;
                for (int c = 0; c < item.tiles * kchunks; ++c, ++gc) {
                    const int s = gc % cstages;
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->c_empty[s]), ((gc / cstages) & 1) ^ 1, abort);
                    if (!ok) break;
                    const uint32_t bar = ptx::smem_addr(&ctl->c_full[s]);
                    ptx::mbar_arrive_expect_tx(bar, S_CHUNK_BYTES);
                    if (BF16S) ptx::tma_load_2d(c_ring + s * S_CHUNK_BYTES, &mat->map_sb, (c % kchunks) * 64, item.row0 + (c / kchunks) * 128, bar);
                    else ptx::tma_load_2d(c_ring + s * S_CHUNK_BYTES, &mat->map_s, (c % kchunks) * 32, item.row0 + (c / kchunks) * 128, bar);
                }
            }
            if (*abort)
                for (int g = max(0, gc - cstages); g < gc; ++g) ptx::mbar_wait(ptx::smem_addr(&ctl->c_full[g % cstages]), (g / cstages) & 1, abort);
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = BF16S ? ptx::umma_idesc_bf16((uint32_t)bn) : ptx::umma_idesc_tf32((uint32_t)bn);
            const uint64_t desc_ring = ptx::umma_desc_k_sw128(c_ring);
            int gt = 0, gc = 0, k = 0;
            bool ok = true;
            for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x, ++k) {
                const K2Item item = items[it];
                const uint64_t desc_slab = ptx::umma_desc_k_sw128(slab0 + (k & 1) * slab_bytes);
                ok = ptx::mbar_wait(ptx::smem_addr(&ctl->slab_full[k & 1]), (k >> 1) & 1, abort);
                for (int i = 0; i < item.tiles && ok; ++i, ++gt) {
                    const uint32_t acc_addr = tmem + (gt & 1) * bn;
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->acc_empty[gt & 1]), ((gt >> 1) & 1) ^ 1, abort);
                    for (int kc = 0; kc < kchunks && ok; ++kc, ++gc) {
                        const int s = gc % cstages;
                        ok = ptx::mbar_wait(ptx::smem_addr(&ctl->c_full[s]), (gc / cstages) & 1, abort);
                        if (!ok) break;
                        ptx::tc_fence_after_sync();
#pragma unroll
                        for (int k8 = 0; k8 < 4; ++k8) {
                            // descriptors differ from the ring / slab base only in the start-address field (16-byte units)
                            const uint64_t da = desc_ring + (uint64_t)((s * S_CHUNK_BYTES + k8 * 32) >> 4);
                            const uint64_t db = desc_slab + (uint64_t)((kc * slab_block + k8 * 32) >> 4);
                            if (BF16S) ptx::umma_bf16(acc_addr, da, db, idesc, (kc | k8) != 0);
                            else ptx::umma_tf32(acc_addr, da, db, idesc, (kc | k8) != 0);
                        }
                        ptx::umma_commit(ptx::smem_addr(&ctl->c_empty[s]));
                    }
                    if (ok) ptx::umma_commit(ptx::smem_addr(&ctl->acc_full[gt & 1]));
                }
                if (ok) ptx::umma_commit(ptx::smem_addr(&ctl->slab_empty[k & 1]));   // every MMA that reads this slab has completed
            }
        }
    } else if (warp == 7) {
        // ------------------------------------------------------------------ W tile stores
        if (lane == 0) {
            int gt = 0;
            bool ok = true;
            const bool lag = slots >= 4;               // with few slots, freeing a slot one tile late costs more than it gains
            for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
                const K2Item item = items[it];
                const TcMatrix* mat = mats + item.mat;
                const int live_boxes = min(boxes, (mat->m - item.col0 + 63) >> 6);
                for (int i = 0; i < item.tiles; ++i, ++gt) {
                    const int s = gt % slots;
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->out_ready[s]), (gt / slots) & 1, abort);
                    if (!ok) break;
                    for (int bx = 0; bx < live_boxes; ++bx)
                        ptx::tma_store_2d(&mat->map_w, item.col0 + bx * 64, item.row0 + i * 128, w_ring + s * slot_bytes + bx * W_BOX_BYTES);
                    ptx::tma_store_commit();
                    if (lag) {
                        // one store stays in flight: wait until all but the newest have read their slot, free that one
                        ptx::tma_store_wait_read<1>();
                        if (gt > 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->w_free[(gt - 1) % slots]));
                    } else {
                        ptx::tma_store_wait_read<0>();          // the slot has been read out: it can be refilled
                        ptx::mbar_arrive(ptx::smem_addr(&ctl->w_free[s]));
                    }
                }
            }
            ptx::tma_store_wait_read<0>();
            if (lag && gt > 0 && ok) ptx::mbar_arrive(ptx::smem_addr(&ctl->w_free[(gt - 1) % slots]));
            ptx::tma_store_wait_all<0>();
        }
    } else if ((warp >= 2 && warp <= 5) || (warp >= 8 && warp <= 11)) {
        // ------------------------------------------------------------------ combine the accumulator with the W tile
        // Eight warps: warp w owns tensor-memory lanes 32*(w%4) .. +31 (rows of the tile); warps 2-5 take the left
        // half of the tile's columns, warps 8-11 the right half.  All accumulator loads of a warp are issued
        // before the first is consumed.
        const int quarter = warp & 3;
        const int half = warp >= 8 ? 1 : 0;
        const int row = quarter * 32 + lane;
        const int per_half = boxes << 1;                       // 16-column chunks per half: 2 (bn 64) or 4 (bn 128)
        int gt = 0;
        bool ok = true;
        for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
            const K2Item item = items[it];
            const int live_chunks = min(boxes, (mats[item.mat].m - item.col0 + 63) >> 6) << 2;
            const int c_begin = half * per_half;
            const int mine = max(0, min(per_half, live_chunks - c_begin));
            for (int i = 0; i < item.tiles; ++i, ++gt) {
                const int s = gt % slots;
                ok = ptx::mbar_wait(ptx::smem_addr(&ctl->acc_full[gt & 1]), (gt >> 1) & 1, abort) &&
                     ptx::mbar_wait(ptx::smem_addr(&ctl->w_full[s]), (gt / slots) & 1, abort);
                if (!ok) break;
                ptx::tc_fence_after_sync();
                const uint32_t wrow = w_ring + s * slot_bytes + row * 128;
                uint32_t acc[4][16];
#pragma unroll
                for (int k = 0; k < 4; ++k)
                    if (k < mine) ptx::tmem_ld_16(tmem + ((uint32_t)(quarter * 32) << 16) + (gt & 1) * bn + (c_begin + k) * 16, acc[k]);
                ptx::tmem_ld_wait();
#pragma unroll
                for (int k = 0; k < 4; ++k) {
                    if (k < mine) {
                        const int c16 = c_begin + k;
                        const uint32_t box = wrow + (c16 >> 2) * W_BOX_BYTES;
#pragma unroll
                        for (int h = 0; h < 2; ++h) {
                            const uint32_t addr = box + (((((c16 & 3) << 1) + h) ^ (row & 7)) << 4);
                            uint32_t x[4];
                            ptx::ld_shared_v4(addr, x[0], x[1], x[2], x[3]);
#pragma unroll
                            for (int u = 0; u < 4; ++u) {
                                const __nv_bfloat162 old = *reinterpret_cast<__nv_bfloat162*>(&x[u]);
                                const float lo = fmaf(-step, __uint_as_float(acc[k][h * 8 + 2 * u]), __low2float(old));
                                const float hi = fmaf(-step, __uint_as_float(acc[k][h * 8 + 2 * u + 1]), __high2float(old));
                                __nv_bfloat162 nw = __floats2bfloat162_rn(lo, hi);
                                x[u] = *reinterpret_cast<uint32_t*>(&nw);
                            }
                            ptx::st_shared_v4(addr, x[0], x[1], x[2], x[3]);
                        }
                    }
                }
                ptx::tc_fence_before_sync();
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) {
                    ptx::mbar_arrive(ptx::smem_addr(&ctl->acc_empty[gt & 1]));
                    ptx::mbar_arrive(ptx::smem_addr(&ctl->out_ready[s]));
                }
            }
        }
    } else {
        // ------------------------------------------------------------------ slab generators
        // Slab of A as the N x K operand: row = column of W, K = index j of the sketch, values rounded to bf16
        // and widened to 32 bits (exact in tf32).  One task makes a 4-column x 4-j block (four Philox blocks) and
        // stores one 16-byte chunk per column; j >= r is written as zero.
        const int g = threadIdx.x - 32 * K2_FIXED_WARPS;
        const int jgroups = kchunks * 8;
        const int tasks = (bn >> 2) * jgroups;
        int k = 0;
        bool ok = true;
        for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x, ++k) {
            const K2Item item = items[it];
            const PhiloxKey key = make_key(seeds.s[item.mat - seed_base]);
            ok = ptx::mbar_wait(ptx::smem_addr(&ctl->slab_empty[k & 1]), ((k >> 1) & 1) ^ 1, abort);
            if (!ok) break;
            const uint32_t slab = slab0 + (k & 1) * slab_bytes;
            for (int t = g; t < tasks; t += 32 * GW) {
                const int jg = t % jgroups, cq = t / jgroups;       // jg: 16-byte chunk along K (4 tf32 or 8 bf16 values)
                const uint32_t blk = slab + (jg >> 3) * slab_block;
                if (BF16S) {
                    uint32_t packed[4][4];
#pragma unroll
                    for (int jj = 0; jj < 8; jj += 2) {
                        float v0[4] = {0.f, 0.f, 0.f, 0.f}, v1[4] = {0.f, 0.f, 0.f, 0.f};
                        const int j = jg * 8 + jj;
                        if (j < r) projection_quad((uint32_t)(item.col0 / 4 + cq), (uint32_t)j, key, scale, v0);
                        if (j + 1 < r) projection_quad((uint32_t)(item.col0 / 4 + cq), (uint32_t)(j + 1), key, scale, v1);
#pragma unroll
                        for (int u = 0; u < 4; ++u) {
                            __nv_bfloat162 pr = __floats2bfloat162_rn(v0[u], v1[u]);
                            packed[u][jj >> 1] = *reinterpret_cast<uint32_t*>(&pr);
                        }
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int c = cq * 4 + u;
                        ptx::st_shared_v4(blk + c * 128 + (((jg & 7) ^ (c & 7)) << 4), packed[u][0], packed[u][1], packed[u][2], packed[u][3]);
                    }
                } else {
                    float v[4][4];
#pragma unroll
                    for (int jj = 0; jj < 4; ++jj) {
                        float q[4] = {0.f, 0.f, 0.f, 0.f};
                        if (jg * 4 + jj < r) projection_quad((uint32_t)(item.col0 / 4 + cq), (uint32_t)(jg * 4 + jj), key, scale, q);
#pragma unroll
                        for (int u = 0; u < 4; ++u) v[u][jj] = bf16_round(q[u]);
                    }
#pragma unroll
                    for (int u = 0; u < 4; ++u) {
                        const int c = cq * 4 + u;
                        ptx::st_shared_v4(blk + c * 128 + (((jg & 7) ^ (c & 7)) << 4), __float_as_uint(v[u][0]), __float_as_uint(v[u][1]),
                                          __float_as_uint(v[u][2]), __float_as_uint(v[u][3]));
                    }
                }
            }
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->slab_full[k & 1]));
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem, tmem_cols);
    }
}

// S <- b S for the listed matrices (those whose rows receive atomic adds from several CTAs); blockIdx.y = list entry.
__global__ void scale_sketches_kernel(const TcMatrix* __restrict__ mats, const int* __restrict__ ids, int r, float b)
{
    ptx::grid_launch_dependents();       // the compression kernel that follows may start streaming G right away
    const TcMatrix* mat = mats + ids[blockIdx.y];
    const int64_t total = (int64_t)mat->n * r;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        float* p = mat->S + (t / r) * mat->lds + (t % r);
        *p = (b == 0.0f) ? 0.0f : *p * b;
    }
}

// bf16 copy of every sketch of the table, n x k_pad with zero padding (the M x K operand of the decompression
// kernel for ranks above 64); blockIdx.y = matrix, one thread per pair of columns.
__global__ void sketch_to_bf16_kernel(const TcMatrix* __restrict__ mats, int r, int k_pad)
{
    const TcMatrix* mat = mats + blockIdx.y;
    const int half = k_pad >> 1;
    const int64_t total = (int64_t)mat->n * half;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x) {
        const int64_t row = t / half;
        const int j = (int)(t % half) * 2;
        const float* src = mat->S + row * mat->lds;
        const float a = j < r ? src[j] : 0.0f, b = j + 1 < r ? src[j + 1] : 0.0f;
        reinterpret_cast<__nv_bfloat162*>(mat->Sb + row * k_pad)[j >> 1] = __floats2bfloat162_rn(a, b);
    }
}

// S <- 0 for every matrix of the table (start of an accumulation cycle); blockIdx.y = matrix.
__global__ void zero_sketches_kernel(const TcMatrix* __restrict__ mats, int r)
{
    const TcMatrix* mat = mats + blockIdx.y;
    const int64_t total = (int64_t)mat->n * r;
    for (int64_t t = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; t < total; t += (int64_t)gridDim.x * blockDim.x)
        mat->S[(t / r) * mat->lds + (t % r)] = 0.0f;
}

// ------------------------------------------------------------------------------------------------
// host side
// ------------------------------------------------------------------------------------------------
struct TcSet {
    bool compress_ready = false;
    bool decompress_ready = false;
    bool transient = false;             // device buffers come from the stream-ordered allocator
    int count = 0, r = 0;
    int T = 1, stages = 2, S = 1, GW = 8, P = 1;
    std::vector<int> k1_launch_first_mat;
    size_t k1_smem = 0;
    TcMatrix* d_mats = nullptr;
    K1Item* d_k1 = nullptr;
    int* d_split = nullptr;
    std::vector<TcMatrix> h_mats;
    std::vector<K1Item> h_k1;
    std::vector<int> k1_launch_begin;   // item ranges per launch (at most SEEDS_PER_LAUNCH matrices each)
    std::vector<int> split_mats;        // matrices whose sketch is updated by several items
    // decompression
    int bn = 128, slots = 2, cstages = 2, k2_gw = 8, k2_grid_max = 148;
    bool k2_bf16 = false;               // ranks above 64: the kernel reads a bf16 copy of the sketches
    __nv_bfloat16* d_sb = nullptr;      // that copy (scratch owned by the set)
    std::vector<int> k2_launch_first_mat;
    size_t k2_smem = 0;
    K2Item* d_k2 = nullptr;
    std::vector<K2Item> h_k2;
    std::vector<int> k2_launch_begin;
};

typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*, const cuuint64_t*,
                                  const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave, CUtensorMapSwizzle,
                                  CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

inline EncodeTiledFn encode_tiled_fn()
{
    static EncodeTiledFn fn = nullptr;
    static bool tried = false;
    if (!tried) {
        tried = true;
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<EncodeTiledFn>(p);
        else
            cudaGetLastError();
    }
    return fn;
}

// bf16 matrix, box = 64 columns x 128 rows, 128-byte swizzle, zero fill outside the matrix
inline bool make_map(CUtensorMap* out, const flora_mat& a)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)a.cols, (cuuint64_t)a.rows};
    cuuint64_t strides[1] = {(cuuint64_t)a.ld * 2};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t estr[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, a.data, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

// fp32 sketch, box = 32 columns x 128 rows, 128-byte swizzle, zero fill outside the matrix
inline bool make_map_f32(CUtensorMap* out, const flora_mat& a)
{
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {(cuuint64_t)a.cols, (cuuint64_t)a.rows};
    cuuint64_t strides[1] = {(cuuint64_t)a.ld * 4};
    cuuint32_t box[2] = {32, 128};
    cuuint32_t estr[2] = {1, 1};
    return fn(out, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, a.data, dims, strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE,
              CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE) == CUDA_SUCCESS;
}

inline bool tc_sketch_ok(const flora_mat& s)
{
    return (reinterpret_cast<uintptr_t>(s.data) & 15) == 0 && (s.ld & 3) == 0 && s.cols >= 1 && s.cols <= 256;
}

inline bool tc_mat_ok(const flora_mat& a)
{
    return a.dtype == FLORA_BF16 && a.rows >= 128 && a.cols >= 64 && (reinterpret_cast<uintptr_t>(a.data) & 15) == 0 &&
           (a.ld & 7) == 0 && a.rows < (1ll << 31) - 256 && a.cols < (1ll << 31) - 256;
}

inline bool tc_compress_supported(const flora_mat* big, const flora_mat* sketch)
{
    return tc_mat_ok(*big) && tc_sketch_ok(*sketch) && encode_tiled_fn() != nullptr;
}

inline int sm_count()
{
    static int n = 0;
    if (!n) {
        int dev = 0;
        cudaGetDevice(&dev);
        cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev);
        if (n <= 0) n = 148;
    }
    return n;
}

constexpr size_t SMEM_BUDGET = 226 * 1024;   // per SM, below the 227 KB limit of sm_100

// Tuning knobs (environment variables, read when a set is planned): they change tile shapes and the
// work split only, never what is computed.
inline int tune_knob(const char* name, int dflt, int lo, int hi)
{
    const char* v = getenv(name);
    if (!v || !*v) return dflt;
    return std::max(lo, std::min(hi, atoi(v)));
}

// Work decomposition of the compression kernel over a set of matrices.
//
// A CTA handles up to T 128-row tiles; S CTAs (a thread-block cluster) handle neighbouring row groups of the
// same matrix over the same columns and share the generation of A.  The generation of one r x 64 tile costs
// about r*64*0.18 ns of one SM's ALUs, the loads of a CTA's T tiles T*0.37 us of its share of HBM: S is chosen
// so that the former stays under half of the latter.
inline void plan_compress(TcSet& set, const std::vector<flora_mat>& G, int r)
{
    const int r_pad = (r + 15) & ~15;
    int64_t max_tiles = 1, total_work = 0;       // work unit: one 128-row tile over one 64-column step
    for (const auto& g : G) {
        const int64_t tiles = (g.rows + 127) / 128, ks = (g.cols + 63) / 64;
        max_tiles = std::max(max_tiles, tiles);
        total_work += tiles * ks;
    }
    // T: bounded by tensor memory (T * r_pad <= 512 columns).  The largest value, unless a smaller one removes
    // more than a fifth of the tile slots that row counts which are no multiple of T * 128 leave empty
    // (empty slots cost MMA issue and shared memory, not HBM traffic).
    // (for r <= 32 at most 3 tiles, so that two CTAs with two stages each fit one SM)
    const int t_cap = (int)std::min<int64_t>(std::min<int64_t>(max_tiles, 512 / r_pad), r_pad <= 32 ? 3 : 4);
    auto padded_work = [&](int cand) {
        double padded = 0;
        for (const auto& g : G) {
            const int64_t tiles = (g.rows + 127) / 128, ks = (g.cols + 63) / 64;
            padded += (double)((tiles + cand - 1) / cand * cand) * ks;
        }
        return padded;
    };
    int T = t_cap;
    for (int cand = t_cap - 1; cand >= 1; --cand)
        if (padded_work(cand) < 0.8 * padded_work(T)) T = cand;
    T = tune_knob("FLORA_K1_T", T, 1, 512 / r_pad);
    const size_t stage = (size_t)T * G_TILE_BYTES + (size_t)r_pad * 128;
    uint32_t cols = 32;
    while ((int)cols < T * r_pad) cols <<= 1;
    // cluster size from the generation / load ratio
    const double ratio = r * 0.045 / T;
    int S = 1;
    while (S < 8 && ratio / S > 0.5) S <<= 1;
    while (S > 1 && (int64_t)S * T > 2 * max_tiles) S >>= 1;         // not more CTAs than there are rows to share
    S = tune_knob("FLORA_K1_CLUSTER", S, 1, 8);
    if (S & (S - 1)) S = 1;
    while (S > 1 && r_pad % (8 * S)) S >>= 1;                     // every CTA's slice of A is whole 8-row groups
    // two CTAs per SM when tensor memory allows it and each still gets two stages: the epilogue of one
    // overlaps the loads of the other (single-CTA clusters only)
    int per_sm = (S == 1 && cols <= 256 && 2 * stage <= SMEM_BUDGET / 2) ? 2 : 1;
    per_sm = tune_knob("FLORA_K1_PER_SM", per_sm, 1, (S == 1 && cols <= 256) ? 2 : 1);
    int stages = (int)std::min<size_t>(8, SMEM_BUDGET / per_sm / stage);
    stages = tune_knob("FLORA_K1_STAGES", stages, 1, std::max(1, stages));
    // generator warps: 16 where one CTA owns the SM and generation is a sizeable share of the work
    int GW = (per_sm == 1 && ratio / S > 0.15) ? 16 : 8;
    GW = tune_knob("FLORA_K1_GEN_WARPS", GW, 4, per_sm == 1 ? K1_MAX_GEN_WARPS : 8);
    set.GW = GW;
    // generator teams: as many as keep every thread of a team busy with at least one task per tile
    {
        const int tile_tasks = (S > 1 ? r_pad / S : r) * 8;
        int P = 1;
        while (2 * P <= stages && GW % (2 * P) == 0 && 32 * GW / (2 * P) >= tile_tasks) P *= 2;
        P = tune_knob("FLORA_K1_TEAMS", P, 1, 8);
        while (P > 1 && (GW % P || P > stages || (P & (P - 1)))) --P;
        set.P = P;
    }
    set.T = T;
    set.S = S;
    set.stages = stages;
    set.k1_smem = (size_t)stages * stage + sizeof(K1Smem) + 1024;
    // column chunks: aim at about `waves` items per slot (a slot is a CTA, or a cluster), at least 8 steps each
    int64_t slots = std::max<int64_t>(1, (int64_t)sm_count() * per_sm / S);
    cudaFuncSetAttribute(compress_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)set.k1_smem);
    if (S > 1) {
        // clusters that can be resident at once (fewer than SMs / S: a cluster must sit inside one GPC)
        cudaFuncSetAttribute(compress_tc_kernel, cudaFuncAttributeNonPortableClusterSizeAllowed, 0);
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(S * 64));
        cfg.blockDim = dim3((unsigned)k1_threads(set.GW));
        cfg.dynamicSmemBytes = set.k1_smem;
        cudaLaunchAttribute attr[1];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = (unsigned)S;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = 1;
        int active = 0;
        if (cudaOccupancyMaxActiveClusters(&active, compress_tc_kernel, &cfg) == cudaSuccess && active > 0) slots = active;
        else cudaGetLastError();
    }
    const int64_t group_tiles = (int64_t)S * T;                      // rows of one slot, in tiles
    struct Unit { int mat; int64_t tile0, tiles, kstep0, ksteps; bool direct; };
    auto build_units = [&](int64_t target, std::vector<Unit>& units, std::vector<int>& split) {
        units.clear();
        split.clear();
        for (size_t i = 0; i < G.size(); ++i) {
            const auto& g = G[i];
            if (g.rows == 0 || g.cols == 0) continue;
            const int64_t tiles = (g.rows + 127) / 128, ks = (g.cols + 63) / 64;
            const int64_t groups = (tiles + group_tiles - 1) / group_tiles;
            const int64_t per_group = (tiles + groups - 1) / groups;     // rows spread evenly over the groups
            int64_t chunk = std::max<int64_t>(8, target / per_group);
            int64_t nchunks = (ks + chunk - 1) / chunk;
            if (nchunks > 1 && ks - (nchunks - 1) * chunk < chunk / 2) --nchunks;    // no short tail item
            chunk = (ks + nchunks - 1) / nchunks;
            nchunks = (ks + chunk - 1) / chunk;
            if (nchunks > 1) split.push_back((int)i);
            for (int64_t t0 = 0; t0 < tiles; t0 += per_group)
                for (int64_t c = 0; c < nchunks; ++c)
                    units.push_back({(int)i, t0, std::min(per_group, tiles - t0), c * chunk, std::min(chunk, ks - c * chunk), nchunks == 1});
        }
    };
    // time of a unit on its slot, in 64-column steps of a full slot: a fixed start-up / epilogue cost plus its steps,
    // scaled by the rows a CTA streams (a cluster moves in lockstep, so its most loaded CTA counts)
    auto unit_time = [&](const Unit& u) {
        const double per_cta = (double)((u.tiles + S - 1) / S);
        return (6.0 + (double)u.ksteps) * std::max(per_cta, 0.5 * T);
    };
    auto makespan = [&](const std::vector<Unit>& units) {
        std::vector<double> tms;
        for (const auto& u : units) tms.push_back(unit_time(u));
        std::sort(tms.begin(), tms.end(), std::greater<double>());
        std::vector<double> free_at((size_t)slots, 0.0);     // min-heap of slot availability
        auto cmp = std::greater<double>();
        for (double t : tms) {
            std::pop_heap(free_at.begin(), free_at.end(), cmp);
            free_at.back() += t;
            std::push_heap(free_at.begin(), free_at.end(), cmp);
        }
        return *std::max_element(free_at.begin(), free_at.end());
    };
    // column chunks: try several granularities (about 1..4 units per slot) and keep the shortest schedule
    std::vector<Unit> units, cand_units;
    std::vector<int> cand_split;
    double best_span = 1e300;
    const int fixed_waves = tune_knob("FLORA_K1_WAVES", 0, 0, 64);
    for (int w = 1; w <= 4; ++w) {
        for (double f : {1.0, 1.1, 1.2, 1.35, 1.5}) {
            if (fixed_waves && (w != fixed_waves || f != 1.0)) continue;
            const int64_t target = (int64_t)((double)total_work / (double)((fixed_waves ? fixed_waves : w) * slots) * f) + 1;
            build_units(target, cand_units, cand_split);
            const double span = makespan(cand_units);
            if (span < best_span * 0.98) {
                best_span = span;
                units = cand_units;
                set.split_mats = cand_split;
            }
        }
    }
    // a schedule without any split over columns is preferred when it is nearly as short: every row of a sketch then
    // has one owner, so a momentum update needs neither the pre-scaling pass nor atomic adds
    if (!fixed_waves) {
        build_units((int64_t)1 << 60, cand_units, cand_split);
        if (makespan(cand_units) <= 1.12 * best_span) {
            units = cand_units;
            set.split_mats = cand_split;
        }
    }
    // launches cover at most SEEDS_PER_LAUNCH consecutive matrices; inside a launch the largest units go first
    set.h_k1.clear();
    set.k1_launch_begin.clear();
    set.k1_launch_first_mat.clear();
    size_t u0 = 0;
    while (u0 < units.size()) {
        size_t u1 = u0;
        while (u1 < units.size() && units[u1].mat < units[u0].mat + SEEDS_PER_LAUNCH) ++u1;
        const int first_mat = units[u0].mat;          // before sorting: units are still in matrix order here
        if (tune_knob("FLORA_K1_SORT", 1, 0, 1))
            std::stable_sort(units.begin() + u0, units.begin() + u1,
                             [](const Unit& x, const Unit& y) { return x.tiles * x.ksteps > y.tiles * y.ksteps; });
        set.k1_launch_begin.push_back((int)set.h_k1.size());
        set.k1_launch_first_mat.push_back(first_mat);
        for (size_t u = u0; u < u1; ++u) {
            // the unit's tiles spread evenly over the S CTAs of the slot (some may get none)
            const Unit& un = units[u];
            int64_t t0 = un.tile0;
            for (int c = 0; c < S; ++c) {
                const int64_t left = un.tile0 + un.tiles - t0;
                const int64_t mine = std::min<int64_t>(T, (left + (S - c) - 1) / (S - c));
                K1Item it;
                it.mat = un.mat;
                it.row0 = (int)(t0 * 128);
                it.tiles = (int)std::max<int64_t>(0, mine);
                it.kstep0 = (int)un.kstep0;
                it.ksteps = (int)un.ksteps;
                it.direct = un.direct;
                set.h_k1.push_back(it);
                t0 += it.tiles;
            }
        }
        u0 = u1;
    }
    set.k1_launch_begin.push_back((int)set.h_k1.size());
}

// Work decomposition of the decompression kernel: column slabs of bn columns, cut into runs of row tiles; the
// persistent CTAs take the items round-robin, largest first.
inline void plan_decompress(TcSet& set, const std::vector<flora_mat>& W, int r)
{
    // ranks up to 64 read the fp32 sketch directly (tf32 MMA); above that the bytes of S that a CTA pulls per W
    // tile exceed what shared memory can keep in flight, so a bf16 copy of S is made first (half the bytes,
    // twice the K depth per 128-byte row) and the MMA runs in bf16
    const bool bf16s = tune_knob("FLORA_K2_BF16S", r > 64 ? 1 : 0, 0, 1) != 0;
    set.k2_bf16 = bf16s;
    const int kchunks = bf16s ? (r + 63) / 64 : (r + 31) / 32;
    // slabs of 128 columns (every chunk of S then serves twice the columns of W) whenever two slabs, two W slots and
    // two S chunks of that width fit; 64 columns otherwise
    const size_t ctl = sizeof(K2Smem) + 1024;
    int bn = (2 * (size_t)kchunks * 128 * 128 + 2 * S_CHUNK_BYTES + 2 * 2 * (size_t)W_BOX_BYTES + ctl <= SMEM_BUDGET) ? 128 : 64;
    bn = tune_knob("FLORA_K2_BN", bn, 64, 128) >= 128 ? 128 : 64;
    const size_t slab_bytes = (size_t)kchunks * bn * 128, slot = (size_t)(bn / 64) * W_BOX_BYTES;
    // two CTAs per SM when two of them fit (each with two slabs, two W slots and one S chunk)
    const size_t per_cta_max = 113 * 1024;                       // half of an SM's shared memory minus the reserve
    int per_sm = (2 * slab_bytes + S_CHUNK_BYTES + 2 * slot + ctl <= per_cta_max) ? 2 : 1;
    per_sm = 1;   // twelve fixed warps plus generators: one CTA per SM
    const size_t budget = (per_sm == 2 ? per_cta_max : SMEM_BUDGET) - ctl - 2 * slab_bytes;
    int cstages = std::max(2, std::min(kchunks + 1, 4));
    cstages = tune_knob("FLORA_K2_CSTAGES", cstages, 1, K2_MAX_CSTAGES);
    while (cstages > 1 && (size_t)cstages * S_CHUNK_BYTES + 2 * slot > budget) --cstages;
    int slots = (int)std::min<size_t>(K2_MAX_SLOTS, (budget - (size_t)cstages * S_CHUNK_BYTES) / slot);
    slots = tune_knob("FLORA_K2_SLOTS", slots, 1, std::max(1, slots));
    int GW = 8;
    GW = tune_knob("FLORA_K2_GEN_WARPS", GW, 1, K2_MAX_GEN_WARPS);
    set.bn = bn;
    set.slots = slots;
    set.cstages = cstages;
    set.k2_gw = GW;
    set.k2_smem = 2 * slab_bytes + (size_t)cstages * S_CHUNK_BYTES + (size_t)slots * slot + sizeof(K2Smem) + 1024;
    const int grid_max = sm_count() * per_sm;
    // cost model (microseconds of one SM): a tile streams bn*128*4 bytes at the SM's share of HBM; a slab costs
    // r*bn normals at the generator warps' rate and overlaps the previous item's streaming
    // (an SM takes in about 60 GB/s whatever the source: the chunks of S count like the W tile itself)
    const double t_tile = std::max((double)bn * 128 * 4 / (6.5e6 / sm_count()),
                                   ((double)bn * 128 * 2 + (double)kchunks * S_CHUNK_BYTES) / 60e3);
    const double t_slab = (double)r * bn / (GW >= 8 ? 2000.0 : 1300.0);   // generator warps share the SM with the streaming warps
    auto build = [&](int run, std::vector<K2Item>& out) {
        out.clear();
        for (size_t i = 0; i < W.size(); ++i) {
            const auto& w = W[i];
            if (w.rows == 0 || w.cols == 0) continue;
            const int64_t rtiles = (w.rows + 127) / 128, slabs = (w.cols + bn - 1) / bn;
            const int64_t groups = (rtiles + run - 1) / run;
            const int64_t per = (rtiles + groups - 1) / groups;
            for (int64_t sl = 0; sl < slabs; ++sl)
                for (int64_t t0 = 0; t0 < rtiles; t0 += per) {
                    K2Item it;
                    it.mat = (int)i;
                    it.col0 = (int)(sl * bn);
                    it.row0 = (int)(t0 * 128);
                    it.tiles = (int)std::min<int64_t>(per, rtiles - t0);
                    out.push_back(it);
                }
        }
    };
    auto sort_items = [&](std::vector<K2Item>& v, size_t b0, size_t b1) {
        std::stable_sort(v.begin() + b0, v.begin() + b1, [](const K2Item& x, const K2Item& y) { return x.tiles > y.tiles; });
    };
    auto makespan = [&](const std::vector<K2Item>& v) {
        const int grid = (int)std::min<size_t>(grid_max, v.size());
        std::vector<K2Item> sorted = v;
        sort_items(sorted, 0, sorted.size());
        std::vector<double> t((size_t)std::max(grid, 1), 0.0);
        for (size_t k = 0; k < sorted.size(); ++k) {
            // generation overlaps the streaming of the previous item, but the two compete for issue slots
            const double stream = sorted[k].tiles * t_tile;
            t[k % t.size()] += std::max(t_slab, stream) + 0.35 * std::min(t_slab, stream) + 0.2;
        }
        return *std::max_element(t.begin(), t.end());
    };
    const int fixed_run = tune_knob("FLORA_K2_TILES", 0, 0, 1 << 20);
    std::vector<K2Item> cand;
    double best = 1e300;
    for (int run : {1 << 20, 48, 32, 24, 16, 12, 11, 8, 6, 4, 3, 2}) {
        if (fixed_run && run != (1 << 20)) continue;
        build(fixed_run ? fixed_run : run, cand);
        const double span = makespan(cand);
        if (span < best * 0.97) {
            best = span;
            set.h_k2 = cand;
        }
    }
    // launches cover at most SEEDS_PER_LAUNCH consecutive matrices; inside a launch the largest items go first
    set.k2_launch_begin.clear();
    set.k2_launch_first_mat.clear();
    size_t u0 = 0;
    while (u0 < set.h_k2.size()) {
        size_t u1 = u0;
        while (u1 < set.h_k2.size() && set.h_k2[u1].mat < set.h_k2[u0].mat + SEEDS_PER_LAUNCH) ++u1;
        set.k2_launch_begin.push_back((int)u0);
        set.k2_launch_first_mat.push_back(set.h_k2[u0].mat);
        sort_items(set.h_k2, u0, u1);
        u0 = u1;
    }
    set.k2_launch_begin.push_back((int)set.h_k2.size());
    set.k2_grid_max = grid_max;
}

inline void tc_set_free_stream(TcSet& s, cudaStream_t st)
{
    if (s.transient) {
        if (s.d_mats) cudaFreeAsync(s.d_mats, st);
        if (s.d_k1) cudaFreeAsync(s.d_k1, st);
        if (s.d_k2) cudaFreeAsync(s.d_k2, st);
        if (s.d_split) cudaFreeAsync(s.d_split, st);
        if (s.d_sb) cudaFreeAsync(s.d_sb, st);
    } else {
        if (s.d_mats) cudaFree(s.d_mats);
        if (s.d_k1) cudaFree(s.d_k1);
        if (s.d_k2) cudaFree(s.d_k2);
        if (s.d_split) cudaFree(s.d_split);
        if (s.d_sb) cudaFree(s.d_sb);
    }
    s.d_mats = nullptr;
    s.d_k1 = nullptr;
    s.d_k2 = nullptr;
    s.d_split = nullptr;
    s.d_sb = nullptr;
    s.compress_ready = s.decompress_ready = false;
}
inline void tc_set_free(TcSet& s) { tc_set_free_stream(s, nullptr); }

template <typename T>
inline flora_status upload(T** dst, const std::vector<T>& src, bool transient, cudaStream_t st)
{
    if (src.empty()) return FLORA_OK;
    const size_t bytes = src.size() * sizeof(T);
    if (!*dst) {
        cudaError_t e = transient ? cudaMallocAsync((void**)dst, bytes, st) : cudaMalloc((void**)dst, bytes);
        if (e != cudaSuccess) {
            cudaGetLastError();
            return FLORA_ERR_ALLOC;
        }
    }
    // pageable source: the runtime stages it before returning, so the vector may change afterwards
    if (cudaMemcpyAsync(*dst, src.data(), bytes, cudaMemcpyHostToDevice, st) != cudaSuccess) return FLORA_ERR_CUDA;
    return FLORA_OK;
}

inline flora_status tc_fill_matrices(TcSet& set, const std::vector<flora_mat>& G, const std::vector<flora_mat>& W,
                                     const std::vector<flora_mat>& S)
{
    set.h_mats.assign(S.size(), TcMatrix());
    for (size_t i = 0; i < S.size(); ++i) {
        TcMatrix& tm = set.h_mats[i];
        memset(&tm, 0, sizeof(tm));
        tm.S = (float*)S[i].data;
        tm.lds = S[i].ld;
        const flora_mat& big = !G.empty() ? G[i] : W[i];
        tm.n = (int32_t)big.rows;
        tm.m = (int32_t)big.cols;
        if (!G.empty() && G[i].rows && G[i].cols && !make_map(&tm.map_g, G[i])) return FLORA_ERR_CUDA;
        if (!W.empty() && W[i].rows && W[i].cols && !make_map(&tm.map_w, W[i])) return FLORA_ERR_CUDA;
        if (S[i].rows && S[i].cols && !make_map_f32(&tm.map_s, S[i])) return FLORA_ERR_CUDA;
    }
    return FLORA_OK;
}

// Builds the tensor-core side of a set; leaves it "not ready" (SIMT kernels are used) if any matrix is not eligible.
inline flora_status tc_set_build_on(TcSet& set, const std::vector<flora_mat>& G, const std::vector<flora_mat>& W,
                                    const std::vector<flora_mat>& S, bool transient, cudaStream_t st)
{
    set.transient = transient;
    set.count = (int)S.size();
    if (S.empty() || !encode_tiled_fn()) return FLORA_OK;
    set.r = (int)S[0].cols;
    bool g_ok = !G.empty(), w_ok = !W.empty();
    for (size_t i = 0; i < S.size(); ++i) {
        if (!G.empty() && !tc_mat_ok(G[i])) g_ok = false;
        if (!W.empty() && (!tc_mat_ok(W[i]) || !tc_sketch_ok(S[i]))) w_ok = false;
    }
    if (!g_ok && !w_ok) return FLORA_OK;
    std::vector<flora_mat> none;
    flora_status rc = tc_fill_matrices(set, g_ok ? G : none, w_ok ? W : none, S);
    if (rc) return rc;
    if (w_ok) {
        plan_decompress(set, W, set.r);
        if (set.k2_bf16) {
            // scratch for the bf16 copies of the sketches: n x k_pad each, 1 KB aligned
            const int k_pad = (set.r + 63) & ~63;
            size_t total = 0;
            std::vector<size_t> offset(S.size());
            for (size_t i = 0; i < S.size(); ++i) {
                offset[i] = total;
                total += (((size_t)S[i].rows * k_pad * 2) + 1023) & ~(size_t)1023;
            }
            if (total) {
                cudaError_t e = transient ? cudaMallocAsync((void**)&set.d_sb, total, st) : cudaMalloc((void**)&set.d_sb, total);
                if (e != cudaSuccess) {
                    cudaGetLastError();
                    return FLORA_ERR_ALLOC;
                }
            }
            for (size_t i = 0; i < S.size(); ++i) {
                if (S[i].rows == 0) continue;
                TcMatrix& tm = set.h_mats[i];
                tm.Sb = reinterpret_cast<__nv_bfloat16*>(reinterpret_cast<uint8_t*>(set.d_sb) + offset[i]);
                flora_mat sb;
                sb.data = tm.Sb;
                sb.rows = S[i].rows;
                sb.cols = k_pad;
                sb.ld = k_pad;
                sb.dtype = FLORA_BF16;
                if (!make_map(&tm.map_sb, sb)) return FLORA_ERR_CUDA;
            }
        }
    }
    rc = upload(&set.d_mats, set.h_mats, transient, st);
    if (rc) return rc;
    if (g_ok) {
        plan_compress(set, G, set.r);
        rc = upload(&set.d_k1, set.h_k1, transient, st);
        if (rc) return rc;
        rc = upload(&set.d_split, set.split_mats, transient, st);
        if (rc) return rc;
        if (cudaFuncSetAttribute(compress_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)set.k1_smem) != cudaSuccess)
            return FLORA_ERR_CUDA;
        set.compress_ready = true;
    }
    if (w_ok) {
        rc = upload(&set.d_k2, set.h_k2, transient, st);
        if (rc) return rc;
        cudaError_t e = set.k2_bf16 ? cudaFuncSetAttribute(decompress_tc_kernel<true>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)set.k2_smem)
                                    : cudaFuncSetAttribute(decompress_tc_kernel<false>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)set.k2_smem);
        if (e != cudaSuccess) return FLORA_ERR_CUDA;
        set.decompress_ready = true;
    }
    return FLORA_OK;
}

inline flora_status tc_set_build(TcSet& set, const std::vector<flora_mat>& G, const std::vector<flora_mat>& W,
                                 const std::vector<flora_mat>& S)
{
    return tc_set_build_on(set, G, W, S, false, nullptr);
}

// New gradient pointers, same shapes: only the tensor maps change.
inline flora_status tc_set_rebind(TcSet& set, const std::vector<flora_mat>& G, cudaStream_t st)
{
    if (!set.compress_ready) return FLORA_OK;
    for (size_t i = 0; i < G.size(); ++i) {
        if (!tc_mat_ok(G[i])) return FLORA_ERR_ALIGN;
        if (G[i].rows && G[i].cols && !make_map(&set.h_mats[i].map_g, G[i])) return FLORA_ERR_CUDA;
    }
    return upload(&set.d_mats, set.h_mats, false, st);
}

// Blocks per matrix for the element-wise helper kernels (zero, scale): about four elements per thread of the
// largest sketch.
inline unsigned helper_blocks(const TcSet& set)
{
    int64_t most = 1;
    for (const auto& tm : set.h_mats) most = std::max<int64_t>(most, (int64_t)tm.n * set.r);
    return (unsigned)std::min<int64_t>(1024, (most + 1023) / 1024);
}

inline flora_status tc_set_compress(TcSet& set, const uint64_t* seeds, float a, float b, cudaStream_t st,
                                    std::atomic<uint64_t>& launches)
{
    const int r = set.r;
    const float scale = 1.0f / sqrtf((float)r);
    int late_wait = 0;
    if (b != 1.0f && !set.split_mats.empty()) {
        late_wait = tune_knob("FLORA_PDL", 1, 0, 1);
        // rows updated by several CTAs receive atomic adds: scale them by b first
        for (size_t begin = 0; begin < set.split_mats.size(); begin += 65535) {
            const size_t jobs_here = std::min<size_t>(65535, set.split_mats.size() - begin);
            // few enough blocks to be resident at once: the compression kernel may only start once all have started
            dim3 grid((unsigned)std::max<size_t>(1, std::min<size_t>(helper_blocks(set), (size_t)sm_count() * 6 / jobs_here)), (unsigned)jobs_here);
            scale_sketches_kernel<<<grid, 256, 0, st>>>(set.d_mats, set.d_split + begin, r, b);
            launches.fetch_add(1, std::memory_order_relaxed);
        }
    }
    for (size_t l = 0; l + 1 < set.k1_launch_begin.size(); ++l) {
        const int begin = set.k1_launch_begin[l], end = set.k1_launch_begin[l + 1];
        if (end == begin) continue;
        const int seed_base = set.k1_launch_first_mat[l];
        SeedTable table;
        for (int i = 0; i < SEEDS_PER_LAUNCH; ++i) table.s[i] = seed_base + i < set.count ? seeds[seed_base + i] : 0;
        cudaLaunchConfig_t cfg = {};
        cfg.gridDim = dim3((unsigned)(end - begin));
        cfg.blockDim = dim3((unsigned)k1_threads(set.GW));
        cfg.dynamicSmemBytes = set.k1_smem;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;     // the kernel waits for its predecessor itself
        attr[0].val.programmaticStreamSerializationAllowed = tune_knob("FLORA_PDL", 1, 0, 1);
        attr[1].id = cudaLaunchAttributeClusterDimension;
        attr[1].val.clusterDim.x = (unsigned)set.S;
        attr[1].val.clusterDim.y = 1;
        attr[1].val.clusterDim.z = 1;
        cfg.attrs = attr;
        cfg.numAttrs = set.S > 1 ? 2 : 1;
        const TcMatrix* mats = set.d_mats;
        const K1Item* items = set.d_k1 + begin;
        if (cudaLaunchKernelEx(&cfg, compress_tc_kernel, mats, items, table, seed_base, r, scale, a, b, set.T, set.stages, set.S, set.GW, set.P, l == 0 ? late_wait : 0) !=
            cudaSuccess)
            return FLORA_ERR_CUDA;
        launches.fetch_add(1, std::memory_order_relaxed);
    }
    return cudaPeekAtLastError() == cudaSuccess ? FLORA_OK : FLORA_ERR_CUDA;
}

inline flora_status tc_compress_single(const flora_mat* G, flora_mat* S, uint64_t seed, float a, float b, cudaStream_t st,
                                       std::atomic<uint64_t>& launches)
{
    TcSet set;
    std::vector<flora_mat> g(1, *G), s(1, *S), none;
    flora_status rc = tc_set_build_on(set, g, none, s, true, st);
    if (rc == FLORA_OK) rc = set.compress_ready ? tc_set_compress(set, &seed, a, b, st, launches) : FLORA_ERR_UNSUPPORTED;
    tc_set_free_stream(set, st);
    return rc;
}

inline flora_status tc_set_decompress(TcSet& set, const uint64_t* seeds, float step, cudaStream_t st,
                                      std::atomic<uint64_t>& launches)
{
    const int r = set.r;
    const float scale = 1.0f / sqrtf((float)r);
    if (set.k2_bf16) {
        const int k_pad = (r + 63) & ~63;
        int max_rows = 1;
        for (const auto& tm : set.h_mats) max_rows = std::max(max_rows, tm.n);
        const unsigned bx = (unsigned)std::min<int64_t>(1024, ((int64_t)max_rows * (k_pad / 2) + 1023) / 1024);   // ~4 pairs per thread
        for (int begin = 0; begin < set.count; begin += 65535) {
            dim3 grid(bx, (unsigned)std::min(65535, set.count - begin));
            sketch_to_bf16_kernel<<<grid, 256, 0, st>>>(set.d_mats + begin, r, k_pad);
            launches.fetch_add(1, std::memory_order_relaxed);
        }
    }
    for (size_t l = 0; l + 1 < set.k2_launch_begin.size(); ++l) {
        const int begin = set.k2_launch_begin[l], end = set.k2_launch_begin[l + 1];
        if (end == begin) continue;
        const int seed_base = set.k2_launch_first_mat[l];
        SeedTable table;
        for (int i = 0; i < SEEDS_PER_LAUNCH; ++i) table.s[i] = seed_base + i < set.count ? seeds[seed_base + i] : 0;
        const int grid = std::min(set.k2_grid_max, end - begin);
        if (set.k2_bf16)
            decompress_tc_kernel<true><<<grid, 32 * (K2_FIXED_WARPS + set.k2_gw), set.k2_smem, st>>>(
                set.d_mats, set.d_k2 + begin, end - begin, table, seed_base, r, scale, step, set.bn, set.slots, set.cstages, set.k2_gw);
        else
            decompress_tc_kernel<false><<<grid, 32 * (K2_FIXED_WARPS + set.k2_gw), set.k2_smem, st>>>(
                set.d_mats, set.d_k2 + begin, end - begin, table, seed_base, r, scale, step, set.bn, set.slots, set.cstages, set.k2_gw);
        launches.fetch_add(1, std::memory_order_relaxed);
    }
    return cudaPeekAtLastError() == cudaSuccess ? FLORA_OK : FLORA_ERR_CUDA;
}

inline flora_status tc_decompress_single(flora_mat* W, const flora_mat* S, uint64_t seed, float step, cudaStream_t st,
                                         std::atomic<uint64_t>& launches)
{
    TcSet set;
    std::vector<flora_mat> w(1, *W), s(1, *S), none;
    flora_status rc = tc_set_build_on(set, none, w, s, true, st);
    if (rc == FLORA_OK) rc = set.decompress_ready ? tc_set_decompress(set, &seed, step, st, launches) : FLORA_ERR_UNSUPPORTED;
    tc_set_free_stream(set, st);
    return rc;
}

inline bool tc_decompress_supported(const flora_mat* big, const flora_mat* sketch)
{
    return tc_mat_ok(*big) && tc_sketch_ok(*sketch) && encode_tiled_fn() != nullptr;
}

inline flora_status tc_set_zero(TcSet& set, cudaStream_t st, std::atomic<uint64_t>& launches)
{
    for (int begin = 0; begin < set.count; begin += 65535) {
        dim3 grid(helper_blocks(set), (unsigned)std::min(65535, set.count - begin));
        zero_sketches_kernel<<<grid, 256, 0, st>>>(set.d_mats + begin, set.r);
        launches.fetch_add(1, std::memory_order_relaxed);
    }
    return cudaPeekAtLastError() == cudaSuccess ? FLORA_OK : FLORA_ERR_CUDA;
}

// Self-test of the bounded waits: one CTA waits on a barrier that nothing ever arrives on, with a one-millisecond
// limit.  The wait gives up, raises the error word and the kernel returns normally.
__global__ void wait_timeout_selftest_kernel(int* gave_up)
{
    __shared__ uint64_t bar;
    __shared__ int abort_flag;
    if (threadIdx.x == 0) {
        ptx::mbar_init(ptx::smem_addr(&bar), 1);
        abort_flag = 0;
        ptx::fence_barrier_init();
    }
    __syncthreads();
    if (threadIdx.x == 0) *gave_up = ptx::mbar_wait(ptx::smem_addr(&bar), 0, &abort_flag, 1000000ull) ? 0 : 1;
}

inline bool tc_read_and_clear_error(int* word)
{
    int zero = 0;
    if (cudaMemcpyFromSymbol(word, g_flora_error_word, sizeof(int)) != cudaSuccess) return false;
    return cudaMemcpyToSymbol(g_flora_error_word, &zero, sizeof(int)) == cudaSuccess;
}

}  // namespace flora
