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

// Position in a ring of `n` stages: stage index and how often the ring has wrapped (its parity is the phase bit of
// the stage's barriers).  Advanced by one step at a time: the loops that use it run once per 64-column step in a single
// thread on the critical path, where a division by a run-time value costs more than the MMAs it feeds.
struct RingPos {
    int s = 0;
    uint32_t wraps = 0;
    __device__ __forceinline__ void advance(int n)
    {
        if (++s == n) {
            s = 0;
            ++wraps;
        }
    }
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
    uint64_t full_g[8], empty_g[8], full_a[8], slice_ready[8], empty_a[8], acc_full, old_full[16];
    uint32_t tmem_base;
    int abort;
    int epi_go[4];
};

__global__ void __launch_bounds__(K1_MAX_THREADS, 1)
compress_tc_kernel(const TcMatrix* __restrict__ mats, const K1Item* __restrict__ items, const __grid_constant__ SeedTable seeds,
                   int seed_base, int r, float scale, float a, float b, int T, int gstages, int astages, int S, int GW, int P, int late_wait)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
    const int r_pad = (r + 15) & ~15;
    const uint32_t a_bytes = (uint32_t)r_pad * 128u;
    // two rings: G tiles (gstages x T tiles; the loads come from HBM and want many bytes in flight) and A tiles
    // (astages x r_pad rows; produced on chip).  Each has its own full / empty barriers.
    const uint32_t g_bytes = (uint32_t)T * G_TILE_BYTES;
    const uint32_t a_ring = smem_base + (uint32_t)gstages * g_bytes;
    K1Smem* ctl = reinterpret_cast<K1Smem*>(smem_raw + (a_ring - ptx::smem_addr(smem_raw)) + (size_t)astages * a_bytes);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;

    ptx::grid_launch_dependents();
    const K1Item item = items[blockIdx.x];                    // tables and descriptors are written at set creation, not by kernels
    const TcMatrix* mat = mats + item.mat;
    uint32_t tmem_cols = 32;
    while ((int)tmem_cols < T * r_pad) tmem_cols <<= 1;

    if (threadIdx.x == 0) {
        for (int s = 0; s < gstages; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->full_g[s]), 1);
            ptx::mbar_init(ptx::smem_addr(&ctl->empty_g[s]), 1);                   // this CTA's MMAs have consumed the G tiles
        }
        for (int s = 0; s < astages; ++s) {
            ptx::mbar_init(ptx::smem_addr(&ctl->full_a[s]), S > 1 ? 1 : GW / P);   // cluster: one arrival + the peers' bytes
            ptx::mbar_init(ptx::smem_addr(&ctl->slice_ready[s]), GW / P);
            ptx::mbar_init(ptx::smem_addr(&ctl->empty_a[s]), S);                   // every CTA of the cluster has consumed the A tile
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
        for (int s = 0; s < astages; ++s)
            for (int t = threadIdx.x; t < pad_chunks; t += (int)blockDim.x)
                ptx::st_shared_v4(a_ring + s * a_bytes + (uint32_t)r * 128u + t * 16u, 0, 0, 0, 0);
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
            RingPos pg;
            for (int ks = 0; ks < item.ksteps; ++ks, pg.advance(gstages)) {
                const int s = pg.s;
                if (!ptx::mbar_wait(ptx::smem_addr(&ctl->empty_g[s]), (pg.wraps & 1u) ^ 1u, abort)) break;
                const uint32_t bar = ptx::smem_addr(&ctl->full_g[s]);
                ptx::mbar_arrive_expect_tx(bar, (uint32_t)item.tiles * G_TILE_BYTES);
                for (int t = 0; t < item.tiles; ++t)
                    ptx::tma_load_2d(smem_base + s * g_bytes + t * G_TILE_BYTES, &mat->map_g, (item.kstep0 + ks) * 64, item.row0 + t * 128, bar);
                issued = ks + 1;
            }
            if (*abort) {
                // nobody consumes any more: wait (bounded) until the copies still in flight have landed
                for (int ks = max(0, issued - gstages); ks < issued; ++ks)
                    ptx::mbar_wait(ptx::smem_addr(&ctl->full_g[ks % gstages]), (ks / gstages) & 1, abort);
            }
        }
    } else if (warp == 1) {
        // ------------------------------------------------------------------ MMA issuer
        if (lane == 0) {
            const uint32_t idesc = ptx::umma_idesc_bf16((uint32_t)r_pad);
            const uint64_t desc_base = ptx::umma_desc_k_sw128(smem_base);
            bool ok = true;
            RingPos rg, ra;
            for (int ks = 0; ks < item.ksteps && ok; ++ks, rg.advance(gstages), ra.advance(astages)) {
                const int sg = rg.s, sa = ra.s;
                const uint32_t pa = ra.wraps & 1u;
                ok = (item.tiles == 0 || ptx::mbar_wait(ptx::smem_addr(&ctl->full_g[sg]), rg.wraps & 1u, abort)) &&
                     (S > 1 ? ptx::mbar_wait_cluster(ptx::smem_addr(&ctl->full_a[sa]), pa, abort)
                            : ptx::mbar_wait(ptx::smem_addr(&ctl->full_a[sa]), pa, abort));
                if (!ok) break;
                ptx::tc_fence_after_sync();
                // descriptors differ from the ring base only in the start-address field (16-byte units)
                const uint64_t dstage = desc_base + (uint64_t)((sg * g_bytes) >> 4);
                const uint64_t da_tile = desc_base + (uint64_t)((a_ring - smem_base + sa * a_bytes) >> 4);
                for (int t = 0; t < item.tiles; ++t) {
#pragma unroll
                    for (int kk = 0; kk < 4; ++kk)
                        ptx::umma_bf16(tmem + t * r_pad, dstage + (uint64_t)((t * G_TILE_BYTES + kk * 32) >> 4), da_tile + (uint64_t)(kk * 2), idesc,
                                       (ks | kk) != 0);
                }
                if (item.tiles > 0) ptx::umma_commit(ptx::smem_addr(&ctl->empty_g[sg]));
                // the A stage is free once every CTA of the cluster has consumed its copy of the tile
                const uint32_t ebar = ptx::smem_addr(&ctl->empty_a[sa]);
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
            RingPos ra;
            for (int ks = 0; ks < item.ksteps; ++ks, ra.advance(astages)) {
                const int s = ra.s;
                if (!ptx::mbar_wait(ptx::smem_addr(&ctl->slice_ready[s]), ra.wraps & 1u, abort)) break;
                const uint32_t fbar = ptx::smem_addr(&ctl->full_a[s]);
                const uint32_t src = a_ring + s * a_bytes + rank * slice_bytes;
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
            const int s = ks % astages, it = ks / astages;
            ok = S > 1 ? ptx::mbar_wait_cluster(ptx::smem_addr(&ctl->empty_a[s]), (it & 1) ^ 1, abort)
                       : ptx::mbar_wait(ptx::smem_addr(&ctl->empty_a[s]), (it & 1) ^ 1, abort);
            if (!ok) break;
            const uint32_t a_tile = a_ring + s * a_bytes;
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
        // The chunk buffers are the tiles of the G ring, which nothing uses once the last MMA has completed (the A ring is
        // left alone: this CTA's last slices may still be on their way to the peers).
        const int gw = warp - 2;
        const int areas = gstages * T;                            // 16 KB areas: the tiles of the G ring
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
                return smem_base + (uint32_t)(grp * NB + u % NB) * G_TILE_BYTES;
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
constexpr int K2_HELPER_WARPS = 8;    // the combine warps, idle until the first tile arrives, generate part of the CTA's first slab
constexpr int K2_MAX_THREADS = 32 * (K2_FIXED_WARPS + K2_MAX_GEN_WARPS);
constexpr int K2_MAX_SLOTS = 6;
constexpr int K2_MAX_CSTAGES = 8;
constexpr int W_BOX_BYTES = 128 * 128;     // 128 rows x 64 bf16
constexpr int S_CHUNK_BYTES = 128 * 128;   // 128 rows x 32 fp32

struct K2Smem {
    uint64_t w_full[K2_MAX_SLOTS], w_free[K2_MAX_SLOTS], out_ready[K2_MAX_SLOTS];
    uint64_t c_full[K2_MAX_CSTAGES], c_empty[K2_MAX_CSTAGES], acc_full[2], acc_empty[2], slab_full[2], slab_empty[2], slab_help;
    uint32_t tmem_base;
    int abort;
};

// Writes the tasks first, first + stride, ... of one r x bn slab of A as the N x K operand: row = column of W,
// K = index j of the sketch, values rounded to bf16 (kept in 32-bit containers, exact in tf32, for the fp32 sketch
// path).  One task makes a 4-column x 4-j (or 8-j) block and stores one 16-byte chunk per column; j >= r is zero.
template <bool BF16S>
__device__ __forceinline__ void k2_generate_slab(uint32_t slab, uint32_t slab_block, int kchunks, int bn, int col0, int r, const PhiloxKey key,
                                                 float scale, int first, int stride)
{
    const int jgroups = kchunks * 8;
    const int tasks = (bn >> 2) * jgroups;
    for (int t = first; t < tasks; t += stride) {
        const int jg = t % jgroups, cq = t / jgroups;       // jg: 16-byte chunk along K (4 tf32 or 8 bf16 values)
        const uint32_t blk = slab + (jg >> 3) * slab_block;
        if (BF16S) {
            uint32_t packed[4][4];
#pragma unroll
            for (int jj = 0; jj < 8; jj += 2) {
                float v0[4] = {0.f, 0.f, 0.f, 0.f}, v1[4] = {0.f, 0.f, 0.f, 0.f};
                const int j = jg * 8 + jj;
                if (j < r) projection_quad((uint32_t)(col0 / 4 + cq), (uint32_t)j, key, scale, v0);
                if (j + 1 < r) projection_quad((uint32_t)(col0 / 4 + cq), (uint32_t)(j + 1), key, scale, v1);
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
                if (jg * 4 + jj < r) projection_quad((uint32_t)(col0 / 4 + cq), (uint32_t)(jg * 4 + jj), key, scale, q);
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
}

template <bool BF16S>
__global__ void __launch_bounds__(K2_MAX_THREADS, 1)
decompress_tc_kernel(const TcMatrix* __restrict__ mats, const K2Item* __restrict__ items, int n_items,
                     const __grid_constant__ SeedTable seeds, int seed_base, int r, float scale, float step, int bn, int slots,
                     int cstages, int GW, int nslabs)
{
    extern __shared__ uint8_t smem_raw[];
    const uint32_t smem_base = (ptx::smem_addr(smem_raw) + 1023u) & ~1023u;
    // K chunks: one 128-byte row of S each (32 fp32 values, or 64 bf16 values when the bf16 copy of S is used)
    const int kchunks = BF16S ? (r + 63) >> 6 : (r + 31) >> 5;
    const int boxes = bn >> 6;                                 // 64-column boxes per W tile
    const uint32_t slab_block = (uint32_t)bn * 128u;           // one K chunk of a slab
    const uint32_t slab_bytes = kchunks * slab_block;
    const uint32_t slab0 = smem_base;
    const uint32_t c_ring = slab0 + nslabs * slab_bytes;
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
        ptx::mbar_init(ptx::smem_addr(&ctl->slab_help), K2_HELPER_WARPS);
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
            RingPos pw;
            bool ok = true;
            for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
                const K2Item item = items[it];
                const TcMatrix* mat = mats + item.mat;
                const int live_boxes = min(boxes, (mat->m - item.col0 + 63) >> 6);
                for (int i = 0; i < item.tiles; ++i, ++gt, pw.advance(slots)) {
                    const int s = pw.s;
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->w_free[s]), (pw.wraps & 1u) ^ 1u, abort);
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
            RingPos pc;
            bool ok = true;
            for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
                const K2Item item = items[it];
                const TcMatrix* mat = mats + item.mat;
                for (int i = 0; i < item.tiles && ok; ++i) {
                    for (int kc = 0; kc < kchunks; ++kc, ++gc, pc.advance(cstages)) {
                        const int s = pc.s;
                        ok = ptx::mbar_wait(ptx::smem_addr(&ctl->c_empty[s]), (pc.wraps & 1u) ^ 1u, abort);
                        if (!ok) break;
                        const uint32_t bar = ptx::smem_addr(&ctl->c_full[s]);
                        ptx::mbar_arrive_expect_tx(bar, S_CHUNK_BYTES);
                        if (BF16S) ptx::tma_load_2d(c_ring + s * S_CHUNK_BYTES, &mat->map_sb, kc * 64, item.row0 + i * 128, bar);
                        else ptx::tma_load_2d(c_ring + s * S_CHUNK_BYTES, &mat->map_s, kc * 32, item.row0 + i * 128, bar);
                    }
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
            RingPos pc;
            bool ok = true;
            for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x, ++k) {
                const K2Item item = items[it];
                const int sb = nslabs == 2 ? (k & 1) : 0, sphase = (nslabs == 2 ? (k >> 1) : k) & 1;
                const uint64_t desc_slab = ptx::umma_desc_k_sw128(slab0 + sb * slab_bytes);
                ok = ptx::mbar_wait(ptx::smem_addr(&ctl->slab_full[sb]), sphase, abort);
                // the combine warps' share: of the first slab, or of every slab when there is only one buffer
                if ((k == 0 || nslabs == 1) && ok) ok = ptx::mbar_wait(ptx::smem_addr(&ctl->slab_help), k & 1, abort);
                for (int i = 0; i < item.tiles && ok; ++i, ++gt) {
                    const uint32_t acc_addr = tmem + (gt & 1) * bn;
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->acc_empty[gt & 1]), ((gt >> 1) & 1) ^ 1, abort);
                    for (int kc = 0; kc < kchunks && ok; ++kc, ++gc, pc.advance(cstages)) {
                        const int s = pc.s;
                        ok = ptx::mbar_wait(ptx::smem_addr(&ctl->c_full[s]), pc.wraps & 1u, abort);
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
                if (ok) ptx::umma_commit(ptx::smem_addr(&ctl->slab_empty[sb]));   // every MMA that reads this slab has completed
            }
        }
    } else if (warp == 7) {
        // ------------------------------------------------------------------ W tile stores
        if (lane == 0) {
            int gt = 0;
            RingPos pw;
            int prev_slot = 0;
            bool ok = true;
            const bool lag = slots >= 4;               // with few slots, freeing a slot one tile late costs more than it gains
            for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x) {
                const K2Item item = items[it];
                const TcMatrix* mat = mats + item.mat;
                const int live_boxes = min(boxes, (mat->m - item.col0 + 63) >> 6);
                for (int i = 0; i < item.tiles; ++i, ++gt, pw.advance(slots)) {
                    const int s = pw.s;
                    ok = ptx::mbar_wait(ptx::smem_addr(&ctl->out_ready[s]), pw.wraps & 1u, abort);
                    if (!ok) break;
                    for (int bx = 0; bx < live_boxes; ++bx)
                        ptx::tma_store_2d(&mat->map_w, item.col0 + bx * 64, item.row0 + i * 128, w_ring + s * slot_bytes + bx * W_BOX_BYTES);
                    ptx::tma_store_commit();
                    if (lag) {
                        // one store stays in flight: wait until all but the newest have read their slot, free that one
                        ptx::tma_store_wait_read<1>();
                        if (gt > 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->w_free[prev_slot]));
                        prev_slot = s;
                    } else {
                        ptx::tma_store_wait_read<0>();          // the slot has been read out: it can be refilled
                        ptx::mbar_arrive(ptx::smem_addr(&ctl->w_free[s]));
                    }
                }
            }
            ptx::tma_store_wait_read<0>();
            if (lag && gt > 0 && ok) ptx::mbar_arrive(ptx::smem_addr(&ctl->w_free[prev_slot]));
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
        RingPos pw;
        bool ok = true;
        const int helper = (half * 4 + (warp - (half ? 8 : 2))) * 32 + lane;              // 0 .. 255
        int k = 0;
        for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x, ++k) {
            const K2Item item = items[it];
            if (k == 0 || nslabs == 1) {
                // Nothing to combine yet (first item), or a single slab buffer whose refill nothing overlaps: write a
                // share of the slab alongside the generator warps.
                ok = ptx::mbar_wait(ptx::smem_addr(&ctl->slab_empty[0]), (((nslabs == 2 ? (k >> 1) : k) & 1) ^ 1), abort);
                if (!ok) break;
                if (item.tiles > 0)     // (an empty item pads a CTA's list: its slab is never read)
                    k2_generate_slab<BF16S>(slab0, slab_block, kchunks, bn, item.col0, r, make_key(seeds.s[item.mat - seed_base]), scale,
                                            32 * GW + helper, 32 * (GW + K2_HELPER_WARPS));
                ptx::fence_proxy_async_smem();
                __syncwarp();
                if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->slab_help));
            }
            const int live_chunks = min(boxes, (mats[item.mat].m - item.col0 + 63) >> 6) << 2;
            const int c_begin = half * per_half;
            const int mine = max(0, min(per_half, live_chunks - c_begin));
            for (int i = 0; i < item.tiles; ++i, ++gt, pw.advance(slots)) {
                const int s = pw.s;
                ok = ptx::mbar_wait(ptx::smem_addr(&ctl->acc_full[gt & 1]), (gt >> 1) & 1, abort) &&
                     ptx::mbar_wait(ptx::smem_addr(&ctl->w_full[s]), pw.wraps & 1u, abort);
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
        int k = 0;
        bool ok = true;
        for (int it = blockIdx.x; it < n_items && ok; it += gridDim.x, ++k) {
            const K2Item item = items[it];
            const PhiloxKey key = make_key(seeds.s[item.mat - seed_base]);
            const int sb = nslabs == 2 ? (k & 1) : 0;
            ok = ptx::mbar_wait(ptx::smem_addr(&ctl->slab_empty[sb]), (((nslabs == 2 ? (k >> 1) : k) & 1) ^ 1), abort);
            if (!ok) break;
            const uint32_t slab = slab0 + sb * slab_bytes;
            // the first slab (every slab, with a single buffer) is shared with the combine warps
            if (item.tiles > 0)
                k2_generate_slab<BF16S>(slab, slab_block, kchunks, bn, item.col0, r, key, scale, g,
                                        (k == 0 || nslabs == 1) ? 32 * (GW + K2_HELPER_WARPS) : 32 * GW);
            ptx::fence_proxy_async_smem();
            __syncwarp();
            if (lane == 0) ptx::mbar_arrive(ptx::smem_addr(&ctl->slab_full[sb]));
        }
    }
    ptx::tc_fence_before_sync();
    __syncthreads();
    if (warp == 1) {
        ptx::tc_fence_after_sync();
        ptx::tmem_dealloc(tmem, tmem_cols);
    }
}

// S <- b S for the listed matrices (those whose rows receive adds), or for matrix first + blockIdx.y of the table
// where there is no list; blockIdx.y = list entry.
__global__ void scale_sketches_kernel(const TcMatrix* __restrict__ mats, const int* __restrict__ ids, int first, int r, float b)
{
    ptx::grid_launch_dependents();       // the compression kernel that follows may start streaming G right away
    const TcMatrix* mat = mats + (ids ? ids[blockIdx.y] : first + (int)blockIdx.y);
    float* S = mat->S;
    const int64_t total = (int64_t)mat->n * r;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, nthreads = (int64_t)gridDim.x * blockDim.x;
    if (mat->lds == r && (reinterpret_cast<uintptr_t>(S) & 15) == 0) {
        // densely stored, 16-byte aligned: four values per access
        float4* S4 = reinterpret_cast<float4*>(S);
        for (int64_t t = tid; t < (total >> 2); t += nthreads) {
            float4 v = S4[t];
            v = (b == 0.0f) ? make_float4(0.f, 0.f, 0.f, 0.f) : make_float4(v.x * b, v.y * b, v.z * b, v.w * b);
            S4[t] = v;
        }
        for (int64_t t = (total & ~(int64_t)3) + tid; t < total; t += nthreads) S[t] = (b == 0.0f) ? 0.0f : S[t] * b;
    } else {
        for (int64_t row = blockIdx.x; row < mat->n; row += gridDim.x)
            for (int j = (int)threadIdx.x; j < r; j += (int)blockDim.x) {
                float* p = S + row * mat->lds + j;
                *p = (b == 0.0f) ? 0.0f : *p * b;
            }
    }
}


// bf16 copy of every sketch of the table, n x k_pad with zero padding (the M x K operand of the decompression
// kernel for ranks above 64); blockIdx.y = matrix.  A thread converts eight neighbouring columns of one row: two
// 16-byte loads (the sketches that reach this kernel have 16-byte aligned rows), one 16-byte store; a block of 256
// threads covers 2048 / k_pad rows at a time.
__global__ void __launch_bounds__(256) sketch_to_bf16_kernel(const TcMatrix* __restrict__ mats, int r, int k_pad)
{
    ptx::grid_launch_dependents();       // the decompression kernel that follows may set up and generate its first slabs meanwhile
    const TcMatrix* mat = mats + blockIdx.y;
    const int groups = k_pad >> 3;                        // 8-column groups per row: 8, 16, 24 or 32
    const int rows_per_block = 256 / groups;
    const int g = (int)threadIdx.x % groups, lr = (int)threadIdx.x / groups;
    if (lr >= rows_per_block) return;
    const int j = g * 8;
    const float* S = mat->S;
    const int64_t lds = mat->lds;
    __nv_bfloat16* Sb = mat->Sb;
    for (int row = (int)blockIdx.x * rows_per_block + lr; row < mat->n; row += (int)gridDim.x * rows_per_block) {
        const float* src = S + (int64_t)row * lds + j;
        float v[8];
        if (j + 7 < r) {
            const float4 a = *reinterpret_cast<const float4*>(src), b = *reinterpret_cast<const float4*>(src + 4);
            v[0] = a.x; v[1] = a.y; v[2] = a.z; v[3] = a.w; v[4] = b.x; v[5] = b.y; v[6] = b.z; v[7] = b.w;
        } else {
#pragma unroll
            for (int e = 0; e < 8; ++e) v[e] = j + e < r ? src[e] : 0.0f;
        }
        uint4 out;
        __nv_bfloat162 p0 = __floats2bfloat162_rn(v[0], v[1]), p1 = __floats2bfloat162_rn(v[2], v[3]);
        __nv_bfloat162 p2 = __floats2bfloat162_rn(v[4], v[5]), p3 = __floats2bfloat162_rn(v[6], v[7]);
        out.x = *reinterpret_cast<uint32_t*>(&p0);
        out.y = *reinterpret_cast<uint32_t*>(&p1);
        out.z = *reinterpret_cast<uint32_t*>(&p2);
        out.w = *reinterpret_cast<uint32_t*>(&p3);
        *reinterpret_cast<uint4*>(Sb + (int64_t)row * k_pad + j) = out;
    }
}

// S <- 0 for every matrix of the table (start of an accumulation cycle); blockIdx.y = matrix.  Densely stored sketches
// with 16-byte aligned storage are cleared with 16-byte stores, others element by element along each row.
__global__ void zero_sketches_kernel(const TcMatrix* __restrict__ mats, int r)
{
    const TcMatrix* mat = mats + blockIdx.y;
    float* S = mat->S;
    const int64_t total = (int64_t)mat->n * r;
    const int64_t tid = (int64_t)blockIdx.x * blockDim.x + threadIdx.x, nthreads = (int64_t)gridDim.x * blockDim.x;
    if (mat->lds == r && (reinterpret_cast<uintptr_t>(S) & 15) == 0) {
        float4* S4 = reinterpret_cast<float4*>(S);
        for (int64_t t = tid; t < (total >> 2); t += nthreads) S4[t] = make_float4(0.f, 0.f, 0.f, 0.f);
        for (int64_t t = (total & ~(int64_t)3) + tid; t < total; t += nthreads) S[t] = 0.0f;
    } else {
        for (int64_t row = blockIdx.x; row < mat->n; row += gridDim.x)
            for (int j = (int)threadIdx.x; j < r; j += (int)blockDim.x) S[row * mat->lds + j] = 0.0f;
    }
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

}  // namespace flora
